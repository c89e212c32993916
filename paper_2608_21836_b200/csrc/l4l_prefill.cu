#include "l4l_internal.h"
namespace l4l {
l4l_status launch_prefill(const l4l_tensor4 &, const l4l_tensor4 &, const l4l_tensor4 &, const l4l_tensor4 &,
                          const l4l_kv_cache &, const int32_t *, int, int, int, int, int, float, float *, void *,
                          cudaStream_t)
{
    return L4L_ERR_UNSUPPORTED;
}
}  // namespace l4l
