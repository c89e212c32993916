// Prefill entry on the host side: one kernel serves every supported shape.
#include "l4l_internal.h"

namespace l4l {

l4l_status launch_prefill(const l4l_tensor4 &q, const l4l_tensor4 &k, const l4l_tensor4 &v,
                          const l4l_tensor4 &o, const l4l_kv_cache &cache, const int32_t *d_seq_lens,
                          int S_max, int B, int Hq, int Hkv, int D, float scale, float *d_lse,
                          void *workspace, cudaStream_t stream)
{
    return launch_prefill_tc(q, k, v, o, cache, d_seq_lens, S_max, B, Hq, Hkv, D, scale, d_lse, workspace, stream);
}

}  // namespace l4l
