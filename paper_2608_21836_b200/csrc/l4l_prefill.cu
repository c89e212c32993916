// Prefill dispatch: picks the kernel for the shape. (Host code only.)
#include <cstdlib>

#include "l4l_internal.h"

namespace l4l {

l4l_status launch_prefill(const l4l_tensor4 &q, const l4l_tensor4 &k, const l4l_tensor4 &v,
                          const l4l_tensor4 &o, const l4l_kv_cache &cache, const int32_t *d_seq_lens,
                          int S_max, int B, int Hq, int Hkv, int D, float scale, float *d_lse,
                          void *workspace, cudaStream_t stream)
{
    // L4L_PREFILL_KERNEL=mma selects the warp-MMA kernel (debugging aid); the default is tcgen05
    static const bool use_mma = [] {
        const char *e = getenv("L4L_PREFILL_KERNEL");
        return e && e[0] == 'm';
    }();
    if (!use_mma)
        return launch_prefill_tc(q, k, v, o, cache, d_seq_lens, S_max, B, Hq, Hkv, D, scale, d_lse, workspace, stream);
    return launch_prefill_mma(q, k, v, o, cache, d_seq_lens, S_max, B, Hq, Hkv, D, scale, d_lse, workspace, stream);
}

}  // namespace l4l
