// Prefill entries on the host side: one kernel serves every supported shape, for a fresh prompt and for a
// chunk of new tokens over an already populated cache.
#include "l4l_internal.h"

namespace l4l {

l4l_status launch_prefill(const l4l_tensor4 &q, const l4l_tensor4 &k, const l4l_tensor4 &v,
                          const l4l_tensor4 &o, const l4l_kv_cache &cache, const int32_t *d_seq_lens,
                          int S_max, int B, int Hq, int Hkv, int D, float scale, float *d_lse,
                          void *workspace, cudaStream_t stream)
{
    return launch_prefill_tc(q, k, v, o, cache, d_seq_lens, S_max, B, Hq, Hkv, D, scale, d_lse, workspace, stream,
                             nullptr, S_max);
}

l4l_status launch_prefill_chunk(const l4l_tensor4 &q, const l4l_tensor4 &o, const l4l_kv_cache &cache,
                                const int32_t *d_past_lens, const int32_t *d_q_lens, int S_max, int B, int Hq,
                                int Hkv, int D, float scale, float *d_lse, void *workspace, cudaStream_t stream)
{
    // keys and values are read straight from the cache: view it as [B, slot, Hkv, D]
    l4l_tensor4 k{cache.k, cache.stride_b, cache.stride_t, cache.stride_h};
    l4l_tensor4 v{cache.v, cache.stride_b, cache.stride_t, cache.stride_h};
    l4l_kv_cache no_write{nullptr, nullptr, 0, 0, 0, 0};       // the caller has already appended the chunk
    return launch_prefill_tc(q, k, v, o, no_write, d_q_lens, S_max, B, Hq, Hkv, D, scale, d_lse, workspace, stream,
                             d_past_lens, cache.max_len);
}

}  // namespace l4l
