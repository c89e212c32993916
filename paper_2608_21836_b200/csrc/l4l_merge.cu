// Log-sum-exp merge of R partial attention results over disjoint parts of one key range: the exchange-side
// half of context-parallel decode (every rank decodes over its shard of a sequence's cache and returns its
// output and log-sum-exp; the partials are gathered; this kernel combines them). The same formula as the
// in-kernel merge of the split decode: o = sum_r w_r o_r / sum_r w_r with w_r = exp(lse_r - max_r lse_r).
// One warp per (sequence, query head); a shard with no keys has lse = -inf and weight 0.
#include "l4l_internal.h"
#include "l4l_ptx.cuh"

namespace l4l {

namespace {

template <int D>
__global__ void __launch_bounds__(256)
attn_merge_kernel(const __nv_bfloat16 *o_parts, const float *lse_parts, int R, __nv_bfloat16 *o, float *lse, int rows)
{
    constexpr int kPer = D / 32;                         // values per lane: 2 (D = 64) or 4 (D = 128)
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    float mx = -INFINITY;
    for (int r = 0; r < R; ++r) mx = fmaxf(mx, __ldg(lse_parts + (size_t)r * rows + row));
    float acc[kPer];
#pragma unroll
    for (int i = 0; i < kPer; ++i) acc[i] = 0.f;
    float wsum = 0.f;
    if (mx > -INFINITY) {
        for (int r = 0; r < R; ++r) {
            const float w = __expf(__ldg(lse_parts + (size_t)r * rows + row) - mx);      // -inf -> 0
            const __nv_bfloat16 *src = o_parts + ((size_t)r * rows + row) * D + lane * kPer;
            if (w > 0.f) {
#pragma unroll
                for (int i = 0; i < kPer; i += 2) {
                    const uint32_t two = *reinterpret_cast<const uint32_t *>(src + i);
                    acc[i] = fmaf(w, __uint_as_float(two << 16), acc[i]);
                    acc[i + 1] = fmaf(w, __uint_as_float(two & 0xffff0000u), acc[i + 1]);
                }
            }
            wsum += w;
        }
    }
    const float inv = wsum > 0.f ? 1.f / wsum : 0.f;
    __nv_bfloat16 *dst = o + (size_t)row * D + lane * kPer;
#pragma unroll
    for (int i = 0; i < kPer; i += 2)
        *reinterpret_cast<uint32_t *>(dst + i) = pack_bf16x2(acc[i] * inv, acc[i + 1] * inv);
    if (lse && lane == 0) lse[row] = wsum > 0.f ? mx + logf(wsum) : -INFINITY;
}

}  // namespace

l4l_status launch_attn_merge(const void *o_parts, const float *lse_parts, int R, void *o, float *d_lse, int B, int Hq,
                             int D, cudaStream_t stream)
{
    const long long rows = (long long)B * Hq;
    if (rows > 0x7fffffffll) return L4L_ERR_UNSUPPORTED;
    const int blocks = (int)((rows + 7) / 8);
    auto *op = static_cast<const __nv_bfloat16 *>(o_parts);
    auto *out = static_cast<__nv_bfloat16 *>(o);
    if (D == 128)
        attn_merge_kernel<128><<<blocks, 256, 0, stream>>>(op, lse_parts, R, out, d_lse, (int)rows);
    else
        attn_merge_kernel<64><<<blocks, 256, 0, stream>>>(op, lse_parts, R, out, d_lse, (int)rows);
    return cudaGetLastError() == cudaSuccess ? L4L_OK : L4L_ERR_CUDA;
}

}  // namespace l4l
