// Cache update for an fp8 (e4m3) KV cache: the new tokens' bf16 K and V rows are divided by the scale
// of their KV head and rounded to e4m3 (nearest even, saturating at +-448) on the way into the cache.
// One thread turns 16 bf16 values of a K row and of the matching V row into 16 bytes each.
#include "l4l_fp8_quant.cuh"
#include "l4l_internal.h"
#include "l4l_ptx.cuh"

namespace l4l {

namespace {

struct AppendFp8Params {
    const uint4 *k_new, *v_new;      // bf16, strides in 16-byte units (8 values)
    uint4 *cache_k, *cache_v;        // e4m3, strides in 16-byte units (16 values)
    int64_t k_sb, k_st, k_sh, v_sb, v_st, v_sh;
    int64_t c_sb, c_sh, c_st;
    const int32_t *write_pos, *n_new;
    const float *k_scale, *v_scale;  // [Hkv]
    int B, T, Hkv, pieces, max_len;
};

__global__ void __launch_bounds__(256) kv_append_fp8_kernel(const AppendFp8Params p)
{
    const long long total = (long long)p.B * p.T * p.Hkv * p.pieces;
    for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int piece = (int)(idx % p.pieces);              // 16 values
        long long rest = idx / p.pieces;
        const int g = (int)(rest % p.Hkv);
        rest /= p.Hkv;
        const int r = (int)(rest % p.T);
        const int b = (int)(rest / p.T);
        const int n = p.n_new ? p.n_new[b] : p.T;
        if (r >= n) continue;
        const long long slot = (long long)p.write_pos[b] + r;
        if (slot < 0 || slot >= p.max_len) continue;          // dropped, never written out of range
        const uint4 *ks = p.k_new + b * p.k_sb + r * p.k_st + g * p.k_sh + 2 * piece;
        const uint4 *vs = p.v_new + b * p.v_sb + r * p.v_st + g * p.v_sh + 2 * piece;
        const float sk = p.k_scale[g], sv = p.v_scale[g];
        const uint2 k0 = quantise8(ks[0], sk), k1 = quantise8(ks[1], sk);
        const uint2 v0 = quantise8(vs[0], sv), v1 = quantise8(vs[1], sv);
        const int64_t dst = b * p.c_sb + g * p.c_sh + slot * p.c_st + piece;
        p.cache_k[dst] = make_uint4(k0.x, k0.y, k1.x, k1.y);
        p.cache_v[dst] = make_uint4(v0.x, v0.y, v1.x, v1.y);
    }
}

}  // namespace

l4l_status launch_kv_append_fp8(const l4l_kv_cache &cache, const l4l_tensor4 &k_new, const l4l_tensor4 &v_new,
                                const int32_t *d_write_pos, const int32_t *d_n_new, int n_new_max, int B, int Hkv,
                                int D, const float *d_k_scale, const float *d_v_scale, cudaStream_t stream)
{
    AppendFp8Params p;
    p.k_new = static_cast<const uint4 *>(k_new.ptr);
    p.v_new = static_cast<const uint4 *>(v_new.ptr);
    p.cache_k = static_cast<uint4 *>(cache.k);
    p.cache_v = static_cast<uint4 *>(cache.v);
    p.k_sb = k_new.stride_b / 8; p.k_st = k_new.stride_t / 8; p.k_sh = k_new.stride_h / 8;
    p.v_sb = v_new.stride_b / 8; p.v_st = v_new.stride_t / 8; p.v_sh = v_new.stride_h / 8;
    p.c_sb = cache.stride_b / 16; p.c_sh = cache.stride_h / 16; p.c_st = cache.stride_t / 16;
    p.write_pos = d_write_pos; p.n_new = d_n_new;
    p.k_scale = d_k_scale; p.v_scale = d_v_scale;
    p.B = B; p.T = n_new_max; p.Hkv = Hkv; p.pieces = D / 16; p.max_len = cache.max_len;
    const long long total = (long long)B * n_new_max * Hkv * p.pieces;
    long long blocks = (total + 255) / 256;
    const long long cap = 8ll * sm_count();
    if (blocks > cap) blocks = cap;
    kv_append_fp8_kernel<<<(int)blocks, 256, 0, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? L4L_OK : L4L_ERR_CUDA;
}

}  // namespace l4l
