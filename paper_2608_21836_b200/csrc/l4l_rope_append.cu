// Rotary position embedding, optional per-head RMS normalisation of q and k, and the cache update in
// one streaming pass over the projection outputs of the new tokens: q is rotated in place, k is
// rotated into its cache slot, v is copied into its cache slot. HBM-bound: every byte is read once
// and written once; the cos / sin rows of a position are shared by all heads of the token and stay
// in cache.
//
// A head row of D values is handled by D/16 neighbouring lanes; lane u holds elements [8u, 8u+8) of
// the first half and the matching elements of the second half (the rotation pairs element i with
// element i + D/2), so every access is a 16-byte piece and a warp touches whole contiguous rows.
#include "l4l_internal.h"
#include "l4l_ptx.cuh"

namespace l4l {

namespace {

struct RopeParams {
    uint4 *q;                        // strides below in 16-byte units
    const uint4 *k_new, *v_new;
    uint4 *cache_k, *cache_v;
    int64_t q_sb, q_st, q_sh, k_sb, k_st, k_sh, v_sb, v_st, v_sh, c_sb, c_sh, c_st;
    const int32_t *pos, *n_new;
    const float4 *cos, *sin;         // [n_pos, D/2] as float4
    const float4 *q_weight, *k_weight;
    float eps;
    int B, T, Hq, Hkv, max_pos;      // max_pos = min(cache.max_len, n_pos)
};

__device__ __forceinline__ void unpack8(const uint4 &v, float (&f)[8])
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

__device__ __forceinline__ uint4 pack8(const float (&f)[8])
{
    return make_uint4(pack_bf16x2(f[0], f[1]), pack_bf16x2(f[2], f[3]), pack_bf16x2(f[4], f[5]),
                      pack_bf16x2(f[6], f[7]));
}

// Six blocks per SM (40 registers): the kernel lives on loads in flight, and the compiler fits the row in 40
// registers without spilling (eight blocks would spill; the unconstrained build took 63 registers, four blocks).
template <int D>
__global__ void __launch_bounds__(256, 6) rope_kv_append_kernel(const RopeParams p)
{
    constexpr int kLanes = D / 16;                  // lanes per head row
    constexpr int kHalfPieces = D / 16;             // 16-byte pieces per half row
    const int heads = p.Hq + 2 * p.Hkv;             // q heads, then k heads, then v heads
    const unsigned rows = (unsigned)p.B * p.T * heads;        // < 2^31, checked by the launcher
    const int u = threadIdx.x % kLanes;
    const uint32_t group_mask = ((1u << kLanes) - 1u) << ((threadIdx.x & 31) & ~(kLanes - 1));
    const unsigned first = (blockIdx.x * blockDim.x + threadIdx.x) / kLanes;
    const unsigned step = gridDim.x * blockDim.x / kLanes;
    // all lanes of a row group take the same trips through the loop (rows is tested per group)
    for (unsigned r = first; r < rows; r += step) {
        const int hh = (int)(r % (unsigned)heads);
        const unsigned bt = r / (unsigned)heads;
        const int t = (int)(bt % (unsigned)p.T), b = (int)(bt / (unsigned)p.T);
        const int n = p.n_new ? p.n_new[b] : p.T;
        const long long P = (long long)p.pos[b] + t;
        // the lanes of a row group skip together, so the group-masked shuffles below see the full group
        if (t >= n || P < 0 || P >= p.max_pos) continue;

        if (hh >= p.Hq + p.Hkv) {                   // v: exact copy
            const int g = hh - p.Hq - p.Hkv;
            const uint4 *src = p.v_new + b * p.v_sb + t * p.v_st + g * p.v_sh;
            uint4 *dst = p.cache_v + b * p.c_sb + g * p.c_sh + P * p.c_st;
            const uint4 a = src[u], c = src[kHalfPieces + u];
            dst[u] = a;
            dst[kHalfPieces + u] = c;
            continue;
        }
        const bool is_q = hh < p.Hq;
        const int g = is_q ? hh : hh - p.Hq;
        const uint4 *src = is_q ? p.q + b * p.q_sb + t * p.q_st + g * p.q_sh
                                : p.k_new + b * p.k_sb + t * p.k_st + g * p.k_sh;
        uint4 *dst = is_q ? p.q + b * p.q_sb + t * p.q_st + g * p.q_sh
                          : p.cache_k + b * p.c_sb + g * p.c_sh + P * p.c_st;
        float x1[8], x2[8];
        unpack8(src[u], x1);
        unpack8(src[kHalfPieces + u], x2);

        const float4 *w = is_q ? p.q_weight : p.k_weight;
        if (w) {
            float ss = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) ss = fmaf(x1[i], x1[i], ss);
#pragma unroll
            for (int i = 0; i < 8; ++i) ss = fmaf(x2[i], x2[i], ss);
#pragma unroll
            for (int off = 1; off < kLanes; off <<= 1) ss += __shfl_xor_sync(group_mask, ss, off);
            const float rinv = rsqrtf(ss * (1.f / D) + p.eps);
            const float4 wa = w[2 * u], wb = w[2 * u + 1], wc = w[D / 8 + 2 * u], wd = w[D / 8 + 2 * u + 1];
            const float w1[8] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
            const float w2[8] = {wc.x, wc.y, wc.z, wc.w, wd.x, wd.y, wd.z, wd.w};
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                x1[i] = x1[i] * rinv * w1[i];
                x2[i] = x2[i] * rinv * w2[i];
            }
        }
        const float4 *cr = p.cos + P * (D / 8) + 2 * u, *sr = p.sin + P * (D / 8) + 2 * u;
        const float4 ca = cr[0], cb = cr[1], sa = sr[0], sb = sr[1];
        const float c[8] = {ca.x, ca.y, ca.z, ca.w, cb.x, cb.y, cb.z, cb.w};
        const float s[8] = {sa.x, sa.y, sa.z, sa.w, sb.x, sb.y, sb.z, sb.w};
        float y1[8], y2[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            y1[i] = fmaf(-x2[i], s[i], x1[i] * c[i]);
            y2[i] = fmaf(x1[i], s[i], x2[i] * c[i]);
        }
        dst[u] = pack8(y1);
        dst[kHalfPieces + u] = pack8(y2);
    }
}

}  // namespace

l4l_status launch_rope_kv_append(const l4l_tensor4 &q, const l4l_tensor4 &k_new, const l4l_tensor4 &v_new,
                                 const l4l_kv_cache &cache, const int32_t *d_pos, const int32_t *d_n_new, int T, int B,
                                 int Hq, int Hkv, int D, const float *d_cos, const float *d_sin, int n_pos,
                                 const float *d_q_weight, const float *d_k_weight, float norm_eps, cudaStream_t stream)
{
    RopeParams p;
    p.q = static_cast<uint4 *>(q.ptr);
    p.k_new = static_cast<const uint4 *>(k_new.ptr);
    p.v_new = static_cast<const uint4 *>(v_new.ptr);
    p.cache_k = static_cast<uint4 *>(cache.k);
    p.cache_v = static_cast<uint4 *>(cache.v);
    p.q_sb = q.stride_b / 8; p.q_st = q.stride_t / 8; p.q_sh = q.stride_h / 8;
    p.k_sb = k_new.stride_b / 8; p.k_st = k_new.stride_t / 8; p.k_sh = k_new.stride_h / 8;
    p.v_sb = v_new.stride_b / 8; p.v_st = v_new.stride_t / 8; p.v_sh = v_new.stride_h / 8;
    p.c_sb = cache.stride_b / 8; p.c_sh = cache.stride_h / 8; p.c_st = cache.stride_t / 8;
    p.pos = d_pos; p.n_new = d_n_new;
    p.cos = reinterpret_cast<const float4 *>(d_cos);
    p.sin = reinterpret_cast<const float4 *>(d_sin);
    p.q_weight = reinterpret_cast<const float4 *>(d_q_weight);
    p.k_weight = reinterpret_cast<const float4 *>(d_k_weight);
    p.eps = norm_eps;
    p.B = B; p.T = T; p.Hq = Hq; p.Hkv = Hkv;
    p.max_pos = cache.max_len < n_pos ? cache.max_len : n_pos;
    const long long rows = (long long)B * T * (Hq + 2 * Hkv);
    if (rows >= (1ll << 31) - (1ll << 24)) return L4L_ERR_UNSUPPORTED;   // the kernel indexes rows in 32 bits
    const long long threads = rows * (D / 16);
    long long blocks = (threads + 255) / 256;
    const long long cap = 16ll * sm_count();      // grid-stride beyond that (6 resident blocks per SM; 6 to 48 per SM measured, 16 best)
    if (blocks > cap) blocks = cap;
    if (D == 128)
        rope_kv_append_kernel<128><<<(int)blocks, 256, 0, stream>>>(p);
    else
        rope_kv_append_kernel<64><<<(int)blocks, 256, 0, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? L4L_OK : L4L_ERR_CUDA;
}

}  // namespace l4l
