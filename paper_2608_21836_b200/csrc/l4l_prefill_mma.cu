// Causal prefill on the legacy warp-level tensor path (mma.sync). A simple flash-style kernel:
// one CTA per (64-row query tile, query head, sequence); a producer warp streams 64-token K/V
// tiles by TMA up to the diagonal; four consumer warps own 16 query rows each and keep
// online-softmax statistics in fp32. The CTA of a KV group's first query head copies its
// diagonal K/V tile from shared memory into the cache (each cache row is written once).
//
// This kernel serves shapes the tcgen05 kernel does not take and is the correctness
// stepping stone it was validated against; it is not the fast path.
#include "l4l_internal.h"
#include "l4l_warp_attn.cuh"

namespace l4l {

namespace {

constexpr int kTile = 64;               // query rows per CTA == tokens per K/V tile
constexpr int kConsumerWarps = 4;
constexpr int kThreads = (kConsumerWarps + 1) * 32;

template <int D>
struct PrefillMmaCfg {
    static constexpr int kHalves = D / 64;
    static constexpr uint32_t kHalfBytes = kTile * 128;
    static constexpr uint32_t kTileBytes = kHalves * kHalfBytes;
    static constexpr uint32_t kStageBytes = 2 * kTileBytes;
    static constexpr int kStages = (D == 128) ? 3 : 4;
    static constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + 2 * kStages * sizeof(uint64_t) + 64;
};

struct PrefillMmaParams {
    const __nv_bfloat16 *q;
    __nv_bfloat16 *o;
    int64_t q_sb, q_st, q_sh, o_sb, o_st, o_sh;
    __nv_bfloat16 *cache_k, *cache_v;     // null: no cache write
    int64_t c_sb, c_sh, c_st;
    int cache_max_len;
    const int32_t *seq_lens;
    float *lse;                            // [B, Hq, S_max] or null
    unsigned *status;
    int S_max, Hq, Hkv, G, n_qtiles;
    float scale_log2e;
    TmapCoord coord;
};

__device__ __forceinline__ void order_coords(const TmapCoord &c, int t, int h, int b, int &c1, int &c2, int &c3)
{
    c1 = (c.pos_t == 1) ? t : (c.pos_h == 1) ? h : b;
    c2 = (c.pos_t == 2) ? t : (c.pos_h == 2) ? h : b;
    c3 = (c.pos_t == 3) ? t : (c.pos_h == 3) ? h : b;
}

template <int D>
__global__ void __launch_bounds__(kThreads)
prefill_mma_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                   const PrefillMmaParams p)
{
    using C = PrefillMmaCfg<D>;
    const int qt = p.n_qtiles - 1 - (int)blockIdx.x;      // heaviest (longest causal span) tiles first
    const int h = blockIdx.y, b = blockIdx.z;
    int L = p.seq_lens[b];
    L = L < 0 ? 0 : (L > p.S_max ? p.S_max : L);
    const int q0 = qt * kTile;
    if (q0 >= L) return;                                  // whole tile beyond the sequence
    const int kvh = h / p.G;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    uint8_t *stages = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
    uint64_t *full = reinterpret_cast<uint64_t *>(stages + (size_t)C::kStages * C::kStageBytes);
    uint64_t *empty = full + C::kStages;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(empty + C::kStages);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], kConsumerWarps);
        }
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
    }
    __syncthreads();

    const int n_kv_tiles = qt + 1;                         // tiles 0 .. diagonal

    if (warp == kConsumerWarps) {
        if (lane == 0) {
            tma_prefetch_desc(&tmap_k);
            tma_prefetch_desc(&tmap_v);
            int c1, c2, c3;
            for (int j = 0; j < n_kv_tiles; ++j) {
                const uint32_t s = j % C::kStages, ph = (j / C::kStages) & 1u;
                if (!mbar_wait(&empty[s], ph ^ 1u, abort_flag)) break;
                mbar_arrive_expect_tx(&full[s], C::kStageBytes);
                uint8_t *dst = stages + (size_t)s * C::kStageBytes;
                order_coords(p.coord, j * kTile, kvh, b, c1, c2, c3);
#pragma unroll
                for (int hf = 0; hf < C::kHalves; ++hf) {
                    tma_load_4d(dst + hf * C::kHalfBytes, &tmap_k, &full[s], hf * 64, c1, c2, c3);
                    tma_load_4d(dst + C::kTileBytes + hf * C::kHalfBytes, &tmap_v, &full[s], hf * 64, c1, c2, c3);
                }
            }
        }
    } else {
        WarpAttnState<D> st;
        st.reset();
        uint32_t qf[D / 16][4];
        const int row_lo = q0 + warp * 16 + (lane >> 2);   // this lane's two query rows (tokens)
        const int row_hi = row_lo + 8;
        {
            const uint32_t *q_lo = reinterpret_cast<const uint32_t *>(p.q + b * p.q_sb + (int64_t)row_lo * p.q_st + h * p.q_sh);
            const uint32_t *q_hi = reinterpret_cast<const uint32_t *>(p.q + b * p.q_sb + (int64_t)row_hi * p.q_st + h * p.q_sh);
            const bool v_lo = row_lo < L, v_hi = row_hi < L;
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                const int w = ks * 8 + (lane & 3);
                qf[ks][0] = v_lo ? __ldg(q_lo + w) : 0u;
                qf[ks][1] = v_hi ? __ldg(q_hi + w) : 0u;
                qf[ks][2] = v_lo ? __ldg(q_lo + w + 4) : 0u;
                qf[ks][3] = v_hi ? __ldg(q_hi + w + 4) : 0u;
            }
        }
        const int warp_row_min = q0 + warp * 16, warp_row_max = warp_row_min + 15;
        const bool writes_cache = p.cache_k != nullptr && (h % p.G) == 0;

        for (int j = 0; j < n_kv_tiles; ++j) {
            const uint32_t s = j % C::kStages, ph = (j / C::kStages) & 1u;
            if (!mbar_wait(&full[s], ph, abort_flag)) break;
            uint8_t *kt = stages + (size_t)s * C::kStageBytes;
            uint8_t *vt = kt + C::kTileBytes;
            const int t0 = j * kTile;
            bool wrote_smem = false;

            if (j == qt) {
                // diagonal tile: tokens q0 .. q0+63
                if (writes_cache) {
                    // copy rows < L of K and V into cache slots (bit-exact; un-swizzle on the way)
                    const int ctid = threadIdx.x;
                    constexpr int kChunks = D / 8;
                    for (int i = ctid; i < kTile * kChunks; i += kConsumerWarps * 32) {
                        const int r = i / kChunks, ch = i % kChunks;
                        const int tok = t0 + r;
                        if (tok < L && tok < p.cache_max_len) {
                            const uint32_t off = (ch >> 3) * C::kHalfBytes + swz128(r, ch & 7);
                            const uint4 kk = *reinterpret_cast<const uint4 *>(kt + off);
                            const uint4 vv = *reinterpret_cast<const uint4 *>(vt + off);
                            const int64_t dst = b * p.c_sb + kvh * p.c_sh + (int64_t)tok * p.c_st + ch * 8;
                            *reinterpret_cast<uint4 *>(p.cache_k + dst) = kk;
                            *reinterpret_cast<uint4 *>(p.cache_v + dst) = vv;
                        }
                    }
                }
                if (t0 + kTile > L) {
                    // V rows past the end of the sequence may hold any bits: clear them so that a zero
                    // weight times garbage cannot appear. Every warp clears all such rows itself (same
                    // values), so no cross-warp ordering is needed; the cache copy above never reads them.
                    constexpr int kChunks = D / 8;
                    const int first = L - t0;
                    for (int i = lane; i < (kTile - first) * kChunks; i += 32) {
                        const int r = first + i / kChunks, ch = i % kChunks;
                        *reinterpret_cast<uint4 *>(vt + (ch >> 3) * C::kHalfBytes + r * 128 + ((ch & 7) << 4)) =
                            make_uint4(0u, 0u, 0u, 0u);
                    }
                    wrote_smem = true;
                    __syncwarp();
                }
            }

#pragma unroll 1
            for (int sl = 0; sl < kTile / 16; ++sl) {
                const int tok0 = t0 + sl * 16;
                if (tok0 > warp_row_max) break;                      // nothing of this slice is visible
                float s_lo[4], s_hi[4];
                warp_qk_16x16<D>(qf, smem_u32(kt), C::kHalfBytes, sl * 16, s_lo, s_hi);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    s_lo[e] *= p.scale_log2e;
                    s_hi[e] *= p.scale_log2e;
                }
                if (tok0 + 15 > warp_row_min) {                      // causal mask inside the slice
                    const int tk = tok0 + 2 * (lane & 3);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int row = (e < 2) ? row_lo : row_hi;
                        if (tk + (e & 1) > row) s_lo[e] = -INFINITY;
                        if (tk + (e & 1) + 8 > row) s_hi[e] = -INFINITY;
                    }
                }
                uint32_t pa[4];
                warp_softmax_16<D>(st, s_lo, s_hi, pa);
                warp_pv_16x16<D>(st, pa, smem_u32(vt), C::kHalfBytes, sl * 16);
            }
            if (wrote_smem) fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[s]);
        }

        // ---- epilogue: O / l -> bf16, optional LSE
        float l0 = st.l[0], l1 = st.l[1];
        l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
        l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
        if (!*abort_flag) {
            if (row_lo < L) {
                const float inv = 1.f / l0;
                uint32_t *orow = reinterpret_cast<uint32_t *>(p.o + b * p.o_sb + (int64_t)row_lo * p.o_st + h * p.o_sh);
#pragma unroll
                for (int nt = 0; nt < D / 8; ++nt)
                    orow[nt * 4 + (lane & 3)] = pack_bf16x2(st.o[nt][0] * inv, st.o[nt][1] * inv);
                if (p.lse && (lane & 3) == 0)
                    p.lse[((size_t)b * p.Hq + h) * p.S_max + row_lo] = (st.m[0] + log2f(l0)) * 0.6931471805599453f;
            }
            if (row_hi < L) {
                const float inv = 1.f / l1;
                uint32_t *orow = reinterpret_cast<uint32_t *>(p.o + b * p.o_sb + (int64_t)row_hi * p.o_st + h * p.o_sh);
#pragma unroll
                for (int nt = 0; nt < D / 8; ++nt)
                    orow[nt * 4 + (lane & 3)] = pack_bf16x2(st.o[nt][2] * inv, st.o[nt][3] * inv);
                if (p.lse && (lane & 3) == 0)
                    p.lse[((size_t)b * p.Hq + h) * p.S_max + row_hi] = (st.m[1] + log2f(l1)) * 0.6931471805599453f;
            }
        }
    }

    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) {
        atomicOr(p.status + kStatusErrWord, kErrPrefillWait);
        p.status[kStatusInfoWord] = 0x10000u | blockIdx.x;
    }
}

template <int D>
l4l_status launch_t(const CUtensorMap &tk, const CUtensorMap &tv, const PrefillMmaParams &p, int B, cudaStream_t stream)
{
    using C = PrefillMmaCfg<D>;
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(prefill_mma_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)C::kSmemBytes) != cudaSuccess)
            return L4L_ERR_CUDA;
        configured = true;
    }
    prefill_mma_kernel<D><<<dim3(p.n_qtiles, p.Hq, B), kThreads, C::kSmemBytes, stream>>>(tk, tv, p);
    return cudaGetLastError() == cudaSuccess ? L4L_OK : L4L_ERR_CUDA;
}

}  // namespace

l4l_status launch_prefill_mma(const l4l_tensor4 &q, const l4l_tensor4 &k, const l4l_tensor4 &v,
                              const l4l_tensor4 &o, const l4l_kv_cache &cache, const int32_t *d_seq_lens,
                              int S_max, int B, int Hq, int Hkv, int D, float scale, float *d_lse,
                              void *workspace, cudaStream_t stream)
{
    CUtensorMap tk, tv;
    TmapCoord ck, cv;
    if (!make_tmap_bf16(&tk, &ck, k.ptr, D, S_max, Hkv, B, k.stride_t, k.stride_h, k.stride_b, 64, kTile) ||
        !make_tmap_bf16(&tv, &cv, v.ptr, D, S_max, Hkv, B, v.stride_t, v.stride_h, v.stride_b, 64, kTile))
        return L4L_ERR_CUDA;
    if (ck.pos_t != cv.pos_t || ck.pos_h != cv.pos_h || ck.pos_b != cv.pos_b) return L4L_ERR_UNSUPPORTED;
    PrefillMmaParams p;
    p.q = static_cast<const __nv_bfloat16 *>(q.ptr);
    p.o = static_cast<__nv_bfloat16 *>(o.ptr);
    p.q_sb = q.stride_b; p.q_st = q.stride_t; p.q_sh = q.stride_h;
    p.o_sb = o.stride_b; p.o_st = o.stride_t; p.o_sh = o.stride_h;
    p.cache_k = static_cast<__nv_bfloat16 *>(cache.k);
    p.cache_v = static_cast<__nv_bfloat16 *>(cache.v);
    p.c_sb = cache.stride_b; p.c_sh = cache.stride_h; p.c_st = cache.stride_t;
    p.cache_max_len = cache.max_len;
    p.seq_lens = d_seq_lens;
    p.lse = d_lse;
    p.status = static_cast<unsigned *>(workspace);
    p.S_max = S_max; p.Hq = Hq; p.Hkv = Hkv; p.G = Hq / Hkv;
    p.n_qtiles = (S_max + kTile - 1) / kTile;
    p.scale_log2e = scale * 1.4426950408889634f;
    p.coord = ck;
    if (B > 65535 || Hq > 65535) return L4L_ERR_UNSUPPORTED;
    return (D == 128) ? launch_t<128>(tk, tv, p, B, stream) : launch_t<64>(tk, tv, p, B, stream);
}

}  // namespace l4l
