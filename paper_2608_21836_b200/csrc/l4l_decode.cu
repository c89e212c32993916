// Decode attention: one query token per sequence over a ragged bf16 KV cache.
//
// Pass 1 (decode_split_kernel): persistent CTAs stream the cache exactly once. A work item is
// (sequence, KV head, chunk of `chunk` tokens); items are enumerated from the device-side
// lengths (prefix sum over sequences) and dealt round-robin to the CTAs. One producer warp
// keeps a ring of TMA tiles (64 tokens of K and V, 128-byte swizzle) full across item
// boundaries; four consumer warps each take 16 tokens of every tile and serve ALL query heads
// of the KV group from it: the group is the M dimension (zero padded to 16) of warp-level
// bf16 MMAs, so the cache bytes are read once per group. Softmax statistics are fp32, row
// maxima are reduced with warp shuffles, and the four warps' partial results are merged
// through shared memory at the end of an item.
// Pass 2 (decode_merge_kernel): log-sum-exp merge of the chunk partials of each
// (sequence, query head); sequences that fit one chunk were already finished by pass 1.
#include "l4l_internal.h"
#include "l4l_warp_attn.cuh"

namespace l4l {

namespace {

constexpr int kTileT = 64;                 // tokens per TMA tile
constexpr int kConsumerWarps = 4;
constexpr int kThreads = (kConsumerWarps + 1) * 32;
constexpr int kMaxB = 1024;                // sequences per launch (prefix sums live in shared memory)

template <int D>
struct DecodeCfg {
    static constexpr int kHalves = D / 64;
    static constexpr uint32_t kHalfBytes = kTileT * 128;          // [64 tokens][64 dims] bf16
    static constexpr uint32_t kTileBytes = kHalves * kHalfBytes;  // one of K or V
    static constexpr uint32_t kStageBytes = 2 * kTileBytes;
    static constexpr int kStages = (D == 128) ? 3 : 6;
};

struct TileMeta {
    int b, kvh, t0, chunk_idx, kv_len, nchunks, flags, pad;
};
constexpr int kFlagFirst = 1, kFlagLast = 2, kFlagStop = 4;

struct DecodeParams {
    const __nv_bfloat16 *q;   // [B, Hq, D]
    __nv_bfloat16 *o;         // [B, Hq, D]
    float *lse;               // [B, Hq] or null
    const int32_t *kv_lens;   // [B]
    float *part_o;            // [B, Hq, nsplit, D]  normalised partial outputs
    float *part_lse;          // [B, Hq, nsplit]     log2-domain log-sum-exp of the chunk
    unsigned *status;
    int B, Hq, Hkv, G, chunk, nsplit;
    float scale_log2e;
    TmapCoord coord;
};

template <int D>
size_t decode_smem_bytes(int G)
{
    using C = DecodeCfg<D>;
    size_t comb = (size_t)kConsumerWarps * G * (D + 2) * sizeof(float);
    return 1024 /*alignment slack*/ + (size_t)C::kStages * C::kStageBytes + comb +
           C::kStages * sizeof(TileMeta) + (2 * C::kStages + 2) * sizeof(uint64_t) + (kMaxB + 1) * sizeof(int) + 64;
}

__device__ __forceinline__ void order_coords(const TmapCoord &c, int t, int h, int b, int &c1, int &c2, int &c3)
{
    c1 = (c.pos_t == 1) ? t : (c.pos_h == 1) ? h : b;
    c2 = (c.pos_t == 2) ? t : (c.pos_h == 2) ? h : b;
    c3 = (c.pos_t == 3) ? t : (c.pos_h == 3) ? h : b;
}

template <int D>
__global__ void __launch_bounds__(kThreads)
decode_split_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                    const DecodeParams p)
{
    using C = DecodeCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    uint8_t *smem = smem_raw + ((1024u - (raw & 1023u)) & 1023u);

    uint8_t *stages = smem;
    float *comb = reinterpret_cast<float *>(stages + (size_t)C::kStages * C::kStageBytes);
    const int comb_floats = kConsumerWarps * p.G * (D + 2);
    TileMeta *meta = reinterpret_cast<TileMeta *>(comb + comb_floats);
    uint64_t *full = reinterpret_cast<uint64_t *>(meta + C::kStages);
    uint64_t *empty = full + C::kStages;
    uint64_t *comb_bar = empty + C::kStages;   // [0]: partials written, [1]: partials consumed
    int *cum = reinterpret_cast<int *>(comb_bar + 2);
    volatile int *abort_flag = cum + (kMaxB + 1);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], kConsumerWarps);
        }
        mbar_init(&comb_bar[0], kConsumerWarps);
        mbar_init(&comb_bar[1], kConsumerWarps);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
    }
    __syncthreads();

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------------ producer warp
        // exclusive prefix sum of chunks per sequence
        int running = 0;
        for (int b0 = 0; b0 < p.B; b0 += 32) {
            const int b = b0 + lane;
            int n = 0;
            if (b < p.B) {
                int len = p.kv_lens[b];
                len = len < 0 ? 0 : len;
                n = (len + p.chunk - 1) / p.chunk;
                n = n > p.nsplit ? p.nsplit : n;   // lengths beyond the host bound are clipped
            }
            int incl = n;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                int t = __shfl_up_sync(0xffffffffu, incl, d);
                if (lane >= d) incl += t;
            }
            if (b < p.B) cum[b] = running + incl - n;
            running += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) cum[p.B] = running;
        __syncwarp();

        if (lane == 0) {
            tma_prefetch_desc(&tmap_k);
            tma_prefetch_desc(&tmap_v);
            const long long total_items = (long long)running * p.Hkv;
            uint32_t it = 0;
            bool ok = true;
            for (long long item = blockIdx.x; ok && item < total_items; item += gridDim.x) {
                const int pair = (int)(item / p.Hkv);
                const int kvh = (int)(item % p.Hkv);
                int lo = 0, hi = p.B;          // largest b with cum[b] <= pair
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (cum[mid] <= pair) lo = mid; else hi = mid;
                }
                const int b = lo;
                const int c = pair - cum[b];
                int len = p.kv_lens[b];
                const int cap = p.nsplit * p.chunk;
                len = len > cap ? cap : len;
                const int nchunks = cum[b + 1] - cum[b];
                const int t_begin = c * p.chunk;
                const int t_end = min(len, t_begin + p.chunk);
                int c1, c2, c3;
                for (int t0 = t_begin; t0 < t_end; t0 += kTileT, ++it) {
                    const uint32_t s = it % C::kStages;
                    const uint32_t ph = (it / C::kStages) & 1u;
                    if (!mbar_wait(&empty[s], ph ^ 1u, abort_flag)) { ok = false; break; }
                    TileMeta &mt = meta[s];
                    mt.b = b; mt.kvh = kvh; mt.t0 = t0; mt.chunk_idx = c; mt.kv_len = len; mt.nchunks = nchunks;
                    mt.flags = (t0 == t_begin ? kFlagFirst : 0) | (t0 + kTileT >= t_end ? kFlagLast : 0);
                    mbar_arrive_expect_tx(&full[s], C::kStageBytes);
                    uint8_t *dst = stages + (size_t)s * C::kStageBytes;
                    order_coords(p.coord, t0, kvh, b, c1, c2, c3);
#pragma unroll
                    for (int hf = 0; hf < C::kHalves; ++hf) {
                        tma_load_4d(dst + hf * C::kHalfBytes, &tmap_k, &full[s], hf * 64, c1, c2, c3);
                        tma_load_4d(dst + C::kTileBytes + hf * C::kHalfBytes, &tmap_v, &full[s], hf * 64, c1, c2, c3);
                    }
                }
            }
            if (ok) {
                const uint32_t s = it % C::kStages;
                const uint32_t ph = (it / C::kStages) & 1u;
                if (mbar_wait(&empty[s], ph ^ 1u, abort_flag)) {
                    meta[s].flags = kFlagStop;
                    mbar_arrive(&full[s]);
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ consumer warps
        WarpAttnState<D> st;
        st.reset();
        uint32_t qf[D / 16][4];
        const int r_lo = lane >> 2;          // query head within the group held in rows lane/4, lane/4+8
        const int r_hi = r_lo + 8;
        const int ctid = threadIdx.x;        // 0..127
        uint32_t item_par = 0;               // parity of the per-item merge barriers

        for (uint32_t it = 0;; ++it) {
            const uint32_t s = it % C::kStages;
            const uint32_t ph = (it / C::kStages) & 1u;
            if (!mbar_wait(&full[s], ph, abort_flag)) break;
            const TileMeta mt = meta[s];
            if (mt.flags & kFlagStop) break;

            if (mt.flags & kFlagFirst) {
                st.reset();
                const uint32_t *qrow_lo = reinterpret_cast<const uint32_t *>(
                    p.q + ((size_t)mt.b * p.Hq + (size_t)mt.kvh * p.G + r_lo) * D);
                const uint32_t *qrow_hi = qrow_lo + (size_t)8 * D / 2;
                const bool v_lo = r_lo < p.G, v_hi = r_hi < p.G;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const int w = ks * 8 + (lane & 3);               // 32-bit word index in the row
                    qf[ks][0] = v_lo ? __ldg(qrow_lo + w) : 0u;
                    qf[ks][1] = v_hi ? __ldg(qrow_hi + w) : 0u;
                    qf[ks][2] = v_lo ? __ldg(qrow_lo + w + 4) : 0u;
                    qf[ks][3] = v_hi ? __ldg(qrow_hi + w + 4) : 0u;
                }
            }

            const uint32_t k_tile = smem_u32(stages + (size_t)s * C::kStageBytes);
            const uint32_t v_tile = k_tile + C::kTileBytes;
            const int row0 = warp * 16;
            const int nvalid = mt.kv_len - (mt.t0 + row0);       // valid tokens in this warp's slice
            bool wrote_smem = false;
            if (nvalid > 0) {
                float s_lo[4], s_hi[4];
                warp_qk_16x16<D>(qf, k_tile, C::kHalfBytes, row0, s_lo, s_hi);
                const int tok = 2 * (lane & 3);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    s_lo[e] *= p.scale_log2e;
                    s_hi[e] *= p.scale_log2e;
                }
                if (nvalid < 16) {
                    // tokens past the end of the sequence: no weight, and their V rows (which may
                    // hold any bits, NaN included) are cleared so that 0 * garbage cannot appear
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        if (tok + (e & 1) >= nvalid) s_lo[e] = -INFINITY;
                        if (tok + (e & 1) + 8 >= nvalid) s_hi[e] = -INFINITY;
                    }
                    uint8_t *vt = stages + (size_t)s * C::kStageBytes + C::kTileBytes;
                    const int chunks_per_row = D / 8;
                    for (int i = lane; i < (16 - nvalid) * chunks_per_row; i += 32) {
                        const int r = row0 + nvalid + i / chunks_per_row;
                        const int ch = i % chunks_per_row;
                        *reinterpret_cast<uint4 *>(vt + (ch >> 3) * C::kHalfBytes + r * 128 + ((ch & 7) << 4)) =
                            make_uint4(0u, 0u, 0u, 0u);
                    }
                    wrote_smem = true;
                    __syncwarp();
                }
                uint32_t pa[4];
                warp_softmax_16<D>(st, s_lo, s_hi, pa);
                warp_pv_16x16<D>(st, pa, v_tile, C::kHalfBytes, row0);
            }

            const bool last = (mt.flags & kFlagLast) != 0;
            if (wrote_smem) fence_proxy_async_smem();   // generic writes before the next TMA fill
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[s]);

            if (last) {
                // ---- merge the four warps' (m, l, O) and emit the item's result
                float l0 = st.l[0], l1 = st.l[1];
                l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
                l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
                l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
                l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
                float *cw = comb + (size_t)warp * p.G * (D + 2);
                if (r_lo < p.G) {
                    float *row = cw + (size_t)r_lo * (D + 2);
                    if ((lane & 3) == 0) { row[D] = st.m[0]; row[D + 1] = l0; }
#pragma unroll
                    for (int nt = 0; nt < D / 8; ++nt) {
                        row[nt * 8 + 2 * (lane & 3)] = st.o[nt][0];
                        row[nt * 8 + 2 * (lane & 3) + 1] = st.o[nt][1];
                    }
                }
                if (r_hi < p.G) {
                    float *row = cw + (size_t)r_hi * (D + 2);
                    if ((lane & 3) == 0) { row[D] = st.m[1]; row[D + 1] = l1; }
#pragma unroll
                    for (int nt = 0; nt < D / 8; ++nt) {
                        row[nt * 8 + 2 * (lane & 3)] = st.o[nt][2];
                        row[nt * 8 + 2 * (lane & 3) + 1] = st.o[nt][3];
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&comb_bar[0]);
                if (!mbar_wait(&comb_bar[0], item_par, abort_flag)) break;
                for (int idx = ctid; idx < p.G * D; idx += kConsumerWarps * 32) {
                    const int r = idx / D, d = idx % D;
                    float mstar = -INFINITY;
#pragma unroll
                    for (int w = 0; w < kConsumerWarps; ++w)
                        mstar = fmaxf(mstar, comb[((size_t)w * p.G + r) * (D + 2) + D]);
                    float acc = 0.f, lsum = 0.f;
#pragma unroll
                    for (int w = 0; w < kConsumerWarps; ++w) {
                        const float *row = comb + ((size_t)w * p.G + r) * (D + 2);
                        const float wgt = fast_exp2(row[D] - mstar);   // idle warp: m = -inf -> 0
                        acc += wgt * row[d];
                        lsum += wgt * row[D + 1];
                    }
                    const float val = acc / lsum;
                    const int head = mt.kvh * p.G + r;
                    const size_t bh = (size_t)mt.b * p.Hq + head;
                    const float lse2 = mstar + log2f(lsum);
                    if (mt.nchunks == 1) {
                        p.o[bh * D + d] = __float2bfloat16_rn(val);
                        if (d == 0 && p.lse) p.lse[bh] = lse2 * 0.6931471805599453f;
                    } else {
                        const size_t slot = bh * p.nsplit + mt.chunk_idx;
                        p.part_o[slot * D + d] = val;
                        if (d == 0) p.part_lse[slot] = lse2;
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&comb_bar[1]);
                if (!mbar_wait(&comb_bar[1], item_par, abort_flag)) break;
                item_par ^= 1u;
            }
        }
    }

    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) {
        atomicOr(p.status + kStatusErrWord, kErrDecodeWait);
        p.status[kStatusInfoWord] = blockIdx.x;
    }
}

// Pass 2: out[b,h,:] = sum_c w_c o_c / sum_c w_c with w_c = 2^(lse_c - max lse).
template <int D>
__global__ void __launch_bounds__(D) decode_merge_kernel(const DecodeParams p)
{
    const int h = blockIdx.x, b = blockIdx.y, d = threadIdx.x;
    int len = p.kv_lens[b];
    len = len < 0 ? 0 : len;
    int n = (len + p.chunk - 1) / p.chunk;
    n = n > p.nsplit ? p.nsplit : n;
    if (n == 1) return;                       // finished by pass 1
    const size_t bh = (size_t)b * p.Hq + h;
    if (n == 0) {
        p.o[bh * D + d] = __float2bfloat16_rn(0.f);
        if (d == 0 && p.lse) p.lse[bh] = -INFINITY;
        return;
    }
    const float *pl = p.part_lse + bh * p.nsplit;
    const float *po = p.part_o + bh * p.nsplit * D;
    float mstar = -INFINITY;
    for (int c = 0; c < n; ++c) mstar = fmaxf(mstar, pl[c]);
    float acc = 0.f, wsum = 0.f;
    for (int c = 0; c < n; ++c) {
        const float w = fast_exp2(pl[c] - mstar);
        acc += w * po[(size_t)c * D + d];
        wsum += w;
    }
    p.o[bh * D + d] = __float2bfloat16_rn(acc / wsum);
    if (d == 0 && p.lse) p.lse[bh] = (mstar + log2f(wsum)) * 0.6931471805599453f;
}

template <int D>
l4l_status launch_decode_t(const CUtensorMap &tk, const CUtensorMap &tv, const DecodeParams &p, int n_items_max,
                           cudaStream_t stream)
{
    static int blocks_per_sm[17] = {0};
    const size_t smem = decode_smem_bytes<D>(p.G);
    if (blocks_per_sm[p.G] == 0) {
        // the opt-in limit is per kernel: set it once to the largest group's need
        if (cudaFuncSetAttribute(decode_split_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)decode_smem_bytes<D>(16)) != cudaSuccess)
            return L4L_ERR_CUDA;
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, decode_split_kernel<D>, kThreads, smem) != cudaSuccess ||
            n < 1)
            return L4L_ERR_CUDA;
        blocks_per_sm[p.G] = n;
    }
    int grid = sm_count() * blocks_per_sm[p.G];
    if (grid > n_items_max) grid = n_items_max;
    if (grid < 1) grid = 1;
    decode_split_kernel<D><<<grid, kThreads, smem, stream>>>(tk, tv, p);
    // always launched: it also covers kv_len == 0 (writes zeros); single-chunk sequences return at once
    decode_merge_kernel<D><<<dim3(p.Hq, p.B), D, 0, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? L4L_OK : L4L_ERR_CUDA;
}

}  // namespace

DecodePlan plan_decode(int B, int Hq, int Hkv, int D, int max_kv_len, size_t ws_limit)
{
    // Largest chunk that still gives every CTA slot several items; then grown (fewer, larger
    // partials) until the partials fit the workspace the caller provided.
    const long long slots = 2ll * sm_count();
    int chunk = 1024;
    while (chunk > kTileT) {
        const long long items = (long long)B * Hkv * ((max_kv_len + chunk - 1) / chunk);
        if (items >= 8 * slots) break;
        chunk >>= 1;
    }
    DecodePlan pl;
    for (;; chunk <<= 1) {
        pl.chunk = chunk;
        pl.nsplit = max_kv_len > 0 ? (max_kv_len + chunk - 1) / chunk : 1;
        pl.ws_bytes = kStatusBytes + (size_t)B * Hq * pl.nsplit * (D + 1) * sizeof(float);
        if (pl.ws_bytes <= ws_limit || pl.nsplit == 1) break;
    }
    return pl;
}

l4l_status launch_decode(const void *q, void *o, const l4l_kv_cache &cache, const int32_t *d_kv_lens,
                         int max_kv_len, int B, int Hq, int Hkv, int D, float scale, float *d_lse,
                         void *workspace, const DecodePlan &plan, cudaStream_t stream)
{
    CUtensorMap tk, tv;
    TmapCoord coord, coord_v;
    if (!make_tmap_bf16(&tk, &coord, cache.k, D, cache.max_len, Hkv, B, cache.stride_t, cache.stride_h,
                        cache.stride_b, 64, kTileT) ||
        !make_tmap_bf16(&tv, &coord_v, cache.v, D, cache.max_len, Hkv, B, cache.stride_t, cache.stride_h,
                        cache.stride_b, 64, kTileT))
        return L4L_ERR_CUDA;

    uint8_t *ws = static_cast<uint8_t *>(workspace);
    for (int b0 = 0; b0 < B; b0 += kMaxB) {
        const int nb = (B - b0 < kMaxB) ? (B - b0) : kMaxB;
        DecodeParams p;
        p.q = static_cast<const __nv_bfloat16 *>(q) + (size_t)b0 * Hq * D;
        p.o = static_cast<__nv_bfloat16 *>(o) + (size_t)b0 * Hq * D;
        p.lse = d_lse ? d_lse + (size_t)b0 * Hq : nullptr;
        p.kv_lens = d_kv_lens + b0;
        p.part_o = reinterpret_cast<float *>(ws + kStatusBytes) + (size_t)b0 * Hq * plan.nsplit * D;
        p.part_lse = reinterpret_cast<float *>(ws + kStatusBytes) + (size_t)B * Hq * plan.nsplit * D +
                     (size_t)b0 * Hq * plan.nsplit;
        p.status = reinterpret_cast<unsigned *>(ws);
        p.B = nb; p.Hq = Hq; p.Hkv = Hkv; p.G = Hq / Hkv; p.chunk = plan.chunk; p.nsplit = plan.nsplit;
        p.scale_log2e = scale * 1.4426950408889634f;
        p.coord = coord;
        // batch slices address the cache through the tensor map: shift the batch coordinate
        // by rebuilding the maps on the slice's base pointer
        CUtensorMap tks = tk, tvs = tv;
        if (b0 > 0) {
            const __nv_bfloat16 *kb = static_cast<const __nv_bfloat16 *>(cache.k) + (size_t)b0 * cache.stride_b;
            const __nv_bfloat16 *vb = static_cast<const __nv_bfloat16 *>(cache.v) + (size_t)b0 * cache.stride_b;
            if (!make_tmap_bf16(&tks, &coord, kb, D, cache.max_len, Hkv, nb, cache.stride_t, cache.stride_h,
                                cache.stride_b, 64, kTileT) ||
                !make_tmap_bf16(&tvs, &coord_v, vb, D, cache.max_len, Hkv, nb, cache.stride_t, cache.stride_h,
                                cache.stride_b, 64, kTileT))
                return L4L_ERR_CUDA;
            p.coord = coord;
        }
        const long long items = (long long)nb * Hkv * plan.nsplit;
        const int n_items_max = items > (1ll << 30) ? (1 << 30) : (int)items;
        l4l_status st = (D == 128) ? launch_decode_t<128>(tks, tvs, p, n_items_max, stream)
                                   : launch_decode_t<64>(tks, tvs, p, n_items_max, stream);
        if (st != L4L_OK) return st;
    }
    return L4L_OK;
}

}  // namespace l4l
