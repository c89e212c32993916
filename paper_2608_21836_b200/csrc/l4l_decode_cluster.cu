// Decode attention for small batches: one thread-block cluster per (sequence, KV head).
//
// When the whole problem is a handful of tiles per SM, a decode step is a chain of latencies, not a stream:
// the split kernel's workspace round trips (partials -> fence -> ticket -> partial loads) then cost more than
// the attention itself. Here the CTAs that share a (sequence, KV head) form a cluster of C = 1, 2, 4 or 8 CTAs: CTA
// `rank` streams the rank-th share of the sequence's 128-token tiles, the eight consumer warps merge their
// results in shared memory, and after ONE cluster barrier every CTA reads the C partials straight out of its
// peers' shared memory (distributed shared memory) and writes its 1/C of the output rows. No workspace, no
// atomics, no global-memory fence.
//
//   warp 8      TMA producer: the group's query rows with the first tile, then K/V tiles (128-byte swizzle)
//               through a small ring; the last tile of a sequence in 16-token groups
//   warps 0-7   16 tokens of every tile each, all query heads of the KV group as the M dimension of the warp
//               MMAs (the same building blocks as the split kernel), fused append of the step's new token
//
// bf16 cache (contiguous or paged, with or without the fused append and the rotary embedding (+ RMS norm) of the step's
// q and k) or fp8 (e4m3) cache with per-KV-head scales (contiguous or paged; 256-token tiles, 32 tokens per warp and
// tile, bytes widened to f16 in registers as in the split kernel).
#include <cstdlib>
#include <mutex>

#include "l4l_fp8_quant.cuh"
#include "l4l_internal.h"
#include "l4l_rope_frag.cuh"
#include "l4l_warp_attn.cuh"

namespace l4l {

namespace {

constexpr int kW = 8;                          // consumer warps
constexpr int kThreads = (kW + 1) * 32;
constexpr int kMaxCluster = 8;             // the portable limit; wider clusters schedule in too few places to pay

// F8: the cache holds e4m3 bytes (one byte per value, head_dim 128); a consumer warp then takes 32 tokens per tile.
template <int D, bool F8>
struct ClusterCfg {
    static_assert(!F8 || D == 128, "the fp8 path wants one 128-byte row per token");
    static constexpr int kSub = F8 ? 2 : 1;                          // 16-token blocks a consumer warp takes per tile
    static constexpr int kTileT = 16 * kW * kSub;                    // tokens per tile
    static constexpr int kRowBytes = F8 ? D : 2 * D;                 // one token of one KV head
    static constexpr int kHalves = kRowBytes / 128;                  // 128-byte column blocks of a tile
    static constexpr int kBoxD = F8 ? 128 : 64;                      // elements per 128-byte box row
    static constexpr uint32_t kHalfBytes = kTileT * 128;             // [tile tokens][128 bytes], swizzled
    static constexpr uint32_t kTileBytes = kHalves * kHalfBytes;     // one of K or V
    static constexpr uint32_t kStageBytes = 2 * kTileBytes;
    static constexpr int kPitch = D + 4;                             // floats per row: O[D], max, sum, pad
    static constexpr int kMaxStages = (kStageBytes >= 65536u) ? 3 : 6;
};

struct ClusterParams {
    const __nv_bfloat16 *q;   // [B, Hq, D]
    __nv_bfloat16 *o;         // [B, Hq, D]
    float *lse;               // [B, Hq] or null
    const int32_t *kv_lens;   // [B]
    const __nv_bfloat16 *k_new, *v_new;       // fused append (null: none): element (b, kv head, d) at b*new_sb + kvh*new_sh + d
    int64_t new_sb, new_sh;
    __nv_bfloat16 *cache_k, *cache_v;
    int64_t c_sb, c_sh, c_st;
    unsigned *status;
    const int32_t *block_table;               // paged cache (null: contiguous)
    int table_stride, page_size, page_shift, num_pages;
    int tail_rows;                            // tokens per box of the tail maps (32, or the page size if that is smaller)
    // rotary embedding (+ optional RMS norm) of the step's q and k_new (null: inputs are final); only with the fused
    // append. The new token's position is kv_len - 1.
    const float *rope_cos, *rope_sin;         // [rope_n_pos, D/2]
    const float *q_weight, *k_weight;         // [D] or null
    float norm_eps;
    int rope_n_pos;
    const float *k_scale, *v_scale;           // fp8 cache: real value = e4m3 value * scale of its KV head, [Hkv]
    int B, Hq, Hkv, G, C, max_kv_len, stages;
    int stream_once;          // load K/V with the L2 evict-first policy (large caches)
    float scale_log2e;
    TmapCoord coord;
};

template <int D, bool F8>
size_t cluster_smem_bytes(int G, int stages)
{
    using C = ClusterCfg<D, F8>;
    return 1024 /*alignment slack*/ + (size_t)stages * C::kStageBytes + (size_t)G * D * 2 +
           (size_t)(kW + 1) * G * C::kPitch * sizeof(float) + 4 * D * sizeof(float) +
           2 * C::kMaxStages * sizeof(uint64_t) + 64;
}

__device__ __forceinline__ void order_coords(const TmapCoord &c, int t, int h, int b, int &c1, int &c2, int &c3)
{
    c1 = (c.pos_t == 1) ? t : (c.pos_h == 1) ? h : b;
    c2 = (c.pos_t == 2) ? t : (c.pos_h == 2) ? h : b;
    c3 = (c.pos_t == 3) ? t : (c.pos_h == 3) ? h : b;
}

// Cluster-wide barrier in two halves, so that work that needs no peer can sit between them. Hardware
// barrier (no spinning): every thread of every CTA of the cluster executes both halves exactly once per use.
__device__ __forceinline__ void cluster_arrive()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait()
{
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Address of the same shared-memory location in the CTA of the given rank of this cluster.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t smem_addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "r"(addr)
                 : "memory");
    return v;
}
__device__ __forceinline__ float2 ld_cluster_f2(uint32_t addr)
{
    float2 v;
    asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr) : "memory");
    return v;
}

template <int D, bool F8>
__global__ void __launch_bounds__(kThreads, 1)
decode_cluster_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                      const __grid_constant__ CUtensorMap tmap_k_tail, const __grid_constant__ CUtensorMap tmap_v_tail,
                      const ClusterParams p)
{
    using C = ClusterCfg<D, F8>;
    constexpr int kPitch = C::kPitch, kVec = D / 4, kTileT = C::kTileT;
    constexpr uint32_t kHalfBytes = C::kHalfBytes;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    // the same offset in every CTA of the cluster (the dynamic segment starts at the same shared address)
    uint8_t *smem = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
    uint8_t *stages = smem;
    uint8_t *q_smem = stages + (size_t)p.stages * C::kStageBytes;
    const uint32_t q_bytes = (uint32_t)p.G * D * 2;
    float *comb = reinterpret_cast<float *>(q_smem + q_bytes);       // [kW][G][kPitch] per-warp results
    float *part = comb + (size_t)kW * p.G * kPitch;                  // [G][kPitch] this CTA's merged partial
    float *rope_cs = part + (size_t)p.G * kPitch;                    // cos | sin of the new token's position
    float *norm_w = rope_cs + D;                                     // q_weight | k_weight
    constexpr uint32_t kRopeBytes = D * 4;
    // fused append: the step's new k row and v row (bf16), fetched with the first tile so that the warp that patches
    // them into the last tile does not wait for global memory there
    uint8_t *new_rows = reinterpret_cast<uint8_t *>(norm_w + 2 * D);
    constexpr uint32_t kNewBytes = 2 * D * 2;
    uint64_t *full = reinterpret_cast<uint64_t *>(new_rows + kNewBytes);
    uint64_t *empty = full + C::kMaxStages;
    uint64_t *q_rotated = empty + C::kMaxStages;     // consumers among themselves: the query rows have been rotated in place
    volatile int *abort_flag = reinterpret_cast<volatile int *>(q_rotated + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = blockIdx.x;                 // cluster = the gridDim.x CTAs of one blockIdx.y
    const int unit = blockIdx.y;
    const int b = unit / p.Hkv, kvh = unit % p.Hkv;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], kW);
        }
        mbar_init(q_rotated, kW);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
    }
    if (warp == kW && lane == 0) {
        tma_prefetch_desc(&tmap_k);
        tma_prefetch_desc(&tmap_v);
        tma_prefetch_desc(&tmap_k_tail);
        tma_prefetch_desc(&tmap_v_tail);
    }
    // Programmatic dependent launch: everything above overlaps the tail of the previous kernel of the stream
    grid_dependency_wait();
    grid_launch_dependents();
    int len = __ldg(p.kv_lens + b);
    len = len < 0 ? 0 : (len > p.max_kv_len ? (p.k_new ? 0 : p.max_kv_len) : len);   // over the host's bound: decode ignores the extra tokens, a fused append treats the sequence as empty
    const bool with_rope = p.rope_cos != nullptr && len - 1 < p.rope_n_pos;   // a position outside the table: rows stay as they are
    // fused append over a paged cache: the page of the new token's slot, looked up now rather than when its tile arrives
    long long new_page = b;
    if (p.k_new != nullptr && p.block_table != nullptr && len > 0)
        new_page = __ldg(p.block_table + (size_t)b * p.table_stride + ((len - 1) >> p.page_shift));
    if (p.rope_cos != nullptr) {
        for (int i = threadIdx.x; i < D; i += kThreads) {
            norm_w[i] = p.q_weight ? __ldg(p.q_weight + i) : 1.f;
            norm_w[D + i] = p.k_weight ? __ldg(p.k_weight + i) : 1.f;
        }
    }
    __syncthreads();

    // this CTA's share of the sequence's tiles: as even as whole tiles allow
    const int tiles_b = (len + kTileT - 1) / kTileT;
    const int t_begin = (int)(((long long)rank * tiles_b) / p.C);
    const int t_end = (int)(((long long)(rank + 1) * tiles_b) / p.C);
    const int n_mine = t_end - t_begin;

    if (warp == kW) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            const bool paged = p.block_table != nullptr;
            const int32_t *pages = paged ? p.block_table + (size_t)b * p.table_stride : nullptr;
            // a large cache is read once per step: its lines go first; a small one stays L2-resident between steps
            const uint64_t stream_policy = p.stream_once ? l2_policy_evict_first() : l2_policy_evict_normal();
            for (int it = 0; it < n_mine; ++it) {
                const int tile = t_begin + it;
                const uint32_t s = it % p.stages, ph = (it / p.stages) & 1u;
                if (!mbar_wait(&empty[s], ph ^ 1u, abort_flag)) break;
                // The last tile of a sequence: if at most half of it holds tokens it comes in groups of p.tail_rows
                // tokens (a few small boxes), else as a whole tile like the others (rows past the end of the sequence are
                // never looked at, rows past the end of the cache arrive as zeros); with pages smaller than a tile only
                // the pages that hold tokens are fetched. Neither a box nor a group straddles pages.
                const int rem = len - tile * kTileT;
                const int groups = (rem + p.tail_rows - 1) / p.tail_rows;
                const bool by_groups = rem < kTileT && groups * p.tail_rows * 2 <= kTileT;
                const int box_rows = by_groups ? p.tail_rows : ((paged && p.page_size < kTileT) ? p.page_size : kTileT);
                const int n_box = by_groups ? groups : ((rem >= kTileT || box_rows == kTileT) ? kTileT / box_rows
                                                                                              : (rem + box_rows - 1) / box_rows);
                const uint32_t kv_bytes = (uint32_t)n_box * box_rows * 128u * C::kHalves * 2u;
                mbar_arrive_expect_tx(&full[s], kv_bytes + (it == 0 ? q_bytes + (with_rope ? kRopeBytes : 0u) +
                                                                              (p.k_new != nullptr ? kNewBytes : 0u) : 0u));
                if (it == 0) {
                    bulk_load_1d(q_smem, p.q + ((size_t)b * p.Hq + (size_t)kvh * p.G) * D, q_bytes, &full[s]);
                    if (p.k_new != nullptr) {
                        const size_t src = (size_t)b * p.new_sb + (size_t)kvh * p.new_sh;
                        bulk_load_1d(new_rows, p.k_new + src, kNewBytes / 2, &full[s]);
                        bulk_load_1d(new_rows + kNewBytes / 2, p.v_new + src, kNewBytes / 2, &full[s]);
                    }
                    if (with_rope) {
                        bulk_load_1d(rope_cs, p.rope_cos + (size_t)(len - 1) * (D / 2), kRopeBytes / 2, &full[s]);
                        bulk_load_1d(rope_cs + D / 2, p.rope_sin + (size_t)(len - 1) * (D / 2), kRopeBytes / 2, &full[s]);
                    }
                }
                uint8_t *dst = stages + (size_t)s * C::kStageBytes;
                int c1, c2, c3;
                const CUtensorMap *tk = by_groups ? &tmap_k_tail : &tmap_k;
                const CUtensorMap *tv = by_groups ? &tmap_v_tail : &tmap_v;
                int page_of[kTileT / 16];                            // looked up together: independent loads
#pragma unroll
                for (int bx = 0; bx < kTileT / 16; ++bx)
                    page_of[bx] = (paged && bx < n_box) ? __ldg(pages + ((tile * kTileT + bx * box_rows) >> p.page_shift)) : b;
#pragma unroll
                for (int bx = 0; bx < kTileT / 16; ++bx) {
                    if (bx >= n_box) break;
                    int tt = tile * kTileT + bx * box_rows;
                    if (paged) tt &= p.page_size - 1;
                    order_coords(p.coord, tt, kvh, page_of[bx], c1, c2, c3);
                    uint8_t *db = dst + bx * box_rows * 128;          // whole 8-row groups: the swizzle phase is kept
#pragma unroll
                    for (int hf = 0; hf < C::kHalves; ++hf) {
                        tma_load_4d_policy(db + hf * kHalfBytes, tk, &full[s], hf * C::kBoxD, c1, c2, c3, stream_policy);
                        tma_load_4d_policy(db + C::kTileBytes + hf * kHalfBytes, tv, &full[s], hf * C::kBoxD, c1, c2, c3, stream_policy);
                    }
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ consumer warps
        WarpAttnState<D> st;
        st.reset();
        uint32_t qf[D / 16][4];
        const int r_lo = lane >> 2, r_hi = r_lo + 8;    // query heads of the group held in rows lane/4, lane/4 + 8
        float k_sc = 1.f, v_sc = 1.f;                   // fp8 cache: scales of this KV head
        if constexpr (F8) {
            k_sc = __ldg(p.k_scale + kvh);
            v_sc = __ldg(p.v_scale + kvh);
        }
        for (int it = 0; it < n_mine; ++it) {
            const uint32_t s = it % p.stages, ph = (it / p.stages) & 1u;
            if (!mbar_wait(&full[s], ph, abort_flag)) break;
            if (it == 0) {
                if (with_rope) {
                    // rope fused into the step: the query rows are rotated in place in shared memory, row g by consumer
                    // warp g mod kW, before anybody builds fragments from them (small code: it runs once, from a cold
                    // instruction cache)
                    for (int g = warp; g < p.G; g += kW)
                        rope_row_in_smem<D>(reinterpret_cast<uint32_t *>(q_smem) + (size_t)g * (D / 2), rope_cs, p.q_weight != nullptr,
                                            p.norm_eps, norm_w, lane);
                    __syncwarp();
                    if (lane == 0) mbar_arrive(q_rotated);
                    if (!mbar_wait(q_rotated, 0u, abort_flag)) break;
                }
                const uint32_t *qs = reinterpret_cast<const uint32_t *>(q_smem);
                const uint32_t *qrow_lo = qs + (size_t)r_lo * D / 2;
                const uint32_t *qrow_hi = qs + (size_t)r_hi * D / 2;
                const bool v_lo = r_lo < p.G, v_hi = r_hi < p.G;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    if constexpr (F8) {
                        // f16 fragments with the k index permuted the way the fp8 K tiles arrive
                        const int w = q_frag_f8_word(ks, 0, lane);
                        qf[ks][0] = v_lo ? bf16x2_to_f16x2(qrow_lo[w]) : 0u;
                        qf[ks][1] = v_hi ? bf16x2_to_f16x2(qrow_hi[w]) : 0u;
                        qf[ks][2] = v_lo ? bf16x2_to_f16x2(qrow_lo[w + 1]) : 0u;
                        qf[ks][3] = v_hi ? bf16x2_to_f16x2(qrow_hi[w + 1]) : 0u;
                    } else {
                        const int w = ks * 8 + (lane & 3);           // 32-bit word index in the row
                        qf[ks][0] = v_lo ? qrow_lo[w] : 0u;
                        qf[ks][1] = v_hi ? qrow_hi[w] : 0u;
                        qf[ks][2] = v_lo ? qrow_lo[w + 4] : 0u;
                        qf[ks][3] = v_hi ? qrow_hi[w + 4] : 0u;
                    }
                }
            }
            const int t0 = (t_begin + it) * kTileT;
            const uint32_t k_tile = smem_u32(stages + (size_t)s * C::kStageBytes);
            const uint32_t v_tile = k_tile + C::kTileBytes;
            const int row0 = warp * 16 * C::kSub;
            const int nvalid = len - (t0 + row0);                    // valid tokens in this warp's slice
            bool wrote_smem = false;
            if (!F8 && p.k_new != nullptr && nvalid > 0 && nvalid <= 16) {
                // fused append: this slice holds the sequence's newest token. Its K/V arrive from the caller, not
                // from the cache: patch the tile in shared memory and write the cache slot (exactly one warp of
                // one CTA owns it)
                const int last = row0 + nvalid - 1;
                constexpr int kChunks = D / 8;
                uint4 kk = make_uint4(0u, 0u, 0u, 0u), vv = kk;
                if (lane < kChunks) {
                    kk = reinterpret_cast<const uint4 *>(new_rows)[lane];
                    vv = reinterpret_cast<const uint4 *>(new_rows + kNewBytes / 2)[lane];
                }
                if (p.rope_cos != nullptr)                                      // all lanes: shuffles inside
                    kk = rope_k_row<D>(kk, p.k_weight != nullptr, p.norm_eps, rope_cs, norm_w + D, with_rope, lane);
                if (lane < kChunks) {
                    // the slot in the cache: with pages, behind the block table. No page there: nothing is written,
                    // and the tile keeps the zeros that the fetch of a missing page delivers.
                    long long outer = b, slot = len - 1;
                    if (p.block_table != nullptr) {
                        outer = new_page;
                        slot &= p.page_size - 1;
                    }
                    if (p.block_table == nullptr || (outer >= 0 && outer < p.num_pages)) {
                        uint8_t *kt = stages + (size_t)s * C::kStageBytes;
                        const uint32_t off = (lane >> 3) * kHalfBytes + swz128(last, lane & 7);
                        *reinterpret_cast<uint4 *>(kt + off) = kk;
                        *reinterpret_cast<uint4 *>(kt + C::kTileBytes + off) = vv;
                        const size_t dst = (size_t)outer * p.c_sb + (size_t)kvh * p.c_sh + (size_t)slot * p.c_st + lane * 8;
                        *reinterpret_cast<uint4 *>(p.cache_k + dst) = kk;
                        *reinterpret_cast<uint4 *>(p.cache_v + dst) = vv;
                    }
                }
                wrote_smem = true;
                __syncwarp();
            }
            if constexpr (F8) {
                if (p.k_new != nullptr && nvalid > 0 && nvalid <= 16 * C::kSub) {
                    // fused append into an fp8 cache: the newest token's K/V rows are quantised here exactly as the
                    // cache update quantises them (same division, same rounding), patched into the tile and written
                    // to their cache slot; 8 lanes, 16 values each
                    const int last = row0 + nvalid - 1;
                    // the k row: straight from the caller, or (rope fused into the step) rotated first, in the
                    // arrangement of the bf16 path (8 values per lane), rounded to bf16 and regrouped
                    uint4 ka = make_uint4(0u, 0u, 0u, 0u), kb = ka;
                    if (p.rope_cos != nullptr) {
                        uint4 kk = make_uint4(0u, 0u, 0u, 0u);
                        if (lane < D / 8) kk = reinterpret_cast<const uint4 *>(new_rows)[lane];
                        kk = rope_k_row<D>(kk, p.k_weight != nullptr, p.norm_eps, rope_cs, norm_w + D, with_rope, lane);
                        regroup_row_16(kk, lane, ka, kb);
                    } else if (lane < 8) {
                        ka = reinterpret_cast<const uint4 *>(new_rows)[2 * lane];
                        kb = reinterpret_cast<const uint4 *>(new_rows)[2 * lane + 1];
                    }
                    if (lane < 8) {
                        const uint4 *vs = reinterpret_cast<const uint4 *>(new_rows + kNewBytes / 2);
                        const uint4 kq = quantise16(ka, kb, k_sc);
                        const uint4 vq = quantise16(vs[2 * lane], vs[2 * lane + 1], v_sc);
                        long long outer = b, slot = len - 1;
                        if (p.block_table != nullptr) {
                            outer = new_page;
                            slot &= p.page_size - 1;
                        }
                        if (p.block_table == nullptr || (outer >= 0 && outer < p.num_pages)) {
                            uint8_t *kt = stages + (size_t)s * C::kStageBytes;
                            const uint32_t off = swz128(last, lane);
                            *reinterpret_cast<uint4 *>(kt + off) = kq;
                            *reinterpret_cast<uint4 *>(kt + C::kTileBytes + off) = vq;
                            // fp8 caches: the strides count bytes
                            const size_t dst = (size_t)outer * p.c_sb + (size_t)kvh * p.c_sh + (size_t)slot * p.c_st + lane * 16;
                            *reinterpret_cast<uint4 *>(reinterpret_cast<uint8_t *>(p.cache_k) + dst) = kq;
                            *reinterpret_cast<uint4 *>(reinterpret_cast<uint8_t *>(p.cache_v) + dst) = vq;
                        }
                    }
                    wrote_smem = true;
                    __syncwarp();
                }
                if (nvalid > 0) {
                    // 32 tokens per step: two 16-token blocks share one softmax update. A block with no valid token is
                    // skipped (its rows may never have been fetched); in the last valid block the tokens past the end
                    // get no weight and their V rows are cleared.
                    constexpr int kSub = C::kSub;
                    float sv[2 * kSub][4];
                    const float sc = p.scale_log2e * k_sc;
#pragma unroll
                    for (int u = 0; u < kSub; ++u) {
                        if (u == 0 || nvalid > 16 * u) {
                            warp_qk_16x16_f8<D>(qf, k_tile, row0 + 16 * u, sv[2 * u], sv[2 * u + 1]);
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                sv[2 * u][e] *= sc;
                                sv[2 * u + 1][e] *= sc;
                            }
                        } else {
#pragma unroll
                            for (int e = 0; e < 4; ++e) sv[2 * u][e] = sv[2 * u + 1][e] = -INFINITY;
                        }
                    }
                    if (nvalid < 16 * kSub) {
                        const int tok = 2 * (lane & 3);
#pragma unroll
                        for (int j = 0; j < 2 * kSub; ++j)
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                if (8 * j + tok + (e & 1) >= nvalid) sv[j][e] = -INFINITY;
                        uint8_t *vt = stages + (size_t)s * C::kStageBytes + C::kTileBytes;
                        const int fetched_end = (nvalid + 15) & ~15;                 // end of the last valid block
                        for (int i = lane; i < (fetched_end - nvalid) * 8; i += 32)
                            *reinterpret_cast<uint4 *>(vt + (row0 + nvalid + i / 8) * 128 + ((i & 7) << 4)) =
                                make_uint4(0u, 0u, 0u, 0u);
                        wrote_smem = true;
                        __syncwarp();
                    }
                    uint32_t pa[kSub][4];
                    warp_softmax_tiles<D, true, 2 * kSub>(st, sv, pa);
#pragma unroll
                    for (int u = 0; u < kSub; ++u)
                        if (u == 0 || nvalid > 16 * u) warp_pv_16x16_f8<D>(st, pa[u], v_tile, row0 + 16 * u);
                }
            } else if (nvalid > 0) {
                float s_lo[4], s_hi[4];
                warp_qk_16x16<D>(qf, k_tile, kHalfBytes, row0, s_lo, s_hi);
                const int tok = 2 * (lane & 3);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    s_lo[e] *= p.scale_log2e;
                    s_hi[e] *= p.scale_log2e;
                }
                if (nvalid < 16) {
                    // tokens past the end of the sequence: no weight, and their V rows (any bits, NaN included)
                    // are cleared so that 0 * garbage cannot appear
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        if (tok + (e & 1) >= nvalid) s_lo[e] = -INFINITY;
                        if (tok + (e & 1) + 8 >= nvalid) s_hi[e] = -INFINITY;
                    }
                    uint8_t *vt = stages + (size_t)s * C::kStageBytes + C::kTileBytes;
                    constexpr int kChunksPerRow = D / 8;
                    for (int i = lane; i < (16 - nvalid) * kChunksPerRow; i += 32) {
                        const int r = row0 + nvalid + i / kChunksPerRow, ch = i % kChunksPerRow;
                        *reinterpret_cast<uint4 *>(vt + (ch >> 3) * kHalfBytes + r * 128 + ((ch & 7) << 4)) =
                            make_uint4(0u, 0u, 0u, 0u);
                    }
                    wrote_smem = true;
                    __syncwarp();
                }
                uint32_t pa[4];
                warp_softmax_16<D>(st, s_lo, s_hi, pa);
                warp_pv_16x16<D>(st, pa, v_tile, kHalfBytes, row0);
            }
            if (wrote_smem) fence_proxy_async_smem();   // generic writes before the next TMA fill
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[s]);
        }
        // ---- this warp's (max, sum, O) into shared memory
        float l0 = st.l[0], l1 = st.l[1];
        l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
        l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
        float *cw = comb + (size_t)warp * p.G * kPitch;
        // fp8: accumulator tiles alternate even / odd head dims (a tile pair gives this lane 4 consecutive dims) and O
        // still lacks the V scale of its KV head
        const float vs = F8 ? v_sc : 1.f;
        if (r_lo < p.G) {
            float *row = cw + (size_t)r_lo * kPitch;
            if ((lane & 3) == 0) { row[D] = st.m[0]; row[D + 1] = l0; }
            if constexpr (F8) {
#pragma unroll
                for (int ch = 0; ch < D / 16; ++ch)
                    *reinterpret_cast<float4 *>(row + ch * 16 + 4 * (lane & 3)) =
                        make_float4(st.o[2 * ch][0] * vs, st.o[2 * ch + 1][0] * vs, st.o[2 * ch][1] * vs, st.o[2 * ch + 1][1] * vs);
            } else {
#pragma unroll
                for (int nt = 0; nt < D / 8; ++nt)
                    *reinterpret_cast<float2 *>(row + nt * 8 + 2 * (lane & 3)) = make_float2(st.o[nt][0], st.o[nt][1]);
            }
        }
        if (r_hi < p.G) {
            float *row = cw + (size_t)r_hi * kPitch;
            if ((lane & 3) == 0) { row[D] = st.m[1]; row[D + 1] = l1; }
            if constexpr (F8) {
#pragma unroll
                for (int ch = 0; ch < D / 16; ++ch)
                    *reinterpret_cast<float4 *>(row + ch * 16 + 4 * (lane & 3)) =
                        make_float4(st.o[2 * ch][2] * vs, st.o[2 * ch + 1][2] * vs, st.o[2 * ch][3] * vs, st.o[2 * ch + 1][3] * vs);
            } else {
#pragma unroll
                for (int nt = 0; nt < D / 8; ++nt)
                    *reinterpret_cast<float2 *>(row + nt * 8 + 2 * (lane & 3)) = make_float2(st.o[nt][2], st.o[nt][3]);
            }
        }
    }
    __syncthreads();

    // ---- merge of the eight warps: every thread owns float4 pieces of the G x D partial (unnormalised, relative
    // to the CTA's row maximum). A warp (or a CTA) that saw no token has max = -inf and weight 0.
    const int items = p.G * kVec;
    for (int item = threadIdx.x; item < items; item += kThreads) {
        const int r = item / kVec, d4 = item % kVec;
        float mw[kW];
        float mstar = -INFINITY;
#pragma unroll
        for (int w = 0; w < kW; ++w) {
            mw[w] = comb[((size_t)w * p.G + r) * kPitch + D];
            mstar = fmaxf(mstar, mw[w]);
        }
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float lsum = 0.f;
#pragma unroll
        for (int w = 0; w < kW; ++w) {
            const float *row = comb + ((size_t)w * p.G + r) * kPitch;
            const float wgt = (mw[w] == -INFINITY) ? 0.f : fast_exp2(mw[w] - mstar);
            const float4 v = *reinterpret_cast<const float4 *>(row + d4 * 4);
            acc.x += wgt * v.x; acc.y += wgt * v.y; acc.z += wgt * v.z; acc.w += wgt * v.w;
            lsum += wgt * row[D + 1];
        }
        *reinterpret_cast<float4 *>(part + (size_t)r * kPitch + d4 * 4) = acc;
        if (d4 == 0) *reinterpret_cast<float2 *>(part + (size_t)r * kPitch + D) = make_float2(mstar, lsum);
    }
    __syncwarp();
    if (p.C > 1) {
        cluster_arrive();
        cluster_wait();
    } else {
        __syncthreads();
    }

    // ---- every CTA merges the C partials for its share of the output (peers' shared memory read directly)
    const int per = (items + p.C - 1) / p.C;
    for (int t = threadIdx.x; t < per; t += kThreads) {
        const int item = rank * per + t;
        if (item >= items) break;
        const int r = item / kVec, d4 = item % kVec;
        const uint32_t a_val = smem_u32(part + (size_t)r * kPitch + d4 * 4);
        const uint32_t a_ml = smem_u32(part + (size_t)r * kPitch + D);
        float2 ml[kMaxCluster];
        float4 val[kMaxCluster];
#pragma unroll
        for (int c = 0; c < kMaxCluster; ++c) {
            if (c < p.C) {
                ml[c] = ld_cluster_f2(map_to_rank(a_ml, c));
                val[c] = ld_cluster_f4(map_to_rank(a_val, c));
            } else {
                ml[c] = make_float2(-INFINITY, 0.f);
                val[c] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
        float mstar = -INFINITY;
#pragma unroll
        for (int c = 0; c < kMaxCluster; ++c) mstar = fmaxf(mstar, ml[c].x);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float lsum = 0.f;
#pragma unroll
        for (int c = 0; c < kMaxCluster; ++c) {
            const float wgt = (ml[c].x == -INFINITY) ? 0.f : fast_exp2(ml[c].x - mstar);
            acc.x += wgt * val[c].x; acc.y += wgt * val[c].y; acc.z += wgt * val[c].z; acc.w += wgt * val[c].w;
            lsum += wgt * ml[c].y;
        }
        // a sequence with no cached token gets o = 0, lse = -inf
        const float inv = len > 0 ? 1.f / lsum : 0.f;
        const size_t bh = (size_t)b * p.Hq + (size_t)kvh * p.G + r;
        uint2 packed;
        packed.x = pack_bf16x2(acc.x * inv, acc.y * inv);
        packed.y = pack_bf16x2(acc.z * inv, acc.w * inv);
        *reinterpret_cast<uint2 *>(p.o + bh * D + d4 * 4) = packed;
        if (d4 == 0 && p.lse) p.lse[bh] = len > 0 ? (mstar + log2f(lsum)) * 0.6931471805599453f : -INFINITY;
    }
    __syncwarp();
    // no CTA may leave while a peer can still read its shared memory
    if (p.C > 1) {
        cluster_arrive();
        cluster_wait();
    }
    if (threadIdx.x == 0 && *abort_flag) {
        atomicOr(p.status + kStatusErrWord, kErrDecodeWait);
        p.status[kStatusInfoWord] = 0x30000u | (blockIdx.y & 0xffffu);
    }
}

template <int D, bool F8>
bool configure_kernel()
{
    static bool done_on[kDeviceSlots] = {}, ok_on[kDeviceSlots] = {};
    const int slot = device_slot();
    if (slot < 0) return false;
    bool &done = done_on[slot], &ok = ok_on[slot];
    std::lock_guard<std::mutex> lock(setup_mutex());
    if (!done) {
        done = true;
        ok = cudaFuncSetAttribute(decode_cluster_kernel<D, F8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) ==
             cudaSuccess;
        if (!ok) (void)cudaGetLastError();
    }
    return ok;
}

// Shared-memory stages that fit beside the merge scratch (0: none do).
template <int D, bool F8>
int pick_stages(int G)
{
    for (int s = ClusterCfg<D, F8>::kMaxStages; s >= 2; --s)
        if (cluster_smem_bytes<D, F8>(G, s) <= 227 * 1024) return s;
    return 0;
}

// Clusters of C CTAs that the device can hold at once (0 if the shape cannot launch). Looked up once per shape.
template <int D, bool F8>
int resident_clusters(int C, size_t smem)
{
    struct Entry { int C; size_t smem; int dev; int n; };
    static Entry cache[32];
    static int n_cached = 0;
    static std::mutex mutex;
    const int dev = device_slot();
    if (dev < 0) return 0;
    if (!configure_kernel<D, F8>()) return 0;
    std::lock_guard<std::mutex> lock(mutex);
    for (int i = 0; i < n_cached; ++i)
        if (cache[i].C == C && cache[i].smem == smem && cache[i].dev == dev) return cache[i].n;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(C, 1, 1);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, decode_cluster_kernel<D, F8>, &cfg) != cudaSuccess) {
        (void)cudaGetLastError();
        n = 0;
    }
    if (n_cached < 32) cache[n_cached++] = Entry{C, smem, dev, n};
    return n;
}

// Host-side view of one instantiation.
struct ClusterShape {
    int tile_t;
    uint32_t stage_bytes;                      // K and V of one tile
    int (*stages)(int G);
    size_t (*smem)(int G, int stages);
    int (*resident)(int C, size_t smem);
    bool (*configure)();
};

template <int D, bool F8>
ClusterShape shape_of()
{
    return ClusterShape{ClusterCfg<D, F8>::kTileT, ClusterCfg<D, F8>::kStageBytes, &pick_stages<D, F8>, &cluster_smem_bytes<D, F8>, &resident_clusters<D, F8>,
                        &configure_kernel<D, F8>};
}

ClusterShape pick_cluster_shape(int D, bool fp8)
{
    if (fp8) return shape_of<128, true>();
    return D == 128 ? shape_of<128, false>() : shape_of<64, false>();
}

}  // namespace

int decode_cluster_width(int B, int Hq, int Hkv, int D, int max_kv_len, bool fp8)
{
    // tuning override: 0 keeps every call on the split kernel, N forces clusters of N where they fit
    const int forced = decode_override().cluster;
    if (forced == 0 || (fp8 && D != 128)) return 0;       // fp8 at head_dim 64 runs on the split kernel only
    const int G = Hq / Hkv;
    const long long units = (long long)B * Hkv;
    const int sms = sm_count();
    if (units <= 0 || units > 65535 || units > sms) return 0;
    const ClusterShape shape = pick_cluster_shape(D, fp8);
    const int stages = shape.stages(G);
    if (stages == 0) return 0;
    const size_t smem = shape.smem(G, stages);
    const int tiles_max = max_kv_len > 0 ? (max_kv_len + shape.tile_t - 1) / shape.tile_t : 1;
    // the widest power of two that keeps every cluster resident at once and gives every CTA at least one tile
    int C = 1;
    while (2 * C <= kMaxCluster && units * 2 * C <= sms && 2 * C <= tiles_max) C *= 2;
    if (forced > 0) {
        C = 1;
        while (2 * C <= forced && 2 * C <= kMaxCluster) C *= 2;
    }
    for (; C >= 1; C /= 2) {
        const int n = shape.resident(C, smem);
        if (n >= units || (forced > 0 && n > 0)) break;
    }
    if (C < 1) return 0;
    if (forced > 0) return C;
    // Beyond these bounds the even split of the whole tile stream over all SMs (the split kernel) wins: a lone CTA
    // per sequence streams at one SM's rate, and ragged lengths leave short sequences' CTAs idle.
    // (measured on ragged batches of 8 to 16 sequences of up to 4096 tokens: with one CTA per sequence the cluster
    // kernel wins up to about 1 MB of cache per CTA, with two or more up to about 2 MB)
    const long long per_cta_bytes = (long long)((tiles_max + C - 1) / C) * shape.stage_bytes;
    if (per_cta_bytes > (C == 1 ? (1ll << 20) : (2ll << 20))) return 0;
    return C;
}

l4l_status launch_decode_cluster(const void *q, void *o, const l4l_kv_cache &cache, const int32_t *d_kv_lens,
                                 int max_kv_len, int B, int Hq, int Hkv, int D, float scale, float *d_lse,
                                 void *workspace, cudaStream_t stream, const l4l_tensor4 *k_new,
                                 const l4l_tensor4 *v_new, const PagedTable *paged, const RopeArgs *rope,
                                 const Fp8Scales *fp8, int width)
{
    if (rope && (!k_new || !v_new)) return L4L_ERR_UNSUPPORTED;               // only with the fused append
    if (fp8 && D != 128) return L4L_ERR_UNSUPPORTED;
    // fp8: cache.k / cache.v point at e4m3 bytes, the strides count bytes (= elements)
    const int esz = fp8 ? 1 : 2, box_d = fp8 ? 128 : 64;
    const int G = Hq / Hkv;
    const ClusterShape shape = pick_cluster_shape(D, fp8 != nullptr);
    const int kTileT = shape.tile_t;
    const int stages = shape.stages(G);
    if (stages == 0 || width < 1 || width > kMaxCluster) return L4L_ERR_UNSUPPORTED;
    const size_t smem = shape.smem(G, stages);
    if (!shape.configure()) return L4L_ERR_CUDA;

    CUtensorMap tk, tv, tk_tail, tv_tail;   // tile-sized boxes, and small boxes for a mostly empty last tile of a sequence
    TmapCoord coord, coord_v;
    const int outer = paged ? paged->num_pages : B;
    // pages smaller than a tile are fetched page by page: no box may exceed the page
    const int box_t = (paged && cache.max_len < kTileT) ? cache.max_len : kTileT;
    const int tail_rows = (paged && cache.max_len < 32) ? cache.max_len : 32;
    if (!make_tmap(&tk, &coord, cache.k, D, cache.max_len, Hkv, outer, cache.stride_t, cache.stride_h, cache.stride_b, box_d,
                   box_t, esz) ||
        !make_tmap(&tv, &coord_v, cache.v, D, cache.max_len, Hkv, outer, cache.stride_t, cache.stride_h, cache.stride_b,
                   box_d, box_t, esz) ||
        !make_tmap(&tk_tail, &coord_v, cache.k, D, cache.max_len, Hkv, outer, cache.stride_t, cache.stride_h,
                   cache.stride_b, box_d, tail_rows, esz) ||
        !make_tmap(&tv_tail, &coord_v, cache.v, D, cache.max_len, Hkv, outer, cache.stride_t, cache.stride_h,
                   cache.stride_b, box_d, tail_rows, esz))
        return L4L_ERR_CUDA;
    ClusterParams p;
    p.q = static_cast<const __nv_bfloat16 *>(q);
    p.o = static_cast<__nv_bfloat16 *>(o);
    p.lse = d_lse;
    p.kv_lens = d_kv_lens;
    p.k_new = p.v_new = nullptr;
    p.new_sb = p.new_sh = 0;
    if (k_new && v_new) {
        if (k_new->stride_b != v_new->stride_b || k_new->stride_h != v_new->stride_h) return L4L_ERR_UNSUPPORTED;
        p.k_new = static_cast<const __nv_bfloat16 *>(k_new->ptr);
        p.v_new = static_cast<const __nv_bfloat16 *>(v_new->ptr);
        p.new_sb = k_new->stride_b; p.new_sh = k_new->stride_h;
    }
    p.cache_k = static_cast<__nv_bfloat16 *>(cache.k);
    p.cache_v = static_cast<__nv_bfloat16 *>(cache.v);
    p.c_sb = cache.stride_b; p.c_sh = cache.stride_h; p.c_st = cache.stride_t;
    p.status = static_cast<unsigned *>(workspace);
    p.block_table = paged ? paged->block_table : nullptr;
    p.table_stride = paged ? paged->table_stride : 0;
    p.page_size = paged ? cache.max_len : 0;
    p.num_pages = paged ? paged->num_pages : 0;
    p.tail_rows = tail_rows;
    p.page_shift = 0;
    while (paged && (1 << p.page_shift) < cache.max_len) ++p.page_shift;
    p.rope_cos = rope ? rope->cos : nullptr;
    p.rope_sin = rope ? rope->sin : nullptr;
    p.q_weight = rope ? rope->q_weight : nullptr;
    p.k_weight = rope ? rope->k_weight : nullptr;
    p.norm_eps = rope ? rope->eps : 0.f;
    p.rope_n_pos = rope ? rope->n_pos : 0;
    p.k_scale = fp8 ? fp8->k_scale : nullptr;
    p.v_scale = fp8 ? fp8->v_scale : nullptr;
    p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.G = G; p.C = width; p.max_kv_len = max_kv_len; p.stages = stages;
    p.stream_once = decode_streams_once(B, Hkv, D, max_kv_len, fp8 != nullptr) ? 1 : 0;
    p.scale_log2e = scale * 1.4426950408889634f;
    p.coord = coord;

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(width, B * Hkv, 1);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = width; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    const cudaError_t err =
        fp8        ? cudaLaunchKernelEx(&cfg, decode_cluster_kernel<128, true>, tk, tv, tk_tail, tv_tail, p)
        : D == 128 ? cudaLaunchKernelEx(&cfg, decode_cluster_kernel<128, false>, tk, tv, tk_tail, tv_tail, p)
                   : cudaLaunchKernelEx(&cfg, decode_cluster_kernel<64, false>, tk, tv, tk_tail, tv_tail, p);
    return err == cudaSuccess ? L4L_OK : L4L_ERR_CUDA;
}

}  // namespace l4l
