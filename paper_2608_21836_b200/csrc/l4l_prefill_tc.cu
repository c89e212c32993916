// Causal prefill on the 5th-generation tensor cores (tcgen05.mma, accumulators in tensor memory).
//
// One CTA owns two 128-row sub-tiles whose S = Q K^T and O += P V products ping-pong on the tensor
// pipe while the other sub-tile's softmax runs on the CUDA cores. The two sub-tiles are the same 128
// query rows of TWO query heads that share a KV head (query-head groups of even size: both sub-tiles
// then visit the same K/V tiles, their causal spans are equal, and work items are half as coarse), or
// 256 consecutive rows of ONE query head (odd group sizes, multi-head attention included).
//
//   warps 0-3   softmax of sub-tile 0: thread t owns row t (= TMEM lane t): reads S from TMEM,
//               keeps the running max / sum in fp32, writes P (bf16) back into TMEM over S
//   warps 4-7   the same for sub-tile 1
//   warp  8     TMA producer: Q once, then K_j, V_j tiles (128 tokens, 128-byte swizzle) through a
//               ring of shared-memory slots; afterwards copies the block's diagonal K/V tiles from
//               shared memory into the KV cache (only for the first query head of a KV group)
//   warp  9     MMA issuer (one lane): S_i = Q_i K_j^T from shared memory, O_i += P_i V_j with P read
//               from TMEM and V as an MN-major shared-memory operand; owns the TMEM allocation
//   warps 10-11 help with the cache copy, which runs beside the last iterations
//
// The same kernel serves a chunk of new tokens over a populated cache. The key axis of a sequence is then two runs
// of 128-token tiles: the `past` tokens cached before (tiles of the cache, contiguous or paged, aligned to slot 0;
// every query row sees all of them, the last tile may be partly filled) followed by the new tokens (tiles aligned
// to the chunk's first token, so the causal diagonal sits exactly as in a fresh prompt, which is the case past = 0).
// The new tokens' K/V come from the caller's tensors (and are written to the cache in the same pass) or, when the
// caller has appended them already, from the cache itself at slot past + row.
// A whole sub-tile's output leaves through the shared memory that held its Q rows and TMA stores.
//
// TMEM columns: S0 [0,128) S1 [128,256) O0 [256,256+D) O1 [256+D,256+2D); P_i aliases the first 64
// columns of S_i. Causal tile skipping: sub-tile i only visits K/V tiles up to its diagonal.
// The tensor pipe executes one thread's MMAs in issue order, which is what makes the S/P aliasing
// safe: QK_{j+1} into S_i is issued after PV_j that reads P_i.
#include "l4l_internal.h"
#include "l4l_ptx.cuh"

namespace l4l {

namespace {

constexpr int kRows = 128;                     // rows per sub-tile == tokens per K/V tile
constexpr int kThreads = 384;                  // 3 warpgroups: softmax 0, softmax 1, {producer, MMA, 2 idle}
constexpr uint32_t kHalfBytes = kRows * 128;   // [128 rows][64 bf16], 128-byte swizzled
constexpr float kRescaleThreshold = 8.f;       // log2 domain: O is rescaled only if the max grew by > 2^8

template <int D>
struct TcCfg {
    static constexpr int kHalves = D / 64;
    static constexpr uint32_t kTileBytes = kHalves * kHalfBytes;        // one Q sub-tile, K tile or V tile
    static constexpr int kSlots = (D == 128) ? 5 : 8;                    // ring of K/V tiles
    static constexpr uint32_t kTmemCols = 512;
    static constexpr uint32_t kColS0 = 0, kColS1 = 128, kColO0 = 256, kColO1 = 256 + D;
    static constexpr int kNumBars = 1 + 2 * kSlots + 8;
    static constexpr size_t kSmemBytes = 1024 + 2 * kTileBytes + (size_t)kSlots * kTileBytes + kNumBars * 8 + 64;
};

struct TcParams {
    __nv_bfloat16 *o;
    int64_t o_sb, o_st, o_sh;
    __nv_bfloat16 *cache_k, *cache_v;   // destination of the fused cache write (null: nothing is written)
    int64_t c_sb, c_sh, c_st;           // its strides (paged: c_sb is the stride between pages)
    int cache_slots;                    // token slots per sequence that may be written
    const int32_t *seq_lens;            // [B] new tokens per sequence (prompt or chunk length)
    const int32_t *past_lens;           // [B] tokens cached ahead of them, or null (none)
    const int32_t *block_table;         // paged cache: [B, table_stride] page ids; null: contiguous cache
    int table_stride, page_shift, page_size, num_pages;
    int new_at_past;                    // the new tokens' K/V are read from the cache itself: row r is slot past + r
    int cache_box_t;                    // token rows per TMA box of a cache tile (128, or the page size if smaller)
    float *lse;
    unsigned *status;
    int S_max, B, Hq, Hkv, G, n_qblocks;
    int pair_heads;                     // the two sub-tiles are two query heads of one KV group at the same 128 rows
    float scale_log2e;
    TmapCoord cq, ckv, co, ckc;         // ckv: maps of the new tokens' K/V; ckc: maps of the cache (tokens before)
};

__device__ __forceinline__ void order_coords(const TmapCoord &c, int t, int h, int b, int &c1, int &c2, int &c3)
{
    c1 = (c.pos_t == 1) ? t : (c.pos_h == 1) ? h : b;
    c2 = (c.pos_t == 2) ? t : (c.pos_h == 2) ? h : b;
    c3 = (c.pos_t == 3) ? t : (c.pos_h == 3) ? h : b;
}

// Shared-memory matrix descriptor, 128-byte swizzle, 8-row groups 1024 bytes apart.
// K-major operands ignore the leading byte offset; MN-major ones use it as the stride between
// 64-element chunks along M/N.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr, uint32_t lbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((1024u >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;                     // descriptor version for sm_100
    d |= (uint64_t)2 << 61;                     // SWIZZLE_128B
    return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, M = 128.
__host__ __device__ constexpr uint32_t make_idesc(int n, bool b_mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(kRows >> 4) << 24);
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                  const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_o,
                  const __grid_constant__ CUtensorMap tmap_kc, const __grid_constant__ CUtensorMap tmap_vc,
                  const TcParams p)
{
    using C = TcCfg<D>;
    // ---- which block: heaviest (longest causal span) blocks first, heads of a KV group adjacent
    grid_dependency_wait();                       // seq_lens may have been written by the previous kernel
    // pair mode: sub-tile i is query head h + i at rows q0 ..; else: head h at rows q0 + 128 i ..
    const bool pair = p.pair_heads != 0;
    const int heads = pair ? p.Hq / 2 : p.Hq;
    const int per_block = heads * p.B;
    const int qb = p.n_qblocks - 1 - (int)(blockIdx.x / per_block);     // block of 128 (pair mode) or 256 rows
    const int hb = blockIdx.x % per_block;
    const int h = pair ? 2 * (hb % heads) : hb % heads, b = hb / heads;
    const int kvh = h / p.G;
    const int sub_rows = pair ? 0 : kRows;                // rows between the two sub-tiles
    const int sub_heads = pair ? 1 : 0;                   // heads between them
    const int diag0 = pair ? qb : 2 * qb;                 // tile (among the new tokens) of sub-tile 0's diagonal
    // The two lengths are requested now and first looked at after the barrier / TMEM set-up below, so that
    // their latency is hidden behind it.
    const int L_raw = __ldg(p.seq_lens + b);
    const int past_raw = p.past_lens ? __ldg(p.past_lens + b) : 0;
    const int q0 = qb * (pair ? kRows : 2 * kRows);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    uint8_t *smem = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
    uint8_t *q_smem = smem;                                       // 2 sub-tiles
    uint8_t *ring = smem + 2 * C::kTileBytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(ring + (size_t)C::kSlots * C::kTileBytes);
    uint64_t *q_full = bars;
    uint64_t *kv_full = bars + 1;
    uint64_t *kv_empty = kv_full + C::kSlots;
    uint64_t *s_full = kv_empty + C::kSlots;      // [2]
    uint64_t *p_full = s_full + 2;                // [2]
    uint64_t *o_full = p_full + 2;                // [2]
    uint64_t *o_staged = o_full + 2;              // [2] a sub-tile's output rows are in shared memory
    uint32_t *tmem_base_smem = reinterpret_cast<uint32_t *>(o_staged + 2);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_base_smem + 1);
    volatile int *copy_go = abort_flag + 1;       // producer -> helper warps: all loads issued

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // The producer's lane sets the barriers up itself, so that it can start the first loads right away, while
    // the other warps are still on their way to the block-wide barrier below (TMEM allocation included).
    const bool producer_lane = threadIdx.x == 8 * 32;
    if (producer_lane) {
        mbar_init(q_full, 1);
        for (int s = 0; s < C::kSlots; ++s) {
            mbar_init(&kv_full[s], 1);
            mbar_init(&kv_empty[s], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&s_full[i], 1);
            mbar_init(&p_full[i], kRows);
            mbar_init(&o_full[i], 1);
            mbar_init(&o_staged[i], kRows);
        }
        *abort_flag = 0;
        *copy_go = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
    }
    // first use of the lengths. A block past the end of its sequence has nothing to do (decided before any
    // TMEM is taken).
    const int L = L_raw < 0 ? 0 : (L_raw > p.S_max ? p.S_max : L_raw);
    if (q0 >= L) return;
    // Tokens already in the cache ahead of these (0 for a fresh prompt): n_cache tiles, seen by every row.
    const int past = past_raw < 0 ? 0 : past_raw;
    const int n_cache = (past + kRows - 1) / kRows;
    // sub-tile i (rows q0 + 128 i ..) visits the tiles of the past and the new tokens' tiles up to its diagonal
    int n_sub[2];
    n_sub[0] = n_cache + min(q0 + kRows - 1, L - 1) / kRows + 1;
    n_sub[1] = (q0 + sub_rows < L) ? n_cache + min(q0 + sub_rows + kRows - 1, L - 1) / kRows + 1 : 0;
    const int n_kv = max(n_sub[0], n_sub[1]);
    // Q and the first ring-ful of K/V tiles need no waiting: requested before the block-wide barrier
    const int n_pre = min(2 * n_kv, C::kSlots);
    auto request_tile = [&](int idx) {
        const uint32_t s = idx % C::kSlots;
        const int j = idx >> 1;
        uint8_t *dst = ring + (size_t)s * C::kTileBytes;
        int c1, c2, c3;
        mbar_arrive_expect_tx(&kv_full[s], C::kTileBytes);
        if (j >= n_cache) {
            // a tile of the new tokens
            order_coords(p.ckv, (p.new_at_past ? past : 0) + (j - n_cache) * kRows, kvh, b, c1, c2, c3);
            const CUtensorMap *tm = (idx & 1) ? &tmap_v : &tmap_k;
#pragma unroll
            for (int hf = 0; hf < C::kHalves; ++hf) tma_load_4d(dst + hf * kHalfBytes, tm, &kv_full[s], hf * 64, c1, c2, c3);
        } else if (p.block_table == nullptr) {
            // a tile of the tokens cached before, contiguous cache
            order_coords(p.ckc, j * kRows, kvh, b, c1, c2, c3);
            const CUtensorMap *tm = (idx & 1) ? &tmap_vc : &tmap_kc;
#pragma unroll
            for (int hf = 0; hf < C::kHalves; ++hf) tma_load_4d(dst + hf * kHalfBytes, tm, &kv_full[s], hf * 64, c1, c2, c3);
        } else {
            // ... paged cache: one box per page that the tile touches (a page never straddles tiles or boxes). A
            // table entry outside the pool becomes an out-of-range coordinate, which reads zeros.
            const CUtensorMap *tm = (idx & 1) ? &tmap_vc : &tmap_kc;
            const int32_t *row = p.block_table + (size_t)b * p.table_stride;
            for (int r0 = 0; r0 < kRows; r0 += p.cache_box_t) {
                const int slot0 = j * kRows + r0, entry = slot0 >> p.page_shift;
                int page = entry < p.table_stride ? __ldg(row + entry) : -1;
                if (page < 0 || page >= p.num_pages) page = p.num_pages;
                order_coords(p.ckc, slot0 & (p.page_size - 1), kvh, page, c1, c2, c3);
#pragma unroll
                for (int hf = 0; hf < C::kHalves; ++hf)
                    tma_load_4d(dst + hf * kHalfBytes + r0 * 128, tm, &kv_full[s], hf * 64, c1, c2, c3);
            }
        }
    };
    if (producer_lane) {
        tma_prefetch_desc(&tmap_q);
        tma_prefetch_desc(&tmap_k);
        tma_prefetch_desc(&tmap_v);
        if (n_cache > 0) {
            tma_prefetch_desc(&tmap_kc);
            tma_prefetch_desc(&tmap_vc);
        }
        int c1, c2, c3;
        mbar_arrive_expect_tx(q_full, 2 * C::kTileBytes);
        order_coords(p.cq, q0, h, b, c1, c2, c3);
#pragma unroll
        for (int hf = 0; hf < C::kHalves; ++hf) tma_load_4d(q_smem + hf * kHalfBytes, &tmap_q, q_full, hf * 64, c1, c2, c3);
        request_tile(0);                                   // K_0 right behind Q_0: the first product needs both
        order_coords(p.cq, q0 + sub_rows, h + sub_heads, b, c1, c2, c3);
#pragma unroll
        for (int hf = 0; hf < C::kHalves; ++hf)
            tma_load_4d(q_smem + C::kTileBytes + hf * kHalfBytes, &tmap_q, q_full, hf * 64, c1, c2, c3);
        for (int idx = 1; idx < n_pre; ++idx) request_tile(idx);
    }
    if (warp == 9) {
        tmem_alloc(tmem_base_smem, C::kTmemCols);
        tmem_relinquish_alloc_permit();
    }
    // Programmatic dependent launch: the next kernel of the stream may start its own prologue now.
    grid_launch_dependents();
    tcgen05_fence_before_sync();
    __syncthreads();
    tcgen05_fence_after_sync();
    const uint32_t tmem_base = *tmem_base_smem;

    // The block's diagonal K/V tiles (one or two tiles of the new tokens, from diag0 on) go to the cache, at slot past + row
    // (first query head of a KV group only, so each row is written once). They are the last tiles loaded, so their
    // ring slots are never refilled; the copy runs beside the last iterations, shared by three warps. Rows >= L
    // and slots the cache does not have are not written.
    const bool writes_cache = p.cache_k != nullptr && (h % p.G) == 0;
    auto copy_diagonal_tiles = [&](int part) {
        if (!writes_cache) return;
        for (int j = n_cache + diag0; j < n_kv; ++j) {
            const int r_base = (j - n_cache) * kRows;              // first row of the tile among the new tokens
            for (int kv = 0; kv < 2; ++kv) {
                const int idx = 2 * j + kv;
                const uint32_t s = idx % C::kSlots, ph = (idx / C::kSlots) & 1u;
                if (!mbar_wait(&kv_full[s], ph, abort_flag)) return;
                const uint8_t *src = ring + (size_t)s * C::kTileBytes;
                __nv_bfloat16 *dst_all = kv ? p.cache_v : p.cache_k;
                constexpr int kChunks = D / 8;
                const int rows = min(min(kRows, L - r_base), p.cache_slots - past - r_base);
                for (int i = part * 32 + lane; i < rows * kChunks; i += 96) {
                    const int r = i / kChunks, ch = i % kChunks;
                    const int slot = past + r_base + r;
                    __nv_bfloat16 *dst;
                    if (p.block_table == nullptr) {
                        dst = dst_all + b * p.c_sb + kvh * p.c_sh + (int64_t)slot * p.c_st;
                    } else {
                        const int page = __ldg(p.block_table + (size_t)b * p.table_stride + (slot >> p.page_shift));
                        if (page < 0 || page >= p.num_pages) continue;          // no page behind this slot
                        dst = dst_all + (int64_t)page * p.c_sb + kvh * p.c_sh + (int64_t)(slot & (p.page_size - 1)) * p.c_st;
                    }
                    const uint4 val = *reinterpret_cast<const uint4 *>(src + (ch >> 3) * kHalfBytes + swz128(r, ch & 7));
                    *reinterpret_cast<uint4 *>(dst + ch * 8) = val;
                }
            }
        }
    };

    // Register reallocation: the data-movement warpgroup gives registers to the softmax warpgroups,
    // whose threads hold a whole 128-column score row.
    if (warp >= 8) {
    setmaxnreg_dec<64>();
    if (warp == 8) {
        // ============================================================ TMA producer (+ cache copy)
        if (lane == 0) {
            for (int idx = n_pre; idx < 2 * n_kv; ++idx) {
                const uint32_t s = idx % C::kSlots, ph = (idx / C::kSlots) & 1u;
                if (!mbar_wait(&kv_empty[s], ph ^ 1u, abort_flag)) break;
                request_tile(idx);
            }
        }
        // all loads are issued: the diagonal tiles' slots are in their last phase, the copy may start
        if (lane == 0) {
            __threadfence_block();
            *copy_go = 1;
        }
        __syncwarp();
        copy_diagonal_tiles(0);
    } else if (warp == 10 || warp == 11) {
        // otherwise idle warps. First: if an earlier CTA of this launch already reported a dead wait, do
        // not repeat its time-out in every remaining CTA. Then: help the producer warp copy the diagonal
        // tiles to the cache.
        if (warp == 10 && lane == 0 && *reinterpret_cast<volatile unsigned *>(p.status + kStatusErrWord) != 0u)
            *abort_flag = 1;
        if (writes_cache) {
            const long long t0 = clock64();
            bool go = true;
            while (*copy_go == 0) {
                if (*abort_flag || clock64() - t0 > kWaitCycleBudget) { go = false; break; }
                __nanosleep(128);
            }
            __threadfence_block();
            if (go) copy_diagonal_tiles(warp - 9);
        }
    } else if (warp == 9) {
        // ============================================================ MMA issuer
        constexpr uint32_t idesc_qk = make_idesc(kRows, false);
        constexpr uint32_t idesc_pv = make_idesc(D, true);
        const uint32_t tmem_s[2] = {tmem_base + C::kColS0, tmem_base + C::kColS1};
        const uint32_t tmem_o[2] = {tmem_base + C::kColO0, tmem_base + C::kColO1};
        const uint32_t q_addr = smem_u32(q_smem), ring_addr = smem_u32(ring);

        auto issue_qk = [&](int i, uint32_t k_addr) {
#pragma unroll
            for (int k = 0; k < D / 16; ++k) {
                const uint32_t off = (k >> 2) * kHalfBytes + (k & 3) * 32;
                tcgen05_mma_ss(tmem_s[i], make_smem_desc(q_addr + i * C::kTileBytes + off, 0),
                               make_smem_desc(k_addr + off, 0), idesc_qk, k > 0 ? 1u : 0u);
            }
        };
        auto issue_pv = [&](int i, uint32_t v_addr, bool first) {
#pragma unroll
            for (int k = 0; k < kRows / 16; ++k)
                tcgen05_mma_ts(tmem_o[i], tmem_s[i] + k * 8, make_smem_desc(v_addr + k * 2048, kHalfBytes), idesc_pv,
                               (first && k == 0) ? 0u : 1u);
        };

        bool ok = mbar_wait(q_full, 0, abort_flag) && mbar_wait(&kv_full[0], 0, abort_flag);
        if (ok) {
            tcgen05_fence_after_sync();
            if (lane == 0) {
                for (int i = 0; i < 2; ++i)
                    if (n_sub[i] > 0) {
                        issue_qk(i, ring_addr);
                        tcgen05_commit(&s_full[i]);
                    }
                tcgen05_commit(&kv_empty[0]);
            }
            __syncwarp();
        }
        for (int j = 0; ok && j < n_kv; ++j) {
            const int iv = 2 * j + 1, ik = 2 * j + 2;
            const uint32_t sv = iv % C::kSlots, sk = ik % C::kSlots;
            if (!mbar_wait(&kv_full[sv], (iv / C::kSlots) & 1u, abort_flag)) { ok = false; break; }
            // V rows >= this hold no valid token (the partly filled last tile of the past, or of the new tokens)
            const int first_dead = j < n_cache ? past - j * kRows : L - (j - n_cache) * kRows;
            if (first_dead < kRows) {
                // may hold any bits (NaN included): clear, so that a zero weight times garbage cannot appear
                uint8_t *vt = ring + (size_t)sv * C::kTileBytes;
                constexpr int kChunks = D / 8;
                for (int i = lane; i < (kRows - first_dead) * kChunks; i += 32) {
                    const int r = first_dead + i / kChunks, ch = i % kChunks;
                    *reinterpret_cast<uint4 *>(vt + (ch >> 3) * kHalfBytes + r * 128 + ((ch & 7) << 4)) =
                        make_uint4(0u, 0u, 0u, 0u);
                }
                fence_proxy_async_smem();
                __syncwarp();
            }
            const bool have_next = j + 1 < n_kv;
            if (have_next && !mbar_wait(&kv_full[sk], (ik / C::kSlots) & 1u, abort_flag)) { ok = false; break; }
            for (int i = 0; i < 2 && ok; ++i) {
                if (j >= n_sub[i]) continue;
                if (!mbar_wait(&p_full[i], j & 1u, abort_flag)) { ok = false; break; }
                tcgen05_fence_after_sync();
                if (lane == 0) {
                    issue_pv(i, ring_addr + sv * C::kTileBytes, j == 0);
                    if (j + 1 < n_sub[i]) {
                        issue_qk(i, ring_addr + sk * C::kTileBytes);
                        tcgen05_commit(&s_full[i]);
                    } else {
                        tcgen05_commit(&o_full[i]);
                    }
                }
                __syncwarp();
            }
            if (ok && lane == 0) {
                tcgen05_commit(&kv_empty[sv]);
                if (have_next) tcgen05_commit(&kv_empty[sk]);
            }
            __syncwarp();
        }
    }
    } else {
        setmaxnreg_inc<216>();
        // ============================================================ softmax + epilogue warpgroups
        const int i = warp >> 2;                                   // sub-tile
        const int t = threadIdx.x & 127;                           // row within the sub-tile == TMEM lane
        const int row = q0 + i * sub_rows + t;                     // token index of this thread's query row
        const int hq = h + i * sub_heads;                          // ... and its query head
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tmem_s = tmem_base + lane_base + (i ? C::kColS1 : C::kColS0);
        const uint32_t tmem_o = tmem_base + lane_base + (i ? C::kColO1 : C::kColO0);
        const int n_mine = n_sub[i];
        // Tiles that need a mask: the last tile of the past when it is partly filled (columns past its end, the same
        // for every row), and the sub-tile's diagonal tile among the new tokens (row t sees columns 0..t).
        const int j_ragged = (past & (kRows - 1)) ? n_cache - 1 : -1;
        const int j_diag = n_cache + (pair ? diag0 : diag0 + i);
        const float c = p.scale_log2e;
        float m = -INFINITY, l = 0.f;
        bool ok = true;

        for (int j = 0; j < n_mine; ++j) {
            if (!mbar_wait(&s_full[i], j & 1u, abort_flag)) { ok = false; break; }
            tcgen05_fence_after_sync();
            uint32_t sr[4][32];
#pragma unroll
            for (int qd = 0; qd < 4; ++qd) tmem_ld_32x32b_x32(tmem_s + qd * 32, sr[qd]);
            tcgen05_wait_ld();

            // Row maximum of the scaled scores (log2 domain). Off the diagonal the maximum is taken over the
            // raw scores with independent 3-input max chains and scaled once (min for a negative scale);
            // on the diagonal tile the causal mask is applied to the scaled scores first.
            const bool diag = (j == j_ragged) || (j >= j_diag);
            float mx;
            if (diag) {
                const int lim = (j == j_ragged) ? (past & (kRows - 1)) - 1 : t;   // columns > lim hold no visible key
                float a0 = -INFINITY, a1 = -INFINITY, a2 = -INFINITY, a3 = -INFINITY;
#pragma unroll
                for (int qd = 0; qd < 4; ++qd)
#pragma unroll
                    for (int e = 0; e < 32; e += 4) {
                        float x[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            x[u] = __uint_as_float(sr[qd][e + u]) * c;
                            x[u] = (qd * 32 + e + u > lim) ? -INFINITY : x[u];
                            sr[qd][e + u] = __float_as_uint(x[u]);
                        }
                        a0 = fmaxf(a0, x[0]); a1 = fmaxf(a1, x[1]); a2 = fmaxf(a2, x[2]); a3 = fmaxf(a3, x[3]);
                    }
                mx = fmaxf(fmaxf(a0, a1), fmaxf(a2, a3));
            } else if (c >= 0.f) {
                float a0 = -INFINITY, a1 = -INFINITY, a2 = -INFINITY, a3 = -INFINITY;
#pragma unroll
                for (int qd = 0; qd < 4; ++qd)
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        a0 = max3(a0, __uint_as_float(sr[qd][e + 0]), __uint_as_float(sr[qd][e + 1]));
                        a1 = max3(a1, __uint_as_float(sr[qd][e + 2]), __uint_as_float(sr[qd][e + 3]));
                        a2 = max3(a2, __uint_as_float(sr[qd][e + 4]), __uint_as_float(sr[qd][e + 5]));
                        a3 = max3(a3, __uint_as_float(sr[qd][e + 6]), __uint_as_float(sr[qd][e + 7]));
                    }
                mx = fmaxf(fmaxf(a0, a1), fmaxf(a2, a3)) * c;
            } else {
                float a0 = INFINITY, a1 = INFINITY, a2 = INFINITY, a3 = INFINITY;
#pragma unroll
                for (int qd = 0; qd < 4; ++qd)
#pragma unroll
                    for (int e = 0; e < 32; e += 4) {
                        a0 = fminf(a0, __uint_as_float(sr[qd][e + 0]));
                        a1 = fminf(a1, __uint_as_float(sr[qd][e + 1]));
                        a2 = fminf(a2, __uint_as_float(sr[qd][e + 2]));
                        a3 = fminf(a3, __uint_as_float(sr[qd][e + 3]));
                    }
                mx = fminf(fminf(a0, a1), fminf(a2, a3)) * c;
            }
            // lazy rescale: keep the old reference max unless the new one is much larger
            const bool grow = (mx > m + kRescaleThreshold) || (j == 0);
            float alpha = 1.f;
            if (grow) {
                const float m_new = (mx == -INFINITY) ? 0.f : mx;
                alpha = fast_exp2(m - m_new);                      // j == 0: exp2(-inf) = 0
                m = m_new;
                l *= alpha;
            }
            if (j > 0 && __any_sync(0xffffffffu, grow)) {
                // PV_{j-1} has completed (s_full is committed after it), PV_j is not issued before p_full
#pragma unroll
                for (int qd = 0; qd < D / 32; ++qd) {
                    uint32_t orr[32];
                    tmem_ld_32x32b_x32(tmem_o + qd * 32, orr);
                    tcgen05_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; ++e) orr[e] = __float_as_uint(__uint_as_float(orr[e]) * alpha);
                    tmem_st_32x32b_x32(tmem_o + qd * 32, orr);
                }
            }
            // p = 2^(x - m): packed fp32x2 FMA feeds the exp2 unit; sums in two independent packed chains
            const float fc = diag ? 1.f : c;                       // diagonal scores are already scaled
            const uint64_t c2 = pack_f32x2(fc, fc), nm2 = pack_f32x2(-m, -m);
            uint64_t sum_a = pack_f32x2(0.f, 0.f), sum_b = sum_a;
#pragma unroll
            for (int qd = 0; qd < 4; ++qd) {
                uint32_t pk[16];
#pragma unroll
                for (int e = 0; e < 16; e += 2) {
                    const uint64_t xa = fma_f32x2(pack_u32x2(sr[qd][2 * e], sr[qd][2 * e + 1]), c2, nm2);
                    const uint64_t xb = fma_f32x2(pack_u32x2(sr[qd][2 * e + 2], sr[qd][2 * e + 3]), c2, nm2);
                    float xa0, xa1, xb0, xb1;
                    unpack_f32x2(xa, xa0, xa1);
                    unpack_f32x2(xb, xb0, xb1);
                    const float pa0 = fast_exp2(xa0), pa1 = fast_exp2(xa1);
                    const float pb0 = fast_exp2(xb0), pb1 = fast_exp2(xb1);
                    sum_a = add_f32x2(sum_a, pack_f32x2(pa0, pa1));
                    sum_b = add_f32x2(sum_b, pack_f32x2(pb0, pb1));
                    pk[e] = pack_bf16x2(pa0, pa1);
                    pk[e + 1] = pack_bf16x2(pb0, pb1);
                }
                tmem_st_32x32b_x16(tmem_s + qd * 16, pk);
            }
            float sa0, sa1, sb0, sb1;
            unpack_f32x2(sum_a, sa0, sa1);
            unpack_f32x2(sum_b, sb0, sb1);
            const float sum = (sa0 + sa1) + (sb0 + sb1);
            l += sum;
            tcgen05_wait_st();
            tcgen05_fence_before_sync();
            mbar_arrive(&p_full[i]);
        }

        if (ok && n_mine > 0 && mbar_wait(&o_full[i], 0, abort_flag)) {
            tcgen05_fence_after_sync();
            const float inv = 1.f / l;
            const bool valid = row < L;
            __nv_bfloat16 *orow = p.o + b * p.o_sb + (int64_t)row * p.o_st + hq * p.o_sh;
            // A sub-tile whose 128 rows are all valid leaves through shared memory and one TMA store per 64
            // columns (coalesced, asynchronous): the rows are staged where Q_i was, which no MMA reads any more
            // (o_full follows the last of them). A ragged sub-tile writes its valid rows directly.
            const bool whole = q0 + i * sub_rows + kRows <= L;
            uint8_t *stage = q_smem + i * C::kTileBytes;
#pragma unroll
            for (int qd = 0; qd < D / 32; ++qd) {
                uint32_t orr[32];
                tmem_ld_32x32b_x32(tmem_o + qd * 32, orr);
                tcgen05_wait_ld();
                if (whole) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        uint4 val;
                        val.x = pack_bf16x2(__uint_as_float(orr[8 * e + 0]) * inv, __uint_as_float(orr[8 * e + 1]) * inv);
                        val.y = pack_bf16x2(__uint_as_float(orr[8 * e + 2]) * inv, __uint_as_float(orr[8 * e + 3]) * inv);
                        val.z = pack_bf16x2(__uint_as_float(orr[8 * e + 4]) * inv, __uint_as_float(orr[8 * e + 5]) * inv);
                        val.w = pack_bf16x2(__uint_as_float(orr[8 * e + 6]) * inv, __uint_as_float(orr[8 * e + 7]) * inv);
                        const int ch = qd * 4 + e;                 // 16-byte chunk of the row
                        *reinterpret_cast<uint4 *>(stage + (ch >> 3) * kHalfBytes + swz128(t, ch & 7)) = val;
                    }
                } else if (valid) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        uint4 val;
                        val.x = pack_bf16x2(__uint_as_float(orr[8 * e + 0]) * inv, __uint_as_float(orr[8 * e + 1]) * inv);
                        val.y = pack_bf16x2(__uint_as_float(orr[8 * e + 2]) * inv, __uint_as_float(orr[8 * e + 3]) * inv);
                        val.z = pack_bf16x2(__uint_as_float(orr[8 * e + 4]) * inv, __uint_as_float(orr[8 * e + 5]) * inv);
                        val.w = pack_bf16x2(__uint_as_float(orr[8 * e + 6]) * inv, __uint_as_float(orr[8 * e + 7]) * inv);
                        *reinterpret_cast<uint4 *>(orow + qd * 32 + e * 8) = val;
                    }
                }
            }
            if (whole) {
                fence_proxy_async_smem();                          // this thread's rows, for the TMA store
                mbar_arrive(&o_staged[i]);
                if (t == 0 && mbar_wait(&o_staged[i], 0, abort_flag)) {
                    int c1, c2, c3;
                    order_coords(p.co, q0 + i * sub_rows, hq, b, c1, c2, c3);
#pragma unroll
                    for (int hf = 0; hf < C::kHalves; ++hf) tma_store_4d(&tmap_o, stage + hf * kHalfBytes, hf * 64, c1, c2, c3);
                    tma_store_commit();
                    tma_store_wait_read_all();                     // shared memory must outlive the reads
                }
            }
            if (valid && p.lse)
                p.lse[((size_t)b * p.Hq + hq) * p.S_max + row] = (m + log2f(l)) * 0.6931471805599453f;
        }
    }

    tcgen05_fence_before_sync();
    __syncthreads();
    if (warp == 9) {
        tcgen05_fence_after_sync();
        tmem_dealloc(tmem_base, C::kTmemCols);
    }
    if (threadIdx.x == 0 && *abort_flag) {
        if (atomicOr(p.status + kStatusErrWord, kErrPrefillWait) == 0u)
            p.status[kStatusInfoWord] = 0x20000u | (blockIdx.x & 0xffffu);
    }
}

template <int D>
l4l_status launch_t(const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv, const CUtensorMap &to,
                    const CUtensorMap &tkc, const CUtensorMap &tvc, const TcParams &p, cudaStream_t stream)
{
    using C = TcCfg<D>;
    static bool configured_on[kDeviceSlots] = {};
    const int slot = device_slot();
    if (slot < 0) return L4L_ERR_CUDA;
    {
        std::lock_guard<std::mutex> lock(setup_mutex());
        bool &configured = configured_on[slot];
        if (!configured) {
            if (cudaFuncSetAttribute(prefill_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)C::kSmemBytes) != cudaSuccess)
                return L4L_ERR_CUDA;
            configured = true;
        }
    }
    const long long grid = (long long)p.n_qblocks * (p.pair_heads ? p.Hq / 2 : p.Hq) * p.B;
    if (grid > 0x7fffffffll) return L4L_ERR_UNSUPPORTED;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = C::kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, prefill_tc_kernel<D>, tq, tk, tv, to, tkc, tvc, p) == cudaSuccess ? L4L_OK : L4L_ERR_CUDA;
}

}  // namespace

l4l_status launch_prefill_tc(const l4l_tensor4 &q, const l4l_tensor4 &o, const PrefillKV &kv, const int32_t *d_seq_lens,
                             const int32_t *d_past_lens, int S_max, int B, int Hq, int Hkv, int D, float scale,
                             float *d_lse, void *workspace, cudaStream_t stream)
{
    CUtensorMap tq, tk, tv, to, tkc, tvc;
    TmapCoord cq, ck, cv, co, ckc, cvc;
    if (!make_tmap_bf16(&tq, &cq, q.ptr, D, S_max, Hq, B, q.stride_t, q.stride_h, q.stride_b, 64, kRows) ||
        !make_tmap_bf16(&to, &co, o.ptr, D, S_max, Hq, B, o.stride_t, o.stride_h, o.stride_b, 64, kRows) ||
        !make_tmap_bf16(&tk, &ck, kv.k_new.ptr, D, kv.new_extent, Hkv, B, kv.k_new.stride_t, kv.k_new.stride_h,
                        kv.k_new.stride_b, 64, kRows) ||
        !make_tmap_bf16(&tv, &cv, kv.v_new.ptr, D, kv.new_extent, Hkv, B, kv.v_new.stride_t, kv.v_new.stride_h,
                        kv.v_new.stride_b, 64, kRows))
        return L4L_ERR_CUDA;
    if (ck.pos_t != cv.pos_t || ck.pos_h != cv.pos_h || ck.pos_b != cv.pos_b) return L4L_ERR_UNSUPPORTED;
    TcParams p = {};
    // the tokens cached before: tiles of the cache (one box per tile), or of the page pool (one box per page if the
    // pages are smaller than a tile); without a past the kernel never touches these two maps
    tkc = tk; tvc = tv; ckc = ck;
    p.cache_box_t = kRows;
    if (kv.past) {
        const l4l_kv_cache &c = *kv.past;
        const int outer = kv.paged ? kv.paged->num_pages : B;
        if (kv.paged && c.max_len < kRows) p.cache_box_t = c.max_len;
        if (!make_tmap_bf16(&tkc, &ckc, c.k, D, c.max_len, Hkv, outer, c.stride_t, c.stride_h, c.stride_b, 64, p.cache_box_t) ||
            !make_tmap_bf16(&tvc, &cvc, c.v, D, c.max_len, Hkv, outer, c.stride_t, c.stride_h, c.stride_b, 64, p.cache_box_t))
            return L4L_ERR_CUDA;
    }
    p.o = static_cast<__nv_bfloat16 *>(o.ptr);
    p.o_sb = o.stride_b; p.o_st = o.stride_t; p.o_sh = o.stride_h;
    if (kv.write) {
        p.cache_k = static_cast<__nv_bfloat16 *>(kv.write->k);
        p.cache_v = static_cast<__nv_bfloat16 *>(kv.write->v);
        p.c_sb = kv.write->stride_b; p.c_sh = kv.write->stride_h; p.c_st = kv.write->stride_t;
        const long long slots = kv.paged ? (long long)kv.paged->table_stride * kv.write->max_len : kv.write->max_len;
        p.cache_slots = slots > 0x7fffffffll ? 0x7fffffff : (int)slots;
    }
    if (kv.paged) {
        const int page_size = kv.past ? kv.past->max_len : kv.write->max_len;
        p.block_table = kv.paged->block_table;
        p.table_stride = kv.paged->table_stride;
        p.num_pages = kv.paged->num_pages;
        p.page_size = page_size;
        while ((1 << p.page_shift) < page_size) ++p.page_shift;
    }
    p.new_at_past = kv.new_at_past ? 1 : 0;
    p.seq_lens = d_seq_lens;
    p.past_lens = d_past_lens;
    p.lse = d_lse;
    p.status = static_cast<unsigned *>(workspace);
    p.S_max = S_max; p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.G = Hq / Hkv;
    p.pair_heads = (p.G % 2 == 0) ? 1 : 0;
    p.n_qblocks = p.pair_heads ? (S_max + kRows - 1) / kRows : (S_max + 2 * kRows - 1) / (2 * kRows);
    p.scale_log2e = scale * 1.4426950408889634f;
    p.cq = cq; p.ckv = ck; p.co = co; p.ckc = ckc;
    return (D == 128) ? launch_t<128>(tq, tk, tv, to, tkc, tvc, p, stream) : launch_t<64>(tq, tk, tv, to, tkc, tvc, p, stream);
}

}  // namespace l4l
