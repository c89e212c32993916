// Decode attention: one query token per sequence over a ragged KV cache (bf16, or e4m3 bytes with a scale
// per KV head; contiguous, or pages behind a block table: the template flag F8 and the optional page table
// change the tile element type and the producer's coordinates, nothing else).
//
// One launch. The cache of every (sequence, KV head) is cut into tiles of 16*W tokens (W = 4 or 8
// consumer warps; twice that for fp8 caches and for 64-wide heads, where a warp takes 32 tokens per step); the
// flattened tile stream (sequence-major, then KV head, then position) is divided
// among persistent CTAs as evenly as whole tiles allow, so every CTA streams the same number of bytes
// (to within one tile) whatever the length mix. A CTA's range may
// start or end inside a sequence: each (sequence, KV head) is thus covered by one or more
// "pieces", one per CTA that touches it.
//
//   producer warp    walks the CTA's tile range and keeps a ring of TMA tiles (K and V, 128-byte
//                    swizzle) full, across piece boundaries
//   W consumer warps each take 16 tokens of every tile and serve ALL query heads of the KV group
//                    from it: the group is the M dimension (zero-padded to 16) of warp-level bf16
//                    MMAs, so cache bytes are read once per group. Softmax statistics are fp32;
//                    row maxima are reduced with warp shuffles. At the end of a piece they drop
//                    their (max, sum, O) into shared memory and go straight on to the next tile.
//   finisher warp    merges the consumer warps' results of a piece off the critical path. A sequence
//                    covered by a single piece is written out directly; otherwise the piece's
//                    normalised fp32 partial and its log-sum-exp go to the workspace, and the LAST
//                    piece to arrive (a self-resetting ticket counter per (sequence, KV head)) runs
//                    the second pass: the log-sum-exp merge of all pieces.
#include <cstdlib>
#include <mutex>

#include "l4l_fp8_quant.cuh"
#include "l4l_internal.h"
#include "l4l_rope_frag.cuh"
#include "l4l_warp_attn.cuh"

namespace l4l {

namespace {

// The kernel comes in two shapes, W = 4 or 8 consumer warps. A tile is 16*W tokens (each consumer warp takes
// 16 of them); with W = 4 two CTAs share an SM, with W = 8 one CTA owns it and streams ranges twice as long,
// so that fewer sequences are cut between CTAs. W + 2 warps in all: consumers, producer, finisher.
constexpr int kPostRing = 16;               // pieces a producer can be ahead of its finisher (ring size)
// The ticket counters sit at a FIXED place and size in the workspace (right after the status block), so
// that calls of different shapes on one workspace can never write partials over counters another call
// relies on being zero.
constexpr size_t kTicketBytes = 128 * 1024;  // 32768 (sequence, KV head) pairs per launch
constexpr int kMaxB = 384;                 // sequences per launch (prefix sums and lengths live in shared memory)

// F8: the cache holds e4m3 bytes (one byte per value) instead of bf16.
template <int D, int W, bool F8>
struct DecodeCfg {
    // 16-token blocks a consumer warp takes per tile: two (one softmax update per 32 tokens) for fp8 caches and for
    // 64-wide heads, where a token is half the bytes and the per-token bookkeeping weighs twice as much
    static constexpr int kSub = (F8 || D == 64) ? 2 : 1;
    static constexpr int kTileT = 16 * W * kSub;                  // tokens per TMA tile
    static constexpr int kRowBytes = F8 ? D : 2 * D;              // one token of one KV head
    // fp8 at head_dim 64: a token is 64 bytes, and two consecutive tokens make one 128-byte row of the tile (the
    // cache must be dense in the token dimension); everywhere else a token is one row of every 128-byte column block
    static constexpr int kTokPerRow = kRowBytes < 128 ? 2 : 1;
    static constexpr int kTokBytes = 128 / kTokPerRow;            // bytes of a token in one column block
    static constexpr int kHalves = kRowBytes < 128 ? 1 : kRowBytes / 128;   // 128-byte column blocks of a tile
    static constexpr int kBoxD = F8 ? 128 : 64;                   // elements per 128-byte box row
    static constexpr uint32_t kHalfBytes = kTileT * kTokBytes;    // [tile rows][128 bytes], swizzled
    static constexpr uint32_t kTileBytes = kHalves * kHalfBytes;  // one of K or V
    static constexpr uint32_t kStageBytes = 2 * kTileBytes;
    static constexpr int kStages = (kStageBytes >= 32768u * (W / 4)) ? 3 : 6;   // 192 KB (96 KB with W = 4) in flight
};

// One row of `comb`: the unnormalised O of one query head of a piece as one consumer warp saw it, then its max and its
// sum. Groups of 5 to 8 query heads at head_dim 128 (BigG) keep O as bf16 there, so that eight warps' rows still fit
// beside the three 64 KB stages; max and sum stay fp32. (One rounding to bf16 per warp and piece, ahead of the merge.)
template <int D, bool BigG>
struct CombRow {
    static constexpr int kBytes = BigG ? D * 2 + 16 : (D + 4) * 4;
    static constexpr int kOffM = BigG ? D * 2 : D * 4;
    static __device__ __forceinline__ float m(const uint8_t *row) { return *reinterpret_cast<const float *>(row + kOffM); }
    static __device__ __forceinline__ float l(const uint8_t *row) { return *reinterpret_cast<const float *>(row + kOffM + 4); }
    static __device__ __forceinline__ float4 v4(const uint8_t *row, int d4)
    {
        if constexpr (BigG) {
            const uint2 u = *reinterpret_cast<const uint2 *>(row + d4 * 8);
            return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u), __uint_as_float(u.y << 16),
                               __uint_as_float(u.y & 0xffff0000u));
        } else {
            return *reinterpret_cast<const float4 *>(row + d4 * 16);
        }
    }
};

struct TileMeta {
    int b, kvh, t0, piece, kv_len, npieces, flags, pad;
};
constexpr int kFlagFirst = 1, kFlagLast = 2, kFlagStop = 4;

struct PieceMeta {
    int b, kvh, piece, npieces, stop, pad0, pad1, pad2;
};

struct DecodeParams {
    const __nv_bfloat16 *q;   // [B, Hq, D]
    __nv_bfloat16 *o;         // [B, Hq, D]
    float *lse;               // [B, Hq] or null
    const int32_t *kv_lens;   // [B]
    float *part_o;            // [B, Hq, nsplit, D]  normalised partial outputs
    float *part_lse;          // [B, Hq, nsplit]     log2-domain log-sum-exp of the piece
    int *tickets;             // [B, Hkv]            pieces arrived; zero between calls
    // fused append (null: none): the newest token of every sequence (slot kv_len-1) comes from here and
    // is written to the cache by the CTA that streams its tile
    const __nv_bfloat16 *k_new, *v_new;       // element (b, kv head, d) at b*new_sb + kvh*new_sh + d
    int64_t new_sb, new_sh;
    __nv_bfloat16 *cache_k, *cache_v;
    int64_t c_sb, c_sh, c_st;
    unsigned *status;
    // fp8 cache: real value = e4m3 value * scale of its KV head
    const float *k_scale, *v_scale;           // [Hkv]
    // rotary embedding (+ optional RMS norm) of the step's q and k_new inside the kernel (null: inputs are final);
    // only together with the fused append. The new token's position is kv_len - 1.
    const float *rope_cos, *rope_sin;         // [rope_n_pos, D/2]
    const float *q_weight, *k_weight;         // [D] or null
    float norm_eps;
    int rope_n_pos;
    // paged cache (null: contiguous): token t of sequence b lives in page block_table[b * table_stride + t / page_size]
    // at offset t % page_size; the tensor maps then describe the page pool [pages, Hkv, page_size, D]
    const int32_t *block_table;
    int table_stride, page_size, page_shift, num_pages;
    int page_box;             // paged: tokens per box of tmap_k / tmap_v (divides the tile, never straddles a page)
    int tail_rows;            // tokens per box of tmap_k_tail / tmap_v_tail (32, or the page size if that is smaller)
    int B, Hq, Hkv, G, min_tiles, nsplit, max_kv_len;
    int stream_once;          // load K/V with the L2 evict-first policy (large caches)
    int nfin;                 // finisher warps (BigG: one per 4 query heads of the group; else 1)
    float scale_log2e;
    TmapCoord coord;
};

template <int D, int W, bool F8, bool BigG>
size_t decode_smem_bytes(int G, int nsplit)
{
    using C = DecodeCfg<D, W, F8>;
    size_t comb = (size_t)W * G * CombRow<D, BigG>::kBytes + (size_t)((G * nsplit + 3) & ~3) * sizeof(float);
    // per stage: the K/V tiles, the piece's query rows and (rope fused into the step) the cos / sin rows of the
    // new token's position; per consumer warp: its private copy of those rows for the piece it is working on
    return 1024 /*alignment slack*/ + (size_t)C::kStages * (C::kStageBytes + (size_t)G * D * 2 + D * 4 + (BigG ? 0 : 2 * D * 2)) + (size_t)W * D * 4 + 2 * D * 4 +
           comb +
           C::kStages * sizeof(TileMeta) +
           sizeof(PieceMeta) + (2 * C::kStages + 2) * sizeof(uint64_t) + (2 * kMaxB + 1) * sizeof(int) + 64 +
           kPostRing * sizeof(PieceMeta);
}

// n / d for 0 <= n < 2^23, 0 < d < 2^23 without the integer-division sequence (the producer lane's partition
// arithmetic sits on the path to the first load of the kernel): a float quotient, corrected by at most one.
__device__ __forceinline__ int small_div(int n, int d)
{
    int q = (int)__fdividef((float)n, (float)d);
    if (q * d > n) --q;
    if ((q + 1) * d <= n) ++q;
    return q;
}

__device__ __forceinline__ void order_coords(const TmapCoord &c, int t, int h, int b, int &c1, int &c2, int &c3)
{
    c1 = (c.pos_t == 1) ? t : (c.pos_h == 1) ? h : b;
    c2 = (c.pos_t == 2) ? t : (c.pos_h == 2) ? h : b;
    c3 = (c.pos_t == 3) ? t : (c.pos_h == 3) ? h : b;
}

// R8: an e4m3-cache kernel that also carries the rope-fused step. A build of its own, so that the rotation code does
// not weigh on the registers of the plain fp8 kernels, which are bound by their consumer warps (bf16 kernels always carry it).
template <int D, int W, bool F8, bool BigG, bool R8 = false>
__global__ void __launch_bounds__((BigG ? 11 : W + 2) * 32)
decode_split_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                    const __grid_constant__ CUtensorMap tmap_k_tail, const __grid_constant__ CUtensorMap tmap_v_tail,
                    const DecodeParams p)
{
    using C = DecodeCfg<D, W, F8>;
    constexpr int kTileT = C::kTileT;
    constexpr int kConsumerWarps = W, kProducerWarp = W, kFinisherWarp = W + 1;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    uint8_t *smem = smem_raw + ((1024u - (raw & 1023u)) & 1023u);

    uint8_t *stages = smem;
    uint8_t *q_slots = stages + (size_t)C::kStages * C::kStageBytes;     // per stage: the piece's G query rows ...
    const uint32_t q_bytes = (uint32_t)p.G * D * 2;
    constexpr uint32_t kRopeBytes = D * 4;                               // ... and cos | sin of the new token's position
    // ... and (fused append; not on the big-group shapes, whose shared memory is full) the step's new k row and v row,
    // which arrive with the tile they are patched into, so that the patching warp does not wait for global memory there
    constexpr uint32_t kNewBytes = BigG ? 0 : 2 * D * 2;
    const uint32_t q_stride = q_bytes + kRopeBytes + kNewBytes;
    float *rope_priv = reinterpret_cast<float *>(q_slots + (size_t)C::kStages * q_stride);   // [W][D] per-warp copy
    float *norm_w = rope_priv + (size_t)W * D;                           // q_weight | k_weight (when given)
    float *comb = norm_w + 2 * D;
    constexpr int kVec = D / 4;
    using CR = CombRow<D, BigG>;
    uint8_t *comb_b = reinterpret_cast<uint8_t *>(comb);
    float *merge_lse = reinterpret_cast<float *>(comb_b + (size_t)kConsumerWarps * p.G * CR::kBytes);   // [G][nsplit] scratch of the finisher's second pass
    TileMeta *meta = reinterpret_cast<TileMeta *>(merge_lse + ((p.G * p.nsplit + 3) & ~3));   // keeps 16-byte alignment
    PieceMeta *piece_meta = reinterpret_cast<PieceMeta *>(meta + C::kStages);
    uint64_t *full = reinterpret_cast<uint64_t *>(piece_meta + 1);
    uint64_t *empty = full + C::kStages;
    uint64_t *comb_full = empty + C::kStages;   // consumers -> finisher: a piece's results are in `comb`
    uint64_t *comb_empty = comb_full + 1;       // finisher -> consumers: `comb` may be overwritten
    int *cum = reinterpret_cast<int *>(comb_empty + 1);   // cum[b] = stream items (tiles + one marker per KV head) of sequences < b
    int *lens_s = cum + (kMaxB + 1);                      // clamped kv_lens
    volatile int *abort_flag = lens_s + kMaxB;
    // producer -> finisher: the pieces this CTA has started, in order (so that the finisher can look at a
    // piece's ticket while the piece is still being streamed)
    volatile uint32_t *posted_count = reinterpret_cast<volatile uint32_t *>(abort_flag + 1);
    // producer -> finisher: how many pieces this CTA has in all (known once the last one has been started); the
    // finisher leaves right after the last one
    volatile uint32_t *pieces_total = posted_count + 1;
    PieceMeta *post_ring = reinterpret_cast<PieceMeta *>(lens_s + kMaxB + 4);
    // consumers among themselves: the piece's query rows have been rotated in place (rope fused into the step)
    uint64_t *q_rotated = reinterpret_cast<uint64_t *>((reinterpret_cast<uintptr_t>(post_ring + kPostRing) + 7) & ~(uintptr_t)7);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], kConsumerWarps);
        }
        mbar_init(comb_full, kConsumerWarps);
        mbar_init(q_rotated, kConsumerWarps);
        mbar_init(comb_empty, BigG ? p.nfin : 1);
        *abort_flag = 0;
        *posted_count = 0u;
        *pieces_total = 0xffffffffu;
        fence_barrier_init();
        fence_proxy_async_smem();
    }
    if (warp == kProducerWarp && lane == 0) {
        tma_prefetch_desc(&tmap_k);
        tma_prefetch_desc(&tmap_v);
        tma_prefetch_desc(&tmap_k_tail);
        tma_prefetch_desc(&tmap_v_tail);
    }
    // Programmatic dependent launch: everything above overlaps the tail of the previous kernel in the
    // stream; nothing below (no global read or write) starts before that kernel has completed. The
    // next kernel in the stream may begin its own prologue as soon as this grid's CTAs retire.
    grid_dependency_wait();
    grid_launch_dependents();
    // the producer's first look at the lengths is requested now, so that its latency passes behind the barrier below
    int early_len = 0;
    if (warp == kProducerWarp && lane < p.B) early_len = p.kv_lens[lane];
    if (p.rope_cos != nullptr) {
        for (int i = threadIdx.x; i < D; i += blockDim.x) {
            norm_w[i] = p.q_weight ? __ldg(p.q_weight + i) : 1.f;
            norm_w[D + i] = p.k_weight ? __ldg(p.k_weight + i) : 1.f;
        }
    }
    __syncthreads();

    if (warp == kProducerWarp) {
        // ------------------------------------------------------------------ producer warp
        // Exclusive prefix sum over sequences of ((tiles + 1) * Hkv): the flattened stream that is divided among
        // the CTAs holds, ahead of the tiles of every (sequence, KV head), one marker that stands for the fixed
        // cost of starting a piece there (query rows, a mostly short last tile, the hand-over to the finisher:
        // about one tile's time). A CTA whose range covers many short sequences thus gets fewer tiles.
        int running = 0;
        for (int b0 = 0; b0 < p.B; b0 += 32) {
            const int b = b0 + lane;
            int n = 0;
            if (b < p.B) {
                int len = b0 == 0 ? early_len : p.kv_lens[b];
                len = len < 0 ? 0 : (len > p.max_kv_len ? (p.k_new ? 0 : p.max_kv_len) : len);   // over the host's bound: decode ignores the extra tokens, a fused append treats the sequence as empty
                lens_s[b] = len;
                n = len > 0 ? ((len + kTileT - 1) / kTileT + 1) * p.Hkv : 0;
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
            const int total = running;
            // Even split of the tile stream: the first `rem` CTAs take q+1 tiles, the others q, so that
            // no CTA idles; if that would be fewer than the floor, every CTA takes the floor instead (and
            // the last CTAs get nothing).
            int q = small_div(total, (int)gridDim.x), rem = total - q * (int)gridDim.x;
            if (q < p.min_tiles) { q = p.min_tiles; rem = 0; }
            const int big = rem * (q + 1);                 // tiles covered by the CTAs that take q+1
            auto range_begin = [&](int c) { return min(total, c * q + min(c, rem)); };
            auto cta_of = [&](int t) { return t < big ? small_div(t, q + 1) : rem + small_div(t - big, q); };
            const int my_begin = range_begin((int)blockIdx.x);
            const int my_end = range_begin((int)blockIdx.x + 1);
            uint32_t it = 0, n_posted = 0;
            bool ok = true;
            // a large cache is read once per step: its lines go first; a small one stays L2-resident between steps
            const uint64_t stream_policy = p.stream_once ? l2_policy_evict_first() : l2_policy_evict_normal();
            // Order of work. If the range ends inside a sequence (the next CTA holds its tail and, walking forward,
            // takes it first), that last piece is streamed FIRST and the rest of the range after it: both halves
            // of a cut sequence are then finished early, their merge through the workspace (several round trips
            // through a memory system that is saturated by the streams) happens in the background, and what a CTA
            // ends with is a whole sequence or a tail whose head was finished long ago: no global round trip at
            // the end of the kernel.
            auto locate = [&](int g, int &b_, int &kvh_, int &len_, int &tiles_, int &first_) {
                int lo = 0, hi = p.B;              // largest b with cum[b] <= g
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (cum[mid] <= g) lo = mid; else hi = mid;
                }
                b_ = lo;
                len_ = lens_s[lo];
                tiles_ = (len_ + kTileT - 1) / kTileT;
                kvh_ = small_div(g - cum[lo], tiles_ + 1);
                first_ = cum[lo] + kvh_ * (tiles_ + 1);          // flattened index of this sequence's marker; tile t at +1+t
            };
            int b = 0, kvh = 0, len = 0, tiles_b = 0, seq_first = 0;
            int split = my_end;                    // [split, my_end) goes first, then [my_begin, split)
            if (my_end > my_begin) {
                locate(my_end - 1, b, kvh, len, tiles_b, seq_first);
                if (my_end - 1 > seq_first && seq_first + tiles_b + 1 > my_end) split = max(seq_first, my_begin);
            }
            // The walk over a range's pieces: the first one is located by a binary search over the prefix sums, every
            // later one starts a sequence (the next KV head of the same sequence, or the next sequence with tokens),
            // so its numbers follow from the previous piece without a search or a division.
            for (int pass = (split < my_end ? 0 : 1); pass < 2 && ok; ++pass) {
            int g = pass == 0 ? split : my_begin;
            const int g_end = pass == 0 ? my_end : split;
            bool located = false;
            while (ok && g < g_end) {
                int first_cta;
                if (!located) {
                    if (pass == 1) locate(g, b, kvh, len, tiles_b, seq_first);   // pass 0 starts in the piece located above
                    first_cta = cta_of(seq_first + 1);
                    located = true;
                } else {
                    seq_first += tiles_b + 1;                     // == g: the previous piece ran to the end of its sequence
                    if (++kvh == p.Hkv) {
                        kvh = 0;
                        do { ++b; } while (lens_s[b] == 0);       // g < total: a sequence with tokens follows
                        len = lens_s[b];
                        tiles_b = (len + kTileT - 1) / kTileT;
                    }
                    first_cta = (int)blockIdx.x;
                }
                const int tile_begin = max(g - seq_first - 1, 0);
                const int tile_end = min(tiles_b, g_end - seq_first - 1);
                if (tile_end <= tile_begin) break;                // only the marker fell into this range (at its very end)
                const int npieces = (seq_first + tiles_b + 1 <= my_end) ? (int)blockIdx.x - first_cta + 1
                                                                        : cta_of(seq_first + tiles_b) - first_cta + 1;
                const int piece = (int)blockIdx.x - first_cta;
                {
                    PieceMeta &pp = post_ring[n_posted % kPostRing];
                    pp.b = b; pp.kvh = kvh; pp.piece = piece; pp.npieces = npieces; pp.stop = 0;
                    __threadfence_block();
                    *posted_count = ++n_posted;
                }
                int c1, c2, c3;
                for (int tile = tile_begin; tile < tile_end; ++tile, ++it) {
                    const uint32_t s = it % C::kStages;
                    const uint32_t ph = (it / C::kStages) & 1u;
                    if (!mbar_wait(&empty[s], ph ^ 1u, abort_flag)) { ok = false; break; }
                    TileMeta &mt = meta[s];
                    mt.b = b; mt.kvh = kvh; mt.t0 = tile * kTileT; mt.piece = piece; mt.kv_len = len;
                    mt.npieces = npieces;
                    mt.flags = (tile == tile_begin ? kFlagFirst : 0) | (tile + 1 == tile_end ? kFlagLast : 0);
                    // the first tile of a piece also brings the group's query rows (contiguous in q)
                    const bool first = (tile == tile_begin);
                    // The last tile of a sequence: if at most half of it holds tokens it is fetched in groups of
                    // p.tail_rows tokens (a few small boxes, nothing past the group that holds the last token); else as
                    // a whole tile like the others (one box; rows past the end of the sequence are never looked at
                    // by the consumers, rows past the end of the cache arrive as zeros). With pages smaller than a
                    // tile only the pages that hold tokens are fetched.
                    const bool paged = p.block_table != nullptr;
                    const int rem = len - tile * kTileT;
                    // (a whole tile of a contiguous cache, which is nearly every tile, is one box: no division on that path)
                    bool by_groups = false;
                    int box_rows = kTileT, n_box = 1;
                    if (rem < kTileT || paged) {
                        const int groups = (rem + p.tail_rows - 1) / p.tail_rows;
                        by_groups = rem < kTileT && groups * p.tail_rows * 2 <= kTileT;
                        box_rows = by_groups ? p.tail_rows : (paged ? p.page_box : kTileT);
                        n_box = by_groups ? groups : ((rem >= kTileT || box_rows == kTileT) ? kTileT / box_rows
                                                                                              : (rem + box_rows - 1) / box_rows);
                    }
                    // Neither a box nor a group straddles pages: page sizes are powers of two >= 16 and p.tail_rows is at
                    // most the page size. A page id outside the pool makes the box read zeros, never memory.
                    const int32_t *pages = paged ? p.block_table + (size_t)b * p.table_stride : nullptr;
                    const CUtensorMap *tk = by_groups ? &tmap_k_tail : &tmap_k;
                    const CUtensorMap *tv = by_groups ? &tmap_v_tail : &tmap_v;
                    int page_of[kTileT / 16];                    // looked up together: independent loads
#pragma unroll
                    for (int bx = 0; bx < kTileT / 16; ++bx)
                        page_of[bx] = (paged && bx < n_box) ? __ldg(pages + ((tile * kTileT + bx * box_rows) >> p.page_shift)) : b;
                    // paged fused append: the page of the newest token's slot (it lies in the last box fetched)
                    if (paged && p.k_new != nullptr && tile + 1 == tiles_b) {
                        int pg = page_of[0];
#pragma unroll
                        for (int bx = 1; bx < kTileT / 16; ++bx) pg = (bx < n_box) ? page_of[bx] : pg;
                        mt.pad = pg;
                    }
                    const uint32_t kv_bytes = (uint32_t)n_box * box_rows * (uint32_t)C::kTokBytes * C::kHalves * 2u;
                    // with the rope fused into the step, the piece's first tile also brings the cos / sin rows of
                    // the new token's position (kv_len - 1), if the table has it
                    const bool with_rope = first && p.rope_cos != nullptr && len - 1 < p.rope_n_pos;
                    const bool with_new = kNewBytes != 0 && p.k_new != nullptr && tile + 1 == tiles_b;   // the tile of the newest token
                    mbar_arrive_expect_tx(&full[s], kv_bytes + (first ? q_bytes : 0u) + (with_rope ? kRopeBytes : 0u) +
                                                        (with_new ? kNewBytes : 0u));
                    if (with_new) {
                        uint8_t *ns = q_slots + (size_t)s * q_stride + q_bytes + kRopeBytes;
                        const size_t src = (size_t)b * p.new_sb + (size_t)kvh * p.new_sh;
                        bulk_load_1d(ns, p.k_new + src, kNewBytes / 2, &full[s]);
                        bulk_load_1d(ns + kNewBytes / 2, p.v_new + src, kNewBytes / 2, &full[s]);
                    }
                    if (first)
                        bulk_load_1d(q_slots + (size_t)s * q_stride, p.q + ((size_t)b * p.Hq + (size_t)kvh * p.G) * D,
                                     q_bytes, &full[s]);
                    if (with_rope) {
                        uint8_t *rs = q_slots + (size_t)s * q_stride + q_bytes;
                        bulk_load_1d(rs, p.rope_cos + (size_t)(len - 1) * (D / 2), kRopeBytes / 2, &full[s]);
                        bulk_load_1d(rs + kRopeBytes / 2, p.rope_sin + (size_t)(len - 1) * (D / 2), kRopeBytes / 2, &full[s]);
                    }
                    uint8_t *dst = stages + (size_t)s * C::kStageBytes;
#pragma unroll
                    for (int bx = 0; bx < kTileT / 16; ++bx) {
                        if (bx >= n_box) break;
                        int tt = tile * kTileT + bx * box_rows;
                        if (paged) tt &= p.page_size - 1;
                        order_coords(p.coord, tt / C::kTokPerRow, kvh, page_of[bx], c1, c2, c3);
                        uint8_t *db = dst + bx * box_rows * C::kTokBytes;  // whole 8-row groups: the swizzle phase is kept
#pragma unroll
                        for (int hf = 0; hf < C::kHalves; ++hf) {
                            tma_load_4d_policy(db + hf * C::kHalfBytes, tk, &full[s], hf * C::kBoxD, c1, c2, c3, stream_policy);
                            tma_load_4d_policy(db + C::kTileBytes + hf * C::kHalfBytes, tv, &full[s], hf * C::kBoxD, c1, c2, c3, stream_policy);
                        }
                    }
                }
                g = seq_first + 1 + tile_end;
            }
            }
            __threadfence_block();
            *pieces_total = n_posted;
            if (ok) {
                const uint32_t s = it % C::kStages;
                const uint32_t ph = (it / C::kStages) & 1u;
                if (mbar_wait(&empty[s], ph ^ 1u, abort_flag)) {
                    meta[s].flags = kFlagStop;
                    mbar_arrive(&full[s]);
                }
            }
        }
    } else if (warp >= kFinisherWarp) {
        // ------------------------------------------------------------------ finisher warp
        // BigG: one finisher warp per 4 query heads of the group (so that a lane never owns more than four float4
        // outputs of a piece), each with its own rows of `comb`, of the outputs and of the workspace, and its own ticket.
        const int fin = BigG ? warp - kFinisherWarp : 0;
        const int nfin = BigG ? p.nfin : 1;
        const int g0 = BigG ? fin * 4 : 0;
        const int gcnt = BigG ? min(4, p.G - g0) : p.G;
        // sequences with no cached token get o = 0, lse = -inf (no tile ever refers to them)
        for (int b = blockIdx.x; fin == 0 && b < p.B; b += gridDim.x) {
            const int raw = p.kv_lens[b];
            if (raw <= 0 || (p.k_new != nullptr && raw > p.max_kv_len)) {      // the same rule as the producer's clamp
                for (int i = lane; i < p.Hq * D; i += 32) p.o[(size_t)b * p.Hq * D + i] = __float2bfloat16_rn(0.f);
                if (p.lse)
                    for (int i = lane; i < p.Hq; i += 32) p.lse[(size_t)b * p.Hq + i] = -INFINITY;
            }
        }
        const bool few_items = (gcnt * kVec <= 4 * 32);     // each lane owns at most four float4 outputs of a piece
        for (uint32_t n = 0;; ++n) {
            // ---- While the consumers are still streaming piece n: if every other piece of its sequence has
            // already arrived (the usual case for the piece a CTA ends with), fetch their partials now, so
            // that nothing but the local merge is left when the piece completes.
            float4 sv[4][4];
            float sl[4][4];
            bool prefetched = false;
            {
                // every decision in this loop is taken by lane 0 and broadcast, so that the warp stays converged
                const long long t0 = clock64();
                bool have_post = false, dead = false, all_done = false;
                while (true) {
                    int st = 0;                                       // 0: keep polling
                    if (lane == 0) {
                        if (*pieces_total == n) st = 4;                                                // nothing left
                        else if (mbar_try_wait(comb_full, n & 1u)) st = 1;                             // piece complete
                        else if (*abort_flag || clock64() - t0 > kWaitCycleBudget) st = 3;             // give up
                        else if (!have_post && (int32_t)(*posted_count - (n + 1u)) >= 0) st = 2;       // piece started
                    }
                    st = __shfl_sync(0xffffffffu, st, 0);
                    if (st == 1) break;
                    if (st == 4) { all_done = true; break; }
                    if (st == 3) { dead = true; break; }
                    if (st == 2) {
                        have_post = true;
                        __threadfence_block();
                        const PieceMeta pp = post_ring[n % kPostRing];
                        if (few_items && pp.npieces > 1 && pp.npieces <= 4) {
                            int *tk = p.tickets + ((size_t)pp.b * p.Hkv + pp.kvh) * nfin + fin;
                            int seen = (lane == 0) ? ld_acquire_gpu(tk) : 0;
                            seen = __shfl_sync(0xffffffffu, seen, 0);
                            if (seen == pp.npieces - 1) {
                                const size_t bh0 = (size_t)pp.b * p.Hq + pp.kvh * p.G + g0;
#pragma unroll
                                for (int u = 0; u < 4; ++u) {
                                    const int item = u * 32 + lane;
                                    const bool on = item < gcnt * kVec;
                                    const int r = on ? item / kVec : 0, d4 = on ? item % kVec : 0;
                                    const float *pl = p.part_lse + (bh0 + r) * p.nsplit;
                                    const float4 *po =
                                        reinterpret_cast<const float4 *>(p.part_o + (bh0 + r) * p.nsplit * D) + d4;
#pragma unroll
                                    for (int c = 0; c < 4; ++c) {
                                        const bool ld = on && c < pp.npieces && c != pp.piece;
                                        sl[u][c] = ld ? __ldcg(pl + c) : -INFINITY;
                                        sv[u][c] = ld ? __ldcg(po + (size_t)c * kVec) : make_float4(0.f, 0.f, 0.f, 0.f);
                                    }
                                }
                                prefetched = true;
                            }
                        }
                    } else {
                        __nanosleep(64);
                    }
                }
                if (dead) {
                    *abort_flag = 1;
                    break;
                }
                if (all_done) break;
                __syncwarp();                                         // lane 0's acquire covers the warp
            }
            const PieceMeta pm = *piece_meta;
            const bool single = (pm.npieces == 1);
            const size_t bh0 = (size_t)pm.b * p.Hq + pm.kvh * p.G + g0;
            int *tk = p.tickets + ((size_t)pm.b * p.Hkv + pm.kvh) * nfin + fin;
            const int np = pm.npieces;

            // ---- merge of the consumer warps' (max, sum, O). With at most 128 float4 outputs per piece (the usual
            // case) a lane owns up to four of them and works on all four in lockstep, stage by stage, so that the
            // four dependent chains overlap; the result is unnormalised, relative to the row maximum mloc.
            float4 acc4[4];
            float lsum4[4], mloc4[4];
            int r4[4], d4s[4];
            bool on4[4];
            if (few_items) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int item = u * 32 + lane;
                    on4[u] = item < gcnt * kVec;
                    r4[u] = on4[u] ? item / kVec : 0;
                    d4s[u] = on4[u] ? item % kVec : 0;
                    mloc4[u] = -INFINITY;
                    acc4[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                    lsum4[u] = 0.f;
                }
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w)
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        mloc4[u] = fmaxf(mloc4[u], CR::m(comb_b + ((size_t)w * p.G + g0 + r4[u]) * CR::kBytes));
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w)
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const uint8_t *row = comb_b + ((size_t)w * p.G + g0 + r4[u]) * CR::kBytes;
                        const float wgt = fast_exp2(CR::m(row) - mloc4[u]);    // warp that saw no token: max = -inf -> 0
                        const float4 v = CR::v4(row, d4s[u]);
                        acc4[u].x += wgt * v.x; acc4[u].y += wgt * v.y; acc4[u].z += wgt * v.z; acc4[u].w += wgt * v.w;
                        lsum4[u] += wgt * CR::l(row);
                    }
            }

            if (prefetched) {
                // ---- this piece completes its sequence: fold in the other pieces' partials fetched above and write
                // the final output; nothing goes through the workspace (prefetched implies few_items)
                float4 out4[4];
                float wsum4[4], mstar4[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    // own piece in the same form as the stored partials: normalised output + log2-sum-exp
                    const float inv_own = 1.f / lsum4[u];
                    const float lse_own = mloc4[u] + log2f(lsum4[u]);
                    mstar4[u] = fmaxf(lse_own, fmaxf(fmaxf(sl[u][0], sl[u][1]), fmaxf(sl[u][2], sl[u][3])));
                    const float e_own = fast_exp2(lse_own - mstar4[u]);
                    const float w_own = e_own * inv_own;
                    out4[u] = make_float4(acc4[u].x * w_own, acc4[u].y * w_own, acc4[u].z * w_own, acc4[u].w * w_own);
                    wsum4[u] = e_own;
                }
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const float wc = fast_exp2(sl[u][c] - mstar4[u]);          // absent piece: 2^-inf = 0
                        out4[u].x += wc * sv[u][c].x; out4[u].y += wc * sv[u][c].y;
                        out4[u].z += wc * sv[u][c].z; out4[u].w += wc * sv[u][c].w;
                        wsum4[u] += wc;
                    }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (on4[u]) {
                        const float inv = 1.f / wsum4[u];
                        uint2 packed;
                        packed.x = pack_bf16x2(out4[u].x * inv, out4[u].y * inv);
                        packed.y = pack_bf16x2(out4[u].z * inv, out4[u].w * inv);
                        *reinterpret_cast<uint2 *>(p.o + (bh0 + r4[u]) * D + d4s[u] * 4) = packed;
                        if (d4s[u] == 0 && p.lse) p.lse[bh0 + r4[u]] = (mstar4[u] + log2f(wsum4[u])) * 0.6931471805599453f;
                    }
                }
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(comb_empty);                // `comb` has been consumed
                    atomicExch(tk, 0);                      // every piece is accounted for: ready for the next call
                }
                continue;
            }

            // this piece alone: straight to the output if it is the whole sequence, else (normalised, with its
            // log2-sum-exp) to the workspace
            auto emit = [&](int r, int d4, float4 acc, float lsum, float mstar) {
                const float inv = 1.f / lsum;
                acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
                const size_t bh = bh0 + r;
                const float lse2 = mstar + log2f(lsum);
                if (single) {
                    uint2 packed;
                    packed.x = pack_bf16x2(acc.x, acc.y);
                    packed.y = pack_bf16x2(acc.z, acc.w);
                    *reinterpret_cast<uint2 *>(p.o + bh * D + d4 * 4) = packed;
                    if (d4 == 0 && p.lse) p.lse[bh] = lse2 * 0.6931471805599453f;
                } else {
                    const size_t slot = bh * p.nsplit + pm.piece;
                    *reinterpret_cast<float4 *>(p.part_o + slot * D + d4 * 4) = acc;
                    if (d4 == 0) p.part_lse[slot] = lse2;
                }
            };
            if (few_items) {
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (on4[u]) emit(r4[u], d4s[u], acc4[u], lsum4[u], mloc4[u]);
            } else {
                for (int item = lane; item < gcnt * kVec; item += 32) {
                    const int r = item / kVec, d4 = item % kVec;
                    float mw[kConsumerWarps];
                    float mstar = -INFINITY;
#pragma unroll
                    for (int w = 0; w < kConsumerWarps; ++w) {
                        mw[w] = CR::m(comb_b + ((size_t)w * p.G + g0 + r) * CR::kBytes);
                        mstar = fmaxf(mstar, mw[w]);
                    }
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                    float lsum = 0.f;
#pragma unroll
                    for (int w = 0; w < kConsumerWarps; ++w) {
                        const uint8_t *row = comb_b + ((size_t)w * p.G + g0 + r) * CR::kBytes;
                        const float wgt = fast_exp2(mw[w] - mstar);    // warp that saw no token: max = -inf -> 0
                        const float4 v = CR::v4(row, d4);
                        acc.x += wgt * v.x; acc.y += wgt * v.y; acc.z += wgt * v.z; acc.w += wgt * v.w;
                        lsum += wgt * CR::l(row);
                    }
                    emit(r, d4, acc, lsum, mstar);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(comb_empty);        // `comb` has been consumed
            if (single) continue;

            // ---- ticket: the last piece of this (sequence, KV head) to arrive merges all of them.
            // The counter is read (acquire) before the fence; if it already shows every other piece, their
            // partials are loaded while this piece's own ticket is in flight (fence, then ticket and loads
            // together: two memory round trips instead of three).
            const bool small = few_items && np <= 4;
            int seen = 0;
            if (small && lane == 0) seen = ld_acquire_gpu(tk);
            __threadfence();                               // this warp's partials visible device-wide
            seen = __shfl_sync(0xffffffffu, seen, 0);
            const bool spec = small && (seen == np - 1);
            auto load_pieces = [&]() {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int item = u * 32 + lane;
                    const bool on = item < gcnt * kVec;
                    const int r = on ? item / kVec : 0, d4 = on ? item % kVec : 0;
                    const float *pl = p.part_lse + (bh0 + r) * p.nsplit;
                    const float4 *po = reinterpret_cast<const float4 *>(p.part_o + (bh0 + r) * p.nsplit * D) + d4;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const bool ld = on && c < np;
                        sl[u][c] = ld ? __ldcg(pl + c) : -INFINITY;
                        sv[u][c] = ld ? __ldcg(po + (size_t)c * kVec) : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
            };
            if (spec) load_pieces();
            int ticket = 0;
            if (lane == 0) {
                ticket = atomicAdd(tk, 1);
                if (ticket == np - 1) atomicExch(tk, 0);               // ready for the next call
            }
            ticket = __shfl_sync(0xffffffffu, ticket, 0);
            if (ticket != np - 1) continue;
            if (!spec) __threadfence();
            if (small) {
                if (!spec) load_pieces();
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int item = u * 32 + lane;
                    if (item < gcnt * kVec) {
                        const int r = item / kVec, d4 = item % kVec;
                        const float mstar = fmaxf(fmaxf(sl[u][0], sl[u][1]), fmaxf(sl[u][2], sl[u][3]));
                        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                        float wsum = 0.f;
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const float w = fast_exp2(sl[u][c] - mstar);           // absent piece: 2^-inf = 0
                            acc.x += w * sv[u][c].x; acc.y += w * sv[u][c].y;
                            acc.z += w * sv[u][c].z; acc.w += w * sv[u][c].w;
                            wsum += w;
                        }
                        const float inv = 1.f / wsum;
                        uint2 packed;
                        packed.x = pack_bf16x2(acc.x * inv, acc.y * inv);
                        packed.y = pack_bf16x2(acc.z * inv, acc.w * inv);
                        *reinterpret_cast<uint2 *>(p.o + (bh0 + r) * D + d4 * 4) = packed;
                        if (d4 == 0 && p.lse) p.lse[bh0 + r] = (mstar + log2f(wsum)) * 0.6931471805599453f;
                    }
                }
                __syncwarp();
                continue;
            }
            // second pass: out = sum_c w_c o_c / sum_c w_c with w_c = 2^(lse_c - max_c lse_c)
            for (int idx = lane; idx < gcnt * np; idx += 32) {
                const int r = idx / np, c = idx % np;
                merge_lse[(g0 + r) * p.nsplit + c] = __ldcg(p.part_lse + (bh0 + r) * p.nsplit + c);
            }
            __syncwarp();
            for (int base = 0; base < gcnt * kVec; base += 4 * 32) {
                float4 res[4];
                float lse_out[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int item = base + u * 32 + lane;
                    res[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                    lse_out[u] = 0.f;
                    if (item < gcnt * kVec) {
                        const int r = item / kVec, d4 = item % kVec;
                        const float *wl = merge_lse + (g0 + r) * p.nsplit;
                        float mstar = -INFINITY;
                        for (int c = 0; c < np; ++c) mstar = fmaxf(mstar, wl[c]);
                        const float4 *po = reinterpret_cast<const float4 *>(p.part_o + (bh0 + r) * p.nsplit * D) + d4;
                        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                        float wsum = 0.f;
#pragma unroll 4
                        for (int c = 0; c < np; ++c) {
                            const float w = fast_exp2(wl[c] - mstar);
                            const float4 v = __ldcg(po + (size_t)c * kVec);
                            acc.x += w * v.x; acc.y += w * v.y; acc.z += w * v.z; acc.w += w * v.w;
                            wsum += w;
                        }
                        const float inv = 1.f / wsum;
                        res[u] = make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
                        lse_out[u] = (mstar + log2f(wsum)) * 0.6931471805599453f;
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int item = base + u * 32 + lane;
                    if (item < gcnt * kVec) {
                        const int r = item / kVec, d4 = item % kVec;
                        uint2 packed;
                        packed.x = pack_bf16x2(res[u].x, res[u].y);
                        packed.y = pack_bf16x2(res[u].z, res[u].w);
                        *reinterpret_cast<uint2 *>(p.o + (bh0 + r) * D + d4 * 4) = packed;
                        if (d4 == 0 && p.lse) p.lse[bh0 + r] = lse_out[u];
                    }
                }
            }
            __syncwarp();
        }
    } else {
        // ------------------------------------------------------------------ consumer warps
        WarpAttnState<D> st;
        st.reset();
        uint32_t qf[D / 16][4];
        const int r_lo = lane >> 2;          // query head within the group held in rows lane/4, lane/4+8
        const int r_hi = r_lo + 8;
        uint32_t n_dumps = 0;                // pieces handed to the finisher so far
        uint32_t n_rotated = 0;              // pieces whose query rows were rotated (phase of q_rotated)
        float k_sc = 1.f, v_sc = 1.f;        // fp8 cache: scales of the piece's KV head (read once per piece)

        for (uint32_t it = 0;; ++it) {
            const uint32_t s = it % C::kStages;
            const uint32_t ph = (it / C::kStages) & 1u;
            if (!mbar_wait(&full[s], ph, abort_flag)) break;
            const TileMeta mt = meta[s];
            // end of this CTA's range: nothing to tell the finisher, which knows the number of pieces from the producer
            if (mt.flags & kFlagStop) break;

            if (mt.flags & kFlagFirst) {
                st.reset();
                if constexpr (F8) {
                    k_sc = __ldg(p.k_scale + mt.kvh);
                    v_sc = __ldg(p.v_scale + mt.kvh);
                }
                if constexpr (!F8 || R8) {
                    if (p.rope_cos != nullptr && mt.kv_len - 1 < p.rope_n_pos) {
                        // Rope fused into the step: the piece's query rows are rotated in place in the stage's slot, row g by
                        // consumer warp g mod W, before anybody builds fragments from them. Every warp also keeps the
                        // cos | sin rows in its own scratch: the stage is recycled long before the tile with the new
                        // token (whose k row needs them) arrives.
                        uint8_t *slot = q_slots + (size_t)s * q_stride;
                        float *mine = rope_priv + (size_t)warp * D;
                        const float4 *src = reinterpret_cast<const float4 *>(slot + q_bytes);
                        for (int i = lane; i < D / 4; i += 32) reinterpret_cast<float4 *>(mine)[i] = src[i];
                        __syncwarp();
                        for (int g = warp; g < p.G; g += kConsumerWarps)
                            rope_row_in_smem<D>(reinterpret_cast<uint32_t *>(slot) + (size_t)g * (D / 2), mine, p.q_weight != nullptr,
                                                p.norm_eps, norm_w, lane);
                        __syncwarp();
                        if (lane == 0) mbar_arrive(q_rotated);
                        if (!mbar_wait(q_rotated, n_rotated & 1u, abort_flag)) break;
                        ++n_rotated;
                    }
                }
                const uint32_t *qs = reinterpret_cast<const uint32_t *>(q_slots + (size_t)s * q_stride);
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

            const uint32_t k_tile = smem_u32(stages + (size_t)s * C::kStageBytes);
            const uint32_t v_tile = k_tile + C::kTileBytes;
            const int row0 = warp * 16 * C::kSub;
            const int nvalid = mt.kv_len - (mt.t0 + row0);       // valid tokens in this warp's slice
            bool wrote_smem = false;
            if (!F8 && p.k_new != nullptr && nvalid > 0 && nvalid <= 16 * C::kSub) {
                // fused append: this slice holds the sequence's newest token (row `last` of the tile). Its K/V
                // arrive from the caller, not from the cache: patch the tile in shared memory and write the
                // cache slot (each slot belongs to exactly one CTA's range and one warp's slice).
                const int last = row0 + nvalid - 1;
                constexpr int kChunks = D / 8;
                uint4 kk = make_uint4(0u, 0u, 0u, 0u), vv = kk;
                if (lane < kChunks) {
                    if constexpr (kNewBytes != 0) {          // the rows came with this tile
                        const uint4 *ns = reinterpret_cast<const uint4 *>(q_slots + (size_t)s * q_stride + q_bytes + kRopeBytes);
                        kk = ns[lane];
                        vv = ns[kChunks + lane];
                    } else {
                        const size_t src = (size_t)mt.b * p.new_sb + (size_t)mt.kvh * p.new_sh + lane * 8;
                        kk = __ldg(reinterpret_cast<const uint4 *>(p.k_new + src));
                        vv = __ldg(reinterpret_cast<const uint4 *>(p.v_new + src));
                    }
                }
                if (p.rope_cos != nullptr)                                      // all lanes: shuffles inside
                    kk = rope_k_row<D>(kk, p.k_weight != nullptr, p.norm_eps, rope_priv + (size_t)warp * D, norm_w + D,
                                        mt.kv_len - 1 < p.rope_n_pos, lane);
                if (lane < kChunks) {
                    // the slot in the cache: with pages, behind the block table. No page there: nothing is written,
                    // and the tile keeps the zeros that the fetch of a missing page delivers.
                    long long outer = mt.b, slot = mt.kv_len - 1;
                    if (p.block_table != nullptr) {
                        outer = mt.pad;                                          // looked up by the producer
                        slot &= p.page_size - 1;
                    }
                    if (p.block_table == nullptr || (outer >= 0 && outer < p.num_pages)) {
                        uint8_t *kt = stages + (size_t)s * C::kStageBytes;
                        const uint32_t off = (lane >> 3) * C::kHalfBytes + swz128(last, lane & 7);
                        *reinterpret_cast<uint4 *>(kt + off) = kk;
                        *reinterpret_cast<uint4 *>(kt + C::kTileBytes + off) = vv;
                        const size_t dst = (size_t)outer * p.c_sb + (size_t)mt.kvh * p.c_sh + (size_t)slot * p.c_st + lane * 8;
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
                    bool rotated = false;
                    if constexpr (R8) {
                        if (p.rope_cos != nullptr) {
                            uint4 kk = make_uint4(0u, 0u, 0u, 0u);
                            if (lane < D / 8) {
                                if constexpr (kNewBytes != 0)
                                    kk = reinterpret_cast<const uint4 *>(q_slots + (size_t)s * q_stride + q_bytes + kRopeBytes)[lane];
                                else
                                    kk = __ldg(reinterpret_cast<const uint4 *>(p.k_new + (size_t)mt.b * p.new_sb + (size_t)mt.kvh * p.new_sh + lane * 8));
                            }
                            kk = rope_k_row<D>(kk, p.k_weight != nullptr, p.norm_eps, rope_priv + (size_t)warp * D, norm_w + D,
                                                mt.kv_len - 1 < p.rope_n_pos, lane);
                            regroup_row_16(kk, lane, ka, kb);
                            rotated = true;
                        }
                    }
                    uint4 va = make_uint4(0u, 0u, 0u, 0u), vb = va;
                    if (lane < D / 16) {
                        if constexpr (kNewBytes != 0) {      // the rows came with this tile
                            const uint4 *ns = reinterpret_cast<const uint4 *>(q_slots + (size_t)s * q_stride + q_bytes + kRopeBytes);
                            if (!rotated) {
                                ka = ns[2 * lane];
                                kb = ns[2 * lane + 1];
                            }
                            va = ns[D / 8 + 2 * lane];
                            vb = ns[D / 8 + 2 * lane + 1];
                        } else {
                            const size_t src = (size_t)mt.b * p.new_sb + (size_t)mt.kvh * p.new_sh + lane * 16;
                            if (!rotated) {
                                ka = __ldg(reinterpret_cast<const uint4 *>(p.k_new + src));
                                kb = __ldg(reinterpret_cast<const uint4 *>(p.k_new + src) + 1);
                            }
                            va = __ldg(reinterpret_cast<const uint4 *>(p.v_new + src));
                            vb = __ldg(reinterpret_cast<const uint4 *>(p.v_new + src) + 1);
                        }
                    }
                    if (lane < D / 16) {
                        const uint4 kq = quantise16(ka, kb, k_sc);
                        const uint4 vq = quantise16(va, vb, v_sc);
                        long long outer = mt.b, slot = mt.kv_len - 1;
                        if (p.block_table != nullptr) {
                            outer = mt.pad;                                      // looked up by the producer
                            slot &= p.page_size - 1;
                        }
                        if (p.block_table == nullptr || (outer >= 0 && outer < p.num_pages)) {
                            uint8_t *kt = stages + (size_t)s * C::kStageBytes;
                            const uint32_t off = tok_chunk_f8<D>(0u, (uint32_t)last, (uint32_t)lane);
                            *reinterpret_cast<uint4 *>(kt + off) = kq;
                            *reinterpret_cast<uint4 *>(kt + C::kTileBytes + off) = vq;
                            // fp8 caches: the strides count bytes
                            const size_t dst = (size_t)outer * p.c_sb + (size_t)mt.kvh * p.c_sh + (size_t)slot * p.c_st + lane * 16;
                            *reinterpret_cast<uint4 *>(reinterpret_cast<uint8_t *>(p.cache_k) + dst) = kq;
                            *reinterpret_cast<uint4 *>(reinterpret_cast<uint8_t *>(p.cache_v) + dst) = vq;
                        }
                    }
                    wrote_smem = true;
                    __syncwarp();
                }
                if (nvalid > 0) {
                    // 32 tokens per step: two 16-token blocks share one softmax update. A block with no valid
                    // token is skipped (its rows may never have been fetched); in the last valid block the
                    // tokens past the end get no weight and their V rows are cleared.
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
                        constexpr int kCh = D / 16;                                   // 16-byte chunks of a token
                        for (int i = lane; i < (fetched_end - nvalid) * kCh; i += 32)
                            *reinterpret_cast<uint4 *>(vt + tok_chunk_f8<D>(0u, (uint32_t)(row0 + nvalid + i / kCh), (uint32_t)(i % kCh))) =
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
                // kSub 16-token blocks per step share one softmax update. A block with no valid token is skipped (its
                // rows may never have been fetched); in the last valid block the tokens past the end of the sequence get
                // no weight, and their V rows (which may hold any bits, NaN included) are cleared so that 0 * garbage
                // cannot appear.
                constexpr int kSub = C::kSub;
                float sv[2 * kSub][4];
                const float sc = p.scale_log2e;
#pragma unroll
                for (int u = 0; u < kSub; ++u) {
                    if (u == 0 || nvalid > 16 * u) {
                        warp_qk_16x16<D>(qf, k_tile, C::kHalfBytes, row0 + 16 * u, sv[2 * u], sv[2 * u + 1]);
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
                    const int chunks_per_row = C::kRowBytes / 16;
                    const int fetched_end = (nvalid + 15) & ~15;                 // end of the last valid block
                    for (int i = lane; i < (fetched_end - nvalid) * chunks_per_row; i += 32) {
                        const int r = row0 + nvalid + i / chunks_per_row;
                        const int ch = i % chunks_per_row;
                        *reinterpret_cast<uint4 *>(vt + (ch >> 3) * C::kHalfBytes + r * 128 + ((ch & 7) << 4)) =
                            make_uint4(0u, 0u, 0u, 0u);
                    }
                    wrote_smem = true;
                    __syncwarp();
                }
                uint32_t pa[kSub][4];
                warp_softmax_tiles<D, false, 2 * kSub>(st, sv, pa);
#pragma unroll
                for (int u = 0; u < kSub; ++u)
                    if (u == 0 || nvalid > 16 * u) warp_pv_16x16<D>(st, pa[u], v_tile, C::kHalfBytes, row0 + 16 * u);
            }

            if (wrote_smem) fence_proxy_async_smem();   // generic writes before the next TMA fill
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[s]);

            if (mt.flags & kFlagLast) {
                // ---- hand this piece's (max, sum, O) to the finisher warp and carry on
                if (!mbar_wait(comb_empty, (n_dumps & 1u) ^ 1u, abort_flag)) break;
                float l0 = st.l[0], l1 = st.l[1];
                l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
                l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
                l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
                l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
                uint8_t *cw = comb_b + (size_t)warp * p.G * CR::kBytes;
                // fp8: accumulator tiles alternate even / odd head dims (a tile pair gives this lane 4 consecutive
                // dims) and O still lacks the V scale of its KV head
                const float vs = F8 ? v_sc : 1.f;
                if (r_lo < p.G) {
                    uint8_t *rowb = cw + (size_t)r_lo * CR::kBytes;
                    float *row = reinterpret_cast<float *>(rowb);
                    if ((lane & 3) == 0) {
                        *reinterpret_cast<float *>(rowb + CR::kOffM) = st.m[0];
                        *reinterpret_cast<float *>(rowb + CR::kOffM + 4) = l0;
                    }
                    if constexpr (BigG) {
                        // bf16 rows (groups of 5 to 8 heads occupy rows lane/4 only): the same elements, half the bytes
                        if constexpr (F8) {
#pragma unroll
                            for (int ch = 0; ch < D / 16; ++ch)
                                *reinterpret_cast<uint2 *>(rowb + (ch * 16 + 4 * (lane & 3)) * 2) =
                                    make_uint2(pack_bf16x2(st.o[2 * ch][0] * vs, st.o[2 * ch + 1][0] * vs),
                                               pack_bf16x2(st.o[2 * ch][1] * vs, st.o[2 * ch + 1][1] * vs));
                        } else {
#pragma unroll
                            for (int nt = 0; nt < D / 8; ++nt)
                                *reinterpret_cast<uint32_t *>(rowb + (nt * 8 + 2 * (lane & 3)) * 2) = pack_bf16x2(st.o[nt][0], st.o[nt][1]);
                        }
                    } else if constexpr (F8) {
#pragma unroll
                        for (int ch = 0; ch < D / 16; ++ch)
                            *reinterpret_cast<float4 *>(row + ch * 16 + 4 * (lane & 3)) =
                                make_float4(st.o[2 * ch][0] * vs, st.o[2 * ch + 1][0] * vs, st.o[2 * ch][1] * vs,
                                            st.o[2 * ch + 1][1] * vs);
                    } else {
#pragma unroll
                        for (int nt = 0; nt < D / 8; ++nt)
                            *reinterpret_cast<float2 *>(row + nt * 8 + 2 * (lane & 3)) = make_float2(st.o[nt][0], st.o[nt][1]);
                    }
                }
                if (r_hi < p.G) {
                    uint8_t *rowb = cw + (size_t)r_hi * CR::kBytes;
                    float *row = reinterpret_cast<float *>(rowb);
                    if ((lane & 3) == 0) {
                        *reinterpret_cast<float *>(rowb + CR::kOffM) = st.m[1];
                        *reinterpret_cast<float *>(rowb + CR::kOffM + 4) = l1;
                    }
                    if constexpr (BigG) {
                        if constexpr (F8) {
#pragma unroll
                            for (int ch = 0; ch < D / 16; ++ch)
                                *reinterpret_cast<uint2 *>(rowb + (ch * 16 + 4 * (lane & 3)) * 2) =
                                    make_uint2(pack_bf16x2(st.o[2 * ch][2] * vs, st.o[2 * ch + 1][2] * vs),
                                               pack_bf16x2(st.o[2 * ch][3] * vs, st.o[2 * ch + 1][3] * vs));
                        } else {
#pragma unroll
                            for (int nt = 0; nt < D / 8; ++nt)
                                *reinterpret_cast<uint32_t *>(rowb + (nt * 8 + 2 * (lane & 3)) * 2) = pack_bf16x2(st.o[nt][2], st.o[nt][3]);
                        }
                    } else if constexpr (F8) {
#pragma unroll
                        for (int ch = 0; ch < D / 16; ++ch)
                            *reinterpret_cast<float4 *>(row + ch * 16 + 4 * (lane & 3)) =
                                make_float4(st.o[2 * ch][2] * vs, st.o[2 * ch + 1][2] * vs, st.o[2 * ch][3] * vs,
                                            st.o[2 * ch + 1][3] * vs);
                    } else {
#pragma unroll
                        for (int nt = 0; nt < D / 8; ++nt)
                            *reinterpret_cast<float2 *>(row + nt * 8 + 2 * (lane & 3)) = make_float2(st.o[nt][2], st.o[nt][3]);
                    }
                }
                if (warp == 0 && lane == 0) {
                    piece_meta->b = mt.b; piece_meta->kvh = mt.kvh; piece_meta->piece = mt.piece;
                    piece_meta->npieces = mt.npieces; piece_meta->stop = 0;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(comb_full);
                ++n_dumps;
            }
        }
    }

    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) {
        atomicOr(p.status + kStatusErrWord, kErrDecodeWait);
        p.status[kStatusInfoWord] = blockIdx.x;
    }
}

// Resident CTAs per SM for a given dynamic shared-memory size (0 on failure).
template <int D, int W, bool F8, bool BigG, bool R8 = false>
int decode_blocks_per_sm(size_t smem)
{
    static bool attr_set_on[kDeviceSlots] = {};
    const int slot = device_slot();
    if (slot < 0) return 0;
    bool &attr_set = attr_set_on[slot];
    std::lock_guard<std::mutex> lock(setup_mutex());
    if (!attr_set) {
        // the opt-in limit is per kernel: allow everything the SM has
        if (cudaFuncSetAttribute(decode_split_kernel<D, W, F8, BigG, R8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) !=
            cudaSuccess)
            return 0;
        attr_set = true;
    }
    if (smem > 227 * 1024) return 0;
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, decode_split_kernel<D, W, F8, BigG, R8>, (BigG ? 11 : W + 2) * 32, smem) != cudaSuccess)
        return 0;
    return n;
}

}  // namespace

namespace {

// Host-side view of one kernel shape.
struct ShapeOps {
    int warps, tile_t;
    size_t (*smem_bytes)(int G, int nsplit);
    int (*blocks_per_sm)(size_t smem);
};

template <int D, int W, bool F8, bool BigG = false, bool R8 = false>
ShapeOps shape_ops()
{
    return ShapeOps{W, DecodeCfg<D, W, F8>::kTileT, &decode_smem_bytes<D, W, F8, BigG>, &decode_blocks_per_sm<D, W, F8, BigG, R8>};
}

// Groups of more than 4 query heads at head_dim 128: 16-bit hand-over rows and one finisher warp per 4 heads. Up to 8
// heads on the 8-warp shape; 9 to 16 heads on a 6-warp shape (96-token tiles: three 48 KB stages leave room for the
// sixteen rows per warp, and 6 + 1 + 4 warps keep the block at 11 warps).
bool is_big_group(int D, int warps, int G)
{
    return D == 128 && ((warps == 8 && G > 4 && G <= 8) || (warps == 6 && G > 8 && G <= 16));
}

ShapeOps pick_shape(int D, int warps, bool fp8, bool big = false, bool rope8 = false)
{
    if (fp8 && rope8) {          // the e4m3-cache kernels that carry the rope-fused step
        if (big && warps == 6) return shape_ops<128, 6, true, true, true>();
        if (big) return shape_ops<128, 8, true, true, true>();
        if (D == 64) return warps == 8 ? shape_ops<64, 8, true, false, true>() : shape_ops<64, 4, true, false, true>();
        return warps == 8 ? shape_ops<128, 8, true, false, true>() : shape_ops<128, 4, true, false, true>();
    }
    if (big && warps == 6) return fp8 ? shape_ops<128, 6, true, true>() : shape_ops<128, 6, false, true>();
    if (big) return fp8 ? shape_ops<128, 8, true, true>() : shape_ops<128, 8, false, true>();
    if (fp8 && D == 64) return warps == 8 ? shape_ops<64, 8, true>() : shape_ops<64, 4, true>();
    if (fp8) return warps == 8 ? shape_ops<128, 8, true>() : shape_ops<128, 4, true>();
    if (D == 128) return warps == 8 ? shape_ops<128, 8, false>() : shape_ops<128, 4, false>();
    return warps == 8 ? shape_ops<64, 8, false>() : shape_ops<64, 4, false>();
}

// Plan for one kernel shape (warps = 4 or 8).
DecodePlan plan_for_shape(int B, int Hq, int Hkv, int D, int max_kv_len, size_t ws_limit, int warps, bool have_dev,
                          bool fp8)
{
    // Grid: every resident CTA slot of the device. A floor on the tiles per CTA bounds the number of
    // pieces a sequence can be cut into (and with it the partials in the workspace and the finisher's
    // scratch) when the real lengths are far below max_kv_len; it is raised until the partials fit the
    // caller's workspace and the shared memory fits the SM.
    DecodePlan pl;
    const int G = Hq / Hkv;
    const ShapeOps ops = pick_shape(D, warps, fp8, is_big_group(D, warps, G));
    pl.warps = warps;
    auto blocks = [&](int nsplit) {
        const size_t smem = ops.smem_bytes(G, nsplit);
        if (!have_dev) return smem <= 227 * 1024 ? (warps == 4 ? 2 : 1) : 0;   // sizing without a device
        return ops.blocks_per_sm(smem);
    };
    int per_sm = blocks(2);
    if (per_sm < 1) per_sm = 1;
    const long long slots = (long long)sm_count() * per_sm;
    const long long tiles_max = max_kv_len > 0 ? (max_kv_len + ops.tile_t - 1) / ops.tile_t : 1;
    const long long total_max = (long long)B * Hkv * tiles_max;
    long long min_tiles = (total_max + 8 * slots - 1) / (8 * slots);
    // small problems are latency-bound: a CTA that streams only a tile or two spends longer in the
    // merge of the many pieces than in the stream, so give every CTA at least 1024 tokens (or a quarter
    // of the longest sequence, if that is less)
    const long long floor_cap = 1024 / ops.tile_t;
    const long long floor_tiles = (tiles_max + 3) / 4 < floor_cap ? (tiles_max + 3) / 4 : floor_cap;
    if (min_tiles < floor_tiles) min_tiles = floor_tiles;
    if (min_tiles < 1) min_tiles = 1;
    for (;; min_tiles *= 2) {
        // a sequence of n tiles meets at most ceil(n / tiles per CTA) + 1 CTAs, never more than it has tiles
        long long nsplit = (tiles_max + min_tiles - 1) / min_tiles + 1;
        if (nsplit > tiles_max) nsplit = tiles_max;
        if (nsplit < 1) nsplit = 1;
        pl.min_tiles = (int)min_tiles;
        pl.nsplit = (int)nsplit;
        pl.ws_bytes = kStatusBytes + kTicketBytes +
                      (size_t)B * Hq * pl.nsplit * (D + 1) * sizeof(float);
        const int n = blocks(pl.nsplit);
        pl.grid = sm_count() * (n > 0 ? n : 1);
        pl.fits = n > 0;
        if ((pl.ws_bytes <= ws_limit && n > 0) || min_tiles >= tiles_max) break;
    }
    return pl;
}

}  // namespace

DecodePlan plan_decode(int B, int Hq, int Hkv, int D, int max_kv_len, size_t ws_limit, bool fp8, int page_size)
{
    int n_dev = 0;
    const bool have_dev = cudaGetDeviceCount(&n_dev) == cudaSuccess && n_dev > 0;
    if (!have_dev) (void)cudaGetLastError();
    // groups of 9 to 16 query heads at head_dim 128: the 6-warp shape (its 96-token tiles are fetched in 32-token
    // boxes from pages they do not line up with)
    if (D == 128 && Hq / Hkv > 8) {
        const DecodePlan six = plan_for_shape(B, Hq, Hkv, D, max_kv_len, ws_limit, 6, have_dev, fp8);
        if (six.fits && six.ws_bytes <= ws_limit) return six;
    }
    // 128-wide heads: prefer the 8-warp shape (one CTA per SM, ranges twice as long, so fewer sequences are cut
    // between CTAs) whenever its shared memory fits, which it does for query-head groups of up to 4; else 4 warps.
    const int forced = decode_override().split_warps;    // tuning override: force a shape
    // With 64-wide heads a tile carries half the bytes for the same per-tile work in the consumer warps, and two
    // 4-warp CTAs per SM (two independent streams) hide that better than one 8-warp CTA: 4 warps first there.
    const bool four_first = forced == 4 || (forced == 0 && D == 64);
    const DecodePlan first = plan_for_shape(B, Hq, Hkv, D, max_kv_len, ws_limit, four_first ? 4 : 8, have_dev, fp8);
    if ((first.fits && first.ws_bytes <= ws_limit) || forced != 0) return first;
    const DecodePlan second = plan_for_shape(B, Hq, Hkv, D, max_kv_len, ws_limit, four_first ? 8 : 4, have_dev, fp8);
    if (second.fits && second.ws_bytes <= ws_limit) return second;
    return four_first ? first : second;          // neither fits: the 4-warp plan carries the diagnosis
}

l4l_status launch_decode(const void *q, void *o, const l4l_kv_cache &cache, const int32_t *d_kv_lens,
                         int max_kv_len, int B, int Hq, int Hkv, int D, float scale, float *d_lse,
                         void *workspace, const DecodePlan &plan, cudaStream_t stream, const l4l_tensor4 *k_new,
                         const l4l_tensor4 *v_new, const PagedTable *paged, const Fp8Scales *fp8, const RopeArgs *rope)
{
    if (rope && (!k_new || !v_new)) return L4L_ERR_UNSUPPORTED;   // only with the fused append
    // fp8: cache.k / cache.v point at e4m3 bytes, the strides count bytes (= elements)
    // fp8 at head_dim 64: two 64-byte tokens make one 128-byte tile row, so the token rows of the cache (or of a page)
    // must lie back to back and come in pairs
    const bool pair_rows = fp8 && D == 64;
    if (pair_rows && (cache.stride_t != 64 || (cache.max_len & 1))) return L4L_ERR_UNSUPPORTED;
    const int esz = fp8 ? 1 : 2;
    // paged: `cache` describes the page pool (stride_b = stride between pages, max_len = page size)
    // hundreds of short sequences: one warp per (sequence, KV head), nothing to merge
    if (decode_warp_eligible(B, Hq, Hkv, D, max_kv_len, fp8 != nullptr, rope != nullptr, k_new != nullptr))
        return launch_decode_warp(q, o, cache, d_kv_lens, max_kv_len, B, Hq, Hkv, D, scale, d_lse, stream, k_new, v_new,
                                  paged, fp8, rope);
    {
        // small batches are latency-bound: one cluster per (sequence, KV head), no workspace round trips
        const int width = decode_cluster_width(B, Hq, Hkv, D, max_kv_len, fp8 != nullptr);
        if (width > 0)
            return launch_decode_cluster(q, o, cache, d_kv_lens, max_kv_len, B, Hq, Hkv, D, scale, d_lse, workspace,
                                         stream, k_new, v_new, paged, rope, fp8, width);
    }
    const int G = Hq / Hkv;
    const bool big = is_big_group(D, plan.warps, G);
    const int nfin = big ? (G + 3) / 4 : 1;
    const bool rope8 = fp8 != nullptr && rope != nullptr;
    const ShapeOps ops = pick_shape(D, plan.warps, fp8 != nullptr, big, rope8);
    const int kTileT = ops.tile_t;
    const size_t smem = ops.smem_bytes(G, plan.nsplit);
    if (ops.blocks_per_sm(smem) == 0) return L4L_ERR_CUDA;
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    int *tickets = reinterpret_cast<int *>(ws + kStatusBytes);
    // partial outputs first: their float4 accesses need 16-byte alignment
    float *part_o = reinterpret_cast<float *>(ws + kStatusBytes + kTicketBytes);
    float *part_lse = part_o + (size_t)B * Hq * plan.nsplit * D;

    // sequences per launch: bounded by the prefix-sum array in shared memory and by the ticket region
    int slice = (int)(kTicketBytes / sizeof(int)) / (Hkv * nfin);
    if (slice > kMaxB) slice = kMaxB;
    if (slice < 1) return L4L_ERR_UNSUPPORTED;
    for (int b0 = 0; b0 < B; b0 += slice) {
        const int nb = (B - b0 < slice) ? (B - b0) : slice;
        CUtensorMap tk, tv, tk_tail, tv_tail;   // tile-sized boxes, and small boxes for a mostly empty last tile of a sequence
        TmapCoord coord, coord_v;
        // contiguous: the maps cover this slice's sequences; paged: the whole pool, whatever the slice
        const size_t first = paged ? 0 : (size_t)b0 * cache.stride_b;
        const int outer = paged ? paged->num_pages : nb;
        const uint8_t *kb = static_cast<const uint8_t *>(cache.k) + first * esz;
        const uint8_t *vb = static_cast<const uint8_t *>(cache.v) + first * esz;
        const int box_d = fp8 ? 128 : 64;
        // no box may straddle pages: pages smaller than a tile are fetched page by page, and tiles that are not a
        // power of two (96 tokens) over larger pages in 32-token boxes (page sizes are powers of two >= 16)
        int box_t = kTileT;
        if (paged) box_t = (kTileT % cache.max_len == 0) ? cache.max_len : (cache.max_len % kTileT == 0 ? kTileT : 32);
        const int tail_rows = (paged && cache.max_len < 32) ? cache.max_len : 32;
        // what the maps see as a row: a token, or (fp8 at head_dim 64) a pair of tokens
        const int tpr = pair_rows ? 2 : 1, map_d = pair_rows ? 128 : D;
        const int64_t map_rows = cache.max_len / tpr, map_st = cache.stride_t * tpr;
        if (!make_tmap(&tk, &coord, kb, map_d, map_rows, Hkv, outer, map_st, cache.stride_h,
                       cache.stride_b, box_d, box_t / tpr, esz) ||
            !make_tmap(&tv, &coord_v, vb, map_d, map_rows, Hkv, outer, map_st, cache.stride_h,
                       cache.stride_b, box_d, box_t / tpr, esz) ||
            !make_tmap(&tk_tail, &coord_v, kb, map_d, map_rows, Hkv, outer, map_st, cache.stride_h,
                       cache.stride_b, box_d, tail_rows / tpr, esz) ||
            !make_tmap(&tv_tail, &coord_v, vb, map_d, map_rows, Hkv, outer, map_st, cache.stride_h,
                       cache.stride_b, box_d, tail_rows / tpr, esz))
            return L4L_ERR_CUDA;
        DecodeParams p;
        p.q = static_cast<const __nv_bfloat16 *>(q) + (size_t)b0 * Hq * D;
        p.o = static_cast<__nv_bfloat16 *>(o) + (size_t)b0 * Hq * D;
        p.lse = d_lse ? d_lse + (size_t)b0 * Hq : nullptr;
        p.kv_lens = d_kv_lens + b0;
        p.part_o = part_o + (size_t)b0 * Hq * plan.nsplit * D;
        p.part_lse = part_lse + (size_t)b0 * Hq * plan.nsplit;
        p.tickets = tickets;                       // every launch leaves them at zero for the next
        p.status = reinterpret_cast<unsigned *>(ws);
        p.B = nb; p.Hq = Hq; p.Hkv = Hkv; p.G = G; p.min_tiles = plan.min_tiles; p.nsplit = plan.nsplit;
        p.max_kv_len = max_kv_len;
        p.stream_once = decode_streams_once(B, Hkv, D, max_kv_len, fp8 != nullptr) ? 1 : 0;
        p.nfin = nfin;
        p.k_new = p.v_new = nullptr;
        p.new_sb = p.new_sh = 0;
        p.rope_cos = rope ? rope->cos : nullptr;
        p.rope_sin = rope ? rope->sin : nullptr;
        p.q_weight = rope ? rope->q_weight : nullptr;
        p.k_weight = rope ? rope->k_weight : nullptr;
        p.norm_eps = rope ? rope->eps : 0.f;
        p.rope_n_pos = rope ? rope->n_pos : 0;
        p.k_scale = fp8 ? fp8->k_scale : nullptr;
        p.v_scale = fp8 ? fp8->v_scale : nullptr;
        p.block_table = paged ? paged->block_table + (size_t)b0 * paged->table_stride : nullptr;
        p.table_stride = paged ? paged->table_stride : 0;
        p.page_size = paged ? cache.max_len : 0;
        p.page_box = box_t;
        p.num_pages = paged ? paged->num_pages : 0;
        p.tail_rows = tail_rows;
        p.page_shift = 0;
        while (paged && (1 << p.page_shift) < cache.max_len) ++p.page_shift;
        // only the fused append writes through these: the slice's sequences, or the whole pool of a paged cache
        const size_t base_bytes = paged ? 0 : (size_t)b0 * cache.stride_b * esz;
        p.cache_k = reinterpret_cast<__nv_bfloat16 *>(static_cast<uint8_t *>(cache.k) + base_bytes);
        p.cache_v = reinterpret_cast<__nv_bfloat16 *>(static_cast<uint8_t *>(cache.v) + base_bytes);
        p.c_sb = cache.stride_b; p.c_sh = cache.stride_h; p.c_st = cache.stride_t;
        if (k_new && v_new) {
            if (k_new->stride_b != v_new->stride_b || k_new->stride_h != v_new->stride_h) return L4L_ERR_UNSUPPORTED;
            p.k_new = static_cast<const __nv_bfloat16 *>(k_new->ptr) + (size_t)b0 * k_new->stride_b;
            p.v_new = static_cast<const __nv_bfloat16 *>(v_new->ptr) + (size_t)b0 * v_new->stride_b;
            p.new_sb = k_new->stride_b; p.new_sh = k_new->stride_h;
        }
        p.scale_log2e = scale * 1.4426950408889634f;
        p.coord = coord;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(plan.grid);
        cfg.blockDim = dim3((plan.warps + 1 + nfin) * 32);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaError_t err;
        if (rope8 && big)
            err = plan.warps == 6 ? cudaLaunchKernelEx(&cfg, decode_split_kernel<128, 6, true, true, true>, tk, tv, tk_tail, tv_tail, p)
                                  : cudaLaunchKernelEx(&cfg, decode_split_kernel<128, 8, true, true, true>, tk, tv, tk_tail, tv_tail, p);
        else if (rope8 && D == 64)
            err = plan.warps == 8 ? cudaLaunchKernelEx(&cfg, decode_split_kernel<64, 8, true, false, true>, tk, tv, tk_tail, tv_tail, p)
                                  : cudaLaunchKernelEx(&cfg, decode_split_kernel<64, 4, true, false, true>, tk, tv, tk_tail, tv_tail, p);
        else if (rope8)
            err = plan.warps == 8 ? cudaLaunchKernelEx(&cfg, decode_split_kernel<128, 8, true, false, true>, tk, tv, tk_tail, tv_tail, p)
                                  : cudaLaunchKernelEx(&cfg, decode_split_kernel<128, 4, true, false, true>, tk, tv, tk_tail, tv_tail, p);
        else if (big && plan.warps == 6)
            err = fp8 ? cudaLaunchKernelEx(&cfg, decode_split_kernel<128, 6, true, true>, tk, tv, tk_tail, tv_tail, p)
                      : cudaLaunchKernelEx(&cfg, decode_split_kernel<128, 6, false, true>, tk, tv, tk_tail, tv_tail, p);
        else if (big)
            err = fp8 ? cudaLaunchKernelEx(&cfg, decode_split_kernel<128, 8, true, true>, tk, tv, tk_tail, tv_tail, p)
                      : cudaLaunchKernelEx(&cfg, decode_split_kernel<128, 8, false, true>, tk, tv, tk_tail, tv_tail, p);
        else if (fp8 && D == 64)
            err = plan.warps == 8 ? cudaLaunchKernelEx(&cfg, decode_split_kernel<64, 8, true, false>, tk, tv, tk_tail, tv_tail, p)
                                  : cudaLaunchKernelEx(&cfg, decode_split_kernel<64, 4, true, false>, tk, tv, tk_tail, tv_tail, p);
        else if (fp8)
            err = plan.warps == 8 ? cudaLaunchKernelEx(&cfg, decode_split_kernel<128, 8, true, false>, tk, tv, tk_tail, tv_tail, p)
                                  : cudaLaunchKernelEx(&cfg, decode_split_kernel<128, 4, true, false>, tk, tv, tk_tail, tv_tail, p);
        else if (D == 128)
            err = plan.warps == 8 ? cudaLaunchKernelEx(&cfg, decode_split_kernel<128, 8, false, false>, tk, tv, tk_tail, tv_tail, p)
                                  : cudaLaunchKernelEx(&cfg, decode_split_kernel<128, 4, false, false>, tk, tv, tk_tail, tv_tail, p);
        else
            err = plan.warps == 8 ? cudaLaunchKernelEx(&cfg, decode_split_kernel<64, 8, false, false>, tk, tv, tk_tail, tv_tail, p)
                                  : cudaLaunchKernelEx(&cfg, decode_split_kernel<64, 4, false, false>, tk, tv, tk_tail, tv_tail, p);
        if (err != cudaSuccess) return L4L_ERR_CUDA;
    }
    return L4L_OK;
}

}  // namespace l4l

// =================================================================================================
// Decode without a caller-provided workspace (and without any allocation).
//
// The scratch that l4l_attn_decode keeps in the caller's workspace (status block, ticket counters,
// fp32 partials) lives here in a fixed array inside the library's device image. Host code cannot use
// the array's name as a pointer: the name is only a handle on the host side, and a kernel handed it
// would fault or scribble over unrelated memory. The device address is looked up once per device with
// cudaGetSymbolAddress (that device being current) and passed to the very same launch path as the
// workspace variant.
namespace l4l {

namespace {

static __device__ __align__(256) unsigned char g_decode_static_scratch[L4L_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void *g_static_scratch_addr[kMaxDevices] = {nullptr};
std::mutex g_static_scratch_mutex;

}  // namespace

// Device address of the scratch array on the current device, or nullptr if the look-up fails.
void *static_scratch_on_current_device()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
    if (g_static_scratch_addr[dev] == nullptr) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_decode_static_scratch) != cudaSuccess || ptr == nullptr) {
            (void)cudaGetLastError();
            return nullptr;
        }
        g_static_scratch_addr[dev] = ptr;
    }
    return g_static_scratch_addr[dev];
}

}  // namespace l4l

extern "C" l4l_status l4l_attn_decode_static(const void *q, void *o, l4l_kv_cache cache, const int32_t *d_kv_lens,
                                             int max_kv_len, int B, int Hq, int Hkv, int head_dim, float scale,
                                             float *d_lse, l4l_stream stream)
{
    using namespace l4l;
    if (B < 0 || Hq <= 0 || Hkv <= 0) return L4L_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return L4L_ERR_UNSUPPORTED;
    if (Hq % Hkv != 0 || Hq / Hkv > 16) return L4L_ERR_UNSUPPORTED;
    auto aligned16 = [](const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };
    auto stride_ok = [](int64_t s) { return s >= 0 && (s % 8) == 0; };
    if (!q || !o || !d_kv_lens || !aligned16(q) || !aligned16(o)) return L4L_ERR_INVALID_ARG;
    if (!cache.k || !cache.v || !aligned16(cache.k) || !aligned16(cache.v) || !stride_ok(cache.stride_b) ||
        !stride_ok(cache.stride_h) || !stride_ok(cache.stride_t) || cache.max_len <= 0)
        return L4L_ERR_INVALID_ARG;
    if (max_kv_len < 0 || max_kv_len > cache.max_len) return L4L_ERR_INVALID_ARG;
    if (B == 0) return L4L_OK;

    // the split is chosen so that its partials fit the fixed array; if even the coarsest split does
    // not fit, the problem is beyond this entry point
    const DecodePlan plan = plan_decode(B, Hq, Hkv, head_dim, max_kv_len, (size_t)L4L_STATIC_SCRATCH_BYTES);
    if (plan.ws_bytes > (size_t)L4L_STATIC_SCRATCH_BYTES) return L4L_ERR_WORKSPACE;

    void *scratch = static_scratch_on_current_device();
    if (!scratch) return L4L_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the array keeps whatever the previous call left: the status block and the ticket counters must
    // start at zero (the partials need no clearing, every slot is written before it is read)
    const size_t zero_bytes = kStatusBytes + kTicketBytes;
    if (cudaMemsetAsync(scratch, 0, zero_bytes, s) != cudaSuccess) return L4L_ERR_CUDA;
    return launch_decode(q, o, cache, d_kv_lens, max_kv_len, B, Hq, Hkv, head_dim, scale, d_lse, scratch, plan, s,
                         nullptr, nullptr, nullptr, nullptr, nullptr);
}
