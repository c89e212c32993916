// Decode attention for MANY SHORT sequences: one warp owns a (sequence, KV head) from its first cached token to
// the output row, so there is nothing to merge and nothing to hand over. The split kernel pays a fixed cost per
// piece of a sequence (query rows, hand-over, finisher); with hundreds of sequences of a few hundred tokens
// that cost is paid every tile or two and the kernel falls to a third of the HBM rate.
//
// Persistent CTAs of 4 to 12 warps (the fewer units per SM, the fewer warps and the deeper their rings). The
// (sequence, KV head) units are laid end to end in 16-token chunks; a CTA
// takes the units that START inside its equal share of that stream (whole units only), puts them in order of
// descending length and hands them to its warps through a counter in shared memory, longest first, so that the
// warps of a CTA finish together. A warp moves its chunks from the cache into a private ring in
// shared memory with 16-byte asynchronous copies (cp.async: no barrier objects, no descriptors, rows past the
// end of a sequence arrive as zeros), in the 128-byte-swizzled layout that the warp-level MMA blocks expect, and
// stays S - 1 chunks ahead of its own arithmetic, across unit boundaries (the query rows of a unit travel with
// the unit's first chunk). Contiguous or paged caches, bf16 or fp8 (e4m3, per-KV-head scales); optional fused
// append of the step's newest token (bf16 caches).
#include <cstdlib>
#include <mutex>

#include "l4l_internal.h"
#include "l4l_ptx.cuh"
#include "l4l_rope_frag.cuh"
#include "l4l_warp_attn.cuh"

namespace l4l {

namespace {

constexpr int kMaxB = 1024;          // sequences per launch (lengths and prefix sums in shared memory)
constexpr int kMetaBytes = 11 * 1024; // lengths, prefix sums, unit order, queue: ahead of the rings
constexpr int kMaxList = 512;        // units of a CTA that can be put in order
constexpr int kFifo = 8;             // units the fetch side of a warp can be ahead of its compute side (power of two)
constexpr int kChunkT = 16;          // tokens per chunk = one MMA step of a warp

struct WarpParams {
    const __nv_bfloat16 *q;   // [B, Hq, D]
    __nv_bfloat16 *o;         // [B, Hq, D]
    float *lse;               // [B, Hq] or null
    const int32_t *kv_lens;   // [B]
    const __nv_bfloat16 *k_new, *v_new;   // fused append (null: none): element (b, kv head, d) at b*new_sb + kvh*new_sh + d
    int64_t new_sb, new_sh;
    __nv_bfloat16 *cache_k, *cache_v;
    int64_t c_sb, c_sh, c_st;
    const int32_t *block_table;           // paged cache (null: contiguous)
    int table_stride, page_size, page_shift, num_pages;
    const float *k_scale, *v_scale;       // fp8 cache: real value = e4m3 value * scale of its KV head, [Hkv]
    // rotary embedding (+ optional RMS norm) of the step's q and k_new inside the kernel (null: inputs are final); only
    // together with the fused append, bf16 caches. The new token's position is kv_len - 1.
    const float *rope_cos, *rope_sin;     // [rope_n_pos, D/2]
    const float *q_weight, *k_weight;     // [D] or null
    float norm_eps;
    int rope_n_pos;
    int B, Hq, Hkv, G, max_kv_len, stages;
    int stream_once;          // copy whole chunks with the L2 evict-first policy (large caches)
    float scale_log2e;
};

template <int D, bool F8>
struct WarpCfg {
    static constexpr int kRowBytes = F8 ? D : 2 * D;                  // one token of one KV head
    static constexpr int kHalves = kRowBytes / 128;                   // 128-byte column blocks of a row
    static constexpr uint32_t kHalfBytes = kChunkT * 128;             // [16 tokens][128 bytes], swizzled
    static constexpr uint32_t kTileBytes = kHalves * kHalfBytes;      // K or V of one chunk
    static constexpr int kRowPieces = kRowBytes / 16;                 // 16-byte pieces per row
    static constexpr int kCopies = kChunkT * kRowPieces / 32;         // cp.async per lane for K (and as many for V)
};

__host__ __device__ inline size_t stage_bytes(int D, int G, bool f8, bool rope)
{
    // K, V, the unit's query rows, and (rope fused into the step) the cos | sin rows of the unit's newest position
    return (size_t)2 * ((f8 ? D : 2 * D) / 128) * kChunkT * 128 + (size_t)G * D * 2 + (rope ? (size_t)D * 4 : 0);
}
// Beside the rings when the rope is fused in: every warp's copy of its unit's cos | sin rows (a unit's first stage is
// recycled long before its last chunk, which holds the new token), and the two norm weight rows.
__host__ __device__ inline size_t rope_extra_bytes(int D, int warps, bool rope) { return rope ? (size_t)(warps + 2) * D * 4 : 0; }

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void *src, uint32_t src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_16_full(uint32_t dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// The same for data that is read once (whole chunks of the cache): an L2 evict-first policy, so that the stream recycles
// its own lines instead of pushing out what an earlier kernel left in the L2.
__device__ __forceinline__ void cp_async_16_stream(uint32_t dst, const void *src, uint64_t policy)
{
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "l"(policy) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Position of a warp in its list of units.
struct Cursor {
    int b, kvh, len, chunks, chunk;   // current unit, its length and chunk count, next chunk of it
    bool valid;                       // false: the queue is empty
};

template <int D, int kWarps, bool F8>
__global__ void __launch_bounds__(kWarps * 32) decode_warp_kernel(const WarpParams p)
{
    static_assert(!F8 || D == 128, "the fp8 path wants one 128-byte row per token");
    using C = WarpCfg<D, F8>;
    constexpr int kEsz = F8 ? 1 : 2;
    constexpr int kThreads = kWarps * 32;
    extern __shared__ __align__(1024) uint8_t smem[];
    int *lens_s = reinterpret_cast<int *>(smem);                 // [kMaxB]
    int *cum_s = lens_s + kMaxB;                                 // [kMaxB + 1] chunks of the sequences before b
    int *warp_sums = cum_s + kMaxB + 1;                          // [kWarps] (16 at most)
    int *ctl = warp_sums + 16;                                   // first unit, end unit, queue position
    int *fifo_s = ctl + 4;                                       // [kWarps][kFifo]
    uint16_t *cnt_s = reinterpret_cast<uint16_t *>(fifo_s + 16 * kFifo);   // [kMaxList] chunks per unit of this CTA
    uint16_t *order_s = cnt_s + kMaxList;                        // [kMaxList] units by descending chunk count
    const bool fused_rope = !F8 && p.rope_cos != nullptr;
    const size_t sbytes = stage_bytes(D, p.G, F8, fused_rope);
    uint8_t *ring_base = smem + kMetaBytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *ring = ring_base + (size_t)warp * p.stages * sbytes;
    float *rope_priv = reinterpret_cast<float *>(ring_base + (size_t)kWarps * p.stages * sbytes) + (size_t)warp * D;   // cos | sin of this warp's unit
    float *norm_w = reinterpret_cast<float *>(ring_base + (size_t)kWarps * p.stages * sbytes) + (size_t)kWarps * D;   // q_weight | k_weight
    if (fused_rope) {
        for (int i = threadIdx.x; i < D; i += kThreads) {
            norm_w[i] = p.q_weight ? __ldg(p.q_weight + i) : 1.f;
            norm_w[D + i] = p.k_weight ? __ldg(p.k_weight + i) : 1.f;
        }
    }

    grid_dependency_wait();
    grid_launch_dependents();

    // ---- lengths and the prefix sum of chunk counts (a sequence without tokens still owns one chunk of the
    // stream, so that some warp writes its zero output)
    constexpr int kPer = (kMaxB + kThreads - 1) / kThreads;
    int mine[kPer], run = 0;
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        const int b = threadIdx.x * kPer + i;
        int len = 0, ch = 0;
        if (b < p.B) {
            len = __ldg(p.kv_lens + b);
            len = len < 0 ? 0 : (len > p.max_kv_len ? (p.k_new ? 0 : p.max_kv_len) : len);   // over the host's bound: decode ignores the extra tokens, a fused append treats the sequence as empty
            lens_s[b] = len;
            ch = len > 0 ? (len + kChunkT - 1) / kChunkT : 1;
        }
        mine[i] = run;
        run += ch;
    }
    int incl = run;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += v;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    int before = incl - run;
    for (int w = 0; w < warp; ++w) before += warp_sums[w];
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
        const int b = threadIdx.x * kPer + i;
        if (b <= p.B) cum_s[b] = before + mine[i];
    }
    if (kThreads * kPer == kMaxB && threadIdx.x == kThreads - 1 && p.B == kMaxB) cum_s[kMaxB] = before + run;
    __syncthreads();

    // ---- this CTA's units: those that start inside its equal share [lo, hi) of the chunk stream. Unit u is
    // (sequence u / Hkv, KV head u % Hkv); units are ordered by their start, and every unit has at least one chunk.
    const long long total = (long long)cum_s[p.B] * p.Hkv;
    auto first_unit_at = [&](long long pos) -> int {          // first unit that starts at or after pos
        if (pos >= total) return p.B * p.Hkv;
        int a = 0, z = p.B;                                   // smallest b with Hkv * cum[b + 1] > pos
        while (a < z) {
            const int mid = (a + z) >> 1;
            if ((long long)cum_s[mid + 1] * p.Hkv > pos) z = mid; else a = mid + 1;
        }
        const int cb = cum_s[a + 1] - cum_s[a];
        const long long base = (long long)cum_s[a] * p.Hkv;
        return a * p.Hkv + (int)((pos - base + cb - 1) / cb);  // KV head Hkv of sequence a = head 0 of a + 1
    };
    if (threadIdx.x < 2) {
        const long long pos = ((long long)blockIdx.x + threadIdx.x) * total / gridDim.x;
        ctl[threadIdx.x] = first_unit_at(pos);
    }
    if (threadIdx.x == 2) ctl[2] = kWarps;                    // queue position of the next unit to hand out
    __syncthreads();
    const int u_first = ctl[0], n_units = ctl[1] - ctl[0];

    // The units are handed to the warps longest first (every warp takes the next one when it has fetched its
    // current one to the end), which evens out the finishing times of the warps: order_s = the CTA's units by
    // descending chunk count (rank sort; a CTA has a few dozen units). Lists too long for the array keep their order.
    const bool sorted = n_units <= kMaxList;
    if (sorted) {
        for (int j = threadIdx.x; j < n_units; j += kThreads) {
            const int b = (u_first + j) / p.Hkv;
            cnt_s[j] = (uint16_t)min(cum_s[b + 1] - cum_s[b], 65535);
        }
        __syncthreads();
        for (int j = threadIdx.x; j < n_units; j += kThreads) {
            const int mine_c = cnt_s[j];
            int rank = 0;
            for (int k = 0; k < n_units; ++k) {
                const int c = cnt_s[k];
                rank += (c > mine_c || (c == mine_c && k < j)) ? 1 : 0;
            }
            order_s[rank] = (uint16_t)j;
        }
        __syncthreads();
    }
    int *fifo = fifo_s + warp * kFifo;            // queue positions that the fetch side took, for the compute side
    int fifo_wr = 0, fifo_rd = 0;
    auto load_unit = [&](Cursor &c, int pos) {    // the unit at queue position pos (pos >= n_units: none)
        c.chunk = 0;
        c.valid = pos < n_units;
        if (!c.valid) return;
        const int u = u_first + (sorted ? (int)order_s[pos] : pos);
        c.b = u / p.Hkv;
        c.kvh = u - c.b * p.Hkv;
        c.len = lens_s[c.b];
        c.chunks = cum_s[c.b + 1] - cum_s[c.b];
    };
    auto live = [&](const Cursor &c) { return c.valid; };
    auto advance_head = [&](Cursor &c) {          // next chunk, or the first chunk of the next unit in the queue
        if (++c.chunk < c.chunks) return;
        int pos = 0;
        if (lane == 0) pos = atomicAdd(&ctl[2], 1);
        pos = __shfl_sync(0xffffffffu, pos, 0);
        fifo[fifo_wr & (kFifo - 1)] = pos;        // all lanes, the same value
        ++fifo_wr;
        load_unit(c, pos);
    };
    auto advance_tail = [&](Cursor &c) {          // the fetch side is ahead: it has taken the next unit already
        if (++c.chunk < c.chunks) return;
        if (fifo_rd == fifo_wr) {
            c.valid = false;
            return;
        }
        load_unit(c, fifo[fifo_rd & (kFifo - 1)]);
        ++fifo_rd;
    };
    Cursor first;
    first.b = first.kvh = first.len = first.chunks = 0;
    load_unit(first, warp);

    // per-lane constants of the copies: piece i of a lane is row (32 i + lane) / kRowPieces, 16-byte piece
    // (32 i + lane) % kRowPieces of the row
    const int piece = lane % C::kRowPieces, row_of_lane = lane / C::kRowPieces;
    constexpr int kRowsPerTrip = 32 / C::kRowPieces;
    const uint32_t dst_half = (uint32_t)(piece >> 3) * C::kHalfBytes;

    uint32_t soff[C::kCopies];                     // where this lane's pieces land inside a K (or V) tile
#pragma unroll
    for (int i = 0; i < C::kCopies; ++i) soff[i] = dst_half + swz128(i * kRowsPerTrip + row_of_lane, piece & 7);

    // a large cache is read once per step: its lines go first; a small one stays L2-resident between steps
    const uint64_t stream_policy = p.stream_once ? l2_policy_evict_first() : l2_policy_evict_normal();
    auto issue = [&](const Cursor &c, int slot) {
        uint8_t *st = ring + (size_t)slot * sbytes;
        const uint32_t k_dst = smem_u32(st), v_dst = k_dst + C::kTileBytes;
        const int t0 = c.chunk * kChunkT;
        long long outer = c.b, slot_t = t0;
        bool have = true;
        if (p.block_table != nullptr) {
            outer = __ldg(p.block_table + (size_t)c.b * p.table_stride + (t0 >> p.page_shift));
            slot_t = t0 & (p.page_size - 1);
            have = outer >= 0 && outer < p.num_pages;     // a page outside the pool reads as zeros
            if (!have) outer = 0;
        }
        // byte addresses: an fp8 cache counts its strides in bytes, a bf16 cache in 2-byte elements
        const size_t base = ((size_t)outer * p.c_sb + (size_t)c.kvh * p.c_sh + (size_t)(slot_t + row_of_lane) * p.c_st) * kEsz +
                            piece * 16;
        const uint8_t *kbase = reinterpret_cast<const uint8_t *>(p.cache_k), *vbase = reinterpret_cast<const uint8_t *>(p.cache_v);
        const uint8_t *ks = kbase + base, *vs = vbase + base;
        const size_t step = (size_t)kRowsPerTrip * p.c_st * kEsz;
        const int nval = c.len - t0;               // rows of the chunk that hold tokens
        if (have && (nval > kChunkT || (nval == kChunkT && p.k_new == nullptr))) {
            // a full chunk of cached tokens (all but the last chunk of a unit): no predicates
#pragma unroll
            for (int i = 0; i < C::kCopies; ++i) {
                cp_async_16_stream(k_dst + soff[i], ks, stream_policy);
                cp_async_16_stream(v_dst + soff[i], vs, stream_policy);
                ks += step;
                vs += step;
            }
        } else {
            const int newest = (p.k_new != nullptr) ? nval - 1 : -1;        // row of the chunk that the caller brings
            const size_t new_off = (size_t)c.b * p.new_sb + (size_t)c.kvh * p.new_sh + piece * 8;
#pragma unroll
            for (int i = 0; i < C::kCopies; ++i) {
                const int row = i * kRowsPerTrip + row_of_lane;
                const bool valid = have && row < nval;
                if (row == newest) {
                    cp_async_16(k_dst + soff[i], p.k_new + new_off, 16u);
                    cp_async_16(v_dst + soff[i], p.v_new + new_off, 16u);
                } else {
                    cp_async_16(k_dst + soff[i], valid ? ks : kbase, valid ? 16u : 0u);
                    cp_async_16(v_dst + soff[i], valid ? vs : vbase, valid ? 16u : 0u);
                }
                ks += step;
                vs += step;
            }
        }
        if (c.chunk == 0) {                        // the unit's query rows: G x D bf16, unswizzled
            const uint32_t q_dst = v_dst + C::kTileBytes;
            const __nv_bfloat16 *qs = p.q + ((size_t)c.b * p.Hq + (size_t)c.kvh * p.G) * D;
            for (int i = lane; i < p.G * (D / 8); i += 32) cp_async_16_full(q_dst + i * 16, qs + i * 8);
            if (fused_rope && c.len >= 1 && c.len - 1 < p.rope_n_pos) {
                // cos | sin of the unit's newest position, behind the query rows: D/8 pieces of 16 bytes each
                const uint32_t r_dst = q_dst + (uint32_t)p.G * D * 2;
                const float *row = (lane < D / 8 ? p.rope_cos : p.rope_sin) + (size_t)(c.len - 1) * (D / 2);
                if (lane < D / 4) cp_async_16_full(r_dst + lane * 16, row + (lane % (D / 8)) * 4);
            }
        }
    };

    // ---- prologue: S - 1 chunks in flight
    Cursor head = first, tail = first;            // head: next chunk to fetch; tail: next chunk to compute
    const int S = p.stages;
    int head_slot = 0, tail_slot = 0;
    for (int i = 0; i < S - 1; ++i) {
        if (live(head)) {
            issue(head, head_slot);
            advance_head(head);
        }
        cp_async_commit();
        head_slot = head_slot + 1 == S ? 0 : head_slot + 1;
    }

    WarpAttnState<D> st;
    st.reset();
    uint32_t qf[D / 16][4];
    const int r_lo = lane >> 2, r_hi = r_lo + 8;
    float k_sc = 1.f, v_sc = 1.f;                  // fp8 cache: scales of the unit's KV head
    while (live(tail)) {
        if (live(head)) {
            issue(head, head_slot);
            advance_head(head);
        }
        cp_async_commit();
        head_slot = head_slot + 1 == S ? 0 : head_slot + 1;
        switch (S) {                               // all but the newest S - 1 groups have landed
        case 2: cp_async_wait<1>(); break;
        case 3: cp_async_wait<2>(); break;
        case 4: cp_async_wait<3>(); break;
        case 5: cp_async_wait<4>(); break;
        default: cp_async_wait<5>(); break;
        }
        __syncwarp();

        uint8_t *stg = ring + (size_t)tail_slot * sbytes;
        const uint32_t k_tile = smem_u32(stg), v_tile = k_tile + C::kTileBytes;
        if (tail.chunk == 0) {
            const uint32_t *qs = reinterpret_cast<const uint32_t *>(stg + 2 * C::kTileBytes);
            const uint32_t *qrow_lo = qs + (size_t)r_lo * D / 2;
            const uint32_t *qrow_hi = qs + (size_t)r_hi * D / 2;
            const bool v_lo = r_lo < p.G, v_hi = r_hi < p.G;
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                if constexpr (F8) {
                    // f16 fragments with the k index permuted the way the fp8 K rows arrive
                    const int w = q_frag_f8_word(ks, 0, lane);
                    qf[ks][0] = v_lo ? bf16x2_to_f16x2(qrow_lo[w]) : 0u;
                    qf[ks][1] = v_hi ? bf16x2_to_f16x2(qrow_hi[w]) : 0u;
                    qf[ks][2] = v_lo ? bf16x2_to_f16x2(qrow_lo[w + 1]) : 0u;
                    qf[ks][3] = v_hi ? bf16x2_to_f16x2(qrow_hi[w + 1]) : 0u;
                } else {
                    const int w = ks * 8 + (lane & 3);
                    qf[ks][0] = v_lo ? qrow_lo[w] : 0u;
                    qf[ks][1] = v_hi ? qrow_hi[w] : 0u;
                    qf[ks][2] = v_lo ? qrow_lo[w + 4] : 0u;
                    qf[ks][3] = v_hi ? qrow_hi[w + 4] : 0u;
                }
            }
            if constexpr (F8) {
                k_sc = __ldg(p.k_scale + tail.kvh);
                v_sc = __ldg(p.v_scale + tail.kvh);
            } else if (fused_rope && tail.len >= 1 && tail.len - 1 < p.rope_n_pos) {
                // keep the unit's cos | sin rows (its first stage is recycled before the chunk with the new token), then
                // rotate the q fragments in registers
                const float4 *src = reinterpret_cast<const float4 *>(stg + 2 * C::kTileBytes + (size_t)p.G * D * 2);
                __syncwarp();
                for (int i = lane; i < D / 4; i += 32) reinterpret_cast<float4 *>(rope_priv)[i] = src[i];
                __syncwarp();
                rope_q_fragments<D>(qf, p.G, p.q_weight != nullptr, p.norm_eps, rope_priv, norm_w, lane);
            }
        }
        const int t0 = tail.chunk * kChunkT;
        const int nvalid = tail.len - t0;
        if (nvalid > 0) {
            if (!F8 && p.k_new != nullptr && nvalid <= kChunkT) {
                // fused append: the newest token came from the caller; its cache slot is written from the copy in
                // shared memory (with pages: behind the block table; no page there: nothing is written)
                const int row = nvalid - 1;
                long long outer = tail.b, slot_t = tail.len - 1;
                if (p.block_table != nullptr) {
                    outer = __ldg(p.block_table + (size_t)tail.b * p.table_stride + (slot_t >> p.page_shift));
                    slot_t &= p.page_size - 1;
                }
                const bool have = p.block_table == nullptr || (outer >= 0 && outer < p.num_pages);
                const uint32_t off = lane < C::kRowPieces ? (uint32_t)(lane >> 3) * C::kHalfBytes + swz128(row, lane & 7) : 0u;
                if (fused_rope) {
                    // the k row arrived as the caller holds it: rotate (+ normalise) it where it sits (all lanes: shuffles)
                    uint4 kk = make_uint4(0u, 0u, 0u, 0u);
                    if (lane < C::kRowPieces) kk = *reinterpret_cast<const uint4 *>(stg + off);
                    kk = rope_k_row<D>(kk, p.k_weight != nullptr, p.norm_eps, rope_priv, norm_w + D, tail.len - 1 < p.rope_n_pos, lane);
                    if (lane < C::kRowPieces) *reinterpret_cast<uint4 *>(stg + off) = kk;
                }
                if (lane < C::kRowPieces) {
                    if (have) {
                        const size_t dst = (size_t)outer * p.c_sb + (size_t)tail.kvh * p.c_sh + (size_t)slot_t * p.c_st + lane * 8;
                        *reinterpret_cast<uint4 *>(p.cache_k + dst) = *reinterpret_cast<const uint4 *>(stg + off);
                        *reinterpret_cast<uint4 *>(p.cache_v + dst) = *reinterpret_cast<const uint4 *>(stg + C::kTileBytes + off);
                    } else {                       // as the cache would read: zeros
                        *reinterpret_cast<uint4 *>(stg + off) = make_uint4(0u, 0u, 0u, 0u);
                        *reinterpret_cast<uint4 *>(stg + C::kTileBytes + off) = make_uint4(0u, 0u, 0u, 0u);
                    }
                }
                __syncwarp();
            }
            float s_lo[4], s_hi[4];
            if constexpr (F8)
                warp_qk_16x16_f8<D>(qf, k_tile, 0, s_lo, s_hi);
            else
                warp_qk_16x16<D>(qf, k_tile, C::kHalfBytes, 0, s_lo, s_hi);
            const float sc = F8 ? p.scale_log2e * k_sc : p.scale_log2e;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                s_lo[e] *= sc;
                s_hi[e] *= sc;
            }
            if (nvalid < kChunkT) {                // tokens past the end: no weight (their V rows arrived as zeros)
                const int tok = 2 * (lane & 3);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (tok + (e & 1) >= nvalid) s_lo[e] = -INFINITY;
                    if (tok + (e & 1) + 8 >= nvalid) s_hi[e] = -INFINITY;
                }
            }
            uint32_t pa[4];
            warp_softmax_16<D, F8>(st, s_lo, s_hi, pa);        // fp8: weights as f16 for the f16 MMAs
            if constexpr (F8)
                warp_pv_16x16_f8<D>(st, pa, v_tile, 0);
            else
                warp_pv_16x16<D>(st, pa, v_tile, C::kHalfBytes, 0);
        }
        if (tail.chunk + 1 == tail.chunks) {
            // ---- the unit is complete: normalise and write its G output rows
            float l0 = st.l[0], l1 = st.l[1];
            l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
            l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
            l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
            l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
            const bool any = tail.len > 0;
            const float i0 = any ? 1.f / l0 : 0.f, i1 = any ? 1.f / l1 : 0.f;
            const size_t bh = (size_t)tail.b * p.Hq + (size_t)tail.kvh * p.G;
            // fp8: accumulator tiles alternate even / odd head dims (a tile pair gives this lane 4 consecutive dims) and O
            // still lacks the V scale of its KV head
            if (r_lo < p.G) {
                if constexpr (F8) {
                    __nv_bfloat16 *row = p.o + (bh + r_lo) * D + 4 * (lane & 3);
                    const float f = i0 * v_sc;
#pragma unroll
                    for (int ch = 0; ch < D / 16; ++ch)
                        *reinterpret_cast<uint2 *>(row + ch * 16) =
                            make_uint2(pack_bf16x2(st.o[2 * ch][0] * f, st.o[2 * ch + 1][0] * f),
                                       pack_bf16x2(st.o[2 * ch][1] * f, st.o[2 * ch + 1][1] * f));
                } else {
                    __nv_bfloat16 *row = p.o + (bh + r_lo) * D + 2 * (lane & 3);
#pragma unroll
                    for (int nt = 0; nt < D / 8; ++nt)
                        *reinterpret_cast<uint32_t *>(row + nt * 8) = pack_bf16x2(st.o[nt][0] * i0, st.o[nt][1] * i0);
                }
                if ((lane & 3) == 0 && p.lse)
                    p.lse[bh + r_lo] = any ? (st.m[0] + log2f(l0)) * 0.6931471805599453f : -INFINITY;
            }
            if (r_hi < p.G) {
                if constexpr (F8) {
                    __nv_bfloat16 *row = p.o + (bh + r_hi) * D + 4 * (lane & 3);
                    const float f = i1 * v_sc;
#pragma unroll
                    for (int ch = 0; ch < D / 16; ++ch)
                        *reinterpret_cast<uint2 *>(row + ch * 16) =
                            make_uint2(pack_bf16x2(st.o[2 * ch][2] * f, st.o[2 * ch + 1][2] * f),
                                       pack_bf16x2(st.o[2 * ch][3] * f, st.o[2 * ch + 1][3] * f));
                } else {
                    __nv_bfloat16 *row = p.o + (bh + r_hi) * D + 2 * (lane & 3);
#pragma unroll
                    for (int nt = 0; nt < D / 8; ++nt)
                        *reinterpret_cast<uint32_t *>(row + nt * 8) = pack_bf16x2(st.o[nt][2] * i1, st.o[nt][3] * i1);
                }
                if ((lane & 3) == 0 && p.lse)
                    p.lse[bh + r_hi] = any ? (st.m[1] + log2f(l1)) * 0.6931471805599453f : -INFINITY;
            }
            st.reset();
        }
        __syncwarp();                              // every lane is done with the slot before it is filled again
        tail_slot = tail_slot + 1 == S ? 0 : tail_slot + 1;
        advance_tail(tail);
    }
    cp_async_wait<0>();
}

size_t warp_smem_bytes(int D, int G, int warps, int stages, bool f8, bool rope)
{
    return kMetaBytes + (size_t)warps * stages * stage_bytes(D, G, f8, rope) + rope_extra_bytes(D, warps, rope);
}

template <int D, int W, bool F8>
int blocks_per_sm(size_t smem)
{
    struct Entry { size_t smem; int dev; int n; };
    static Entry cache[16];
    static int n_cached = 0;
    static std::mutex mutex;
    const int dev = device_slot();
    if (dev < 0) return 0;
    std::lock_guard<std::mutex> lock(mutex);
    for (int i = 0; i < n_cached; ++i)
        if (cache[i].smem == smem && cache[i].dev == dev) return cache[i].n;
    int n = 0;
    if (cudaFuncSetAttribute(decode_warp_kernel<D, W, F8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, decode_warp_kernel<D, W, F8>, W * 32, smem) != cudaSuccess) {
        (void)cudaGetLastError();
        n = 0;
    }
    if (n_cached < 16) cache[n_cached++] = {smem, dev, n};
    return n;
}

// Warps per CTA and ring depth. A CTA's shared memory holds a fixed number of chunks (24 at head_dim 128 with groups
// of up to 4 query heads); it is divided among as many warps as the CTA has units to work on at a time. With many
// units per SM the arithmetic of a warp (one dependent chain per chunk) is the bound and 12 warps with 2-chunk
// rings are fastest; with few units per SM a warp's chain of memory round trips is the bound and fewer warps with
// deeper rings (up to 6 chunks) are. head_dim 64 runs two CTAs per SM (of 8 warps at most: registers).
struct WarpShape { int warps, stages, ctas_per_sm; };
WarpShape pick_warp_shape(int D, int G, long long units, bool f8, bool rope = false)
{
    const int cps = D == 64 ? 2 : 1;
    const size_t budget = (D == 64 ? 113u : 227u) * 1024u - kMetaBytes - rope_extra_bytes(D, 12, rope);
    const int total = (int)(budget / stage_bytes(D, G, f8, rope));   // chunks of ring per CTA
    const long long ctas = (long long)sm_count() * cps;
    const long long per_cta = (units + ctas - 1) / ctas;
    const int wmax = (D == 128 && total >= 24) ? 12 : 8;
    int warps = 4;
    for (int w : {4, 6, 8, 12}) {
        if (w > wmax) break;
        warps = w;
        if (w >= per_cta) break;
    }
    const int stages = total / warps < 6 ? total / warps : 6;
    return {warps, stages >= 2 ? stages : 0, cps};
}

using WarpKernel = void (*)(const WarpParams);
struct KernelEntry { WarpKernel fn; int (*blocks)(size_t); };
template <int D, int W, bool F8>
KernelEntry entry() { return {decode_warp_kernel<D, W, F8>, &blocks_per_sm<D, W, F8>}; }
KernelEntry pick_kernel(int D, int warps, bool f8)
{
    if (f8)                                                       // head_dim 128 only
        return warps == 4 ? entry<128, 4, true>() : warps == 6 ? entry<128, 6, true>()
               : warps == 8 ? entry<128, 8, true>() : entry<128, 12, true>();
    if (D == 64) return warps == 4 ? entry<64, 4, false>() : warps == 6 ? entry<64, 6, false>() : entry<64, 8, false>();
    return warps == 4 ? entry<128, 4, false>() : warps == 6 ? entry<128, 6, false>()
           : warps == 8 ? entry<128, 8, false>() : entry<128, 12, false>();
}

}  // namespace

// Whether the warp-per-unit kernel should serve this decode call. The tuning override (l4l_set_decode_override) forces the answer (for
// tests); shapes it cannot run are refused either way.
bool decode_warp_eligible(int B, int Hq, int Hkv, int D, int max_kv_len, bool fp8, bool rope, bool append)
{
    const int G = Hq / Hkv;
    const long long units = (long long)B * Hkv;
    // fp8 caches: plain decode only (the fused append of an fp8 cache quantises the new token, which this kernel's
    // copy path cannot do on the way)
    if ((rope && (fp8 || !append)) || (fp8 && (append || D != 128)) || G > 16 ||
        pick_warp_shape(D, G, units, fp8, rope).stages == 0)
        return false;
    if (const int forced = decode_override().warp; forced >= 0) return forced != 0;
    // many units of a few chunks each: the regime where the split kernel pays its per-piece cost every tile or two.
    // Thresholds measured against the split kernel in CUDA graphs (8 KV heads at head_dim 128, 12 at head_dim 64),
    // in units per SM: with at most 256 tokens per sequence it wins from 3 units per SM (8 at head_dim 64), with
    // at most 512 from 10 (30).
    const long long sms = sm_count();
    if (max_kv_len <= 256) return units >= (D == 64 ? 8 : 3) * sms;
    if (max_kv_len <= 512) return units >= (D == 64 ? 30 : 10) * sms;
    return false;
}

l4l_status launch_decode_warp(const void *q, void *o, const l4l_kv_cache &cache, const int32_t *d_kv_lens,
                              int max_kv_len, int B, int Hq, int Hkv, int D, float scale, float *d_lse,
                              cudaStream_t stream, const l4l_tensor4 *k_new, const l4l_tensor4 *v_new,
                              const PagedTable *paged, const Fp8Scales *fp8, const RopeArgs *rope)
{
    const int G = Hq / Hkv;
    const bool f8 = fp8 != nullptr;
    if (G > 16 || (k_new == nullptr) != (v_new == nullptr) || (f8 && (k_new || D != 128))) return L4L_ERR_UNSUPPORTED;
    if (rope && (f8 || !k_new)) return L4L_ERR_UNSUPPORTED;
    for (int b0 = 0; b0 < B; b0 += kMaxB) {
        const int nb = B - b0 < kMaxB ? B - b0 : kMaxB;
        const long long units = (long long)nb * Hkv;
        const WarpShape shape = pick_warp_shape(D, G, units, f8, rope != nullptr);
        const int stages = shape.stages, kWarps = shape.warps;
        if (stages == 0) return L4L_ERR_UNSUPPORTED;
        const size_t smem = warp_smem_bytes(D, G, kWarps, stages, f8, rope != nullptr);
        const KernelEntry kernel = pick_kernel(D, kWarps, f8);
        const int per_sm = kernel.blocks(smem);
        if (per_sm == 0) return L4L_ERR_CUDA;
        WarpParams p = {};
        p.q = static_cast<const __nv_bfloat16 *>(q) + (size_t)b0 * Hq * D;
        p.o = static_cast<__nv_bfloat16 *>(o) + (size_t)b0 * Hq * D;
        p.lse = d_lse ? d_lse + (size_t)b0 * Hq : nullptr;
        p.kv_lens = d_kv_lens + b0;
        if (k_new) {
            p.k_new = static_cast<const __nv_bfloat16 *>(k_new->ptr) + (size_t)b0 * k_new->stride_b;
            p.v_new = static_cast<const __nv_bfloat16 *>(v_new->ptr) + (size_t)b0 * v_new->stride_b;
            if (k_new->stride_b != v_new->stride_b || k_new->stride_h != v_new->stride_h) return L4L_ERR_UNSUPPORTED;
            p.new_sb = k_new->stride_b;
            p.new_sh = k_new->stride_h;
        }
        // paged: the pool as a whole, whatever the slice; contiguous: this slice's sequences
        // (fp8: the strides count bytes)
        const size_t base_bytes = paged ? 0 : (size_t)b0 * cache.stride_b * (f8 ? 1 : 2);
        p.cache_k = reinterpret_cast<__nv_bfloat16 *>(static_cast<uint8_t *>(cache.k) + base_bytes);
        p.cache_v = reinterpret_cast<__nv_bfloat16 *>(static_cast<uint8_t *>(cache.v) + base_bytes);
        p.k_scale = f8 ? fp8->k_scale : nullptr;
        p.v_scale = f8 ? fp8->v_scale : nullptr;
        p.rope_cos = rope ? rope->cos : nullptr;
        p.rope_sin = rope ? rope->sin : nullptr;
        p.q_weight = rope ? rope->q_weight : nullptr;
        p.k_weight = rope ? rope->k_weight : nullptr;
        p.norm_eps = rope ? rope->eps : 0.f;
        p.rope_n_pos = rope ? rope->n_pos : 0;
        p.c_sb = cache.stride_b; p.c_sh = cache.stride_h; p.c_st = cache.stride_t;
        p.block_table = paged ? paged->block_table + (size_t)b0 * paged->table_stride : nullptr;
        p.table_stride = paged ? paged->table_stride : 0;
        p.page_size = paged ? cache.max_len : 0;
        p.num_pages = paged ? paged->num_pages : 0;
        p.page_shift = 0;
        while (paged && (1 << p.page_shift) < cache.max_len) ++p.page_shift;
        p.B = nb; p.Hq = Hq; p.Hkv = Hkv; p.G = G; p.max_kv_len = max_kv_len; p.stages = stages;
        p.stream_once = decode_streams_once(B, Hkv, D, max_kv_len, fp8 != nullptr) ? 1 : 0;
        p.scale_log2e = scale * 1.4426950408889634f;

        // persistent: every resident CTA gets its share of the stream; never more CTAs than units
        long long blocks = (long long)per_sm * sm_count();
        if (blocks > units) blocks = units;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)blocks, 1, 1);
        cfg.blockDim = dim3(kWarps * 32, 1, 1);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        const cudaError_t err = cudaLaunchKernelEx(&cfg, kernel.fn, p);
        if (err != cudaSuccess) {
            (void)cudaGetLastError();
            return L4L_ERR_CUDA;
        }
    }
    return L4L_OK;
}

}  // namespace l4l
