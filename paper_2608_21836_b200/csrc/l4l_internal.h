// Host-side declarations shared by the translation units of libl4l (not part of the ABI).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <mutex>
#include <stddef.h>
#include <stdint.h>

#include "../../include/l4l.h"

namespace l4l {

// One-time set-up of a kernel (the shared-memory opt-in, occupancy look-ups) holds for one device only, so the
// "already done" flags are kept per device ordinal. Slot of the current device, or -1 if it cannot be had.
constexpr int kDeviceSlots = 64;
inline int device_slot()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kDeviceSlots) return -1;
    return dev;
}

// One mutex for every "first call on this device" set-up (shared-memory opt-ins, occupancy look-ups): those
// flags are read and written from whichever host thread launches first.
std::mutex &setup_mutex();

// Tuning overrides of the decode kernel choice (tests and benchmarks use them to hold a call on one kernel).
// Seeded once, when the library is loaded, from L4L_DECODE_CLUSTER / L4L_DECODE_WARP / L4L_DECODE_WARPS, and
// changed afterwards only through l4l_set_decode_override: no decode call reads the environment.
struct DecodeOverride {
    int cluster;       // -1: library's choice, 0: never the cluster kernel, N > 0: clusters of N where they fit
    int warp;          // -1: library's choice, 0: never the warp-per-unit kernel, 1: always where it can run
    int split_warps;   // 0: library's choice, 4 or 8: consumer warps of the split kernel
};
DecodeOverride decode_override();

// Where each logical coordinate (token, head, batch) sits among coordinates 1..3 of a 4-D
// tensor map whose coordinate 0 is head_dim. Dimensions are ordered by ascending stride.
struct TmapCoord {
    int pos_t, pos_h, pos_b;
};

// Builds a tiled tensor map over a [batch, head, token, D]-indexable buffer of bf16 (elem_bytes = 2) or
// single bytes (elem_bytes = 1) with the given element strides; the box is box_d x box_t (x1x1) with the
// 128-byte swizzle (box_d * elem_bytes must be 128). Returns false (and leaves *out undefined) if the
// driver refuses.
bool make_tmap(CUtensorMap *out, TmapCoord *coord, const void *base, int D, int64_t n_t, int64_t n_h, int64_t n_b,
               int64_t stride_t, int64_t stride_h, int64_t stride_b, int box_d, int box_t, int elem_bytes);
inline bool make_tmap_bf16(CUtensorMap *out, TmapCoord *coord, const void *base, int D, int64_t n_t, int64_t n_h,
                           int64_t n_b, int64_t stride_t, int64_t stride_h, int64_t stride_b, int box_d, int box_t)
{
    return make_tmap(out, coord, base, D, n_t, n_h, n_b, stride_t, stride_h, stride_b, box_d, box_t, 2);
}

// Tiled bf16 tensor map without swizzle over a dense [outer, rows, cols] array (cols contiguous): box =
// box_cols x box_rows x 1. Coordinates are (col, row, outer).
bool make_tmap_rows_bf16(CUtensorMap *out, const void *base, int64_t n_cols, int64_t n_rows, int64_t n_outer,
                         int64_t stride_row, int64_t stride_outer, int box_cols, int box_rows);

int sm_count();

// Whether a decode launch should load its K/V with the L2 evict-first policy: yes when the cache it may stream is large
// against the L2 (it is read once per step and would otherwise push out what earlier kernels left there, dirty lines
// included); no for small caches, which stay L2-resident from one step to the next and are better off without the hint.
inline bool decode_streams_once(int B, int Hkv, int D, int max_kv_len, bool fp8)
{
    return (size_t)B * Hkv * (size_t)max_kv_len * D * (fp8 ? 1 : 2) * 2 >= ((size_t)64 << 20);
}

struct DecodePlan {
    int warps;       // kernel shape: 4, 6 or 8 consumer warps (tile = 16 tokens per warp)
    bool fits;       // the shape's shared memory fits an SM
    int grid;        // persistent CTAs
    int min_tiles;   // floor on the 64-token tiles per CTA (bounds the pieces per sequence)
    int nsplit;      // max pieces a (sequence, KV head) can be cut into
    size_t ws_bytes; // status block + ticket counters + partials
};
// page_size: 0 for a contiguous cache, else the tokens per page of a paged cache (kept for shapes whose tiles must
// line up with pages; none does at present)
DecodePlan plan_decode(int B, int Hq, int Hkv, int D, int max_kv_len, size_t ws_limit, bool fp8 = false,
                       int page_size = 0);

// Block table of a paged cache: token t of sequence b is in page block_table[b * table_stride + t / page_size].
struct PagedTable {
    const int32_t *block_table;   // device
    int table_stride;             // entries per sequence
    int num_pages;                // pages in the pool
};

// Scales of an fp8 (e4m3) cache: real value = stored value * scale of its KV head.
struct Fp8Scales {
    const float *k_scale, *v_scale;   // device, [Hkv]
};

// Rotary embedding (+ optional RMS norm) of the step's q and k_new inside the decode kernel.
struct RopeArgs {
    const float *cos, *sin;           // device, [n_pos, D/2]
    const float *q_weight, *k_weight; // device [D] or null
    float eps;
    int n_pos;
};

// With `paged`, `cache` describes the page pool: stride_b = stride between pages, max_len = page size.
// With `fp8`, cache.k / cache.v hold e4m3 bytes and the strides count bytes.
l4l_status launch_decode(const void *q, void *o, const l4l_kv_cache &cache, const int32_t *d_kv_lens,
                         int max_kv_len, int B, int Hq, int Hkv, int D, float scale, float *d_lse,
                         void *workspace, const DecodePlan &plan, cudaStream_t stream,
                         const l4l_tensor4 *k_new = nullptr, const l4l_tensor4 *v_new = nullptr,
                         const PagedTable *paged = nullptr, const Fp8Scales *fp8 = nullptr,
                         const RopeArgs *rope = nullptr);

// Small batches: one thread-block cluster per (sequence, KV head), partials merged through distributed shared
// memory. decode_cluster_width returns the cluster size to use, or 0 if the split kernel should run.
int decode_cluster_width(int B, int Hq, int Hkv, int D, int max_kv_len, bool fp8);
l4l_status launch_decode_cluster(const void *q, void *o, const l4l_kv_cache &cache, const int32_t *d_kv_lens,
                                 int max_kv_len, int B, int Hq, int Hkv, int D, float scale, float *d_lse,
                                 void *workspace, cudaStream_t stream, const l4l_tensor4 *k_new,
                                 const l4l_tensor4 *v_new, const PagedTable *paged, const RopeArgs *rope,
                                 const Fp8Scales *fp8, int width);

// Many short sequences: one warp per (sequence, KV head), no merge (bf16 caches with or without the fused append and
// the rotary fusion, fp8 caches without them, groups of up to 16 query heads). decode_warp_eligible says whether launch_decode should hand the call over.
bool decode_warp_eligible(int B, int Hq, int Hkv, int D, int max_kv_len, bool fp8, bool rope, bool append);
l4l_status launch_decode_warp(const void *q, void *o, const l4l_kv_cache &cache, const int32_t *d_kv_lens,
                              int max_kv_len, int B, int Hq, int Hkv, int D, float scale, float *d_lse,
                              cudaStream_t stream, const l4l_tensor4 *k_new, const l4l_tensor4 *v_new,
                              const PagedTable *paged, const Fp8Scales *fp8, const RopeArgs *rope);

l4l_status launch_rope_kv_append(const l4l_tensor4 &q, const l4l_tensor4 &k_new, const l4l_tensor4 &v_new,
                                 const l4l_kv_cache &cache, const int32_t *d_pos, const int32_t *d_n_new, int T, int B,
                                 int Hq, int Hkv, int D, const float *d_cos, const float *d_sin, int n_pos,
                                 const float *d_q_weight, const float *d_k_weight, float norm_eps, cudaStream_t stream);
l4l_status launch_kv_append(const l4l_kv_cache &cache, const l4l_tensor4 &k_new, const l4l_tensor4 &v_new,
                            const int32_t *d_write_pos, const int32_t *d_n_new, int n_new_max, int B, int Hkv,
                            int D, cudaStream_t stream, const PagedTable *paged = nullptr);

l4l_status launch_kv_append_fp8(const l4l_kv_cache &cache, const l4l_tensor4 &k_new, const l4l_tensor4 &v_new,
                                const int32_t *d_write_pos, const int32_t *d_n_new, int n_new_max, int B, int Hkv,
                                int D, const float *d_k_scale, const float *d_v_scale, cudaStream_t stream);

l4l_status launch_attn_merge(const void *o_parts, const float *lse_parts, int R, void *o, float *d_lse, int B, int Hq,
                             int D, cudaStream_t stream);

l4l_status launch_rglru_scan(const void *x, const void *gate_x, const void *gate_a, const float *d_a_param,
                             const int32_t *d_position, const int32_t *d_seq_lens, float *d_state, void *y, int B, int T,
                             int W, void *workspace, size_t ws_bytes, cudaStream_t stream);
size_t rglru_workspace_bytes(int B, int T, int W);
// the scan's shape for these sizes on the current device: 0 = 64-channel strips, teams of 16 warps; 1, 2, 4 = teams of
// 8 warps on strips of 64, 32, 16 channels
int rglru_strip_split(int B, int T, int W);

// Where one prefill launch takes its keys and values from, and where it puts them.
struct PrefillKV {
    l4l_tensor4 k_new, v_new;     // K/V of the new tokens (a prompt, or a chunk) as [B, T, Hkv, D] views ...
    int new_extent;               // ... with this many token rows
    bool new_at_past;             // those views are the cache itself: row r of sequence b is slot past[b] + r
    const l4l_kv_cache *past;     // the tokens cached before are read from here (a contiguous cache, or with `paged`
                                  // the page pool: stride_b = stride between pages, max_len = page size); null: none
    const PagedTable *paged;      // block table of a paged cache; null: contiguous
    const l4l_kv_cache *write;    // the new tokens' K/V are written here in the same pass; null: nothing is written
};

// tcgen05 / tensor-memory prefill kernel: a fresh prompt (no past), or a chunk of new tokens over a populated
// cache. d_past_lens (may be null): tokens ahead of the chunk, per sequence.
l4l_status launch_prefill_tc(const l4l_tensor4 &q, const l4l_tensor4 &o, const PrefillKV &kv, const int32_t *d_seq_lens,
                             const int32_t *d_past_lens, int S_max, int B, int Hq, int Hkv, int D, float scale,
                             float *d_lse, void *workspace, cudaStream_t stream);

}  // namespace l4l
