/*
 * l4l.h — C ABI of the B200 (sm_100a) causal-attention hot path.
 *
 * The operations are the ones the paper's appendix on accepted kernels ("Transformer
 * attention", Table A.4) names as the attention module's two phases plus the cache
 * update that surrounds them:
 *
 *   l4l_attn_prefill   q_len > 1 : causal grouped-query attention over the prompt; the KV
 *                                  head of a query head follows from the grouped-query
 *                                  structure, the causal mask is part of the score update,
 *                                  softmax statistics are kept in fp32; the prompt's K and V
 *                                  are written to the cache in the same pass.
 *   l4l_attn_decode    q_len = 1 : one query token per sequence over a populated, ragged KV
 *                                  cache; all query heads of a KV group are served by one
 *                                  pass over that group's cache.
 *   l4l_kv_append                : the cache update (an exact copy).
 *
 * Further entry points widen that path, each documented at its declaration:
 *   l4l_attn_prefill_chunk (new tokens over a populated cache; _append / _paged_append with the cache
 *   update fused in, over a contiguous or a paged cache), l4l_attn_decode_append (cache
 *   update fused into the decode step), l4l_rope_kv_append (rotary embedding and QK-norm fused
 *   with the cache update), l4l_attn_decode_paged / l4l_kv_append_paged / l4l_attn_decode_paged_append
 *   (page pool + block table), l4l_attn_decode_fp8 / l4l_kv_append_fp8 / l4l_attn_decode_append_fp8 /
 *   l4l_attn_decode_rope_append_fp8 (e4m3 cache), l4l_attn_decode_static (no caller workspace), and a second workload,
 *   l4l_rglru_scan (gated linear recurrence).
 *
 * Conventions shared by every call
 *   - All tensors are bf16 (16-bit words) in DEVICE memory unless a parameter says "host".
 *     head_dim (D) is the contiguous innermost dimension; the other strides are passed in
 *     ELEMENTS. Every base pointer must be 16-byte aligned and every stride a multiple of 8
 *     elements (16 bytes), because tiles move with TMA.
 *   - Query head h reads KV head h / (Hq / Hkv): consecutive query heads share a KV head.
 *   - The caller owns every buffer. The library allocates no device memory, enqueues its
 *     kernels on the caller's stream and never synchronises (l4l_last_device_error excepted).
 *     Sequence lengths live in device memory; only upper bounds come from the host.
 *   - Every call works on the device that is current in the calling thread (all its pointers
 *     belong to that device); the one-time set-up of each kernel is kept per device, so one
 *     process may drive several GPUs, one at a time per call.
 *   - Errors: arguments are validated on the host BEFORE anything is launched; a non-zero
 *     status means no kernel of that call ran. Nothing throws, nothing traps on the device.
 *     Unsupported shapes return L4L_ERR_UNSUPPORTED; there is no fallback path.
 *       supported: head_dim in {64, 128}; Hq % Hkv == 0; Hq / Hkv <= 16.
 *   - Device-side waits (TMA / tensor-core pipeline barriers) are bounded. If one ever runs
 *     out, the kernel records a code in the workspace's status block and returns; the host
 *     sees it through l4l_last_device_error().
 */
#ifndef L4L_H
#define L4L_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    L4L_OK = 0,
    L4L_ERR_INVALID_ARG = 1, /* null pointer, negative size, misaligned pointer or stride      */
    L4L_ERR_UNSUPPORTED = 2, /* head_dim / head grouping outside the supported set             */
    L4L_ERR_WORKSPACE = 3,   /* workspace missing or too small                                  */
    L4L_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed (launch, tensor-map encode) */
    L4L_ERR_TIMEOUT = 5      /* a bounded device-side wait ran out (returned by l4l_check_status) */
} l4l_status;

/* A cudaStream_t, passed as an opaque pointer (NULL = the legacy default stream). */
typedef void *l4l_stream;

/* bf16 [B, T, H, D] view: element (b, t, h, d) is at ptr + b*stride_b + t*stride_t + h*stride_h + d. */
typedef struct {
    void *ptr;
    int64_t stride_b, stride_t, stride_h;
} l4l_tensor4;

/* bf16 KV cache: element (b, kv_head, slot, d) of K is at k + b*stride_b + kv_head*stride_h +
 * slot*stride_t + d (V likewise). The default dense layout is [B, Hkv, max_len, D]; any
 * layout expressible by these strides (e.g. [B, max_len, Hkv, D]) is accepted. Not paged.
 * max_len = number of token slots per sequence. */
typedef struct {
    void *k;
    void *v;
    int64_t stride_b, stride_h, stride_t;
    int32_t max_len;
} l4l_kv_cache;

/*
 * A paged KV cache: a pool of fixed-size pages, element (page, kv head g, slot t, d) at
 * k + page*stride_page + g*stride_h + t*stride_t + d. A per-sequence block table (device int32,
 * [B, table_stride]) names the page that holds tokens [i*page_size, (i+1)*page_size) of a
 * sequence in entry i. page_size must be a power of two >= 16. The dense layout is
 * [num_pages, Hkv, page_size, D].
 */
typedef struct {
    void *k;
    void *v;
    int64_t stride_page, stride_h, stride_t;
    int32_t page_size;
    int32_t num_pages;
} l4l_paged_kv;

enum { L4L_OP_PREFILL = 0, L4L_OP_DECODE = 1 };

/*
 * Bytes of device workspace the given operation needs for these sizes (max_len = the largest
 * S_max / max_kv_len it will be called with). Always >= 256: the first 256 bytes are the
 * status block. Returns 0 for unsupported arguments.
 */
size_t l4l_workspace_bytes(int op, int B, int Hq, int Hkv, int head_dim, int max_len);

/*
 * Zero the workspace (status block and the decode ticket counters; enqueued on `stream`).
 * Call once after allocating a workspace and again after a reported device error. The
 * kernels leave the counters at zero, so no re-initialisation is needed between calls. A
 * workspace serves one call at a time: calls that may overlap on the device need their own.
 */
l4l_status l4l_workspace_init(void *workspace, size_t ws_bytes, l4l_stream stream);

/*
 * Cache update: for every sequence b, copy n_new[b] tokens of k_new / v_new ([B, T, Hkv, D],
 * T = n_new_max) into cache slots write_pos[b] .. write_pos[b] + n_new[b] - 1, bit for bit.
 * (In the paper the cache update is the module code around the two kernels; it must happen
 * exactly once per token.) Every other cache slot is left untouched. Writes that would fall
 * outside [0, max_len) are dropped on the device, never performed.
 *   d_write_pos  device int32 [B]
 *   d_n_new      device int32 [B], or NULL meaning n_new[b] = n_new_max for all b
 */
l4l_status l4l_kv_append(l4l_kv_cache cache, l4l_tensor4 k_new, l4l_tensor4 v_new,
                         const int32_t *d_write_pos, const int32_t *d_n_new, int n_new_max,
                         int B, int Hkv, int head_dim, l4l_stream stream);

/*
 * The same two operations over a paged cache (what serving runtimes hold: the paper's related-work
 * discussion of KV-cache management; the paper's own kernels read a contiguous cache, so this
 * layout has no counterpart there). Results are those of l4l_kv_append / l4l_attn_decode on the
 * contiguous cache one gets by laying every sequence's pages end to end.
 *   l4l_kv_append_paged : token slot s of sequence b goes to page block_table[b][s / page_size],
 *                         offset s % page_size; slots beyond table_stride * page_size and slots
 *                         whose table entry is outside [0, num_pages) are dropped.
 *   l4l_attn_decode_paged : kv_lens[b] <= table_stride * page_size; a table entry outside
 *                         [0, num_pages) reads as zeros (never as memory); entries past the last
 *                         token of a sequence are not looked at. Workspace as for l4l_attn_decode
 *                         with max_len = max_kv_len.
 */
l4l_status l4l_kv_append_paged(l4l_paged_kv pool, const int32_t *d_block_table, int table_stride,
                               l4l_tensor4 k_new, l4l_tensor4 v_new, const int32_t *d_write_pos,
                               const int32_t *d_n_new, int n_new_max, int B, int Hkv, int head_dim,
                               l4l_stream stream);
l4l_status l4l_attn_decode_paged(const void *q, void *o, l4l_paged_kv pool, const int32_t *d_block_table,
                                 int table_stride, const int32_t *d_kv_lens, int max_kv_len,
                                 int B, int Hq, int Hkv, int head_dim, float scale, float *d_lse,
                                 void *workspace, size_t ws_bytes, l4l_stream stream);
/*
 * l4l_attn_decode_append over a paged cache: the step's newest token (k_new / v_new, [B, 1, Hkv, D]) goes to
 * slot kv_lens[b] - 1 of sequence b, i.e. to page block_table[b][(kv_lens[b]-1) / page_size], bit for bit, and
 * is attended with the rest in the same launch. Equivalent to l4l_kv_append_paged at that slot followed by
 * l4l_attn_decode_paged; a sequence whose table has no valid page for the slot gets no write (as in
 * l4l_kv_append_paged) and attends over zeros there. Sequences with kv_lens[b] = 0 append nothing.
 */
l4l_status l4l_attn_decode_paged_append(const void *q, void *o, l4l_paged_kv pool, const int32_t *d_block_table,
                                        int table_stride, l4l_tensor4 k_new, l4l_tensor4 v_new,
                                        const int32_t *d_kv_lens, int max_kv_len, int B, int Hq, int Hkv,
                                        int head_dim, float scale, float *d_lse, void *workspace, size_t ws_bytes,
                                        l4l_stream stream);

/*
 * The same two operations over an fp8 cache (e4m3: 1 sign, 4 exponent, 3 mantissa bits, largest
 * finite value 448, no infinities), which halves the bytes decode has to stream. The paper's
 * kernels read a bf16 cache; this layout has no counterpart there. `cache8` uses the l4l_kv_cache
 * struct with k / v pointing at bytes and strides counted in bytes (multiples of 16); a stored
 * byte c of KV head g stands for the real value e4m3(c) * scale[g].
 *   l4l_kv_append_fp8  : stores RN_e4m3( fp32(x) / k_scale[g] ) (IEEE fp32 division, then round to
 *                        nearest even, saturating at +-448; NaN stays NaN); other rules as l4l_kv_append.
 *   l4l_attn_decode_fp8: l4l_attn_decode over the values the bytes stand for (the widening to f16 in
 *                        the kernel is exact; q and the softmax weights are used as f16). At head_dim 64 (this
 *                        entry point and the other fp8 decode calls) two tokens share a 128-byte tile row, so the
 *                        token rows of the cache (of each page) must lie back to back (stride_t = 64) and the
 *                        number of slots must be even, else L4L_ERR_UNSUPPORTED.
 *   d_k_scale, d_v_scale   device float [Hkv], > 0
 */
l4l_status l4l_kv_append_fp8(l4l_kv_cache cache8, l4l_tensor4 k_new, l4l_tensor4 v_new,
                             const int32_t *d_write_pos, const int32_t *d_n_new, int n_new_max,
                             int B, int Hkv, int head_dim, const float *d_k_scale, const float *d_v_scale,
                             l4l_stream stream);
l4l_status l4l_attn_decode_fp8(const void *q, void *o, l4l_kv_cache cache8, const float *d_k_scale,
                               const float *d_v_scale, const int32_t *d_kv_lens, int max_kv_len,
                               int B, int Hq, int Hkv, int head_dim, float scale, float *d_lse,
                               void *workspace, size_t ws_bytes, l4l_stream stream);
/* Both at once: an fp8 page pool (l4l_paged_kv with k / v pointing at bytes, strides in bytes, multiples
 * of 16) read through a block table. Rules of l4l_attn_decode_paged and l4l_attn_decode_fp8 combined. */
l4l_status l4l_attn_decode_paged_fp8(const void *q, void *o, l4l_paged_kv pool8, const float *d_k_scale,
                                     const float *d_v_scale, const int32_t *d_block_table, int table_stride,
                                     const int32_t *d_kv_lens, int max_kv_len, int B, int Hq, int Hkv,
                                     int head_dim, float scale, float *d_lse, void *workspace,
                                     size_t ws_bytes, l4l_stream stream);
/* l4l_attn_decode_append over an fp8 cache: the step's newest token (bf16 k_new / v_new, [B, 1, Hkv, D]) is
 * quantised with the arithmetic of l4l_kv_append_fp8 (the stored codes are the same, bit for bit), written to
 * slot kv_lens[b] - 1 and attended with the rest in the same launch. Contiguous cache, or page pool + block
 * table (rules of l4l_attn_decode_paged_append). */
l4l_status l4l_attn_decode_append_fp8(const void *q, void *o, l4l_kv_cache cache8, const float *d_k_scale,
                                      const float *d_v_scale, l4l_tensor4 k_new, l4l_tensor4 v_new,
                                      const int32_t *d_kv_lens, int max_kv_len, int B, int Hq, int Hkv,
                                      int head_dim, float scale, float *d_lse, void *workspace, size_t ws_bytes,
                                      l4l_stream stream);
l4l_status l4l_attn_decode_paged_append_fp8(const void *q, void *o, l4l_paged_kv pool8, const float *d_k_scale,
                                            const float *d_v_scale, const int32_t *d_block_table, int table_stride,
                                            l4l_tensor4 k_new, l4l_tensor4 v_new, const int32_t *d_kv_lens,
                                            int max_kv_len, int B, int Hq, int Hkv, int head_dim, float scale,
                                            float *d_lse, void *workspace, size_t ws_bytes, l4l_stream stream);

/*
 * The whole decode step of one attention layer in ONE launch: rotary embedding (and optional per-head RMS
 * normalisation) of the step's q and k, the cache update, and the attention. For sequence b the new token
 * sits at position kv_lens[b] - 1: q[b] and k_new[b] (projection outputs) go through the arithmetic of
 * l4l_rope_kv_append at that position, the rotated k and v_new are written to cache slot kv_lens[b] - 1, and
 * the rotated q attends over slots 0 .. kv_lens[b] - 1. Same result as l4l_rope_kv_append (T = 1) followed by
 * l4l_attn_decode, up to the last bf16 bit of the rotated values (the sum of squares of the norm is reduced
 * in a different order). q is NOT modified (the rotated values live on chip only). A position outside
 * [0, n_pos) leaves q and k unrotated.
 *   arguments as for l4l_attn_decode_append and l4l_rope_kv_append
 */
l4l_status l4l_attn_decode_rope_append(const void *q, void *o, l4l_kv_cache cache, l4l_tensor4 k_new, l4l_tensor4 v_new,
                                       const int32_t *d_kv_lens, int max_kv_len, int B, int Hq, int Hkv,
                                       int head_dim, float scale, const float *d_cos, const float *d_sin, int n_pos,
                                       const float *d_q_weight, const float *d_k_weight, float norm_eps,
                                       float *d_lse, void *workspace, size_t ws_bytes, l4l_stream stream);
/* The same step over a paged cache (l4l_attn_decode_paged_append with the rotation and normalisation of
 * l4l_attn_decode_rope_append): the rotated k and v_new go to the page slot of position kv_lens[b] - 1. */
l4l_status l4l_attn_decode_paged_rope_append(const void *q, void *o, l4l_paged_kv pool, const int32_t *d_block_table,
                                             int table_stride, l4l_tensor4 k_new, l4l_tensor4 v_new,
                                             const int32_t *d_kv_lens, int max_kv_len, int B, int Hq, int Hkv,
                                             int head_dim, float scale, const float *d_cos, const float *d_sin, int n_pos,
                                             const float *d_q_weight, const float *d_k_weight, float norm_eps,
                                             float *d_lse, void *workspace, size_t ws_bytes, l4l_stream stream);
/* The same step over an e4m3 cache (contiguous, or a page pool behind a block table): k_new is rotated (and
 * normalised) as above, rounded to bf16, and then quantised with the arithmetic of l4l_kv_append_fp8, so the stored
 * codes are those of l4l_rope_kv_append followed by l4l_kv_append_fp8 (up to the last bf16 bit of the rotated values
 * when the norm is on, as above); v_new is quantised as it is. Rules of l4l_attn_decode_append_fp8 /
 * l4l_attn_decode_paged_append_fp8 for the cache, of l4l_attn_decode_rope_append for the tables. */
l4l_status l4l_attn_decode_rope_append_fp8(const void *q, void *o, l4l_kv_cache cache8, const float *d_k_scale,
                                           const float *d_v_scale, l4l_tensor4 k_new, l4l_tensor4 v_new,
                                           const int32_t *d_kv_lens, int max_kv_len, int B, int Hq, int Hkv,
                                           int head_dim, float scale, const float *d_cos, const float *d_sin, int n_pos,
                                           const float *d_q_weight, const float *d_k_weight, float norm_eps,
                                           float *d_lse, void *workspace, size_t ws_bytes, l4l_stream stream);
l4l_status l4l_attn_decode_paged_rope_append_fp8(const void *q, void *o, l4l_paged_kv pool8, const float *d_k_scale,
                                                 const float *d_v_scale, const int32_t *d_block_table, int table_stride,
                                                 l4l_tensor4 k_new, l4l_tensor4 v_new, const int32_t *d_kv_lens,
                                                 int max_kv_len, int B, int Hq, int Hkv, int head_dim, float scale,
                                                 const float *d_cos, const float *d_sin, int n_pos,
                                                 const float *d_q_weight, const float *d_k_weight, float norm_eps,
                                                 float *d_lse, void *workspace, size_t ws_bytes, l4l_stream stream);

/*
 * Merge of R partial decode results over DISJOINT parts of the same sequences' caches: the step that
 * context-parallel decode adds (one sequence's cache sharded over R GPUs: every rank calls
 * l4l_attn_decode over its shard with d_lse set, the R (o, lse) pairs are gathered, this call combines
 * them). The paper runs on one GPU and has no counterpart; the formula is the one the split decode
 * kernel uses between its pieces:
 *     o = sum_r w_r o_r / sum_r w_r,   lse = m + ln sum_r w_r,   w_r = exp(lse_r - m),  m = max_r lse_r
 * A shard without keys has lse_r = -inf and weight 0; if all are empty, o = 0 and lse = -inf.
 *   o_parts      device bf16 [R, B, Hq, D] dense        d_lse_parts  device float [R, B, Hq]
 *   o            device bf16 [B, Hq, D] dense           d_lse        device float [B, Hq] or NULL
 */
l4l_status l4l_attn_merge(const void *o_parts, const float *d_lse_parts, int R, void *o, float *d_lse,
                          int B, int Hq, int head_dim, l4l_stream stream);

/*
 * Second workload: the gated linear recurrence of the RecurrentGemma block (RG-LRU). The paper's
 * appendix ("RecurrentGemma RGLRU", Table A.4) describes the accepted kernel as fusing sigmoid,
 * softplus-derived recurrent gating, reset handling, normalisation and the recurrent scan, with the
 * state carried through the sequence inside the kernel and the final state written once; it prints
 * no formula, so the recurrence is the published one of that block. For sequence b, channel c,
 * step t < seq_lens[b]:
 *     i = sigmoid(gate_x[b,t,c]),  r = sigmoid(gate_a[b,t,c]),  a = exp(-8 r softplus(a_param[c])),
 *     m = sqrt(1 - a^2);   if position[b,t] == 0:  a = 0, m = 1        (first token of a segment)
 *     h <- a h + m i x[b,t,c];   y[b,t,c] = h
 * with h starting from state[b,c] and state[b,c] receiving the last h (after seq_lens[b] steps).
 * fp32 arithmetic, y rounded to bf16. Rows t >= seq_lens[b] of y are left untouched.
 *   x, gate_x, gate_a, y   device bf16, dense [B, T, W] (W a multiple of 8; x / gate_x / gate_a 16-byte aligned)
 *   d_a_param    device float [W]
 *   d_position   device int32 [B, T], or NULL: no resets (a chunk that continues its sequence)
 *   d_seq_lens   device int32 [B], or NULL meaning T for all
 *   d_state      device float [B, W], read and written
 *   workspace    >= l4l_rglru_workspace_bytes(B, T, W) bytes, initialised once (at present the 256-byte
 *                status block: the state is handed from tile to tile on chip)
 */
size_t l4l_rglru_workspace_bytes(int B, int T, int W);

/*
 * Channels per strip (64, 32 or 16) that l4l_rglru_scan would give one thread block for these sizes on the
 * current device, without launching anything (for tests and tuning; no counterpart in the paper): narrower
 * strips are taken when 64-channel ones would load the SMs unevenly. -1 for sizes the scan rejects.
 */
int l4l_rglru_strip_channels(int B, int T, int W);
l4l_status l4l_rglru_scan(const void *x, const void *gate_x, const void *gate_a, const float *d_a_param,
                          const int32_t *d_position, const int32_t *d_seq_lens, float *d_state, void *y,
                          int B, int T, int W, void *workspace, size_t ws_bytes, l4l_stream stream);

/*
 * Rotary position embedding (and optional per-head RMS normalisation of q and k) fused with the
 * cache update: the projection outputs of the new tokens go through ONE streaming pass that
 * leaves q ready for the attention calls and K, V in the cache. (The paper's prefill kernel is
 * described as causal attention "with fused QKV wiring" and its decode path as keeping the cache
 * update's tensor contract; the paper prints no formula for the rotation, so the reading is the
 * half-split convention of the Llama / Qwen3 modules it names.) For sequence b, new token
 * t < n_new[b] at position P = pos[b] + t, every head row x of q and k_new (D values):
 *     if a norm weight w is given:   x[d] <- x[d] / sqrt(mean_d(x[d]^2) + eps) * w[d]
 *     for i < D/2:   y[i]       = x[i] * cos[P, i] - x[i + D/2] * sin[P, i]
 *                    y[i + D/2] = x[i + D/2] * cos[P, i] + x[i] * sin[P, i]
 * computed in fp32 and rounded once to bf16 (round to nearest even). q is overwritten with its y;
 * cache_k slot P of (b, kv head) receives k_new's y; cache_v slot P receives v_new bit for bit.
 * Tokens whose position falls outside [0, min(cache.max_len, n_pos)) are skipped entirely (q row
 * left as it was, nothing written). Afterwards: l4l_attn_prefill_chunk(q, ..., past = pos,
 * q_lens = n_new) for a prompt or a chunk, l4l_attn_decode for single tokens.
 *   q            [B, T, Hq, D] view, read and written     k_new, v_new  [B, T, Hkv, D] views, read
 *   d_pos        device int32 [B]      d_n_new  device int32 [B] or NULL (= T for all)
 *   d_cos, d_sin device float [n_pos, D/2], row P holding cos / sin of P * theta_i
 *   d_q_weight, d_k_weight   device float [D] or NULL (no normalisation of that tensor)
 */
l4l_status l4l_rope_kv_append(l4l_tensor4 q, l4l_tensor4 k_new, l4l_tensor4 v_new, l4l_kv_cache cache,
                              const int32_t *d_pos, const int32_t *d_n_new, int T,
                              int B, int Hq, int Hkv, int head_dim,
                              const float *d_cos, const float *d_sin, int n_pos,
                              const float *d_q_weight, const float *d_k_weight, float norm_eps,
                              l4l_stream stream);

/*
 * Causal prefill. For every sequence b with L = seq_lens[b] tokens, query head h, row i < L:
 *     o[b, i, h, :] = softmax_j( scale * q[b, i, h, :] . k[b, j, h/G, :],  j = 0..i ) @ v[b, 0..i, h/G, :]
 * and, when cache.k != NULL, cache slots 0..L-1 of sequence b receive k and v bit for bit
 * (the prompt starts an empty cache; for new tokens over a populated cache see
 * l4l_attn_prefill_chunk_append). Rows i >= L of o / lse and cache slots >= L are left untouched; q/k/v rows
 * >= L may hold anything.
 *   q, o         [B, S_max, Hq, D] views       k, v   [B, S_max, Hkv, D] views
 *   d_seq_lens   device int32 [B], each 0 <= L <= S_max (and <= cache.max_len when caching)
 *   S_max        host upper bound of the lengths = extent of the token dimension
 *   d_lse        device float [B, Hq, S_max] receiving max + ln(sum) of the scaled scores, or NULL
 *   workspace    >= l4l_workspace_bytes(L4L_OP_PREFILL, ...) bytes, initialised once
 */
l4l_status l4l_attn_prefill(l4l_tensor4 q, l4l_tensor4 k, l4l_tensor4 v, l4l_tensor4 o,
                            l4l_kv_cache cache, const int32_t *d_seq_lens, int S_max,
                            int B, int Hq, int Hkv, int head_dim, float scale,
                            float *d_lse, void *workspace, size_t ws_bytes, l4l_stream stream);

/*
 * Prefill of a chunk of new tokens over an already populated cache (the regime between the paper's
 * two phases: q_len > 1 AND a populated cache; bottom-right causal alignment). For sequence b with
 * P = past_lens[b] tokens already cached and L = q_lens[b] new tokens, whose K and V the caller has
 * ALREADY written to cache slots P .. P+L-1 (l4l_kv_append), query row i < L and query head h:
 *     o[b, i, h, :] = softmax_j( scale * q[b, i, h, :] . K[b, h/G, j, :],  j = 0 .. P+i ) @ V[b, h/G, 0..P+i, :]
 * Keys and values are read from the cache; nothing is written to it. P = 0 is an ordinary prefill
 * whose keys happen to live in the cache. Rows i >= L of o / lse are left untouched; cache slots
 * >= P+L may hold anything.
 *   q, o          [B, S_max, Hq, D] views (the chunk's tokens)
 *   d_past_lens   device int32 [B], P >= 0;   d_q_lens  device int32 [B], 0 <= L <= S_max; P + L <= cache.max_len
 *   d_lse         device float [B, Hq, S_max] or NULL;   workspace as for l4l_attn_prefill
 */
l4l_status l4l_attn_prefill_chunk(l4l_tensor4 q, l4l_tensor4 o, l4l_kv_cache cache,
                                  const int32_t *d_past_lens, const int32_t *d_q_lens, int S_max,
                                  int B, int Hq, int Hkv, int head_dim, float scale,
                                  float *d_lse, void *workspace, size_t ws_bytes, l4l_stream stream);

/*
 * The same chunk prefill with the cache update fused in (the paper's cache contract: the phase that produces
 * tokens updates the state exactly once; here in the same launch, as l4l_attn_prefill does for a prompt). The
 * chunk's K and V come from k_new / v_new; for sequence b with P = past_lens[b] and L = q_lens[b]:
 *     cache slots P .. P+L-1 receive k_new[b, 0..L-1] and v_new[b, 0..L-1] bit for bit, and
 *     o[b, i, h, :] = attention of q[b, i, h, :] over the cached tokens 0..P-1 and the new tokens 0..i.
 * Equivalent to l4l_kv_append at slot P followed by l4l_attn_prefill_chunk. Cache slots below P are only read,
 * slots from P+L on are neither read into a result nor written; new tokens whose slot lies outside the cache
 * (P + i >= cache.max_len) are still attended (from k_new / v_new) but not stored. P = 0 is an ordinary prefill.
 *   q, o          [B, S_max, Hq, D] views;   k_new, v_new  [B, S_max, Hkv, D] views (the chunk's tokens)
 *   everything else as in l4l_attn_prefill_chunk
 */
l4l_status l4l_attn_prefill_chunk_append(l4l_tensor4 q, l4l_tensor4 k_new, l4l_tensor4 v_new, l4l_tensor4 o,
                                         l4l_kv_cache cache, const int32_t *d_past_lens, const int32_t *d_q_lens,
                                         int S_max, int B, int Hq, int Hkv, int head_dim, float scale,
                                         float *d_lse, void *workspace, size_t ws_bytes, l4l_stream stream);

/*
 * l4l_attn_prefill_chunk_append over a paged cache (pool + block table, as in l4l_attn_decode_paged): the tokens
 * cached before are read page by page, the chunk's K and V are written to the page slots the block table names.
 * A slot whose table entry is not a page of the pool (or lies beyond table_stride entries) is read as zeros
 * (only slots >= P can be in that state in a well-formed table) and is not written.
 */
l4l_status l4l_attn_prefill_chunk_paged_append(l4l_tensor4 q, l4l_tensor4 k_new, l4l_tensor4 v_new, l4l_tensor4 o,
                                               l4l_paged_kv pool, const int32_t *d_block_table, int table_stride,
                                               const int32_t *d_past_lens, const int32_t *d_q_lens, int S_max,
                                               int B, int Hq, int Hkv, int head_dim, float scale,
                                               float *d_lse, void *workspace, size_t ws_bytes, l4l_stream stream);

/*
 * Decode. For every sequence b with n = kv_lens[b] cached tokens (the current token has
 * already been appended and is included), query head h:
 *     o[b, h, :] = softmax_j( scale * q[b, h, :] . K[b, h/G, j, :],  j = 0..n-1 ) @ V[b, h/G, 0..n-1, :]
 * with no mask. n = 0 gives o = 0 and lse = -inf. Cache slots >= n are never allowed to
 * influence the result, whatever bits they hold (slots up to the end of the 256-token block that
 * holds slot n-1 may be READ, inside cache.max_len only). Small batches (every (sequence, KV head)
 * on its own thread-block cluster at once) run a kernel that merges through shared memory, and
 * hundreds of sequences of at most a few hundred tokens (by max_kv_len) one that gives every
 * (sequence, KV head) to a single warp; both leave the workspace's partials unused; the
 * workspace is required all the same.
 *   q, o         dense [B, Hq, D]
 *   d_kv_lens    device int32 [B], each 0 <= n <= max_kv_len
 *   max_kv_len   host upper bound of kv_lens (<= cache.max_len); used to size the split
 *   d_lse        device float [B, Hq] or NULL
 *   workspace    >= l4l_workspace_bytes(L4L_OP_DECODE, ...) bytes; holds the fp32 partial
 *                results of the KV splits between the two passes
 */
l4l_status l4l_attn_decode(const void *q, void *o, l4l_kv_cache cache,
                           const int32_t *d_kv_lens, int max_kv_len,
                           int B, int Hq, int Hkv, int head_dim, float scale,
                           float *d_lse, void *workspace, size_t ws_bytes, l4l_stream stream);

/*
 * Decode with the cache update fused in (one launch per decode step instead of two; the paper leaves
 * the cache update to the module code around its decode kernel, and notes that the state must be
 * updated exactly once). For every sequence b with n = kv_lens[b] >= 1: cache slot n-1 receives
 * k_new[b, 0, :, :] and v_new[b, 0, :, :] bit for bit, and o[b] is the attention of q[b] over slots
 * 0..n-1 with that newest token taken from k_new / v_new. Equivalent to l4l_kv_append at slot n-1
 * followed by l4l_attn_decode; sequences with n = 0 append nothing and give o = 0.
 *   k_new, v_new  [B, 1, Hkv, D] views (stride_t unused); both with the same strides
 * Everything else as in l4l_attn_decode, except for a sequence whose kv_lens[b] exceeds the host bound
 * max_kv_len (a caller error): l4l_attn_decode ignores the tokens past the bound, whereas here the new token
 * has no slot inside the bound, so the sequence is treated as empty: nothing is written to the cache, o[b] = 0
 * and lse[b] = -inf. The same holds for every other entry point that fuses the append.
 */
l4l_status l4l_attn_decode_append(const void *q, void *o, l4l_kv_cache cache,
                                  l4l_tensor4 k_new, l4l_tensor4 v_new,
                                  const int32_t *d_kv_lens, int max_kv_len,
                                  int B, int Hq, int Hkv, int head_dim, float scale,
                                  float *d_lse, void *workspace, size_t ws_bytes, l4l_stream stream);

/*
 * Decode for callers that cannot allocate device memory (no counterpart in the paper: it is the
 * same operation as l4l_attn_decode, with the scratch moved inside the library).
 *
 * Who needs it: code that runs where cudaMalloc / cudaFree (or a framework allocator that may fall
 * back to them) is off limits at the moment decode is needed. Typical cases are a serving loop whose
 * memory plan is frozen after start-up because every spare byte of HBM already belongs to the KV
 * pool, and a plug-in inside someone else's runtime, where an allocation would synchronise the
 * device, stall the other streams and break the host's latency guarantees. Such callers have no
 * workspace to hand over and no safe way to make one.
 *
 * What it does instead: the status block, the ticket counters and the fp32 partials live in a fixed
 * array of L4L_STATIC_SCRATCH_BYTES inside the library's device image. Every GPU that loads the
 * library carries that array until the process exits, whether or not this entry point is used. The
 * call itself allocates nothing and frees nothing, through CUDA or any other library.
 *
 * Arguments, layouts, results and host-side validation are exactly those of l4l_attn_decode (inputs
 * and outputs are still the caller's buffers); there is no workspace argument. Differences:
 *   - Limit: the split of the KV axis is chosen so that its partials fit the fixed array. If even the
 *     coarsest split needs more than L4L_STATIC_SCRATCH_BYTES (roughly B * Hq * (head_dim + 1) * 8
 *     bytes plus 128 KiB of counters), the call returns L4L_ERR_WORKSPACE and launches nothing; use l4l_attn_decode
 *     with a workspace of your own for such sizes.
 *   - First call on each device: the device address of the array is looked up (with that device
 *     current) and remembered. Make this first call during start-up, before any stream capture.
 *   - Shared state: all calls on a device use the same array, which keeps what the previous call left
 *     in it; each call therefore clears the status block and the ticket counters on `stream` before its
 *     kernel. Two calls that can overlap on the GPU (different streams, no ordering between them) race
 *     on the array and give wrong results: order them, or give one of them a workspace.
 *   - A bounded device-side wait that runs out is recorded in the array's status block;
 *     l4l_check_status(NULL, stream) reads it.
 */
#define L4L_STATIC_SCRATCH_BYTES (8u << 20)
l4l_status l4l_attn_decode_static(const void *q, void *o, l4l_kv_cache cache,
                                  const int32_t *d_kv_lens, int max_kv_len,
                                  int B, int Hq, int Hkv, int head_dim, float scale,
                                  float *d_lse, l4l_stream stream);

/* Static, human-readable name of a status code. */
const char *l4l_status_string(l4l_status status);

/*
 * Which kernel the decode entry points would run for these sizes on the current device, without launching
 * anything (for tests and tuning): 0 = the split kernel (*detail = consumer warps per CTA), 1 = the cluster
 * kernel (*detail = CTAs per cluster), 2 = the warp-per-unit kernel, -1 = sizes the decode calls reject.
 * fp8: non-zero for an e4m3 cache. detail may be NULL. The overrides of l4l_set_decode_override are honoured
 * here as in the decode calls.
 */
int l4l_decode_kernel_choice(int B, int Hq, int Hkv, int head_dim, int max_kv_len, int fp8, int *detail);

/*
 * Tuning override of the decode kernel choice, process-wide (for tests and benchmarks that must hold a call on
 * one kernel; a serving loop has no reason to call it). No counterpart in the paper.
 *   cluster      -1 library's choice; 0 never the cluster kernel; N > 0 clusters of N CTAs where they fit
 *   warp         -1 library's choice; 0 never the warp-per-unit kernel; 1 that kernel wherever it can run
 *   split_warps   0 library's choice; 4 or 8 consumer warps per CTA of the split kernel
 * The decode calls never read the environment; L4L_DECODE_CLUSTER, L4L_DECODE_WARP and L4L_DECODE_WARPS are
 * read once, when the library is loaded, as the initial values of these three settings.
 */
void l4l_set_decode_override(int cluster, int warp, int split_warps);

/*
 * Synchronises `stream`, reads the workspace's status block and returns 0 if no bounded wait
 * has run out since the last l4l_workspace_init(), else a non-zero code identifying the wait
 * (bit 0: decode pipeline, bit 1: prefill pipeline, bit 2: scan pipeline, bit 3: the self-test). Returns -1 if
 * the read itself fails.
 */
int l4l_last_device_error(void *workspace, l4l_stream stream);

/*
 * The same check as a status: synchronises `stream` and returns L4L_OK if no bounded device-side wait has run
 * out since the status block was last cleared, L4L_ERR_TIMEOUT if one has (the kernels of that call gave up and
 * returned; their outputs are not valid), L4L_ERR_CUDA if the block cannot be read. workspace = NULL checks the
 * status block of the library's own scratch array on the current device, the one l4l_attn_decode_static uses
 * (that entry point clears it at every call, so the answer is about the latest such call). After
 * L4L_ERR_TIMEOUT, l4l_workspace_init makes the workspace usable again.
 */
l4l_status l4l_check_status(void *workspace, l4l_stream stream);

/*
 * Self-test of the time-out path (no counterpart in the paper; not part of the hot path). Launches one warp
 * that waits, with the library's bounded-wait routine and a budget of `budget_cycles` SM clock cycles (clamped
 * to [1000, 2^24], i.e. a few milliseconds at most), on a pipeline barrier that nothing ever completes. The wait
 * runs out, the kernel records bit 3 in the workspace's status block and returns normally: the context stays
 * usable, nothing traps. Afterwards l4l_last_device_error() reports a non-zero code and l4l_check_status()
 * L4L_ERR_TIMEOUT until l4l_workspace_init() is called. workspace: any workspace of this library (>= 256 bytes).
 */
l4l_status l4l_selftest_wait_expiry(void *workspace, size_t ws_bytes, long long budget_cycles, l4l_stream stream);

/* Library version, "major.minor". */
const char *l4l_version(void);

#ifdef __cplusplus
}
#endif
#endif /* L4L_H */
