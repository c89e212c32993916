// Warp-level building blocks on the legacy tensor path (mma.sync m16n8k16, bf16 -> fp32):
// one warp holds 16 query rows and consumes 16 tokens of K and V at a time from a shared-
// memory tile written by TMA with the 128-byte swizzle. Used by the decode kernel, where
// the 16 rows are the (zero-padded) query-head group of one KV head. (Prefill runs on
// tcgen05 instead: see l4l_prefill_tc.cu.)
//
// Tile layout in shared memory: D/64 "halves", each [tile_tokens][64] bf16 (128-byte rows,
// swizzled), half h covering head_dim [64h, 64h+64).
#pragma once

#include "l4l_ptx.cuh"

namespace l4l {

template <int D>
struct WarpAttnState {
    float m[2];           // running max (log2 domain) of rows lane/4 and lane/4 + 8
    float l[2];           // this lane's share of the running sum
    float o[D / 8][4];    // accumulator fragments: n-tile nt covers head_dim [8nt, 8nt+8)

    __device__ __forceinline__ void reset()
    {
        m[0] = m[1] = -INFINITY;
        l[0] = l[1] = 0.f;
#pragma unroll
        for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    }
};

// S(16 rows x 16 tokens) = Q(16 x D) . K(tokens row0..row0+15)^T.
// s_lo: tokens row0 + 2*(lane%4) + {0,1}   (elements 0,1: row lane/4; 2,3: row lane/4 + 8)
// s_hi: the same for tokens + 8.
template <int D>
__device__ __forceinline__ void warp_qk_16x16(const uint32_t (&qf)[D / 16][4], uint32_t k_tile, uint32_t half_bytes,
                                              int row0, float (&s_lo)[4], float (&s_hi)[4])
{
    const int lane = threadIdx.x & 31;
    s_lo[0] = s_lo[1] = s_lo[2] = s_lo[3] = 0.f;
    s_hi[0] = s_hi[1] = s_hi[2] = s_hi[3] = 0.f;
    const uint32_t row = row0 + ((lane >> 4) << 3) + (lane & 7);   // matrices 2,3: tokens +8
    const uint32_t csel = (lane >> 3) & 1;                          // matrices 1,3: head_dim +8
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
        const uint32_t chunk = 2 * ks + csel;                       // 16-byte chunk of the full row
        const uint32_t addr = k_tile + (chunk >> 3) * half_bytes + swz128(row, chunk & 7);
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4(addr, b0, b1, b2, b3);
        mma_bf16_16816(s_lo, qf[ks], b0, b1);
        mma_bf16_16816(s_hi, qf[ks], b2, b3);
    }
}

// Online-softmax update for 16 tokens. Scores arrive already multiplied by scale*log2(e)
// and with masked positions set to -inf. Produces the bf16 A-fragment of P and rescales O.
// kF16: P is packed as f16 (for the f16 MMAs of the fp8-cache path) instead of bf16.
template <int D, bool kF16 = false>
__device__ __forceinline__ void warp_softmax_16(WarpAttnState<D> &st, const float (&s_lo)[4], const float (&s_hi)[4],
                                                uint32_t (&pa)[4])
{
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const float a0 = s_lo[2 * h], a1 = s_lo[2 * h + 1], a2 = s_hi[2 * h], a3 = s_hi[2 * h + 1];
        float mx = fmaxf(fmaxf(a0, a1), fmaxf(a2, a3));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(st.m[h], mx);
        const float m_use = (m_new == -INFINITY) ? 0.f : m_new;     // row with nothing visible yet
        const float corr = fast_exp2(st.m[h] - m_use);
        const float e0 = fast_exp2(a0 - m_use), e1 = fast_exp2(a1 - m_use);
        const float e2 = fast_exp2(a2 - m_use), e3 = fast_exp2(a3 - m_use);
        const uint32_t p01 = kF16 ? pack_f16x2(e0, e1) : pack_bf16x2(e0, e1);
        const uint32_t p23 = kF16 ? pack_f16x2(e2, e3) : pack_bf16x2(e2, e3);
        pa[h] = p01;          // tokens +0,+1
        pa[2 + h] = p23;      // tokens +8,+9
        // the denominator sums exactly the rounded weights that multiply V
        const float psum = kF16 ? sum_f16x2(p01) + sum_f16x2(p23)
                                : __uint_as_float(p01 << 16) + __uint_as_float(p01 & 0xffff0000u) +
                                      __uint_as_float(p23 << 16) + __uint_as_float(p23 & 0xffff0000u);
        st.l[h] = st.l[h] * corr + psum;
        st.m[h] = m_new;
        // O is rescaled only if some row of this half saw its maximum grow (after the first tiles of a long
        // sequence that is rare): corr == 1 exactly otherwise
        if (__any_sync(0xffffffffu, corr != 1.f)) {
#pragma unroll
            for (int nt = 0; nt < D / 8; ++nt) {
                st.o[nt][2 * h] *= corr;
                st.o[nt][2 * h + 1] *= corr;
            }
        }
    }
}

// O(16 x D) += P(16 x 16 tokens) . V(tokens row0..row0+15, D)
template <int D>
__device__ __forceinline__ void warp_pv_16x16(WarpAttnState<D> &st, const uint32_t (&pa)[4], uint32_t v_tile,
                                              uint32_t half_bytes, int row0)
{
    const int lane = threadIdx.x & 31;
    const uint32_t row = row0 + (((lane >> 3) & 1) << 3) + (lane & 7);   // matrices 1,3: tokens +8
    const uint32_t csel = lane >> 4;                                      // matrices 2,3: head_dim +8
#pragma unroll
    for (int np = 0; np < D / 16; ++np) {
        const uint32_t chunk = 2 * np + csel;
        const uint32_t addr = v_tile + (chunk >> 3) * half_bytes + swz128(row, chunk & 7);
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4_trans(addr, b0, b1, b2, b3);
        mma_bf16_16816(st.o[2 * np], pa, b0, b1);
        mma_bf16_16816(st.o[2 * np + 1], pa, b2, b3);
    }
}

// Online-softmax update over NT 8-token score tiles at once (NT = 2 is warp_softmax_16; the fp8 path takes 32
// tokens per step so that the shuffles and the bookkeeping are paid once per 32 tokens). s[j] holds tokens
// 8j + 2*(lane%4) + {0,1} (elements 0,1: row lane/4; 2,3: row lane/4 + 8); pa[u] is the A fragment of P for
// tokens 16u .. 16u+15.
template <int D, bool kF16, int NT>
__device__ __forceinline__ void warp_softmax_tiles(WarpAttnState<D> &st, const float (&s)[NT][4], uint32_t (&pa)[NT / 2][4])
{
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        float mx = -INFINITY;
#pragma unroll
        for (int j = 0; j < NT; ++j) mx = fmaxf(mx, fmaxf(s[j][2 * h], s[j][2 * h + 1]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(st.m[h], mx);
        const float m_use = (m_new == -INFINITY) ? 0.f : m_new;     // row with nothing visible yet
        const float corr = fast_exp2(st.m[h] - m_use);
        float psum = 0.f;
#pragma unroll
        for (int j = 0; j < NT; ++j) {
            const float e0 = fast_exp2(s[j][2 * h] - m_use), e1 = fast_exp2(s[j][2 * h + 1] - m_use);
            const uint32_t pk = kF16 ? pack_f16x2(e0, e1) : pack_bf16x2(e0, e1);
            pa[j >> 1][(j & 1) * 2 + h] = pk;
            // the denominator sums exactly the rounded weights that multiply V
            psum += kF16 ? sum_f16x2(pk) : __uint_as_float(pk << 16) + __uint_as_float(pk & 0xffff0000u);
        }
        st.l[h] = st.l[h] * corr + psum;
        st.m[h] = m_new;
        if (__any_sync(0xffffffffu, corr != 1.f)) {
#pragma unroll
            for (int nt = 0; nt < D / 8; ++nt) {
                st.o[nt][2 * h] *= corr;
                st.o[nt][2 * h + 1] *= corr;
            }
        }
    }
}

// ----------------------------------------------------------------------------- fp8 (e4m3) K/V tiles
// A tile is rows of 128 bytes, 128-byte swizzled: one token per row at D = 128, TWO consecutive tokens per row at
// D = 64 (token 2r in bytes 0..63 of row r, token 2r+1 in bytes 64..127: a dense cache of 64-byte token rows seen as
// rows of 128). tok_chunk_f8 gives the address of 16-byte chunk c (16 head dims) of a token either way. The values are
// widened to f16 in registers (exact) and multiplied with f16 MMAs. ldmatrix moves 16-bit units, so a
// thread receives 4 consecutive head-dim bytes of a K row where the MMA wants two separate pairs: the
// k index of QK^T is therefore permuted (MMA slots 2c, 2c+1, 2c+8, 2c+9 of a 16-block hold head dims
// 4c .. 4c+3), and the q fragments are built with the same permutation (see q_frag_f8_word). For V the
// transposing ldmatrix delivers, per thread, two tokens of an EVEN and an ODD head dim: the 8-column
// MMA tiles of O alternate even / odd dims (tile 2j: dims 16j + 2x, tile 2j+1: dims 16j + 2x + 1 in
// column x); a thread's accumulators of a tile pair are then 4 consecutive head dims.

// Shared-memory address of head dims [16c, 16c+16) of token `tok` of an fp8 tile.
template <int D>
__device__ __forceinline__ uint32_t tok_chunk_f8(uint32_t tile, uint32_t tok, uint32_t c)
{
    static_assert(D == 128 || D == 64, "one or two tokens per 128-byte row");
    if constexpr (D == 128) return tile + swz128(tok, c);
    else return tile + swz128(tok >> 1, ((tok & 1u) << 2) + c);
}

// 32-bit word (two bf16) of a q row that feeds A-fragment register `reg` (0..3) of k-step ks, as f16x2.
__device__ __forceinline__ int q_frag_f8_word(int ks, int reg, int lane) { return ks * 8 + 2 * (lane & 3) + (reg >> 1); }

__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t v)
{
    return pack_f16x2(__uint_as_float(v << 16), __uint_as_float(v & 0xffff0000u));
}

template <int D>
__device__ __forceinline__ void warp_qk_16x16_f8(const uint32_t (&qf)[D / 16][4], uint32_t k_tile, int row0,
                                                 float (&s_lo)[4], float (&s_hi)[4])
{
    const int lane = threadIdx.x & 31;
    s_lo[0] = s_lo[1] = s_lo[2] = s_lo[3] = 0.f;
    s_hi[0] = s_hi[1] = s_hi[2] = s_hi[3] = 0.f;
    const uint32_t row = row0 + ((lane >> 4) << 3) + (lane & 7);   // matrices 2,3: tokens +8
    const uint32_t csel = (lane >> 3) & 1;                          // matrices 1,3: next 16 head dims
#pragma unroll
    for (int qd = 0; qd < D / 32; ++qd) {
        uint32_t r0, r1, r2, r3;
        ldmatrix_x4(tok_chunk_f8<D>(k_tile, row, 2 * qd + csel), r0, r1, r2, r3);
        mma_f16_16816(s_lo, qf[2 * qd], e4m3x2_to_f16x2(r0), e4m3x2_to_f16x2(r0 >> 16));
        mma_f16_16816(s_lo, qf[2 * qd + 1], e4m3x2_to_f16x2(r1), e4m3x2_to_f16x2(r1 >> 16));
        mma_f16_16816(s_hi, qf[2 * qd], e4m3x2_to_f16x2(r2), e4m3x2_to_f16x2(r2 >> 16));
        mma_f16_16816(s_hi, qf[2 * qd + 1], e4m3x2_to_f16x2(r3), e4m3x2_to_f16x2(r3 >> 16));
    }
}

template <int D>
__device__ __forceinline__ void warp_pv_16x16_f8(WarpAttnState<D> &st, const uint32_t (&pa)[4], uint32_t v_tile, int row0)
{
    const int lane = threadIdx.x & 31;
    const uint32_t row = row0 + (((lane >> 3) & 1) << 3) + (lane & 7);   // matrices 1,3: tokens +8
    const uint32_t csel = lane >> 4;                                      // matrices 2,3: next 16 head dims
#pragma unroll
    for (int qd = 0; qd < D / 32; ++qd) {
        uint32_t r0, r1, r2, r3;
        ldmatrix_x4_trans(tok_chunk_f8<D>(v_tile, row, 2 * qd + csel), r0, r1, r2, r3);
        // bytes (tok, even) (tok, odd) (tok+1, even) (tok+1, odd) -> (tok, even) (tok+1, even) | (tok, odd) (tok+1, odd)
        const uint32_t x0 = __byte_perm(r0, 0u, 0x3120), x1 = __byte_perm(r1, 0u, 0x3120);
        const uint32_t x2 = __byte_perm(r2, 0u, 0x3120), x3 = __byte_perm(r3, 0u, 0x3120);
        mma_f16_16816(st.o[4 * qd], pa, e4m3x2_to_f16x2(x0), e4m3x2_to_f16x2(x1));
        mma_f16_16816(st.o[4 * qd + 1], pa, e4m3x2_to_f16x2(x0 >> 16), e4m3x2_to_f16x2(x1 >> 16));
        mma_f16_16816(st.o[4 * qd + 2], pa, e4m3x2_to_f16x2(x2), e4m3x2_to_f16x2(x3));
        mma_f16_16816(st.o[4 * qd + 3], pa, e4m3x2_to_f16x2(x2 >> 16), e4m3x2_to_f16x2(x3 >> 16));
    }
}

}  // namespace l4l
