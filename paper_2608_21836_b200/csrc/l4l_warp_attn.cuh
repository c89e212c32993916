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
template <int D>
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
        const uint32_t p01 = pack_bf16x2(fast_exp2(a0 - m_use), fast_exp2(a1 - m_use));
        const uint32_t p23 = pack_bf16x2(fast_exp2(a2 - m_use), fast_exp2(a3 - m_use));
        pa[h] = p01;          // tokens +0,+1
        pa[2 + h] = p23;      // tokens +8,+9
        // the denominator sums exactly the rounded weights that multiply V
        const float psum = __uint_as_float(p01 << 16) + __uint_as_float(p01 & 0xffff0000u) +
                           __uint_as_float(p23 << 16) + __uint_as_float(p23 & 0xffff0000u);
        st.l[h] = st.l[h] * corr + psum;
        st.m[h] = m_new;
#pragma unroll
        for (int nt = 0; nt < D / 8; ++nt) {
            st.o[nt][2 * h] *= corr;
            st.o[nt][2 * h + 1] *= corr;
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

}  // namespace l4l
