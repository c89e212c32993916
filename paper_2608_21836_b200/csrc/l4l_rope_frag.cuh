// Rotary embedding (+ optional per-head RMS norm) of a decode step's own token on the data layouts of the decode
// kernels: the query rows as warp-MMA A fragments in registers, the new key row as 16-byte pieces across a warp.
#pragma once

#include "l4l_ptx.cuh"

namespace l4l {

// Same arithmetic as the streaming rope kernel: xn = (x * rinv) * w, y1 = fma(-x2, sin, x1 * cos),
// y2 = fma(x1, sin, x2 * cos) in fp32, one rounding to bf16. A position outside the table leaves the row as it is.
// The cos | sin rows of the position come from shared memory: the producer fetches them with the piece's first tile.

// The q rows live in the A fragments of the warp MMA: a thread holds, per 16-column k-step, columns 2c, 2c+1
// (registers 0: row lane/4, 1: row lane/4 + 8) and 2c+8, 2c+9 (registers 2, 3), c = lane % 4. The partner of
// column i is column i + D/2, i.e. the same register of the k-step D/32 further on: no data leaves the thread.
// (The warp-per-unit kernel rotates this way: every warp has its own query rows. The split and the cluster kernel,
// where all warps of a CTA share the rows, rotate them once in shared memory instead: rope_row_in_smem below.)
template <int D>
__device__ __forceinline__ void rope_q_fragments(uint32_t (&qf)[D / 16][4], int G, bool with_norm, float norm_eps,
                                                 const float *cos_sin, const float *weight, int lane)
{
    constexpr int kSteps = D / 16, kHalf = kSteps / 2;
    const int c = lane & 3;
    const bool valid[2] = {(lane >> 2) < G, (lane >> 2) + 8 < G};
    float rinv[2] = {1.f, 1.f};
    if (with_norm) {
        float ss[2] = {0.f, 0.f};
#pragma unroll
        for (int ks = 0; ks < kSteps; ++ks)
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const float a = __uint_as_float(qf[ks][r] << 16), b = __uint_as_float(qf[ks][r] & 0xffff0000u);
                ss[r & 1] = fmaf(a, a, fmaf(b, b, ss[r & 1]));
            }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            ss[h] += __shfl_xor_sync(0xffffffffu, ss[h], 1);
            ss[h] += __shfl_xor_sync(0xffffffffu, ss[h], 2);
            rinv[h] = valid[h] ? rsqrtf(ss[h] * (1.f / D) + norm_eps) : 0.f;
        }
    }
    const float *cr = cos_sin, *sr = cos_sin + D / 2;              // shared memory: cos | sin of the position
#pragma unroll
    for (int ks = 0; ks < kHalf; ++ks)
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int col = 16 * ks + 2 * c + ((r >> 1) << 3);               // first-half column of element 0
            float x1[2] = {__uint_as_float(qf[ks][r] << 16), __uint_as_float(qf[ks][r] & 0xffff0000u)};
            float x2[2] = {__uint_as_float(qf[ks + kHalf][r] << 16), __uint_as_float(qf[ks + kHalf][r] & 0xffff0000u)};
            float y1[2], y2[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                if (with_norm) {
                    x1[e] = x1[e] * rinv[r & 1] * weight[col + e];
                    x2[e] = x2[e] * rinv[r & 1] * weight[col + e + D / 2];
                }
                const float cs = cr[col + e], sn = sr[col + e];
                y1[e] = fmaf(-x2[e], sn, x1[e] * cs);
                y2[e] = fmaf(x1[e], sn, x2[e] * cs);
            }
            if (valid[r & 1]) {
                qf[ks][r] = pack_bf16x2(y1[0], y1[1]);
                qf[ks + kHalf][r] = pack_bf16x2(y2[0], y2[1]);
            }
        }
}

// One query row rotated in place in shared memory by one warp: lane l owns the words l (elements 2l, 2l+1) and
// D/4 + l (their partners, D/2 columns further on); lanes >= D/4 idle. Small code on purpose: it runs once per
// piece, from a cold instruction cache. All lanes of the warp must call this (shuffles).
template <int D>
__device__ __forceinline__ void rope_row_in_smem(uint32_t *row, const float *cos_sin, bool with_norm, float norm_eps,
                                                 const float *weight, int lane)
{
    constexpr int kWords = D / 4;                       // 32-bit words per half row
    const bool on = lane < kWords;
    const uint32_t w1 = on ? row[lane] : 0u, w2 = on ? row[kWords + lane] : 0u;
    float x1[2] = {__uint_as_float(w1 << 16), __uint_as_float(w1 & 0xffff0000u)};
    float x2[2] = {__uint_as_float(w2 << 16), __uint_as_float(w2 & 0xffff0000u)};
    if (with_norm) {
        float ss = fmaf(x1[0], x1[0], fmaf(x1[1], x1[1], fmaf(x2[0], x2[0], x2[1] * x2[1])));
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, d);
        const float rinv = rsqrtf(ss * (1.f / D) + norm_eps);
        if (on) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                x1[e] = x1[e] * rinv * weight[2 * lane + e];
                x2[e] = x2[e] * rinv * weight[D / 2 + 2 * lane + e];
            }
        }
    }
    if (on) {
        float y1[2], y2[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const float cs = cos_sin[2 * lane + e], sn = cos_sin[D / 2 + 2 * lane + e];
            y1[e] = fmaf(-x2[e], sn, x1[e] * cs);
            y2[e] = fmaf(x1[e], sn, x2[e] * cs);
        }
        row[lane] = pack_bf16x2(y1[0], y1[1]);
        row[kWords + lane] = pack_bf16x2(y2[0], y2[1]);
    }
}

// The new token's k row as the patching warp holds it: lane l < D/8 has elements [8l, 8l + 8). The partner chunk
// is D/16 lanes away. Every lane of the warp must call this (shuffles); lanes >= D/8 pass zeros.
template <int D>
__device__ __forceinline__ uint4 rope_k_row(uint4 kk, bool with_norm, float norm_eps, const float *cos_sin,
                                            const float *weight, bool in_table, int lane)
{
    constexpr int kChunks = D / 8, kHalfChunks = D / 16;
    float x[8];
    const uint32_t w[4] = {kk.x, kk.y, kk.z, kk.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        x[2 * i] = __uint_as_float(w[i] << 16);
        x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
    if (with_norm) {
        float ss = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) ss = fmaf(x[i], x[i], ss);
#pragma unroll
        for (int off = 1; off < kChunks; off <<= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
        const float rinv = rsqrtf(ss * (1.f / D) + norm_eps);
        if (lane < kChunks && in_table) {
#pragma unroll
            for (int i = 0; i < 8; ++i) x[i] = x[i] * rinv * weight[8 * lane + i];
        }
    }
    float y[8];
    const bool first = (lane & kHalfChunks) == 0;
    const int col0 = 8 * (lane & (kHalfChunks - 1));
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float px = __shfl_xor_sync(0xffffffffu, x[i], kHalfChunks);
        float cs = 1.f, sn = 0.f;
        if (lane < kChunks && in_table) {
            cs = cos_sin[col0 + i];
            sn = cos_sin[D / 2 + col0 + i];
        }
        y[i] = first ? fmaf(-px, sn, x[i] * cs) : fmaf(px, sn, x[i] * cs);
    }
    if (!in_table) return kk;
    return make_uint4(pack_bf16x2(y[0], y[1]), pack_bf16x2(y[2], y[3]), pack_bf16x2(y[4], y[5]), pack_bf16x2(y[6], y[7]));
}

// The rotated row regrouped for the e4m3 quantiser: from 8 values per lane (lanes < D/8) to 16 values per lane
// (lanes < D/16) as two 16-byte pieces. Every lane of the warp must call this.
__device__ __forceinline__ void regroup_row_16(const uint4 &kk, int lane, uint4 &a, uint4 &b)
{
    const int src = (2 * lane) & 31;
    a.x = __shfl_sync(0xffffffffu, kk.x, src);     a.y = __shfl_sync(0xffffffffu, kk.y, src);
    a.z = __shfl_sync(0xffffffffu, kk.z, src);     a.w = __shfl_sync(0xffffffffu, kk.w, src);
    b.x = __shfl_sync(0xffffffffu, kk.x, src + 1); b.y = __shfl_sync(0xffffffffu, kk.y, src + 1);
    b.z = __shfl_sync(0xffffffffu, kk.z, src + 1); b.w = __shfl_sync(0xffffffffu, kk.w, src + 1);
}

}  // namespace l4l
