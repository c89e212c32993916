// Gated linear recurrence of the RecurrentGemma block (RG-LRU): gates, normalisation, reset handling and
// the scan over the sequence in one kernel; the state stays in registers for the whole sequence and is
// written once at the end.
//
// The recurrence is sequential in time and independent across (sequence, channel), so a consumer warp owns
// 64 channels of one sequence (two per lane, packed fp32x2 arithmetic) and walks the time axis. What lets
// that stream is that the loads do not wait for the arithmetic: the warp keeps two TMA tiles (16 time steps x
// 64 channels of x, gate_x and gate_a each) in flight and reads its inputs from shared memory; as soon as a
// tile's values are in registers its buffer is refilled with the tile after next. A CTA is that one warp
// (no producer warp holding registers it does not need), so that up to 18 of them share an SM.
//
// With few sequences there are too few such warps to fill the GPU (B * W / 64; 160 for 4 sequences of 2560
// channels), and each is bound by its own latency. The time axis is then cut into S segments that run in
// parallel, using the linearity of the recurrence: pass 1 computes for every segment the product A of its a_t
// and its end state E from a zero start; a small pass 2 chains h <- A h + E over the segments to get every
// segment's true start state (and the final state); pass 3 is the plain scan of every segment from that
// state. This reads the inputs twice (14 instead of 8 bytes per element) but runs S times as many warps. Per 16 steps the gates of all steps are evaluated first (independent, so MUFU and FMA latencies
// overlap), then the recurrence runs as a chain of 16 packed FMAs. 8 bytes per (step, channel) move through
// HBM (3 bf16 read, 1 written) against about 20 issued instructions and 4 MUFU operations per channel pair
// and step, so the kernel needs several resident warps per scheduler to approach the memory roofline, and
// B * W / 64 warps is all the parallelism there is: small batches are latency-bound.
#include "l4l_internal.h"
#include "l4l_ptx.cuh"

namespace l4l {

namespace {

constexpr int kTb = 16;          // time steps per tile
constexpr int kCb = 64;          // channels per tile (two per consumer lane)
constexpr int kStages = 2;
constexpr uint32_t kArrayBytes = kTb * kCb * 2;
constexpr uint32_t kStageBytes = 3 * kArrayBytes;

struct RglruParams {
    const float *a_param;        // [W]
    const int32_t *position;     // [B, T] or null
    const int32_t *seq_lens;     // [B] or null
    float *state;                // [B, W] in/out (single pass), or the start states [B, S, W] of pass 3
    float *agg_a, *agg_e;        // [B, S, W] outputs of pass 1
    __nv_bfloat16 *y;            // [B, T, W]
    unsigned *status;
    int B, T, W;
    int S, seg_len;              // segments per sequence and steps per segment (a multiple of kTb); S = 1: one pass
};

__device__ __forceinline__ float tanh_approx(float x)
{
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float sqrt_approx(float x)
{
    float y;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// two bf16 in one word -> packed fp32x2 (low half first)
__device__ __forceinline__ uint64_t widen2(uint32_t w) { return pack_u32x2(w << 16, w & 0xffff0000u); }

// sigmoid(z) = 0.5 tanh(z / 2) + 0.5 on both halves
__device__ __forceinline__ uint64_t sigmoid2(uint64_t z, uint64_t half2)
{
    float lo, hi;
    unpack_f32x2(mul_f32x2(z, half2), lo, hi);
    return fma_f32x2(pack_f32x2(tanh_approx(lo), tanh_approx(hi)), half2, half2);
}

// kAgg: pass 1 (segment aggregates, nothing written to y). Otherwise the scan proper.
template <bool kAgg>
__global__ void __launch_bounds__(32)
rglru_scan_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_gx,
                  const __grid_constant__ CUtensorMap tmap_ga, const RglruParams p)
{
    __shared__ __align__(128) uint8_t stages[kStages * kStageBytes];
    __shared__ uint64_t full[kStages];
    __shared__ int abort_word;
    volatile int *abort_flag = &abort_word;

    const int lane = threadIdx.x;
    const int b = blockIdx.y / p.S, seg = blockIdx.y % p.S, c0 = blockIdx.x * kCb;
    int L = p.seq_lens ? p.seq_lens[b] : p.T;
    L = L < 0 ? 0 : (L > p.T ? p.T : L);
    const int t_begin = seg * p.seg_len;                          // a multiple of kTb
    if (p.S > 1) L = min(L, t_begin + p.seg_len);                 // this segment's steps: [t_begin, L)
    const int tile0 = t_begin / kTb;
    const int n_tiles = L > t_begin ? (L - t_begin + kTb - 1) / kTb : 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) mbar_init(&full[s], 1);
        abort_word = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
    }
    __syncthreads();

    // lane 0 requests tile `it` into its buffer (rows past T arrive as zeros and still count)
    auto request = [&](int it) {
        if (lane == 0 && it < n_tiles) {
            const uint32_t s = it % kStages;
            mbar_arrive_expect_tx(&full[s], kStageBytes);
            uint8_t *dst = stages + s * kStageBytes;
            tma_load_3d(dst, &tmap_x, &full[s], c0, (tile0 + it) * kTb, b);
            tma_load_3d(dst + kArrayBytes, &tmap_gx, &full[s], c0, (tile0 + it) * kTb, b);
            tma_load_3d(dst + 2 * kArrayBytes, &tmap_ga, &full[s], c0, (tile0 + it) * kTb, b);
        }
    };
    if (lane == 0) {
        tma_prefetch_desc(&tmap_x);
        tma_prefetch_desc(&tmap_gx);
        tma_prefetch_desc(&tmap_ga);
    }
    for (int it = 0; it < kStages; ++it) request(it);
    {
        // ------------------------------------------------------------------ consumer: lane = channels c, c + 1
        const int c = c0 + 2 * lane;
        const bool live = c < p.W;                       // W is even: both channels or neither
        uint64_t h2 = pack_f32x2(0.f, 0.f);
        uint64_t k2 = h2;                                // -8 softplus(a_param) log2(e), per channel
        uint64_t prod2 = pack_f32x2(1.f, 1.f);           // pass 1: product of the a_t of this segment
        const size_t state_idx = (size_t)blockIdx.y * p.W + c;          // [B, W] or [B, S, W]
        if (live) {
            if (!kAgg) {
                const float2 st = *reinterpret_cast<const float2 *>(p.state + state_idx);
                h2 = pack_f32x2(st.x, st.y);
            }
            const float2 lam = *reinterpret_cast<const float2 *>(p.a_param + c);
            const float sp0 = lam.x > 15.f ? lam.x : log1pf(expf(lam.x));
            const float sp1 = lam.y > 15.f ? lam.y : log1pf(expf(lam.y));
            k2 = pack_f32x2(-8.f * 1.4426950408889634f * sp0, -8.f * 1.4426950408889634f * sp1);
        }
        const uint64_t half2 = pack_f32x2(0.5f, 0.5f), one2 = pack_f32x2(1.f, 1.f);
        const uint64_t two_ln2 = pack_f32x2(1.3862943611198906f, 1.3862943611198906f);
        const uint64_t c24 = pack_f32x2(1.f / 24.f, 1.f / 24.f), c6 = pack_f32x2(1.f / 6.f, 1.f / 6.f);
        const uint64_t neg1 = pack_f32x2(-1.f, -1.f);
        uint32_t *yrow = reinterpret_cast<uint32_t *>(p.y + (size_t)b * p.T * p.W + c);
        const size_t y_step = (size_t)p.W / 2;           // 32-bit words between time steps
        unsigned reset_next = 0u;
        auto resets_of = [&](int it) -> unsigned {
            // bit t: step it*kTb + t is the first token of a segment (position 0)
            if (!p.position) return 0u;
            const int t = (tile0 + it) * kTb + lane;
            const int pos = (lane < kTb && t < L) ? __ldg(p.position + (size_t)b * p.T + t) : 1;
            return __ballot_sync(0xffffffffu, pos == 0);
        };
        if (n_tiles > 0) reset_next = resets_of(0);
        for (int it = 0; it < n_tiles; ++it) {
            const uint32_t s = it % kStages, ph = (it / kStages) & 1u;
            const unsigned resets = reset_next;
            if (it + 1 < n_tiles) reset_next = resets_of(it + 1);     // in flight while this tile is processed
            if (!mbar_wait(&full[s], ph, abort_flag)) break;
            const uint32_t *xs = reinterpret_cast<const uint32_t *>(stages + s * kStageBytes) + lane;
            const uint32_t *gxs = xs + kTb * kCb / 2, *gas = gxs + kTb * kCb / 2;
            const int t0 = (tile0 + it) * kTb;
            const int n = min(kTb, L - t0);
            // Phase 1: a_t and b_t = m_t i_t x_t of all steps of the tile (independent of the state)
            uint64_t av[kTb], bv[kTb];
#pragma unroll
            for (int t = 0; t < kTb; ++t) {
                const uint64_t xv = widen2(xs[t * (kCb / 2)]);
                const uint64_t in_gate = sigmoid2(widen2(gxs[t * (kCb / 2)]), half2);
                const uint64_t rec_gate = sigmoid2(widen2(gas[t * (kCb / 2)]), half2);
                const uint64_t la2 = mul_f32x2(k2, rec_gate);                  // log2(a)
                float l0, l1;
                unpack_f32x2(la2, l0, l1);
                const float a0 = fast_exp2(l0), a1 = fast_exp2(l1);
                uint64_t a = pack_f32x2(a0, a1);
                // 1 - a^2 = -expm1(z), z = 2 ln a: a short series when a is close to 1, where 1 - a*a cancels
                const uint64_t z = mul_f32x2(la2, two_ln2);
                const uint64_t poly = fma_f32x2(z, fma_f32x2(z, fma_f32x2(z, c24, c6), half2), one2);
                float s0, s1, d0, d1, z0, z1;
                unpack_f32x2(mul_f32x2(mul_f32x2(z, neg1), poly), s0, s1);
                unpack_f32x2(fma_f32x2(mul_f32x2(a, neg1), a, one2), d0, d1);
                unpack_f32x2(z, z0, z1);
                float m0 = sqrt_approx(z0 > -0.0625f ? s0 : d0), m1 = sqrt_approx(z1 > -0.0625f ? s1 : d1);
                if ((resets >> t) & 1u) {                                      // uniform across the warp
                    a = pack_f32x2(0.f, 0.f);
                    m0 = m1 = 1.f;
                }
                av[t] = a;
                bv[t] = mul_f32x2(mul_f32x2(pack_f32x2(m0, m1), in_gate), xv);
            }
            // every lane has its values of this tile in registers: the buffer can take the tile after next
            __syncwarp();
            request(it + kStages);
            // Phase 2: the recurrence, one packed FMA per step
#pragma unroll
            for (int t = 0; t < kTb; ++t) {
                if (t < n) {                                                   // uniform across the warp
                    h2 = fma_f32x2(av[t], h2, bv[t]);
                    if constexpr (kAgg) {
                        prod2 = mul_f32x2(prod2, av[t]);
                    } else {
                        float h0, h1;
                        unpack_f32x2(h2, h0, h1);
                        if (live) yrow[(size_t)(t0 + t) * y_step] = pack_bf16x2(h0, h1);
                    }
                }
            }
        }
        if (live) {
            float h0, h1;
            unpack_f32x2(h2, h0, h1);
            if constexpr (kAgg) {
                float a0, a1;
                unpack_f32x2(prod2, a0, a1);
                *reinterpret_cast<float2 *>(p.agg_a + state_idx) = make_float2(a0, a1);
                *reinterpret_cast<float2 *>(p.agg_e + state_idx) = make_float2(h0, h1);
            } else if (p.S == 1) {
                *reinterpret_cast<float2 *>(p.state + state_idx) = make_float2(h0, h1);   // pass 2 writes it otherwise
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0 && abort_word) atomicOr(p.status + kStatusErrWord, kErrScanWait);
}

// Pass 2: chains the segment aggregates. start[b, seg, c] = state before the segment; the state after the last
// segment goes back to state[b, c].
__global__ void __launch_bounds__(256)
rglru_carry_kernel(const float *agg_a, const float *agg_e, float *start, float *state, int B, int S, int W)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= B * W) return;
    const int b = i / W, c = i % W;
    float h = state[i];
    for (int seg = 0; seg < S; ++seg) {
        const size_t k = ((size_t)b * S + seg) * W + c;
        start[k] = h;
        h = fmaf(agg_a[k], h, agg_e[k]);
    }
    state[i] = h;
}

}  // namespace

// Segments per sequence: enough warps to fill the GPU (about 16 per SM), no segment shorter than 64 steps.
int rglru_segments(int B, int T, int W)
{
    const long long warps = (long long)B * ((W + kCb - 1) / kCb);
    const long long want = 16ll * sm_count();
    long long S = (want + warps - 1) / warps;
    const long long max_s = T / 64 > 1 ? T / 64 : 1;
    if (S > max_s) S = max_s;
    if (S < 2) return 1;
    return (int)S;
}

size_t rglru_workspace_bytes(int B, int T, int W)
{
    const int S = rglru_segments(B, T, W);
    return kStatusBytes + (S > 1 ? (size_t)3 * B * S * W * sizeof(float) : 0);
}

l4l_status launch_rglru_scan(const void *x, const void *gate_x, const void *gate_a, const float *d_a_param,
                             const int32_t *d_position, const int32_t *d_seq_lens, float *d_state, void *y, int B, int T,
                             int W, void *workspace, size_t ws_bytes, cudaStream_t stream)
{
    CUtensorMap tx, tgx, tga;
    if (!make_tmap_rows_bf16(&tx, x, W, T, B, W, (int64_t)T * W, kCb, kTb) ||
        !make_tmap_rows_bf16(&tgx, gate_x, W, T, B, W, (int64_t)T * W, kCb, kTb) ||
        !make_tmap_rows_bf16(&tga, gate_a, W, T, B, W, (int64_t)T * W, kCb, kTb))
        return L4L_ERR_CUDA;
    // segments only if the caller's workspace has room for the aggregates and start states
    int S = rglru_segments(B, T, W);
    if (ws_bytes < kStatusBytes + (size_t)3 * B * S * W * sizeof(float)) S = 1;
    if ((long long)B * S > 65535) S = 1;
    RglruParams p;
    p.a_param = d_a_param; p.position = d_position; p.seq_lens = d_seq_lens; p.state = d_state;
    p.agg_a = p.agg_e = nullptr;
    p.y = static_cast<__nv_bfloat16 *>(y);
    p.status = static_cast<unsigned *>(workspace);
    p.B = B; p.T = T; p.W = W;
    p.S = S;
    p.seg_len = ((T + S - 1) / S + kTb - 1) / kTb * kTb;
    const dim3 grid((W + kCb - 1) / kCb, B * S);
    if (S > 1) {
        float *scratch = reinterpret_cast<float *>(static_cast<uint8_t *>(workspace) + kStatusBytes);
        const size_t n = (size_t)B * S * W;
        p.agg_a = scratch;
        p.agg_e = scratch + n;
        float *start = scratch + 2 * n;
        rglru_scan_kernel<true><<<grid, 32, 0, stream>>>(tx, tgx, tga, p);
        rglru_carry_kernel<<<(B * W + 255) / 256, 256, 0, stream>>>(p.agg_a, p.agg_e, start, d_state, B, S, W);
        p.state = start;
    }
    rglru_scan_kernel<false><<<grid, 32, 0, stream>>>(tx, tgx, tga, p);
    return cudaGetLastError() == cudaSuccess ? L4L_OK : L4L_ERR_CUDA;
}

}  // namespace l4l
