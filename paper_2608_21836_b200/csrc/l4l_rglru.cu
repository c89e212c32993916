// Gated linear recurrence of the RecurrentGemma block (RG-LRU): gates, normalisation, reset handling and
// the scan over the sequence in one kernel; the state stays in a register for the whole sequence and is
// written once at the end.
//
// The recurrence is sequential in time and independent across (sequence, channel), so a consumer warp owns
// 32 channels of one sequence (one per lane) and walks the time axis. What makes that stream at memory
// speed is that the loads do not wait for the arithmetic: a producer thread keeps a ring of TMA tiles
// (32 time steps x 32 channels of x, gate_x and gate_a) full, and the consumer reads its inputs from shared
// memory. HBM-bound for enough channels (B * W / 32 warps; 4 MUFU operations per element keep a warp at
// about 8 bytes per cycle): 8 bytes per (step, channel), 3 bf16 read and 1 written.
#include "l4l_internal.h"
#include "l4l_ptx.cuh"

namespace l4l {

namespace {

constexpr int kTb = 32;          // time steps per tile
constexpr int kCb = 32;          // channels per tile (one per consumer lane)
constexpr int kStages = 6;
constexpr uint32_t kArrayBytes = kTb * kCb * 2;
constexpr uint32_t kStageBytes = 3 * kArrayBytes;

struct RglruParams {
    const float *a_param;        // [W]
    const int32_t *position;     // [B, T] or null
    const int32_t *seq_lens;     // [B] or null
    float *state;                // [B, W] in/out
    __nv_bfloat16 *y;            // [B, T, W]
    unsigned *status;
    int B, T, W;
};

__device__ __forceinline__ float tanh_approx(float x)
{
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float sigmoid_fast(float z) { return fmaf(0.5f, tanh_approx(0.5f * z), 0.5f); }

__device__ __forceinline__ float bf16_bits_to_float(unsigned short v) { return __uint_as_float((uint32_t)v << 16); }

__global__ void __launch_bounds__(64)
rglru_scan_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_gx,
                  const __grid_constant__ CUtensorMap tmap_ga, const RglruParams p)
{
    __shared__ __align__(128) uint8_t stages[kStages * kStageBytes];
    __shared__ uint64_t full[kStages], empty[kStages];
    __shared__ int abort_word;
    volatile int *abort_flag = &abort_word;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.y, c0 = blockIdx.x * kCb;
    int L = p.seq_lens ? p.seq_lens[b] : p.T;
    L = L < 0 ? 0 : (L > p.T ? p.T : L);
    const int n_tiles = (L + kTb - 1) / kTb;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        abort_word = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
    }
    __syncthreads();

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            tma_prefetch_desc(&tmap_x);
            tma_prefetch_desc(&tmap_gx);
            tma_prefetch_desc(&tmap_ga);
            for (int it = 0; it < n_tiles; ++it) {
                const uint32_t s = it % kStages, ph = (it / kStages) & 1u;
                if (!mbar_wait(&empty[s], ph ^ 1u, abort_flag)) break;
                mbar_arrive_expect_tx(&full[s], kStageBytes);    // rows past T arrive as zeros and still count
                uint8_t *dst = stages + s * kStageBytes;
                tma_load_3d(dst, &tmap_x, &full[s], c0, it * kTb, b);
                tma_load_3d(dst + kArrayBytes, &tmap_gx, &full[s], c0, it * kTb, b);
                tma_load_3d(dst + 2 * kArrayBytes, &tmap_ga, &full[s], c0, it * kTb, b);
            }
        }
    } else {
        // ------------------------------------------------------------------ consumer: lane = channel
        const int c = c0 + lane;
        const bool live = c < p.W;
        float h = live ? p.state[(size_t)b * p.W + c] : 0.f;
        // -8 * softplus(a_param), in the log2 domain for ex2
        const float lam = live ? p.a_param[c] : 0.f;
        const float sp = lam > 15.f ? lam : log1pf(expf(lam));
        const float k2 = -8.f * sp * 1.4426950408889634f;
        __nv_bfloat16 *yrow = p.y + (size_t)b * p.T * p.W + c;
        unsigned reset_next = 0u;
        auto resets_of = [&](int it) -> unsigned {
            // bit t: step it*kTb + t is the first token of a segment (position 0)
            if (!p.position) return 0u;
            const int t = it * kTb + lane;
            const int pos = (t < L) ? __ldg(p.position + (size_t)b * p.T + t) : 1;
            return __ballot_sync(0xffffffffu, pos == 0);
        };
        if (n_tiles > 0) reset_next = resets_of(0);
        for (int it = 0; it < n_tiles; ++it) {
            const uint32_t s = it % kStages, ph = (it / kStages) & 1u;
            const unsigned resets = reset_next;
            if (it + 1 < n_tiles) reset_next = resets_of(it + 1);     // in flight while this tile is processed
            if (!mbar_wait(&full[s], ph, abort_flag)) break;
            const unsigned short *xs = reinterpret_cast<const unsigned short *>(stages + s * kStageBytes) + lane;
            const unsigned short *gxs = xs + kTb * kCb, *gas = gxs + kTb * kCb;
            const int t0 = it * kTb;
            const int n = min(kTb, L - t0);
#pragma unroll 4
            for (int t = 0; t < n; ++t) {
                const float xv = bf16_bits_to_float(xs[t * kCb]);
                const float in_gate = sigmoid_fast(bf16_bits_to_float(gxs[t * kCb]));
                const float rec_gate = sigmoid_fast(bf16_bits_to_float(gas[t * kCb]));
                const float la2 = k2 * rec_gate;                       // log2(a)
                float a = fast_exp2(la2);
                // 1 - a^2 = -expm1(z), z = 2 ln a: a short series when a is close to 1, where 1 - a*a cancels
                const float z = la2 * (2.f * 0.6931471805599453f);
                float m2 = (z > -0.0625f) ? -z * fmaf(z, fmaf(z, fmaf(z, 1.f / 24.f, 1.f / 6.f), 0.5f), 1.f)
                                          : fmaf(-a, a, 1.f);
                float m = sqrtf(m2);
                if ((resets >> t) & 1u) {
                    a = 0.f;
                    m = 1.f;
                }
                h = fmaf(a, h, m * in_gate * xv);
                if (live) yrow[(size_t)(t0 + t) * p.W] = __float2bfloat16_rn(h);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[s]);
        }
        if (live) p.state[(size_t)b * p.W + c] = h;
    }
    __syncthreads();
    if (threadIdx.x == 0 && abort_word) atomicOr(p.status + kStatusErrWord, kErrScanWait);
}

}  // namespace

l4l_status launch_rglru_scan(const void *x, const void *gate_x, const void *gate_a, const float *d_a_param,
                             const int32_t *d_position, const int32_t *d_seq_lens, float *d_state, void *y, int B, int T,
                             int W, void *workspace, cudaStream_t stream)
{
    CUtensorMap tx, tgx, tga;
    if (!make_tmap_rows_bf16(&tx, x, W, T, B, W, (int64_t)T * W, kCb, kTb) ||
        !make_tmap_rows_bf16(&tgx, gate_x, W, T, B, W, (int64_t)T * W, kCb, kTb) ||
        !make_tmap_rows_bf16(&tga, gate_a, W, T, B, W, (int64_t)T * W, kCb, kTb))
        return L4L_ERR_CUDA;
    RglruParams p;
    p.a_param = d_a_param; p.position = d_position; p.seq_lens = d_seq_lens; p.state = d_state;
    p.y = static_cast<__nv_bfloat16 *>(y);
    p.status = static_cast<unsigned *>(workspace);
    p.B = B; p.T = T; p.W = W;
    const dim3 grid((W + kCb - 1) / kCb, B);
    rglru_scan_kernel<<<grid, 64, 0, stream>>>(tx, tgx, tga, p);
    return cudaGetLastError() == cudaSuccess ? L4L_OK : L4L_ERR_CUDA;
}

}  // namespace l4l
