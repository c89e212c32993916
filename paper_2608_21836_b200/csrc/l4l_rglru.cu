// Gated linear recurrence of the RecurrentGemma block (RG-LRU): gates, normalisation, reset handling and
// the scan over the sequence in one kernel and one pass over the data; the state is handed from tile to
// tile on chip and written once at the end.
//
// The recurrence is sequential in time and independent across (sequence, channel). A CTA owns 64 channels
// of one sequence (two per lane, packed fp32x2 arithmetic) and walks the time axis in tiles of 16 steps,
// its 8 warps taking the tiles in turn (warp w: tiles w, w + 8, ...; a single warp when there is only one tile). Per tile a warp
//   1. has the tile's x, gate_x and gate_a in shared memory (its own TMA double buffer: as soon as a tile's
//      values are in registers the buffer is refilled with the warp's tile after next),
//   2. evaluates a_t and b_t of all 16 steps (independent of the state, so MUFU and FMA latencies overlap)
//      and, by linearity, the tile's aggregate: A = prod a_t and E = the end state from a zero start,
//   3. waits for the state at the start of the tile from the warp that owns the previous tile (shared
//      memory), hands A h + E on to the next warp at once,
//   4. and only then runs the recurrence proper from its start state and stores y.
// Only step 3 is serial along the sequence (a hand-off of 64 floats through shared memory per 16 steps);
// everything else runs 8 tiles at a time, which is what lets ONE sequence of 64 channels stream at a
// rate near an SM's share of HBM instead of at the latency of one warp.
// 8 bytes per (step, channel) move through HBM (3 bf16 read, 1 written) against 4 MUFU operations per
// channel (two tanh.approx sigmoids, ex2.approx, sqrt.approx) and about 25 issued instructions per channel
// pair and step.
#include <type_traits>

#include "l4l_internal.h"
#include "l4l_ptx.cuh"

namespace l4l {

namespace {

constexpr int kTb = 16;          // time steps per tile
constexpr int kCb = 64;          // channels per CTA (two per lane)
constexpr int kStages = 2;       // TMA buffers per warp
constexpr uint32_t kArrayBytes = kTb * kCb * 2;
constexpr uint32_t kStageBytes = 3 * kArrayBytes;
// kTeam warps per CTA, each taking every kTeam-th tile: 8 for sequences, 16 when the launch has no more strips
// than the GPU has SMs (one CTA per SM then, and a strip's rate is set by how many tiles it has in flight),
// 1 for a single tile (decode steps)
constexpr size_t smem_bytes(int team)
{
    return 128 + (size_t)team * kStages * kStageBytes + (team * kStages + team) * 8 + 2 * kCb * 4 + 64;
}

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

__device__ __forceinline__ float sqrt_approx(float x)
{
    float y;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// two bf16 in one word -> packed fp32x2 (low half first)
__device__ __forceinline__ uint64_t widen2(uint32_t w) { return pack_u32x2(w << 16, w & 0xffff0000u); }

template <int kTeam>
__global__ void __launch_bounds__(kTeam * 32)
rglru_scan_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_gx,
                  const __grid_constant__ CUtensorMap tmap_ga, const RglruParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u);
    uint8_t *stages = smem;                                                    // [warp][stage][3 arrays]
    uint64_t *full = reinterpret_cast<uint64_t *>(stages + (size_t)kTeam * kStages * kStageBytes);   // [warp][stage]
    uint64_t *handed = full + kTeam * kStages;                                 // [warp]: the start state of its next tile is there
    float *carry = reinterpret_cast<float *>(handed + kTeam);                  // [2][kCb]: start state of tile j in slot j & 1
    volatile int *abort_flag = reinterpret_cast<volatile int *>(carry + 2 * kCb);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.y, c0 = blockIdx.x * kCb;
    int L = p.seq_lens ? p.seq_lens[b] : p.T;
    L = L < 0 ? 0 : (L > p.T ? p.T : L);
    const int n_tiles = (L + kTb - 1) / kTb;
    const int c = c0 + 2 * lane;
    const bool live = c < p.W;                           // W is even: both channels or neither

    if (threadIdx.x == 0) {
        for (int s = 0; s < kTeam * kStages; ++s) mbar_init(&full[s], 1);
        for (int w = 0; w < kTeam; ++w) mbar_init(&handed[w], 1);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
    }
    if (warp == 0) {
        const float2 st = live ? *reinterpret_cast<const float2 *>(p.state + (size_t)b * p.W + c) : make_float2(0.f, 0.f);
        *reinterpret_cast<float2 *>(carry + 2 * lane) = st;                    // slot 0: the caller's state starts tile 0
    }
    __syncthreads();
    if (threadIdx.x == 0) mbar_arrive(&handed[0]);

    uint8_t *my_stages = stages + (size_t)warp * kStages * kStageBytes;
    uint64_t *my_full = full + warp * kStages;
    // lane 0 requests this warp's k-th tile (tile warp + k * kTeam) into its buffer k % kStages
    // (rows past T arrive as zeros and still count)
    auto request = [&](int k) {
        const int tile = warp + k * kTeam;
        if (lane == 0 && tile < n_tiles) {
            const uint32_t s = k % kStages;
            mbar_arrive_expect_tx(&my_full[s], kStageBytes);
            uint8_t *dst = my_stages + s * kStageBytes;
            tma_load_3d(dst, &tmap_x, &my_full[s], c0, tile * kTb, b);
            tma_load_3d(dst + kArrayBytes, &tmap_gx, &my_full[s], c0, tile * kTb, b);
            tma_load_3d(dst + 2 * kArrayBytes, &tmap_ga, &my_full[s], c0, tile * kTb, b);
        }
    };
    if (lane == 0) {
        tma_prefetch_desc(&tmap_x);
        tma_prefetch_desc(&tmap_gx);
        tma_prefetch_desc(&tmap_ga);
    }
    for (int k = 0; k < kStages; ++k) request(k);

    uint64_t k2 = pack_f32x2(0.f, 0.f);                  // -8 softplus(a_param) log2(e), per channel
    if (live) {
        const float2 lam = *reinterpret_cast<const float2 *>(p.a_param + c);
        const float sp0 = lam.x > 15.f ? lam.x : log1pf(expf(lam.x));
        const float sp1 = lam.y > 15.f ? lam.y : log1pf(expf(lam.y));
        k2 = pack_f32x2(-8.f * 1.4426950408889634f * sp0, -8.f * 1.4426950408889634f * sp1);
    }
    const uint64_t half2 = pack_f32x2(0.5f, 0.5f), one2 = pack_f32x2(1.f, 1.f), zero2 = pack_f32x2(0.f, 0.f);
    const uint64_t k2h = mul_f32x2(k2, half2);
    const uint64_t two_ln2 = pack_f32x2(1.3862943611198906f, 1.3862943611198906f);
    const uint64_t nc24 = pack_f32x2(-1.f / 24.f, -1.f / 24.f), nc6 = pack_f32x2(-1.f / 6.f, -1.f / 6.f);
    const uint64_t nhalf2 = pack_f32x2(-0.5f, -0.5f), neg1 = pack_f32x2(-1.f, -1.f);
    uint32_t *yrow = reinterpret_cast<uint32_t *>(p.y + (size_t)b * p.T * p.W + c);
    const size_t y_step = (size_t)p.W / 2;               // 32-bit words between time steps
    auto resets_of = [&](int tile) -> unsigned {
        // bit t: step tile*kTb + t is the first token of a segment (position 0)
        if (!p.position || tile >= n_tiles) return 0u;
        const int t = tile * kTb + lane;
        const int pos = (lane < kTb && t < L) ? __ldg(p.position + (size_t)b * p.T + t) : 1;
        return __ballot_sync(0xffffffffu, pos == 0);
    };
    unsigned reset_next = resets_of(warp);

    for (int k = 0, tile = warp; tile < n_tiles; ++k, tile += kTeam) {
        const uint32_t s = k % kStages, ph = (k / kStages) & 1u;
        const unsigned resets = reset_next;
        reset_next = resets_of(tile + kTeam);            // in flight while this tile is processed
        if (!mbar_wait(&my_full[s], ph, abort_flag)) break;
        const uint32_t *xs = reinterpret_cast<const uint32_t *>(my_stages + s * kStageBytes) + lane;
        const uint32_t *gxs = xs + kTb * kCb / 2, *gas = gxs + kTb * kCb / 2;
        const int t0 = tile * kTb;
        const int n = min(kTb, L - t0);
        // ---- a_t and b_t = m_t i_t x_t of all steps of the tile (independent of the state). Tiles without a
        // reset and without a ragged end (nearly all) take the version without the per-step selects.
        uint64_t av[kTb], bv[kTb];
        auto gates = [&](auto plain_tag) {
            constexpr bool kPlain = decltype(plain_tag)::value;
#pragma unroll
            for (int t = 0; t < kTb; ++t) {
                const uint64_t xv = widen2(xs[t * (kCb / 2)]);
                float g0, g1, r0, r1;
                unpack_f32x2(mul_f32x2(widen2(gxs[t * (kCb / 2)]), half2), g0, g1);
                unpack_f32x2(mul_f32x2(widen2(gas[t * (kCb / 2)]), half2), r0, r1);
                const uint64_t th_x = pack_f32x2(tanh_approx(g0), tanh_approx(g1));   // sigmoid = 0.5 tanh(z/2) + 0.5
                const uint64_t th_a = pack_f32x2(tanh_approx(r0), tanh_approx(r1));
                const uint64_t la2 = fma_f32x2(th_a, k2h, k2h);                        // log2(a) = k2 * sigmoid(gate_a)
                float l0, l1;
                unpack_f32x2(la2, l0, l1);
                uint64_t a = pack_f32x2(fast_exp2(l0), fast_exp2(l1));
                // 1 - a^2 = -expm1(z), z = 2 ln a: a short series when a is close to 1, where 1 - a*a cancels
                const uint64_t z = mul_f32x2(la2, two_ln2);
                const uint64_t npoly = fma_f32x2(z, fma_f32x2(z, fma_f32x2(z, nc24, nc6), nhalf2), neg1);
                float s0, s1, d0, d1, z0, z1;
                unpack_f32x2(mul_f32x2(z, npoly), s0, s1);
                unpack_f32x2(fma_f32x2(mul_f32x2(a, neg1), a, one2), d0, d1);
                unpack_f32x2(z, z0, z1);
                float m0 = sqrt_approx(z0 > -0.0625f ? s0 : d0), m1 = sqrt_approx(z1 > -0.0625f ? s1 : d1);
                if constexpr (!kPlain) {
                    if ((resets >> t) & 1u) {                                          // uniform across the warp
                        a = zero2;
                        m0 = m1 = 1.f;
                    }
                    if (t >= n) {                                                      // past the end: the identity step
                        a = one2;
                        m0 = m1 = 0.f;
                    }
                }
                av[t] = a;
                const uint64_t mxh = mul_f32x2(mul_f32x2(pack_f32x2(m0, m1), half2), xv);   // m x / 2
                bv[t] = fma_f32x2(th_x, mxh, mxh);                                         // m x sigmoid(gate_x)
                if constexpr (!kPlain) {
                    // rows past the end are caller memory that may hold anything (0 * NaN is NaN): select, not multiply
                    if (t >= n) bv[t] = zero2;
                }
            }
        };
        if (resets == 0u && n == kTb)
            gates(std::true_type{});
        else
            gates(std::false_type{});
        // every lane has its values of this tile in registers: the buffer can take this warp's tile after next
        __syncwarp();
        request(k + kStages);
        // ---- the tile's aggregate: h_end = A h_start + E
        uint64_t A = one2, E = zero2;
#pragma unroll
        for (int t = 0; t < kTb; ++t) {
            E = fma_f32x2(av[t], E, bv[t]);
            A = mul_f32x2(A, av[t]);
        }
        // ---- the start state, from the owner of the previous tile (bounded wait); pass the end state on at once.
        // Every warp has its own barrier, completed once per tile it owns by the owner of the tile before; that
        // warp cannot reach its next arrival here before this warp has handed the present tile on, so the
        // phases are seen one by one.
        if (!mbar_wait(&handed[warp], k & 1u, abort_flag)) break;
        const float2 hs = *reinterpret_cast<const float2 *>(carry + (tile & 1) * kCb + 2 * lane);
        uint64_t h2 = pack_f32x2(hs.x, hs.y);
        {
            float e0, e1;
            unpack_f32x2(fma_f32x2(A, h2, E), e0, e1);
            *reinterpret_cast<float2 *>(carry + ((tile + 1) & 1) * kCb + 2 * lane) = make_float2(e0, e1);
            __syncwarp();
            if (lane == 0) mbar_arrive(&handed[(warp + 1) % kTeam]);           // release: the slot is written
            if (tile + 1 == n_tiles && live)                                   // the sequence ends here
                *reinterpret_cast<float2 *>(p.state + (size_t)b * p.W + c) = make_float2(e0, e1);
        }
        // ---- the recurrence proper, one packed FMA per step, and the outputs
#pragma unroll
        for (int t = 0; t < kTb; ++t) {
            if (t < n) {                                                       // uniform across the warp
                h2 = fma_f32x2(av[t], h2, bv[t]);
                float h0, h1;
                unpack_f32x2(h2, h0, h1);
                if (live) yrow[(size_t)(t0 + t) * y_step] = pack_bf16x2(h0, h1);
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.status + kStatusErrWord, kErrScanWait);
}

}  // namespace

size_t rglru_workspace_bytes(int, int, int) { return kStatusBytes; }

l4l_status launch_rglru_scan(const void *x, const void *gate_x, const void *gate_a, const float *d_a_param,
                             const int32_t *d_position, const int32_t *d_seq_lens, float *d_state, void *y, int B, int T,
                             int W, void *workspace, size_t, cudaStream_t stream)
{
    CUtensorMap tx, tgx, tga;
    if (!make_tmap_rows_bf16(&tx, x, W, T, B, W, (int64_t)T * W, kCb, kTb) ||
        !make_tmap_rows_bf16(&tgx, gate_x, W, T, B, W, (int64_t)T * W, kCb, kTb) ||
        !make_tmap_rows_bf16(&tga, gate_a, W, T, B, W, (int64_t)T * W, kCb, kTb))
        return L4L_ERR_CUDA;
    static bool configured_on[kDeviceSlots] = {};
    static int sm_count_on[kDeviceSlots] = {};
    const int slot = device_slot();
    if (slot < 0) return L4L_ERR_CUDA;
    int sm_count;
    {
        std::lock_guard<std::mutex> lock(setup_mutex());
        bool &configured = configured_on[slot];
        if (!configured) {
            if (cudaDeviceGetAttribute(&sm_count_on[slot], cudaDevAttrMultiProcessorCount, slot) != cudaSuccess ||
                cudaFuncSetAttribute(rglru_scan_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)smem_bytes(8)) != cudaSuccess ||
                cudaFuncSetAttribute(rglru_scan_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)smem_bytes(16)) != cudaSuccess)
                return L4L_ERR_CUDA;
            configured = true;
        }
        sm_count = sm_count_on[slot];
    }
    RglruParams p;
    p.a_param = d_a_param; p.position = d_position; p.seq_lens = d_seq_lens; p.state = d_state;
    p.y = static_cast<__nv_bfloat16 *>(y);
    p.status = static_cast<unsigned *>(workspace);
    p.B = B; p.T = T; p.W = W;
    const dim3 grid((W + kCb - 1) / kCb, B);
    if (T <= kTb)
        rglru_scan_kernel<1><<<grid, 32, smem_bytes(1), stream>>>(tx, tgx, tga, p);
    else if ((long long)grid.x * grid.y <= sm_count && T >= 16 * 2 * kTb)
        rglru_scan_kernel<16><<<grid, 16 * 32, smem_bytes(16), stream>>>(tx, tgx, tga, p);
    else
        rglru_scan_kernel<8><<<grid, 8 * 32, smem_bytes(8), stream>>>(tx, tgx, tga, p);
    return cudaGetLastError() == cudaSuccess ? L4L_OK : L4L_ERR_CUDA;
}

}  // namespace l4l
