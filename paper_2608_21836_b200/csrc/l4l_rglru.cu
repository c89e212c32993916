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
//
// Narrow strips (template parameter kSplit = 2 or 4). A strip is one serial chain, so a launch is as long as the
// most loaded SM's chains: 160 strips on 148 SMs put two on twelve SMs and take twice the time of 148. For such
// launches the strips are made 32 or 16 channels wide, and a warp then owns kSplit CONSECUTIVE time tiles at once:
// lane = (sub-tile, channel pair), so every instruction still does 32 lanes' worth of work. Everything per lane is
// unchanged; the start states of a warp's later sub-tiles come from the earlier ones by kSplit - 1 shuffles
// (h <- A h + E) inside step 3. Twice or four times as many CTAs of half or a quarter of the work spread evenly.
#include <type_traits>

#include "l4l_internal.h"
#include "l4l_ptx.cuh"

namespace l4l {

namespace {

constexpr int kTb = 16;          // time steps per tile
constexpr int kCb = 64;          // channels per CTA at kSplit = 1 (two per lane); kCb / kSplit otherwise
constexpr int kStages = 2;       // TMA buffers per warp
constexpr uint32_t kArrayBytes = kTb * kCb * 2;   // one array of a warp's tile: (kTb * kSplit) steps x (kCb / kSplit) channels
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

template <int kTeam, int kSplit>
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

    constexpr int kCw = kCb / kSplit;                    // channels of this CTA's strip
    constexpr int kPairs = kCw / 2;                      // lanes per sub-tile (one channel pair each)
    constexpr int kSteps = kTb * kSplit;                 // time steps a warp owns at a time (kSplit sub-tiles of kTb)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane / kPairs, cp = lane % kPairs;   // this lane's sub-tile and channel pair
    const int b = blockIdx.y, c0 = blockIdx.x * kCw;
    int L = p.seq_lens ? p.seq_lens[b] : p.T;
    L = L < 0 ? 0 : (L > p.T ? p.T : L);
    const int n_tiles = (L + kSteps - 1) / kSteps;
    const int c = c0 + 2 * cp;
    const bool live = c < p.W;                           // W is even: both channels or neither

    if (threadIdx.x == 0) {
        for (int s = 0; s < kTeam * kStages; ++s) mbar_init(&full[s], 1);
        for (int w = 0; w < kTeam; ++w) mbar_init(&handed[w], 1);
        *abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async_smem();
    }
    if (warp == 0 && sub == 0) {
        const float2 st = live ? *reinterpret_cast<const float2 *>(p.state + (size_t)b * p.W + c) : make_float2(0.f, 0.f);
        *reinterpret_cast<float2 *>(carry + 2 * cp) = st;                      // slot 0: the caller's state starts tile 0
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
            tma_load_3d(dst, &tmap_x, &my_full[s], c0, tile * kSteps, b);
            tma_load_3d(dst + kArrayBytes, &tmap_gx, &my_full[s], c0, tile * kSteps, b);
            tma_load_3d(dst + 2 * kArrayBytes, &tmap_ga, &my_full[s], c0, tile * kSteps, b);
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
        // bit t: step t of THIS LANE'S sub-tile is the first token of a segment (position 0)
        if (!p.position || tile >= n_tiles) return 0u;
        unsigned mine = 0u;
#pragma unroll
        for (int part = 0; part < (kSteps + 31) / 32; ++part) {
            const int t = tile * kSteps + part * 32 + lane;
            const int pos = (part * 32 + lane < kSteps && t < L) ? __ldg(p.position + (size_t)b * p.T + t) : 1;
            const unsigned bits = __ballot_sync(0xffffffffu, pos == 0);
            if ((sub * kTb) / 32 == part) mine = (bits >> ((sub * kTb) % 32)) & 0xffffu;
        }
        return mine;
    };
    unsigned reset_next = resets_of(warp);

    for (int k = 0, tile = warp; tile < n_tiles; ++k, tile += kTeam) {
        const uint32_t s = k % kStages, ph = (k / kStages) & 1u;
        const unsigned resets = reset_next;
        reset_next = resets_of(tile + kTeam);            // in flight while this tile is processed
        if (!mbar_wait(&my_full[s], ph, abort_flag)) break;
        // the tile in shared memory: kSteps rows of kPairs words; this lane reads rows sub * kTb .. of column cp
        const uint32_t *xs = reinterpret_cast<const uint32_t *>(my_stages + s * kStageBytes) + sub * kTb * kPairs + cp;
        const uint32_t *gxs = xs + kTb * kCb / 2, *gas = gxs + kTb * kCb / 2;
        const int t0 = tile * kSteps + sub * kTb;            // first step of this lane's sub-tile
        const int n = max(0, min(kTb, L - t0));
        // ---- a_t and b_t = m_t i_t x_t of all steps of the tile (independent of the state). Tiles without a
        // reset and without a ragged end (nearly all) take the version without the per-step selects.
        uint64_t av[kTb], bv[kTb];
        auto gates = [&](auto plain_tag) {
            constexpr bool kPlain = decltype(plain_tag)::value;
#pragma unroll
            for (int t = 0; t < kTb; ++t) {
                const uint64_t xv = widen2(xs[t * kPairs]);
                float g0, g1, r0, r1;
                unpack_f32x2(mul_f32x2(widen2(gxs[t * kPairs]), half2), g0, g1);
                unpack_f32x2(mul_f32x2(widen2(gas[t * kPairs]), half2), r0, r1);
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
                    if ((resets >> t) & 1u) {                                          // uniform across a sub-tile's lanes
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
        if (__all_sync(0xffffffffu, resets == 0u && n == kTb))
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
        const float2 hs = *reinterpret_cast<const float2 *>(carry + (tile & 1) * kCb + 2 * cp);
        uint64_t h2 = pack_f32x2(hs.x, hs.y);                                  // start state of the warp's first sub-tile
        {
            // start states of the later sub-tiles, and the end state of the warp's steps: h <- A h + E along the
            // sub-tiles, the state travelling kPairs lanes up at each step
            float e0, e1;
            unpack_f32x2(fma_f32x2(A, h2, E), e0, e1);
#pragma unroll
            for (int u = 1; u < kSplit; ++u) {
                const float i0 = __shfl_up_sync(0xffffffffu, e0, kPairs), i1 = __shfl_up_sync(0xffffffffu, e1, kPairs);
                if (sub == u) {
                    h2 = pack_f32x2(i0, i1);
                    unpack_f32x2(fma_f32x2(A, h2, E), e0, e1);
                }
            }
            if (sub == kSplit - 1) *reinterpret_cast<float2 *>(carry + ((tile + 1) & 1) * kCb + 2 * cp) = make_float2(e0, e1);
            __syncwarp();
            if (lane == 0) mbar_arrive(&handed[(warp + 1) % kTeam]);           // release: the slot is written
            if (tile + 1 == n_tiles && live && sub == kSplit - 1)              // the sequence ends here
                *reinterpret_cast<float2 *>(p.state + (size_t)b * p.W + c) = make_float2(e0, e1);
        }
        // ---- the recurrence proper, one packed FMA per step, and the outputs
#pragma unroll
        for (int t = 0; t < kTb; ++t) {
            if (t < n) {                                                       // uniform across a sub-tile's lanes
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

namespace {

template <int kTeam, int kSplit>
l4l_status launch_shape(const void *x, const void *gate_x, const void *gate_a, const RglruParams &p, cudaStream_t stream)
{
    // one opt-in per instantiation and device
    static bool configured_on[kDeviceSlots] = {};
    const int slot = device_slot();
    if (slot < 0) return L4L_ERR_CUDA;
    {
        std::lock_guard<std::mutex> lock(setup_mutex());
        if (!configured_on[slot]) {
            if (cudaFuncSetAttribute(rglru_scan_kernel<kTeam, kSplit>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)smem_bytes(kTeam)) != cudaSuccess)
                return L4L_ERR_CUDA;
            configured_on[slot] = true;
        }
    }
    constexpr int kCw = kCb / kSplit;
    CUtensorMap tx, tgx, tga;
    if (!make_tmap_rows_bf16(&tx, x, p.W, p.T, p.B, p.W, (int64_t)p.T * p.W, kCw, kTb * kSplit) ||
        !make_tmap_rows_bf16(&tgx, gate_x, p.W, p.T, p.B, p.W, (int64_t)p.T * p.W, kCw, kTb * kSplit) ||
        !make_tmap_rows_bf16(&tga, gate_a, p.W, p.T, p.B, p.W, (int64_t)p.T * p.W, kCw, kTb * kSplit))
        return L4L_ERR_CUDA;
    const dim3 grid((p.W + kCw - 1) / kCw, p.B);
    rglru_scan_kernel<kTeam, kSplit><<<grid, kTeam * 32, smem_bytes(kTeam), stream>>>(tx, tgx, tga, p);
    return cudaGetLastError() == cudaSuccess ? L4L_OK : L4L_ERR_CUDA;
}

}  // namespace

l4l_status launch_rglru_scan(const void *x, const void *gate_x, const void *gate_a, const float *d_a_param,
                             const int32_t *d_position, const int32_t *d_seq_lens, float *d_state, void *y, int B, int T,
                             int W, void *workspace, size_t, cudaStream_t stream)
{
    RglruParams p;
    p.a_param = d_a_param; p.position = d_position; p.seq_lens = d_seq_lens; p.state = d_state;
    p.y = static_cast<__nv_bfloat16 *>(y);
    p.status = static_cast<unsigned *>(workspace);
    p.B = B; p.T = T; p.W = W;
    if (T <= kTb) return launch_shape<1, 1>(x, gate_x, gate_a, p, stream);
    const int split = rglru_strip_split(B, T, W);
    if (split == 0) return launch_shape<16, 1>(x, gate_x, gate_a, p, stream);
    if (split == 4) return launch_shape<8, 4>(x, gate_x, gate_a, p, stream);
    if (split == 2) return launch_shape<8, 2>(x, gate_x, gate_a, p, stream);
    return launch_shape<8, 1>(x, gate_x, gate_a, p, stream);
}

// 0: 64-channel strips with teams of 16 warps; 1, 2, 4: teams of 8 warps on strips of 64, 32, 16 channels.
int rglru_strip_split(int B, int T, int W)
{
    if (T <= kTb) return 1;
    const long long sms = sm_count();
    // A strip is a serial chain that keeps an SM's issue slots busy, so a launch takes as long as the most loaded
    // SM. Estimated time of that SM, in units of one 64-channel strip on an SM of its own: k CTAs of 1/s strip each
    // take k / s; a lone team of 8 warps reaches about three quarters of the issue rate that two co-resident teams
    // or one team of 16 warps reach.
    auto fullest = [&](int s) { return ((long long)((W + kCb / s - 1) / (kCb / s)) * B + sms - 1) / sms; };
    int best = 1;
    double best_time = fullest(1) >= 2 ? (double)fullest(1) : 1.0 / 0.74;
    if (fullest(1) == 1 && T >= 16 * 2 * kTb) {
        best = 0;
        best_time = 1.0;
    }
    // narrower strips have to win by a tenth or more (their warps pay two or four dependent steps in the hand-off
    // instead of one), and the sequence has to be long enough for their wider tiles
    for (int s = 2; s <= 4; s *= 2) {
        const long long k = fullest(s);
        const double time = k >= 2 ? (double)k / s : (1.0 / s) / 0.74;
        if (time < 0.9 * best_time && T >= 8 * kTb * s) {
            best = s;
            best_time = time;
        }
    }
    return best;
}

}  // namespace l4l
