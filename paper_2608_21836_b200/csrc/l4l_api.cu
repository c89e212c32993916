// C-ABI entry points: host-side validation, workspace sizing, tensor-map construction.
// Nothing here touches the data path; every operation runs in the kernels of the other
// translation units.
#include <atomic>
#include <cstdlib>
#include <mutex>

#include "l4l_internal.h"
#include "l4l_ptx.cuh"

namespace l4l {

namespace {

using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    });
    return fn;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool stride_ok(int64_t s) { return s >= 0 && (s % 8) == 0; }

bool tensor4_ok(const l4l_tensor4 &t)
{
    return t.ptr && aligned16(t.ptr) && stride_ok(t.stride_b) && stride_ok(t.stride_t) && stride_ok(t.stride_h);
}

bool cache_ok(const l4l_kv_cache &c)
{
    return c.k && c.v && aligned16(c.k) && aligned16(c.v) && stride_ok(c.stride_b) && stride_ok(c.stride_h) &&
           stride_ok(c.stride_t) && c.max_len > 0;
}

l4l_status shape_status(int B, int Hq, int Hkv, int D)
{
    if (B < 0 || Hq <= 0 || Hkv <= 0) return L4L_ERR_INVALID_ARG;
    if (D != 64 && D != 128) return L4L_ERR_UNSUPPORTED;
    if (Hq % Hkv != 0 || Hq / Hkv > 16) return L4L_ERR_UNSUPPORTED;
    return L4L_OK;
}

}  // namespace

int sm_count()
{
    // per device: one process may drive GPUs that differ in SM count (or in how they are partitioned)
    static std::atomic<int> n_on[kDeviceSlots];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kDeviceSlots) {
        (void)cudaGetLastError();
        return 148;
    }
    int n = n_on[dev].load(std::memory_order_relaxed);
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
            (void)cudaGetLastError();
            n = 148;
        }
        n_on[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}

std::mutex &setup_mutex()
{
    static std::mutex m;
    return m;
}

namespace {

std::atomic<int> g_override_cluster{-1}, g_override_warp{-1}, g_override_split_warps{0};

// The environment is read once, when the library is loaded.
const bool g_override_seeded = [] {
    if (const char *e = getenv("L4L_DECODE_CLUSTER")) g_override_cluster = atoi(e);
    if (const char *e = getenv("L4L_DECODE_WARP")) g_override_warp = (e[0] != '0') ? 1 : 0;
    if (const char *e = getenv("L4L_DECODE_WARPS")) g_override_split_warps = atoi(e);
    return true;
}();

}  // namespace

DecodeOverride decode_override()
{
    return DecodeOverride{g_override_cluster.load(std::memory_order_relaxed), g_override_warp.load(std::memory_order_relaxed),
                          g_override_split_warps.load(std::memory_order_relaxed)};
}

namespace {

// A serving loop calls with the same buffers step after step: remember the last few encoded maps
// (a tensor map is a pure function of these arguments; it encodes an address and a layout, nothing of the
// device, and under unified addressing an address names one device's memory, so the key needs no device).
struct TmapKey {
    const void *base;
    int D, box_d, box_t, elem_bytes;
    int64_t n_t, n_h, n_b, stride_t, stride_h, stride_b;
    bool operator==(const TmapKey &o) const
    {
        return base == o.base && D == o.D && elem_bytes == o.elem_bytes && box_d == o.box_d && box_t == o.box_t && n_t == o.n_t && n_h == o.n_h &&
               n_b == o.n_b && stride_t == o.stride_t && stride_h == o.stride_h && stride_b == o.stride_b;
    }
};
struct TmapEntry {
    TmapKey key;
    CUtensorMap map;
    TmapCoord coord;
    bool valid = false;
};
constexpr int kTmapCache = 32;
TmapEntry g_tmap_cache[kTmapCache];
int g_tmap_next = 0;
std::mutex g_tmap_mutex;

bool encode_tmap(CUtensorMap *out, TmapCoord *coord, const void *base, int D, int64_t n_t, int64_t n_h, int64_t n_b,
                 int64_t stride_t, int64_t stride_h, int64_t stride_b, int box_d, int box_t, int elem_bytes);

}  // namespace

bool make_tmap_rows_bf16(CUtensorMap *out, const void *base, int64_t n_cols, int64_t n_rows, int64_t n_outer,
                         int64_t stride_row, int64_t stride_outer, int box_cols, int box_rows)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t gdim[3] = {(cuuint64_t)n_cols, (cuuint64_t)(n_rows < 1 ? 1 : n_rows), (cuuint64_t)(n_outer < 1 ? 1 : n_outer)};
    cuuint64_t gstride[2] = {(cuuint64_t)stride_row * 2, (cuuint64_t)stride_outer * 2};
    if (gstride[1] < gstride[0] * gdim[1]) gstride[1] = gstride[0] * gdim[1];      // extent-1 outer dimension
    cuuint32_t box[3] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), gdim, gstride, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_tmap(CUtensorMap *out, TmapCoord *coord, const void *base, int D, int64_t n_t, int64_t n_h, int64_t n_b,
               int64_t stride_t, int64_t stride_h, int64_t stride_b, int box_d, int box_t, int elem_bytes)
{
    const TmapKey key{base, D, box_d, box_t, elem_bytes, n_t, n_h, n_b, stride_t, stride_h, stride_b};
    {
        std::lock_guard<std::mutex> lock(g_tmap_mutex);
        for (int i = 0; i < kTmapCache; ++i)
            if (g_tmap_cache[i].valid && g_tmap_cache[i].key == key) {
                *out = g_tmap_cache[i].map;
                *coord = g_tmap_cache[i].coord;
                return true;
            }
    }
    if (!encode_tmap(out, coord, base, D, n_t, n_h, n_b, stride_t, stride_h, stride_b, box_d, box_t, elem_bytes))
        return false;
    std::lock_guard<std::mutex> lock(g_tmap_mutex);
    TmapEntry &e = g_tmap_cache[g_tmap_next];
    g_tmap_next = (g_tmap_next + 1) % kTmapCache;
    e.key = key; e.map = *out; e.coord = *coord; e.valid = true;
    return true;
}

namespace {

bool encode_tmap(CUtensorMap *out, TmapCoord *coord, const void *base, int D, int64_t n_t, int64_t n_h, int64_t n_b,
                 int64_t stride_t, int64_t stride_h, int64_t stride_b, int box_d, int box_t, int elem_bytes)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    // order the three outer dimensions by ascending stride (extent-1 dimensions last)
    struct Dim { int64_t n, stride; int which; int box; };
    Dim dims[3] = {{n_t, stride_t, 0, box_t}, {n_h, stride_h, 1, 1}, {n_b, stride_b, 2, 1}};
    auto key = [](const Dim &d) { return d.n <= 1 ? INT64_MAX : d.stride; };
    for (int i = 0; i < 3; ++i)
        for (int j = i + 1; j < 3; ++j)
            if (key(dims[j]) < key(dims[i])) { Dim t = dims[i]; dims[i] = dims[j]; dims[j] = t; }
    cuuint64_t gdim[4] = {(cuuint64_t)D, 0, 0, 0};
    cuuint64_t gstride[3];
    cuuint32_t box[4] = {(cuuint32_t)box_d, 1, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    int64_t prev_extent_bytes = (int64_t)D * elem_bytes;
    for (int i = 0; i < 3; ++i) {
        gdim[i + 1] = (cuuint64_t)(dims[i].n < 1 ? 1 : dims[i].n);
        int64_t sb = dims[i].stride * elem_bytes;
        if (dims[i].n <= 1 && sb < prev_extent_bytes) sb = prev_extent_bytes;   // never used for addressing
        gstride[i] = (cuuint64_t)sb;
        prev_extent_bytes = sb * (int64_t)gdim[i + 1];
        box[i + 1] = (cuuint32_t)dims[i].box;
        if (dims[i].which == 0) coord->pos_t = i + 1;
        if (dims[i].which == 1) coord->pos_h = i + 1;
        if (dims[i].which == 2) coord->pos_b = i + 1;
    }
    CUresult r = fn(out, elem_bytes == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), gdim, gstride, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

}  // namespace

}  // namespace l4l

using namespace l4l;

extern "C" {

const char *l4l_version(void) { return "0.1"; }

const char *l4l_status_string(l4l_status s)
{
    switch (s) {
        case L4L_OK: return "ok";
        case L4L_ERR_INVALID_ARG: return "invalid argument";
        case L4L_ERR_UNSUPPORTED: return "unsupported shape";
        case L4L_ERR_WORKSPACE: return "workspace missing or too small";
        case L4L_ERR_CUDA: return "CUDA call failed";
        case L4L_ERR_TIMEOUT: return "bounded device-side wait ran out";
    }
    return "unknown status";
}

size_t l4l_workspace_bytes(int op, int B, int Hq, int Hkv, int head_dim, int max_len)
{
    if (shape_status(B, Hq, Hkv, head_dim) != L4L_OK || max_len < 0) return 0;
    if (op == L4L_OP_PREFILL) return kStatusBytes;
    if (op == L4L_OP_DECODE) {
        // the contiguous and the paged entry points may pick different kernel shapes: enough for either
        const size_t a = plan_decode(B, Hq, Hkv, head_dim, max_len, (size_t)-1, false, 0).ws_bytes;
        const size_t b = plan_decode(B, Hq, Hkv, head_dim, max_len, (size_t)-1, false, 64).ws_bytes;
        return a > b ? a : b;
    }
    return 0;
}

l4l_status l4l_workspace_init(void *workspace, size_t ws_bytes, l4l_stream stream)
{
    if (!workspace || ws_bytes < kStatusBytes) return L4L_ERR_WORKSPACE;
    return cudaMemsetAsync(workspace, 0, ws_bytes, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? L4L_OK
               : L4L_ERR_CUDA;
}

int l4l_last_device_error(void *workspace, l4l_stream stream)
{
    if (!workspace) return -1;
    unsigned words[2] = {0, 0};
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(words, workspace, sizeof(words), cudaMemcpyDeviceToHost, s) != cudaSuccess) return -1;
    if (cudaStreamSynchronize(s) != cudaSuccess) return -1;
    return (int)words[kStatusErrWord];
}

l4l_status l4l_kv_append(l4l_kv_cache cache, l4l_tensor4 k_new, l4l_tensor4 v_new, const int32_t *d_write_pos,
                         const int32_t *d_n_new, int n_new_max, int B, int Hkv, int head_dim, l4l_stream stream)
{
    if (B < 0 || Hkv <= 0 || n_new_max < 0) return L4L_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return L4L_ERR_UNSUPPORTED;
    if (!cache_ok(cache) || !tensor4_ok(k_new) || !tensor4_ok(v_new) || !d_write_pos) return L4L_ERR_INVALID_ARG;
    if (B == 0 || n_new_max == 0) return L4L_OK;
    return launch_kv_append(cache, k_new, v_new, d_write_pos, d_n_new, n_new_max, B, Hkv, head_dim,
                            static_cast<cudaStream_t>(stream));
}

namespace {

// A page pool is valid if a page size is a power of two >= 16 (tiles are fetched in 16-token groups).
bool pool_ok(const l4l_paged_kv &pool)
{
    return pool.k && pool.v && aligned16(pool.k) && aligned16(pool.v) && stride_ok(pool.stride_page) &&
           stride_ok(pool.stride_h) && stride_ok(pool.stride_t) && pool.num_pages > 0 && pool.page_size >= 16 &&
           pool.page_size <= (1 << 20) && (pool.page_size & (pool.page_size - 1)) == 0;
}

l4l_kv_cache pool_as_cache(const l4l_paged_kv &pool)
{
    l4l_kv_cache c;
    c.k = pool.k; c.v = pool.v;
    c.stride_b = pool.stride_page; c.stride_h = pool.stride_h; c.stride_t = pool.stride_t;
    c.max_len = pool.page_size;
    return c;
}

}  // namespace

l4l_status l4l_kv_append_paged(l4l_paged_kv pool, const int32_t *d_block_table, int table_stride, l4l_tensor4 k_new,
                               l4l_tensor4 v_new, const int32_t *d_write_pos, const int32_t *d_n_new, int n_new_max,
                               int B, int Hkv, int head_dim, l4l_stream stream)
{
    if (B < 0 || Hkv <= 0 || n_new_max < 0 || table_stride <= 0) return L4L_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return L4L_ERR_UNSUPPORTED;
    if (!pool_ok(pool) || !tensor4_ok(k_new) || !tensor4_ok(v_new) || !d_write_pos || !d_block_table)
        return L4L_ERR_INVALID_ARG;
    if (B == 0 || n_new_max == 0) return L4L_OK;
    const PagedTable pt{d_block_table, table_stride, pool.num_pages};
    return launch_kv_append(pool_as_cache(pool), k_new, v_new, d_write_pos, d_n_new, n_new_max, B, Hkv, head_dim,
                            static_cast<cudaStream_t>(stream), &pt);
}

l4l_status l4l_attn_decode_paged(const void *q, void *o, l4l_paged_kv pool, const int32_t *d_block_table,
                                 int table_stride, const int32_t *d_kv_lens, int max_kv_len, int B, int Hq, int Hkv,
                                 int head_dim, float scale, float *d_lse, void *workspace, size_t ws_bytes,
                                 l4l_stream stream)
{
    l4l_status st = shape_status(B, Hq, Hkv, head_dim);
    if (st != L4L_OK) return st;
    if (!q || !o || !d_kv_lens || !d_block_table || !aligned16(q) || !aligned16(o)) return L4L_ERR_INVALID_ARG;
    if (!pool_ok(pool) || table_stride <= 0) return L4L_ERR_INVALID_ARG;
    if (max_kv_len < 0 || (long long)max_kv_len > (long long)table_stride * pool.page_size) return L4L_ERR_INVALID_ARG;
    if (!workspace || ws_bytes < kStatusBytes) return L4L_ERR_WORKSPACE;
    if (B == 0) return L4L_OK;
    const DecodePlan plan = plan_decode(B, Hq, Hkv, head_dim, max_kv_len, ws_bytes, false, pool.page_size);
    if (plan.ws_bytes > ws_bytes) return L4L_ERR_WORKSPACE;
    const PagedTable pt{d_block_table, table_stride, pool.num_pages};
    return launch_decode(q, o, pool_as_cache(pool), d_kv_lens, max_kv_len, B, Hq, Hkv, head_dim, scale, d_lse, workspace,
                         plan, static_cast<cudaStream_t>(stream), nullptr, nullptr, &pt);
}

l4l_status l4l_attn_decode_paged_append(const void *q, void *o, l4l_paged_kv pool, const int32_t *d_block_table,
                                        int table_stride, l4l_tensor4 k_new, l4l_tensor4 v_new,
                                        const int32_t *d_kv_lens, int max_kv_len, int B, int Hq, int Hkv, int head_dim,
                                        float scale, float *d_lse, void *workspace, size_t ws_bytes, l4l_stream stream)
{
    l4l_status st = shape_status(B, Hq, Hkv, head_dim);
    if (st != L4L_OK) return st;
    if (!q || !o || !d_kv_lens || !d_block_table || !aligned16(q) || !aligned16(o)) return L4L_ERR_INVALID_ARG;
    if (!pool_ok(pool) || table_stride <= 0) return L4L_ERR_INVALID_ARG;
    if (!tensor4_ok(k_new) || !tensor4_ok(v_new)) return L4L_ERR_INVALID_ARG;
    if (max_kv_len < 0 || (long long)max_kv_len > (long long)table_stride * pool.page_size) return L4L_ERR_INVALID_ARG;
    if (!workspace || ws_bytes < kStatusBytes) return L4L_ERR_WORKSPACE;
    if (B == 0) return L4L_OK;
    const DecodePlan plan = plan_decode(B, Hq, Hkv, head_dim, max_kv_len, ws_bytes, false, pool.page_size);
    if (plan.ws_bytes > ws_bytes) return L4L_ERR_WORKSPACE;
    const PagedTable pt{d_block_table, table_stride, pool.num_pages};
    return launch_decode(q, o, pool_as_cache(pool), d_kv_lens, max_kv_len, B, Hq, Hkv, head_dim, scale, d_lse, workspace,
                         plan, static_cast<cudaStream_t>(stream), &k_new, &v_new, &pt);
}

namespace {

// An fp8 cache: byte elements, every row start 16-byte aligned.
bool cache8_ok(const l4l_kv_cache &c)
{
    auto s16 = [](int64_t s) { return s >= 0 && (s % 16) == 0; };
    return c.k && c.v && aligned16(c.k) && aligned16(c.v) && s16(c.stride_b) && s16(c.stride_h) && s16(c.stride_t) &&
           c.max_len > 0;
}

}  // namespace

l4l_status l4l_kv_append_fp8(l4l_kv_cache cache8, l4l_tensor4 k_new, l4l_tensor4 v_new, const int32_t *d_write_pos,
                             const int32_t *d_n_new, int n_new_max, int B, int Hkv, int head_dim,
                             const float *d_k_scale, const float *d_v_scale, l4l_stream stream)
{
    if (B < 0 || Hkv <= 0 || n_new_max < 0) return L4L_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return L4L_ERR_UNSUPPORTED;
    if (!cache8_ok(cache8) || !tensor4_ok(k_new) || !tensor4_ok(v_new) || !d_write_pos || !d_k_scale || !d_v_scale)
        return L4L_ERR_INVALID_ARG;
    if (B == 0 || n_new_max == 0) return L4L_OK;
    return launch_kv_append_fp8(cache8, k_new, v_new, d_write_pos, d_n_new, n_new_max, B, Hkv, head_dim, d_k_scale,
                                d_v_scale, static_cast<cudaStream_t>(stream));
}

l4l_status l4l_attn_decode_fp8(const void *q, void *o, l4l_kv_cache cache8, const float *d_k_scale,
                               const float *d_v_scale, const int32_t *d_kv_lens, int max_kv_len, int B, int Hq, int Hkv,
                               int head_dim, float scale, float *d_lse, void *workspace, size_t ws_bytes,
                               l4l_stream stream)
{
    l4l_status st = shape_status(B, Hq, Hkv, head_dim);
    if (st != L4L_OK) return st;
    if (!q || !o || !d_kv_lens || !d_k_scale || !d_v_scale || !aligned16(q) || !aligned16(o)) return L4L_ERR_INVALID_ARG;
    if (!cache8_ok(cache8)) return L4L_ERR_INVALID_ARG;
    if (max_kv_len < 0 || max_kv_len > cache8.max_len) return L4L_ERR_INVALID_ARG;
    if (!workspace || ws_bytes < kStatusBytes) return L4L_ERR_WORKSPACE;
    if (B == 0) return L4L_OK;
    const DecodePlan plan = plan_decode(B, Hq, Hkv, head_dim, max_kv_len, ws_bytes, true);
    if (plan.ws_bytes > ws_bytes) return L4L_ERR_WORKSPACE;
    const Fp8Scales sc{d_k_scale, d_v_scale};
    return launch_decode(q, o, cache8, d_kv_lens, max_kv_len, B, Hq, Hkv, head_dim, scale, d_lse, workspace, plan,
                         static_cast<cudaStream_t>(stream), nullptr, nullptr, nullptr, &sc);
}

l4l_status l4l_attn_decode_paged_fp8(const void *q, void *o, l4l_paged_kv pool8, const float *d_k_scale,
                                     const float *d_v_scale, const int32_t *d_block_table, int table_stride,
                                     const int32_t *d_kv_lens, int max_kv_len, int B, int Hq, int Hkv, int head_dim,
                                     float scale, float *d_lse, void *workspace, size_t ws_bytes, l4l_stream stream)
{
    l4l_status st = shape_status(B, Hq, Hkv, head_dim);
    if (st != L4L_OK) return st;
    if (!q || !o || !d_kv_lens || !d_block_table || !d_k_scale || !d_v_scale || !aligned16(q) || !aligned16(o))
        return L4L_ERR_INVALID_ARG;
    auto s16 = [](int64_t s) { return s >= 0 && (s % 16) == 0; };
    if (!pool8.k || !pool8.v || !aligned16(pool8.k) || !aligned16(pool8.v) || !s16(pool8.stride_page) ||
        !s16(pool8.stride_h) || !s16(pool8.stride_t) || pool8.num_pages <= 0 || pool8.page_size < 16 ||
        pool8.page_size > (1 << 20) || (pool8.page_size & (pool8.page_size - 1)) != 0 || table_stride <= 0)
        return L4L_ERR_INVALID_ARG;
    if (max_kv_len < 0 || (long long)max_kv_len > (long long)table_stride * pool8.page_size) return L4L_ERR_INVALID_ARG;
    if (!workspace || ws_bytes < kStatusBytes) return L4L_ERR_WORKSPACE;
    if (B == 0) return L4L_OK;
    const DecodePlan plan = plan_decode(B, Hq, Hkv, head_dim, max_kv_len, ws_bytes, true, pool8.page_size);
    if (plan.ws_bytes > ws_bytes) return L4L_ERR_WORKSPACE;
    const PagedTable pt{d_block_table, table_stride, pool8.num_pages};
    const Fp8Scales sc{d_k_scale, d_v_scale};
    return launch_decode(q, o, pool_as_cache(pool8), d_kv_lens, max_kv_len, B, Hq, Hkv, head_dim, scale, d_lse, workspace,
                         plan, static_cast<cudaStream_t>(stream), nullptr, nullptr, &pt, &sc);
}

l4l_status l4l_attn_decode_append_fp8(const void *q, void *o, l4l_kv_cache cache8, const float *d_k_scale,
                                      const float *d_v_scale, l4l_tensor4 k_new, l4l_tensor4 v_new,
                                      const int32_t *d_kv_lens, int max_kv_len, int B, int Hq, int Hkv, int head_dim,
                                      float scale, float *d_lse, void *workspace, size_t ws_bytes, l4l_stream stream)
{
    l4l_status st = shape_status(B, Hq, Hkv, head_dim);
    if (st != L4L_OK) return st;
    if (!q || !o || !d_kv_lens || !d_k_scale || !d_v_scale || !aligned16(q) || !aligned16(o)) return L4L_ERR_INVALID_ARG;
    if (!cache8_ok(cache8) || !tensor4_ok(k_new) || !tensor4_ok(v_new)) return L4L_ERR_INVALID_ARG;
    if (max_kv_len < 0 || max_kv_len > cache8.max_len) return L4L_ERR_INVALID_ARG;
    if (!workspace || ws_bytes < kStatusBytes) return L4L_ERR_WORKSPACE;
    if (B == 0) return L4L_OK;
    const DecodePlan plan = plan_decode(B, Hq, Hkv, head_dim, max_kv_len, ws_bytes, true);
    if (plan.ws_bytes > ws_bytes) return L4L_ERR_WORKSPACE;
    const Fp8Scales sc{d_k_scale, d_v_scale};
    return launch_decode(q, o, cache8, d_kv_lens, max_kv_len, B, Hq, Hkv, head_dim, scale, d_lse, workspace, plan,
                         static_cast<cudaStream_t>(stream), &k_new, &v_new, nullptr, &sc);
}

l4l_status l4l_attn_decode_paged_append_fp8(const void *q, void *o, l4l_paged_kv pool8, const float *d_k_scale,
                                            const float *d_v_scale, const int32_t *d_block_table, int table_stride,
                                            l4l_tensor4 k_new, l4l_tensor4 v_new, const int32_t *d_kv_lens,
                                            int max_kv_len, int B, int Hq, int Hkv, int head_dim, float scale,
                                            float *d_lse, void *workspace, size_t ws_bytes, l4l_stream stream)
{
    l4l_status st = shape_status(B, Hq, Hkv, head_dim);
    if (st != L4L_OK) return st;
    if (!q || !o || !d_kv_lens || !d_block_table || !d_k_scale || !d_v_scale || !aligned16(q) || !aligned16(o))
        return L4L_ERR_INVALID_ARG;
    auto s16 = [](int64_t s) { return s >= 0 && (s % 16) == 0; };
    if (!pool8.k || !pool8.v || !aligned16(pool8.k) || !aligned16(pool8.v) || !s16(pool8.stride_page) ||
        !s16(pool8.stride_h) || !s16(pool8.stride_t) || pool8.num_pages <= 0 || pool8.page_size < 16 ||
        pool8.page_size > (1 << 20) || (pool8.page_size & (pool8.page_size - 1)) != 0 || table_stride <= 0)
        return L4L_ERR_INVALID_ARG;
    if (!tensor4_ok(k_new) || !tensor4_ok(v_new)) return L4L_ERR_INVALID_ARG;
    if (max_kv_len < 0 || (long long)max_kv_len > (long long)table_stride * pool8.page_size) return L4L_ERR_INVALID_ARG;
    if (!workspace || ws_bytes < kStatusBytes) return L4L_ERR_WORKSPACE;
    if (B == 0) return L4L_OK;
    const DecodePlan plan = plan_decode(B, Hq, Hkv, head_dim, max_kv_len, ws_bytes, true, pool8.page_size);
    if (plan.ws_bytes > ws_bytes) return L4L_ERR_WORKSPACE;
    const PagedTable pt{d_block_table, table_stride, pool8.num_pages};
    const Fp8Scales sc{d_k_scale, d_v_scale};
    return launch_decode(q, o, pool_as_cache(pool8), d_kv_lens, max_kv_len, B, Hq, Hkv, head_dim, scale, d_lse, workspace,
                         plan, static_cast<cudaStream_t>(stream), &k_new, &v_new, &pt, &sc);
}

l4l_status l4l_attn_merge(const void *o_parts, const float *d_lse_parts, int R, void *o, float *d_lse, int B, int Hq,
                          int head_dim, l4l_stream stream)
{
    if (B < 0 || Hq <= 0 || R <= 0) return L4L_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return L4L_ERR_UNSUPPORTED;
    if (B == 0) return L4L_OK;
    if (!o_parts || !d_lse_parts || !o || !aligned16(o_parts) || !aligned16(o)) return L4L_ERR_INVALID_ARG;
    return launch_attn_merge(o_parts, d_lse_parts, R, o, d_lse, B, Hq, head_dim, static_cast<cudaStream_t>(stream));
}

l4l_status l4l_rglru_scan(const void *x, const void *gate_x, const void *gate_a, const float *d_a_param,
                          const int32_t *d_position, const int32_t *d_seq_lens, float *d_state, void *y, int B, int T,
                          int W, void *workspace, size_t ws_bytes, l4l_stream stream)
{
    if (B < 0 || T < 0 || W <= 0) return L4L_ERR_INVALID_ARG;
    if (W % 8 != 0 || B > 65535) return L4L_ERR_UNSUPPORTED;       // 16-byte rows for the tensor maps; grid.y
    if (B == 0 || T == 0) return L4L_OK;                            // nothing to do (empty tensors have no address)
    if (!x || !gate_x || !gate_a || !d_a_param || !d_state || !y) return L4L_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(gate_x) || !aligned16(gate_a)) return L4L_ERR_INVALID_ARG;
    if (!workspace || ws_bytes < kStatusBytes) return L4L_ERR_WORKSPACE;
    if (B == 0 || T == 0) return L4L_OK;
    return launch_rglru_scan(x, gate_x, gate_a, d_a_param, d_position, d_seq_lens, d_state, y, B, T, W, workspace,
                             ws_bytes, static_cast<cudaStream_t>(stream));
}

int l4l_rglru_strip_channels(int B, int T, int W)
{
    if (B <= 0 || T <= 0 || W <= 0 || W % 8 != 0) return -1;
    const int split = rglru_strip_split(B, T, W);
    return split == 0 ? 64 : 64 / split;
}

size_t l4l_rglru_workspace_bytes(int B, int T, int W)
{
    if (B < 0 || T < 0 || W <= 0) return 0;
    return rglru_workspace_bytes(B, T, W);
}

l4l_status l4l_rope_kv_append(l4l_tensor4 q, l4l_tensor4 k_new, l4l_tensor4 v_new, l4l_kv_cache cache,
                              const int32_t *d_pos, const int32_t *d_n_new, int T, int B, int Hq, int Hkv, int head_dim,
                              const float *d_cos, const float *d_sin, int n_pos, const float *d_q_weight,
                              const float *d_k_weight, float norm_eps, l4l_stream stream)
{
    l4l_status st = shape_status(B, Hq, Hkv, head_dim);
    if (st != L4L_OK) return st;
    if (T < 0 || n_pos < 0 || !d_pos || !d_cos || !d_sin || !(norm_eps >= 0.f)) return L4L_ERR_INVALID_ARG;
    if (!tensor4_ok(q) || !tensor4_ok(k_new) || !tensor4_ok(v_new) || !cache_ok(cache)) return L4L_ERR_INVALID_ARG;
    if (!aligned16(d_cos) || !aligned16(d_sin) || !aligned16(d_q_weight) || !aligned16(d_k_weight))
        return L4L_ERR_INVALID_ARG;
    if (B == 0 || T == 0) return L4L_OK;
    return launch_rope_kv_append(q, k_new, v_new, cache, d_pos, d_n_new, T, B, Hq, Hkv, head_dim, d_cos, d_sin, n_pos,
                                 d_q_weight, d_k_weight, norm_eps, static_cast<cudaStream_t>(stream));
}

l4l_status l4l_attn_prefill(l4l_tensor4 q, l4l_tensor4 k, l4l_tensor4 v, l4l_tensor4 o, l4l_kv_cache cache,
                            const int32_t *d_seq_lens, int S_max, int B, int Hq, int Hkv, int head_dim, float scale,
                            float *d_lse, void *workspace, size_t ws_bytes, l4l_stream stream)
{
    l4l_status st = shape_status(B, Hq, Hkv, head_dim);
    if (st != L4L_OK) return st;
    if (S_max < 0 || !d_seq_lens) return L4L_ERR_INVALID_ARG;
    if (!tensor4_ok(q) || !tensor4_ok(k) || !tensor4_ok(v) || !tensor4_ok(o)) return L4L_ERR_INVALID_ARG;
    if (cache.k || cache.v) {
        if (!cache_ok(cache)) return L4L_ERR_INVALID_ARG;
    }
    if (!workspace || ws_bytes < kStatusBytes) return L4L_ERR_WORKSPACE;
    if (B == 0 || S_max == 0) return L4L_OK;
    // a fresh prompt: every key comes from k / v, nothing is cached before; the cache (if given) is written
    const PrefillKV kv{k, v, S_max, false, nullptr, nullptr, (cache.k && cache.v) ? &cache : nullptr};
    return launch_prefill_tc(q, o, kv, d_seq_lens, nullptr, S_max, B, Hq, Hkv, head_dim, scale, d_lse, workspace,
                             static_cast<cudaStream_t>(stream));
}

l4l_status l4l_attn_prefill_chunk(l4l_tensor4 q, l4l_tensor4 o, l4l_kv_cache cache, const int32_t *d_past_lens,
                                  const int32_t *d_q_lens, int S_max, int B, int Hq, int Hkv, int head_dim,
                                  float scale, float *d_lse, void *workspace, size_t ws_bytes, l4l_stream stream)
{
    l4l_status st = shape_status(B, Hq, Hkv, head_dim);
    if (st != L4L_OK) return st;
    if (S_max < 0 || !d_past_lens || !d_q_lens) return L4L_ERR_INVALID_ARG;
    if (!tensor4_ok(q) || !tensor4_ok(o) || !cache_ok(cache)) return L4L_ERR_INVALID_ARG;
    if (!workspace || ws_bytes < kStatusBytes) return L4L_ERR_WORKSPACE;
    if (B == 0 || S_max == 0) return L4L_OK;
    // the caller has appended the chunk already: its keys are read from the cache too, viewed as [B, slot, Hkv, D]
    const l4l_tensor4 k{cache.k, cache.stride_b, cache.stride_t, cache.stride_h};
    const l4l_tensor4 v{cache.v, cache.stride_b, cache.stride_t, cache.stride_h};
    const PrefillKV kv{k, v, cache.max_len, true, &cache, nullptr, nullptr};
    return launch_prefill_tc(q, o, kv, d_q_lens, d_past_lens, S_max, B, Hq, Hkv, head_dim, scale, d_lse, workspace,
                             static_cast<cudaStream_t>(stream));
}

l4l_status l4l_attn_prefill_chunk_append(l4l_tensor4 q, l4l_tensor4 k_new, l4l_tensor4 v_new, l4l_tensor4 o,
                                         l4l_kv_cache cache, const int32_t *d_past_lens, const int32_t *d_q_lens,
                                         int S_max, int B, int Hq, int Hkv, int head_dim, float scale, float *d_lse,
                                         void *workspace, size_t ws_bytes, l4l_stream stream)
{
    l4l_status st = shape_status(B, Hq, Hkv, head_dim);
    if (st != L4L_OK) return st;
    if (S_max < 0 || !d_past_lens || !d_q_lens) return L4L_ERR_INVALID_ARG;
    if (!tensor4_ok(q) || !tensor4_ok(k_new) || !tensor4_ok(v_new) || !tensor4_ok(o) || !cache_ok(cache))
        return L4L_ERR_INVALID_ARG;
    if (!workspace || ws_bytes < kStatusBytes) return L4L_ERR_WORKSPACE;
    if (B == 0 || S_max == 0) return L4L_OK;
    const PrefillKV kv{k_new, v_new, S_max, false, &cache, nullptr, &cache};
    return launch_prefill_tc(q, o, kv, d_q_lens, d_past_lens, S_max, B, Hq, Hkv, head_dim, scale, d_lse, workspace,
                             static_cast<cudaStream_t>(stream));
}

l4l_status l4l_attn_prefill_chunk_paged_append(l4l_tensor4 q, l4l_tensor4 k_new, l4l_tensor4 v_new, l4l_tensor4 o,
                                               l4l_paged_kv pool, const int32_t *d_block_table, int table_stride,
                                               const int32_t *d_past_lens, const int32_t *d_q_lens, int S_max, int B,
                                               int Hq, int Hkv, int head_dim, float scale, float *d_lse, void *workspace,
                                               size_t ws_bytes, l4l_stream stream)
{
    l4l_status st = shape_status(B, Hq, Hkv, head_dim);
    if (st != L4L_OK) return st;
    if (S_max < 0 || !d_past_lens || !d_q_lens || !d_block_table || table_stride <= 0) return L4L_ERR_INVALID_ARG;
    if (!tensor4_ok(q) || !tensor4_ok(k_new) || !tensor4_ok(v_new) || !tensor4_ok(o) || !pool_ok(pool))
        return L4L_ERR_INVALID_ARG;
    if (!workspace || ws_bytes < kStatusBytes) return L4L_ERR_WORKSPACE;
    if (B == 0 || S_max == 0) return L4L_OK;
    const l4l_kv_cache as_cache = pool_as_cache(pool);
    const PagedTable pt{d_block_table, table_stride, pool.num_pages};
    const PrefillKV kv{k_new, v_new, S_max, false, &as_cache, &pt, &as_cache};
    return launch_prefill_tc(q, o, kv, d_q_lens, d_past_lens, S_max, B, Hq, Hkv, head_dim, scale, d_lse, workspace,
                             static_cast<cudaStream_t>(stream));
}

l4l_status l4l_attn_decode(const void *q, void *o, l4l_kv_cache cache, const int32_t *d_kv_lens, int max_kv_len,
                           int B, int Hq, int Hkv, int head_dim, float scale, float *d_lse, void *workspace,
                           size_t ws_bytes, l4l_stream stream)
{
    l4l_status st = shape_status(B, Hq, Hkv, head_dim);
    if (st != L4L_OK) return st;
    if (!q || !o || !d_kv_lens || !aligned16(q) || !aligned16(o)) return L4L_ERR_INVALID_ARG;
    if (!cache_ok(cache) || max_kv_len < 0 || max_kv_len > cache.max_len) return L4L_ERR_INVALID_ARG;
    if (!workspace || ws_bytes < kStatusBytes) return L4L_ERR_WORKSPACE;
    if (B == 0) return L4L_OK;
    const DecodePlan plan = plan_decode(B, Hq, Hkv, head_dim, max_kv_len, ws_bytes);
    if (plan.ws_bytes > ws_bytes) return L4L_ERR_WORKSPACE;
    return launch_decode(q, o, cache, d_kv_lens, max_kv_len, B, Hq, Hkv, head_dim, scale, d_lse, workspace, plan,
                         static_cast<cudaStream_t>(stream));
}

l4l_status l4l_attn_decode_append(const void *q, void *o, l4l_kv_cache cache, l4l_tensor4 k_new, l4l_tensor4 v_new,
                                  const int32_t *d_kv_lens, int max_kv_len, int B, int Hq, int Hkv, int head_dim,
                                  float scale, float *d_lse, void *workspace, size_t ws_bytes, l4l_stream stream)
{
    l4l_status st = shape_status(B, Hq, Hkv, head_dim);
    if (st != L4L_OK) return st;
    if (!q || !o || !d_kv_lens || !aligned16(q) || !aligned16(o)) return L4L_ERR_INVALID_ARG;
    if (!cache_ok(cache) || max_kv_len < 0 || max_kv_len > cache.max_len) return L4L_ERR_INVALID_ARG;
    if (!tensor4_ok(k_new) || !tensor4_ok(v_new)) return L4L_ERR_INVALID_ARG;
    if (!workspace || ws_bytes < kStatusBytes) return L4L_ERR_WORKSPACE;
    if (B == 0) return L4L_OK;
    const DecodePlan plan = plan_decode(B, Hq, Hkv, head_dim, max_kv_len, ws_bytes);
    if (plan.ws_bytes > ws_bytes) return L4L_ERR_WORKSPACE;
    return launch_decode(q, o, cache, d_kv_lens, max_kv_len, B, Hq, Hkv, head_dim, scale, d_lse, workspace, plan,
                         static_cast<cudaStream_t>(stream), &k_new, &v_new);
}

l4l_status l4l_attn_decode_rope_append(const void *q, void *o, l4l_kv_cache cache, l4l_tensor4 k_new, l4l_tensor4 v_new,
                                       const int32_t *d_kv_lens, int max_kv_len, int B, int Hq, int Hkv, int head_dim,
                                       float scale, const float *d_cos, const float *d_sin, int n_pos,
                                       const float *d_q_weight, const float *d_k_weight, float norm_eps, float *d_lse,
                                       void *workspace, size_t ws_bytes, l4l_stream stream)
{
    l4l_status st = shape_status(B, Hq, Hkv, head_dim);
    if (st != L4L_OK) return st;
    if (!q || !o || !d_kv_lens || !aligned16(q) || !aligned16(o)) return L4L_ERR_INVALID_ARG;
    if (!cache_ok(cache) || max_kv_len < 0 || max_kv_len > cache.max_len) return L4L_ERR_INVALID_ARG;
    if (!tensor4_ok(k_new) || !tensor4_ok(v_new)) return L4L_ERR_INVALID_ARG;
    if (!d_cos || !d_sin || n_pos < 0 || !(norm_eps >= 0.f)) return L4L_ERR_INVALID_ARG;
    if (!aligned16(d_cos) || !aligned16(d_sin)) return L4L_ERR_INVALID_ARG;      // rows are fetched with bulk copies
    if (!workspace || ws_bytes < kStatusBytes) return L4L_ERR_WORKSPACE;
    if (B == 0) return L4L_OK;
    const DecodePlan plan = plan_decode(B, Hq, Hkv, head_dim, max_kv_len, ws_bytes);
    if (plan.ws_bytes > ws_bytes) return L4L_ERR_WORKSPACE;
    const RopeArgs rope{d_cos, d_sin, d_q_weight, d_k_weight, norm_eps, n_pos};
    return launch_decode(q, o, cache, d_kv_lens, max_kv_len, B, Hq, Hkv, head_dim, scale, d_lse, workspace, plan,
                         static_cast<cudaStream_t>(stream), &k_new, &v_new, nullptr, nullptr, &rope);
}

l4l_status l4l_attn_decode_paged_rope_append(const void *q, void *o, l4l_paged_kv pool, const int32_t *d_block_table,
                                             int table_stride, l4l_tensor4 k_new, l4l_tensor4 v_new,
                                             const int32_t *d_kv_lens, int max_kv_len, int B, int Hq, int Hkv,
                                             int head_dim, float scale, const float *d_cos, const float *d_sin, int n_pos,
                                             const float *d_q_weight, const float *d_k_weight, float norm_eps,
                                             float *d_lse, void *workspace, size_t ws_bytes, l4l_stream stream)
{
    l4l_status st = shape_status(B, Hq, Hkv, head_dim);
    if (st != L4L_OK) return st;
    if (!q || !o || !d_kv_lens || !d_block_table || !aligned16(q) || !aligned16(o)) return L4L_ERR_INVALID_ARG;
    if (!pool_ok(pool) || table_stride <= 0) return L4L_ERR_INVALID_ARG;
    if (!tensor4_ok(k_new) || !tensor4_ok(v_new)) return L4L_ERR_INVALID_ARG;
    if (max_kv_len < 0 || (long long)max_kv_len > (long long)table_stride * pool.page_size) return L4L_ERR_INVALID_ARG;
    if (!d_cos || !d_sin || n_pos < 0 || !(norm_eps >= 0.f)) return L4L_ERR_INVALID_ARG;
    if (!aligned16(d_cos) || !aligned16(d_sin)) return L4L_ERR_INVALID_ARG;      // rows are fetched with bulk copies
    if (!workspace || ws_bytes < kStatusBytes) return L4L_ERR_WORKSPACE;
    if (B == 0) return L4L_OK;
    const DecodePlan plan = plan_decode(B, Hq, Hkv, head_dim, max_kv_len, ws_bytes, false, pool.page_size);
    if (plan.ws_bytes > ws_bytes) return L4L_ERR_WORKSPACE;
    const PagedTable pt{d_block_table, table_stride, pool.num_pages};
    const RopeArgs rope{d_cos, d_sin, d_q_weight, d_k_weight, norm_eps, n_pos};
    return launch_decode(q, o, pool_as_cache(pool), d_kv_lens, max_kv_len, B, Hq, Hkv, head_dim, scale, d_lse, workspace,
                         plan, static_cast<cudaStream_t>(stream), &k_new, &v_new, &pt, nullptr, &rope);
}

l4l_status l4l_attn_decode_rope_append_fp8(const void *q, void *o, l4l_kv_cache cache8, const float *d_k_scale,
                                           const float *d_v_scale, l4l_tensor4 k_new, l4l_tensor4 v_new,
                                           const int32_t *d_kv_lens, int max_kv_len, int B, int Hq, int Hkv, int head_dim,
                                           float scale, const float *d_cos, const float *d_sin, int n_pos,
                                           const float *d_q_weight, const float *d_k_weight, float norm_eps, float *d_lse,
                                           void *workspace, size_t ws_bytes, l4l_stream stream)
{
    l4l_status st = shape_status(B, Hq, Hkv, head_dim);
    if (st != L4L_OK) return st;
    if (!q || !o || !d_kv_lens || !d_k_scale || !d_v_scale || !aligned16(q) || !aligned16(o)) return L4L_ERR_INVALID_ARG;
    if (!cache8_ok(cache8) || !tensor4_ok(k_new) || !tensor4_ok(v_new)) return L4L_ERR_INVALID_ARG;
    if (max_kv_len < 0 || max_kv_len > cache8.max_len) return L4L_ERR_INVALID_ARG;
    if (!d_cos || !d_sin || n_pos < 0 || !(norm_eps >= 0.f)) return L4L_ERR_INVALID_ARG;
    if (!aligned16(d_cos) || !aligned16(d_sin)) return L4L_ERR_INVALID_ARG;      // rows are fetched with bulk copies
    if (!workspace || ws_bytes < kStatusBytes) return L4L_ERR_WORKSPACE;
    if (B == 0) return L4L_OK;
    const DecodePlan plan = plan_decode(B, Hq, Hkv, head_dim, max_kv_len, ws_bytes, true);
    if (plan.ws_bytes > ws_bytes) return L4L_ERR_WORKSPACE;
    const Fp8Scales sc{d_k_scale, d_v_scale};
    const RopeArgs rope{d_cos, d_sin, d_q_weight, d_k_weight, norm_eps, n_pos};
    return launch_decode(q, o, cache8, d_kv_lens, max_kv_len, B, Hq, Hkv, head_dim, scale, d_lse, workspace, plan,
                         static_cast<cudaStream_t>(stream), &k_new, &v_new, nullptr, &sc, &rope);
}

l4l_status l4l_attn_decode_paged_rope_append_fp8(const void *q, void *o, l4l_paged_kv pool8, const float *d_k_scale,
                                                 const float *d_v_scale, const int32_t *d_block_table, int table_stride,
                                                 l4l_tensor4 k_new, l4l_tensor4 v_new, const int32_t *d_kv_lens,
                                                 int max_kv_len, int B, int Hq, int Hkv, int head_dim, float scale,
                                                 const float *d_cos, const float *d_sin, int n_pos,
                                                 const float *d_q_weight, const float *d_k_weight, float norm_eps,
                                                 float *d_lse, void *workspace, size_t ws_bytes, l4l_stream stream)
{
    l4l_status st = shape_status(B, Hq, Hkv, head_dim);
    if (st != L4L_OK) return st;
    if (!q || !o || !d_kv_lens || !d_block_table || !d_k_scale || !d_v_scale || !aligned16(q) || !aligned16(o))
        return L4L_ERR_INVALID_ARG;
    auto s16 = [](int64_t s) { return s >= 0 && (s % 16) == 0; };
    if (!pool8.k || !pool8.v || !aligned16(pool8.k) || !aligned16(pool8.v) || !s16(pool8.stride_page) ||
        !s16(pool8.stride_h) || !s16(pool8.stride_t) || pool8.num_pages <= 0 || pool8.page_size < 16 ||
        pool8.page_size > (1 << 20) || (pool8.page_size & (pool8.page_size - 1)) != 0 || table_stride <= 0)
        return L4L_ERR_INVALID_ARG;
    if (!tensor4_ok(k_new) || !tensor4_ok(v_new)) return L4L_ERR_INVALID_ARG;
    if (max_kv_len < 0 || (long long)max_kv_len > (long long)table_stride * pool8.page_size) return L4L_ERR_INVALID_ARG;
    if (!d_cos || !d_sin || n_pos < 0 || !(norm_eps >= 0.f)) return L4L_ERR_INVALID_ARG;
    if (!aligned16(d_cos) || !aligned16(d_sin)) return L4L_ERR_INVALID_ARG;      // rows are fetched with bulk copies
    if (!workspace || ws_bytes < kStatusBytes) return L4L_ERR_WORKSPACE;
    if (B == 0) return L4L_OK;
    const DecodePlan plan = plan_decode(B, Hq, Hkv, head_dim, max_kv_len, ws_bytes, true, pool8.page_size);
    if (plan.ws_bytes > ws_bytes) return L4L_ERR_WORKSPACE;
    const PagedTable pt{d_block_table, table_stride, pool8.num_pages};
    const Fp8Scales sc{d_k_scale, d_v_scale};
    const RopeArgs rope{d_cos, d_sin, d_q_weight, d_k_weight, norm_eps, n_pos};
    return launch_decode(q, o, pool_as_cache(pool8), d_kv_lens, max_kv_len, B, Hq, Hkv, head_dim, scale, d_lse, workspace,
                         plan, static_cast<cudaStream_t>(stream), &k_new, &v_new, &pt, &sc, &rope);
}

void l4l_set_decode_override(int cluster, int warp, int split_warps)
{
    g_override_cluster = cluster < 0 ? -1 : cluster;
    g_override_warp = warp < 0 ? -1 : (warp ? 1 : 0);
    g_override_split_warps = (split_warps == 4 || split_warps == 8) ? split_warps : 0;
}

int l4l_decode_kernel_choice(int B, int Hq, int Hkv, int head_dim, int max_kv_len, int fp8, int *detail)
{
    if (detail) *detail = 0;
    if (shape_status(B, Hq, Hkv, head_dim) != L4L_OK || B == 0 || max_kv_len < 0) return -1;
    // the order launch_decode asks in
    if (decode_warp_eligible(B, Hq, Hkv, head_dim, max_kv_len, fp8 != 0, false, false)) return 2;
    const int width = decode_cluster_width(B, Hq, Hkv, head_dim, max_kv_len, fp8 != 0);
    if (width > 0) {
        if (detail) *detail = width;
        return 1;
    }
    const DecodePlan plan = plan_decode(B, Hq, Hkv, head_dim, max_kv_len, ~(size_t)0, fp8 != 0);
    if (detail) *detail = plan.warps;
    return 0;
}

}  // extern "C"
