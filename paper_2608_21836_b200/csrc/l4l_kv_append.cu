// KV-cache append: an exact copy of the new tokens' K and V rows into their cache slots.
// One thread moves one 16-byte piece of a K row and the matching piece of the V row, so a
// warp reads and writes whole contiguous rows (coalesced both ways).
#include "l4l_internal.h"
#include "l4l_ptx.cuh"

namespace l4l {

namespace {

struct AppendParams {
    const uint4 *k_new, *v_new;     // strides below are in 16-byte units
    uint4 *cache_k, *cache_v;
    int64_t new_sb, new_st, new_sh, vnew_sb, vnew_st, vnew_sh;
    int64_t c_sb, c_sh, c_st;
    const int32_t *write_pos, *n_new;
    const int32_t *block_table;     // paged cache (null: contiguous): c_sb is then the stride between pages
    int table_stride, page_size, num_pages;
    int B, T, Hkv, pieces, max_len;
};

// Idx: unsigned 32-bit when the piece count fits (the index arithmetic is four divisions per piece, which in 64 bits
// cost more than the copy), 64-bit otherwise.
template <typename Idx>
__global__ void __launch_bounds__(256) kv_append_kernel(const AppendParams p)
{
    const Idx total = (Idx)p.B * (Idx)p.T * (Idx)p.Hkv * (Idx)p.pieces;
    const Idx step = (Idx)gridDim.x * blockDim.x;
    for (Idx idx = (Idx)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += step) {
        const int piece = (int)(idx % (Idx)p.pieces);
        Idx rest = idx / (Idx)p.pieces;
        const int g = (int)(rest % (Idx)p.Hkv);
        rest /= (Idx)p.Hkv;
        const int r = (int)(rest % (Idx)p.T);
        const int b = (int)(rest / (Idx)p.T);
        const int n = p.n_new ? p.n_new[b] : p.T;
        if (r >= n) continue;
        long long slot = (long long)p.write_pos[b] + r;
        if (slot < 0 || slot >= p.max_len) continue;          // dropped, never written out of range
        long long outer = b;
        if (p.block_table) {                                   // max_len = table_stride * page_size here
            outer = p.block_table[(long long)b * p.table_stride + slot / p.page_size];
            if (outer < 0 || outer >= p.num_pages) continue;  // no page behind this slot: dropped
            slot %= p.page_size;
        }
        const uint4 kk = p.k_new[b * p.new_sb + r * p.new_st + g * p.new_sh + piece];
        const uint4 vv = p.v_new[b * p.vnew_sb + r * p.vnew_st + g * p.vnew_sh + piece];
        const int64_t dst = outer * p.c_sb + g * p.c_sh + slot * p.c_st + piece;
        p.cache_k[dst] = kk;
        p.cache_v[dst] = vv;
    }
}

}  // namespace

l4l_status launch_kv_append(const l4l_kv_cache &cache, const l4l_tensor4 &k_new, const l4l_tensor4 &v_new,
                            const int32_t *d_write_pos, const int32_t *d_n_new, int n_new_max, int B, int Hkv,
                            int D, cudaStream_t stream, const PagedTable *paged)
{
    AppendParams p;
    p.k_new = static_cast<const uint4 *>(k_new.ptr);
    p.v_new = static_cast<const uint4 *>(v_new.ptr);
    p.cache_k = static_cast<uint4 *>(cache.k);
    p.cache_v = static_cast<uint4 *>(cache.v);
    p.new_sb = k_new.stride_b / 8; p.new_st = k_new.stride_t / 8; p.new_sh = k_new.stride_h / 8;
    p.vnew_sb = v_new.stride_b / 8; p.vnew_st = v_new.stride_t / 8; p.vnew_sh = v_new.stride_h / 8;
    p.c_sb = cache.stride_b / 8; p.c_sh = cache.stride_h / 8; p.c_st = cache.stride_t / 8;
    p.write_pos = d_write_pos; p.n_new = d_n_new;
    p.B = B; p.T = n_new_max; p.Hkv = Hkv; p.pieces = D / 8; p.max_len = cache.max_len;
    p.block_table = nullptr;
    p.table_stride = p.page_size = p.num_pages = 0;
    if (paged) {                                               // `cache` is the page pool, max_len the page size
        p.block_table = paged->block_table;
        p.table_stride = paged->table_stride;
        p.page_size = cache.max_len;
        p.num_pages = paged->num_pages;
        const long long cap = (long long)paged->table_stride * cache.max_len;
        p.max_len = cap > 0x7fffffffll ? 0x7fffffff : (int)cap;
    }
    const long long total = (long long)B * n_new_max * Hkv * p.pieces;
    long long blocks = (total + 255) / 256;
    const long long cap = 8ll * sm_count();
    if (blocks > cap) blocks = cap;
    // (the 32-bit index also has to hold idx + grid step without wrapping)
    if (total + blocks * 256 < (1ll << 32))
        kv_append_kernel<uint32_t><<<(int)blocks, 256, 0, stream>>>(p);
    else
        kv_append_kernel<unsigned long long><<<(int)blocks, 256, 0, stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? L4L_OK : L4L_ERR_CUDA;
}

}  // namespace l4l
