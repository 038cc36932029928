// ec_kv_refresh: scatter the active rows' fresh K/V into the cache in place
// (Section 4.2 of the paper: on a partial step only the mask tokens and the
// selected recent tokens get new K,V; Appendix A, partial branch).
//
//   k_cache[b, h, idx[b,i], :] = k_new[b, i, h, :]        (same for V)
//
// Pure data movement, bit-exact: one thread moves one 16-byte piece of a
// (row, kv-head) vector; consecutive threads cover consecutive pieces of the
// source, so reads are fully coalesced and writes are coalesced per head row.
// With idx == nullptr the list is the identity (recompute step) and the kernel
// is a [n, H, D] -> [H, n, D] layout-changing copy.
#include "ec_common.cuh"

namespace ec {
namespace {

__global__ void __launch_bounds__(256) refresh_kernel(uint4* __restrict__ k_cache, uint4* __restrict__ v_cache,
                                                      const uint4* __restrict__ k_new,
                                                      const uint4* __restrict__ v_new,
                                                      const int32_t* __restrict__ idx, int n_active,
                                                      int ctx_len, int n_kv_heads, int row_vecs,
                                                      long long total_vecs) {
    // flat source index over [b, i, h, piece]; blockIdx.y selects K or V
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= total_vecs) return;
    const int piece = (int)(t % row_vecs);
    const long long bih = t / row_vecs;
    const int h = (int)(bih % n_kv_heads);
    const long long bi = bih / n_kv_heads;
    const int i = (int)(bi % n_active);
    const long long b = bi / n_active;
    const int pos = idx ? __ldg(idx + bi) : i;
    if (pos < 0 || pos >= ctx_len) return;  // never write outside the cache
    const long long dst = ((b * n_kv_heads + h) * ctx_len + pos) * row_vecs + piece;
    if (blockIdx.y == 0)
        k_cache[dst] = __ldg(k_new + t);
    else
        v_cache[dst] = __ldg(v_new + t);
}

}  // namespace

cudaError_t launch_refresh(const ec_attn_desc& d, void* k_cache, void* v_cache, const void* k_new,
                           const void* v_new, const int32_t* active_idx, int n_active,
                           cudaStream_t stream) {
    const int esize = d.dtype == EC_BF16 ? 2 : 4;
    const int row_vecs = d.head_dim * esize / 16;
    const long long total = (long long)d.batch * n_active * d.n_kv_heads * row_vecs;
    if (total == 0) return cudaSuccess;
    const dim3 grid((unsigned)((total + 255) / 256), 2);
    refresh_kernel<<<grid, 256, 0, stream>>>(static_cast<uint4*>(k_cache), static_cast<uint4*>(v_cache),
                                             static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new),
                                             active_idx, n_active, d.ctx_len, d.n_kv_heads, row_vecs, total);
    return cudaGetLastError();
}

}  // namespace ec
