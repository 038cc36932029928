// ec_attend, bf16 storage, warp-level tensor-core path (mma.sync m16n8k16, fp32
// accumulation): active-row bidirectional attention over the full cache
// (Appendix A of the paper, partial branch; the full branch when n_active == L).
//
// Work decomposition
//   - The query rows that share one kv head -- n_active rows x g = H_q/H_kv query
//     heads -- are flattened into one row axis r = i*g + j (GQA packing), cut into
//     64-row tiles; one CTA (4 warps x 16 rows) owns one tile.
//   - Keys are cut into 64-key tiles.  When there are few row tiles (skip step:
//     34 active rows) the key axis is also split across CTAs ("split-KV"): each
//     split writes an un-normalised partial (m, l, O) to the workspace and a small
//     combine kernel merges them.  Every K/V byte is read by exactly one CTA per
//     row tile, so the skip step streams the cache once.
//   - K/V tiles are staged in shared memory with 16-byte cp.async copies (two
//     stages), XOR-swizzled so ldmatrix is bank-conflict free.
//   - Softmax is online (running max / sum per row, exp2 with the scale folded
//     in); P is re-packed from the S accumulators into A fragments in registers.
#include "ec_common.cuh"

namespace ec {
namespace {

constexpr int BM = 64;   // query rows per CTA
constexpr int BN = 64;   // keys per tile
constexpr int kThreads = 128;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    const int sz = valid ? 16 : 0;  // src-size 0: the 16 bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// byte offset of 16-byte chunk `chunk` of row `row` in a swizzled [rows, D] bf16 tile
template <int D>
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
    return (uint32_t)(row * (D * 2) + ((chunk ^ (row & 7)) << 4));
}

struct MmaParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k_cache;
    const __nv_bfloat16* v_cache;
    __nv_bfloat16* out;
    float* part_o;   // [B*Hkv, n_splits, rows_total, D]
    float2* part_ml; // [B*Hkv, n_splits, rows_total]  (m in log2 units, l)
    int n_active, ctx_len, n_q_heads, n_kv_heads, group;  // group = H_q / H_kv
    int rows_total;   // n_active * group
    int n_splits, tiles_per_split;
    float scale_log2;  // scale * log2(e)
};

template <int D>
__global__ void __launch_bounds__(kThreads) attend_mma_kernel(const MmaParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int TILE_BYTES = BN * D * 2;
    constexpr int CHUNKS = D / 8;  // 16-byte chunks per row
    unsigned char* sQ = smem;                       // BM x D
    unsigned char* sK = smem + BM * D * 2;          // 2 stages
    unsigned char* sV = sK + 2 * TILE_BYTES;        // 2 stages

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int row_tile = blockIdx.x, split = blockIdx.y, bh = blockIdx.z;
    const int b = bh / p.n_kv_heads, hk = bh % p.n_kv_heads;
    const int r0 = row_tile * BM;

    const int n_tiles_total = (p.ctx_len + BN - 1) / BN;
    const int t_begin = split * p.tiles_per_split;
    const int t_end = min(n_tiles_total, t_begin + p.tiles_per_split);

    const __nv_bfloat16* kbase = p.k_cache + ((long long)bh * p.ctx_len) * D;
    const __nv_bfloat16* vbase = p.v_cache + ((long long)bh * p.ctx_len) * D;

    // ---- stage Q (rows beyond rows_total are zero-filled) --------------------------
    for (int c = tid; c < BM * CHUNKS; c += kThreads) {
        const int row = c / CHUNKS, ch = c % CHUNKS;
        const int r = r0 + row;
        const bool ok = r < p.rows_total;
        const int i = ok ? r / p.group : 0, j = ok ? r % p.group : 0;
        const __nv_bfloat16* src =
            p.q + (((long long)b * p.n_active + i) * p.n_q_heads + hk * p.group + j) * D + ch * 8;
        cp_async16(smem_u32(sQ) + swz<D>(row, ch), src, ok);
    }
    auto load_kv = [&](int tile, int stage) {
        const int key0 = tile * BN;
        for (int c = tid; c < BN * CHUNKS; c += kThreads) {
            const int row = c / CHUNKS, ch = c % CHUNKS;
            const bool ok = key0 + row < p.ctx_len;
            const long long off = (long long)(ok ? key0 + row : 0) * D + ch * 8;
            cp_async16(smem_u32(sK) + stage * TILE_BYTES + swz<D>(row, ch), kbase + off, ok);
            cp_async16(smem_u32(sV) + stage * TILE_BYTES + swz<D>(row, ch), vbase + off, ok);
        }
    };
    if (t_begin < t_end) load_kv(t_begin, 0);
    cp_async_commit();

    // ---- per-thread state ----------------------------------------------------------
    uint32_t qf[D / 16][4];
    float o[D / 8][4];
#pragma unroll
    for (int n = 0; n < D / 8; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};  // rows g and g+8 of the warp's 16

    bool q_loaded = false;
    for (int t = t_begin; t < t_end; ++t) {
        const int stage = (t - t_begin) & 1;
        if (t + 1 < t_end) load_kv(t + 1, stage ^ 1);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();

        if (!q_loaded) {
            q_loaded = true;
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks)
                ldsm_x4(smem_u32(sQ) + swz<D>(warp * 16 + (lane & 15), ks * 2 + (lane >> 4)), qf[ks]);
        }

        // ---- S = Q K^T --------------------------------------------------------------
        float s[BN / 8][4];
#pragma unroll
        for (int n = 0; n < BN / 8; ++n) { s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f; }
        const uint32_t kst = smem_u32(sK) + stage * TILE_BYTES;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
#pragma unroll
            for (int nb = 0; nb < BN / 16; ++nb) {
                uint32_t kf[4];
                const int key = nb * 16 + (lane & 7) + ((lane >> 4) << 3);
                ldsm_x4(kst + swz<D>(key, ks * 2 + ((lane >> 3) & 1)), kf);
                mma_bf16(s[2 * nb], qf[ks], kf[0], kf[1]);
                mma_bf16(s[2 * nb + 1], qf[ks], kf[2], kf[3]);
            }
        }
        // ---- mask keys beyond the context (ragged last tile) ------------------------
        const int key0 = t * BN;
        if (key0 + BN > p.ctx_len) {
#pragma unroll
            for (int n = 0; n < BN / 8; ++n) {
                const int kcol = key0 + n * 8 + 2 * (lane & 3);
                if (kcol >= p.ctx_len) { s[n][0] = -INFINITY; s[n][2] = -INFINITY; }
                if (kcol + 1 >= p.ctx_len) { s[n][1] = -INFINITY; s[n][3] = -INFINITY; }
            }
        }
        // ---- online softmax ---------------------------------------------------------
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int n = 0; n < BN / 8; ++n) {
            mx[0] = fmaxf(mx[0], fmaxf(s[n][0], s[n][1]));
            mx[1] = fmaxf(mx[1], fmaxf(s[n][2], s[n][3]));
        }
        float corr[2], mneg[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
            const float m_new = fmaxf(m_run[h], mx[h] * p.scale_log2);
            corr[h] = (m_run[h] == -INFINITY) ? 0.f : fast_exp2(m_run[h] - m_new);
            m_run[h] = m_new;
            mneg[h] = -m_new;
        }
        float rs[2] = {0.f, 0.f};
#pragma unroll
        for (int n = 0; n < BN / 8; ++n) {
            s[n][0] = fast_exp2(fmaf(s[n][0], p.scale_log2, mneg[0]));
            s[n][1] = fast_exp2(fmaf(s[n][1], p.scale_log2, mneg[0]));
            s[n][2] = fast_exp2(fmaf(s[n][2], p.scale_log2, mneg[1]));
            s[n][3] = fast_exp2(fmaf(s[n][3], p.scale_log2, mneg[1]));
            rs[0] += s[n][0] + s[n][1];
            rs[1] += s[n][2] + s[n][3];
        }
        l_run[0] = fmaf(l_run[0], corr[0], rs[0]);
        l_run[1] = fmaf(l_run[1], corr[1], rs[1]);
#pragma unroll
        for (int n = 0; n < D / 8; ++n) {
            o[n][0] *= corr[0]; o[n][1] *= corr[0];
            o[n][2] *= corr[1]; o[n][3] *= corr[1];
        }
        // ---- O += P V ---------------------------------------------------------------
        const uint32_t vst = smem_u32(sV) + stage * TILE_BYTES;
#pragma unroll
        for (int ks = 0; ks < BN / 16; ++ks) {
            uint32_t pf[4];
            pf[0] = pack_bf16(s[2 * ks][0], s[2 * ks][1]);
            pf[1] = pack_bf16(s[2 * ks][2], s[2 * ks][3]);
            pf[2] = pack_bf16(s[2 * ks + 1][0], s[2 * ks + 1][1]);
            pf[3] = pack_bf16(s[2 * ks + 1][2], s[2 * ks + 1][3]);
#pragma unroll
            for (int db = 0; db < D / 16; ++db) {
                uint32_t vf[4];
                ldsm_x4_t(vst + swz<D>(ks * 16 + (lane & 15), db * 2 + (lane >> 4)), vf);
                mma_bf16(o[2 * db], pf, vf[0], vf[1]);
                mma_bf16(o[2 * db + 1], pf, vf[2], vf[3]);
            }
        }
        __syncthreads();  // everyone is done with this stage before it is refilled
    }
    cp_async_wait<0>();

    // ---- epilogue ------------------------------------------------------------------
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 1);
        l_run[h] += __shfl_xor_sync(0xffffffffu, l_run[h], 2);
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int r = r0 + warp * 16 + (lane >> 2) + 8 * h;
        if (r >= p.rows_total) continue;
        if (p.n_splits == 1) {
            const int i = r / p.group, j = r % p.group;
            __nv_bfloat16* dst = p.out + (((long long)b * p.n_active + i) * p.n_q_heads + hk * p.group + j) * D;
            const float inv = 1.f / l_run[h];
#pragma unroll
            for (int n = 0; n < D / 8; ++n) {
                const uint32_t v = pack_bf16(o[n][2 * h] * inv, o[n][2 * h + 1] * inv);
                *reinterpret_cast<uint32_t*>(dst + n * 8 + 2 * (lane & 3)) = v;
            }
        } else {
            const long long slot = ((long long)bh * p.n_splits + split) * p.rows_total + r;
            float* dst = p.part_o + slot * D;
#pragma unroll
            for (int n = 0; n < D / 8; ++n)
                *reinterpret_cast<float2*>(dst + n * 8 + 2 * (lane & 3)) = make_float2(o[n][2 * h], o[n][2 * h + 1]);
            if ((lane & 3) == 0) p.part_ml[slot] = make_float2(m_run[h], l_run[h]);
        }
    }
}

// merge the split-KV partials of one (sequence, kv head, row): out = sum_s w_s O_s / sum_s w_s l_s,
// w_s = 2^(m_s - max m)
template <int D>
__global__ void __launch_bounds__(128) attend_combine_kernel(const MmaParams p) {
    const int lane = threadIdx.x & 31;
    const int bh = blockIdx.z;
    const int r = blockIdx.x * 4 + (threadIdx.x >> 5);  // one warp per flattened row
    if (r >= p.rows_total) return;
    const int b = bh / p.n_kv_heads, hk = bh % p.n_kv_heads;
    float m = -INFINITY;
    for (int s = 0; s < p.n_splits; ++s)
        m = fmaxf(m, __ldcg(&p.part_ml[((long long)bh * p.n_splits + s) * p.rows_total + r]).x);
    constexpr int DPL = D / 32;
    float acc[DPL];
#pragma unroll
    for (int t = 0; t < DPL; ++t) acc[t] = 0.f;
    float l = 0.f;
    for (int s = 0; s < p.n_splits; ++s) {
        const long long slot = ((long long)bh * p.n_splits + s) * p.rows_total + r;
        const float2 ml = __ldcg(&p.part_ml[slot]);
        if (ml.y <= 0.f) continue;  // an empty split
        const float w = fast_exp2(ml.x - m);
        l = fmaf(w, ml.y, l);
        const float* src = p.part_o + slot * D;
#pragma unroll
        for (int t = 0; t < DPL; ++t) acc[t] = fmaf(w, __ldcg(src + lane + 32 * t), acc[t]);
    }
    const int i = r / p.group, j = r % p.group;
    __nv_bfloat16* dst = p.out + (((long long)b * p.n_active + i) * p.n_q_heads + hk * p.group + j) * D;
    const float inv = 1.f / l;
#pragma unroll
    for (int t = 0; t < DPL; ++t) dst[lane + 32 * t] = __float2bfloat16_rn(acc[t] * inv);
}

struct Plan {
    int row_tiles, n_splits, tiles_per_split, rows_total;
};
Plan make_plan(const ec_attn_desc& d, int n_active) {
    Plan pl;
    const int g = d.n_q_heads / d.n_kv_heads;
    pl.rows_total = n_active * g;
    pl.row_tiles = (pl.rows_total + BM - 1) / BM;
    const int key_tiles = (d.ctx_len + BN - 1) / BN;
    const long long base = (long long)pl.row_tiles * d.batch * d.n_kv_heads;
    const long long want = 2LL * sm_count();
    int splits = (int)((want + base - 1) / base);
    if (splits < 1) splits = 1;
    if (splits > key_tiles) splits = key_tiles;
    pl.tiles_per_split = (key_tiles + splits - 1) / splits;
    pl.n_splits = (key_tiles + pl.tiles_per_split - 1) / pl.tiles_per_split;
    return pl;
}

template <int D>
cudaError_t launch_d(const AttendArgs& a, const Plan& pl, cudaStream_t stream) {
    MmaParams p;
    p.q = static_cast<const __nv_bfloat16*>(a.q);
    p.k_cache = static_cast<const __nv_bfloat16*>(a.k_cache);
    p.v_cache = static_cast<const __nv_bfloat16*>(a.v_cache);
    p.out = static_cast<__nv_bfloat16*>(a.out);
    p.n_active = a.n_active;
    p.ctx_len = a.d.ctx_len;
    p.n_q_heads = a.d.n_q_heads;
    p.n_kv_heads = a.d.n_kv_heads;
    p.group = a.d.n_q_heads / a.d.n_kv_heads;
    p.rows_total = pl.rows_total;
    p.n_splits = pl.n_splits;
    p.tiles_per_split = pl.tiles_per_split;
    p.scale_log2 = a.scale * kLog2e;
    const long long slots = (long long)a.d.batch * a.d.n_kv_heads * pl.n_splits * pl.rows_total;
    p.part_o = static_cast<float*>(a.workspace);
    p.part_ml = reinterpret_cast<float2*>(static_cast<char*>(a.workspace) + (size_t)slots * D * sizeof(float));
    constexpr int smem = (BM + 4 * BN) * D * 2;
    static PerDeviceOnce attr_once;
    if (const cudaError_t ea = ensure_dynamic_smem(attr_once, attend_mma_kernel<D>, smem); ea != cudaSuccess) return ea;
    const dim3 grid(pl.row_tiles, pl.n_splits, a.d.batch * a.d.n_kv_heads);
    attend_mma_kernel<D><<<grid, kThreads, smem, stream>>>(p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (pl.n_splits > 1) {
        const dim3 cgrid((pl.rows_total + 3) / 4, 1, a.d.batch * a.d.n_kv_heads);
        attend_combine_kernel<D><<<cgrid, 128, 0, stream>>>(p);
        e = cudaGetLastError();
    }
    return e;
}

}  // namespace

size_t attend_workspace_bytes(const ec_attn_desc& d, int n_active) {
    if (d.dtype != EC_BF16 || n_active <= 0) return 16;
    const Plan pl = make_plan(d, n_active);
    if (pl.n_splits <= 1) return 16;
    const size_t slots = (size_t)d.batch * d.n_kv_heads * pl.n_splits * pl.rows_total;
    return slots * ((size_t)d.head_dim * sizeof(float) + sizeof(float2)) + 16;
}

cudaError_t launch_attend_bf16(const AttendArgs& a, cudaStream_t stream) {
    if (a.n_active == 0) return cudaSuccess;
    const Plan pl = make_plan(a.d, a.n_active);
    return a.d.head_dim == 64 ? launch_d<64>(a, pl, stream) : launch_d<128>(a, pl, stream);
}

}  // namespace ec
