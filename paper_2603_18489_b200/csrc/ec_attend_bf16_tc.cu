// ec_attend, bf16 storage, head_dim 128: Blackwell tensor-core path (tcgen05 + TMEM + TMA).
//
// Active-row bidirectional attention over the full cache (Appendix A of the paper:
// partial branch with the active rows as queries, full branch when every row is
// active).  One CTA owns a 128-row tile of the flattened (active row x query heads
// of one kv head) axis and a contiguous range of 128-key tiles of that kv head.
//
// Roles (192 threads, warp-specialised):
//   warp 0      TMA producer: K and V tiles, [128 keys x 128 d] bf16 each, as two
//               64-column boxes with the 128-byte swizzle, two stages per operand,
//               full/empty mbarriers;
//   warp 1      MMA issuer (one elected thread): S = Q K^T (8 x tcgen05.mma
//               M128 N128 K16, both operands K-major in shared memory) into one of
//               two TMEM S buffers, then O += P V (P K-major from shared memory, V
//               MN-major) into the TMEM O accumulator; completion is signalled
//               with tcgen05.commit on mbarriers.  S of tile j+1 is issued before
//               P V of tile j so the tensor pipe works while the softmax runs;
//   warps 2..5  softmax: thread = one query row (TMEM lane).  tcgen05.ld of the
//               128 scores, running max / sum, exp2 with the scale folded in, P
//               rounded to bf16 and written to swizzled shared memory; the O
//               accumulator is only rescaled when a row maximum grows by more than
//               2^8 (the stale maximum stays the reference otherwise), epilogue
//               normalises and stores (or writes a split-KV partial).
// TMEM: columns [0,128) S0, [128,256) S1, [256,384) O (fp32), 512 allocated.
// Every mbarrier wait is bounded; a wait that runs out sets EC_ERR_TIMEOUT in the
// caller's dev_status word, raises a CTA-wide abort flag that makes all later
// waits fall through, and the CTA still frees its TMEM and exits.
#include "ec_common.cuh"
#include "ec_tc_ptx.cuh"

#include <cuda.h>

namespace ec {
namespace {

constexpr int BM = 128, BN = 128, HD = 128;
constexpr int kThreads = 192;
constexpr uint32_t SUB = 128 * 128;      // bytes of a [128 rows x 64 bf16] swizzled sub-tile
constexpr uint32_t TILE = 2 * SUB;       // [128 x 128] bf16
constexpr uint32_t OFF_Q = 0;
constexpr uint32_t OFF_K = TILE;                 // 2 stages
constexpr uint32_t OFF_V = OFF_K + 2 * TILE;     // 2 stages
constexpr uint32_t OFF_P = OFF_V + 2 * TILE;     // 2 buffers
constexpr uint32_t OFF_BAR = OFF_P + 2 * TILE;   // 224 KiB
constexpr uint32_t SMEM_BYTES = OFF_BAR + 256 + 1024;  // + barrier block + alignment slack

constexpr uint32_t TM_S0 = 0, TM_S1 = 128, TM_O = 256, TM_COLS = 512;

// barrier indices (8 bytes each) inside the barrier block
enum { B_KFULL = 0, B_KEMPTY = 2, B_VFULL = 4, B_VEMPTY = 6, B_SFULL = 8, B_PFULL = 10, B_PVDONE = 12, B_COUNT = 14 };

// ---- PTX wrappers -----------------------------------------------------------------
// mbarriers (bounded waits), shared-memory addresses and the async-proxy fence are the shared wrappers
using tc::s2u;
using tc::mbar_init;
using tc::mbar_arrive;
using tc::mbar_expect_tx;
using tc::mbar_try;
using tc::mbar_wait;
using tc::fence_async_smem;
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float* v) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_st32(uint32_t taddr, const float* v) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
        ::"r"(taddr),
          "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
          "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
          "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
          "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
          "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
          "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
          "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
          "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
        : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor version 1
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// instruction descriptor: D fp32, A/B bf16, M = 128, N = 128; b_mn = 1 when B is MN-major
__host__ __device__ constexpr uint32_t instr_desc(int b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn << 16) | ((uint32_t)(BN >> 3) << 17) |
           ((uint32_t)(BM >> 4) << 24);
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

struct TcParams {
    const __nv_bfloat16* q;
    __nv_bfloat16* out;
    float* part_o;    // [B*Hkv, n_splits, rows_total, 128]
    float2* part_ml;  // [B*Hkv, n_splits, rows_total] (m in log2 units, l)
    int32_t* dev_status;
    int n_active, ctx_len, n_q_heads, n_kv_heads, group, rows_total;
    int n_splits, tiles_per_split;
    float scale_log2;
};

__global__ void __launch_bounds__(kThreads, 1)
attend_tc_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v, const TcParams p) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (s2u(smem_raw) + 1023u) & ~1023u;
    unsigned char* gbase = smem_raw + (base - s2u(smem_raw));
    const uint32_t bars = base + OFF_BAR;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gbase + OFF_BAR + B_COUNT * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gbase + OFF_BAR + B_COUNT * 8 + 4);
    auto bar = [&](int idx) { return bars + idx * 8; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int row_tile = blockIdx.x, split = blockIdx.y, bh = blockIdx.z;
    const int b = bh / p.n_kv_heads, hk = bh % p.n_kv_heads;
    const int r0 = row_tile * BM;
    const int n_tiles_total = (p.ctx_len + BN - 1) / BN;
    const int t_begin = split * p.tiles_per_split;
    const int t_end = min(n_tiles_total, t_begin + p.tiles_per_split);
    const int T = t_end - t_begin;  // >= 1 by construction of the plan

    // ---- set-up: barriers, TMEM, Q tile ---------------------------------------------
    if (tid == 0) {
        for (int i = 0; i < B_COUNT; ++i) mbar_init(bar(i), (i == B_PFULL || i == B_PFULL + 1) ? 128u : 1u);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s2u(tmem_slot)), "r"(TM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // Q rows of this tile -> swizzled K-major tile (rows beyond rows_total are zero)
    for (int c = tid; c < BM * (HD / 8); c += kThreads) {
        const int row = c >> 4, ch = c & 15;
        const int r = r0 + row;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (r < p.rows_total) {
            const int i = r / p.group, j = r % p.group;
            v = __ldg(reinterpret_cast<const uint4*>(
                p.q + (((long long)b * p.n_active + i) * p.n_q_heads + hk * p.group + j) * HD + ch * 8));
        }
        const uint32_t off = OFF_Q + (ch >> 3) * SUB + (row >> 3) * 1024 + (row & 7) * 128 + (((ch & 7) ^ (row & 7)) << 4);
        *reinterpret_cast<uint4*>(gbase + off) = v;
    }
    fence_async_smem();  // generic-proxy writes of Q -> visible to the tensor core (async proxy)
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        // ================================ TMA producer ==================================
        if (lane == 0) {
            for (int j = 0; j < T; ++j) {
                const int s = j & 1, u = j >> 1;
                const int key0 = (t_begin + j) * BN;
                if (u > 0) mbar_wait(bar(B_KEMPTY + s), (u - 1) & 1, abort_flag, p.dev_status);
                mbar_expect_tx(bar(B_KFULL + s), TILE);
                tma_load_3d(base + OFF_K + s * TILE, &map_k, 0, key0, bh, bar(B_KFULL + s));
                tma_load_3d(base + OFF_K + s * TILE + SUB, &map_k, 64, key0, bh, bar(B_KFULL + s));
                if (u > 0) mbar_wait(bar(B_VEMPTY + s), (u - 1) & 1, abort_flag, p.dev_status);
                mbar_expect_tx(bar(B_VFULL + s), TILE);
                tma_load_3d(base + OFF_V + s * TILE, &map_v, 0, key0, bh, bar(B_VFULL + s));
                tma_load_3d(base + OFF_V + s * TILE + SUB, &map_v, 64, key0, bh, bar(B_VFULL + s));
            }
        }
    } else if (warp == 1) {
        // ================================ MMA issuer ====================================
        if (lane == 0) {
            constexpr uint32_t IDESC_S = instr_desc(0), IDESC_PV = instr_desc(1);
            auto issue_s = [&](int j) {
                const int s = j & 1;
                const uint32_t d = tmem + (s ? TM_S1 : TM_S0);
#pragma unroll
                for (int k = 0; k < HD / 16; ++k) {
                    const uint32_t koff = (k >> 2) * SUB + (k & 3) * 32;
                    tc_mma_ss(d, smem_desc(base + OFF_Q + koff, 16, 1024),
                              smem_desc(base + OFF_K + s * TILE + koff, 16, 1024), IDESC_S, k > 0);
                }
                tc_commit(bar(B_SFULL + s));
                tc_commit(bar(B_KEMPTY + s));
            };
            mbar_wait(bar(B_KFULL + 0), 0, abort_flag, p.dev_status);
            tc_fence_after();
            issue_s(0);
            for (int j = 0; j < T; ++j) {
                const int s = j & 1, u = j >> 1;
                if (j + 1 < T) {
                    mbar_wait(bar(B_KFULL + ((j + 1) & 1)), ((j + 1) >> 1) & 1, abort_flag, p.dev_status);
                    tc_fence_after();
                    issue_s(j + 1);
                }
                mbar_wait(bar(B_PFULL + s), u & 1, abort_flag, p.dev_status);
                mbar_wait(bar(B_VFULL + s), u & 1, abort_flag, p.dev_status);
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < BN / 16; ++k) {
                    const uint32_t poff = (k >> 2) * SUB + (k & 3) * 32;
                    tc_mma_ss(tmem + TM_O, smem_desc(base + OFF_P + s * TILE + poff, 16, 1024),
                              smem_desc(base + OFF_V + s * TILE + k * 2048, SUB, 1024), IDESC_PV, (j > 0 || k > 0));
                }
                tc_commit(bar(B_PVDONE + s));
                tc_commit(bar(B_VEMPTY + s));
            }
        }
    } else {
        // ================================ softmax warps =================================
        const int quarter = warp & 3;               // TMEM lanes this warp may touch
        const int row = quarter * 32 + lane;        // row of the tile == TMEM lane
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const int r = r0 + row;
        float m_used = -INFINITY, l_run = 0.f;
        const float sl2 = p.scale_log2;

        for (int j = 0; j < T; ++j) {
            const int s = j & 1, u = j >> 1;
            mbar_wait(bar(B_SFULL + s), u & 1, abort_flag, p.dev_status);
            tc_fence_after();
            float sc[BN];
            const uint32_t s_addr = tmem + lane_addr + (s ? TM_S1 : TM_S0);
#pragma unroll
            for (int c = 0; c < BN / 32; ++c) tc_ld32(s_addr + c * 32, sc + c * 32);
            tc_wait_ld();

            const int key0 = (t_begin + j) * BN;
            if (key0 + BN > p.ctx_len) {
#pragma unroll
                for (int c = 0; c < BN; ++c)
                    if (key0 + c >= p.ctx_len) sc[c] = -INFINITY;
            }
            float mx = sc[0];
#pragma unroll
            for (int c = 1; c < BN; ++c) mx = fmaxf(mx, sc[c]);
            const float m_tile = mx * sl2;
            float factor = 1.f;
            if (m_tile > m_used + 8.f || m_used == -INFINITY) {  // stale maximum allowed up to 2^8
                factor = (m_used == -INFINITY) ? 0.f : fast_exp2(m_used - m_tile);
                m_used = m_tile;
            }
            const bool need_rescale = (j > 0) && __any_sync(0xffffffffu, factor != 1.f);
            float rs = 0.f;
            const float mneg = -m_used;
#pragma unroll
            for (int c = 0; c < BN; ++c) {
                sc[c] = fast_exp2(fmaf(sc[c], sl2, mneg));
                rs += sc[c];
            }
            l_run = fmaf(l_run, factor, rs);

            if (u > 0) mbar_wait(bar(B_PVDONE + s), (u - 1) & 1, abort_flag, p.dev_status);  // P buffer s is free
            unsigned char* prow = gbase + OFF_P + s * TILE + (row >> 3) * 1024 + (row & 7) * 128;
#pragma unroll
            for (int ch = 0; ch < 16; ++ch) {
                uint4 v;
                v.x = pack2(sc[ch * 8 + 0], sc[ch * 8 + 1]);
                v.y = pack2(sc[ch * 8 + 2], sc[ch * 8 + 3]);
                v.z = pack2(sc[ch * 8 + 4], sc[ch * 8 + 5]);
                v.w = pack2(sc[ch * 8 + 6], sc[ch * 8 + 7]);
                *reinterpret_cast<uint4*>(prow + (ch >> 3) * SUB + (((ch & 7) ^ (row & 7)) << 4)) = v;
            }
            if (need_rescale) {
                // O holds tiles < j: wait for P V of tile j-1, then scale this row's accumulator
                mbar_wait(bar(B_PVDONE + ((j - 1) & 1)), ((j - 1) >> 1) & 1, abort_flag, p.dev_status);
                tc_fence_after();
#pragma unroll
                for (int c = 0; c < HD / 32; ++c) {
                    float o[32];
                    tc_ld32(tmem + lane_addr + TM_O + c * 32, o);
                    tc_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] *= factor;
                    tc_st32(tmem + lane_addr + TM_O + c * 32, o);
                }
                tc_wait_st();
            }
            fence_async_smem();
            tc_fence_before();
            mbar_arrive(bar(B_PFULL + s));
        }

        // ---- epilogue ------------------------------------------------------------------
        mbar_wait(bar(B_PVDONE + ((T - 1) & 1)), ((T - 1) >> 1) & 1, abort_flag, p.dev_status);
        tc_fence_after();
        const bool valid = r < p.rows_total;
        if (p.n_splits == 1) {
            const int i = valid ? r / p.group : 0, jh = valid ? r % p.group : 0;
            __nv_bfloat16* dst = p.out + (((long long)b * p.n_active + i) * p.n_q_heads + hk * p.group + jh) * HD;
            const float inv = 1.f / l_run;
#pragma unroll
            for (int c = 0; c < HD / 32; ++c) {
                float o[32];
                tc_ld32(tmem + lane_addr + TM_O + c * 32, o);
                tc_wait_ld();
                if (valid && !*abort_flag) {   // a CTA whose wait gave up stores nothing
#pragma unroll
                    for (int v4 = 0; v4 < 4; ++v4) {
                        uint4 w;
                        w.x = pack2(o[v4 * 8 + 0] * inv, o[v4 * 8 + 1] * inv);
                        w.y = pack2(o[v4 * 8 + 2] * inv, o[v4 * 8 + 3] * inv);
                        w.z = pack2(o[v4 * 8 + 4] * inv, o[v4 * 8 + 5] * inv);
                        w.w = pack2(o[v4 * 8 + 6] * inv, o[v4 * 8 + 7] * inv);
                        *reinterpret_cast<uint4*>(dst + c * 32 + v4 * 8) = w;
                    }
                }
            }
        } else {
            const long long slot = ((long long)bh * p.n_splits + split) * p.rows_total + (valid ? r : 0);
            float* dst = p.part_o + slot * HD;
#pragma unroll
            for (int c = 0; c < HD / 32; ++c) {
                float o[32];
                tc_ld32(tmem + lane_addr + TM_O + c * 32, o);
                tc_wait_ld();
                if (valid) {
#pragma unroll
                    for (int v4 = 0; v4 < 8; ++v4)
                        *reinterpret_cast<float4*>(dst + c * 32 + v4 * 4) =
                            make_float4(o[v4 * 4], o[v4 * 4 + 1], o[v4 * 4 + 2], o[v4 * 4 + 3]);
                }
            }
            if (valid) p.part_ml[slot] = make_float2(m_used, l_run);
        }
        tc_fence_before();
    }

    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TM_COLS) : "memory");
    }
}

// split-KV merge: out = sum_s 2^(m_s - m) O_s / sum_s 2^(m_s - m) l_s
__global__ void __launch_bounds__(128) attend_tc_combine_kernel(const TcParams p) {
    const int lane = threadIdx.x & 31;
    const int bh = blockIdx.z;
    const int r = blockIdx.x * 4 + (threadIdx.x >> 5);
    if (r >= p.rows_total) return;
    const int b = bh / p.n_kv_heads, hk = bh % p.n_kv_heads;
    float m = -INFINITY;
    for (int s = 0; s < p.n_splits; ++s)
        m = fmaxf(m, __ldcg(&p.part_ml[((long long)bh * p.n_splits + s) * p.rows_total + r]).x);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float l = 0.f;
    for (int s = 0; s < p.n_splits; ++s) {
        const long long slot = ((long long)bh * p.n_splits + s) * p.rows_total + r;
        const float2 ml = __ldcg(&p.part_ml[slot]);
        if (ml.y <= 0.f) continue;
        const float w = fast_exp2(ml.x - m);
        l = fmaf(w, ml.y, l);
        const float4 o = __ldcg(reinterpret_cast<const float4*>(p.part_o + slot * HD) + lane);
        acc.x = fmaf(w, o.x, acc.x);
        acc.y = fmaf(w, o.y, acc.y);
        acc.z = fmaf(w, o.z, acc.z);
        acc.w = fmaf(w, o.w, acc.w);
    }
    const int i = r / p.group, j = r % p.group;
    __nv_bfloat16* dst = p.out + (((long long)b * p.n_active + i) * p.n_q_heads + hk * p.group + j) * HD;
    const float inv = 1.f / l;
    uint2 w2;
    w2.x = pack2(acc.x * inv, acc.y * inv);
    w2.y = pack2(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2*>(dst + lane * 4) = w2;
}

// ---- host side ---------------------------------------------------------------------------
using tc::EncodeTiledFn;
using tc::encode_fn;

// cache [B*Hkv, L, 128] bf16 -> 3-D map {d, key, head}; box {64, 128, 1}; 128-byte swizzle; keys beyond L read as zero
bool make_cache_map(CUtensorMap* map, const void* cache, int bh, int ctx_len) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)HD, (cuuint64_t)ctx_len, (cuuint64_t)bh};
    const cuuint64_t strides[2] = {(cuuint64_t)HD * 2, (cuuint64_t)ctx_len * HD * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)BN, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(cache), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct TcPlan {
    int row_tiles, n_splits, tiles_per_split, rows_total;
};
TcPlan make_tc_plan(const ec_attn_desc& d, int n_active) {
    TcPlan pl;
    const int g = d.n_q_heads / d.n_kv_heads;
    pl.rows_total = n_active * g;
    pl.row_tiles = (pl.rows_total + BM - 1) / BM;
    const int key_tiles = (d.ctx_len + BN - 1) / BN;
    const long long base = (long long)pl.row_tiles * d.batch * d.n_kv_heads;
    const long long want = sm_count();  // one CTA per SM (224 KiB of shared memory each)
    int splits = (int)((want + base - 1) / base);
    if (splits < 1) splits = 1;
    if (splits > key_tiles) splits = key_tiles;
    pl.tiles_per_split = (key_tiles + splits - 1) / splits;
    pl.n_splits = (key_tiles + pl.tiles_per_split - 1) / pl.tiles_per_split;
    return pl;
}

}  // namespace

size_t attend_tc_workspace_bytes(const ec_attn_desc& d, int n_active) {
    if (n_active <= 0) return 16;
    const TcPlan pl = make_tc_plan(d, n_active);
    if (pl.n_splits <= 1) return 16;
    const size_t slots = (size_t)d.batch * d.n_kv_heads * pl.n_splits * pl.rows_total;
    return slots * ((size_t)HD * sizeof(float) + sizeof(float2)) + 16;
}

cudaError_t launch_attend_bf16_tc(const AttendArgs& a, cudaStream_t stream) {
    if (a.n_active == 0) return cudaSuccess;
    const TcPlan pl = make_tc_plan(a.d, a.n_active);
    const int bh = a.d.batch * a.d.n_kv_heads;
    CUtensorMap map_k, map_v;
    if (!make_cache_map(&map_k, a.k_cache, bh, a.d.ctx_len) || !make_cache_map(&map_v, a.v_cache, bh, a.d.ctx_len))
        return cudaErrorInvalidValue;
    TcParams p;
    p.q = static_cast<const __nv_bfloat16*>(a.q);
    p.out = static_cast<__nv_bfloat16*>(a.out);
    p.dev_status = a.dev_status;
    p.n_active = a.n_active;
    p.ctx_len = a.d.ctx_len;
    p.n_q_heads = a.d.n_q_heads;
    p.n_kv_heads = a.d.n_kv_heads;
    p.group = a.d.n_q_heads / a.d.n_kv_heads;
    p.rows_total = pl.rows_total;
    p.n_splits = pl.n_splits;
    p.tiles_per_split = pl.tiles_per_split;
    p.scale_log2 = a.scale * kLog2e;
    const size_t slots = (size_t)bh * pl.n_splits * pl.rows_total;
    p.part_o = static_cast<float*>(a.workspace);
    p.part_ml = reinterpret_cast<float2*>(static_cast<char*>(a.workspace) + slots * HD * sizeof(float));
    static PerDeviceOnce attr_once;
    if (const cudaError_t ea = ensure_dynamic_smem(attr_once, attend_tc_kernel, (int)SMEM_BYTES); ea != cudaSuccess) return ea;
    const dim3 grid(pl.row_tiles, pl.n_splits, bh);
    attend_tc_kernel<<<grid, kThreads, SMEM_BYTES, stream>>>(map_k, map_v, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (pl.n_splits > 1) {
        const dim3 cgrid((pl.rows_total + 3) / 4, 1, bh);
        attend_tc_combine_kernel<<<cgrid, 128, 0, stream>>>(p);
        e = cudaGetLastError();
    }
    return e;
}

}  // namespace ec
