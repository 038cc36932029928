// ec_attend, skip step (bf16, head_dim 128, at most 256 packed query rows per kv head):
// ONE launch that refreshes the active rows' K/V in the cache, attends from the active
// rows over the whole cache and merges the key-range partials -- no workspace, no second
// kernel.  (Section 4.2 and Appendix A of the paper, partial branch:
// TransformerBlock(Q[M u R], K[I], V[I]) after the rows M u R got fresh K, V.)
//
// The step is HBM-bound (every K/V byte of the cache is read exactly once) and, at the
// context lengths of a diffusion LM block, latency-bound: the design keeps every
// global round trip off the path between kernel start and the first K/V tile, and off
// the path between the last tile and the output.
//   grid     (C, B*H_kv), launched as clusters of C CTAs: the C CTAs of a cluster share
//            one (sequence, kv head) and split its 64-key tiles into C contiguous ranges;
//   rows     the n_active x (H_q/H_kv) query rows that share the kv head are packed
//            into one or two 128-row M tiles (NT); the same K/V tile serves both;
//   warp 1   scans active_idx for positions inside this CTA's key range (the refresh
//            list), then issues the tcgen05.mma (S = Q K^T, M128 N64 K16 x 8, into one of
//            two TMEM S buffers; O += P V, M128 N128 K16 x 4, P from shared memory, V
//            MN-major);
//   refresh  a CTA refreshes the cache rows of its own key range (no other CTA reads
//            them).  Its tiles are visited in rotated order, starting behind the last
//            tile that holds a refreshed position, so the tiles that need no refresh
//            stream while softmax warps without query rows copy the fresh rows into the
//            cache; the producer waits for that copy (generic-proxy writes, then a
//            proxy fence) only before the first tile that holds a refreshed position;
//   warp 0   TMA producer: one 4-D box per operand tile ([2 halves][64 keys][64 columns],
//            128-byte swizzle), NS stages, full/empty mbarriers;
//   warps 2+ load Q into swizzled shared memory, then run the softmax: thread = query
//            row = TMEM lane, running max and sum, exp2 with the scale folded in, lazy
//            rescale of O;
//   merge    the un-normalised rows (O, m, l) go from TMEM to a staging area grouped by
//            owner (row r belongs to CTA r mod C of the cluster) and from there with one
//            bulk shared-to-shared copy per owner into the owner's receive buffer,
//            completing on the owner's mbarrier; the owner combines the C partials,
//            normalises and writes out[b, i, h, :].
// Shared memory only holds the rows that exist: the tensor core always multiplies 128
// rows, and the rows past the last packed query row read whatever follows in the CTA's
// own allocation; rows of S, P and O are independent, so those values never reach a
// real row and are never stored.
// The kernel is launched with programmatic stream serialisation: everything before
// griddepcontrol.wait (barrier set-up, TMEM allocation, descriptor prefetch) may overlap
// the previous kernel of the stream; nothing in global memory is touched before it.
// Every mbarrier wait is bounded: a wait that runs out sets EC_ERR_TIMEOUT in the
// caller's dev_status word and a CTA-wide abort flag that makes all later waits fall
// through; the CTA still frees its TMEM and exits.
#include "ec_common.cuh"
#include "ec_tc_ptx.cuh"

#include <cuda.h>

#include <cstdio>

namespace ec {
namespace {

constexpr int BM = 128, BN = 64, HD = 128;
constexpr uint32_t KV_SUB = BN * 128;      // [64 keys x 64 bf16], 128-byte swizzle: 8 KB
constexpr uint32_t KV_TILE = 2 * KV_SUB;   // [64 keys x 128 bf16]
constexpr uint32_t STAGE = 2 * KV_TILE;    // K tile + V tile: 32 KB
constexpr int kMaxStages = 6;
constexpr int kRec = HD + 4;               // floats per exchanged row: O[128], m, l, pad (16-byte multiple)
constexpr int kMaxRows = 2 * BM;
constexpr int kMaxCluster = 8;

// barrier slots (8 bytes each)
enum {
    B_FULL = 0,                       // [kMaxStages] K/V tile landed
    B_EMPTY = kMaxStages,             // [kMaxStages] tile consumed
    B_SFULL = 2 * kMaxStages,         // [tile][2]
    B_PFULL = B_SFULL + 4,            // [tile]
    B_PVDONE = B_PFULL + 2,           // [tile]
    B_QFULL = B_PVDONE + 2,           // Q tiles staged
    B_LIST = B_QFULL + 1,             // refresh list built
    B_REFRESHED = B_LIST + 1,         // fresh rows of this CTA's key range are in the cache
    B_RECV = B_REFRESHED + 1,              // all partial rows this CTA owns have arrived
    B_COUNT = B_RECV + 1
};

// ---- PTX wrappers -----------------------------------------------------------------
// mbarriers (bounded waits), shared-memory addresses and the async-proxy fence are the shared wrappers
using tc::s2u;
using tc::mbar_init;
using tc::mbar_arrive;
using tc::mbar_expect_tx;
using tc::mbar_try;
using tc::mbar_wait;
using tc::fence_async_smem;
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

__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, int w, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(w), "r"(bar) : "memory");
}
// bulk copy from this CTA's shared memory into a peer's, completing (bytes) on the peer's mbarrier
__device__ __forceinline__ void bulk_copy_to_peer(uint32_t dst_cluster, uint32_t src_local, uint32_t bytes, uint32_t bar_cluster) {
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_cluster), "r"(src_local), "r"(bytes), "r"(bar_cluster) : "memory");
}
__device__ __forceinline__ void fence_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }
__device__ __forceinline__ void prefetch_map(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_smem_addr, uint32_t cta_rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_smem_addr), "r"(cta_rank));
    return r;
}

// shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor version 1
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// instruction descriptor: D fp32, A/B bf16, M = 128, N = n; b_mn = 1 when B is MN-major
__host__ __device__ constexpr uint32_t instr_desc(int n, int b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn << 16) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(BM >> 4) << 24);
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

struct SkipParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k_new;   // nullptr: attend without refreshing
    const __nv_bfloat16* v_new;
    __nv_bfloat16* k_cache;
    __nv_bfloat16* v_cache;
    const int32_t* active_idx;    // nullptr: identity
    __nv_bfloat16* out;
    int32_t* dev_status;
    int n_active, ctx_len, n_q_heads, n_kv_heads, group, rows_total;
    int n_splits, tiles_per_split, n_stages, rows_per_cta;
    // shared-memory carve (bytes from the 1024-aligned base)
    uint32_t off_q[2], off_p[2], rows_pad[2], off_stage, off_recv, off_list, off_bar;
    float scale_log2;
};

// words after the barrier block
struct SkipShared {
    uint32_t tmem;
    int abort_flag;
    int n_mine;       // entries of the refresh list
    int first_tile;   // rotation: the CTA visits its tiles in the order (first_tile + j) mod T
    int j_refreshed;  // first visit index j whose tile holds a refreshed position (T if none)
};

template <int NT>
__global__ void __launch_bounds__(64 + NT * 128, NT == 1 ? 2 : 1)
attend_skip_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v, const SkipParams p) {
    constexpr int kThreads = 64 + NT * 128;
    constexpr int kSoftThreads = NT * 128;
    constexpr uint32_t TM_COLS = NT * 256;   // per row tile: S0 [0,64), S1 [64,128), O [128,256)
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (s2u(smem_raw) + 1023u) & ~1023u;
    unsigned char* gbase = smem_raw + (base - s2u(smem_raw));
    const uint32_t bars = base + p.off_bar;
    SkipShared* sh = reinterpret_cast<SkipShared*>(gbase + p.off_bar + B_COUNT * 8);
    volatile int* abort_flag = &sh->abort_flag;
    int2* list = reinterpret_cast<int2*>(gbase + p.off_list);   // (active row i, position) pairs of this CTA's key range
    auto bar = [&](int idx) { return bars + idx * 8; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int split = blockIdx.x, bh = blockIdx.y;
    const int b = bh / p.n_kv_heads, hk = bh % p.n_kv_heads;
    const int C = p.n_splits;
    const int n_tiles_total = (p.ctx_len + BN - 1) / BN;
    const int t_begin = split * p.tiles_per_split;
    const int t_end = min(n_tiles_total, t_begin + p.tiles_per_split);
    const int T = t_end - t_begin;   // >= 1 by construction of the plan
    const int NS = p.n_stages;
    const int n_own = (p.rows_total - split + C - 1) / C;   // packed rows r = split + q * C merged by this CTA
    const bool refresh = p.k_new != nullptr;

    // softmax warps that own no query row copy the fresh rows; when every warp owns rows, all of them share it
    int n_idle = 0, my_idle = -1;
#pragma unroll
    for (int w = 2; w < 2 + NT * 4; ++w) {
        const int rows_w = min(BM, p.rows_total - ((w - 2) >> 2) * BM);
        if (!((w & 3) * 32 < rows_w)) {
            if (w == warp) my_idle = n_idle;
            ++n_idle;
        }
    }
    const int n_copy_threads = n_idle == 0 ? kSoftThreads : n_idle * 32;

    // ---- set-up (touches no global memory) -------------------------------------------------
    if (tid == 0) {
        prefetch_map(&map_k);
        prefetch_map(&map_v);
        for (int i = 0; i < B_COUNT; ++i) {
            uint32_t count = 1;
            if (i >= B_PFULL && i < B_PFULL + 2) {
                const int rows_t = min(BM, p.rows_total - (i - B_PFULL) * BM);
                count = rows_t > 0 ? 32u * ((rows_t + 31) / 32) : 1u;
            } else if (i == B_QFULL) {
                count = kSoftThreads;
            } else if (i == B_REFRESHED) {
                count = (uint32_t)n_copy_threads;
            }
            mbar_init(bar(i), count);
        }
        sh->abort_flag = 0;
        sh->n_mine = 0;
        sh->first_tile = 0;
        sh->j_refreshed = T;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (C > 1 && n_own > 0) mbar_expect_tx(bar(B_RECV), (uint32_t)(C * n_own * kRec * 4));
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s2u(&sh->tmem)), "r"(TM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        tc_fence_before();
    }
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh->tmem;
    pdl_wait();                    // the previous kernel of the stream has completed; global memory may be touched
    pdl_launch_dependents();

    // softmax role: warp w >= 2 owns TMEM lanes 32 * (w % 4) of row tile (w - 2) / 4; thread = query row
    const int soft_tile = warp >= 2 ? (warp - 2) >> 2 : 0;
    const int soft_row = (warp & 3) * 32 + lane;
    const int soft_rows_t = min(BM, p.rows_total - soft_tile * BM);
    const bool soft_active = warp >= 2 && (warp & 3) * 32 < soft_rows_t;   // warp-uniform
    const bool valid = soft_active && soft_row < soft_rows_t;
    const uint32_t tm_t = tmem + ((uint32_t)((warp & 3) * 32) << 16) + soft_tile * 256;
    float m_used = -INFINITY, l_run = 0.f;
    const int key_lo = t_begin * BN, key_hi = min(p.ctx_len, t_end * BN);

    if (warp == 0) {
        // ================================ TMA producer ======================================
        if (lane == 0) {
            int first_tile = 0, j_refreshed = T;
            if (refresh) {
                mbar_wait(bar(B_LIST), 0, abort_flag, p.dev_status);
                first_tile = sh->first_tile;
                j_refreshed = sh->j_refreshed;
            }
            for (int j = 0; j < T; ++j) {
                const int s = j % NS, u = j / NS;
                int tile = first_tile + j;
                if (tile >= T) tile -= T;
                const int key0 = (t_begin + tile) * BN;
                if (j == j_refreshed) mbar_wait(bar(B_REFRESHED), 0, abort_flag, p.dev_status);
                if (u > 0) mbar_wait(bar(B_EMPTY + s), (u - 1) & 1, abort_flag, p.dev_status);
                const uint32_t dst = base + p.off_stage + s * STAGE;
                mbar_expect_tx(bar(B_FULL + s), STAGE);
                tma_load_4d(dst, &map_k, 0, key0, 0, bh, bar(B_FULL + s));
                tma_load_4d(dst + KV_TILE, &map_v, 0, key0, 0, bh, bar(B_FULL + s));
            }
        }
    } else if (warp == 1) {
        // ================= refresh list, then MMA issue (lane 0) =================================
        if (refresh) {
            int posv[kMaxRows / 32];
#pragma unroll
            for (int k = 0; k < kMaxRows / 32; ++k) {
                const int i = k * 32 + lane;
                posv[k] = -1;
                if (i < p.n_active) posv[k] = p.active_idx ? __ldg(p.active_idx + (long long)b * p.n_active + i) : i;
            }
            int n_mine = 0;
            int hi_tile = -1;   // last local tile that holds a refreshed position
#pragma unroll
            for (int k = 0; k < kMaxRows / 32; ++k) {
                const bool hit = posv[k] >= key_lo && posv[k] < key_hi;
                const unsigned m = __ballot_sync(0xffffffffu, hit);
                if (hit) {
                    list[n_mine + __popc(m & ((1u << lane) - 1u))] = make_int2(k * 32 + lane, posv[k]);
                    hi_tile = max(hi_tile, (posv[k] - key_lo) / BN);
                }
                n_mine += __popc(m);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) hi_tile = max(hi_tile, __shfl_xor_sync(0xffffffffu, hi_tile, o));
            // rotate so that the last refreshed tile comes last; the first refreshed tile in that order:
            const int first_tile = n_mine > 0 ? (hi_tile + 1) % T : 0;
            int j_ref = T;
#pragma unroll
            for (int k = 0; k < kMaxRows / 32; ++k) {
                if (posv[k] >= key_lo && posv[k] < key_hi) {
                    int j = (posv[k] - key_lo) / BN - first_tile;
                    if (j < 0) j += T;
                    j_ref = min(j_ref, j);
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) j_ref = min(j_ref, __shfl_xor_sync(0xffffffffu, j_ref, o));
            __syncwarp();
            if (lane == 0) {
                sh->n_mine = n_mine;
                sh->first_tile = first_tile;
                sh->j_refreshed = j_ref;
                mbar_arrive(bar(B_LIST));
            }
        }
        if (lane == 0) {
            constexpr uint32_t IDESC_S = instr_desc(BN, 0), IDESC_PV = instr_desc(HD, 1);
            auto issue_s = [&](int j) {
                const uint32_t kst = base + p.off_stage + (j % NS) * STAGE;
#pragma unroll
                for (int t = 0; t < NT; ++t) {
                    const uint32_t d = tmem + t * 256 + (j & 1) * 64;
                    const uint32_t qh = p.rows_pad[t] * 128u;   // bytes of one 64-column half of the Q tile
#pragma unroll
                    for (int k = 0; k < HD / 16; ++k) {
                        tc_mma_ss(d, smem_desc(base + p.off_q[t] + (k >> 2) * qh + (k & 3) * 32, 16, 1024),
                                  smem_desc(kst + (k >> 2) * KV_SUB + (k & 3) * 32, 16, 1024), IDESC_S, k > 0);
                    }
                    tc_commit(bar(B_SFULL + t * 2 + (j & 1)));
                }
            };
            mbar_wait(bar(B_QFULL), 0, abort_flag, p.dev_status);
            mbar_wait(bar(B_FULL + 0), 0, abort_flag, p.dev_status);
            tc_fence_after();
            issue_s(0);
            for (int j = 0; j < T; ++j) {
                if (j + 1 < T) {
                    mbar_wait(bar(B_FULL + (j + 1) % NS), ((j + 1) / NS) & 1, abort_flag, p.dev_status);
                    tc_fence_after();
                    issue_s(j + 1);
                }
                const uint32_t vst = base + p.off_stage + (j % NS) * STAGE + KV_TILE;
#pragma unroll
                for (int t = 0; t < NT; ++t) {
                    mbar_wait(bar(B_PFULL + t), j & 1, abort_flag, p.dev_status);
                    tc_fence_after();
#pragma unroll
                    for (int k = 0; k < BN / 16; ++k) {
                        tc_mma_ss(tmem + t * 256 + 128, smem_desc(base + p.off_p[t] + k * 32, 16, 1024),
                                  smem_desc(vst + k * 2048, KV_SUB, 1024), IDESC_PV, (j > 0 || k > 0));
                    }
                    tc_commit(bar(B_PVDONE + t));
                }
                tc_commit(bar(B_EMPTY + j % NS));
            }
        }
    } else {
        // ================== Q staging, cache refresh, softmax (warps 2..) ========================
        const int stid = tid - 64;
        // Q rows of this kv head -> swizzled K-major tiles (rows past rows_total inside the padded tile are zero)
        for (int t = 0; t < NT; ++t) {
            const int rows_pad = (int)p.rows_pad[t];
            for (int c = stid; c < rows_pad * (HD / 8); c += kSoftThreads) {
                const int row = c >> 4, ch = c & 15;
                const int r = t * BM + row;
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                if (r < p.rows_total) {
                    const int i = r / p.group, j = r % p.group;
                    v = __ldg(reinterpret_cast<const uint4*>(
                        p.q + (((long long)b * p.n_active + i) * p.n_q_heads + hk * p.group + j) * HD + ch * 8));
                }
                const uint32_t off = p.off_q[t] + (ch >> 3) * (uint32_t)rows_pad * 128u + (row >> 3) * 1024 + (row & 7) * 128 +
                                     (((ch & 7) ^ (row & 7)) << 4);
                *reinterpret_cast<uint4*>(gbase + off) = v;
            }
        }
        fence_async_smem();         // Q tiles (generic proxy) -> visible to the tensor core (async proxy)
        mbar_arrive(bar(B_QFULL));

        int first_tile = 0;
        if (refresh) {
            mbar_wait(bar(B_LIST), 0, abort_flag, p.dev_status);
            first_tile = sh->first_tile;
            // fresh rows of this CTA's key range -> cache in global memory, eight 16-byte pieces in flight per thread
            if (n_idle == 0 || my_idle >= 0) {
                const int wid = n_idle == 0 ? stid : my_idle * 32 + lane;
                const int wn = n_copy_threads;
                const int chunks = sh->n_mine * 32;
                for (int c0 = wid; c0 < chunks; c0 += 8 * wn) {
                    uint4 v[8];
                    long long dsto[8];
                    int isv[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const int c = c0 + u * wn;
                        isv[u] = -1;
                        if (c < chunks) {
                            const int e = c >> 5, piece = c & 15;
                            isv[u] = (c >> 4) & 1;
                            const int2 ip = list[e];
                            const long long src = (((long long)b * p.n_active + ip.x) * p.n_kv_heads + hk) * HD + piece * 8;
                            dsto[u] = ((long long)bh * p.ctx_len + ip.y) * HD + piece * 8;
                            v[u] = __ldg(reinterpret_cast<const uint4*>((isv[u] ? p.v_new : p.k_new) + src));
                        }
                    }
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        if (isv[u] >= 0) *reinterpret_cast<uint4*>((isv[u] ? p.v_cache : p.k_cache) + dsto[u]) = v[u];
                }
                if (chunks > 0) {
                    __threadfence();
                    fence_async_global();   // generic-proxy writes above before this CTA's TMA reads of the same rows
                }
                mbar_arrive(bar(B_REFRESHED));
            }
        }

        if (soft_active) {
            const float sl2 = p.scale_log2;
            const int t = soft_tile;
            unsigned char* prow = gbase + p.off_p[t] + (soft_row >> 3) * 1024 + (soft_row & 7) * 128;
            const bool store_p = soft_row < (int)p.rows_pad[t];   // rows past the padded tile have no storage

            for (int j = 0; j < T; ++j) {
                mbar_wait(bar(B_SFULL + t * 2 + (j & 1)), (j >> 1) & 1, abort_flag, p.dev_status);
                tc_fence_after();
                float sc[BN];
                tc_ld32(tm_t + (j & 1) * 64, sc);
                tc_ld32(tm_t + (j & 1) * 64 + 32, sc + 32);
                tc_wait_ld();
                int tile = first_tile + j;
                if (tile >= T) tile -= T;
                const int key0 = (t_begin + tile) * BN;
                if (key0 + BN > p.ctx_len) {
#pragma unroll
                    for (int c = 0; c < BN; ++c)
                        if (key0 + c >= p.ctx_len) sc[c] = -INFINITY;
                }
                float mx4[4] = {sc[0], sc[1], sc[2], sc[3]};
#pragma unroll
                for (int c = 4; c < BN; ++c) mx4[c & 3] = fmaxf(mx4[c & 3], sc[c]);
                float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                if (!valid) mx = 0.f;                // padded lanes never ask for a rescale
                const float m_tile = mx * sl2;
                float factor = 1.f;
                if (m_tile > m_used + 8.f || m_used == -INFINITY) {   // stale maximum allowed up to 2^8
                    factor = (m_used == -INFINITY) ? 0.f : fast_exp2(m_used - m_tile);
                    m_used = m_tile;
                }
                const bool need_rescale = (j > 0) && __any_sync(0xffffffffu, factor != 1.f);
                float rs4[4] = {0.f, 0.f, 0.f, 0.f};
                const float mneg = -m_used;
#pragma unroll
                for (int c = 0; c < BN; ++c) {
                    sc[c] = fast_exp2(fmaf(sc[c], sl2, mneg));
                    rs4[c & 3] += sc[c];
                }
                l_run = fmaf(l_run, factor, (rs4[0] + rs4[1]) + (rs4[2] + rs4[3]));

                // P buffer free and O stable once P V of the previous tile has completed
                if (j > 0) mbar_wait(bar(B_PVDONE + t), (j - 1) & 1, abort_flag, p.dev_status);
                if (store_p) {
#pragma unroll
                    for (int ch = 0; ch < BN / 8; ++ch) {
                        uint4 v;
                        v.x = pack2(sc[ch * 8 + 0], sc[ch * 8 + 1]);
                        v.y = pack2(sc[ch * 8 + 2], sc[ch * 8 + 3]);
                        v.z = pack2(sc[ch * 8 + 4], sc[ch * 8 + 5]);
                        v.w = pack2(sc[ch * 8 + 6], sc[ch * 8 + 7]);
                        *reinterpret_cast<uint4*>(prow + ((ch ^ (soft_row & 7)) << 4)) = v;
                    }
                }
                if (need_rescale) {
                    tc_fence_after();
#pragma unroll
                    for (int c = 0; c < HD / 32; ++c) {
                        float o[32];
                        tc_ld32(tm_t + 128 + c * 32, o);
                        tc_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] *= factor;
                        tc_st32(tm_t + 128 + c * 32, o);
                    }
                    tc_wait_st();
                }
                fence_async_smem();
                tc_fence_before();
                mbar_arrive(bar(B_PFULL + t));
            }
            // all row tiles have finished their last P V: Q, P and the K/V stages are dead from here on
#pragma unroll
            for (int tt = 0; tt < NT; ++tt) mbar_wait(bar(B_PVDONE + tt), (T - 1) & 1, abort_flag, p.dev_status);
            tc_fence_after();

            const int r = t * BM + soft_row;
            if (C == 1) {
                // ---- single CTA per (sequence, kv head): normalise and store -------------------
                const int i = valid ? r / p.group : 0, jh = valid ? r % p.group : 0;
                __nv_bfloat16* dst = p.out + (((long long)b * p.n_active + i) * p.n_q_heads + hk * p.group + jh) * HD;
                const float inv = 1.f / l_run;
#pragma unroll
                for (int c = 0; c < HD / 32; ++c) {
                    float o[32];
                    tc_ld32(tm_t + 128 + c * 32, o);
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
                // ---- un-normalised row -> staging, grouped by owner (CTA r mod C) -----------------
                float* rec = reinterpret_cast<float*>(gbase) +
                             (valid ? ((r % C) * p.rows_per_cta + r / C) : 0) * kRec;   // staging reuses the dead Q/P/stage memory
#pragma unroll
                for (int c = 0; c < HD / 32; ++c) {
                    float o[32];
                    tc_ld32(tm_t + 128 + c * 32, o);
                    tc_wait_ld();
                    if (valid) {
#pragma unroll
                        for (int v4 = 0; v4 < 8; ++v4)
                            *reinterpret_cast<float4*>(rec + c * 32 + v4 * 4) =
                                make_float4(o[v4 * 4], o[v4 * 4 + 1], o[v4 * 4 + 2], o[v4 * 4 + 3]);
                    }
                }
                if (valid) *reinterpret_cast<float4*>(rec + HD) = make_float4(m_used, l_run, 0.f, 0.f);
                fence_async_smem();   // staging (generic proxy) -> bulk copies (async proxy)
            }
        }
    }

    if (C > 1) {
        // every CTA of the cluster is past its main loop (its Q, P and K/V stages are dead, its barriers
        // initialised) and has staged its rows
        __syncwarp();
        cluster_arrive();
        cluster_wait();
        // one bulk copy per owner into the owner's receive buffer, issued by the first C lanes of warp 0
        if (warp == 0 && lane < C) {
            const int owner = lane;
            const int n_rows_owner = (p.rows_total - owner + C - 1) / C;
            if (n_rows_owner > 0) {
                const uint32_t src = base + (uint32_t)(owner * p.rows_per_cta * kRec) * 4u;
                const uint32_t dst = map_to_cta(base + p.off_recv + (uint32_t)(split * p.rows_per_cta * kRec) * 4u, owner);
                bulk_copy_to_peer(dst, src, (uint32_t)(n_rows_owner * kRec) * 4u, map_to_cta(bar(B_RECV), owner));
            }
        }
        // ---- merge the C partials of the rows this CTA owns ------------------------------------
        if (n_own > 0) {
            mbar_wait(bar(B_RECV), 0, abort_flag, p.dev_status);
            const float* recv = reinterpret_cast<const float*>(gbase + p.off_recv);
            for (int qi = warp; qi < n_own; qi += kThreads / 32) {
                const int r = split + qi * C;
                // lane s < C holds (m_s, l_s); the weights are shared through shuffles
                float ms = -INFINITY, ls = 0.f;
                if (lane < C) {
                    const float2 ml = *reinterpret_cast<const float2*>(recv + (lane * p.rows_per_cta + qi) * kRec + HD);
                    ms = ml.x;
                    ls = ml.y;
                }
                float m = ms;
#pragma unroll
                for (int o = 4; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
                m = __shfl_sync(0xffffffffu, m, 0);
                const float ws = lane < C ? fast_exp2(ms - m) : 0.f;
                float l = ws * ls;
#pragma unroll
                for (int o = 4; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
                l = __shfl_sync(0xffffffffu, l, 0);
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int s = 0; s < kMaxCluster; ++s) {
                    if (s < C) {
                        const float w = __shfl_sync(0xffffffffu, ws, s);
                        const float4 o = *reinterpret_cast<const float4*>(recv + (s * p.rows_per_cta + qi) * kRec + lane * 4);
                        acc.x = fmaf(w, o.x, acc.x);
                        acc.y = fmaf(w, o.y, acc.y);
                        acc.z = fmaf(w, o.z, acc.z);
                        acc.w = fmaf(w, o.w, acc.w);
                    }
                }
                const int i = r / p.group, jh = r % p.group;
                __nv_bfloat16* dst = p.out + (((long long)b * p.n_active + i) * p.n_q_heads + hk * p.group + jh) * HD;
                const float inv = 1.f / l;
                uint2 w2;
                w2.x = pack2(acc.x * inv, acc.y * inv);
                w2.y = pack2(acc.z * inv, acc.w * inv);
                if (!*abort_flag) *reinterpret_cast<uint2*>(dst + lane * 4) = w2;   // nothing from a CTA whose wait gave up
            }
        }
        // no CTA leaves while a peer may still copy out of or into its shared memory
        __syncwarp();
        cluster_arrive();
        cluster_wait();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TM_COLS) : "memory");
    }
}

// ---- host side ---------------------------------------------------------------------------
using tc::EncodeTiledFn;
using tc::encode_fn;

// cache [B*Hkv, L, 128] bf16 seen as 4-D {64 columns, key, half, head}: one box {64, 64, 2, 1} lands as
// [half][key][64 columns], i.e. the two 128-byte-swizzled halves of a [64 keys x 128] tile back to back; keys
// beyond L read as zero
bool make_cache_map(CUtensorMap* map, const void* cache, int bh, int ctx_len) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[4] = {64, (cuuint64_t)ctx_len, 2, (cuuint64_t)bh};
    const cuuint64_t strides[3] = {(cuuint64_t)HD * 2, 128, (cuuint64_t)ctx_len * HD * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)BN, 2, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(cache), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct SkipPlan {
    int nt, rows_total, n_splits, tiles_per_split, n_stages, rows_per_cta;
    uint32_t off_q[2], off_p[2], rows_pad[2], off_stage, off_recv, off_list, off_bar, smem_bytes;
};

constexpr uint32_t kSmemTwoPerSm = 115712;   // (228 KB per SM - 2 x 1 KB reserved) / 2
constexpr uint32_t kSmemMax = 232448;        // 227 KB: largest dynamic allocation of one CTA

SkipPlan make_skip_plan(const ec_attn_desc& d, int n_active) {
    SkipPlan pl{};
    const int g = d.n_q_heads / d.n_kv_heads;
    pl.rows_total = n_active * g;
    pl.nt = pl.rows_total > BM ? 2 : 1;
    const int key_tiles = (d.ctx_len + BN - 1) / BN;
    const int bh = d.batch * d.n_kv_heads;
    const int slots = (pl.nt == 1 ? 2 : 1) * sm_count();   // co-resident CTAs
    int c = slots / bh;
    if (c < 1) c = 1;
    if (c > kMaxCluster) c = kMaxCluster;
    if (c > key_tiles) c = key_tiles;
    pl.tiles_per_split = (key_tiles + c - 1) / c;
    pl.n_splits = (key_tiles + pl.tiles_per_split - 1) / pl.tiles_per_split;
    pl.rows_per_cta = (pl.rows_total + pl.n_splits - 1) / pl.n_splits;
    uint32_t off = 0;
    for (int t = 0; t < 2; ++t) {
        const int rows_t = t < pl.nt ? (pl.rows_total - t * BM < BM ? pl.rows_total - t * BM : BM) : 0;
        pl.rows_pad[t] = (uint32_t)((rows_t + 7) / 8 * 8);
        pl.off_q[t] = off;
        off += pl.rows_pad[t] * 256u;
    }
    for (int t = 0; t < 2; ++t) {
        pl.off_p[t] = off;
        off += pl.rows_pad[t] * 128u;
    }
    pl.off_stage = off;   // multiple of 1024: every piece above is a multiple of 8 rows x 128 bytes
    // the exchange areas (staging, then receive buffer) reuse the memory below the list once the main loop is over
    const uint32_t recv = pl.n_splits > 1 ? (uint32_t)(pl.n_splits * pl.rows_per_cta * kRec * 4) : 0u;
    const uint32_t list = ((uint32_t)n_active * 8u + 15u) & ~15u;
    const uint32_t tail = list + B_COUNT * 8u + 32u + 1024u;   // + barrier block + alignment slack
    int ns = 0;
    if (pl.nt == 1) {   // two CTAs per SM when at least two stages fit in half an SM
        ns = off + tail < kSmemTwoPerSm ? (int)((kSmemTwoPerSm - off - tail) / STAGE) : 0;
        if (ns > 3) ns = 3;
    }
    if (ns < 2) {
        ns = off + tail < kSmemMax ? (int)((kSmemMax - off - tail) / STAGE) : 0;
        if (ns > kMaxStages) ns = kMaxStages;
    }
    if (ns > pl.tiles_per_split && ns > 2) ns = pl.tiles_per_split < 2 ? 2 : pl.tiles_per_split;
    pl.n_stages = ns;
    off += (uint32_t)ns * STAGE;
    pl.off_recv = recv;   // right behind the staging area, which starts at 0
    pl.off_list = off;
    off += list;
    pl.off_bar = off;
    off += B_COUNT * 8u + 32u;
    pl.smem_bytes = off + 1024u;
    return pl;
}

template <int NT>
cudaError_t launch_nt(const SkipPlan& pl, const SkipParams& p, const CUtensorMap& mk, const CUtensorMap& mv, int bh,
                      cudaStream_t stream) {
    static PerDeviceOnce attr_once;
    if (const cudaError_t ea = ensure_dynamic_smem(attr_once, attend_skip_kernel<NT>, (int)kSmemMax); ea != cudaSuccess) return ea;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(pl.n_splits, bh, 1);
    cfg.blockDim = dim3(64 + NT * 128, 1, 1);
    cfg.dynamicSmemBytes = pl.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = pl.n_splits;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // set-up may overlap the previous kernel's tail
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, attend_skip_kernel<NT>, mk, mv, p);
}

}  // namespace

bool attend_skip_supported(const ec_attn_desc& d, int n_active) {
    if (d.dtype != EC_BF16 || d.head_dim != HD || n_active < 1) return false;
    const long long rows = (long long)n_active * (d.n_q_heads / d.n_kv_heads);
    if (rows > kMaxRows) return false;
    if ((long long)d.batch * d.n_kv_heads > 65535) return false;                       // grid.y
    const SkipPlan pl = make_skip_plan(d, n_active);
    const size_t exchange = pl.n_splits > 1 ? 2 * (size_t)pl.n_splits * pl.rows_per_cta * kRec * 4 : 0;
    return pl.n_stages >= 2 && pl.smem_bytes <= kSmemMax && exchange <= pl.off_list;
}

void attend_skip_describe(const ec_attn_desc& d, int n_active, char* buf, size_t len) {
    const SkipPlan pl = make_skip_plan(d, n_active);
    snprintf(buf, len, "attend_skip_kernel<%d> grid=(%d,%d) cluster=%d stages=%d smem=%u", pl.nt, pl.n_splits,
             d.batch * d.n_kv_heads, pl.n_splits, pl.n_stages, pl.smem_bytes);
}

cudaError_t launch_attend_skip(const AttendArgs& a, const void* k_new, const void* v_new, const int32_t* active_idx,
                               cudaStream_t stream) {
    const SkipPlan pl = make_skip_plan(a.d, a.n_active);
    const int bh = a.d.batch * a.d.n_kv_heads;
    CUtensorMap map_k, map_v;
    if (!make_cache_map(&map_k, a.k_cache, bh, a.d.ctx_len) || !make_cache_map(&map_v, a.v_cache, bh, a.d.ctx_len))
        return cudaErrorInvalidValue;
    SkipParams p{};
    p.q = static_cast<const __nv_bfloat16*>(a.q);
    p.k_new = static_cast<const __nv_bfloat16*>(k_new);
    p.v_new = static_cast<const __nv_bfloat16*>(v_new);
    p.k_cache = static_cast<__nv_bfloat16*>(const_cast<void*>(a.k_cache));
    p.v_cache = static_cast<__nv_bfloat16*>(const_cast<void*>(a.v_cache));
    p.active_idx = active_idx;
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
    p.n_stages = pl.n_stages;
    p.rows_per_cta = pl.rows_per_cta;
    for (int t = 0; t < 2; ++t) {
        p.off_q[t] = pl.off_q[t];
        p.off_p[t] = pl.off_p[t];
        p.rows_pad[t] = pl.rows_pad[t];
    }
    p.off_stage = pl.off_stage;
    p.off_recv = pl.off_recv;
    p.off_list = pl.off_list;
    p.off_bar = pl.off_bar;
    p.scale_log2 = a.scale * kLog2e;
    return pl.nt == 1 ? launch_nt<1>(pl, p, map_k, map_v, bh, stream) : launch_nt<2>(pl, p, map_k, map_v, bh, stream);
}

}  // namespace ec
