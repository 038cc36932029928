// ec_attend, skip step with FEW query rows (bf16, head_dim 128, at most 64 packed query rows per kv head):
// ONE launch that refreshes the active rows' K/V in the cache, attends from the active rows over the whole
// cache and merges the key-range partials.  (Section 4.2 and Appendix A of the paper, partial branch:
// TransformerBlock(Q[M u R], K[I], V[I]) after the rows M u R got fresh K, V.)
//
// With 34 query rows a 128-row M tile would be three quarters padding, and a thread per query row would
// leave most softmax lanes idle.  Here the KEYS take the M axis of the tensor core and the query rows the N
// axis (N = 48 or 64):
//     S^T[128 keys x N]  = K_tile[128 keys x 128] . Q[N x 128]^T          (A = K tile, B = Q, both K-major)
//     O^T[128 d    x N] += V_tile^T[128 d x 128 keys] . P^T[128 keys x N]  (A = V tile MN-major, B = P^T MN-major)
// so a softmax thread owns one KEY (TMEM lane) and N scores: all 128 softmax lanes work, one exponential per
// (key, query) and no padding rows, and a step of the pipeline covers 128 keys.
//   softmax  the reference maxima m[q] (log2 units) are shared by all keys of the CTA and live in shared memory.
//            The common path computes p = 2^(s*scale*log2e - m[q]) with no reduction at all; a barrier-wide OR
//            tells whether any score exceeds its reference by more than 2^8 (always true on the first tile):
//            only then the column maxima are reduced (integer warp reductions + shared memory), m is raised,
//            and O^T and the partial row sums are rescaled.  Row sums are kept per thread (sum over its own
//            keys) and reduced across the CTA once, at the end;
//   grid     (C, B*H_kv*n_sub) as clusters of C in {1, 2, 4, 8} CTAs that split one head's 128-key tiles.  With
//            grouped-query attention the g = H_q/H_kv query heads of a kv head are packed into the N axis; when
//            n*g exceeds the 64 slots the heads are spread over n_sub CTA columns (each takes g/n_sub heads and
//            streams the same K/V, which the other columns' reads keep in L2).  Every column refreshes the rows of
//            its key range itself: the columns of a kv head write identical bytes, and each orders its own copy
//            before its own TMA reads, so whichever copy a read observes holds the fresh row;
//   refresh  as in the row-major skip kernel: a CTA refreshes the cache rows of its own key range, visits its
//            tiles in rotated order and waits for the copy only before the first tile that holds one;
//   merge    CTA c of the cluster owns the output columns d in [c*128/C, (c+1)*128/C): every CTA sends that
//            slice of its O^T (rows of the TMEM accumulator) plus its m and l vectors with one bulk
//            shared-to-shared copy per owner; the owner combines, normalises and writes out[b, i, h, d].
// warp 0: TMA producer (K and V tiles of 128 keys, one 4-D box each, NS stages of 64 KB); warp 1: refresh list
// and tcgen05.mma issue; warps 2..5: Q staging, refresh copy, softmax, exchange.  One CTA per SM.
// Launched with programmatic stream serialisation; global memory is touched only after griddepcontrol.wait.
// Every mbarrier wait is bounded (EC_ERR_TIMEOUT in dev_status, CTA-wide abort flag); the CTA always frees its
// TMEM and exits.
#include "ec_common.cuh"
#include "ec_tc_ptx.cuh"

#include <cstdio>

namespace ec {
namespace {

using namespace tc;

constexpr int BK = 128, HD = 128;
constexpr int kThreads = 192;
constexpr int kSoft = 128;
constexpr uint32_t SUB = 128 * 128;        // [128 rows x 64 bf16], 128-byte swizzle: 16 KB
constexpr uint32_t TILE = 2 * SUB;         // [128 x 128] bf16
constexpr uint32_t STAGE = 2 * TILE;       // K tile + V tile: 64 KB
constexpr uint32_t P_BYTES = SUB;          // P^T [128 keys x 64 query slots] bf16
constexpr int kMaxStages = 3;
constexpr int kMaxRowsT = 64;            // query slots (packed rows) of one CTA
constexpr int kMaxActive = 256;          // active rows of a sequence (refresh list, row chunks)
constexpr uint32_t TM_COLS = 256;          // S^T buffers at columns 0 and 64, O^T at 128
constexpr uint32_t TM_S = 0, TM_O = 128;
// exchange areas, reusing the dead staging memory after the main loop (bytes from the aligned base)
constexpr uint32_t kStagingOff = 36864;                       // row-sum scratch [128][N + 1] floats sits below it
constexpr uint32_t kExchangeMax = (128 * 65 + 2 * 64 * 8) * 4;   // C chunks of (128/C) x (N + 1) + 2N floats, N <= 64, C <= 8
constexpr uint32_t kRecvOff = kStagingOff + 40960;

enum { B_FULL = 0, B_EMPTY = kMaxStages, B_SFULL = 2 * kMaxStages, B_PFULL = B_SFULL + 2, B_PVDONE = B_PFULL + 1,
       B_QFULL = B_PVDONE + 1, B_LIST = B_QFULL + 1, B_REFRESHED = B_LIST + 1, B_RECV = B_REFRESHED + 1, B_COUNT = B_RECV + 1 };

typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pk(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void upk(f32x2 v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
// order-preserving map float -> int (for integer warp reductions of a maximum) and back
__device__ __forceinline__ int f2ord(float f) {
    const int i = __float_as_int(f);
    return i >= 0 ? i : (i ^ 0x7fffffff);
}
__device__ __forceinline__ float ord2f(int i) { return __int_as_float(i >= 0 ? i : (i ^ 0x7fffffff)); }

struct KeysParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k_new;   // nullptr: attend without refreshing
    const __nv_bfloat16* v_new;
    __nv_bfloat16* k_cache;
    __nv_bfloat16* v_cache;
    const int32_t* active_idx;    // nullptr: identity
    __nv_bfloat16* out;
    int32_t* dev_status;
    int n_active, ctx_len, n_q_heads, n_kv_heads;
    int group;        // query heads of one kv head handled by one CTA column (a divisor of H_q / H_kv)
    int rows_chunk;   // active rows handled by one CTA column (the last chunk may hold fewer)
    int n_sub_r;      // row chunks = ceil(n_active / rows_chunk)
    int n_sub;        // CTA columns per kv head = ((H_q / H_kv) / group) * n_sub_r
    int n_splits, tiles_per_split, n_stages;
    int q_tma;                    // 1: the producer fetches Q with one TMA box (MHA); 0: the softmax warps stage it
    uint32_t off_p, off_stage, off_list, off_bar;   // shared-memory carve (bytes from the 1024-aligned base); Q is at 0
    float scale_log2;
};

// words after the barrier block
struct alignas(16) KeysShared {
    uint32_t tmem;
    int abort_flag;
    int n_mine;       // entries of the refresh list
    int spec_ok;      // 1: the first tile of the range, loaded before the list was known, holds no refreshed row
    int first_tile;   // rotation of the visiting order, see tile_of()
    int j_refreshed;  // first visit index j whose tile holds a refreshed position (T if none)
    alignas(16) float m[kMaxRowsT];        // reference maxima of the query rows, log2 units (read as float2)
    alignas(16) float factor[kMaxRowsT];   // rescale factors of the current slow path; the row sums at the end
    int colmax[4][kMaxRowsT];      // per-warp column maxima (ordered ints) of the current slow path
};

template <int N>
__global__ void __launch_bounds__(kThreads, 1)
attend_skip_keys_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                        const __grid_constant__ CUtensorMap map_q, const KeysParams p) {
    static_assert(N == 48 || N == 64, "query-row slots per CTA");
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (s2u(smem_raw) + 1023u) & ~1023u;
    unsigned char* gbase = smem_raw + (base - s2u(smem_raw));
    const uint32_t bars = base + p.off_bar;
    KeysShared* sh = reinterpret_cast<KeysShared*>(gbase + p.off_bar + B_COUNT * 8);
    volatile int* abort_flag = &sh->abort_flag;
    int2* list = reinterpret_cast<int2*>(gbase + p.off_list);   // (active row i, position) pairs of this CTA's key range
    auto bar = [&](int idx) { return bars + idx * 8; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int split = blockIdx.x, bh = blockIdx.y / p.n_sub, sub = blockIdx.y % p.n_sub;
    const int b = bh / p.n_kv_heads, hk = bh % p.n_kv_heads;
    const int hq0 = (hk * (p.n_sub / p.n_sub_r) + sub / p.n_sub_r) * p.group;   // first query head of this CTA
    const int i0 = (sub % p.n_sub_r) * p.rows_chunk;                           // first active row of this CTA
    const int rows_total = min(p.rows_chunk, p.n_active - i0) * p.group;       // packed query rows of this CTA
    const int C = p.n_splits;
    const int DL = HD / C;                                 // output columns this CTA merges
    const int n_tiles_total = (p.ctx_len + BK - 1) / BK;
    const int t_begin = split * p.tiles_per_split;
    const int t_end = min(n_tiles_total, t_begin + p.tiles_per_split);
    const int T = t_end - t_begin;   // >= 1 by construction of the plan
    const int NS = p.n_stages;
    const bool refresh = p.k_new != nullptr;
    constexpr int NP = N + 1;   // odd row stride (floats) of the transposing buffers: conflict-free by row and by column
    const uint32_t chunk_bytes = (uint32_t)(DL * NP + 2 * N) * 4u;   // one owner's slice of O^T, then m[N], l[N]

    // ---- set-up (touches no global memory) -------------------------------------------------
    if (tid == 0) {
        prefetch_map(&map_k);
        prefetch_map(&map_v);
        if (p.q_tma) prefetch_map(&map_q);
        for (int i = 0; i < B_COUNT; ++i) {
            uint32_t count = 1;
            if (i == B_PFULL || i == B_REFRESHED || (i == B_QFULL && !p.q_tma)) count = kSoft;
            mbar_init(bar(i), count);
        }
        sh->abort_flag = 0;
        sh->n_mine = 0;
        sh->spec_ok = 1;
        sh->first_tile = 0;
        sh->j_refreshed = T;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (C > 1) mbar_expect_tx(bar(B_RECV), (uint32_t)C * chunk_bytes);
    }
    if (tid < N) sh->m[tid] = -INFINITY;
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s2u(&sh->tmem)), "r"(TM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        fence_before();
    }
    __syncthreads();
    fence_after();
    const uint32_t tmem = sh->tmem;
    pdl_wait();                    // the previous kernel of the stream has completed; global memory may be touched
    pdl_launch_dependents();

    const int key_lo = t_begin * BK, key_hi = min(p.ctx_len, t_end * BK);
    // Visiting order of the CTA's T tiles.  The producer loads the first tile of the range at once, before the
    // refresh list is known.  If that tile holds no refreshed row (spec_ok) it is visit 0 and the other tiles
    // follow in rotated order, those without refreshed rows first; otherwise its data are discarded (that stage
    // is simply filled again later) and all T tiles are visited in rotated order, shifted by one stage.
    auto tile_of = [&](int j, int spec_ok, int rot) {
        if (spec_ok) return j == 0 ? 0 : 1 + (rot + j - 1) % (T - 1);
        return (rot + j) % T;
    };

    if (warp == 0) {
        // ================================ TMA producer ======================================
        if (lane == 0) {
            if (p.q_tma) {   // Q first: [half][row][64 columns] of this head's rows, rows past n_active read as zero
                mbar_expect_tx(bar(B_QFULL), (uint32_t)N * 256u);
                tma_load_5d(base, &map_q, 0, i0, hq0, 0, b, bar(B_QFULL));   // rows past the chunk land in unused slots
            }
            auto load_tile = [&](int tile, int stage) {
                const int key0 = (t_begin + tile) * BK;
                const uint32_t dst = base + p.off_stage + stage * STAGE;
                mbar_expect_tx(bar(B_FULL + stage), STAGE);
                tma_load_4d(dst, &map_k, 0, key0, 0, bh, bar(B_FULL + stage));
                tma_load_4d(dst + TILE, &map_v, 0, key0, 0, bh, bar(B_FULL + stage));
            };
            int spec_ok = 1, rot = 0, j_refreshed = T;
            load_tile(0, 0);   // visit 0 if it turns out to hold no refreshed row
            if (refresh) {
                mbar_wait(bar(B_LIST), 0, abort_flag, p.dev_status);
                spec_ok = sh->spec_ok;
                rot = sh->first_tile;
                j_refreshed = sh->j_refreshed;
            }
            const int soff = spec_ok ? 0 : 1;   // stage shift: the discarded fill took stage 0's first phase
            bool discard_seen = spec_ok != 0;
            for (int j = spec_ok ? 1 : 0; j < T; ++j) {
                const int s = (j + soff) % NS, u = (j + soff) / NS;
                if (j == j_refreshed) mbar_wait(bar(B_REFRESHED), 0, abort_flag, p.dev_status);
                if (u > 0) {
                    if (soff == 1 && s == 0) {
                        // stage 0: its phase 0 was the discarded fill, which nobody consumes or releases
                        if (u == 1) {
                            mbar_wait(bar(B_FULL + 0), 0, abort_flag, p.dev_status);
                            discard_seen = true;
                        } else {
                            mbar_wait(bar(B_EMPTY + 0), (u - 2) & 1, abort_flag, p.dev_status);
                        }
                    } else {
                        mbar_wait(bar(B_EMPTY + s), (u - 1) & 1, abort_flag, p.dev_status);
                    }
                }
                load_tile(tile_of(j, spec_ok, rot), s);
            }
            if (!discard_seen) mbar_wait(bar(B_FULL + 0), 0, abort_flag, p.dev_status);   // no copy in flight at exit
        }
        if (C > 1) {   // this warp no longer touches the memory the peers' partials will land in
            __syncwarp();
            cluster_arrive();
        }
    } else if (warp == 1) {
        // ================= refresh list, then MMA issue (lane 0) =================================
        bool spec_ok_w1 = true;
        if (refresh) {
            int posv[kMaxActive / 32];
#pragma unroll
            for (int k = 0; k < kMaxActive / 32; ++k) {
                const int i = k * 32 + lane;
                posv[k] = -1;
                if (k * 32 >= p.n_active) continue;   // uniform: nothing of the list left
                if (i < p.n_active) posv[k] = p.active_idx ? __ldg(p.active_idx + (long long)b * p.n_active + i) : i;
            }
            int n_mine = 0, hi_tile = -1, lo_tile = T;   // last / first local tile that holds a refreshed position
#pragma unroll
            for (int k = 0; k < kMaxActive / 32; ++k) {
                if (k * 32 >= p.n_active) break;
                const bool hit = posv[k] >= key_lo && posv[k] < key_hi;
                const unsigned mk = __ballot_sync(0xffffffffu, hit);
                if (hit) {
                    list[n_mine + __popc(mk & ((1u << lane) - 1u))] = make_int2(k * 32 + lane, posv[k]);
                    hi_tile = max(hi_tile, (posv[k] - key_lo) / BK);
                    lo_tile = min(lo_tile, (posv[k] - key_lo) / BK);
                }
                n_mine += __popc(mk);
            }
            hi_tile = __reduce_max_sync(0xffffffffu, hi_tile);
            lo_tile = __reduce_min_sync(0xffffffffu, lo_tile);
            spec_ok_w1 = lo_tile > 0;   // the tile loaded ahead of this list holds no refreshed row
            int rot = 0;
            if (n_mine > 0) rot = spec_ok_w1 ? hi_tile % (T - 1) : (hi_tile + 1) % T;   // (spec_ok and n_mine > 0 imply T > 1)
            int j_ref = T;
#pragma unroll
            for (int k = 0; k < kMaxActive / 32; ++k) {
                if (k * 32 >= p.n_active) break;
                if (posv[k] >= key_lo && posv[k] < key_hi) {
                    const int tile = (posv[k] - key_lo) / BK;
                    int j;
                    if (spec_ok_w1) {
                        j = tile - 1 - rot;
                        if (j < 0) j += T - 1;
                        j += 1;
                    } else {
                        j = tile - rot;
                        if (j < 0) j += T;
                    }
                    j_ref = min(j_ref, j);
                }
            }
            j_ref = __reduce_min_sync(0xffffffffu, j_ref);
            __syncwarp();
            if (lane == 0) {
                sh->n_mine = n_mine;
                sh->spec_ok = spec_ok_w1 ? 1 : 0;
                sh->first_tile = rot;
                sh->j_refreshed = j_ref;
                mbar_arrive(bar(B_LIST));
            }
        }
        if (lane == 0) {
            constexpr uint32_t IDESC_S = instr_desc2(N, 0, 0);    // A = K tile (K-major), B = Q (K-major)
            constexpr uint32_t IDESC_PV = instr_desc2(N, 1, 1);   // A = V tile (MN-major: d contiguous), B = P^T (MN-major)
            constexpr uint32_t QHALF = N * 128;                   // bytes of one 64-column half of the Q tile
            const int soff = spec_ok_w1 ? 0 : 1;
            auto stage_of = [&](int j) { return (j + soff) % NS; };
            auto wait_stage = [&](int j) { mbar_wait(bar(B_FULL + stage_of(j)), ((j + soff) / NS) & 1, abort_flag, p.dev_status); };
            auto issue_s = [&](int j) {
                const uint32_t kst = base + p.off_stage + stage_of(j) * STAGE;
#pragma unroll
                for (int k = 0; k < HD / 16; ++k) {
                    const uint32_t koff = (k & 3) * 32;
                    mma_ss(tmem + TM_S + (j & 1) * 64, smem_desc(kst + (k >> 2) * SUB + koff, 16, 1024),
                           smem_desc(base + (k >> 2) * QHALF + koff, 16, 1024), IDESC_S, k > 0);
                }
                commit(bar(B_SFULL + (j & 1)));
            };
            mbar_wait(bar(B_QFULL), 0, abort_flag, p.dev_status);
            wait_stage(0);
            fence_after();
            issue_s(0);
            for (int j = 0; j < T; ++j) {
                if (j + 1 < T) {
                    wait_stage(j + 1);
                    fence_after();
                    issue_s(j + 1);
                }
                const uint32_t vst = base + p.off_stage + stage_of(j) * STAGE + TILE;
                mbar_wait(bar(B_PFULL), j & 1, abort_flag, p.dev_status);
                fence_after();
#pragma unroll
                for (int k = 0; k < BK / 16; ++k)
                    mma_ss(tmem + TM_O, smem_desc(vst + k * 2048, SUB, 1024), smem_desc(base + p.off_p + k * 2048, SUB, 1024),
                           IDESC_PV, (j > 0 || k > 0));
                commit(bar(B_PVDONE));
                commit(bar(B_EMPTY + stage_of(j)));
            }
        }
        if (C > 1) {   // (the products still in flight are covered by the softmax warps, which arrive after the last one)
            __syncwarp();
            cluster_arrive();
        }
    } else {
        // ================== Q staging, cache refresh, softmax (warps 2..5) ========================
        const int stid = tid - 64;
        constexpr uint32_t QHALF = N * 128;
        // Q rows of this kv head -> swizzled K-major tile of N rows (rows past rows_total are zero)
        for (int c = stid; c < (p.q_tma ? 0 : N * (HD / 8)); c += kSoft) {
            const int row = c >> 4, ch = c & 15;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (row < rows_total) {
                const int i = i0 + row / p.group, jh = row % p.group;
                v = __ldg(reinterpret_cast<const uint4*>(
                    p.q + (((long long)b * p.n_active + i) * p.n_q_heads + hq0 + jh) * HD + ch * 8));
            }
            const uint32_t off = (ch >> 3) * QHALF + (row >> 3) * 1024 + (row & 7) * 128 + (((ch & 7) ^ (row & 7)) << 4);
            *reinterpret_cast<uint4*>(gbase + off) = v;
        }
        if (!p.q_tma) {
            fence_async_smem();     // Q (generic proxy) -> visible to the tensor core (async proxy)
            mbar_arrive(bar(B_QFULL));
        }

        int spec_ok = 1, rot = 0;
        if (refresh) {
            mbar_wait(bar(B_LIST), 0, abort_flag, p.dev_status);
            spec_ok = sh->spec_ok;
            rot = sh->first_tile;
            // fresh rows of this CTA's key range -> cache in global memory, eight 16-byte pieces in flight per thread
            const int chunks = sh->n_mine * 32;
            for (int c0 = stid; c0 < chunks; c0 += 8 * kSoft) {
                uint4 v[8];
                long long dsto[8];
                int isv[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int c = c0 + u * kSoft;
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

        const int quarter = warp & 3;
        const int kk = quarter * 32 + lane;          // key of the tile == TMEM lane == output column d later on
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const float sl2 = p.scale_log2;
        const f32x2 sl2_2 = pk(sl2, sl2);
        f32x2 l2[N / 2];
#pragma unroll
        for (int i = 0; i < N / 2; ++i) l2[i] = pk(0.f, 0.f);
        unsigned char* prow = gbase + p.off_p + (kk >> 3) * 1024 + (kk & 7) * 128;

        for (int j = 0; j < T; ++j) {
            mbar_wait(bar(B_SFULL + (j & 1)), (j >> 1) & 1, abort_flag, p.dev_status);
            fence_after();
            uint32_t sr[N];
            const uint32_t s_addr = tmem + lane_addr + TM_S + (j & 1) * 64;
            ld32(s_addr, sr);
            if (N == 48) ld16(s_addr + 32, sr + 32); else ld32(s_addr + 32, sr + 32);
            wait_ld();
            const int key = (t_begin + tile_of(j, spec_ok, rot)) * BK + kk;
            if (key >= p.ctx_len) {   // only in the ragged last tile of the context
#pragma unroll
                for (int c = 0; c < N; ++c) sr[c] = 0xff800000u;   // -inf: probability 0 for every query
            }
            // d = s * scale * log2(e) - m[q]; does any score exceed its reference by more than 2^8?
            f32x2 d2[N / 2];
            float dmx0 = -INFINITY, dmx1 = -INFINITY;
#pragma unroll
            for (int i = 0; i < N / 2; ++i) {
                const float2 mm = *reinterpret_cast<const float2*>(&sh->m[2 * i]);
                d2[i] = fma2(pk(__uint_as_float(sr[2 * i]), __uint_as_float(sr[2 * i + 1])), sl2_2, pk(-mm.x, -mm.y));
                float d0, d1;
                upk(d2[i], d0, d1);
                if (i & 1) dmx1 = max3(dmx1, d0, d1); else dmx0 = max3(dmx0, d0, d1);
            }
            const bool slow = named_barrier_or(2, kSoft, fmaxf(dmx0, dmx1) > 8.f);
            if (slow) {
                // ---- rare path: raise the references to the column maxima of this tile, rescale l and O^T ----
#pragma unroll
                for (int c = 0; c < N; ++c) {
                    const int o = __reduce_max_sync(0xffffffffu, f2ord(__uint_as_float(sr[c])));
                    if (lane == (c & 31)) sh->colmax[quarter][c] = o;
                }
                named_barrier(3, kSoft);
                if (stid < N) {
                    const int o = max(max(sh->colmax[0][stid], sh->colmax[1][stid]), max(sh->colmax[2][stid], sh->colmax[3][stid]));
                    const float m_old = sh->m[stid];
                    const float m_new = fmaxf(m_old, ord2f(o) * sl2);
                    sh->factor[stid] = (m_old == -INFINITY) ? 0.f : fast_exp2(m_old - m_new);
                    sh->m[stid] = m_new;
                }
                named_barrier(3, kSoft);
#pragma unroll
                for (int i = 0; i < N / 2; ++i) {
                    const float2 ff = *reinterpret_cast<const float2*>(&sh->factor[2 * i]);
                    l2[i] = mul2(l2[i], pk(ff.x, ff.y));
                }
                if (j > 0) {   // O^T holds the tiles before j: P V of tile j - 1 must have completed
                    mbar_wait(bar(B_PVDONE), (j - 1) & 1, abort_flag, p.dev_status);
                    fence_after();
                    uint32_t o[N];
                    const uint32_t o_addr = tmem + lane_addr + TM_O;
                    ld32(o_addr, o);
                    if (N == 48) ld16(o_addr + 32, o + 32); else ld32(o_addr + 32, o + 32);
                    wait_ld();
#pragma unroll
                    for (int c = 0; c < N; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * sh->factor[c]);
                    st32(o_addr, o);
                    if (N == 48) st16(o_addr + 32, o + 32); else st32(o_addr + 32, o + 32);
                    wait_st();
                }
#pragma unroll
                for (int i = 0; i < N / 2; ++i) {
                    const float2 mm = *reinterpret_cast<const float2*>(&sh->m[2 * i]);
                    d2[i] = fma2(pk(__uint_as_float(sr[2 * i]), __uint_as_float(sr[2 * i + 1])), sl2_2, pk(-mm.x, -mm.y));
                }
            }
            uint32_t pw[N / 2];
#pragma unroll
            for (int i = 0; i < N / 2; ++i) {
                float d0, d1;
                upk(d2[i], d0, d1);
                const float e0 = fast_exp2(d0), e1 = fast_exp2(d1);
                l2[i] = add2(l2[i], pk(e0, e1));
                pw[i] = pack_bf16x2(e0, e1);
            }
            // the P^T buffer is free once P V of the previous tile has completed
            if (j > 0) mbar_wait(bar(B_PVDONE), (j - 1) & 1, abort_flag, p.dev_status);
#pragma unroll
            for (int ch = 0; ch < N / 8; ++ch)
                *reinterpret_cast<uint4*>(prow + ((ch ^ (kk & 7)) << 4)) = make_uint4(pw[4 * ch], pw[4 * ch + 1], pw[4 * ch + 2], pw[4 * ch + 3]);
            fence_async_smem();
            fence_before();
            mbar_arrive(bar(B_PFULL));
        }
        mbar_wait(bar(B_PVDONE), (T - 1) & 1, abort_flag, p.dev_status);   // Q, P^T and the K/V stages are dead from here on
        fence_after();
        if (C > 1) {
            // first cluster barrier, arrive half: from here on the peers may write their partials into this CTA's
            // receive buffer (dead stage memory that the reduction and the staging below do not touch)
            __syncwarp();
            cluster_arrive();
        }

        // ---- row sums over the CTA's keys: per-thread partials -> shared memory -> one thread per query ----
        float* lred = reinterpret_cast<float*>(gbase);   // [128 keys][NP]
#pragma unroll
        for (int i = 0; i < N / 2; ++i) {
            float a0, a1;
            upk(l2[i], a0, a1);
            lred[kk * NP + 2 * i] = a0;
            lred[kk * NP + 2 * i + 1] = a1;
        }
        named_barrier(3, kSoft);
        {   // two threads per query column, 64 keys each
            const int qc = stid & 63, half = stid >> 6;
            float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            if (qc < N) {
#pragma unroll
                for (int k = 0; k < 64; ++k) acc[k & 7] += lred[(half * 64 + k) * NP + qc];
            }
            const float part = ((acc[0] + acc[1]) + (acc[2] + acc[3])) + ((acc[4] + acc[5]) + (acc[6] + acc[7]));
            named_barrier(3, kSoft);   // every partial sum has been read out of lred
            if (qc < N) lred[half * N + qc] = part;
            named_barrier(3, kSoft);
            if (stid < N) sh->factor[stid] = lred[stid] + lred[N + stid];   // l[q] of this CTA
        }
        named_barrier(3, kSoft);

        uint32_t o[N];
        {
            const uint32_t o_addr = tmem + lane_addr + TM_O;
            ld32(o_addr, o);
            if (N == 48) ld16(o_addr + 32, o + 32); else ld32(o_addr + 32, o + 32);
            wait_ld();
        }
        if (C == 1) {
            // ---- single CTA per (sequence, kv head): normalise and store column kk of every query row ----
#pragma unroll
            for (int c = 0; c < N; ++c) {
                if (c < rows_total) {
                    const int i = i0 + c / p.group, jh = c % p.group;
                    __nv_bfloat16* dst = p.out + (((long long)b * p.n_active + i) * p.n_q_heads + hq0 + jh) * HD;
                    dst[kk] = __float2bfloat16_rn(__uint_as_float(o[c]) / sh->factor[c]);
                }
            }
        } else {
            // ---- this CTA's O^T row kk -> staging chunk of the CTA that owns output column kk ----
            float* stg = reinterpret_cast<float*>(gbase + kStagingOff) + (kk / DL) * (chunk_bytes / 4) + (kk % DL) * NP;
#pragma unroll
            for (int c = 0; c < N; ++c) stg[c] = __uint_as_float(o[c]);
            if (stid < N) {   // every owner also gets this CTA's m[q] and l[q]
                for (int c = 0; c < C; ++c) {
                    float* ml = reinterpret_cast<float*>(gbase + kStagingOff) + c * (chunk_bytes / 4) + DL * NP;
                    ml[stid] = sh->m[stid];
                    ml[N + stid] = sh->factor[stid];
                }
            }
            fence_async_smem();   // staging (generic proxy) -> bulk copies (async proxy)
        }
        fence_before();
    }

    if (C > 1) {
        // the slices are staged (CTA barrier: the softmax warps wrote them, warp 0 sends them) and every CTA of
        // the cluster is past its main loop (its Q, P^T and K/V stages are dead, its barriers initialised)
        __syncthreads();
        cluster_wait();
        if (warp == 0 && lane < C) {   // one bulk copy per owner into the owner's receive buffer
            const uint32_t src = base + kStagingOff + (uint32_t)lane * chunk_bytes;
            const uint32_t dst = map_to_cta(base + kRecvOff + (uint32_t)split * chunk_bytes, lane);
            bulk_copy_to_peer(dst, src, chunk_bytes, map_to_cta(bar(B_RECV), lane));
        }
        // ---- merge the C partials of the output columns this CTA owns -------------------------
        mbar_wait(bar(B_RECV), 0, abort_flag, p.dev_status);
        // second cluster barrier, arrive half: this CTA holds every peer's partial, i.e. the peers' copies out of
        // their staging areas have completed; the wait half, before leaving, overlaps the merge
        __syncwarp();
        cluster_arrive();
        const float* recv = reinterpret_cast<const float*>(gbase + kRecvOff);
        const int cf = (int)(chunk_bytes / 4);
        float* wgt = reinterpret_cast<float*>(gbase);   // [C][N] normalised weights 2^(m_s - m) / l, over the dead row-sum scratch
        long long* qoff = reinterpret_cast<long long*>(gbase + 4096);   // [N] element offset of each query row in out
        if (tid < N) {
            float m = -INFINITY;
            for (int s = 0; s < C; ++s) m = fmaxf(m, recv[s * cf + DL * NP + tid]);
            float l = 0.f;
            for (int s = 0; s < C; ++s) l = fmaf(fast_exp2(recv[s * cf + DL * NP + tid] - m), recv[s * cf + DL * NP + N + tid], l);
            const float inv = 1.f / l;
            for (int s = 0; s < C; ++s) wgt[s * N + tid] = fast_exp2(recv[s * cf + DL * NP + tid] - m) * inv;
            const int i = i0 + tid / p.group, jh = tid % p.group;
            qoff[tid] = (((long long)b * p.n_active + i) * p.n_q_heads + hq0 + jh) * HD + split * DL;
        }
        __syncthreads();
        // a thread owns two adjacent output columns of a query row: one 4-byte store
        const int half_dl = DL / 2;
        const int dp = tid % half_dl;
        for (int qq = tid / half_dl; qq < rows_total; qq += kThreads / half_dl) {
            float a0 = 0.f, a1 = 0.f;
            for (int s = 0; s < C; ++s) {
                const float w = wgt[s * N + qq];
                a0 = fmaf(w, recv[s * cf + (2 * dp) * NP + qq], a0);
                a1 = fmaf(w, recv[s * cf + (2 * dp + 1) * NP + qq], a1);
            }
            *reinterpret_cast<uint32_t*>(p.out + qoff[qq] + 2 * dp) = pack_bf16x2(a0, a1);
        }
        // no CTA leaves while a peer may still copy out of or into its shared memory
        __syncwarp();
        cluster_wait();
    }

    fence_before();
    __syncthreads();
    if (warp == 1) {
        fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TM_COLS) : "memory");
    }
}

// ---- host side ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// cache [B*Hkv, L, 128] bf16 seen as 4-D {64 columns, key, half, head}: one box {64, 128, 2, 1} lands as
// [half][key][64 columns], the two 128-byte-swizzled halves of a [128 keys x 128] tile; keys beyond L read as zero
bool make_cache_map(CUtensorMap* map, const void* cache, int bh, int ctx_len) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[4] = {64, (cuuint64_t)ctx_len, 2, (cuuint64_t)bh};
    const cuuint64_t strides[3] = {(cuuint64_t)HD * 2, 128, (cuuint64_t)ctx_len * HD * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)BK, 2, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(cache), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// q [B, n, H_q, 128] bf16 (MHA: one query head per kv head) seen as 5-D {64 columns, row, head, half, sequence}:
// the box {64, N, 1, 2, 1} lands as [half][row][64 columns], the K-major Q tile; rows past n read as zero
bool make_q_map(CUtensorMap* map, const void* q, int batch, int n_active, int n_q_heads, int n_slots) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[5] = {64, (cuuint64_t)n_active, (cuuint64_t)n_q_heads, 2, (cuuint64_t)batch};
    const cuuint64_t strides[4] = {(cuuint64_t)n_q_heads * HD * 2, (cuuint64_t)HD * 2, 128,
                                   (cuuint64_t)n_active * n_q_heads * HD * 2};
    const cuuint32_t box[5] = {64, (cuuint32_t)n_slots, 1, 2, 1};
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(q), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct KeysPlan {
    int group, rows_chunk, n_sub_r, n_sub;   // heads and active rows per CTA column, row chunks, CTA columns per kv head
    int n_slots, n_splits, tiles_per_split, n_stages;
    uint32_t off_p, off_stage, off_list, off_bar, smem_bytes;
};

constexpr uint32_t kSmemMax = 232448;   // 227 KB: largest dynamic allocation of one CTA

KeysPlan make_keys_plan(const ec_attn_desc& d, int n_active) {
    KeysPlan pl{};
    // a CTA column takes the largest divisor of the H_q / H_kv heads of a kv head whose packed rows fit the 64
    // query slots; the other columns of that kv head stream the same K/V (from L2) for their own heads
    const int g = d.n_q_heads / d.n_kv_heads;
    pl.group = g;
    while (pl.group > 1 && (g % pl.group != 0 || (long long)n_active * pl.group > kMaxRowsT)) --pl.group;
    // more active rows than slots (the paper's default budget k = 64 gives 96): the rows are cut into equal chunks,
    // one CTA column each
    pl.n_sub_r = (n_active * pl.group + kMaxRowsT - 1) / kMaxRowsT;
    pl.rows_chunk = (n_active + pl.n_sub_r - 1) / pl.n_sub_r;
    pl.n_sub_r = (n_active + pl.rows_chunk - 1) / pl.rows_chunk;
    pl.n_sub = (g / pl.group) * pl.n_sub_r;
    const int rows = pl.rows_chunk * pl.group;
    pl.n_slots = rows <= 48 ? 48 : 64;
    const int key_tiles = (d.ctx_len + BK - 1) / BK;
    const int bh = d.batch * d.n_kv_heads * pl.n_sub;
    // one CTA per SM; the cluster size divides the 128 output columns, every CTA gets at least one tile
    int c = 1;
    while (c < 8 && 2 * c * bh <= sm_count() && 2 * c <= key_tiles) c *= 2;
    pl.tiles_per_split = (key_tiles + c - 1) / c;
    while (c > 1 && (key_tiles + pl.tiles_per_split - 1) / pl.tiles_per_split < c) {   // no empty CTA
        c /= 2;
        pl.tiles_per_split = (key_tiles + c - 1) / c;
    }
    pl.n_splits = c;
    uint32_t off = (uint32_t)pl.n_slots * 256u;   // Q
    pl.off_p = off;
    off += P_BYTES;
    pl.off_stage = off;
    const uint32_t list = ((uint32_t)n_active * 8u + 15u) & ~15u;
    const uint32_t tail = list + B_COUNT * 8u + (uint32_t)sizeof(KeysShared) + 16u + 1024u;
    int ns = (int)((kSmemMax - off - tail) / STAGE);
    if (ns > kMaxStages) ns = kMaxStages;
    if (ns > pl.tiles_per_split && ns > 2) ns = pl.tiles_per_split < 2 ? 2 : pl.tiles_per_split;
    pl.n_stages = ns;
    off += (uint32_t)ns * STAGE;
    pl.off_list = off;
    off += list;
    pl.off_bar = off;
    off += B_COUNT * 8u + (uint32_t)sizeof(KeysShared) + 16u;
    pl.smem_bytes = off + 1024u;
    return pl;
}

template <int N>
cudaError_t launch_n(const KeysPlan& pl, const KeysParams& p, const CUtensorMap& mk, const CUtensorMap& mv,
                     const CUtensorMap& mq, int bh, cudaStream_t stream) {
    static PerDeviceOnce attr_once;
    if (const cudaError_t ea = ensure_dynamic_smem(attr_once, attend_skip_keys_kernel<N>, (int)kSmemMax); ea != cudaSuccess)
        return ea;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(pl.n_splits, bh, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
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
    return cudaLaunchKernelEx(&cfg, attend_skip_keys_kernel<N>, mk, mv, mq, p);
}

}  // namespace

bool attend_skip_keys_supported(const ec_attn_desc& d, int n_active) {
    if (d.dtype != EC_BF16 || d.head_dim != HD || n_active < 1) return false;
    if (n_active > kMaxActive) return false;
    const KeysPlan pl = make_keys_plan(d, n_active);
    if ((long long)d.batch * d.n_kv_heads * pl.n_sub > 65535) return false;   // grid.y
    // the exchange areas (row-sum scratch, staging, receive buffer) reuse the memory below the refresh list
    // one CTA per SM: beyond one wave of CTAs the row-major skip kernel (two CTAs per SM) streams better
    if ((long long)pl.n_splits * d.batch * d.n_kv_heads * pl.n_sub > sm_count()) return false;
    // row chunks re-read the K/V of a head once per chunk: only worth it while the keys can still be split
    if (pl.n_sub_r > 1 && pl.n_splits < 2) return false;
    return pl.n_stages >= 2 && pl.smem_bytes <= kSmemMax && kRecvOff + kExchangeMax <= pl.off_list;
}

void attend_skip_keys_describe(const ec_attn_desc& d, int n_active, char* buf, size_t len) {
    const KeysPlan pl = make_keys_plan(d, n_active);
    snprintf(buf, len, "attend_skip_keys_kernel<%d> grid=(%d,%d) cluster=%d stages=%d smem=%u", pl.n_slots, pl.n_splits,
             d.batch * d.n_kv_heads * pl.n_sub, pl.n_splits, pl.n_stages, pl.smem_bytes);
}

cudaError_t launch_attend_skip_keys(const AttendArgs& a, const void* k_new, const void* v_new, const int32_t* active_idx,
                                    cudaStream_t stream) {
    const KeysPlan pl = make_keys_plan(a.d, a.n_active);
    const int bh = a.d.batch * a.d.n_kv_heads;
    CUtensorMap map_k, map_v;
    if (!make_cache_map(&map_k, a.k_cache, bh, a.d.ctx_len) || !make_cache_map(&map_v, a.v_cache, bh, a.d.ctx_len))
        return cudaErrorInvalidValue;
    KeysParams p{};
    CUtensorMap map_q = map_k;   // unused unless q_tma
    p.q_tma = (pl.group == 1) ? 1 : 0;   // one query head per CTA column: its rows are one TMA box
    if (p.q_tma && !make_q_map(&map_q, a.q, a.d.batch, a.n_active, a.d.n_q_heads, pl.n_slots)) return cudaErrorInvalidValue;
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
    p.group = pl.group;
    p.rows_chunk = pl.rows_chunk;
    p.n_sub_r = pl.n_sub_r;
    p.n_sub = pl.n_sub;
    p.n_splits = pl.n_splits;
    p.tiles_per_split = pl.tiles_per_split;
    p.n_stages = pl.n_stages;
    p.off_p = pl.off_p;
    p.off_stage = pl.off_stage;
    p.off_list = pl.off_list;
    p.off_bar = pl.off_bar;
    p.scale_log2 = a.scale * kLog2e;
    return pl.n_slots == 48 ? launch_n<48>(pl, p, map_k, map_v, map_q, bh * pl.n_sub, stream)
                            : launch_n<64>(pl, p, map_k, map_v, map_q, bh * pl.n_sub, stream);
}

}  // namespace ec
