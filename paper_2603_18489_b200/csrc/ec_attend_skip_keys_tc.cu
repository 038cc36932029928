// ec_attend, skip step with FEW query rows (bf16, head_dim 128, at most 96 packed query rows per CTA column):
// ONE launch that refreshes the active rows' K/V in the cache, attends from the active rows over the whole
// cache and merges the key-range partials.  (Section 4.2 and Appendix A of the paper, partial branch:
// TransformerBlock(Q[M u R], K[I], V[I]) after the rows M u R got fresh K, V.)
//
// With 34 query rows a 128-row M tile would be three quarters padding, and a thread per query row would
// leave most softmax lanes idle.  Here the KEYS take the M axis of the tensor core and the query rows the N
// axis (N = 48, 64 or 96 slots):
//     S^T[128 keys x N]  = K_tile[128 keys x 128] . Q[N x 128]^T          (A = K tile, B = Q, both K-major)
//     O^T[128 d    x N] += V_tile^T[128 d x 128 keys] . P^T[128 keys x N]  (A = V tile MN-major, B = P^T MN-major)
// so a softmax thread owns one KEY (TMEM lane) and its scores against the query slots: all 128 lanes work, one
// exponential per (key, query), no padding rows, a pipeline step covers 128 keys.  The row sums sum_keys P are
// taken by two auxiliary warps that read P^T back from shared memory (where the softmax threads put it for the
// second product), so the softmax threads carry no running sums.  With N = 96 (the paper's default budget k = 64
// gives 96 active rows) two softmax warpgroups share the columns of a key.
//   softmax  the reference maxima m[q] (log2 units) are shared by all keys of the CTA and live in shared memory.
//            The common path computes p = 2^(s*scale*log2e - m[q]) with no reduction at all; a barrier-wide OR
//            tells whether any score exceeds its reference by more than 2^8 (always true on the first tile):
//            only then the column maxima are reduced, m is raised, and O^T and the row sums are rescaled;
//   grid     (C, B*H_kv*n_sub) as clusters of C <= 8 CTAs (any count, not only powers of two) that split one
//            head's 128-key tiles, chosen so that the most-loaded SM streams the fewest tiles; CTAs that hold a
//            single tile are small enough for two per SM.  With grouped-query attention the query heads of a kv
//            head are packed into the N axis; when they exceed the slots the heads (and, beyond 96 active rows,
//            the rows) are spread over n_sub CTA columns that stream the same K/V (L2 serves the repeats);
//   K/V      the producer warp issues its TMA loads in key order through a ring of NS slots of 32 KB (K_0 V_0 K_1 V_1
//            ...: a K slot is free again as soon as the scores of its tile are computed, a V slot after the second
//            product, and an odd slot count is possible, which is what lets the 96-slot instantiation keep two and
//            a half tiles in flight); the loads depend on nothing, and the first fill of the ring is spaced in time
//            (one tile of every CTA per interval) so that the memory system always has requests queued while the
//            first tiles are consumed;
//   refresh  the active rows' fresh K/V reach the attention straight from k_new / v_new, not through the cache: one
//            CTA of every cluster (the last) attends to them as one or two EXTRA key tiles, fetched by TMA from the
//            fresh tensors (a [128 rows x 128] box of k_new is laid out exactly like a cache tile) after its cache
//            tiles (visited first they held a ring stage through the start of the stream and set that CTA two tile
//            times behind its peers), while every CTA masks the stale cached keys of the refreshed positions (a bit per key, built from
//            the index list).  The attention therefore never waits for the cache update: the auxiliary warps of that
//            CTA copy the fresh rows from the landed tile to the cache in global memory with plain 16-byte stores,
//            for later steps, ordered against nothing.  (Keys
//            in a different order, the same sum.)  When a CTA holds a single cache tile the extra tiles get a CTA of
//            their own, so that nobody streams two tiles through one stage;
//   merge    CTA c of the cluster owns the output columns d in [c*DL, (c+1)*DL): once every CTA of the cluster is
//            past its last product (first cluster barrier, arrive early / wait late) each softmax thread puts its
//            O^T row (one output column, all queries) into a local staging chunk per owner, next to m and l; one
//            bulk copy per owner moves the chunk into the owner's shared memory and completes on the owner's
//            mbarrier; the owner combines the C partials, normalises and writes out[b, i, h, d]; a second cluster
//            barrier keeps every CTA's shared memory alive until its peers have read it.
// warp 0: TMA producer; warp 1: stale-key masks, then tcgen05.mma issue; next 4 (or 8) warps: softmax; last two
// warps: cache update and row sums.  Launched with programmatic stream serialisation; global memory is touched only after
// griddepcontrol.wait.  Every mbarrier wait is bounded (EC_ERR_TIMEOUT in dev_status, CTA-wide abort flag: an
// aborted CTA stores no output); the CTA always frees its TMEM and exits.
#include "ec_common.cuh"
#include "ec_tc_ptx.cuh"

#include <cstdio>
#include <mutex>
#include <vector>

namespace ec {
namespace {

using namespace tc;

constexpr int BK = 128, HD = 128;
// auxiliary warps (cache update and row sums): two, or four for the 96-slot instantiation, whose row sums over twice
// the columns otherwise trail the softmax and hold up the merge
__host__ __device__ constexpr int aux_threads(int n) { return n > 64 ? 128 : 64; }
constexpr uint32_t SUB = 128 * 128;        // [128 rows x 64 bf16], 128-byte swizzle: 16 KB
constexpr uint32_t TILE = 2 * SUB;         // [128 x 128] bf16
constexpr uint32_t STAGE = 2 * TILE;       // K tile + V tile: 64 KB
constexpr int kMaxStages = 6;              // ring slots of one tile (32 KB) each
constexpr int kMaxSlots = 96;              // query slots (packed rows) of one CTA column
constexpr int kMaxActive = 256;            // active rows of a sequence (refresh list, row chunks)
constexpr int kMaxTiles = 1024;            // key tiles of one CTA (bits of the patch mask)

enum { B_FULL = 0, B_EMPTY = kMaxStages, B_SFULL = 2 * kMaxStages, B_PFULL = B_SFULL + 2, B_PVDONE = B_PFULL + 1,
       B_PSUM = B_PVDONE + 1, B_QFULL = B_PSUM + 1, B_LIST = B_QFULL + 1, B_RECV = B_LIST + 1,
       B_COUNT = B_RECV + 1 };

constexpr uint32_t kBarBytes = (B_COUNT * 8u + 15u) & ~15u;   // the barrier block, padded so that what follows is 16-byte aligned

// order-preserving map float -> int (for integer warp reductions of a maximum) and back
__device__ __forceinline__ int f2ord(float f) {
    const int i = __float_as_int(f);
    return i >= 0 ? i : (i ^ 0x7fffffff);
}
__device__ __forceinline__ float ord2f(int i) { return __int_as_float(i >= 0 ? i : (i ^ 0x7fffffff)); }

// COLS consecutive 32-bit columns of this thread's TMEM lane -> registers (and back).  ALIGNED32: the first column is
// a multiple of 32 (one 32-column access, then the rest); otherwise 16-column accesses at multiples of 16.
template <int COLS, bool ALIGNED32>
__device__ __forceinline__ void ld_row(uint32_t taddr, uint32_t* r) {
    static_assert(COLS == 48 || COLS == 64, "columns per thread");
    if (ALIGNED32) {
        ld32(taddr, r);
        if (COLS == 48) ld16(taddr + 32, r + 32); else ld32(taddr + 32, r + 32);
    } else {
#pragma unroll
        for (int c = 0; c < COLS; c += 16) ld16(taddr + c, r + c);
    }
    wait_ld();
}
template <int COLS, bool ALIGNED32>
__device__ __forceinline__ void st_row(uint32_t taddr, const uint32_t* r) {
    if (ALIGNED32) {
        st32(taddr, r);
        if (COLS == 48) st16(taddr + 32, r + 32); else st32(taddr + 32, r + 32);
    } else {
#pragma unroll
        for (int c = 0; c < COLS; c += 16) st16(taddr + c, r + c);
    }
    wait_st();
}

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
    int shift;        // 1: the first CTA of the cluster takes one cache tile more and the last, which also visits the
                      // fresh tiles, one less (ranges of the CTAs in between move up by one tile)
    int n_extra;      // key tiles of fresh rows attended by the last CTA of every cluster (0: nothing to refresh)
    int dl;           // output columns merged by one CTA of the cluster (even; the last CTA may own fewer)
    int q_tma;        // 1: the producer fetches Q with one TMA box (one query head per column); 0: softmax warps stage it
    uint32_t off_p, off_stage, off_list, off_bar;   // shared-memory carve (bytes from the 1024-aligned base); Q is at 0;
                                                    // off_list: the stale-key bits, 16 bytes per refreshed cache tile
    float scale_log2;
    // Nanoseconds the memory system needs for one stage of every CTA that streams its own K/V: the producer spaces
    // the first fill of its ring by this much per stage, so that the stages of the launch arrive one wave after the
    // other instead of all together (0: no spacing).
    uint32_t stagger_ns;
    // 1: the caller stated (EC_ATTN_CACHE_SETTLED) that nothing still running on the stream writes the caches, so the
    // first cache tile is asked for before the dependency wait
    int early_cache;
};

// words after the barrier block
struct alignas(16) KeysShared {
    uint32_t tmem;
    int abort_flag;
    int pad[2];
    int slow_flag[2][2];                       // [tile parity][warpgroup]: the softmax of that tile raised its references
    uint32_t patch_mask[kMaxTiles / 32];       // bit t: cache tile t of this CTA holds a refreshed (stale) position
    uint16_t slot_base[kMaxTiles / 32];        // refreshed tiles before word w of the mask: tile -> row of the stale-key bits
    alignas(16) float m[kMaxSlots];            // reference maxima of the query rows, log2 units (read as float2)
    alignas(16) float factor[2][kMaxSlots];    // [tile parity]: rescale factors of that tile's slow path
    alignas(16) float lpart[2][kMaxSlots];     // row sums of the CTA's keys, one partial per group of row-sum threads
    int colmax[4][kMaxSlots];                  // per-warp column maxima (ordered ints) of the current slow path
};

template <int N>
__global__ void __launch_bounds__(64 + (N > 64 ? 256 : 128) + aux_threads(N), N <= 64 ? 2 : 1)
attend_skip_keys_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                        const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kn,
                        const __grid_constant__ CUtensorMap map_vn, const KeysParams p) {
    static_assert(N == 48 || N == 64 || N == 96, "query-row slots per CTA");
    constexpr int WG = N > 64 ? 2 : 1;          // softmax warpgroups: each takes NH of a key's N scores
    constexpr int NH = N / WG;
    constexpr int kSoft = 128 * WG;
    constexpr int kAuxThreads = aux_threads(N);
    constexpr int kThreads = 64 + kSoft + kAuxThreads;
    // tensor-memory columns: S^T x 2 and O^T at multiples of NP (the slots rounded up to 64 or 128)
    constexpr uint32_t NP = N <= 64 ? 64 : 128;
    constexpr uint32_t TM_S = 0, TM_O = 2 * NP;
    constexpr uint32_t TM_COLS = (3 * NP <= 256) ? 256 : 512;
    // row-sum threads: a column pair and a share of the tile's keys each
    constexpr int kPairs = N / 2, kParts = (kAuxThreads / kPairs) >= 2 ? 2 : 1;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (s2u(smem_raw) + 1023u) & ~1023u;
    unsigned char* gbase = smem_raw + (base - s2u(smem_raw));
    const uint32_t bars = base + p.off_bar;
    KeysShared* sh = reinterpret_cast<KeysShared*>(gbase + p.off_bar + kBarBytes);
    volatile int* abort_flag = &sh->abort_flag;
    uint32_t* stale = reinterpret_cast<uint32_t*>(gbase + p.off_list);   // [refreshed cache tile][4]: a bit per stale key
    auto bar = [&](int idx) { return bars + idx * 8; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int split = blockIdx.x, bh = blockIdx.y / p.n_sub, sub = blockIdx.y % p.n_sub;
    const int b = bh / p.n_kv_heads, hk = bh % p.n_kv_heads;
    const int hq0 = (hk * (p.n_sub / p.n_sub_r) + sub / p.n_sub_r) * p.group;   // first query head of this CTA
    const int i0 = (sub % p.n_sub_r) * p.rows_chunk;                           // first active row of this CTA
    const int rows_total = min(p.rows_chunk, p.n_active - i0) * p.group;       // packed query rows of this CTA
    const int C = p.n_splits;
    const int DL = p.dl;
    const int n_tiles_total = (p.ctx_len + BK - 1) / BK;
    const int t_begin = split * p.tiles_per_split + (split > 0 ? p.shift : 0);
    const int t_end = min(n_tiles_total, (split + 1) * p.tiles_per_split + p.shift);
    const int TC = max(0, t_end - t_begin);                  // cache tiles of this CTA
    const int NS = p.n_stages;       // ring slots: tile j has K in slot 2j mod NS and V in slot (2j + 1) mod NS
    const bool refresh = p.k_new != nullptr;
    // the last CTA of the cluster attends to the fresh rows too, after its cache tiles, as XT extra key tiles read from
    // k_new / v_new: visits [0, TC) are cache tiles, visits [TC, T) fresh tiles
    const int XT = (refresh && split == p.n_splits - 1) ? p.n_extra : 0;
    const int T = XT + TC;           // tiles this CTA visits: >= 1 by construction of the plan
    const int key_lo = t_begin * BK, key_hi = min(p.ctx_len, t_end * BK);
    // exchange areas of the merge, from the start of the (then dead) Q / P^T / stage memory: C staging chunks (one per
    // owner), C receive chunks (one per source).  A chunk holds
    // [N queries][DL columns] floats of O^T, then m[N], then l[N].
    const uint32_t chunk_floats = (uint32_t)(N * DL + 2 * N);
    const uint32_t chunk_bytes = chunk_floats * 4u;
    const uint32_t stg_off = 0, recv_off = (uint32_t)C * chunk_bytes;

    // ---- set-up ------------------------------------------------------------------------------
    // Under programmatic dependent launch this CTA starts while the tail of the previous kernel still runs.  Whatever
    // that kernel produces (q, k_new, v_new, the index list) is read after the dependency wait below.  The caches are
    // read before it only when the caller has stated that nothing in flight writes them: the producer thread then asks
    // for its first cache tile as soon as the barriers exist, and the memory system works through the rest of the
    // set-up, the previous kernel's tail and the wait.
    unsigned long long t_fill = 0;
    if (tid == 0) {
        for (int i = 0; i < B_COUNT; ++i) {
            uint32_t count = 1;
            if (i == B_PFULL || (i == B_QFULL && !p.q_tma)) count = kSoft;
            if (i == B_PSUM) count = kAuxThreads;
            mbar_init(bar(i), count);
        }
        sh->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (p.early_cache && TC > 0) {   // ring entry 0: the first cache tile
            t_fill = global_timer_ns();
            const uint32_t dst = base + p.off_stage;
            mbar_expect_tx(bar(B_FULL + 0), TILE);
            tma_load_4d(dst, &map_k, 0, t_begin * BK, 0, bh, bar(B_FULL + 0));
            mbar_expect_tx(bar(B_FULL + 1), TILE);
            tma_load_4d(dst + TILE, &map_v, 0, t_begin * BK, 0, bh, bar(B_FULL + 1));
        } else {
            prefetch_map(&map_k);
            prefetch_map(&map_v);
        }
        if (p.q_tma) prefetch_map(&map_q);
        if (p.k_new) {
            prefetch_map(&map_kn);
            prefetch_map(&map_vn);
        }
        if (C > 1) mbar_expect_tx(bar(B_RECV), (uint32_t)C * chunk_bytes);   // the peers' partials, one chunk each
    }
    if (tid < kMaxTiles / 32) sh->patch_mask[tid] = 0u;
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

    if (warp == 0) {
        // ================================ TMA producer ======================================
        if (lane == 0) {
            if (p.q_tma) {   // Q first: [half][row][64 columns] of this head's rows, rows past n_active read as zero
                mbar_expect_tx(bar(B_QFULL), (uint32_t)N * 256u);
                tma_load_5d(base, &map_q, 0, i0, hq0, 0, b, bar(B_QFULL));   // rows past the chunk land in unused slots
            }
            const bool first_asked = t_fill != 0;   // ring entry 0 (the first cache tile) is already on its way
            if (!first_asked) t_fill = global_timer_ns();
            for (int n = 0; n < 2 * T; ++n) {   // ring entry n: K of tile n / 2 (even n) or its V (odd n)
                const int j = n >> 1, s = n % NS, u = n / NS;
                if (first_asked && j == 0) continue;
                if (u == 0 && !(n & 1) && j > 0 && j < TC && p.stagger_ns) {
                    // First fill of the ring: cache tile j of every CTA is asked for j * stagger_ns after the first, so
                    // the first tiles of all CTAs land before anybody's second, and requests stay queued while they
                    // are consumed.  (Asked for all at once, the tiles of the whole launch arrive together after
                    // the time of all of them, and the memory system then idles until the first slot is free again.)
                    const unsigned long long due = t_fill + (unsigned long long)j * p.stagger_ns;
                    while (global_timer_ns() < due) __nanosleep(64);
                }
                if (u > 0) mbar_wait(bar(B_EMPTY + s), (u - 1) & 1, abort_flag, p.dev_status);
                const uint32_t dst = base + p.off_stage + s * TILE;
                mbar_expect_tx(bar(B_FULL + s), TILE);
                if (j >= TC) {   // active rows [128 x, 128 x + 128) of this kv head, fresh; rows past n_active read as zero
                    tma_load_5d(dst, (n & 1) ? &map_vn : &map_kn, 0, (j - TC) * BK, 0, hk, b, bar(B_FULL + s));
                } else {
                    tma_load_4d(dst, (n & 1) ? &map_v : &map_k, 0, (t_begin + j) * BK, 0, bh, bar(B_FULL + s));
                }
            }
        }
    } else if (warp == 1) {
        // ================= stale-key masks, then MMA issue (lane 0) =================================
        if (refresh) {
            // which cached keys of this CTA's range are about to be refreshed: they are attended from k_new / v_new (as
            // extra tiles, by the last CTA of the cluster), so their cached copies must not count
            int posv[kMaxActive / 32];
#pragma unroll
            for (int k = 0; k < kMaxActive / 32; ++k) {
                const int i = k * 32 + lane;
                posv[k] = -1;
                if (k * 32 >= p.n_active) continue;   // uniform: nothing of the list left
                if (i < p.n_active) posv[k] = p.active_idx ? __ldg(p.active_idx + (long long)b * p.n_active + i) : i;
            }
#pragma unroll
            for (int k = 0; k < kMaxActive / 32; ++k) {
                if (k * 32 >= p.n_active) break;
                if (posv[k] >= key_lo && posv[k] < key_hi) {
                    const int tile = (posv[k] - key_lo) / BK;
                    atomicOr(&sh->patch_mask[tile >> 5], 1u << (tile & 31));
                }
            }
            __syncwarp();
            {   // rows of the bit table: refreshed tiles in tile order (exclusive prefix count over the mask words)
                const int cnt = __popc(sh->patch_mask[lane]);
                int incl = cnt;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int v = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += v;
                }
                sh->slot_base[lane] = (uint16_t)(incl - cnt);
                const int total = __shfl_sync(0xffffffffu, incl, 31);
                for (int w = lane; w < total * 4; w += 32) stale[w] = 0u;
            }
            __syncwarp();
#pragma unroll
            for (int k = 0; k < kMaxActive / 32; ++k) {
                if (k * 32 >= p.n_active) break;
                if (posv[k] >= key_lo && posv[k] < key_hi) {
                    const int r = posv[k] - key_lo, tile = r / BK, kk = r % BK;
                    const int slot = sh->slot_base[tile >> 5] + __popc(sh->patch_mask[tile >> 5] & ((1u << (tile & 31)) - 1u));
                    atomicOr(&stale[slot * 4 + (kk >> 5)], 1u << (kk & 31));
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(B_LIST));   // release: the masks above are visible to whoever waits
            __syncwarp();
        }
        if (lane == 0) {
            constexpr uint32_t IDESC_S = instr_desc2(N, 0, 0);    // A = K tile (K-major), B = Q (K-major)
            constexpr uint32_t IDESC_PV = instr_desc2(N, 1, 1);   // A = V tile (MN-major: d contiguous), B = P^T (MN-major)
            constexpr uint32_t QHALF = N * 128;                   // bytes of one 64-column half of the Q tile
            auto issue_s = [&](int j) {
                const int s = (2 * j) % NS;
                fence_after();
                const uint32_t kst = base + p.off_stage + s * TILE;
#pragma unroll
                for (int k = 0; k < HD / 16; ++k) {
                    const uint32_t koff = (k & 3) * 32;
                    mma_ss(tmem + TM_S + (j & 1) * NP, smem_desc(kst + (k >> 2) * SUB + koff, 16, 1024),
                           smem_desc(base + (k >> 2) * QHALF + koff, 16, 1024), IDESC_S, k > 0);
                }
                commit(bar(B_SFULL + (j & 1)));
                commit(bar(B_EMPTY + s));   // the K slot is free once these products have run
            };
            // S of tile j needs the tile (and its patch); P V of tile j needs P^T from the softmax.  Whichever is ready
            // is issued: P V of a tile does not wait for the next tile to land (its commit frees the stage for the
            // producer), S may run one tile ahead of P V (two S^T buffers).
            mbar_wait(bar(B_QFULL), 0, abort_flag, p.dev_status);
            int next_s = 0, next_pv = 0;
            SpinGuard guard;
            while (next_pv < T) {
                bool progressed = false;
                if (next_s < T && next_s <= next_pv + 1 && mbar_try(bar(B_FULL + (2 * next_s) % NS), ((2 * next_s) / NS) & 1)) {
                    issue_s(next_s);   // (the tile has landed)
                    ++next_s;
                    progressed = true;
                }
                if (mbar_try(bar(B_PFULL), next_pv & 1) &&
                    mbar_try(bar(B_FULL + (2 * next_pv + 1) % NS), ((2 * next_pv + 1) / NS) & 1)) {   // P^T is there, V has landed
                    const int j = next_pv;
                    const uint32_t vst = base + p.off_stage + ((2 * j + 1) % NS) * TILE;
                    fence_after();
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        mma_ss(tmem + TM_O, smem_desc(vst + k * 2048, SUB, 1024), smem_desc(base + p.off_p + k * 2048, SUB, 1024),
                               IDESC_PV, (j > 0 || k > 0));
                    commit(bar(B_PVDONE));
                    commit(bar(B_EMPTY + (2 * j + 1) % NS));
                    ++next_pv;
                    progressed = true;
                }
                if (progressed) guard.progress();
                else if (!guard.tick(abort_flag, p.dev_status)) break;
            }
        }
    } else if (warp >= 2 + 4 * WG) {
        // ===== auxiliary warps: the fresh rows into the cache (for later steps); row sums of P^T =====
        const int atid = tid - (64 + kSoft);
        // row sums: this thread adds up column pair cp of the keys [k_lo, k_lo + BK / kParts) of every tile
        const bool summer = atid < kPairs * kParts;
        const int cp = atid % kPairs, col = 2 * cp, gch = col >> 3;
        const int k_lo = (atid / kPairs) * (BK / kParts);
        const unsigned char* pcol = gbase + p.off_p + (gch >> 3) * SUB + (col & 7) * 2;
        float acc0 = 0.f, acc1 = 0.f;

        for (int j = 0; j < T; ++j) {
            if (j >= TC && sub == 0) {
                // One CTA per (sequence, kv head) -- the one that attends to the fresh tiles -- also puts the active
                // rows' K/V into the cache, for later steps: the fresh tile is in shared memory once its stage is full,
                // so the rows leave from there as plain 16-byte stores (thread = one 16-byte piece of a row, four rows
                // per pass; the tile is 128-byte swizzled).  Nothing in this launch depends on these stores.  The stage
                // is overwritten (by the merge's exchange areas) only after the row sums of the last visit, which this
                // thread reports after it has read its pieces.  (One TMA store per row and half took 3.5 us for 34
                // rows: 136 requests of 128 bytes, served one after the other.)
                const int x = j - TC;
                mbar_wait(bar(B_FULL + (2 * j) % NS), ((2 * j) / NS) & 1, abort_flag, p.dev_status);           // the fresh K tile
                mbar_wait(bar(B_FULL + (2 * j + 1) % NS), ((2 * j + 1) / NS) & 1, abort_flag, p.dev_status);   // and V tile
                const unsigned char* ktile = gbase + p.off_stage + ((2 * j) % NS) * TILE;
                const unsigned char* vtile = gbase + p.off_stage + ((2 * j + 1) % NS) * TILE;
                const int ch = atid & 15;   // piece of the row: columns [8 ch, 8 ch + 8)
                const int n_rows = min(BK, p.n_active - x * BK);
                for (int r = atid >> 4; r < n_rows; r += kAuxThreads / 16) {
                    const int i = x * BK + r;
                    const int pos = p.active_idx ? __ldg(p.active_idx + (long long)b * p.n_active + i) : i;
                    if (pos < 0 || pos >= p.ctx_len) continue;
                    const uint32_t off = (ch >> 3) * SUB + (r >> 3) * 1024 + (r & 7) * 128 + (((ch & 7) ^ (r & 7)) << 4);
                    const long long dst = (((long long)bh * p.ctx_len + pos) * HD + ch * 8);
                    *reinterpret_cast<uint4*>(p.k_cache + dst) = *reinterpret_cast<const uint4*>(ktile + off);
                    *reinterpret_cast<uint4*>(p.v_cache + dst) = *reinterpret_cast<const uint4*>(vtile + off);
                }
            }
            // P^T of tile j is in shared memory
            mbar_wait(bar(B_PFULL), j & 1, abort_flag, p.dev_status);
            if (summer) {
                if (sh->slow_flag[j & 1][col / NH]) {   // the references of these columns were raised at this tile
                    acc0 *= sh->factor[j & 1][col];
                    acc1 *= sh->factor[j & 1][col + 1];
                }
#pragma unroll 4
                for (int k8 = 0; k8 < BK / kParts; k8 += 8) {
#pragma unroll
                    for (int r = 0; r < 8; ++r) {
                        const int k = k_lo + k8 + r;
                        const uint32_t w = *reinterpret_cast<const uint32_t*>(pcol + (k >> 3) * 1024 + r * 128 + (((gch & 7) ^ r) << 4));
                        acc0 += __uint_as_float(w << 16);
                        acc1 += __uint_as_float(w & 0xffff0000u);
                    }
                }
                if (j == T - 1) {
                    sh->lpart[atid / kPairs][col] = acc0;
                    sh->lpart[atid / kPairs][col + 1] = acc1;
                }
            }
            mbar_arrive(bar(B_PSUM));   // P^T of tile j has been read (release: the row sums above are visible)
        }
    } else {
        // ================== Q staging (grouped heads), softmax (warps 2 ..) ========================
        const int stid = tid - 64;
        const int wg = stid >> 7;                    // warpgroup: columns [wg * NH, (wg + 1) * NH) of every key
        const int c0 = wg * NH;
        const int st_w = stid & 127;
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

        const int quarter = warp & 3;
        const int kk = quarter * 32 + lane;          // key of the tile == TMEM lane == output column d later on
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const float sl2 = p.scale_log2;
        const f32x2 sl2_2 = pk(sl2, sl2);
        // P^T row of this key: [64-slot half][key][64 slots], 128-byte swizzle
        unsigned char* prow = gbase + p.off_p + (kk >> 3) * 1024 + (kk & 7) * 128;
        const int bar_or = 2 + 2 * wg, bar_sync = 3 + 2 * wg;   // named barriers of this warpgroup
        // which keys of the fresh tiles exist: active rows with a position inside the context (bit x: row 128 x + kk)
        uint32_t fresh_ok = 0;
        for (int x = 0; x < XT; ++x) {
            const int i = x * BK + kk;
            if (i < p.n_active) {
                const int pos = p.active_idx ? __ldg(p.active_idx + (long long)b * p.n_active + i) : i;
                if (pos >= 0 && pos < p.ctx_len) fresh_ok |= 1u << x;
            }
        }
        bool masks_ready = !refresh;   // the stale-key bits are awaited once, before the first cache tile

        for (int j = 0; j < T; ++j) {
            mbar_wait(bar(B_SFULL + (j & 1)), (j >> 1) & 1, abort_flag, p.dev_status);
            fence_after();
            const uint32_t s_addr = tmem + lane_addr + TM_S + (j & 1) * NP + c0;
            // this thread's key does not count: a missing row of a fresh tile, a key past the end of the context (ragged
            // last tile), a cached key whose position is being refreshed (it is attended from the fresh tile instead)
            bool past_end;
            if (j >= TC) {
                past_end = !((fresh_ok >> (j - TC)) & 1u);
            } else {
                const int t = j;
                past_end = (t_begin + t) * BK + kk >= p.ctx_len;
                if (!masks_ready) {
                    mbar_wait(bar(B_LIST), 0, abort_flag, p.dev_status);
                    masks_ready = true;
                }
                if (refresh && ((sh->patch_mask[t >> 5] >> (t & 31)) & 1u)) {
                    const int slot = sh->slot_base[t >> 5] + __popc(sh->patch_mask[t >> 5] & ((1u << (t & 31)) - 1u));
                    past_end = past_end || ((stale[slot * 4 + (kk >> 5)] >> (kk & 31)) & 1u);
                }
            }
            // d = s * scale * log2(e) - m[q]; does any score exceed its reference by more than 2^8?
            f32x2 d2[NH / 2];
            auto load_d = [&]() {
                uint32_t sr[NH];
                ld_row<NH, WG == 1>(s_addr, sr);
#pragma unroll
                for (int i = 0; i < NH / 2; ++i) {
                    const float2 mm = *reinterpret_cast<const float2*>(&sh->m[c0 + 2 * i]);
                    d2[i] = fma2(pk(__uint_as_float(sr[2 * i]), __uint_as_float(sr[2 * i + 1])), sl2_2, pk(-mm.x, -mm.y));
                    if (past_end) d2[i] = pk(-INFINITY, -INFINITY);   // probability 0 for every query
                }
            };
            load_d();
            float dmx0 = -INFINITY, dmx1 = -INFINITY;
#pragma unroll
            for (int i = 0; i < NH / 2; ++i) {
                float d0, d1;
                upk(d2[i], d0, d1);
                if (i & 1) dmx1 = max3(dmx1, d0, d1); else dmx0 = max3(dmx0, d0, d1);
            }
            const bool slow = named_barrier_or(bar_or, 128, fmaxf(dmx0, dmx1) > 8.f);
            if (st_w == 0) sh->slow_flag[j & 1][wg] = slow ? 1 : 0;   // for the row-sum threads (read after "P full")
            if (slow) {
                // ---- rare path: raise the references to the column maxima of this tile, rescale O^T (the row-sum
                //      threads rescale their sums by the same factors) ----
                {
                    uint32_t sr[NH];   // the raw scores once more (they stay in tensor memory until S of tile j + 2)
                    ld_row<NH, WG == 1>(s_addr, sr);
#pragma unroll
                    for (int c = 0; c < NH; ++c) {
                        const int o = __reduce_max_sync(0xffffffffu, f2ord(past_end ? -INFINITY : __uint_as_float(sr[c])));
                        if (lane == (c & 31)) sh->colmax[quarter][c0 + c] = o;
                    }
                }
                named_barrier(bar_sync, 128);
                if (st_w < NH) {
                    const int c = c0 + st_w;
                    const int o = max(max(sh->colmax[0][c], sh->colmax[1][c]), max(sh->colmax[2][c], sh->colmax[3][c]));
                    const float m_old = sh->m[c];
                    const float m_new = fmaxf(m_old, ord2f(o) * sl2);
                    sh->factor[j & 1][c] = (m_old == -INFINITY) ? 0.f : fast_exp2(m_old - m_new);
                    sh->m[c] = m_new;
                }
                named_barrier(bar_sync, 128);
                if (j > 0) {   // O^T holds the tiles before j: P V of tile j - 1 must have completed
                    mbar_wait(bar(B_PVDONE), (j - 1) & 1, abort_flag, p.dev_status);
                    fence_after();
                    uint32_t o[NH];
                    const uint32_t o_addr = tmem + lane_addr + TM_O + c0;
                    ld_row<NH, WG == 1>(o_addr, o);
#pragma unroll
                    for (int c = 0; c < NH; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * sh->factor[j & 1][c0 + c]);
                    st_row<NH, WG == 1>(o_addr, o);
                }
                load_d();   // against the raised references
            }
            uint32_t pw[NH / 2];
#pragma unroll
            for (int i = 0; i < NH / 2; ++i) {
                float d0, d1;
                upk(d2[i], d0, d1);
                pw[i] = pack_bf16x2(fast_exp2(d0), fast_exp2(d1));
            }
            // the P^T buffer is free once P V of the previous tile has completed and its row sums have been taken
            if (j > 0) {
                mbar_wait(bar(B_PVDONE), (j - 1) & 1, abort_flag, p.dev_status);
                mbar_wait(bar(B_PSUM), (j - 1) & 1, abort_flag, p.dev_status);
            }
#pragma unroll
            for (int ch = 0; ch < NH / 8; ++ch) {
                const int gch = (c0 >> 3) + ch;      // 16-byte chunk (8 slots) of the whole P^T row
                *reinterpret_cast<uint4*>(prow + (gch >> 3) * SUB + (((gch & 7) ^ (kk & 7)) << 4)) =
                    make_uint4(pw[4 * ch], pw[4 * ch + 1], pw[4 * ch + 2], pw[4 * ch + 3]);
            }
            fence_async_smem();
            fence_before();
            mbar_arrive(bar(B_PFULL));
        }
        mbar_wait(bar(B_PVDONE), (T - 1) & 1, abort_flag, p.dev_status);   // Q, P^T and the K/V stages are dead from here on
        fence_after();
        if (C > 1) {
            // first cluster barrier, arrive half: the peers may write their partials into this CTA's receive chunks
            // (nothing is published by it, so no memory ordering is attached)
            __syncwarp();
            cluster_arrive_relaxed();
        }
        mbar_wait(bar(B_PSUM), (T - 1) & 1, abort_flag, p.dev_status);     // the row sums are complete

        uint32_t o[NH];
        ld_row<NH, WG == 1>(tmem + lane_addr + TM_O + c0, o);
        if (C == 1) {
            // ---- single CTA per (sequence, kv head): normalise and store column kk of every query row ----
            if (!*abort_flag) {
#pragma unroll
                for (int c = 0; c < NH; ++c) {
                    if (c0 + c < rows_total) {
                        const float l = sh->lpart[0][c0 + c] + (kParts == 2 ? sh->lpart[1][c0 + c] : 0.f);
                        const int i = i0 + (c0 + c) / p.group, jh = (c0 + c) % p.group;
                        __nv_bfloat16* dst = p.out + (((long long)b * p.n_active + i) * p.n_q_heads + hq0 + jh) * HD;
                        dst[kk] = __float2bfloat16_rn(__uint_as_float(o[c]) / l);
                    }
                }
            }
        } else {
            // ---- this thread's O^T row (output column kk, its warpgroup's queries) -> the staging chunk of the
            //      CTA that owns column kk; consecutive lanes write consecutive words ----
            float* stg = reinterpret_cast<float*>(gbase + stg_off) + (kk / DL) * chunk_floats + (kk % DL);
#pragma unroll
            for (int c = 0; c < NH; ++c)
                if (c0 + c < rows_total) stg[(c0 + c) * DL] = __uint_as_float(o[c]);
            if (st_w < NH) {   // every owner also gets this CTA's m[q] and l[q]
                const int c = c0 + st_w;
                const float l = sh->lpart[0][c] + (kParts == 2 ? sh->lpart[1][c] : 0.f);
                for (int ow = 0; ow < C; ++ow) {
                    float* ml = reinterpret_cast<float*>(gbase + stg_off) + ow * chunk_floats + N * DL;
                    ml[c] = sh->m[c];
                    ml[N + c] = l;
                }
            }
            fence_async_smem();   // staging (generic proxy) -> bulk copies (async proxy)
            named_barrier(6, kSoft);
            __syncwarp();
            cluster_wait();       // every CTA of the cluster is past its main loop
            if (stid < C) {       // one bulk copy per owner into the owner's receive chunk of this source
                const uint32_t src = base + stg_off + (uint32_t)stid * chunk_bytes;
                const uint32_t dst = map_to_cta(base + recv_off + (uint32_t)split * chunk_bytes, stid);
                bulk_copy_to_peer(dst, src, chunk_bytes, map_to_cta(bar(B_RECV), stid));
            }
        }
    }

    if (C > 1) {
        if (!(warp >= 2 && warp < 2 + 4 * WG)) {   // the other warps' halves of the first cluster barrier
            __syncwarp();
            cluster_arrive_relaxed();
            cluster_wait();
        }
        // ---- merge the C partials of the output columns this CTA owns -------------------------
        mbar_wait(bar(B_RECV), 0, abort_flag, p.dev_status);
        // second cluster barrier, arrive half: this CTA holds every peer's partial, so the peers' copies out of their
        // staging chunks have completed; the wait half, before leaving, overlaps the merge
        __syncwarp();
        cluster_arrive_relaxed();
        const float* recv = reinterpret_cast<const float*>(gbase + recv_off);
        // a thread owns two adjacent output columns of a query row (one 4-byte store) and works out the row's weights
        // 2^(m_s - m) / l itself: the sixteen or so threads of a row repeat that, but nobody waits for a table
        const int own_dl = min(DL, HD - split * DL);   // output columns this CTA owns (even)
        if (!*abort_flag && (DL & 3) == 0 && (own_dl & 3) == 0) {
            // four adjacent output columns of a query row per item (one 8-byte store)
            const int quads = own_dl / 4;
            for (int idx = tid; idx < rows_total * quads; idx += kThreads) {
                const int qq = idx / quads, dq = idx % quads;
                float m = -INFINITY;
#pragma unroll
                for (int s = 0; s < 8; ++s)
                    if (s < C) m = fmaxf(m, recv[s * chunk_floats + N * DL + qq]);
                float l = 0.f;
                float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int s = 0; s < 8; ++s) {
                    if (s < C) {
                        const float* ch = recv + s * chunk_floats;
                        const float e = fast_exp2(ch[N * DL + qq] - m);
                        const float4 v = *reinterpret_cast<const float4*>(ch + qq * DL + 4 * dq);
                        l = fmaf(e, ch[N * DL + N + qq], l);
                        a.x = fmaf(e, v.x, a.x);
                        a.y = fmaf(e, v.y, a.y);
                        a.z = fmaf(e, v.z, a.z);
                        a.w = fmaf(e, v.w, a.w);
                    }
                }
                const float inv = 1.f / l;
                const int i = i0 + qq / p.group, jh = qq % p.group;
                __nv_bfloat16* dst = p.out + (((long long)b * p.n_active + i) * p.n_q_heads + hq0 + jh) * HD + split * DL + 4 * dq;
                *reinterpret_cast<uint2*>(dst) = make_uint2(pack_bf16x2(a.x * inv, a.y * inv), pack_bf16x2(a.z * inv, a.w * inv));
            }
        } else if (!*abort_flag) {
            const int half_dl = own_dl / 2;
            for (int idx = tid; idx < rows_total * half_dl; idx += kThreads) {
                const int qq = idx / half_dl, dp = idx % half_dl;
                float ms[8], ls[8];
                float2 v[8];
#pragma unroll
                for (int s = 0; s < 8; ++s) {
                    if (s < C) {
                        const float* ch = recv + s * chunk_floats;
                        ms[s] = ch[N * DL + qq];
                        ls[s] = ch[N * DL + N + qq];
                        v[s] = *reinterpret_cast<const float2*>(ch + qq * DL + 2 * dp);
                    } else {
                        ms[s] = -INFINITY;
                        ls[s] = 0.f;
                        v[s] = make_float2(0.f, 0.f);
                    }
                }
                const float m = fmaxf(fmaxf(fmaxf(ms[0], ms[1]), fmaxf(ms[2], ms[3])), fmaxf(fmaxf(ms[4], ms[5]), fmaxf(ms[6], ms[7])));
                float l = 0.f, a0 = 0.f, a1 = 0.f;
#pragma unroll
                for (int s = 0; s < 8; ++s) {
                    const float e = fast_exp2(ms[s] - m);   // 0 for the sources that do not exist
                    l = fmaf(e, ls[s], l);
                    a0 = fmaf(e, v[s].x, a0);
                    a1 = fmaf(e, v[s].y, a1);
                }
                const float inv = 1.f / l;
                const int i = i0 + qq / p.group, jh = qq % p.group;
                __nv_bfloat16* dst = p.out + (((long long)b * p.n_active + i) * p.n_q_heads + hq0 + jh) * HD + split * DL + 2 * dp;
                *reinterpret_cast<uint32_t*>(dst) = pack_bf16x2(a0 * inv, a1 * inv);
            }
        }
        // no CTA leaves while a peer may still copy out of its staging chunks
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

// q [B, n, H_q, 128] bf16 (one query head per CTA column) seen as 5-D {64 columns, row, head, half, sequence}:
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
    bool ok;
    int group, rows_chunk, n_sub_r, n_sub;   // heads and active rows per CTA column, row chunks, CTA columns per kv head
    int n_slots, n_splits, tiles_per_split, n_stages, n_extra, dl, ctas_per_sm, shift;
    uint32_t off_p, off_stage, off_list, off_bar, smem_bytes;
};

constexpr uint32_t kSmemMax = 232448;        // 227 KB: largest dynamic allocation of one CTA
constexpr uint32_t kSmemTwoPerSm = 115712;   // (228 KB per SM - 2 x 1 KB reserved) / 2

// tensor-memory columns the instantiation for n_slots allocates (see TM_COLS in the kernel)
constexpr int tm_columns(int n_slots) { return 3 * (n_slots <= 64 ? 64 : 128) <= 256 ? 256 : 512; }

// shared-memory carve for n_slots query slots and ns stages; `fresh`: room for the stale-key bits (16 bytes per
// refreshed cache tile, of which there are at most n_active)
void carve(KeysPlan& pl, int n_active, int ns, bool fresh) {
    uint32_t off = (uint32_t)pl.n_slots * 256u;   // Q
    off = (off + 1023u) & ~1023u;
    pl.off_p = off;
    off += (uint32_t)((pl.n_slots + 63) / 64) * SUB;
    pl.off_stage = off;
    off += (uint32_t)ns * TILE;
    pl.off_list = off;
    off += fresh ? (uint32_t)n_active * 16u : 0u;
    pl.off_bar = off;
    off += kBarBytes + (uint32_t)sizeof(KeysShared) + 16u;
    pl.smem_bytes = off + 1024u;
    // an instantiation that allocates all 512 columns of tensor memory must never share an SM with a CTA of its own
    // cluster (the second allocation would wait for the first CTA, which waits for it at the cluster barrier): ask for
    // more than half an SM's shared memory
    if (tm_columns(pl.n_slots) > 256 && pl.smem_bytes <= kSmemTwoPerSm) pl.smem_bytes = kSmemTwoPerSm + 1024u;
    pl.n_stages = ns;
}

// How many clusters of c CTAs with this much dynamic shared memory the current device keeps resident at once (clusters
// are placed inside one GPC, so this can be fewer than SMs x CTAs per SM / c); -1 when it cannot be asked (no device).
// Asked once per (device, instantiation, cluster size, shared memory) and remembered.
template <int N>
int resident_clusters_of(int c, uint32_t smem) {
    static PerDeviceOnce attr_once;
    if (ensure_dynamic_smem(attr_once, attend_skip_keys_kernel<N>, (int)kSmemMax) != cudaSuccess) {
        (void)cudaGetLastError();
        return -1;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(c, 1, 1);
    cfg.blockDim = dim3(64 + (N > 64 ? 256 : 128) + aux_threads(N), 1, 1);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = c;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, attend_skip_keys_kernel<N>, &cfg) != cudaSuccess) {
        (void)cudaGetLastError();
        return -1;
    }
    return n;
}

int resident_clusters(int n_slots, int c, uint32_t smem) {
    struct Entry { int dev, n_slots, c; uint32_t smem; int clusters; };
    static std::mutex mu;
    static std::vector<Entry> seen;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return -1;
    }
    std::lock_guard<std::mutex> lock(mu);
    for (const Entry& e : seen)
        if (e.dev == dev && e.n_slots == n_slots && e.c == c && e.smem == smem) return e.clusters;
    const int n = n_slots == 48 ? resident_clusters_of<48>(c, smem) : n_slots == 64 ? resident_clusters_of<64>(c, smem)
                                                                                      : resident_clusters_of<96>(c, smem);
    seen.push_back({dev, n_slots, c, smem, n});
    return n;
}

// fresh: the call refreshes (k_new / v_new given), so the last CTA of every cluster also visits the fresh tiles
KeysPlan make_keys_plan(const ec_attn_desc& d, int n_active, bool fresh) {
    KeysPlan pl{};
    // a CTA column takes the largest divisor of the H_q / H_kv heads of a kv head whose packed rows fit the query
    // slots; the other columns of that kv head stream the same K/V (from L2) for their own heads
    const int g = d.n_q_heads / d.n_kv_heads;
    pl.group = g;
    while (pl.group > 1 && (g % pl.group != 0 || (long long)n_active * pl.group > kMaxSlots)) --pl.group;
    // more active rows than slots: the rows are cut into equal chunks, one CTA column each
    pl.n_sub_r = (n_active * pl.group + kMaxSlots - 1) / kMaxSlots;
    pl.rows_chunk = (n_active + pl.n_sub_r - 1) / pl.n_sub_r;
    pl.n_sub_r = (n_active + pl.rows_chunk - 1) / pl.rows_chunk;
    pl.n_sub = (g / pl.group) * pl.n_sub_r;
    const int rows = pl.rows_chunk * pl.group;
    pl.n_slots = rows <= 48 ? 48 : rows <= 64 ? 64 : 96;
    pl.n_extra = fresh ? (n_active + BK - 1) / BK : 0;
    const int tm_cols = tm_columns(pl.n_slots);
    const int key_tiles = (d.ctx_len + BK - 1) / BK;
    const long long columns = (long long)d.batch * d.n_kv_heads * pl.n_sub;   // grid.y
    const int sms = sm_count();
    // Cluster shape: cs CTAs split the cache tiles (every one at least one tile); the fresh tiles go to the last of
    // them, or to one more CTA of their own (worth it when a CTA holds so few tiles that one more would be felt, and
    // needed when it has a single stage).  All CTAs resident at once (two per SM when they are small); the most-loaded SM
    // streams as few tiles as possible; among equals, more CTAs (more SMs pulling).
    long long best_cost = -1, best_ctas = 0;
    for (int cs = 1; cs <= 8 && cs <= key_tiles; ++cs) {
        const int tps = (key_tiles + cs - 1) / cs;
        if ((key_tiles + tps - 1) / tps != cs || tps > kMaxTiles) continue;   // this cs leaves a CTA empty
        for (int own = 0; own <= (fresh ? 1 : 0); ++own) {                     // own: the fresh tiles get their own CTA
            const int c = cs + own;
            if (c > 8) continue;
            int dl = (HD + c - 1) / c;
            dl += dl & 1;
            if ((c - 1) * dl >= HD) continue;                                  // an owner without columns
            const int last_tiles = key_tiles - (cs - 1) * tps;
            const int visits = own ? (tps > pl.n_extra ? tps : pl.n_extra)
                                   : (tps > last_tiles + pl.n_extra ? tps : last_tiles + pl.n_extra);
            KeysPlan t = pl;
            int ns = 2 * visits < kMaxStages ? 2 * visits : kMaxStages;   // ring slots: a K and a V slot per tile in flight
            carve(t, n_active, ns, fresh);
            while (ns > 2 && t.smem_bytes > kSmemMax) carve(t, n_active, --ns, fresh);
            if (t.smem_bytes > kSmemMax || (ns < 4 && visits > 1)) continue;
            // the exchange areas of the merge (2 c chunks) reuse the Q / P^T / stage memory
            if (c > 1 && 2 * (size_t)c * (pl.n_slots * dl + 2 * pl.n_slots) * 4 > t.off_list) continue;
            const int per_sm = (t.smem_bytes <= kSmemTwoPerSm && tm_cols <= 256) ? 2 : 1;
            const long long ctas = columns * c;
            if (ctas > (long long)per_sm * sms) continue;
            const int fit = resident_clusters(pl.n_slots, c, t.smem_bytes);   // (-1: no device to ask, keep the estimate)
            if (fit >= 0 && columns > fit) continue;
            // cost in quarter tiles: the fresh tiles arrive early (they are small and mostly in L2), so on a shared CTA
            // they count a quarter of a cache tile
            const long long cost = 4LL * tps * ((ctas + sms - 1) / sms) + ((fresh && !own) ? pl.n_extra : 0);
            if (best_cost < 0 || cost < best_cost || (cost == best_cost && ctas > best_ctas)) {
                best_cost = cost;
                best_ctas = ctas;
                pl.n_splits = c;
                pl.tiles_per_split = tps;
                // The CTA that also visits the fresh tiles has one visit more than its peers, and the cluster waits for
                // it at the merge.  The memory system serves whoever asks, so giving that CTA one cache tile less (and
                // the first CTA one more) lets it finish its stream early and spend the difference on the extra visit.
                pl.shift = (fresh && !own && cs >= 2 && tps >= 2 && last_tiles == tps) ? 1 : 0;
                pl.dl = dl;
                pl.ctas_per_sm = per_sm;
                pl.n_stages = ns;
            }
        }
    }
    pl.ok = best_cost >= 0;
    if (pl.ok) carve(pl, n_active, pl.n_stages, fresh);
    return pl;
}

// k_new / v_new [B, n, H_kv, 128] bf16 seen as 5-D {64 columns, active row, half, kv head, sequence}: one box
// {64, 128, 2, 1, 1} lands as [half][row][64 columns], i.e. exactly like a cache tile whose keys are the active rows
// 128 j .. 128 j + 127 of one kv head; rows past n read as zero
bool make_fresh_map(CUtensorMap* map, const void* fresh, int batch, int n_active, int n_kv_heads) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[5] = {64, (cuuint64_t)n_active, 2, (cuuint64_t)n_kv_heads, (cuuint64_t)batch};
    const cuuint64_t strides[4] = {(cuuint64_t)n_kv_heads * HD * 2, 128, (cuuint64_t)HD * 2,
                                   (cuuint64_t)n_active * n_kv_heads * HD * 2};
    const cuuint32_t box[5] = {64, (cuuint32_t)BK, 2, 1, 1};
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(fresh), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bytes per nanosecond assumed for a streaming read when spacing the first ring fill: 0.7 of the nominal rate of the
// device (clock x bus width, double data rate; a spacing between 1.0 and 1.3 times the measured copy rate's stage
// time timed best), cached per device
double stream_bytes_per_ns() {
    static std::atomic<uint64_t> cached[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 5700.0;
    const bool slot = dev >= 0 && dev < kMaxDevices;
    if (slot) {
        const uint64_t v = cached[dev].load(std::memory_order_relaxed);
        if (v) return (double)v;
    }
    int khz = 0, bits = 0;
    if (cudaDeviceGetAttribute(&khz, cudaDevAttrMemoryClockRate, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&bits, cudaDevAttrGlobalMemoryBusWidth, dev) != cudaSuccess || khz <= 0 || bits <= 0) {
        (void)cudaGetLastError();
        return 5700.0;
    }
    const double rate = 0.7 * 2.0 * (double)khz * 1e3 * (bits / 8.0) * 1e-9;
    if (slot) cached[dev].store((uint64_t)rate, std::memory_order_relaxed);
    return rate;
}

template <int N>
cudaError_t launch_n(const KeysPlan& pl, const KeysParams& p, const CUtensorMap& mk, const CUtensorMap& mv,
                     const CUtensorMap& mq, const CUtensorMap& mkn, const CUtensorMap& mvn,
                     int bh, cudaStream_t stream) {
    static PerDeviceOnce attr_once;
    if (const cudaError_t ea = ensure_dynamic_smem(attr_once, attend_skip_keys_kernel<N>, (int)kSmemMax); ea != cudaSuccess)
        return ea;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(pl.n_splits, bh, 1);
    cfg.blockDim = dim3(64 + (N > 64 ? 256 : 128) + aux_threads(N), 1, 1);
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
    return cudaLaunchKernelEx(&cfg, attend_skip_keys_kernel<N>, mk, mv, mq, mkn, mvn, p);
}

}  // namespace

bool attend_skip_keys_supported(const ec_attn_desc& d, int n_active, bool fresh) {
    if (d.dtype != EC_BF16 || d.head_dim != HD || n_active < 1) return false;
    if (n_active > kMaxActive) return false;
    const KeysPlan pl = make_keys_plan(d, n_active, fresh);
    if (!pl.ok) return false;   // no cluster shape keeps all CTAs resident: the row-major skip kernel streams better
    if ((long long)d.batch * d.n_kv_heads * pl.n_sub > 65535) return false;   // grid.y
    // row chunks re-read the K/V of a head once per chunk: only worth it while the keys can still be split
    if (pl.n_sub_r > 1 && pl.n_splits < 2) return false;
    return true;
}

void attend_skip_keys_describe(const ec_attn_desc& d, int n_active, bool fresh, char* buf, size_t len) {
    const KeysPlan pl = make_keys_plan(d, n_active, fresh);
    snprintf(buf, len, "attend_skip_keys_kernel<%d> grid=(%d,%d) cluster=%d ring_slots=%d smem=%u ctas_per_sm=%d fresh_tiles=%d",
             pl.n_slots, pl.n_splits, d.batch * d.n_kv_heads * pl.n_sub, pl.n_splits, pl.n_stages, pl.smem_bytes, pl.ctas_per_sm,
             pl.n_extra);
}

cudaError_t launch_attend_skip_keys(const AttendArgs& a, const void* k_new, const void* v_new, const int32_t* active_idx,
                                    cudaStream_t stream) {
    const bool fresh = k_new != nullptr;
    const KeysPlan pl = make_keys_plan(a.d, a.n_active, fresh);
    if (!pl.ok) return cudaErrorInvalidConfiguration;
    const int bh = a.d.batch * a.d.n_kv_heads;
    CUtensorMap map_k, map_v;
    if (!make_cache_map(&map_k, a.k_cache, bh, a.d.ctx_len) || !make_cache_map(&map_v, a.v_cache, bh, a.d.ctx_len))
        return cudaErrorInvalidValue;
    KeysParams p{};
    CUtensorMap map_q = map_k, map_kn = map_k, map_vn = map_v;   // placeholders unless q_tma / fresh
    p.q_tma = (pl.group == 1) ? 1 : 0;   // one query head per CTA column: its rows are one TMA box
    if (p.q_tma && !make_q_map(&map_q, a.q, a.d.batch, a.n_active, a.d.n_q_heads, pl.n_slots)) return cudaErrorInvalidValue;
    if (fresh && (!make_fresh_map(&map_kn, k_new, a.d.batch, a.n_active, a.d.n_kv_heads) ||
                  !make_fresh_map(&map_vn, v_new, a.d.batch, a.n_active, a.d.n_kv_heads)))
        return cudaErrorInvalidValue;
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
    p.shift = pl.shift;
    p.n_stages = pl.n_stages;
    p.n_extra = pl.n_extra;
    p.dl = pl.dl;
    p.off_p = pl.off_p;
    p.off_stage = pl.off_stage;
    p.off_list = pl.off_list;
    p.off_bar = pl.off_bar;
    p.scale_log2 = a.scale * kLog2e;
    p.early_cache = (a.d.flags & EC_ATTN_CACHE_SETTLED) ? 1 : 0;
    p.stagger_ns = 0;
    if (pl.tiles_per_split > 1) {
        const double streams = (double)pl.n_splits * bh;   // CTAs with K/V of their own (columns of one head share it through L2)
        const double ns = streams * STAGE / stream_bytes_per_ns();
        p.stagger_ns = (uint32_t)(ns < 3000.0 ? ns : 3000.0);
    }
    const int cols = bh * pl.n_sub;
    return pl.n_slots == 48   ? launch_n<48>(pl, p, map_k, map_v, map_q, map_kn, map_vn, cols, stream)
           : pl.n_slots == 64 ? launch_n<64>(pl, p, map_k, map_v, map_q, map_kn, map_vn, cols, stream)
                              : launch_n<96>(pl, p, map_k, map_v, map_q, map_kn, map_vn, cols, stream);
}

}  // namespace ec
