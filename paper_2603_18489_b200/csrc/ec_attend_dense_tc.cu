// ec_attend, recompute step and other dense cases (bf16, head_dim 128, more than 256 packed query rows per
// kv head): bidirectional attention of every active row over the whole cache on the Blackwell tensor cores
// (Appendix A of the paper, full branch; Algorithm 1 FullPrefill / FullRecompute).
//
// The step is bound by the tensor pipe and, next to it, by the exponentials of the softmax.  One CTA owns
// TWO 128-row tiles of the packed (active row x query heads of one kv head) axis and walks over all
// 128-key tiles of that kv head; while the softmax of one row tile runs, the tensor core works for the other.
//   warp 0      TMA producer: K and V tiles ([128 keys x 128] bf16, one 4-D box each: [2 halves][128 keys]
//               [64 columns], 128-byte swizzle) through a ring of five 32 KB slots (K0 V0 K1 V1 ...), and the
//               two Q tiles of the unit, one box each.  (Grouped-query shapes are launched with one unit per
//               QUERY head, so a row tile is always 128 active rows of one head; the query heads of a kv head
//               stream the same K/V, which L2 serves.)
//   warp 1      tcgen05.mma issuer (one thread): S_t = Q_t K^T (both operands K-major in shared memory) into
//               the TMEM columns of row tile t, and O_t += P_t V with P_t read from TENSOR MEMORY (it
//               overwrites the first 64 columns of S_t as packed bf16) and V MN-major from shared memory.
//               Order per key tile j:  P V_0(j), S_0(j+1), P V_1(j), S_1(j+1): the pipe executes in order,
//               so S_t(j+1) cannot overwrite P_t(j) before P V_t(j) has read it;
//   warps 2..17 softmax, four warpgroups: (row tile 0 / 1) x (keys 0..63 / 64..127 of the tile).  A query row
//               (= TMEM lane) is shared by two threads in warps that own the same lanes; they exchange
//               their half-row maxima through shared memory (a 64-thread named barrier), then each does
//               tcgen05.ld of its 64 scores, exp2 with the scale folded in (packed fp32x2 FMA), its share of
//               the row sum, P rounded to bf16 and stored back with tcgen05.st; the O accumulator is only
//               rescaled when a row maximum grows by more than 2^8 (the stale maximum stays the reference
//               otherwise).  Halving the per-thread row shortens the softmax that sits between two uses of
//               the tensor pipe for the same row tile.
//   warp 18     recompute steps only: every cache row is overwritten by the fresh row of the same position, so the
//               launch reads K/V straight from the token-major k_new / v_new (only the tensor map's strides
//               differ) and this warp copies them into the cache meanwhile: no separate refresh pass.
// TMEM (512 columns): S_0 [0,128), S_1 [128,256), O_0 [256,384), O_1 [384,512).
// Shared memory: Q_0, Q_1 (32 KB each, staged once), five 32 KB K/V slots, barriers: 225 KB, one CTA per SM.
// Every mbarrier wait is bounded; a wait that runs out sets EC_ERR_TIMEOUT in the caller's dev_status word and
// a CTA-wide abort flag that makes all later waits fall through; the CTA still frees its TMEM and exits.
#include "ec_common.cuh"
#include "ec_tc_ptx.cuh"

#include <cstdio>

namespace ec {
namespace {

using namespace tc;

constexpr int BM = 128, BN = 128, HD = 128;
constexpr int kSoftThreads = 512;          // four softmax warpgroups: (row tile) x (64-column half)
constexpr int kThreads = 64 + kSoftThreads + 32;   // + one warp that copies fresh K/V into the cache (recompute steps)
constexpr uint32_t SUB = 128 * 128;        // [128 rows x 64 bf16], 128-byte swizzle: 16 KB
constexpr uint32_t TILE = 2 * SUB;         // [128 x 128] bf16
constexpr int kSlots = 5;
constexpr uint32_t OFF_Q = 0;              // two tiles
constexpr uint32_t OFF_RING = 2 * TILE;
constexpr uint32_t OFF_BAR = OFF_RING + kSlots * TILE;   // 224 KB
constexpr uint32_t OFF_XCH = OFF_BAR + 256;               // [2 tiles][2 halves][128 rows] floats
constexpr uint32_t SMEM_BYTES = 232448;                   // all of a CTA's 227 KB; the rest is alignment slack
constexpr uint32_t SMEM_NEEDED = OFF_XCH + 2 * 2 * BM * 4;
constexpr uint32_t TM_COLS = 512;
constexpr uint32_t TM_S = 0, TM_O = 256;   // + 128 * tile

enum { B_FULL = 0, B_EMPTY = kSlots, B_SFULL = 2 * kSlots, B_PFULL = B_SFULL + 2, B_PVDONE = B_PFULL + 2,
       B_QFULL = B_PVDONE + 2, B_COUNT = B_QFULL + 1 };

struct DenseParams {
    const __nv_bfloat16* q;
    __nv_bfloat16* out;
    // recompute step: the K/V this launch reads are the token-major fresh tensors [B, L, Hkv, 128]; its copy warp
    // writes them into the caches [B, Hkv, L, 128] (nullptr: nothing to copy)
    const uint4* k_src;
    const uint4* v_src;
    uint4* k_dst;
    uint4* v_dst;
    int32_t* dev_status;
    int n_active, ctx_len, n_q_heads, n_kv_heads, group, rows_total;
    // Grouped-query shapes run with one unit per QUERY head (the kernel then sees n_kv_heads = n_q_heads = H_q and
    // group = 1, so its row tiles are 128 active rows of one head and come by TMA); the K/V of unit head h are
    // those of the real kv head h / kv_div, of which there are n_kv_real.  kv_div = 1 otherwise.
    int kv_div, n_kv_real;
    float scale_log2;
    // Launch order = unit order (row-tile pair fastest, then head).  The first n_full units are whole; each later
    // unit (the last, partial wave of the launch) is cut along the keys into `split` CTAs that leave un-normalised
    // partials in the workspace for combine_cut_units_kernel.  split = 1: no cuts.
    int n_pairs, n_full, split;
    float* part;      // [cut unit][part][row tile][128 rows x 128 floats, then m[128], then l[128]]
};
constexpr int kPartFloats = BM * (HD + 2);   // one row tile of one part

__global__ void __launch_bounds__(kThreads, 1)
attend_dense_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                    const __grid_constant__ CUtensorMap map_q, const DenseParams p) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (s2u(smem_raw) + 1023u) & ~1023u;
    unsigned char* gbase = smem_raw + (base - s2u(smem_raw));
    const uint32_t bars = base + OFF_BAR;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gbase + OFF_BAR + B_COUNT * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gbase + OFF_BAR + B_COUNT * 8 + 4);
    float* xch = reinterpret_cast<float*>(gbase + OFF_XCH);
    auto bar = [&](int idx) { return bars + idx * 8; };
    if (base - s2u(smem_raw) + SMEM_NEEDED > SMEM_BYTES) {   // never with the 1024-byte alignment the runtime gives
        if (threadIdx.x == 0 && p.dev_status) atomicExch(p.dev_status, (int)EC_ERR_CUDA);
        return;
    }

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int lin = blockIdx.x;
    const bool cut = lin >= p.n_full;
    const int unit = cut ? p.n_full + (lin - p.n_full) / p.split : lin;
    const int part = cut ? (lin - p.n_full) % p.split : 0;
    const int pair = unit % p.n_pairs, bh = unit / p.n_pairs;
    const int b = bh / p.n_kv_heads, hk = bh % p.n_kv_heads;
    const int r_pair = pair * 2 * BM;
    const int n_tiles_q = (p.rows_total - r_pair > BM) ? 2 : 1;   // row tiles of this CTA that hold rows
    const int T_all = (p.ctx_len + BN - 1) / BN;
    const int tiles_per_part = cut ? (T_all + p.split - 1) / p.split : T_all;
    const int j0 = part * tiles_per_part;                        // first key tile of this CTA
    const int T = min(T_all, j0 + tiles_per_part) - j0;          // >= 1 by construction of the plan

    if (tid == 0) {
        prefetch_map(&map_k);
        prefetch_map(&map_v);
        for (int i = 0; i < B_COUNT; ++i)
            mbar_init(bar(i), (i >= B_PFULL && i < B_PFULL + 2) ? 256u : 1u);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s2u(tmem_slot)), "r"(TM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        fence_before();
    }
    __syncthreads();
    fence_after();
    const uint32_t tmem = *tmem_slot;
    pdl_wait();   // the previous kernel of the stream has completed; global memory may be touched
    pdl_launch_dependents();

    if (warp == 0) {
        // ================================ TMA producer ======================================
        if (lane == 0) {
            const int hk_kv = hk / p.kv_div;
            // Q first: [half][row][64 columns] per row tile; rows past n_active read as zero
            prefetch_map(&map_q);
            mbar_expect_tx(bar(B_QFULL), (uint32_t)n_tiles_q * TILE);
            for (int t = 0; t < n_tiles_q; ++t)
                tma_load_5d(base + OFF_Q + t * TILE, &map_q, 0, r_pair + t * BM, hk, 0, b, bar(B_QFULL));
            for (int n = 0; n < 2 * T; ++n) {   // ring index: K_j = 2j, V_j = 2j + 1
                const int slot = n % kSlots, u = n / kSlots;
                if (u > 0) mbar_wait(bar(B_EMPTY + slot), (u - 1) & 1, abort_flag, p.dev_status);
                mbar_expect_tx(bar(B_FULL + slot), TILE);
                tma_load_5d(base + OFF_RING + slot * TILE, (n & 1) ? &map_v : &map_k, 0, (j0 + (n >> 1)) * BN, 0, hk_kv, b, bar(B_FULL + slot));
            }
        }
    } else if (warp == 1) {
        // ================================ MMA issuer ========================================
        if (lane == 0) {
            constexpr uint32_t IDESC_S = instr_desc(BN, 0), IDESC_PV = instr_desc(HD, 1);
            auto wait_full = [&](int n) { mbar_wait(bar(B_FULL + n % kSlots), (n / kSlots) & 1, abort_flag, p.dev_status); };
            auto issue_s = [&](int t, int j) {
                const uint32_t kst = base + OFF_RING + ((2 * j) % kSlots) * TILE;
#pragma unroll
                for (int k = 0; k < HD / 16; ++k) {
                    const uint32_t koff = (k >> 2) * SUB + (k & 3) * 32;
                    mma_ss(tmem + TM_S + t * 128, smem_desc(base + OFF_Q + t * TILE + koff, 16, 1024),
                           smem_desc(kst + koff, 16, 1024), IDESC_S, k > 0);
                }
                commit(bar(B_SFULL + t));
            };
            mbar_wait(bar(B_QFULL), 0, abort_flag, p.dev_status);
            wait_full(0);
            fence_after();
            for (int t = 0; t < n_tiles_q; ++t) issue_s(t, 0);
            commit(bar(B_EMPTY + 0));   // K_0 is free once both S(0) have run
            for (int j = 0; j < T; ++j) {
                wait_full(2 * j + 1);   // V_j
                if (j + 1 < T) wait_full(2 * j + 2);   // K_{j+1}
                const uint32_t vst = base + OFF_RING + ((2 * j + 1) % kSlots) * TILE;
                for (int t = 0; t < n_tiles_q; ++t) {
                    mbar_wait(bar(B_PFULL + t), j & 1, abort_flag, p.dev_status);
                    fence_after();
#pragma unroll
                    for (int k = 0; k < BN / 16; ++k)
                        mma_ts(tmem + TM_O + t * 128, tmem + TM_S + t * 128 + k * 8, smem_desc(vst + k * 2048, SUB, 1024),
                               IDESC_PV, (j > 0 || k > 0));
                    commit(bar(B_PVDONE + t));
                    if (j + 1 < T) issue_s(t, j + 1);
                }
                commit(bar(B_EMPTY + (2 * j + 1) % kSlots));              // V_j
                if (j + 1 < T) commit(bar(B_EMPTY + (2 * j + 2) % kSlots));   // K_{j+1}
            }
        }
    } else if (warp < 2 + kSoftThreads / 32) {
        // ================================ softmax (warps 2..17) ================================
        // A row of a tile is shared by two threads, one per 64-column half, in warps that own the same TMEM
        // lanes: softmax warp ws = warp - 2 -> row tile ws / 8, column half (ws / 4) % 2, lanes 32 * (warp % 4).
        const int ws = warp - 2;
        const int t = ws >> 3, h = (ws >> 2) & 1;
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;        // row of the tile == TMEM lane
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const uint32_t tm_s = tmem + lane_addr + TM_S + t * 128;
        const uint32_t tm_o = tmem + lane_addr + TM_O + t * 128;
        const int r = r_pair + t * BM + row;
        float* xch_mine = xch + (t * 2 + h) * BM + row;        // exchanged with the partner thread of the row
        const float* xch_other = xch + (t * 2 + (1 - h)) * BM + row;
        const int pair_bar = 1 + t * 4 + quarter;              // named barrier of the two warps that share these rows
        if (t < n_tiles_q) {
            float m_used = -INFINITY, l_run = 0.f;
            const float sl2 = p.scale_log2;
            const f32x2 sl2_2 = pk(sl2, sl2);
            for (int j = 0; j < T; ++j) {
                mbar_wait(bar(B_SFULL + t), j & 1, abort_flag, p.dev_status);
                fence_after();
                uint32_t sr[BN / 2];
                ld32(tm_s + h * 64, sr);
                ld32(tm_s + h * 64 + 32, sr + 32);
                wait_ld();
                const int key0 = (j0 + j) * BN + h * 64;
                if (key0 + 64 > p.ctx_len) {
#pragma unroll
                    for (int c = 0; c < 64; ++c)
                        if (key0 + c >= p.ctx_len) sr[c] = 0xff800000u;   // -inf
                }
                float mx[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) mx[c] = __uint_as_float(sr[c]);
#pragma unroll
                for (int c = 4; c < 64; c += 2) mx[(c >> 1) & 3] = max3(mx[(c >> 1) & 3], __uint_as_float(sr[c]), __uint_as_float(sr[c + 1]));
                const float mloc = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
                *xch_mine = mloc;
                named_barrier(pair_bar, 64);   // both halves of the row have loaded their scores and posted their maxima
                const float m_tile = fmaxf(mloc, *xch_other) * sl2;
                float factor = 1.f;
                if (m_tile > m_used + 8.f || m_used == -INFINITY) {   // stale maximum allowed up to 2^8
                    factor = (m_used == -INFINITY) ? 0.f : fast_exp2(m_used - m_tile);
                    m_used = m_tile;
                }
                const bool need_rescale = (j > 0) && __any_sync(0xffffffffu, factor != 1.f);
                const f32x2 mneg2 = pk(-m_used, -m_used);
                f32x2 sum2[2] = {pk(0.f, 0.f), pk(0.f, 0.f)};
                uint32_t pw[32];
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    const f32x2 d2 = fma2(pk(__uint_as_float(sr[2 * c]), __uint_as_float(sr[2 * c + 1])), sl2_2, mneg2);
                    float d0, d1;
                    upk(d2, d0, d1);
                    const float e0 = fast_exp2(d0), e1 = fast_exp2(d1);
                    sum2[c & 1] = add2(sum2[c & 1], pk(e0, e1));
                    pw[c] = pack_bf16x2(e0, e1);
                }
                {
                    float a0, a1, b0, b1;
                    upk(sum2[0], a0, a1);
                    upk(sum2[1], b0, b1);
                    l_run = fmaf(l_run, factor, (a0 + a1) + (b0 + b1));   // this half's share of the row sum
                }
                if (need_rescale) {
                    // O holds tiles < j: P V of tile j - 1 must have completed before the accumulator is scaled;
                    // each of the two threads of a row scales its 64 columns
                    mbar_wait(bar(B_PVDONE + t), (j - 1) & 1, abort_flag, p.dev_status);
                    fence_after();
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t o[32];
                        ld32(tm_o + h * 64 + c * 32, o);
                        wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * factor);
                        st32(tm_o + h * 64 + c * 32, o);
                    }
                }
                // P (bf16 pairs) over the first 64 columns of S_t: this thread's 64 keys are columns [32 h, 32 h + 32)
                st32(tm_s + h * 32, pw);
                wait_st();
                fence_before();
                mbar_arrive(bar(B_PFULL + t));
            }

            // ---- epilogue ------------------------------------------------------------------------
            mbar_wait(bar(B_PVDONE + t), (T - 1) & 1, abort_flag, p.dev_status);
            fence_after();
            *xch_mine = l_run;
            named_barrier(pair_bar, 64);
            const float l_row = l_run + *xch_other;   // both halves of a row carry the same reference maximum
            const bool valid = r < p.rows_total;
            const int i = valid ? r / p.group : 0, jh = valid ? r % p.group : 0;
            __nv_bfloat16* dst = p.out + (((long long)b * p.n_active + i) * p.n_q_heads + hk * p.group + jh) * HD + h * 64;
            if (!cut) {
                // whole unit: normalise and store this thread's 64 columns
                const float inv = 1.f / l_row;
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t o[32];
                    ld32(tm_o + h * 64 + c * 32, o);
                    wait_ld();
                    if (valid && !*abort_flag) {   // a CTA whose wait gave up stores nothing
#pragma unroll
                        for (int v4 = 0; v4 < 4; ++v4) {
                            uint4 w;
                            w.x = pack_bf16x2(__uint_as_float(o[v4 * 8 + 0]) * inv, __uint_as_float(o[v4 * 8 + 1]) * inv);
                            w.y = pack_bf16x2(__uint_as_float(o[v4 * 8 + 2]) * inv, __uint_as_float(o[v4 * 8 + 3]) * inv);
                            w.z = pack_bf16x2(__uint_as_float(o[v4 * 8 + 4]) * inv, __uint_as_float(o[v4 * 8 + 5]) * inv);
                            w.w = pack_bf16x2(__uint_as_float(o[v4 * 8 + 6]) * inv, __uint_as_float(o[v4 * 8 + 7]) * inv);
                            *reinterpret_cast<uint4*>(dst + c * 32 + v4 * 8) = w;
                        }
                    }
                }
            } else {
                // part of a cut unit: the un-normalised row (relative to m_used), m and l go to the workspace; the
                // combine kernel that follows in the stream merges the parts (one CTA combining a unit on its own is
                // bound by what a single SM can pull out of L2: 11 us per extra part)
                const int cu = unit - p.n_full;
                float* mine = p.part + ((size_t)(cu * p.split + part) * 2 + t) * kPartFloats;
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t o[32];
                    ld32(tm_o + h * 64 + c * 32, o);
                    wait_ld();
                    if (!*abort_flag) {
#pragma unroll
                        for (int v4 = 0; v4 < 8; ++v4)
                            *reinterpret_cast<uint4*>(mine + row * HD + h * 64 + c * 32 + v4 * 4) =
                                make_uint4(o[v4 * 4], o[v4 * 4 + 1], o[v4 * 4 + 2], o[v4 * 4 + 3]);
                    }
                }
                if (h == 0 && !*abort_flag) {
                    mine[BM * HD + row] = m_used;
                    mine[BM * HD + BM + row] = l_row;
                }
            }
        }
        fence_before();
    } else if (p.k_dst != nullptr && part == 0) {
        // ====================== copy warp: this CTA's share of the refresh ============================
        // The (row-tile pair, kv head) CTAs of a head split its positions evenly; a position's K and V rows
        // (256 bytes each) go from [b, pos, hk, :] to [b, hk, pos, :].  Two rows per warp instruction, eight
        // instructions in flight.  Nobody reads the cache in this launch.
        // (with one unit per query head, the kv_div units of a real kv head share its positions as well)
        const int hk_kv = hk / p.kv_div;
        const int n_share = p.n_pairs * p.kv_div;
        const int per = (p.ctx_len + n_share - 1) / n_share;
        const int pos0 = ((hk % p.kv_div) * p.n_pairs + pair) * per, pos1 = min(p.ctx_len, pos0 + per);
        const int sub = lane >> 4, piece = lane & 15;
        for (int pos = pos0; pos < pos1; pos += 16) {
            uint4 kv[8], vv[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int pp = pos + 2 * u + sub;
                if (pp < pos1) {
                    const long long src = (((long long)b * p.ctx_len + pp) * p.n_kv_real + hk_kv) * 16 + piece;
                    kv[u] = __ldg(p.k_src + src);
                    vv[u] = __ldg(p.v_src + src);
                }
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int pp = pos + 2 * u + sub;
                if (pp < pos1) {
                    const long long dst = (((long long)b * p.n_kv_real + hk_kv) * p.ctx_len + pp) * 16 + piece;
                    p.k_dst[dst] = kv[u];
                    p.v_dst[dst] = vv[u];
                }
            }
        }
    }

    __syncthreads();
    if (warp == 1) {
        fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TM_COLS) : "memory");
    }
}

// Merges the parts of the cut units: CTA = 32 rows of one row tile of one cut unit, thread = 16 columns of a row.
// With M the largest reference maximum of the row's parts and w_q = 2^(m_q - M):  out = sum_q w_q O_q / sum_q w_q l_q.
struct CombineParams {
    const float* part;
    __nv_bfloat16* out;
    int n_pairs, n_full, split, n_active, n_q_heads, rows_total;
};
__global__ void __launch_bounds__(256) combine_cut_units_kernel(const CombineParams p) {
    pdl_wait();   // the partials of the attention launch are complete
    pdl_launch_dependents();
    const int cu = blockIdx.x >> 3, t = (blockIdx.x >> 2) & 1, row = (blockIdx.x & 3) * 32 + (threadIdx.x >> 3);
    const int c0 = (threadIdx.x & 7) * 16;
    const int unit = p.n_full + cu;
    const int pair = unit % p.n_pairs, bh = unit / p.n_pairs;
    const int b = bh / p.n_q_heads, hq = bh % p.n_q_heads;
    const int r = pair * 2 * BM + t * BM + row;
    if (r >= p.rows_total) return;
    float w[8], M = -INFINITY, L = 0.f;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        w[q] = -INFINITY;
        if (q < p.split) {
            w[q] = __ldcg(p.part + ((size_t)(cu * p.split + q) * 2 + t) * kPartFloats + BM * HD + row);
            M = fmaxf(M, w[q]);
        }
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        if (q < p.split) {
            w[q] = fast_exp2(w[q] - M);
            L = fmaf(w[q], __ldcg(p.part + ((size_t)(cu * p.split + q) * 2 + t) * kPartFloats + BM * HD + BM + row), L);
        }
    }
    float acc[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) acc[e] = 0.f;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        if (q < p.split) {
            const float4* src = reinterpret_cast<const float4*>(
                p.part + ((size_t)(cu * p.split + q) * 2 + t) * kPartFloats + row * HD + c0);
#pragma unroll
            for (int v4 = 0; v4 < 4; ++v4) {
                const float4 f = __ldcg(src + v4);
                acc[v4 * 4 + 0] = fmaf(w[q], f.x, acc[v4 * 4 + 0]);
                acc[v4 * 4 + 1] = fmaf(w[q], f.y, acc[v4 * 4 + 1]);
                acc[v4 * 4 + 2] = fmaf(w[q], f.z, acc[v4 * 4 + 2]);
                acc[v4 * 4 + 3] = fmaf(w[q], f.w, acc[v4 * 4 + 3]);
            }
        }
    }
    const float inv = 1.f / L;
    __nv_bfloat16* dst = p.out + (((long long)b * p.n_active + r) * p.n_q_heads + hq) * HD + c0;
    uint4 o0, o1;
    o0.x = pack_bf16x2(acc[0] * inv, acc[1] * inv);   o0.y = pack_bf16x2(acc[2] * inv, acc[3] * inv);
    o0.z = pack_bf16x2(acc[4] * inv, acc[5] * inv);   o0.w = pack_bf16x2(acc[6] * inv, acc[7] * inv);
    o1.x = pack_bf16x2(acc[8] * inv, acc[9] * inv);   o1.y = pack_bf16x2(acc[10] * inv, acc[11] * inv);
    o1.z = pack_bf16x2(acc[12] * inv, acc[13] * inv); o1.w = pack_bf16x2(acc[14] * inv, acc[15] * inv);
    *reinterpret_cast<uint4*>(dst) = o0;
    *reinterpret_cast<uint4*>(dst + 8) = o1;
}

// ---- host side ---------------------------------------------------------------------------
// Q of an MHA step seen as 5-D {64 columns, active row, head, half, sequence}: one box {64, 128, 1, 2, 1} lands as the
// two 128-byte-swizzled halves of a [128 rows x 128] tile; rows past n_active read as zero.
// K or V seen as 5-D {64 columns, key, half, kv head, sequence}: one box {64, 128, 2, 1, 1} lands as
// [half][key][64 columns], the two 128-byte-swizzled halves of a [128 keys x 128] tile; keys beyond L read as zero.
// Cache layout [B, Hkv, L, 128] or token-major [B, L, Hkv, 128] (the fresh K/V of a recompute step): only the
// strides differ.
bool make_kv_map(CUtensorMap* map, const void* ptr, int batch, int n_kv_heads, int ctx_len, bool token_major) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t row = (cuuint64_t)HD * 2;
    const cuuint64_t dims[5] = {64, (cuuint64_t)ctx_len, 2, (cuuint64_t)n_kv_heads, (cuuint64_t)batch};
    const cuuint64_t strides[4] = {token_major ? row * n_kv_heads : row, 128, token_major ? row : row * ctx_len,
                                   row * ctx_len * n_kv_heads};
    const cuuint32_t box[5] = {64, (cuuint32_t)BN, 2, 1, 1};
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// How the launch is cut.  Units = (sequence, query head, row-tile pair); a unit walks over all T key tiles.  The
// hardware deals the CTAs to the SMs in launch order, so the last units form a partial wave: `tail` units on `sms` SMs.
// Cutting each of them along the keys into s CTAs (s = 2, 4 or 8, at least four key tiles each) fills that wave:
// cost in key-tile times, with two tiles' worth of fixed cost per CTA, one more for writing the partials, and four
// for the combine launch that follows:
//     waves_full * (T + 2) + ceil(tail * s / sms) * (ceil(T / s) + 3) + 4
// s = 1 (no cut) unless a cut saves at least 3 %.
struct DensePlan {
    int n_pairs, units, n_full, split, n_ctas;
};
DensePlan make_dense_plan(const ec_attn_desc& d, int n_active) {
    DensePlan pl;
    pl.n_pairs = (n_active + 2 * BM - 1) / (2 * BM);
    pl.units = pl.n_pairs * d.batch * d.n_q_heads;
    pl.n_full = pl.units;
    pl.split = 1;
    const int sms = sm_count();
    const long long T = (d.ctx_len + BN - 1) / BN;
    const long long waves_full = pl.units / sms, tail = pl.units % sms;
    if (tail > 0) {
        long long best = (waves_full + 1) * (T + 2);
        const long long need = best - best * 3 / 100;
        for (int s = 2; s <= 8; s *= 2) {
            if (T / s < 4) break;
            const long long cost = waves_full * (T + 2) + ((tail * s + sms - 1) / sms) * ((T + s - 1) / s + 3) + 4;
            if (cost < best && cost <= need) {
                best = cost;
                pl.split = s;
            }
        }
        if (pl.split > 1) pl.n_full = pl.units - (int)tail;
    }
    pl.n_ctas = pl.n_full + (pl.units - pl.n_full) * pl.split;
    return pl;
}


}  // namespace

// the two-tile kernel is used when its (row-tile pair, head) units fill the GPU
bool attend_dense_supported(const ec_attn_desc& d, int n_active) {
    if (d.dtype != EC_BF16 || d.head_dim != HD || n_active < 1) return false;
    // one unit per (sequence, query head, row-tile pair): grouped-query shapes are run head by head
    const long long pairs = ((long long)n_active + 2 * BM - 1) / (2 * BM);
    const long long bh = (long long)d.batch * d.n_q_heads;
    if (pairs * bh > 0x3fffffffLL) return false;
    return pairs * bh >= sm_count() / 2;
}

size_t attend_dense_workspace_bytes(const ec_attn_desc& d, int n_active) {
    if (!attend_dense_supported(d, n_active)) return 0;
    const DensePlan pl = make_dense_plan(d, n_active);
    if (pl.split == 1) return 0;
    return (size_t)(pl.units - pl.n_full) * pl.split * 2 * kPartFloats * sizeof(float);
}

void attend_dense_describe(const ec_attn_desc& d, int n_active, char* buf, size_t len) {
    const DensePlan pl = make_dense_plan(d, n_active);
    snprintf(buf, len, "attend_dense_kernel grid=(%d,%d) cluster=1 whole_units=%d cut_units=%dx%d", pl.n_pairs,
             d.batch * d.n_q_heads, pl.n_full, pl.units - pl.n_full, pl.split);
}

cudaError_t launch_attend_dense(const AttendArgs& a, cudaStream_t stream) {
    CUtensorMap map_k, map_v;
    if (!make_kv_map(&map_k, a.k_cache, a.d.batch, a.d.n_kv_heads, a.d.ctx_len, a.kv_token_major) ||
        !make_kv_map(&map_v, a.v_cache, a.d.batch, a.d.n_kv_heads, a.d.ctx_len, a.kv_token_major))
        return cudaErrorInvalidValue;
    DenseParams p;
    p.q = static_cast<const __nv_bfloat16*>(a.q);
    p.out = static_cast<__nv_bfloat16*>(a.out);
    const bool copy = a.kv_token_major && a.refresh_k_dst && a.refresh_v_dst;
    p.k_src = copy ? static_cast<const uint4*>(a.k_cache) : nullptr;
    p.v_src = copy ? static_cast<const uint4*>(a.v_cache) : nullptr;
    p.k_dst = copy ? static_cast<uint4*>(a.refresh_k_dst) : nullptr;
    p.v_dst = copy ? static_cast<uint4*>(a.refresh_v_dst) : nullptr;
    p.dev_status = a.dev_status;
    p.n_active = a.n_active;
    p.ctx_len = a.d.ctx_len;
    p.n_q_heads = a.d.n_q_heads;
    p.n_kv_heads = a.d.n_q_heads;   // the kernel's heads are the query heads, see kv_div
    p.group = 1;
    p.rows_total = a.n_active;
    p.kv_div = a.d.n_q_heads / a.d.n_kv_heads;
    p.n_kv_real = a.d.n_kv_heads;
    p.scale_log2 = a.scale * kLog2e;
    const DensePlan pl = make_dense_plan(a.d, a.n_active);
    p.n_pairs = pl.n_pairs;
    p.n_full = pl.n_full;
    p.split = pl.split;
    p.part = nullptr;
    if (pl.split > 1) {
        if (!a.workspace || a.workspace_bytes < attend_dense_workspace_bytes(a.d, a.n_active)) return cudaErrorInvalidValue;
        p.part = static_cast<float*>(a.workspace);
    }
    CUtensorMap map_q;
    {
        EncodeTiledFn fn = encode_fn();
        if (!fn) return cudaErrorInvalidValue;
        const cuuint64_t dims[5] = {64, (cuuint64_t)a.n_active, (cuuint64_t)a.d.n_q_heads, 2, (cuuint64_t)a.d.batch};
        const cuuint64_t strides[4] = {(cuuint64_t)a.d.n_q_heads * HD * 2, (cuuint64_t)HD * 2, 128,
                                       (cuuint64_t)a.n_active * a.d.n_q_heads * HD * 2};
        const cuuint32_t box[5] = {64, (cuuint32_t)BM, 1, 2, 1};
        const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
        if (fn(&map_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(a.q), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    static PerDeviceOnce attr_once;
    if (const cudaError_t ea = ensure_dynamic_smem(attr_once, attend_dense_kernel, (int)SMEM_BYTES); ea != cudaSuccess) return ea;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(pl.n_ctas, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    if (const cudaError_t el = cudaLaunchKernelEx(&cfg, attend_dense_kernel, map_k, map_v, map_q, p); el != cudaSuccess) return el;
    if (pl.split == 1) return cudaSuccess;
    CombineParams c{p.part, p.out, pl.n_pairs, pl.n_full, pl.split, a.n_active, a.d.n_q_heads, a.n_active};
    cfg.gridDim = dim3((pl.units - pl.n_full) * 8, 1, 1);   // (cut unit, row tile, 32-row group)
    cfg.blockDim = dim3(256, 1, 1);
    cfg.dynamicSmemBytes = 0;
    return cudaLaunchKernelEx(&cfg, combine_cut_units_kernel, c);
}

}  // namespace ec
