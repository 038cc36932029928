// ec_entropy_gate: one streaming pass over the logits (Eq. 1 of the paper) that
// yields, per row, argmax / confidence / Shannon entropy, then the maximum
// entropy over the rows flagged "newly decoded" and its comparison with tau
// (Algorithm 1: E > tau -> recompute, else skip).
//
// R*V*sizeof(elem) bytes are read exactly once; the arithmetic is about seven instructions per element.
//   grid  = (splits, R): CTA (s, r) owns the columns [s*chunk, (s+1)*chunk) of row r; the split count is
//           chosen so that the whole grid is about one resident wave (4 CTAs per SM);
//   CTA   : (inputs below 24 MB; larger ones: every thread loads its own vectors through four rolling registers,
//           no producer warp)  8 consumer warps and one producer warp.  The producer's lane 0 moves the chunk through a ring of
//           three 16 KB stages in shared memory with bulk copies (cp.async.bulk, completion on an mbarrier, L2
//           evict-first), as far ahead as the ring allows, so the bytes in flight per SM are the rings of its
//           resident CTAs and do not depend on the consumers' registers;
//   loop  : a consumer thread takes the 16-byte vectors (bf16x8 / f32x4) t, t + 256, ... of the chunk in ascending
//           order, four per stage, and keeps a running
//           (max, S, T) with S = sum 2^d, T = sum 2^d * d, d = x*log2(e) - base: one ex2.approx per element
//           and one packed fp32x2 FMA, add and FMA per pair of elements.  The base follows the maximum lazily: it moves, and S and T
//           are rescaled (S' = 2^dl S, T' = 2^dl (T + dl S), dl = old base - new base), only when a value
//           exceeds it by more than 2^64, so the common path has no data-dependent branch.  Logits are
//           clamped from below at -1e38 (packed bf16 max on the raw words), which keeps d finite:
//           -inf and finfo.min-style masks get probability 0 without a per-element special case;
//   argmax: the thread remembers the iteration that raised its maximum; after the CTA-wide maximum is
//           known, only the threads that attained it look at that iteration's vectors again for the
//           first column (ties -> smallest index, through every reduction stage);
//   reduce: sums rescaled to the CTA's base and added (shuffles + shared memory);
//   merge : CTA partial (M, S, T, idx) -> workspace, one atomic ticket; the last CTA of a sequence
//           (no spinning: tickets only count arrivals) merges the partials of every row of the
//           sequence, writes H = ln S - ln2 * T / S, conf = 2^(M*log2e - base) / S and argmax, takes
//           the flagged maximum and the decision.  Sequences of more than 64 rows, or rows cut into more
//           than 32 splits, use two ticket levels instead (last CTA of a row, then last row of the sequence).
// The entropy identity used: with p_j = 2^{d_j} / S,  -sum p_j ln p_j = ln S - ln2 * T / S
// for any common base, so no partial ever needs the true row maximum.
// The kernel is launched with programmatic stream serialisation and touches global memory only after
// griddepcontrol.wait.  Every mbarrier wait is bounded (one second); a CTA whose wait gave up waits, bounded
// again, for its copies in flight, still arrives at its ticket with a poison bit, and the sequence then reports
// decision -1 instead of a value computed from missing data.
#include "ec_common.cuh"
#include "ec_tc_ptx.cuh"

#include <float.h>

namespace ec {
namespace {

constexpr int kGateThreads = 256;      // consumer threads of a CTA (a producer warp comes on top)
constexpr int kCtasPerSm = 4;
constexpr int kVec = 8;  // columns per thread in one slab of kGateThreads * kVec columns (chunk granularity)
constexpr int kMaxSplits = 96;
constexpr float kDClamp = -150.0f;  // 2^-150 flushes to 0 (ftz)
constexpr int kStages = 3;                          // ring of staged buffers per CTA
constexpr int kInFlight = 4;                        // rolling variant: 16-byte vectors a thread keeps in flight
constexpr int kStageVecs = 4 * kGateThreads;        // 16-byte vectors per stage: four per consumer thread
constexpr uint32_t kStageBytes = kStageVecs * 16u;
constexpr int kPoison = 1 << 20;                    // added to a ticket by a CTA whose wait gave up
constexpr int kSingleLevelMaxRows = 64;
constexpr float kRebase = 64.f;     // the base moves when a value exceeds it by more than 2^kRebase
constexpr unsigned int kXMinBf16x2 = 0xFE96FE96u;   // two bf16 of about -1e38: lower clamp of the logits
constexpr unsigned int kXMinF32 = 0xFE960000u;      // the same value as fp32 bits

struct Partial {
    float M;  // maximum of the chunk (clamped logits)
    float S;  // sum 2^(x*log2e - base(M))
    float T;  // sum 2^(..) * (x*log2e - base(M))
    int idx;  // first column attaining M
};

__device__ __forceinline__ float base_of(float M) { return fmaxf(M * kLog2e, -3.0e38f); }

__device__ __forceinline__ Partial merge(Partial a, Partial b) {
    const bool a_wins = (a.M > b.M) || (a.M == b.M && a.idx <= b.idx);
    Partial hi = a_wins ? a : b;
    const Partial lo = a_wins ? b : a;
    const float dl = base_of(lo.M) - base_of(hi.M);  // <= 0
    if (lo.S > 0.f && dl > kDClamp) {
        const float c = fast_exp2(dl);
        hi.S = fmaf(c, lo.S, hi.S);
        hi.T = fmaf(c, fmaf(dl, lo.S, lo.T), hi.T);
    }
    return hi;
}

// ticket: release (the partial written just before by this thread is visible to whoever sees the count) and
// acquire (whoever completes the count sees every earlier partial)
__device__ __forceinline__ int ticket_add(int* addr, int v) {
    int old;
    asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], %2;" : "=r"(old) : "l"(addr), "r"(v) : "memory");
    return old;
}
// packed pairs of fp32 (one 64-bit register): two lanes per FMA / add issue slot
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
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
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
// global -> shared bulk copy that completes on an mbarrier; the source is read once, so it leaves L2 first
__device__ __forceinline__ uint64_t evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ uint4 lds_v4(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
// barrier of the 256 consumer threads (the producer warp leaves early)
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kGateThreads) : "memory"); }
__device__ __forceinline__ unsigned int max_bf16x2(unsigned int a, unsigned int b) {
    unsigned int d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// One 16-byte vector of a row: EPV elements, kept raw (packed) while in flight.
//   clamp()    lower clamp of all elements, on the raw words
//   vec_max()  maximum of the (clamped) vector as fp32
//   widen()    raw -> fp32
template <typename T>
struct Loader;

template <>
struct Loader<__nv_bfloat16> {
    static constexpr int EPV = 8;
    static __device__ __forceinline__ void clamp(uint4& u) {
        u.x = max_bf16x2(u.x, kXMinBf16x2); u.y = max_bf16x2(u.y, kXMinBf16x2);
        u.z = max_bf16x2(u.z, kXMinBf16x2); u.w = max_bf16x2(u.w, kXMinBf16x2);
    }
    static __device__ __forceinline__ unsigned int max_word(const uint4& u) {
        return max_bf16x2(max_bf16x2(u.x, u.y), max_bf16x2(u.z, u.w));
    }
    static __device__ __forceinline__ unsigned int max_words(unsigned int a, unsigned int b) { return max_bf16x2(a, b); }
    static __device__ __forceinline__ float word_max(unsigned int w) {
        return fmaxf(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
    }
    static __device__ __forceinline__ void widen(const uint4& u, float (&x)[8]) {
        const unsigned int w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    static __device__ __forceinline__ void widen2(const uint4& u, f32x2 (&x)[4]) {
        const unsigned int w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) x[i] = pack2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xffff0000u));
    }
    static __device__ __forceinline__ float one(const __nv_bfloat16* p) {
        return fmaxf(__bfloat162float(*p), __uint_as_float(kXMinF32));
    }
};

template <>
struct Loader<float> {
    static constexpr int EPV = 4;
    static __device__ __forceinline__ void clamp(uint4& u) {
        const float lo = __uint_as_float(kXMinF32);
        u.x = __float_as_uint(fmaxf(__uint_as_float(u.x), lo)); u.y = __float_as_uint(fmaxf(__uint_as_float(u.y), lo));
        u.z = __float_as_uint(fmaxf(__uint_as_float(u.z), lo)); u.w = __float_as_uint(fmaxf(__uint_as_float(u.w), lo));
    }
    // "word" = one fp32 value here
    static __device__ __forceinline__ unsigned int max_word(const uint4& u) {
        return __float_as_uint(fmaxf(fmaxf(__uint_as_float(u.x), __uint_as_float(u.y)),
                                     fmaxf(__uint_as_float(u.z), __uint_as_float(u.w))));
    }
    static __device__ __forceinline__ unsigned int max_words(unsigned int a, unsigned int b) {
        return __float_as_uint(fmaxf(__uint_as_float(a), __uint_as_float(b)));
    }
    static __device__ __forceinline__ float word_max(unsigned int w) { return __uint_as_float(w); }
    static __device__ __forceinline__ void widen(const uint4& u, float (&x)[4]) {
        x[0] = __uint_as_float(u.x); x[1] = __uint_as_float(u.y);
        x[2] = __uint_as_float(u.z); x[3] = __uint_as_float(u.w);
    }
    static __device__ __forceinline__ void widen2(const uint4& u, f32x2 (&x)[2]) {
        x[0] = pack2(__uint_as_float(u.x), __uint_as_float(u.y));
        x[1] = pack2(__uint_as_float(u.z), __uint_as_float(u.w));
    }
    static __device__ __forceinline__ float one(const float* p) { return fmaxf(*p, __uint_as_float(kXMinF32)); }
};

struct GateParams {
    const void* logits;
    long long row_stride;
    int n_rows, vocab, rows_per_seq, splits;
    int chunk;          // columns per CTA, a multiple of kGateThreads * kVec
    int single_level;   // 1: the last CTA of a sequence finishes all its rows; 0: per-row then per-sequence tickets
    const uint8_t* flags;
    float tau;
    int* argmax_out;
    float* conf_out;
    float* entropy_out;  // never null inside the kernel (workspace scratch if the caller gave none)
    float* max_entropy_out;
    int* decision_out;
    int* row_ticket;  // [n_rows], zero on entry, zero on exit
    int* seq_ticket;  // [n_seq],  zero on entry, zero on exit
    Partial* partials;  // [n_rows, splits]
    // decode mode (masked != nullptr, single_level only): the decoded set comes from the confidences
    uint8_t* masked;       // in/out [n_rows]: rows still masked; cleared for the rows decoded here
    float conf_thr;
    uint8_t* decoded_out;  // [n_rows]
    int* tokens;           // [n_rows]: argmax written for the decoded rows
    // Section 5.3's other candidate metrics over the decoded rows (single_level only; either may be null)
    float* ent_sum_out;    // [n_seq]
    float* max_conf_out;   // [n_seq]
};

// warp-collective: merge the split partials of one row, write the row's outputs, return its entropy (all lanes)
__device__ __forceinline__ float finish_row(const GateParams& p, int row, int lane) {
    Partial acc;
    acc.M = -INFINITY; acc.S = 0.f; acc.T = 0.f; acc.idx = 0x7fffffff;
    for (int s = lane; s < p.splits; s += 32) {
        const float4 f = __ldcg(reinterpret_cast<const float4*>(&p.partials[(long long)row * p.splits + s]));
        Partial q;
        q.M = f.x; q.S = f.y; q.T = f.z; q.idx = __float_as_int(f.w);
        acc = merge(acc, q);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Partial q;
        q.M = __shfl_xor_sync(0xffffffffu, acc.M, o);
        q.S = __shfl_xor_sync(0xffffffffu, acc.S, o);
        q.T = __shfl_xor_sync(0xffffffffu, acc.T, o);
        q.idx = __shfl_xor_sync(0xffffffffu, acc.idx, o);
        acc = merge(acc, q);
    }
    const float H = fmaxf(logf(acc.S) - kLn2 * acc.T / acc.S, 0.f);
    if (lane == 0) {
        const float conf = fast_exp2(fmaf(acc.M, kLog2e, -base_of(acc.M))) / acc.S;
        if (p.argmax_out) p.argmax_out[row] = acc.idx;
        if (p.conf_out) p.conf_out[row] = conf;
        p.entropy_out[row] = H;
    }
    return H;
}

// kStaged: the logits come through the bulk-copy ring (a producer warp on top of the consumers); otherwise every
// thread loads its own vectors into a rolling set of kInFlight registers.  The ring wins on small inputs (three
// stages are on their way before any consumer has started: 7.5 against 8.3 us at [32, 126464]), the rolling loads on
// large ones (17.8 against 19.7 us at [256, 126464]): the host picks by size.
template <typename T, bool kStaged>
__global__ void __launch_bounds__(kGateThreads + (kStaged ? 32 : 0), kCtasPerSm) gate_kernel(const GateParams p) {
    __shared__ float s_m[kGateThreads / 32];
    __shared__ int s_i[kGateThreads / 32];
    __shared__ float s_S[kGateThreads / 32], s_T[kGateThreads / 32];
    __shared__ float s_H[kSingleLevelMaxRows];
    __shared__ float s_conf[kSingleLevelMaxRows];
    __shared__ int s_arg[kSingleLevelMaxRows];
    __shared__ int s_last;
    __shared__ __align__(8) unsigned long long s_bar[2 * kStages];
    __shared__ volatile int s_abort;
    __shared__ volatile int s_issued;
    extern __shared__ __align__(128) unsigned char s_ring[];
    const uint32_t ring0 = tc::s2u(s_ring), full0 = tc::s2u(&s_bar[0]), empty0 = tc::s2u(&s_bar[kStages]);

    constexpr int EPV = Loader<T>::EPV;
    const int row = blockIdx.y, split = blockIdx.x, tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    const T* rowp = reinterpret_cast<const T*>(p.logits) + (long long)row * p.row_stride;
    const int c0 = split * p.chunk;
    const int c_end = min(p.vocab, c0 + p.chunk);

    // running state: maximum, exponent base, and S, T as two packed lanes each
    float m = -INFINITY, base = base_of(-INFINITY);
    f32x2 S2 = pack2(0.f, 0.f), T2 = pack2(0.f, 0.f);
    int mcol = -1, mspan = 0;   // where the maximum was raised: first column, and how many elements (a vector or one)
    const f32x2 kL2 = pack2(kLog2e, kLog2e);
    auto rebase_if_needed = [&](float vmax) {
        if (fmaf(vmax, kLog2e, -base) > kRebase) {   // rare
            const float nb = base_of(vmax);
            const float dl = fmaxf(base - nb, kDClamp);
            const float c = fast_exp2(dl);
            float s0, s1, t0, t1;
            unpack2(S2, s0, s1);
            unpack2(T2, t0, t1);
            t0 = s0 > 0.f ? c * fmaf(dl, s0, t0) : 0.f;
            t1 = s1 > 0.f ? c * fmaf(dl, s1, t1) : 0.f;
            S2 = pack2(s0 * c, s1 * c);
            T2 = pack2(t0, t1);
            base = nb;
        }
    };

    // ---- the chunk's whole vectors, staged through shared memory --------------------------------------------------
    // Warp 8 lane 0 issues one bulk copy per stage (16 KB = four vectors per consumer thread) into a ring of kStages
    // buffers, as far ahead as the ring allows; the bytes in flight per SM (the ring of every resident CTA) are what
    // the pass lives on, not the consumers' registers.  Consumer thread t takes the vectors t, t + 256, t + 512, ...
    // of the chunk in ascending order.  The ragged end of a row (a vocabulary that is no multiple of the vector
    // length) is handled element by element below.
    const int n_vec = (c_end - c0) / EPV;                                  // whole vectors of the chunk
    const int n_stage = (n_vec + kStageVecs - 1) / kStageVecs;
    if (tid == 0) {
        if (kStaged) {
#pragma unroll
            for (int i = 0; i < kStages; ++i) { tc::mbar_init(full0 + 8u * i, 1); tc::mbar_init(empty0 + 8u * i, kGateThreads / 32); }
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        s_abort = 0;
        s_issued = -1;
    }
    __syncthreads();
    pdl_wait();                 // the previous kernel of the stream has completed: the logits are final
    pdl_launch_dependents();
    if (kStaged && warp == kGateThreads / 32) {            // the producer warp
        if (lane == 0) {
            const unsigned char* src = reinterpret_cast<const unsigned char*>(rowp + c0);
            const uint64_t policy = evict_first_policy();
            int s = 0;
            for (; s < n_stage; ++s) {
                const int slot = s % kStages;
                if (s >= kStages) tc::mbar_wait(empty0 + 8u * slot, ((s / kStages) - 1) & 1, &s_abort, nullptr);
                if (s_abort) break;
                const uint32_t bytes = (uint32_t)min(kStageVecs, n_vec - s * kStageVecs) * 16u;
                tc::mbar_expect_tx(full0 + 8u * slot, bytes);
                bulk_load(ring0 + (uint32_t)slot * kStageBytes, src + (size_t)s * kStageBytes, bytes, full0 + 8u * slot, policy);
            }
            s_issued = s;
        }
        return;
    }
    auto consume = [&](uint4 raw, int col) {
        Loader<T>::clamp(raw);
        const float vmax = Loader<T>::word_max(Loader<T>::max_word(raw));
        rebase_if_needed(vmax);
        const bool up = vmax > m;   // strictly greater: the first vector of a tie survives
        m = up ? vmax : m;
        mcol = up ? col : mcol;
        mspan = up ? EPV : mspan;
        const f32x2 nb2 = pack2(-base, -base);
        f32x2 x2[EPV / 2];
        Loader<T>::widen2(raw, x2);
#pragma unroll
        for (int i = 0; i < EPV / 2; ++i) {
            const f32x2 d2 = fma2(x2[i], kL2, nb2);
            float d0, d1;
            unpack2(d2, d0, d1);
            const f32x2 e2 = pack2(fast_exp2(d0), fast_exp2(d1));
            S2 = add2(S2, e2);
            T2 = fma2(e2, d2, T2);
        }
    };
    if (!kStaged) {
        // Thread t owns the vectors t, t + 256, ... of the chunk.  They pass through a rolling set of kInFlight
        // registers: as soon as a vector has been consumed its register is given to the load kInFlight vectors ahead.
        constexpr int kVStride = kGateThreads * EPV;
        const int n_mine = n_vec > tid ? (n_vec - tid + kGateThreads - 1) / kGateThreads : 0;
        const T* mine = rowp + c0 + tid * EPV;
        uint4 raw[kInFlight];
#pragma unroll
        for (int v = 0; v < kInFlight; ++v)
            if (v < n_mine) raw[v] = __ldcs(reinterpret_cast<const uint4*>(mine + (long long)v * kVStride));   // streamed once
        int i0 = 0;
        for (; i0 + kInFlight <= n_mine; i0 += kInFlight) {
#pragma unroll
            for (int v = 0; v < kInFlight; ++v) {
                consume(raw[v], c0 + (i0 + v) * kVStride + tid * EPV);
                if (i0 + v + kInFlight < n_mine)
                    raw[v] = __ldcs(reinterpret_cast<const uint4*>(mine + (long long)(i0 + v + kInFlight) * kVStride));
            }
        }
#pragma unroll
        for (int v = 0; v < kInFlight; ++v)
            if (i0 + v < n_mine) consume(raw[v], c0 + (i0 + v) * kVStride + tid * EPV);
    }
    for (int s = 0; kStaged && s < n_stage; ++s) {
        const int slot = s % kStages;
        tc::mbar_wait(full0 + 8u * slot, (s / kStages) & 1, &s_abort, nullptr);
        if (s_abort) break;
        const uint32_t at = ring0 + (uint32_t)slot * kStageBytes + (uint32_t)tid * 16u;
        uint4 raw[kStageVecs / kGateThreads];
#pragma unroll
        for (int k = 0; k < kStageVecs / kGateThreads; ++k) raw[k] = lds_v4(at + (uint32_t)k * kGateThreads * 16u);
#pragma unroll
        for (int k = 0; k < kStageVecs / kGateThreads; ++k) {
            const int v = s * kStageVecs + k * kGateThreads + tid;
            if (v < n_vec) consume(raw[k], c0 + v * EPV);
        }
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(empty0 + 8u * slot);   // the stage's bytes are in registers or consumed
    }
    consumer_sync();
    if (s_abort) {      // uniform: nothing raises the flag after the barrier above
        // a wait gave up (one second): the copies already issued still target this CTA's shared memory, so the CTA
        // stays until they have landed (bounded again) and reports through the poisoned ticket below
        if (tid == 0) {
            unsigned long long t0 = tc::global_timer_ns();
            while (s_issued < 0 && tc::global_timer_ns() - t0 < tc::kWaitLimitNs) {}
            const int issued = max(0, s_issued);
            for (int s = max(0, issued - kStages); s < issued; ++s) {
                t0 = tc::global_timer_ns();
                while (!tc::mbar_try(full0 + 8u * (s % kStages), (s / kStages) & 1) && tc::global_timer_ns() - t0 < tc::kWaitLimitNs) {}
            }
        }
        consumer_sync();
    }
    {   // the ragged end of the chunk: fewer than EPV columns, one element per thread
        const int col = c0 + n_vec * EPV + tid;
        if (col < c_end) {
            const float x = Loader<T>::one(rowp + col);
            rebase_if_needed(x);
            const bool up = x > m;
            m = up ? x : m;
            mcol = up ? col : mcol;
            mspan = up ? 1 : mspan;
            float s0, s1, t0, t1;
            unpack2(S2, s0, s1);
            unpack2(T2, t0, t1);
            const float d = fmaf(x, kLog2e, -base);
            const float e = fast_exp2(d);
            S2 = pack2(s0 + e, s1);
            T2 = pack2(fmaf(e, d, t0), t1);
        }
    }

    // ---- CTA-wide maximum; the threads that attained it find its first column ---------------------------
    // every thread asks again for the vector that raised its maximum (an L2 hit, in flight during the reduction); only
    // the threads that attained the CTA's maximum will look at it
    uint4 again = make_uint4(0u, 0u, 0u, 0u);
    if (mspan == EPV) again = __ldg(reinterpret_cast<const uint4*>(rowp + mcol));
    float wm = m;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, o));
    if (lane == 0) s_m[warp] = wm;
    consumer_sync();
    float M = s_m[0];
#pragma unroll
    for (int w = 1; w < kGateThreads / 32; ++w) M = fmaxf(M, s_m[w]);
    int idx = 0x7fffffff;
    if (m == M && mcol >= 0) {
        if (mspan == EPV) {
            float x[EPV];
            Loader<T>::clamp(again);
            Loader<T>::widen(again, x);
#pragma unroll
            for (int i = EPV - 1; i >= 0; --i)   // descending: the smallest column survives
                if (x[i] == M) idx = mcol + i;
        } else {
            idx = mcol;   // a single element of the ragged end
        }
    }
    // ---- sums against the CTA's base, first column of the maximum --------------------------------------
    float S, Tt;
    {
        float s0, s1, t0, t1;
        unpack2(S2, s0, s1);
        unpack2(T2, t0, t1);
        S = s0 + s1;
        Tt = t0 + t1;
    }
    if (S > 0.f) {
        const float dl = fmaxf(base - base_of(M), kDClamp);
        const float c = fast_exp2(dl);
        Tt = c * fmaf(dl, S, Tt);
        S *= c;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        S += __shfl_xor_sync(0xffffffffu, S, o);
        Tt += __shfl_xor_sync(0xffffffffu, Tt, o);
        idx = min(idx, __shfl_xor_sync(0xffffffffu, idx, o));
    }
    if (lane == 0) { s_S[warp] = S; s_T[warp] = Tt; s_i[warp] = idx; }
    consumer_sync();

    // ---- publish the partial; count arrivals (tickets only count, nothing spins) --------------------
    const int seq = row / p.rows_per_seq;
    if (tid == 0) {
        float Ss = 0.f, Ts = 0.f;
        int Midx = 0x7fffffff;
#pragma unroll
        for (int w = 0; w < kGateThreads / 32; ++w) { Ss += s_S[w]; Ts += s_T[w]; Midx = min(Midx, s_i[w]); }
        *reinterpret_cast<float4*>(&p.partials[(long long)row * p.splits + split]) =
            make_float4(M, Ss, Ts, __int_as_float(Midx));
        // a CTA whose wait gave up still arrives, with the poison bit: the sequence then reports decision -1
        const int mine = 1 + (s_abort ? kPoison : 0);
        const int old = p.single_level ? ticket_add(&p.seq_ticket[seq], mine) : ticket_add(&p.row_ticket[row], mine);
        const int expected = p.single_level ? p.rows_per_seq * p.splits : p.splits;
        s_last = ((old & (kPoison - 1)) == expected - 1 ? 1 : 0) | (old + mine >= kPoison ? 2 : 0);
    }
    consumer_sync();   // orders the ticket's acquire before the other threads' reads of the partials
    if (!(s_last & 1)) return;
    const bool poisoned = (s_last & 2) != 0;

    if (p.single_level) {
        // ---- last CTA of the sequence: finish every row, then the masked maximum and the decision ----
        // eight threads per row (each merges up to four split partials, then three shuffle steps), 32 rows per pass
        for (int r0 = 0; r0 < p.rows_per_seq; r0 += kGateThreads / 8) {
            const int r = r0 + (tid >> 3), j = tid & 7;
            const bool ok = r < p.rows_per_seq;
            const int rr = seq * p.rows_per_seq + (ok ? r : 0);
            float4 f[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int sp = j + 8 * k;
                f[k] = make_float4(-INFINITY, 0.f, 0.f, __int_as_float(0x7fffffff));
                if (ok && sp < p.splits) f[k] = __ldcg(reinterpret_cast<const float4*>(&p.partials[(long long)rr * p.splits + sp]));
            }
            Partial acc;
            acc.M = f[0].x; acc.S = f[0].y; acc.T = f[0].z; acc.idx = __float_as_int(f[0].w);
#pragma unroll
            for (int k = 1; k < 4; ++k) {
                Partial q;
                q.M = f[k].x; q.S = f[k].y; q.T = f[k].z; q.idx = __float_as_int(f[k].w);
                acc = merge(acc, q);
            }
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) {
                Partial q;
                q.M = __shfl_xor_sync(0xffffffffu, acc.M, o);
                q.S = __shfl_xor_sync(0xffffffffu, acc.S, o);
                q.T = __shfl_xor_sync(0xffffffffu, acc.T, o);
                q.idx = __shfl_xor_sync(0xffffffffu, acc.idx, o);
                acc = merge(acc, q);
            }
            if (ok && j == 0) {
                const float H = fmaxf(logf(acc.S) - kLn2 * acc.T / acc.S, 0.f);
                const float conf = fast_exp2(fmaf(acc.M, kLog2e, -base_of(acc.M))) / acc.S;
                if (p.argmax_out) p.argmax_out[rr] = acc.idx;
                if (p.conf_out) p.conf_out[rr] = conf;
                p.entropy_out[rr] = H;
                if (p.masked) {
                    s_H[r] = H;
                    s_conf[r] = conf;
                    s_arg[r] = acc.idx;
                } else {
                    s_H[r] = p.flags[rr] ? H : -INFINITY;
                    s_conf[r] = p.flags[rr] ? conf : -INFINITY;
                }
            }
        }
        consumer_sync();
        if (warp == 0 && p.masked) {
            // ---- confidence-based parallel decoding (Section 2.1 of the paper; threshold 0.9 in its experiments):
            // every masked row above the threshold is decoded; if none is, the masked row of highest confidence
            // (smallest index on ties).  Lane l owns rows l and l + 32 (rows_per_seq <= 64).
            bool msk[2], dec[2];
            float best = -1.f;
            int best_r = 0x7fffffff;
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int r = lane + 32 * q;
                msk[q] = r < p.rows_per_seq && p.masked[seq * p.rows_per_seq + r] != 0;
                dec[q] = msk[q] && s_conf[r] > p.conf_thr;
                if (msk[q] && s_conf[r] > best) { best = s_conf[r]; best_r = r; }   // rows ascend: the first maximum stays
            }
            if (!__any_sync(0xffffffffu, dec[0] || dec[1])) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    const float ob = __shfl_xor_sync(0xffffffffu, best, o);
                    const int orow = __shfl_xor_sync(0xffffffffu, best_r, o);
                    if (ob > best || (ob == best && orow < best_r)) { best = ob; best_r = orow; }
                }
#pragma unroll
                for (int q = 0; q < 2; ++q) dec[q] = msk[q] && (lane + 32 * q == best_r);
            }
            float E = -INFINITY, Hsum = 0.f, Cmax = -INFINITY;
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int r = lane + 32 * q;
                if (r < p.rows_per_seq) {
                    const int rr = seq * p.rows_per_seq + r;
                    p.decoded_out[rr] = dec[q] ? 1 : 0;
                    if (dec[q]) {
                        p.tokens[rr] = s_arg[r];
                        p.masked[rr] = 0;
                        E = fmaxf(E, s_H[r]);
                        Hsum += s_H[r];
                        Cmax = fmaxf(Cmax, s_conf[r]);
                    }
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                E = fmaxf(E, __shfl_xor_sync(0xffffffffu, E, o));
                Hsum += __shfl_xor_sync(0xffffffffu, Hsum, o);
                Cmax = fmaxf(Cmax, __shfl_xor_sync(0xffffffffu, Cmax, o));
            }
            if (lane == 0) {
                if (p.ent_sum_out) p.ent_sum_out[seq] = Hsum;
                if (p.max_conf_out) p.max_conf_out[seq] = Cmax;
                p.max_entropy_out[seq] = E;
                p.decision_out[seq] = poisoned ? -1 : (E > p.tau) ? EC_RECOMPUTE : EC_SKIP;
                p.seq_ticket[seq] = 0;   // ready for the next call
            }
        } else if (warp == 0) {
            float E = -INFINITY, Hsum = 0.f, Cmax = -INFINITY;
            for (int r = lane; r < p.rows_per_seq; r += 32) {
                E = fmaxf(E, s_H[r]);
                Hsum += (s_H[r] == -INFINITY) ? 0.f : s_H[r];   // rows outside the decoded set carry -inf
                Cmax = fmaxf(Cmax, s_conf[r]);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                E = fmaxf(E, __shfl_xor_sync(0xffffffffu, E, o));
                Hsum += __shfl_xor_sync(0xffffffffu, Hsum, o);
                Cmax = fmaxf(Cmax, __shfl_xor_sync(0xffffffffu, Cmax, o));
            }
            if (lane == 0) {
                if (p.ent_sum_out) p.ent_sum_out[seq] = Hsum;
                if (p.max_conf_out) p.max_conf_out[seq] = Cmax;
                p.max_entropy_out[seq] = E;
                p.decision_out[seq] = poisoned ? -1 : (E > p.tau) ? EC_RECOMPUTE : EC_SKIP;
                p.seq_ticket[seq] = 0;   // ready for the next call
            }
        }
        return;
    }

    // ---- last CTA of the row finishes the row; the last row of the sequence finishes the sequence ----
    if (warp != 0) return;
    finish_row(p, row, lane);
    int seq_last = 0;
    if (lane == 0) {
        p.row_ticket[row] = 0;
        const int mine = 1 + (poisoned ? kPoison : 0);
        const int old = ticket_add(&p.seq_ticket[seq], mine);
        seq_last = ((old & (kPoison - 1)) == p.rows_per_seq - 1 ? 1 : 0) | (old + mine >= kPoison ? 2 : 0);
    }
    seq_last = __shfl_sync(0xffffffffu, seq_last, 0);
    if (!(seq_last & 1)) return;
    float E = -INFINITY;
    for (int r = lane; r < p.rows_per_seq; r += 32) {
        const int rr = seq * p.rows_per_seq + r;
        if (p.flags[rr]) E = fmaxf(E, __ldcg(&p.entropy_out[rr]));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) E = fmaxf(E, __shfl_xor_sync(0xffffffffu, E, o));
    if (lane == 0) {
        p.max_entropy_out[seq] = E;
        p.decision_out[seq] = (seq_last & 2) ? -1 : (E > p.tau) ? EC_RECOMPUTE : EC_SKIP;
        p.seq_ticket[seq] = 0;
    }
}

// workspace carving: [row_ticket: R i32][seq_ticket: R i32][entropy scratch: R f32][pad to 16][partials]
struct GateWs {
    size_t off_row, off_seq, off_ent, off_part, total;
};
GateWs carve(int n_rows) {
    GateWs w;
    const size_t r = (size_t)n_rows;
    w.off_row = 0;
    w.off_seq = r * 4;
    w.off_ent = r * 8;
    w.off_part = ((r * 12) + 15) & ~(size_t)15;
    w.total = w.off_part + r * kMaxSplits * sizeof(Partial);
    return w;
}

// split count and columns per CTA: about one resident wave (4 CTAs of 256 threads per SM), every CTA a whole number
// of 2048-column slabs, at most kMaxSplits partials per row
void plan_chunks(int n_rows, int vocab, int* splits, int* chunk, int max_splits = kMaxSplits) {
    const int slab = kGateThreads * kVec;
    const long long slots = (long long)kCtasPerSm * sm_count();
    long long want = slots / n_rows;
    if (want < 1) want = 1;
    if (want > max_splits) want = max_splits;
    long long per = (vocab + want - 1) / want;
    const long long per_min = (vocab + kMaxSplits - 1) / kMaxSplits;
    if (per < per_min) per = per_min;
    per = (per + slab - 1) / slab * slab;
    *chunk = (int)per;
    *splits = (int)((vocab + per - 1) / per);
}

template <typename T, bool kStaged>
cudaError_t launch_t(const GateParams& p, cudaStream_t stream) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(p.splits, p.n_rows, 1);
    cfg.blockDim = dim3(kGateThreads + (kStaged ? 32 : 0), 1, 1);    // the consumer warps (and the producer warp)
    cfg.dynamicSmemBytes = kStaged ? kStages * kStageBytes : 0;
    if (kStaged) {
        static PerDeviceOnce once;
        const cudaError_t e = ensure_dynamic_smem(once, gate_kernel<T, kStaged>, kStages * kStageBytes);
        if (e != cudaSuccess) return e;
    }
    cfg.stream = stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // launch latency may overlap the previous kernel's tail
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gate_kernel<T, kStaged>, p);
}

}  // namespace

size_t gate_workspace_bytes(int n_rows, int vocab) {
    if (n_rows <= 0 || vocab <= 0) return 0;
    return carve(n_rows).total;
}

size_t gate_ticket_bytes(int n_rows) { return n_rows > 0 ? carve(n_rows).off_ent : 0; }   // row + sequence tickets

cudaError_t launch_gate(const GateArgs& a, cudaStream_t stream) {
    const GateWs w = carve(a.n_rows);
    char* ws = static_cast<char*>(a.workspace);
    GateParams p;
    p.logits = a.logits;
    p.row_stride = a.row_stride;
    p.n_rows = a.n_rows;
    p.vocab = a.vocab;
    p.rows_per_seq = a.rows_per_seq;
    p.splits = 0;
    p.chunk = 0;
    p.single_level = 0;
    p.flags = a.flags;
    p.tau = a.tau;
    p.argmax_out = a.argmax_out;
    p.conf_out = a.conf_out;
    p.entropy_out = a.entropy_out ? a.entropy_out : reinterpret_cast<float*>(ws + w.off_ent);
    p.max_entropy_out = a.max_entropy_out;
    p.decision_out = a.decision_out;
    p.row_ticket = reinterpret_cast<int*>(ws + w.off_row);
    p.seq_ticket = reinterpret_cast<int*>(ws + w.off_seq);
    p.partials = reinterpret_cast<Partial*>(ws + w.off_part);
    p.masked = a.masked;
    p.conf_thr = a.conf_threshold;
    p.decoded_out = a.decoded_out;
    p.tokens = a.tokens;
    p.ent_sum_out = a.entropy_sum_out;
    p.max_conf_out = a.max_conf_out;
    // decode mode and the extra metrics need all rows of a sequence in one CTA's hands at the end: the single-level
    // finish (at most 32 splits)
    const bool one_cta_finish = a.masked || a.entropy_sum_out || a.max_conf_out;
    plan_chunks(a.n_rows, a.vocab, &p.splits, &p.chunk, one_cta_finish ? 32 : kMaxSplits);
    if (p.splits > kMaxSplits) return cudaErrorInvalidValue;   // vocab > 96 * 8192: rejected by the API layer before this
    p.single_level = (a.rows_per_seq <= kSingleLevelMaxRows && p.splits <= 32) ? 1 : 0;
    if (one_cta_finish && !p.single_level) return cudaErrorInvalidValue;   // rows_per_seq > 64 or vocab > 32 * 8192 * ...: rejected by the API layer
    // small inputs through the bulk-copy ring, large ones (more than a few chunks per CTA slot) with per-thread loads
    const size_t bytes = (size_t)a.n_rows * a.vocab * (a.dtype == EC_BF16 ? 2 : 4);
    const bool staged = bytes < ((size_t)24 << 20);
    if (a.dtype == EC_BF16)
        return staged ? launch_t<__nv_bfloat16, true>(p, stream) : launch_t<__nv_bfloat16, false>(p, stream);
    return staged ? launch_t<float, true>(p, stream) : launch_t<float, false>(p, stream);
}

}  // namespace ec
