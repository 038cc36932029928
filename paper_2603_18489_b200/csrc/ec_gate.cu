// ec_entropy_gate: one streaming pass over the logits (Eq. 1 of the paper) that
// yields, per row, argmax / confidence / Shannon entropy, then the maximum
// entropy over the rows flagged "newly decoded" and its comparison with tau
// (Algorithm 1: E > tau -> recompute, else skip).
//
// The pass is HBM-bound: R*V*sizeof(elem) bytes are read exactly once; the arithmetic is kept to about
// six instructions per element so that the issue slots do not become the limit first.
//   grid  = (splits, R): CTA (s, r) owns the columns [s*chunk, (s+1)*chunk) of row r; the split count is
//           chosen so that the whole grid is about one resident wave (4 CTAs of 256 threads per SM);
//   loop  : a thread visits its columns in ascending order, four 16-byte vectors (bf16x8 / f32x4) per
//           iteration, the next four already in flight (register double buffer), and keeps a running
//           (max, S, T) with S = sum 2^d, T = sum 2^d * d, d = x*log2(e) - base: one ex2.approx per element
//           and one packed fp32x2 FMA, add and FMA per pair of elements.  The base follows the maximum lazily: it moves, and S and T
//           are rescaled (S' = 2^dl S, T' = 2^dl (T + dl S), dl = old base - new base), only when a value
//           exceeds it by more than 2^64, so the common path has no data-dependent branch.  Logits are
//           clamped from below at -1e38 (packed bf16 max on the raw words), which keeps d finite:
//           -inf and finfo.min-style masks get probability 0 without a per-element special case;
//   argmax: the thread remembers the iteration that raised its maximum; after the CTA-wide maximum is
//           known, only the threads that attained it look at that iteration's vectors again for the
//           first column (ties -> smallest index, through every reduction stage);
//   CTA   : sums rescaled to the CTA's base and added (shuffles + shared memory);
//   merge : CTA partial (M, S, T, idx) -> workspace, one atomic ticket; the last CTA of a sequence
//           (no spinning: tickets only count arrivals) merges the partials of every row of the
//           sequence, writes H = ln S - ln2 * T / S, conf = 2^(M*log2e - base) / S and argmax, takes
//           the flagged maximum and the decision.  Sequences of more than 64 rows, or rows cut into more
//           than 32 splits, use two ticket levels instead (last CTA of a row, then last row of the sequence).
// The entropy identity used: with p_j = 2^{d_j} / S,  -sum p_j ln p_j = ln S - ln2 * T / S
// for any common base, so no partial ever needs the true row maximum.
// The kernel is launched with programmatic stream serialisation and touches global memory only after
// griddepcontrol.wait.
#include "ec_common.cuh"

#include <float.h>

namespace ec {
namespace {

constexpr int kGateThreads = 256;
constexpr int kVec = 8;  // columns per thread in one slab of kGateThreads * kVec columns (chunk granularity)
constexpr int kMaxSplits = 96;
constexpr float kDClamp = -150.0f;  // 2^-150 flushes to 0 (ftz)
constexpr int kUnroll = 4;          // 16-byte vectors per thread per iteration
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

template <typename T>
__global__ void __launch_bounds__(kGateThreads, 4) gate_kernel(const GateParams p) {
    __shared__ float s_m[kGateThreads / 32];
    __shared__ int s_i[kGateThreads / 32];
    __shared__ float s_S[kGateThreads / 32], s_T[kGateThreads / 32];
    __shared__ float s_H[kSingleLevelMaxRows];
    __shared__ float s_conf[kSingleLevelMaxRows];
    __shared__ int s_arg[kSingleLevelMaxRows];
    __shared__ int s_last;

    constexpr int EPV = Loader<T>::EPV;
    constexpr int kVStride = kGateThreads * EPV;     // columns between a thread's consecutive vectors
    constexpr int kStep = kUnroll * kVStride;        // columns per loop iteration
    const int row = blockIdx.y, split = blockIdx.x, tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    const T* rowp = reinterpret_cast<const T*>(p.logits) + (long long)row * p.row_stride;
    const int c0 = split * p.chunk;
    const int c_end = min(p.vocab, c0 + p.chunk);

    pdl_wait();                 // the previous kernel of the stream has completed: the logits are final
    pdl_launch_dependents();

    // running state: maximum, exponent base, and S, T as two packed lanes each
    float m = -INFINITY, base = base_of(-INFINITY);
    f32x2 S2 = pack2(0.f, 0.f), T2 = pack2(0.f, 0.f);
    int mcol = -1, mspan = 0;   // where the maximum was raised: first column of the vectors to look at again, and how many
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

    // ---- kUnroll vectors per thread per iteration, the next kUnroll already in flight ------------------------
    // Only the chunk's last iteration can hold vectors that are ragged or past the end; it takes the guarded path.
    const int n_full = (c_end - c0) / kStep;
    const int n_iter = (c_end - c0 + kStep - 1) / kStep;
    auto fetch = [&](int it, uint4 (&raw)[kUnroll]) {
        const int col0 = c0 + it * kStep + tid * EPV;
        if (it < n_full) {
#pragma unroll
            for (int v = 0; v < kUnroll; ++v) raw[v] = __ldcs(reinterpret_cast<const uint4*>(rowp + col0 + v * kVStride));   // streamed once
        } else {
#pragma unroll
            for (int v = 0; v < kUnroll; ++v)
                if (col0 + v * kVStride + EPV <= c_end) raw[v] = __ldcs(reinterpret_cast<const uint4*>(rowp + col0 + v * kVStride));
        }
    };
    auto consume = [&](int it, uint4 (&raw)[kUnroll]) {
        const int col0 = c0 + it * kStep + tid * EPV;
        if (it < n_full) {
            unsigned int w = 0;
#pragma unroll
            for (int v = 0; v < kUnroll; ++v) {
                Loader<T>::clamp(raw[v]);
                const unsigned int wv = Loader<T>::max_word(raw[v]);
                w = v == 0 ? wv : Loader<T>::max_words(w, wv);
            }
            const float it_max = Loader<T>::word_max(w);
            rebase_if_needed(it_max);
            const bool up = it_max > m;   // strictly greater: the first iteration of a tie survives
            m = up ? it_max : m;
            mcol = up ? col0 : mcol;
            mspan = up ? kUnroll : mspan;
            const f32x2 nb2 = pack2(-base, -base);
#pragma unroll
            for (int v = 0; v < kUnroll; ++v) {
                f32x2 x2[EPV / 2];
                Loader<T>::widen2(raw[v], x2);
#pragma unroll
                for (int i = 0; i < EPV / 2; ++i) {
                    const f32x2 d2 = fma2(x2[i], kL2, nb2);
                    float d0, d1;
                    unpack2(d2, d0, d1);
                    const f32x2 e2 = pack2(fast_exp2(d0), fast_exp2(d1));
                    S2 = add2(S2, e2);
                    T2 = fma2(e2, d2, T2);
                }
            }
        } else {
#pragma unroll
            for (int v = 0; v < kUnroll; ++v) {
                const int col = col0 + v * kVStride;
                if (col >= c_end) continue;
                float x[EPV];
                if (col + EPV <= c_end) {
                    Loader<T>::clamp(raw[v]);
                    Loader<T>::widen(raw[v], x);
                } else {   // ragged end of the row: -inf stands for "no column"
#pragma unroll
                    for (int i = 0; i < EPV; ++i) x[i] = (col + i < c_end) ? Loader<T>::one(rowp + col + i) : -INFINITY;
                }
                float vmax = x[0];
#pragma unroll
                for (int i = 1; i < EPV; ++i) vmax = fmaxf(vmax, x[i]);
                rebase_if_needed(vmax);
                const bool up = vmax > m;
                m = up ? vmax : m;
                mcol = up ? col : mcol;
                mspan = up ? 1 : mspan;
                float s0, s1, t0, t1;
                unpack2(S2, s0, s1);
                unpack2(T2, t0, t1);
#pragma unroll
                for (int i = 0; i < EPV; ++i) {   // 2^-inf = 0, and that product is kept out of T
                    const float d = fmaf(x[i], kLog2e, -base);
                    const float e = fast_exp2(d);
                    s0 += e;
                    t0 = (x[i] == -INFINITY) ? t0 : fmaf(e, d, t0);
                }
                S2 = pack2(s0, s1);
                T2 = pack2(t0, t1);
            }
        }
    };
    {
        uint4 ra[kUnroll], rb[kUnroll];
        fetch(0, ra);
        for (int it = 0; it < n_iter; it += 2) {
            if (it + 1 < n_iter) fetch(it + 1, rb);
            consume(it, ra);
            if (it + 1 < n_iter) {
                if (it + 2 < n_iter) fetch(it + 2, ra);
                consume(it + 1, rb);
            }
        }
    }

    // ---- CTA-wide maximum; the threads that attained it find its first column ---------------------------
    // every thread asks again for the vectors that raised its maximum (L2 hits, in flight during the reduction);
    // only the threads that attained the CTA's maximum will look at them
    uint4 again[kUnroll];
#pragma unroll
    for (int v = 0; v < kUnroll; ++v) {
        again[v] = make_uint4(0u, 0u, 0u, 0u);
        const int col = mcol + v * kVStride;
        if (v < mspan && mcol >= 0 && col + EPV <= c_end) again[v] = __ldg(reinterpret_cast<const uint4*>(rowp + col));
    }
    float wm = m;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, o));
    if (lane == 0) s_m[warp] = wm;
    __syncthreads();
    float M = s_m[0];
#pragma unroll
    for (int w = 1; w < kGateThreads / 32; ++w) M = fmaxf(M, s_m[w]);
    int idx = 0x7fffffff;
    if (m == M && mcol >= 0) {
#pragma unroll
        for (int v = kUnroll - 1; v >= 0; --v) {   // descending: the smallest column survives
            const int col = mcol + v * kVStride;
            if (v >= mspan) continue;
            if (col + EPV <= c_end) {
                float x[EPV];
                Loader<T>::clamp(again[v]);
                Loader<T>::widen(again[v], x);
#pragma unroll
                for (int i = EPV - 1; i >= 0; --i)
                    if (x[i] == M) idx = col + i;
            } else {   // the chunk's ragged last vector
#pragma unroll
                for (int i = EPV - 1; i >= 0; --i)
                    if (col + i < c_end && Loader<T>::one(rowp + col + i) == M) idx = col + i;
            }
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
    __syncthreads();

    // ---- publish the partial; count arrivals (tickets only count, nothing spins) --------------------
    const int seq = row / p.rows_per_seq;
    if (tid == 0) {
        float Ss = 0.f, Ts = 0.f;
        int Midx = 0x7fffffff;
#pragma unroll
        for (int w = 0; w < kGateThreads / 32; ++w) { Ss += s_S[w]; Ts += s_T[w]; Midx = min(Midx, s_i[w]); }
        *reinterpret_cast<float4*>(&p.partials[(long long)row * p.splits + split]) =
            make_float4(M, Ss, Ts, __int_as_float(Midx));
        int last;
        if (p.single_level)
            last = (ticket_add(&p.seq_ticket[seq], 1) == p.rows_per_seq * p.splits - 1);
        else
            last = (ticket_add(&p.row_ticket[row], 1) == p.splits - 1);
        s_last = last;
    }
    __syncthreads();   // orders the ticket's acquire before the other threads' reads of the partials
    if (!s_last) return;

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
        __syncthreads();
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
                p.decision_out[seq] = (E > p.tau) ? EC_RECOMPUTE : EC_SKIP;
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
                p.decision_out[seq] = (E > p.tau) ? EC_RECOMPUTE : EC_SKIP;
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
        seq_last = (ticket_add(&p.seq_ticket[seq], 1) == p.rows_per_seq - 1);
    }
    seq_last = __shfl_sync(0xffffffffu, seq_last, 0);
    if (!seq_last) return;
    float E = -INFINITY;
    for (int r = lane; r < p.rows_per_seq; r += 32) {
        const int rr = seq * p.rows_per_seq + r;
        if (p.flags[rr]) E = fmaxf(E, __ldcg(&p.entropy_out[rr]));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) E = fmaxf(E, __shfl_xor_sync(0xffffffffu, E, o));
    if (lane == 0) {
        p.max_entropy_out[seq] = E;
        p.decision_out[seq] = (E > p.tau) ? EC_RECOMPUTE : EC_SKIP;
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
    const long long slots = 4LL * sm_count();
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

template <typename T>
cudaError_t launch_t(const GateParams& p, cudaStream_t stream) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(p.splits, p.n_rows, 1);
    cfg.blockDim = dim3(kGateThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // launch latency may overlap the previous kernel's tail
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gate_kernel<T>, p);
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
    return a.dtype == EC_BF16 ? launch_t<__nv_bfloat16>(p, stream) : launch_t<float>(p, stream);
}

}  // namespace ec
