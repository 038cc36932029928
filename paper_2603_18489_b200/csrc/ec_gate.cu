// ec_entropy_gate: one streaming pass over the logits (Eq. 1 of the paper) that
// yields, per row, argmax / confidence / Shannon entropy, then the maximum
// entropy over the rows flagged "newly decoded" and its comparison with tau
// (Algorithm 1: E > tau -> recompute, else skip).
//
// The pass is HBM-bound: R*V*sizeof(elem) bytes are read exactly once.
//   grid  = (splits, R): CTA (s, r) owns the column chunk [s*chunk, (s+1)*chunk) of row r,
//           chunk = 256 threads * 8 elements * NV vectors, all loads issued up front
//           as 16-byte vectors (bf16x8 / 2 x f32x4) and held in registers;
//   max   : thread max -> CTA max (shuffles + shared memory), with the first index
//           attaining it (order-preserving 64-bit key, ties -> smallest index);
//   sums  : S = sum 2^d, T = sum 2^d * d with d = x*log2(e) - base, base = fl(M*log2(e)),
//           one ex2.approx + one FMA-formed exponent per element;
//   merge : CTA partial (M, S, T, idx) -> workspace; the last CTA of a row (atomic
//           ticket, no spinning) merges the row's partials and writes
//           H = ln S - ln2 * T / S, conf = 2^(M*log2e - base) / S, argmax;
//           the last row of a sequence takes the flagged maximum and the decision.
// The entropy identity used: with p_j = 2^{d_j} / S,  -sum p_j ln p_j = ln S - ln2 * T / S
// for any common base, so no partial ever needs the true row maximum.
#include "ec_common.cuh"

#include <float.h>

namespace ec {
namespace {

constexpr int kGateThreads = 256;
constexpr int kVec = 8;  // elements per thread per vector
constexpr int kMaxSplits = 96;
constexpr float kDClamp = -150.0f;  // 2^-150 flushes to 0 (ftz): masked / -inf logits add nothing

struct Partial {
    float M;  // raw maximum of the chunk (-inf if the chunk holds no finite value)
    float S;  // sum 2^(x*log2e - base(M))
    float T;  // sum 2^(..) * (x*log2e - base(M))
    int idx;  // first column attaining M
};

__device__ __forceinline__ float base_of(float M) { return fmaxf(M * kLog2e, -3.0e38f); }

__device__ __forceinline__ unsigned int orderable(float f) {
    unsigned int u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float unorderable(unsigned int k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// (M desc, idx asc) lexicographic maximum
__device__ __forceinline__ unsigned long long make_key(float M, int idx) {
    return ((unsigned long long)orderable(M) << 32) | (unsigned int)(0x7fffffff - idx);
}

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

template <typename T>
struct Loader;

template <>
struct Loader<__nv_bfloat16> {
    static __device__ __forceinline__ void vec(const __nv_bfloat16* p, float (&x)[kVec]) {
        const uint4 u = __ldcs(reinterpret_cast<const uint4*>(p));  // streamed once: evict first
        const unsigned int w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    static __device__ __forceinline__ float one(const __nv_bfloat16* p) { return __bfloat162float(*p); }
};

template <>
struct Loader<float> {
    static __device__ __forceinline__ void vec(const float* p, float (&x)[kVec]) {
        const float4 a = __ldcs(reinterpret_cast<const float4*>(p));
        const float4 b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
        x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
        x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
    }
    static __device__ __forceinline__ float one(const float* p) { return *p; }
};

struct GateParams {
    const void* logits;
    long long row_stride;
    int n_rows, vocab, rows_per_seq, splits;
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
};

template <typename T, int NV>
__global__ void __launch_bounds__(kGateThreads) gate_kernel(const GateParams p) {
    __shared__ unsigned long long s_key[kGateThreads / 32];
    __shared__ float s_S[kGateThreads / 32], s_T[kGateThreads / 32];
    __shared__ int s_last;

    const int row = blockIdx.y, split = blockIdx.x, tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    const T* rowp = reinterpret_cast<const T*>(p.logits) + (long long)row * p.row_stride;
    const int c0 = split * (kGateThreads * kVec * NV);
    const int V = p.vocab;

    // ---- load everything this thread owns -----------------------------------------
    float x[NV][kVec];
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const int col = c0 + (v * kGateThreads + tid) * kVec;
        if (col + kVec <= V) {
            Loader<T>::vec(rowp + col, x[v]);
        } else {
#pragma unroll
            for (int i = 0; i < kVec; ++i) x[v][i] = (col + i < V) ? Loader<T>::one(rowp + col + i) : -INFINITY;
        }
    }

    // ---- maximum and its first index ----------------------------------------------
    float tmax = -INFINITY;
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const float m01 = fmaxf(x[v][0], x[v][1]), m23 = fmaxf(x[v][2], x[v][3]);
        const float m45 = fmaxf(x[v][4], x[v][5]), m67 = fmaxf(x[v][6], x[v][7]);
        tmax = fmaxf(tmax, fmaxf(fmaxf(m01, m23), fmaxf(m45, m67)));
    }
    int tidx = 0x7fffffff;
#pragma unroll
    for (int v = NV - 1; v >= 0; --v) {
        const int col = c0 + (v * kGateThreads + tid) * kVec;
#pragma unroll
        for (int i = kVec - 1; i >= 0; --i)
            if (x[v][i] == tmax) tidx = col + i;  // descending scan: the smallest index survives
    }
    unsigned long long key = make_key(tmax, tidx);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, key, o);
        key = other > key ? other : key;
    }
    if (lane == 0) s_key[warp] = key;
    __syncthreads();
    key = s_key[0];
#pragma unroll
    for (int w = 1; w < kGateThreads / 32; ++w) key = s_key[w] > key ? s_key[w] : key;
    const float M = unorderable((unsigned int)(key >> 32));
    const int idx = 0x7fffffff - (int)(unsigned int)(key & 0xffffffffu);
    const float base = base_of(M);

    // ---- exponent sums against the CTA-wide base ----------------------------------
    float S = 0.f, Tt = 0.f;
#pragma unroll
    for (int v = 0; v < NV; ++v) {
#pragma unroll
        for (int i = 0; i < kVec; ++i) {
            const float d = fmaxf(fmaf(x[v][i], kLog2e, -base), kDClamp);
            const float e = fast_exp2(d);
            S += e;
            Tt = fmaf(e, d, Tt);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        S += __shfl_xor_sync(0xffffffffu, S, o);
        Tt += __shfl_xor_sync(0xffffffffu, Tt, o);
    }
    if (lane == 0) { s_S[warp] = S; s_T[warp] = Tt; }
    __syncthreads();

    // ---- publish the partial; the last CTA of the row finishes the row ------------
    if (tid == 0) {
        float Ss = 0.f, Ts = 0.f;
#pragma unroll
        for (int w = 0; w < kGateThreads / 32; ++w) { Ss += s_S[w]; Ts += s_T[w]; }
        Partial out;
        out.M = M; out.S = Ss; out.T = Ts; out.idx = idx;
        int last = 1;
        if (p.splits > 1) {
            *reinterpret_cast<float4*>(&p.partials[(long long)row * p.splits + split]) =
                make_float4(out.M, out.S, out.T, __int_as_float(out.idx));
            __threadfence();
            last = (atomicAdd(&p.row_ticket[row], 1) == p.splits - 1);
        }
        s_last = last;
    }
    __syncthreads();
    if (!s_last || warp != 0) return;

    Partial acc;
    if (p.splits > 1) {
        __threadfence();
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
    } else {
        float Ss = 0.f, Ts = 0.f;
#pragma unroll
        for (int w = 0; w < kGateThreads / 32; ++w) { Ss += s_S[w]; Ts += s_T[w]; }
        acc.M = M; acc.S = Ss; acc.T = Ts; acc.idx = idx;
    }

    int seq_last = 0;
    const int seq = row / p.rows_per_seq;
    if (lane == 0) {
        const float H = fmaxf(logf(acc.S) - kLn2 * acc.T / acc.S, 0.f);
        const float conf = fast_exp2(fmaf(acc.M, kLog2e, -base_of(acc.M))) / acc.S;
        if (p.argmax_out) p.argmax_out[row] = acc.idx;
        if (p.conf_out) p.conf_out[row] = conf;
        p.entropy_out[row] = H;
        if (p.splits > 1) p.row_ticket[row] = 0;  // ready for the next call
        __threadfence();
        seq_last = (atomicAdd(&p.seq_ticket[seq], 1) == p.rows_per_seq - 1);
    }
    seq_last = __shfl_sync(0xffffffffu, seq_last, 0);
    if (!seq_last) return;

    // ---- masked maximum over the sequence's rows and the decision -----------------
    __threadfence();
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

int pick_nv(int n_rows, int vocab) {
    // prefer the largest per-CTA chunk that still gives every SM a few CTAs
    const long long want = 3LL * sm_count();
    for (int nv = 4; nv > 1; nv >>= 1) {
        const long long per = (long long)kGateThreads * kVec * nv;
        const long long ctas = ((vocab + per - 1) / per) * n_rows;
        if (ctas >= want) return nv;
    }
    return 1;
}

template <typename T>
cudaError_t launch_t(const GateParams& p0, int nv, cudaStream_t stream) {
    GateParams p = p0;
    const int per = kGateThreads * kVec * nv;
    p.splits = (p.vocab + per - 1) / per;
    const dim3 grid(p.splits, p.n_rows);
    switch (nv) {
        case 4: gate_kernel<T, 4><<<grid, kGateThreads, 0, stream>>>(p); break;
        case 2: gate_kernel<T, 2><<<grid, kGateThreads, 0, stream>>>(p); break;
        default: gate_kernel<T, 1><<<grid, kGateThreads, 0, stream>>>(p); break;
    }
    return cudaGetLastError();
}

}  // namespace

size_t gate_workspace_bytes(int n_rows, int vocab) {
    if (n_rows <= 0 || vocab <= 0) return 0;
    return carve(n_rows).total;
}

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
    int nv = pick_nv(a.n_rows, a.vocab);
    // the split count must fit the workspace
    while ((a.vocab + kGateThreads * kVec * nv - 1) / (kGateThreads * kVec * nv) > kMaxSplits) nv *= 2;
    if (nv > 4) return cudaErrorInvalidValue;  // vocab > 96 * 8192: rejected by the API layer before this
    return a.dtype == EC_BF16 ? launch_t<__nv_bfloat16>(p, nv, stream) : launch_t<float>(p, nv, stream);
}

}  // namespace ec
