// ec_select_recent: decode history, recent-token selection and the skip_flag / dt bookkeeping of the cached
// denoising loop on the device (Eq. 2-3 and Appendix A of the paper), so that the row list of the next partial
// step never leaves the GPU.
//
// One CTA of 256 threads per sequence.  Thread i owns the contiguous positions [i*per, (i+1)*per), held in
// registers, so a block-wide exclusive scan of the per-thread counts yields R in ascending order.
//   min over K   history values are step indices <= t, so the k-th largest value is found by bisection on the
//                value: the largest v in [vmin, t] with |{i : H_i >= v}| >= k; each probe is one block-wide count.
//                If fewer than k positions were ever decoded the minimum is "-infinity" and only t - dt limits R.
// The kernel has no waits; an out-of-range window (block mode) or a window list that does not consist of masked
// positions (sliding mode) leaves the sequence untouched and reports n_active = -1.
#include "ec_common.cuh"

namespace ec {
namespace {

constexpr int kSelThreads = 256;
constexpr int kSelMaxPer = 64;   // positions per thread: ctx_len <= 16384

struct SelectParams {
    int32_t* history;
    ec_step_state* state;
    const uint8_t* decoded;
    const int32_t* window_start;
    const int32_t* decision;
    int32_t* active_idx;
    uint8_t* masked;   // sliding-window mode: [batch, ctx_len] positions still masked (in/out); nullptr: block mode
    int ctx_len, block, k, n_cap;
};

__device__ __forceinline__ int block_sum(int v, int* scratch) {   // every thread gets the total
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v = __reduce_add_sync(0xffffffffu, v);
    __syncthreads();   // scratch from the previous use has been read
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    int total = 0;
#pragma unroll
    for (int w = 0; w < kSelThreads / 32; ++w) total += scratch[w];
    return total;
}

template <int PER>   // positions per thread held in registers: ctx_len <= PER * 256
__global__ void __launch_bounds__(kSelThreads) select_recent_kernel(const SelectParams p) {
    __shared__ int scratch[kSelThreads / 32];
    __shared__ int warp_base[kSelThreads / 32];
    const int b = blockIdx.x, tid = threadIdx.x;
    int32_t* H = p.history + (long long)b * p.ctx_len;
    ec_step_state st = p.state[b];
    const bool sliding = p.masked != nullptr;
    uint8_t* M = sliding ? p.masked + (long long)b * p.ctx_len : nullptr;
    int32_t* idx = p.active_idx + (long long)b * p.n_cap;
    const int w0 = sliding ? 0 : p.window_start[b];
    if (!sliding && (w0 < 0 || w0 > p.ctx_len - p.block)) {   // uniform over the CTA
        if (tid == 0) p.state[b].n_active = -1;
        return;
    }
    // sliding mode: the current window holds min(block, masked positions left) rows; the list entries behind it are
    // recent rows, not window rows, whatever their flags say
    int n_cur = p.block;
    if (sliding) {
        const int per0 = (p.ctx_len + kSelThreads - 1) / kSelThreads;
        int c = 0;
        for (int j = 0; j < per0; ++j) {
            const int pos = tid * per0 + j;
            c += (pos < p.ctx_len && M[pos] != 0) ? 1 : 0;
        }
        c = block_sum(c, scratch);
        n_cur = c < p.block ? c : p.block;
        __syncthreads();
        // the window rows must be the list the previous call (or, before the first call, the caller) wrote: in range
        // and still masked.  Anything else would credit the decoded flags to the wrong positions, so the sequence is
        // left untouched and reports n_active = -1, as an out-of-range window does in block mode.
        int bad = 0;
        for (int r = tid; r < n_cur; r += kSelThreads) {
            const int pos = idx[r];
            bad += (pos < 0 || pos >= p.ctx_len || M[pos] == 0) ? 1 : 0;
        }
        bad = block_sum(bad, scratch);
        __syncthreads();
        if (bad) {   // uniform over the CTA
            if (tid == 0) p.state[b].n_active = -1;
            return;
        }
    }
    // ---- Eq. 2: the positions decoded in this step get the step's index -----------------------------
    // block mode: window row r is position w0 + r; sliding mode: it is entry r of the row list of the previous call
    for (int r = tid; r < n_cur; r += kSelThreads) {
        if (p.decoded[(long long)b * p.block + r]) {
            const int pos = sliding ? idx[r] : w0 + r;
            if (pos >= 0 && pos < p.ctx_len) {
                H[pos] = st.t;
                if (sliding) M[pos] = 0;
            }
        }
    }
    __syncthreads();

    const int per = (p.ctx_len + kSelThreads - 1) / kSelThreads;
    const int i0 = tid * per;
    int32_t h[PER];
    int vmin_local = INT32_MAX;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
        h[j] = (j < per && i0 + j < p.ctx_len) ? H[i0 + j] : EC_H_NEVER;
        if (h[j] != EC_H_NEVER) vmin_local = min(vmin_local, h[j]);
    }
    auto count_ge = [&](int v) {
        int c = 0;
#pragma unroll
        for (int j = 0; j < PER; ++j) c += (h[j] != EC_H_NEVER && h[j] >= v) ? 1 : 0;
        return block_sum(c, scratch);
    };
    // ---- Eq. 3: min over the k largest = largest v with at least k entries >= v -----------------------
    long long tau = (long long)st.t - st.dt_recompute;   // t - dt; the k-th largest can only raise it
    bool empty = false;
    if (p.k == 0) {
        empty = true;   // minimum over the empty set: nothing reaches it
    } else {
        // smallest decoded value of the sequence (or "none")
        int vmin = vmin_local;
        vmin = __reduce_min_sync(0xffffffffu, vmin);
        __syncthreads();
        if ((tid & 31) == 0) scratch[tid >> 5] = vmin;
        __syncthreads();
        vmin = INT32_MAX;
#pragma unroll
        for (int w = 0; w < kSelThreads / 32; ++w) vmin = min(vmin, scratch[w]);
        if (vmin != INT32_MAX && count_ge(vmin) >= p.k) {
            // at least k decoded positions: bisect for the k-th largest value in [vmin, vmax]; no entry exceeds t
            long long lo = vmin, hi = st.t;   // count_ge(lo) >= k holds; find the largest such v
            if (count_ge((int)hi) >= p.k) {
                lo = hi;
            } else {
                while (hi - lo > 1) {   // invariant: count_ge(lo) >= k > count_ge(hi)
                    const long long mid = lo + (hi - lo) / 2;
                    if (count_ge((int)mid) >= p.k) lo = mid; else hi = mid;
                }
            }
            tau = tau > lo ? tau : lo;
        }
    }
    // exclusive scan of per-thread counts over the CTA (threads own ascending position ranges): base of this thread, total
    const int lane = tid & 31, warp = tid >> 5;
    auto block_scan = [&](int mine, int& base, int& total) {
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int n = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += n;
        }
        __syncthreads();
        if (lane == 31) scratch[warp] = incl;
        __syncthreads();
        if (tid == 0) {
            int run = 0;
            for (int w = 0; w < kSelThreads / 32; ++w) {
                warp_base[w] = run;
                run += scratch[w];
            }
            scratch[0] = run;
        }
        __syncthreads();
        total = scratch[0];
        base = warp_base[warp] + incl - mine;
    };
    // ---- the window's rows ---------------------------------------------------------------------------
    int n_win = p.block;
    if (!sliding) {
        for (int r = tid; r < p.block; r += kSelThreads) idx[r] = w0 + r;   // block <= n_cap (checked on the host)
    } else {
        // sliding window: the first `block` positions that are still masked (fewer when fewer remain)
        unsigned long long mbits = 0ull;
        int mine_m = 0;
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            const int pos = i0 + j;
            if (j < per && pos < p.ctx_len && M[pos] != 0) {
                mbits |= 1ull << j;
                ++mine_m;
            }
        }
        int base_m, total_m;
        block_scan(mine_m, base_m, total_m);
        n_win = total_m < p.block ? total_m : p.block;
        int at_m = base_m;
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            if ((mbits >> j) & 1ull) {
                if (at_m < p.block) idx[at_m] = i0 + j;
                ++at_m;
            }
        }
    }
    // ---- R (outside the block in block mode; a decoded position is never in a sliding window), ascending ----
    int mine = 0;
    if (!empty) {
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            const int pos = i0 + j;
            const bool in_r = h[j] != EC_H_NEVER && (long long)h[j] >= tau;
            mine += (in_r && (sliding || pos < w0 || pos >= w0 + p.block)) ? 1 : 0;
        }
    }
    int base_r, n_out;
    block_scan(mine, base_r, n_out);
    int at = n_win + base_r;
    if (!empty) {
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            const int pos = i0 + j;
            const bool in_r = h[j] != EC_H_NEVER && (long long)h[j] >= tau;
            if (in_r && (sliding || pos < w0 || pos >= w0 + p.block)) {
                if (at < p.n_cap) idx[at] = pos;
                ++at;
            }
        }
    }
    for (int r = n_win + n_out + tid; r < p.n_cap; r += kSelThreads) idx[r] = -1;
    // ---- Appendix A: skip_flag, dt, t ------------------------------------------------------------------
    if (tid == 0) {
        const int skip = p.decision[b] == EC_SKIP ? 1 : 0;
        st.skip_flag = skip;
        st.dt_recompute = skip ? st.dt_recompute + 1 : 0;
        st.t = st.t + 1;
        st.n_active = n_win + n_out;
        p.state[b] = st;
    }
}

}  // namespace

int select_recent_max_ctx() { return kSelMaxPer * kSelThreads; }

cudaError_t launch_select_recent(int32_t* history, int ctx_len, int batch, ec_step_state* state, const uint8_t* decoded,
                                 const int32_t* window_start, int block, const int32_t* decision, int k,
                                 int32_t* active_idx, int n_cap, uint8_t* masked, cudaStream_t stream) {
    SelectParams p{history, state, decoded, window_start, decision, active_idx, masked, ctx_len, block, k, n_cap};
    if (ctx_len <= 4 * kSelThreads) select_recent_kernel<4><<<batch, kSelThreads, 0, stream>>>(p);
    else if (ctx_len <= 16 * kSelThreads) select_recent_kernel<16><<<batch, kSelThreads, 0, stream>>>(p);
    else select_recent_kernel<kSelMaxPer><<<batch, kSelThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace ec
