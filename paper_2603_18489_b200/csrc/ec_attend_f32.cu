// ec_attend, fp32 storage: active-row bidirectional attention over the full
// cache (Appendix A of the paper, partial branch; the full branch when every row
// is active) computed entirely in fp32 on the FMA pipes.
//
// fp32 tensors are the small validation geometry; the tight tolerance that goes
// with them (1e-5 relative) rules out tf32 tensor cores, so this is a plain SIMT
// kernel: one warp per (sequence, active row, query head).
//   scores : lane l takes key c*32+l of a 32-key chunk and dots its K row with
//            the query (staged in shared memory, read as broadcast float4);
//   softmax: online over chunks (running max m, running sum l), accurate expf;
//   PV     : every lane owns head_dim/32 output columns; the chunk's 32
//            probabilities are broadcast by shuffle and V rows are read coalesced.
#include "ec_common.cuh"

namespace ec {
namespace {

constexpr int kWarpsPerCta = 4;

template <int D>
__global__ void __launch_bounds__(kWarpsPerCta * 32) attend_f32_kernel(
    const float* __restrict__ q, const float* __restrict__ k_cache, const float* __restrict__ v_cache,
    float* __restrict__ out, int batch, int n_active, int ctx_len, int n_q_heads, int n_kv_heads, float scale) {
    __shared__ __align__(16) float s_q[kWarpsPerCta][D];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long job = (long long)blockIdx.x * kWarpsPerCta + warp;
    const long long n_jobs = (long long)batch * n_active * n_q_heads;
    if (job >= n_jobs) return;  // whole warp leaves together; no block-wide barrier below
    const int hq = (int)(job % n_q_heads);
    const long long bi = job / n_q_heads;
    const long long b = bi / n_active;
    const int hk = hq / (n_q_heads / n_kv_heads);
    constexpr int DPL = D / 32;  // output columns per lane

    const float* qrow = q + job * D;
#pragma unroll
    for (int t = 0; t < DPL; ++t) s_q[warp][lane + 32 * t] = qrow[lane + 32 * t];
    __syncwarp();

    const float* kb = k_cache + ((b * n_kv_heads + hk) * (long long)ctx_len) * D;
    const float* vb = v_cache + ((b * n_kv_heads + hk) * (long long)ctx_len) * D;

    float m = -INFINITY, l = 0.f;
    float acc[DPL];
#pragma unroll
    for (int t = 0; t < DPL; ++t) acc[t] = 0.f;

    for (int c0 = 0; c0 < ctx_len; c0 += 32) {
        const int j = c0 + lane;
        float s = -INFINITY;
        if (j < ctx_len) {
            const float4* kr = reinterpret_cast<const float4*>(kb + (long long)j * D);
            const float4* qs = reinterpret_cast<const float4*>(s_q[warp]);
            float d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;  // four partial sums: shorter chains, smaller error
#pragma unroll
            for (int d4 = 0; d4 < D / 4; ++d4) {
                const float4 kv = __ldg(kr + d4);
                const float4 qv = qs[d4];
                d0 = fmaf(qv.x, kv.x, d0);
                d1 = fmaf(qv.y, kv.y, d1);
                d2 = fmaf(qv.z, kv.z, d2);
                d3 = fmaf(qv.w, kv.w, d3);
            }
            s = ((d0 + d1) + (d2 + d3)) * scale;
        }
        float cmax = s;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, o));
        const float m_new = fmaxf(m, cmax);
        const float corr = (m == -INFINITY) ? 0.f : expf(m - m_new);
        const float p = (j < ctx_len) ? expf(s - m_new) : 0.f;
        float psum = p;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, o);
        l = fmaf(l, corr, psum);
        m = m_new;
#pragma unroll
        for (int t = 0; t < DPL; ++t) acc[t] *= corr;
        const int cnt = min(32, ctx_len - c0);
        for (int jj = 0; jj < cnt; ++jj) {
            const float pj = __shfl_sync(0xffffffffu, p, jj);
            const float* vr = vb + (long long)(c0 + jj) * D;
#pragma unroll
            for (int t = 0; t < DPL; ++t) acc[t] = fmaf(pj, __ldg(vr + lane + 32 * t), acc[t]);
        }
    }
    float* orow = out + job * D;
    const float inv = 1.f / l;
#pragma unroll
    for (int t = 0; t < DPL; ++t) orow[lane + 32 * t] = acc[t] * inv;
}

}  // namespace

cudaError_t launch_attend_f32(const AttendArgs& a, cudaStream_t stream) {
    const long long n_jobs = (long long)a.d.batch * a.n_active * a.d.n_q_heads;
    if (n_jobs == 0) return cudaSuccess;
    const unsigned grid = (unsigned)((n_jobs + kWarpsPerCta - 1) / kWarpsPerCta);
    const float* q = static_cast<const float*>(a.q);
    const float* k = static_cast<const float*>(a.k_cache);
    const float* v = static_cast<const float*>(a.v_cache);
    float* o = static_cast<float*>(a.out);
    if (a.d.head_dim == 64)
        attend_f32_kernel<64><<<grid, kWarpsPerCta * 32, 0, stream>>>(
            q, k, v, o, a.d.batch, a.n_active, a.d.ctx_len, a.d.n_q_heads, a.d.n_kv_heads, a.scale);
    else
        attend_f32_kernel<128><<<grid, kWarpsPerCta * 32, 0, stream>>>(
            q, k, v, o, a.d.batch, a.n_active, a.d.ctx_len, a.d.n_q_heads, a.d.n_kv_heads, a.scale);
    return cudaGetLastError();
}

}  // namespace ec
