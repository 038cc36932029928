// Shared declarations of libentropycache's CUDA translation units (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include <atomic>

#include "entropycache.h"

namespace ec {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Number of SMs the launch heuristics assume when the device cannot be queried
// (B200: 148).
constexpr int kDefaultSmCount = 148;

constexpr int kMaxDevices = 64;   // device ordinals with a slot in the per-device caches below

int sm_count();  // cudaDevAttrMultiProcessorCount of the CURRENT device, cached per device ordinal

// "this per-device set-up has been done" flags (cudaFuncSetAttribute is per device): one bit per ordinal, safe
// to query and set from several host threads (a repeated set-up is harmless, a torn flag is not)
struct PerDeviceOnce {
    std::atomic<unsigned long long> mask{0};
    bool done(int dev) const { return dev >= 0 && dev < kMaxDevices && ((mask.load(std::memory_order_acquire) >> dev) & 1ull); }
    void set(int dev) {
        if (dev >= 0 && dev < kMaxDevices) mask.fetch_or(1ull << dev, std::memory_order_release);
    }
};

// raises a kernel's dynamic shared-memory limit once per device
template <typename Kernel>
cudaError_t ensure_dynamic_smem(PerDeviceOnce& once, Kernel kernel, int bytes) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorInvalidDevice;
    if (once.done(dev)) return cudaSuccess;
    const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) once.set(dev);
    return e;
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float fast_log2(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// ---- internal launchers (host), one per translation unit ------------------
struct GateArgs {
    const void* logits;
    int dtype;
    int n_rows;
    int vocab;
    long long row_stride;
    int rows_per_seq;
    const uint8_t* flags;
    float tau;
    int* argmax_out;
    float* conf_out;
    float* entropy_out;
    float* max_entropy_out;
    int* decision_out;
    void* workspace;
    // decode mode (ec_entropy_gate_decode): the decoded set is formed inside the launch from the confidences
    uint8_t* masked = nullptr;        // in/out, nullptr: the decoded set is `flags`
    float conf_threshold = 0.f;
    uint8_t* decoded_out = nullptr;
    int* tokens = nullptr;
    // the other two candidate metrics of Section 5.3 over the decoded rows (optional, per sequence)
    float* entropy_sum_out = nullptr;
    float* max_conf_out = nullptr;
};
constexpr int kGateDecodeMaxRowsPerSeq = 64;
size_t gate_workspace_bytes(int n_rows, int vocab);
size_t gate_ticket_bytes(int n_rows);   // leading bytes of a gate workspace that must be zero when a call starts
// all host-side argument checks of the gate entry points (EC_OK: a launch with these arguments is well-formed)
ec_status gate_validate(const void* logits, int32_t dtype, int32_t n_rows, int32_t vocab, int64_t row_stride_elems,
                        int32_t rows_per_seq, const uint8_t* decoded_flags, uint8_t* masked, float conf_threshold,
                        uint8_t* decoded_out, int32_t* tokens, float tau, int32_t* argmax_out, float* conf_out,
                        float* entropy_out, float* max_entropy_out, int32_t* decision_out, float* entropy_sum_out,
                        float* max_conf_out, const void* workspace, size_t workspace_bytes);
cudaError_t launch_gate(const GateArgs& a, cudaStream_t stream);
int select_recent_max_ctx();
cudaError_t launch_select_recent(int32_t* history, int ctx_len, int batch, ec_step_state* state, const uint8_t* decoded,
                                 const int32_t* window_start, int block, const int32_t* decision, int k,
                                 int32_t* active_idx, int n_cap, uint8_t* masked, cudaStream_t stream);

cudaError_t launch_refresh(const ec_attn_desc& d, void* k_cache, void* v_cache, const void* k_new,
                           const void* v_new, const int32_t* active_idx, int n_active,
                           cudaStream_t stream);

struct AttendArgs {
    ec_attn_desc d;
    const void* q;
    const void* k_cache;
    const void* v_cache;
    int n_active;
    void* out;
    void* workspace;
    size_t workspace_bytes;
    int32_t* dev_status;
    float scale;  // resolved (never 0)
    // dense path only: k_cache / v_cache point at token-major tensors [batch, ctx_len, n_kv_heads, head_dim]
    // (the fresh K/V of a recompute step) instead of the cache layout
    bool kv_token_major = false;
    // with kv_token_major: the caches those tensors are copied into by the same launch (nullptr: no copy)
    void* refresh_k_dst = nullptr;
    void* refresh_v_dst = nullptr;
};
size_t attend_workspace_bytes(const ec_attn_desc& d, int n_active);
cudaError_t launch_attend_f32(const AttendArgs& a, cudaStream_t stream);
cudaError_t launch_attend_bf16(const AttendArgs& a, cudaStream_t stream);      // mma.sync path (any head_dim)
// fused skip-step path (bf16, head_dim 128, n_active * H_q/H_kv <= 256): refresh + attention + merge in one launch
bool attend_skip_supported(const ec_attn_desc& d, int n_active);
// host-only descriptions of the launch the plan functions choose ("kernel<instantiation> grid=... cluster=..."),
// written into buf (always terminated)
void attend_skip_describe(const ec_attn_desc& d, int n_active, char* buf, size_t len);
void attend_skip_keys_describe(const ec_attn_desc& d, int n_active, bool fresh, char* buf, size_t len);
void attend_dense_describe(const ec_attn_desc& d, int n_active, char* buf, size_t len);
cudaError_t launch_attend_skip(const AttendArgs& a, const void* k_new, const void* v_new, const int32_t* active_idx,
                               cudaStream_t stream);
// skip-step path with the keys on the M axis (bf16, head_dim 128, n_active * H_q/H_kv <= 64)
bool attend_skip_keys_supported(const ec_attn_desc& d, int n_active, bool fresh);   // fresh: k_new / v_new are given
cudaError_t launch_attend_skip_keys(const AttendArgs& a, const void* k_new, const void* v_new, const int32_t* active_idx,
                                    cudaStream_t stream);
// two-row-tile dense path (bf16, head_dim 128): used when its (row-tile pair, kv head) units fill the GPU
bool attend_dense_supported(const ec_attn_desc& d, int n_active);
size_t attend_dense_workspace_bytes(const ec_attn_desc& d, int n_active);   // partials of the cut last wave (0: none)
cudaError_t launch_attend_dense(const AttendArgs& a, cudaStream_t stream);
size_t attend_tc_workspace_bytes(const ec_attn_desc& d, int n_active);
cudaError_t launch_attend_bf16_tc(const AttendArgs& a, cudaStream_t stream);   // tcgen05 path (head_dim 128)

}  // namespace ec
