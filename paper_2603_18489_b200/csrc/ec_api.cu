// C-ABI entry points of libentropycache: argument validation and dispatch.
// Every check here is host-side; nothing in this file touches device memory.
#include "ec_common.cuh"

#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>

namespace ec {

int sm_count() {
    static std::atomic<int> cached[kMaxDevices] = {};   // per device ordinal: a process may drive unlike GPUs
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        (void)cudaGetLastError();  // no device (host-only use of the size queries): not sticky
        return kDefaultSmCount;
    }
    const bool slot = dev >= 0 && dev < kMaxDevices;
    if (slot) {
        const int v = cached[dev].load(std::memory_order_relaxed);
        if (v > 0) return v;
    }
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
        (void)cudaGetLastError();
        return kDefaultSmCount;
    }
    if (slot) cached[dev].store(n, std::memory_order_relaxed);
    return n;
}

namespace {

// bf16 with head_dim 128 runs on the tcgen05 kernels (the fused skip-step kernel when the packed
// query rows fit two M tiles, the dense kernel otherwise); everything else bf16 on the mma.sync kernel.
// EC_ATTEND_IMPL (environment, read once) = "mma" forces the mma.sync kernel, "dense" the one-tile dense
// tcgen05 kernel with a separate refresh launch, "rows" the skip kernel with query rows on the M axis: for A/B
// measurements only.
int forced_impl() {
    static const int f = [] {
        const char* e = std::getenv("EC_ATTEND_IMPL");
        if (e && std::strcmp(e, "mma") == 0) return 1;
        if (e && std::strcmp(e, "dense") == 0) return 2;
        if (e && std::strcmp(e, "rows") == 0) return 3;
        return 0;
    }();
    return f;
}
bool use_tc(const ec_attn_desc& d) { return d.dtype == EC_BF16 && d.head_dim == 128 && forced_impl() != 1; }
bool use_skip_keys(const ec_attn_desc& d, int n_active, bool fresh) {
    return forced_impl() == 0 && attend_skip_keys_supported(d, n_active, fresh);
}
bool use_skip(const ec_attn_desc& d, int n_active) {
    return (forced_impl() == 0 || forced_impl() == 3) && attend_skip_supported(d, n_active);
}

size_t attend_ws(const ec_attn_desc& d, int n_active) {
    size_t n = attend_workspace_bytes(d, n_active);
    if (d.dtype == EC_BF16 && d.head_dim == 128) {
        const size_t t = attend_tc_workspace_bytes(d, n_active);
        if (t > n) n = t;
        const size_t dn = attend_dense_workspace_bytes(d, n_active);
        if (dn > n) n = dn;
    }
    return n;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// which kernel serves a call of ec_attend: the one place the dispatch order is written down
enum AttendPath { PATH_SKIP_KEYS, PATH_SKIP_ROWS, PATH_DENSE_FROM_NEW, PATH_DENSE, PATH_TC_ONE_TILE, PATH_MMA, PATH_F32 };
AttendPath choose_path(const ec_attn_desc& d, int n_active, bool fresh_kv, bool index_list) {
    if (use_skip_keys(d, n_active, fresh_kv)) return PATH_SKIP_KEYS;
    if (use_skip(d, n_active)) return PATH_SKIP_ROWS;
    if (d.dtype != EC_BF16) return PATH_F32;
    if (use_tc(d) && forced_impl() != 2 && attend_dense_supported(d, n_active))
        return fresh_kv && !index_list ? PATH_DENSE_FROM_NEW : PATH_DENSE;
    return use_tc(d) ? PATH_TC_ONE_TILE : PATH_MMA;
}

ec_status check_desc(const ec_attn_desc* d) {
    if (!d) return EC_ERR_NULL;
    if (d->dtype != EC_F32 && d->dtype != EC_BF16) return EC_ERR_DTYPE;
    if (d->batch < 1 || d->ctx_len < 1 || d->n_q_heads < 1 || d->n_kv_heads < 1) return EC_ERR_SHAPE;
    if (d->n_q_heads % d->n_kv_heads != 0) return EC_ERR_SHAPE;
    if (d->head_dim != 64 && d->head_dim != 128) return EC_ERR_UNSUPPORTED;
    if (!(d->scale >= 0.f) || d->scale > 1.0e30f) return EC_ERR_SHAPE;  // also rejects NaN
    if (d->flags & ~(uint32_t)EC_ATTN_CACHE_SETTLED) return EC_ERR_UNSUPPORTED;   // unknown bits
    return EC_OK;
}

ec_status check_active(const ec_attn_desc* d, const int32_t* active_idx, int32_t n_active) {
    if (n_active < 0) return EC_ERR_SHAPE;
    if (!active_idx && n_active != 0 && n_active != d->ctx_len) return EC_ERR_SHAPE;
    if (active_idx && n_active > d->ctx_len) return EC_ERR_SHAPE;  // unique positions cannot exceed L
    if (active_idx && (reinterpret_cast<uintptr_t>(active_idx) & 3u)) return EC_ERR_ALIGN;
    return EC_OK;
}

}  // namespace
}  // namespace ec

namespace ec {

// every host-side check of the gate entry points; EC_OK means a launch with these arguments is well-formed
// (n_rows == 0 is EC_OK too: the callers return before launching)
ec_status gate_validate(const void* logits, int32_t dtype, int32_t n_rows, int32_t vocab, int64_t row_stride_elems,
                        int32_t rows_per_seq, const uint8_t* decoded_flags, uint8_t* masked, float conf_threshold,
                        uint8_t* decoded_out, int32_t* tokens, float tau, int32_t* argmax_out, float* conf_out,
                        float* entropy_out, float* max_entropy_out, int32_t* decision_out, float* entropy_sum_out,
                        float* max_conf_out, const void* workspace, size_t workspace_bytes) {
    if (dtype != EC_F32 && dtype != EC_BF16) return EC_ERR_DTYPE;
    if (n_rows < 0 || vocab < 1 || rows_per_seq < 1 || row_stride_elems < vocab) return EC_ERR_SHAPE;
    if (n_rows % rows_per_seq != 0) return EC_ERR_SHAPE;
    if (n_rows > 65535) return EC_ERR_UNSUPPORTED;          // grid.y limit
    if (vocab > 96 * 8192) return EC_ERR_UNSUPPORTED;       // split table of the workspace
    if (tau != tau) return EC_ERR_SHAPE;
    const bool decode = masked != nullptr || decoded_out != nullptr || tokens != nullptr;
    if (decode && (conf_threshold != conf_threshold)) return EC_ERR_SHAPE;
    const bool one_cta_finish = decode || entropy_sum_out != nullptr || max_conf_out != nullptr;
    if (one_cta_finish && rows_per_seq > kGateDecodeMaxRowsPerSeq) return EC_ERR_UNSUPPORTED;
    if (n_rows == 0) return EC_OK;
    if (!logits || !max_entropy_out || !decision_out) return EC_ERR_NULL;
    if (decode ? (!masked || !decoded_out || !tokens) : !decoded_flags) return EC_ERR_NULL;
    const size_t esize = dtype == EC_BF16 ? 2 : 4;
    if ((reinterpret_cast<uintptr_t>(logits) & 15u) || ((size_t)row_stride_elems * esize) % 16 != 0) return EC_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(argmax_out) | reinterpret_cast<uintptr_t>(conf_out) |
         reinterpret_cast<uintptr_t>(entropy_out) | reinterpret_cast<uintptr_t>(max_entropy_out) |
         reinterpret_cast<uintptr_t>(decision_out) | reinterpret_cast<uintptr_t>(tokens) |
         reinterpret_cast<uintptr_t>(entropy_sum_out) | reinterpret_cast<uintptr_t>(max_conf_out)) & 3u)
        return EC_ERR_ALIGN;
    const size_t need = gate_workspace_bytes(n_rows, vocab);
    if (!workspace || workspace_bytes < need) return EC_ERR_WORKSPACE;
    return EC_OK;
}

}  // namespace ec

using namespace ec;

extern "C" {

ec_status ec_kv_refresh(const ec_attn_desc* desc, void* k_cache, void* v_cache, const void* k_new,
                        const void* v_new, const int32_t* active_idx, int32_t n_active, void* stream) {
    ec_status st = check_desc(desc);
    if (st != EC_OK) return st;
    st = check_active(desc, active_idx, n_active);
    if (st != EC_OK) return st;
    if (n_active == 0) return EC_OK;
    if (!k_cache || !v_cache || !k_new || !v_new) return EC_ERR_NULL;
    if (!aligned16(k_cache) || !aligned16(v_cache) || !aligned16(k_new) || !aligned16(v_new)) return EC_ERR_ALIGN;
    const cudaError_t e =
        launch_refresh(*desc, k_cache, v_cache, k_new, v_new, active_idx, n_active, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? EC_OK : EC_ERR_CUDA;
}

ec_status ec_select_recent(int32_t* history, int32_t ctx_len, int32_t batch, ec_step_state* state,
                           const uint8_t* decoded_flags, const int32_t* window_start, int32_t block,
                           const int32_t* decision, int32_t k, int32_t* active_idx, int32_t n_cap, void* stream) {
    if (!history || !state || !decoded_flags || !window_start || !decision || !active_idx) return EC_ERR_NULL;
    if (ctx_len < 1 || batch < 1 || block < 1 || block > ctx_len || k < 0 || k > ctx_len || n_cap < block)
        return EC_ERR_SHAPE;
    if (ctx_len > select_recent_max_ctx() || batch > 65535) return EC_ERR_UNSUPPORTED;
    const cudaError_t e = launch_select_recent(history, ctx_len, batch, state, decoded_flags, window_start, block,
                                               decision, k, active_idx, n_cap, nullptr, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? EC_OK : EC_ERR_CUDA;
}

ec_status ec_select_recent_sliding(int32_t* history, int32_t ctx_len, int32_t batch, ec_step_state* state,
                                   uint8_t* masked, const uint8_t* decoded_flags, int32_t window,
                                   const int32_t* decision, int32_t k, int32_t* active_idx, int32_t n_cap, void* stream) {
    if (!history || !state || !masked || !decoded_flags || !decision || !active_idx) return EC_ERR_NULL;
    if (ctx_len < 1 || batch < 1 || window < 1 || window > ctx_len || k < 0 || k > ctx_len || n_cap < window)
        return EC_ERR_SHAPE;
    if (ctx_len > select_recent_max_ctx() || batch > 65535) return EC_ERR_UNSUPPORTED;
    const cudaError_t e = launch_select_recent(history, ctx_len, batch, state, decoded_flags, nullptr, window, decision, k,
                                               active_idx, n_cap, masked, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? EC_OK : EC_ERR_CUDA;
}

size_t ec_attend_workspace_bytes(const ec_attn_desc* desc, int32_t n_active) {
    if (check_desc(desc) != EC_OK || n_active < 0 || n_active > desc->ctx_len) return 0;
    return attend_ws(*desc, n_active);
}

ec_status ec_attend(const ec_attn_desc* desc, const void* q, const void* k_new, const void* v_new, void* k_cache,
                    void* v_cache, const int32_t* active_idx, int32_t n_active, void* out, void* workspace,
                    size_t workspace_bytes, int32_t* dev_status, void* stream) {
    ec_status st = check_desc(desc);
    if (st != EC_OK) return st;
    st = check_active(desc, active_idx, n_active);
    if (st != EC_OK) return st;
    if (n_active == 0) return EC_OK;
    if (!q || !k_cache || !v_cache || !out) return EC_ERR_NULL;
    if ((k_new == nullptr) != (v_new == nullptr)) return EC_ERR_NULL;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(out) || !aligned16(k_new) ||
        !aligned16(v_new))
        return EC_ERR_ALIGN;
    if (dev_status && (reinterpret_cast<uintptr_t>(dev_status) & 3u)) return EC_ERR_ALIGN;
    const size_t need = attend_ws(*desc, n_active);
    if (!workspace || workspace_bytes < need) return EC_ERR_WORKSPACE;
    if (!aligned16(workspace)) return EC_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const AttendPath path = choose_path(*desc, n_active, k_new != nullptr, active_idx != nullptr);
    const bool fused_keys = path == PATH_SKIP_KEYS;
    const bool fused = fused_keys || path == PATH_SKIP_ROWS;
    // recompute step on the dense path: every cache row is overwritten by the fresh row of the same position, so
    // attention reads K/V straight from k_new / v_new and a spare warp of the same launch copies them into the cache
    const bool from_new = path == PATH_DENSE_FROM_NEW;
    if (k_new && !fused && !from_new) {
        if (launch_refresh(*desc, k_cache, v_cache, k_new, v_new, active_idx, n_active, s) != cudaSuccess)
            return EC_ERR_CUDA;
    }
    AttendArgs a;
    a.d = *desc;
    a.q = q;
    a.k_cache = k_cache;
    a.v_cache = v_cache;
    a.n_active = n_active;
    a.out = out;
    a.workspace = workspace;
    a.workspace_bytes = workspace_bytes;
    a.dev_status = dev_status;
    a.scale = desc->scale > 0.f ? desc->scale : 1.0f / sqrtf((float)desc->head_dim);
    if (from_new) {
        a.k_cache = k_new;
        a.v_cache = v_new;
        a.kv_token_major = true;
        a.refresh_k_dst = k_cache;
        a.refresh_v_dst = v_cache;
    }
    cudaError_t e;
    switch (path) {
        case PATH_SKIP_KEYS: e = launch_attend_skip_keys(a, k_new, v_new, active_idx, s); break;
        case PATH_SKIP_ROWS: e = launch_attend_skip(a, k_new, v_new, active_idx, s); break;
        case PATH_F32: e = launch_attend_f32(a, s); break;
        case PATH_DENSE_FROM_NEW:
        case PATH_DENSE: e = launch_attend_dense(a, s); break;
        case PATH_TC_ONE_TILE: e = launch_attend_bf16_tc(a, s); break;
        default: e = launch_attend_bf16(a, s); break;
    }
    return e == cudaSuccess ? EC_OK : EC_ERR_CUDA;
}

const char* ec_attend_kernel_name(const ec_attn_desc* desc, int32_t n_active, int32_t with_fresh_kv,
                                  int32_t with_index_list) {
    static thread_local char buf[192];
    if (check_desc(desc) != EC_OK || n_active < 1 || n_active > desc->ctx_len ||
        (!with_index_list && n_active != desc->ctx_len))
        return "";
    const bool fresh = with_fresh_kv != 0;
    switch (choose_path(*desc, n_active, fresh, with_index_list != 0)) {
        case PATH_SKIP_KEYS: attend_skip_keys_describe(*desc, n_active, fresh, buf, sizeof buf); return buf;
        case PATH_SKIP_ROWS: attend_skip_describe(*desc, n_active, buf, sizeof buf); return buf;
        case PATH_F32: return fresh ? "refresh_kernel + attend_f32_kernel" : "attend_f32_kernel";
        case PATH_DENSE_FROM_NEW: attend_dense_describe(*desc, n_active, buf, sizeof buf); return buf;
        case PATH_DENSE: {
            char inner[160];
            attend_dense_describe(*desc, n_active, inner, sizeof inner);
            snprintf(buf, sizeof buf, "%s%s", fresh ? "refresh_kernel + " : "", inner);
            return buf;
        }
        case PATH_TC_ONE_TILE: return fresh ? "refresh_kernel + attend_tc_kernel" : "attend_tc_kernel";
        default: return fresh ? "refresh_kernel + attend_mma_kernel" : "attend_mma_kernel";
    }
}

size_t ec_entropy_gate_workspace_bytes(int32_t n_rows, int32_t vocab) { return gate_workspace_bytes(n_rows, vocab); }

namespace {

// shared by ec_entropy_gate, ec_entropy_gate_metrics and ec_entropy_gate_decode: `masked` selects the decode mode
ec_status gate_call(const void* logits, int32_t dtype, int32_t n_rows, int32_t vocab, int64_t row_stride_elems,
                    int32_t rows_per_seq, const uint8_t* decoded_flags, uint8_t* masked, float conf_threshold,
                    uint8_t* decoded_out, int32_t* tokens, float tau, int32_t* argmax_out, float* conf_out,
                    float* entropy_out, float* max_entropy_out, int32_t* decision_out, float* entropy_sum_out,
                    float* max_conf_out, void* workspace, size_t workspace_bytes, void* stream) {
    const ec_status st = gate_validate(logits, dtype, n_rows, vocab, row_stride_elems, rows_per_seq, decoded_flags, masked,
                                       conf_threshold, decoded_out, tokens, tau, argmax_out, conf_out, entropy_out,
                                       max_entropy_out, decision_out, entropy_sum_out, max_conf_out, workspace,
                                       workspace_bytes);
    if (st != EC_OK || n_rows == 0) return st;
    GateArgs a;
    a.logits = logits;
    a.dtype = dtype;
    a.n_rows = n_rows;
    a.vocab = vocab;
    a.row_stride = row_stride_elems;
    a.rows_per_seq = rows_per_seq;
    a.flags = decoded_flags;
    a.tau = tau;
    a.argmax_out = argmax_out;
    a.conf_out = conf_out;
    a.entropy_out = entropy_out;
    a.max_entropy_out = max_entropy_out;
    a.decision_out = decision_out;
    a.workspace = workspace;
    a.masked = masked;
    a.conf_threshold = conf_threshold;
    a.decoded_out = decoded_out;
    a.tokens = tokens;
    a.entropy_sum_out = entropy_sum_out;
    a.max_conf_out = max_conf_out;
    const cudaError_t e = launch_gate(a, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? EC_OK : EC_ERR_CUDA;
}

}  // namespace

ec_status ec_entropy_gate(const void* logits, int32_t dtype, int32_t n_rows, int32_t vocab, int64_t row_stride_elems,
                          int32_t rows_per_seq, const uint8_t* decoded_flags, float tau, int32_t* argmax_out,
                          float* conf_out, float* entropy_out, float* max_entropy_out, int32_t* decision_out,
                          void* workspace, size_t workspace_bytes, void* stream) {
    return gate_call(logits, dtype, n_rows, vocab, row_stride_elems, rows_per_seq, decoded_flags, nullptr, 0.f, nullptr,
                     nullptr, tau, argmax_out, conf_out, entropy_out, max_entropy_out, decision_out, nullptr, nullptr,
                     workspace, workspace_bytes, stream);
}

ec_status ec_entropy_gate_metrics(const void* logits, int32_t dtype, int32_t n_rows, int32_t vocab,
                                  int64_t row_stride_elems, int32_t rows_per_seq, const uint8_t* decoded_flags, float tau,
                                  int32_t* argmax_out, float* conf_out, float* entropy_out, float* max_entropy_out,
                                  int32_t* decision_out, float* entropy_sum_out, float* max_conf_out, void* workspace,
                                  size_t workspace_bytes, void* stream) {
    return gate_call(logits, dtype, n_rows, vocab, row_stride_elems, rows_per_seq, decoded_flags, nullptr, 0.f, nullptr,
                     nullptr, tau, argmax_out, conf_out, entropy_out, max_entropy_out, decision_out, entropy_sum_out,
                     max_conf_out, workspace, workspace_bytes, stream);
}

ec_status ec_entropy_gate_decode(const void* logits, int32_t dtype, int32_t n_rows, int32_t vocab,
                                 int64_t row_stride_elems, int32_t rows_per_seq, uint8_t* masked, float conf_threshold,
                                 float tau, uint8_t* decoded_flags_out, int32_t* tokens, int32_t* argmax_out,
                                 float* conf_out, float* entropy_out, float* max_entropy_out, int32_t* decision_out,
                                 void* workspace, size_t workspace_bytes, void* stream) {
    if (!masked || !decoded_flags_out || !tokens) return n_rows == 0 ? EC_OK : EC_ERR_NULL;
    return gate_call(logits, dtype, n_rows, vocab, row_stride_elems, rows_per_seq, nullptr, masked, conf_threshold,
                     decoded_flags_out, tokens, tau, argmax_out, conf_out, entropy_out, max_entropy_out, decision_out,
                     nullptr, nullptr, workspace, workspace_bytes, stream);
}

ec_status ec_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
    if (workspace_bytes == 0) return EC_OK;
    if (!workspace) return EC_ERR_NULL;
    return cudaMemsetAsync(workspace, 0, workspace_bytes, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? EC_OK
               : EC_ERR_CUDA;
}

const char* ec_status_string(int32_t status) {
    switch (status) {
        case EC_OK: return "EC_OK";
        case EC_ERR_NULL: return "EC_ERR_NULL: a required pointer is NULL";
        case EC_ERR_SHAPE: return "EC_ERR_SHAPE: a size is non-positive, inconsistent or out of range";
        case EC_ERR_DTYPE: return "EC_ERR_DTYPE: unknown element type";
        case EC_ERR_ALIGN: return "EC_ERR_ALIGN: a pointer or row is not 16-byte aligned";
        case EC_ERR_WORKSPACE: return "EC_ERR_WORKSPACE: workspace missing or too small";
        case EC_ERR_UNSUPPORTED: return "EC_ERR_UNSUPPORTED: outside what the kernels implement";
        case EC_ERR_CUDA: return "EC_ERR_CUDA: a CUDA runtime call or launch failed";
        case EC_ERR_TIMEOUT: return "EC_ERR_TIMEOUT: a bounded device-side wait gave up";
        default: return "unknown ec_status";
    }
}

int32_t ec_version(void) { return 100; }

}  // extern "C"
