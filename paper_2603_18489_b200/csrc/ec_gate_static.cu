// ec_entropy_gate_static: the entropy gate for callers that cannot hand the
// library a workspace because they cannot allocate device memory at all.
//
// Who that is: code running where a cudaMalloc is either forbidden or harmful --
// a serving loop whose HBM was carved up in advance (every byte already belongs
// to a KV cache, so a late allocation can fail), a plug-in that lives inside
// another runtime's memory pool and must not touch the allocator, or a
// latency-critical step where cudaMalloc's implicit device synchronisation would
// stall every stream.  Such a caller still owns its inputs and outputs; what it
// lacks is a place for the gate's scratch (row/sequence tickets, per-split
// partial sums, per-row entropies).
//
// Here that scratch lives in a file-scope __device__ array of fixed size, part of
// the library image: every GPU that loads the library holds these bytes until the
// process exits.  Consequences the caller must know:
//   - sizes are capped (EC_GATE_STATIC_MAX_ROWS logits rows); larger requests are
//     refused with EC_ERR_UNSUPPORTED;
//   - all calls on one GPU share the one array, so two calls that may overlap on
//     the GPU (different streams, no ordering) race; serialise them;
//   - the array keeps whatever the previous call left, so each call first clears
//     the ticket words it needs to start from zero (an asynchronous memset on the
//     caller's stream; no allocation);
//   - the first call on each device looks up the array's device address
//     (cudaGetSymbolAddress).  Make that first call outside any stream capture.
// The kernel and its arithmetic are those of ec_entropy_gate; only the scratch differs.
#include "ec_common.cuh"

#include <mutex>

namespace {

constexpr int kStaticMaxRows = EC_GATE_STATIC_MAX_ROWS;
// tickets (2 x int32) + entropy scratch (f32) per row, then 96 splits x 16-byte partials per row
constexpr size_t kStaticBytes = (size_t)kStaticMaxRows * 12 + (size_t)kStaticMaxRows * 96 * 16;

static __device__ __align__(256) unsigned char g_gate_scratch[kStaticBytes];

std::mutex g_mu;
void* g_scratch_addr[ec::kMaxDevices] = {};  // device address of g_gate_scratch, per device ordinal

// In host code `g_gate_scratch` is only a handle for the runtime, not a device address:
// the address a kernel can use comes from cudaGetSymbolAddress, asked once per device with
// that device current.
ec_status scratch_for_current_device(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= ec::kMaxDevices) return EC_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_gate_scratch) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return EC_ERR_CUDA;
        }
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return EC_OK;
}

}  // namespace

extern "C" ec_status ec_entropy_gate_static(const void* logits, int32_t dtype, int32_t n_rows, int32_t vocab,
                                            int64_t row_stride_elems, int32_t rows_per_seq,
                                            const uint8_t* decoded_flags, float tau, int32_t* argmax_out,
                                            float* conf_out, float* entropy_out, float* max_entropy_out,
                                            int32_t* decision_out, void* stream) {
    if (n_rows > kStaticMaxRows) return EC_ERR_UNSUPPORTED;  // beyond the built-in scratch
    if (n_rows > 0 && vocab > 0 && ec::gate_workspace_bytes(n_rows, vocab) > kStaticBytes) return EC_ERR_UNSUPPORTED;
    // every argument check comes BEFORE anything is enqueued or looked up: a rejected call must leave the shared
    // scratch alone (an earlier call's kernel may still be using it on another stream).  The checks only ask whether
    // a workspace of kStaticBytes exists, not where it is, so they run against a placeholder address.
    char placeholder;
    const ec_status ok = ec::gate_validate(logits, dtype, n_rows, vocab, row_stride_elems, rows_per_seq, decoded_flags,
                                           nullptr, 0.f, nullptr, nullptr, tau, argmax_out, conf_out, entropy_out,
                                           max_entropy_out, decision_out, nullptr, nullptr, &placeholder, kStaticBytes);
    if (ok != EC_OK || n_rows == 0) return ok;
    void* scratch = nullptr;
    const ec_status st = scratch_for_current_device(&scratch);
    if (st != EC_OK) return st;
    // tickets must start at zero whatever an earlier (possibly abandoned) call left behind
    if (cudaMemsetAsync(scratch, 0, ec::gate_ticket_bytes(n_rows), static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return EC_ERR_CUDA;
    return ec_entropy_gate(logits, dtype, n_rows, vocab, row_stride_elems, rows_per_seq, decoded_flags, tau,
                           argmax_out, conf_out, entropy_out, max_entropy_out, decision_out, scratch, kStaticBytes,
                           stream);
}
