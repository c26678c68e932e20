// Forward pass for callers that may not allocate device memory.
//
// Some hosts of this library cannot hand it a workspace: a plug-in running under a framework
// that owns every byte of device memory and forbids cudaMalloc, a latency-critical serving loop
// whose memory pool is frozen after start-up (cudaMalloc also synchronises the whole device), or
// a component that is only given input and output tensors.  For them the scratch of the forward
// pass (status block, work items, keys regrouped by head) lives in a fixed array that is part of
// the library image: every GPU that loads the library holds kStaticScratchBytes for the lifetime
// of the process, and problems that need more are refused.
#include "common.cuh"

namespace {

constexpr size_t kStaticScratchBytes = KMIP_STATIC_SCRATCH_BYTES;

// The array itself.  In host code this name is only a handle for the runtime's symbol table, not
// a device address - it must never be passed to a kernel or to pointer arithmetic directly.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {nullptr};  // device address of the array, per device ordinal

// Device address of this device's copy of the array; resolved once per device with that device
// current.  Returns nullptr (and leaves the slot empty) if the runtime call fails.
void* scratch_address_for_current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    if (g_scratch_addr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return nullptr;
        g_scratch_addr[dev] = p;
    }
    return g_scratch_addr[dev];
}

}  // namespace

extern "C" int kmip_attn_forward_static_scratch(const void* Q, const void* K, const void* V,
                                                const int32_t* graph_offsets, int32_t G, int64_t N, int32_t H,
                                                int32_t d, int32_t k, int mode, void* out, int32_t* topk_idx,
                                                float* topk_score, int32_t* device_status, void* stream) {
    // size check first: host arithmetic only, and the answer does not depend on the device
    size_t need = 0;
    const int rc = kmip_attn_workspace_bytes(N, graph_offsets ? G : 1, H, d, k, mode, KMIP_PASS_FORWARD, &need);
    if (rc != KMIP_OK) return rc;
    if (need > kStaticScratchBytes) return KMIP_ERR_TOO_LARGE;
    if (N == 0) {
        // nothing to enqueue, but a caller that polls device_status must not read the previous call's word
        if (device_status != nullptr &&
            cudaMemsetAsync(device_status, 0, sizeof(int32_t), static_cast<cudaStream_t>(stream)) != cudaSuccess)
            return KMIP_ERR_CUDA;
        return KMIP_OK;
    }
    void* scratch = scratch_address_for_current_device();
    if (scratch == nullptr) return KMIP_ERR_CUDA;
    // The regular entry point clears the status block and rewrites the work items and the regrouped
    // keys in full, so nothing of the previous call's contents survives where it matters.
    const int st = kmip_attn_forward(Q, K, V, graph_offsets, G, N, H, d, k, mode, out, topk_idx, topk_score,
                                     scratch, kStaticScratchBytes, stream);
    if (st != KMIP_OK) return st;
    if (device_status != nullptr &&
        cudaMemcpyAsync(device_status, scratch, sizeof(int32_t), cudaMemcpyDeviceToDevice,
                        static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return KMIP_ERR_CUDA;
    return KMIP_OK;
}
