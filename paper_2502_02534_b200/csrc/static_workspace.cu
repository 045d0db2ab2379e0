// psa_decode_static: the decode step for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc (or any allocating routine) around a
// decode step: code running inside a serving engine that has already handed the whole
// device to its own KV-cache pool, plugins loaded into a process whose allocator is
// owned by someone else, or latency-critical loops where an allocation would
// synchronise the device.  For them the scratch memory the step needs -- the planner's
// work lists and the partial results that the prefix and suffix stages hand to the merge
// stage -- lives in a fixed array inside the library image instead of a caller buffer.
//
// The array is a file-scope __device__ object: every GPU that loads the library carries
// its PSA_STATIC_WORKSPACE_BYTES until the process exits.  In host code the array's
// name is only a handle for the runtime, not a device address, so the address each
// device uses is looked up once per device with cudaGetSymbolAddress (with that device
// current) and cached; the kernels receive that pointer.
#include <cuda_runtime.h>

#include <mutex>
#include <string>

#include "psa_internal.h"

namespace {

constexpr size_t kStaticBytes = PSA_STATIC_WORKSPACE_BYTES;
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_static_workspace[kStaticBytes];

std::mutex g_lookup_mutex;
void *g_device_address[kMaxDevices] = {};

// Device address of the array on the current device; looked up on the first call per device.
psa_status_t static_workspace_address(void **out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return psa::set_last_error(PSA_ERR_CUDA, std::string("cudaGetDevice: ") + cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices) return psa::set_last_error(PSA_ERR_UNSUPPORTED, "device ordinal beyond the static workspace table");
    std::lock_guard<std::mutex> lock(g_lookup_mutex);
    if (!g_device_address[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_workspace);
        if (e != cudaSuccess || !p)
            return psa::set_last_error(PSA_ERR_CUDA, std::string("cudaGetSymbolAddress(static workspace): ") + cudaGetErrorString(e));
        g_device_address[dev] = p;
    }
    *out = g_device_address[dev];
    return PSA_OK;
}

}  // namespace

extern "C" psa_status_t psa_decode_static(const psa_plan_t *plan, const void *q, const void *prefix_k, const void *prefix_v,
                                          const int64_t prefix_strides[2], const void *suffix_k_pool,
                                          const void *suffix_v_pool, const int64_t pool_strides[3],
                                          const int32_t *page_indptr, const int32_t *page_indices,
                                          const int32_t *suffix_lens, void *out, float *lse, void *cuda_stream)
{
    if (!plan) return psa::set_last_error(PSA_ERR_INVALID_ARG, "null plan");
    if (plan->ws.total > kStaticBytes)
        return psa::set_last_error(PSA_ERR_WORKSPACE,
                                   "this plan needs " + std::to_string(plan->ws.total) + " bytes of workspace; psa_decode_static holds " +
                                       std::to_string(kStaticBytes) + " (PSA_STATIC_WORKSPACE_BYTES): use psa_decode with a caller workspace");
    void *ws = nullptr;
    psa_status_t st = static_workspace_address(&ws);
    if (st != PSA_OK) return st;
    // The array still holds the previous call's lists, status word and partial results (maybe another
    // plan's).  The upload rewrites the lists and zeroes the status word; partial results need no
    // clearing because every row the merge stage reads is written by this call's prefix / suffix stages.
    cudaError_t e = cudaMemcpyAsync(ws, plan->upload.data(), plan->upload.size(), cudaMemcpyHostToDevice,
                                    static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return psa::set_last_error(PSA_ERR_CUDA, std::string("uploading the work lists: ") + cudaGetErrorString(e));
    return psa_decode(plan, q, prefix_k, prefix_v, prefix_strides, suffix_k_pool, suffix_v_pool, pool_strides, page_indptr,
                      page_indices, suffix_lens, out, lse, ws, kStaticBytes, cuda_stream);
}
