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
//
// When the memory is taken: a __device__ array belongs to this file's CUDA module and comes
// into being when the driver loads that module on a device.  With the runtime's default lazy
// module loading that is the symbol lookup of the FIRST call on the device (so that one call
// can still run out of memory or take a while); with CUDA_MODULE_LOADING=EAGER it is the
// moment the library is loaded.  Every later call allocates nothing at all.  Callers should
// therefore make one warm-up call per device while they initialise, before their pool takes
// the rest of the memory.
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

// Device-side status of the steps run through psa_decode_static.  psa_check_status needs the workspace's
// address, which for this path is private to the library, so the static array gets the same service here:
// synchronise the stream, return the status word, clear the status area.  Allocates nothing.
extern "C" psa_status_t psa_static_check_status(void *cuda_stream)
{
    void *ws = nullptr;
    psa_status_t st = static_workspace_address(&ws);
    if (st != PSA_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int32_t word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, ws, sizeof word, cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return psa::set_last_error(PSA_ERR_CUDA, std::string("reading the static status word: ") + cudaGetErrorString(e));
    if (word != 0) {
        // the stream is idle (synchronised above): the prefix counters in the same area restart from zero together
        e = cudaMemsetAsync(ws, 0, sizeof(int32_t) * psa::kStatusWords, stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
        if (e != cudaSuccess) return psa::set_last_error(PSA_ERR_CUDA, std::string("clearing the static status word: ") + cudaGetErrorString(e));
        return psa::set_last_error(psa_status_t(word), "device-side status word of the static workspace was set");
    }
    return PSA_OK;
}

// The bounded-wait self-test (see psa_selftest_bounded_wait) reporting into the static array's status word.
extern "C" psa_status_t psa_static_selftest_bounded_wait(uint64_t limit_ns, void *cuda_stream)
{
    if (limit_ns == 0 || limit_ns > 1000000000ull) return psa::set_last_error(PSA_ERR_INVALID_ARG, "limit_ns must be in (0, 1e9]");
    void *ws = nullptr;
    psa_status_t st = static_workspace_address(&ws);
    if (st != PSA_OK) return st;
    const int rc = psa::launch_bounded_wait_selftest(static_cast<int32_t *>(ws), limit_ns, cuda_stream);
    if (rc != 0) return psa::set_last_error(PSA_ERR_CUDA, std::string("self-test launch: ") + cudaGetErrorString(cudaError_t(rc)));
    return PSA_OK;
}
