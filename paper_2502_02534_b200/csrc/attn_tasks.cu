// The paper's three "attn" tasks as selectable kernels: three algebraically equal ways to fold a stream of
// (score, value) pairs into softmax(S) V (appendix "Benchmark details", attn group):
//   task 0  "MaxSum":      running maximum m, running sum l, output normalised at EVERY step
//   task 1  "ExpMaxDiff" -> "DivSum": stage one emits e = exp(s - m_new) and the decay d = exp(m_old - m_new) of what
//                          was accumulated so far, stage two keeps (l, o) with o normalised at every step
//   task 2  "ExpMaxDiff" -> two weighted sums (r, acc) divided once at the end: the deferred division every fast
//                          kernel of this library uses
// They exist to tie the library to the paper's own operator forms and to show on the GPU that the forms agree; they are
// plain CUDA-core code (one warp per query row, keys taken one at a time, fp32), not a fast path.
// State starts at (m, l, o) = (-inf, 0, 0) as in the paper; an empty key stream returns exactly that.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <string>

#include "psa_internal.h"

namespace psa {
namespace {

constexpr int kMaxPerLane = 8;   // head_dim <= 256

template <int kTask>
__global__ void attn_task_kernel(const __nv_bfloat16 *__restrict__ q, const __nv_bfloat16 *__restrict__ k,
                                 const __nv_bfloat16 *__restrict__ v, int num_rows, int num_keys, int head_dim, float sm_scale,
                                 float *__restrict__ out, float *__restrict__ m_out, float *__restrict__ l_out)
{
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (row >= num_rows) return;
    const int per = head_dim / 32;   // elements of a row this lane owns: [lane * per, lane * per + per)
    float qv[kMaxPerLane], o[kMaxPerLane];
#pragma unroll
    for (int i = 0; i < kMaxPerLane; ++i) {
        qv[i] = i < per ? __bfloat162float(q[size_t(row) * head_dim + lane * per + i]) : 0.f;
        o[i] = 0.f;
    }
    float m = -INFINITY, l = 0.f;   // task 2 calls its running sum r; it plays the part of l
    for (int j = 0; j < num_keys; ++j) {
        float dot = 0.f;
#pragma unroll
        for (int i = 0; i < kMaxPerLane; ++i)
            if (i < per) dot = fmaf(qv[i], __bfloat162float(k[size_t(j) * head_dim + lane * per + i]), dot);
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, s);
        // One key: the running sum is brought to the new maximum and takes the key's weight, l <- l 2^... in natural
        // units: l <- l exp(m - m') + exp(s - m').  What differs between the forms is what the output carries.
        const float score = sm_scale * dot;
        const float top = fmaxf(m, score);
        const float weight = expf(score - top);
        const float keep = expf(m - top);            // share of the old maximum's scale that survives; 0 on the first key
        l = fmaf(l, keep, weight);
        if constexpr (kTask == 2) {
            // deferred division: the output stays un-normalised at the scale of the running maximum
#pragma unroll
            for (int i = 0; i < kMaxPerLane; ++i)
                if (i < per) o[i] = fmaf(weight, __bfloat162float(v[size_t(j) * head_dim + lane * per + i]), o[i] * keep);
        } else {
            // normalised at every step (tasks 0 and 1 carry the same numbers; the paper splits the step into one
            // operator or two): the normalised output is a running weighted mean, and a new key moves it toward its
            // value by the key's share of the sum so far, o <- o + (weight / l) (v - o)
            const float share = weight / l;
#pragma unroll
            for (int i = 0; i < kMaxPerLane; ++i)
                if (i < per) o[i] = fmaf(share, __bfloat162float(v[size_t(j) * head_dim + lane * per + i]) - o[i], o[i]);
        }
        m = top;
    }
    const float fin = (kTask == 2 && l > 0.f) ? 1.f / l : 1.f;   // the one deferred division
#pragma unroll
    for (int i = 0; i < kMaxPerLane; ++i)
        if (i < per) out[size_t(row) * head_dim + lane * per + i] = o[i] * fin;
    if (lane == 0) { m_out[row] = m; l_out[row] = l; }
}

}  // namespace
}  // namespace psa

extern "C" psa_status_t psa_attn_task(int32_t task, const void *q, const void *k, const void *v, int32_t num_rows, int32_t num_keys,
                                      int32_t head_dim, float sm_scale, float *out, float *m_out, float *l_out, void *cuda_stream)
{
    using psa::set_last_error;
    if (task < 0 || task > 2) return set_last_error(PSA_ERR_INVALID_ARG, "task must be 0, 1 or 2");
    if (num_rows < 0 || num_keys < 0) return set_last_error(PSA_ERR_INVALID_ARG, "negative num_rows or num_keys");
    if (head_dim <= 0 || head_dim % 32 || head_dim > 32 * psa::kMaxPerLane)
        return set_last_error(PSA_ERR_UNSUPPORTED, "head_dim must be a multiple of 32, at most 256");
    if (num_rows == 0) return PSA_OK;
    if (!q || !out || !m_out || !l_out || (num_keys > 0 && (!k || !v))) return set_last_error(PSA_ERR_INVALID_ARG, "null argument");
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int warps = 4;
    const dim3 grid((num_rows + warps - 1) / warps), block(warps * 32);
    const auto *qq = static_cast<const __nv_bfloat16 *>(q);
    const auto *kk = static_cast<const __nv_bfloat16 *>(k);
    const auto *vv = static_cast<const __nv_bfloat16 *>(v);
    if (task == 0) psa::attn_task_kernel<0><<<grid, block, 0, st>>>(qq, kk, vv, num_rows, num_keys, head_dim, sm_scale, out, m_out, l_out);
    else if (task == 1) psa::attn_task_kernel<1><<<grid, block, 0, st>>>(qq, kk, vv, num_rows, num_keys, head_dim, sm_scale, out, m_out, l_out);
    else psa::attn_task_kernel<2><<<grid, block, 0, st>>>(qq, kk, vv, num_rows, num_keys, head_dim, sm_scale, out, m_out, l_out);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return set_last_error(PSA_ERR_CUDA, std::string("attn task launch: ") + cudaGetErrorString(e));
    return PSA_OK;
}
