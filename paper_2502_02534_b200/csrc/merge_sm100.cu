// Merge stage: log-sum-exp combination of every (sample, query head) row's partial results.
//
// Each partial i carries a normalised output O_i and lse_i = ln sum_j exp(x_j) over its
// own keys.  Because the un-normalised accumulators of the paper's deferred-division
// recurrence (attn Task 2) add once they are brought to a common maximum,
//     lse = ln sum_i exp(lse_i),   out = sum_i exp(lse_i - lse) O_i .
// A row with no partial at all (empty prefix and empty suffix) gives out = 0, lse = -inf.
//
// One warp per row; lane l owns D/32 consecutive output elements.  The stage moves
// (#partials * D * 4 + D * 2) bytes per row and is bound by L2 / HBM bandwidth.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "psa_internal.h"

namespace psa {
namespace {

constexpr int kMergeWarps = 8;

template <int D>
__global__ void __launch_bounds__(kMergeWarps * 32)
merge_kernel(const SampleInfo *__restrict__ sample_info, const int32_t *__restrict__ suffix_lens,
             const float *__restrict__ partial_o, const float *__restrict__ partial_lse,
             int num_rows, int num_q_heads, int group, int chunk_tokens, int out_is_f32,
             void *__restrict__ out, float *__restrict__ lse_out)
{
    constexpr int V = D / 32;  // floats per lane: 2 or 4
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * kMergeWarps + (threadIdx.x >> 5);
    if (row >= num_rows) return;
    const int s = row / num_q_heads, h = row % num_q_heads;
    const int kv = h / group, g = h % group;

    const int4 *ip = reinterpret_cast<const int4 *>(sample_info + s);
    const int4 a = __ldg(ip), b = __ldg(ip + 1);
    const int pre_row0 = a.x, pre_split_stride = a.y, pre_splits = a.z, pre_head_stride = a.w;
    const int suf_row0 = b.x, suf_chunks = b.y, suf_bound = b.z;
    int S = __ldg(suffix_lens + s);
    S = min(max(S, 0), suf_bound);
    const int n_suf = (S + chunk_tokens - 1) / chunk_tokens;
    const int n_total = pre_splits + n_suf;

    const int pre_first = pre_row0 + kv * pre_head_stride + g;
    const int suf_first = suf_row0 + kv * suf_chunks * group + g;
    auto partial_row = [&](int i) {
        return i < pre_splits ? pre_first + i * pre_split_stride : suf_first + (i - pre_splits) * group;
    };

    // pass 1: the largest lse (lanes stride over the partials)
    float top = -INFINITY;
    for (int i = lane; i < n_total; i += 32) top = fmaxf(top, __ldg(partial_lse + partial_row(i)));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) top = fmaxf(top, __shfl_xor_sync(0xffffffffu, top, o));

    float acc[V];
#pragma unroll
    for (int v = 0; v < V; ++v) acc[v] = 0.f;
    float z = 0.f;
    if (top != -INFINITY) {
        for (int i = 0; i < n_total; ++i) {
            const int r = partial_row(i);
            const float w = __expf(__ldg(partial_lse + r) - top);  // 0 for an empty piece (lse = -inf)
            z += w;
            const float *src = partial_o + size_t(r) * D + lane * V;
            if constexpr (V == 4) {
                const float4 x = __ldg(reinterpret_cast<const float4 *>(src));
                acc[0] += w * x.x; acc[1] += w * x.y; acc[2] += w * x.z; acc[3] += w * x.w;
            } else {
                const float2 x = __ldg(reinterpret_cast<const float2 *>(src));
                acc[0] += w * x.x; acc[1] += w * x.y;
            }
        }
        const float inv = 1.f / z;
#pragma unroll
        for (int v = 0; v < V; ++v) acc[v] *= inv;
    }
    if (out_is_f32) {
        float *dst = static_cast<float *>(out) + size_t(row) * D + lane * V;
        if constexpr (V == 4) *reinterpret_cast<float4 *>(dst) = make_float4(acc[0], acc[1], acc[2], acc[3]);
        else *reinterpret_cast<float2 *>(dst) = make_float2(acc[0], acc[1]);
    } else {
        __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(out) + size_t(row) * D + lane * V;
        __nv_bfloat162 lo = __floats2bfloat162_rn(acc[0], acc[1]);
        if constexpr (V == 4) {
            __nv_bfloat162 hi = __floats2bfloat162_rn(acc[2], acc[3]);
            uint2 pk;
            pk.x = *reinterpret_cast<uint32_t *>(&lo);
            pk.y = *reinterpret_cast<uint32_t *>(&hi);
            *reinterpret_cast<uint2 *>(dst) = pk;
        } else {
            *reinterpret_cast<__nv_bfloat162 *>(dst) = lo;
        }
    }
    if (lane == 0) lse_out[row] = (top == -INFINITY) ? -INFINITY : top + logf(z);
}

}  // namespace

int launch_merge(const MergeArgs &a, void *stream, std::string *err)
{
    const int rows = a.num_samples * a.num_q_heads;
    if (rows == 0) return 0;
    const int group = a.num_q_heads / a.num_kv_heads;
    const dim3 grid((rows + kMergeWarps - 1) / kMergeWarps), block(kMergeWarps * 32);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (a.head_dim == 128)
        merge_kernel<128><<<grid, block, 0, st>>>(a.sample_info, a.suffix_lens, a.partial_o, a.partial_lse, rows,
                                                  a.num_q_heads, group, a.chunk_tokens, a.out_dtype == PSA_OUT_F32, a.out, a.lse);
    else
        merge_kernel<64><<<grid, block, 0, st>>>(a.sample_info, a.suffix_lens, a.partial_o, a.partial_lse, rows,
                                                 a.num_q_heads, group, a.chunk_tokens, a.out_dtype == PSA_OUT_F32, a.out, a.lse);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess && err) *err = std::string("merge launch: ") + cudaGetErrorString(e);
    return int(e);
}

}  // namespace psa
