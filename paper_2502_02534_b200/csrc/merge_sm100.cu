// Merge stage: log-sum-exp combination of every (sample, query head) row's partial results.
//
// Each partial i carries a normalised output O_i and lse_i = ln sum_j exp(x_j) over its
// own keys.  Because the un-normalised accumulators of the paper's deferred-division
// recurrence (attn Task 2) add once they are brought to a common maximum,
//     lse = ln sum_i exp(lse_i),   out = sum_i exp(lse_i - lse) O_i .
// A row with no partial at all (empty prefix and empty suffix) gives out = 0, lse = -inf.
//
// One warp per row; lane l owns D/32 consecutive output elements.  Partials are read with
// L2-only loads (they were written by other blocks moments ago).  The stage moves
// (#partials * D * 4 + D * 2) bytes per row and is bound by L2 / HBM bandwidth.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "psa_internal.h"

namespace psa {
namespace {

constexpr int kMergeWarps = 4;

template <int D, int kChunk>
__global__ void __launch_bounds__(kMergeWarps * 32)
merge_kernel(const SampleInfo *__restrict__ sample_info, const int32_t *__restrict__ suffix_lens,
             const float *__restrict__ partial_o, const float *__restrict__ partial_lse,
             int num_rows, int num_q_heads, int group, int chunk_tokens, int out_is_f32,
             void *__restrict__ out, float *__restrict__ lse_out, const int *prefix_counters, int prefix_blocks, int *__restrict__ status)
{
    constexpr int V = D / 32;  // floats per lane: 2 or 4
    // kChunk rows are fetched together (registers: kChunk float4 per lane)
    const int lane = threadIdx.x & 31;
    // a warp past the last row repeats the last row's work and stores nothing: every warp of the block then reaches
    // the block-wide barrier below
    const int row_id = blockIdx.x * kMergeWarps + (threadIdx.x >> 5);
    const bool live = row_id < num_rows;
    const int row = live ? row_id : num_rows - 1;
    const int s = row / num_q_heads, h = row % num_q_heads;
    const int kv = h / group, g = h % group;

    // head of the sample's record, then one int4 per prefix level (a sample of a cascade belongs to several groups)
    const int4 *ip = reinterpret_cast<const int4 *>(sample_info + s);
    const int4 head = __ldg(ip);
    const int suf_row0 = head.x, suf_chunks = head.y, suf_bound = head.z, n_levels = head.w;
    int lv_first[kMaxPrefixLevels], lv_stride[kMaxPrefixLevels], lv_end[kMaxPrefixLevels];   // lv_end: running count of splits
    int n_pre = 0;
#pragma unroll
    for (int l = 0; l < kMaxPrefixLevels; ++l) {
        int4 lv = make_int4(0, 0, 0, 0);
        if (l < n_levels) lv = __ldg(ip + 1 + l);
        lv_first[l] = lv.x + kv * lv.w + g;
        lv_stride[l] = lv.y;
        n_pre += lv.z;
        lv_end[l] = n_pre;
    }
    int S = __ldg(suffix_lens + s);
    S = min(max(S, 0), suf_bound);
    const int n_suf = (S + chunk_tokens - 1) / chunk_tokens;
    const int n_total = n_pre + n_suf;

    const int suf_first = suf_row0 + kv * suf_chunks * group + g;
    auto partial_row = [&](int i) {
        if (i >= n_pre) return suf_first + (i - n_pre) * group;
        int r = lv_first[0] + i * lv_stride[0];
#pragma unroll
        for (int l = 1; l < kMaxPrefixLevels; ++l)
            if (i >= lv_end[l - 1]) r = lv_first[l] + (i - lv_end[l - 1]) * lv_stride[l];
        return r;
    };

    // In a fused step that has both stages the preceding grid is the suffix stage, which ran beside the prefix
    // stage; prefix blocks count themselves off after storing their results (launches x blocks in total, both
    // counters wrap together).  The launch was announced before the suffix grid could start and every prefix block
    // was running before the first suffix block, so the count is complete or about to be; the wait is bounded all
    // the same.  It sits BEFORE the wait for the suffix grid, off the critical path.
    int lag = 0;
    if (prefix_blocks > 0) {
        if (lane == 0) {
            unsigned long long t0 = 0;
            for (uint32_t spins = 0;; ++spins) {
                // both words in one load (they are adjacent and 8-byte aligned): launches in the low half, blocks done in the high half
                unsigned long long both;
                asm volatile("ld.acquire.gpu.global.b64 %0, [%1];" : "=l"(both) : "l"(prefix_counters) : "memory");
                lag = int(uint32_t(both) * uint32_t(prefix_blocks) - uint32_t(both >> 32));
                if (lag <= 0) break;
                __nanosleep(200);   // the prefix stage may still run for a while (long prompts, short suffixes): poll gently
                if ((spins & 255u) == 255u) {
                    unsigned long long now;
                    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
                    if (t0 == 0) t0 = now;
                    else if (now - t0 > 2000000000ull) { atomicCAS(status, 0, int(PSA_ERR_TIMEOUT)); break; }
                }
            }
        }
        lag = __shfl_sync(0xffffffffu, lag, 0);
        __syncwarp();   // lane 0's acquire load orders the other lanes' reads of the partial results as well
    }
    // EVERY warp of the block must have read the counters before ANY warp lets the next kernel start: the block
    // counts as having released its dependents as soon as one of its threads has, and the next step's prefix grid
    // announces itself in the same counters the moment it is scheduled -- a warp still polling (it sleeps 200 ns
    // between polls) would then wait for a launch that itself waits for this grid.
    __syncthreads();
    if (prefix_blocks > 0 && lag > 0) return;   // timed out: the row stays unwritten, the status word says why
    // launched as a programmatic dependent: the partial results exist only after the preceding grids completed
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // the next kernel in the stream (typically the next step's prefix stage) may set itself up meanwhile;
    // it waits for this grid to complete before it touches memory
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // Single pass with a running maximum (the same deferred-division bookkeeping as inside the kernels):
    // per group of 32 partials, lane i loads lse_i while the first kChunk output rows of the group are already
    // being fetched -- row addresses do not depend on the lse values -- so the lse round trip
    // and the first row round trip overlap.
    float acc[V];
#pragma unroll
    for (int v = 0; v < V; ++v) acc[v] = 0.f;
    float top = -INFINITY, z = 0.f;   // z: this lane's share of sum_i exp(lse_i - top)
    auto fetch = [&](int r) {
        const float *src = partial_o + size_t(r) * D + lane * V;
        if constexpr (V == 4) return __ldcg(reinterpret_cast<const float4 *>(src));
        else { const float2 x = __ldcg(reinterpret_cast<const float2 *>(src)); return make_float4(x.x, x.y, 0.f, 0.f); }
    };
    for (int base = 0; base < n_total; base += 32) {
        const int mine = base + lane;
        const int my_row = mine < n_total ? partial_row(mine) : 0;
        const float my_lse = mine < n_total ? __ldcg(partial_lse + my_row) : -INFINITY;
        const int cnt = min(32, n_total - base);
        float my_w = 0.f;
        for (int c0 = 0; c0 < cnt; c0 += kChunk) {
            float4 x[kChunk];
#pragma unroll
            for (int u = 0; u < kChunk; ++u) {
                const int r = __shfl_sync(0xffffffffu, my_row, (c0 + u) & 31);
                x[u] = (c0 + u < cnt) ? fetch(r) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            if (c0 == 0) {   // first use of the lse values of this group
                float gmax = my_lse;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) gmax = fmaxf(gmax, __shfl_xor_sync(0xffffffffu, gmax, o));
                const float new_top = fmaxf(top, gmax);
                if (new_top != -INFINITY) {
                    const float scale = __expf(top - new_top);   // 0 when nothing was accumulated yet
#pragma unroll
                    for (int v = 0; v < V; ++v) acc[v] *= scale;
                    z *= scale;
                    top = new_top;
                    my_w = __expf(my_lse - top);                 // an empty piece (lse = -inf) gets weight 0
                    z += my_w;
                }
            }
#pragma unroll
            for (int u = 0; u < kChunk; ++u) {
                const float w = __shfl_sync(0xffffffffu, my_w, (c0 + u) & 31);
                if (c0 + u < cnt) {
                    acc[0] += w * x[u].x; acc[1] += w * x[u].y;
                    if constexpr (V == 4) { acc[2] += w * x[u].z; acc[3] += w * x[u].w; }
                }
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    if (top != -INFINITY) {
        const float inv = 1.f / z;
#pragma unroll
        for (int v = 0; v < V; ++v) acc[v] *= inv;
    }
    if (!live) return;
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
    cudaLaunchConfig_t lc{};
    lc.gridDim = grid;
    lc.blockDim = block;
    lc.stream = st;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = &attr;
    lc.numAttrs = a.after_stage ? 1 : 0;   // start filling in while the preceding stage drains
    const int f32 = a.out_dtype == PSA_OUT_F32;
    const int counted_blocks = (a.prefix_counters && a.status) ? a.prefix_blocks : 0;
    cudaError_t e;
    const bool small = rows <= 4096;   // few rows: latency matters, fetch 16 partial rows at a time
    const bool large = rows > 8192;    // many rows: occupancy matters more than loads in flight per warp (4 rows at a time, 2x the warps per SM)
    if (a.head_dim == 128 && large)
        e = cudaLaunchKernelEx(&lc, merge_kernel<128, 4>, a.sample_info, a.suffix_lens, a.partial_o, a.partial_lse, rows,
                               a.num_q_heads, group, a.chunk_tokens, f32, a.out, a.lse, a.prefix_counters, counted_blocks, a.status);
    else if (a.head_dim == 128 && small)
        e = cudaLaunchKernelEx(&lc, merge_kernel<128, 16>, a.sample_info, a.suffix_lens, a.partial_o, a.partial_lse, rows,
                               a.num_q_heads, group, a.chunk_tokens, f32, a.out, a.lse, a.prefix_counters, counted_blocks, a.status);
    else if (a.head_dim == 128)
        e = cudaLaunchKernelEx(&lc, merge_kernel<128, 8>, a.sample_info, a.suffix_lens, a.partial_o, a.partial_lse, rows,
                               a.num_q_heads, group, a.chunk_tokens, f32, a.out, a.lse, a.prefix_counters, counted_blocks, a.status);
    else
        e = cudaLaunchKernelEx(&lc, merge_kernel<64, 16>, a.sample_info, a.suffix_lens, a.partial_o, a.partial_lse, rows,
                               a.num_q_heads, group, a.chunk_tokens, f32, a.out, a.lse, a.prefix_counters, counted_blocks, a.status);
    if (e != cudaSuccess && err) *err = std::string("merge launch: ") + cudaGetErrorString(e);
    return int(e);
}

}  // namespace psa
