// The step after the path, second half: draw the next token of every sample from its logits at a temperature.
//
// The paper samples its candidate answers at temperature T in {0.4, 0.7, 1.0} with a seed (appendix "Experiment
// details").  Token i is drawn with probability softmax(logits / T)_i through the Gumbel-max identity:
//     token = argmax_i ( logits_i / T + g_i ),   g_i = -ln(-ln u_i),   u_i uniform on (0, 1),
// which needs no normalisation pass and no prefix sum: one streaming pass over the row.  T = 0 is greedy decoding.
// The uniforms come from the counter-based generator Philox4x32-10 (Salmon et al., SC'11), written from its published
// definition: counter = (index / 4, step, row, 0), key = the two words of the row's seed, u = ((x >> 9) + 0.5) 2^-23 for
// the output word x = output[index % 4] -- so a draw is a pure function of (seed, step, row, index).
//
// Layout of the work: a row is cut into `splits` contiguous pieces, one thread block each (so that few rows still fill
// the machine); a thread handles groups of four consecutive logits (one 16-byte or 8-byte load, one Philox call), keeps
// its best (score, index), the block reduces by shuffles and one 64-bit atomicMax per warp folds it into the row's cell
// of the scratch array: key = (order-preserving bits of the fp32 score) << 32 | (2^32 - 1 - index), so that equal scores
// go to the lowest index.  A second tiny kernel turns the cells into token ids.
// Bound: about 10 integer multiplies / xors and two logarithms per logit next to 2 or 4 bytes of HBM traffic: ALU and HBM
// are of the same order and the ALU side wins: 256 rows x 131072 bf16 logits take about 80 us on a B200 (0.84 TB/s).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <string>
#include <type_traits>

#include "psa_internal.h"

namespace psa {
namespace {

constexpr int kSampleThreads = 256;

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1,
                                              uint32_t (&out)[4])
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// g = -ln(-ln u) for u = (m + 0.5) 2^-23, m < 2^23 (the top 23 bits of a Philox word).  u is assembled from the bits
// (1.m as a float in [1, 2), minus 1, plus 2^-24: all exact), without an integer-to-float conversion.  The draws that
// win a large vocabulary are those with u next to 1, where ln u cancels: within 1/64 of 1, E = -ln u is taken from
// w = 1 - u (exact as well) as the series w + w^2/2 + w^3/3 + w^4/4 (remainder below 2e-10 relative).  Elsewhere the
// fast logarithm is accurate to 2.3e-5 relative or better in E, i.e. absolute in g.
__device__ __forceinline__ float gumbel(uint32_t m)
{
    const float f = __uint_as_float(0x3F800000u | m);                  // 1 + m 2^-23
    const float u = (f - 1.f) + 5.9604644775390625e-8f;                // + 2^-24
    const float w = (2.f - f) - 5.9604644775390625e-8f;                // 1 - u
    const float series = w * fmaf(w, fmaf(w, fmaf(w, 0.25f, 0.333333343f), 0.5f), 1.f);
    const float e = w < 0.015625f ? series : -__logf(u);
    return -__logf(e);
}

__device__ __forceinline__ unsigned long long make_key(float score, uint32_t index)
{
    const uint32_t b = __float_as_uint(score);
    const uint32_t ord = (b & 0x80000000u) ? ~b : (b | 0x80000000u);   // unsigned order == float order
    return (static_cast<unsigned long long>(ord) << 32) | (0xFFFFFFFFu - index);
}

template <bool kF32>
__global__ void __launch_bounds__(kSampleThreads)
sample_kernel(const void *__restrict__ logits, int64_t row_stride, int vocab, int splits, const float *__restrict__ temperature,
              const unsigned long long *__restrict__ seeds, uint32_t step_value, const uint32_t *__restrict__ step_device,
              unsigned long long *__restrict__ cells)
{
    const uint32_t step = step_device ? __ldg(step_device) : step_value;   // a replayed graph reads the step from memory
    const int row = blockIdx.y, split = blockIdx.x;
    const float T = __ldg(temperature + row);
    const bool greedy = !(T > 0.f);
    const float inv_t = greedy ? 1.f : 1.f / T;
    const unsigned long long seed = __ldg(seeds + row);
    const uint32_t k0 = uint32_t(seed), k1 = uint32_t(seed >> 32);
    // groups of four logits; this block owns groups [g0, g1)
    const int n_groups = (vocab + 3) / 4;
    const int per = (n_groups + splits - 1) / splits;
    const int g0 = split * per, g1 = min(n_groups, g0 + per);
    float best = -INFINITY;
    uint32_t best_i = 0xFFFFFFFFu;   // "nothing seen": loses against every real index at equal score
    // scores of the four logits x[] of group g (indices 4g .. 4g+3, the first `valid` of them inside the row)
    auto consume = [&](int g, const float (&x)[4], int valid) {
        uint32_t r[4] = {0u, 0u, 0u, 0u};
        if (!greedy) philox4x32_10(uint32_t(g), step, uint32_t(row), 0u, k0, k1, r);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float s = x[e];
            if (!greedy) s = fmaf(x[e], inv_t, gumbel(r[e] >> 9));
            if (e < valid && (s > best || best_i == 0xFFFFFFFFu)) { best = s; best_i = uint32_t(4 * g + e); }   // first maximum wins
        }
    };
    // full groups: one vector load each, the next one in flight while this one is worked on
    using Vec = typename std::conditional<kF32, float4, uint2>::type;
    const Vec *base = reinterpret_cast<const Vec *>(kF32 ? static_cast<const void *>(static_cast<const float *>(logits) + row * row_stride)
                                                         : static_cast<const void *>(static_cast<const __nv_bfloat16 *>(logits) + row * row_stride));
    const int full_end = min(g1, vocab / 4);
    int g = g0 + threadIdx.x;
    Vec cur{};
    if (g < full_end) cur = __ldcs(base + g);
    for (; g < full_end; g += kSampleThreads) {
        Vec nxt{};
        if (g + kSampleThreads < full_end) nxt = __ldcs(base + g + kSampleThreads);
        float x[4];
        if constexpr (kF32) {
            x[0] = cur.x; x[1] = cur.y; x[2] = cur.z; x[3] = cur.w;
        } else {
            x[0] = __uint_as_float(cur.x << 16); x[1] = __uint_as_float(cur.x & 0xFFFF0000u);
            x[2] = __uint_as_float(cur.y << 16); x[3] = __uint_as_float(cur.y & 0xFFFF0000u);
        }
        consume(g, x, 4);
        cur = nxt;
    }
    // the ragged last group of the row (vocab not a multiple of 4): one thread of the block that owns it
    const int tail = vocab / 4;
    if ((vocab & 3) && tail >= g0 && tail < g1 && threadIdx.x == 0) {
        float x[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            x[e] = -INFINITY;
            if (4 * tail + e < vocab) {
                if constexpr (kF32) x[e] = static_cast<const float *>(logits)[row * row_stride + 4 * tail + e];
                else x[e] = __bfloat162float(static_cast<const __nv_bfloat16 *>(logits)[row * row_stride + 4 * tail + e]);
            }
        }
        consume(tail, x, vocab & 3);
    }
    unsigned long long key = best_i == 0xFFFFFFFFu ? 0ull : make_key(best, best_i);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, key, o);
        key = other > key ? other : key;
    }
    if ((threadIdx.x & 31) == 0 && key != 0ull) atomicMax(cells + row, key);
}

__global__ void sample_finalize_kernel(const unsigned long long *__restrict__ cells, int num_rows, int32_t *__restrict__ tokens,
                                       uint32_t *step_device, uint32_t advance)
{
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r < num_rows) tokens[r] = int32_t(0xFFFFFFFFu - uint32_t(cells[r]));
    // every block of the drawing kernel has read the step by now (this kernel follows it in the stream)
    if (step_device != nullptr && r == 0) *step_device += advance;
}

}  // namespace
}  // namespace psa

extern "C" size_t psa_sample_scratch_bytes(int32_t num_rows) { return num_rows > 0 ? size_t(num_rows) * 8 : 0; }

static psa_status_t sample_impl(const void *logits, int32_t logits_dtype, int64_t row_stride, int32_t num_rows, int32_t vocab,
                                const float *temperature, const uint64_t *seeds, uint32_t step, uint32_t *step_device, uint32_t advance,
                                int32_t *tokens, void *scratch, size_t scratch_bytes, void *cuda_stream)
{
    using psa::set_last_error;
    if (num_rows < 0 || vocab < 0) return set_last_error(PSA_ERR_INVALID_ARG, "negative num_rows or vocab");
    if (num_rows == 0) return PSA_OK;
    if (vocab == 0) return set_last_error(PSA_ERR_INVALID_ARG, "vocab must be positive");
    if (num_rows > 65535) return set_last_error(PSA_ERR_UNSUPPORTED, "at most 65535 rows per call");
    if (logits_dtype != PSA_OUT_BF16 && logits_dtype != PSA_OUT_F32) return set_last_error(PSA_ERR_UNSUPPORTED, "logits_dtype must be PSA_OUT_BF16 or PSA_OUT_F32");
    if (!logits || !temperature || !seeds || !tokens || !scratch) return set_last_error(PSA_ERR_INVALID_ARG, "null argument");
    if (reinterpret_cast<uintptr_t>(logits) % 16 || row_stride < vocab || row_stride % 8)
        return set_last_error(PSA_ERR_INVALID_ARG, "logits must be 16-byte aligned with a row stride >= vocab that is a multiple of 8 elements");
    if (reinterpret_cast<uintptr_t>(scratch) % 8 || scratch_bytes < psa_sample_scratch_bytes(num_rows))
        return set_last_error(PSA_ERR_WORKSPACE, "scratch must be 8-byte aligned and hold psa_sample_scratch_bytes(num_rows)");
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return set_last_error(PSA_ERR_CUDA, std::string("querying the SM count: ") + cudaGetErrorString(e));
    // enough blocks for about four per SM, each with at least 2048 logits
    const int n_groups = (vocab + 3) / 4;
    int splits = (4 * sms + num_rows - 1) / num_rows;
    splits = std::max(1, std::min(splits, (n_groups + 511) / 512));
    e = cudaMemsetAsync(scratch, 0, size_t(num_rows) * 8, st);
    if (e != cudaSuccess) return set_last_error(PSA_ERR_CUDA, std::string("clearing the scratch cells: ") + cudaGetErrorString(e));
    const dim3 grid(splits, num_rows);
    auto *cells = static_cast<unsigned long long *>(scratch);
    const auto *sd = reinterpret_cast<const unsigned long long *>(seeds);
    if (logits_dtype == PSA_OUT_F32)
        psa::sample_kernel<true><<<grid, psa::kSampleThreads, 0, st>>>(logits, row_stride, vocab, splits, temperature, sd, step, step_device, cells);
    else
        psa::sample_kernel<false><<<grid, psa::kSampleThreads, 0, st>>>(logits, row_stride, vocab, splits, temperature, sd, step, step_device, cells);
    psa::sample_finalize_kernel<<<(num_rows + 255) / 256, 256, 0, st>>>(cells, num_rows, tokens, step_device, advance);
    e = cudaGetLastError();
    if (e != cudaSuccess) return set_last_error(PSA_ERR_CUDA, std::string("sampling launch: ") + cudaGetErrorString(e));
    return PSA_OK;
}

extern "C" psa_status_t psa_sample_tokens(const void *logits, int32_t logits_dtype, int64_t row_stride, int32_t num_rows, int32_t vocab,
                                          const float *temperature, const uint64_t *seeds, uint32_t step, int32_t *tokens,
                                          void *scratch, size_t scratch_bytes, void *cuda_stream)
{
    return sample_impl(logits, logits_dtype, row_stride, num_rows, vocab, temperature, seeds, step, nullptr, 0u, tokens, scratch,
                       scratch_bytes, cuda_stream);
}

extern "C" psa_status_t psa_sample_tokens_at(const void *logits, int32_t logits_dtype, int64_t row_stride, int32_t num_rows, int32_t vocab,
                                             const float *temperature, const uint64_t *seeds, uint32_t *step_device, uint32_t advance,
                                             int32_t *tokens, void *scratch, size_t scratch_bytes, void *cuda_stream)
{
    if (!step_device || reinterpret_cast<uintptr_t>(step_device) % 4)
        return psa::set_last_error(PSA_ERR_INVALID_ARG, "step_device must be a 4-byte aligned device pointer");
    return sample_impl(logits, logits_dtype, row_stride, num_rows, vocab, temperature, seeds, 0u, step_device, advance, tokens, scratch,
                       scratch_bytes, cuda_stream);
}
