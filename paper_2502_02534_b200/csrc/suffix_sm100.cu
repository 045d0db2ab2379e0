// Suffix stage: each sample's G query rows (one KV head) against its own generated
// tokens, stored in 16-token pages scattered through a pool.
//
// Arithmetic is the deferred-division online softmax (the paper's attn Task 2
// recurrence: running maximum m, running sum l, un-normalised accumulator O), applied
// page by page; the division happens once, when the block writes its partial result.
//
// The stage is bound by HBM: every K and V byte is read exactly once and there are only
// G (<= 8) flops per byte.  Design for that bound:
//   * one thread block per (sample, kv head, token chunk); its 4 warps take pages
//     round-robin, each with a private ring of kStages (K page + V page) buffers that
//     it fills with 16-byte cp.async copies -- a page of one head is 16 x D bf16 =
//     4 KB contiguous (D = 128), so every copy instruction of a warp reads 512
//     consecutive bytes.  No block-wide barrier in the main loop.
//   * the dot products run on warp-level tensor-core MMAs (m16n8k16, bf16 in, fp32
//     accumulate), computed TRANSPOSED so that the G (<= 8) query rows are the MMA's
//     8-wide side and nothing is padded: S^T = K Q^T (16 tokens x 8 rows) and
//     O^T = V^T P^T (16 channels x 8 rows), one MMA per 16 channels each -- half the
//     MMAs of the untransposed form, whose 16-row side would be half zeros.  Plain FMAs
//     could not keep up with HBM at G = 8.  K fragments come from ldmatrix, V^T
//     fragments from ldmatrix.trans, both conflict-free through a 16-byte XOR swizzle
//     of the rows; P^T comes from the S^T accumulators through two movmatrix transposes.
//   * row maxima are refreshed lazily: the shuffles + rescale only run when some
//     logit exceeds the reference maximum by more than 2^8.
//   * slots of the last page beyond the sample's length are zero-filled by the copy
//     (source size 0), never read from memory, and masked to -inf before the softmax.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "psa_internal.h"

namespace psa {
namespace {

constexpr int kWarps = 4;
constexpr int kStages = 3;
constexpr float kRescaleThreshold = 8.f;  // log2 units

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return uint32_t(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// D(16x8, f32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// transpose of an 8x8 matrix of 16-bit elements held in the fragment layout (row = lane / 4, columns 2 * (lane % 4), +1)
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a)
{
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

template <int D>
struct SuffixSmem {
    static constexpr int kRowBytes = D * 2;            // one token of one head
    static constexpr int kPageBytes = kPageSize * kRowBytes;
    static constexpr int kStageBytes = 2 * kPageBytes; // K page + V page
    static constexpr int kWarpBytes = kStages * kStageBytes;
    static constexpr int kTotal = kWarps * kWarpBytes;
};

template <int D, int G>
__global__ void __launch_bounds__(kWarps * 32, 2)
suffix_kernel(const __nv_bfloat16 *__restrict__ q, const __nv_bfloat16 *__restrict__ pool_k,
              const __nv_bfloat16 *__restrict__ pool_v, int64_t stride_page, int64_t stride_head, int64_t stride_tok,
              const int32_t *__restrict__ page_indptr, const int32_t *__restrict__ page_indices,
              const int32_t *__restrict__ suffix_lens, const SuffixItem *__restrict__ items,
              const SampleInfo *__restrict__ sample_info, int num_q_heads, int chunk_tokens, float scale_log2,
              float *__restrict__ partial_o, float *__restrict__ partial_lse, int first_of_step)
{
    using L = SuffixSmem<D>;
    constexpr int KK = D / 16;           // k-steps of QK^T
    constexpr int DT = D / 16;           // 16-channel tiles of O^T
    constexpr int CPR = L::kRowBytes / 16;  // 16-byte chunks per token row
    extern __shared__ __align__(128) unsigned char smem_raw[];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int4 item = __ldg(reinterpret_cast<const int4 *>(items + blockIdx.x));   // plan data, bound long before
    const int s = item.x, kv = item.y, tok0 = item.z, prow0 = item.w;
    // Not behind a prefix stage: this grid is launched as a programmatic dependent of whatever precedes it in the
    // stream, its blocks got here while that kernel drained, and they wait for it before they touch anything it may
    // have written (lengths, page table, K/V, Q) or still be reading (partial results).  The next kernel may then
    // set itself up under this grid.  Behind a prefix stage there is nothing to wait for: the prefix blocks have.
    if (first_of_step) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    }
    int S = __ldg(suffix_lens + s);
    S = min(S, __ldg(&sample_info[s].suf_len_bound));
    const int n_tok = min(S - tok0, chunk_tokens);
    if (n_tok <= 0) return;  // the merge stage derives the chunk count from the same length
    const int n_pages = (n_tok + kPageSize - 1) / kPageSize;
    const int my_pages = (n_pages - warp + kWarps - 1) / kWarps;  // pages warp, warp+4, ...
    const int32_t *my_page_ids = page_indices + __ldg(page_indptr + s) + tok0 / kPageSize;

    // ---- Q^T as the B operand (16 channels x 8 rows per k-step): row lane / 4, channels 2 * (lane % 4), +1 and those
    // + 8; rows >= G stay zero
    const int qrow = lane >> 2, qcol = (lane & 3) * 2;
    uint32_t qb0[KK], qb1[KK];
    {
        const __nv_bfloat16 *qp = q + (size_t(s) * num_q_heads + size_t(kv) * G + qrow) * D + qcol;
#pragma unroll
        for (int kk = 0; kk < KK; ++kk) {
            qb0[kk] = qrow < G ? __ldg(reinterpret_cast<const uint32_t *>(qp + kk * 16)) : 0u;
            qb1[kk] = qrow < G ? __ldg(reinterpret_cast<const uint32_t *>(qp + kk * 16 + 8)) : 0u;
        }
    }

    const uint32_t warp_smem = smem_u32(smem_raw) + warp * L::kWarpBytes;
    const __nv_bfloat16 *head_k = pool_k + int64_t(kv) * stride_head;
    const __nv_bfloat16 *head_v = pool_v + int64_t(kv) * stride_head;

    // Page ids of this warp's pages, 32 at a time: lane l holds the id of page number 32 g + l of the warp, for the
    // group g in use (ids_cur) and the next one (ids_nxt).  One coalesced load per group instead of one dependent
    // load per page: otherwise every copy would wait a full L2 round trip for its address first.
    auto load_ids = [&](int g) {
        const int i = g * 32 + lane;
        return i < my_pages ? __ldg(my_page_ids + warp + i * kWarps) : 0;
    };
    int ids_cur = load_ids(0), ids_nxt = load_ids(1);

    // copy page number i of this warp (tokens [16*(warp+4i), +16) of the chunk) into ring slot i % kStages;
    // called with i = 0, 1, 2, ... in order
    auto issue_page = [&](int i) {
        if (i > 0 && (i & 31) == 0) {   // warp-uniform: the next group of ids becomes the current one
            ids_cur = ids_nxt;
            ids_nxt = load_ids((i >> 5) + 1);
        }
        const int64_t page = __shfl_sync(0xffffffffu, ids_cur, i & 31);
        if (i < my_pages) {
            const int page_in_chunk = warp + i * kWarps;
            const int valid = min(kPageSize, n_tok - page_in_chunk * kPageSize);
            const uint32_t dst = warp_smem + (i % kStages) * L::kStageBytes;
            const __nv_bfloat16 *src_k = head_k + page * stride_page;
            const __nv_bfloat16 *src_v = head_v + page * stride_page;
#pragma unroll
            for (int c = lane; c < kPageSize * CPR; c += 32) {
                const int row = c / CPR, col = c % CPR;
                const int bytes = row < valid ? 16 : 0;              // 0: nothing is read, the slot is zero-filled
                const int64_t off = bytes ? row * stride_tok + col * 8 : 0;
                const uint32_t d = dst + row * L::kRowBytes + ((col ^ (row & 7)) << 4);
                cp_async16(d, src_k + off, bytes);
                cp_async16(d + L::kPageBytes, src_v + off, bytes);
            }
        }
        cp_async_commit();  // an empty group keeps the group count uniform
    };

    // Accumulator layout of the transposed products: a thread holds query rows r0 = 2 * (lane % 4) and r0 + 1, for
    // tokens (S^T) or channels (O^T) lane / 4 and lane / 4 + 8 of each 16-wide tile: [0], [1] = rows r0, r0 + 1 of the
    // first, [2], [3] of the second.
    const int trow = lane >> 2, r0 = (lane & 3) * 2;
    float o[DT][4];
#pragma unroll
    for (int n = 0; n < DT; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
    float m_ref[2] = {-INFINITY, -INFINITY};  // reference maxima of rows r0, r0 + 1, log2 units (same in all 8 lanes that hold the row)
    float l_part[2] = {0.f, 0.f};             // this thread's share of the two row sums

#pragma unroll
    for (int i = 0; i < kStages - 1; ++i) issue_page(i);

    for (int i = 0; i < my_pages; ++i) {
        // Refill the slot read in iteration i - 1 BEFORE waiting for page i: while the warp waits, kStages pages are
        // in flight, not kStages - 1 (the blocks of a small step are bound by the latency of their own copies).
        __syncwarp();
        issue_page(i + kStages - 1);
        cp_async_wait<kStages - 1>();
        __syncwarp();

        const int page_in_chunk = warp + i * kWarps;
        const int valid = min(kPageSize, n_tok - page_in_chunk * kPageSize);
        const uint32_t sk = warp_smem + (i % kStages) * L::kStageBytes;
        const uint32_t sv = sk + L::kPageBytes;

        // ---- S^T = K Q^T for 16 tokens x 8 rows; two accumulators halve the dependent chain
        float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
        {
            const int mat = lane >> 3, r = lane & 7;
            const int tok = (mat & 1) * 8 + r;
            const uint32_t row_addr = sk + tok * L::kRowBytes;
#pragma unroll
            for (int kk = 0; kk < KK; kk += 2) {
                uint32_t a0, a1, a2, a3;
                ldmatrix_x4(row_addr + (((2 * kk + (mat >> 1)) ^ (tok & 7)) << 4), a0, a1, a2, a3);
                mma_bf16(sa, a0, a1, a2, a3, qb0[kk], qb1[kk]);
                ldmatrix_x4(row_addr + (((2 * kk + 2 + (mat >> 1)) ^ (tok & 7)) << 4), a0, a1, a2, a3);
                mma_bf16(sb, a0, a1, a2, a3, qb0[kk + 1], qb1[kk + 1]);
            }
        }
        // x[0], x[1]: token trow, rows r0, r0 + 1;  x[2], x[3]: token trow + 8
        float x[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) x[t] = (sa[t] + sb[t]) * scale_log2;
        if (valid < kPageSize) {
            if (trow >= valid) x[0] = x[1] = -INFINITY;
            if (trow + 8 >= valid) x[2] = x[3] = -INFINITY;
        }
        const float tmax0 = fmaxf(x[0], x[2]), tmax1 = fmaxf(x[1], x[3]);
        if (__any_sync(0xffffffffu, tmax0 > m_ref[0] + kRescaleThreshold || tmax1 > m_ref[1] + kRescaleThreshold)) {
            float rmax0 = tmax0, rmax1 = tmax1;   // over the 8 lanes that hold the same rows
#pragma unroll
            for (int sh = 4; sh < 32; sh <<= 1) {
                rmax0 = fmaxf(rmax0, __shfl_xor_sync(0xffffffffu, rmax0, sh));
                rmax1 = fmaxf(rmax1, __shfl_xor_sync(0xffffffffu, rmax1, sh));
            }
            const float m_new0 = fmaxf(m_ref[0], rmax0), m_new1 = fmaxf(m_ref[1], rmax1);
            if (m_new0 > m_ref[0] || m_new1 > m_ref[1]) {
                const float alpha0 = m_new0 > m_ref[0] ? fast_exp2(m_ref[0] - m_new0) : 1.f;  // m_ref = -inf gives 0
                const float alpha1 = m_new1 > m_ref[1] ? fast_exp2(m_ref[1] - m_new1) : 1.f;
                l_part[0] *= alpha0; l_part[1] *= alpha1;
#pragma unroll
                for (int n = 0; n < DT; ++n) { o[n][0] *= alpha0; o[n][1] *= alpha1; o[n][2] *= alpha0; o[n][3] *= alpha1; }
                m_ref[0] = m_new0; m_ref[1] = m_new1;
            }
        }
        float p[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) p[t] = fast_exp2(x[t] - m_ref[t & 1]);  // masked slots: exp2(-inf) = 0
        l_part[0] += p[0] + p[2];
        l_part[1] += p[1] + p[3];
        // P^T as the B operand (16 tokens x 8 rows): the two 8x8 halves of S^T's layout, transposed
        const uint32_t pb0 = movmatrix_trans(pack_bf16(p[0], p[1])), pb1 = movmatrix_trans(pack_bf16(p[2], p[3]));

        // ---- O^T += V^T P^T : V[16 tokens x D] read transposed, 16 channels per MMA
        {
            const int mat = lane >> 3, r = lane & 7;
            const int tok = (mat >> 1) * 8 + r;
            const uint32_t row_addr = sv + tok * L::kRowBytes;
#pragma unroll
            for (int n = 0; n < DT; ++n) {
                uint32_t a0, a1, a2, a3;
                ldmatrix_x4_trans(row_addr + (((2 * n + (mat & 1)) ^ (tok & 7)) << 4), a0, a1, a2, a3);
                mma_bf16(o[n], a0, a1, a2, a3, pb0, pb1);
            }
        }
    }
    cp_async_wait<0>();

    // ---- finish the row sums over the 8 lanes that share the rows, then combine the 4 warps through shared memory
    float l_row[2] = {l_part[0], l_part[1]};
#pragma unroll
    for (int sh = 4; sh < 32; sh <<= 1) {
        l_row[0] += __shfl_xor_sync(0xffffffffu, l_row[0], sh);
        l_row[1] += __shfl_xor_sync(0xffffffffu, l_row[1], sh);
    }
    __syncthreads();  // every warp is done with its ring: reuse the memory
    float *sm_o = reinterpret_cast<float *>(smem_raw);           // [kWarps][G][D]
    float *sm_m = sm_o + kWarps * G * D;                          // [kWarps][G]
    float *sm_l = sm_m + kWarps * G;                              // [kWarps][G]
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int g = r0 + h;
        if (g < G) {
            float *dst = sm_o + (warp * G + g) * D + trow;
#pragma unroll
            for (int n = 0; n < DT; ++n) { dst[n * 16] = o[n][h]; dst[n * 16 + 8] = o[n][2 + h]; }
            if (trow == 0) { sm_m[warp * G + g] = m_ref[h]; sm_l[warp * G + g] = l_row[h]; }
        }
    }
    __syncthreads();
    for (int e = threadIdx.x; e < G * D; e += kWarps * 32) {
        const int g = e / D, d = e % D;
        float top = -INFINITY;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) top = fmaxf(top, sm_m[w * G + g]);
        float z = 0.f, acc = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float mw = sm_m[w * G + g];
            const float f = mw == -INFINITY ? 0.f : fast_exp2(mw - top);
            z += f * sm_l[w * G + g];
            acc += f * sm_o[(w * G + g) * D + d];
        }
        partial_o[size_t(prow0 + g) * D + d] = acc / z;
        if (d == 0) partial_lse[prow0 + g] = (top + log2f(z)) * 0.6931471805599453f;
    }
    // When launched as a programmatic dependent of the prefix stage this grid runs beside it, and its blocks retire
    // as soon as they are done (so that the next ones take their place while prefix blocks still run): the merge
    // stage, ordered behind this grid, learns of the prefix grid's completion through a counter.  It may be
    // scheduled once every block is here.
    if (!first_of_step) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

template <int D, int G>
int launch_one(const SuffixArgs &a, cudaStream_t st)
{
    using L = SuffixSmem<D>;
    static_assert(L::kTotal >= int(sizeof(float)) * kWarps * G * (D + 2), "combine buffer must fit in the ring");
    auto kern = suffix_kernel<D, G>;
    static PerDeviceOnce once;   // per instantiation
    const int cfg_rc = once.ensure([&] {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        return int(e);
    });
    if (cfg_rc != 0) return cfg_rc;
    const float scale_log2 = a.sm_scale * 1.4426950408889634f;
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(a.num_items);
    lc.blockDim = dim3(kWarps * 32);
    lc.dynamicSmemBytes = L::kTotal;
    lc.stream = st;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = &attr;
    lc.numAttrs = 1;   // behind a prefix stage: runs beside it; else: set-up under the tail of the preceding kernel
    return int(cudaLaunchKernelEx(&lc, kern, static_cast<const __nv_bfloat16 *>(a.q), static_cast<const __nv_bfloat16 *>(a.pool_k),
                                  static_cast<const __nv_bfloat16 *>(a.pool_v), a.stride_page, a.stride_head, a.stride_tok,
                                  a.page_indptr, a.page_indices, a.suffix_lens, a.items, a.sample_info, a.num_q_heads,
                                  a.chunk_tokens, scale_log2, a.partial_o, a.partial_lse, a.after_prefix ? 0 : 1));
}

}  // namespace

int launch_suffix(const SuffixArgs &a, void *stream, std::string *err)
{
    if (a.num_items == 0) return 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int G = a.num_q_heads / a.num_kv_heads;
    int rc = -1;
#define PSA_CASE(DD, GG) if (a.head_dim == DD && G == GG) rc = launch_one<DD, GG>(a, st);
    PSA_CASE(128, 1) PSA_CASE(128, 2) PSA_CASE(128, 4) PSA_CASE(128, 8)
    PSA_CASE(64, 1) PSA_CASE(64, 2) PSA_CASE(64, 4) PSA_CASE(64, 8)
#undef PSA_CASE
    if (rc != 0 && err) *err = rc < 0 ? "suffix: unsupported shape" : std::string("suffix launch: ") + cudaGetErrorString(cudaError_t(rc));
    return rc;
}

}  // namespace psa
