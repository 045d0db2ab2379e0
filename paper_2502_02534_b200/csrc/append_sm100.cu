// Step after the path: append one generated token's K and V per sample to the paged suffix pool.
//
// The paper's samples each grow by one token per decode step (appendix "Experiment details": at most 1024
// output tokens per sample), so between two psa_decode calls every sample's new K/V rows go to position S_s of
// its page list and S_s becomes S_s + 1.  The plan's suffix lengths are upper bounds, so the same plan serves
// every step of the loop until a sample reaches its bound.
//
// One block per sample: it reads S_s once, copies H_kv x D bf16 for K and for V with 16-byte vectors, and
// only then stores S_s + 1.  A sample that is already at its planned bound, or whose page list has no page for
// the new position, is left untouched and PSA_ERR_BOUNDS is raised in the status word.
#include <cuda_runtime.h>

#include "psa_internal.h"

namespace psa {
namespace {

__global__ void __launch_bounds__(128)
append_kernel(const uint4 *__restrict__ new_k, const uint4 *__restrict__ new_v, uint4 *__restrict__ pool_k,
              uint4 *__restrict__ pool_v, int64_t stride_page, int64_t stride_head, int64_t stride_tok,
              const int32_t *__restrict__ page_indptr, const int32_t *__restrict__ page_indices,
              int32_t *__restrict__ suffix_lens, const SampleInfo *__restrict__ sample_info, int num_kv_heads, int head_dim,
              int *__restrict__ status)
{
    const int s = blockIdx.x;
    __shared__ int sh_pos, sh_page;
    if (threadIdx.x == 0) {
        const int S = suffix_lens[s];
        const int first = page_indptr[s], n_pages = page_indptr[s + 1] - first;
        bool ok = S >= 0 && S < sample_info[s].suf_len_bound && S / kPageSize < n_pages;
        const int page = ok ? page_indices[first + S / kPageSize] : 0;
        ok = ok && page >= 0;   // a negative id marks a slot of the list that no page has been assigned to
        sh_pos = ok ? S : -1;
        sh_page = page;
        if (!ok) atomicCAS(status, 0, int(PSA_ERR_BOUNDS));
    }
    __syncthreads();
    const int pos = sh_pos;
    if (pos < 0) return;
    const int vec_per_head = head_dim / 8;   // 16-byte vectors per (token, head)
    // strides are multiples of 8 elements, so element offsets divide into uint4 units exactly
    const int64_t base = (int64_t(sh_page) * stride_page + int64_t(pos % kPageSize) * stride_tok) / 8;
    for (int i = threadIdx.x; i < num_kv_heads * vec_per_head; i += blockDim.x) {
        const int kv = i / vec_per_head, v = i % vec_per_head;
        const int64_t dst = base + int64_t(kv) * (stride_head / 8) + v;
        const int64_t src = (int64_t(s) * num_kv_heads + kv) * vec_per_head + v;
        pool_k[dst] = new_k[src];
        pool_v[dst] = new_v[src];
    }
    __syncthreads();
    if (threadIdx.x == 0) suffix_lens[s] = pos + 1;
}

// Page allocation for the append: a sample whose length is a multiple of the page size needs a fresh page for its
// next token.  One block walks the samples IN ORDER (so that the assignment does not depend on scheduling): the r-th
// sample that needs a page takes free_pages[*free_count - 1 - r], the top of the caller's stack of free page ids, and
// the id goes into the sample's page list at slot S / 16.  When the stack runs out the remaining samples get nothing:
// their slot keeps its negative id, the append kernel then leaves them untouched and reports PSA_ERR_BOUNDS.
// A sample at its planned bound, or whose list has no slot left, asks for nothing (the append kernel reports it).
__global__ void __launch_bounds__(1024)
allocate_pages_kernel(const int32_t *__restrict__ page_indptr, int32_t *__restrict__ page_indices,
                      const int32_t *__restrict__ suffix_lens, const SampleInfo *__restrict__ sample_info, int num_samples,
                      const int32_t *__restrict__ free_pages, int32_t *__restrict__ free_count, int *__restrict__ status)
{
    __shared__ int warp_sums[32];
    __shared__ int base, available;
    if (threadIdx.x == 0) { base = 0; available = max(0, *free_count); }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int s0 = 0; s0 < num_samples; s0 += blockDim.x) {
        const int s = s0 + threadIdx.x;
        int need = 0, slot = 0, first = 0;
        if (s < num_samples) {
            const int S = suffix_lens[s];
            first = page_indptr[s];
            slot = S / kPageSize;
            need = S >= 0 && S < sample_info[s].suf_len_bound && S % kPageSize == 0 && slot < page_indptr[s + 1] - first;
        }
        // rank of this sample among the samples of the chunk that need a page (block-wide exclusive scan)
        int incl = need;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) warp_sums[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            int w = lane < int(blockDim.x >> 5) ? warp_sums[lane] : 0;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, w, o);
                if (lane >= o) w += v;
            }
            warp_sums[lane] = w;   // inclusive sums over warps
        }
        __syncthreads();
        const int rank = base + (warp ? warp_sums[warp - 1] : 0) + incl - need;
        if (need) {
            if (rank < available) page_indices[first + slot] = free_pages[available - 1 - rank];
            else atomicCAS(status, 0, int(PSA_ERR_BOUNDS));   // the stack is empty: the slot stays unassigned
        }
        __syncthreads();
        if (threadIdx.x == 0) base += warp_sums[(blockDim.x >> 5) - 1];
        __syncthreads();
    }
    if (threadIdx.x == 0) *free_count = available - min(available, base);
}

// Debug aid: check a page table against the plan before trusting it to the suffix stage.  One thread per sample:
// 0 <= S_s <= planned bound, enough pages for S_s tokens, every page id inside the pool.  The first violation
// raises PSA_ERR_BOUNDS in the status word; nothing is dereferenced beyond the tables themselves.
__global__ void validate_kernel(const int32_t *__restrict__ page_indptr, const int32_t *__restrict__ page_indices,
                                const int32_t *__restrict__ suffix_lens, const SampleInfo *__restrict__ sample_info,
                                int num_samples, int num_pool_pages, int *__restrict__ status)
{
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= num_samples) return;
    const int S = suffix_lens[s], first = page_indptr[s], n_pages = page_indptr[s + 1] - first;
    bool ok = S >= 0 && S <= sample_info[s].suf_len_bound && first >= 0 && n_pages >= 0 &&
              n_pages >= (S + kPageSize - 1) / kPageSize;
    if (ok)
        for (int i = 0; i < (S + kPageSize - 1) / kPageSize; ++i) {
            const int pg = page_indices[first + i];
            ok = ok && pg >= 0 && pg < num_pool_pages;
        }
    if (!ok) atomicCAS(status, 0, int(PSA_ERR_BOUNDS));
}

}  // namespace

int launch_validate(const int32_t *page_indptr, const int32_t *page_indices, const int32_t *suffix_lens,
                    const SampleInfo *sample_info, int num_samples, int num_pool_pages, int32_t *status, void *stream)
{
    if (num_samples == 0) return 0;
    validate_kernel<<<(num_samples + 127) / 128, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        page_indptr, page_indices, suffix_lens, sample_info, num_samples, num_pool_pages, status);
    return int(cudaGetLastError());
}

int launch_append(const AppendArgs &a, void *stream)
{
    if (a.num_samples == 0) return 0;
    if (a.free_pages != nullptr) {
        allocate_pages_kernel<<<1, 1024, 0, static_cast<cudaStream_t>(stream)>>>(
            a.page_indptr, a.page_indices_rw, a.suffix_lens, a.sample_info, a.num_samples, a.free_pages, a.free_count, a.status);
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return int(e);
    }
    append_kernel<<<a.num_samples, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4 *>(a.new_k), static_cast<const uint4 *>(a.new_v), static_cast<uint4 *>(a.pool_k),
        static_cast<uint4 *>(a.pool_v), a.stride_page, a.stride_head, a.stride_tok, a.page_indptr, a.page_indices,
        a.suffix_lens, a.sample_info, a.num_kv_heads, a.head_dim, a.status);
    return int(cudaGetLastError());
}

}  // namespace psa
