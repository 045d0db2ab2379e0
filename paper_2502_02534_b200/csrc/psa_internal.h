// Internal declarations shared by the planner, the launchers and the C ABI.
// Nothing here is part of the public interface (include/psa.h).
#pragma once

#include <atomic>
#include <cstddef>
#include <cstdint>
#include <string>
#include <vector>

#include "psa.h"

namespace psa {

constexpr int kPageSize = 16;          // tokens per suffix page
constexpr int kPrefixTileKeys = 128;   // keys per tensor-core tile (N of QK^T, K of PV)
constexpr int kPrefixTileRows = 128;   // query rows per softmax warpgroup (M of one MMA)
constexpr int kPrefixRowsPerItem = 256;// two row tiles share the K/V stream of one thread block
constexpr int kStatusWords = 64;       // int32 words reserved at the start of the workspace
// Words of that area besides word 0 (the status).  Within one fused step the suffix grid runs beside the prefix grid
// and the merge grid is ordered behind the SUFFIX grid only, so the prefix grid announces itself and counts its
// blocks off here, and merge warps wait (bounded) until the count reaches launches x blocks.  Neither word is ever
// reset by a kernel (both wrap around together); binding a workspace zeroes them.
constexpr int kPrefixLaunchWord = 8;   // counted prefix launches so far (block 0 adds 1 before it releases the suffix grid)
static_assert(kPrefixLaunchWord % 2 == 0, "the two counters are read as one aligned 64-bit word");
constexpr int kPrefixDoneWord = kPrefixLaunchWord + 1;     // prefix blocks of all those launches that have stored their partial results

// One thread block of the prefix stage: a (prompt, kv head, row group, key range).
struct PrefixItem {
    int32_t first_token;   // index into the packed prefix arrays
    int32_t n_keys;        // > 0
    int32_t kv_head;
    int32_t first_sample;  // sample index of row 0
    int32_t n_rows;        // valid rows, 1..256 (row = local_sample * G + g)
    int32_t partial_row0;  // row of the partial arrays that receives row 0
    int32_t prompt;
    int32_t split;
};
static_assert(sizeof(PrefixItem) == 32, "PrefixItem is read as two int4");

// One thread block of the suffix stage: a (sample, kv head, token chunk).
struct SuffixItem {
    int32_t sample;
    int32_t kv_head;
    int32_t first_token;   // multiple of the chunk size
    int32_t partial_row0;  // row of the partial arrays that receives query head g = 0
};
static_assert(sizeof(SuffixItem) == 16, "SuffixItem is read as one int4");

// Where the merge stage finds the partial results of one sample.  A sample belongs to up to kMaxPrefixLevels
// shared-prefix groups (one per level of a cascade: demonstrations shared by every task, task text shared by the
// task's samples, ...).
// prefix row of (level l, kv head, split j, g): level[l].row0 + kv*level[l].head_stride + j*level[l].split_stride + g
// suffix row of (kv head, chunk c, g):          suf_row0 + (kv*suf_chunks + c)*G + g
constexpr int kMaxPrefixLevels = 4;
struct PrefixLevel {
    int32_t row0;
    int32_t split_stride;
    int32_t splits;
    int32_t head_stride;
};
struct SampleInfo {
    int32_t suf_row0;
    int32_t suf_chunks;     // chunks at the planned suffix length
    int32_t suf_len_bound;  // planned suffix length
    int32_t n_levels;
    PrefixLevel level[kMaxPrefixLevels];
};
static_assert(sizeof(SampleInfo) == 80, "SampleInfo is read as five int4");

struct WorkspaceLayout {
    size_t status_off = 0;       // kStatusWords int32
    size_t prefix_items_off = 0;
    size_t suffix_items_off = 0;
    size_t sample_info_off = 0;
    size_t zero_lens_off = 0;     // int32 [B] of zeros: the suffix lengths of a prefill plan
    size_t lists_end = 0;        // bytes copied by bind_workspace
    size_t partial_lse_off = 0;  // float [num_partial_rows]
    size_t partial_o_off = 0;    // float [num_partial_rows, D]
    size_t total = 0;
};

}  // namespace psa

struct psa_plan {
    psa_config_t cfg{};
    int32_t num_prefixes = 0;
    int32_t num_samples = 0;
    int32_t group = 1;  // G
    int64_t total_prefix_tokens = 0;
    std::vector<int32_t> group_first_sample, group_n_samples, group_token_len, suffix_len_bounds;
    std::vector<psa::PrefixItem> prefix_items;
    std::vector<psa::SuffixItem> suffix_items;
    std::vector<psa::SampleInfo> sample_info;
    int32_t prefix_tiles_per_item = 0;
    int32_t prefix_max_rows_per_item = 0;
    bool causal = false;          // a prefill plan
    int32_t suffix_chunk_tokens = 0;
    int64_t num_partial_rows = 0;
    psa::WorkspaceLayout ws;
    std::vector<unsigned char> upload;  // host image of [0, ws.lists_end)
    int64_t total_suffix_bound_hint() const { int64_t t = 0; for (int32_t v : suffix_len_bounds) t += v; return t; }
};

namespace psa {

// api.cu: records the thread-local message psa_last_error_message returns; returns `status`
psa_status_t set_last_error(psa_status_t status, const std::string &message);

// Kernel attributes (dynamic shared memory size, carve-out preference) are per device: this remembers, for one
// kernel instantiation, on which devices they have been set.  Thread-safe.
struct PerDeviceOnce {
    static constexpr int kMaxDevices = 64;
    std::atomic<unsigned char> done[kMaxDevices];
    PerDeviceOnce() { for (auto &d : done) d.store(0); }
    // Runs `configure()` (returning a CUDA error code, 0 = ok) the first time it is called on the current device.
    template <class F>
    int ensure(F configure)
    {
        int dev = 0;
        if (int e = device_ordinal(&dev)) return e;
        if (dev < 0 || dev >= kMaxDevices) return configure();   // beyond the table: just set them every time
        if (done[dev].load(std::memory_order_acquire)) return 0;
        const int e = configure();                                 // setting twice from two threads is harmless
        if (e == 0) done[dev].store(1, std::memory_order_release);
        return e;
    }
    static int device_ordinal(int *dev);   // api.cu (cudaGetDevice)
};

// plan.cpp
// Shared-prefix group g: `token_len[g]` consecutive tokens of the packed prefix arrays (groups back to back, in
// order) attended by samples [first_sample[g], first_sample[g] + n_samples[g]).
// token_begin == nullptr: group g starts where group g-1 ends.  causal: keys beyond a row's own packed token index
// are masked (prefill: "samples" are the prompt's tokens).
psa_status_t build_plan(const psa_config_t &cfg, int32_t num_groups, const int32_t *first_sample, const int32_t *n_samples,
                        const int32_t *token_len, const int32_t *token_begin, int64_t total_tokens, bool causal,
                        int32_t num_samples, const int32_t *suffix_lens, psa_plan *plan, std::string *err);

// Launchers (one per .cu file). All enqueue on `stream` and return a CUDA error code (0 = ok).
struct PrefixArgs {
    const void *q, *k, *v;
    int64_t stride_tok, stride_head;  // elements
    int64_t total_tokens;
    int32_t num_samples, num_q_heads, num_kv_heads, head_dim;
    float sm_scale;
    const PrefixItem *items;  // device
    int32_t num_items;
    int32_t max_rows_per_item, max_tiles_per_item;  // over all items of the plan
    bool causal = false;  // prefill: row (token) i sees keys up to its own packed token index
    int32_t kernel_choice = 0;   // PSA_PREFIX_KERNEL_*: 0 = by the shape of the items
    bool no_suffix_stage = false;   // the plan has no suffix work at all: the prefix grid has the SMs to itself
    float *partial_o, *partial_lse;  // device
    int32_t *status;                 // device
    int32_t *launch_counter = nullptr, *done_counter = nullptr;   // device; when set: block 0 adds 1 to the first at its start,
                                                                  // every block adds 1 to the second after storing its results
};
int launch_prefix(const PrefixArgs &a, void *stream, std::string *err);
int launch_bounded_wait_selftest(int32_t *status, unsigned long long limit_ns, void *stream);

struct SuffixArgs {
    const void *q, *pool_k, *pool_v;
    int64_t stride_page, stride_head, stride_tok;  // elements
    const int32_t *page_indptr, *page_indices, *suffix_lens;  // device
    int32_t num_q_heads, num_kv_heads, head_dim;
    float sm_scale;
    const SuffixItem *items;      // device
    const SampleInfo *sample_info;// device
    int32_t num_items, chunk_tokens;
    float *partial_o, *partial_lse;
    int32_t *status;
    bool after_prefix = false;  // launched right behind the prefix stage of the same step: may overlap it
};
int launch_suffix(const SuffixArgs &a, void *stream, std::string *err);

struct MergeArgs {
    const SampleInfo *sample_info;  // device
    const int32_t *suffix_lens;     // device
    const float *partial_o, *partial_lse;
    int32_t num_samples, num_q_heads, num_kv_heads, head_dim, chunk_tokens, out_dtype;
    void *out;
    float *lse;
    bool after_stage = false;  // launched right behind a prefix / suffix stage of the same step
    // fused step with both stages: wait until *prefix_done reaches *prefix_launches x prefix_blocks before reading
    // prefix partials
    const int32_t *prefix_counters = nullptr;   // the pair (kPrefixLaunchWord, kPrefixDoneWord), read as one 64-bit word
    int32_t *status = nullptr;
    int32_t prefix_blocks = 0;
};
int launch_merge(const MergeArgs &a, void *stream, std::string *err);

struct AppendArgs {
    const void *new_k, *new_v;   // [B, Hkv, D] bf16, device
    void *pool_k, *pool_v;
    int64_t stride_page, stride_head, stride_tok;  // elements
    const int32_t *page_indptr, *page_indices;
    int32_t *suffix_lens;        // in/out
    const SampleInfo *sample_info;
    int32_t num_samples, num_kv_heads, head_dim;
    int32_t *status;
    // page allocation (all null: every page is already in the lists): a stack of free page ids and its height,
    // and the page lists as writable memory
    const int32_t *free_pages = nullptr;
    int32_t *free_count = nullptr;
    int32_t *page_indices_rw = nullptr;
};
int launch_append(const AppendArgs &a, void *stream);
int launch_validate(const int32_t *page_indptr, const int32_t *page_indices, const int32_t *suffix_lens,
                    const SampleInfo *sample_info, int num_samples, int num_pool_pages, int32_t *status, void *stream);

}  // namespace psa
