// C ABI of the library (include/psa.h): argument checks, workspace carving, stage launches.
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <algorithm>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "psa_internal.h"

namespace {

thread_local std::string g_last_error;

psa_status_t fail(psa_status_t st, const std::string &msg)
{
    g_last_error = msg;
    return st;
}
psa_status_t cuda_fail(cudaError_t e, const char *what)
{
    return fail(PSA_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}
bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// A named range on the host timeline of profilers (NVTX; a pointer check when no tool is attached).
struct TraceRange {
    explicit TraceRange(const char *name) { nvtxRangePushA(name); }
    ~TraceRange() { nvtxRangePop(); }
    TraceRange(const TraceRange &) = delete;
    TraceRange &operator=(const TraceRange &) = delete;
};

struct Carved {
    int32_t *status;
    const psa::PrefixItem *prefix_items;
    const psa::SuffixItem *suffix_items;
    const psa::SampleInfo *sample_info;
    float *partial_lse, *partial_o;
};

psa_status_t carve(const psa_plan_t *plan, void *workspace, size_t bytes, Carved *c)
{
    if (!plan) return fail(PSA_ERR_INVALID_ARG, "null plan");
    if (!workspace) return fail(PSA_ERR_WORKSPACE, "null workspace");
    if (!aligned(workspace, 256)) return fail(PSA_ERR_WORKSPACE, "workspace must be 256-byte aligned");
    if (bytes < plan->ws.total) return fail(PSA_ERR_WORKSPACE, "workspace smaller than psa_plan_workspace_bytes");
    unsigned char *b = static_cast<unsigned char *>(workspace);
    c->status = reinterpret_cast<int32_t *>(b + plan->ws.status_off);
    c->prefix_items = reinterpret_cast<const psa::PrefixItem *>(b + plan->ws.prefix_items_off);
    c->suffix_items = reinterpret_cast<const psa::SuffixItem *>(b + plan->ws.suffix_items_off);
    c->sample_info = reinterpret_cast<const psa::SampleInfo *>(b + plan->ws.sample_info_off);
    c->partial_lse = reinterpret_cast<float *>(b + plan->ws.partial_lse_off);
    c->partial_o = reinterpret_cast<float *>(b + plan->ws.partial_o_off);
    return PSA_OK;
}

}  // namespace

namespace psa {
int PerDeviceOnce::device_ordinal(int *dev) { return int(cudaGetDevice(dev)); }
psa_status_t set_last_error(psa_status_t status, const std::string &message) { return fail(status, message); }
}  // namespace psa

extern "C" {

static psa_status_t create_impl(const psa_config_t *cfg, int32_t num_groups, const int32_t *first_sample,
                                const int32_t *n_samples, const int32_t *token_len, int32_t num_samples,
                                const int32_t *suffix_lens, psa_plan_t **out_plan, const int32_t *token_begin = nullptr,
                                int64_t total_tokens = 0, bool causal = false)
{
    if (!cfg || !out_plan) return fail(PSA_ERR_INVALID_ARG, "null cfg or out_plan");
    *out_plan = nullptr;
    psa_config_t c = *cfg;
    if (c.num_sms == 0) {
        int dev = 0, sms = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return cuda_fail(e, "querying the SM count");
        c.num_sms = sms;
    }
    psa_plan *plan = new (std::nothrow) psa_plan();
    if (!plan) return fail(PSA_ERR_INVALID_ARG, "out of host memory");
    std::string err;
    psa_status_t st = psa::build_plan(c, num_groups, first_sample, n_samples, token_len, token_begin, total_tokens, causal, num_samples,
                                      suffix_lens, plan, &err);
    if (st != PSA_OK) {
        delete plan;
        return fail(st, err);
    }
    *out_plan = plan;
    return PSA_OK;
}

psa_status_t psa_plan_create(const psa_config_t *cfg, int32_t num_prefixes, const int32_t *prefix_lens,
                             const int32_t *n_samples_per_prefix, const int32_t *suffix_lens, psa_plan_t **out_plan)
{
    if (num_prefixes < 0 || (num_prefixes > 0 && !n_samples_per_prefix)) return fail(PSA_ERR_INVALID_ARG, "null length arrays");
    // prompt p is the prefix group of the next n_samples_per_prefix[p] samples
    std::vector<int32_t> first(static_cast<size_t>(num_prefixes), 0);
    int64_t B = 0;
    for (int32_t p = 0; p < num_prefixes; ++p) {
        if (n_samples_per_prefix[p] < 0) return fail(PSA_ERR_INVALID_ARG, "negative length or sample count");
        first[size_t(p)] = int32_t(B);
        B += n_samples_per_prefix[p];
        if (B > (1 << 24)) return fail(PSA_ERR_UNSUPPORTED, "problem too large");
    }
    return create_impl(cfg, num_prefixes, first.data(), n_samples_per_prefix, prefix_lens, int32_t(B), suffix_lens, out_plan);
}

psa_status_t psa_plan_create_cascade(const psa_config_t *cfg, int32_t num_groups, const int32_t *group_first_sample,
                                     const int32_t *group_n_samples, const int32_t *group_token_len, int32_t num_samples,
                                     const int32_t *suffix_lens, psa_plan_t **out_plan)
{
    return create_impl(cfg, num_groups, group_first_sample, group_n_samples, group_token_len, num_samples, suffix_lens, out_plan);
}

psa_status_t psa_plan_create_prefill(const psa_config_t *cfg, int32_t num_prompts, const int32_t *prompt_lens,
                                     psa_plan_t **out_plan)
{
    if (!cfg || !out_plan) return fail(PSA_ERR_INVALID_ARG, "null cfg or out_plan");
    if (num_prompts < 0 || (num_prompts > 0 && !prompt_lens)) return fail(PSA_ERR_INVALID_ARG, "null prompt_lens");
    if (cfg->num_kv_heads <= 0 || cfg->num_q_heads <= 0 || cfg->num_q_heads % cfg->num_kv_heads)
        return fail(PSA_ERR_INVALID_ARG, "num_q_heads must be a positive multiple of num_kv_heads");
    const int G = cfg->num_q_heads / cfg->num_kv_heads;
    if (G > 8) return fail(PSA_ERR_UNSUPPORTED, "group size must be 1, 2, 4 or 8");
    // Every query token is a "sample" without a suffix.  The tokens of one row group (256 query rows = 256 / G
    // tokens) form a prefix group whose keys are the prompt's tokens up to the group's last token; the causal
    // mask inside the kernel trims the diagonal.
    const int tokens_per_group = psa::kPrefixRowsPerItem / G;
    std::vector<int32_t> first, count, len, begin;
    int64_t total = 0;
    for (int32_t p = 0; p < num_prompts; ++p) {
        if (prompt_lens[p] < 0) return fail(PSA_ERR_INVALID_ARG, "negative prompt length");
        for (int64_t t0 = 0; t0 < prompt_lens[p]; t0 += tokens_per_group) {
            const int64_t n = std::min<int64_t>(tokens_per_group, prompt_lens[p] - t0);
            first.push_back(int32_t(total + t0));
            count.push_back(int32_t(n));
            len.push_back(int32_t(t0 + n));
            begin.push_back(int32_t(total));
        }
        total += prompt_lens[p];
        if (total > (1 << 24)) return fail(PSA_ERR_UNSUPPORTED, "problem too large");
    }
    std::vector<int32_t> zero_suffix(size_t(total), 0);
    psa_config_t c = *cfg;
    if (c.prefix_rows_per_item == 0) c.prefix_rows_per_item = psa::kPrefixRowsPerItem;
    return create_impl(&c, int32_t(first.size()), first.data(), count.data(), len.data(), int32_t(total), zero_suffix.data(),
                       out_plan, begin.data(), total, true);
}

psa_status_t psa_plan_destroy(psa_plan_t *plan)
{
    delete plan;
    return PSA_OK;
}

psa_status_t psa_plan_get_info(const psa_plan_t *plan, psa_plan_info_t *info)
{
    if (!plan || !info) return fail(PSA_ERR_INVALID_ARG, "null plan or info");
    info->num_sms = plan->cfg.num_sms;
    info->num_samples = plan->num_samples;
    info->num_prefix_items = int32_t(plan->prefix_items.size());
    info->num_suffix_items = int32_t(plan->suffix_items.size());
    info->prefix_tile_keys = psa::kPrefixTileKeys;
    info->prefix_tiles_per_item = plan->prefix_tiles_per_item;
    info->suffix_chunk_tokens = plan->suffix_chunk_tokens;
    info->kernel_launches = (plan->prefix_items.empty() ? 0 : 1) + (plan->suffix_items.empty() ? 0 : 1) +
                            (plan->num_samples > 0 ? 1 : 0);
    info->num_partial_rows = plan->num_partial_rows;
    return PSA_OK;
}

size_t psa_plan_workspace_bytes(const psa_plan_t *plan) { return plan ? plan->ws.total : 0; }

psa_status_t psa_plan_bind_workspace(const psa_plan_t *plan, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    Carved c;
    psa_status_t st = carve(plan, workspace, workspace_bytes, &c);
    if (st != PSA_OK) return st;
    cudaError_t e = cudaMemcpyAsync(workspace, plan->upload.data(), plan->upload.size(), cudaMemcpyHostToDevice,
                                    static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(e, "uploading the work lists");
    return PSA_OK;
}

int32_t psa_plan_prefix_items(const psa_plan_t *plan, int32_t *items8)
{
    if (!plan) return -1;
    if (items8 && !plan->prefix_items.empty())
        std::memcpy(items8, plan->prefix_items.data(), sizeof(psa::PrefixItem) * plan->prefix_items.size());
    return int32_t(plan->prefix_items.size());
}

int32_t psa_plan_suffix_items(const psa_plan_t *plan, int32_t *items4)
{
    if (!plan) return -1;
    if (items4 && !plan->suffix_items.empty())
        std::memcpy(items4, plan->suffix_items.data(), sizeof(psa::SuffixItem) * plan->suffix_items.size());
    return int32_t(plan->suffix_items.size());
}

static psa_status_t prefix_impl(const psa_plan_t *plan, const void *q, const void *prefix_k, const void *prefix_v,
                                const int64_t prefix_strides[2], void *workspace, size_t workspace_bytes, void *cuda_stream,
                                bool count_blocks)
{
    TraceRange trace("psa prefix stage");
    Carved c;
    psa_status_t st = carve(plan, workspace, workspace_bytes, &c);
    if (st != PSA_OK) return st;
    if (plan->prefix_items.empty()) return PSA_OK;
    if (!q || !prefix_k || !prefix_v || !prefix_strides) return fail(PSA_ERR_INVALID_ARG, "null q / prefix_k / prefix_v / prefix_strides");
    if (!aligned(q, 16) || !aligned(prefix_k, 16) || !aligned(prefix_v, 16))
        return fail(PSA_ERR_INVALID_ARG, "q, prefix_k and prefix_v must be 16-byte aligned");
    if (prefix_strides[0] <= 0 || prefix_strides[1] <= 0 || prefix_strides[0] % 8 || prefix_strides[1] % 8)
        return fail(PSA_ERR_INVALID_ARG, "prefix strides must be positive multiples of 8 elements");
    psa::PrefixArgs a{};
    a.q = q; a.k = prefix_k; a.v = prefix_v;
    a.stride_tok = prefix_strides[0]; a.stride_head = prefix_strides[1];
    a.total_tokens = plan->total_prefix_tokens;
    a.num_samples = plan->num_samples;
    a.num_q_heads = plan->cfg.num_q_heads; a.num_kv_heads = plan->cfg.num_kv_heads; a.head_dim = plan->cfg.head_dim;
    a.sm_scale = plan->cfg.sm_scale;
    a.items = c.prefix_items; a.num_items = int32_t(plan->prefix_items.size());
    a.max_rows_per_item = plan->prefix_max_rows_per_item; a.max_tiles_per_item = plan->prefix_tiles_per_item;
    a.causal = plan->causal;
    a.kernel_choice = plan->cfg.prefix_kernel;
    a.no_suffix_stage = plan->suffix_items.empty();
    a.partial_o = c.partial_o; a.partial_lse = c.partial_lse; a.status = c.status;
    a.launch_counter = count_blocks ? c.status + psa::kPrefixLaunchWord : nullptr;
    a.done_counter = count_blocks ? c.status + psa::kPrefixDoneWord : nullptr;
    std::string err;
    if (psa::launch_prefix(a, cuda_stream, &err) != 0) return fail(PSA_ERR_CUDA, err);
    return PSA_OK;
}

psa_status_t psa_decode_prefix(const psa_plan_t *plan, const void *q, const void *prefix_k, const void *prefix_v,
                               const int64_t prefix_strides[2], void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    return prefix_impl(plan, q, prefix_k, prefix_v, prefix_strides, workspace, workspace_bytes, cuda_stream, false);
}

static psa_status_t suffix_impl(const psa_plan_t *plan, const void *q, const void *suffix_k_pool, const void *suffix_v_pool,
                                const int64_t pool_strides[3], const int32_t *page_indptr, const int32_t *page_indices,
                                const int32_t *suffix_lens, void *workspace, size_t workspace_bytes, void *cuda_stream,
                                bool after_prefix)
{
    TraceRange trace("psa suffix stage");
    Carved c;
    psa_status_t st = carve(plan, workspace, workspace_bytes, &c);
    if (st != PSA_OK) return st;
    if (plan->suffix_items.empty()) return PSA_OK;
    if (!q || !suffix_k_pool || !suffix_v_pool || !pool_strides || !page_indptr || !page_indices || !suffix_lens)
        return fail(PSA_ERR_INVALID_ARG, "null suffix argument");
    if (!aligned(q, 16) || !aligned(suffix_k_pool, 16) || !aligned(suffix_v_pool, 16))
        return fail(PSA_ERR_INVALID_ARG, "q and the pools must be 16-byte aligned");
    for (int i = 0; i < 3; ++i)
        if (pool_strides[i] <= 0 || pool_strides[i] % 8) return fail(PSA_ERR_INVALID_ARG, "pool strides must be positive multiples of 8 elements");
    psa::SuffixArgs a{};
    a.q = q; a.pool_k = suffix_k_pool; a.pool_v = suffix_v_pool;
    a.stride_page = pool_strides[0]; a.stride_head = pool_strides[1]; a.stride_tok = pool_strides[2];
    a.page_indptr = page_indptr; a.page_indices = page_indices; a.suffix_lens = suffix_lens;
    a.num_q_heads = plan->cfg.num_q_heads; a.num_kv_heads = plan->cfg.num_kv_heads; a.head_dim = plan->cfg.head_dim;
    a.sm_scale = plan->cfg.sm_scale;
    a.items = c.suffix_items; a.sample_info = c.sample_info;
    a.num_items = int32_t(plan->suffix_items.size()); a.chunk_tokens = plan->suffix_chunk_tokens;
    a.partial_o = c.partial_o; a.partial_lse = c.partial_lse; a.status = c.status;
    a.after_prefix = after_prefix;
    std::string err;
    if (psa::launch_suffix(a, cuda_stream, &err) != 0) return fail(PSA_ERR_CUDA, err);
    return PSA_OK;
}

psa_status_t psa_decode_suffix(const psa_plan_t *plan, const void *q, const void *suffix_k_pool, const void *suffix_v_pool,
                               const int64_t pool_strides[3], const int32_t *page_indptr, const int32_t *page_indices,
                               const int32_t *suffix_lens, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    return suffix_impl(plan, q, suffix_k_pool, suffix_v_pool, pool_strides, page_indptr, page_indices, suffix_lens, workspace,
                       workspace_bytes, cuda_stream, false);
}

static psa_status_t merge_impl(const psa_plan_t *plan, const int32_t *suffix_lens, void *out, float *lse, void *workspace,
                               size_t workspace_bytes, void *cuda_stream, bool after_stage, bool wait_for_prefix_count = false)
{
    TraceRange trace("psa merge stage");
    Carved c;
    psa_status_t st = carve(plan, workspace, workspace_bytes, &c);
    if (st != PSA_OK) return st;
    if (plan->num_samples == 0) return PSA_OK;
    if (!suffix_lens || !out || !lse) return fail(PSA_ERR_INVALID_ARG, "null suffix_lens / out / lse");
    if (!aligned(out, 16) || !aligned(lse, 4)) return fail(PSA_ERR_INVALID_ARG, "out must be 16-byte aligned");
    psa::MergeArgs a{};
    a.sample_info = c.sample_info; a.suffix_lens = suffix_lens;
    a.partial_o = c.partial_o; a.partial_lse = c.partial_lse;
    a.num_samples = plan->num_samples;
    a.num_q_heads = plan->cfg.num_q_heads; a.num_kv_heads = plan->cfg.num_kv_heads; a.head_dim = plan->cfg.head_dim;
    a.chunk_tokens = plan->suffix_chunk_tokens; a.out_dtype = plan->cfg.out_dtype;
    a.out = out; a.lse = lse;
    a.after_stage = after_stage;
    if (wait_for_prefix_count) {
        a.prefix_counters = c.status + psa::kPrefixLaunchWord;
        a.status = c.status;
        a.prefix_blocks = int32_t(plan->prefix_items.size());
    }
    std::string err;
    if (psa::launch_merge(a, cuda_stream, &err) != 0) return fail(PSA_ERR_CUDA, err);
    return PSA_OK;
}

psa_status_t psa_decode_merge(const psa_plan_t *plan, const int32_t *suffix_lens, void *out, float *lse, void *workspace,
                              size_t workspace_bytes, void *cuda_stream)
{
    return merge_impl(plan, suffix_lens, out, lse, workspace, workspace_bytes, cuda_stream, false);
}

psa_status_t psa_prefill(const psa_plan_t *plan, const void *q, const void *k, const void *v, const int64_t kv_strides[2],
                         void *out, float *lse, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    Carved c;
    psa_status_t st = carve(plan, workspace, workspace_bytes, &c);
    if (st != PSA_OK) return st;
    if (!plan->causal) return fail(PSA_ERR_INVALID_ARG, "psa_prefill needs a plan made by psa_plan_create_prefill");
    st = psa_decode_prefix(plan, q, k, v, kv_strides, workspace, workspace_bytes, cuda_stream);
    if (st != PSA_OK) return st;
    const int32_t *zero_lens = reinterpret_cast<const int32_t *>(static_cast<unsigned char *>(workspace) + plan->ws.zero_lens_off);
    return merge_impl(plan, zero_lens, out, lse, workspace, workspace_bytes, cuda_stream, !plan->prefix_items.empty());
}

psa_status_t psa_decode(const psa_plan_t *plan, const void *q, const void *prefix_k, const void *prefix_v,
                        const int64_t prefix_strides[2], const void *suffix_k_pool, const void *suffix_v_pool,
                        const int64_t pool_strides[3], const int32_t *page_indptr, const int32_t *page_indices,
                        const int32_t *suffix_lens, void *out, float *lse, void *workspace, size_t workspace_bytes,
                        void *cuda_stream)
{
    if (!plan) return fail(PSA_ERR_INVALID_ARG, "null plan");
    TraceRange trace("psa_decode");
    // The suffix stage is independent of the prefix stage: launched as its programmatic dependent it runs
    // beside it.  The merge stage needs both, but stream order (and the programmatic dependency) only puts it
    // behind the suffix grid, so with both stages present the prefix blocks count themselves off in the workspace
    // and the merge stage waits for the count.
    const bool have_prefix = !plan->prefix_items.empty(), have_suffix = !plan->suffix_items.empty();
    psa_status_t st = prefix_impl(plan, q, prefix_k, prefix_v, prefix_strides, workspace, workspace_bytes, cuda_stream,
                                  have_prefix && have_suffix);
    if (st != PSA_OK) return st;
    st = suffix_impl(plan, q, suffix_k_pool, suffix_v_pool, pool_strides, page_indptr, page_indices, suffix_lens, workspace,
                     workspace_bytes, cuda_stream, have_prefix);
    if (st != PSA_OK) return st;
    return merge_impl(plan, suffix_lens, out, lse, workspace, workspace_bytes, cuda_stream, have_prefix || have_suffix,
                      have_prefix && have_suffix);
}

namespace {
struct HostStaging {
    size_t q, pk, pv, sk, sv, indptr, indices, lens, out, lse, total;
};
HostStaging staging_layout(const psa_plan_t *plan, int64_t tokens, int64_t pages, int64_t n_indices)
{
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    const size_t Hq = plan->cfg.num_q_heads, Hkv = plan->cfg.num_kv_heads, D = plan->cfg.head_dim, B = plan->num_samples;
    HostStaging s{};
    size_t off = 0;
    s.q = off;       off = up(off + B * Hq * D * 2);
    s.pk = off;      off = up(off + size_t(tokens) * Hkv * D * 2);
    s.pv = off;      off = up(off + size_t(tokens) * Hkv * D * 2);
    s.sk = off;      off = up(off + size_t(pages) * Hkv * psa::kPageSize * D * 2);
    s.sv = off;      off = up(off + size_t(pages) * Hkv * psa::kPageSize * D * 2);
    s.indptr = off;  off = up(off + (B + 1) * 4);
    s.indices = off; off = up(off + size_t(n_indices) * 4);
    s.lens = off;    off = up(off + B * 4);
    s.out = off;     off = up(off + B * Hq * D * (plan->cfg.out_dtype == PSA_OUT_F32 ? 4 : 2));
    s.lse = off;     off = up(off + B * Hq * 4);
    s.total = off;
    return s;
}
}  // namespace

size_t psa_decode_host_staging_bytes(const psa_plan_t *plan, int64_t num_prefix_tokens, int64_t num_pool_pages,
                                     int64_t num_page_indices)
{
    if (!plan || num_prefix_tokens < 0 || num_pool_pages < 0 || num_page_indices < 0) return 0;
    return staging_layout(plan, num_prefix_tokens, num_pool_pages, num_page_indices).total;
}

psa_status_t psa_decode_host(const psa_plan_t *plan, const void *q_host, const void *prefix_k_host, const void *prefix_v_host,
                             int64_t num_prefix_tokens, const void *suffix_k_pool_host, const void *suffix_v_pool_host,
                             int64_t num_pool_pages, const int32_t *page_indptr_host, const int32_t *page_indices_host,
                             int64_t num_page_indices, const int32_t *suffix_lens_host, void *out_host, float *lse_host,
                             void *staging, size_t staging_bytes, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!plan) return fail(PSA_ERR_INVALID_ARG, "null plan");
    if (num_prefix_tokens < plan->total_prefix_tokens) return fail(PSA_ERR_INVALID_ARG, "num_prefix_tokens smaller than the plan's prompts");
    if (num_pool_pages < 0 || num_page_indices < 0) return fail(PSA_ERR_INVALID_ARG, "negative sizes");
    if (!staging || !aligned(staging, 256)) return fail(PSA_ERR_WORKSPACE, "staging must be a 256-byte aligned device buffer");
    const HostStaging s = staging_layout(plan, num_prefix_tokens, num_pool_pages, num_page_indices);
    if (staging_bytes < s.total) return fail(PSA_ERR_WORKSPACE, "staging smaller than psa_decode_host_staging_bytes");
    if (plan->num_samples == 0) return PSA_OK;
    if (!q_host || !page_indptr_host || !suffix_lens_host || !out_host || !lse_host) return fail(PSA_ERR_INVALID_ARG, "null host buffer");
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    unsigned char *b = static_cast<unsigned char *>(staging);
    const size_t Hq = plan->cfg.num_q_heads, Hkv = plan->cfg.num_kv_heads, D = plan->cfg.head_dim, B = plan->num_samples;
    auto h2d = [&](size_t off, const void *src, size_t bytes) -> cudaError_t {
        if (bytes == 0) return cudaSuccess;
        if (!src) return cudaErrorInvalidValue;
        return cudaMemcpyAsync(b + off, src, bytes, cudaMemcpyHostToDevice, st);
    };
    cudaError_t e = h2d(s.q, q_host, B * Hq * D * 2);
    if (e == cudaSuccess) e = h2d(s.pk, prefix_k_host, size_t(num_prefix_tokens) * Hkv * D * 2);
    if (e == cudaSuccess) e = h2d(s.pv, prefix_v_host, size_t(num_prefix_tokens) * Hkv * D * 2);
    if (e == cudaSuccess) e = h2d(s.sk, suffix_k_pool_host, size_t(num_pool_pages) * Hkv * psa::kPageSize * D * 2);
    if (e == cudaSuccess) e = h2d(s.sv, suffix_v_pool_host, size_t(num_pool_pages) * Hkv * psa::kPageSize * D * 2);
    if (e == cudaSuccess) e = h2d(s.indptr, page_indptr_host, (B + 1) * 4);
    if (e == cudaSuccess) e = h2d(s.indices, page_indices_host, size_t(num_page_indices) * 4);
    if (e == cudaSuccess) e = h2d(s.lens, suffix_lens_host, B * 4);
    if (e != cudaSuccess) return cuda_fail(e, "host to device copy");
    const int64_t pst[2] = {int64_t(Hkv * D), int64_t(D)};
    const int64_t qst[3] = {int64_t(Hkv * psa::kPageSize * D), int64_t(psa::kPageSize * D), int64_t(D)};
    psa_status_t rc = psa_decode(plan, b + s.q, b + s.pk, b + s.pv, pst, b + s.sk, b + s.sv, qst,
                                 reinterpret_cast<const int32_t *>(b + s.indptr), reinterpret_cast<const int32_t *>(b + s.indices),
                                 reinterpret_cast<const int32_t *>(b + s.lens), b + s.out, reinterpret_cast<float *>(b + s.lse),
                                 workspace, workspace_bytes, cuda_stream);
    if (rc != PSA_OK) return rc;
    e = cudaMemcpyAsync(out_host, b + s.out, B * Hq * D * (plan->cfg.out_dtype == PSA_OUT_F32 ? 4 : 2), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(lse_host, b + s.lse, B * Hq * 4, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(e, "device to host copy");
    return PSA_OK;
}

psa_status_t psa_check_status(const psa_plan_t *plan, void *workspace, void *cuda_stream)
{
    if (!plan || !workspace) return fail(PSA_ERR_INVALID_ARG, "null plan or workspace");
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int32_t word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, workspace, sizeof word, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e, "reading the status word");
    if (word != 0) {
        // The whole status area is cleared, the two prefix counters (launches, blocks done) with it.  That is safe
        // because the stream is idle here (synchronised above) and the merge stage only compares
        // launches x blocks with blocks done: both restart from zero together.
        e = cudaMemsetAsync(workspace, 0, sizeof(int32_t) * psa::kStatusWords, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) return cuda_fail(e, "clearing the status word");
        return fail(psa_status_t(word), "device-side status word was set");
    }
    return PSA_OK;
}

static psa_status_t append_impl(const psa_plan_t *plan, const void *new_k, const void *new_v, void *suffix_k_pool,
                                void *suffix_v_pool, const int64_t pool_strides[3], const int32_t *page_indptr,
                                const int32_t *page_indices, int32_t *suffix_lens, void *workspace, size_t workspace_bytes,
                                void *cuda_stream, const int32_t *free_pages, int32_t *free_count, int32_t *page_indices_rw);

psa_status_t psa_append_kv(const psa_plan_t *plan, const void *new_k, const void *new_v, void *suffix_k_pool,
                           void *suffix_v_pool, const int64_t pool_strides[3], const int32_t *page_indptr,
                           const int32_t *page_indices, int32_t *suffix_lens, void *workspace, size_t workspace_bytes,
                           void *cuda_stream)
{
    return append_impl(plan, new_k, new_v, suffix_k_pool, suffix_v_pool, pool_strides, page_indptr, page_indices, suffix_lens,
                       workspace, workspace_bytes, cuda_stream, nullptr, nullptr, nullptr);
}

psa_status_t psa_append_kv_alloc(const psa_plan_t *plan, const void *new_k, const void *new_v, void *suffix_k_pool,
                                 void *suffix_v_pool, const int64_t pool_strides[3], const int32_t *page_indptr,
                                 int32_t *page_indices, int32_t *suffix_lens, const int32_t *free_pages, int32_t *free_count,
                                 void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!free_pages || !free_count) return fail(PSA_ERR_INVALID_ARG, "null free_pages / free_count");
    return append_impl(plan, new_k, new_v, suffix_k_pool, suffix_v_pool, pool_strides, page_indptr, page_indices, suffix_lens,
                       workspace, workspace_bytes, cuda_stream, free_pages, free_count, page_indices);
}

static psa_status_t append_impl(const psa_plan_t *plan, const void *new_k, const void *new_v, void *suffix_k_pool,
                                void *suffix_v_pool, const int64_t pool_strides[3], const int32_t *page_indptr,
                                const int32_t *page_indices, int32_t *suffix_lens, void *workspace, size_t workspace_bytes,
                                void *cuda_stream, const int32_t *free_pages, int32_t *free_count, int32_t *page_indices_rw)
{
    Carved c;
    psa_status_t st = carve(plan, workspace, workspace_bytes, &c);
    if (st != PSA_OK) return st;
    if (plan->num_samples == 0) return PSA_OK;
    if (!new_k || !new_v || !suffix_k_pool || !suffix_v_pool || !pool_strides || !page_indptr || !page_indices || !suffix_lens)
        return fail(PSA_ERR_INVALID_ARG, "null append argument");
    if (!aligned(new_k, 16) || !aligned(new_v, 16) || !aligned(suffix_k_pool, 16) || !aligned(suffix_v_pool, 16))
        return fail(PSA_ERR_INVALID_ARG, "new_k, new_v and the pools must be 16-byte aligned");
    for (int i = 0; i < 3; ++i)
        if (pool_strides[i] <= 0 || pool_strides[i] % 8) return fail(PSA_ERR_INVALID_ARG, "pool strides must be positive multiples of 8 elements");
    psa::AppendArgs a{};
    a.new_k = new_k; a.new_v = new_v; a.pool_k = suffix_k_pool; a.pool_v = suffix_v_pool;
    a.stride_page = pool_strides[0]; a.stride_head = pool_strides[1]; a.stride_tok = pool_strides[2];
    a.page_indptr = page_indptr; a.page_indices = page_indices; a.suffix_lens = suffix_lens;
    a.sample_info = c.sample_info;
    a.num_samples = plan->num_samples; a.num_kv_heads = plan->cfg.num_kv_heads; a.head_dim = plan->cfg.head_dim;
    a.status = c.status;
    a.free_pages = free_pages; a.free_count = free_count; a.page_indices_rw = page_indices_rw;
    const int rc = psa::launch_append(a, cuda_stream);
    if (rc != 0) return cuda_fail(cudaError_t(rc), "append launch");
    return PSA_OK;
}

psa_status_t psa_validate_page_table(const psa_plan_t *plan, const int32_t *page_indptr, const int32_t *page_indices,
                                     const int32_t *suffix_lens, int64_t num_pool_pages, void *workspace,
                                     size_t workspace_bytes, void *cuda_stream)
{
    Carved c;
    psa_status_t st = carve(plan, workspace, workspace_bytes, &c);
    if (st != PSA_OK) return st;
    if (!page_indptr || !suffix_lens || (!page_indices && plan->total_suffix_bound_hint() > 0))
        return fail(PSA_ERR_INVALID_ARG, "null page table");
    if (num_pool_pages < 0 || num_pool_pages > (int64_t(1) << 31) - 1) return fail(PSA_ERR_INVALID_ARG, "num_pool_pages out of range");
    const int rc = psa::launch_validate(page_indptr, page_indices, suffix_lens, c.sample_info, plan->num_samples,
                                        int(num_pool_pages), c.status, cuda_stream);
    if (rc != 0) return cuda_fail(cudaError_t(rc), "validate launch");
    return PSA_OK;
}

psa_status_t psa_selftest_bounded_wait(void *workspace, size_t workspace_bytes, uint64_t limit_ns, void *cuda_stream)
{
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < sizeof(int32_t) * psa::kStatusWords)
        return fail(PSA_ERR_WORKSPACE, "workspace must be a 256-byte aligned device buffer of at least 256 bytes");
    if (limit_ns == 0 || limit_ns > 1000000000ull) return fail(PSA_ERR_INVALID_ARG, "limit_ns must be in (0, 1e9]");
    const int rc = psa::launch_bounded_wait_selftest(static_cast<int32_t *>(workspace), limit_ns, cuda_stream);
    if (rc != 0) return cuda_fail(cudaError_t(rc), "self-test launch");
    return PSA_OK;
}

const char *psa_status_string(psa_status_t status)
{
    switch (status) {
        case PSA_OK: return "ok";
        case PSA_ERR_INVALID_ARG: return "invalid argument";
        case PSA_ERR_UNSUPPORTED: return "unsupported shape or dtype";
        case PSA_ERR_WORKSPACE: return "workspace missing, too small or misaligned";
        case PSA_ERR_CUDA: return "CUDA call failed";
        case PSA_ERR_TIMEOUT: return "device-side bounded wait expired";
        case PSA_ERR_BOUNDS: return "device-side index out of bounds";
    }
    return "unknown status";
}

const char *psa_last_error_message(void) { return g_last_error.c_str(); }

int32_t psa_version(void) { return 100; }

}  // extern "C"
