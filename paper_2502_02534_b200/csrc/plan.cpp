// Planner: cuts the prefix and suffix stages into work items that fill every SM.
// Host only, integer arithmetic only.
//
// The shape it plans for is the paper's parallel-sampling step (Algorithm 1): a few
// prompts, each sampled N_p times, so that the N_p * G query rows of a KV head share
// the prompt's K/V.  Prefix work is counted in (key tile x row group) steps, suffix
// work in tokens; both cost models charge a fixed start-up per item so that very
// small pieces are not preferred.
#include <algorithm>
#include <cstring>
#include <functional>
#include <limits>
#include <queue>

#include "psa_internal.h"

namespace psa {
namespace {

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Prefix: every (group, kv head, row group) streams ceil(L / 128) key tiles; with at most T tiles per item a
// group of `tiles` tiles is cut into ceil(tiles / T) items.  Items are dispatched longest first to the SMs, so
// the stage takes about max(longest item, sum of items / SMs); every split also costs a partial result per row
// (4*D bytes written, read again by the merge stage).  Costs are in tile steps of a one-row-tile block (~1.5 us);
// a step of a two-row-tile block counts 1.3.  In a step that also has a suffix stage the two grids run side by side
// and the suffix stage (HBM-bound, the longer one) wants every SM, so the SM time the prefix items take is charged
// once more at `sm_time_weight` (measured on 32 samples x 4096 + U[0,1024] tokens: 88 items of 3 tiles give a 22.2 us
// step, 128 items of 2 tiles 23.4 us, although the prefix stage alone is faster with 128).  Pick the T with the
// smallest estimate, larger T on ties.
//
// Blocks of two row tiles own their SM (no suffix block fits beside them) and work in the tensor-bound regime, where
// they need little of the HBM bandwidth.  There the whole step is estimated instead: while the prefix items run,
// the suffix stage streams on the SMs they leave free, at up to 72 GB/s per SM (measured: 84 free SMs sustain
// 6.1 TB/s) and at most what the prefix stage leaves of 6.4 TB/s; afterwards it has the machine to itself.  Few long
// items then beat many short ones: 2048 rows x 8192 keys x 8 heads beside 2.1 GB of suffix K/V take 338 us as 64
// items of 64 tiles against 385 us as 128 items of 32 tiles.
int choose_prefix_tiles_per_item(const std::vector<int64_t> &tiles, const std::vector<int64_t> &groups,
                                 const std::vector<int64_t> &partial_rows_per_split, double step_weight, int head_dim, int num_sms,
                                 double sm_time_weight, bool owns_sm, double prefix_bytes, double suffix_bytes)
{
    int64_t max_tiles = 0;
    for (int64_t t : tiles) max_tiles = std::max(max_tiles, t);
    if (max_tiles == 0) return 1;
    const double overhead = 2.0;                                   // prologue + epilogue of one item, in tile steps
    const double steps_per_partial_row = double(head_dim) * 8.0 / 4.0e12 / 1.5e-6;   // bytes / (4 TB/s) / step time
    double best_cost = std::numeric_limits<double>::infinity();
    int best_T = 1;
    for (int64_t T = 1; T <= max_tiles; ++T) {
        double sum = 0.0, longest = 0.0, partial = 0.0, items = 0.0;
        for (size_t p = 0; p < tiles.size(); ++p) {
            if (tiles[p] == 0) continue;
            const int64_t splits = ceil_div(tiles[p], T);
            const double len = step_weight * double(ceil_div(tiles[p], splits)) + overhead;
            sum += double(groups[p] * splits) * len;
            items += double(groups[p] * splits);
            longest = std::max(longest, len);
            partial += double(partial_rows_per_split[p] * splits) * steps_per_partial_row;
        }
        // Blocks that own their SM (two row tiles, or a step without a suffix stage) run in waves of num_sms: the stage
        // lasts as long as the busiest SM when the items are dealt out longest first, and 144 items of 17 steps beat
        // 160 items of 16 (measured on 2 x 128 rows x 16384 keys x 8 heads: 21.3 against 33.6 us).
        double stage = std::max(longest, 1.1 * sum / num_sms);
        if (owns_sm || sm_time_weight == 0.0) {
            std::vector<double> lens;
            for (size_t p = 0; p < tiles.size(); ++p) {
                if (tiles[p] == 0) continue;
                const int64_t splits = ceil_div(tiles[p], T);
                const int64_t per = tiles[p] / splits, extra = tiles[p] % splits;
                for (int64_t j = 0; j < splits; ++j)
                    lens.insert(lens.end(), size_t(groups[p]), step_weight * double(per + (j < extra ? 1 : 0)) + overhead);
            }
            std::sort(lens.begin(), lens.end(), std::greater<double>());
            std::priority_queue<double, std::vector<double>, std::greater<double>> sms;   // finish time of every SM
            for (int i = 0; i < num_sms; ++i) sms.push(0.0);
            double makespan = 0.0;
            for (double len : lens) {
                const double t = sms.top() + len;
                sms.pop();
                sms.push(t);
                makespan = std::max(makespan, t);
            }
            stage = makespan;
        }
        double cost = stage + partial;
        if (owns_sm && suffix_bytes > 0.0) {
            const double step_us = 1.5, hbm = 6.4e6 /* bytes per us */, per_sm = 7.2e4;
            const double t_prefix = stage * step_us;
            const double free_sms = std::max(0.0, double(num_sms) - items);
            const double rate = std::max(0.0, std::min(hbm - prefix_bytes / t_prefix, free_sms * per_sm));
            cost += std::max(0.0, suffix_bytes - rate * t_prefix) / hbm / step_us;
        } else {
            cost += sm_time_weight * sum / num_sms;
        }
        if (cost <= best_cost) { best_cost = cost; best_T = int(T); }
    }
    return best_T;
}

// Suffix: items are dispatched greedily (longest first) to 2 resident blocks per SM and the stage is bound by HBM
// as a whole, not block by block: a block alone can stream about three times its fair share of the bandwidth, so
// one long item is no tail as long as it needs less than a third of the stage.  Estimate, in tokens streamed by
// one slot at its fair share:
//     max( (sum of tokens + 384 per item) / min(slots, items),  longest item / 3 + 384 ).
// The 384 is what a block spends finding its pages (three dependent loads) and combining its warps, expressed
// in tokens.  Measured on B200: 64 samples x U[0,2048] tokens take 41.9 us as whole-sample items (0.98 of the
// copy bandwidth), 45.4 us in 1024-token chunks, 48.7 us in 512-token chunks; 32 samples x U[0,1024] tokens beside a
// 4096-token prefix: the step takes 21.3 us with 896-token chunks, 21.7 with 768, 22.1 with 1024, 22.8 with 512.
int choose_suffix_chunk(const int32_t *lens, int n, int num_kv_heads, int num_sms)
{
    const double overhead = 384.0;
    const double slots = 2.0 * num_sms;
    double best_cost = std::numeric_limits<double>::infinity();
    int best = 64;
    // candidates: every 64 tokens up to 1024, every 256 up to 4096, every 1024 up to 8192
    for (int C = 64; C <= 8192; C += (C < 1024 ? 64 : (C < 4096 ? 256 : 1024))) {
        double sum = 0.0, items = 0.0;
        int64_t longest = 0;
        for (int s = 0; s < n; ++s) {
            int64_t S = lens[s];
            if (S <= 0) continue;
            int64_t chunks = ceil_div(S, C);
            sum += double(num_kv_heads) * (double(S) + overhead * double(chunks));
            items += double(num_kv_heads) * double(chunks);
            longest = std::max<int64_t>(longest, std::min<int64_t>(S, C));
        }
        if (items == 0.0) break;
        const double cost = std::max(sum / std::min(slots, items), double(longest) / 3.0 + overhead);
        if (cost < best_cost * 0.999) { best_cost = cost; best = C; }
    }
    return best;
}

}  // namespace

psa_status_t build_plan(const psa_config_t &cfg, int32_t P, const int32_t *first_sample, const int32_t *n_samples,
                        const int32_t *prefix_lens, const int32_t *token_begin, int64_t total_tokens_arg, bool causal,
                        int32_t num_samples, const int32_t *suffix_lens, psa_plan *plan, std::string *err)
{
    auto fail = [&](psa_status_t st, const char *msg) { if (err) *err = msg; return st; };
    if (cfg.num_q_heads <= 0 || cfg.num_kv_heads <= 0 || cfg.num_q_heads % cfg.num_kv_heads != 0)
        return fail(PSA_ERR_INVALID_ARG, "num_q_heads must be a positive multiple of num_kv_heads");
    const int G = cfg.num_q_heads / cfg.num_kv_heads;
    if (cfg.head_dim != 64 && cfg.head_dim != 128) return fail(PSA_ERR_UNSUPPORTED, "head_dim must be 64 or 128");
    if (G != 1 && G != 2 && G != 4 && G != 8) return fail(PSA_ERR_UNSUPPORTED, "group size must be 1, 2, 4 or 8");
    if (cfg.page_size != kPageSize) return fail(PSA_ERR_UNSUPPORTED, "page_size must be 16");
    if (!(cfg.sm_scale > 0.0f) || !(cfg.sm_scale < std::numeric_limits<float>::infinity()))
        return fail(PSA_ERR_INVALID_ARG, "sm_scale must be positive and finite");
    if (cfg.out_dtype != PSA_OUT_BF16 && cfg.out_dtype != PSA_OUT_F32)
        return fail(PSA_ERR_UNSUPPORTED, "out_dtype must be PSA_OUT_BF16 or PSA_OUT_F32");
    if (cfg.prefix_kernel < 0 || cfg.prefix_kernel > PSA_PREFIX_KERNEL_COUPLED) return fail(PSA_ERR_INVALID_ARG, "prefix_kernel out of range");
    if (cfg.suffix_chunk_tokens < 0 || cfg.suffix_chunk_tokens % 64 != 0)
        return fail(PSA_ERR_INVALID_ARG, "suffix_chunk_tokens must be 0 or a multiple of 64");
    if (cfg.prefix_tiles_per_item < 0) return fail(PSA_ERR_INVALID_ARG, "prefix_tiles_per_item must be >= 0");
    if (cfg.prefix_rows_per_item != 0 && cfg.prefix_rows_per_item != 128 && cfg.prefix_rows_per_item != 256)
        return fail(PSA_ERR_INVALID_ARG, "prefix_rows_per_item must be 0, 128 or 256");
    if (cfg.num_sms <= 0) return fail(PSA_ERR_INVALID_ARG, "num_sms must be positive here");
    if (P < 0 || (P > 0 && (!prefix_lens || !n_samples || !first_sample))) return fail(PSA_ERR_INVALID_ARG, "null length arrays");
    if (num_samples < 0) return fail(PSA_ERR_INVALID_ARG, "negative sample count");

    plan->cfg = cfg;
    plan->causal = causal;
    plan->group = G;
    plan->num_prefixes = P;
    plan->group_first_sample.assign(first_sample, first_sample + P);
    plan->group_n_samples.assign(n_samples, n_samples + P);
    plan->group_token_len.assign(prefix_lens, prefix_lens + P);
    const int64_t B = num_samples;
    int64_t total_tokens = 0;
    for (int p = 0; p < P; ++p) {
        if (prefix_lens[p] < 0 || n_samples[p] < 0) return fail(PSA_ERR_INVALID_ARG, "negative length or sample count");
        if (first_sample[p] < 0 || int64_t(first_sample[p]) + n_samples[p] > B)
            return fail(PSA_ERR_INVALID_ARG, "a prefix group reaches outside the samples");
        total_tokens += prefix_lens[p];
    }
    if (token_begin) {   // explicit key ranges (they may overlap): the caller says how long the packed arrays are
        total_tokens = total_tokens_arg;
        for (int p = 0; p < P; ++p)
            if (token_begin[p] < 0 || int64_t(token_begin[p]) + prefix_lens[p] > total_tokens)
                return fail(PSA_ERR_INVALID_ARG, "a prefix group reaches outside the packed prefix arrays");
    }
    if (B > (1 << 24) || total_tokens > (int64_t(1) << 30)) return fail(PSA_ERR_UNSUPPORTED, "problem too large");
    if (B > 0 && !suffix_lens) return fail(PSA_ERR_INVALID_ARG, "null suffix_lens");
    for (int64_t s = 0; s < B; ++s)
        if (suffix_lens[s] < 0 || suffix_lens[s] > (1 << 24)) return fail(PSA_ERR_INVALID_ARG, "suffix length out of range");
    plan->num_samples = int32_t(B);
    plan->total_prefix_tokens = total_tokens;
    plan->suffix_len_bounds.assign(suffix_lens, suffix_lens + B);

    // ---- prefix items
    // Rows per item.  Two row tiles (256 rows) per block halve the K/V traffic into the SM, which pays once
    // the stage is tensor-bound (R_p >= 512, above the machine's flop/byte ridge); below that a block of
    // one row tile is small enough to share its SM with a suffix block, and the overlap is worth more.
    int64_t max_rows = 0;
    for (int p = 0; p < P; ++p) max_rows = std::max<int64_t>(max_rows, int64_t(n_samples[p]) * G);
    const int rows_per_item = cfg.prefix_rows_per_item > 0 ? cfg.prefix_rows_per_item
                                                           : (max_rows >= 2 * kPrefixRowsPerItem ? kPrefixRowsPerItem : kPrefixTileRows);
    const int samples_per_group = rows_per_item / G;
    bool any_suffix = false;
    double suffix_kv_bytes = 0.0, prefix_kv_bytes = 0.0;   // K and V, bf16, all heads
    for (int64_t s = 0; s < B; ++s) {
        any_suffix = any_suffix || suffix_lens[s] > 0;
        suffix_kv_bytes += 4.0 * double(suffix_lens[s]) * cfg.num_kv_heads * cfg.head_dim;
    }
    for (int p = 0; p < P; ++p)
        if (n_samples[p] > 0) prefix_kv_bytes += 4.0 * double(prefix_lens[p]) * cfg.num_kv_heads * cfg.head_dim;
    std::vector<int64_t> tiles(P), groups(P), rows_per_split(P);
    for (int p = 0; p < P; ++p) {
        tiles[p] = n_samples[p] > 0 ? ceil_div(prefix_lens[p], kPrefixTileKeys) : 0;
        groups[p] = int64_t(cfg.num_kv_heads) * ceil_div(n_samples[p], samples_per_group);
        rows_per_split[p] = int64_t(cfg.num_kv_heads) * n_samples[p] * G;
    }
    const int T = cfg.prefix_tiles_per_item > 0
                      ? cfg.prefix_tiles_per_item
                      : choose_prefix_tiles_per_item(tiles, groups, rows_per_split, rows_per_item > kPrefixTileRows ? 1.3 : 1.0,
                                                     cfg.head_dim, cfg.num_sms, any_suffix ? 0.35 : 0.0,
                                                     rows_per_item > kPrefixTileRows, prefix_kv_bytes, suffix_kv_bytes);
    plan->prefix_tiles_per_item = T;

    plan->sample_info.assign(size_t(B), SampleInfo{});
    plan->prefix_items.clear();
    int64_t next_row = 0;  // partial rows are handed out prefix first, then suffix
    int64_t tok_off = 0;
    int longest_item_tiles = 0;
    for (int p = 0; p < P; ++p) {
        const int64_t N = n_samples[p], L = prefix_lens[p], R = N * G, samp_off = first_sample[p];
        if (token_begin) tok_off = token_begin[p];
        const int64_t splits = tiles[p] > 0 ? ceil_div(tiles[p], T) : 0;
        const int64_t base = next_row;
        for (int64_t i = 0; splits > 0 && i < N; ++i) {
            SampleInfo &si = plan->sample_info[size_t(samp_off + i)];
            if (si.n_levels >= kMaxPrefixLevels) return fail(PSA_ERR_UNSUPPORTED, "a sample belongs to more than 4 prefix groups");
            PrefixLevel &lv = si.level[si.n_levels++];
            lv.row0 = int32_t(base + i * G);
            lv.split_stride = int32_t(R);
            lv.splits = int32_t(splits);
            lv.head_stride = int32_t(R * splits);
        }
        if (splits > 0) {
            // key tiles are dealt out as evenly as possible: the first `extra` splits get one more
            const int64_t per = tiles[p] / splits, extra = tiles[p] % splits;
            for (int kv = 0; kv < cfg.num_kv_heads; ++kv) {
                int64_t tile0 = 0;
                for (int64_t j = 0; j < splits; ++j) {
                    const int64_t nt = per + (j < extra ? 1 : 0);
                    const int64_t key0 = tile0 * kPrefixTileKeys;
                    const int64_t key1 = std::min<int64_t>(L, (tile0 + nt) * kPrefixTileKeys);
                    longest_item_tiles = std::max<int>(longest_item_tiles, int(nt));
                    for (int64_t s0 = 0; s0 < N; s0 += samples_per_group) {
                        PrefixItem it;
                        it.first_token = int32_t(tok_off + key0);
                        it.n_keys = int32_t(key1 - key0);
                        it.kv_head = kv;
                        it.first_sample = int32_t(samp_off + s0);
                        it.n_rows = int32_t(std::min<int64_t>(samples_per_group, N - s0) * G);
                        it.partial_row0 = int32_t(base + (int64_t(kv) * splits + j) * R + s0 * G);
                        it.prompt = p;
                        it.split = int32_t(j);
                        plan->prefix_items.push_back(it);
                    }
                    tile0 += nt;
                }
            }
            next_row += int64_t(cfg.num_kv_heads) * splits * R;
        }
        tok_off += L;
    }
    plan->prefix_tiles_per_item = std::max(1, longest_item_tiles);
    plan->prefix_max_rows_per_item = 0;
    for (const PrefixItem &it : plan->prefix_items) plan->prefix_max_rows_per_item = std::max(plan->prefix_max_rows_per_item, it.n_rows);
    // longest items first: the hardware scheduler then fills the tail with short ones
    std::stable_sort(plan->prefix_items.begin(), plan->prefix_items.end(), [](const PrefixItem &a, const PrefixItem &b) {
        const int64_t ca = int64_t(ceil_div(a.n_keys, kPrefixTileKeys)) * (a.n_rows > kPrefixTileRows ? 2 : 1);
        const int64_t cb = int64_t(ceil_div(b.n_keys, kPrefixTileKeys)) * (b.n_rows > kPrefixTileRows ? 2 : 1);
        return ca > cb;
    });

    // ---- suffix items
    const int C = cfg.suffix_chunk_tokens > 0 ? cfg.suffix_chunk_tokens : choose_suffix_chunk(suffix_lens, int(B), cfg.num_kv_heads, cfg.num_sms);
    plan->suffix_chunk_tokens = C;
    plan->suffix_items.clear();
    for (int64_t s = 0; s < B; ++s) {
        SampleInfo &si = plan->sample_info[size_t(s)];
        const int64_t S = suffix_lens[s];
        const int64_t chunks = ceil_div(S, C);
        si.suf_row0 = int32_t(next_row);
        si.suf_chunks = int32_t(chunks);
        si.suf_len_bound = int32_t(S);
        for (int kv = 0; kv < cfg.num_kv_heads; ++kv)
            for (int64_t c = 0; c < chunks; ++c) {
                SuffixItem it;
                it.sample = int32_t(s);
                it.kv_head = kv;
                it.first_token = int32_t(c * C);
                it.partial_row0 = int32_t(next_row + (int64_t(kv) * chunks + c) * G);
                plan->suffix_items.push_back(it);
            }
        next_row += int64_t(cfg.num_kv_heads) * chunks * G;
    }
    // full chunks first, ragged last chunks after them (longest first)
    std::stable_sort(plan->suffix_items.begin(), plan->suffix_items.end(), [&](const SuffixItem &a, const SuffixItem &b) {
        const int la = std::min<int>(C, suffix_lens[a.sample] - a.first_token);
        const int lb = std::min<int>(C, suffix_lens[b.sample] - b.first_token);
        return la > lb;
    });
    if (next_row >= (int64_t(1) << 31)) return fail(PSA_ERR_UNSUPPORTED, "too many partial rows");
    plan->num_partial_rows = next_row;

    // ---- workspace layout and the host image of the lists
    WorkspaceLayout &ws = plan->ws;
    size_t off = 0;
    ws.status_off = off;          off = align_up(off + sizeof(int32_t) * kStatusWords, 256);
    ws.prefix_items_off = off;    off = align_up(off + sizeof(PrefixItem) * plan->prefix_items.size(), 256);
    ws.suffix_items_off = off;    off = align_up(off + sizeof(SuffixItem) * plan->suffix_items.size(), 256);
    ws.sample_info_off = off;     off = align_up(off + sizeof(SampleInfo) * plan->sample_info.size(), 256);
    ws.zero_lens_off = off;       off = align_up(off + (causal ? sizeof(int32_t) * size_t(B) : 0), 256);
    ws.lists_end = off;
    ws.partial_lse_off = off;     off = align_up(off + sizeof(float) * size_t(next_row), 256);
    ws.partial_o_off = off;       off = align_up(off + sizeof(float) * size_t(next_row) * size_t(cfg.head_dim), 256);
    ws.total = off;

    plan->upload.assign(ws.lists_end, 0);
    if (!plan->prefix_items.empty())
        std::memcpy(plan->upload.data() + ws.prefix_items_off, plan->prefix_items.data(), sizeof(PrefixItem) * plan->prefix_items.size());
    if (!plan->suffix_items.empty())
        std::memcpy(plan->upload.data() + ws.suffix_items_off, plan->suffix_items.data(), sizeof(SuffixItem) * plan->suffix_items.size());
    if (!plan->sample_info.empty())
        std::memcpy(plan->upload.data() + ws.sample_info_off, plan->sample_info.data(), sizeof(SampleInfo) * plan->sample_info.size());
    return PSA_OK;
}

}  // namespace psa
