// Host-side entry points: error names, Algorithm 1 step 2, Algorithm 2, and the decode work plan.
// Nothing here touches the device.
#include <algorithm>
#include <cstdint>
#include <cstring>
#include <numeric>
#include <vector>

#include "baklava.h"
#include "common.h"

extern "C" __attribute__((visibility("default"))) const char* baklava_strerror(int code) {
    switch (code) {
        case BAKLAVA_OK: return "ok";
        case BAKLAVA_ERR_INVALID_ARG: return "invalid argument";
        case BAKLAVA_ERR_SHAPE: return "unsupported shape";
        case BAKLAVA_ERR_CAPACITY: return "budget cannot be met within the capacity bounds";
        case BAKLAVA_ERR_WORKSPACE: return "workspace or output buffer too small";
        case BAKLAVA_ERR_CUDA: return "CUDA runtime error";
        case BAKLAVA_ERR_TIMEOUT: return "device wait timed out";
        case BAKLAVA_ERR_UNSUPPORTED: return "not supported by this build";
        default: return "unknown error code";
    }
}

int baklava_check_shape(const baklava_shape* s) {
    if (!s) return BAKLAVA_ERR_INVALID_ARG;
    if (s->L <= 0 || s->Hq <= 0 || s->Hkv <= 0) return BAKLAVA_ERR_SHAPE;
    if (s->D != 64 && s->D != 128) return BAKLAVA_ERR_SHAPE;
    if (s->Hq % s->Hkv != 0 || s->Hq / s->Hkv > BAKLAVA_MAX_GROUP) return BAKLAVA_ERR_SHAPE;
    if (s->page <= 0 || s->page % 16 != 0) return BAKLAVA_ERR_SHAPE;
    if (s->n_sink < 0 || s->recent_den <= 0 || s->recent_num < 0 || s->recent_num > s->recent_den)
        return BAKLAVA_ERR_SHAPE;
    return BAKLAVA_OK;
}

// ---------------------------------------------------------------- Algorithm 1, step 2
extern "C" __attribute__((visibility("default"))) int baklava_importance(const baklava_shape* shape, const float* head_cos, int32_t P,
                                  double* kv_importance) {
    int rc = baklava_check_shape(shape);
    if (rc) return rc;
    if (!head_cos || !kv_importance || P <= 0) return BAKLAVA_ERR_INVALID_ARG;
    const int L = shape->L, Hq = shape->Hq, Hkv = shape->Hkv, g = Hq / Hkv;
    for (int l = 0; l < L; ++l)
        for (int c = 0; c < Hkv; ++c) {
            double group = 0.0;
            for (int a = 0; a < g; ++a) {
                const int h = c * g + a;
                double over_prompts = 0.0;
                for (int p = 0; p < P; ++p) over_prompts += (double)head_cos[((size_t)p * L + l) * Hq + h];
                const double sim = over_prompts / P;        // mean over prompts of the per-prompt means
                group += (sim + 1.0) * 0.5;                 // cosine range [-1, 1] -> [0, 1]
            }
            kv_importance[l * Hkv + c] = 1.0 - group / g;   // complement of the group's similarity
        }
    return BAKLAVA_OK;
}

// ---------------------------------------------------------------- Algorithm 2
namespace {

void even_split(int64_t total, int m, std::vector<int64_t>& out) {
    out.assign(m, total / m);
    for (int i = 0; i < (int)(total % m); ++i) out[i] += 1;
}

// One group of m caches, sizes in pages.  Returns 0 or BAKLAVA_ERR_CAPACITY.
int reallocate_group(const double* imp, int m, double t, int64_t r_num, int64_t r_den, int64_t total,
                     int64_t lo, int64_t hi, std::vector<int64_t>& size) {
    even_split(total, m, size);
    for (int i = 0; i < m; ++i)
        if (size[i] < lo || size[i] > hi) return BAKLAVA_ERR_CAPACITY;

    std::vector<int> reduced, others;
    for (int i = 0; i < m; ++i) (imp[i] < t ? reduced : others).push_back(i);
    const int n = (int)reduced.size();
    if (n == 0 || n == m) return BAKLAVA_OK;

    auto more_important = [&](int a, int b) { return imp[a] > imp[b] || (imp[a] == imp[b] && a < b); };
    std::sort(others.begin(), others.end(), more_important);
    std::sort(reduced.begin(), reduced.end(), more_important);

    int64_t pool = 0;
    for (int i : reduced) {
        const int64_t give = std::min(size[i] * r_num / r_den, size[i] - lo);
        size[i] -= give;
        pool += give;
    }
    const int k = std::min(n, m - n);
    for (int rank = 0; rank < k; ++rank) size[others[rank]] += pool / k + (rank < pool % k ? 1 : 0);

    int64_t spill = 0;
    for (int rank = 0; rank < k; ++rank) {
        int64_t& s = size[others[rank]];
        if (s > hi) { spill += s - hi; s = hi; }
    }
    const std::vector<int>* passes[2] = {&others, &reduced};
    for (const std::vector<int>* order : passes) {
        bool placed = true;
        while (spill > 0 && placed) {
            placed = false;
            for (int j : *order) {
                if (spill == 0) break;
                if (size[j] < hi) { size[j] += 1; spill -= 1; placed = true; }
            }
        }
    }
    return spill > 0 ? BAKLAVA_ERR_CAPACITY : BAKLAVA_OK;
}

}  // namespace

extern "C" __attribute__((visibility("default"))) int baklava_allocate(const baklava_shape* shape, const double* kv_importance,
                                const baklava_alloc_params* p, int64_t total_tokens,
                                int32_t* cap_out, int64_t* slab_off_out, int64_t* seq_stride_out) {
    int rc = baklava_check_shape(shape);
    if (rc) return rc;
    if (!kv_importance || !p || !cap_out || !slab_off_out || !seq_stride_out) return BAKLAVA_ERR_INVALID_ARG;
    if (p->r_den <= 0 || p->r_num < 0 || p->r_num > p->r_den) return BAKLAVA_ERR_INVALID_ARG;
    if (p->scope != BAKLAVA_SCOPE_LAYER && p->scope != BAKLAVA_SCOPE_MODEL) return BAKLAVA_ERR_INVALID_ARG;
    const int64_t page = shape->page;
    if (total_tokens <= 0 || total_tokens % page != 0) return BAKLAVA_ERR_INVALID_ARG;
    if (p->min_tokens <= 0 || p->max_tokens < p->min_tokens) return BAKLAVA_ERR_INVALID_ARG;
    const int L = shape->L, Hkv = shape->Hkv;
    const int64_t total = total_tokens / page;
    const int64_t lo = (p->min_tokens + page - 1) / page, hi = (p->max_tokens + page - 1) / page;

    std::vector<int64_t> pages((size_t)L * Hkv), group;
    if (p->scope == BAKLAVA_SCOPE_MODEL) {
        rc = reallocate_group(kv_importance, L * Hkv, p->t, p->r_num, p->r_den, total, lo, hi, group);
        if (rc) return rc;
        pages = group;
    } else {
        std::vector<int64_t> per_layer;
        if (p->layer_importance) {
            if (p->rl_den <= 0 || p->rl_num < 0 || p->rl_num > p->rl_den) return BAKLAVA_ERR_INVALID_ARG;
            rc = reallocate_group(p->layer_importance, L, p->t_layer, p->rl_num, p->rl_den, total,
                                  lo * Hkv, hi * Hkv, per_layer);
            if (rc) return rc;
        } else {
            even_split(total, L, per_layer);
        }
        for (int l = 0; l < L; ++l) {
            rc = reallocate_group(kv_importance + (size_t)l * Hkv, Hkv, p->t, p->r_num, p->r_den,
                                  per_layer[l], lo, hi, group);
            if (rc) return rc;
            std::copy(group.begin(), group.end(), pages.begin() + (size_t)l * Hkv);
        }
    }
    int64_t run = 0;
    for (size_t i = 0; i < pages.size(); ++i) {
        const int64_t tokens = pages[i] * page;
        if (tokens > INT32_MAX) return BAKLAVA_ERR_CAPACITY;
        cap_out[i] = (int32_t)tokens;
        slab_off_out[i] = run;
        run += tokens;
    }
    *seq_stride_out = run;
    return BAKLAVA_OK;
}

// ---------------------------------------------------------------- decode work plan
size_t baklava_decode_ws_bytes(const baklava_shape* s, int64_t n_items, int64_t n_score_items, int64_t n_units, int32_t B,
                               int64_t seq_stride_tokens, DecodeWorkspace* lay) {
    const int g = s->Hq / s->Hkv;
    DecodeWorkspace w;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off += (bytes + 255) / 256 * 256; return at; };
    w.control_off = take(sizeof(int32_t) * 64);
    w.arrive_off = take(sizeof(int32_t) * (size_t)n_units);
    w.stats_off = take(sizeof(float) * (size_t)n_units * (2 * BAKLAVA_MAX_GROUP + 4));
    w.best_off = take(16 * (size_t)n_score_items);
    w.partial_off = take(sizeof(float) * (size_t)n_items * partial_floats(g, s->D));
    w.logit_off = take(sizeof(float) * (size_t)B * (size_t)seq_stride_tokens * g);
    w.total = off;
    if (lay) *lay = w;
    return off;
}

extern "C" __attribute__((visibility("default"))) int baklava_decode_plan(const baklava_shape* shape, const int32_t* cap, int32_t B,
                                   int32_t layer_begin, int32_t layer_end, int32_t chunk_tokens, int32_t n_sm,
                                   int32_t kv_dtype, int64_t seq_stride_tokens, int32_t* items_out, int64_t items_capacity,
                                   baklava_plan_info* info) {
    int rc = baklava_check_shape(shape);
    if (rc) return rc;
    if (!cap || !info || B <= 0 || seq_stride_tokens <= 0) return BAKLAVA_ERR_INVALID_ARG;
    if (layer_begin < 0 || layer_end > shape->L || layer_begin >= layer_end) return BAKLAVA_ERR_INVALID_ARG;
    if (chunk_tokens < 0 || (chunk_tokens == 0 && n_sm <= 0)) return BAKLAVA_ERR_INVALID_ARG;
    if (kv_dtype != BAKLAVA_KV_BF16 && kv_dtype != BAKLAVA_KV_FP8_E4M3) return BAKLAVA_ERR_INVALID_ARG;
    const int Hkv = shape->Hkv, layers = layer_end - layer_begin;

    std::vector<int> heads((size_t)layers * Hkv);       // index (li * Hkv + h) inside the range
    std::iota(heads.begin(), heads.end(), 0);
    int64_t tokens = 0;
    for (int i : heads) {
        const int32_t c = cap[(size_t)layer_begin * Hkv + i];
        if (c <= 0 || c % shape->page != 0) return BAKLAVA_ERR_INVALID_ARG;
        tokens += c;
    }
    tokens *= B;
    std::stable_sort(heads.begin(), heads.end(), [&](int a, int b) {
        return cap[(size_t)layer_begin * Hkv + a] > cap[(size_t)layer_begin * Hkv + b];
    });

    // Chunk length.  A fixed request is used as given.  Otherwise the launch is self-balancing: CTAs are
    // dispatched in item order, so the list starts with long chunks (about half of a CTA slot's share of
    // the tokens: little per-chunk overhead) and ends with short ones (a short tail).
    bool guided = chunk_tokens == 0;
    int64_t target = chunk_tokens, min_chunk = kMinChunk;
    if (guided) {
        const int64_t slots = (int64_t)n_sm * kCtasPerSm;
        // what a chunk costs besides its rows (start-up, partial, arrival) is paid per chunk, not per byte: with
        // one-byte rows the same balance between that and the tail of the launch is struck at twice the length
        const int64_t wide = kv_dtype == BAKLAVA_KV_FP8_E4M3 ? 2 : 1;
        min_chunk = wide * kMinChunk;
        target = (wide * tokens / (2 * slots) + kTile - 1) / kTile * kTile;
        target = std::max<int64_t>(kMinChunk, std::min<int64_t>(target, wide * 4096));
        if (target == kMinChunk) {
            // A short launch (one layer of a model): nothing balances a second, partly filled wave, so all chunks
            // get the same length, the shortest (from the minimum up) with which every chunk is resident at once.
            guided = false;
            for (; target < 4096; target += kTile) {
                int64_t count = 0;
                for (int i : heads) {
                    const int64_t c = cap[(size_t)layer_begin * Hkv + i];
                    const int64_t pieces = (c + target - 1) / target;
                    const int64_t len = ((c + pieces - 1) / pieces + kTile - 1) / kTile * kTile;
                    count += (c + len - 1) / len * B;
                }
                if (count <= slots) break;
            }
        }
    }
    target = std::max<int64_t>(kTile, (target + kTile - 1) / kTile * kTile);

    // cut every head into equal pieces of about `want` tokens and list them, head after head
    int64_t n_written = 0;
    auto emit = [&](int64_t base, bool shrink, int64_t* count) -> int {
        *count = 0;
        int64_t done = 0;                                  // tokens listed so far
        for (int i : heads) {
            const int64_t c = cap[(size_t)layer_begin * Hkv + i];
            int64_t want = base;
            if (shrink) {
                if (done * 20 >= tokens * 19) want = base / 8;          // last 5 % of the tokens
                else if (done * 5 >= tokens * 4) want = base / 4;       // 80 % .. 95 %
                else if (done * 2 >= tokens) want = base / 2;           // 50 % .. 80 %
                want = std::max<int64_t>(min_chunk, want);
            }
            done += c * B;
            int64_t pieces = (c + want - 1) / want;
            const int64_t len = ((c + pieces - 1) / pieces + kTile - 1) / kTile * kTile;
            pieces = (c + len - 1) / len;
            if (pieces > 32767 || pieces * (shape->Hq / Hkv) > max_merge_entries(shape->D)) return BAKLAVA_ERR_UNSUPPORTED;
            const int li = i / Hkv, h = i % Hkv;
            for (int b = 0; b < B; ++b) {
                const int64_t unit = ((int64_t)li * B + b) * Hkv + h;
                for (int64_t pc = 0; pc < pieces; ++pc, ++*count, ++n_written) {
                    if (!items_out) continue;
                    if (n_written >= items_capacity) return BAKLAVA_ERR_WORKSPACE;
                    int32_t* it = items_out + 4 * n_written;
                    it[0] = (int32_t)unit;
                    it[1] = (int32_t)(pc * len);
                    it[2] = (int32_t)len;
                    it[3] = (int32_t)(pc | (pieces << 16));
                }
            }
        }
        return BAKLAVA_OK;
    };
    int64_t n_items = 0, n_score = 0;
    rc = emit(target, guided, &n_items);
    if (rc) return rc;
    if (n_items > INT32_MAX) return BAKLAVA_ERR_UNSUPPORTED;
    // A launch whose chunks are all resident at once ends with its few longest heads; the plan then also lists
    // pieces of the heads for a score / eviction pass that runs as a kernel of its own (about two per SM).
    const bool short_launch = n_sm > 0 && n_items <= (int64_t)n_sm * kCtasPerSm;
    if (short_launch) {
        const int64_t len = std::min<int64_t>(kScoreChunk, std::max<int64_t>(kMinChunk, (tokens / (2 * (int64_t)n_sm) + kTile - 1) / kTile * kTile));
        rc = emit(len, false, &n_score);
        if (rc) return rc;
    }
    info->n_items = (int32_t)n_items;
    info->n_score_items = (int32_t)n_score;
    info->n_units = layers * B * Hkv;
    info->chunk_tokens = (int32_t)target;
    info->layer_begin = layer_begin;
    info->layer_end = layer_end;
    info->B = B;
    info->ws_bytes = (int64_t)baklava_decode_ws_bytes(shape, n_items, n_score, info->n_units, B, seq_stride_tokens, nullptr);
    return BAKLAVA_OK;
}

// ---------------------------------------------------------------- Algorithm 3: which configuration wins
extern "C" __attribute__((visibility("default"))) int baklava_search_pick(const double* avg_loss, int32_t n,
                                                                          int32_t* best) {
    if (!best || n < 0 || (n > 0 && !avg_loss)) return BAKLAVA_ERR_INVALID_ARG;
    int32_t at = -1;
    double min_loss = __builtin_inf();
    for (int32_t i = 0; i < n; ++i)
        if (avg_loss[i] < min_loss) { min_loss = avg_loss[i]; at = i; }   // strict: the first minimum stays; NaN never wins
    *best = at;
    return BAKLAVA_OK;
}
