// Internal declarations shared by the library's translation units (not part of the ABI).
#pragma once
#include <cstddef>
#include <cstdint>

#include "baklava.h"

constexpr int kTile = 64;          // chunk lengths are multiples of this many tokens
constexpr int kCtasPerSm = 3;       // resident CTAs of the attention kernel per SM (its launch bounds)
constexpr int kMinChunk = 256;      // shortest chunk the automatic plan makes
constexpr int kScoreChunk = 2048;   // longest piece of the score / eviction pass of a short launch
// chunks of a head x group size that the merge of partials can stage in the attention kernel's idle ring
#ifdef __CUDACC__
__host__ __device__
#endif
constexpr int max_merge_entries(int D) { return 48 * D; }

// Byte offsets of the regions of the decode workspace.
struct DecodeWorkspace {
    size_t control_off;    // 64 int32: launch-wide counters
    size_t arrive_off;     // int32 [n_units]: chunks of a head that have delivered their partial result
    size_t stats_off;      // fp32 [n_units][2 * 8 + 4]: final (max, 1 / sum) of each query head, log2 domain, and where the
                           //   head's partials are (split tail)
    size_t best_off;       // uint64 [n_score_items] + int32 [n_score_items]: each score piece's eviction candidate
    size_t partial_off;    // fp32 [n_items][g * D + 2 * g + 2]: per-chunk (o, m, l) and its oldest evictable row (pos, slot)
    size_t logit_off;      // per head: fp16 [g][C] unnormalised probabilities of this step and fp32 [g][C / 16] reference
                           //   maxima, at 4 * g bytes per slab row
    size_t total;
};

// floats of one chunk's partial result: o [g][D], m [g], l [g], (pos, slot) of its oldest evictable row; padded
// so that every record starts 16-byte aligned
#ifdef __CUDACC__
__host__ __device__
#endif
constexpr int partial_floats(int g, int D) { return (g * D + 2 * g + 2 + 3) / 4 * 4; }

int baklava_check_shape(const baklava_shape* s);
size_t baklava_decode_ws_bytes(const baklava_shape* s, int64_t n_items, int64_t n_score_items, int64_t n_units, int32_t B,
                               int64_t seq_stride_tokens, DecodeWorkspace* layout);

inline bool baklava_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// prefill.cu: log2-domain largest logit of every causal query row (+inf past the prompt) into lse2 [B, Hq, T],
// for the 128-row blocks listed in `list` (flat index ((b * Hq + h) * n_blk + blk), *list_count entries, both on
// the device); `grid` CTAs share the list
struct CUstream_st;
int baklava_launch_row_max(const baklava_shape* shape, const void* q, const void* k, const int32_t* prompt_len,
                           int32_t B, int32_t T, float* lse2, const int32_t* list, const int32_t* list_count,
                           int32_t grid, uint32_t* error, CUstream_st* stream);
