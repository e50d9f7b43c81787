// Bulk eviction (Eq. 5-6 applied to a whole prefilled head): choose which of T dense rows stay
// under the head's budget and copy them, in position order, into the head's slab.
//
// Kernel 1 (one CTA per head) finds the score threshold of the heavy-hitter quota with an
// 8-bit-per-pass radix select and lists the kept rows in ascending position.  Kernel 2 copies
// the listed rows.  Ties at the threshold go to the earlier positions, so the kept set is the
// first R rows of the order (sinks, recent window, then score descending / position ascending).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <climits>
#include <cstdint>

#include "baklava.h"
#include "common.h"
#include "fp8.cuh"

namespace {

constexpr int kSelThreads = 1024;
constexpr int kCopyThreads = 256;
constexpr int kCopyRows = 64;   // rows per CTA of the copy kernel

struct EvictParams {
    __nv_bfloat16* k_slab;
    __nv_bfloat16* v_slab;
    int32_t* pos;
    float* score;
    int32_t* len;
    int32_t* free_slot;
    const int32_t* cap;
    const int64_t* slab_off;
    int64_t seq_stride;
    uint32_t* status;
    int32_t B, L, Hkv, n_sink, recent_num, recent_den;
    int32_t layer_begin;
    const __nv_bfloat16* k_dense;
    const __nv_bfloat16* v_dense;
    const float* score_dense;
    int32_t T, reserve;
    const int32_t* seq_len;   // [B] tokens of each sequence's prompt (clamped to 0 .. T) or NULL: T for all
    int64_t stride_layer, stride_seq, stride_head;
    int32_t* kept;   // [n_units][T]
    const float* kv_scale;   // FP8 slabs: [L, Hkv, 4] (K scale, its reciprocal, V scale, its reciprocal)
};

struct Where {
    int head, st, b;
    int64_t dense0, slab0;
};

__device__ __forceinline__ Where locate(const EvictParams& p, int unit) {
    const int li = unit / (p.B * p.Hkv);
    const int rem = unit - li * (p.B * p.Hkv);
    const int b = rem / p.Hkv, h = rem - b * p.Hkv;
    const int l = p.layer_begin + li;
    Where w;
    w.head = l * p.Hkv + h;
    w.b = b;
    w.st = (b * p.L + l) * p.Hkv + h;
    w.dense0 = (int64_t)li * p.stride_layer + (int64_t)b * p.stride_seq + (int64_t)h * p.stride_head;
    w.slab0 = (int64_t)b * p.seq_stride + p.slab_off[w.head];
    return w;
}

// fp32 -> uint32 whose unsigned order is the float order (-0 counted as +0)
__device__ __forceinline__ uint32_t ordered_bits(float x) {
    const uint32_t b = __float_as_uint(x + 0.0f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// exclusive prefix sum of one int per thread over the CTA; returns the CTA total in `total`
__device__ __forceinline__ int block_exclusive_scan(int x, int* warp_sums, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = warp_sums[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, w, o);
            if (lane >= o) w += y;
        }
        warp_sums[lane] = w;   // inclusive over warps
    }
    __syncthreads();
    const int before = warp > 0 ? warp_sums[warp - 1] : 0;
    total = warp_sums[31];
    __syncthreads();
    return before + incl - x;
}

__global__ void __launch_bounds__(kSelThreads) evict_select_kernel(const EvictParams p) {
    __shared__ int hist[256];
    __shared__ int warp_sums[32];
    __shared__ uint32_t sh_prefix;
    __shared__ int sh_want;

    const int unit = blockIdx.x, tid = threadIdx.x;
    const Where w = locate(p, unit);
    const int C = p.cap[w.head];
    const int R = C - p.reserve;
    int32_t* kept = p.kept + (int64_t)unit * p.T;
    const int T = p.seq_len ? min(max(p.seq_len[w.b], 0), p.T) : p.T;
    if (R < 1) {
        if (tid == 0) { atomicOr(p.status, BAKLAVA_STATUS_BAD_STATE); p.len[w.st] = 0; p.free_slot[w.st] = 0; }
        return;
    }
    if (T <= R) {
        for (int j = tid; j < T; j += kSelThreads) kept[j] = j;
        if (tid == 0) { p.len[w.st] = T; p.free_slot[w.st] = T; }
        return;
    }
    const int W = max(0, (int)(((int64_t)(R - p.n_sink) * p.recent_num) / p.recent_den));
    const int lo = min(p.n_sink, T);          // candidates are positions lo .. hi-1
    const int hi = max(lo, T - W);
    const int quota = R - lo - (T - hi);      // heavy hitters to pick among the candidates
    if (quota < 0 || quota > hi - lo) {
        if (tid == 0) { atomicOr(p.status, BAKLAVA_STATUS_BAD_STATE); p.len[w.st] = 0; p.free_slot[w.st] = 0; }
        return;
    }
    const float* sc = p.score_dense ? p.score_dense + w.dense0 : nullptr;

    // radix select: the `quota`-th largest ordered score among the candidates
    uint32_t prefix = 0;      // bits decided so far (from the top)
    int want = quota;         // how many still to take among rows matching the prefix
    if (quota > 0) {
        for (int shift = 24; shift >= 0; shift -= 8) {
            for (int i = tid; i < 256; i += kSelThreads) hist[i] = 0;
            __syncthreads();
            const uint32_t mask = shift == 24 ? 0u : (0xffffffffu << (shift + 8));
            for (int j = lo + tid; j < hi; j += kSelThreads) {
                const uint32_t key = ordered_bits(sc ? sc[j] : 0.0f);
                if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1);
            }
            __syncthreads();
            if (tid == 0) {
                int left = want, bin = 255;
                for (; bin > 0; --bin) {
                    if (hist[bin] >= left) break;
                    left -= hist[bin];
                }
                sh_prefix = prefix | ((uint32_t)bin << shift);
                sh_want = left;
            }
            __syncthreads();
            prefix = sh_prefix;
            want = sh_want;
            __syncthreads();
        }
    }
    // rows with key > prefix are in; of the rows with key == prefix the first `want` by position

    int base_eq = 0, base_out = 0;
    for (int j0 = 0; j0 < T; j0 += kSelThreads) {
        const int j = j0 + tid;
        const bool in_range = j < T;
        const bool cand = in_range && j >= lo && j < hi;
        uint32_t key = 0;
        if (cand) key = ordered_bits(sc ? sc[j] : 0.0f);
        const int is_eq = (cand && quota > 0 && key == prefix) ? 1 : 0;
        int total_eq;
        const int eq_rank = base_eq + block_exclusive_scan(is_eq, warp_sums, total_eq);
        bool keep = in_range && !cand;                       // sinks and the recent window
        if (cand && quota > 0) keep = key > prefix || (is_eq && eq_rank < want);
        int total_keep;
        const int rank = base_out + block_exclusive_scan(keep ? 1 : 0, warp_sums, total_keep);
        if (keep) kept[rank] = j;
        base_eq += total_eq;
        base_out += total_keep;
    }
    if (tid == 0) { p.len[w.st] = R; p.free_slot[w.st] = R; }
}

template <int D, bool kFp8>
__global__ void __launch_bounds__(kCopyThreads) evict_copy_kernel(const EvictParams p) {
    const int unit = blockIdx.x;
    const Where w = locate(p, unit);
    const int n = p.len[w.st];
    const int r0 = blockIdx.y * kCopyRows;
    if (r0 >= n) return;
    const int32_t* kept = p.kept + (int64_t)unit * p.T;
    constexpr int kVec = D / 8;                       // 16-byte pieces per row
    constexpr int kPerRow = 2 * kVec;                 // K and V
    constexpr int kRowsPerPass = kCopyThreads / kPerRow;
    const int sub = threadIdx.x / kPerRow, piece = threadIdx.x % kPerRow;
    for (int r = r0 + sub; r < min(r0 + kCopyRows, n); r += kRowsPerPass) {
        const int src = kept[r];
        const bool is_v = piece >= kVec;
        const int c = is_v ? piece - kVec : piece;
        const uint4* from = reinterpret_cast<const uint4*>((is_v ? p.v_dense : p.k_dense) + (w.dense0 + src) * D) + c;
        if (kFp8) {          // the row is quantised on its way into the slab: D bytes per row
            const float inv_scale = p.kv_scale[w.head * 4 + (is_v ? 3 : 1)];
            uint8_t* slab = reinterpret_cast<uint8_t*>(is_v ? p.v_slab : p.k_slab);
            *(reinterpret_cast<uint2*>(slab + (w.slab0 + r) * D) + c) = fp8::quantise8(__ldg(from), inv_scale);
        } else {
            uint4* to = reinterpret_cast<uint4*>((is_v ? p.v_slab : p.k_slab) + (w.slab0 + r) * D) + c;
            *to = __ldg(from);
        }
        if (piece == 0) {
            p.pos[w.slab0 + r] = src;
            p.score[w.slab0 + r] = p.score_dense ? p.score_dense[w.dense0 + src] + 0.0f : 0.0f;
        }
    }
}

// ---------------------------------------------------------------- in place (no dense source)
// The same rule applied to the rows a slab already holds (a budget that shrank, a cache that filled up under
// NO_EVICT, a freed slot to close).  Eq. 5-6 remove rows and keep the order of the others, so the kept rows move
// down to slots 0 .. n'-1 in the order they have in the slab; for a slab filled by baklava_evict that is
// ascending position.  Rows only ever move to lower slots, so one CTA per head can move them block by block
// (read a block of sources, synchronise, write) without staging a copy of the head.
//
// Rows are not in position order here, so ties at the score threshold are settled by a second radix select on
// the position (earliest positions stay).

// k-th largest 32-bit key among the rows for which key_of(j, &key) is true; returns the key and, in `want`,
// how many rows with exactly that key belong to the top k.  Whole CTA.
template <typename KeyOf>
__device__ __forceinline__ uint32_t radix_select(int n, int k, KeyOf key_of, int* hist, uint32_t* sh_prefix,
                                                 int* sh_want, int& want) {
    uint32_t prefix = 0;
    want = k;
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = threadIdx.x; i < 256; i += kSelThreads) hist[i] = 0;
        __syncthreads();
        const uint32_t mask = shift == 24 ? 0u : (0xffffffffu << (shift + 8));
        for (int j = threadIdx.x; j < n; j += kSelThreads) {
            uint32_t key;
            if (key_of(j, key) && (key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int left = want, bin = 255;
            for (; bin > 0; --bin) {
                if (hist[bin] >= left) break;
                left -= hist[bin];
            }
            *sh_prefix = prefix | ((uint32_t)bin << shift);
            *sh_want = left;
        }
        __syncthreads();
        prefix = *sh_prefix;
        want = *sh_want;
        __syncthreads();
    }
    return prefix;
}

template <int kRowBytes>
__global__ void __launch_bounds__(kSelThreads) evict_inplace_kernel(const EvictParams p) {
    __shared__ int hist[256];
    __shared__ int warp_sums[32];
    __shared__ uint32_t sh_prefix;
    __shared__ int sh_want;
    __shared__ int sh_red[32];

    const int unit = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const Where w = locate(p, unit);
    const int C = p.cap[w.head];
    const int R = C - p.reserve;
    const int n = p.len[w.st], f = p.free_slot[w.st];
    int32_t* order = p.kept + (int64_t)unit * p.T;           // source slot of every kept row, in slab order
    if (R < 1 || C > p.T || n < 0 || n > C || f < 0 || f > n || (f < n && n >= C)) {
        if (tid == 0) atomicOr(p.status, BAKLAVA_STATUS_BAD_STATE);
        return;                                              // the head is left as it is
    }
    const int span = n + (f < n ? 1 : 0);                    // slots 0 .. span-1 hold the n rows and, maybe, the hole
    const int32_t* pos = p.pos + w.slab0;
    float* score = p.score + w.slab0;

    uint32_t thr_key = 0, thr_pos = 0;
    int t_max = INT32_MIN, quota = 0;
    const bool cut = n > R;
    int W = 0;
    if (cut) {
        // the latest position present, the sinks and the rows of the recent window
        for (int j = tid; j < span; j += kSelThreads)
            if (j != f) t_max = max(t_max, pos[j]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) t_max = max(t_max, __shfl_xor_sync(0xffffffffu, t_max, o));
        if (lane == 0) sh_red[warp] = t_max;
        __syncthreads();
        t_max = sh_red[0];
        for (int i = 1; i < kSelThreads / 32; ++i) t_max = max(t_max, sh_red[i]);
        __syncthreads();
        W = max(0, (int)(((int64_t)(R - p.n_sink) * p.recent_num) / p.recent_den));
        int fixed = 0;
        for (int j = tid; j < span; j += kSelThreads)
            if (j != f && (pos[j] < p.n_sink || pos[j] > t_max - W)) ++fixed;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) fixed += __shfl_xor_sync(0xffffffffu, fixed, o);
        if (lane == 0) sh_red[warp] = fixed;
        __syncthreads();
        fixed = 0;
        for (int i = 0; i < kSelThreads / 32; ++i) fixed += sh_red[i];
        __syncthreads();
        quota = R - fixed;
        if (quota < 0 || quota > n - fixed) {
            if (tid == 0) atomicOr(p.status, BAKLAVA_STATUS_BAD_STATE);
            return;
        }
        if (quota > 0) {
            const int lo_pos = p.n_sink, hi_pos = t_max - W;
            auto is_cand = [&](int j) { return j != f && pos[j] >= lo_pos && pos[j] <= hi_pos; };
            int want = 0;
            thr_key = radix_select(span, quota, [&](int j, uint32_t& key) {
                if (!is_cand(j)) return false;
                key = ordered_bits(score[j]);
                return true;
            }, hist, &sh_prefix, &sh_want, want);
            // of the rows exactly at the threshold the `want` earliest positions stay
            int unused = 0;
            const uint32_t inv = radix_select(span, want, [&](int j, uint32_t& key) {
                if (!is_cand(j) || ordered_bits(score[j]) != thr_key) return false;
                key = ~(uint32_t)pos[j];
                return true;
            }, hist, &sh_prefix, &sh_want, unused);
            thr_pos = ~inv;                                   // rows at the threshold with pos <= thr_pos stay
        }
    }
    // list the kept rows in slab order
    int base = 0;
    for (int j0 = 0; j0 < span; j0 += kSelThreads) {
        const int j = j0 + tid;
        bool keep = j < span && j != f;
        if (keep && cut) {
            const int ps = pos[j];
            if (ps >= p.n_sink && ps <= t_max - W) {
                const uint32_t key = ordered_bits(score[j]);
                keep = quota > 0 && (key > thr_key || (key == thr_key && (uint32_t)ps <= thr_pos));
            }
        }
        int total;
        const int rank = base + block_exclusive_scan(keep ? 1 : 0, warp_sums, total);
        if (keep) order[rank] = j;
        base += total;
    }
    const int n_keep = base;
    __syncthreads();
    // move: row order[r] -> slot r, r ascending; order[r] >= r, so a block's writes never reach a later source
    constexpr int kVec = kRowBytes / 16;                     // 16-byte pieces per row and operand
    constexpr int kRows = kSelThreads / kVec;                // rows per pass
    uint8_t* ks = reinterpret_cast<uint8_t*>(p.k_slab) + w.slab0 * kRowBytes;
    uint8_t* vs = reinterpret_cast<uint8_t*>(p.v_slab) + w.slab0 * kRowBytes;
    int32_t* pos_w = p.pos + w.slab0;
    for (int r0 = 0; r0 < n_keep; r0 += kRows) {
        const int r = r0 + tid / kVec, c = tid % kVec;
        const bool on = r < n_keep;
        int src = 0, ps = 0;
        float sc = 0.0f;
        uint4 kv = make_uint4(0, 0, 0, 0), vv = kv;
        if (on) {
            src = __ldcg(order + r);
            if (src != r) {
                kv = *(reinterpret_cast<const uint4*>(ks + (int64_t)src * kRowBytes) + c);
                vv = *(reinterpret_cast<const uint4*>(vs + (int64_t)src * kRowBytes) + c);
                if (c == 0) { ps = pos_w[src]; sc = score[src]; }
            }
        }
        __syncthreads();
        if (on && src != r) {
            *(reinterpret_cast<uint4*>(ks + (int64_t)r * kRowBytes) + c) = kv;
            *(reinterpret_cast<uint4*>(vs + (int64_t)r * kRowBytes) + c) = vv;
            if (c == 0) { pos_w[r] = ps; score[r] = sc; }
        }
        __syncthreads();
    }
    if (tid == 0) { p.len[w.st] = n_keep; p.free_slot[w.st] = n_keep; }
}

}  // namespace

extern "C" __attribute__((visibility("default"))) size_t baklava_evict_workspace_size(const baklava_shape* shape, int32_t B, int32_t layers, int32_t T) {
    if (!shape || B <= 0 || layers <= 0 || T <= 0) return 0;
    return (size_t)B * layers * shape->Hkv * (size_t)T * sizeof(int32_t);
}

namespace {

// Argument checks and launches shared by the three entry points; `kept` has room for units * T entries.
int evict_impl(const baklava_shape* shape, const baklava_cache* cache, int32_t layer_begin, int32_t layer_end,
               const void* k_dense, const void* v_dense, const float* score_dense, int32_t T, const int32_t* seq_len,
               int64_t stride_layer, int64_t stride_seq, int64_t stride_head, int32_t reserve,
               int32_t* kept, void* stream) {
    const bool in_place = !k_dense && !v_dense;
    if (!in_place && (!k_dense || !v_dense)) return BAKLAVA_ERR_INVALID_ARG;
    if (in_place && (score_dense || seq_len)) return BAKLAVA_ERR_INVALID_ARG;   // the slab's own scores and lengths rule
    if (T <= 0 || reserve < 1) return BAKLAVA_ERR_INVALID_ARG;
    if (!in_place && (stride_layer < 0 || stride_seq < 0 || stride_head < T)) return BAKLAVA_ERR_INVALID_ARG;
    const void* ptrs[] = {k_dense, v_dense, cache->k_slab, cache->v_slab};
    for (const void* ptr : ptrs)
        if (ptr && !baklava_aligned16(ptr)) return BAKLAVA_ERR_INVALID_ARG;
    const int64_t units = (int64_t)(layer_end - layer_begin) * cache->B * shape->Hkv;
    const int64_t row_blocks = ((int64_t)T + kCopyRows - 1) / kCopyRows;
    if (units > INT32_MAX || row_blocks > 65535) return BAKLAVA_ERR_UNSUPPORTED;

    EvictParams p;
    p.k_slab = static_cast<__nv_bfloat16*>(cache->k_slab);
    p.v_slab = static_cast<__nv_bfloat16*>(cache->v_slab);
    p.pos = cache->pos; p.score = cache->score; p.len = cache->len; p.free_slot = cache->free_slot;
    p.cap = cache->cap; p.slab_off = cache->slab_off; p.seq_stride = cache->seq_stride_tokens;
    p.status = cache->status;
    p.B = cache->B; p.L = shape->L; p.Hkv = shape->Hkv;
    p.n_sink = shape->n_sink; p.recent_num = shape->recent_num; p.recent_den = shape->recent_den;
    p.layer_begin = layer_begin;
    p.k_dense = static_cast<const __nv_bfloat16*>(k_dense);
    p.v_dense = static_cast<const __nv_bfloat16*>(v_dense);
    p.score_dense = score_dense;
    p.T = T; p.reserve = reserve;
    p.seq_len = seq_len;
    p.stride_layer = stride_layer; p.stride_seq = stride_seq; p.stride_head = stride_head;
    p.kept = kept;
    p.kv_scale = cache->kv_scale;
    const bool quantised = cache->kv_dtype == BAKLAVA_KV_FP8_E4M3;
    if (cache->kv_dtype != BAKLAVA_KV_BF16 && !quantised) return BAKLAVA_ERR_INVALID_ARG;
    if (quantised && !cache->kv_scale) return BAKLAVA_ERR_INVALID_ARG;
    if (quantised && shape->D != 128) return BAKLAVA_ERR_UNSUPPORTED;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (in_place) {
        if (quantised) evict_inplace_kernel<128><<<(unsigned)units, kSelThreads, 0, s>>>(p);
        else if (shape->D == 128) evict_inplace_kernel<256><<<(unsigned)units, kSelThreads, 0, s>>>(p);
        else evict_inplace_kernel<128><<<(unsigned)units, kSelThreads, 0, s>>>(p);
        return cudaGetLastError() == cudaSuccess ? BAKLAVA_OK : BAKLAVA_ERR_CUDA;
    }
    evict_select_kernel<<<(unsigned)units, kSelThreads, 0, s>>>(p);
    if (cudaGetLastError() != cudaSuccess) return BAKLAVA_ERR_CUDA;
    const dim3 grid((unsigned)units, (unsigned)row_blocks);
    if (quantised) evict_copy_kernel<128, true><<<grid, kCopyThreads, 0, s>>>(p);
    else if (shape->D == 128) evict_copy_kernel<128, false><<<grid, kCopyThreads, 0, s>>>(p);
    else evict_copy_kernel<64, false><<<grid, kCopyThreads, 0, s>>>(p);
    return cudaGetLastError() == cudaSuccess ? BAKLAVA_OK : BAKLAVA_ERR_CUDA;
}

int check_cache_and_layers(const baklava_shape* shape, const baklava_cache* cache, int32_t layer_begin,
                           int32_t layer_end) {
    int rc = baklava_check_shape(shape);
    if (rc) return rc;
    if (!cache) return BAKLAVA_ERR_INVALID_ARG;
    if (!cache->k_slab || !cache->v_slab || !cache->pos || !cache->score || !cache->len || !cache->free_slot ||
        !cache->cap || !cache->slab_off || !cache->status || cache->B <= 0 || cache->seq_stride_tokens <= 0)
        return BAKLAVA_ERR_INVALID_ARG;
    if (layer_begin < 0 || layer_end > shape->L || layer_begin >= layer_end) return BAKLAVA_ERR_INVALID_ARG;
    return BAKLAVA_OK;
}

}  // namespace

extern "C" __attribute__((visibility("default"))) int baklava_evict_varlen(
        const baklava_shape* shape, const baklava_cache* cache, int32_t layer_begin, int32_t layer_end,
        const void* k_dense, const void* v_dense, const float* score_dense, int32_t T, const int32_t* prompt_len,
        int64_t stride_layer, int64_t stride_seq, int64_t stride_head, int32_t reserve,
        void* ws, size_t ws_bytes, void* stream) {
    int rc = check_cache_and_layers(shape, cache, layer_begin, layer_end);
    if (rc) return rc;
    if (!ws || !baklava_aligned16(ws)) return BAKLAVA_ERR_INVALID_ARG;
    if (T > 0 && ws_bytes < baklava_evict_workspace_size(shape, cache->B, layer_end - layer_begin, T))
        return BAKLAVA_ERR_WORKSPACE;
    return evict_impl(shape, cache, layer_begin, layer_end, k_dense, v_dense, score_dense, T, prompt_len,
                      stride_layer, stride_seq, stride_head, reserve, static_cast<int32_t*>(ws), stream);
}

extern "C" __attribute__((visibility("default"))) int baklava_evict(const baklava_shape* shape, const baklava_cache* cache,
                             int32_t layer_begin, int32_t layer_end,
                             const void* k_dense, const void* v_dense, const float* score_dense, int32_t T,
                             int64_t stride_layer, int64_t stride_seq, int64_t stride_head, int32_t reserve,
                             void* ws, size_t ws_bytes, void* stream) {
    return baklava_evict_varlen(shape, cache, layer_begin, layer_end, k_dense, v_dense, score_dense, T, nullptr,
                                stride_layer, stride_seq, stride_head, reserve, ws, ws_bytes, stream);
}

// ---------------------------------------------------------------- bulk eviction without a workspace
// Some callers of this library cannot hand over a workspace because they cannot allocate device
// memory at the point of the call: code running under a memory pool that is already full or
// frozen, a plug-in that is only given its input and output tensors, a start-up path that runs
// before the host framework's allocator exists.  For them the list of kept rows lives in a
// fixed array inside the library image instead of in caller memory.
namespace {

constexpr size_t kStaticKeptEntries = BAKLAVA_EVICT_STATIC_MAX_ENTRIES;   // 4 MiB per GPU that loads the library
static __device__ __align__(256) int32_t g_static_kept[kStaticKeptEntries];

constexpr int kMaxDevices = 64;
std::atomic<int32_t*> g_static_kept_addr[kMaxDevices];   // device address of the array, per device (zero-initialised)

// The array's name is only a host-side handle; the kernels need its address on the current device.
int static_kept_address(int32_t** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return BAKLAVA_ERR_CUDA;
    int32_t* known = g_static_kept_addr[dev].load(std::memory_order_acquire);
    if (!known) {                                            // threads that race here all look up the same address
        void* addr = nullptr;
        if (cudaGetSymbolAddress(&addr, g_static_kept) != cudaSuccess || !addr) return BAKLAVA_ERR_CUDA;
        known = static_cast<int32_t*>(addr);
        g_static_kept_addr[dev].store(known, std::memory_order_release);
    }
    *out = known;
    return BAKLAVA_OK;
}

}  // namespace

extern "C" __attribute__((visibility("default"))) int baklava_evict_static(
        const baklava_shape* shape, const baklava_cache* cache, int32_t layer_begin, int32_t layer_end,
        const void* k_dense, const void* v_dense, const float* score_dense, int32_t T,
        int64_t stride_layer, int64_t stride_seq, int64_t stride_head, int32_t reserve, void* stream) {
    int rc = check_cache_and_layers(shape, cache, layer_begin, layer_end);
    if (rc) return rc;
    if (T <= 0) return BAKLAVA_ERR_INVALID_ARG;
    const int64_t units = (int64_t)(layer_end - layer_begin) * cache->B * shape->Hkv;
    if (units * (int64_t)T > (int64_t)kStaticKeptEntries) return BAKLAVA_ERR_WORKSPACE;   // beyond the fixed array
    int32_t* kept = nullptr;
    rc = static_kept_address(&kept);
    if (rc) return rc;
    return evict_impl(shape, cache, layer_begin, layer_end, k_dense, v_dense, score_dense, T, nullptr,
                      stride_layer, stride_seq, stride_head, reserve, kept, stream);
}
