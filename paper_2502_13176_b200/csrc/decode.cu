// Decode step over budgeted KV caches (Eq. 4-7): append, attention for the g query heads of a
// group in one pass over K and V, accumulated-attention update, and single-row eviction.
//
// One launch covers every (layer, sequence, KV head) of a layer range.  A head is cut into
// chunks (the host plan); one CTA reduces one chunk to a partial (o, m, l) and leaves the
// chunk's logits in the workspace.  The CTA that delivers the last partial of a head merges
// them in chunk order, writes the output, turns the logits into probabilities with the final
// normaliser, adds them to the scores and picks the row to evict in the same sweep.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>

#include "baklava.h"
#include "common.h"

namespace {

constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct DecodeParams {
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
    int32_t B, L, Hq, Hkv, n_sink, recent_num, recent_den;
    int32_t layer_begin, layers;
    const __nv_bfloat16* q;
    const __nv_bfloat16* k_new;
    const __nv_bfloat16* v_new;
    __nv_bfloat16* out;
    float* lse;
    int32_t t_pos;
    uint32_t flags;
    const int4* items;
    int32_t n_items;
    int32_t* arrive;
    int32_t* appended;
    float* partial;
    float* logit;
    float scale_log2;   // log2(e) / sqrt(D)
};

struct Unit {
    int li, b, h, head, st;
};

__device__ __forceinline__ Unit decode_unit(const DecodeParams& p, int unit) {
    Unit u;
    u.li = unit / (p.B * p.Hkv);
    const int rem = unit - u.li * (p.B * p.Hkv);
    u.b = rem / p.Hkv;
    u.h = rem - u.b * p.Hkv;
    const int l = p.layer_begin + u.li;
    u.head = l * p.Hkv + u.h;
    u.st = (u.b * p.L + l) * p.Hkv + u.h;
    return u;
}

// ---------------------------------------------------------------- step 1: append (Eq. 4)
template <int D>
__global__ void append_kernel(const DecodeParams p) {
    const int unit = blockIdx.x;
    const Unit u = decode_unit(p, unit);
    const int C = p.cap[u.head];
    const int n = p.len[u.st];
    const int f = p.free_slot[u.st];
    int ok = 1;
    if (n < 0 || n > C || f < 0 || f > n) {
        if (threadIdx.x == 0) atomicOr(p.status, BAKLAVA_STATUS_BAD_STATE);
        ok = 0;
    } else if (n >= C) {
        if (threadIdx.x == 0) atomicOr(p.status, BAKLAVA_STATUS_OVERFLOW);
        ok = 0;
    }
    if (ok) {
        const int64_t row = (int64_t)u.b * p.seq_stride + p.slab_off[u.head] + f;
        const int64_t src = ((int64_t)(u.li * p.B + u.b) * p.Hkv + u.h) * D;
        constexpr int kVec = D / 8;   // 16-byte pieces per row
        for (int i = threadIdx.x; i < 2 * kVec; i += blockDim.x) {
            const bool is_v = i >= kVec;
            const int c = is_v ? i - kVec : i;
            const uint4* from = reinterpret_cast<const uint4*>((is_v ? p.v_new : p.k_new) + src) + c;
            uint4* to = reinterpret_cast<uint4*>((is_v ? p.v_slab : p.k_slab) + row * D) + c;
            *to = *from;
        }
        if (threadIdx.x == 0) {
            p.pos[row] = p.t_pos;
            p.score[row] = 0.0f;
            p.len[u.st] = n + 1;
        }
    }
    if (threadIdx.x == 0) p.appended[unit] = ok;
}

// ---------------------------------------------------------------- steps 2-4
template <int E>
__device__ __forceinline__ void load_row(const __nv_bfloat16* row, int lane, float (&x)[E]) {
    if constexpr (E == 4) {
        const uint2 raw = __ldg(reinterpret_cast<const uint2*>(row) + lane);
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
        const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
        x[0] = a.x; x[1] = a.y; x[2] = b.x; x[3] = b.y;
    } else {
        const uint32_t raw = __ldg(reinterpret_cast<const uint32_t*>(row) + lane);
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw));
        x[0] = a.x; x[1] = a.y;
    }
}

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}
__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}

template <int D, int G>
__global__ void __launch_bounds__(kThreads) decode_chunk_kernel(const DecodeParams p) {
    constexpr int E = D / 32;   // elements of a row held by one lane
    __shared__ float sm_o[kWarps][G][D];
    __shared__ float sm_m[kWarps][G];
    __shared__ float sm_l[kWarps][G];
    __shared__ float sm_M[G];
    __shared__ float sm_invL[G];
    __shared__ unsigned long long sm_key[kWarps];
    __shared__ int sm_slot[kWarps];
    __shared__ int sm_last;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int4 item = p.items[blockIdx.x];
    const int unit = item.x, begin = item.y, chunk_len = item.z, piece = item.w & 0xffff;
    const Unit u = decode_unit(p, unit);
    const int C = p.cap[u.head];
    const int n = p.len[u.st];
    const int f = p.free_slot[u.st];
    if (n < 0 || n > C || f < 0 || f > C) {
        if (tid == 0 && piece == 0) atomicOr(p.status, BAKLAVA_STATUS_BAD_STATE);
        return;
    }
    const bool no_append = (p.flags & BAKLAVA_FLAG_NO_APPEND) != 0;
    const int hole = (no_append && f < n) ? f : -1;       // a freed slot in the middle of the rows
    const int n_hi = n + (hole >= 0 ? 1 : 0);             // rows 0 .. n_hi-1 are scanned
    const int active = n_hi > 0 ? (n_hi + chunk_len - 1) / chunk_len : 1;
    if (piece >= active) return;
    const int end = min(begin + chunk_len, n_hi);
    const bool keep_logits = (p.flags & BAKLAVA_FLAG_NO_SCORE) == 0;

    const int64_t row0 = (int64_t)u.b * p.seq_stride + p.slab_off[u.head];
    const __nv_bfloat16* Kh = p.k_slab + row0 * D;
    const __nv_bfloat16* Vh = p.v_slab + row0 * D;
    float* logit_h = p.logit + row0 * G;

    float qf[G][E];
    {
        const __nv_bfloat16* qrow = p.q + ((int64_t)(u.li * p.B + u.b) * p.Hq + u.h * G) * D;
#pragma unroll
        for (int a = 0; a < G; ++a) {
            load_row<E>(qrow + a * D, lane, qf[a]);
#pragma unroll
            for (int e = 0; e < E; ++e) qf[a][e] *= p.scale_log2;
        }
    }
    float m[G], l[G], o[G][E];
#pragma unroll
    for (int a = 0; a < G; ++a) {
        m[a] = -INFINITY;
        l[a] = 0.0f;
#pragma unroll
        for (int e = 0; e < E; ++e) o[a][e] = 0.0f;
    }

    for (int tile = begin + warp * 32; tile < end; tile += kWarps * 32) {
        const int cnt = min(32, end - tile);
        float s_mine[G];
#pragma unroll
        for (int a = 0; a < G; ++a) s_mine[a] = -INFINITY;
#pragma unroll 4
        for (int j = 0; j < cnt; ++j) {
            float kx[E];
            load_row<E>(Kh + (int64_t)(tile + j) * D, lane, kx);
#pragma unroll
            for (int a = 0; a < G; ++a) {
                float part = 0.0f;
#pragma unroll
                for (int e = 0; e < E; ++e) part = fmaf(qf[a][e], kx[e], part);
                part = warp_sum(part);
                if (lane == j) s_mine[a] = part;
            }
        }
        const bool valid = lane < cnt && (tile + lane) != hole;
        if (keep_logits && lane < cnt) {
#pragma unroll
            for (int a = 0; a < G; ++a) logit_h[(int64_t)(tile + lane) * G + a] = s_mine[a];
        }
        float pr[G];
#pragma unroll
        for (int a = 0; a < G; ++a) {
            const float s = valid ? s_mine[a] : -INFINITY;
            const float m_new = fmaxf(m[a], warp_max(s));
            const float corr = (m_new == -INFINITY) ? 1.0f : exp2f(m[a] - m_new);
            pr[a] = valid ? exp2f(s - m_new) : 0.0f;
            l[a] = l[a] * corr + warp_sum(pr[a]);
#pragma unroll
            for (int e = 0; e < E; ++e) o[a][e] *= corr;
            m[a] = m_new;
        }
#pragma unroll 4
        for (int j = 0; j < cnt; ++j) {
            if (tile + j == hole) continue;
            float vx[E];
            load_row<E>(Vh + (int64_t)(tile + j) * D, lane, vx);
#pragma unroll
            for (int a = 0; a < G; ++a) {
                const float pj = __shfl_sync(0xffffffffu, pr[a], j);
#pragma unroll
                for (int e = 0; e < E; ++e) o[a][e] = fmaf(pj, vx[e], o[a][e]);
            }
        }
    }

    // the four warps' states -> one partial for the chunk
#pragma unroll
    for (int a = 0; a < G; ++a) {
#pragma unroll
        for (int e = 0; e < E; ++e) sm_o[warp][a][lane * E + e] = o[a][e];
        if (lane == 0) { sm_m[warp][a] = m[a]; sm_l[warp][a] = l[a]; }
    }
    __syncthreads();
    float* part = p.partial + (int64_t)blockIdx.x * (G * D + 2 * G);
    for (int i = tid; i < G * D; i += kThreads) {
        const int a = i / D, d = i - a * D;
        float mm = -INFINITY;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) mm = fmaxf(mm, sm_m[w][a]);
        float acc = 0.0f, lsum = 0.0f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float c = (sm_m[w][a] == -INFINITY) ? 0.0f : exp2f(sm_m[w][a] - mm);
            acc = fmaf(sm_o[w][a][d], c, acc);
            lsum = fmaf(sm_l[w][a], c, lsum);
        }
        part[i] = acc;
        if (d == 0) { part[G * D + a] = mm; part[G * D + G + a] = lsum; }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int before = atomicAdd(p.arrive + unit, 1);
        sm_last = (before == active - 1);
    }
    __syncthreads();
    if (!sm_last) return;
    __threadfence();

    // ---- this CTA delivered the head's last partial: merge in chunk order and finish the step
    const float* part0 = p.partial + (int64_t)(blockIdx.x - piece) * (G * D + 2 * G);
    if (tid < G) {
        float mm = -INFINITY;
        for (int c = 0; c < active; ++c) mm = fmaxf(mm, __ldcg(part0 + (int64_t)c * (G * D + 2 * G) + G * D + tid));
        float ll = 0.0f;
        for (int c = 0; c < active; ++c) {
            const float* pc = part0 + (int64_t)c * (G * D + 2 * G);
            const float mc = __ldcg(pc + G * D + tid);
            if (mc != -INFINITY) ll = fmaf(__ldcg(pc + G * D + G + tid), exp2f(mc - mm), ll);
        }
        sm_M[tid] = mm;
        sm_invL[tid] = ll > 0.0f ? 1.0f / ll : 0.0f;
        if (p.lse) p.lse[(int64_t)(u.li * p.B + u.b) * p.Hq + u.h * G + tid] = ll > 0.0f ? (mm + log2f(ll)) * kLn2 : -INFINITY;
    }
    __syncthreads();
    __nv_bfloat16* orow = p.out + ((int64_t)(u.li * p.B + u.b) * p.Hq + u.h * G) * D;
    for (int i = tid; i < G * D; i += kThreads) {
        const int a = i / D;
        float acc = 0.0f;
        for (int c = 0; c < active; ++c) {
            const float* pc = part0 + (int64_t)c * (G * D + 2 * G);
            const float mc = __ldcg(pc + G * D + a);
            if (mc != -INFINITY) acc = fmaf(__ldcg(pc + i), exp2f(mc - sm_M[a]), acc);
        }
        orow[i] = __float2bfloat16_rn(acc * sm_invL[a]);
    }

    const bool appended = !no_append && p.appended[unit] != 0;
    const int R = C - 1;
    const bool evict = appended && keep_logits && (p.flags & BAKLAVA_FLAG_NO_EVICT) == 0 && n > R;
    unsigned long long best = ~0ull;
    int best_slot = -1;
    if (keep_logits) {
        const int W = max(0, (int)(((int64_t)(R - p.n_sink) * p.recent_num) / p.recent_den));
        float Mq[G], iL[G];
#pragma unroll
        for (int a = 0; a < G; ++a) { Mq[a] = sm_M[a]; iL[a] = sm_invL[a]; }
        for (int j = tid; j < n_hi; j += kThreads) {
            if (j == hole) continue;
            float inc = 0.0f;
#pragma unroll
            for (int a = 0; a < G; ++a) inc += exp2f(__ldcg(logit_h + (int64_t)j * G + a) - Mq[a]) * iL[a];
            const float sc = p.score[row0 + j] + inc;
            p.score[row0 + j] = sc;
            if (evict) {
                const int ps = p.pos[row0 + j];
                if (ps >= p.n_sink && ps <= p.t_pos - W) {
                    // lowest score goes; among equal scores the latest position goes
                    const unsigned long long key =
                        ((unsigned long long)__float_as_uint(sc) << 32) | (uint32_t)(~(uint32_t)ps);
                    if (key < best) { best = key; best_slot = j; }
                }
            }
        }
    }
    if (evict) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const unsigned long long ok = __shfl_xor_sync(0xffffffffu, best, off);
            const int os = __shfl_xor_sync(0xffffffffu, best_slot, off);
            if (ok < best) { best = ok; best_slot = os; }
        }
        if (lane == 0) { sm_key[warp] = best; sm_slot[warp] = best_slot; }
    }
    __syncthreads();
    if (tid == 0) {
        if (appended) {
            if (evict) {
                for (int w = 0; w < kWarps; ++w)
                    if (sm_key[w] < best) { best = sm_key[w]; best_slot = sm_slot[w]; }
                if (best_slot >= 0) {
                    p.free_slot[u.st] = best_slot;
                    p.len[u.st] = n - 1;
                } else {
                    atomicOr(p.status, BAKLAVA_STATUS_BAD_STATE);   // capacity too small for sinks + window
                    p.free_slot[u.st] = n;
                }
            } else {
                p.free_slot[u.st] = n;
            }
        }
        p.arrive[unit] = 0;
        p.appended[unit] = 0;
    }
}

template <int D, int G>
cudaError_t launch_chunks(const DecodeParams& p, cudaStream_t s) {
    decode_chunk_kernel<D, G><<<p.n_items, kThreads, 0, s>>>(p);
    return cudaGetLastError();
}

template <int D>
cudaError_t launch_for_group(int g, const DecodeParams& p, cudaStream_t s) {
    switch (g) {
        case 1: return launch_chunks<D, 1>(p, s);
        case 2: return launch_chunks<D, 2>(p, s);
        case 3: return launch_chunks<D, 3>(p, s);
        case 4: return launch_chunks<D, 4>(p, s);
        case 5: return launch_chunks<D, 5>(p, s);
        case 6: return launch_chunks<D, 6>(p, s);
        case 7: return launch_chunks<D, 7>(p, s);
        default: return launch_chunks<D, 8>(p, s);
    }
}

}  // namespace

extern "C" __attribute__((visibility("default"))) int baklava_decode_attn(const baklava_shape* shape, const baklava_cache* cache,
                                   const void* q, const void* k_new, const void* v_new, int32_t t_pos,
                                   void* out, float* lse, uint32_t flags,
                                   const int32_t* items, const baklava_plan_info* info,
                                   void* ws, size_t ws_bytes, void* stream) {
    int rc = baklava_check_shape(shape);
    if (rc) return rc;
    if (!cache || !q || !out || !items || !info || !ws) return BAKLAVA_ERR_INVALID_ARG;
    if (flags & ~(BAKLAVA_FLAG_NO_APPEND | BAKLAVA_FLAG_NO_SCORE | BAKLAVA_FLAG_NO_EVICT)) return BAKLAVA_ERR_INVALID_ARG;
    const bool no_append = flags & BAKLAVA_FLAG_NO_APPEND;
    if (!no_append && (!k_new || !v_new)) return BAKLAVA_ERR_INVALID_ARG;
    if (!cache->k_slab || !cache->v_slab || !cache->pos || !cache->score || !cache->len || !cache->free_slot ||
        !cache->cap || !cache->slab_off || !cache->status || cache->B <= 0 || cache->seq_stride_tokens <= 0)
        return BAKLAVA_ERR_INVALID_ARG;
    const void* ptrs[] = {q, k_new, v_new, out, cache->k_slab, cache->v_slab, items, ws};
    for (const void* ptr : ptrs)
        if (ptr && !baklava_aligned16(ptr)) return BAKLAVA_ERR_INVALID_ARG;
    if (info->layer_begin < 0 || info->layer_end > shape->L || info->layer_begin >= info->layer_end ||
        info->B != cache->B || info->n_items <= 0 ||
        info->n_units != (info->layer_end - info->layer_begin) * cache->B * shape->Hkv)
        return BAKLAVA_ERR_INVALID_ARG;
    DecodeWorkspace lay;
    const size_t need = baklava_decode_ws_bytes(shape, info->n_items, info->n_units, cache->B,
                                                cache->seq_stride_tokens, &lay);
    if (ws_bytes < need) return BAKLAVA_ERR_WORKSPACE;

    DecodeParams p;
    p.k_slab = static_cast<__nv_bfloat16*>(cache->k_slab);
    p.v_slab = static_cast<__nv_bfloat16*>(cache->v_slab);
    p.pos = cache->pos;
    p.score = cache->score;
    p.len = cache->len;
    p.free_slot = cache->free_slot;
    p.cap = cache->cap;
    p.slab_off = cache->slab_off;
    p.seq_stride = cache->seq_stride_tokens;
    p.status = cache->status;
    p.B = cache->B;
    p.L = shape->L; p.Hq = shape->Hq; p.Hkv = shape->Hkv;
    p.n_sink = shape->n_sink; p.recent_num = shape->recent_num; p.recent_den = shape->recent_den;
    p.layer_begin = info->layer_begin;
    p.layers = info->layer_end - info->layer_begin;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k_new = static_cast<const __nv_bfloat16*>(k_new);
    p.v_new = static_cast<const __nv_bfloat16*>(v_new);
    p.out = static_cast<__nv_bfloat16*>(out);
    p.lse = lse;
    p.t_pos = t_pos;
    p.flags = (flags & BAKLAVA_FLAG_NO_SCORE) ? (flags | BAKLAVA_FLAG_NO_EVICT) : flags;
    p.items = reinterpret_cast<const int4*>(items);
    p.n_items = info->n_items;
    char* base = static_cast<char*>(ws);
    p.arrive = reinterpret_cast<int32_t*>(base + lay.arrive_off);
    p.appended = reinterpret_cast<int32_t*>(base + lay.appended_off);
    p.partial = reinterpret_cast<float*>(base + lay.partial_off);
    p.logit = reinterpret_cast<float*>(base + lay.logit_off);
    p.scale_log2 = kLog2e / sqrtf((float)shape->D);

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int g = shape->Hq / shape->Hkv;
    cudaError_t err = cudaSuccess;
    if (!no_append) {
        if (shape->D == 128) append_kernel<128><<<info->n_units, 32, 0, s>>>(p);
        else append_kernel<64><<<info->n_units, 32, 0, s>>>(p);
        err = cudaGetLastError();
        if (err != cudaSuccess) return BAKLAVA_ERR_CUDA;
    }
    err = shape->D == 128 ? launch_for_group<128>(g, p, s) : launch_for_group<64>(g, p, s);
    return err == cudaSuccess ? BAKLAVA_OK : BAKLAVA_ERR_CUDA;
}
