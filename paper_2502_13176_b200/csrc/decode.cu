// Decode step over budgeted KV caches (Eq. 4-7): append, attention for the g query heads of a
// group in one pass over K and V, accumulated-attention update, and single-row eviction.
//
// One launch covers every (layer, sequence, KV head) of a layer range.  A head is cut into
// chunks (the host plan); one CTA reduces one chunk to a partial (o, m, l) and leaves the
// chunk's unnormalised probabilities in the workspace.  The CTA that delivers the last partial of a
// head finishes the head: it merges the partials in chunk order, writes the output, brings the
// probabilities to the final normaliser, adds them to the scores and picks the row to evict.
//
// Inside a chunk: a producer warp streams 64-token K and V tiles with TMA (128-byte swizzle)
// into a ring of shared-memory stages guarded by full/empty mbarriers; four consumer warps take
// 16 tokens of each tile (the tokens are the M side of both contractions: S^T = K Q^T and
// O^T += V^T P^T, bf16 mma.sync with fp32 accumulation) and keep an online-softmax state each.
// What the step writes besides the cache (probabilities, partials) is dropped from L2 once it has
// been read, and the scores and positions are kept in L2 from one step to the next where they fit.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <climits>
#include <cmath>
#include <cstdint>
#include <type_traits>

#include "baklava.h"
#include "common.h"
#include "fp8.cuh"
#include "ptx.cuh"

namespace {

using ptx::ldmatrix_x4;
using ptx::mbar_arrive_expect_tx;
using ptx::mbar_init;
using ptx::mbar_wait;
using ptx::smem_u32;
using ptx::tile_offset;          // tiles here are 64 tokens of 64-element boxes: the same swizzled layout
using tc::mbar_arrive;

constexpr int kConsumerWarps = 4;
constexpr int kThreads = (kConsumerWarps + 1) * 32;     // + one producer warp
constexpr int kTileTokens = kTile;                      // 64 tokens per stage
constexpr int kWarpTokens = kTileTokens / kConsumerWarps;
constexpr int kStages = 2;                              // bf16 slabs: two 32 KB stages, 64 KB per CTA, three CTAs per SM
// FP8 slabs: 128-token stages of the same 32 KB (64-token stages, three of them and four CTAs per SM were
// measured slower: 151 us against 137 us per step on the Llama-shaped workload)
constexpr int kFp8StageTokens = 128;
constexpr int kFp8Stages = 2;
constexpr int kFp8CtasPerSm = 3;
constexpr int kMaxStages = 4;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kStatsStride = 2 * BAKLAVA_MAX_GROUP + 4;   // per head: final max [8], 1 / sum [8], first item, chunks
static_assert(kWarpTokens == 16, "a consumer warp owns one 16-token MMA block of each tile");

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
    int32_t B, L, Hq, Hkv, G, D, n_sink, recent_num, recent_den;
    int32_t layer_begin, layers;
    const __nv_bfloat16* q;
    const __nv_bfloat16* k_new;
    const __nv_bfloat16* v_new;
    __nv_bfloat16* out;
    float* lse;
    int32_t t_pos;
    const int32_t* t_pos_seq;      // per-sequence positions [B] (negative: the sequence sits this step out) or NULL
    uint32_t flags;
    int32_t window_evict;          // 1: no scores are kept and the policy is sinks + window: evict by position
    const int4* items;             // the plan's work items
    int32_t n_items;
    int32_t split_tail;            // 1: the score update and the eviction run as a second kernel (short launches)
    int32_t* arrive;               // [n_units]: chunks of a head that have delivered their partial
    float* partial;
    float* logit;
    float* stats;                  // [n_units][kStatsStride]: final (max, 1 / sum) of every query head, the head's first
                                   //   item and its number of chunks (split tail only)
    unsigned long long* best_key;  // [n_score_items]: each piece's eviction candidate (split tail only)
    int32_t* best_slot;            // [n_score_items]
    float scale_log2;   // log2(e) / sqrt(D)
    const float* kv_scale;   // FP8 slabs: [L, Hkv, 4] (K scale, its reciprocal, V scale, its reciprocal)
    long long wait_cycles;   // SM clock cycles after which a wait on a tile gives up
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

// What a step does to one head, derived identically by every CTA that touches it.
struct HeadState {
    int C, n, f;        // capacity, valid rows and free slot before the step
    int n_att;          // rows 0 .. n_att-1 are scanned by attention
    int hole;           // a scanned slot that is not a row (-1: none)
    bool bad;           // inconsistent state: the head is skipped
    bool overflow;      // a row was offered but the cache has no free slot
    bool do_append;     // this step writes the new row at slot f (Eq. 4)
};

__device__ __forceinline__ HeadState head_state(const DecodeParams& p, const Unit& u) {
    HeadState h;
    h.C = p.cap[u.head];
    h.n = p.len[u.st];
    h.f = p.free_slot[u.st];
    const bool no_append = (p.flags & BAKLAVA_FLAG_NO_APPEND) != 0;
    h.bad = h.n < 0 || h.n > h.C || h.f < 0 || h.f > h.C || (!no_append && h.f > h.n) ||
            (p.slab_off[u.head] & 15) != 0 || (h.C & 15) != 0;   // rows are read in 16-byte vectors of pos / score
    h.overflow = !no_append && h.n >= h.C;
    h.do_append = !no_append && !h.overflow && !h.bad;
    h.hole = (no_append && h.f < h.n) ? h.f : -1;
    h.n_att = h.n + ((h.do_append || h.hole >= 0) ? 1 : 0);
    return h;
}

// ---------------------------------------------------------------- PTX wrappers
// Programmatic dependent launch: both kernels of a step are launched with the stream-serialisation
// attribute.  launch_dependents lets the next kernel's CTAs become resident while this grid drains;
// grid_dependency_wait returns once the previous grid has completed and its writes are visible.
__device__ __forceinline__ void launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// one arrival on a counter in global memory that also publishes this CTA's earlier writes and acquires the
// other arrivers' (the thread calling it has been through a CTA barrier with the writers)
__device__ __forceinline__ int arrive_acq_rel(int32_t* ptr) {
    int before;
    asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;" : "=r"(before) : "l"(ptr) : "memory");
    return before;
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
__device__ __forceinline__ void prefetch_l2_keep(const void* ptr) {
    asm volatile("prefetch.global.L2::evict_last [%0];" ::"l"(ptr));
}
// Scores and positions are read and rewritten once per step while a thousand times their size streams past: they
// are accessed with the keep-longest priority, so that they are still in L2 a step later where they fit.
__device__ __forceinline__ uint64_t l2_evict_last_policy() {
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(policy));
    return policy;
}
__device__ __forceinline__ float4 ld_keep(const float4* ptr, uint64_t policy) {
    float4 v;
    asm volatile("ld.global.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(ptr), "l"(policy));
    return v;
}
__device__ __forceinline__ int4 ld_keep(const int4* ptr, uint64_t policy) {
    int4 v;
    asm volatile("ld.global.L2::cache_hint.v4.s32 {%0, %1, %2, %3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(ptr), "l"(policy));
    return v;
}
__device__ __forceinline__ void st_keep(float4* ptr, const float4 v, uint64_t policy) {
    asm volatile("st.global.L2::cache_hint.v4.f32 [%0], {%1, %2, %3, %4}, %5;"
                 ::"l"(ptr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "l"(policy) : "memory");
}
__device__ __forceinline__ int ld_acquire(const int32_t* ptr) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
    return v;
}
__device__ __forceinline__ void st_release(int32_t* ptr, int v) {
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(ptr), "r"(v) : "memory");
}

// Scratch that has been read for the last time: its lines are dropped from L2 where they stand, so that they are
// never written back to device memory (what they hold afterwards is undefined; it is rewritten before it is read).
// Only lines that lie wholly inside [lo, hi) are touched.
template <int NT>
__device__ __forceinline__ void drop_lines(const void* lo, const void* hi) {
    const uintptr_t first = (reinterpret_cast<uintptr_t>(lo) + 127u) & ~(uintptr_t)127u;
    const uintptr_t last = reinterpret_cast<uintptr_t>(hi) & ~(uintptr_t)127u;
    for (uintptr_t x = first + 128u * threadIdx.x; x < last; x += 128u * NT)
        asm volatile("discard.global.L2 [%0], 128;" ::"l"(x) : "memory");
}

// K and V are read once per step and never fit in L2: ask L2 to drop them first, so that the
// step's logits, scores and positions (which the score pass re-reads) stay resident.
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    return policy;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar,
                                            uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D (16x8, fp32) += A (16x16, bf16, row) * B (16x8, bf16, col); rows 8..15 of A are zero here
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
    const uint32_t zero = 0u;
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(zero), "r"(a2), "r"(zero), "r"(b0), "r"(b1));
}
// the same with fp16 operands (FP8 slabs: the codes convert to fp16 exactly)
__device__ __forceinline__ void mma_f16(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
    const uint32_t zero = 0u;
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(zero), "r"(a2), "r"(zero), "r"(b0), "r"(b1));
}
// D (16x8, fp32) += A (16x16, row) * B (16x8, col), all four A registers in use
__device__ __forceinline__ void mma_bf16_full(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                              uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_f16_full(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                             uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// transpose of an 8 x 8 matrix of 16-bit elements held one row per quad of lanes (lane / 4 = row, two
// consecutive elements per lane): afterwards lane (g, t) holds elements (2 t, g) and (2 t + 1, g)
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
// 2^x on the special-function unit (one instruction; -inf gives 0, results below 2^-126 flush to 0)
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    const __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// ---------------------------------------------------------------- steps 3-4: scores and the row to evict
// Run over the whole head by the CTA that delivered its last partial, or over a piece of it by a CTA of the
// second kernel of a short launch.  Every row's stored probabilities
// are brought to the head's final normaliser and added to its score; rows that may be evicted compete on the
// 64-bit key (score bits, inverted position): the smallest key is the lowest score and, among equal scores,
// the latest token.  Eight consecutive rows per thread and group (they share one 16-row block, hence one
// reference maximum per query head), two or three groups in flight.  Each warp leaves its best candidate in shared
// memory.
template <int G>
struct SweepGroup {
    uint4 pr[G];
    float fac[G];
    float4 s0, s1;
    int4 p0, p1;
};

template <int G, int NT = kThreads>
__device__ __forceinline__ void sweep_head(const float* logit_h, float* score, const int32_t* pos, int n_sink, int C,
                                           int j_begin, int n_hi, int hole, bool evict, int newest_candidate,
                                           const float* sm_M, const float* sm_invL, unsigned long long* sm_key,
                                           int* sm_slot) {                // rows j_begin (a multiple of 64) .. n_hi - 1
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const __half* prob_h = reinterpret_cast<const __half*>(logit_h);
    const float* mref_h = reinterpret_cast<const float*>(prob_h + (int64_t)G * C);
    float Mq[G], iL[G];
#pragma unroll
    for (int a = 0; a < G; ++a) { Mq[a] = sm_M[a]; iL[a] = sm_invL[a]; }
    unsigned long long best = ~0ull;
    int best_slot = -1;
    const uint64_t keep = l2_evict_last_policy();

    auto load = [&](SweepGroup<G>& g, int j0) {              // a full group: rows j0 .. j0 + 7 all inside the head
#pragma unroll
        for (int a = 0; a < G; ++a) {
            g.fac[a] = __ldcg(mref_h + a * (C >> 4) + (j0 >> 4));
            g.pr[a] = __ldcg(reinterpret_cast<const uint4*>(prob_h + (int64_t)a * C + j0));
        }
        g.s0 = ld_keep(reinterpret_cast<const float4*>(score + j0), keep);
        g.s1 = ld_keep(reinterpret_cast<const float4*>(score + j0 + 4), keep);
        if (evict) {
            g.p0 = ld_keep(reinterpret_cast<const int4*>(pos + j0), keep);
            g.p1 = ld_keep(reinterpret_cast<const int4*>(pos + j0 + 4), keep);
        }
    };
    auto finish = [&](SweepGroup<G>& g, int j0) {
        float inc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) inc[e] = 0.0f;
#pragma unroll
        for (int a = 0; a < G; ++a) {
            const float f = (g.fac[a] == -INFINITY) ? 0.0f : exp2f(g.fac[a] - Mq[a]) * iL[a];
            const uint32_t w[4] = {g.pr[a].x, g.pr[a].y, g.pr[a].z, g.pr[a].w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float2 pe = __half22float2(*reinterpret_cast<const __half2*>(&w[k]));
                inc[2 * k] = fmaf(pe.x, f, inc[2 * k]);
                inc[2 * k + 1] = fmaf(pe.y, f, inc[2 * k + 1]);
            }
        }
        const float old[8] = {g.s0.x, g.s0.y, g.s0.z, g.s0.w, g.s1.x, g.s1.y, g.s1.z, g.s1.w};
        float sc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) sc[e] = (j0 + e == hole) ? old[e] : old[e] + inc[e];   // the freed slot is not a row
        st_keep(reinterpret_cast<float4*>(score + j0), make_float4(sc[0], sc[1], sc[2], sc[3]), keep);
        st_keep(reinterpret_cast<float4*>(score + j0 + 4), make_float4(sc[4], sc[5], sc[6], sc[7]), keep);
        if (evict) {
            const int ps[8] = {g.p0.x, g.p0.y, g.p0.z, g.p0.w, g.p1.x, g.p1.y, g.p1.z, g.p1.w};
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                if (j0 + e != hole && ps[e] >= n_sink && ps[e] <= newest_candidate) {
                    const unsigned long long key =
                        ((unsigned long long)__float_as_uint(sc[e]) << 32) | (uint32_t)(~(uint32_t)ps[e]);
                    if (key < best) { best = key; best_slot = j0 + e; }
                }
            }
        }
    };

    constexpr int kStride = 8 * NT;
    const int n_full = n_hi & ~7;                          // rows covered by full groups
    int j0 = j_begin + 8 * tid;
    if (G <= 4) {
        for (; j0 + 2 * kStride < n_full; j0 += 3 * kStride) {   // three full groups of this thread in flight
            SweepGroup<G> g0, g1, g2;
            load(g0, j0);
            load(g1, j0 + kStride);
            load(g2, j0 + 2 * kStride);
            finish(g0, j0);
            finish(g1, j0 + kStride);
            finish(g2, j0 + 2 * kStride);
        }
    }
    for (; j0 + kStride < n_full; j0 += 2 * kStride) {     // two full groups of this thread in flight
        SweepGroup<G> g0, g1;
        load(g0, j0);
        load(g1, j0 + kStride);
        finish(g0, j0);
        finish(g1, j0 + kStride);
    }
    if (j0 < n_full) {
        SweepGroup<G> g0;
        load(g0, j0);
        finish(g0, j0);
    }
    // the ragged end of the head: fewer than eight rows, one thread
    if (tid == (((n_full - j_begin) >> 3) % NT) && n_full < n_hi) {
        float f[G];
#pragma unroll
        for (int a = 0; a < G; ++a) {
            const float mr = __ldcg(mref_h + a * (C >> 4) + (n_full >> 4));
            f[a] = (mr == -INFINITY) ? 0.0f : exp2f(mr - Mq[a]) * iL[a];
        }
        for (int j = n_full; j < n_hi; ++j) {
            if (j == hole) continue;
            float inc = 0.0f;
#pragma unroll
            for (int a = 0; a < G; ++a) inc = fmaf(__half2float(__ldcg(prob_h + (int64_t)a * C + j)), f[a], inc);
            const float sc = score[j] + inc;
            score[j] = sc;
            if (evict) {
                const int ps = pos[j];
                if (ps >= n_sink && ps <= newest_candidate) {
                    const unsigned long long key = ((unsigned long long)__float_as_uint(sc) << 32) | (uint32_t)(~(uint32_t)ps);
                    if (key < best) { best = key; best_slot = j; }
                }
            }
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const unsigned long long ok = __shfl_xor_sync(0xffffffffu, best, off);
        const int os = __shfl_xor_sync(0xffffffffu, best_slot, off);
        if (ok < best) { best = ok; best_slot = os; }
    }
    if (lane == 0) { sm_key[warp] = best; sm_slot[warp] = best_slot; }
}

// ---------------------------------------------------------------- the end of a head
// Run by the CTA that delivered a head's last partial: final (max, 1 / sum) of every query head, the merged
// output (chunks in order: the result does not depend on which CTA comes last), then the score update over the
// whole head, the row to evict and the bookkeeping.  Other heads' CTAs keep streaming meanwhile; the plan puts
// the largest heads first, so the long tails fall into the middle of a launch.  Not inlined: its registers are
// its own and do not weigh on the streaming loop.
struct TailArgs {
    const float* part0;            // the head's first partial
    float* scratch;                // idle shared memory, 2 * max_merge_entries(D) floats
    int32_t* arrive;               // the head's arrival counter
    float* lse;                    // the group's entries of lse, or NULL
    __nv_bfloat16* out;            // the group's rows of out
    const float* logit_h;          // the head's probability scratch
    float* score;                  // the head's rows of score / pos
    const int32_t* pos;
    int32_t* len;
    int32_t* free_slot;
    uint32_t* status;
    float* stats;                  // the head's final (max, 1 / sum), for a score pass that runs as a second kernel
    int active, G, C, n, n_hi, hole, n_sink, newest_candidate;
    bool keep_logits, do_append, may_evict, pos_evict, overlap, split;
};

template <int D, bool kByPosition, int NT = kThreads>
__device__ __noinline__ void finish_head(const DecodeParams* pp, float* scratch, int unit, int piece, int active) {
    // everything about the head is derived again from the parameters, so that the call passes five values
    const DecodeParams& p = *pp;
    const Unit u = decode_unit(p, unit);
    const HeadState hs = head_state(p, u);
    const int t_pos = p.t_pos_seq ? p.t_pos_seq[u.b] : p.t_pos;
    const int64_t row0 = (int64_t)u.b * p.seq_stride + p.slab_off[u.head];
    TailArgs t;
    t.part0 = p.partial + (int64_t)((int)blockIdx.x - piece) * partial_floats(p.G, D);
    t.scratch = scratch;
    t.arrive = p.arrive + unit;
    t.lse = p.lse ? p.lse + (int64_t)(u.li * p.B + u.b) * p.Hq + u.h * p.G : nullptr;
    t.out = p.out + ((int64_t)(u.li * p.B + u.b) * p.Hq + u.h * p.G) * D;
    t.logit_h = p.logit + row0 * p.G;
    t.score = p.score + row0;
    t.pos = p.pos + row0;
    t.len = p.len + u.st;
    t.free_slot = p.free_slot + u.st;
    t.status = p.status;
    t.stats = p.stats + (int64_t)unit * kStatsStride;
    t.active = active; t.G = p.G; t.C = hs.C; t.n = hs.n; t.n_hi = hs.n_att; t.hole = hs.hole; t.n_sink = p.n_sink;
    // rows with a later position are in the recent window
    t.newest_candidate = t_pos - max(0, (int)(((int64_t)(hs.C - 1 - p.n_sink) * p.recent_num) / p.recent_den));
    t.keep_logits = (p.flags & BAKLAVA_FLAG_NO_SCORE) == 0;
    t.do_append = hs.do_append;
    t.may_evict = hs.do_append && (p.flags & BAKLAVA_FLAG_NO_EVICT) == 0 && hs.n_att > hs.C - 1;
    t.pos_evict = kByPosition && hs.do_append && hs.n_att > hs.C - 1;
    t.overlap = (p.flags & BAKLAVA_FLAG_OVERLAP_PREV) != 0;
    t.split = !kByPosition && t.keep_logits && p.split_tail != 0;
    constexpr int kG = BAKLAVA_MAX_GROUP;
    __shared__ float sm_M[kG];
    __shared__ float sm_invL[kG];
    __shared__ int sm_gave_up;
    __shared__ unsigned long long sm_key[NT / 32];   // each warp's eviction candidate
    __shared__ int sm_slot[NT / 32];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = t.G;
    const int psz = partial_floats(G, D);
    const float* part0 = t.part0;
    // every chunk's (max, sum) into shared memory with one round of loads (the plan keeps chunks x group
    // within max_merge_entries(D))
    float* sm_mc = t.scratch;
    float* sm_lc = sm_mc + max_merge_entries(D);
    const int n_ml = active * G;
    if (tid == 0) sm_gave_up = 0;
    __syncthreads();
    for (int i = tid; i < n_ml; i += NT) {
        const int c = i / G, a = i - c * G;
        const float* pc = part0 + (int64_t)c * psz + G * D;
        const float mc = __ldcg(pc + a);
        if (mc != mc) sm_gave_up = 1;                       // a chunk of this head ran out of time
        sm_mc[i] = mc;
        sm_lc[i] = __ldcg(pc + G + a);
    }
    __syncthreads();
    if (sm_gave_up) {
        // lost step: no output, no score update, no bookkeeping; the counter goes back to zero
        if (tid == 0) {
            *t.arrive = 0;
            if (t.split) t.stats[0] = __int_as_float(0x7fc00000);   // the second kernel is told
            if (t.overlap) grid_dependency_wait();
        }
        return;
    }
    for (int a = warp; a < G; a += NT / 32) {         // one warp per query head, lanes over the chunks
        float mm = -INFINITY;
        for (int c = lane; c < active; c += 32) mm = fmaxf(mm, sm_mc[c * G + a]);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, off));
        float ll = 0.0f;
        for (int c = lane; c < active; c += 32) {
            const float mc = sm_mc[c * G + a];
            if (mc != -INFINITY) ll = fmaf(sm_lc[c * G + a], exp2f(mc - mm), ll);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) ll += __shfl_xor_sync(0xffffffffu, ll, off);
        if (lane == 0) {
            sm_M[a] = mm;
            sm_invL[a] = ll > 0.0f ? 1.0f / ll : 0.0f;
            if (t.split) { t.stats[a] = mm; t.stats[kG + a] = sm_invL[a]; }
            if (t.lse) t.lse[a] = ll > 0.0f ? (mm + log2f(ll)) * kLn2 : -INFINITY;
        }
    }
    __syncthreads();
    if (t.split) {
        // steps 3-4 follow as a kernel of their own, whose pieces also merge the partial outputs (a share of the
        // output columns each): it is told where the head's partials are
        if (tid == 0) {
            reinterpret_cast<int32_t*>(t.stats)[2 * kG] = (int32_t)(part0 - pp->partial) / psz;
            reinterpret_cast<int32_t*>(t.stats)[2 * kG + 1] = t.active;
            *t.arrive = 0;
        }
        return;
    }
    for (int i = tid; i < n_ml; i += NT) {            // each chunk's weight in the merged output
        const int a = i % G;
        const float mc = sm_mc[i];
        sm_lc[i] = (mc == -INFINITY) ? 0.0f : exp2f(mc - sm_M[a]);
    }
    __syncthreads();
    for (int grp = tid; grp < G * D / 4; grp += NT) { // four output elements per thread, chunks in order
        const int a = (grp * 4) / D;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        int c = 0;
        for (; c + 16 <= active; c += 16) {                 // sixteen chunks' loads in flight
            float4 oc[16];
#pragma unroll
            for (int k = 0; k < 16; ++k)
                oc[k] = __ldcg(reinterpret_cast<const float4*>(part0 + (int64_t)(c + k) * psz) + grp);
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                const float wgt = sm_lc[(c + k) * G + a];
                acc.x = fmaf(oc[k].x, wgt, acc.x); acc.y = fmaf(oc[k].y, wgt, acc.y);
                acc.z = fmaf(oc[k].z, wgt, acc.z); acc.w = fmaf(oc[k].w, wgt, acc.w);
            }
        }
        for (; c + 4 <= active; c += 4) {
            float4 oc[4];
#pragma unroll
            for (int k = 0; k < 4; ++k)
                oc[k] = __ldcg(reinterpret_cast<const float4*>(part0 + (int64_t)(c + k) * psz) + grp);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float wgt = sm_lc[(c + k) * G + a];
                acc.x = fmaf(oc[k].x, wgt, acc.x); acc.y = fmaf(oc[k].y, wgt, acc.y);
                acc.z = fmaf(oc[k].z, wgt, acc.z); acc.w = fmaf(oc[k].w, wgt, acc.w);
            }
        }
        for (; c < active; ++c) {
            const float4 oc = __ldcg(reinterpret_cast<const float4*>(part0 + (int64_t)c * psz) + grp);
            const float wgt = sm_lc[c * G + a];
            acc.x = fmaf(oc.x, wgt, acc.x); acc.y = fmaf(oc.y, wgt, acc.y);
            acc.z = fmaf(oc.z, wgt, acc.z); acc.w = fmaf(oc.w, wgt, acc.w);
        }
        const float inv = sm_invL[a];
        const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
        const __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
        uint2 packed;
        packed.x = *reinterpret_cast<const uint32_t*>(&lo);
        packed.y = *reinterpret_cast<const uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(t.out + grp * 4) = packed;
    }

    // ---- steps 3-4
    const bool evict = !kByPosition && t.keep_logits && t.may_evict;
    if (!kByPosition && t.keep_logits) {
        switch (G) {
            case 1: sweep_head<1, NT>(t.logit_h, t.score, t.pos, t.n_sink, t.C, 0, t.n_hi, t.hole, evict, t.newest_candidate, sm_M, sm_invL, sm_key, sm_slot); break;
            case 2: sweep_head<2, NT>(t.logit_h, t.score, t.pos, t.n_sink, t.C, 0, t.n_hi, t.hole, evict, t.newest_candidate, sm_M, sm_invL, sm_key, sm_slot); break;
            case 3: sweep_head<3, NT>(t.logit_h, t.score, t.pos, t.n_sink, t.C, 0, t.n_hi, t.hole, evict, t.newest_candidate, sm_M, sm_invL, sm_key, sm_slot); break;
            case 4: sweep_head<4, NT>(t.logit_h, t.score, t.pos, t.n_sink, t.C, 0, t.n_hi, t.hole, evict, t.newest_candidate, sm_M, sm_invL, sm_key, sm_slot); break;
            case 5: sweep_head<5, NT>(t.logit_h, t.score, t.pos, t.n_sink, t.C, 0, t.n_hi, t.hole, evict, t.newest_candidate, sm_M, sm_invL, sm_key, sm_slot); break;
            case 6: sweep_head<6, NT>(t.logit_h, t.score, t.pos, t.n_sink, t.C, 0, t.n_hi, t.hole, evict, t.newest_candidate, sm_M, sm_invL, sm_key, sm_slot); break;
            case 7: sweep_head<7, NT>(t.logit_h, t.score, t.pos, t.n_sink, t.C, 0, t.n_hi, t.hole, evict, t.newest_candidate, sm_M, sm_invL, sm_key, sm_slot); break;
            default: sweep_head<8, NT>(t.logit_h, t.score, t.pos, t.n_sink, t.C, 0, t.n_hi, t.hole, evict, t.newest_candidate, sm_M, sm_invL, sm_key, sm_slot); break;
        }
    }
    __syncthreads();                                        // output, scores and the warps' candidates are written
    if (!kByPosition && t.keep_logits) {                    // the head's probabilities and reference maxima are spent
        const char* h0 = reinterpret_cast<const char*>(t.logit_h);
        drop_lines<NT>(h0, h0 + (size_t)G * t.C * 2 + (size_t)G * (t.C >> 4) * 4);
    }
    // and so are the chunks' partials (the sinks + window policy still reads its candidates from them below)
    if (!kByPosition) drop_lines<NT>(part0, part0 + (int64_t)active * psz);
    if (tid == 0) {
        *t.arrive = 0;
        if (t.do_append) {
            int victim = -1;
            bool wanted = false;                            // a row has to go
            if (kByPosition && t.pos_evict) {
                wanted = true;
                int bp = INT32_MAX;
                for (int c = 0; c < active; ++c) {
                    const float* pc = part0 + (int64_t)c * psz + G * D + 2 * G;
                    const int cp = __float_as_int(__ldcg(pc));
                    if (cp < bp) { bp = cp; victim = __float_as_int(__ldcg(pc + 1)); }
                }
            } else if (evict) {
                wanted = true;
                unsigned long long bk = ~0ull;
                for (int w = 0; w < NT / 32; ++w)
                    if (sm_key[w] < bk) { bk = sm_key[w]; victim = sm_slot[w]; }
            }
            if (wanted && victim < 0) atomicOr(t.status, BAKLAVA_STATUS_BAD_STATE);   // nothing outside sinks + window
            if (victim >= 0) {
                *t.free_slot = victim;                      // len stays n: one row in, one row out (Eq. 5-6)
            } else {
                *t.len = t.n + 1;
                *t.free_slot = t.n + 1;
            }
        }
        // an overlapping call has not looked behind yet: a grid of this library never completes before the grid
        // in front of it, which keeps "complete" transitive along the stream
        if (t.overlap) grid_dependency_wait();
    }
}

// ---------------------------------------------------------------- steps 2-4
// kByPosition: the score-free sinks + window policy (a second instantiation, so that the default
// path carries none of its registers or branches).
// kFp8: K and V rows are FP8 E4M3 codes (one byte per element, per-head scales).  A stage then holds 128
// tokens (the same 32 KB), every consumer warp takes two 16-token blocks of it, the codes are widened to fp16
// in registers (exactly) and the MMAs run in fp16 with the scales applied to the fp32 results.  The
// contraction index of an MMA may be permuted freely as long as both operands agree, which is what lets
// ldmatrix (16-bit granules) serve one-byte data: four consecutive bytes of a K row land in one register
// and become two fp16 pairs; V comes through ldmatrix.trans as two tokens x two adjacent channels per
// register, which a byte permute splits into an even-channel and an odd-channel operand.
template <int D, bool kByPosition, bool kFp8>
__global__ void __launch_bounds__(kThreads, kFp8 ? kFp8CtasPerSm : kCtasPerSm) decode_chunk_kernel(const __grid_constant__ DecodeParams p,
                                                                const __grid_constant__ CUtensorMap k_map,
                                                                const __grid_constant__ CUtensorMap v_map) {
    constexpr int kKSteps = D / 16;                    // MMA k-steps over the head dimension
    constexpr int kNTiles = D / 8;                     // 8-wide output column blocks
    constexpr int kTT = kFp8 ? kFp8StageTokens : kTileTokens;       // tokens per stage
    constexpr int kNS = kFp8 ? kFp8Stages : kStages;            // stages of the ring
    constexpr int kBlocks = kTT / (kConsumerWarps * kWarpTokens);    // 16-token blocks per warp and stage
    static_assert(kBlocks >= 1 && kNS <= kMaxStages, "a stage holds at least one 16-token block per warp");
    constexpr int kRowBytes = kFp8 ? D : 2 * D;
    constexpr int kTileBytes = kTT * kRowBytes;        // one K (or V) tile
    constexpr int kStageBytes = 2 * kTileBytes;
    constexpr int kG = BAKLAVA_MAX_GROUP;

    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[kMaxStages];
    __shared__ __align__(8) uint64_t bar_empty[kMaxStages];
    __shared__ float sm_m[kConsumerWarps][kG];
    __shared__ float sm_l[kConsumerWarps][kG];
    __shared__ int sm_last;
    __shared__ int sm_abort;
    __shared__ int sm_issued;
    __shared__ int sm_old_pos[kConsumerWarps];
    __shared__ int sm_old_slot[kConsumerWarps];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = p.G;
    // BAKLAVA_FLAG_OVERLAP_PREV: the caller vouches that nothing still in flight on the stream touches this call's
    // data, so the chunk starts streaming at once and releases what follows at once.  The dependency wait is still
    // made, at the very end, by the CTAs that finish a head (and by thread 0 of a CTA with nothing to do): a grid
    // of this library never completes before the grid in front of it, so an unflagged call, whose CTAs all wait
    // before they read anything, finds everything before it complete.
    const bool overlap = (p.flags & BAKLAVA_FLAG_OVERLAP_PREV) != 0;
    // what needs no memory of an earlier kernel comes first: the barriers and the tensor maps (kernel parameters)
    if (tid == kConsumerWarps * 32) {
        for (int s = 0; s < kNS; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), kConsumerWarps);
        }
        sm_abort = 0;
        sm_issued = 0;
        ptx::fence_mbar_init();
        prefetch_tensormap(&k_map);
        prefetch_tensormap(&v_map);
    }
    if (!overlap) grid_dependency_wait();                 // len / free_slot / slab rows / items come from earlier kernels
    else launch_dependents();
    const int4 item = p.items[blockIdx.x];
    const int unit = item.x, begin = item.y, chunk_len = item.z, piece = item.w & 0xffff;
    const Unit u = decode_unit(p, unit);
    // Only now may the score kernel's CTAs become resident: they read len / free_slot before their own
    // dependency wait, and this order guarantees that the previous step's bookkeeping is complete by then
    // even when the whole grid is resident at once.
    if (!overlap) launch_dependents();
    const int t_pos = p.t_pos_seq ? p.t_pos_seq[u.b] : p.t_pos;
    const HeadState hs = head_state(p, u);                // (its loads go out together with the one above)
    const int C = hs.C, n = hs.n, hole = hs.hole, n_hi = hs.n_att;
    const int active = n_hi > 0 ? (n_hi + chunk_len - 1) / chunk_len : 1;
    // idle sequence (none of its rows, outputs or bookkeeping is touched), inconsistent head, chunk past the rows
    if (t_pos < 0 || hs.bad || piece >= active) {
        if (t_pos >= 0 && hs.bad && tid == 0 && piece == 0) atomicOr(p.status, BAKLAVA_STATUS_BAD_STATE);
        if (overlap && tid == 0) grid_dependency_wait();
        return;
    }
    if (hs.overflow && tid == 0 && piece == 0) atomicOr(p.status, BAKLAVA_STATUS_OVERFLOW);
    const int end = min(begin + chunk_len, n_hi);
    const int n_tiles = end > begin ? (end - begin + kTT - 1) / kTT : 0;
    const bool keep_logits = (p.flags & BAKLAVA_FLAG_NO_SCORE) == 0;
    // sinks + window without scores: the one row that is neither a sink nor in the window (the oldest) goes
    const bool pos_evict = kByPosition && hs.do_append && n_hi > C - 1;
    const int window_from = t_pos - max(0, (int)(((int64_t)(C - 1 - p.n_sink) * p.recent_num) / p.recent_den));
    int old_pos = INT32_MAX, old_slot = -1;                // per lane, then per warp: oldest evictable row seen

    const int64_t row0 = (int64_t)u.b * p.seq_stride + p.slab_off[u.head];
    const float scale_k = kFp8 ? p.scale_log2 * p.kv_scale[u.head * 4 + 0] : p.scale_log2;   // logits -> log2 domain
    // this head's share of the scratch: unnormalised probabilities [G][C] in fp16, each relative to the
    // running maximum its 16-token block was computed under, and those maxima [G][C / 16] in fp32
    __half* prob_h = reinterpret_cast<__half*>(p.logit + row0 * G);
    float* mref_h = reinterpret_cast<float*>(prob_h + (int64_t)G * C);

    // 1024-byte aligned stage ring inside the dynamic shared memory
    const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* ring_ptr = smem_raw + (ring - smem_u32(smem_raw));

    // The head's tail reads and rewrites the score (and reads the position) of every row; those lines were last
    // touched a whole step ago.  Each chunk asks for its own share now, so that the tail finds them in L2.
    if (!kByPosition && keep_logits) {
        for (int r = begin + 32 * tid; r < end; r += 32 * kThreads) {
            prefetch_l2_keep(p.score + row0 + r);
            prefetch_l2_keep(p.pos + row0 + r);
        }
    }
    __syncthreads();                                      // the barriers are initialised

    // Tokens sit on the M side of both contractions (S^T = K Q^T and O^T = V^T P^T): a 16-token block costs
    // D / 16 MMAs each, with every accumulator row in use.  Lane (g, t) = (lane / 4, lane % 4) of a consumer warp
    // holds, of S^T, tokens g and g + 8 of the block for the query heads 2 t and 2 t + 1, and, of O^T, two
    // channels of every 16-channel group for the same two heads; its online-softmax state is that of those two
    // heads (the maximum shared by the warp, the sum its own rows' share, added up at the end of the chunk).
    const int g8 = lane >> 2, t4 = lane & 3;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.0f, 0.0f};
    float o[D / 16][4];
#pragma unroll
    for (int j = 0; j < D / 16; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.0f; }

    if (warp == kConsumerWarps) {
        // ---------------- producer: one lane issues the TMA loads
        if (lane == 0) {
            const uint64_t stream_policy = l2_evict_first_policy();
            int it = 0;
            for (; it < n_tiles; ++it) {
                const int s = it % kNS;
                // test aid (BAKLAVA_FLAG_TEST_STALL): the first chunk of a head gets its first tile only, so that
                // the consumers' bounded wait for the second one runs out; nothing is in flight by then
                if ((p.flags & BAKLAVA_FLAG_TEST_STALL) && piece == 0 && it == 1) break;
                if (it >= kNS) {
                    if (!mbar_wait(smem_u32(&bar_empty[s]), ((it / kNS) - 1) & 1, p.wait_cycles)) {
                        atomicOr(p.status, BAKLAVA_STATUS_TIMEOUT);
                        sm_abort = 1;
                        break;
                    }
                }
                const uint32_t full = smem_u32(&bar_full[s]);
                const uint32_t dst = ring + s * kStageBytes;
                const int y = (int)(row0 + begin + it * kTT);
                mbar_arrive_expect_tx(full, kStageBytes);
                if (kFp8) {                                  // one 128-byte-wide box holds the whole row
                    tma_load_2d(dst, &k_map, 0, y, full, stream_policy);
                    tma_load_2d(dst + kTileBytes, &v_map, 0, y, full, stream_policy);
                } else {
#pragma unroll
                    for (int bx = 0; bx < D / 64; ++bx) {
                        tma_load_2d(dst + bx * (kTileTokens * 128), &k_map, bx * 64, y, full, stream_policy);
                        tma_load_2d(dst + kTileBytes + bx * (kTileTokens * 128), &v_map, bx * 64, y, full, stream_policy);
                    }
                }
            }
            sm_issued = it;
        }
    } else {
        // ---------------- consumers
        // query fragments (B operand of S^T): head g of the group (zero from G on), per 16-channel step the
        // channels 2 t, 2 t + 1 (q0) and 8 + 2 t, 9 + 2 t (q1); for FP8 slabs the channels 4 t .. 4 t + 3, the order
        // in which the four bytes of a K register arrive (the contraction index may be permuted at will)
        uint32_t qq[2 * kKSteps];                          // (q0, q1) of step ks side by side, as the MMA takes them
        {
            const __nv_bfloat16* q_ptr = p.q + ((int64_t)(u.li * p.B + u.b) * p.Hq + u.h * G + g8) * D;
#pragma unroll
            for (int ks = 0; ks < kKSteps; ++ks) {
                if (kFp8) {
                    const uint2 raw = g8 < G ? *reinterpret_cast<const uint2*>(q_ptr + ks * 16 + 4 * t4) : make_uint2(0u, 0u);
                    const float2 f0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
                    const float2 f1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
                    qq[2 * ks] = pack_f16(f0.x, f0.y);
                    qq[2 * ks + 1] = pack_f16(f1.x, f1.y);
                } else {
                    qq[2 * ks] = g8 < G ? *reinterpret_cast<const uint32_t*>(q_ptr + ks * 16 + 2 * t4) : 0u;
                    qq[2 * ks + 1] = g8 < G ? *reinterpret_cast<const uint32_t*>(q_ptr + ks * 16 + 8 + 2 * t4) : 0u;
                }
            }
        }
        const int lm = lane >> 3, li8 = lane & 7;          // ldmatrix: matrix index and row inside it
        const int w0 = warp * kBlocks * kWarpTokens;       // this warp's rows inside a tile
        // This lane's row address inside a 16-token block for the two kinds of ldmatrix.  A tile is stored with
        // the 128-byte swizzle (16-byte piece c of row r at position c ^ (r % 8)); with the piece index
        // 2 c + b (b = one bit of the matrix index) that is a constant exclusive-or on a per-lane address:
        //   offset(r, 2 c + b) = (c / 4) * 8192 + ((r * 128 + ((b ^ r % 8) << 4)) ^ ((2 c % 8) << 4))
        // The four matrices of a load come out in the order of the MMA's A registers (a0 .. a3), so that no register
        // has to be moved in between: for K (rows = tokens) matrix 1 is the second token half and matrix 2 the
        // second channel half (bf16; for FP8 bytes the order of the conversions is free anyway), for the transposed
        // V load (rows of the MMA = channels) it is the other way round.
        const uint32_t k_lane = kFp8 ? (uint32_t)(((lm >> 1) * 8 + li8) * 128 + ((li8 ^ (lm & 1)) << 4))    // rows (lm / 2) * 8 + .., b = lm % 2
                                     : (uint32_t)(((lm & 1) * 8 + li8) * 128 + ((li8 ^ (lm >> 1)) << 4));   // rows (lm % 2) * 8 + .., b = lm / 2
        const uint32_t v_lane = kFp8 ? (uint32_t)(((lm & 1) * 8 + li8) * 128 + ((li8 ^ (lm >> 1)) << 4))
                                     : (uint32_t)(((lm >> 1) * 8 + li8) * 128 + ((li8 ^ (lm & 1)) << 4));
        // where this lane leaves the probabilities of head g8 (tokens 2 t4, 2 t4 + 1 of a block) for the score pass
        __half* const prob_lane = prob_h + (int64_t)g8 * C + 2 * t4;
        bool alive = true;
        for (int it = 0; it < n_tiles && alive; ++it) {
            const int s = it % kNS;
            if (!mbar_wait(smem_u32(&bar_full[s]), (it / kNS) & 1, p.wait_cycles)) {
                if (lane == 0) atomicOr(p.status, BAKLAVA_STATUS_TIMEOUT);
                alive = false;
                break;
            }
            const uint32_t k_tile = ring + s * kStageBytes;
            const uint32_t v_tile = k_tile + kTileBytes;
            const int wtok0 = begin + it * kTT + w0;                 // first token of this warp's share of the stage
            constexpr int kWarpSpan = kBlocks * kWarpTokens;
            // One body for the warp's tokens of the stage, compiled twice: the plain form for a span that lies
            // inside the chunk and holds neither the slot to append to nor a freed slot (nearly always), and the
            // careful form that patches the tile and masks rows.
            auto stage_body = [&](auto careful_tag) {
                constexpr bool kCareful = decltype(careful_tag)::value;
                if (kCareful) {
#pragma unroll
                    for (int blk = 0; blk < kBlocks; ++blk) {        // per 16-token block: patch the tile where needed
                        const int r0 = w0 + blk * kWarpTokens;
                        const int tok0 = wtok0 + blk * kWarpTokens;
                        const int valid = max(0, min(kWarpTokens, end - tok0));   // rows of the block inside the chunk
                        if (hs.do_append && hs.f >= tok0 && hs.f < tok0 + valid) {
                            // step 1 (Eq. 4): the new token's row replaces whatever the tile holds at the free slot,
                            // in shared memory for this pass and in the slab for the steps to come
                            constexpr int kVec = D / 8;
                            const int64_t src = ((int64_t)(u.li * p.B + u.b) * p.Hkv + u.h) * D;
                            const int64_t row = row0 + hs.f;
                            uint8_t* k_ptr = ring_ptr + s * kStageBytes;
                            if (kFp8) {                      // quantise the row: eight elements per lane and operand
                                for (int i = lane; i < 2 * kVec; i += 32) {
                                    const bool is_v = i >= kVec;
                                    const int c = is_v ? i - kVec : i;
                                    const uint4 raw = *(reinterpret_cast<const uint4*>((is_v ? p.v_new : p.k_new) + src) + c);
                                    const uint2 val = fp8::quantise8(raw, p.kv_scale[u.head * 4 + (is_v ? 3 : 1)]);
                                    *reinterpret_cast<uint2*>(k_ptr + (is_v ? kTileBytes : 0) + tile_offset(r0 + (hs.f - tok0), c >> 1) +
                                                              (c & 1) * 8) = val;
                                    uint8_t* slab = reinterpret_cast<uint8_t*>(is_v ? p.v_slab : p.k_slab);
                                    *(reinterpret_cast<uint2*>(slab + row * D) + c) = val;
                                }
                            } else {
                                for (int i = lane; i < 2 * kVec; i += 32) {
                                    const bool is_v = i >= kVec;
                                    const int c = is_v ? i - kVec : i;
                                    const uint4 val = *(reinterpret_cast<const uint4*>((is_v ? p.v_new : p.k_new) + src) + c);
                                    *reinterpret_cast<uint4*>(k_ptr + (is_v ? kTileBytes : 0) + tile_offset(r0 + (hs.f - tok0), c)) = val;
                                    *(reinterpret_cast<uint4*>((is_v ? p.v_slab : p.k_slab) + row * D) + c) = val;
                                }
                            }
                            if (lane == 0) { p.pos[row] = t_pos; p.score[row] = 0.0f; }
                            __syncwarp();
                        }
                        // rows past the end of the head (or the freed slot) may hold anything: keep them out of P.V
                        if (valid < kWarpTokens || (hole >= tok0 && hole < tok0 + kWarpTokens)) {
                            uint8_t* v_ptr = ring_ptr + s * kStageBytes + kTileBytes;
                            constexpr int kPieces = kRowBytes / 16;     // 16-byte pieces of a row
                            for (int i = lane; i < kWarpTokens * kPieces; i += 32) {
                                const int r = i / kPieces, c = i % kPieces;
                                if (r >= valid || tok0 + r == hole)
                                    *reinterpret_cast<uint4*>(v_ptr + tile_offset(r0 + r, c)) = make_uint4(0, 0, 0, 0);
                            }
                            __syncwarp();
                        }
                    }
                }
                // S^T = K Q^T for the warp's tokens: st[blk] = (token g: heads 2 t, 2 t + 1; token g + 8: the same)
                float st[kBlocks][4];
#pragma unroll
                for (int blk = 0; blk < kBlocks; ++blk) {
                    st[blk][0] = st[blk][1] = st[blk][2] = st[blk][3] = 0.0f;
                    const uint32_t k_row = k_tile + (uint32_t)((w0 + blk * kWarpTokens) * 128) + k_lane;
                    if (kFp8) {
#pragma unroll
                        for (int kk = 0; kk < D / 32; ++kk) {     // 32 channels per load: two steps of 16
                            uint32_t kb[4];      // (tokens 0-7 | 8-15) x (channels 0-15 | 16-31), four bytes per lane
                            ldmatrix_x4((k_row ^ (uint32_t)(((2 * kk) & 7) << 4)) + (kk >> 2) * 8192, kb);
#pragma unroll
                            for (int c = 0; c < 2; ++c) {
                                uint32_t a0, a2, a1, a3;
                                fp8::f16x4_from_e4m3x4(kb[c], a0, a2);
                                fp8::f16x4_from_e4m3x4(kb[2 + c], a1, a3);
                                mma_f16_full(st[blk], a0, a1, a2, a3, qq[2 * (2 * kk + c)], qq[2 * (2 * kk + c) + 1]);
                            }
                        }
                    } else {
#pragma unroll
                        for (int ks = 0; ks < kKSteps; ++ks) {
                            uint32_t kb[4];      // channels 0-7 of the step: tokens 0-7, 8-15; channels 8-15: tokens 0-7, 8-15
                            ldmatrix_x4((k_row ^ (uint32_t)(((2 * ks) & 7) << 4)) + (ks >> 2) * 8192, kb);
                            mma_bf16_full(st[blk], kb[0], kb[1], kb[2], kb[3], qq[2 * ks], qq[2 * ks + 1]);
                        }
                    }
                }
                // online softmax for the two heads of this lane over the warp's tokens of the stage
                float mx[2] = {-INFINITY, -INFINITY};
                bool ok[kBlocks][2];
#pragma unroll
                for (int blk = 0; blk < kBlocks; ++blk)
#pragma unroll
                    for (int r = 0; r < 2; ++r) {
                        const int tok = wtok0 + blk * kWarpTokens + g8 + 8 * r;
                        ok[blk][r] = !kCareful || (tok < end && tok != hole);
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            st[blk][2 * r + e] *= scale_k;
                            if (ok[blk][r]) mx[e] = fmaxf(mx[e], st[blk][2 * r + e]);
                        }
                    }
                float corr[2];
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    mx[e] = fmaxf(mx[e], __shfl_xor_sync(0xffffffffu, mx[e], 4));
                    mx[e] = fmaxf(mx[e], __shfl_xor_sync(0xffffffffu, mx[e], 8));
                    mx[e] = fmaxf(mx[e], __shfl_xor_sync(0xffffffffu, mx[e], 16));
                    const float m_new = fmaxf(m_run[e], mx[e]);
                    corr[e] = (m_new == -INFINITY) ? 1.0f : fast_exp2(m_run[e] - m_new);
                    m_run[e] = m_new;
                }
                float psum[2] = {0.0f, 0.0f};
#pragma unroll
                for (int blk = 0; blk < kBlocks; ++blk)
#pragma unroll
                    for (int r = 0; r < 2; ++r)
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const float pv = ok[blk][r] ? fast_exp2(st[blk][2 * r + e] - m_run[e]) : 0.0f;
                            st[blk][2 * r + e] = pv;
                            psum[e] += pv;
                        }
                l_run[0] = l_run[0] * corr[0] + psum[0];
                l_run[1] = l_run[1] * corr[1] + psum[1];
                if (__any_sync(0xffffffffu, corr[0] != 1.0f || corr[1] != 1.0f)) {
#pragma unroll
                    for (int j = 0; j < D / 16; ++j) { o[j][0] *= corr[0]; o[j][1] *= corr[1]; o[j][2] *= corr[0]; o[j][3] *= corr[1]; }
                }
                // P^T as the B operand of O^T += V^T P^T: the 8 x 8 blocks (tokens x heads) this warp holds one
                // row per quad are transposed, so that lane (g, t) gets head g, tokens 2 t, 2 t + 1 (and + 8)
                uint32_t pb[kBlocks][2];
#pragma unroll
                for (int blk = 0; blk < kBlocks; ++blk) {
                    const int tok0 = wtok0 + blk * kWarpTokens;
                    const uint32_t h0 = movmatrix_trans(pack_f16(st[blk][0], st[blk][1]));
                    const uint32_t h1 = movmatrix_trans(pack_f16(st[blk][2], st[blk][3]));
                    if (kFp8) {
                        pb[blk][0] = h0; pb[blk][1] = h1;
                    } else {
                        pb[blk][0] = movmatrix_trans(pack_bf16(st[blk][0], st[blk][1]));
                        pb[blk][1] = movmatrix_trans(pack_bf16(st[blk][2], st[blk][3]));
                    }
                    if (keep_logits) {
                        // the unnormalised probabilities of head g, in fp16, and the maximum they were taken under
                        __half* dst = prob_lane + tok0;
                        if (!kCareful) {
                            if (g8 < G) {
                                *reinterpret_cast<uint32_t*>(dst) = h0;
                                *reinterpret_cast<uint32_t*>(dst + 8) = h1;
                            }
                        } else if (g8 < G && tok0 < end) {
                            if (tok0 + 2 * t4 + 1 < end) *reinterpret_cast<uint32_t*>(dst) = h0;
                            else if (tok0 + 2 * t4 < end) dst[0] = __ushort_as_half((unsigned short)(h0 & 0xffffu));
                            if (tok0 + 8 + 2 * t4 + 1 < end) *reinterpret_cast<uint32_t*>(dst + 8) = h1;
                            else if (tok0 + 8 + 2 * t4 < end) dst[8] = __ushort_as_half((unsigned short)(h1 & 0xffffu));
                        }
                        if (g8 == 0 && (!kCareful || tok0 < end)) {
                            if (2 * t4 < G) mref_h[(2 * t4) * (C >> 4) + (tok0 >> 4)] = m_run[0];
                            if (2 * t4 + 1 < G) mref_h[(2 * t4 + 1) * (C >> 4) + (tok0 >> 4)] = m_run[1];
                        }
                    }
                }
                // O^T += V^T P^T: V^T fragments through ldmatrix.trans
#pragma unroll
                for (int blk = 0; blk < kBlocks; ++blk) {
                    const uint32_t v_row = v_tile + (uint32_t)((w0 + blk * kWarpTokens) * 128) + v_lane;
                    if (kFp8) {
                        // a register of the transposed load = two tokens x two adjacent channels; the permute puts the
                        // even channel's token pair in the low half and the odd channel's in the high half.  Row g of
                        // the MMA is channel 2 g of the 16-channel group, row g + 8 channel 2 g + 1.
#pragma unroll
                        for (int c2 = 0; c2 < D / 32; ++c2) {
                            uint32_t vb[4];      // (tokens 0-7 | 8-15) x (channels 0-15 | 16-31)
                            ldmatrix_x4_trans((v_row ^ (uint32_t)(((2 * c2) & 7) << 4)) + (c2 >> 2) * 8192, vb);
#pragma unroll
                            for (int h2 = 0; h2 < 2; ++h2) {
                                const uint32_t lo = __byte_perm(vb[2 * h2], 0u, 0x3120), hi = __byte_perm(vb[2 * h2 + 1], 0u, 0x3120);
                                uint32_t even0, odd0, even1, odd1;               // tokens 0-7 and 8-15 of the block
                                fp8::f16x4_from_e4m3x4(lo, even0, odd0);
                                fp8::f16x4_from_e4m3x4(hi, even1, odd1);
                                mma_f16_full(o[2 * c2 + h2], even0, odd0, even1, odd1, pb[blk][0], pb[blk][1]);
                            }
                        }
                    } else {
#pragma unroll
                        for (int c = 0; c < D / 16; ++c) {
                            uint32_t vb[4];      // tokens 0-7: channels 0-7, 8-15 of the group; tokens 8-15: channels 0-7, 8-15
                            ldmatrix_x4_trans((v_row ^ (uint32_t)(((2 * c) & 7) << 4)) + (c >> 2) * 8192, vb);
                            mma_bf16_full(o[c], vb[0], vb[1], vb[2], vb[3], pb[blk][0], pb[blk][1]);
                        }
                    }
                }
            };
            if (wtok0 < end) {
                if (kByPosition && pos_evict) {
                    for (int tok = wtok0 + lane; tok < min(end, wtok0 + kWarpSpan); tok += 32) {
                        if (tok == hs.f) continue;
                        const int ps = p.pos[row0 + tok];
                        if (ps >= p.n_sink && ps <= window_from && ps < old_pos) { old_pos = ps; old_slot = tok; }
                    }
                }
                const bool inside = wtok0 + kWarpSpan <= end;
                const bool has_hole = hole >= wtok0 && hole < wtok0 + kWarpSpan;
                const bool has_slot = hs.do_append && hs.f >= wtok0 && hs.f < wtok0 + kWarpSpan;
                if (inside && !has_hole && !has_slot) stage_body(std::false_type{});
                else stage_body(std::true_type{});
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bar_empty[s]));
        }
        if (!alive && lane == 0) sm_abort = 1;
    }
    __syncthreads();
    const int psz = partial_floats(G, D);                   // o, m, l, and the chunk's oldest evictable row
    float* part = p.partial + (int64_t)blockIdx.x * psz;
    const bool aborted = sm_abort != 0;                     // a bounded wait gave up: the status word says so
    if (aborted) {
        // The head's step is lost, but the launch stays consistent: no copy into this CTA's shared memory may be
        // left in flight when it exits (bounded wait for every tile that was requested), and the chunk still
        // arrives, with a mark, so that the head's counters return to zero and its bookkeeping is skipped.
        if (tid == 0)
            for (int t = max(0, sm_issued - kNS); t < sm_issued; ++t)
                mbar_wait(smem_u32(&bar_full[t % kNS]), (t / kNS) & 1, p.wait_cycles);
        if (tid < G) part[G * D + tid] = __int_as_float(0x7fc00000);
    }
    if (!aborted) {
    // ---- the four warps' states -> one partial for the chunk (the ring is idle now: reuse it)
    float* sm_o = reinterpret_cast<float*>(ring_ptr);       // [kConsumerWarps][G][D]
    if (warp < kConsumerWarps) {
        if (kByPosition && pos_evict) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                const int op = __shfl_xor_sync(0xffffffffu, old_pos, off);
                const int os = __shfl_xor_sync(0xffffffffu, old_slot, off);
                if (op < old_pos) { old_pos = op; old_slot = os; }
            }
            if (lane == 0) { sm_old_pos[warp] = old_pos; sm_old_slot[warp] = old_slot; }
        }
        // the sums were kept per lane (its own token rows): add them up over the eight row groups
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            l_run[e] += __shfl_xor_sync(0xffffffffu, l_run[e], 4);
            l_run[e] += __shfl_xor_sync(0xffffffffu, l_run[e], 8);
            l_run[e] += __shfl_xor_sync(0xffffffffu, l_run[e], 16);
        }
        const float sv_ = kFp8 ? p.kv_scale[u.head * 4 + 2] : 1.0f;
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int head = 2 * t4 + e;
            if (head < G) {
                float* dst = sm_o + (warp * G + head) * D;
#pragma unroll
                for (int c = 0; c < D / 16; ++c) {
                    if (kFp8) {                             // rows g and g + 8 of the MMA are channels 2 g and 2 g + 1
                        *reinterpret_cast<float2*>(dst + 16 * c + 2 * g8) = make_float2(o[c][e] * sv_, o[c][2 + e] * sv_);
                    } else {
                        dst[16 * c + g8] = o[c][e];
                        dst[16 * c + 8 + g8] = o[c][2 + e];
                    }
                }
                if (g8 == 0) { sm_m[warp][head] = m_run[e]; sm_l[warp][head] = l_run[e]; }
            }
        }
    }
    __syncthreads();
    for (int i = tid; i < G * D; i += kThreads) {
        const int a = i / D, d = i - a * D;
        float mm = -INFINITY;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) mm = fmaxf(mm, sm_m[w][a]);
        float acc = 0.0f, lsum = 0.0f;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) {
            const float c = (sm_m[w][a] == -INFINITY) ? 0.0f : exp2f(sm_m[w][a] - mm);
            acc = fmaf(sm_o[(w * G + a) * D + d], c, acc);
            lsum = fmaf(sm_l[w][a], c, lsum);
        }
        part[i] = acc;
        if (d == 0) { part[G * D + a] = mm; part[G * D + G + a] = lsum; }
    }
    if (kByPosition && pos_evict && tid == 0) {
        int bp = INT32_MAX, bs = -1;
        for (int w = 0; w < kConsumerWarps; ++w)
            if (sm_old_pos[w] < bp) { bp = sm_old_pos[w]; bs = sm_old_slot[w]; }
        part[G * D + 2 * G] = __int_as_float(bp);
        part[G * D + 2 * G + 1] = __int_as_float(bs);
    }
    }
    __syncthreads();                                        // the whole partial is written ...
    if (tid == 0) sm_last = (arrive_acq_rel(p.arrive + unit) == active - 1);   // ... and published with the arrival
    __syncthreads();
    if (!sm_last) return;

    // ---- this CTA delivered the head's last partial and finishes the head
    finish_head<D, kByPosition>(&p, reinterpret_cast<float*>(ring_ptr), unit, piece, active);   // the ring is idle now
}

// ---------------------------------------------------------------- steps 3-4 as a kernel of their own
// A short launch (one layer of one sequence) ends with a few long heads, and one CTA sweeping a long head would
// be most of the call's time.  There the attention kernel stops after the heads' final statistics and this
// kernel follows: one CTA per piece of a head does the score update of its rows and merges its share of the
// output columns; the CTA that finishes a head last picks the head's victim among the pieces' candidates and
// does the bookkeeping.
__global__ void __launch_bounds__(kThreads) sweep_kernel(const DecodeParams p) {
    constexpr int kG = BAKLAVA_MAX_GROUP;
    __shared__ float sm_M[kG];
    __shared__ float sm_invL[kG];
    __shared__ unsigned long long sm_key[kThreads / 32];
    __shared__ int sm_slot[kThreads / 32];
    __shared__ int sm_last;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = p.G;
    launch_dependents();                                  // what follows waits for this grid by itself
    // The piece and the head's state are read while the attention kernel is still running: that kernel (never an
    // overlapping call here) released this one only after its own dependency wait, so the previous step's
    // bookkeeping is complete, and it leaves len / free_slot alone when this kernel follows.
    const int4 item = p.items[p.n_items + blockIdx.x];
    const int unit = item.x, begin = item.y, chunk_len = item.z, piece = item.w & 0xffff;
    const Unit u = decode_unit(p, unit);
    const int t_pos = p.t_pos_seq ? p.t_pos_seq[u.b] : p.t_pos;
    const HeadState hs = head_state(p, u);
    const int C = hs.C, n = hs.n, n_hi = hs.n_att;
    const int active = n_hi > 0 ? (n_hi + chunk_len - 1) / chunk_len : 1;
    const int end = min(begin + chunk_len, n_hi);
    const int64_t row0 = (int64_t)u.b * p.seq_stride + p.slab_off[u.head];
    if (tid == 0 || !(hs.bad || t_pos < 0 || piece >= active))
        grid_dependency_wait();                           // the attention kernel: statistics, scratch, partials, appended rows
    if (hs.bad || t_pos < 0) return;                      // reported by the attention kernel / idle sequence
    if (piece >= active) return;
    const float* stats = p.stats + (int64_t)unit * kStatsStride;
    if (tid < G) {
        sm_M[tid] = stats[tid];
        sm_invL[tid] = stats[kG + tid];
    }
    const int D = p.D;
    const int psz = partial_floats(G, D);
    const float* part0 = p.partial + (int64_t)reinterpret_cast<const int32_t*>(stats)[2 * kG] * psz;
    const int n_chunks = reinterpret_cast<const int32_t*>(stats)[2 * kG + 1];
    __syncthreads();
    const bool lost = sm_M[0] != sm_M[0];                  // the attention kernel gave the head's step up
    const bool appended = hs.do_append && !lost;
    const bool evict = appended && (p.flags & BAKLAVA_FLAG_NO_EVICT) == 0 && n_hi > C - 1;
    const int newest_candidate = t_pos - max(0, (int)(((int64_t)(C - 1 - p.n_sink) * p.recent_num) / p.recent_den));
    if (!lost && begin < end) {
        const float* logit_h = p.logit + row0 * G;
        float* score = p.score + row0;
        const int32_t* pos = p.pos + row0;
        switch (G) {
            case 1: sweep_head<1>(logit_h, score, pos, p.n_sink, C, begin, end, hs.hole, evict, newest_candidate, sm_M, sm_invL, sm_key, sm_slot); break;
            case 2: sweep_head<2>(logit_h, score, pos, p.n_sink, C, begin, end, hs.hole, evict, newest_candidate, sm_M, sm_invL, sm_key, sm_slot); break;
            case 3: sweep_head<3>(logit_h, score, pos, p.n_sink, C, begin, end, hs.hole, evict, newest_candidate, sm_M, sm_invL, sm_key, sm_slot); break;
            case 4: sweep_head<4>(logit_h, score, pos, p.n_sink, C, begin, end, hs.hole, evict, newest_candidate, sm_M, sm_invL, sm_key, sm_slot); break;
            case 5: sweep_head<5>(logit_h, score, pos, p.n_sink, C, begin, end, hs.hole, evict, newest_candidate, sm_M, sm_invL, sm_key, sm_slot); break;
            case 6: sweep_head<6>(logit_h, score, pos, p.n_sink, C, begin, end, hs.hole, evict, newest_candidate, sm_M, sm_invL, sm_key, sm_slot); break;
            case 7: sweep_head<7>(logit_h, score, pos, p.n_sink, C, begin, end, hs.hole, evict, newest_candidate, sm_M, sm_invL, sm_key, sm_slot); break;
            default: sweep_head<8>(logit_h, score, pos, p.n_sink, C, begin, end, hs.hole, evict, newest_candidate, sm_M, sm_invL, sm_key, sm_slot); break;
        }
    } else if (lane == 0) {
        sm_key[warp] = ~0ull;
        sm_slot[warp] = -1;
    }
    // ---- this piece's share of the output: column groups [lo, hi) of the g * D / 4 four-element groups, summed
    // over the chunks.  Up to kMergeSplit threads share a group (each takes every P-th chunk, in ascending
    // order) and the group's first thread adds their sums in thread order: the result does not depend on timing.
    if (!lost) {
        constexpr int kMergeSplit = 16;
        __shared__ float4 sm_acc[kThreads];
        const int n_grp = G * D / 4;
        const int lo = (int)(((int64_t)piece * n_grp) / active), hi = (int)(((int64_t)(piece + 1) * n_grp) / active);
        __nv_bfloat16* orow = p.out + ((int64_t)(u.li * p.B + u.b) * p.Hq + u.h * G) * D;
        for (int g0 = lo; g0 < hi; g0 += kThreads) {
            const int n_here = min(kThreads, hi - g0);
            const int P = max(1, min(min(kMergeSplit, kThreads / n_here), n_chunks));
            const int gl = tid / P, r = tid - gl * P;
            const bool on = gl < n_here;
            const int grp = g0 + gl;
            const int a = on ? (grp * 4) / D : 0;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            if (on) {
                const float Ma = sm_M[a];
#pragma unroll 4
                for (int c = r; c < n_chunks; c += P) {
                    const float* pc = part0 + (int64_t)c * psz;
                    const float mc = __ldcg(pc + G * D + a);
                    const float4 oc = __ldcg(reinterpret_cast<const float4*>(pc) + grp);
                    const float wgt = (mc == -INFINITY) ? 0.0f : exp2f(mc - Ma);
                    acc.x = fmaf(oc.x, wgt, acc.x); acc.y = fmaf(oc.y, wgt, acc.y);
                    acc.z = fmaf(oc.z, wgt, acc.z); acc.w = fmaf(oc.w, wgt, acc.w);
                }
            }
            sm_acc[tid] = acc;
            __syncthreads();
            if (on && r == 0) {
                for (int k = 1; k < P; ++k) {
                    const float4 o2 = sm_acc[tid + k];
                    acc.x += o2.x; acc.y += o2.y; acc.z += o2.z; acc.w += o2.w;
                }
                const float inv = sm_invL[a];
                const __nv_bfloat162 lo2 = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
                const __nv_bfloat162 hi2 = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
                uint2 packed;
                packed.x = *reinterpret_cast<const uint32_t*>(&lo2);
                packed.y = *reinterpret_cast<const uint32_t*>(&hi2);
                *reinterpret_cast<uint2*>(orow + grp * 4) = packed;
            }
            __syncthreads();
        }
    }
    __syncthreads();
    if (!lost && begin < end) {                             // this piece's probabilities are spent
        const char* h0 = reinterpret_cast<const char*>(p.logit + row0 * G);
        for (int a = 0; a < G; ++a)
            drop_lines<kThreads>(h0 + ((size_t)a * C + begin) * 2, h0 + ((size_t)a * C + end) * 2);
    }
    if (tid == 0) {
        unsigned long long bk = ~0ull;
        int bs = -1;
        for (int w = 0; w < kThreads / 32; ++w)
            if (sm_key[w] < bk) { bk = sm_key[w]; bs = sm_slot[w]; }
        p.best_key[blockIdx.x] = bk;
        p.best_slot[blockIdx.x] = bs;
        sm_last = (arrive_acq_rel(p.arrive + unit) == active - 1);
    }
    __syncthreads();
    if (!sm_last || warp != 0) return;
    // the head's victim among the pieces' candidates: lanes take every 32nd piece, then the warp reduces
    unsigned long long bk = ~0ull;
    int bs = -1;
    if (evict) {
        const int64_t first = (int64_t)blockIdx.x - piece;
        for (int c = lane; c < active; c += 32) {
            const unsigned long long kc = __ldcg(p.best_key + first + c);
            const int sc = __ldcg(p.best_slot + first + c);
            if (kc < bk) { bk = kc; bs = sc; }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const unsigned long long ok = __shfl_xor_sync(0xffffffffu, bk, off);
            const int os = __shfl_xor_sync(0xffffffffu, bs, off);
            if (ok < bk) { bk = ok; bs = os; }
        }
    }
    if (lane == 0) {
        if (appended) {
            if (evict && bs >= 0) {
                p.free_slot[u.st] = bs;                     // len stays n: one row in, one row out (Eq. 5-6)
            } else {
                if (evict) atomicOr(p.status, BAKLAVA_STATUS_BAD_STATE);   // capacity too small for sinks + window
                p.len[u.st] = n + 1;
                p.free_slot[u.st] = n + 1;
            }
        }
        p.arrive[unit] = 0;
    }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult res;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &res) != cudaSuccess ||
            res != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// bf16 [rows, D] row-major, boxes of 64 rows x 64 elements (128 bytes), 128-byte swizzle, zero fill
bool make_slab_map(CUtensorMap* map, void* base, int64_t rows, int D) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)D * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)kTileTokens};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// FP8 slabs: one byte per element, boxes of one stage's rows x 128 bytes (the whole row), 128-byte swizzle
bool make_slab_map_fp8(CUtensorMap* map, void* base, int64_t rows, int D) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)D};
    const cuuint32_t box[2] = {128, (cuuint32_t)kFp8StageTokens};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, bool kByPosition, bool kFp8 = false>
cudaError_t launch_chunks(const DecodeParams& p, const CUtensorMap& km, const CUtensorMap& vm, cudaStream_t s) {
    constexpr int kSmem = (kFp8 ? kFp8Stages * 2 * kFp8StageTokens * D : kStages * 2 * kTileTokens * D * 2) + 1024;
    // the attribute belongs to the function on the current device: set once per device and instantiation
    static std::atomic<uint64_t> configured{0};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 64 || !(configured.load(std::memory_order_acquire) >> dev & 1)) {
        e = cudaFuncSetAttribute(decode_chunk_kernel<D, kByPosition, kFp8>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
        if (e != cudaSuccess) return e;
        if (dev < 64) configured.fetch_or(1ull << dev, std::memory_order_release);
    }
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.n_items);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmem;
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, decode_chunk_kernel<D, kByPosition, kFp8>, p, km, vm);
}

}  // namespace

namespace {
std::atomic<long long> g_wait_cycles{ptx::kWaitCycles};

int decode_attn_impl(
        const baklava_shape* shape, const baklava_cache* cache,
        const void* q, const void* k_new, const void* v_new, int32_t t_pos, const int32_t* t_pos_seq,
        void* out, float* lse, uint32_t flags,
        const int32_t* items, const baklava_plan_info* info,
        void* ws, size_t ws_bytes, void* stream) {
    int rc = baklava_check_shape(shape);
    if (rc) return rc;
    if (!cache || !q || !out || !items || !info || !ws) return BAKLAVA_ERR_INVALID_ARG;
    if (flags & ~(BAKLAVA_FLAG_NO_APPEND | BAKLAVA_FLAG_NO_SCORE | BAKLAVA_FLAG_NO_EVICT | BAKLAVA_FLAG_OVERLAP_PREV |
                  BAKLAVA_FLAG_TEST_STALL))
        return BAKLAVA_ERR_INVALID_ARG;
    const bool no_append = flags & BAKLAVA_FLAG_NO_APPEND;
    if (!no_append && (!k_new || !v_new)) return BAKLAVA_ERR_INVALID_ARG;
    if (!cache->k_slab || !cache->v_slab || !cache->pos || !cache->score || !cache->len || !cache->free_slot ||
        !cache->cap || !cache->slab_off || !cache->status || cache->B <= 0 || cache->seq_stride_tokens <= 0)
        return BAKLAVA_ERR_INVALID_ARG;
    const void* ptrs[] = {q, k_new, v_new, out, cache->k_slab, cache->v_slab, cache->pos, cache->score, items, ws};
    for (const void* ptr : ptrs)
        if (ptr && !baklava_aligned16(ptr)) return BAKLAVA_ERR_INVALID_ARG;
    if (cache->seq_stride_tokens % 16 != 0) return BAKLAVA_ERR_INVALID_ARG;   // rows of pos / score go in 16-byte vectors
    if (info->layer_begin < 0 || info->layer_end > shape->L || info->layer_begin >= info->layer_end ||
        info->B != cache->B || info->n_items <= 0 || info->n_score_items < 0 ||
        info->n_units != (info->layer_end - info->layer_begin) * cache->B * shape->Hkv)
        return BAKLAVA_ERR_INVALID_ARG;
    const int64_t rows = (int64_t)cache->B * cache->seq_stride_tokens;
    if (rows > INT32_MAX) return BAKLAVA_ERR_UNSUPPORTED;
    DecodeWorkspace lay;
    const size_t need = baklava_decode_ws_bytes(shape, info->n_items, info->n_score_items, info->n_units, cache->B,
                                                cache->seq_stride_tokens, &lay);
    if (ws_bytes < need) return BAKLAVA_ERR_WORKSPACE;

    const bool quantised = cache->kv_dtype == BAKLAVA_KV_FP8_E4M3;
    if (cache->kv_dtype != BAKLAVA_KV_BF16 && !quantised) return BAKLAVA_ERR_INVALID_ARG;
    if (quantised && !cache->kv_scale) return BAKLAVA_ERR_INVALID_ARG;
    if (quantised && shape->D != 128) return BAKLAVA_ERR_UNSUPPORTED;
    CUtensorMap k_map, v_map;
    if (quantised) {
        if (!make_slab_map_fp8(&k_map, cache->k_slab, rows, shape->D) || !make_slab_map_fp8(&v_map, cache->v_slab, rows, shape->D))
            return BAKLAVA_ERR_CUDA;
    } else if (!make_slab_map(&k_map, cache->k_slab, rows, shape->D) || !make_slab_map(&v_map, cache->v_slab, rows, shape->D)) {
        return BAKLAVA_ERR_CUDA;
    }

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
    p.L = shape->L; p.Hq = shape->Hq; p.Hkv = shape->Hkv; p.G = shape->Hq / shape->Hkv;
    p.D = shape->D;
    p.n_sink = shape->n_sink; p.recent_num = shape->recent_num; p.recent_den = shape->recent_den;
    p.layer_begin = info->layer_begin;
    p.layers = info->layer_end - info->layer_begin;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k_new = static_cast<const __nv_bfloat16*>(k_new);
    p.v_new = static_cast<const __nv_bfloat16*>(v_new);
    p.out = static_cast<__nv_bfloat16*>(out);
    p.lse = lse;
    p.t_pos = t_pos;
    p.t_pos_seq = t_pos_seq;
    // without scores only the pure sinks + window policy can still choose a victim (by position)
    p.window_evict = (flags & BAKLAVA_FLAG_NO_SCORE) && !(flags & BAKLAVA_FLAG_NO_EVICT) &&
                     shape->recent_num == shape->recent_den;
    p.flags = ((flags & BAKLAVA_FLAG_NO_SCORE) && !p.window_evict) ? (flags | BAKLAVA_FLAG_NO_EVICT) : flags;
    p.items = reinterpret_cast<const int4*>(items);
    p.n_items = info->n_items;
    char* base = static_cast<char*>(ws);
    p.arrive = reinterpret_cast<int32_t*>(base + lay.arrive_off);
    p.partial = reinterpret_cast<float*>(base + lay.partial_off);
    p.logit = reinterpret_cast<float*>(base + lay.logit_off);
    p.stats = reinterpret_cast<float*>(base + lay.stats_off);
    p.best_key = reinterpret_cast<unsigned long long*>(base + lay.best_off);
    p.best_slot = reinterpret_cast<int32_t*>(base + lay.best_off + 8 * (size_t)info->n_score_items);
    // A short launch that may not overlap what follows it ends in a kernel of its own for the score update
    // (the plan lists its pieces); otherwise the CTA that finishes a head does it all.
    p.split_tail = info->n_score_items > 0 && !(p.flags & (BAKLAVA_FLAG_NO_SCORE | BAKLAVA_FLAG_OVERLAP_PREV));
    p.scale_log2 = kLog2e / sqrtf((float)shape->D);
    p.kv_scale = cache->kv_scale;
    p.wait_cycles = g_wait_cycles.load(std::memory_order_relaxed);

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t err = cudaSuccess;
    if (quantised) err = p.window_evict ? launch_chunks<128, true, true>(p, k_map, v_map, s) : launch_chunks<128, false, true>(p, k_map, v_map, s);
    else if (p.window_evict) err = shape->D == 128 ? launch_chunks<128, true>(p, k_map, v_map, s) : launch_chunks<64, true>(p, k_map, v_map, s);
    else err = shape->D == 128 ? launch_chunks<128, false>(p, k_map, v_map, s) : launch_chunks<64, false>(p, k_map, v_map, s);
    if (err != cudaSuccess) return BAKLAVA_ERR_CUDA;
    if (p.split_tail) {
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)info->n_score_items);
        cfg.blockDim = dim3(kThreads);
        cfg.stream = s;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, sweep_kernel, p) != cudaSuccess) return BAKLAVA_ERR_CUDA;
    }
    if (cudaGetLastError() != cudaSuccess) return BAKLAVA_ERR_CUDA;
    return BAKLAVA_OK;
}
}  // namespace

extern "C" __attribute__((visibility("default"))) int baklava_decode_attn(
        const baklava_shape* shape, const baklava_cache* cache,
        const void* q, const void* k_new, const void* v_new, int32_t t_pos,
        void* out, float* lse, uint32_t flags,
        const int32_t* items, const baklava_plan_info* info,
        void* ws, size_t ws_bytes, void* stream) {
    if (t_pos < 0) return BAKLAVA_ERR_INVALID_ARG;
    return decode_attn_impl(shape, cache, q, k_new, v_new, t_pos, nullptr, out, lse, flags, items, info, ws, ws_bytes,
                            stream);
}

extern "C" __attribute__((visibility("default"))) int baklava_decode_attn_varlen(
        const baklava_shape* shape, const baklava_cache* cache,
        const void* q, const void* k_new, const void* v_new, const int32_t* t_pos,
        void* out, float* lse, uint32_t flags,
        const int32_t* items, const baklava_plan_info* info,
        void* ws, size_t ws_bytes, void* stream) {
    if (!t_pos) return BAKLAVA_ERR_INVALID_ARG;
    return decode_attn_impl(shape, cache, q, k_new, v_new, 0, t_pos, out, lse, flags, items, info, ws, ws_bytes,
                            stream);
}

extern "C" __attribute__((visibility("default"))) int baklava_set_wait_limit(int64_t sm_cycles) {
    if (sm_cycles <= 0) return BAKLAVA_ERR_INVALID_ARG;
    g_wait_cycles.store(sm_cycles, std::memory_order_relaxed);
    return BAKLAVA_OK;
}
