// Seed of the heavy-hitter scores: the attention mass every prompt token received while the prompt was
// processed, i.e. the column sums of the causal attention matrix of Eq. 1, added over the g query heads
// that share a KV head.
//
// Two passes over Q K^T (V is not needed; one pass when the caller brings the rows' log-sum-exp), both on the
// 5th-generation tensor cores.  A CTA keeps one
// 128-row operand tile resident in shared memory and streams the other operand's tiles through a
// two-stage TMA ring; one thread issues tcgen05.mma into a double-buffered 128 x 128 fp32 accumulator in
// tensor memory; two groups of four epilogue warps, one per accumulator, read it back with tcgen05.ld, a thread
// owning an accumulator row of every other tile.
//   pass 1 (rows = queries): every query row's log-sum-exp, a running max / sum kept by its thread;
//   pass 2 (rows = keys):    exp2(logit - lse[query]) summed along each key's row, again by its thread.
// The only reduction across threads joins the two groups' shares of a row in a fixed order, so the result is
// reproducible bit for bit.
#include <cmath>
#include <cstdint>

#include "baklava.h"
#include "common.h"
#include "ptx.cuh"

namespace {

using namespace ptx;

constexpr int kTileRows = 128;       // rows of an operand tile = accumulator rows = accumulator columns
constexpr int kThreads = 320;        // warp 0: TMA producer, warp 1: MMA issuer + TMEM owner, warps 2-9: epilogue
constexpr int kEpilogueThreads = 256; // two groups of 128, one per accumulator; a thread owns an accumulator row
constexpr uint32_t kTmemColumns = 256;   // two 128-column accumulators
constexpr float kLog2e = 1.4426950408889634f;
constexpr int kPassLse = 0, kPassColumnSums = 1, kPassRowMax = 2;   // row passes: kPassLse and kPassRowMax

// 2^x on the special-function unit (one instruction; -inf gives 0)
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

struct PrefillParams {
    const int32_t* prompt_len;   // [B] or null
    float* lse2;                 // [B, Hq, T] log2-domain log-sum-exp of every query row (+inf past the prompt)
    const float* lse_nat;        // caller's natural-log log-sum-exp [B, Hq, T] (then lse2 is not used), or null
    float* score;                // [B, Hkv, T]
    uint32_t* error;
    int32_t B, T, Hq, Hkv, n_blk;
    float scale_log2;
};

// One CTA's work: the row block / key block (bx, by, bz) of the grid the pass is normally launched with.
template <int D, int PASS>
__device__ __forceinline__ void qk_pass_block(const PrefillParams& p, const CUtensorMap& q_map, const CUtensorMap& k_map,
                                              const int bx, const int by, const int bz) {
    constexpr int kKSteps = D / 16;                         // one MMA covers 16 elements of the head dimension
    constexpr int kBoxBytes = kTileRows * 128;              // one TMA box: 128 rows x 64 elements
    constexpr int kTileBytes = kTileRows * D * 2;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_res, bar_full[2], bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t tmem_slot;
    __shared__ __align__(16) float sm_lse[2][2][kTileRows];   // [group][tile parity inside the group][streamed row]
    __shared__ int sm_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = p.Hq / p.Hkv;
    const int b = bz;
    const int len = p.prompt_len ? min(max(p.prompt_len[b], 0), p.T) : p.T;
    int blk, n_it, nq = 1, head_res, head_first;            // resident block, streamed tiles, heads
    if (PASS != kPassColumnSums) {
        blk = p.n_blk - 1 - bx;                             // long rows of the causal triangle first
        const int h = by;
        head_res = b * p.Hq + h;
        head_first = b * p.Hkv + h / g;
        n_it = blk + 1;
        if (blk * kTileRows >= len) {
            for (int r = tid; r < kTileRows; r += kThreads)
                if (blk * kTileRows + r < p.T) p.lse2[(int64_t)head_res * p.T + blk * kTileRows + r] = INFINITY;
            return;
        }
    } else {
        blk = bx;                                           // early key blocks meet the most query tiles: first
        const int kvh = by;
        head_res = b * p.Hkv + kvh;
        head_first = b * p.Hq + kvh * g;
        if (blk * kTileRows >= len) {                       // keys past the prompt receive nothing
            for (int r = tid; r < kTileRows; r += kThreads)
                if (blk * kTileRows + r < p.T) p.score[(int64_t)head_res * p.T + blk * kTileRows + r] = 0.0f;
            return;
        }
        nq = (len + kTileRows - 1) / kTileRows - blk;       // query tiles of the prompt at or below this key block
        n_it = g * nq;
    }
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t res_tile = base;
    if (tid == 0) {
        mbar_init(smem_u32(&bar_res), 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_acc_full[s]), 1);
            mbar_init(smem_u32(&bar_acc_empty[s]), kEpilogueThreads / 64);   // the four warps of accumulator s
        }
        sm_abort = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tc::tmem_alloc(smem_u32(&tmem_slot), kTmemColumns);
        tc::tmem_relinquish();
    }
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    const uint32_t tmem_base = tmem_slot;

    // which streamed tile iteration `it` is: (head of the group, row block)
    auto stream_head = [&](int it) { return PASS != kPassColumnSums ? head_first : head_first + it / nq; };
    auto stream_blk = [&](int it) { return PASS != kPassColumnSums ? it : blk + it % nq; };

    if (warp == 0) {
        // ---------------- TMA producer
        if (lane == 0) {
            const CUtensorMap* res_map = PASS != kPassColumnSums ? &q_map : &k_map;
            const CUtensorMap* str_map = PASS != kPassColumnSums ? &k_map : &q_map;
            mbar_arrive_expect_tx(smem_u32(&bar_res), kTileBytes);
#pragma unroll
            for (int bx = 0; bx < D / 64; ++bx)
                tma_load_3d(res_tile + bx * kBoxBytes, res_map, bx * 64, blk * kTileRows, head_res, smem_u32(&bar_res));
            for (int it = 0; it < n_it; ++it) {
                const int s = it & 1;
                // the stage is free once the MMAs of the tile two back have completed: their commit says so
                if (it >= 2 && !mbar_wait(smem_u32(&bar_acc_full[s]), ((it >> 1) - 1) & 1)) { sm_abort = 1; break; }
                const uint32_t bar = smem_u32(&bar_full[s]);
                mbar_arrive_expect_tx(bar, kTileBytes);
#pragma unroll
                for (int bx = 0; bx < D / 64; ++bx)
                    tma_load_3d(base + (1 + s) * kTileBytes + bx * kBoxBytes, str_map, bx * 64,
                                stream_blk(it) * kTileRows, stream_head(it), bar);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer: D[128 x 128] = resident (A) x streamed^T (B), both K-major
        if (lane == 0) {
            constexpr uint32_t idesc = tc::idesc_bf16_f32(kTileRows, kTileRows);
            bool ok = mbar_wait(smem_u32(&bar_res), 0);
            for (int it = 0; it < n_it && ok; ++it) {
                const int s = it & 1;
                ok = mbar_wait(smem_u32(&bar_full[s]), (it >> 1) & 1);
                if (ok && it >= 2) ok = mbar_wait(smem_u32(&bar_acc_empty[s]), ((it >> 1) - 1) & 1);
                if (!ok) break;
                tc::fence_after_sync();
                const uint32_t str_tile = base + (1 + s) * kTileBytes;
                const uint64_t da = tc::desc_k_major_sw128(res_tile), db = tc::desc_k_major_sw128(str_tile);
#pragma unroll
                for (int ks = 0; ks < kKSteps; ++ks) {
                    // 64-element span, then 32 B per step; the descriptor's address field counts 16-byte units
                    const uint32_t off = ((ks >> 2) * kBoxBytes + (ks & 3) * 32) >> 4;
                    tc::umma_bf16(tmem_base + s * kTileRows, da + off, db + off, idesc, ks > 0);
                }
                // one commit per tile (a commit costs the tensor pipe about as much as a third of this tile's
                // MMAs): it tells the epilogue that the accumulator is complete and the producer that the stage is free
                tc::umma_commit(smem_u32(&bar_acc_full[s]));
            }
            if (!ok) sm_abort = 1;
        }
    } else {
        // ---------------- epilogue: a warp reads its quarter of the TMEM lanes (thread = accumulator row).
        // Warps 2-5 take the tiles of accumulator 0 (the even ones), warps 6-9 those of accumulator 1: the two groups
        // never wait for each other, so one of them has exponentials to do while the other waits for its next tile.
        const int grp = (warp - 2) >> 2;
        const int row = 32 * (warp & 3) + lane;              // = this thread's index inside its group
        const uint32_t lane_addr = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16) + grp * kTileRows;
        float m_run = -INFINITY, l_run = 0.0f, colsum = 0.0f;
        auto fetch_lse = [&](int it) -> float {              // the log-sum-exp of streamed query row `row` of tile it
            const int t = stream_blk(it) * kTileRows + row;
            if (p.lse_nat)                                   // the caller's own (natural logarithm; rows past the prompt: none)
                return t < len ? p.lse_nat[(int64_t)stream_head(it) * p.T + t] * kLog2e : INFINITY;
            return t < p.T ? p.lse2[(int64_t)stream_head(it) * p.T + t] : INFINITY;
        };
        auto group_barrier = [&]() {
            if (grp == 0) asm volatile("bar.sync 1, 128;" ::: "memory");
            else asm volatile("bar.sync 2, 128;" ::: "memory");
        };
        if (PASS == kPassColumnSums) {
            if (grp < n_it) sm_lse[grp][0][row] = fetch_lse(grp);
            group_barrier();
        }
        bool ok = true;
        for (int it = grp; it < n_it; it += 2) {
            const int par = (it >> 1) & 1;
            float next_lse = 0.0f;
            if (PASS == kPassColumnSums && it + 2 < n_it) next_lse = fetch_lse(it + 2);
            if (!mbar_wait(smem_u32(&bar_acc_full[grp]), par)) { ok = false; break; }
            tc::fence_after_sync();
            const bool diagonal = stream_blk(it) == blk;
            if (PASS == kPassRowMax) {
                // row = query, columns = keys: only the largest logit of the row is wanted (no exponentials)
#pragma unroll
                for (int c0 = 0; c0 < kTileRows; c0 += 32) {
                    uint32_t v[32];
                    tc::tmem_ld_32x32(lane_addr + c0, v);
                    tc::tmem_ld_wait();
                    if (diagonal) {
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c0 + c > row) v[c] = 0xff800000u;    // -inf
                    }
                    float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int c = 0; c < 32; ++c) mx[c & 3] = fmaxf(mx[c & 3], __uint_as_float(v[c]));
                    m_run = fmaxf(m_run, fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])));
                }
            } else if (PASS == kPassLse) {
                // row = query, columns = keys: keys above the query are masked on the diagonal tile.
                // Online softmax statistics, 32 columns at a time.
#pragma unroll
                for (int c0 = 0; c0 < kTileRows; c0 += 32) {
                    uint32_t v[32];
                    tc::tmem_ld_32x32(lane_addr + c0, v);
                    tc::tmem_ld_wait();
                    if (diagonal) {                            // keys above the query do not exist for it
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (c0 + c > row) v[c] = 0xff800000u;    // -inf
                    }
                    float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int c = 0; c < 32; ++c) mx[c & 3] = fmaxf(mx[c & 3], __uint_as_float(v[c]));
                    const float m_new = fmaxf(m_run, fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * p.scale_log2);
                    if (m_new != -INFINITY) {                 // (a diagonal tile's first rows see none of the upper columns)
                        float sum[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            sum[c & 3] += fast_exp2(fmaf(__uint_as_float(v[c]), p.scale_log2, -m_new));
                        l_run = l_run * fast_exp2(m_run - m_new) + ((sum[0] + sum[1]) + (sum[2] + sum[3]));
                        m_run = m_new;
                    }
                }
            } else {
                // row = key, columns = queries: queries before the key are masked on the diagonal tile;
                // queries past the prompt carry lse = +inf and contribute exp2(-inf) = 0
                const float* lse = sm_lse[grp][par];
#pragma unroll
                for (int c0 = 0; c0 < kTileRows; c0 += 64) {
                    uint32_t v0[32], v1[32];                 // 64 columns of the tile at a time
                    tc::tmem_ld_32x32(lane_addr + c0, v0);
                    tc::tmem_ld_32x32(lane_addr + c0 + 32, v1);
                    tc::tmem_ld_wait();
                    if (diagonal) {                            // queries before the key do not see it
#pragma unroll
                        for (int c = 0; c < 32; ++c) {
                            if (row > c0 + c) v0[c] = 0xff800000u;               // -inf
                            if (row > c0 + 32 + c) v1[c] = 0xff800000u;
                        }
                    }
                    float sum[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                    const float4* lse4 = reinterpret_cast<const float4*>(lse + c0);
#pragma unroll
                    for (int c4 = 0; c4 < 8; ++c4) {           // four streamed rows' log-sum-exp per shared-memory load
                        const float4 la = lse4[c4], lb = lse4[8 + c4];
                        const float l0[4] = {la.x, la.y, la.z, la.w}, l1[4] = {lb.x, lb.y, lb.z, lb.w};
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            sum[k] += fast_exp2(fmaf(__uint_as_float(v0[4 * c4 + k]), p.scale_log2, -l0[k]));
                            sum[(k + 2) & 3] += fast_exp2(fmaf(__uint_as_float(v1[4 * c4 + k]), p.scale_log2, -l1[k]));
                        }
                    }
                    colsum += (sum[0] + sum[1]) + (sum[2] + sum[3]);
                }
            }
            tc::fence_before_sync();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(smem_u32(&bar_acc_empty[grp]));
            if (PASS == kPassColumnSums) {
                sm_lse[grp][par ^ 1][row] = next_lse;         // (the buffer of this group's tile before this one)
                group_barrier();
            }
        }
        // join the two groups' shares of every row: the second group hands its state over through shared memory
        asm volatile("bar.sync 3, 256;" ::: "memory");
        if (grp == 1) { sm_lse[0][0][row] = PASS != kPassColumnSums ? m_run : colsum; sm_lse[0][1][row] = l_run; }
        asm volatile("bar.sync 3, 256;" ::: "memory");
        if (!ok) {
            sm_abort = 1;
        } else if (grp == 0) {
            const int t = blk * kTileRows + row;
            if (PASS == kPassRowMax) {
                // scaled to the log2 domain like the log-sum-exp it stands in for
                if (t < p.T) p.lse2[(int64_t)head_res * p.T + t] = t < len ? fmaxf(m_run, sm_lse[0][0][row]) * p.scale_log2 : INFINITY;
            } else if (PASS == kPassLse) {
                const float m_hi = sm_lse[0][0][row], l_hi = sm_lse[0][1][row];
                const float m_all = fmaxf(m_run, m_hi);      // m_run is finite: tile 0, with key 0, belongs to the first group
                const float l_all = l_run * exp2f(m_run - m_all) + (m_hi == -INFINITY ? 0.0f : l_hi * exp2f(m_hi - m_all));
                if (t < p.T) p.lse2[(int64_t)head_res * p.T + t] = t < len ? m_all + log2f(l_all) : INFINITY;
            } else {
                if (t < p.T) p.score[(int64_t)head_res * p.T + t] = colsum + sm_lse[0][0][row];
            }
        }
    }
    tc::fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc::fence_after_sync();
        tc::tmem_dealloc(tmem_base, kTmemColumns);
    }
    if (tid == 0 && sm_abort) atomicOr(p.error, 1u);
    if (tid == 0) {                                         // the barriers may be set up again by the next block of this CTA
        mbar_inval(smem_u32(&bar_res));
        for (int s = 0; s < 2; ++s) {
            mbar_inval(smem_u32(&bar_full[s]));
            mbar_inval(smem_u32(&bar_acc_full[s]));
            mbar_inval(smem_u32(&bar_acc_empty[s]));
        }
    }
    __syncthreads();
}

template <int D, int PASS>
__global__ void __launch_bounds__(kThreads, 2) qk_pass_kernel(const PrefillParams p,
                                                           const __grid_constant__ CUtensorMap q_map,
                                                           const __grid_constant__ CUtensorMap k_map) {
    qk_pass_block<D, PASS>(p, q_map, k_map, blockIdx.x, blockIdx.y, blockIdx.z);
}

// The row-maximum pass over a list of row blocks (entries = flat index ((b * Hq + h) * n_blk + blk), count
// in *list_count): a small fixed grid whose CTAs take the entries in turn, so that an empty list costs nothing.
template <int D>
__global__ void __launch_bounds__(kThreads, 2) row_max_list_kernel(const PrefillParams p, const int32_t* list,
                                                                const int32_t* list_count,
                                                                const __grid_constant__ CUtensorMap q_map,
                                                                const __grid_constant__ CUtensorMap k_map) {
    const int n = *list_count;
    for (int w = blockIdx.x; w < n; w += gridDim.x) {
        const int flat = list[w];
        const int blk = flat % p.n_blk, h = (flat / p.n_blk) % p.Hq, b = flat / (p.n_blk * p.Hq);
        qk_pass_block<D, kPassRowMax>(p, q_map, k_map, p.n_blk - 1 - blk, h, b);
    }
}

template <int D, int PASS>
cudaError_t launch_pass(const PrefillParams& p, const CUtensorMap& qm, const CUtensorMap& km, dim3 grid, cudaStream_t s) {
    // at least 100 KB per CTA, so that never more than two CTAs (2 x 256 TMEM columns) share an SM
    constexpr int kSmem = (3 * kTileRows * D * 2 + 1024) > 100 * 1024 ? (3 * kTileRows * D * 2 + 1024) : 100 * 1024;
    cudaError_t e = cudaFuncSetAttribute(qk_pass_kernel<D, PASS>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    qk_pass_kernel<D, PASS><<<grid, kThreads, kSmem, s>>>(p, qm, km);
    return cudaGetLastError();
}

template <int D>
cudaError_t launch_prefill(const PrefillParams& p, const CUtensorMap& qm, const CUtensorMap& km, cudaStream_t s) {
    if (!p.lse_nat) {                                       // the rows' log-sum-exp first, unless the caller has it
        cudaError_t e = launch_pass<D, kPassLse>(p, qm, km, dim3(p.n_blk, p.Hq, p.B), s);
        if (e != cudaSuccess) return e;
    }
    return launch_pass<D, kPassColumnSums>(p, qm, km, dim3(p.n_blk, p.Hkv, p.B), s);
}

}  // namespace

// A row pass alone, for the profiling kernel: log2-domain largest logit of every causal query row
// (+inf past the prompt).  The cosine of Algorithm 1 does not depend on the scale of a head's output
// row, so the row maximum serves as the softmax's stabiliser and its sum is never needed.
int baklava_launch_row_max(const baklava_shape* shape, const void* q, const void* k, const int32_t* prompt_len,
                           int32_t B, int32_t T, float* lse2, const int32_t* list, const int32_t* list_count,
                           int32_t grid, uint32_t* error, cudaStream_t s) {
    PrefillParams p;
    p.prompt_len = prompt_len;
    p.error = error;
    p.lse2 = lse2;
    p.lse_nat = nullptr;
    p.score = nullptr;
    p.B = B; p.T = T; p.Hq = shape->Hq; p.Hkv = shape->Hkv;
    p.n_blk = (T + kTileRows - 1) / kTileRows;
    p.scale_log2 = kLog2e / sqrtf((float)shape->D);
    CUtensorMap qm, km;
    if (!make_head_map(&qm, q, (int64_t)B * shape->Hq, T, shape->D, kTileRows) ||
        !make_head_map(&km, k, (int64_t)B * shape->Hkv, T, shape->D, kTileRows))
        return BAKLAVA_ERR_CUDA;
    constexpr int kSmem128 = 100 * 1024, kSmem64 = 100 * 1024;   // as launch_pass: at most two CTAs (2 x 256 TMEM columns) per SM
    cudaError_t e;
    if (shape->D == 128) {
        e = cudaFuncSetAttribute(row_max_list_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem128);
        if (e == cudaSuccess) row_max_list_kernel<128><<<grid, kThreads, kSmem128, s>>>(p, list, list_count, qm, km);
    } else {
        e = cudaFuncSetAttribute(row_max_list_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem64);
        if (e == cudaSuccess) row_max_list_kernel<64><<<grid, kThreads, kSmem64, s>>>(p, list, list_count, qm, km);
    }
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? BAKLAVA_OK : BAKLAVA_ERR_CUDA;
}

extern "C" __attribute__((visibility("default"))) size_t baklava_prefill_workspace_size(const baklava_shape* shape,
                                                                                    int32_t B, int32_t T) {
    if (!shape || B <= 0 || T <= 0) return 0;
    return 256 + sizeof(float) * (size_t)B * shape->Hq * (size_t)T;
}

extern "C" __attribute__((visibility("default"))) int baklava_prefill_scores(
        const baklava_shape* shape, const void* q, const void* k, const int32_t* prompt_len, const float* lse,
        int32_t B, int32_t T, float* score, void* ws, size_t ws_bytes, void* stream) {
    int rc = baklava_check_shape(shape);
    if (rc) return rc;
    if (!q || !k || !score || !ws || B <= 0 || T <= 0) return BAKLAVA_ERR_INVALID_ARG;
    const void* ptrs[] = {q, k, ws};
    for (const void* ptr : ptrs)
        if (!baklava_aligned16(ptr)) return BAKLAVA_ERR_INVALID_ARG;
    if (lse && (reinterpret_cast<uintptr_t>(lse) & 3u)) return BAKLAVA_ERR_INVALID_ARG;
    if (B > 65535 || shape->Hq > 65535) return BAKLAVA_ERR_UNSUPPORTED;
    if (ws_bytes < baklava_prefill_workspace_size(shape, B, T)) return BAKLAVA_ERR_WORKSPACE;

    PrefillParams p;
    p.prompt_len = prompt_len;
    p.error = static_cast<uint32_t*>(ws);
    p.lse2 = reinterpret_cast<float*>(static_cast<char*>(ws) + 256);
    p.lse_nat = lse;
    p.score = score;
    p.B = B; p.T = T; p.Hq = shape->Hq; p.Hkv = shape->Hkv;
    p.n_blk = (T + kTileRows - 1) / kTileRows;
    p.scale_log2 = kLog2e / sqrtf((float)shape->D);

    CUtensorMap qm, km;
    if (!make_head_map(&qm, q, (int64_t)B * shape->Hq, T, shape->D, kTileRows) ||
        !make_head_map(&km, k, (int64_t)B * shape->Hkv, T, shape->D, kTileRows))
        return BAKLAVA_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(ws, 0, 256, s) != cudaSuccess) return BAKLAVA_ERR_CUDA;
    cudaError_t err = shape->D == 128 ? launch_prefill<128>(p, qm, km, s) : launch_prefill<64>(p, qm, km, s);
    return err == cudaSuccess ? BAKLAVA_OK : BAKLAVA_ERR_CUDA;
}
