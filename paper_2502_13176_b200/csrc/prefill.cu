// Seed of the heavy-hitter scores: the attention mass every prompt token received while the prompt was
// processed, i.e. the column sums of the causal attention matrix of Eq. 1, added over the g query heads
// that share a KV head.
//
// Two passes over Q K^T (V is not needed).  Pass 1 gives every query row its log-sum-exp; pass 2 owns
// key blocks: a CTA keeps 64 keys as the A operand in registers, streams every query tile at or below
// them through a two-stage TMA ring, turns logits into probabilities with the rows' log-sum-exp and
// adds them up per key.  Every sum has a fixed order, so the result is reproducible bit for bit.
#include <cmath>
#include <cstdint>

#include "baklava.h"
#include "common.h"
#include "ptx.cuh"

namespace {

using namespace ptx;

constexpr int kRows = 64;          // query rows / keys per tile
constexpr int kThreads = 128;
constexpr float kLog2e = 1.4426950408889634f;

struct PrefillParams {
    const int32_t* prompt_len;   // [B] or null
    float* lse2;                 // [B, Hq, T] log2-domain log-sum-exp of every query row (+inf past the prompt)
    float* score;                // [B, Hkv, T]
    uint32_t* error;
    int32_t B, T, Hq, Hkv, n_blk;
    float scale_log2;
};

// ---------------------------------------------------------------- pass 1: row log-sum-exp
template <int D>
__global__ void __launch_bounds__(kThreads) prefill_lse_kernel(const PrefillParams p,
                                                               const __grid_constant__ CUtensorMap q_map,
                                                               const __grid_constant__ CUtensorMap k_map) {
    constexpr int kKSteps = D / 16;
    constexpr int kTileBytes = kRows * D * 2;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_q;
    __shared__ __align__(8) uint64_t bar_k[2];
    __shared__ int sm_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int qb = p.n_blk - 1 - blockIdx.x;               // long rows of the causal triangle first
    const int h = blockIdx.y, b = blockIdx.z;
    const int kvh = h / (p.Hq / p.Hkv);
    const int len = p.prompt_len ? min(max(p.prompt_len[b], 0), p.T) : p.T;
    float* lse_row = p.lse2 + ((int64_t)b * p.Hq + h) * p.T;
    if (qb * kRows >= len) {
        for (int r = tid; r < kRows; r += kThreads)
            if (qb * kRows + r < p.T) lse_row[qb * kRows + r] = INFINITY;
        return;
    }
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t q_tile = base;
    if (tid == 0) {
        mbar_init(smem_u32(&bar_q), 1);
        mbar_init(smem_u32(&bar_k[0]), 1);
        mbar_init(smem_u32(&bar_k[1]), 1);
        sm_abort = 0;
        fence_mbar_init();
    }
    __syncthreads();
    auto issue_k = [&](int kb) {
        const uint32_t bar = smem_u32(&bar_k[kb & 1]);
        mbar_arrive_expect_tx(bar, kTileBytes);
#pragma unroll
        for (int bx = 0; bx < D / 64; ++bx)
            tma_load_3d(base + (1 + (kb & 1)) * kTileBytes + bx * (kRows * 128), &k_map, bx * 64, kb * kRows,
                        b * p.Hkv + kvh, bar);
    };
    if (tid == 0) {
        mbar_arrive_expect_tx(smem_u32(&bar_q), kTileBytes);
#pragma unroll
        for (int bx = 0; bx < D / 64; ++bx)
            tma_load_3d(q_tile + bx * (kRows * 128), &q_map, bx * 64, qb * kRows, b * p.Hq + h, smem_u32(&bar_q));
        issue_k(0);
    }
    const int r0 = warp * 16;
    const int lm = lane >> 3, li8 = lane & 7;
    const int qrow = lane >> 2, qcol = (lane & 3) * 2;
    bool alive = mbar_wait(smem_u32(&bar_q), 0);
    uint32_t qa[kKSteps][4];
    if (alive) {
#pragma unroll
        for (int ks = 0; ks < kKSteps; ++ks)
            ldmatrix_x4(q_tile + tile_offset(r0 + (lm & 1) * 8 + li8, 2 * ks + (lm >> 1)), qa[ks]);
    }
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.0f, 0.0f};
    for (int kb = 0; kb <= qb; ++kb) {
        __syncthreads();
        if (sm_abort) break;
        if (tid == 0 && kb + 1 <= qb) issue_k(kb + 1);
        if (!alive || !mbar_wait(smem_u32(&bar_k[kb & 1]), (kb >> 1) & 1)) {
            alive = false;
            sm_abort = 1;
            continue;
        }
        const uint32_t k_tile = base + (1 + (kb & 1)) * kTileBytes;
        float sacc[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) { sacc[nt][0] = sacc[nt][1] = sacc[nt][2] = sacc[nt][3] = 0.0f; }
#pragma unroll
        for (int ks = 0; ks < kKSteps; ++ks)
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                uint32_t kf[4];
                ldmatrix_x4(k_tile + tile_offset(16 * kk + (lm >> 1) * 8 + li8, 2 * ks + (lm & 1)), kf);
                mma_bf16(sacc[2 * kk], qa[ks], kf[0], kf[1]);
                mma_bf16(sacc[2 * kk + 1], qa[ks], kf[2], kf[3]);
            }
        const bool diagonal = kb == qb;
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float v = sacc[nt][e] * p.scale_log2;
                if (diagonal && 8 * nt + qcol + (e & 1) > r0 + qrow + (e >> 1) * 8) v = -INFINITY;   // causal mask
                sacc[nt][e] = v;
                mx[e >> 1] = fmaxf(mx[e >> 1], v);
            }
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
            const float m_new = fmaxf(m_run[r], mx[r]);      // finite: key 0 is never masked
            l_run[r] *= exp2f(m_run[r] - m_new);
            m_run[r] = m_new;
        }
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) l_run[e >> 1] += exp2f(sacc[nt][e] - m_run[e >> 1]);
    }
    __syncthreads();
    if (sm_abort) {
        if (tid == 0) atomicOr(p.error, 1u);
        return;
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        float l = l_run[r];
        l += __shfl_xor_sync(0xffffffffu, l, 1);
        l += __shfl_xor_sync(0xffffffffu, l, 2);
        const int t = qb * kRows + r0 + qrow + r * 8;
        if ((lane & 3) == 0 && t < p.T) lse_row[t] = t < len ? m_run[r] + log2f(l) : INFINITY;
    }
}

// ---------------------------------------------------------------- pass 2: column sums per key block
template <int D>
__global__ void __launch_bounds__(kThreads) prefill_colsum_kernel(const PrefillParams p,
                                                                  const __grid_constant__ CUtensorMap q_map,
                                                                  const __grid_constant__ CUtensorMap k_map) {
    constexpr int kKSteps = D / 16;
    constexpr int kTileBytes = kRows * D * 2;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_k;
    __shared__ __align__(8) uint64_t bar_q[2];
    __shared__ float sm_lse[2][kRows];
    __shared__ int sm_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int kb = blockIdx.x;                              // early key blocks have the most query tiles: first
    const int kvh = blockIdx.y, b = blockIdx.z;
    const int g = p.Hq / p.Hkv;
    const int len = p.prompt_len ? min(max(p.prompt_len[b], 0), p.T) : p.T;
    if (kb * kRows >= len) {                                // keys past the prompt receive nothing
        for (int r = tid; r < kRows; r += kThreads)
            if (kb * kRows + r < p.T) p.score[((int64_t)b * p.Hkv + kvh) * p.T + kb * kRows + r] = 0.0f;
        return;
    }
    const int nq = (len + kRows - 1) / kRows - kb;          // query tiles of the prompt at or below this key block
    const int n_it = g * nq;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t k_tile = base;
    if (tid == 0) {
        mbar_init(smem_u32(&bar_k), 1);
        mbar_init(smem_u32(&bar_q[0]), 1);
        mbar_init(smem_u32(&bar_q[1]), 1);
        sm_abort = 0;
        fence_mbar_init();
    }
    __syncthreads();
    auto issue_q = [&](int it) {
        const int a = it / nq, qb = kb + it % nq;
        const uint32_t bar = smem_u32(&bar_q[it & 1]);
        mbar_arrive_expect_tx(bar, kTileBytes);
#pragma unroll
        for (int bx = 0; bx < D / 64; ++bx)
            tma_load_3d(base + (1 + (it & 1)) * kTileBytes + bx * (kRows * 128), &q_map, bx * 64, qb * kRows,
                        b * p.Hq + kvh * g + a, bar);
    };
    auto fetch_lse = [&](int it) -> float {                  // threads 0..63: one query row of tile `it`
        const int a = it / nq, qb = kb + it % nq;
        const int t = qb * kRows + tid;
        return t < p.T ? p.lse2[((int64_t)b * p.Hq + kvh * g + a) * p.T + t] : INFINITY;
    };
    if (tid == 0) {
        mbar_arrive_expect_tx(smem_u32(&bar_k), kTileBytes);
#pragma unroll
        for (int bx = 0; bx < D / 64; ++bx)
            tma_load_3d(k_tile + bx * (kRows * 128), &k_map, bx * 64, kb * kRows, b * p.Hkv + kvh, smem_u32(&bar_k));
        issue_q(0);
    }
    if (tid < kRows) sm_lse[0][tid] = fetch_lse(0);

    const int r0 = warp * 16;                               // this warp's keys inside the block
    const int lm = lane >> 3, li8 = lane & 7;
    const int qrow = lane >> 2, qcol = (lane & 3) * 2;
    bool alive = mbar_wait(smem_u32(&bar_k), 0);
    uint32_t ka[kKSteps][4];                                // the warp's 16 keys as the A operand, kept all along
    if (alive) {
#pragma unroll
        for (int ks = 0; ks < kKSteps; ++ks)
            ldmatrix_x4(k_tile + tile_offset(r0 + (lm & 1) * 8 + li8, 2 * ks + (lm >> 1)), ka[ks]);
    }
    float colsum[2] = {0.0f, 0.0f};                          // keys r0 + qrow and r0 + qrow + 8
    for (int it = 0; it < n_it; ++it) {
        __syncthreads();                                    // tile it - 1 is consumed; sm_lse[it & 1] is in place
        if (sm_abort) break;
        if (it + 1 < n_it) {
            if (tid == 0) issue_q(it + 1);
            if (tid < kRows) sm_lse[(it + 1) & 1][tid] = fetch_lse(it + 1);
        }
        if (!alive || !mbar_wait(smem_u32(&bar_q[it & 1]), (it >> 1) & 1)) {
            alive = false;
            sm_abort = 1;
            continue;
        }
        const uint32_t q_tile = base + (1 + (it & 1)) * kTileBytes;
        const bool diagonal = (it % nq) == 0;
        // S^T = K Q^T: rows are this warp's keys, columns the tile's 64 queries
        float sacc[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) { sacc[nt][0] = sacc[nt][1] = sacc[nt][2] = sacc[nt][3] = 0.0f; }
#pragma unroll
        for (int ks = 0; ks < kKSteps; ++ks)
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                uint32_t qf[4];
                ldmatrix_x4(q_tile + tile_offset(16 * kk + (lm >> 1) * 8 + li8, 2 * ks + (lm & 1)), qf);
                mma_bf16(sacc[2 * kk], ka[ks], qf[0], qf[1]);
                mma_bf16(sacc[2 * kk + 1], ka[ks], qf[2], qf[3]);
            }
        const float* lse = sm_lse[it & 1];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int query = 8 * nt + qcol + (e & 1);          // inside the tile
                const int key = r0 + qrow + (e >> 1) * 8;
                float pe = exp2f(sacc[nt][e] * p.scale_log2 - lse[query]);   // lse = +inf past the prompt: 0
                if (diagonal && key > query) pe = 0.0f;             // causal mask
                colsum[e >> 1] += pe;
            }
    }
    __syncthreads();
    if (sm_abort) {
        if (tid == 0) atomicOr(p.error, 1u);
        return;
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        float c = colsum[r];
        c += __shfl_xor_sync(0xffffffffu, c, 1);
        c += __shfl_xor_sync(0xffffffffu, c, 2);
        const int t = kb * kRows + r0 + qrow + r * 8;
        if ((lane & 3) == 0 && t < p.T) p.score[((int64_t)b * p.Hkv + kvh) * p.T + t] = c;
    }
}

template <int D>
cudaError_t launch_prefill(const PrefillParams& p, const CUtensorMap& qm, const CUtensorMap& km, cudaStream_t s) {
    constexpr int kSmem = 3 * kRows * D * 2 + 1024;      // one resident tile + a two-stage ring
    cudaError_t e = cudaFuncSetAttribute(prefill_lse_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(prefill_colsum_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    prefill_lse_kernel<D><<<dim3(p.n_blk, p.Hq, p.B), kThreads, kSmem, s>>>(p, qm, km);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    prefill_colsum_kernel<D><<<dim3(p.n_blk, p.Hkv, p.B), kThreads, kSmem, s>>>(p, qm, km);
    return cudaGetLastError();
}

}  // namespace

extern "C" __attribute__((visibility("default"))) size_t baklava_prefill_workspace_size(const baklava_shape* shape,
                                                                                    int32_t B, int32_t T) {
    if (!shape || B <= 0 || T <= 0) return 0;
    return 256 + sizeof(float) * (size_t)B * shape->Hq * (size_t)T;
}

extern "C" __attribute__((visibility("default"))) int baklava_prefill_scores(
        const baklava_shape* shape, const void* q, const void* k, const int32_t* prompt_len, int32_t B, int32_t T,
        float* score, void* ws, size_t ws_bytes, void* stream) {
    int rc = baklava_check_shape(shape);
    if (rc) return rc;
    if (!q || !k || !score || !ws || B <= 0 || T <= 0) return BAKLAVA_ERR_INVALID_ARG;
    const void* ptrs[] = {q, k, ws};
    for (const void* ptr : ptrs)
        if (!baklava_aligned16(ptr)) return BAKLAVA_ERR_INVALID_ARG;
    if (B > 65535 || shape->Hq > 65535) return BAKLAVA_ERR_UNSUPPORTED;
    if (ws_bytes < baklava_prefill_workspace_size(shape, B, T)) return BAKLAVA_ERR_WORKSPACE;

    PrefillParams p;
    p.prompt_len = prompt_len;
    p.error = static_cast<uint32_t*>(ws);
    p.lse2 = reinterpret_cast<float*>(static_cast<char*>(ws) + 256);
    p.score = score;
    p.B = B; p.T = T; p.Hq = shape->Hq; p.Hkv = shape->Hkv;
    p.n_blk = (T + kRows - 1) / kRows;
    p.scale_log2 = kLog2e / sqrtf((float)shape->D);

    CUtensorMap qm, km;
    if (!make_head_map(&qm, q, (int64_t)B * shape->Hq, T, shape->D) ||
        !make_head_map(&km, k, (int64_t)B * shape->Hkv, T, shape->D))
        return BAKLAVA_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(ws, 0, 256, s) != cudaSuccess) return BAKLAVA_ERR_CUDA;
    cudaError_t err = shape->D == 128 ? launch_prefill<128>(p, qm, km, s) : launch_prefill<64>(p, qm, km, s);
    return err == cudaSuccess ? BAKLAVA_OK : BAKLAVA_ERR_CUDA;
}
