// Head-similarity profiling (Algorithm 1, step 1): for every prompt and query head of one layer,
// causal softmax attention O = softmax(Q K^T / sqrt(D)) V and the token-wise cosine between the
// head's input V_t and its output O_t, averaged over the prompt's tokens.
//
// One pass on the 5th-generation tensor cores.  The cosine does not change when a row of O is scaled, so
// the softmax is left unnormalised and needs only a stabiliser per row, for which the row's largest logit
// among its first eight keys serves: p = exp2(s - reference), no running maximum, no sum, no rescaling of O, no
// division.  (Rows whose later logits leave the fp32 range that way are detected in the epilogue and redone
// by a second instantiation that takes the true row maxima from a row pass; see profile_pv_block.)
// A CTA owns 128 query rows: the Q tile stays in shared memory, K and V tiles of 128 keys stream through
// three-stage TMA rings; one thread issues S = Q K^T into tensor memory (double-buffered), sixteen softmax
// warps read S back, form the probabilities in bf16 and write them back to tensor memory, from where the next
// MMA takes them as its A operand, and the same thread issues O += P V with V as an MN-major B operand; O
// accumulates in tensor memory over all key tiles and is never written.  The last key tile is the
// diagonal one, whose V rows are exactly the rows the cosine needs, so the final epilogue reads them from
// shared memory.
// Per-CTA cosine sums go to the workspace and a small kernel adds them in a fixed order.
#include <cmath>
#include <cstdint>

#include "baklava.h"
#include "common.h"
#include "ptx.cuh"

namespace {

using namespace ptx;

constexpr int kTileRows = 128;        // query rows per CTA = keys per streamed tile
constexpr int kSoftmaxWarps = 16;     // four threads per query row, 32 keys of a tile each
constexpr int kThreads = (2 + kSoftmaxWarps) * 32;   // warp 0: TMA producer, warp 1: MMA issuer + TMEM owner, then softmax
constexpr int kGroupRing = 4;         // mbarriers that track the MMA groups in flight
constexpr int kKvStages = 3;          // K and V tiles in flight: the streamed operands come from L2 at a bounded rate
constexpr uint32_t kTmemColumns = 512;    // S: 2 x 128 columns, O: D columns (at most 128), P: 2 x 64 columns
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kCosEps = 1e-12f;

struct ProfileParams {
    const int32_t* prompt_len;   // [P] or null
    const float* lse2;           // [P, Hq, T] from the row pass: every row's largest logit, log2 domain (exact mode)
    int32_t* redo_list;          // flat indices ((pr * Hq + h) * n_blk + qb) of the row blocks the one-pass kernel
    int32_t* redo_count;         //   could not finish in range, and how many there are
    float* head_cos;             // [P, Hq]
    float* token_cos;            // [P, Hq, T] or null
    float* block_sum;            // [P, Hq, n_blk]
    uint32_t* error;
    int32_t P, T, Hq, Hkv, n_blk;
    float scale_log2;
};

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// kExact = false: one pass.  The softmax needs a stabiliser per row, not the row's true maximum: the
// largest logit among the row's first eight keys serves (every row sees key 0, so it exists),
// probabilities of later keys may then exceed 1, which bf16 and the fp32 accumulator hold up to 2^127.
// A row whose later logits are so far above that reference that O or its norm leaves the fp32 range
// shows up as a non-finite cosine term in the epilogue; its row block is flagged in `redo` and done again
// by the kExact = true instantiation, which takes every row's true maximum from a row pass and runs only
// on flagged blocks.  Results that stayed finite are exact up to rounding, because scaling a row of O by
// a power of two changes nothing in its cosine.
template <int D, bool kExact>
__device__ __forceinline__ void profile_pv_block(const ProfileParams& p, const CUtensorMap& q_map, const CUtensorMap& k_map,
                                                 const CUtensorMap& v_map, const int qb, const int h, const int pr) {
    constexpr int kKSteps = D / 16;                          // MMA steps over the head dimension (S = Q K^T)
    constexpr int kPvSteps = kTileRows / 16;                 // MMA steps over the keys (O += P V)
    constexpr int kBoxBytes = kTileRows * 128;               // one TMA box: 128 rows x 64 elements
    constexpr int kTileBytes = kTileRows * D * 2;            // a Q, K or V tile
    constexpr int kStageBytes = 2 * kTileBytes;              // K then V
    constexpr uint32_t kOColumn = 2 * kTileRows;             // O sits after the two S buffers in tensor memory
    constexpr uint32_t kPColumn = 3 * kTileRows;             // then two probability tiles: 128 keys in bf16 = 64 columns
    constexpr uint32_t kPColumns = kTileRows / 2;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_q, bar_k01[2], bar_in[kGroupRing], bar_group[kGroupRing];
    __shared__ uint32_t tmem_slot;
    __shared__ float sm_warp_sum[kSoftmaxWarps];
    __shared__ int sm_abort;
    __shared__ int sm_redo;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int kvh = h / (p.Hq / p.Hkv);
    const int len = p.prompt_len ? min(max(p.prompt_len[pr], 0), p.T) : p.T;
    float* out_sum = p.block_sum + ((int64_t)pr * p.Hq + h) * p.n_blk + qb;
    if (qb * kTileRows >= len) {
        if (tid == 0) *out_sum = 0.0f;
        return;
    }
    const int n_it = qb + 1;                                 // key tiles 0 .. qb
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t q_tile = base;
    const uint32_t stage0 = base + kTileBytes;

    if (tid == 0) {
        mbar_init(smem_u32(&bar_q), 1);
        for (int s = 0; s < 2; ++s) mbar_init(smem_u32(&bar_k01[s]), 1);
        for (int s = 0; s < kGroupRing; ++s) {
            mbar_init(smem_u32(&bar_in[s]), kSoftmaxWarps + 2);   // P(it) written, V(it) landed, K(it + 2) landed
            mbar_init(smem_u32(&bar_group[s]), 1);
        }
        sm_abort = 0;
        sm_redo = 0;
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
    // completion of MMA group g (see the MMA issuer); a slot of the ring is reused four groups later,
    // and no waiter can be that far behind
    auto group_wait = [&](int g) { return mbar_wait(smem_u32(&bar_group[g % kGroupRing]), (g / kGroupRing) & 1); };

    if (warp == 0) {
        // ---------------- TMA producer
        if (lane == 0) {
            mbar_arrive_expect_tx(smem_u32(&bar_q), kTileBytes);
#pragma unroll
            for (int bx = 0; bx < D / 64; ++bx)
                tma_load_3d(q_tile + bx * kBoxBytes, &q_map, bx * 64, qb * kTileRows, pr * p.Hq + h, smem_u32(&bar_q));
            // The single MMA thread pays well over a hundred cycles for every mbarrier it looks at, so
            // everything group it + 2 = { P(it) V(it), S(it + 2) } needs arrives on ONE barrier, bar_in[it % 4]:
            // the sixteen softmax warps (P(it) written) and the two loads V(it) and K(it + 2).
            // K(j) reuses the stage of K(j - 3), consumed by S(j - 3) = MMA group j - 3; V(j) the stage of
            // V(j - 3), consumed by P V of tile j - 3 = MMA group j - 1: both loads of bar_in[j % 4] wait for
            // group j - 1.
            auto load = [&](const CUtensorMap* map, uint32_t bar, uint32_t dst, int it) {
                mbar_arrive_expect_tx(bar, kTileBytes);
#pragma unroll
                for (int bx = 0; bx < D / 64; ++bx)
                    tma_load_3d(dst + (it % kKvStages) * kStageBytes + bx * kBoxBytes, map, bx * 64, it * kTileRows,
                                pr * p.Hkv + kvh, bar);
            };
            for (int j = 0; j < 2 && j < n_it; ++j) load(&k_map, smem_u32(&bar_k01[j]), stage0, j);
            bool ok = true;
            for (int j = 0; j < n_it && ok; ++j) {
                if (j >= 1) ok = group_wait(j - 1);           // (K(3) and K(4) already reuse a stage)
                if (!ok) break;
                const uint32_t bar = smem_u32(&bar_in[j % kGroupRing]);
                load(&v_map, bar, stage0 + kTileBytes, j);
                if (j + 2 < n_it) load(&k_map, bar, stage0, j + 2);
                else tc::mbar_arrive(bar);
            }
            if (!ok) sm_abort = 1;
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_s = tc::idesc_bf16_f32(kTileRows, kTileRows);      // S[128 q x 128 keys]
            constexpr uint32_t idesc_o = tc::idesc_bf16_f32_b_mn(kTileRows, D);         // O[128 q x D]
            // A tcgen05.commit occupies the tensor pipe for about as long as a quarter of a 128 x 128 x 128
            // MMA, so the work is issued in groups with ONE commit each: group 0 = S(0), group 1 = S(1),
            // group it + 2 = { O += P(it) V(it), S(it + 2) }.  Completion of group g therefore tells the
            // softmax warps that S(g) is ready and that the probability buffer of tile g - 2 is free, and
            // the producer that K(g) and V(g - 2) are consumed.
            bool ok = mbar_wait(smem_u32(&bar_q), 0);
            auto issue_s = [&](int it) {                     // S_it = Q K_it^T into S buffer it & 1
                const int s = it & 1, kv = it % kKvStages;
                const uint32_t k_tile = stage0 + kv * kStageBytes;
                // a descriptor's address field is (address >> 4), so stepping through a tile is an addition: the
                // issuing thread's instruction count per MMA is what bounds this kernel
                const uint64_t dq = tc::desc_k_major_sw128(q_tile), dk = tc::desc_k_major_sw128(k_tile);
#pragma unroll
                for (int ks = 0; ks < kKSteps; ++ks) {
                    const uint32_t off = ((ks >> 2) * kBoxBytes + (ks & 3) * 32) >> 4;
                    tc::umma_bf16(tmem_base + s * kTileRows, dq + off, dk + off, idesc_s, ks > 0);
                }
            };
            for (int g = 0; g < 2 && g < n_it && ok; ++g) {
                ok = mbar_wait(smem_u32(&bar_k01[g]), 0);
                if (!ok) break;
                tc::fence_after_sync();
                issue_s(g);
                tc::umma_commit(smem_u32(&bar_group[g % kGroupRing]));
            }
            for (int it = 0; it < n_it && ok; ++it) {
                const int s = it & 1, kv = it % kKvStages;
                // P(it) is written (so S(it) has been read), V(it) and K(it + 2) have landed
                ok = mbar_wait(smem_u32(&bar_in[it % kGroupRing]), (it / kGroupRing) & 1);
                if (!ok) break;
                tc::fence_after_sync();
                const uint32_t v_tile = stage0 + kv * kStageBytes + kTileBytes;
                const uint64_t dv = tc::desc_mn_major_sw128(v_tile, kBoxBytes);
#pragma unroll
                for (int ks = 0; ks < kPvSteps; ++ks) {      // 16 keys per step = 8 columns of the probability tile
                    tc::umma_bf16_ts(tmem_base + kOColumn, tmem_base + kPColumn + s * kPColumns + ks * 8,
                                     dv + (ks * 2048 >> 4), idesc_o, (it > 0) || (ks > 0));
                }
                if (it + 2 < n_it) issue_s(it + 2);          // into the S buffer tile `it` has just left
                tc::umma_commit(smem_u32(&bar_group[(it + 2) % kGroupRing]));
            }
            if (!ok) sm_abort = 1;
        }
    } else {
        // ---------------- softmax warps: a warp reads its quarter of the TMEM lanes (thread = query row);
        // warps 2-5 take keys 0..31 of every tile, warps 6-9 keys 32..63, and so on
        const int row = 32 * (warp & 3) + lane;
        const int part = (warp - 2) >> 2;                     // 0 .. 3
        const int col_base = part * 32;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16);
        const int t = qb * kTileRows + row;
        // the softmax's reference logit of this row, log2 domain (exact mode: the row's maximum; +inf past the prompt)
        float lse = 0.0f;
        if (kExact) lse = t < p.T ? p.lse2[((int64_t)pr * p.Hq + h) * p.T + t] : INFINITY;
        bool ok = true;
        for (int it = 0; it < n_it; ++it) {
            const int s = it & 1;
            if (!group_wait(it)) { ok = false; break; }        // S(it) is ready and P V of tile it - 2 has read its P
            tc::fence_after_sync();
            uint32_t v[32];
            if (!kExact && it == 0) {
                // reference = the row's largest logit among the first eight keys (those of them it may see):
                // every thread of the row reads the same eight columns, so the four agree without talking
                uint32_t first[8];
                tc::tmem_ld_32x32_x8(lane_addr, first);
                tc::tmem_ld_wait();
                float mx = __uint_as_float(first[0]);
#pragma unroll
                for (int c = 1; c < 8; ++c)
                    if (qb > 0 || c <= row) mx = fmaxf(mx, __uint_as_float(first[c]));
                lse = mx * p.scale_log2;
            }
            tc::tmem_ld_32x32(lane_addr + s * kTileRows + col_base, v);
            tc::tmem_ld_wait();
            if (it == qb) {                                   // diagonal tile: keys above the query do not exist
#pragma unroll
                for (int c = 0; c < 32; ++c)
                    if (col_base + c > row) v[c] = 0xff800000u;
            }
            // probabilities of this thread's 32 keys -> bf16, two per 32-bit column of the A operand
            uint32_t w[16];
#pragma unroll
            for (int c = 0; c < 16; ++c)
                w[c] = pack_bf16(fast_exp2(fmaf(__uint_as_float(v[2 * c]), p.scale_log2, -lse)),
                                 fast_exp2(fmaf(__uint_as_float(v[2 * c + 1]), p.scale_log2, -lse)));
            tc::tmem_st_32x32_x16(lane_addr + kPColumn + s * kPColumns + part * 16, w);
            tc::tmem_st_wait();
            tc::fence_before_sync();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(smem_u32(&bar_in[it % kGroupRing]));
        }
        // ---- O is complete: cosine between V_t and O_t; the V rows of this CTA's tokens are the diagonal tile.
        // Four threads per row take 32 columns of the head dimension each (two of them when D = 64).
        if (ok) ok = group_wait(n_it + 1);                    // the last group: O is complete
        float dot = 0.0f, vv = 0.0f, oo = 0.0f;
        if (ok && part * 32 < D) {
            tc::fence_after_sync();
            const uint8_t* v_row = base_ptr + (stage0 - base) + (qb % kKvStages) * kStageBytes + kTileBytes + row * 128;
            uint32_t o[32];
            tc::tmem_ld_32x32(lane_addr + kOColumn + part * 32, o);
            tc::tmem_ld_wait();
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {                  // 16-byte pieces of 8 elements
                const int piece = part * 4 + cc;              // within the row: 0 .. D/8 - 1
                const uint4 raw = *reinterpret_cast<const uint4*>(v_row + (piece >> 3) * kBoxBytes +
                                                                  (((piece & 7) ^ (row & 7)) << 4));
                const uint32_t wv[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                for (int k2 = 0; k2 < 4; ++k2) {
                    const float2 vx = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&wv[k2]));
                    const float o0 = __uint_as_float(o[cc * 8 + k2 * 2]), o1 = __uint_as_float(o[cc * 8 + k2 * 2 + 1]);
                    dot = fmaf(vx.x, o0, fmaf(vx.y, o1, dot));
                    vv = fmaf(vx.x, vx.x, fmaf(vx.y, vx.y, vv));
                    oo = fmaf(o0, o0, fmaf(o1, o1, oo));
                }
            }
        }
        // join the four parts of every row through shared memory (the stage without the diagonal tile is idle)
        float* sm_part = reinterpret_cast<float*>(base_ptr + (stage0 - base) + ((qb + 1) % kKvStages) * kStageBytes);   // [3][4][128]
        sm_part[(0 * 4 + part) * kTileRows + row] = dot;
        sm_part[(1 * 4 + part) * kTileRows + row] = vv;
        sm_part[(2 * 4 + part) * kTileRows + row] = oo;
        asm volatile("bar.sync 1, 512;" ::: "memory");
        float c = 0.0f;
        if (part == 0 && ok && t < len) {
            float d4 = 0.0f, v4 = 0.0f, o4 = 0.0f;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                d4 += sm_part[(0 * 4 + k) * kTileRows + row];
                v4 += sm_part[(1 * 4 + k) * kTileRows + row];
                o4 += sm_part[(2 * 4 + k) * kTileRows + row];
            }
            c = d4 / fmaxf(sqrtf(v4) * sqrtf(o4), kCosEps);
            if (!kExact && !(fabsf(d4) <= 3.0e38f && o4 <= 3.0e38f)) {   // left the fp32 range (or NaN): redo this block
                sm_redo = 1;
                c = 0.0f;
            }
            if (p.token_cos) p.token_cos[((int64_t)pr * p.Hq + h) * p.T + t] = c;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) c += __shfl_xor_sync(0xffffffffu, c, off);
        if (lane == 0) sm_warp_sum[warp - 2] = c;
        if (!ok) sm_abort = 1;
    }
    tc::fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc::fence_after_sync();
        tc::tmem_dealloc(tmem_base, kTmemColumns);
    }
    if (tid == 0) {
        if (sm_abort) atomicOr(p.error, 1u);
        const bool again = !kExact && sm_redo != 0;
        *out_sum = (sm_abort || again) ? 0.0f : (sm_warp_sum[0] + sm_warp_sum[1]) + (sm_warp_sum[2] + sm_warp_sum[3]);
        if (again) p.redo_list[atomicAdd(p.redo_count, 1)] = (pr * p.Hq + h) * p.n_blk + qb;
        // the barriers may be set up again by the next row block of this CTA (exact mode)
        mbar_inval(smem_u32(&bar_q));
        for (int s = 0; s < 2; ++s) mbar_inval(smem_u32(&bar_k01[s]));
        for (int s = 0; s < kGroupRing; ++s) {
            mbar_inval(smem_u32(&bar_in[s]));
            mbar_inval(smem_u32(&bar_group[s]));
        }
    }
    __syncthreads();
}

// One pass over every row block of the layer: grid (row blocks, query heads, prompts), long blocks first.
template <int D>
__global__ void __launch_bounds__(kThreads, 1) profile_pv_kernel(const ProfileParams p,
                                                                 const __grid_constant__ CUtensorMap q_map,
                                                                 const __grid_constant__ CUtensorMap k_map,
                                                                 const __grid_constant__ CUtensorMap v_map) {
    profile_pv_block<D, false>(p, q_map, k_map, v_map, p.n_blk - 1 - (int)blockIdx.x, blockIdx.y, blockIdx.z);
}

// The exact form over the row blocks the one-pass kernel listed: a small fixed grid whose CTAs take the
// entries in turn, so that the usual empty list costs nothing.
template <int D>
__global__ void __launch_bounds__(kThreads, 1) profile_pv_redo_kernel(const ProfileParams p,
                                                                      const __grid_constant__ CUtensorMap q_map,
                                                                      const __grid_constant__ CUtensorMap k_map,
                                                                      const __grid_constant__ CUtensorMap v_map) {
    const int n = *p.redo_count;
    for (int w = blockIdx.x; w < n; w += gridDim.x) {
        const int flat = p.redo_list[w];
        profile_pv_block<D, true>(p, q_map, k_map, v_map, flat % p.n_blk, (flat / p.n_blk) % p.Hq,
                                  flat / (p.n_blk * p.Hq));
    }
}

__global__ void profile_mean_kernel(const ProfileParams p) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;   // (prompt, head)
    if (i >= p.P * p.Hq) return;
    const int pr = i / p.Hq;
    const int len = p.prompt_len ? min(max(p.prompt_len[pr], 0), p.T) : p.T;
    float acc = 0.0f;
    for (int b = 0; b < p.n_blk; ++b) acc += p.block_sum[(int64_t)i * p.n_blk + b];
    p.head_cos[i] = len > 0 ? acc / (float)len : 0.0f;
}

constexpr int kRedoGrid = 148;        // CTAs that share the list of row blocks to redo

template <int D, bool kExact>
cudaError_t launch_profile(const ProfileParams& p, const CUtensorMap& qm, const CUtensorMap& km, const CUtensorMap& vm,
                           cudaStream_t s) {
    // Q tile and the (K, V) stages
    constexpr int kSmem = kTileRows * D * 2 * (1 + 2 * kKvStages) + 1024;
    if (kExact) {
        cudaError_t e = cudaFuncSetAttribute(profile_pv_redo_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
        if (e != cudaSuccess) return e;
        profile_pv_redo_kernel<D><<<kRedoGrid, kThreads, kSmem, s>>>(p, qm, km, vm);
        return cudaGetLastError();
    }
    cudaError_t e = cudaFuncSetAttribute(profile_pv_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    const dim3 grid(p.n_blk, p.Hq, p.P);
    profile_pv_kernel<D><<<grid, kThreads, kSmem, s>>>(p, qm, km, vm);
    return cudaGetLastError();
}

}  // namespace

extern "C" __attribute__((visibility("default"))) size_t baklava_profile_workspace_size(const baklava_shape* shape,
                                                                                    int32_t P, int32_t T) {
    if (!shape || P <= 0 || T <= 0) return 0;
    const size_t n_blk = ((size_t)T + kTileRows - 1) / kTileRows;
    return 256 + sizeof(float) * (size_t)P * shape->Hq * ((size_t)T + 2 * n_blk);
}

extern "C" __attribute__((visibility("default"))) int baklava_profile_heads(
        const baklava_shape* shape, const void* q, const void* k, const void* v,
        const int32_t* prompt_len, int32_t P, int32_t T,
        float* head_cos, float* token_cos, void* ws, size_t ws_bytes, void* stream) {
    int rc = baklava_check_shape(shape);
    if (rc) return rc;
    if (!q || !k || !v || !head_cos || !ws || P <= 0 || T <= 0) return BAKLAVA_ERR_INVALID_ARG;
    const void* ptrs[] = {q, k, v, ws};
    for (const void* ptr : ptrs)
        if (!baklava_aligned16(ptr)) return BAKLAVA_ERR_INVALID_ARG;
    if (P > 65535 || shape->Hq > 65535) return BAKLAVA_ERR_UNSUPPORTED;
    if (ws_bytes < baklava_profile_workspace_size(shape, P, T)) return BAKLAVA_ERR_WORKSPACE;

    ProfileParams p;
    p.prompt_len = prompt_len;
    p.head_cos = head_cos;
    p.token_cos = token_cos;
    p.error = static_cast<uint32_t*>(ws);
    float* lse2 = reinterpret_cast<float*>(static_cast<char*>(ws) + 256);
    p.lse2 = lse2;
    p.block_sum = lse2 + (size_t)P * shape->Hq * (size_t)T;
    p.redo_list = reinterpret_cast<int32_t*>(p.block_sum + (size_t)P * shape->Hq * ((size_t)(T + kTileRows - 1) / kTileRows));
    p.redo_count = reinterpret_cast<int32_t*>(ws) + 1;       // inside the header that is cleared below
    p.P = P; p.T = T; p.Hq = shape->Hq; p.Hkv = shape->Hkv;
    p.n_blk = (T + kTileRows - 1) / kTileRows;
    p.scale_log2 = kLog2e / sqrtf((float)shape->D);

    CUtensorMap qm, km, vm;
    if (!make_head_map(&qm, q, (int64_t)P * shape->Hq, T, shape->D, kTileRows) ||
        !make_head_map(&km, k, (int64_t)P * shape->Hkv, T, shape->D, kTileRows) ||
        !make_head_map(&vm, v, (int64_t)P * shape->Hkv, T, shape->D, kTileRows))
        return BAKLAVA_ERR_CUDA;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(ws, 0, 256, s) != cudaSuccess) return BAKLAVA_ERR_CUDA;
    // one pass for everything, then the exact two-pass form for the row blocks it listed (normally none:
    // both follow-up launches then find an empty list and return at once)
    cudaError_t err = shape->D == 128 ? launch_profile<128, false>(p, qm, km, vm, s) : launch_profile<64, false>(p, qm, km, vm, s);
    if (err != cudaSuccess) return BAKLAVA_ERR_CUDA;
    rc = baklava_launch_row_max(shape, q, k, prompt_len, P, T, lse2, p.redo_list, p.redo_count, 2 * kRedoGrid, p.error, s);
    if (rc) return rc;
    err = shape->D == 128 ? launch_profile<128, true>(p, qm, km, vm, s) : launch_profile<64, true>(p, qm, km, vm, s);
    if (err != cudaSuccess) return BAKLAVA_ERR_CUDA;
    const int n = P * shape->Hq;
    profile_mean_kernel<<<(n + 127) / 128, 128, 0, s>>>(p);
    return cudaGetLastError() == cudaSuccess ? BAKLAVA_OK : BAKLAVA_ERR_CUDA;
}
