// Head-similarity profiling (Algorithm 1, step 1): for every prompt and query head of one layer,
// causal softmax attention O = softmax(Q K^T / sqrt(D)) V and the token-wise cosine between the
// head's input V_t and its output O_t, averaged over the prompt's tokens.
//
// One pass on the 5th-generation tensor cores.  The cosine does not change when a row of O is scaled, so
// the softmax is left unnormalised and needs only a stabiliser per row, for which the row's largest logit
// among its first eight keys serves: p = exp2(s - reference), no running maximum, no sum, no rescaling of O, no
// division.  (Rows whose later logits leave the fp32 range that way are detected in the epilogue and redone
// by a second instantiation that takes the true row maxima from a row pass; see profile_pv_block.)
// A CTA owns 128 query rows and half an SM: the Q tile, one K tile and one V tile of 128 keys in shared memory
// (96 KB), 256 columns of tensor memory (S, with the probabilities written over it, and O), ten warps.  Per key
// tile one thread issues O += P V for the tile before and S = Q K^T for this one (one commit), eight softmax warps
// read S back, form the probabilities in bf16 and write them over the logits they came from, from where the next
// MMA takes them as its A operand; V is an MN-major B operand; O accumulates in tensor memory over all key
// tiles and is never written.  Inside one CTA these steps follow one another, each waiting for the one before it
// and for the next tiles to land; the SM's second CTA, at another point of its own chain (or in its start-up or
// its epilogue), uses the tensor pipe and the special-function unit meanwhile.  The last key tile is the diagonal
// one, whose V rows are exactly the rows the cosine needs, so the final epilogue reads them from shared memory.
// Per-CTA cosine sums go to the workspace and a small kernel adds them in a fixed order.
#include <cmath>
#include <cstdint>

#include "baklava.h"
#include "common.h"
#include "ptx.cuh"

namespace {

using namespace ptx;

constexpr int kTileRows = 128;        // query rows per CTA = keys per streamed tile
constexpr int kSoftmaxWarps = 8;      // two threads per query row, 64 keys of a tile each
constexpr int kThreads = (2 + kSoftmaxWarps) * 32;   // warp 0: TMA producer, warp 1: MMA issuer + TMEM owner, then softmax
constexpr int kGroupRing = 4;         // mbarriers that track the MMA groups in flight
constexpr uint32_t kTmemColumns = 256;    // S / P: 128 columns, O: D columns (at most 128)
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
    constexpr uint32_t kOColumn = kTileRows;                 // O sits after S in tensor memory
    // A thread turns its 64 logits (64 columns) into 64 probabilities in bf16 in two halves, and writes each half
    // (16 columns) over the first columns of the 32 logits it came from: nobody else reads or writes those (but for
    // the tile's first columns, which every thread of a row reads once for the reference, see below).  The MMA
    // thread is told about each half by itself, so that P V of the first half runs while the second is computed.
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_q, bar_k0, bar_pa[kGroupRing], bar_pb[kGroupRing], bar_group[kGroupRing];
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
    const uint32_t q_tile = base, k_tile = base + kTileBytes, v_tile = base + 2 * kTileBytes;

    if (tid == 0) {
        mbar_init(smem_u32(&bar_q), 1);
        mbar_init(smem_u32(&bar_k0), 1);
        for (int s = 0; s < kGroupRing; ++s) {
            mbar_init(smem_u32(&bar_pa[s]), kSoftmaxWarps + 1);   // first half of P(it) written, V(it) landed
            mbar_init(smem_u32(&bar_pb[s]), kSoftmaxWarps + 1);   // second half of P(it) written, K(it + 1) landed
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
            auto load = [&](const CUtensorMap* map, uint32_t bar, uint32_t dst, int row0, int head) {
                mbar_arrive_expect_tx(bar, kTileBytes);
#pragma unroll
                for (int bx = 0; bx < D / 64; ++bx) tma_load_3d(dst + bx * kBoxBytes, map, bx * 64, row0, head, bar);
            };
            load(&q_map, smem_u32(&bar_q), q_tile, qb * kTileRows, pr * p.Hq + h);
            load(&k_map, smem_u32(&bar_k0), k_tile, 0, pr * p.Hkv + kvh);
            // The MMA thread pays well over a hundred cycles for every mbarrier it looks at, so what it needs for
            // tile `it` arrives on TWO barriers: bar_pa[it % 4] collects the eight softmax warps (first half of P(it)
            // written) and the load V(it), bar_pb[it % 4] the same warps (second half) and the load K(it + 1).  There
            // is one K and one V tile: K(j + 1) takes the place of K(j) once S(j) is complete and V(j) that of
            // V(j - 1) once P V of tile j - 1 is, and both are in MMA group j.
            bool ok = true;
            for (int j = 0; j < n_it && ok; ++j) {
                if (j >= 1) ok = group_wait(j);
                if (!ok) break;
                load(&v_map, smem_u32(&bar_pa[j % kGroupRing]), v_tile, j * kTileRows, pr * p.Hkv + kvh);
                if (j == 0) ok = group_wait(0);
                if (!ok) break;
                const uint32_t bar = smem_u32(&bar_pb[j % kGroupRing]);
                if (j + 1 < n_it) load(&k_map, bar, k_tile, (j + 1) * kTileRows, pr * p.Hkv + kvh);
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
            // MMA, so the work is issued in groups with ONE commit each: group 0 = S(0),
            // group it + 1 = { O += P(it) V(it), S(it + 1) }.  S(it + 1) overwrites the logits and probabilities of
            // tile it, which P V has just read (the tensor pipe runs its work in order).  Completion of group g
            // tells the softmax warps that S(g) is ready and the producer that K(g) and V(g - 1) are consumed.
            // A descriptor's address field is (address >> 4), so stepping through a tile is an addition: the
            // issuing thread's instruction count per MMA matters.
            const uint64_t dq = tc::desc_k_major_sw128(q_tile), dk = tc::desc_k_major_sw128(k_tile);
            const uint64_t dv = tc::desc_mn_major_sw128(v_tile, kBoxBytes);
            auto issue_s = [&]() {
#pragma unroll
                for (int ks = 0; ks < kKSteps; ++ks) {
                    const uint32_t off = ((ks >> 2) * kBoxBytes + (ks & 3) * 32) >> 4;
                    tc::umma_bf16(tmem_base, dq + off, dk + off, idesc_s, ks > 0);
                }
            };
            bool ok = mbar_wait(smem_u32(&bar_q), 0);
            if (ok) ok = mbar_wait(smem_u32(&bar_k0), 0);
            if (ok) {
                tc::fence_after_sync();
                issue_s();
                tc::umma_commit(smem_u32(&bar_group[0]));
            }
            for (int it = 0; it < n_it && ok; ++it) {
                // 16 keys per step = 8 columns of probabilities; a thread's halves are keys 0..31 and 32..63 of its 64
                auto issue_pv = [&](int hh) {
#pragma unroll
                    for (int k4 = 0; k4 < kPvSteps / 2; ++k4) {
                        const int ks = (k4 >> 1) * 4 + hh * 2 + (k4 & 1);
                        tc::umma_bf16_ts(tmem_base + kOColumn, tmem_base + (ks >> 2) * 64 + hh * 32 + (ks & 1) * 8,
                                         dv + (ks * 2048 >> 4), idesc_o, (it > 0) || (hh > 0) || (k4 > 0));
                    }
                };
                // the first half of P(it) is written and V(it) has landed
                ok = mbar_wait(smem_u32(&bar_pa[it % kGroupRing]), (it / kGroupRing) & 1);
                if (!ok) break;
                tc::fence_after_sync();
                issue_pv(0);
                // the second half is written (so all of S(it) has been read) and K(it + 1) has landed
                ok = mbar_wait(smem_u32(&bar_pb[it % kGroupRing]), (it / kGroupRing) & 1);
                if (!ok) break;
                tc::fence_after_sync();
                issue_pv(1);
                if (it + 1 < n_it) issue_s();
                tc::umma_commit(smem_u32(&bar_group[(it + 1) % kGroupRing]));
            }
            if (!ok) sm_abort = 1;
        }
    } else {
        // ---------------- softmax warps: a warp reads its quarter of the TMEM lanes (thread = query row);
        // the first four of them take keys 0..63 of every tile, the others keys 64..127
        const int row = 32 * (warp & 3) + lane;
        const int part = (warp - 2) >> 2;                     // 0 .. 1
        const int col_base = part * 64;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16);
        const int t = qb * kTileRows + row;
        // the softmax's reference logit of this row, log2 domain (exact mode: the row's maximum; +inf past the prompt)
        float lse = 0.0f;
        if (kExact) lse = t < p.T ? p.lse2[((int64_t)pr * p.Hq + h) * p.T + t] : INFINITY;
        bool ok = true;
        for (int it = 0; it < n_it; ++it) {
            if (!group_wait(it)) { ok = false; break; }        // S(it) is ready
            tc::fence_after_sync();
            if (!kExact && it == 0) {
                // reference = the row's largest logit among the first eight keys (those of them it may see):
                // every thread of the row reads the same eight columns, so the two agree without talking
                uint32_t first[8];
                tc::tmem_ld_32x32_x8(lane_addr, first);
                tc::tmem_ld_wait();
                float mx = __uint_as_float(first[0]);
#pragma unroll
                for (int c = 1; c < 8; ++c)
                    if (qb > 0 || c <= row) mx = fmaxf(mx, __uint_as_float(first[c]));
                lse = mx * p.scale_log2;
                // (the first probabilities go over these columns: not before every thread has read them)
                asm volatile("bar.sync 1, 256;" ::: "memory");
            }
            // probabilities of this thread's 64 keys -> bf16, two per 32-bit column of the A operand
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                uint32_t v[32];
                tc::tmem_ld_32x32(lane_addr + col_base + hh * 32, v);
                tc::tmem_ld_wait();
                if (it == qb) {                               // diagonal tile: keys above the query do not exist
#pragma unroll
                    for (int c = 0; c < 32; ++c)
                        if (col_base + hh * 32 + c > row) v[c] = 0xff800000u;
                }
                uint32_t w[16];
#pragma unroll
                for (int c = 0; c < 16; ++c)
                    w[c] = pack_bf16(fast_exp2(fmaf(__uint_as_float(v[2 * c]), p.scale_log2, -lse)),
                                     fast_exp2(fmaf(__uint_as_float(v[2 * c + 1]), p.scale_log2, -lse)));
                tc::tmem_st_32x32_x16(lane_addr + col_base + hh * 32, w);
                tc::tmem_st_wait();
                tc::fence_before_sync();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(smem_u32(hh == 0 ? &bar_pa[it % kGroupRing] : &bar_pb[it % kGroupRing]));
            }
        }
        // ---- O is complete: cosine between V_t and O_t; the V rows of this CTA's tokens are the diagonal tile,
        // the last one loaded.  Two threads per row take half of the head dimension each.
        if (ok) ok = group_wait(n_it);                        // the last group: O is complete
        float dot = 0.0f, vv = 0.0f, oo = 0.0f;
        if (ok) {
            tc::fence_after_sync();
            const uint8_t* v_row = base_ptr + 2 * kTileBytes + row * 128;
#pragma unroll
            for (int ch = 0; ch < D / 64; ++ch) {             // 32 columns of the head dimension at a time
                const int col0 = part * (D / 2) + ch * 32;
                uint32_t o[32];
                tc::tmem_ld_32x32(lane_addr + kOColumn + col0, o);
                tc::tmem_ld_wait();
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {              // 16-byte pieces of 8 elements
                    const int piece = col0 / 8 + cc;          // within the row: 0 .. D/8 - 1
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
        }
        // join the two halves of every row through shared memory (the K tile is idle by now)
        float* sm_part = reinterpret_cast<float*>(base_ptr + kTileBytes);   // [3][2][128]
        sm_part[(0 * 2 + part) * kTileRows + row] = dot;
        sm_part[(1 * 2 + part) * kTileRows + row] = vv;
        sm_part[(2 * 2 + part) * kTileRows + row] = oo;
        asm volatile("bar.sync 1, 256;" ::: "memory");
        float c = 0.0f;
        if (part == 0 && ok && t < len) {
            const float d2 = sm_part[(0 * 2 + 0) * kTileRows + row] + sm_part[(0 * 2 + 1) * kTileRows + row];
            const float v2 = sm_part[(1 * 2 + 0) * kTileRows + row] + sm_part[(1 * 2 + 1) * kTileRows + row];
            const float o2 = sm_part[(2 * 2 + 0) * kTileRows + row] + sm_part[(2 * 2 + 1) * kTileRows + row];
            c = d2 / fmaxf(sqrtf(v2) * sqrtf(o2), kCosEps);
            if (!kExact && !(fabsf(d2) <= 3.0e38f && o2 <= 3.0e38f)) {   // left the fp32 range (or NaN): redo this block
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
        mbar_inval(smem_u32(&bar_k0));
        for (int s = 0; s < kGroupRing; ++s) {
            mbar_inval(smem_u32(&bar_pa[s]));
            mbar_inval(smem_u32(&bar_pb[s]));
            mbar_inval(smem_u32(&bar_group[s]));
        }
    }
    __syncthreads();
}

// One pass over every row block of the layer: grid (row blocks, query heads, prompts), long blocks first.
template <int D>
__global__ void __launch_bounds__(kThreads, 2) profile_pv_kernel(const ProfileParams p,
                                                                 const __grid_constant__ CUtensorMap q_map,
                                                                 const __grid_constant__ CUtensorMap k_map,
                                                                 const __grid_constant__ CUtensorMap v_map) {
    profile_pv_block<D, false>(p, q_map, k_map, v_map, p.n_blk - 1 - (int)blockIdx.x, blockIdx.y, blockIdx.z);
}

// The exact form over the row blocks the one-pass kernel listed: a small fixed grid whose CTAs take the
// entries in turn, so that the usual empty list costs nothing.
template <int D>
__global__ void __launch_bounds__(kThreads, 2) profile_pv_redo_kernel(const ProfileParams p,
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
    // the Q, K and V tiles; at least 80 KB, so that never more than two CTAs (2 x 256 TMEM columns) share an SM
    constexpr int kSmem = (3 * kTileRows * D * 2 + 1024) > 80 * 1024 ? (3 * kTileRows * D * 2 + 1024) : 80 * 1024;
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
