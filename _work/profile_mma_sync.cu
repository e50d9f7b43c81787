// Head-similarity profiling (Algorithm 1, step 1): for every prompt and query head of one layer,
// causal softmax attention O = softmax(Q K^T / sqrt(D)) V and the token-wise cosine between the
// head's input V_t and its output O_t, averaged over the prompt's tokens.
//
// One CTA owns 64 query rows of one (prompt, head): four warps of 16 rows each.  K and V tiles of
// 64 keys are brought in by TMA (128-byte swizzle) into a two-stage ring; logits and P.V run on
// the tensor cores (bf16 mma.sync, fp32 accumulate) with an online softmax.  O is never written:
// the last key tile is the diagonal one, whose V rows are exactly the rows the cosine needs, so
// the epilogue reads them from shared memory.  Per-CTA cosine sums go to the workspace and a
// second kernel adds them in a fixed order (deterministic mean).
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>

#include "baklava.h"
#include "common.h"

namespace {

constexpr int kRows = 64;          // query rows per CTA = keys per tile
constexpr int kThreads = 128;
constexpr uint32_t kWaitLimit = 1u << 22;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kCosEps = 1e-12f;

struct ProfileParams {
    const int32_t* prompt_len;   // [P] or null
    float* head_cos;             // [P, Hq]
    float* token_cos;            // [P, Hq, T] or null
    float* block_sum;            // [P, Hq, n_qb]
    uint32_t* error;             // one word in the workspace, set when a bounded wait gives up
    int32_t P, T, Hq, Hkv, n_qb;
    float scale_log2;
};

__device__ __forceinline__ uint32_t smem_u32(const void* ptr) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(ptr));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kWaitLimit; ++i) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}
// 16-byte piece `piece` of row `row` in a [64][D] bf16 tile written by TMA with the 128-byte swizzle
__device__ __forceinline__ uint32_t tile_offset(int row, int piece) {
    return (uint32_t)((piece >> 3) * (kRows * 128) + row * 128 + (((piece & 7) ^ (row & 7)) << 4));
}

template <int D>
__global__ void __launch_bounds__(kThreads) profile_kernel(const ProfileParams p,
                                                           const __grid_constant__ CUtensorMap q_map,
                                                           const __grid_constant__ CUtensorMap k_map,
                                                           const __grid_constant__ CUtensorMap v_map) {
    constexpr int kKSteps = D / 16;
    constexpr int kNTiles = D / 8;
    constexpr int kTileBytes = kRows * D * 2;

    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_q;
    __shared__ __align__(8) uint64_t bar_kv[2];
    __shared__ float sm_sum[kThreads / 32];
    __shared__ int sm_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int qb = p.n_qb - 1 - blockIdx.x;               // long rows of the causal triangle first
    const int h = blockIdx.y, pr = blockIdx.z;
    const int kvh = h / (p.Hq / p.Hkv);
    const int len = p.prompt_len ? min(max(p.prompt_len[pr], 0), p.T) : p.T;
    float* out_sum = p.block_sum + ((int64_t)pr * p.Hq + h) * p.n_qb + qb;
    if (qb * kRows >= len) {
        if (tid == 0) *out_sum = 0.0f;
        return;
    }
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t q_tile = base;
    auto k_tile = [&](int s) { return base + kTileBytes + s * 2 * kTileBytes; };
    auto v_tile = [&](int s) { return base + 2 * kTileBytes + s * 2 * kTileBytes; };

    if (tid == 0) {
        mbar_init(smem_u32(&bar_q), 1);
        mbar_init(smem_u32(&bar_kv[0]), 1);
        mbar_init(smem_u32(&bar_kv[1]), 1);
        sm_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    auto issue_kv = [&](int kb) {
        const int s = kb & 1;
        const uint32_t bar = smem_u32(&bar_kv[s]);
        mbar_arrive_expect_tx(bar, 2 * kTileBytes);
#pragma unroll
        for (int bx = 0; bx < D / 64; ++bx) {
            tma_load_3d(k_tile(s) + bx * (kRows * 128), &k_map, bx * 64, kb * kRows, pr * p.Hkv + kvh, bar);
            tma_load_3d(v_tile(s) + bx * (kRows * 128), &v_map, bx * 64, kb * kRows, pr * p.Hkv + kvh, bar);
        }
    };
    if (tid == 0) {
        mbar_arrive_expect_tx(smem_u32(&bar_q), kTileBytes);
#pragma unroll
        for (int bx = 0; bx < D / 64; ++bx)
            tma_load_3d(q_tile + bx * (kRows * 128), &q_map, bx * 64, qb * kRows, pr * p.Hq + h, smem_u32(&bar_q));
        issue_kv(0);
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
    float o[kNTiles][4];
#pragma unroll
    for (int j = 0; j < kNTiles; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.0f; }

    for (int kb = 0; kb <= qb; ++kb) {
        __syncthreads();                                   // everyone is done with the stage kb + 1 will overwrite
        if (sm_abort) break;
        if (tid == 0 && kb + 1 <= qb) issue_kv(kb + 1);
        const int s = kb & 1;
        if (!alive || !mbar_wait(smem_u32(&bar_kv[s]), (kb >> 1) & 1)) {
            alive = false;
            sm_abort = 1;
            continue;
        }
        float sacc[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) { sacc[nt][0] = sacc[nt][1] = sacc[nt][2] = sacc[nt][3] = 0.0f; }
#pragma unroll
        for (int ks = 0; ks < kKSteps; ++ks) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                uint32_t kf[4];
                ldmatrix_x4(k_tile(s) + tile_offset(16 * kk + (lm >> 1) * 8 + li8, 2 * ks + (lm & 1)), kf);
                mma_bf16(sacc[2 * kk], qa[ks], kf[0], kf[1]);
                mma_bf16(sacc[2 * kk + 1], qa[ks], kf[2], kf[3]);
            }
        }
        const bool diagonal = kb == qb;
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int key = 8 * nt + qcol + (e & 1);            // inside the tile
                const int row = r0 + qrow + (e >> 1) * 8;
                float v = sacc[nt][e] * p.scale_log2;
                if (diagonal && key > row) v = -INFINITY;           // causal mask
                sacc[nt][e] = v;
                mx[e >> 1] = fmaxf(mx[e >> 1], v);
            }
        float corr[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
            const float m_new = fmaxf(m_run[r], mx[r]);             // finite: key 0 is never masked
            corr[r] = exp2f(m_run[r] - m_new);
            m_run[r] = m_new;
        }
        float rs[2] = {0.0f, 0.0f};
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float pe = exp2f(sacc[nt][e] - m_run[e >> 1]);
                sacc[nt][e] = pe;
                rs[e >> 1] += pe;
            }
        l_run[0] = l_run[0] * corr[0] + rs[0];
        l_run[1] = l_run[1] * corr[1] + rs[1];
#pragma unroll
        for (int j = 0; j < kNTiles; ++j) {
            o[j][0] *= corr[0]; o[j][1] *= corr[0];
            o[j][2] *= corr[1]; o[j][3] *= corr[1];
        }
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            uint32_t pa[4];
            pa[0] = pack_bf16(sacc[2 * kk][0], sacc[2 * kk][1]);
            pa[1] = pack_bf16(sacc[2 * kk][2], sacc[2 * kk][3]);
            pa[2] = pack_bf16(sacc[2 * kk + 1][0], sacc[2 * kk + 1][1]);
            pa[3] = pack_bf16(sacc[2 * kk + 1][2], sacc[2 * kk + 1][3]);
#pragma unroll
            for (int j2 = 0; j2 < kNTiles / 2; ++j2) {
                uint32_t vf[4];
                ldmatrix_x4_trans(v_tile(s) + tile_offset(16 * kk + (lm & 1) * 8 + li8, 2 * j2 + (lm >> 1)), vf);
                mma_bf16(o[2 * j2], pa, vf[0], vf[1]);
                mma_bf16(o[2 * j2 + 1], pa, vf[2], vf[3]);
            }
        }
    }
    __syncthreads();
    if (sm_abort) {
        if (tid == 0) { atomicOr(p.error, 1u); *out_sum = 0.0f; }
        return;
    }

    // ---- cosine between V_t and O_t; the V rows of this CTA's tokens are the diagonal tile (stage qb & 1)
    const uint8_t* v_rows = base_ptr + 2 * kTileBytes + (qb & 1) * 2 * kTileBytes;
    float my_sum = 0.0f;
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int row = r0 + qrow + r * 8;
        float dot = 0.0f, vv = 0.0f, oo = 0.0f;
#pragma unroll
        for (int j = 0; j < kNTiles; ++j) {
            const uint32_t raw = *reinterpret_cast<const uint32_t*>(v_rows + tile_offset(row, j) + qcol * 2);
            const float2 vx = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw));
            const float o0 = o[j][2 * r], o1 = o[j][2 * r + 1];
            dot = fmaf(vx.x, o0, fmaf(vx.y, o1, dot));
            vv = fmaf(vx.x, vx.x, fmaf(vx.y, vx.y, vv));
            oo = fmaf(o0, o0, fmaf(o1, o1, oo));
        }
#pragma unroll
        for (int off = 1; off <= 2; off <<= 1) {
            dot += __shfl_xor_sync(0xffffffffu, dot, off);
            vv += __shfl_xor_sync(0xffffffffu, vv, off);
            oo += __shfl_xor_sync(0xffffffffu, oo, off);
        }
        // O here is unnormalised (missing 1 / l): the cosine does not depend on a positive scale,
        // except through the floor on the denominator, so apply 1 / l to the norm product
        float lr = l_run[r];
        lr += __shfl_xor_sync(0xffffffffu, lr, 1);
        lr += __shfl_xor_sync(0xffffffffu, lr, 2);
        const float inv_l = 1.0f / lr;
        const float c = (dot * inv_l) / fmaxf(sqrtf(vv) * sqrtf(oo) * inv_l, kCosEps);
        const int t = qb * kRows + row;
        if (t < len && (lane & 3) == 0) {
            my_sum += c;
            if (p.token_cos) p.token_cos[((int64_t)pr * p.Hq + h) * p.T + t] = c;
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) my_sum += __shfl_xor_sync(0xffffffffu, my_sum, off);
    if (lane == 0) sm_sum[warp] = my_sum;
    __syncthreads();
    if (tid == 0) *out_sum = (sm_sum[0] + sm_sum[1]) + (sm_sum[2] + sm_sum[3]);
}

__global__ void profile_mean_kernel(const ProfileParams p) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;   // (prompt, head)
    if (i >= p.P * p.Hq) return;
    const int pr = i / p.Hq;
    const int len = p.prompt_len ? min(max(p.prompt_len[pr], 0), p.T) : p.T;
    float acc = 0.0f;
    for (int b = 0; b < p.n_qb; ++b) acc += p.block_sum[(int64_t)i * p.n_qb + b];
    p.head_cos[i] = len > 0 ? acc / (float)len : 0.0f;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// bf16 [heads, T, D]: boxes of 64 tokens x 64 elements of one head, 128-byte swizzle, zero fill past T
bool make_map(CUtensorMap* map, const void* base, int64_t heads, int T, int D) {
    static EncodeTiledFn enc = nullptr;
    if (!enc) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult res;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &res) != cudaSuccess ||
            res != cudaDriverEntryPointSuccess)
            return false;
        enc = reinterpret_cast<EncodeTiledFn>(sym);
    }
    const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)T, (cuuint64_t)heads};
    const cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)T * D * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)kRows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D>
cudaError_t launch_profile(const ProfileParams& p, const CUtensorMap& qm, const CUtensorMap& km, const CUtensorMap& vm,
                           cudaStream_t s) {
    constexpr int kSmem = 5 * kRows * D * 2 + 1024;      // Q tile + two (K, V) stages
    cudaError_t e = cudaFuncSetAttribute(profile_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    const dim3 grid(p.n_qb, p.Hq, p.P);
    profile_kernel<D><<<grid, kThreads, kSmem, s>>>(p, qm, km, vm);
    return cudaGetLastError();
}

}  // namespace

extern "C" __attribute__((visibility("default"))) size_t baklava_profile_workspace_size(const baklava_shape* shape,
                                                                                    int32_t P, int32_t T) {
    if (!shape || P <= 0 || T <= 0) return 0;
    const size_t n_qb = ((size_t)T + kRows - 1) / kRows;
    return 256 + sizeof(float) * (size_t)P * shape->Hq * n_qb;
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
    p.block_sum = reinterpret_cast<float*>(static_cast<char*>(ws) + 256);
    p.P = P; p.T = T; p.Hq = shape->Hq; p.Hkv = shape->Hkv;
    p.n_qb = (T + kRows - 1) / kRows;
    p.scale_log2 = kLog2e / sqrtf((float)shape->D);

    CUtensorMap qm, km, vm;
    if (!make_map(&qm, q, (int64_t)P * shape->Hq, T, shape->D) ||
        !make_map(&km, k, (int64_t)P * shape->Hkv, T, shape->D) ||
        !make_map(&vm, v, (int64_t)P * shape->Hkv, T, shape->D))
        return BAKLAVA_ERR_CUDA;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(ws, 0, 256, s) != cudaSuccess) return BAKLAVA_ERR_CUDA;
    cudaError_t err = shape->D == 128 ? launch_profile<128>(p, qm, km, vm, s) : launch_profile<64>(p, qm, km, vm, s);
    if (err != cudaSuccess) return BAKLAVA_ERR_CUDA;
    const int n = P * shape->Hq;
    profile_mean_kernel<<<(n + 127) / 128, 128, 0, s>>>(p);
    return cudaGetLastError() == cudaSuccess ? BAKLAVA_OK : BAKLAVA_ERR_CUDA;
}
