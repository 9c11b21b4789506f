// Dense bf16 GEMM on tcgen05 for the frozen LM head (the one genuinely compute-bound part
// of the path):
//     logits = y W_lm^T          [M x d] x [V x d]^T     B operand K-major  (rows of W_lm)
//     dy     = dlogits W_lm      [M x V] x [V x d]       B operand MN-major (W_lm as stored)
// C[M][N] (fp32) = A[M][K] (bf16, row-major) x B, 128 x 256 output tiles, K steps of 64,
// TMA-fed shared-memory ring, accumulators double-buffered in TMEM (2 x 256 columns) so the
// epilogue of one tile overlaps the MMAs of the next.  Persistent CTAs walk tiles with the M
// index fastest, so the CTAs running at the same time share B tiles through L2.
#pragma once
#include "pac_tensor.cuh"

namespace pac {

constexpr int GT_BM = 128, GT_BN = 256, GT_BK = 64, GT_STAGES = 4;
constexpr uint32_t GT_A_BYTES = GT_BM * GT_BK * 2, GT_B_BYTES = GT_BN * GT_BK * 2, GT_STAGE = GT_A_BYTES + GT_B_BYTES;
constexpr size_t GT_SMEM = (size_t)GT_STAGES * GT_STAGE + 1024;

struct GemmParams {
    int M, N, K;
    int m_tiles, n_tiles, k_chunks;
    int b_mn_major;            // 0: B stored [N][K] (K contiguous); 1: B stored [K][N] (N contiguous)
    float* C; long long ldc;
    unsigned* status;
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}

__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, GemmParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) unsigned long long bars[2 * GT_STAGES + 4];
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[GT_STAGES]);
    const uint32_t accf0 = smem_u32(&bars[2 * GT_STAGES]), acce0 = smem_u32(&bars[2 * GT_STAGES + 2]);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = p.m_tiles * p.n_tiles;

    if (threadIdx.x == 0) {
        abort_sh = 0;
        for (int s = 0; s < GT_STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(accf0 + 8 * b, 1); mbar_init(acce0 + 8 * b, 4); }
        fence_mbar_init();
        tma_prefetch_desc(&map_a);
        tma_prefetch_desc(&map_b);
    }
    if (warp == 1) { tmem_alloc(smem_u32(&tmem_base_sh), 512u); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_sh;
    volatile int* abort_flag = &abort_sh;

    // Both pipeline loops are run by whole converged warps with one elected lane issuing, so that
    // addresses, coordinates and descriptors stay warp-uniform values.
    if (warp == 0) {
        uint32_t it = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
            const int m0 = (t % p.m_tiles) * GT_BM, n0 = (t / p.m_tiles) * GT_BN;
            for (int kc = 0; kc < p.k_chunks; ++kc, ++it) {
                const int s = it % GT_STAGES;
                const uint32_t ph = (it / GT_STAGES) & 1;
                if (!mbar_wait_uniform(empty0 + 8 * s, ph ^ 1, abort_flag, p.status)) { ok = false; break; }
                const uint32_t dst = smem_u32(smem + (size_t)s * GT_STAGE);
                if (elect_one()) {
                    mbar_expect_tx(full0 + 8 * s, GT_STAGE);
                    tma_load_2d(dst, &map_a, full0 + 8 * s, kc * GT_BK, m0);
                    if (p.b_mn_major) {
                        for (int q = 0; q < GT_BN / 64; ++q)       // [64 k][64 n] boxes, one per 64 columns of N
                            tma_load_2d(dst + GT_A_BYTES + q * 8192, &map_b, full0 + 8 * s, n0 + q * 64, kc * GT_BK);
                    } else {
                        tma_load_2d(dst + GT_A_BYTES, &map_b, full0 + 8 * s, kc * GT_BK, n0);
                    }
                }
                __syncwarp();
            }
        }
    } else if (warp == 1) {
        const uint32_t idesc = instr_desc_bf16(GT_BM, GT_BN, 0, p.b_mn_major);
        uint32_t it = 0, tile_n = 0;
        for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++tile_n) {
            const int buf = tile_n & 1;
            const uint32_t aph = (tile_n >> 1) & 1;
            if (!mbar_wait_uniform(acce0 + 8 * buf, aph ^ 1, abort_flag, p.status)) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(buf * GT_BN);
            bool ok = true;
            for (int kc = 0; kc < p.k_chunks; ++kc, ++it) {
                const int s = it % GT_STAGES;
                const uint32_t ph = (it / GT_STAGES) & 1;
                if (!mbar_wait_uniform(full0 + 8 * s, ph, abort_flag, p.status)) { ok = false; break; }
                tc_fence_after();
                const uint32_t a0 = smem_u32(smem + (size_t)s * GT_STAGE), b0 = a0 + GT_A_BYTES;
                const uint64_t ad0 = smem_desc_sw128(a0, 16, 1024);
                // K-major B: 256 rows of 128 B; MN-major B: four [64 k][128 B] blocks 8192 B apart
                const uint64_t bd0 = p.b_mn_major ? smem_desc_sw128(b0, 8192, 1024) : smem_desc_sw128(b0, 16, 1024);
                const uint64_t bstep = p.b_mn_major ? 128u : 2u;     // 16 K elements further, in 16-byte units
                if (elect_one()) {
#pragma unroll
                    for (int k = 0; k < GT_BK / 16; ++k)
                        umma_bf16(d_tmem, ad0 + (uint64_t)(k * 2), bd0 + bstep * k, idesc, (kc | k) ? 1u : 0u);
                    umma_commit(empty0 + 8 * s);
                }
                __syncwarp();
            }
            if (!ok) break;
            if (elect_one()) umma_commit(accf0 + 8 * buf);
            __syncwarp();
        }
    } else {
        const int q = warp & 3;
        uint32_t tile_n = 0;
        for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++tile_n) {
            const int m0 = (t % p.m_tiles) * GT_BM, n0 = (t / p.m_tiles) * GT_BN;
            const int buf = tile_n & 1;
            const uint32_t aph = (tile_n >> 1) & 1;
            if (!mbar_wait_warp(accf0 + 8 * buf, aph, abort_flag, p.status)) break;
            tc_fence_after();
            const int row = m0 + q * 32 + lane;
            float* dst = p.C + (long long)row * p.ldc + n0;
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * GT_BN);
            const bool vec_ok = (p.ldc & 3) == 0;
            for (int c0 = 0; c0 < GT_BN; c0 += 32) {
                float v[32];
                tmem_ld32(taddr + c0, v);
                tmem_ld_wait();
                if (row < p.M) {
                    if (vec_ok && n0 + c0 + 32 <= p.N) {
#pragma unroll
                        for (int c = 0; c < 32; c += 4) *reinterpret_cast<float4*>(dst + c0 + c) = make_float4(v[c], v[c + 1], v[c + 2], v[c + 3]);
                    } else {
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (n0 + c0 + c < p.N) dst[c0 + c] = v[c];
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acce0 + 8 * buf);
        }
    }
    tc_fence_before();
    __syncthreads();
    drain_after_abort(abort_flag);
    if (warp == 1) tmem_dealloc(tmem_base, 512u);
}

// Host side: tensor maps and launch for one GEMM shape.
struct GemmPlan {
    bool ready = false;
    CUtensorMap map_a, map_b;
    int b_mn_major = 0, N = 0, K = 0, sms = 0;
};

// A: [rows_a][K] bf16 row-major.  B: K-major [N][K], or MN-major [K][N].
inline pac_status gemm_plan_create(GemmPlan& gp, int device, const bf16* A, long long rows_a, const bf16* B, int N, int K,
                                   int b_mn_major) {
    gp.ready = false;
    if (N % 8 != 0 || K % 8 != 0) { tensor_err() = "GEMM operand rows are not 16-byte multiples"; return PAC_ERR_UNSUPPORTED; }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { tensor_err() = "cudaGetDeviceProperties failed"; return PAC_ERR_CUDA; }
    if (prop.major != 10) { tensor_err() = "device is not sm_100"; return PAC_ERR_UNSUPPORTED; }
    gp.sms = prop.multiProcessorCount;
    {
        cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows_a};
        cuuint64_t str[1] = {(cuuint64_t)K * 2};
        cuuint32_t box[2] = {GT_BK, GT_BM};
        if (!make_map(&gp.map_a, A, 2, dims, str, box)) return PAC_ERR_UNSUPPORTED;
    }
    if (b_mn_major) {
        cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)K};
        cuuint64_t str[1] = {(cuuint64_t)N * 2};
        cuuint32_t box[2] = {64, GT_BK};
        if (!make_map(&gp.map_b, B, 2, dims, str, box)) return PAC_ERR_UNSUPPORTED;
    } else {
        cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)N};
        cuuint64_t str[1] = {(cuuint64_t)K * 2};
        cuuint32_t box[2] = {GT_BK, GT_BN};
        if (!make_map(&gp.map_b, B, 2, dims, str, box)) return PAC_ERR_UNSUPPORTED;
    }
    if (cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GT_SMEM) != cudaSuccess) {
        tensor_err() = "cudaFuncSetAttribute(MaxDynamicSharedMemorySize) failed";
        cudaGetLastError();
        return PAC_ERR_CUDA;
    }
    gp.b_mn_major = b_mn_major; gp.N = N; gp.K = K;
    gp.ready = true;
    return PAC_OK;
}

inline pac_status gemm_launch(const GemmPlan& gp, cudaStream_t stream, int M, float* C, long long ldc, unsigned* status,
                              long long* launches) {
    GemmParams p{};
    p.M = M; p.N = gp.N; p.K = gp.K;
    p.m_tiles = (M + GT_BM - 1) / GT_BM;
    p.n_tiles = (gp.N + GT_BN - 1) / GT_BN;
    p.k_chunks = (gp.K + GT_BK - 1) / GT_BK;
    p.b_mn_major = gp.b_mn_major;
    p.C = C; p.ldc = ldc; p.status = status;
    const int tiles = p.m_tiles * p.n_tiles;
    const int grid = tiles < gp.sms ? tiles : gp.sms;
    gemm_tc_kernel<<<grid, TC_THREADS, GT_SMEM, stream>>>(gp.map_a, gp.map_b, p);
    (*launches)++;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { tensor_err() = cudaGetErrorString(e); return PAC_ERR_CUDA; }
    return PAC_OK;
}

}  // namespace pac
