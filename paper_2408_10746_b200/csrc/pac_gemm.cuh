// Dense bf16 GEMM on tcgen05 for the frozen LM head (the one genuinely compute-bound part
// of the path):
//     logits = y W_lm^T          [M x d] x [V x d]^T     B operand K-major  (rows of W_lm)
//     dy     = dlogits W_lm      [M x V] x [V x d]       B operand MN-major (W_lm as stored)
// C[M][N] (fp32) = A[M][K] (bf16, row-major) x B, 128 x 256 output tiles, K steps of 64,
// TMA-fed shared-memory ring, accumulators double-buffered in TMEM (2 x 256 columns) so the
// epilogue of one tile overlaps the MMAs of the next.  Persistent CTAs walk tiles with the M
// index fastest, so the CTAs running at the same time share B tiles through L2.
//
// PAIR: the CTAs work as 2-CTA clusters on 256 x 256 tiles (tcgen05.mma.cta_group::2): each CTA loads
// its own 128 rows of A and HALF of the B tile (128 of the 256 columns), the CTA of rank 0 counts the
// bytes of both on its barriers and issues the MMAs.  A single CTA takes in 48 KB per K step for 512
// clocks of tensor work, more than the 64 bytes per clock an SM receives from L2; a CTA of a pair
// takes in 32 KB, and its ring is six stages deep instead of four.
#pragma once
#include <cooperative_groups.h>

#include "pac_tensor.cuh"

namespace pac {

constexpr int GT_BM = 128, GT_BN = 256, GT_BK = 64, GT_STAGES = 4;
constexpr uint32_t GT_A_BYTES = GT_BM * GT_BK * 2, GT_B_BYTES = GT_BN * GT_BK * 2, GT_STAGE = GT_A_BYTES + GT_B_BYTES;
constexpr size_t GT_SMEM = (size_t)GT_STAGES * GT_STAGE + 1024;
constexpr int GT_STAGES_PAIR = 6;
constexpr uint32_t GT_STAGE_PAIR = GT_A_BYTES + GT_B_BYTES / 2;
constexpr size_t GT_SMEM_PAIR = (size_t)GT_STAGES_PAIR * GT_STAGE_PAIR + 1024;

struct GemmParams {
    int M, N, K;
    int m_tiles, n_tiles, k_chunks;
    int b_mn_major;            // 0: B stored [N][K] (K contiguous); 1: B stored [K][N] (N contiguous)
    float* C; long long ldc;   // fp32 output (may be null when only the bf16 output is wanted)
    bf16* C16; long long ldc16; // optional second output: the same values rounded to bf16
    // optional: add the last cached layer's row to every output row before storing, so that
    // y = h_L + a_L W_up (Section IV-A) leaves the GEMM ready for the LM head; N == d then
    const bf16* add_cache; const int* ids; long long n_cache; int L, S;
    unsigned* status;
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}

__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1) : "memory");
}

// map_b: PAIR and K-major B: boxes of 128 rows; otherwise as in the single-CTA form.
template <bool PAIR>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, GemmParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    constexpr int STAGES = PAIR ? GT_STAGES_PAIR : GT_STAGES;
    constexpr uint32_t STAGE = PAIR ? GT_STAGE_PAIR : GT_STAGE;
    __shared__ __align__(8) unsigned long long bars[2 * GT_STAGES_PAIR + 4];
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[STAGES]);
    const uint32_t accf0 = smem_u32(&bars[2 * STAGES]), acce0 = smem_u32(&bars[2 * STAGES + 2]);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint32_t rank = 0;                                         // in the pair; 0 issues the MMAs
    if constexpr (PAIR) rank = cooperative_groups::this_cluster().block_rank();
    // a unit of work: one tile, or the two tiles of a pair (M indices 2i and 2i + 1, one N index)
    const int m_units = PAIR ? (p.m_tiles + 1) / 2 : p.m_tiles;
    const int n_units = m_units * p.n_tiles;
    const int unit0 = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x, unit_step = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;

    if (threadIdx.x == 0) {
        abort_sh = 0;
        for (int s = 0; s < STAGES; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(accf0 + 8 * b, 1); mbar_init(acce0 + 8 * b, PAIR ? 8 : 4); }
        fence_mbar_init();
        tma_prefetch_desc(&map_a);
        tma_prefetch_desc(&map_b);
    }
    if (warp == 1) {
        if constexpr (PAIR) { tmem_alloc_pair(smem_u32(&tmem_base_sh), 512u); tmem_relinquish_pair(); }
        else { tmem_alloc(smem_u32(&tmem_base_sh), 512u); tmem_relinquish(); }
    }
    tc_fence_before();
    __syncthreads();
    if constexpr (PAIR) cooperative_groups::this_cluster().sync();     // the peer's barriers exist before anything arrives at them
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_sh;
    volatile int* abort_flag = &abort_sh;

    // Both pipeline loops are run by whole converged warps with one elected lane issuing, so that
    // addresses, coordinates and descriptors stay warp-uniform values.
    if (warp == 0) {
        uint32_t s = 0, eph = 1;                               // eph: parity of the "stage free" phase to wait for
        const uint32_t ring0 = smem_u32(smem);
        uint32_t dst = ring0;
        bool ok = true;
        for (int t = unit0; t < n_units && ok; t += unit_step) {
            const int m0 = ((t % m_units) * (PAIR ? 2 : 1) + (int)rank) * GT_BM, n0 = (t / m_units) * GT_BN;
            for (int kc = 0; kc < p.k_chunks; ++kc) {
                if (!mbar_wait_uniform(empty0 + 8 * s, eph, abort_flag, p.status)) { ok = false; break; }
                if (elect_one()) {
                    if constexpr (PAIR) {
                        // both CTAs: own rows of A, own half of B's columns, counted on the barrier of CTA 0
                        const uint32_t full = mapa_shared(full0 + 8 * s, 0u);
                        if (rank == 0) mbar_expect_tx(full0 + 8 * s, 2 * STAGE);
                        tma_load_2d_pair(dst, &map_a, full, kc * GT_BK, m0);
                        if (p.b_mn_major) {
                            for (int q = 0; q < GT_BN / 128; ++q)  // [64 k][64 n] boxes, one per 64 columns of N
                                tma_load_2d_pair(dst + GT_A_BYTES + q * 8192, &map_b, full, n0 + ((int)rank * 2 + q) * 64, kc * GT_BK);
                        } else {
                            tma_load_2d_pair(dst + GT_A_BYTES, &map_b, full, kc * GT_BK, n0 + (int)rank * (GT_BN / 2));
                        }
                    } else {
                        const uint32_t full = full0 + 8 * s;
                        mbar_expect_tx(full, STAGE);
                        tma_load_2d(dst, &map_a, full, kc * GT_BK, m0);
                        if (p.b_mn_major) {
                            for (int q = 0; q < GT_BN / 64; ++q)   // [64 k][64 n] boxes, one per 64 columns of N
                                tma_load_2d(dst + GT_A_BYTES + q * 8192, &map_b, full, n0 + q * 64, kc * GT_BK);
                        } else {
                            tma_load_2d(dst + GT_A_BYTES, &map_b, full, kc * GT_BK, n0);
                        }
                    }
                }
                __syncwarp();
                dst += STAGE;
                if (++s == (uint32_t)STAGES) { s = 0; eph ^= 1u; dst = ring0; }
            }
        }
    } else if (warp == 1) {
        if (!PAIR || rank == 0) {
            const uint32_t idesc = instr_desc_bf16(PAIR ? 2 * GT_BM : GT_BM, GT_BN, 0, p.b_mn_major);
            // descriptors of a stage's first K step (start-address field in 16-byte units).  K-major B: rows of
            // 128 B; MN-major B: [64 k][128 B] blocks 8192 B apart
            const uint32_t ring0 = smem_u32(smem);
            const uint64_t a_desc0 = smem_desc_sw128(ring0, 16, 1024);
            const uint64_t b_desc0 = p.b_mn_major ? smem_desc_sw128(ring0 + GT_A_BYTES, 8192, 1024) : smem_desc_sw128(ring0 + GT_A_BYTES, 16, 1024);
            const uint64_t bstep = p.b_mn_major ? 128u : 2u;     // 16 K elements further, in 16-byte units
            const uint64_t desc_step = (uint64_t)(STAGE >> 4);
            uint64_t doff = 0;
            uint32_t s = 0, ph = 0, tile_n = 0;
            for (int t = unit0; t < n_units; t += unit_step, ++tile_n) {
                const int buf = tile_n & 1;
                const uint32_t aph = (tile_n >> 1) & 1;
                if (!mbar_wait_uniform(acce0 + 8 * buf, aph ^ 1, abort_flag, p.status)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * GT_BN);
                bool ok = true;
                for (int kc = 0; kc < p.k_chunks; ++kc) {
                    if (!mbar_wait_uniform(full0 + 8 * s, ph, abort_flag, p.status)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t ad0 = a_desc0 + doff, bd0 = b_desc0 + doff;
                    if (elect_one()) {
#pragma unroll
                        for (int k = 0; k < GT_BK / 16; ++k) {
                            if constexpr (PAIR) umma_bf16_pair(d_tmem, ad0 + (uint64_t)(k * 2), bd0 + bstep * k, idesc, (kc | k) ? 1u : 0u);
                            else umma_bf16(d_tmem, ad0 + (uint64_t)(k * 2), bd0 + bstep * k, idesc, (kc | k) ? 1u : 0u);
                        }
                        if constexpr (PAIR) umma_commit_pair(empty0 + 8 * s, (uint16_t)3);
                        else umma_commit(empty0 + 8 * s);
                    }
                    __syncwarp();
                    doff += desc_step;
                    if (++s == (uint32_t)STAGES) { s = 0; ph ^= 1u; doff = 0; }
                }
                if (!ok) break;
                if (elect_one()) {
                    if constexpr (PAIR) umma_commit_pair(accf0 + 8 * buf, (uint16_t)3);
                    else umma_commit(accf0 + 8 * buf);
                }
                __syncwarp();
            }
        }
    } else {
        const int q = warp & 3;
        const uint32_t acce_arrive0 = PAIR ? mapa_shared(acce0, 0u) : acce0;     // the "drained" barriers of the CTA that issues the MMAs
        uint32_t tile_n = 0;
        for (int t = unit0; t < n_units; t += unit_step, ++tile_n) {
            const int m0 = ((t % m_units) * (PAIR ? 2 : 1) + (int)rank) * GT_BM, n0 = (t / m_units) * GT_BN;
            const int buf = tile_n & 1;
            const uint32_t aph = (tile_n >> 1) & 1;
            if (!mbar_wait_warp(accf0 + 8 * buf, aph, abort_flag, p.status)) break;
            tc_fence_after();
            const int row = m0 + q * 32 + lane;
            float* dst = p.C ? p.C + (long long)row * p.ldc + n0 : nullptr;
            bf16* dst16 = p.C16 ? p.C16 + (long long)row * p.ldc16 + n0 : nullptr;
            const bf16* hrow = nullptr;
            if (p.add_cache && row < p.M) {
                const int b = row / p.S, sidx = row - b * p.S;
                const long long id = safe_id(p.ids, b, p.n_cache, nullptr);
                hrow = p.add_cache + (((id * p.L) + (p.L - 1)) * p.S + sidx) * (long long)p.N + n0;
            }
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * GT_BN);
            const bool vec_ok = (p.ldc & 3) == 0, vec16_ok = (p.ldc16 & 7) == 0 && (p.N & 7) == 0;
            const bool vec32_ok = (p.ldc & 7) == 0 && (reinterpret_cast<uintptr_t>(p.C) & 31) == 0;
            for (int c0 = 0; c0 < GT_BN; c0 += 32) {
                float v[32];
                tmem_ld32(taddr + c0, v);
                tmem_ld_wait();
                if (row < p.M) {
                    const bool full = n0 + c0 + 32 <= p.N;
                    if (hrow) {
                        if (full && vec16_ok) {
#pragma unroll
                            for (int c = 0; c < 32; c += 8) {
                                const uint4 hv = *reinterpret_cast<const uint4*>(hrow + c0 + c);
                                const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&hv);
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const float2 f2 = __bfloat1622float2(h2[e]);
                                    v[c + 2 * e] += f2.x;
                                    v[c + 2 * e + 1] += f2.y;
                                }
                            }
                        } else {
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                if (n0 + c0 + c < p.N) v[c] += __bfloat162float(hrow[c0 + c]);
                        }
                    }
                    if (dst) {
                        if (vec32_ok && full) {
                            // whole 32-byte sectors
#pragma unroll
                            for (int c = 0; c < 32; c += 8)
                                st_global_32(dst + c0 + c, make_uint4(__float_as_uint(v[c]), __float_as_uint(v[c + 1]), __float_as_uint(v[c + 2]), __float_as_uint(v[c + 3])),
                                             make_uint4(__float_as_uint(v[c + 4]), __float_as_uint(v[c + 5]), __float_as_uint(v[c + 6]), __float_as_uint(v[c + 7])));
                        } else if (vec_ok && full) {
#pragma unroll
                            for (int c = 0; c < 32; c += 4) *reinterpret_cast<float4*>(dst + c0 + c) = make_float4(v[c], v[c + 1], v[c + 2], v[c + 3]);
                        } else {
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                if (n0 + c0 + c < p.N) dst[c0 + c] = v[c];
                        }
                    }
                    if (dst16) {
                        if (vec16_ok && full) {
#pragma unroll
                            for (int c = 0; c < 32; c += 8) {
                                __align__(16) __nv_bfloat162 o2[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) o2[e] = __floats2bfloat162_rn(v[c + 2 * e], v[c + 2 * e + 1]);
                                *reinterpret_cast<uint4*>(dst16 + c0 + c) = *reinterpret_cast<const uint4*>(o2);
                            }
                        } else {
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                if (n0 + c0 + c < p.N) dst16[c0 + c] = __float2bfloat16(v[c]);
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if constexpr (PAIR) mbar_arrive_cluster(acce_arrive0 + 8 * buf);
                else mbar_arrive(acce0 + 8 * buf);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    drain_after_abort(abort_flag);
    if constexpr (PAIR) {
        cooperative_groups::this_cluster().sync();     // neither CTA frees TMEM or leaves while the pair's MMAs or arrivals may still touch it
        if (warp == 1) tmem_dealloc_pair(tmem_base, 512u);
    } else {
        if (warp == 1) tmem_dealloc(tmem_base, 512u);
    }
}

// ---------------------------------------------------------------------------
// Cross-entropy of the LM head as a stream over the logits: rows of [M][V] fp32 in, loss per row
// and dlogits = (softmax - onehot) / M as bf16 out (the A operand of dy = dlogits W_lm).
// Persistent CTAs of 512 threads, one row at a time: the row (V <= 32768, V % 4 == 0) is held in
// registers, 16 float4 per thread, while the NEXT row is already on its way into shared memory
// as bulk asynchronous copies, so the logits are read from HBM exactly once and the read of one
// row overlaps the arithmetic and the write of the row before it.  All sums have a fixed order.
// ---------------------------------------------------------------------------
constexpr int CE_THREADS = 512, CE_V4_PER_THREAD = 16, CE_MAX_V = CE_THREADS * CE_V4_PER_THREAD * 4;
constexpr uint32_t CE_COPY_BYTES = 32768;                 // size of one bulk copy

__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

__global__ void __launch_bounds__(CE_THREADS, 1)
lm_ce_stream_kernel(const float* __restrict__ logits, const int* __restrict__ ids, long long N, const int* __restrict__ targets,
                    int S, int V, int M, float* __restrict__ loss_row, bf16* __restrict__ dlog16, unsigned* status) {
    extern __shared__ __align__(128) unsigned char ce_smem[];
    float4* row_s = reinterpret_cast<float4*>(ce_smem);
    __shared__ __align__(8) unsigned long long bar_sh;
    __shared__ float red[32];
    __shared__ int abort_sh;
    const uint32_t bar = smem_u32(&bar_sh);
    const int t = threadIdx.x;
    const uint32_t row_bytes = (uint32_t)V * 4u;
    const int n4 = V >> 2;
    volatile int* abort_flag = &abort_sh;
    if (t == 0) {
        abort_sh = 0;
        mbar_init(bar, 1);
        fence_mbar_init();
    }
    __syncthreads();
    auto issue = [&](int m) {                              // thread 0: the whole row as 32 KB pieces
        mbar_expect_tx(bar, row_bytes);
        const unsigned char* src = reinterpret_cast<const unsigned char*>(logits + (long long)m * V);
        for (uint32_t off = 0; off < row_bytes; off += CE_COPY_BYTES)
            bulk_load_1d(smem_u32(ce_smem) + off, src + off, min(CE_COPY_BYTES, row_bytes - off), bar);
    };
    int m = blockIdx.x;
    if (t == 0 && m < M) issue(m);
    uint32_t phase = 0;
    for (; m < M; m += gridDim.x, phase ^= 1) {
        // the row has landed -> registers; then the buffer is free for the next row
        int ok = 1;
        if ((t & 31) == 0) ok = mbar_wait(bar, phase, abort_flag, status) ? 1 : 0;
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!__syncthreads_and(ok)) break;
        float4 v[CE_V4_PER_THREAD];
#pragma unroll
        for (int i = 0; i < CE_V4_PER_THREAD; ++i) {
            const int e = i * CE_THREADS + t;
            v[i] = e < n4 ? row_s[e] : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        }
        __syncthreads();
        const int m_next = m + gridDim.x;
        if (t == 0 && m_next < M) { fence_proxy_async(); issue(m_next); }

        const int b = m / S, s = m - b * S;
        const long long id = safe_id(ids, b, N, (t == 0 && s == 0) ? status : nullptr);
        const int tgt = targets[id * S + s];
        float mx = -INFINITY;
#pragma unroll
        for (int i = 0; i < CE_V4_PER_THREAD; ++i) mx = fmaxf(mx, fmaxf(fmaxf(v[i].x, v[i].y), fmaxf(v[i].z, v[i].w)));
        mx = block_max(mx, red);
        float se = 0.f, tl = 0.f;                          // sum of exponentials; the target's logit (one thread has it)
#pragma unroll
        for (int i = 0; i < CE_V4_PER_THREAD; ++i) {
            const int e0 = (i * CE_THREADS + t) * 4;
            if (tgt >= e0 && tgt < e0 + 4) tl = tgt == e0 ? v[i].x : tgt == e0 + 1 ? v[i].y : tgt == e0 + 2 ? v[i].z : v[i].w;
            v[i].x = expf(v[i].x - mx); v[i].y = expf(v[i].y - mx); v[i].z = expf(v[i].z - mx); v[i].w = expf(v[i].w - mx);
            se += (v[i].x + v[i].y) + (v[i].z + v[i].w);
        }
        se = block_sum(se, red);
        tl = block_sum(tl, red);                           // every other thread contributes 0
        if (t == 0) loss_row[m] = mx + logf(se) - tl;
        if (dlog16) {
            const float inv = 1.f / se, invM = 1.f / (float)M;
            bf16* out = dlog16 + (long long)m * V;
#pragma unroll
            for (int i = 0; i < CE_V4_PER_THREAD; ++i) {
                const int e = i * CE_THREADS + t, e0 = e * 4;
                if (e < n4) {
                    const float g0 = (v[i].x * inv - (tgt == e0 ? 1.f : 0.f)) * invM, g1 = (v[i].y * inv - (tgt == e0 + 1 ? 1.f : 0.f)) * invM;
                    const float g2 = (v[i].z * inv - (tgt == e0 + 2 ? 1.f : 0.f)) * invM, g3 = (v[i].w * inv - (tgt == e0 + 3 ? 1.f : 0.f)) * invM;
                    __nv_bfloat162 lo = __floats2bfloat162_rn(g0, g1), hi = __floats2bfloat162_rn(g2, g3);
                    uint2 pk;
                    pk.x = *reinterpret_cast<unsigned*>(&lo);
                    pk.y = *reinterpret_cast<unsigned*>(&hi);
                    *reinterpret_cast<uint2*>(out + e0) = pk;
                }
            }
        }
    }
    __syncthreads();
    drain_after_abort(abort_flag);
}

inline bool lm_ce_stream_supported(int V, int max_smem) {
    return V % 4 == 0 && V <= CE_MAX_V && (size_t)V * 4 + 1024 <= (size_t)max_smem;
}

// rows [M][V] fp32 -> loss_row [M], dlog16 [M][V] (may be null: loss only)
inline cudaError_t lm_ce_stream_launch(cudaStream_t stream, int sms, const float* logits, const int* ids, long long N,
                                       const int* targets, int S, int V, int M, float* loss_row, bf16* dlog16, unsigned* status) {
    const size_t smem = (size_t)V * 4;
    {
        cudaError_t e = smem_opt_in((const void*)lm_ce_stream_kernel, smem);
        if (e != cudaSuccess) return e;
    }
    const int grid = M < sms ? M : sms;
    lm_ce_stream_kernel<<<grid, CE_THREADS, smem, stream>>>(logits, ids, N, targets, S, V, M, loss_row, dlog16, status);
    return cudaGetLastError();
}

// fp32 -> bf16 copies of GEMM operands (a_L, W_up), 4 elements per thread (n a multiple of 4).  W_up sits
// behind lambda[L] in the flat parameter vector, so its address is 16-byte aligned only when L % 4 == 0:
// src_vec says whether the source may be read as float4.
__global__ void to_bf16_kernel(const float* __restrict__ x, long long n, bf16* __restrict__ out, int src_vec) {
    const long long i = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i >= n) return;
    const float4 v = src_vec ? *reinterpret_cast<const float4*>(x + i) : make_float4(x[i], x[i + 1], x[i + 2], x[i + 3]);
    __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
    uint2 pk;
    pk.x = *reinterpret_cast<unsigned*>(&lo);
    pk.y = *reinterpret_cast<unsigned*>(&hi);
    *reinterpret_cast<uint2*>(out + i) = pk;
}

// Host side: tensor maps and launch for one GEMM shape.
struct GemmPlan {
    bool ready = false;
    CUtensorMap map_a, map_b;
    CUtensorMap map_b_pair;        // K-major B in boxes of 128 rows, for CTA pairs (MN-major B: the same boxes as map_b)
    bool pair = false;             // run as 2-CTA clusters on 256 x 256 tiles
    int b_mn_major = 0, N = 0, K = 0, sms = 0;
};

// A: [rows_a][K] bf16 row-major.  B: K-major [N][K], or MN-major [K][N].
inline pac_status gemm_plan_create(GemmPlan& gp, int device, const bf16* A, long long rows_a, const bf16* B, int N, int K,
                                   int b_mn_major, bool pair = true) {
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
        gp.map_b_pair = gp.map_b;
    } else {
        cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)N};
        cuuint64_t str[1] = {(cuuint64_t)K * 2};
        cuuint32_t box[2] = {GT_BK, GT_BN}, box_pair[2] = {GT_BK, GT_BN / 2};
        if (!make_map(&gp.map_b, B, 2, dims, str, box)) return PAC_ERR_UNSUPPORTED;
        if (!make_map(&gp.map_b_pair, B, 2, dims, str, box_pair)) return PAC_ERR_UNSUPPORTED;
    }
    gp.pair = pair && gp.sms >= 2;
    if (smem_opt_in((const void*)gemm_tc_kernel<false>, GT_SMEM) != cudaSuccess ||
        smem_opt_in((const void*)gemm_tc_kernel<true>, GT_SMEM_PAIR) != cudaSuccess) {
        tensor_err() = "cudaFuncSetAttribute(MaxDynamicSharedMemorySize) failed";
        cudaGetLastError();
        return PAC_ERR_CUDA;
    }
    gp.b_mn_major = b_mn_major; gp.N = N; gp.K = K;
    gp.ready = true;
    return PAC_OK;
}

// Optional extras of a launch: a bf16 copy of the output and / or the residual rows of the last cached layer.
struct GemmExtras {
    bf16* C16 = nullptr; long long ldc16 = 0;
    const bf16* add_cache = nullptr; const int* ids = nullptr; long long n_cache = 0; int L = 0, S = 0;
};

inline pac_status gemm_launch(const GemmPlan& gp, cudaStream_t stream, int M, float* C, long long ldc, unsigned* status,
                              long long* launches, const GemmExtras* ex = nullptr) {
    GemmParams p{};
    if (ex) {
        p.C16 = ex->C16; p.ldc16 = ex->ldc16;
        p.add_cache = ex->add_cache; p.ids = ex->ids; p.n_cache = ex->n_cache; p.L = ex->L; p.S = ex->S;
    }
    p.M = M; p.N = gp.N; p.K = gp.K;
    p.m_tiles = (M + GT_BM - 1) / GT_BM;
    p.n_tiles = (gp.N + GT_BN - 1) / GT_BN;
    p.k_chunks = (gp.K + GT_BK - 1) / GT_BK;
    p.b_mn_major = gp.b_mn_major;
    p.C = C; p.ldc = ldc; p.status = status;
    cudaError_t e;
    if (gp.pair) {
        const int units = ((p.m_tiles + 1) / 2) * p.n_tiles, clusters = units < gp.sms / 2 ? units : gp.sms / 2;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(2 * clusters), 1, 1);
        cfg.blockDim = dim3(TC_THREADS, 1, 1);
        cfg.dynamicSmemBytes = GT_SMEM_PAIR;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, gemm_tc_kernel<true>, gp.map_a, gp.map_b_pair, p);
    } else {
        const int tiles = p.m_tiles * p.n_tiles;
        const int grid = tiles < gp.sms ? tiles : gp.sms;
        gemm_tc_kernel<false><<<grid, TC_THREADS, GT_SMEM, stream>>>(gp.map_a, gp.map_b, p);
        e = cudaGetLastError();
    }
    (*launches)++;
    if (e != cudaSuccess) { tensor_err() = cudaGetErrorString(e); return PAC_ERR_CUDA; }
    return PAC_OK;
}

}  // namespace pac
