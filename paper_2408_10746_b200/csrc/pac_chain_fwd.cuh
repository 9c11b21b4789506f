// Down-projections with the forward chain in the epilogue, for sequences of 128 tokens or more
// (classifier head).  One CTA owns a tile of 128 tokens of one sample and walks ALL layers:
//     u_l = h_l W_down^l  (TMA -> tcgen05.mma, hi | lo weights side by side along N, accumulators
//                          double-buffered in TMEM)
//     z_l = lambda_l u_l + (1 - lambda_l) a_{l-1},   a_l = phi(z_l)        (Section IV-A)
// The epilogue warps own one token row each and keep a_{l-1} in registers from layer to layer, so
// while the tensor cores work on layer l+1 they finish layer l: u never reaches memory.  What the
// reverse pass needs is left behind in compact form: u_l - a_{l-1} (= d z_l / d lambda_l) as bf16 in
// the slot of the du buffer that du_l will overwrite later, the ReLU gates of all layers as one
// 32-bit word per element, and the token sums of a_L per 32-token group for the pooled head.
#pragma once
#include "pac_simt.cuh"
#include "pac_tensor.cuh"

namespace pac {

constexpr int CF_EPI_WARPS = 8;                      // two per TMEM lane quadrant, each takes half of the adapter columns
constexpr int CF_THREADS = 64 + 32 * CF_EPI_WARPS;   // warp 0: TMA producer, warp 1: MMA issuer, then the epilogue warps
constexpr int CF_POOL_PARTS = 4;                     // 32-token groups per tile

struct ChainFwdParams {
    const int* ids; long long N;
    int L, S, d, r, B;
    int s_chunks, k_chunks, stages;
    int train;                             // 0: evaluation, nothing but the token sums is written
    const float* lam;                      // [L]
    bf16* parked; long long layer_stride;  // [L][max_rows][r]: u_l - a_{l-1} in bf16 (the du buffer's slots)
    unsigned* gates;                       // [max_rows][r]: bit l set = the ReLU of layer l let the element through
    float* pool_part;                      // [B][s_chunks * CF_POOL_PARTS][r]: token sums of a_L per 32-token group
    unsigned* status;
    unsigned long long* stamp;
};

// The epilogue of one warp (see the kernel below).  acce0: "accumulator drained" barriers, in this CTA, or - acce_remote -
// an address in the cluster's shared-memory window (the barriers of the CTA that issues the pair's MMAs).
template <int ACT, int CH>
__device__ __forceinline__ void chain_epilogue(const ChainFwdParams& p, const float* lam_s, uint32_t tmem_base, uint32_t acc_stride,
                                               uint32_t accf0, uint32_t acce0, bool acce_remote, volatile int* abort_flag,
                                               int warp, int lane, int sc, int b) {
    // ---- epilogue: one token row per thread, CH chunks of 16 adapter columns; a_{l-1} and the gate words
    // stay in registers across the layers ----
    const int ew = warp - 2, quad = warp & 3, half = ew >> 2;
    const int srow = sc * FWD_ROWS + quad * 32 + lane;             // token inside the sample
    const bool row_ok = srow < p.S;
    const long long m = (long long)b * p.S + srow;
    const int col_base = half * (CH * 16);
    float a[CH][16];
    unsigned gate[CH][16];
#pragma unroll
    for (int c = 0; c < CH; ++c)
#pragma unroll
        for (int e = 0; e < 16; ++e) { a[c][e] = 0.f; gate[c][e] = 0u; }     // a_0 = 0
    bool ok = true;
    for (int l = 0; l < p.L; ++l) {
        const int buf = l & 1;
        const uint32_t aph = (uint32_t)(l >> 1) & 1u;
        if (!mbar_wait_warp(accf0 + 8 * buf, aph, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        if (threadIdx.x == 64 && l == p.L - 1) stamp_end(p.stamp);
        const float lm = lam_s[l], om = 1.f - lm;
        const uint32_t trow = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)buf * acc_stride;
        bf16* pk = p.parked + (long long)l * p.layer_stride + m * p.r;
#pragma unroll
        for (int c = 0; c < CH; ++c) {
            const int c0 = col_base + c * 16;
            // column c0 of u: hi part at TMEM column (c0/64)*128 + c0%64, lo part 64 columns further
            const uint32_t col = (uint32_t)((c0 >> 6) * 128 + (c0 & 63));
            float v[16], w[16];
            tmem_ld16(trow + col, v);
            tmem_ld16(trow + col + 64, w);
            tmem_ld_wait();
            __align__(16) bf16 park[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                const float u = v[e] + w[e];
                const float z = lm * u + om * a[c][e];
                park[e] = __float2bfloat16(u - a[c][e]);           // d z_l / d lambda_l
                if (ACT == PAC_ACT_RELU) {
                    const bool on = z > 0.f;
                    gate[c][e] |= (on ? 1u : 0u) << l;
                    a[c][e] = on ? z : 0.f;
                } else {
                    a[c][e] = z;
                }
            }
            if (p.train && row_ok)          // 16 bf16 = one whole 32-byte sector
                st_global_32(pk + c0, *reinterpret_cast<const uint4*>(park), *reinterpret_cast<const uint4*>(park + 8));
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
            if (acce_remote) mbar_arrive_cluster(acce0 + 8 * buf); else mbar_arrive(acce0 + 8 * buf);
        }
    }
    if (ok) {
        // the gates of all layers, one word per element
        if (p.train && row_ok && ACT == PAC_ACT_RELU) {
            unsigned* g = p.gates + m * p.r;
#pragma unroll
            for (int c = 0; c < CH; ++c)
#pragma unroll
                for (int e = 0; e < 16; e += 8)
                    st_global_32(g + col_base + c * 16 + e, make_uint4(gate[c][e], gate[c][e + 1], gate[c][e + 2], gate[c][e + 3]),
                                 make_uint4(gate[c][e + 4], gate[c][e + 5], gate[c][e + 6], gate[c][e + 7]));
        }
        // token sums of a_L over this warp's 32 rows (fixed shuffle order); lane e of chunk c keeps column e
        float* pp = p.pool_part + ((long long)b * (p.s_chunks * CF_POOL_PARTS) + sc * CF_POOL_PARTS + quad) * p.r;
#pragma unroll
        for (int c = 0; c < CH; ++c)
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                const float tot = warp_sum(row_ok ? a[c][e] : 0.f);
                if (lane == e) pp[col_base + c * 16 + e] = tot;
            }
    }
}

// CH: 16-column chunks per epilogue warp (r = 32 * CH).
template <int ACT, int CH>
__global__ void __launch_bounds__(CF_THREADS, 1)
down_chain_tc_kernel(const __grid_constant__ CUtensorMap map_cache, const __grid_constant__ CUtensorMap map_w, ChainFwdParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int r_blocks = (p.r + 63) >> 6;
    const uint32_t a_bytes = FWD_ROWS * KC * 2, b_box = KC * 128;
    const uint32_t b_bytes = (uint32_t)r_blocks * 2 * b_box, b_off = a_bytes, stage_bytes = a_bytes + b_bytes;
    const uint32_t acc_stride = 256u;                      // TMEM columns per accumulator (r <= 128: at most 2 x 128)
    __shared__ __align__(8) unsigned long long bars[2 * 16 + 4];
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;
    __shared__ float lam_s[32];
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[16]);
    const uint32_t accf0 = smem_u32(&bars[32]), acce0 = smem_u32(&bars[34]);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sc = blockIdx.x % p.s_chunks, b = blockIdx.x / p.s_chunks;      // this CTA's tile: sample b, token chunk sc

    if (threadIdx.x == 0) {
        abort_sh = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(accf0 + 8 * i, 1); mbar_init(acce0 + 8 * i, CF_EPI_WARPS); }
        fence_mbar_init();
        tma_prefetch_desc(&map_cache);
        tma_prefetch_desc(&map_w);
    }
    if (warp == 1) { tmem_alloc(smem_u32(&tmem_base_sh), 512u); tmem_relinquish(); }
    pdl_trigger();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_sh;
    volatile int* abort_flag = &abort_sh;
    pdl_wait();            // the weights (updated by the predecessor) and device ids are final from here on
    if (warp >= 2) {
        // lambda of every layer for the epilogue warps (a barrier of their own: the pipeline warps never join it)
        if (warp == 2) lam_s[lane] = lane < p.L ? p.lam[lane] : 0.f;
        asm volatile("bar.sync 1, %0;" ::"r"(32 * CF_EPI_WARPS) : "memory");
    }
    const int id = (int)safe_id(p.ids, b, p.N, (threadIdx.x == 0 && sc == 0) ? p.status : nullptr);

    // Both pipeline loops carry ring positions, parities, addresses and descriptors from step to step: their own
    // instruction streams are on the critical path of a K step.
    if (warp == 0) {
        const uint64_t pol = l2_policy_evict_first();
        uint32_t s = 0, eph = 1;                                   // eph: parity of the "stage free" phase to wait for
        const uint32_t ring0 = smem_u32(smem);
        uint32_t dst = ring0;
        bool ok = true;
        if (lane == 0) stamp_begin(p.stamp);
        for (int l = 0; l < p.L && ok; ++l) {
            for (int kc = 0; kc < p.k_chunks; ++kc) {
                if (!mbar_wait_uniform(empty0 + 8 * s, eph, abort_flag, p.status)) { ok = false; break; }
                if (elect_one()) {
                    const uint32_t full = full0 + 8 * s;
                    mbar_expect_tx(full, stage_bytes);
                    tma_load_4d_hint(dst, &map_cache, full, kc * KC, sc * FWD_ROWS, l, id, pol);
                    for (int rb = 0; rb < r_blocks; ++rb)
                        tma_load_4d(dst + b_off + rb * 2 * b_box, &map_w, full, rb * 64, kc * KC, 0, l);
                }
                __syncwarp();
                dst += stage_bytes;
                if (++s == (uint32_t)p.stages) { s = 0; eph ^= 1u; dst = ring0; }
            }
        }
    } else if (warp == 1) {
        // hi and lo blocks lie side by side along N ([r block][hi|lo], 64 columns each): one MMA of
        // N = 128 * r_blocks per K step leaves u_hi | u_lo next to each other in TMEM
        const uint32_t idesc = instr_desc_bf16(FWD_ROWS, 128 * r_blocks, 0, 1);
        // descriptors hold addresses in units of 16 bytes
        const uint64_t a_desc0 = smem_desc_sw128(smem_u32(smem), 16, 1024), w_desc0 = smem_desc_sw128(smem_u32(smem) + b_off, b_box, 1024);
        const uint64_t desc_step = (uint64_t)(stage_bytes >> 4);
        uint64_t ad0 = a_desc0, bw0 = w_desc0;
        uint32_t s = 0, ph = 0;
        bool ok = true;
        for (int l = 0; l < p.L && ok; ++l) {
            const int buf = l & 1;
            const uint32_t aph = (uint32_t)(l >> 1) & 1u;
            if (!mbar_wait_uniform(acce0 + 8 * buf, aph ^ 1, abort_flag, p.status)) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)buf * acc_stride;
            for (int kc = 0; kc < p.k_chunks; ++kc) {
                if (!mbar_wait_uniform(full0 + 8 * s, ph, abort_flag, p.status)) { ok = false; break; }
                tc_fence_after();
                if (elect_one()) {
#pragma unroll
                    for (int k = 0; k < KC / 16; ++k)
                        umma_bf16(d_tmem, ad0 + (uint64_t)(k * 2), bw0 + (uint64_t)(k * 128), idesc, (kc | k) ? 1u : 0u);
                    umma_commit(empty0 + 8 * s);
                }
                __syncwarp();
                ad0 += desc_step; bw0 += desc_step;
                if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1u; ad0 = a_desc0; bw0 = w_desc0; }
            }
            if (!ok) break;
            if (elect_one()) umma_commit(accf0 + 8 * buf);
            __syncwarp();
        }
    } else {
        chain_epilogue<ACT, CH>(p, lam_s, tmem_base, acc_stride, accf0, acce0, false, abort_flag, warp, lane, sc, b);
    }
    tc_fence_before();
    __syncthreads();
    drain_after_abort(abort_flag);
    if (warp == 1) tmem_dealloc(tmem_base, 512u);
}

// The same with CTA pairs (r > 64, an even number of tiles): a 2-CTA cluster takes two tiles and runs one MMA of
// M = 256, N = 256 per K step; each CTA loads its own cache tile and one of the two 128-column weight blocks
// ([hi | lo] of 64 adapter columns), half the weight bytes per CTA, which is what the kernel is short of: per
// SM it takes in L2 data at close to the 64 bytes per clock an SM can.  The CTA of rank 0 waits for the
// bytes of both (one barrier, counted from both sides), issues the MMAs and frees the stages and
// accumulators of both with multicast commits; the epilogue warps of both arrive at its "drained" barrier.
template <int ACT, int CH>
__global__ void __launch_bounds__(CF_THREADS, 1)
down_chain_pair_kernel(const __grid_constant__ CUtensorMap map_cache, const __grid_constant__ CUtensorMap map_w, ChainFwdParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const uint32_t rank = cluster.block_rank();              // 0: issues the MMAs
    const uint32_t a_bytes = FWD_ROWS * KC * 2, b_box = KC * 128;
    const uint32_t b_bytes = 2 * b_box, stage_bytes = a_bytes + b_bytes;      // own cache tile + ONE [hi | lo] weight block
    const uint32_t acc_stride = 256u;
    __shared__ __align__(8) unsigned long long bars[2 * 16 + 4];
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;
    __shared__ float lam_s[32];
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[16]);
    const uint32_t accf0 = smem_u32(&bars[32]), acce0 = smem_u32(&bars[34]);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sc = blockIdx.x % p.s_chunks, b = blockIdx.x / p.s_chunks;

    if (threadIdx.x == 0) {
        abort_sh = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(accf0 + 8 * i, 1); mbar_init(acce0 + 8 * i, 2 * CF_EPI_WARPS); }
        fence_mbar_init();
        tma_prefetch_desc(&map_cache);
        tma_prefetch_desc(&map_w);
    }
    if (warp == 1) { tmem_alloc_pair(smem_u32(&tmem_base_sh), 512u); tmem_relinquish_pair(); }
    pdl_trigger();
    tc_fence_before();
    __syncthreads();
    cluster.sync();                        // the peer's barriers exist before anything arrives at them
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_sh;
    volatile int* abort_flag = &abort_sh;
    pdl_wait();
    if (warp >= 2) {
        if (warp == 2) lam_s[lane] = lane < p.L ? p.lam[lane] : 0.f;
        asm volatile("bar.sync 1, %0;" ::"r"(32 * CF_EPI_WARPS) : "memory");
    }
    const int id = (int)safe_id(p.ids, b, p.N, (threadIdx.x == 0 && sc == 0) ? p.status : nullptr);

    if (warp == 0) {
        // both CTAs: own cache tile and weight block `rank`, counted on the barrier of CTA 0
        const uint64_t pol = l2_policy_evict_first();
        uint32_t s = 0, eph = 1;
        const uint32_t ring0 = smem_u32(smem);
        uint32_t dst = ring0;
        bool ok = true;
        if (lane == 0) stamp_begin(p.stamp);
        for (int l = 0; l < p.L && ok; ++l) {
            for (int kc = 0; kc < p.k_chunks; ++kc) {
                if (!mbar_wait_uniform(empty0 + 8 * s, eph, abort_flag, p.status)) { ok = false; break; }
                if (elect_one()) {
                    const uint32_t full = mapa_shared(full0 + 8 * s, 0u);
                    if (rank == 0) mbar_expect_tx(full0 + 8 * s, 2 * stage_bytes);
                    tma_load_4d_pair_hint(dst, &map_cache, full, kc * KC, sc * FWD_ROWS, l, id, pol);
                    tma_load_4d_pair(dst + a_bytes, &map_w, full, (int)rank * 64, kc * KC, 0, l);
                }
                __syncwarp();
                dst += stage_bytes;
                if (++s == (uint32_t)p.stages) { s = 0; eph ^= 1u; dst = ring0; }
            }
        }
    } else if (warp == 1) {
        if (rank == 0) {
            const uint32_t idesc = instr_desc_bf16(2 * FWD_ROWS, 256, 0, 1);
            const uint64_t a_desc0 = smem_desc_sw128(smem_u32(smem), 16, 1024), w_desc0 = smem_desc_sw128(smem_u32(smem) + a_bytes, b_box, 1024);
            const uint64_t desc_step = (uint64_t)(stage_bytes >> 4);
            uint64_t ad0 = a_desc0, bw0 = w_desc0;
            uint32_t s = 0, ph = 0;
            bool ok = true;
            for (int l = 0; l < p.L && ok; ++l) {
                const int buf = l & 1;
                const uint32_t aph = (uint32_t)(l >> 1) & 1u;
                if (!mbar_wait_uniform(acce0 + 8 * buf, aph ^ 1, abort_flag, p.status)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)buf * acc_stride;
                for (int kc = 0; kc < p.k_chunks; ++kc) {
                    if (!mbar_wait_uniform(full0 + 8 * s, ph, abort_flag, p.status)) { ok = false; break; }
                    tc_fence_after();
                    if (elect_one()) {
#pragma unroll
                        for (int k = 0; k < KC / 16; ++k)
                            umma_bf16_pair(d_tmem, ad0 + (uint64_t)(k * 2), bw0 + (uint64_t)(k * 128), idesc, (kc | k) ? 1u : 0u);
                        umma_commit_pair(empty0 + 8 * s, (uint16_t)3);
                    }
                    __syncwarp();
                    ad0 += desc_step; bw0 += desc_step;
                    if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1u; ad0 = a_desc0; bw0 = w_desc0; }
                }
                if (!ok) break;
                if (elect_one()) umma_commit_pair(accf0 + 8 * buf, (uint16_t)3);
                __syncwarp();
            }
        }
    } else {
        chain_epilogue<ACT, CH>(p, lam_s, tmem_base, acc_stride, accf0, mapa_shared(acce0, 0u), true, abort_flag, warp, lane, sc, b);
    }
    tc_fence_before();
    __syncthreads();
    drain_after_abort(abort_flag);
    cluster.sync();                        // neither CTA frees TMEM or leaves while the pair's MMAs or arrivals may still touch it
    if (warp == 1) tmem_dealloc_pair(tmem_base, 512u);
}

// Shapes the kernel takes: r a multiple of 32 up to 128 (hi | lo fit one MMA and the epilogue's register
// budget), any S (tiles of 128 tokens), at most 32 layers (gate bits).
inline bool chain_fwd_supported(const Dims& dm) { return dm.r % 32 == 0 && dm.r >= 32 && dm.r <= 128 && dm.L <= 32 && dm.d % 8 == 0 && dm.d >= 64; }

template <int ACT>
inline cudaError_t chain_fwd_launch_act(const CUtensorMap& map_cache, const CUtensorMap& map_w, const ChainFwdParams& p, size_t smem,
                                        cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    pdl_launch_config(&cfg, attr, dim3((unsigned)(p.B * p.s_chunks)), dim3(CF_THREADS), smem, stream);
    cudaError_t e;
    switch (p.r / 32) {
        case 1: if ((e = smem_opt_in((const void*)down_chain_tc_kernel<ACT, 1>, smem)) != cudaSuccess) return e;
                return cudaLaunchKernelEx(&cfg, down_chain_tc_kernel<ACT, 1>, map_cache, map_w, p);
        case 2: if ((e = smem_opt_in((const void*)down_chain_tc_kernel<ACT, 2>, smem)) != cudaSuccess) return e;
                return cudaLaunchKernelEx(&cfg, down_chain_tc_kernel<ACT, 2>, map_cache, map_w, p);
        case 3: if ((e = smem_opt_in((const void*)down_chain_tc_kernel<ACT, 3>, smem)) != cudaSuccess) return e;
                return cudaLaunchKernelEx(&cfg, down_chain_tc_kernel<ACT, 3>, map_cache, map_w, p);
        default: if ((e = smem_opt_in((const void*)down_chain_tc_kernel<ACT, 4>, smem)) != cudaSuccess) return e;
                 return cudaLaunchKernelEx(&cfg, down_chain_tc_kernel<ACT, 4>, map_cache, map_w, p);
    }
}

// CTA pairs: shapes, stage count and launch.
inline bool chain_pair_supported(const Dims& dm) { return chain_fwd_supported(dm) && dm.r > 64; }
inline int chain_pair_stages(int max_smem) {
    int st = (max_smem - 2048) / (FWD_ROWS * KC * 2 + 2 * KC * 128);
    return st > 16 ? 16 : st;
}
inline size_t chain_pair_smem(int stages) { return (size_t)stages * (FWD_ROWS * KC * 2 + 2 * KC * 128) + 1024; }

template <int ACT, int CH>
inline cudaError_t chain_pair_launch_one(const CUtensorMap& map_cache, const CUtensorMap& map_w, const ChainFwdParams& p, size_t smem,
                                         cudaStream_t stream) {
    cudaError_t e = smem_opt_in((const void*)down_chain_pair_kernel<ACT, CH>, smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.B * p.s_chunks), 1, 1);
    cfg.blockDim = dim3(CF_THREADS, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, down_chain_pair_kernel<ACT, CH>, map_cache, map_w, p);
}
// p.stages: stages of the pair kernel's ring; the grid (B * s_chunks) must be even.
inline cudaError_t chain_pair_launch(const CUtensorMap& map_cache, const CUtensorMap& map_w, const ChainFwdParams& p, size_t smem, int act,
                                     cudaStream_t stream) {
    const bool relu = act == PAC_ACT_RELU;
    if (p.r / 32 == 3)
        return relu ? chain_pair_launch_one<PAC_ACT_RELU, 3>(map_cache, map_w, p, smem, stream)
                    : chain_pair_launch_one<PAC_ACT_IDENTITY, 3>(map_cache, map_w, p, smem, stream);
    return relu ? chain_pair_launch_one<PAC_ACT_RELU, 4>(map_cache, map_w, p, smem, stream)
                : chain_pair_launch_one<PAC_ACT_IDENTITY, 4>(map_cache, map_w, p, smem, stream);
}

inline cudaError_t chain_fwd_launch(const CUtensorMap& map_cache, const CUtensorMap& map_w, const ChainFwdParams& p, size_t smem, int act,
                                    cudaStream_t stream) {
    return act == PAC_ACT_RELU ? chain_fwd_launch_act<PAC_ACT_RELU>(map_cache, map_w, p, smem, stream)
                               : chain_fwd_launch_act<PAC_ACT_IDENTITY>(map_cache, map_w, p, smem, stream);
}

}  // namespace pac
