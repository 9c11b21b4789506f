// One-launch forward for short sequences (S <= 128, r <= 64, classifier head): one thread-block
// cluster per batch sample does
//   1. the down-projections u_l = h_l W_down^l (Section IV-A) of the sample's 128-token tile, the
//      L layers split over the cluster's CTAs (each CTA: TMA-fed tcgen05 MMAs into one TMEM
//      accumulator per layer; the weights enter as bf16 hi + lo, side by side along N when at most
//      four layers fall to a CTA, else as two products summed in the same accumulator); meanwhile the
//      other warps fetch the head operands, form the head's product matrix (mid_head_products) and
//      then drain every accumulator to the u buffer in global memory AS SOON AS ITS LAYER IS COMPLETE,
//      while the later layers still stream: when the last cache tile has arrived only the last
//      layer's rows are still to be written,
//   2. one cluster barrier, behind which every CTA fetches the u rows of the tokens it owns (all
//      layers, written by its peers a moment ago and still in L2) into its shared memory,
//   3. everything the stand-alone fused kernel does afterwards (mid_body): merge/activation chain,
//      pooling, head, loss, reverse chain -> du_l and dlambda partials.
#pragma once
#include "pac_mid.cuh"
#include "pac_tensor.cuh"

namespace pac {

struct FusedFwdParams {
    MidParams mid;             // G, Sg, dg, layers_per_cta, head operands, u buffer, outputs
    int k_chunks;              // ceil(d / 64)
    int stages;                // pipeline depth of the GEMM phase
    int wide_n;                // 1: hi | lo side by side (N = 128, 128 TMEM columns per layer); 0: two N = 64 products per K step
    size_t mid_offset;         // byte offset of the head vectors behind the stage / chain-state region
    unsigned long long* stamp; // optional stream-phase timestamps (see stamp_begin)
};

constexpr int FUSED_N = 128;        // MMA N with hi and lo side by side: 64 hi columns | 64 lo columns
constexpr int FUSED_MAX_LPC = 8;    // layers per CTA: 8 x 64 TMEM columns (two products per K step), or 4 x 128
constexpr int FUSED_DRAIN_WARP0 = 4;   // warps 4 .. 15 drain accumulators; warp & 3 is the TMEM lane quadrant a warp may read

template <int ACT>
__global__ void __launch_bounds__(512, 1)
fwd_cluster_kernel(const __grid_constant__ CUtensorMap map_cache, const __grid_constant__ CUtensorMap map_w, FusedFwdParams fp) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    cg::cluster_group cluster = cg::this_cluster();
    const MidParams& p = fp.mid;
    const int q = (int)cluster.block_rank();
    const int b = blockIdx.x / p.G;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    const uint32_t a_bytes = FWD_ROWS * KC * 2, b_bytes = 2 * KC * 128, stage_bytes = a_bytes + b_bytes;
    const MidShared h = mid_carve(reinterpret_cast<float*>(smem + fp.mid_offset), p);
    __shared__ __align__(8) unsigned long long bars[2 * 16 + FUSED_MAX_LPC];
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;
    __shared__ long long id_sh;
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[16]), accf0 = smem_u32(&bars[32]);
    const int l_begin = q * p.layers_per_cta, l_end = min(p.L, l_begin + p.layers_per_cta);
    const int n_layers = max(0, l_end - l_begin);
    const uint32_t acc_cols = fp.wide_n ? (uint32_t)FUSED_N : 64u;            // TMEM columns per layer

    if (threadIdx.x == 0) {
        abort_sh = 0;
        for (int s = 0; s < fp.stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int li = 0; li < FUSED_MAX_LPC; ++li) mbar_init(accf0 + 8 * li, 1);
        fence_mbar_init();
        tma_prefetch_desc(&map_cache);
        tma_prefetch_desc(&map_w);
    }
    if (warp == 1) { tmem_alloc(smem_u32(&tmem_base_sh), 512u); tmem_relinquish(); }
    pdl_trigger();
    // Ids that were final before this launch (written by the host, or device ids no kernel ahead of this one
    // touches) are read while the predecessor still drains, and so are the first cache tiles: the cache never
    // changes, only the weights (updated by the predecessor) have to wait.  One thread fetches the id for the
    // whole CTA: with ids in host memory every reading warp would be a transaction on the host link.
    const bool early = p.host_ids || p.early_ids;
    if (early && threadIdx.x == 64) {
        const bool pref = p.host_ids && p.pref_tag && ld_acquire_gpu(p.pref_tag) == p.pref_seq;
        id_sh = safe_id(pref ? p.pref_ids : p.ids, b, p.N, q == 0 ? p.status : nullptr);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_sh;
    volatile int* abort_flag = &abort_sh;
    long long id = early ? id_sh : -1;
    const uint64_t pol = l2_policy_evict_first();
    uint32_t pre = 0;                                            // stages whose cache tile is already on its way
    if (early && warp == 0 && n_layers > 0) {
        pre = (uint32_t)min(n_layers * fp.k_chunks, fp.stages);
        if (elect_one()) {
            for (uint32_t s = 0; s < pre; ++s) {
                mbar_expect_tx(full0 + 8 * s, stage_bytes);
                tma_load_4d_hint(smem_u32(smem + (size_t)s * stage_bytes), &map_cache, full0 + 8 * s,
                                 (int)(s % fp.k_chunks) * KC, 0, l_begin + (int)(s / fp.k_chunks), (int)id, pol);
            }
        }
        __syncwarp();
    }
    pdl_wait();                 // weights, parameters and (device) ids of this step are final from here on
    if (!early) id = safe_id(p.ids, b, p.N, (threadIdx.x == 0 && q == 0) ? p.status : nullptr);
    if (p.ids_copy && q == 0 && threadIdx.x == 0) p.ids_copy[b] = (int)id;

    // ---- phase 1: the GEMMs of this CTA's layers; the other warps fetch the head operands, then drain
    // finished accumulators.  Both pipeline loops are run by a whole converged warp, one elected lane issues. ----
    if (warp == 0) {
        uint32_t it = 0;
        bool ok = true;
        if (lane == 0 && n_layers > 0) stamp_begin(fp.stamp);      // first copy after the predecessor has finished
        for (int l = l_begin; l < l_end && ok; ++l) {
            for (int kc = 0; kc < fp.k_chunks; ++kc, ++it) {
                const int s = it % fp.stages;
                const uint32_t dst = smem_u32(smem + (size_t)s * stage_bytes);
                if (it < pre) {
                    // first round: the cache tile was requested before the wait above, the weight tile follows
                    if (elect_one()) tma_load_4d(dst + a_bytes, &map_w, full0 + 8 * s, 0, kc * KC, 0, l);
                    __syncwarp();
                    continue;
                }
                const uint32_t ph = (it / fp.stages) & 1;
                if (!mbar_wait_uniform(empty0 + 8 * s, ph ^ 1, abort_flag, p.status)) { ok = false; break; }
                if (elect_one()) {
                    mbar_expect_tx(full0 + 8 * s, stage_bytes);
                    tma_load_4d_hint(dst, &map_cache, full0 + 8 * s, kc * KC, 0, l, (int)id, pol);
                    tma_load_4d(dst + a_bytes, &map_w, full0 + 8 * s, 0, kc * KC, 0, l);
                }
                __syncwarp();
            }
        }
    } else if (warp == 1) {
        const uint32_t idesc = fp.wide_n ? instr_desc_bf16(FWD_ROWS, FUSED_N, 0, 1) : instr_desc_bf16(FWD_ROWS, 64, 0, 1);
        uint32_t it = 0;
        bool ok = true;
        for (int l = l_begin; l < l_end && ok; ++l) {
            const uint32_t d_tmem = tmem_base + (uint32_t)(l - l_begin) * acc_cols;
            for (int kc = 0; kc < fp.k_chunks; ++kc, ++it) {
                const int s = it % fp.stages;
                const uint32_t ph = (it / fp.stages) & 1;
                if (!mbar_wait_uniform(full0 + 8 * s, ph, abort_flag, p.status)) { ok = false; break; }
                tc_fence_after();
                const uint32_t a0 = smem_u32(smem + (size_t)s * stage_bytes), b0 = a0 + a_bytes;
                const uint64_t ad0 = smem_desc_sw128(a0, 16, 1024), bw0 = smem_desc_sw128(b0, KC * 128, 1024);
                if (elect_one()) {
                    if (fp.wide_n) {
#pragma unroll
                        for (int k = 0; k < KC / 16; ++k)
                            umma_bf16(d_tmem, ad0 + (uint64_t)(k * 2), bw0 + (uint64_t)(k * 128), idesc, (kc | k) ? 1u : 0u);
                    } else {
                        // the lo block lies KC * 128 bytes behind the hi block of the same stage
                        const uint64_t bl0 = smem_desc_sw128(b0 + KC * 128, KC * 128, 1024);
#pragma unroll
                        for (int k = 0; k < KC / 16; ++k) {
                            umma_bf16(d_tmem, ad0 + (uint64_t)(k * 2), bw0 + (uint64_t)(k * 128), idesc, (kc | k) ? 1u : 0u);
                            umma_bf16(d_tmem, ad0 + (uint64_t)(k * 2), bl0 + (uint64_t)(k * 128), idesc, 1u);
                        }
                    }
                    umma_commit(empty0 + 8 * s);
                }
                __syncwarp();
            }
            if (ok) {
                if (elect_one()) umma_commit(accf0 + 8 * (l - l_begin));      // this layer's accumulator is complete
                __syncwarp();
            }
        }
        if (ok && n_layers > 0) {
            // the last accumulator complete = every load consumed: the stage buffers may be reused
            mbar_wait_uniform(accf0 + 8 * (n_layers - 1), 0, abort_flag, p.status);
            if (lane == 0) stamp_end(fp.stamp);
        }
    } else {
        // head operands -> shared memory, then this CTA's slice of the head products; the barrier
        // covers these warps only (ids 2 .. nwarps-1), the two pipeline warps never join it
        mid_prefetch_head(p, h, q, id, (int)threadIdx.x - 64, (int)blockDim.x - 64);
        cp_async_commit();
        cp_async_wait_group<0>();
        asm volatile("bar.sync 1, %0;" ::"r"((int)blockDim.x - 64) : "memory");
        mid_head_products(p, h, q, warp - 2, nwarps - 2, lane);
        const int part = (warp - FUSED_DRAIN_WARP0) >> 2, nparts = (nwarps - FUSED_DRAIN_WARP0) >> 2;   // whole sets of four quadrants
        if (warp >= FUSED_DRAIN_WARP0 && part < nparts) {
            // accumulator rows (hi + lo) -> u[l][token][:] in global memory, layer by layer as they complete
            const int quad = warp & 3;
            const int row = quad * 32 + lane;                         // token
            for (int li = 0; li < n_layers; ++li) {
                if (!mbar_wait_warp(accf0 + 8 * li, 0, abort_flag, p.status)) break;
                tc_fence_after();
                float* dst = const_cast<float*>(p.u) + (long long)(l_begin + li) * p.lstride + ((long long)b * p.S + row) * p.r;
                for (int c0 = part * 16; c0 < p.r; c0 += 16 * nparts) {
                    float v[16];
                    const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)li * acc_cols + (uint32_t)c0;
                    tmem_ld16(taddr, v);
                    if (fp.wide_n) {
                        float w[16];
                        tmem_ld16(taddr + 64, w);
                        tmem_ld_wait();
#pragma unroll
                        for (int c = 0; c < 16; ++c) v[c] += w[c];
                    } else {
                        tmem_ld_wait();
                    }
                    if (row < p.S) {
#pragma unroll
                        for (int c = 0; c < 16; c += 4)
                            *reinterpret_cast<float4*>(dst + c0 + c) = make_float4(v[c], v[c + 1], v[c + 2], v[c + 3]);
                    }
                }
            }
        }
    }

    // ---- phase 2: every CTA's u rows are in global memory (L2); hand the stage buffers over to the chain ----
    tc_fence_before();
    __syncthreads();
    drain_after_abort(abort_flag);
    if (warp == 1) tmem_dealloc(tmem_base, 512u);
    cluster.sync();         // the peers' u rows are visible; head products are published

    // ---- phase 3: chain, head, loss, reverse chain; each thread fetches its own u values (all layers) first ----
    mid_body<ACT, bf16, 1, STATE_SMEM>(p, cluster, reinterpret_cast<float4*>(smem), h, true, id);
}

// Launch geometry: smallest cluster that gives one 4-column group per thread, at most FUSED_MAX_LPC
// layers per CTA and fits shared memory.
struct FusedFwdPlan {
    bool ok = false;
    MidPlan mp;
    int layers_per_cta = 0, stages = 0, k_chunks = 0, wide_n = 1;
    int max_clusters = 0;          // clusters of this shape the device runs at the same time
    size_t mid_offset = 0, smem = 0;
};

inline FusedFwdPlan fused_fwd_plan(const Dims& dm, int max_smem) {
    FusedFwdPlan fp;
    if (dm.S > FWD_ROWS || dm.r > 64 || dm.r % 16 != 0 || dm.d % 8 != 0 || dm.d < 64 || dm.C > MID_MAX_C || dm.L > MID_MAX_L) return fp;
    const size_t stage = FWD_ROWS * KC * 2 + 2 * KC * 128;
    for (int G = 1; G <= 8; G *= 2) {
        const int Sg = (dm.S + G - 1) / G, dg = (dm.d + G - 1) / G, lpc = (dm.L + G - 1) / G;
        const long long need = (long long)Sg * (dm.r / 4);
        if (need > 512 || lpc > FUSED_MAX_LPC) continue;
        int th = (int)((need + 31) / 32 * 32);
        if (th < 256) th = 256;                                  // producer, MMA, prefetch and drain warps
        int scratch;
        size_t floats = mid_base_floats(dm, Sg, dg, th, &scratch);
        const size_t state = (size_t)dm.L * th * sizeof(float4);   // chain state of mid_body: [L][threads] float4
        const size_t budget = (size_t)max_smem - 2048;
        // stage ring / chain state share one region, head vectors behind it
        {
            const size_t mid_bytes = floats * sizeof(float);
            if (mid_bytes + state > budget) continue;
            int st = (int)((budget - mid_bytes) / stage);
            if (st > 16) st = 16;
            if (st < 2) continue;
            size_t region = (size_t)st * stage;
            if (region < state) region = (state + 1023) & ~(size_t)1023;
            fp.mp.ok = true; fp.mp.G = G; fp.mp.Sg = Sg; fp.mp.dg = dg; fp.mp.threads = th; fp.mp.scratch = scratch;
            fp.mp.gpt = 1; fp.mp.smem_state = 1;
            fp.layers_per_cta = lpc; fp.stages = st; fp.k_chunks = (dm.d + KC - 1) / KC;
            fp.wide_n = lpc <= 4 ? 1 : 0;
            fp.mid_offset = region;
            fp.smem = fp.mid_offset + mid_bytes + 1024;
            fp.ok = true;
            return fp;
        }
    }
    return fp;
}

// How many of the plan's clusters can be resident at once (0 when the query fails).
template <int ACT>
inline int fused_fwd_max_clusters_act(const FusedFwdPlan& pl) {
    if (smem_opt_in((const void*)fwd_cluster_kernel<ACT>, pl.smem) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(pl.mp.G * 1024), 1, 1);
    cfg.blockDim = dim3((unsigned)pl.mp.threads, 1, 1);
    cfg.dynamicSmemBytes = pl.smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)pl.mp.G;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, fwd_cluster_kernel<ACT>, &cfg) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return n;
}
inline int fused_fwd_max_clusters(const FusedFwdPlan& pl, int act) {
    return act == PAC_ACT_RELU ? fused_fwd_max_clusters_act<PAC_ACT_RELU>(pl) : fused_fwd_max_clusters_act<PAC_ACT_IDENTITY>(pl);
}

template <int ACT>
inline cudaError_t fused_fwd_launch_act(const FusedFwdPlan& pl, const CUtensorMap& map_cache, const CUtensorMap& map_w,
                                        const FusedFwdParams& fp, cudaStream_t stream) {
    {
        cudaError_t e = smem_opt_in((const void*)fwd_cluster_kernel<ACT>, pl.smem);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(fp.mid.B * pl.mp.G), 1, 1);
    cfg.blockDim = dim3((unsigned)pl.mp.threads, 1, 1);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)pl.mp.G;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, fwd_cluster_kernel<ACT>, map_cache, map_w, fp);
}

inline cudaError_t fused_fwd_launch(const FusedFwdPlan& pl, const CUtensorMap& map_cache, const CUtensorMap& map_w,
                                    const FusedFwdParams& fp, int act, cudaStream_t stream) {
    return act == PAC_ACT_RELU ? fused_fwd_launch_act<PAC_ACT_RELU>(pl, map_cache, map_w, fp, stream)
                               : fused_fwd_launch_act<PAC_ACT_IDENTITY>(pl, map_cache, map_w, fp, stream);
}

}  // namespace pac
