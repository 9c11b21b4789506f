// One-launch forward for short sequences (S <= 128, r <= 64, classifier head): one thread-block
// cluster of G CTAs per batch sample does
//   1. the down-projections u_l = h_l W_down^l (Section IV-A) of the sample's 128-token tile, CTA q
//      taking layers q, q + G, ... (TMA-fed tcgen05 MMAs into one TMEM accumulator per layer; the
//      weights enter as bf16 hi + lo, side by side along N when at most four layers fall to a CTA,
//      else as two products summed in the same accumulator); meanwhile the other warps fetch the head
//      operands, form the head's product matrix (mid_head_products) and then drain every accumulator
//      AS SOON AS ITS LAYER IS COMPLETE, while the later layers still stream.  All but a CTA's last
//      layer go to the u buffer in global memory and are released to the peers with the arrival at a
//      cluster barrier, long before the stream ends.  A CTA's last layer (together the cluster's top
//      min(G, L) layers) is complete only when the stream is over: its rows go straight into the
//      shared memory of the CTA that owns the token (st.async), which counts the bytes on an mbarrier
//      of its own: no store has to be acknowledged and no barrier crossed behind the stream,
//   2. the wait at that cluster barrier (long satisfied), behind which every CTA fetches the u rows of
//      its tokens for the lower layers (L2 hits) into the shared memory the pipeline no longer needs,
//   3. everything the stand-alone fused kernel does afterwards (mid_body): merge/activation chain
//      (the handed-over top layers are awaited only where the chain reaches them), pooling, head,
//      loss, reverse chain -> du_l and dlambda partials.
#pragma once
#include "pac_mid.cuh"
#include "pac_tensor.cuh"

namespace pac {

struct FusedFwdParams {
    MidParams mid;             // G, Sg, dg, layers_per_cta, head operands, u buffer, outputs
    int k_chunks;              // ceil(d / 64)
    int stages;                // pipeline depth: stages of one cache tile + one weight tile (hi | lo)
    int wide_n;                // 1: hi | lo side by side (N = 128, 128 TMEM columns per layer); 0: two N = 64 products per K step
    size_t mid_offset;         // byte offset of the head vectors behind the stage / chain-state region
    size_t state_offset;       // byte offset of the chain state [L][threads] float4; its top n_land layers lie behind the stage ring
    int n_land;                // top layers handed over through shared memory (0: every layer goes through the u buffer)
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
    __shared__ __align__(8) unsigned long long bars[2 * 16 + FUSED_MAX_LPC + 1];
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;
    __shared__ long long id_sh;
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[16]), accf0 = smem_u32(&bars[32]);
    const uint32_t land_bar = smem_u32(&bars[32 + FUSED_MAX_LPC]);
    const int n_layers = q < p.L ? (p.L - q + p.G - 1) / p.G : 0;          // this CTA's layers: q, q + G, ...
    const int n_land = fp.n_land;                                           // 0, or min(G, L): the last layer of every CTA that has one
    float4* state = reinterpret_cast<float4*>(smem + fp.state_offset);      // [L][threads]
    const uint32_t acc_cols = fp.wide_n ? (uint32_t)FUSED_N : 64u;            // TMEM columns per layer

    if (threadIdx.x == 0) {
        abort_sh = 0;
        for (int s = 0; s < fp.stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int li = 0; li < FUSED_MAX_LPC; ++li) mbar_init(accf0 + 8 * li, 1);
        // the handed-over layers: n_land rows of r floats for each of this CTA's tokens, from the whole cluster
        mbar_init(land_bar, 1);
        const int rows_owned = max(0, min(p.Sg, p.S - q * p.Sg));
        mbar_expect_tx(land_bar, (uint32_t)(n_land * rows_owned * p.r) * 4u);
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
    // Cluster barrier, first round: its completion tells a CTA that the peers' hand-over mbarriers exist.  Second
    // round: a thread arrives when everything it writes for the peers outside the hand-over (u rows in global
    // memory, head products in shared memory) is written; the wait follows the stream.
    cluster.barrier_arrive();
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
                                 (int)(s % fp.k_chunks) * KC, 0, q + (int)(s / fp.k_chunks) * p.G, (int)id, pol);
            }
        }
        __syncwarp();
    }
    pdl_wait();                 // weights, parameters and (device) ids of this step are final from here on
    if (!early) id = safe_id(p.ids, b, p.N, (threadIdx.x == 0 && q == 0) ? p.status : nullptr);
    if (p.ids_copy && q == 0 && threadIdx.x == 0) p.ids_copy[b] = (int)id;

    // ---- phase 1: the GEMMs of this CTA's layers; the other warps fetch the head operands, then drain
    // finished accumulators.  The pipeline loops are run by whole converged warps, one elected lane issues. ----
    // Both loops are run by a whole converged warp, one elected lane issues; their own instruction streams, not
    // the copies or the tensor pipe, set the pace of a K step (an empty pipeline, with no copies and no MMAs,
    // steps barely faster), so ring positions, parities, addresses and descriptors are carried from step to
    // step instead of being recomputed.
    if (warp == 0) {
        cluster.barrier_wait();
        cluster.barrier_arrive();                                  // nothing of this warp's is read by the peers
        uint32_t it = 0, s = 0, eph = 1;                           // eph: parity of the "stage free" phase to wait for
        uint32_t dst = smem_u32(smem);
        const uint32_t ring_end = dst + (uint32_t)fp.stages * stage_bytes;
        bool ok = true;
        if (lane == 0 && n_layers > 0) stamp_begin(fp.stamp);      // first copy after the predecessor has finished
        for (int l = q; l < p.L && ok; l += p.G) {
            for (int kc = 0; kc < fp.k_chunks; ++kc, ++it) {
                const uint32_t full = full0 + 8 * s;
                if (it < pre) {
                    // first round: the cache tile was requested before the wait above, the weight tile follows
                    if (elect_one()) tma_load_4d(dst + a_bytes, &map_w, full, 0, kc * KC, 0, l);
                } else {
                    if (!mbar_wait_uniform(empty0 + 8 * s, eph, abort_flag, p.status)) { ok = false; break; }
                    if (elect_one()) {
                        mbar_expect_tx(full, stage_bytes);
                        tma_load_4d_hint(dst, &map_cache, full, kc * KC, 0, l, (int)id, pol);
                        tma_load_4d(dst + a_bytes, &map_w, full, 0, kc * KC, 0, l);
                    }
                }
                __syncwarp();
                dst += stage_bytes;
                if (++s == (uint32_t)fp.stages) { s = 0; eph ^= 1u; dst = ring_end - (uint32_t)fp.stages * stage_bytes; }
            }
        }
    } else if (warp == 1) {
        cluster.barrier_wait();
        cluster.barrier_arrive();
        const uint32_t idesc = fp.wide_n ? instr_desc_bf16(FWD_ROWS, FUSED_N, 0, 1) : instr_desc_bf16(FWD_ROWS, 64, 0, 1);
        // descriptors hold addresses in units of 16 bytes
        const uint64_t a_desc0 = smem_desc_sw128(smem_u32(smem), 16, 1024), w_desc0 = smem_desc_sw128(smem_u32(smem) + a_bytes, KC * 128, 1024);
        const uint64_t desc_step = (uint64_t)(stage_bytes >> 4), desc_ring = desc_step * (uint64_t)fp.stages;
        uint64_t ad0 = a_desc0, bw0 = w_desc0;
        uint32_t s = 0, ph = 0;
        bool ok = true;
        for (int li = 0; li < n_layers && ok; ++li) {
            const uint32_t d_tmem = tmem_base + (uint32_t)li * acc_cols;
            for (int kc = 0; kc < fp.k_chunks; ++kc) {
                if (!mbar_wait_uniform(full0 + 8 * s, ph, abort_flag, p.status)) { ok = false; break; }
                tc_fence_after();
                if (elect_one()) {
                    if (fp.wide_n) {
#pragma unroll
                        for (int k = 0; k < KC / 16; ++k)
                            umma_bf16(d_tmem, ad0 + (uint64_t)(k * 2), bw0 + (uint64_t)(k * 128), idesc, (kc | k) ? 1u : 0u);
                    } else {
                        // the lo block lies KC * 128 bytes behind the hi block of the same stage
                        const uint64_t bl0 = bw0 + (uint64_t)((KC * 128) >> 4);
#pragma unroll
                        for (int k = 0; k < KC / 16; ++k) {
                            umma_bf16(d_tmem, ad0 + (uint64_t)(k * 2), bw0 + (uint64_t)(k * 128), idesc, (kc | k) ? 1u : 0u);
                            umma_bf16(d_tmem, ad0 + (uint64_t)(k * 2), bl0 + (uint64_t)(k * 128), idesc, 1u);
                        }
                    }
                    umma_commit(empty0 + 8 * s);
                }
                __syncwarp();
                ad0 += desc_step; bw0 += desc_step;
                if (++s == (uint32_t)fp.stages) { s = 0; ph ^= 1u; ad0 -= desc_ring; bw0 -= desc_ring; }
            }
            if (ok) {
                if (elect_one()) umma_commit(accf0 + 8 * li);      // this layer's accumulator is complete
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
        bool arrived = false;
        if (warp >= FUSED_DRAIN_WARP0 && part < nparts) {
            // accumulator rows (hi + lo), layer by layer as they complete
            const int quad = warp & 3;
            const int row = quad * 32 + lane;                         // token
            const int gpt = p.r >> 2;                                 // 16-byte groups per token
            bool ok = true;
            for (int li = 0; li < n_layers; ++li) {
                const int l = q + li * p.G;
                const bool handed = n_land > 0 && li == n_layers - 1;
                if (handed) {
                    // the rows written so far are released to the peers now, under the stream of the last layer
                    cluster.barrier_wait();
                    cluster.barrier_arrive();
                    arrived = true;
                }
                if (!mbar_wait_warp(accf0 + 8 * li, 0, abort_flag, p.status)) { ok = false; break; }
                tc_fence_after();
                // the last layer is complete: so is every MMA, and the stage ring is free.  Its rows are laid out at the
                // ring's base exactly as the owners' chain state wants them (token-major, 16-byte groups swizzled as in
                // state_slot) and go out as one bulk copy per owner below.
                float* dst = handed ? reinterpret_cast<float*>(smem) + (size_t)row * p.r
                                    : const_cast<float*>(p.u) + (long long)l * p.lstride + ((long long)b * p.S + row) * p.r;
                const int sw = handed ? state_swizzle(row % p.Sg, gpt) : 0;
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
                        if (handed) {
#pragma unroll
                            for (int c = 0; c < 16; c += 4)
                                *reinterpret_cast<float4*>(dst + ((((c0 + c) >> 2) ^ sw) << 2)) = make_float4(v[c], v[c + 1], v[c + 2], v[c + 3]);
                        } else {
                            // whole 32-byte sectors
#pragma unroll
                            for (int c = 0; c < 16; c += 8)
                                st_global_32(dst + c0 + c, make_uint4(__float_as_uint(v[c]), __float_as_uint(v[c + 1]), __float_as_uint(v[c + 2]), __float_as_uint(v[c + 3])),
                                             make_uint4(__float_as_uint(v[c + 4]), __float_as_uint(v[c + 5]), __float_as_uint(v[c + 6]), __float_as_uint(v[c + 7])));
                        }
                    }
                }
            }
            if (n_land > 0) {
                // every draining warp passes here exactly once, whatever happened above
                fence_proxy_async();                                  // the rows above are read by the copy engine
                asm volatile("bar.sync 2, %0;" ::"r"(nparts * 128) : "memory");
                if (ok && n_layers > 0 && warp == FUSED_DRAIN_WARP0 && elect_one()) {
                    const int l = q + (n_layers - 1) * p.G;
                    for (int o = 0; o < p.G; ++o) {
                        const int rows = min(p.Sg, p.S - o * p.Sg);
                        if (rows <= 0) break;
                        dsmem_bulk_copy(mapa_shared(smem_u32(state + (size_t)l * blockDim.x), (uint32_t)o),
                                        smem_u32(smem) + (uint32_t)(o * p.Sg * p.r) * 4u, (uint32_t)(rows * p.r) * 4u,
                                        mapa_shared(land_bar, (uint32_t)o));
                    }
                }
                __syncwarp();
            }
        }
        if (!arrived) {
            cluster.barrier_wait();
            cluster.barrier_arrive();                             // head products and, without a hand-over, every u row
        }
    }

    // ---- phase 2: this CTA's pipeline is finished; hand the stage buffers over to the chain ----
    tc_fence_before();
    __syncthreads();
    drain_after_abort(abort_flag);
    if (warp == 1) tmem_dealloc(tmem_base, 512u);
    cluster.barrier_wait();         // the peers' u rows of the lower layers are visible; head products are published

    // ---- phase 3: chain, head, loss, reverse chain; each thread fetches its own u values of the lower layers first ----
    mid_body<ACT, bf16, 1, STATE_SMEM>(p, cluster, state, h, true, id, n_land, land_bar, abort_flag);
}

// Launch geometry: smallest cluster that gives one 4-column group per thread, at most FUSED_MAX_LPC
// layers per CTA and fits shared memory.
struct FusedFwdPlan {
    bool ok = false;
    MidPlan mp;
    int layers_per_cta = 0, stages = 0, k_chunks = 0, wide_n = 1;
    int max_clusters = 0;          // clusters of this shape the device runs at the same time
    size_t mid_offset = 0, state_offset = 0, smem = 0;
    int n_land = 0;                // top layers handed over through shared memory
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
        const int n_top = dm.L < G ? dm.L : G;                      // the last layer of every CTA that has one
        const size_t land = (size_t)n_top * th * sizeof(float4);
        const size_t budget = (size_t)max_smem - 2048;
        {
            const size_t mid_bytes = floats * sizeof(float);
            if (mid_bytes + state > budget) continue;
            // Without a hand-over the stage ring and the chain state share one region, head vectors behind it.
            int st = (int)((budget - mid_bytes) / stage);
            if (st > 16) st = 16;
            if (st < 3) continue;
            size_t region = (size_t)st * stage;
            if (region < state) region = (state + 1023) & ~(size_t)1023;
            fp.state_offset = 0;
            fp.n_land = 0;
            // With it the state's top layers, which the peers write while the ring is live, lie behind the ring; the
            // outgoing rows are staged at the ring's base, below the state.  Taken when that costs one stage at most
            // (the pipeline is not bound by its depth: four stages stream as fast as six).
            if (mid_bytes + land + 3 * stage <= budget) {
                int st2 = (int)((budget - mid_bytes - land) / stage);
                if (st2 > 16) st2 = 16;
                size_t region2 = (size_t)st2 * stage;
                if (region2 < state - land) region2 = (state - land + 1023) & ~(size_t)1023;
                region2 += land;
                const size_t staging = (size_t)FWD_ROWS * dm.r * sizeof(float);
                if (st2 >= 3 && st2 + 1 >= st && region2 - state >= staging) {
                    st = st2; region = region2;
                    fp.state_offset = region2 - state;
                    fp.n_land = n_top;
                }
            }
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
