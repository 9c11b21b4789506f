// The part of a classifier-head train step that sits between the two passes over the
// cache, fused into one kernel, and the gradient finalisation (+ AdamW) fused into another.
//
// mid_cls_kernel: one thread-block cluster per batch sample.  From the down-projections
// u_l it runs the lambda-merge / adapter-body chain (Section IV-A) for all layers keeping
// what the reverse pass needs (u_l - a_{l-1} in shared memory, the ReLU masks in registers), pools a_L over
// the sample's tokens through distributed shared memory, evaluates head, loss and their
// gradients for the sample, and walks the chain backwards to emit du_l (bf16 or fp32) and
// per-block partial sums of dlambda_l.  Nothing but u is read and nothing but du and a few
// per-sample vectors is written.
//
// All cross-thread sums use a fixed order, so results are bit-reproducible.
#pragma once
#include <cooperative_groups.h>
#include <type_traits>

#include "pac_common.cuh"
#include "pac_simt.cuh"
#include "pac_tensor.cuh"

namespace pac {

namespace cg = cooperative_groups;

struct MidParams {
    const int* ids; long long N; const int* labels;
    int L, S, d, r, C, B;
    int G;                      // cluster size: CTAs per sample
    int Sg;                     // tokens per CTA = ceil(S / G)
    int dg;                     // head columns per CTA = ceil(d / G)
    int train;
    int scratch;                // floats of block-local reduction scratch
    int aL_floats;              // floats of the a_L tile in shared memory (Sg * r; 0 when the chain ran elsewhere)
    int layers_per_cta;         // one-kernel forward: layers whose down-projections each CTA of the cluster computes
    int host_ids;               // 1: ids points at host memory the device can read (written before the launch, so
                                // it may be read ahead of the predecessor's completion); read once per CTA
    int early_ids;              // 1: no kernel ahead of this one in the stream writes the ids (device memory)
    // host_ids only: where the previous step's finalisation may already have left this step's ids in device
    // memory (valid when *pref_tag == pref_seq); otherwise the ids are fetched across the host link
    const int* pref_ids; const unsigned* pref_tag; unsigned pref_seq;
    int* ids_copy;              // one-kernel forward: device copy of the batch's (clamped) ids for the later kernels, or null
    // STATE_PARKED: what the down-projection kernel's epilogue left behind
    const unsigned* gates;      // [max_rows][r] bit l = gate of layer l
    const float* pool_part;     // [B][n_pool_parts][r] token sums of a_L per token group
    int n_pool_parts;
    const float* u; long long lstride;
    const float* lam; const float* W_up; const float* W_head; const float* b_head; const float* hbar;
    void* du;                   // [L][max_rows][r] bf16 or fp32
    float* pooled_a;            // [B][r]   mean_s a_L, for the gradient finalisation
    float* dlogits;             // [B][C]
    float* loss_b;              // [B]
    float* lam_part;            // [L][B*G]
    float* logits_out;          // [B][C] (train: scratch copy; eval: caller's buffer)
    unsigned* status;
    const float* prodW;         // optional [r][C]: W_up W_head, formed once per step by head_matrix_kernel (else per CTA)
};

constexpr int MID_MAX_C = 32;
constexpr size_t MID_SMEM_BUDGET = 220 * 1024;    // dynamic shared memory the fused kernel may use
constexpr int MID_RING = 4;       // layers of parked state in flight per thread in the reverse pass of long sequences
constexpr int MID_MAX_L = 32;     // ReLU masks of all layers live in one 32-bit word per element

__device__ __forceinline__ void cp_async_4(void* smem_dst, const void* gsrc) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_8(void* smem_dst, const void* gsrc) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_group() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Shared-memory chain state, [layer][thread] 16-byte groups: group c4 of a CTA's token s_local sits at group
// c4 ^ state_swizzle(s_local, groups per token) of the token's row, so that rows written one per lane (an
// accumulator row per thread) and rows read one group per lane are both free of bank conflicts.
__device__ __forceinline__ int state_swizzle(int s_local, int groups_per_tok) {
    const int m = (groups_per_tok & (groups_per_tok - 1)) ? 0 : min(groups_per_tok, 8) - 1;
    return s_local & m;
}

// Where the per-layer chain state (u_l on the way in, u_l - a_{l-1} for the reverse pass) lives.
enum {
    STATE_SMEM = 0,      // this CTA's shared memory, prefetched from the global u buffer with cp.async
    STATE_DU = 1,        // u read from global memory; u_l - a_{l-1} parked, in du's type, in the du slot
                         // that the reverse pass overwrites with du_l once it has consumed it
    STATE_PARKED = 2     // the forward chain already ran in the down-projection kernel's epilogue: u_l - a_{l-1} is
                         // parked in the du slots, the gates of all layers are one word per element in global
                         // memory, and the token sums of a_L come as per-group partial sums
};

// The small per-CTA vectors of the head computation, carved from one shared-memory region.
struct MidShared {
    float *aL, *colsum, *prodq, *prod, *plq, *daL, *py, *lg, *lam_s, *cprod, *wh_s, *lred;
};
__device__ __forceinline__ MidShared mid_carve(float* sm, const MidParams& p) {
    MidShared h;
    const size_t rc = (size_t)(p.r + 1) * p.C;
    h.aL = sm;                                        // [Sg][r]   a_L of this CTA's tokens
    h.colsum = h.aL + (size_t)p.aL_floats;            // [r]       exchanged through DSMEM
    h.prodq = h.colsum + p.r;                         // [r+1][C]  this CTA's partial head products, exchanged
    h.prod = h.prodq + rc;                            // [r+1][C]  their sum over the cluster
    h.plq = h.prod + rc;                              // [MID_MAX_C] this CTA's tokens' share of S * (mean_s a_L)(W_up W_head), exchanged
    h.daL = h.plq + MID_MAX_C;                        // [r]
    h.py = h.daL + p.r;                               // [dg]  slice of mean_s h_L
    h.lg = h.py + p.dg;                               // [MID_MAX_C] logits, then dlogits
    h.lam_s = h.lg + MID_MAX_C;                       // [MID_MAX_L]
    h.cprod = h.lam_s + MID_MAX_L;                    // [MID_MAX_L] prod_{l' > l} (1 - lambda_l')
    h.wh_s = h.cprod + MID_MAX_L;                     // [dg][C] slice of W_head
    h.lred = h.wh_s + (size_t)p.dg * p.C;             // [nwarps][MID_MAX_L]; also [parts][r] scratch
    return h;
}

// cp.async requests for the head operands of CTA rank q (hbar slice of sample `id`, W_head slice)
// and plain loads of lambda, issued by threads t0 .. t0 + nthr - 1 of the block.
__device__ __forceinline__ void mid_prefetch_head(const MidParams& p, const MidShared& h, int q, long long id, int t, int nthr) {
    const int k0 = q * p.dg, kn = max(0, min(p.dg, p.d - k0));
    for (int kk = t; kk < kn; kk += nthr) cp_async_4(h.py + kk, p.hbar + id * p.d + k0 + kk);
    for (int e = t; e < kn * p.C; e += nthr) cp_async_4(h.wh_s + e, p.W_head + (long long)k0 * p.C + e);
    for (int l = t; l < MID_MAX_L; l += nthr) h.lam_s[l] = l < p.L ? p.lam[l] : 0.f;
    if (t == nthr - 1) {
        // prod_{l' > l} (1 - lambda_l'), multiplied in the order the reverse recursion meets the layers
        float c = 1.f;
        for (int l = p.L - 1; l >= 0; --l) {
            h.cprod[l] = c;
            c *= 1.f - p.lam[l];
        }
    }
}

// The head is linear in mean_s a_L, so both directions through it reduce to one small matrix:
//   logits = b_head + hbar W_head + (mean_s a_L) (W_up W_head),      d loss / d mean_s a_L = (W_up W_head) dlogits.
// Each CTA forms the products over its own slice of the hidden width (operands already in shared
// memory):  prodq[j][c] = sum_k W_up[j][k] W_head[k][c]  (j < r),  prodq[r][c] = sum_k hbar[k] W_head[k][c];
// the slices are added across the cluster afterwards.  Called by nw whole warps, w = the caller's
// index among them; none of it depends on u, so it can run while u is still being produced.
__device__ __forceinline__ void mid_head_products(const MidParams& p, const MidShared& h, int q, int w, int nw, int lane) {
    const int k0 = q * p.dg, kn = max(0, min(p.dg, p.d - k0));
    // with the sample-independent rows already formed for the whole step only the hbar row is left
    for (int j = p.prodW ? p.r + w : w; j <= p.r; j += nw) {
        for (int c0 = 0; c0 < p.C; c0 += 4) {
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            for (int kk = lane; kk < kn; kk += 32) {
                const float a = j == p.r ? h.py[kk] : p.W_up[(long long)j * p.d + k0 + kk];     // each W_up element is read once
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (c0 + c < p.C) acc[c] = fmaf(a, h.wh_s[kk * p.C + c0 + c], acc[c]);
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const float v = warp_sum(acc[c]);
                if (lane == 0 && c0 + c < p.C) h.prodq[j * p.C + c0 + c] = v;
            }
        }
    }
}
// prodW[j][c] = sum_k W_up[j][k] W_head[k][c], one warp per entry, k in lane order then a fixed shuffle tree.  The
// product does not depend on the sample: the stand-alone head kernels take it from here instead of forming
// it again in every CTA (the one-launch forward forms it on warps that would otherwise idle under the stream).
__global__ void __launch_bounds__(256) head_matrix_kernel(const float* __restrict__ W_up, const float* __restrict__ W_head, int d, int r,
                                                          int C, float* __restrict__ prodW) {
    pdl_trigger();
    pdl_wait();                      // the parameters come from the optimizer update before this kernel
    const int e = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (e >= r * C) return;
    const int j = e / C, c = e - j * C;
    float acc = 0.f;
    for (int k = lane; k < d; k += 32) acc = fmaf(W_up[(long long)j * d + k], W_head[(long long)k * C + c], acc);
    acc = warp_sum(acc);
    if (lane == 0) prodW[e] = acc;
}

// After a cluster-wide barrier behind mid_head_products: the sum over the cluster, in rank order.  The
// last row also takes the classifier bias, so the head needs no global load of its own later on.
__device__ __forceinline__ void mid_sum_products(const MidParams& p, const MidShared& h, cg::cluster_group& cluster, int t, int nthr) {
    for (int e = t; e < (p.r + 1) * p.C; e += nthr) {
        if (p.prodW && e < p.r * p.C) { h.prod[e] = p.prodW[e]; continue; }
        float acc = 0.f;
        for (int g = 0; g < p.G; ++g) acc += cluster.map_shared_rank(h.prodq, g)[e];
        if (e >= p.r * p.C) acc = p.b_head[e - p.r * p.C] + acc;      // b_head + (mean_s h_L) W_head
        h.prod[e] = acc;
    }
}

// Everything after the down-projections for one sample, executed by one CTA (rank q) of the
// sample's cluster.  GPT: 4-column groups per thread.  u_s: STATE_SMEM: [L][GPT][nt] float4 state;
// products_ready: the caller has already prefetched the head
// operands, run mid_head_products and passed a cluster barrier.  n_landed > 0 (STATE_SMEM): the state of the
// top n_landed layers is not fetched from the u buffer: the cluster's CTAs write it into u_s directly and the
// mbarrier land_bar (shared-memory address, phase 0) completes when all of it has arrived.
template <int ACT, typename DU, int GPT, int STATE>
__device__ __forceinline__ void mid_body(const MidParams& p, cg::cluster_group& cluster, float4* u_s, const MidShared& h,
                                         bool products_ready, long long known_id = -1, int n_landed = 0, uint32_t land_bar = 0,
                                         volatile int* abort_flag = nullptr) {
    constexpr int LT = MID_MAX_L;
    const int q = (int)cluster.block_rank();
    const int b = blockIdx.x / p.G;
    const int t = threadIdx.x, nt = blockDim.x;
    const int r = p.r, L = p.L, C = p.C;
    const int warp = t >> 5, lane = t & 31, nwarps = nt >> 5;
    float *aL = h.aL, *colsum = h.colsum, *prod = h.prod, *plq = h.plq,
          *lg = h.lg, *lam_s = h.lam_s, *lred = h.lred, *cprod = h.cprod, *daL = h.daL;

    const int groups_per_tok = r >> 2;
    int s_local[GPT], j4[GPT], ts[GPT];                   // ts: this thread's slot in a layer's plane of the shared-memory state
    bool live[GPT];
    long long base[GPT];
#pragma unroll
    for (int g = 0; g < GPT; ++g) {
        const int gi = t + g * nt;                       // this thread's g-th group of 4 adapter columns
        s_local[g] = gi / groups_per_tok;
        j4[g] = (gi - s_local[g] * groups_per_tok) << 2;
        const int s = q * p.Sg + s_local[g];
        live[g] = s_local[g] < p.Sg && s < p.S;
        base[g] = ((long long)b * p.S + s) * r + j4[g];
        ts[g] = t ^ state_swizzle(s_local[g], groups_per_tok);
    }
    DU* du = reinterpret_cast<DU*>(p.du);
    // layer l of group g: read u, park / fetch the reverse-pass state
    auto load_u = [&](int l, int g) -> float4 {
        if constexpr (STATE == STATE_SMEM) return u_s[((size_t)l * GPT + g) * nt + ts[g]];
        else return *reinterpret_cast<const float4*>(p.u + (long long)l * p.lstride + base[g]);
    };
    auto store_w = [&](int l, int g, const float* wv) {
        if constexpr (STATE == STATE_SMEM) {
            u_s[((size_t)l * GPT + g) * nt + ts[g]] = make_float4(wv[0], wv[1], wv[2], wv[3]);
        } else if constexpr (sizeof(DU) == 2) {
            __nv_bfloat162 lo = __floats2bfloat162_rn(wv[0], wv[1]), hi = __floats2bfloat162_rn(wv[2], wv[3]);
            uint2 pk;
            pk.x = *reinterpret_cast<unsigned*>(&lo);
            pk.y = *reinterpret_cast<unsigned*>(&hi);
            *reinterpret_cast<uint2*>(du + (long long)l * p.lstride + base[g]) = pk;
        } else {
            *reinterpret_cast<float4*>(du + (long long)l * p.lstride + base[g]) = make_float4(wv[0], wv[1], wv[2], wv[3]);
        }
    };
    auto load_w = [&](int l, int g) -> float4 {
        if constexpr (STATE == STATE_SMEM) {
            return u_s[((size_t)l * GPT + g) * nt + ts[g]];
        } else if constexpr (sizeof(DU) == 2) {
            const uint2 pk = *reinterpret_cast<const uint2*>(du + (long long)l * p.lstride + base[g]);
            const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pk.x));
            const float2 c = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pk.y));
            return make_float4(a.x, a.y, c.x, c.y);
        } else {
            return *reinterpret_cast<const float4*>(du + (long long)l * p.lstride + base[g]);
        }
    };
    const long long id = known_id >= 0 ? known_id : safe_id(p.ids, b, p.N, (t == 0 && q == 0) ? p.status : nullptr);
    if (!products_ready) mid_prefetch_head(p, h, q, id, t, nt);
    cp_async_commit();                                                          // group: head operands
    if constexpr (STATE == STATE_SMEM) {
#pragma unroll
        for (int g = 0; g < GPT; ++g)
            if (live[g])
                for (int l = 0; l < L - n_landed; ++l) cp_async_16(u_s + ((size_t)l * GPT + g) * nt + ts[g], p.u + (long long)l * p.lstride + base[g]);
    }
    cp_async_commit();                                                          // group: u
    const int label = p.train ? p.labels[id] : 0;                               // fetched long before the head needs it
    if (!products_ready) {
        cp_async_wait_group<1>();                                               // head operands have landed ...
        __syncthreads();                                                        // ... those of every thread
        mid_head_products(p, h, q, warp, nwarps, lane);                         // overlaps the u copies in flight
        cluster.sync();
    }
    mid_sum_products(p, h, cluster, t, nt);              // read after the block barriers below
    cp_async_wait_group<0>();                            // own u values have landed

    // ---- forward chain over each group of 4 adapter columns of one token.  The slot that held
    // u_l is overwritten with u_l - a_{l-1} (= d z_l / d lambda_l) for the reverse pass; the ReLU
    // masks stay in registers (bit l of mask[g][e]).  Layers are taken four at a time so that the
    // loads of a batch are in flight together; the outer loops stay rolled (every CTA runs this
    // code once, so small code beats unrolled code).
    unsigned mask[GPT][4];
    float ap[GPT][4];
    bool landed = false;
    // column sums of a_L straight from registers when a warp holds whole tokens (one group per thread, 4, 8 or 16 groups per token)
    const bool shuffle_sums = GPT == 1 && STATE != STATE_PARKED && groups_per_tok <= 32 && (32 % groups_per_tok) == 0;
#pragma unroll
    for (int g = 0; g < GPT; ++g) {
#pragma unroll
        for (int e = 0; e < 4; ++e) { mask[g][e] = 0u; ap[g][e] = 0.f; }      // a_0 = 0
        if constexpr (STATE == STATE_PARKED) {
            // the chain ran in the down-projection kernel's epilogue: only the gate words are fetched
            if (live[g] && ACT == PAC_ACT_RELU && p.train) {
                const uint4 gw = *reinterpret_cast<const uint4*>(p.gates + base[g]);
                mask[g][0] = gw.x; mask[g][1] = gw.y; mask[g][2] = gw.z; mask[g][3] = gw.w;
            }
            continue;
        }
        if (live[g]) {
#pragma unroll 1
            for (int l0 = 0; l0 < L; l0 += 4) {
                if (n_landed > 0 && !landed && l0 + 4 > L - n_landed) {
                    mbar_wait(land_bar, 0, abort_flag, p.status);      // the handed-over layers have arrived
                    landed = true;
                }
                float4 uq[4];
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (l0 + i < L) uq[i] = load_u(l0 + i, g);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int l = l0 + i;
                    if (l < L) {
                        const float uv[4] = {uq[i].x, uq[i].y, uq[i].z, uq[i].w};
                        const float lm = lam_s[l];
                        float wv[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float z = lm * uv[e] + (1.f - lm) * ap[g][e];
                            wv[e] = uv[e] - ap[g][e];
                            if (ACT == PAC_ACT_RELU) {
                                const bool on = z > 0.f;
                                mask[g][e] |= (on ? 1u : 0u) << l;
                                ap[g][e] = on ? z : 0.f;
                            } else {
                                ap[g][e] = z;
                            }
                        }
                        store_w(l, g, wv);
                    }
                }
            }
        }
        if (!shuffle_sums && s_local[g] < p.Sg) {
#pragma unroll
            for (int e = 0; e < 4; ++e) aL[(size_t)s_local[g] * r + j4[g] + e] = live[g] ? ap[g][e] : 0.f;
        }
    }
    if (shuffle_sums) {
        // the lanes of a warp that hold the same four columns (one per token of the warp) add up by shuffles, in a
        // fixed order; one partial sum per warp and column goes to shared memory
        float v[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) v[e] = live[0] ? ap[0][e] : 0.f;
        for (int off = groups_per_tok; off < 32; off <<= 1)
#pragma unroll
            for (int e = 0; e < 4; ++e) v[e] += __shfl_xor_sync(0xffffffffu, v[e], off);
        if (lane < groups_per_tok)
#pragma unroll
            for (int e = 0; e < 4; ++e) lred[warp * r + (lane << 2) + e] = v[e];
    }
    __syncthreads();
    // column sums over this CTA's tokens: `parts` partial sums per column over contiguous token
    // ranges, then added in range order
    {
        int parts = 1;
        if (shuffle_sums) {
            parts = nwarps;
        } else if constexpr (STATE == STATE_PARKED) {
            // token-group sums from the down-projection kernel; CTA q of the cluster takes groups q, q + G, ...
            if (t < r) {
                float acc = 0.f;
                for (int pp = q; pp < p.n_pool_parts; pp += p.G) acc += p.pool_part[((long long)b * p.n_pool_parts + pp) * r + t];
                lred[t] = acc;
            }
        } else {
            parts = max(1, min(nt / r, p.Sg));
            const int per = (p.Sg + parts - 1) / parts;
            if (t < parts * r) {
                const int j = t % r, part = t / r;
                float acc = 0.f;
                for (int sl = part * per; sl < min(p.Sg, (part + 1) * per); ++sl) acc += aL[(size_t)sl * r + j];
                lred[part * r + j] = acc;
            }
        }
        if (!shuffle_sums) __syncthreads();
        if (t < r) {
            float acc = 0.f;
            for (int part = 0; part < parts; ++part) acc += lred[part * r + t];
            colsum[t] = acc;
        }
        // What the head needs of a_L is its token sum times the head's product matrix; this CTA's tokens'
        // share of that, plq[c] = sum_j colsum[j] prod[j][c], is formed here (warp c), so that only C numbers
        // per CTA cross the cluster on the way to the logits.
        for (int c = warp; c < C; c += nwarps) {
            float pl = 0.f;
            for (int j = lane; j < r; j += 32) {
                float cs = 0.f;
                for (int part = 0; part < parts; ++part) cs += lred[part * r + j];
                pl = fmaf(cs, prod[j * C + c], pl);
            }
            pl = warp_sum(pl);
            if (lane == 0) plq[c] = pl;
        }
    }
    cluster.sync();
    // ---- head, by ONE warp: logits from the cluster's C-vectors, loss, dlogits, d loss / d a_L; everybody
    // else waits at one block barrier.  The same in every CTA of the cluster.  A second warp of the first
    // CTA forms mean_s a_L for the gradient finalisation meanwhile.
    if (warp == 0) {
        float mylogit = -INFINITY;                        // lane c holds logit c (C <= 32)
        if (lane < C) {
            float acc = 0.f;
            for (int g = 0; g < p.G; ++g) acc += cluster.map_shared_rank(plq, g)[lane];
            mylogit = prod[r * C + lane] + acc / (float)p.S;      // b_head + (mean_s h_L) W_head + (mean_s a_L)(W_up W_head)
            if (q == 0) p.logits_out[(long long)b * C + lane] = mylogit;
        }
        if (p.train) {
            const float mx = warp_max(mylogit);
            const float ex = lane < C ? expf(mylogit - mx) : 0.f;
            const float se = warp_sum(ex);
            const float lab_logit = __shfl_sync(0xffffffffu, mylogit, label);
            if (lane == 0 && q == 0) p.loss_b[b] = mx + logf(se) - lab_logit;
            const float my = lane < C ? (ex / se - (lane == label ? 1.f : 0.f)) / (float)p.B : 0.f;     // dlogits
            if (lane < C) {
                lg[lane] = my;
                if (q == 0) p.dlogits[(long long)b * C + lane] = my;
            }
            __syncwarp();
            for (int j = lane; j < r; j += 32) {
                float acc = 0.f;
                for (int c = 0; c < C; ++c) acc = fmaf(prod[j * C + c], lg[c], acc);
                daL[j] = acc / (float)p.S;                // da_L, the same for every token of the sample
            }
        }
    } else if (warp == 1 && q == 0 && p.train) {
        for (int j = lane; j < r; j += 32) {
            float acc = 0.f;
            for (int g = 0; g < p.G; ++g) acc += cluster.map_shared_rank(colsum, g)[j];
            p.pooled_a[(long long)b * r + j] = acc / (float)p.S;      // mean_s a_L
        }
    }
    // That was this CTA's last access to a peer's shared memory: say so now and wait, at the very end, only
    // for the peers to have said the same (a CTA must not exit while a peer may still read its memory).
    cluster.barrier_arrive();
    __syncthreads();
    if (!p.train) {
        cluster.barrier_wait();                           // peers may still be reading this CTA's shared memory
        return;
    }

    // ---- reverse chain, in closed form.  da_L is the same vector for every token of the sample and a ReLU
    // gate only ever multiplies by exactly 1 or 0, so for an element whose gates l..L are all open
    //     dz_l = da_L[j] * prod_{l' > l} (1 - lambda_l'),   du_l = lambda_l dz_l,
    // and 0 as soon as one gate at or above l is closed (cprod[l] holds the product, formed once per CTA in
    // layer order).  No value depends on another layer's, so four layers are in flight at a time, the warp
    // sums of this thread's shares of dlambda_l = sum gate * dz_l * (u_l - a_{l-1}) included. ----
    float daLr[GPT][4];
#pragma unroll
    for (int g = 0; g < GPT; ++g)
#pragma unroll
        for (int e = 0; e < 4; ++e) daLr[g][e] = live[g] ? daL[j4[g] + e] : 0.f;
    int top_closed[GPT][4];                               // highest layer whose gate is closed (-1: none): open from there up only
#pragma unroll
    for (int g = 0; g < GPT; ++g)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const unsigned closed = (ACT == PAC_ACT_RELU) ? (~mask[g][e] & (L >= 32 ? 0xffffffffu : ((1u << L) - 1u))) : 0u;
            top_closed[g][e] = 31 - __clz(closed);        // __clz(0) = 32
        }
    // one layer of one group: du_l out, this thread's share of dlambda_l added to `part`
    auto reverse_step = [&](int l, int g, const float4& w4, float& part, float cp, float lm, DU* dst) {
        const float wv[4] = {w4.x, w4.y, w4.z, w4.w};
        float dv[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const bool open = l > top_closed[g][e];            // gates l .. L all open
            const float dz = open ? daLr[g][e] * cp : 0.f;
            part = fmaf(dz, wv[e], part);
            dv[e] = lm * dz;                                   // du_l
        }
        if constexpr (sizeof(DU) == 2) {
            __nv_bfloat162 lo = __floats2bfloat162_rn(dv[0], dv[1]), hi = __floats2bfloat162_rn(dv[2], dv[3]);
            uint2 pk;
            pk.x = *reinterpret_cast<unsigned*>(&lo);
            pk.y = *reinterpret_cast<unsigned*>(&hi);
            *reinterpret_cast<uint2*>(dst) = pk;
        } else {
            *reinterpret_cast<float4*>(dst) = make_float4(dv[0], dv[1], dv[2], dv[3]);
        }
    };
    if constexpr (STATE == STATE_PARKED) {
        // Long sequences: the reverse pass is a pure stream over the parked state.  It is fetched through a
        // ring of MID_RING layers in shared memory (cp.async, each thread reads back only what it requested),
        // so that GPT * MID_RING loads per thread are in flight without holding registers.
        uint2* ring = reinterpret_cast<uint2*>(u_s);
        // Running pointers instead of per-layer index arithmetic: src[g] walks the parked rows MID_RING layers
        // ahead of dst[g] (the same slots of the du buffer), slot walks the ring.
        DU* dst[GPT];
        const DU* src[GPT];
#pragma unroll
        for (int g = 0; g < GPT; ++g) { dst[g] = du + (long long)(L - 1) * p.lstride + base[g]; src[g] = dst[g]; }
        uint2* const ring_t = ring + t;
        const size_t slot_stride = (size_t)GPT * nt;
        int slot = 0;                                            // ring slot of the layer consumed next
        for (int i = 0; i < MID_RING; ++i) {
            if (L - 1 - i >= 0) {
#pragma unroll
                for (int g = 0; g < GPT; ++g) {
                    if (live[g]) cp_async_8(ring_t + (size_t)i * slot_stride + (size_t)g * nt, src[g]);
                    src[g] -= p.lstride;
                }
            }
            cp_async_commit();
        }
        // the launch geometry of this mode gives every group of a thread the same four columns, so the
        // per-layer coefficients are formed once per thread and layer
#pragma unroll 1
        for (int l = L - 1; l >= 0; --l) {
            cp_async_wait_group<MID_RING - 1>();
            float part = 0.f;
            const float cp = cprod[l], lm = lam_s[l];          // read once per layer (the stores below could alias them)
            float dzc[4], duc[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) { dzc[e] = daLr[0][e] * cp; duc[e] = lm * dzc[e]; }
            uint2* const rp = ring_t + (size_t)slot * slot_stride;
            uint2 x[GPT];
#pragma unroll
            for (int g = 0; g < GPT; ++g)
                if (live[g]) x[g] = rp[(size_t)g * nt];
#pragma unroll
            for (int g = 0; g < GPT; ++g) {
                if (live[g]) {
                    const float2 a2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&x[g].x));
                    const float2 c2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&x[g].y));
                    const float wv[4] = {a2.x, a2.y, c2.x, c2.y};
                    float dv[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const bool open = l > top_closed[g][e];
                        part = fmaf(open ? dzc[e] : 0.f, wv[e], part);
                        dv[e] = open ? duc[e] : 0.f;
                    }
                    __nv_bfloat162 lo = __floats2bfloat162_rn(dv[0], dv[1]), hi = __floats2bfloat162_rn(dv[2], dv[3]);
                    uint2 pk;
                    pk.x = *reinterpret_cast<unsigned*>(&lo);
                    pk.y = *reinterpret_cast<unsigned*>(&hi);
                    *reinterpret_cast<uint2*>(dst[g]) = pk;
                }
                dst[g] -= p.lstride;
            }
            // the slot just consumed takes the layer MID_RING further down
            if (l - MID_RING >= 0) {
#pragma unroll
                for (int g = 0; g < GPT; ++g) {
                    if (live[g]) cp_async_8(rp + (size_t)g * nt, src[g]);
                    src[g] -= p.lstride;
                }
            }
            cp_async_commit();
            if (++slot == MID_RING) slot = 0;
            part = warp_sum(part);
            if (lane == 0) lred[warp * LT + l] = part;
        }
    } else {
        // layers per batch: about four state loads in flight per thread whatever the number of groups it owns
        constexpr int LB = GPT >= 4 ? 1 : 4 / GPT;
        DU* dstp[GPT];                                        // running pointers into du, one layer down per step
#pragma unroll
        for (int g = 0; g < GPT; ++g) dstp[g] = du + (long long)(L - 1) * p.lstride + base[g];
#pragma unroll 1
        for (int l0 = L - 1; l0 >= 0; l0 -= LB) {
            float4 wq[LB][GPT];
#pragma unroll
            for (int i = 0; i < LB; ++i)
#pragma unroll
                for (int g = 0; g < GPT; ++g)
                    if (l0 - i >= 0 && live[g]) wq[i][g] = load_w(l0 - i, g);
            float part[LB];
#pragma unroll
            for (int i = 0; i < LB; ++i) {
                part[i] = 0.f;
                if (l0 - i >= 0) {
                    const float cp = cprod[l0 - i], lm = lam_s[l0 - i];
#pragma unroll
                    for (int g = 0; g < GPT; ++g) {
                        if (live[g]) reverse_step(l0 - i, g, wq[i][g], part[i], cp, lm, dstp[g]);
                        dstp[g] -= p.lstride;
                    }
                }
            }
            // this warp's shares of dlambda of the batch's layers: independent shuffle trees
#pragma unroll
            for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                for (int i = 0; i < LB; ++i) part[i] += __shfl_xor_sync(0xffffffffu, part[i], o);
            if (lane == 0)
#pragma unroll
                for (int i = 0; i < LB; ++i)
                    if (l0 - i >= 0) lred[warp * LT + (l0 - i)] = part[i];
        }
    }
    __syncthreads();
    if (t < L) {
        float acc = 0.f;
        for (int wv = 0; wv < nwarps; ++wv) acc += lred[wv * LT + t];
        p.lam_part[(long long)t * (p.B * p.G) + blockIdx.x] = acc;
    }
    cluster.barrier_wait();                               // keep shared memory alive until every peer has read it
}

// The stand-alone kernel: u comes from the global buffer written by the down-projection kernel.
template <int ACT, typename DU, int GPT, int STATE>
__global__ void __launch_bounds__(512, STATE == STATE_SMEM ? 1 : 2) mid_cls_kernel(MidParams p) {
    cg::cluster_group cluster = cg::this_cluster();
    extern __shared__ float4 sm4[];
    float4* u_s = sm4;                           // [L][GPT][nt] each thread's own u values, later u_l - a_{l-1}
    float* sm = reinterpret_cast<float*>(sm4 + (STATE == STATE_SMEM ? (size_t)p.L * GPT * blockDim.x
                                               : STATE == STATE_PARKED ? (size_t)MID_RING * GPT * blockDim.x / 2 : 0));
    const MidShared h = mid_carve(sm, p);
    pdl_trigger();
    pdl_wait();             // u (or the parked chain state) comes from the kernel before this one
    mid_body<ACT, DU, GPT, STATE>(p, cluster, u_s, h, false);
}

// ---------------------------------------------------------------------------
// Gradient finalisation for the classifier head, one thread per flat parameter index:
//   W_down : sum of the row-split partials of h^T du (split order), or already final
//   lambda : sum of per-block partials (block order)
//   W_up   : pooled_a^T g        W_head : pooled_y^T dlogits        b_head : sum_b dlogits
// plus the mean loss.  With adam != 0 the AdamW update of the same element follows at once.
// ---------------------------------------------------------------------------
struct FinalizeParams {
    ParamLayout lay;
    int B, d, r, C, L;
    const float* dw_part; int splits; long long dw_elems;     // splits <= 1: W_down gradient already in grads
    const float* lam_part; int lam_blocks;
    const float *pooled_a, *dlogits, *loss_b;                // per-sample vectors the forward half left: mean_s a_L, dlogits, loss
    const float* hbar; const int* ids; long long N;          // token mean of the last cached layer, per cache sample; the batch's ids
    const float* params_in;                                  // the parameters the forward half used (W_up, W_head are read)
    float* grads; float* loss_out;
    int wd_blocks;                                           // blocks that handle W_down, 4 elements per thread
    int rest_blocks;                                         // blocks that handle the head side: FIN_KB columns of the hidden width each
    // AdamW
    int adam;
    float *params, *m, *v;
    pac_adamw hp; float bc1, bc2;
    float grad_scale;                                        // factor on every gradient entering the fused update
    bf16* wdT;                                               // [L][2][d][r] bf16 hi/lo shadow of W_down (may be null)
    // Ids of the NEXT step (pac_train_step_async): if the host has already published them in its page-locked
    // ring (tag == next_seq), block 0 copies them to device memory, off every kernel's critical path.
    const int* next_host_ids; const unsigned* next_host_tag; unsigned next_seq; int next_n;
    int* next_dev_ids; unsigned* next_dev_tag;
    // Device status words: when a bounded wait of this or an earlier step has run out, the gradients
    // are not trustworthy, so nothing is written to the gradients, parameters or moments.
    unsigned* status;
};

constexpr int FIN_KB = 4;       // hidden-width columns per head-side block of the finalisation kernel

__device__ __forceinline__ unsigned ld_acquire_sys(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// (five blocks per SM: 48 registers, no spills; T5-Base step 51.0 -> 50.3 us against the 63 registers of an open bound)
__global__ void __launch_bounds__(256, 5) finalize_cls_kernel(FinalizeParams f) {
    pdl_trigger();
    const ParamLayout& lay = f.lay;
    // W_down blocks fetch the old parameter and moments while the predecessor still runs: nothing since the
    // previous finalisation writes them, and that one was over before the predecessor's own predecessor
    // finished (every kernel of a step lets its successor start only after its own wait has returned or
    // does not touch these arrays before its wait)
    // block 0 takes dlambda and the loss (scheduled first, so it runs at once), the next rest_blocks blocks the
    // head parameters, the remaining wd_blocks blocks W_down
    const int blk = (int)blockIdx.x - 1;
    const long long i_wd = ((long long)(blk - f.rest_blocks) * blockDim.x + threadIdx.x) * 4;
    const bool wd_thread = blk >= f.rest_blocks && i_wd < lay.lam;
    float4 p4 = make_float4(0.f, 0.f, 0.f, 0.f), m4 = p4, v4 = p4;
    if (wd_thread && f.adam) {
        p4 = *reinterpret_cast<const float4*>(f.params + i_wd);
        m4 = *reinterpret_cast<const float4*>(f.m + i_wd);
        v4 = *reinterpret_cast<const float4*>(f.v + i_wd);
    }
    // Block 0 (dlambda and the mean loss) needs only what the forward half left behind, which is
    // complete whenever this kernel runs (see above): it does not wait for the second pass at all, so a loss
    // that goes straight to host memory is on its way long before the step ends.
    // Set by a wait that ran out in this step's forward half or in any earlier step since the last
    // pac_sync (the forward half has completed whenever this kernel runs); a wait that runs out in this
    // step's second pass is seen by the W_down blocks behind their own wait below.
    const bool dead = status_timed_out(f.status);
    if (blk < 0) {
        // dlambda_l (one warp per layer, lanes over the per-block partials, fixed
        // shuffle order) and the mean loss
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
        if (dead && f.adam && threadIdx.x == 0) atomicAdd(&f.status[ST_SKIPPED_STEPS], 1u);
        for (int l = warp; l < f.L && !dead; l += nw) {
            float acc = 0.f;
            for (int k = lane; k < f.lam_blocks; k += 32) acc += f.lam_part[(long long)l * f.lam_blocks + k];
            acc = warp_sum(acc);
            if (lane == 0) {
                const long long i = lay.lam + l;
                f.grads[i] = acc;
                if (f.adam) adamw_element(f.params, f.m, f.v, i, acc * f.grad_scale, f.lay, f.hp, f.bc1, f.bc2, f.wdT, f.d, f.r);
            }
        }
        if (warp == nw - 1) {
            float acc = 0.f;
            for (int b = lane; b < f.B; b += 32) acc += f.loss_b[b];
            acc = warp_sum(acc);
            if (lane == 0) *f.loss_out = acc / (float)f.B;
        }
        if (warp == 0 && f.next_host_tag) {
            // the host writes a slot's ids first and its tag last; tag read first here, ids after it
            const unsigned tag = ld_acquire_sys(f.next_host_tag);
            if (tag == f.next_seq) {
                for (int b = lane; b < f.next_n; b += 32) f.next_dev_ids[b] = *reinterpret_cast<const volatile int*>(f.next_host_ids + b);
                // publish: the warp barrier orders every lane's id stores before lane 0, whose fence then
                // comes between them and the tag
                __syncwarp();
                if (lane == 0) {
                    __threadfence();
                    atomicExch(f.next_dev_tag, f.next_seq);
                }
            }
        }
        return;
    }
    if (blk < f.rest_blocks) {
        // Head-side parameters: like block 0 these blocks need only what the forward half left behind, so
        // they finish (and make room for the W_down blocks) while the second pass still runs.  A block owns
        // FIN_KB columns k of the hidden width: W_up[:, k] and W_head[k, :] (the last block also b_head).
        // It first rebuilds, for its columns, the two per-sample vectors of the head's backward,
        //     g[b][k]  = d loss / d mean_s y = sum_c W_head[k][c] dlogits[b][c]
        //     py[b][k] = mean_s y = hbar[id_b][k] + sum_j pooled_a[b][j] W_up[j][k]
        // from the OLD values of exactly the parameters it owns (read before any of them is updated), then
        //     dW_up[j][k] = sum_b pooled_a[b][j] g[b][k],   dW_head[k][c] = sum_b py[b][k] dlogits[b][c].
        extern __shared__ float fsm[];
        float* g_s = fsm;                                    // [B][FIN_KB]
        float* py_s = g_s + (size_t)f.B * FIN_KB;            // [B][FIN_KB]
        float* wup_s = py_s + (size_t)f.B * FIN_KB;          // [r][FIN_KB]   old W_up[:, k0..]
        float* wh_s = wup_s + (size_t)f.r * FIN_KB;          // [FIN_KB][C]   old W_head[k0.., :]
        const int k0 = blk * FIN_KB, kn = min(FIN_KB, f.d - k0), t = threadIdx.x, nt = blockDim.x;
        const float* W_up = f.params_in + lay.w_up;
        const float* W_head = f.params_in + lay.w_head;
        if (dead) return;
        for (int e = t; e < f.r * FIN_KB; e += nt) {
            const int j = e / FIN_KB, kk = e - j * FIN_KB;
            wup_s[e] = kk < kn ? W_up[(long long)j * f.d + k0 + kk] : 0.f;
        }
        for (int e = t; e < FIN_KB * f.C; e += nt) {
            const int kk = e / f.C;
            wh_s[e] = kk < kn ? W_head[(long long)k0 * f.C + e] : 0.f;
        }
        __syncthreads();
        for (int e = t; e < f.B * FIN_KB; e += nt) {
            const int b = e / FIN_KB, kk = e - b * FIN_KB;
            float gv = 0.f, acc = 0.f;
            for (int c = 0; c < f.C; ++c) gv = fmaf(wh_s[kk * f.C + c], f.dlogits[(long long)b * f.C + c], gv);
            for (int j = 0; j < f.r; ++j) acc = fmaf(f.pooled_a[(long long)b * f.r + j], wup_s[j * FIN_KB + kk], acc);
            const long long id = safe_id(f.ids, b, f.N, nullptr);
            g_s[e] = gv;
            py_s[e] = kk < kn ? f.hbar[id * f.d + k0 + kk] + acc : 0.f;
        }
        __syncthreads();
        const int n_up = f.r * FIN_KB, n_head = FIN_KB * f.C;
        const bool last = blk == f.rest_blocks - 1;
        for (int e = t; e < n_up + n_head + (last ? f.C : 0); e += nt) {
            long long i;
            float g = 0.f;
            if (e < n_up) {
                const int j = e / FIN_KB, kk = e - j * FIN_KB;
                if (kk >= kn) continue;
                i = lay.w_up + (long long)j * f.d + k0 + kk;
#pragma unroll 8
                for (int b = 0; b < f.B; ++b) g = fmaf(f.pooled_a[(long long)b * f.r + j], g_s[b * FIN_KB + kk], g);
            } else if (e < n_up + n_head) {
                const int kk = (e - n_up) / f.C, c = (e - n_up) - kk * f.C;
                if (kk >= kn) continue;
                i = lay.w_head + (long long)(k0 + kk) * f.C + c;
#pragma unroll 8
                for (int b = 0; b < f.B; ++b) g = fmaf(py_s[b * FIN_KB + kk], f.dlogits[(long long)b * f.C + c], g);
            } else {
                const int c = e - n_up - n_head;
                i = lay.b_head + c;
                for (int b = 0; b < f.B; ++b) g += f.dlogits[(long long)b * f.C + c];
            }
            f.grads[i] = g;
            if (f.adam) adamw_element(f.params, f.m, f.v, i, g * f.grad_scale, f.lay, f.hp, f.bc1, f.bc2, f.wdT, f.d, f.r);
        }
        return;
    }
    pdl_wait();
    {
        // W_down block, four consecutive elements per thread
        const long long i = i_wd;
        if (i >= lay.lam || status_timed_out(f.status)) return;
        float4 g4;
        if (f.splits > 1) {
            g4 = *reinterpret_cast<const float4*>(f.dw_part + i);
            for (int j = 1; j < f.splits; ++j) {                 // split order
                const float4 q = *reinterpret_cast<const float4*>(f.dw_part + (long long)j * f.dw_elems + i);
                g4.x += q.x; g4.y += q.y; g4.z += q.z; g4.w += q.w;
            }
            *reinterpret_cast<float4*>(f.grads + i) = g4;
        } else {
            g4 = *reinterpret_cast<const float4*>(f.grads + i);
        }
        if (f.adam) {
            g4.x *= f.grad_scale; g4.y *= f.grad_scale; g4.z *= f.grad_scale; g4.w *= f.grad_scale;
            adamw_w_down4_loaded(f.params, f.m, f.v, i, p4, m4, v4, g4, f.hp, f.bc1, f.bc2, f.wdT, f.d, f.r);
        }
        return;
    }
}

// Shape test and launch geometry of the fused kernel: G CTAs per sample, one 4-column
// group per thread, chain state in shared memory.
struct MidPlan {
    bool ok = false;
    int G = 1, Sg = 0, dg = 0, threads = 0, scratch = 0;
    int gpt = 1, smem_state = 1;      // 4-column groups per thread; chain state in shared memory or parked in the du buffer
    int aL_floats = 0;                // a_L tile in shared memory (0: the chain ran in the down-projection kernel)
    size_t smem = 0;
};

// Shared-memory floats the kernel needs besides the chain state and the W_up slice.
inline size_t mid_base_floats(const Dims& dm, int Sg, int dg, int th, int* scratch_out, bool with_aL = true) {
    const int nw = th / 32;
    int scratch = nw * MID_MAX_L;
    const int parts = th / dm.r > 0 ? th / dm.r : 1;
    if (parts * dm.r > scratch) scratch = parts * dm.r;
    if (nw * dm.r > scratch) scratch = nw * dm.r;              // one partial column sum per warp
    *scratch_out = scratch;
    return (with_aL ? (size_t)Sg * dm.r : 0) + 2 * (size_t)dm.r + MID_MAX_C + 2 * (size_t)(dm.r + 1) * dm.C + (size_t)dg + MID_MAX_C + MID_MAX_L + scratch +
           (size_t)dg * dm.C + MID_MAX_L + 4;
}

inline MidPlan mid_plan(const Dims& dm) {
    MidPlan mp;
    if (dm.r % 4 != 0 || dm.C > MID_MAX_C || dm.L > MID_MAX_L) return mp;
    const size_t budget = MID_SMEM_BUDGET / sizeof(float);
    // first choice: one group per thread, chain state in shared memory, fewest CTAs per sample
    for (int G = 1; G <= 8; G *= 2) {
        const int Sg = (dm.S + G - 1) / G, dg = (dm.d + G - 1) / G;
        const long long need = (long long)Sg * (dm.r / 4);
        if (need > 512) continue;
        int th = (int)((need + 31) / 32 * 32);
        if (th < 128) th = 128;
        int scratch;
        size_t floats = mid_base_floats(dm, Sg, dg, th, &scratch) + 4 * (size_t)dm.L * th;
        if (floats > budget) continue;
        mp.G = G; mp.Sg = Sg; mp.dg = dg; mp.threads = th; mp.scratch = scratch; mp.gpt = 1; mp.smem_state = 1;
        mp.smem = sizeof(float) * floats;
        mp.ok = true;
        return mp;
    }
    // otherwise: 8 CTAs per sample, up to 4 groups per thread, state parked in the du buffer
    {
        const int G = 8, Sg = (dm.S + G - 1) / G, dg = (dm.d + G - 1) / G;
        const long long need = (long long)Sg * (dm.r / 4);
        if (need > 4 * 512) return mp;
        const int gpt = need <= 512 ? 1 : need <= 1024 ? 2 : 4;
        int th = (int)(((need + gpt - 1) / gpt + 31) / 32 * 32);
        if (th < 128) th = 128;
        int scratch;
        size_t floats = mid_base_floats(dm, Sg, dg, th, &scratch);
        if (floats > budget) return mp;
        mp.G = G; mp.Sg = Sg; mp.dg = dg; mp.threads = th; mp.scratch = scratch; mp.gpt = gpt; mp.smem_state = 0;
        mp.smem = sizeof(float) * floats;
        mp.ok = true;
    }
    return mp;
}

// Geometry for the parked mode: the chain state never needs shared memory, so the smallest cluster with at
// most four 4-column groups per thread serves (fewer, fuller CTAs than the plan above).
inline MidPlan mid_plan_parked(const Dims& dm) {
    MidPlan mp;
    if (dm.r % 4 != 0 || dm.C > MID_MAX_C || dm.L > MID_MAX_L) return mp;
    for (int G = 1; G <= 8; G *= 2) {
        const int Sg = (dm.S + G - 1) / G, dg = (dm.d + G - 1) / G;
        const long long need = (long long)Sg * (dm.r / 4);
        if (need > 4 * 512) continue;
        const int gpt = need <= 512 ? 1 : need <= 1024 ? 2 : 4;
        // every group of a thread must land on the same four columns: threads a multiple of the groups per token
        const int gtok = dm.r / 4;
        int unit = 32;
        while (unit % gtok != 0) unit += 32;                    // lcm(32, r/4)
        int th = (int)(((need + gpt - 1) / gpt + unit - 1) / unit * unit);
        if (th < 128) th = (128 + unit - 1) / unit * unit;
        if (th > 512) continue;
        int scratch;
        const size_t floats = mid_base_floats(dm, Sg, dg, th, &scratch, false) + (size_t)MID_RING * gpt * th * 2;    // + the state ring (8 bytes per slot)
        if (floats > 110 * 1024 / sizeof(float)) continue;                // two CTAs per SM
        mp.G = G; mp.Sg = Sg; mp.dg = dg; mp.threads = th; mp.scratch = scratch; mp.gpt = gpt; mp.smem_state = 0;
        mp.smem = sizeof(float) * floats;
        mp.ok = true;
        return mp;
    }
    return mp;
}

template <int ACT, typename DU, int GPT, int STATE>
inline cudaError_t mid_launch_one(const MidPlan& mp, const MidParams& p, cudaStream_t stream) {
    {
        cudaError_t e = smem_opt_in((const void*)mid_cls_kernel<ACT, DU, GPT, STATE>, MID_SMEM_BUDGET);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.B * mp.G), 1, 1);
    cfg.blockDim = dim3((unsigned)mp.threads, 1, 1);
    cfg.dynamicSmemBytes = mp.smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)mp.G;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, mid_cls_kernel<ACT, DU, GPT, STATE>, p);
}

template <int ACT, typename DU>
inline cudaError_t mid_launch_shape(const MidPlan& mp, const MidParams& p, cudaStream_t stream) {
    if (mp.smem_state) return mid_launch_one<ACT, DU, 1, STATE_SMEM>(mp, p, stream);
    switch (mp.gpt) {
        case 1: return mid_launch_one<ACT, DU, 1, STATE_DU>(mp, p, stream);
        case 2: return mid_launch_one<ACT, DU, 2, STATE_DU>(mp, p, stream);
        default: return mid_launch_one<ACT, DU, 4, STATE_DU>(mp, p, stream);
    }
}

// The same kernel behind a down-projection kernel that already ran the forward chain (bf16 state parked in du).
template <int ACT>
inline cudaError_t mid_launch_parked_act(const MidPlan& mp, const MidParams& p, cudaStream_t stream) {
    switch (mp.gpt) {
        case 1: return mid_launch_one<ACT, bf16, 1, STATE_PARKED>(mp, p, stream);
        case 2: return mid_launch_one<ACT, bf16, 2, STATE_PARKED>(mp, p, stream);
        default: return mid_launch_one<ACT, bf16, 4, STATE_PARKED>(mp, p, stream);
    }
}
inline cudaError_t mid_launch_parked(const MidPlan& mp, const MidParams& p, int act, cudaStream_t stream) {
    return act == PAC_ACT_RELU ? mid_launch_parked_act<PAC_ACT_RELU>(mp, p, stream) : mid_launch_parked_act<PAC_ACT_IDENTITY>(mp, p, stream);
}

inline cudaError_t mid_launch(const MidPlan& mp, const MidParams& p, int act, bool du_bf16, cudaStream_t stream) {
    if (act == PAC_ACT_RELU)
        return du_bf16 ? mid_launch_shape<PAC_ACT_RELU, bf16>(mp, p, stream) : mid_launch_shape<PAC_ACT_RELU, float>(mp, p, stream);
    return du_bf16 ? mid_launch_shape<PAC_ACT_IDENTITY, bf16>(mp, p, stream) : mid_launch_shape<PAC_ACT_IDENTITY, float>(mp, p, stream);
}

}  // namespace pac
