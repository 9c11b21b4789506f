// Transformer-body adapters in plain fp32 (correctness-grade kernels, any shape).
//
// Section IV-A of the paper describes the side network as "a lightweight version of the backbone
// transformer-based LLM"; Section VI-A sets every weight and hidden dimension of an adapter to
// 1/rho of the backbone's.  Adapter l is therefore one pre-norm encoder layer at width r over the S
// tokens of a sample:
//     x   = lambda_l u_l + (1 - lambda_l) a_{l-1}
//     n1  = LayerNorm(x; g1, b1);   q, k, v = n1 Wq, n1 Wk, n1 Wv   (H heads of width r / H, no bias)
//     P_h = softmax(q_h k_h^T / sqrt(r / H)) over the keys;   x' = x + concat_h(P_h v_h) Wo
//     n2  = LayerNorm(x'; g2, b2);  a_l = x' + relu(n2 W1 + c1) W2 + c2
// The matrix products run through the generic tiled GEMM of pac_simt.cuh with element functors; this
// file holds the kernels that are not matrix products and the functors the products need.
// Flat parameter layout of one layer's body (floats): g1 | b1 | Wq | Wk | Wv | Wo | g2 | b2 | W1 | c1 | W2 | c2.
#pragma once
#include "pac_common.cuh"
#include "pac_simt.cuh"

namespace pac {

constexpr float TB_LN_EPS = 1e-5f;

struct BodyLayout {                  // offsets inside one layer's block, in floats
    int r, f;
    long long g1, b1, wq, wk, wv, wo, g2, b2, w1, c1, w2, c2, per_layer;
    __host__ __device__ static BodyLayout make(int r, int f) {
        BodyLayout b;
        b.r = r; b.f = f;
        b.g1 = 0; b.b1 = b.g1 + r; b.wq = b.b1 + r; b.wk = b.wq + (long long)r * r; b.wv = b.wk + (long long)r * r;
        b.wo = b.wv + (long long)r * r; b.g2 = b.wo + (long long)r * r; b.b2 = b.g2 + r; b.w1 = b.b2 + r;
        b.c1 = b.w1 + (long long)r * f; b.w2 = b.c1 + f; b.c2 = b.w2 + (long long)f * r; b.per_layer = b.c2 + r;
        return b;
    }
    // decoupled weight decay acts on the weight matrices only
    __host__ __device__ bool decays(long long off) const {
        return (off >= wq && off < g2) || (off >= w1 && off < c1) || (off >= w2 && off < c2);
    }
};

// x = lambda u + (1 - lambda) a_prev   (a_prev == nullptr: a_0 = 0)
__global__ void tb_merge_kernel(const float* __restrict__ u, const float* __restrict__ a_prev, const float* __restrict__ lam, int l,
                                long long n, float* __restrict__ x) {
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n) return;
    const float lm = lam[l];
    x[e] = lm * u[e] + (1.f - lm) * (a_prev ? a_prev[e] : 0.f);
}

// One warp per row: xhat = (x - mean) * rstd, n = xhat * g + b.
__global__ void tb_layernorm_fwd_kernel(const float* __restrict__ x, const float* __restrict__ g, const float* __restrict__ b, int M,
                                        int r, float* __restrict__ n, float* __restrict__ xhat, float* __restrict__ rstd) {
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (row >= M) return;
    const float* xr = x + (long long)row * r;
    float s = 0.f;
    for (int j = lane; j < r; j += 32) s += xr[j];
    const float mu = warp_sum(s) / (float)r;
    float v = 0.f;
    for (int j = lane; j < r; j += 32) { const float c = xr[j] - mu; v = fmaf(c, c, v); }
    const float rs = 1.f / sqrtf(warp_sum(v) / (float)r + TB_LN_EPS);
    for (int j = lane; j < r; j += 32) {
        const float xh = (xr[j] - mu) * rs;
        xhat[(long long)row * r + j] = xh;
        n[(long long)row * r + j] = xh * g[j] + b[j];
    }
    if (lane == 0) rstd[row] = rs;
}

// dx = add + (dxhat - mean(dxhat) - xhat * mean(dxhat * xhat)) * rstd,  dxhat = dn * g.  One warp per row.
__global__ void tb_layernorm_bwd_kernel(const float* __restrict__ dn, const float* __restrict__ xhat, const float* __restrict__ rstd,
                                        const float* __restrict__ g, const float* __restrict__ add, int M, int r, float* __restrict__ dx) {
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (row >= M) return;
    const long long o = (long long)row * r;
    float s1 = 0.f, s2 = 0.f;
    for (int j = lane; j < r; j += 32) {
        const float dh = dn[o + j] * g[j];
        s1 += dh;
        s2 = fmaf(dh, xhat[o + j], s2);
    }
    s1 = warp_sum(s1) / (float)r;
    s2 = warp_sum(s2) / (float)r;
    const float rs = rstd[row];
    for (int j = lane; j < r; j += 32) dx[o + j] = add[o + j] + (dn[o + j] * g[j] - s1 - xhat[o + j] * s2) * rs;
}

// Column sums over the M rows, in row order: out_a[j] = sum_i A[i][j] * (B ? B[i][j] : 1).
__global__ void tb_colsum_kernel(const float* __restrict__ A, const float* __restrict__ Bm, int M, int n, float* __restrict__ out) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n) return;
    float acc = 0.f;
    for (int i = 0; i < M; ++i) acc += Bm ? A[(long long)i * n + j] * Bm[(long long)i * n + j] : A[(long long)i * n + j];
    out[j] = acc;
}

// Attention forward, one thread per (sample, head, query token): softmax row P[b][h][s][:] and
// o[b][s][h*dh + :] = sum_t P[s][t] v[t][h*dh + :].  q, k, v, o: [M][r].
__global__ void tb_attn_fwd_kernel(const float* __restrict__ q, const float* __restrict__ k, const float* __restrict__ v, int B, int S,
                                   int r, int H, float* __restrict__ P, float* __restrict__ o) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)B * H * S) return;
    const int s = (int)(idx % S), h = (int)((idx / S) % H), b = (int)(idx / ((long long)S * H));
    const int dh = r / H, c0 = h * dh;
    const float scale = 1.f / sqrtf((float)dh);
    const float* qr = q + ((long long)b * S + s) * r + c0;
    float* Pr = P + (((long long)b * H + h) * S + s) * S;
    float mx = -INFINITY;
    for (int t = 0; t < S; ++t) {
        const float* kr = k + ((long long)b * S + t) * r + c0;
        float acc = 0.f;
        for (int i = 0; i < dh; ++i) acc = fmaf(qr[i], kr[i], acc);
        acc *= scale;
        Pr[t] = acc;
        mx = fmaxf(mx, acc);
    }
    float se = 0.f;
    for (int t = 0; t < S; ++t) { const float e = expf(Pr[t] - mx); Pr[t] = e; se += e; }
    for (int t = 0; t < S; ++t) Pr[t] = Pr[t] / se;
    float* orow = o + ((long long)b * S + s) * r + c0;
    for (int i = 0; i < dh; ++i) {
        float acc = 0.f;
        for (int t = 0; t < S; ++t) acc = fmaf(Pr[t], v[((long long)b * S + t) * r + c0 + i], acc);
        orow[i] = acc;
    }
}

// Attention backward in three steps (do = d loss / d o, [M][r]).
// (1) one thread per (b, h, key t):   dv[t][:] = sum_s P[s][t] do[s][:]
__global__ void tb_attn_bwd_dv_kernel(const float* __restrict__ P, const float* __restrict__ d_o, int B, int S, int r, int H,
                                      float* __restrict__ dv) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)B * H * S) return;
    const int t = (int)(idx % S), h = (int)((idx / S) % H), b = (int)(idx / ((long long)S * H));
    const int dh = r / H, c0 = h * dh;
    const float* Pb = P + ((long long)b * H + h) * S * S;
    for (int i = 0; i < dh; ++i) {
        float acc = 0.f;
        for (int s = 0; s < S; ++s) acc = fmaf(Pb[(long long)s * S + t], d_o[((long long)b * S + s) * r + c0 + i], acc);
        dv[((long long)b * S + t) * r + c0 + i] = acc;
    }
}
// (2) one thread per (b, h, query s):  dP[s][t] = <do[s], v[t]>,  ds = P * (dP - sum_t dP P)  (written over P),
//     dq[s][:] = scale * sum_t ds[s][t] k[t][:]
__global__ void tb_attn_bwd_dq_kernel(float* __restrict__ P, const float* __restrict__ d_o, const float* __restrict__ k,
                                      const float* __restrict__ v, int B, int S, int r, int H, float* __restrict__ dq) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)B * H * S) return;
    const int s = (int)(idx % S), h = (int)((idx / S) % H), b = (int)(idx / ((long long)S * H));
    const int dh = r / H, c0 = h * dh;
    const float scale = 1.f / sqrtf((float)dh);
    float* Pr = P + (((long long)b * H + h) * S + s) * S;
    const float* dor = d_o + ((long long)b * S + s) * r + c0;
    float dot = 0.f;
    for (int t = 0; t < S; ++t) {
        const float* vr = v + ((long long)b * S + t) * r + c0;
        float dp = 0.f;
        for (int i = 0; i < dh; ++i) dp = fmaf(dor[i], vr[i], dp);
        dot = fmaf(dp, Pr[t], dot);
    }
    for (int t = 0; t < S; ++t) {
        const float* vr = v + ((long long)b * S + t) * r + c0;
        float dp = 0.f;
        for (int i = 0; i < dh; ++i) dp = fmaf(dor[i], vr[i], dp);
        Pr[t] = Pr[t] * (dp - dot);                           // ds
    }
    float* dqr = dq + ((long long)b * S + s) * r + c0;
    for (int i = 0; i < dh; ++i) {
        float acc = 0.f;
        for (int t = 0; t < S; ++t) acc = fmaf(Pr[t], k[((long long)b * S + t) * r + c0 + i], acc);
        dqr[i] = acc * scale;
    }
}
// (3) one thread per (b, h, key t):    dk[t][:] = scale * sum_s ds[s][t] q[s][:]   (ds in the P buffer)
__global__ void tb_attn_bwd_dk_kernel(const float* __restrict__ dS, const float* __restrict__ q, int B, int S, int r, int H,
                                      float* __restrict__ dk) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)B * H * S) return;
    const int t = (int)(idx % S), h = (int)((idx / S) % H), b = (int)(idx / ((long long)S * H));
    const int dh = r / H, c0 = h * dh;
    const float scale = 1.f / sqrtf((float)dh);
    const float* Sb = dS + ((long long)b * H + h) * S * S;
    for (int i = 0; i < dh; ++i) {
        float acc = 0.f;
        for (int s = 0; s < S; ++s) acc = fmaf(Sb[(long long)s * S + t], q[((long long)b * S + s) * r + c0 + i], acc);
        dk[((long long)b * S + t) * r + c0 + i] = acc * scale;
    }
}

// dx -> dlambda_l = <dx, u - a_prev> (single block, fixed order), du_l = lambda dx, da_{l-1} = (1 - lambda) dx
__global__ void tb_unmerge_kernel(const float* __restrict__ dx, const float* __restrict__ u, const float* __restrict__ a_prev,
                                  const float* __restrict__ lam, int l, long long n, float* __restrict__ du, float* __restrict__ da_prev,
                                  float* __restrict__ dlam) {
    __shared__ float red[32];
    const float lm = lam[l];
    float acc = 0.f;
    for (long long e = threadIdx.x; e < n; e += blockDim.x) {
        const float g = dx[e];
        acc = fmaf(g, u[e] - (a_prev ? a_prev[e] : 0.f), acc);
        du[e] = lm * g;
        da_prev[e] = (1.f - lm) * g;
    }
    const float tot = block_sum(acc, red);
    if (threadIdx.x == 0) dlam[l] = tot;
}

// da[m][j] = daL[b(m)][j]: the classifier's d loss / d a_L is the same vector for every token of a sample
__global__ void tb_expand_kernel(const float* __restrict__ daL, int S, int r, long long n, float* __restrict__ da) {
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n) return;
    const long long m = e / r;
    da[e] = daL[(m / S) * r + (e - m * r)];
}

// ---- functors for the generic GEMM ----
struct MatA_ReluRowMajor {          // A(i,k) = max(pre[i][k], 0)
    static constexpr bool k_contiguous = true;
    const float* base; int ld;
    __device__ float operator()(int, int i, int k) const { return fmaxf(base[(long long)i * ld + k], 0.f); }
};
struct MatA_ReluColMajor {          // A(i,k) = max(pre[k][i], 0)    (hid^T)
    static constexpr bool k_contiguous = false;
    const float* base; int ld;
    __device__ float operator()(int, int i, int k) const { return fmaxf(base[(long long)k * ld + i], 0.f); }
};
struct StoreAddBias {               // out = v + add[i][j] + bias[j]   (add, bias may be null)
    float* out; const float* add; const float* bias; int ld;
    __device__ void operator()(int, int i, int j, float v) const {
        out[(long long)i * ld + j] = v + (add ? add[(long long)i * ld + j] : 0.f) + (bias ? bias[j] : 0.f);
    }
};
struct StoreAccumulate {            // out += v
    float* out; int ld;
    __device__ void operator()(int, int i, int j, float v) const { out[(long long)i * ld + j] += v; }
};
struct StoreMaskedByPositive {      // out = pre[i][j] > 0 ? v : 0
    float* out; const float* pre; int ld;
    __device__ void operator()(int, int i, int j, float v) const { out[(long long)i * ld + j] = pre[(long long)i * ld + j] > 0.f ? v : 0.f; }
};

}  // namespace pac
