// Plain fp32-FMA kernels: every step of the path for any shape and both cache
// dtypes.  They serve the fp32 configuration (whose 1e-4 tolerance rules out
// reduced-precision tensor-core operands) and shapes the tensor-core path does not
// take; the small per-sample head/chain kernels here are shared by both paths.
//
// Notation follows Section IV-A of the paper: h_l cached state of layer l,
// u_l = h_l W_down^l, z_l = lambda_l u_l + (1-lambda_l) a_{l-1}, a_l = phi(z_l),
// y = h_L + a_L W_up.
#pragma once
#include "pac_common.cuh"

namespace pac {

// ---------------------------------------------------------------------------
// Cache gather (Section IV-B): out[l][b] = cache[ids[b]][l], 16-byte vectors.
// One block per (b, l) slab; slab_bytes is a multiple of 16 when vec16 is set.
// ---------------------------------------------------------------------------
__global__ void gather_kernel(const unsigned char* __restrict__ cache, const int* __restrict__ ids, long long N,
                              int L, int B, long long slab_bytes, unsigned char* __restrict__ out, int vec16,
                              unsigned* status) {
    int l = blockIdx.x % L, b = blockIdx.x / L;
    long long id = safe_id(ids, b, N, threadIdx.x == 0 && blockIdx.y == 0 ? status : nullptr);
    const unsigned char* src = cache + (id * L + l) * slab_bytes;
    unsigned char* dst = out + ((long long)l * B + b) * slab_bytes;
    long long t = (long long)blockIdx.y * blockDim.x + threadIdx.x, step = (long long)gridDim.y * blockDim.x;
    if (vec16) {
        const uint4* s4 = reinterpret_cast<const uint4*>(src);
        uint4* d4 = reinterpret_cast<uint4*>(dst);
        for (long long i = t; i < slab_bytes / 16; i += step) d4[i] = __ldg(s4 + i);
    } else {
        for (long long i = t; i < slab_bytes; i += step) dst[i] = src[i];
    }
}

// ---------------------------------------------------------------------------
// Generic tiled fp32 GEMM  C(z; i, j) = sum_k A(z; i, k) * B(z; k, j)  with element
// access through functors, so the gathered cache, transposes and fused epilogues need
// no staging copies.  64x64x16 tiles, 256 threads, 4x4 outputs per thread; each output
// is summed by one thread in k order, so results do not depend on the launch shape.
// ---------------------------------------------------------------------------
constexpr int SG_BM = 64, SG_BN = 64, SG_BK = 16;

// The k loop of one 64x64 output tile over [k_begin, k_end): 4x4 partial sums per thread.
template <class AF, class BF>
__device__ __forceinline__ void gemm_simt_tile(int M, int N, int K, int k_begin, int k_end, const AF& A, const BF& B, int z,
                                               int i0, int j0, float (&acc)[4][4], float (*As)[SG_BM + 4], float (*Bs)[SG_BN + 4]) {
    const int t = threadIdx.x, ty = t / 16, tx = t % 16;
    for (int k0 = k_begin; k0 < k_end; k0 += SG_BK) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            int i, k;
            if (AF::k_contiguous) { k = t % 16; i = t / 16 + 16 * q; } else { i = t % 64; k = t / 64 + 4 * q; }
            int gi = i0 + i, gk = k0 + k;
            As[k][i] = (gi < M && gk < k_end && gk < K) ? A(z, gi, gk) : 0.f;
            int j;
            if (BF::k_contiguous) { k = t % 16; j = t / 16 + 16 * q; } else { j = t % 64; k = t / 64 + 4 * q; }
            int gj = j0 + j; gk = k0 + k;
            Bs[k][j] = (gj < N && gk < k_end && gk < K) ? B(z, gk, gj) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < SG_BK; ++k) {
            float av[4], bv[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) { av[q] = As[k][ty * 4 + q]; bv[q] = Bs[k][tx * 4 + q]; }
#pragma unroll
            for (int p = 0; p < 4; ++p)
#pragma unroll
                for (int q = 0; q < 4; ++q) acc[p][q] = fmaf(av[p], bv[q], acc[p][q]);
        }
        __syncthreads();
    }
}

template <class AF, class BF, class EF>
__global__ void __launch_bounds__(256) gemm_simt(int M, int N, int K, AF A, BF B, EF E) {
    __shared__ float As[SG_BK][SG_BM + 4];
    __shared__ float Bs[SG_BK][SG_BN + 4];
    const int z = blockIdx.z;
    const int i0 = blockIdx.y * SG_BM, j0 = blockIdx.x * SG_BN;
    const int t = threadIdx.x, ty = t / 16, tx = t % 16;
    float acc[4][4] = {};
    gemm_simt_tile(M, N, K, 0, K, A, B, z, i0, j0, acc, As, Bs);
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            int gi = i0 + ty * 4 + p, gj = j0 + tx * 4 + q;
            if (gi < M && gj < N) E(z, gi, gj, acc[p][q]);
        }
}

// The same product with the k range cut into gridDim.z slices (a multiple of 16 each) for shapes
// with few output tiles and a long reduction: slice s writes its partial sums to part[s][M][N];
// the caller adds the slices up in slice order (reduce_splits_kernel), so the result is still
// independent of timing.
template <class AF, class BF>
__global__ void __launch_bounds__(256) gemm_simt_ksplit(int M, int N, int K, int k_slice, AF A, BF B, float* __restrict__ part) {
    __shared__ float As[SG_BK][SG_BM + 4];
    __shared__ float Bs[SG_BK][SG_BN + 4];
    const int i0 = blockIdx.y * SG_BM, j0 = blockIdx.x * SG_BN;
    const int t = threadIdx.x, ty = t / 16, tx = t % 16;
    const int k_begin = blockIdx.z * k_slice, k_end = min(K, k_begin + k_slice);
    float acc[4][4] = {};
    gemm_simt_tile(M, N, K, k_begin, k_end, A, B, 0, i0, j0, acc, As, Bs);
    float* out = part + (long long)blockIdx.z * M * N;
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            int gi = i0 + ty * 4 + p, gj = j0 + tx * 4 + q;
            if (gi < M && gj < N) out[(long long)gi * N + gj] = acc[p][q];
        }
}

// Row i of the batch = token s of batch sample b; the element comes straight from the cache.
template <typename T>
struct CacheRows {            // A(z=l; i=row, k) = h_l[row][k]
    static constexpr bool k_contiguous = true;
    const T* cache; const int* ids; long long N; int L, S, d, layer0;
    __device__ float operator()(int z, int i, int k) const {
        int b = i / S, s = i - b * S;
        long long id = safe_id(ids, b, N, nullptr);
        return to_f32(cache[(((id * L) + (layer0 + z)) * S + s) * (long long)d + k]);
    }
};
template <typename T>
struct CacheRowsT {           // A(z=l; i=k_d, k=row) = h_l[row][k_d]   (for dW_down = h^T du)
    static constexpr bool k_contiguous = false;
    const T* cache; const int* ids; long long N; int L, S, d;
    __device__ float operator()(int z, int i, int k) const {
        int b = k / S, s = k - b * S;
        long long id = safe_id(ids, b, N, nullptr);
        return to_f32(cache[(((id * L) + z) * S + s) * (long long)d + i]);
    }
};
struct RowMajor {             // X(z; p, q) = base[z*zstride + p*ld + q]; q contiguous
    const float* base; long long zstride; int ld;
};
struct MatA_RowMajor : RowMajor {      // A(i,k) with k contiguous
    static constexpr bool k_contiguous = true;
    __device__ float operator()(int z, int i, int k) const { return base[z * zstride + (long long)i * ld + k]; }
};
struct MatA_ColMajor : RowMajor {      // A(i,k) = base[k*ld + i]  (transposed view)
    static constexpr bool k_contiguous = false;
    __device__ float operator()(int z, int i, int k) const { return base[z * zstride + (long long)k * ld + i]; }
};
struct MatB_RowMajor : RowMajor {      // B(k,j) with j contiguous
    static constexpr bool k_contiguous = false;
    __device__ float operator()(int z, int k, int j) const { return base[z * zstride + (long long)k * ld + j]; }
};
struct MatB_ColMajor : RowMajor {      // B(k,j) = base[j*ld + k]
    static constexpr bool k_contiguous = true;
    __device__ float operator()(int z, int k, int j) const { return base[z * zstride + (long long)j * ld + k]; }
};
struct MatB_Bf16Rows {                 // B(k,j) = W[j][k]   (logits = y W_lm^T)
    static constexpr bool k_contiguous = true;
    const bf16* W; int ld;
    __device__ float operator()(int, int k, int j) const { return to_f32(W[(long long)j * ld + k]); }
};
struct MatB_Bf16Cols {                 // B(k,j) = W[k][j]   (dy = dlogits W_lm)
    static constexpr bool k_contiguous = false;
    const bf16* W; int ld;
    __device__ float operator()(int, int k, int j) const { return to_f32(W[(long long)k * ld + j]); }
};
struct StoreRowMajor {
    float* out; long long zstride; int ld;
    __device__ void operator()(int z, int i, int j, float v) const { out[z * zstride + (long long)i * ld + j] = v; }
};
template <typename T>
struct StorePlusLastLayer {            // y = h_L + a_L W_up
    float* out; int ld; CacheRows<T> h;
    __device__ void operator()(int, int i, int j, float v) const { out[(long long)i * ld + j] = v + h(0, i, j); }
};

template <typename T>
struct StorePlusLastLayerBf16 {        // the same, rounded to bf16 (A operand of the tensor-core LM-head GEMM)
    bf16* out; int ld; CacheRows<T> h;
    __device__ void operator()(int, int i, int j, float v) const { out[(long long)i * ld + j] = __float2bfloat16(v + h(0, i, j)); }
};

// ---------------------------------------------------------------------------
// The lambda-merge / adapter-body chain over saved u (forward) and its reverse.
// One thread per (row, column) element e < n = M*r of the [M][r] state; layer l of a
// saved stack starts at l * lstride (lstride = max_rows * r, fixed per context).
// ---------------------------------------------------------------------------
template <int ACT>
__global__ void chain_fwd_kernel(const float* __restrict__ u, float* __restrict__ a, const float* __restrict__ lam,
                                 int L, long long n, long long lstride) {
    long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n) return;
    float prev = 0.f;                                   // a_0 = 0
    for (int l = 0; l < L; ++l) {
        float lm = lam[l];
        float z = lm * u[l * lstride + e] + (1.f - lm) * prev;
        prev = (ACT == PAC_ACT_RELU) ? (z > 0.f ? z : 0.f) : z;
        a[l * lstride + e] = prev;
    }
}

// pooled_a[b][j] = mean_s a_L[b][s][j]
__global__ void pool_tokens_kernel(const float* __restrict__ aL, float* __restrict__ pooled, int S, int r) {
    int b = blockIdx.x;
    for (int j = threadIdx.x; j < r; j += blockDim.x) {
        float acc = 0.f;
        for (int s = 0; s < S; ++s) acc += aL[((long long)b * S + s) * r + j];
        pooled[(long long)b * r + j] = acc / (float)S;
    }
}

// mean over tokens of the last cached layer of every sample: hbar[n][k]
template <typename T>
__global__ void pool_last_layer_kernel(const T* __restrict__ cache, float* __restrict__ hbar, int L, int S, int d) {
    long long n = blockIdx.x;
    const T* base = cache + ((n * L) + (L - 1)) * (long long)S * d;
    for (int k = threadIdx.x; k < d; k += blockDim.x) {
        float acc = 0.f;
        for (int s = 0; s < S; ++s) acc += to_f32(base[(long long)s * d + k]);
        hbar[n * d + k] = acc / (float)S;
    }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
// Block-wide sum with a fixed combination order (deterministic); red: >= 32 floats of smem.
__device__ __forceinline__ float block_sum(float v, float* red) {
    int w = threadIdx.x >> 5, ln = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (ln == 0) red[w] = v;
    __syncthreads();
    float t = (threadIdx.x < nw) ? red[threadIdx.x] : 0.f;
    if (w == 0) t = warp_sum(t);
    if (threadIdx.x == 0) red[0] = t;
    __syncthreads();
    t = red[0];
    return t;
}
__device__ __forceinline__ float block_max(float v, float* red) {
    int w = threadIdx.x >> 5, ln = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
    v = warp_max(v);
    __syncthreads();
    if (ln == 0) red[w] = v;
    __syncthreads();
    float t = (threadIdx.x < nw) ? red[threadIdx.x] : -INFINITY;
    if (w == 0) t = warp_max(t);
    if (threadIdx.x == 0) red[0] = t;
    __syncthreads();
    t = red[0];
    return t;
}

// ---------------------------------------------------------------------------
// Classifier head, one block per batch sample.  By linearity of the token mean,
//   mean_s y = hbar[id] + (mean_s a_L) W_up,
// so the head needs only per-sample vectors.  Writes logits; when train != 0 also the
// per-sample loss, dlogits = (softmax - onehot)/B, g = W_head dlogits (d loss / d mean_s y)
// and da_L (identical for every token of the sample) = W_up g / S.
// Dynamic shared memory: (d + C + 32) floats.
// ---------------------------------------------------------------------------
__global__ void cls_head_kernel(const float* __restrict__ hbar, const int* __restrict__ ids, long long N,
                                const int* __restrict__ labels, const float* __restrict__ pooled_a,
                                const float* __restrict__ W_up, const float* __restrict__ W_head,
                                const float* __restrict__ b_head, int B, int S, int d, int r, int C, int train,
                                float* __restrict__ pooled_y, float* __restrict__ logits_out,
                                float* __restrict__ loss_b, float* __restrict__ dlogits, float* __restrict__ gvec,
                                float* __restrict__ daL, unsigned* status) {
    extern __shared__ float sm[];
    float* py = sm;            // [d]   mean_s y, later g
    float* lg = sm + d;        // [C]
    float* red = lg + C;       // [32]
    const int b = blockIdx.x;
    const long long id = safe_id(ids, b, N, threadIdx.x == 0 ? status : nullptr);
    for (int k = threadIdx.x; k < d; k += blockDim.x) {
        float acc = 0.f;
        for (int j = 0; j < r; ++j) acc = fmaf(pooled_a[(long long)b * r + j], W_up[(long long)j * d + k], acc);
        float v = hbar[id * d + k] + acc;
        py[k] = v;
        if (train) pooled_y[(long long)b * d + k] = v;
    }
    __syncthreads();
    for (int c = 0; c < C; ++c) {
        float part = 0.f;
        for (int k = threadIdx.x; k < d; k += blockDim.x) part = fmaf(py[k], W_head[(long long)k * C + c], part);
        float tot = block_sum(part, red);
        if (threadIdx.x == 0) lg[c] = tot + b_head[c];
    }
    __syncthreads();
    for (int c = threadIdx.x; c < C; c += blockDim.x) logits_out[(long long)b * C + c] = lg[c];
    if (!train) return;
    float mx = -INFINITY;
    for (int c = 0; c < C; ++c) mx = fmaxf(mx, lg[c]);
    float se = 0.f;
    for (int c = 0; c < C; ++c) se += expf(lg[c] - mx);
    const int label = labels[id];
    if (threadIdx.x == 0) loss_b[b] = mx + logf(se) - lg[label];
    __syncthreads();
    for (int c = threadIdx.x; c < C; c += blockDim.x) {
        float p = expf(lg[c] - mx) / se;
        float g = (p - (c == label ? 1.f : 0.f)) / (float)B;
        lg[c] = g;
        dlogits[(long long)b * C + c] = g;
    }
    __syncthreads();
    for (int k = threadIdx.x; k < d; k += blockDim.x) {
        float acc = 0.f;
        for (int c = 0; c < C; ++c) acc = fmaf(W_head[(long long)k * C + c], lg[c], acc);
        py[k] = acc;
        gvec[(long long)b * d + k] = acc;
    }
    __syncthreads();
    const int w = threadIdx.x >> 5, ln = threadIdx.x & 31, nw = blockDim.x >> 5;
    for (int j = w; j < r; j += nw) {
        float part = 0.f;
        for (int k = ln; k < d; k += 32) part = fmaf(W_up[(long long)j * d + k], py[k], part);
        part = warp_sum(part);
        if (ln == 0) daL[(long long)b * r + j] = part / (float)S;
    }
}

// Gradients of the head-side parameters from the per-sample vectors, summed over the
// batch in sample order:  dW_up = pooled_a^T g,  dW_head = pooled_y^T dlogits,
// db_head = sum_b dlogits, and the mean loss.  One thread per output element.
__global__ void cls_grads_kernel(const float* __restrict__ pooled_a, const float* __restrict__ gvec,
                                 const float* __restrict__ pooled_y, const float* __restrict__ dlogits,
                                 const float* __restrict__ loss_b, int B, int d, int r, int C,
                                 float* __restrict__ gW_up, float* __restrict__ gW_head,
                                 float* __restrict__ gb_head, float* __restrict__ loss_out) {
    long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long n_up = (long long)r * d, n_head = (long long)d * C;
    if (e < n_up) {
        int j = e / d, k = e - (long long)j * d;
        float acc = 0.f;
        for (int b = 0; b < B; ++b) acc = fmaf(pooled_a[(long long)b * r + j], gvec[(long long)b * d + k], acc);
        gW_up[e] = acc;
    } else if (e < n_up + n_head) {
        long long q = e - n_up;
        int k = q / C, c = q - (long long)k * C;
        float acc = 0.f;
        for (int b = 0; b < B; ++b) acc = fmaf(pooled_y[(long long)b * d + k], dlogits[(long long)b * C + c], acc);
        gW_head[q] = acc;
    } else if (e < n_up + n_head + C) {
        int c = e - n_up - n_head;
        float acc = 0.f;
        for (int b = 0; b < B; ++b) acc += dlogits[(long long)b * C + c];
        gb_head[c] = acc;
    } else if (e == n_up + n_head + C) {
        float acc = 0.f;
        for (int b = 0; b < B; ++b) acc += loss_b[b];
        *loss_out = acc / (float)B;
    }
}

// ---------------------------------------------------------------------------
// Reverse chain.  da_L comes either per sample (classifier: the same vector for every
// token, daL[b][j]) or per row (LM head: daL[m][j]).  For l = L..1:
//   dz = da * phi'(z_l)   (ReLU: z_l > 0 <=> a_l > 0),  dlambda_l += dz (u_l - a_{l-1}),
//   du_l = lambda_l dz,  da = (1 - lambda_l) dz.
// du is stored in DU (float or bf16).  dlambda: per-block partials, reduced afterwards
// in block order.  blockDim = 256.
// ---------------------------------------------------------------------------
template <int ACT, typename DU>
__global__ void __launch_bounds__(256) chain_bwd_kernel(const float* __restrict__ u, const float* __restrict__ a,
                                                        const float* __restrict__ lam,
                                                        const float* __restrict__ daL, int per_sample, int S,
                                                        int r, int L, long long n, long long stride,
                                                        DU* __restrict__ du, float* __restrict__ lam_part) {
    __shared__ float red[32];
    long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const bool live = e < n;
    float da = 0.f;
    if (live) {
        if (per_sample) {
            long long m = e / r;
            int j = e - m * r;
            da = daL[(m / S) * r + j];
        } else {
            da = daL[e];
        }
    }
    float a_l = live ? a[(long long)(L - 1) * stride + e] : 0.f;
    for (int l = L - 1; l >= 0; --l) {
        float lm = lam[l];
        float a_prev = (live && l > 0) ? a[(long long)(l - 1) * stride + e] : 0.f;
        float dz = (ACT == PAC_ACT_RELU) ? (a_l > 0.f ? da : 0.f) : da;
        float part = live ? dz * (u[(long long)l * stride + e] - a_prev) : 0.f;
        if (live) {
            float v = lm * dz;
            if constexpr (sizeof(DU) == 2) du[(long long)l * stride + e] = __float2bfloat16(v);
            else du[(long long)l * stride + e] = v;
        }
        da = (1.f - lm) * dz;
        a_l = a_prev;
        float tot = block_sum(part, red);
        if (threadIdx.x == 0) lam_part[(long long)l * gridDim.x + blockIdx.x] = tot;
    }
}

// out[l] = sum over blocks of part[l][*], in block order.
__global__ void reduce_rows_kernel(const float* __restrict__ part, int n, float* __restrict__ out) {
    __shared__ float red[32];
    int l = blockIdx.x;
    float acc = 0.f;
    for (int i = threadIdx.x; i < n; i += blockDim.x) acc += part[(long long)l * n + i];
    float tot = block_sum(acc, red);
    if (threadIdx.x == 0) out[l] = tot;
}

// ---------------------------------------------------------------------------
// LM head cross-entropy, one block per row of logits [M][V]: loss_row = logsumexp -
// logit[target]; when train != 0 the row is overwritten by (softmax - onehot)/M, or, when
// dlog16 is given, that gradient goes to dlog16 [M][V] in bf16 instead (A operand of dy = dlogits W_lm).
// ---------------------------------------------------------------------------
__global__ void lm_ce_kernel(float* __restrict__ logits, const int* __restrict__ ids, long long N,
                             const int* __restrict__ targets, int S, int V, int M, int train,
                             float* __restrict__ loss_row, unsigned* status, bf16* __restrict__ dlog16) {
    __shared__ float red[32];
    const int m = blockIdx.x;
    float* row = logits + (long long)m * V;
    float mx = -INFINITY;
    for (int v = threadIdx.x; v < V; v += blockDim.x) mx = fmaxf(mx, row[v]);
    mx = block_max(mx, red);
    float se = 0.f;
    for (int v = threadIdx.x; v < V; v += blockDim.x) se += expf(row[v] - mx);
    se = block_sum(se, red);
    const int b = m / S, s = m - b * S;
    const long long id = safe_id(ids, b, N, (threadIdx.x == 0 && s == 0) ? status : nullptr);
    const int tgt = targets[id * S + s];
    if (threadIdx.x == 0) loss_row[m] = mx + logf(se) - row[tgt];
    if (!train) return;
    __syncthreads();
    const float inv = 1.f / se, invM = 1.f / (float)M;
    if (dlog16) {
        bf16* out = dlog16 + (long long)m * V;
        for (int v = threadIdx.x; v < V; v += blockDim.x)
            out[v] = __float2bfloat16((expf(row[v] - mx) * inv - (v == tgt ? 1.f : 0.f)) * invM);
    } else {
        for (int v = threadIdx.x; v < V; v += blockDim.x) row[v] = (expf(row[v] - mx) * inv - (v == tgt ? 1.f : 0.f)) * invM;
    }
}

// mean of n values in index order (single block).
__global__ void mean_kernel(const float* __restrict__ x, int n, float* __restrict__ out) {
    __shared__ float red[32];
    float acc = 0.f;
    for (int i = threadIdx.x; i < n; i += blockDim.x) acc += x[i];
    float tot = block_sum(acc, red);
    if (threadIdx.x == 0) *out = tot / (float)n;
}

// ---------------------------------------------------------------------------
// Fused AdamW over the flat parameter vector (decoupled decay on the weight matrices
// only).  bc1 = 1-beta1^t, bc2 = 1-beta2^t (bias corrections, computed on the host in double).  Also refreshes the bf16
// hi/lo shadow of W_down ([L][2][d][r]) that the tensor-core path multiplies with.
// ---------------------------------------------------------------------------
// One element of the update, shared by every kernel that applies AdamW so that fused and
// separate updates are bit-identical.
// The arithmetic of one element: returns the new parameter, updates mi / vi in place.
__device__ __forceinline__ float adamw_math(float th, float& mi, float& vi, float gi, bool decays, const pac_adamw& hp,
                                            float bc1, float bc2) {
    // every rounding is spelled out (no contraction into FMAs), in the order the update is written:
    // m = b1 m + (1-b1) g;  v = b2 v + ((1-b2) g) g;  theta = (theta - lr wd theta) - (lr mhat)/(sqrt(vhat)+eps)
    mi = __fadd_rn(__fmul_rn(hp.beta1, mi), __fmul_rn(__fsub_rn(1.f, hp.beta1), gi));
    vi = __fadd_rn(__fmul_rn(hp.beta2, vi), __fmul_rn(__fmul_rn(__fsub_rn(1.f, hp.beta2), gi), gi));
    const float mhat = __fdiv_rn(mi, bc1), vhat = __fdiv_rn(vi, bc2);
    const float decay = decays ? __fmul_rn(__fmul_rn(hp.lr, hp.weight_decay), th) : 0.f;
    return __fsub_rn(__fsub_rn(th, decay), __fdiv_rn(__fmul_rn(hp.lr, mhat), __fadd_rn(__fsqrt_rn(vhat), hp.eps)));
}

__device__ __forceinline__ void adamw_element(float* __restrict__ p, float* __restrict__ m, float* __restrict__ v,
                                              long long i, float gi, const ParamLayout& lay, const pac_adamw& hp,
                                              float bc1, float bc2, bf16* __restrict__ wdT, int d, int r) {
    const bool decays = lay.decays(i);
    float mi = m[i], vi = v[i];
    const float th = adamw_math(p[i], mi, vi, gi, decays, hp, bc1, bc2);
    m[i] = mi;
    v[i] = vi;
    p[i] = th;
    if (wdT && i < lay.lam) {
        const long long dr = (long long)d * r, l = i / dr, rem = i - l * dr;
        const bf16 hi = __float2bfloat16(th);
        wdT[(l * 2 + 0) * dr + rem] = hi;
        wdT[(l * 2 + 1) * dr + rem] = __float2bfloat16(th - __bfloat162float(hi));
    }
}

// Four consecutive elements of the W_down block (i a multiple of 4; d*r is a multiple of 4, so
// the four share a layer): vector loads and stores, the same arithmetic per element.
// The same with the old parameter and moments already in registers (a caller may fetch them early).
__device__ __forceinline__ void adamw_w_down4_loaded(float* __restrict__ p, float* __restrict__ m, float* __restrict__ v,
                                                     long long i, float4 p4, float4 m4, float4 v4, float4 g4, const pac_adamw& hp,
                                                     float bc1, float bc2, bf16* __restrict__ wdT, int d, int r);
__device__ __forceinline__ void adamw_w_down4(float* __restrict__ p, float* __restrict__ m, float* __restrict__ v,
                                              long long i, float4 g4, const pac_adamw& hp, float bc1, float bc2,
                                              bf16* __restrict__ wdT, int d, int r) {
    const float4 p4 = *reinterpret_cast<float4*>(p + i), m4 = *reinterpret_cast<float4*>(m + i), v4 = *reinterpret_cast<float4*>(v + i);
    adamw_w_down4_loaded(p, m, v, i, p4, m4, v4, g4, hp, bc1, bc2, wdT, d, r);
}
__device__ __forceinline__ void adamw_w_down4_loaded(float* __restrict__ p, float* __restrict__ m, float* __restrict__ v,
                                                     long long i, float4 p4, float4 m4, float4 v4, float4 g4, const pac_adamw& hp,
                                                     float bc1, float bc2, bf16* __restrict__ wdT, int d, int r) {
    p4.x = adamw_math(p4.x, m4.x, v4.x, g4.x, true, hp, bc1, bc2);
    p4.y = adamw_math(p4.y, m4.y, v4.y, g4.y, true, hp, bc1, bc2);
    p4.z = adamw_math(p4.z, m4.z, v4.z, g4.z, true, hp, bc1, bc2);
    p4.w = adamw_math(p4.w, m4.w, v4.w, g4.w, true, hp, bc1, bc2);
    *reinterpret_cast<float4*>(p + i) = p4;
    *reinterpret_cast<float4*>(m + i) = m4;
    *reinterpret_cast<float4*>(v + i) = v4;
    if (wdT) {
        const long long dr = (long long)d * r, l = i / dr, rem = i - l * dr;
        const float th[4] = {p4.x, p4.y, p4.z, p4.w};
        bf16 hi[4], lo[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            hi[e] = __float2bfloat16(th[e]);
            lo[e] = __float2bfloat16(th[e] - __bfloat162float(hi[e]));
        }
        *reinterpret_cast<uint2*>(wdT + (l * 2 + 0) * dr + rem) = *reinterpret_cast<const uint2*>(hi);
        *reinterpret_cast<uint2*>(wdT + (l * 2 + 1) * dr + rem) = *reinterpret_cast<const uint2*>(lo);
    }
}

// wd_blocks leading blocks take the W_down block four elements per thread (0 when its size is
// not a multiple of 4); the remaining blocks take everything else one element per thread.
// grad_scale multiplies every gradient on its way into the update (1 for a single device; 1/world
// when the gradient buffer holds the SUM over data-parallel ranks); the buffer itself is not changed.
__global__ void adamw_kernel(float* __restrict__ p, const float* __restrict__ g, float* __restrict__ m,
                             float* __restrict__ v, long long n, ParamLayout lay, pac_adamw hp, float bc1,
                             float bc2, bf16* __restrict__ wdT, int d, int r, int wd_blocks, unsigned* status,
                             float grad_scale) {
    // gradients computed after a bounded wait ran out are not trustworthy: leave the state alone
    if (status_timed_out(status)) {
        if (blockIdx.x == 0 && threadIdx.x == 0) atomicAdd(&status[ST_SKIPPED_STEPS], 1u);
        return;
    }
    if ((int)blockIdx.x < wd_blocks) {
        const long long i = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 4;
        if (i < lay.lam) {
            float4 g4 = *reinterpret_cast<const float4*>(g + i);
            g4.x *= grad_scale; g4.y *= grad_scale; g4.z *= grad_scale; g4.w *= grad_scale;
            adamw_w_down4(p, m, v, i, g4, hp, bc1, bc2, wdT, d, r);
        }
        return;
    }
    const long long i = (wd_blocks ? lay.lam : 0) + (long long)(blockIdx.x - wd_blocks) * blockDim.x + threadIdx.x;
    if (i >= n) return;
    adamw_element(p, m, v, i, g[i] * grad_scale, lay, hp, bc1, bc2, wdT, d, r);
}

// bf16 hi/lo shadow of W_down from the fp32 master, same [d][r] order:
// wdT[l][0][k][j] = bf16(W_down[l][k][j]), wdT[l][1][k][j] = bf16(W_down[l][k][j] - hi).
__global__ void shadow_wdown_kernel(const float* __restrict__ w, bf16* __restrict__ wdT, int L, int d, int r) {
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)L * d * r) return;
    long long l = i / ((long long)d * r), rem = i - l * (long long)d * r;
    const bf16 hi = __float2bfloat16(w[i]);
    wdT[(l * 2 + 0) * (long long)d * r + rem] = hi;
    wdT[(l * 2 + 1) * (long long)d * r + rem] = __float2bfloat16(w[i] - __bfloat162float(hi));
}

}  // namespace pac
