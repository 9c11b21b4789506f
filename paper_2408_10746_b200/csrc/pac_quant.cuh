// Block-wise absmax INT8 quantisation and dequantisation (paper Section IV-D, Eq. 1-2):
//   c = 127 / absmax(block),  code = round(c * x)  (ties to even),  dequant = code / c,
// every block of `block` consecutive elements on its own; an all-zero block has c = 0.
// All arithmetic in fp32 with explicitly rounded operations, so the integer codes are the same
// on every implementation that follows the equations in fp32.  Both kernels stream: 5 bytes per
// element (4 read + 1 written, or the reverse).
#pragma once
#include "pac_common.cuh"

namespace pac {

// One warp per quantisation block (block <= QUANT_WARP_MAX), several blocks per CTA.
constexpr int QUANT_WARP_MAX = 4096;

__global__ void __launch_bounds__(256) quantize_absmax_warp_kernel(const float* __restrict__ x, long long n, int block,
                                                                   long long n_blocks, signed char* __restrict__ q,
                                                                   float* __restrict__ c) {
    const int lane = threadIdx.x & 31;
    const long long wid = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5, nw = ((long long)gridDim.x * blockDim.x) >> 5;
    for (long long j = wid; j < n_blocks; j += nw) {
        const long long i0 = j * block;
        const int len = (int)((n - i0) < block ? (n - i0) : block);
        float amax = 0.f;
        for (int i = lane; i < len; i += 32) amax = fmaxf(amax, fabsf(x[i0 + i]));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        const float cj = amax > 0.f ? __fdiv_rn(127.f, amax) : 0.f;
        if (lane == 0) c[j] = cj;
        for (int i = lane; i < len; i += 32)                        // second read comes from L1/L2
            q[i0 + i] = (signed char)__float2int_rn(__fmul_rn(cj, x[i0 + i]));
    }
}

// One CTA per quantisation block (large blocks).
__global__ void __launch_bounds__(256) quantize_absmax_cta_kernel(const float* __restrict__ x, long long n, int block,
                                                                  signed char* __restrict__ q, float* __restrict__ c) {
    __shared__ float red[8];
    __shared__ float c_sh;
    const long long j = blockIdx.x, i0 = j * block;
    const int len = (int)((n - i0) < block ? (n - i0) : block);
    float amax = 0.f;
    for (int i = threadIdx.x; i < len; i += blockDim.x) amax = fmaxf(amax, fabsf(x[i0 + i]));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
    __syncthreads();
    if (threadIdx.x == 0) {
        float m = 0.f;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) m = fmaxf(m, red[w]);
        c_sh = m > 0.f ? __fdiv_rn(127.f, m) : 0.f;
        c[j] = c_sh;
    }
    __syncthreads();
    const float cj = c_sh;
    for (int i = threadIdx.x; i < len; i += blockDim.x) q[i0 + i] = (signed char)__float2int_rn(__fmul_rn(cj, x[i0 + i]));
}

__device__ __forceinline__ float absmax4(float4 v) { return fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))); }
__device__ __forceinline__ char4 quant4(float4 v, float cj) {
    return make_char4((signed char)__float2int_rn(__fmul_rn(cj, v.x)), (signed char)__float2int_rn(__fmul_rn(cj, v.y)),
                      (signed char)__float2int_rn(__fmul_rn(cj, v.z)), (signed char)__float2int_rn(__fmul_rn(cj, v.w)));
}

// Single pass, block in {16, 32, 64, 128} and n a multiple of 4: block/4 lanes share one
// quantisation block, every lane keeps its four values in registers between absmax and rounding.
__global__ void __launch_bounds__(256) quantize_absmax_subwarp_kernel(const float4* __restrict__ x4, long long n4, int lanes,
                                                                      char4* __restrict__ q4, float* __restrict__ c) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    const long long n4_pad = (n4 + 31) & ~31LL;                  // whole warps stay together for the shuffles
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4_pad; i += stride) {
        const bool live = i < n4;
        const float4 v = live ? x4[i] : make_float4(0.f, 0.f, 0.f, 0.f);
        float amax = absmax4(v);
        for (int o = lanes >> 1; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        const float cj = amax > 0.f ? __fdiv_rn(127.f, amax) : 0.f;
        if (live) {
            q4[i] = quant4(v, cj);
            if ((i & (lanes - 1)) == 0) c[i / lanes] = cj;
        }
    }
}

// Single pass, one CTA of 256 threads per block, block = 1024 * K (K <= 4), n a multiple of 4.
template <int K>
__global__ void __launch_bounds__(256) quantize_absmax_cta_reg_kernel(const float4* __restrict__ x4, long long n4,
                                                                      char4* __restrict__ q4, float* __restrict__ c) {
    __shared__ float red[8];
    __shared__ float c_sh;
    const long long base = (long long)blockIdx.x * (256 * K);
    float4 v[K];
    float amax = 0.f;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const long long i = base + k * 256 + threadIdx.x;
        v[k] = i < n4 ? x4[i] : make_float4(0.f, 0.f, 0.f, 0.f);
        amax = fmaxf(amax, absmax4(v[k]));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
    __syncthreads();
    if (threadIdx.x == 0) {
        float m = 0.f;
        for (int w = 0; w < 8; ++w) m = fmaxf(m, red[w]);
        c_sh = m > 0.f ? __fdiv_rn(127.f, m) : 0.f;
        c[blockIdx.x] = c_sh;
    }
    __syncthreads();
    const float cj = c_sh;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const long long i = base + k * 256 + threadIdx.x;
        if (i < n4) q4[i] = quant4(v[k], cj);
    }
}

// Four codes per lane (block and n multiples of 4): a warp reads 128 contiguous bytes and writes
// 512 contiguous bytes per instruction; four independent iterations per thread are in flight.
__global__ void __launch_bounds__(256) dequantize_absmax_vec_kernel(const char4* __restrict__ q4, const float* __restrict__ c,
                                                                    long long n4, int block4, float4* __restrict__ out4) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x; i0 < n4; i0 += 4 * stride) {
        char4 b[4];
        float cj[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const long long i = i0 + k * stride;
            if (i < n4) { b[k] = q4[i]; cj[k] = c[i / block4]; }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const long long i = i0 + k * stride;
            if (i < n4) {
                float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
                if (cj[k] != 0.f)
                    o = make_float4(__fdiv_rn((float)b[k].x, cj[k]), __fdiv_rn((float)b[k].y, cj[k]), __fdiv_rn((float)b[k].z, cj[k]),
                                    __fdiv_rn((float)b[k].w, cj[k]));
                out4[i] = o;
            }
        }
    }
}

__global__ void __launch_bounds__(256) dequantize_absmax_kernel(const signed char* __restrict__ q, const float* __restrict__ c,
                                                                long long n, int block, float* __restrict__ out) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        const float cj = c[i / block];
        out[i] = cj != 0.f ? __fdiv_rn((float)q[i], cj) : 0.f;
    }
}

}  // namespace pac
