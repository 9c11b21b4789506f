// Shared device helpers and the context structure of the adapter-over-cache trainer.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cstdint>
#include <cstdio>
#include <map>
#include <mutex>
#include <string>
#include <utility>

#include "pac.h"

namespace pac {

typedef __nv_bfloat16 bf16;

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(bf16 x) { return __bfloat162float(x); }

// Device-side status words (one small array per context).
// ST_SKIPPED_STEPS: optimizer updates that were left out because ST_TIMEOUT was already set when they ran.
enum { ST_CLAMPED_IDS = 0, ST_TIMEOUT = 1, ST_SKIPPED_STEPS = 2, ST_WORDS = 4 };
__device__ __forceinline__ bool status_timed_out(const unsigned* status) {
    return status && *reinterpret_cast<const volatile unsigned*>(status + ST_TIMEOUT) != 0u;
}

// Sample id of batch row b, clamped into [0, N) so that no kernel can read outside
// the cache even if a device-resident id is bad; clamps are counted.
__device__ __forceinline__ long long safe_id(const int* __restrict__ ids, int b, long long N, unsigned* status) {
    long long id = ids[b];
    if (id < 0 || id >= N) {
        if (status) atomicAdd(&status[ST_CLAMPED_IDS], 1u);
        id = id < 0 ? 0 : N - 1;
    }
    return id;
}

// Dynamic shared memory above 48 KB needs an opt-in per kernel, and the attribute belongs to the
// device the call is made on.  Several contexts (other shapes, other devices) share the kernels, so
// the largest size granted so far is kept per (device, kernel) and never lowered.
inline cudaError_t smem_opt_in(const void* kernel, size_t bytes) {
    static std::mutex mu;
    static std::map<std::pair<int, const void*>, size_t> granted;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    size_t& g = granted[std::make_pair(dev, kernel)];
    if (bytes <= g) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess) g = bytes;
    return e;
}

struct Dims {
    long long N;   // samples in the cache
    int L, S, d;   // layers, tokens, hidden width
    int r;         // adapter width
    int C;         // classes or vocabulary
};

// Offsets of the flat fp32 parameter vector:
// W_down[L][d][r] | lambda[L] | W_up[r][d] | W_head[d][C] | b_head[C]
// With transformer-body adapters the per-layer body blocks follow, layer after layer:
// ... | body[0] | body[1] | ... | body[L-1],  body[l] = g1 | b1 | Wq | Wk | Wv | Wo | g2 | b2 | W1 | c1 | W2 | c2
struct ParamLayout {
    long long w_down, lam, w_up, w_head, b_head, total;
    long long body, body_per;        // first body block and floats per block (body_per == 0: point-wise adapters)
    int br, bf;                      // adapter width and FFN width of the body blocks
    __host__ __device__ static ParamLayout make(int L, int d, int r, int C, bool cls) {
        ParamLayout p;
        p.w_down = 0;
        p.lam = (long long)L * d * r;
        p.w_up = p.lam + L;
        p.w_head = p.w_up + (long long)r * d;
        p.b_head = p.w_head + (cls ? (long long)d * C : 0);
        p.total = p.b_head + (cls ? C : 0);
        p.body = p.total; p.body_per = 0; p.br = r; p.bf = 0;
        return p;
    }
    // decoupled weight decay: the weight matrices, not lambda, biases or LayerNorm parameters
    __host__ __device__ bool decays(long long i) const {
        if (i < lam) return true;
        if (i < body) return i >= w_up && i < b_head;
        const long long off = (i - body) % body_per, rr = (long long)br * br, rf = (long long)br * bf;
        const long long wq = 2LL * br, g2 = wq + 4 * rr, w1 = g2 + 2LL * br, c1 = w1 + rf, w2 = c1 + bf, c2 = w2 + rf;
        return (off >= wq && off < g2) || (off >= w1 && off < c1) || (off >= w2 && off < c2);
    }
};

}  // namespace pac
