// Tensor-core path for bf16 caches on sm_100a: the two passes over the cached
// activations, written with TMA (cp.async.bulk.tensor) loads, tcgen05.mma and TMEM
// accumulators.
//
//   down-projection (Section IV-A):  u_l = h_l W_down^l        for every layer l and row tile
//   its weight gradient:             dW_down^l = h_l^T du_l    (reduction over all B*S rows)
//
// The cache gather (Section IV-B) is fused into the loads: a tile's TMA coordinates are
// (column, token, layer, sample id), so gathered activations are never materialised.
// Both kernels are bound by the HBM stream of the cache; the tensor cores are the means
// to keep up with it (about r flop per cached byte and pass).
//
// Every wait on an mbarrier is bounded: when a limit runs out the CTA records
// ST_TIMEOUT in the context's status words, stops issuing work, releases its TMEM and
// returns, so a broken pipeline shows up as PAC_ERR_TIMEOUT instead of a hang.
#pragma once
#include <cuda.h>
#include <cmath>

#include "pac_common.cuh"

namespace pac {

// ---------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------
// One 32-byte store (a whole L2 sector) from two 16-byte halves; p must be 32-byte aligned.
__device__ __forceinline__ void st_global_32(void* p, uint4 a, uint4 b) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"l"(p), "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w) : "memory");
}
// Programmatic dependent launch: a kernel launched with the programmatic-serialization
// attribute may start while its predecessor in the stream is still running; pdl_wait() blocks
// until the predecessor grid has completed and its writes are visible, pdl_trigger() lets the
// successor start launching.  Without the attribute both are no-ops.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// The address, in the cluster's shared-memory window, of this CTA's location `addr` in the CTA of rank `rank`.
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank) {
    uint32_t out;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(out) : "r"(addr), "r"(rank));
    return out;
}
// Bulk copy from this CTA's shared memory into the shared memory of a CTA of this cluster (its own included);
// the mbarrier, which lies in the destination CTA, is credited with the bytes once they are visible there.
// dst and bar from mapa_shared; addresses and size multiples of 16 bytes; the source must have been made
// visible to the copy engine (fence_proxy_async) by its writers.
__device__ __forceinline__ void dsmem_bulk_copy(uint32_t dst_cluster, uint32_t src_cta, uint32_t bytes, uint32_t bar_cluster) {
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_cluster), "r"(src_cta), "r"(bytes), "r"(bar_cluster) : "memory");
}
// One arrival at an mbarrier of a CTA of this cluster (address from mapa_shared).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait (about one second of wall time).  Returns false when the limit ran out or
// another role of this CTA gave up; the caller then stops issuing work.
constexpr unsigned long long WAIT_LIMIT_NS = 1000000000ull;
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned* status,
                                            unsigned long long limit_ns) {
    const unsigned long long t0 = global_ns();
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 63u) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > limit_ns) break;
        }
    }
    *abort_flag = 1;
    if (status) atomicAdd(&status[ST_TIMEOUT], 1u);
    return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned* status,
                                          unsigned long long limit_ns = WAIT_LIMIT_NS) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag, status, limit_ns);
}
// The same for a whole warp: lane 0 waits, every lane gets the same answer.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned* status,
                                               unsigned long long limit_ns = WAIT_LIMIT_NS) {
    int ok = 1;
    if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity, abort_flag, status, limit_ns) ? 1 : 0;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    return ok != 0;
}
// The same with every lane of a converged warp waiting; all lanes get the same answer.  Loops that
// issue TMA copies or MMAs are run by the whole warp with one elected lane issuing, so that
// addresses and descriptors stay warp-uniform values for the compiler.
__device__ __forceinline__ bool mbar_wait_uniform(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned* status) {
    const bool ok = mbar_wait(bar, parity, abort_flag, status);
    return __all_sync(0xffffffffu, ok) != 0;
}
// True in exactly one lane of a converged warp.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n .reg .pred p;\n elect.sync _|p, 0xffffffff;\n selp.u32 %0, 1, 0, p;\n}" : "=r"(pred));
    return pred != 0;
}
// Optional device-side timing of a pass's stream phase: stamp[0] receives the earliest first-copy
// time over the grid's CTAs, stamp[1] the latest accumulator-complete time (%globaltimer, ns).
// The host presets {all ones, 0}.  Unlike event brackets this leaves the launch overlap between the
// kernels of a step untouched.
__device__ __forceinline__ void stamp_begin(unsigned long long* stamp) {
    if (stamp) atomicMin(&stamp[0], global_ns());
}
__device__ __forceinline__ void stamp_end(unsigned long long* stamp) {
    if (stamp) atomicMax(&stamp[1], global_ns());
}
// After a wait gave up: give copies that are still in flight time to land before the CTA ends.
__device__ __forceinline__ void drain_after_abort(volatile int* abort_flag) {
    if (*abort_flag)
        for (int i = 0; i < 100; ++i) __nanosleep(1000);
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
// The same with an L2 eviction-priority hint (a policy word from createpolicy).
__device__ __forceinline__ void tma_load_4d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3,
                                                 uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy) : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem], bf16 operands, fp32 accumulate, issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// The mbarrier receives one arrival once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// ---- CTA pairs (cta_group::2): the two CTAs of a 2-CTA cluster run ONE MMA of M = 256: each holds its own 128
// rows of A and HALF of B's columns in its shared memory and receives its 128 rows of D in its own TMEM, so a
// weight tile crosses from L2 to the pair once instead of twice.  The CTA of rank 0 issues the MMAs. ----
// Executed by the same warp index in both CTAs.
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// Descriptors name shared-memory offsets that are valid in both CTAs of the pair.
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// One arrival at the mbarrier at this shared-memory offset in every CTA of cta_mask, once every MMA issued so far has completed.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar, uint16_t cta_mask) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(cta_mask) : "memory");
}
// Tile load whose bytes are counted on an mbarrier of either CTA of the pair (bar_cluster from mapa_shared).
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_load_4d_pair_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster, int c0, int c1, int c2,
                                                      int c3, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
        ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy) : "memory");
}

// 32 TMEM lanes (this warp's quadrant) x 32 consecutive fp32 columns -> 32 registers per thread.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Self-test of the bounded-wait discipline: one CTA allocates TMEM like the pipeline kernels, waits
// on an mbarrier that nobody will ever arrive at, and, once limit_ns have passed, leaves exactly the
// way the pipeline kernels leave after an abort (status word, abort flag, drain, TMEM release).
// result[0] = 1 if the wait reported expiry, result[1] = the abort flag.
__global__ void __launch_bounds__(64, 1) selftest_wait_expiry_kernel(unsigned* status, unsigned long long limit_ns, unsigned* result) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        abort_sh = 0;
        mbar_init(smem_u32(&bar), 1);
        fence_mbar_init();
    }
    if (warp == 1) { tmem_alloc(smem_u32(&tmem_base_sh), 32u); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    volatile int* abort_flag = &abort_sh;
    if (warp == 0) {
        const bool ok = mbar_wait_warp(smem_u32(&bar), 0, abort_flag, status, limit_ns);
        if (threadIdx.x == 0) result[0] = ok ? 0u : 1u;
    }
    tc_fence_before();
    __syncthreads();
    drain_after_abort(abort_flag);
    if (threadIdx.x == 0) result[1] = (unsigned)abort_sh;
    if (warp == 1) tmem_dealloc(tmem_base_sh, 32u);
}

// Shared-memory matrix descriptor for tcgen05.mma, 128-byte swizzle.
//   bits [0,14) start address >> 4, [16,30) leading byte offset >> 4, [32,46) stride byte
//   offset >> 4, [46,48) descriptor version 1, [61,64) layout type 2 (128-byte swizzle).
// K-major operand (rows of 64 bf16 = 128 B, 8-row groups 1024 B apart): SBO = 1024.
// MN-major operand (each K index is a 128-byte row of 64 MN elements; 8 such rows form a
// 1024-byte group): SBO = 1024 between K groups, LBO = distance between 64-element MN blocks.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}
// Instruction descriptor, kind::f16: D fp32 (bit 4), A and B bf16 (bits 7, 10), operand majors
// (bits 15, 16; 0 = K-major, 1 = MN-major), N >> 3 at bit 17, M >> 4 at bit 24.
__host__ __device__ constexpr uint32_t instr_desc_bf16(int M, int N, int a_mn_major, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

constexpr int TC_THREADS = 192;            // warp 0: TMA producer, warp 1: MMA issuer, warps 2-5: epilogue
constexpr int DW_THREADS = 320;            // dW_down: two epilogue warps per TMEM lane quadrant (warps 2-9)
constexpr int KC = 64;                     // bf16 elements per 128-byte swizzled row
constexpr int FWD_ROWS = 128;              // token rows per forward tile (MMA M)
constexpr int BWD_KR = 64;                 // token rows per backward stage (MMA K extent per stage)

struct FwdParams {
    const int* ids; long long N;
    int L, S, d, r, B;
    int s_chunks;                          // ceil(S / FWD_ROWS)
    int k_chunks;                          // ceil(d / KC)
    int stages;
    int tmem_cols;                         // power of two >= 2 * r_pad
    int acc_stride;                        // column offset of the second accumulator
    int wide_n;                            // 1: hi and lo blocks form one N = 128*r_blocks MMA, summed in the epilogue
    float* u; long long layer_stride;      // u[l][m][j], layer_stride = max_rows * r
    unsigned* status;
    unsigned long long* stamp;             // optional stream-phase timestamps (see stamp_begin)
};

// ---------------------------------------------------------------------------
// u_l = h_l W_down^l.  A tile: 128 tokens of one (sample, layer) x 64 columns, K-major,
// straight from the cache.  B tile: 64 rows of W_down^l in its natural [d][r] order (an
// MN-major operand), split into two bf16 terms (hi = bf16(W), lo = bf16(W - hi); shadow
// [L][2][d][r]); both products accumulate into the same fp32 accumulator, so the weights
// enter with about 16 mantissa bits.  (With bf16-rounded weights alone the ReLU masks of about one element in a
// thousand flip, which alone costs ~3% relative error in dW_down and dlambda.)
// Persistent CTAs walk tiles (layer, sample, token chunk); accumulators are double-buffered
// in TMEM so the epilogue of one tile overlaps the loads and MMAs of the next.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(TC_THREADS, 1)
down_fwd_tc_kernel(const __grid_constant__ CUtensorMap map_cache, const __grid_constant__ CUtensorMap map_w, FwdParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int r_pad = (p.r + 7) & ~7;
    const int r_blocks = (p.r + 63) >> 6;
    const uint32_t a_bytes = FWD_ROWS * KC * 2, b_box = KC * 128;            // one [64 k][64 columns of r] box
    const uint32_t b_bytes = (uint32_t)r_blocks * 2 * b_box;                 // [r block][hi|lo][64 k][128 B]
    const uint32_t b_off = a_bytes, stage_bytes = a_bytes + b_bytes;
    __shared__ __align__(8) unsigned long long bars[2 * 16 + 4];
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[16]);
    const uint32_t accf0 = smem_u32(&bars[32]), acce0 = smem_u32(&bars[34]);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = p.L * p.B * p.s_chunks;

    if (threadIdx.x == 0) {
        abort_sh = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(accf0 + 8 * b, 1); mbar_init(acce0 + 8 * b, 4); }
        fence_mbar_init();
        tma_prefetch_desc(&map_cache);
        tma_prefetch_desc(&map_w);
    }
    if (warp == 1) { tmem_alloc(smem_u32(&tmem_base_sh), (uint32_t)p.tmem_cols); tmem_relinquish(); }
    pdl_trigger();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_sh;
    volatile int* abort_flag = &abort_sh;
    pdl_wait();            // everything above overlapped the previous kernel; its results are needed from here on

    // The two pipeline loops are run by whole converged warps with one elected lane issuing, so that
    // addresses, coordinates and descriptors stay warp-uniform values.
    // Both pipeline loops carry ring positions, parities, addresses and descriptors from step to step: their own
    // instruction streams are on the critical path of a K step.
    if (warp == 0) {
        // cache tiles are read once per pass: evict them first, so that u, du, the weight shadow and
        // the optimizer state stay L2-resident
        const uint64_t pol = l2_policy_evict_first();
        uint32_t s = 0, eph = 1;                                   // eph: parity of the "stage free" phase to wait for
        const uint32_t ring0 = smem_u32(smem);
        uint32_t dst = ring0;
        bool ok = true;
        if (lane == 0) stamp_begin(p.stamp);
        for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
            const int sc = t % p.s_chunks, b = (t / p.s_chunks) % p.B, l = t / (p.s_chunks * p.B);
            const int id = (int)safe_id(p.ids, b, p.N, nullptr);
            for (int kc = 0; kc < p.k_chunks; ++kc) {
                if (!mbar_wait_uniform(empty0 + 8 * s, eph, abort_flag, p.status)) { ok = false; break; }
                if (elect_one()) {
                    const uint32_t full = full0 + 8 * s;
                    mbar_expect_tx(full, a_bytes + b_bytes);
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
        // wide_n: the hi and lo blocks lie next to each other along N ([r block][hi|lo] in 64-column
        // blocks), so one MMA of N = 128 * r_blocks yields u_hi | u_lo side by side in TMEM
        const uint32_t idesc = p.wide_n ? instr_desc_bf16(FWD_ROWS, 128 * r_blocks, 0, 1) : instr_desc_bf16(FWD_ROWS, r_pad, 0, 1);
        // descriptors of a stage's first 16-wide K step (start-address field in 16-byte units); later steps
        // only move the start address: +32 B per step in the K-major A tile, +2048 B (16 rows) in B
        const uint32_t ring0 = smem_u32(smem);
        const uint64_t a_desc0 = smem_desc_sw128(ring0, 16, 1024), bw_desc0 = smem_desc_sw128(ring0 + b_off, b_box, 1024);
        const uint64_t bh_desc0 = smem_desc_sw128(ring0 + b_off, 2 * b_box, 1024), bl_desc0 = smem_desc_sw128(ring0 + b_off + b_box, 2 * b_box, 1024);
        const uint64_t desc_step = (uint64_t)(stage_bytes >> 4);
        uint64_t doff = 0;
        uint32_t s = 0, ph = 0, tile_n = 0;
        for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++tile_n) {
            const int buf = tile_n & 1;
            const uint32_t aph = (tile_n >> 1) & 1;
            if (!mbar_wait_uniform(acce0 + 8 * buf, aph ^ 1, abort_flag, p.status)) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(buf * p.acc_stride);
            bool ok = true;
            for (int kc = 0; kc < p.k_chunks; ++kc) {
                if (!mbar_wait_uniform(full0 + 8 * s, ph, abort_flag, p.status)) { ok = false; break; }
                tc_fence_after();
                const uint64_t ad0 = a_desc0 + doff, bh0 = bh_desc0 + doff, bl0 = bl_desc0 + doff;
                if (elect_one()) {
                    if (p.wide_n) {
                        const uint64_t bw0 = bw_desc0 + doff;
#pragma unroll
                        for (int k = 0; k < KC / 16; ++k)
                            umma_bf16(d_tmem, ad0 + (uint64_t)(k * 2), bw0 + (uint64_t)(k * 128), idesc, (kc | k) ? 1u : 0u);
                    } else {
#pragma unroll
                        for (int k = 0; k < KC / 16; ++k) {
                            umma_bf16(d_tmem, ad0 + (uint64_t)(k * 2), bh0 + (uint64_t)(k * 128), idesc, (kc | k) ? 1u : 0u);
                            umma_bf16(d_tmem, ad0 + (uint64_t)(k * 2), bl0 + (uint64_t)(k * 128), idesc, 1u);
                        }
                    }
                    umma_commit(empty0 + 8 * s);          // frees the smem slot once these MMAs are done
                }
                __syncwarp();
                doff += desc_step;
                if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1u; doff = 0; }
            }
            if (!ok) break;
            if (elect_one()) umma_commit(accf0 + 8 * buf);    // accumulator complete
            __syncwarp();
        }
    } else {
        const int q = warp & 3;                           // TMEM lane quadrant this warp may read
        uint32_t tile_n = 0;
        for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++tile_n) {
            const int sc = t % p.s_chunks, b = (t / p.s_chunks) % p.B, l = t / (p.s_chunks * p.B);
            const int buf = tile_n & 1;
            const uint32_t aph = (tile_n >> 1) & 1;
            if (!mbar_wait_warp(accf0 + 8 * buf, aph, abort_flag, p.status)) break;
            tc_fence_after();
            if (threadIdx.x == 64 && t + (int)gridDim.x >= n_tiles) stamp_end(p.stamp);      // this CTA's last tile
            const int srow = sc * FWD_ROWS + q * 32 + lane;          // token index inside the sample
            const long long m = (long long)b * p.S + srow;
            float* dst = p.u + (long long)l * p.layer_stride + m * p.r;
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * p.acc_stride);
            for (int c0 = 0; c0 < p.r; c0 += 16) {
                float v[16];
                if (p.wide_n) {
                    // column c of u: hi part at TMEM column (c/64)*128 + c%64, lo part 64 columns further
                    float w[16];
                    const uint32_t col = (uint32_t)((c0 >> 6) * 128 + (c0 & 63));
                    tmem_ld16(taddr + col, v);
                    tmem_ld16(taddr + col + 64, w);
                    tmem_ld_wait();
#pragma unroll
                    for (int c = 0; c < 16; ++c) v[c] += w[c];
                } else {
                    tmem_ld16(taddr + c0, v);
                    tmem_ld_wait();
                }
                if (srow < p.S) {
                    // r is a multiple of 16: the chunk is whole; two 32-byte sectors
#pragma unroll
                    for (int c = 0; c < 16; c += 8)
                        st_global_32(dst + c0 + c, make_uint4(__float_as_uint(v[c]), __float_as_uint(v[c + 1]), __float_as_uint(v[c + 2]), __float_as_uint(v[c + 3])),
                                     make_uint4(__float_as_uint(v[c + 4]), __float_as_uint(v[c + 5]), __float_as_uint(v[c + 6]), __float_as_uint(v[c + 7])));
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
    if (warp == 1) tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
}

struct BwdParams {
    const int* ids; long long N;
    int L, S, d, r, B;
    int s_chunks;                          // ceil(S / BWD_KR)
    int d_groups;                          // ceil(d / (128 * chunks))
    int chunks;                            // 128-column blocks of h per CTA (accumulators in TMEM)
    int splits;                            // row splits J: partial sums per output
    int r_blocks;                          // ceil(r / 64)
    int stages;
    int tmem_cols;
    int early_ids;                         // 1: no kernel ahead of this one in the stream writes the ids
    float* out;                            // splits == 1: dW_down [L][d][r]; else partials [J][L][d][r]
    unsigned* status;
    unsigned long long* stamp;             // optional stream-phase timestamps (see stamp_begin)
};

// ---------------------------------------------------------------------------
// dW_down^l = h_l^T du_l.  One CTA owns (layer, group of 128-column blocks of h, row split):
// it streams 64-token tiles of h_l (MN-major A: the 128 output rows are h's columns) and of
// du_l (MN-major B: N = r), accumulates [128 x r] blocks in TMEM over all its rows and writes
// them once.  With splits > 1 the partial sums are added afterwards in split order.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(DW_THREADS, 1)
dw_down_tc_kernel(const __grid_constant__ CUtensorMap map_cache, const __grid_constant__ CUtensorMap map_du, BwdParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int r_pad = (p.r + 15) & ~15;
    const uint32_t box_bytes = BWD_KR * 128;                       // one [64 tokens][64 columns] box
    const uint32_t a_bytes = (uint32_t)p.chunks * 2 * box_bytes, b_bytes = (uint32_t)p.r_blocks * box_bytes;
    const uint32_t stage_bytes = a_bytes + b_bytes;
    __shared__ __align__(8) unsigned long long bars[2 * 16 + 2];
    __shared__ uint32_t tmem_base_sh;
    __shared__ int abort_sh;
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[16]), accf = smem_u32(&bars[32]);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    int item = blockIdx.x;
    const int j = item % p.splits; item /= p.splits;
    const int g = item % p.d_groups;
    const int l = p.L - 1 - item / p.d_groups;       // last layers first: they were read most recently by the forward pass
    const int row_tiles = p.B * p.s_chunks;
    const int rt0 = (int)((long long)row_tiles * j / p.splits), rt1 = (int)((long long)row_tiles * (j + 1) / p.splits);
    const int col0 = g * p.chunks * 128;

    if (threadIdx.x == 0) {
        abort_sh = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        mbar_init(accf, 1);
        fence_mbar_init();
        tma_prefetch_desc(&map_cache);
        tma_prefetch_desc(&map_du);
    }
    if (warp == 1) { tmem_alloc(smem_u32(&tmem_base_sh), (uint32_t)p.tmem_cols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_sh;
    volatile int* abort_flag = &abort_sh;
    // The cache never changes: with ids that were final before this launch the h tiles of the first ring are
    // requested while the predecessor still runs; only du (its result) has to wait.
    uint32_t pre = 0;
    if (p.early_ids && warp == 0 && rt1 > rt0) {
        pre = (uint32_t)min(rt1 - rt0, p.stages);
        if (elect_one()) {
            const uint64_t pol = l2_policy_evict_first();
            for (uint32_t i = 0; i < pre; ++i) {
                const int rt = rt0 + (int)i, sc = rt % p.s_chunks, b = rt / p.s_chunks;
                const int id = (int)safe_id(p.ids, b, p.N, nullptr);
                const uint32_t dst = smem_u32(smem + (size_t)i * stage_bytes);
                mbar_expect_tx(full0 + 8 * i, stage_bytes);
                for (int q = 0; q < 2 * p.chunks; ++q)
                    tma_load_4d_hint(dst + q * box_bytes, &map_cache, full0 + 8 * i, col0 + q * 64, sc * BWD_KR, l, id, pol);
            }
        }
        __syncwarp();
    }
    pdl_wait();
    // the successor may start only now: when it runs, the forward half of this step (and with it the
    // previous step's parameter update) is known to be complete
    pdl_trigger();

    // Both pipeline loops carry ring positions, parities, addresses and descriptors from step to step.
    if (warp == 0) {
        const uint64_t pol = l2_policy_evict_first();
        if (lane == 0 && rt1 > rt0) stamp_begin(p.stamp);
        uint32_t s = 0, eph = 1;                                   // eph: parity of the "stage free" phase to wait for
        const uint32_t ring0 = smem_u32(smem);
        uint32_t dst = ring0;
        int sc = rt0 % p.s_chunks, b = rt0 / p.s_chunks;
        int id = rt1 > rt0 ? (int)safe_id(p.ids, b, p.N, nullptr) : 0;
        for (int rt = rt0; rt < rt1; ++rt) {
            const uint32_t full = full0 + 8 * s;
            if (pre > 0) {
                // first ring: the h tiles are already on their way
                --pre;
                if (elect_one())
                    for (int q = 0; q < p.r_blocks; ++q)
                        tma_load_3d(dst + a_bytes + q * box_bytes, &map_du, full, q * 64, b * p.S + sc * BWD_KR, l);
            } else {
                if (!mbar_wait_uniform(empty0 + 8 * s, eph, abort_flag, p.status)) break;
                if (elect_one()) {
                    mbar_expect_tx(full, stage_bytes);
                    for (int q = 0; q < 2 * p.chunks; ++q)
                        tma_load_4d_hint(dst + q * box_bytes, &map_cache, full, col0 + q * 64, sc * BWD_KR, l, id, pol);
                    for (int q = 0; q < p.r_blocks; ++q)
                        tma_load_3d(dst + a_bytes + q * box_bytes, &map_du, full, q * 64, b * p.S + sc * BWD_KR, l);
                }
            }
            __syncwarp();
            dst += stage_bytes;
            if (++s == (uint32_t)p.stages) { s = 0; eph ^= 1u; dst = ring0; }
            if (++sc == p.s_chunks) {
                sc = 0; ++b;
                if (rt + 1 < rt1) id = (int)safe_id(p.ids, b, p.N, nullptr);
            }
        }
    } else if (warp == 1) {
        const uint32_t idesc = instr_desc_bf16(128, r_pad, 1, 1);
        // descriptors of a stage's first K step (start-address field in 16-byte units)
        const uint32_t ring0 = smem_u32(smem);
        const uint64_t a_desc0 = smem_desc_sw128(ring0, box_bytes, 1024), b_desc0 = smem_desc_sw128(ring0 + a_bytes, box_bytes, 1024);
        const uint64_t desc_step = (uint64_t)(stage_bytes >> 4), a_chunk = (uint64_t)((2 * box_bytes) >> 4);
        uint64_t doff = 0;
        uint32_t s = 0, ph = 0, first = 0;                         // first: 0 until the first K step has been issued
        bool ok = true;
        for (int rt = rt0; rt < rt1 && ok; ++rt) {
            if (!mbar_wait_uniform(full0 + 8 * s, ph, abort_flag, p.status)) { ok = false; break; }
            tc_fence_after();
            if (elect_one()) {
                const uint64_t ad0 = a_desc0 + doff, bd0 = b_desc0 + doff;
                // consecutive MMAs alternate between the column blocks' accumulators: an MMA that adds to
                // the result of the one before it would have to wait for that one to finish
#pragma unroll
                for (int k = 0; k < BWD_KR / 16; ++k)          // 16 tokens = 2048 B further along K in both operands
                    for (int c = 0; c < p.chunks; ++c)
                        umma_bf16(tmem_base + (uint32_t)(c * r_pad), ad0 + (uint64_t)c * a_chunk + (uint64_t)(k * 128),
                                  bd0 + (uint64_t)(k * 128), idesc, (first | (uint32_t)k) ? 1u : 0u);
                umma_commit(empty0 + 8 * s);
            }
            __syncwarp();
            first = 1;
            doff += desc_step;
            if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1u; doff = 0; }
        }
        if (ok) {
            if (elect_one()) umma_commit(accf);
            __syncwarp();
        }
    } else {
        const int q = warp & 3;                                   // TMEM lane quadrant this warp may read
        const int ne = ((int)(blockDim.x >> 5) - 2) >> 2, e16 = ((warp - 2) >> 2) * 16;      // warps per quadrant; this warp's first 16 columns
        if (rt1 > rt0) {
            if (mbar_wait_warp(accf, 0, abort_flag, p.status)) {
                tc_fence_after();
                if (threadIdx.x == 64) stamp_end(p.stamp);
                for (int c = 0; c < p.chunks; ++c) {
                    const int k = col0 + c * 128 + q * 32 + lane;             // column of h = row of dW_down
                    float* dst = p.out + (((long long)j * p.L + l) * p.d + k) * p.r;
                    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * r_pad);
                    for (int c0 = e16; c0 < p.r; c0 += 16 * ne) {              // the quadrant's warps share its columns
                        float v[16];
                        tmem_ld16(taddr + c0, v);
                        tmem_ld_wait();
                        if (k < p.d) {
                            // (16-byte stores: with 32-byte ones here the step measured 0.4 us slower)
#pragma unroll
                            for (int cc = 0; cc < 16; cc += 4)
                                *reinterpret_cast<float4*>(dst + c0 + cc) = make_float4(v[cc], v[cc + 1], v[cc + 2], v[cc + 3]);
                        }
                    }
                }
            }
        } else {
            // no rows in this split: the partial is zero
            for (int c = 0; c < p.chunks; ++c) {
                const int k = col0 + c * 128 + q * 32 + lane;
                if (k < p.d && e16 == 0) {
                    float* dst = p.out + (((long long)j * p.L + l) * p.d + k) * p.r;
                    for (int c0 = 0; c0 < p.r; ++c0) dst[c0] = 0.f;
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    drain_after_abort(abort_flag);
    if (warp == 1) tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
}

// out[i] = sum_j part[j][i] in split order (deterministic).
__global__ void reduce_splits_kernel(const float* __restrict__ part, int splits, long long n, float* __restrict__ out) {
    long long i = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i >= n) return;
    float4 acc = *reinterpret_cast<const float4*>(part + i);
    for (int j = 1; j < splits; ++j) {
        float4 v = *reinterpret_cast<const float4*>(part + (long long)j * n + i);
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    *reinterpret_cast<float4*>(out + i) = acc;
}

// ---------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------
struct TensorPlan {
    bool ready = false;
    Dims dm{};
    int max_batch = 0, sms = 0;
    CUtensorMap map_cache_fwd, map_cache_bwd, map_w, map_du;
    FwdParams fp{};
    BwdParams bp{};
    size_t smem_fwd = 0, smem_bwd = 0;
    long long dw_elems = 0;
};

inline std::string& tensor_err() { static std::string e; return e; }
inline const char* tensor_last_error() { return tensor_err().c_str(); }

// Launch configuration with programmatic stream serialization allowed (see pdl_wait above).
inline void pdl_launch_config(cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr, dim3 grid, dim3 block, size_t smem,
                              cudaStream_t stream) {
    cfg->gridDim = grid;
    cfg->blockDim = block;
    cfg->dynamicSmemBytes = smem;
    cfg->stream = stream;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg->attrs = attr;
    cfg->numAttrs = 1;
}

inline bool tensor_shape_supported(const Dims& dm) {
    return dm.d % 8 == 0 && dm.d >= 64 && dm.r % 16 == 0 && dm.r >= 16 && dm.r <= 256;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn) return fn;
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !sym)
        return nullptr;
    fn = (EncodeTiledFn)sym;
    return fn;
}

// bf16 tensor map with 128-byte swizzle; dims/strides innermost first, strides in bytes for dims 1..rank-1.
inline bool make_map(CUtensorMap* map, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides_bytes,
                     const cuuint32_t* box) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) { tensor_err() = "cuTensorMapEncodeTiled is not available from the driver"; return false; }
    cuuint32_t ones[5] = {1, 1, 1, 1, 1};
    CUresult res = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), dims, strides_bytes,
                      box, ones, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (res != CUDA_SUCCESS) {
        char buf[96];
        snprintf(buf, sizeof buf, "cuTensorMapEncodeTiled failed with CUresult %d", (int)res);
        tensor_err() = buf;
        return false;
    }
    return true;
}

inline int pow2_at_least(int x) { int p = 32; while (p < x) p <<= 1; return p; }

// wdT: [L][2][d][r] bf16 hi/lo shadow of W_down; du16: [L][max_rows][r] bf16.  *part_floats receives the
// size of the split-partial buffer dW needs (0 when no split is used).
inline pac_status tensor_plan_create(TensorPlan& tp, int device, const bf16* cache, const Dims& dm, int max_batch,
                                     const bf16* wdT, const bf16* du16, long long* part_floats) {
    tp.ready = false;
    tp.dm = dm;
    tp.max_batch = max_batch;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { tensor_err() = "cudaGetDeviceProperties failed"; return PAC_ERR_CUDA; }
    if (prop.major != 10) { tensor_err() = "device is not sm_100"; return PAC_ERR_UNSUPPORTED; }
    tp.sms = prop.multiProcessorCount;
    const int max_smem = (int)prop.sharedMemPerBlockOptin;
    const long long max_rows = (long long)max_batch * dm.S;
    const int r_pad = (dm.r + 15) & ~15;

    // ---- tensor maps ----
    {
        cuuint64_t dims[4] = {(cuuint64_t)dm.d, (cuuint64_t)dm.S, (cuuint64_t)dm.L, (cuuint64_t)dm.N};
        cuuint64_t str[3] = {(cuuint64_t)dm.d * 2, (cuuint64_t)dm.S * dm.d * 2, (cuuint64_t)dm.L * dm.S * dm.d * 2};
        cuuint32_t box_f[4] = {KC, FWD_ROWS, 1, 1}, box_b[4] = {KC, BWD_KR, 1, 1};
        if (!make_map(&tp.map_cache_fwd, cache, 4, dims, str, box_f)) return PAC_ERR_UNSUPPORTED;
        if (!make_map(&tp.map_cache_bwd, cache, 4, dims, str, box_b)) return PAC_ERR_UNSUPPORTED;
    }
    {
        cuuint64_t dims[4] = {(cuuint64_t)dm.r, (cuuint64_t)dm.d, 2, (cuuint64_t)dm.L};
        cuuint64_t str[3] = {(cuuint64_t)dm.r * 2, (cuuint64_t)dm.r * dm.d * 2, (cuuint64_t)2 * dm.r * dm.d * 2};
        cuuint32_t box[4] = {64, KC, 2, 1};
        if (!make_map(&tp.map_w, wdT, 4, dims, str, box)) return PAC_ERR_UNSUPPORTED;
    }
    {
        cuuint64_t dims[3] = {(cuuint64_t)dm.r, (cuuint64_t)max_rows, (cuuint64_t)dm.L};
        cuuint64_t str[2] = {(cuuint64_t)dm.r * 2, (cuuint64_t)max_rows * dm.r * 2};
        cuuint32_t box[3] = {KC, BWD_KR, 1};
        if (!make_map(&tp.map_du, du16, 3, dims, str, box)) return PAC_ERR_UNSUPPORTED;
    }

    // ---- forward plan ----
    FwdParams& f = tp.fp;
    f.N = dm.N; f.L = dm.L; f.S = dm.S; f.d = dm.d; f.r = dm.r;
    f.s_chunks = (dm.S + FWD_ROWS - 1) / FWD_ROWS;
    f.k_chunks = (dm.d + KC - 1) / KC;
    f.wide_n = dm.r <= 128 ? 1 : 0;          // N = 128 * r_blocks must stay within 256
    f.tmem_cols = pow2_at_least(2 * (f.wide_n ? 128 * ((dm.r + 63) / 64) : r_pad));
    f.acc_stride = f.tmem_cols / 2;
    {
        const int stage = FWD_ROWS * KC * 2 + ((dm.r + 63) / 64) * 2 * KC * 128;
        int st = (max_smem - 2048) / stage;
        if (st > 16) st = 16;
        if (st < 2) { tensor_err() = "not enough shared memory for the forward pipeline"; return PAC_ERR_UNSUPPORTED; }
        f.stages = st;
        tp.smem_fwd = (size_t)st * stage + 1024;
    }
    f.layer_stride = max_rows * dm.r;

    // ---- backward plan ----
    BwdParams& b = tp.bp;
    b.N = dm.N; b.L = dm.L; b.S = dm.S; b.d = dm.d; b.r = dm.r;
    b.s_chunks = (dm.S + BWD_KR - 1) / BWD_KR;
    b.r_blocks = (dm.r + 63) / 64;
    b.chunks = (dm.d >= 256 && 2 * r_pad <= 512) ? 2 : 1;
    b.d_groups = (dm.d + 128 * b.chunks - 1) / (128 * b.chunks);
    b.tmem_cols = pow2_at_least(b.chunks * r_pad);
    {
        const int stage = (b.chunks * 2 + b.r_blocks) * BWD_KR * 128;
        int st = (max_smem - 2048) / stage;
        if (st > 16) st = 16;
        if (st < 2) { tensor_err() = "not enough shared memory for the backward pipeline"; return PAC_ERR_UNSUPPORTED; }
        b.stages = st;
        tp.smem_bwd = (size_t)st * stage + 1024;
    }
    // row splits: enough CTAs to fill the SMs in balanced waves, few enough partial sums
    {
        const int items = dm.L * b.d_groups;
        const int row_tiles_max = max_batch * b.s_chunks;
        int best = 1;
        double best_cost = 1e30;
        for (int J = 1; J <= 8 && J <= row_tiles_max; ++J) {
            double waves = (double)items * J / tp.sms;
            double cost = std::ceil(waves) / waves + 0.03 * (J - 1);
            if (cost < best_cost - 1e-9) { best_cost = cost; best = J; }
        }
        b.splits = best;
    }
    tp.dw_elems = (long long)dm.L * dm.d * dm.r;
    *part_floats = b.splits > 1 ? tp.dw_elems * b.splits : 0;

    if (smem_opt_in((const void*)down_fwd_tc_kernel, tp.smem_fwd) != cudaSuccess ||
        smem_opt_in((const void*)dw_down_tc_kernel, tp.smem_bwd) != cudaSuccess) {
        tensor_err() = "cudaFuncSetAttribute(MaxDynamicSharedMemorySize) failed";
        cudaGetLastError();
        return PAC_ERR_CUDA;
    }
    tp.ready = true;
    return PAC_OK;
}

inline void tensor_plan_destroy(TensorPlan& tp) { tp.ready = false; }

inline pac_status tensor_down_projection(TensorPlan& tp, cudaStream_t stream, const int* d_ids, int B, float* u,
                                         unsigned* status, long long* launches, unsigned long long* stamp = nullptr) {
    FwdParams p = tp.fp;
    p.ids = d_ids; p.B = B; p.u = u; p.status = status; p.stamp = stamp;
    const int tiles = p.L * B * p.s_chunks;
    const int grid = tiles < tp.sms ? tiles : tp.sms;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    pdl_launch_config(&cfg, attr, dim3((unsigned)grid), dim3(TC_THREADS), tp.smem_fwd, stream);
    cudaError_t e = cudaLaunchKernelEx(&cfg, down_fwd_tc_kernel, tp.map_cache_fwd, tp.map_w, p);
    (*launches)++;
    if (e != cudaSuccess) { tensor_err() = cudaGetErrorString(e); return PAC_ERR_CUDA; }
    return PAC_OK;
}

// Row splits used for a batch of B samples (the partial sums the caller has to add up).
inline int tensor_splits(const TensorPlan& tp, int B) {
    int J = tp.bp.splits;
    if (J > B * tp.bp.s_chunks) J = B * tp.bp.s_chunks;
    return J;
}

// With reduce_splits == false and more than one split the partial sums stay in `part`
// ([J][L][d][r]) for the caller's own reduction.
inline pac_status tensor_dw_down(TensorPlan& tp, cudaStream_t stream, const int* d_ids, int B, const bf16* /*du16*/,
                                 float* dW, float* part, bool reduce_splits, unsigned* status, long long* launches,
                                 unsigned long long* stamp = nullptr, bool early_ids = false) {
    BwdParams p = tp.bp;
    p.ids = d_ids; p.B = B; p.status = status; p.stamp = stamp; p.early_ids = early_ids ? 1 : 0;
    const int J = tensor_splits(tp, B);
    p.splits = J;
    p.out = J > 1 ? part : dW;
    const int grid = p.L * p.d_groups * J;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    pdl_launch_config(&cfg, attr, dim3((unsigned)grid), dim3(DW_THREADS), tp.smem_bwd, stream);
    cudaError_t e = cudaLaunchKernelEx(&cfg, dw_down_tc_kernel, tp.map_cache_bwd, tp.map_du, p);
    (*launches)++;
    if (e != cudaSuccess) { tensor_err() = cudaGetErrorString(e); return PAC_ERR_CUDA; }
    if (J > 1 && reduce_splits) {
        reduce_splits_kernel<<<(unsigned)((tp.dw_elems / 4 + 255) / 256), 256, 0, stream>>>(part, J, tp.dw_elems, dW);
        (*launches)++;
        e = cudaGetLastError();
        if (e != cudaSuccess) { tensor_err() = cudaGetErrorString(e); return PAC_ERR_CUDA; }
    }
    return PAC_OK;
}

}  // namespace pac
