// Host runtime and C ABI of the adapter-over-cache trainer (declarations: include/pac.h).
#include <cmath>
#include <cstdarg>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include <fcntl.h>
#include <sys/mman.h>
#include <sys/stat.h>
#include <unistd.h>

#include "pac_common.cuh"
#include "pac_simt.cuh"
#include "pac_tensor.cuh"
#include "pac_mid.cuh"
#include "pac_fused_fwd.cuh"
#include "pac_chain_fwd.cuh"
#include "pac_gemm.cuh"
#include "pac_quant.cuh"
#include "pac_tbody.cuh"

using namespace pac;

namespace {

constexpr int STAGE_SLOTS = 8;
constexpr int LM_MAX_K_SLICES = 8;
constexpr int ZC_SLOTS = 64;

struct Scratch {
    // per-step state, sized for max_batch
    int* ids = nullptr;            // [max_batch] device copy of the current ids
    float* u = nullptr;            // [L][M][r] down-projections
    float* a = nullptr;            // [L][M][r] adapter states
    float* du = nullptr;           // [L][M][r] fp32 (plain path)
    bf16* du16 = nullptr;          // [L][M][r] bf16 (tensor path)
    float* lam_part = nullptr;     // [L][blocks]
    float* loss = nullptr;         // [1]
    // classifier head
    float* hbar = nullptr;         // [N][d] token mean of the last cached layer
    float* pooled_a = nullptr;     // [B][r]
    float* pooled_y = nullptr;     // [B][d]
    float* logits = nullptr;       // [B][C]
    float* dlogits = nullptr;      // [B][C]
    float* loss_b = nullptr;       // [B] (classifier) or [M] (LM rows)
    float* gvec = nullptr;         // [B][d]
    float* daL = nullptr;          // [B][r] (classifier) or [M][r] (LM)
    // LM head
    float* y = nullptr;            // [M][d]
    float* lm_logits = nullptr;    // [M][V]
    float* dy = nullptr;           // [M][d]
    bf16* y16 = nullptr;           // [M][d] bf16 y (tensor-core LM head)
    bf16* dlog16 = nullptr;        // [M][V] bf16 dlogits (tensor-core LM head)
    bf16* aL16 = nullptr;          // [M][r] bf16 a_L, bf16 W_up [r][d], bf16 dy [M][d]: operands of the LM path's skinny products
    bf16* wup16 = nullptr;
    bf16* dy16 = nullptr;
    // tensor path
    bf16* wdT = nullptr;           // [L][2][d][r] bf16 hi/lo shadow of W_down
    float* lm_part = nullptr;      // [slices][...] partial sums of the LM path's two skinny products (dW_up, da_L)
    float* dw_part = nullptr;      // split partials of dW_down
    unsigned* gates = nullptr;     // [M][r] ReLU gates of all layers, one word per element (chain-in-epilogue forward)
    float* pool_part = nullptr;    // [B][s_chunks * 4][r] token sums of a_L per 32-token group (chain-in-epilogue forward)
    float* prodW = nullptr;        // [r][C] W_up W_head of the current parameters (stand-alone head kernels)
};

// Saved activations and work buffers of the transformer-body adapters (fp32, sized for max_batch).
struct TBody {
    bool on = false;
    int H = 0, f = 0;
    BodyLayout bl{};
    float* buf = nullptr;          // one allocation, carved below
    // per layer stacks [L][...]
    float *x = nullptr, *xhat1 = nullptr, *n1 = nullptr, *qkv = nullptr, *o = nullptr, *x1 = nullptr, *xhat2 = nullptr,
          *n2 = nullptr, *pre = nullptr, *P = nullptr, *rstd1 = nullptr, *rstd2 = nullptr;
    // work buffers of the backward pass
    float *da = nullptr, *dx1 = nullptr, *dn = nullptr, *dqkv = nullptr, *dpre = nullptr, *dtmp = nullptr;
    long long sMr = 0, sMf = 0, sP = 0, sM = 0;      // per-layer strides of the stacks
};

// A cache that lives in host memory (Section V-B, storage cost analysis: the cache is kept on
// storage and reloaded per micro-batch).  The device holds two staging slots of max_batch samples;
// a step's slabs are copied into a slot by the copy engine on a stream of their own while the step
// before it computes on the other slot.  The kernels see a slot as a cache of max_batch samples and
// the ids 0 .. B-1.
struct HostCache {
    bool on = false;
    const unsigned char* host = nullptr;    // [N][L][S][d], host memory (page-locked for asynchronous copies)
    const int* host_labels = nullptr;       // [N][labels_per_sample], host memory
    long long N = 0;                        // samples in the host cache
    long long sample_bytes = 0;             // L * S * d * element size
    int cur = 0;                            // slot the next step uses
    unsigned char* stage[2] = {nullptr, nullptr};   // device [max_batch][L][S][d]
    int* lab_stage[2] = {nullptr, nullptr};         // device [max_batch][labels_per_sample]
    int* h_lab[2] = {nullptr, nullptr};             // page-locked staging of the labels
    float* hbar_stage[2] = {nullptr, nullptr};      // device [max_batch][d]
    int* iota = nullptr;                            // device 0 .. max_batch-1
    TensorPlan tplan[2];
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ready[2] = {nullptr, nullptr};      // slot filled (copy stream)
    cudaEvent_t freed[2] = {nullptr, nullptr};      // slot's step enqueued and done (compute stream)
    // a cache file mapped by pac_cache_register_file (owned: unmapped in pac_destroy)
    void* map_base = nullptr;
    size_t map_bytes = 0;
};

// ---------------------------------------------------------------------------
// Cache files (Section IV-B: the activations are recorded during the first epoch and kept on
// storage; Section V-B, storage cost analysis: reloaded per micro-batch).  Layout: a 64-byte
// header, the cache [N][L][S][d] in its dtype, then the labels [N][labels_per_sample] as int32.
// ---------------------------------------------------------------------------
struct CacheFileHeader {
    char magic[8];                 // "PACCACHE"
    unsigned version;              // 1
    int dtype;                     // pac_dtype
    long long N;
    int L, S, d, labels_per_sample;
    char pad[24];
};
static_assert(sizeof(CacheFileHeader) == 64, "cache file header is 64 bytes");
const char CACHE_MAGIC[8] = {'P', 'A', 'C', 'C', 'A', 'C', 'H', 'E'};

inline size_t cache_file_data_bytes(const CacheFileHeader& h) {
    return (size_t)h.N * h.L * h.S * h.d * (h.dtype == PAC_F32 ? 4 : 2);
}
// the labels start at the next multiple of 64 bytes behind the data
inline size_t cache_file_labels_offset(const CacheFileHeader& h) {
    return sizeof(CacheFileHeader) + ((cache_file_data_bytes(h) + 63) & ~(size_t)63);
}
inline size_t cache_file_bytes(const CacheFileHeader& h) {
    return cache_file_labels_offset(h) + (size_t)h.N * h.labels_per_sample * sizeof(int);
}
inline bool cache_file_header_ok(const CacheFileHeader& h) {
    return std::memcmp(h.magic, CACHE_MAGIC, 8) == 0 && h.version == 1u && (h.dtype == PAC_F32 || h.dtype == PAC_BF16) &&
           h.N >= 1 && h.N <= 0x7fffffffLL && h.L >= 1 && h.S >= 1 && h.d >= 1 &&
           (h.labels_per_sample == 1 || h.labels_per_sample == h.S);
}

}  // namespace

struct pac_ctx {
    int device = 0;
    cudaStream_t stream = nullptr;
    bool own_stream = false;
    // cache
    const void* cache = nullptr;
    int dtype = PAC_F32;
    Dims dm{};
    const int* labels = nullptr;
    int labels_per_sample = 0;
    bool registered = false;
    // adapters
    bool inited = false;
    pac_adapter_cfg cfg{};
    ParamLayout lay{};
    float *params = nullptr, *grads = nullptr, *m = nullptr, *v = nullptr;
    long long step = 0;
    float grad_scale = 1.f;        // factor the optimizer applies to every gradient (data parallel: 1 / world)
    int max_rows = 0;              // max_batch * S
    int chain_blocks_max = 0;
    Scratch sc;
    unsigned* status = nullptr;    // device status words
    // host staging (pinned)
    int* h_ids = nullptr;          // [STAGE_SLOTS][max_batch]
    cudaEvent_t slot_ev[STAGE_SLOTS] = {};
    int slot = 0;
    float* h_loss = nullptr;
    unsigned* h_status = nullptr;
    // epoch buffers
    int* d_perm = nullptr; long long perm_cap = 0;
    float* d_losses = nullptr; long long losses_cap = 0;
    // options / bookkeeping
    int force_simt = 0;
    int timing = 0;
    std::vector<cudaEvent_t> tev[4];   // start/stop pairs per bracketed kernel group
    size_t tev_used[4] = {0, 0, 0, 0};
    // device-side stream-phase timestamps (timing == 2): [pass][slot]{earliest first copy, latest accumulator complete}
    unsigned long long* d_stamps = nullptr;
    size_t stamps_used[2] = {0, 0};
    bool tensor_ok = false;
    long long launches = 0;
    TensorPlan tplan{};
    MidPlan mplan{};               // fused classifier-head kernel (when the shape allows)
    FusedFwdPlan fplan{};          // down-projections + classifier-head kernel in one launch (short sequences)
    MidPlan pplan{};               // head / reverse-chain kernel behind the chain-in-epilogue forward
    bool chain_ok = false;         // the chain-in-epilogue forward can take this shape
    int chain_pair_stages = 0;     // > 0: its CTA-pair form can too, with this many stages
    int forward_mode = 0;          // 0: automatic, 2: down-projections and head phase as two plain launches, 3: one-launch
                                   // forward whenever the shape allows, 4: chain-in-epilogue forward whenever the shape allows
    GemmPlan g_logits{}, g_dy{};   // tensor-core GEMMs of the frozen LM head
    GemmPlan g_y{}, g_daL{};       // y = a_L W_up (+ h_L in the epilogue) and da_L = dy W_up^T on the tensor cores
    bool lm_tensor = false;
    bool lm_skinny_tensor = false; // the three products around W_up also run on the tensor cores
    int sms = 0;                   // multiprocessors of the device
    bool lm_ce_stream = false;     // LM cross-entropy as a register-resident stream over the logits (V <= 32768, V % 4 == 0)
    HostCache hc;                  // out-of-core mode (pac_cache_register_host)
    TBody tb;                      // transformer-body adapters (plain fp32 kernels)
    // pac_train_step_async without copy nodes in the stream: a ring of id slots in page-locked host memory that
    // the forward kernel reads directly (two halves, an event per half orders the reuse)
    int* zc_ids = nullptr;         // [ZC_SLOTS][max_batch]
    unsigned* zc_tags = nullptr;   // [ZC_SLOTS] page-locked: sequence number of the step whose ids the slot holds (written last)
    int* zc_dev_ids = nullptr;     // [2][max_batch] device: ids a finalisation kernel fetched for the step after it
    unsigned* zc_dev_tag = nullptr;// [2] device: sequence number those ids belong to
    cudaEvent_t zc_ev[2] = {nullptr, nullptr};
    unsigned long long zc_count = 0;
    bool step_host_ids = false;    // the step being enqueued reads its ids from the ring
    bool step_early_ids = false;   // the step's device ids were final before any kernel still in flight was launched
    std::string err;
};

namespace {

pac_status fail(pac_ctx* c, pac_status s, const char* fmt, ...) {
    if (c) {
        char buf[512];
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(buf, sizeof buf, fmt, ap);
        va_end(ap);
        c->err = buf;
    }
    return s;
}

#define CU_OK(c, call)                                                                              \
    do {                                                                                            \
        cudaError_t e_ = (call);                                                                    \
        if (e_ != cudaSuccess)                                                                      \
            return fail(c, e_ == cudaErrorMemoryAllocation ? PAC_ERR_NOMEM : PAC_ERR_CUDA,          \
                        "%s failed: %s", #call, cudaGetErrorString(e_));                            \
    } while (0)

#define LAUNCH_CHECK(c)                                                                             \
    do {                                                                                            \
        (c)->launches++;                                                                            \
        cudaError_t e_ = cudaGetLastError();                                                        \
        if (e_ != cudaSuccess) return fail(c, PAC_ERR_CUDA, "kernel launch failed: %s (%s:%d)",     \
                                           cudaGetErrorString(e_), __FILE__, __LINE__);             \
    } while (0)

template <typename T>
pac_status dmalloc(pac_ctx* c, T** p, long long n) {
    if (n <= 0) n = 1;
    CU_OK(c, cudaMalloc((void**)p, (size_t)n * sizeof(T)));
    return PAC_OK;
}

bool use_tensor(const pac_ctx* c) { return c->tensor_ok && !c->force_simt; }
pac_status adam_enqueue(pac_ctx* c, const pac_adamw* hp);
pac_status down_projection(pac_ctx* c, const int* d_ids, int B);
pac_status dw_down(pac_ctx* c, const int* d_ids, int B, bool reduce_splits);

inline unsigned cdiv(long long a, long long b) { return (unsigned)((a + b - 1) / b); }

// ---- counter-based initial parameters (splitmix64 output function on a keyed counter;
// twelve 16-bit fields per element summed to a centred Irwin-Hall(12) value) ----
const unsigned long long GOLD = 0x9E3779B97F4A7C15ull;
unsigned long long mix64(unsigned long long x) {
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
    return x ^ (x >> 31);
}
float unit_normal(unsigned long long key, unsigned long long idx) {
    long long total = 0;
    for (int j = 0; j < 3; ++j) {
        unsigned long long w = mix64((idx * 3 + j) * GOLD + key);
        total += (long long)(w & 0xFFFF) + (long long)((w >> 16) & 0xFFFF) + (long long)((w >> 32) & 0xFFFF) +
                 (long long)(w >> 48);
    }
    return (float)(total - 6 * 65535) * 0x1p-16f;
}

void fill_initial_params(const pac_ctx* c, unsigned long long seed, std::vector<float>& out) {
    const int TAG_PARAM = 4;
    unsigned long long key = mix64(mix64(seed) ^ ((unsigned long long)TAG_PARAM * GOLD));
    const ParamLayout& lay = c->lay;
    out.assign((size_t)lay.total, 0.f);
    const float inv = (float)(1.0 / std::sqrt((double)c->dm.d));
    for (long long i = 0; i < lay.lam; ++i) out[i] = unit_normal(key, (unsigned long long)i) * inv;
    for (long long i = lay.lam; i < lay.w_up; ++i) out[i] = c->cfg.lambda_init;
    for (long long i = lay.w_head; i < lay.b_head; ++i) out[i] = unit_normal(key, (unsigned long long)i) * inv;
    if (c->tb.on) {
        // transformer bodies: LayerNorm gains 1, biases 0, Gaussian matrices scaled by 1/sqrt(fan-in)
        const BodyLayout& bl = c->tb.bl;
        const float ir = (float)(1.0 / std::sqrt((double)bl.r)), jf = (float)(1.0 / std::sqrt((double)bl.f));
        for (int l = 0; l < c->dm.L; ++l) {
            const long long o = lay.body + (long long)l * bl.per_layer;
            for (int j = 0; j < bl.r; ++j) { out[o + bl.g1 + j] = 1.f; out[o + bl.g2 + j] = 1.f; }
            for (long long i = o + bl.wq; i < o + bl.g2; ++i) out[i] = unit_normal(key, (unsigned long long)i) * ir;
            for (long long i = o + bl.w1; i < o + bl.c1; ++i) out[i] = unit_normal(key, (unsigned long long)i) * ir;
            for (long long i = o + bl.w2; i < o + bl.c2; ++i) out[i] = unit_normal(key, (unsigned long long)i) * jf;
        }
    }
}

// ---- optional event brackets around the two cache-stream kernels ----
constexpr size_t MAX_TIMED = 4096;
constexpr size_t STAMP_SLOTS = 1024;
// Slot for the next launch of pass `which` (0: first pass over the cache, 1: second), or null.
unsigned long long* next_stamp(pac_ctx* c, int which) {
    if (c->timing != 2 || !c->d_stamps || c->stamps_used[which] >= STAMP_SLOTS) return nullptr;
    return c->d_stamps + ((size_t)which * STAMP_SLOTS + c->stamps_used[which]++) * 2;
}
pac_status reset_stamps(pac_ctx* c) {
    std::vector<unsigned long long> init(2 * STAMP_SLOTS * 2);
    for (size_t i = 0; i < init.size(); i += 2) { init[i] = ~0ull; init[i + 1] = 0ull; }
    if (!c->d_stamps) CU_OK(c, cudaMalloc((void**)&c->d_stamps, sizeof(unsigned long long) * init.size()));
    CU_OK(c, cudaStreamSynchronize(c->stream));
    CU_OK(c, cudaMemcpy(c->d_stamps, init.data(), sizeof(unsigned long long) * init.size(), cudaMemcpyHostToDevice));
    c->stamps_used[0] = c->stamps_used[1] = 0;
    return PAC_OK;
}

void time_mark(pac_ctx* c, int which, bool stop) {
    if (c->timing != 1) return;
    size_t pair = c->tev_used[which] / 2;
    if (pair >= MAX_TIMED) return;
    if (c->tev[which].size() < 2 * (pair + 1)) {
        cudaEvent_t a, b;
        if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) return;
        c->tev[which].push_back(a);
        c->tev[which].push_back(b);
    }
    cudaEventRecord(c->tev[which][c->tev_used[which]], c->stream);
    c->tev_used[which] += 1;
    (void)stop;
}

// ---- staging of host ids ----
pac_status stage_ids(pac_ctx* c, const int* ids, int B, const char* who) {
    if (!ids) return fail(c, PAC_ERR_INVALID_ARG, "%s: sample_ids is NULL", who);
    if (B < 1 || B > c->cfg.max_batch)
        return fail(c, PAC_ERR_INVALID_ARG, "%s: B=%d outside [1, max_batch=%d]", who, B, c->cfg.max_batch);
    for (int b = 0; b < B; ++b)
        if (ids[b] < 0 || ids[b] >= c->dm.N)
            return fail(c, PAC_ERR_SAMPLE_ID_RANGE, "%s: sample_ids[%d]=%d outside [0, %lld)", who, b, ids[b], c->dm.N);
    int s = c->slot;
    c->slot = (c->slot + 1) % STAGE_SLOTS;
    CU_OK(c, cudaEventSynchronize(c->slot_ev[s]));
    int* h = c->h_ids + (size_t)s * c->cfg.max_batch;
    std::memcpy(h, ids, sizeof(int) * B);
    CU_OK(c, cudaMemcpyAsync(c->sc.ids, h, sizeof(int) * B, cudaMemcpyHostToDevice, c->stream));
    CU_OK(c, cudaEventRecord(c->slot_ev[s], c->stream));
    return PAC_OK;
}

// ---------------------------------------------------------------------------
// Forward: u_l for every layer, the chain, and the head.  ids are on the device.
// ---------------------------------------------------------------------------
template <typename T>
pac_status down_projection_simt(pac_ctx* c, const int* d_ids, int B) {
    const Dims& dm = c->dm;
    const int M = B * dm.S;
    CacheRows<T> A{(const T*)c->cache, d_ids, dm.N, dm.L, dm.S, dm.d, 0};
    MatB_RowMajor Bm{{c->params + c->lay.w_down, (long long)dm.d * dm.r, dm.r}};
    StoreRowMajor E{c->sc.u, (long long)c->max_rows * dm.r, dm.r};
    dim3 grid(cdiv(dm.r, SG_BN), cdiv(M, SG_BM), dm.L);
    gemm_simt<<<grid, 256, 0, c->stream>>>(M, dm.r, dm.d, A, Bm, E);
    LAUNCH_CHECK(c);
    return PAC_OK;
}

pac_status forward(pac_ctx* c, const int* d_ids, int B, bool train, float* d_logits_out) {
    const Dims& dm = c->dm;
    const int M = B * dm.S;
    const long long n = (long long)M * dm.r, stride = (long long)c->max_rows * dm.r;
    Scratch& sc = c->sc;
    pac_status st = down_projection(c, d_ids, B);
    if (st != PAC_OK) return st;
    const float* lam = c->params + c->lay.lam;
    if (c->cfg.act == PAC_ACT_RELU)
        chain_fwd_kernel<PAC_ACT_RELU><<<cdiv(n, 256), 256, 0, c->stream>>>(sc.u, sc.a, lam, dm.L, n, stride);
    else
        chain_fwd_kernel<PAC_ACT_IDENTITY><<<cdiv(n, 256), 256, 0, c->stream>>>(sc.u, sc.a, lam, dm.L, n, stride);
    LAUNCH_CHECK(c);
    const float* aL = sc.a + (long long)(dm.L - 1) * stride;
    const float* W_up = c->params + c->lay.w_up;
    if (c->cfg.head == PAC_HEAD_MEANPOOL_CLS) {
        pool_tokens_kernel<<<B, 128, 0, c->stream>>>(aL, sc.pooled_a, dm.S, dm.r);
        LAUNCH_CHECK(c);
        size_t smem = sizeof(float) * (dm.d + dm.C + 32);
        cls_head_kernel<<<B, 256, smem, c->stream>>>(sc.hbar, d_ids, dm.N, c->labels, sc.pooled_a, W_up,
                                                     c->params + c->lay.w_head, c->params + c->lay.b_head, B, dm.S,
                                                     dm.d, dm.r, dm.C, train ? 1 : 0, sc.pooled_y,
                                                     train ? sc.logits : d_logits_out, sc.loss_b, sc.dlogits,
                                                     sc.gvec, sc.daL, c->status);
        LAUNCH_CHECK(c);
    } else {
        // y = h_L + a_L W_up
        dim3 g1(cdiv(dm.d, SG_BN), cdiv(M, SG_BM), 1);
        MatA_RowMajor Aa{{aL, 0, dm.r}};
        MatB_RowMajor Bu{{W_up, 0, dm.d}};
        if (c->lm_tensor && c->lm_skinny_tensor) {
            // bf16 copies of a_L and W_up, then y16 = bf16(a_L W_up + h_L) in one tensor-core GEMM whose epilogue adds
            // the last cached layer's rows (y enters the LM head rounded to bf16 anyway)
            to_bf16_kernel<<<cdiv((long long)M * dm.r / 4, 256), 256, 0, c->stream>>>(aL, (long long)M * dm.r, sc.aL16, ((uintptr_t)aL & 15) == 0);
            LAUNCH_CHECK(c);
            to_bf16_kernel<<<cdiv((long long)dm.r * dm.d / 4, 256), 256, 0, c->stream>>>(W_up, (long long)dm.r * dm.d, sc.wup16, ((uintptr_t)W_up & 15) == 0);
            LAUNCH_CHECK(c);
            GemmExtras ex;
            ex.C16 = sc.y16; ex.ldc16 = dm.d;
            ex.add_cache = (const bf16*)c->cache; ex.ids = d_ids; ex.n_cache = dm.N; ex.L = dm.L; ex.S = dm.S;
            st = gemm_launch(c->g_y, c->stream, M, nullptr, 0, c->status, &c->launches, &ex);
            if (st != PAC_OK) return fail(c, st, "tensor-core y GEMM launch failed: %s", tensor_last_error());
        } else if (c->lm_tensor) {
            StorePlusLastLayerBf16<bf16> E{sc.y16, dm.d, CacheRows<bf16>{(const bf16*)c->cache, d_ids, dm.N, dm.L, dm.S, dm.d, dm.L - 1}};
            gemm_simt<<<g1, 256, 0, c->stream>>>(M, dm.d, dm.r, Aa, Bu, E);
        } else if (c->dtype == PAC_F32) {
            StorePlusLastLayer<float> E{sc.y, dm.d, CacheRows<float>{(const float*)c->cache, d_ids, dm.N, dm.L, dm.S, dm.d, dm.L - 1}};
            gemm_simt<<<g1, 256, 0, c->stream>>>(M, dm.d, dm.r, Aa, Bu, E);
        } else {
            StorePlusLastLayer<bf16> E{sc.y, dm.d, CacheRows<bf16>{(const bf16*)c->cache, d_ids, dm.N, dm.L, dm.S, dm.d, dm.L - 1}};
            gemm_simt<<<g1, 256, 0, c->stream>>>(M, dm.d, dm.r, Aa, Bu, E);
        }
        LAUNCH_CHECK(c);
        // logits = y W_lm^T
        float* lg = train ? sc.lm_logits : d_logits_out;
        if (c->lm_tensor) {
            time_mark(c, 1, false);
            st = gemm_launch(c->g_logits, c->stream, M, lg, dm.C, c->status, &c->launches);
            time_mark(c, 1, true);
            if (st != PAC_OK) return fail(c, st, "tensor-core logits GEMM launch failed: %s", tensor_last_error());
        } else {
            dim3 g2(cdiv(dm.C, SG_BN), cdiv(M, SG_BM), 1);
            MatA_RowMajor Ay{{sc.y, 0, dm.d}};
            MatB_Bf16Rows Bw{(const bf16*)c->cfg.lm_head, dm.d};
            StoreRowMajor El{lg, 0, dm.C};
            gemm_simt<<<g2, 256, 0, c->stream>>>(M, dm.C, dm.d, Ay, Bw, El);
            LAUNCH_CHECK(c);
        }
        if (train && c->lm_tensor && c->lm_ce_stream) {
            // logits read once, dlogits written as bf16: a stream bound by HBM
            cudaError_t e = lm_ce_stream_launch(c->stream, c->sms, lg, d_ids, dm.N, c->labels, dm.S, dm.C, M, sc.loss_b,
                                                sc.dlog16, c->status);
            c->launches++;
            if (e != cudaSuccess) return fail(c, PAC_ERR_CUDA, "LM cross-entropy launch failed: %s", cudaGetErrorString(e));
        } else if (train) {
            lm_ce_kernel<<<M, 256, 0, c->stream>>>(lg, d_ids, dm.N, c->labels, dm.S, dm.C, M, 1, sc.loss_b, c->status,
                                                   c->lm_tensor ? sc.dlog16 : nullptr);
            LAUNCH_CHECK(c);
        }
    }
    return PAC_OK;
}

template <typename T>
pac_status dw_down_simt(pac_ctx* c, const int* d_ids, int B) {
    const Dims& dm = c->dm;
    const int M = B * dm.S;
    CacheRowsT<T> A{(const T*)c->cache, d_ids, dm.N, dm.L, dm.S, dm.d};
    MatB_RowMajor Bm{{c->sc.du, (long long)c->max_rows * dm.r, dm.r}};
    StoreRowMajor E{c->grads + c->lay.w_down, (long long)dm.d * dm.r, dm.r};
    dim3 grid(cdiv(dm.r, SG_BN), cdiv(dm.d, SG_BM), dm.L);
    gemm_simt<<<grid, 256, 0, c->stream>>>(dm.d, dm.r, M, A, Bm, E);
    LAUNCH_CHECK(c);
    return PAC_OK;
}

// Backward through the adapters only, after forward(train=true).  d_loss receives the mean loss.
pac_status backward(pac_ctx* c, const int* d_ids, int B, float* d_loss) {
    const Dims& dm = c->dm;
    const int M = B * dm.S;
    const long long n = (long long)M * dm.r, stride = (long long)c->max_rows * dm.r;
    Scratch& sc = c->sc;
    const float* aL = sc.a + (long long)(dm.L - 1) * stride;
    const float* W_up = c->params + c->lay.w_up;
    int per_sample;
    if (c->cfg.head == PAC_HEAD_MEANPOOL_CLS) {
        long long n = (long long)dm.r * dm.d + (long long)dm.d * dm.C + dm.C + 1;
        cls_grads_kernel<<<cdiv(n, 256), 256, 0, c->stream>>>(sc.pooled_a, sc.gvec, sc.pooled_y, sc.dlogits, sc.loss_b,
                                                              B, dm.d, dm.r, dm.C, c->grads + c->lay.w_up,
                                                              c->grads + c->lay.w_head, c->grads + c->lay.b_head, d_loss);
        LAUNCH_CHECK(c);
        per_sample = 1;
    } else {
        mean_kernel<<<1, 1024, 0, c->stream>>>(sc.loss_b, M, d_loss);
        LAUNCH_CHECK(c);
        // dy = dlogits W_lm   (the head is frozen: it receives no gradient)
        if (c->lm_tensor) {
            time_mark(c, 3, false);
            GemmExtras ex;
            if (c->lm_skinny_tensor) { ex.C16 = sc.dy16; ex.ldc16 = dm.d; }        // bf16 copy for the two products below
            pac_status gs = gemm_launch(c->g_dy, c->stream, M, sc.dy, dm.d, c->status, &c->launches, c->lm_skinny_tensor ? &ex : nullptr);
            time_mark(c, 3, true);
            if (gs != PAC_OK) return fail(c, gs, "tensor-core dy GEMM launch failed: %s", tensor_last_error());
        } else {
            dim3 g1(cdiv(dm.d, SG_BN), cdiv(M, SG_BM), 1);
            MatA_RowMajor Ad{{sc.lm_logits, 0, dm.C}};
            MatB_Bf16Cols Bw{(const bf16*)c->cfg.lm_head, dm.d};
            StoreRowMajor Ed{sc.dy, 0, dm.d};
            gemm_simt<<<g1, 256, 0, c->stream>>>(M, dm.d, dm.C, Ad, Bw, Ed);
            LAUNCH_CHECK(c);
        }
        // Both products below have few output tiles and a long reduction: the reduction is cut into
        // slices when that fills the device (partial sums added in slice order).
        auto k_slices = [&](long long tiles, int K, long long out_elems) {
            if (!sc.lm_part || out_elems % 4 != 0) return 1;
            long long s = (2LL * c->sms + tiles - 1) / tiles;
            s = std::min<long long>(s, std::min<long long>(LM_MAX_K_SLICES, K / 256));
            return (int)std::max<long long>(1, s);
        };
        // dW_up = a_L^T dy
        dim3 g2(cdiv(dm.d, SG_BN), cdiv(dm.r, SG_BM), 1);
        MatA_ColMajor At{{aL, 0, dm.r}};
        MatB_RowMajor Bd{{sc.dy, 0, dm.d}};
        const int s2 = k_slices((long long)g2.x * g2.y, M, (long long)dm.r * dm.d);
        if (s2 > 1) {
            const int k_slice = (int)cdiv(cdiv(M, s2), SG_BK) * SG_BK;
            g2.z = cdiv(M, k_slice);
            gemm_simt_ksplit<<<g2, 256, 0, c->stream>>>(dm.r, dm.d, M, k_slice, At, Bd, sc.lm_part);
            LAUNCH_CHECK(c);
            const long long ne = (long long)dm.r * dm.d;
            reduce_splits_kernel<<<cdiv(ne / 4, 256), 256, 0, c->stream>>>(sc.lm_part, (int)g2.z, ne, c->grads + c->lay.w_up);
            c->launches++;
        } else {
            StoreRowMajor Eu{c->grads + c->lay.w_up, 0, dm.d};
            gemm_simt<<<g2, 256, 0, c->stream>>>(dm.r, dm.d, M, At, Bd, Eu);
        }
        LAUNCH_CHECK(c);
        // da_L = dy W_up^T: on the tensor cores when the bf16 copy of dy exists (da_L only feeds du, which is
        // rounded to bf16 anyway).  dW_up above stays in fp32 FMA: with a_L and dy rounded to bf16 its error,
        // amplified by Adam, took the parameters after ten steps past the 1e-2 bound (1.1e-2 measured).
        if (c->lm_tensor && c->lm_skinny_tensor) {
            pac_status gs = gemm_launch(c->g_daL, c->stream, M, sc.daL, dm.r, c->status, &c->launches);
            if (gs != PAC_OK) return fail(c, gs, "tensor-core da_L GEMM launch failed: %s", tensor_last_error());
        } else {
        dim3 g3(cdiv(dm.r, SG_BN), cdiv(M, SG_BM), 1);
        MatA_RowMajor Ady{{sc.dy, 0, dm.d}};
        MatB_ColMajor But{{W_up, 0, dm.d}};
        const int s3 = k_slices((long long)g3.x * g3.y, dm.d, (long long)M * dm.r);
        if (s3 > 1) {
            const int k_slice = (int)cdiv(cdiv(dm.d, s3), SG_BK) * SG_BK;
            g3.z = cdiv(dm.d, k_slice);
            gemm_simt_ksplit<<<g3, 256, 0, c->stream>>>(M, dm.r, dm.d, k_slice, Ady, But, sc.lm_part);
            LAUNCH_CHECK(c);
            const long long ne = (long long)M * dm.r;
            reduce_splits_kernel<<<cdiv(ne / 4, 256), 256, 0, c->stream>>>(sc.lm_part, (int)g3.z, ne, sc.daL);
            c->launches++;
        } else {
            StoreRowMajor Ea{sc.daL, 0, dm.r};
            gemm_simt<<<g3, 256, 0, c->stream>>>(M, dm.r, dm.d, Ady, But, Ea);
        }
        LAUNCH_CHECK(c);
        }
        per_sample = 0;
    }
    const float* lam = c->params + c->lay.lam;
    const unsigned blocks = cdiv(n, 256);
    const bool tens = use_tensor(c);
#define CHAIN_BWD(ACT, DUT, DUP)                                                                              \
    chain_bwd_kernel<ACT, DUT><<<blocks, 256, 0, c->stream>>>(sc.u, sc.a, lam, sc.daL, per_sample, dm.S, dm.r, \
                                                              dm.L, n, stride, DUP, sc.lam_part)
    if (c->cfg.act == PAC_ACT_RELU) {
        if (tens) CHAIN_BWD(PAC_ACT_RELU, bf16, sc.du16); else CHAIN_BWD(PAC_ACT_RELU, float, sc.du);
    } else {
        if (tens) CHAIN_BWD(PAC_ACT_IDENTITY, bf16, sc.du16); else CHAIN_BWD(PAC_ACT_IDENTITY, float, sc.du);
    }
#undef CHAIN_BWD
    LAUNCH_CHECK(c);
    reduce_rows_kernel<<<dm.L, 256, 0, c->stream>>>(sc.lam_part, (int)blocks, c->grads + c->lay.lam);
    LAUNCH_CHECK(c);
    return dw_down(c, d_ids, B, true);
}

// ---------------------------------------------------------------------------
// Transformer-body adapters (plain fp32 kernels; see pac_tbody.cuh).  ids are on the device.
// ---------------------------------------------------------------------------
template <class AF, class BF, class EF>
pac_status tb_gemm(pac_ctx* c, int M, int N, int K, int Z, const AF& A, const BF& Bm, const EF& E) {
    dim3 grid(cdiv(N, SG_BN), cdiv(M, SG_BM), (unsigned)Z);
    gemm_simt<<<grid, 256, 0, c->stream>>>(M, N, K, A, Bm, E);
    LAUNCH_CHECK(c);
    return PAC_OK;
}
#define TB_OK(call) do { pac_status s_ = (call); if (s_ != PAC_OK) return s_; } while (0)

pac_status tb_forward(pac_ctx* c, const int* d_ids, int B, bool train, float* d_logits_out) {
    const Dims& dm = c->dm;
    TBody& t = c->tb;
    const BodyLayout& bl = t.bl;
    Scratch& sc = c->sc;
    const int M = B * dm.S, r = dm.r, f = t.f;
    const long long n = (long long)M * r, stride = (long long)c->max_rows * r;
    cudaStream_t st = c->stream;
    TB_OK(down_projection(c, d_ids, B));
    const float* lam = c->params + c->lay.lam;
    const unsigned rows_grid = cdiv(M, 8), heads_grid = cdiv((long long)B * t.H * dm.S, 128);
    for (int l = 0; l < dm.L; ++l) {
        const float* w = c->params + c->lay.body + (long long)l * bl.per_layer;
        float *x = t.x + l * t.sMr, *xhat1 = t.xhat1 + l * t.sMr, *n1 = t.n1 + l * t.sMr, *qkv = t.qkv + 3 * l * t.sMr,
              *o = t.o + l * t.sMr, *x1 = t.x1 + l * t.sMr, *xhat2 = t.xhat2 + l * t.sMr, *n2 = t.n2 + l * t.sMr,
              *pre = t.pre + l * t.sMf, *P = t.P + l * t.sP, *a = sc.a + l * stride;
        tb_merge_kernel<<<cdiv(n, 256), 256, 0, st>>>(sc.u + l * stride, l ? sc.a + (l - 1) * stride : nullptr, lam, l, n, x);
        LAUNCH_CHECK(c);
        tb_layernorm_fwd_kernel<<<rows_grid, 256, 0, st>>>(x, w + bl.g1, w + bl.b1, M, r, n1, xhat1, t.rstd1 + l * t.sM);
        LAUNCH_CHECK(c);
        // q | k | v = n1 [Wq | Wk | Wv]  (three products in one launch: the weights are consecutive in the layout)
        TB_OK(tb_gemm(c, M, r, r, 3, MatA_RowMajor{{n1, 0, r}}, MatB_RowMajor{{w + bl.wq, (long long)r * r, r}},
                      StoreRowMajor{qkv, t.sMr, r}));
        tb_attn_fwd_kernel<<<heads_grid, 128, 0, st>>>(qkv, qkv + t.sMr, qkv + 2 * t.sMr, B, dm.S, r, t.H, P, o);
        LAUNCH_CHECK(c);
        TB_OK(tb_gemm(c, M, r, r, 1, MatA_RowMajor{{o, 0, r}}, MatB_RowMajor{{w + bl.wo, 0, r}}, StoreAddBias{x1, x, nullptr, r}));
        tb_layernorm_fwd_kernel<<<rows_grid, 256, 0, st>>>(x1, w + bl.g2, w + bl.b2, M, r, n2, xhat2, t.rstd2 + l * t.sM);
        LAUNCH_CHECK(c);
        TB_OK(tb_gemm(c, M, f, r, 1, MatA_RowMajor{{n2, 0, r}}, MatB_RowMajor{{w + bl.w1, 0, f}}, StoreAddBias{pre, nullptr, w + bl.c1, f}));
        TB_OK(tb_gemm(c, M, r, f, 1, MatA_ReluRowMajor{pre, f}, MatB_RowMajor{{w + bl.w2, 0, r}}, StoreAddBias{a, x1, w + bl.c2, r}));
    }
    // head: the same kernels as the point-wise plain path
    const float* aL = sc.a + (long long)(dm.L - 1) * stride;
    pool_tokens_kernel<<<B, 128, 0, st>>>(aL, sc.pooled_a, dm.S, r);
    LAUNCH_CHECK(c);
    const size_t smem = sizeof(float) * (dm.d + dm.C + 32);
    cls_head_kernel<<<B, 256, smem, st>>>(sc.hbar, d_ids, dm.N, c->labels, sc.pooled_a, c->params + c->lay.w_up,
                                          c->params + c->lay.w_head, c->params + c->lay.b_head, B, dm.S, dm.d, r, dm.C,
                                          train ? 1 : 0, sc.pooled_y, train ? sc.logits : d_logits_out, sc.loss_b, sc.dlogits,
                                          sc.gvec, sc.daL, c->status);
    LAUNCH_CHECK(c);
    return PAC_OK;
}

pac_status tb_backward(pac_ctx* c, const int* d_ids, int B, float* d_loss) {
    const Dims& dm = c->dm;
    TBody& t = c->tb;
    const BodyLayout& bl = t.bl;
    Scratch& sc = c->sc;
    const int M = B * dm.S, r = dm.r, f = t.f;
    const long long n = (long long)M * r, stride = (long long)c->max_rows * r;
    cudaStream_t st = c->stream;
    {
        const long long ne = (long long)r * dm.d + (long long)dm.d * dm.C + dm.C + 1;
        cls_grads_kernel<<<cdiv(ne, 256), 256, 0, st>>>(sc.pooled_a, sc.gvec, sc.pooled_y, sc.dlogits, sc.loss_b, B, dm.d, r, dm.C,
                                                        c->grads + c->lay.w_up, c->grads + c->lay.w_head, c->grads + c->lay.b_head, d_loss);
        LAUNCH_CHECK(c);
    }
    tb_expand_kernel<<<cdiv(n, 256), 256, 0, st>>>(sc.daL, dm.S, r, n, t.da);
    LAUNCH_CHECK(c);
    const float* lam = c->params + c->lay.lam;
    const unsigned rows_grid = cdiv(M, 8), heads_grid = cdiv((long long)B * t.H * dm.S, 128);
    for (int l = dm.L - 1; l >= 0; --l) {
        const float* w = c->params + c->lay.body + (long long)l * bl.per_layer;
        float* g = c->grads + c->lay.body + (long long)l * bl.per_layer;
        float *xhat1 = t.xhat1 + l * t.sMr, *n1 = t.n1 + l * t.sMr, *qkv = t.qkv + 3 * l * t.sMr, *o = t.o + l * t.sMr,
              *xhat2 = t.xhat2 + l * t.sMr, *n2 = t.n2 + l * t.sMr, *pre = t.pre + l * t.sMf, *P = t.P + l * t.sP;
        float *da = t.da, *dx1 = t.dx1, *dn = t.dn, *dqkv = t.dqkv, *dpre = t.dpre, *dtmp = t.dtmp;
        // a = x1 + relu(pre) W2 + c2
        tb_colsum_kernel<<<cdiv(r, 128), 128, 0, st>>>(da, nullptr, M, r, g + bl.c2);
        LAUNCH_CHECK(c);
        TB_OK(tb_gemm(c, f, r, M, 1, MatA_ReluColMajor{pre, f}, MatB_RowMajor{{da, 0, r}}, StoreRowMajor{g + bl.w2, 0, r}));
        TB_OK(tb_gemm(c, M, f, r, 1, MatA_RowMajor{{da, 0, r}}, MatB_ColMajor{{w + bl.w2, 0, r}}, StoreMaskedByPositive{dpre, pre, f}));
        tb_colsum_kernel<<<cdiv(f, 128), 128, 0, st>>>(dpre, nullptr, M, f, g + bl.c1);
        LAUNCH_CHECK(c);
        TB_OK(tb_gemm(c, r, f, M, 1, MatA_ColMajor{{n2, 0, r}}, MatB_RowMajor{{dpre, 0, f}}, StoreRowMajor{g + bl.w1, 0, f}));
        TB_OK(tb_gemm(c, M, r, f, 1, MatA_RowMajor{{dpre, 0, f}}, MatB_ColMajor{{w + bl.w1, 0, f}}, StoreRowMajor{dn, 0, r}));     // dn2
        tb_colsum_kernel<<<cdiv(r, 128), 128, 0, st>>>(dn, xhat2, M, r, g + bl.g2);
        LAUNCH_CHECK(c);
        tb_colsum_kernel<<<cdiv(r, 128), 128, 0, st>>>(dn, nullptr, M, r, g + bl.b2);
        LAUNCH_CHECK(c);
        tb_layernorm_bwd_kernel<<<rows_grid, 256, 0, st>>>(dn, xhat2, t.rstd2 + l * t.sM, w + bl.g2, da, M, r, dx1);             // dx1 = da + LN2 backward
        LAUNCH_CHECK(c);
        // x1 = x + o Wo
        TB_OK(tb_gemm(c, r, r, M, 1, MatA_ColMajor{{o, 0, r}}, MatB_RowMajor{{dx1, 0, r}}, StoreRowMajor{g + bl.wo, 0, r}));
        TB_OK(tb_gemm(c, M, r, r, 1, MatA_RowMajor{{dx1, 0, r}}, MatB_ColMajor{{w + bl.wo, 0, r}}, StoreRowMajor{dtmp, 0, r}));   // do
        float *dq = dqkv, *dk = dqkv + t.sMr, *dv = dqkv + 2 * t.sMr;
        tb_attn_bwd_dv_kernel<<<heads_grid, 128, 0, st>>>(P, dtmp, B, dm.S, r, t.H, dv);
        LAUNCH_CHECK(c);
        tb_attn_bwd_dq_kernel<<<heads_grid, 128, 0, st>>>(P, dtmp, qkv + t.sMr, qkv + 2 * t.sMr, B, dm.S, r, t.H, dq);
        LAUNCH_CHECK(c);
        tb_attn_bwd_dk_kernel<<<heads_grid, 128, 0, st>>>(P, qkv, B, dm.S, r, t.H, dk);
        LAUNCH_CHECK(c);
        // dWq | dWk | dWv = n1^T [dq | dk | dv]
        TB_OK(tb_gemm(c, r, r, M, 3, MatA_ColMajor{{n1, 0, r}}, MatB_RowMajor{{dqkv, t.sMr, r}}, StoreRowMajor{g + bl.wq, (long long)r * r, r}));
        // dn1 = dq Wq^T + dk Wk^T + dv Wv^T
        TB_OK(tb_gemm(c, M, r, r, 1, MatA_RowMajor{{dq, 0, r}}, MatB_ColMajor{{w + bl.wq, 0, r}}, StoreRowMajor{dn, 0, r}));
        TB_OK(tb_gemm(c, M, r, r, 1, MatA_RowMajor{{dk, 0, r}}, MatB_ColMajor{{w + bl.wk, 0, r}}, StoreAccumulate{dn, r}));
        TB_OK(tb_gemm(c, M, r, r, 1, MatA_RowMajor{{dv, 0, r}}, MatB_ColMajor{{w + bl.wv, 0, r}}, StoreAccumulate{dn, r}));
        tb_colsum_kernel<<<cdiv(r, 128), 128, 0, st>>>(dn, xhat1, M, r, g + bl.g1);
        LAUNCH_CHECK(c);
        tb_colsum_kernel<<<cdiv(r, 128), 128, 0, st>>>(dn, nullptr, M, r, g + bl.b1);
        LAUNCH_CHECK(c);
        tb_layernorm_bwd_kernel<<<rows_grid, 256, 0, st>>>(dn, xhat1, t.rstd1 + l * t.sM, w + bl.g1, dx1, M, r, dtmp);           // dx = dx1 + LN1 backward
        LAUNCH_CHECK(c);
        // x = lambda u + (1 - lambda) a_prev
        tb_unmerge_kernel<<<1, 1024, 0, st>>>(dtmp, sc.u + l * stride, l ? sc.a + (l - 1) * stride : nullptr, lam, l, n,
                                              sc.du + l * stride, da, c->grads + c->lay.lam);
        LAUNCH_CHECK(c);
    }
    return dw_down(c, d_ids, B, true);
}
#undef TB_OK

bool use_fused_cls(const pac_ctx* c) { return c->cfg.head == PAC_HEAD_MEANPOOL_CLS && c->mplan.ok; }
// The one-launch forward pays off when all of the batch's clusters run at the same time (its GEMM
// and chain phases do not overlap across waves); larger batches keep the two separate kernels.
bool use_fused_fwd(const pac_ctx* c, int B) {
    if (!use_fused_cls(c) || !use_tensor(c) || !c->fplan.ok) return false;
    if ((c->forward_mode == 4 || c->forward_mode == 5) && c->chain_ok) return false;
    return c->forward_mode == 3 || B <= c->fplan.max_clusters;
}
// Chain-in-epilogue forward: one CTA per 128-token tile walks all layers, so it needs enough tiles to fill
// the device (long sequences or large batches); the one-launch cluster forward keeps the short shapes.
bool use_chain_fwd(const pac_ctx* c, int B) {
    if (!use_fused_cls(c) || !use_tensor(c) || !c->chain_ok || c->forward_mode == 2 || c->forward_mode == 3) return false;
    if (c->forward_mode == 4 || c->forward_mode == 5) return true;
    if (use_fused_fwd(c, B)) return false;
    return 2 * B * c->tplan.fp.s_chunks >= c->sms;
}
int cls_cluster_size(const pac_ctx* c, int B) {
    return use_chain_fwd(c, B) ? c->pplan.G : use_fused_fwd(c, B) ? c->fplan.mp.G : c->mplan.G;
}

pac_status down_projection(pac_ctx* c, const int* d_ids, int B) {
    pac_status st;
    time_mark(c, 0, false);
    if (use_tensor(c)) {
        st = tensor_down_projection(c->tplan, c->stream, d_ids, B, c->sc.u, c->status, &c->launches, next_stamp(c, 0));
        if (st != PAC_OK) return fail(c, st, "tensor-core down-projection launch failed: %s", tensor_last_error());
    } else {
        st = c->dtype == PAC_F32 ? down_projection_simt<float>(c, d_ids, B) : down_projection_simt<bf16>(c, d_ids, B);
        if (st != PAC_OK) return st;
    }
    time_mark(c, 0, true);
    return PAC_OK;
}

pac_status dw_down(pac_ctx* c, const int* d_ids, int B, bool reduce_splits) {
    pac_status st;
    time_mark(c, 2, false);
    if (use_tensor(c)) {
        st = tensor_dw_down(c->tplan, c->stream, d_ids, B, c->sc.du16, c->grads + c->lay.w_down, c->sc.dw_part,
                            reduce_splits, c->status, &c->launches, next_stamp(c, 1),
                            c->step_early_ids && !c->step_host_ids);       // ids no kernel in flight writes
        if (st != PAC_OK) return fail(c, st, "tensor-core dW_down launch failed: %s", tensor_last_error());
    } else {
        st = c->dtype == PAC_F32 ? dw_down_simt<float>(c, d_ids, B) : dw_down_simt<bf16>(c, d_ids, B);
        if (st != PAC_OK) return st;
    }
    time_mark(c, 2, true);
    return PAC_OK;
}

MidParams mid_params(pac_ctx* c, const MidPlan& mp, const int* d_ids, int B, bool train, float* d_logits_out) {
    const Dims& dm = c->dm;
    Scratch& sc = c->sc;
    MidParams p{};
    p.ids = d_ids; p.N = dm.N; p.labels = c->labels;
    p.L = dm.L; p.S = dm.S; p.d = dm.d; p.r = dm.r; p.C = dm.C; p.B = B;
    p.G = mp.G; p.Sg = mp.Sg; p.dg = mp.dg; p.train = train ? 1 : 0;
    p.scratch = mp.scratch; p.aL_floats = (&mp == &c->pplan) ? 0 : mp.Sg * dm.r;
    p.u = sc.u; p.lstride = (long long)c->max_rows * dm.r;
    p.lam = c->params + c->lay.lam; p.W_up = c->params + c->lay.w_up;
    p.W_head = c->params + c->lay.w_head; p.b_head = c->params + c->lay.b_head; p.hbar = sc.hbar;
    p.du = use_tensor(c) ? (void*)sc.du16 : (void*)sc.du;
    p.pooled_a = sc.pooled_a; p.dlogits = sc.dlogits;
    p.loss_b = sc.loss_b; p.lam_part = sc.lam_part; p.logits_out = train ? sc.logits : d_logits_out;
    p.status = c->status;
    p.prodW = nullptr;
    return p;
}

// W_up W_head for the stand-alone head kernels, once per forward (launched ahead of the down-projections so that
// it overlaps the tail of the previous step's optimizer update).
pac_status head_matrix_enqueue(pac_ctx* c) {
    const Dims& dm = c->dm;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    pdl_launch_config(&cfg, attr, dim3(cdiv((long long)dm.r * dm.C, 8)), dim3(256), 0, c->stream);
    cudaError_t e = cudaLaunchKernelEx(&cfg, head_matrix_kernel, (const float*)(c->params + c->lay.w_up),
                                       (const float*)(c->params + c->lay.w_head), dm.d, dm.r, dm.C, c->sc.prodW);
    c->launches++;
    if (e != cudaSuccess) return fail(c, PAC_ERR_CUDA, "head matrix kernel launch failed: %s", cudaGetErrorString(e));
    return PAC_OK;
}

pac_status mid_enqueue(pac_ctx* c, const int* d_ids, int B, bool train, float* d_logits_out) {
    MidParams p = mid_params(c, c->mplan, d_ids, B, train, d_logits_out);
    p.prodW = c->sc.prodW;
    cudaError_t e = mid_launch(c->mplan, p, c->cfg.act, use_tensor(c), c->stream);
    c->launches++;
    if (e != cudaSuccess) return fail(c, PAC_ERR_CUDA, "fused head kernel launch failed: %s", cudaGetErrorString(e));
    return PAC_OK;
}

// Down-projections, chain, head, loss and reverse chain of a batch in one cluster launch.
pac_status fused_fwd_enqueue(pac_ctx* c, const int* d_ids, int B, bool train, float* d_logits_out) {
    const FusedFwdPlan& pl = c->fplan;
    FusedFwdParams fp{};
    fp.mid = mid_params(c, pl.mp, d_ids, B, train, d_logits_out);
    fp.mid.layers_per_cta = pl.layers_per_cta;
    if (c->step_host_ids) {
        fp.mid.host_ids = 1; fp.mid.ids_copy = c->sc.ids;
        const unsigned seq = (unsigned)(c->zc_count + 1);
        fp.mid.pref_ids = c->zc_dev_ids + (size_t)(seq & 1u) * c->cfg.max_batch;
        fp.mid.pref_tag = c->zc_dev_tag + (seq & 1u);
        fp.mid.pref_seq = seq;
    }
    fp.mid.early_ids = c->step_early_ids ? 1 : 0;
    fp.k_chunks = pl.k_chunks; fp.stages = pl.stages; fp.mid_offset = pl.mid_offset; fp.state_offset = pl.state_offset; fp.n_land = pl.n_land; fp.wide_n = pl.wide_n;
    fp.stamp = next_stamp(c, 0);
    cudaError_t e = fused_fwd_launch(pl, c->tplan.map_cache_fwd, c->tplan.map_w, fp, c->cfg.act, c->stream);
    c->launches++;
    if (e != cudaSuccess) return fail(c, PAC_ERR_CUDA, "fused forward kernel launch failed: %s", cudaGetErrorString(e));
    return PAC_OK;
}

// Down-projections with the chain in their epilogue, then head / loss / reverse chain from the parked state.
pac_status chain_fwd_enqueue(pac_ctx* c, const int* d_ids, int B, bool train, float* d_logits_out) {
    const Dims& dm = c->dm;
    ChainFwdParams cp{};
    cp.ids = d_ids; cp.N = dm.N; cp.L = dm.L; cp.S = dm.S; cp.d = dm.d; cp.r = dm.r; cp.B = B;
    cp.s_chunks = c->tplan.fp.s_chunks; cp.k_chunks = c->tplan.fp.k_chunks; cp.stages = c->tplan.fp.stages;
    cp.train = train ? 1 : 0;
    cp.lam = c->params + c->lay.lam;
    cp.parked = c->sc.du16; cp.layer_stride = (long long)c->max_rows * dm.r;
    cp.gates = c->sc.gates; cp.pool_part = c->sc.pool_part;
    cp.status = c->status; cp.stamp = next_stamp(c, 0);
    pac_status hs = head_matrix_enqueue(c);
    if (hs != PAC_OK) return hs;
    time_mark(c, 0, false);
    const bool pair = c->chain_pair_stages > 0 && c->forward_mode != 5 && ((B * cp.s_chunks) & 1) == 0;
    if (pair) cp.stages = c->chain_pair_stages;
    cudaError_t e = pair ? chain_pair_launch(c->tplan.map_cache_fwd, c->tplan.map_w, cp, chain_pair_smem(cp.stages), c->cfg.act, c->stream)
                         : chain_fwd_launch(c->tplan.map_cache_fwd, c->tplan.map_w, cp, c->tplan.smem_fwd, c->cfg.act, c->stream);
    c->launches++;
    time_mark(c, 0, true);
    if (e != cudaSuccess) return fail(c, PAC_ERR_CUDA, "chain-in-epilogue forward launch failed: %s", cudaGetErrorString(e));
    MidParams p = mid_params(c, c->pplan, d_ids, B, train, d_logits_out);
    p.gates = c->sc.gates; p.pool_part = c->sc.pool_part; p.n_pool_parts = cp.s_chunks * CF_POOL_PARTS;
    p.prodW = c->sc.prodW;
    time_mark(c, 1, false);
    e = mid_launch_parked(c->pplan, p, c->cfg.act, c->stream);
    c->launches++;
    time_mark(c, 1, true);
    if (e != cudaSuccess) return fail(c, PAC_ERR_CUDA, "head kernel launch failed: %s", cudaGetErrorString(e));
    return PAC_OK;
}

// Forward half of a classifier-head step (everything up to du and the per-sample head vectors).
pac_status cls_forward_enqueue(pac_ctx* c, const int* d_ids, int B, bool train, float* d_logits_out) {
    pac_status st;
    if (use_chain_fwd(c, B)) return chain_fwd_enqueue(c, d_ids, B, train, d_logits_out);
    if (use_fused_fwd(c, B)) {
        time_mark(c, 0, false);
        st = fused_fwd_enqueue(c, d_ids, B, train, d_logits_out);
        time_mark(c, 0, true);
        return st;
    }
    if ((st = head_matrix_enqueue(c)) != PAC_OK) return st;
    if ((st = down_projection(c, d_ids, B)) != PAC_OK) return st;
    time_mark(c, 1, false);
    st = mid_enqueue(c, d_ids, B, train, d_logits_out);
    time_mark(c, 1, true);
    return st;
}

void bias_corrections(const pac_adamw* hp, long long step, float* bc1, float* bc2) {
    *bc1 = (float)(1.0 - std::pow((double)hp->beta1, (double)step));
    *bc2 = (float)(1.0 - std::pow((double)hp->beta2, (double)step));
}

pac_status finalize_enqueue(pac_ctx* c, const int* d_ids, int B, float* d_loss, const pac_adamw* hp) {
    const Dims& dm = c->dm;
    Scratch& sc = c->sc;
    FinalizeParams f{};
    f.lay = c->lay; f.B = B; f.d = dm.d; f.r = dm.r; f.C = dm.C; f.L = dm.L;
    f.dw_part = sc.dw_part;
    f.splits = use_tensor(c) ? tensor_splits(c->tplan, B) : 1;
    f.dw_elems = (long long)dm.L * dm.d * dm.r;
    f.lam_part = sc.lam_part; f.lam_blocks = B * cls_cluster_size(c, B);
    f.pooled_a = sc.pooled_a; f.dlogits = sc.dlogits; f.loss_b = sc.loss_b;
    f.hbar = sc.hbar; f.ids = d_ids; f.N = dm.N; f.params_in = c->params;
    f.grads = c->grads; f.loss_out = d_loss;
    f.adam = hp ? 1 : 0;
    if (hp) {
        c->step += 1;
        f.params = c->params; f.m = c->m; f.v = c->v; f.hp = *hp;
        bias_corrections(hp, c->step, &f.bc1, &f.bc2);
        f.wdT = sc.wdT;
        f.grad_scale = c->grad_scale;
    }
    f.wd_blocks = (int)cdiv(c->lay.lam / 4, 256);
    if (c->step_host_ids) {
        // the step after this one will look for its ids under sequence number zc_count + 2 in the next ring slot
        const unsigned next_seq = (unsigned)(c->zc_count + 2);
        const int next_slot = (int)((c->zc_count + 1) % ZC_SLOTS);
        f.next_host_ids = c->zc_ids + (size_t)next_slot * c->cfg.max_batch;
        f.next_host_tag = c->zc_tags + next_slot;
        f.next_seq = next_seq; f.next_n = c->cfg.max_batch;
        f.next_dev_ids = c->zc_dev_ids + (size_t)(next_seq & 1u) * c->cfg.max_batch;
        f.next_dev_tag = c->zc_dev_tag + (next_seq & 1u);
    }
    f.status = c->status;
    const unsigned rest_blocks = cdiv(dm.d, FIN_KB);
    f.rest_blocks = (int)rest_blocks;
    const size_t fin_smem = sizeof(float) * ((size_t)2 * B * FIN_KB + (size_t)dm.r * FIN_KB + (size_t)FIN_KB * dm.C);
    if (fin_smem > 48 * 1024) return fail(c, PAC_ERR_UNSUPPORTED, "finalisation: batch or adapter width beyond its shared memory");
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    pdl_launch_config(&cfg, attr, dim3(f.wd_blocks + rest_blocks + 1), dim3(256), fin_smem, c->stream);   // + one block for lambda and the loss
    cudaError_t le = cudaLaunchKernelEx(&cfg, finalize_cls_kernel, f);
    c->launches++;
    if (le != cudaSuccess) return fail(c, PAC_ERR_CUDA, "finalize kernel launch failed: %s", cudaGetErrorString(le));
    return PAC_OK;
}

// One whole train step; with hp != NULL the AdamW update is fused into the last kernel.
pac_status train_enqueue(pac_ctx* c, const int* d_ids, int B, float* d_loss, const pac_adamw* hp) {
    pac_status st;
    if (c->tb.on) {
        if ((st = tb_forward(c, d_ids, B, true, nullptr)) != PAC_OK) return st;
        if ((st = tb_backward(c, d_ids, B, d_loss)) != PAC_OK) return st;
        return hp ? adam_enqueue(c, hp) : PAC_OK;
    }
    if (use_fused_cls(c)) {
        if ((st = cls_forward_enqueue(c, d_ids, B, true, nullptr)) != PAC_OK) return st;
        if (c->step_host_ids) d_ids = c->sc.ids;          // the forward kernel left a device copy for the later kernels
        if ((st = dw_down(c, d_ids, B, false)) != PAC_OK) return st;
        time_mark(c, 3, false);
        st = finalize_enqueue(c, d_ids, B, d_loss, hp);
        time_mark(c, 3, true);
        return st;
    }
    if ((st = forward(c, d_ids, B, true, nullptr)) != PAC_OK) return st;
    if ((st = backward(c, d_ids, B, d_loss)) != PAC_OK) return st;
    if (hp) return adam_enqueue(c, hp);
    return PAC_OK;
}

pac_status adam_enqueue(pac_ctx* c, const pac_adamw* hp) {
    c->step += 1;
    float bc1, bc2;
    bias_corrections(hp, c->step, &bc1, &bc2);
    const int wd_blocks = (c->lay.lam % 4 == 0) ? (int)cdiv(c->lay.lam / 4, 256) : 0;
    const unsigned rest = cdiv(c->lay.total - (wd_blocks ? c->lay.lam : 0), 256);
    adamw_kernel<<<wd_blocks + rest, 256, 0, c->stream>>>(c->params, c->grads, c->m, c->v, c->lay.total, c->lay, *hp, bc1, bc2,
                                                          c->sc.wdT, c->dm.d, c->dm.r, wd_blocks, c->status, c->grad_scale);
    LAUNCH_CHECK(c);
    return PAC_OK;
}

pac_status check_hp(pac_ctx* c, const pac_adamw* hp) {
    if (!hp) return fail(c, PAC_ERR_INVALID_ARG, "AdamW hyper-parameters are NULL");
    if (!(hp->lr >= 0.f) || !(hp->beta1 >= 0.f && hp->beta1 < 1.f) || !(hp->beta2 >= 0.f && hp->beta2 < 1.f) ||
        !(hp->eps > 0.f) || !(hp->weight_decay >= 0.f))
        return fail(c, PAC_ERR_INVALID_ARG, "AdamW hyper-parameters out of range");
    return PAC_OK;
}

pac_status refresh_shadow(pac_ctx* c) {
    if (!c->sc.wdT) return PAC_OK;
    long long n = (long long)c->dm.L * c->dm.d * c->dm.r;
    shadow_wdown_kernel<<<cdiv(n, 256), 256, 0, c->stream>>>(c->params, c->sc.wdT, c->dm.L, c->dm.d, c->dm.r);
    LAUNCH_CHECK(c);
    return PAC_OK;
}

void free_all(pac_ctx* c) {
    Scratch& s = c->sc;
    if (c->hc.on) s.hbar = nullptr;            // points into a staging slot, freed below
    void* ptrs[] = {s.ids, s.u, s.a, s.du, s.du16, s.lam_part, s.loss, s.hbar, s.pooled_a, s.pooled_y, s.logits,
                    s.dlogits, s.loss_b, s.gvec, s.daL, s.y, s.lm_logits, s.dy, s.y16, s.dlog16, s.aL16, s.wup16, s.dy16, s.wdT, s.lm_part, s.dw_part, s.gates, s.pool_part, s.prodW, c->tb.buf, c->params, c->grads,
                    c->m, c->v, c->status, c->d_perm, c->d_losses, c->d_stamps};
    for (void* p : ptrs)
        if (p) cudaFree(p);
    for (int k = 0; k < 2; ++k) {
        if (c->hc.stage[k]) cudaFree(c->hc.stage[k]);
        if (c->hc.lab_stage[k]) cudaFree(c->hc.lab_stage[k]);
        if (c->hc.hbar_stage[k]) cudaFree(c->hc.hbar_stage[k]);
        if (c->hc.h_lab[k]) cudaFreeHost(c->hc.h_lab[k]);
        if (c->hc.ready[k]) cudaEventDestroy(c->hc.ready[k]);
        if (c->hc.freed[k]) cudaEventDestroy(c->hc.freed[k]);
    }
    if (c->hc.iota) cudaFree(c->hc.iota);
    if (c->hc.copy_stream) cudaStreamDestroy(c->hc.copy_stream);
    if (c->hc.map_base) munmap(c->hc.map_base, c->hc.map_bytes);
    if (c->zc_ids) cudaFreeHost(c->zc_ids);
    if (c->zc_tags) cudaFreeHost(c->zc_tags);
    if (c->zc_dev_ids) cudaFree(c->zc_dev_ids);
    if (c->zc_dev_tag) cudaFree(c->zc_dev_tag);
    for (auto& e : c->zc_ev)
        if (e) cudaEventDestroy(e);
    if (c->h_ids) cudaFreeHost(c->h_ids);
    if (c->h_loss) cudaFreeHost(c->h_loss);
    if (c->h_status) cudaFreeHost(c->h_status);
    for (auto& e : c->slot_ev)
        if (e) cudaEventDestroy(e);
    for (auto& vec : c->tev)
        for (auto& e : vec) cudaEventDestroy(e);
    if (c->own_stream && c->stream) cudaStreamDestroy(c->stream);
}

#define NEED_CTX(c) do { if (!(c)) return PAC_ERR_INVALID_ARG; } while (0)
#define NEED_INIT(c, who)                                                                          \
    do {                                                                                           \
        NEED_CTX(c);                                                                               \
        if (!(c)->inited) return fail(c, PAC_ERR_BAD_STATE, "%s: call pac_adapter_init first", who); \
        cudaError_t e_ = cudaSetDevice((c)->device);                                               \
        if (e_ != cudaSuccess) return fail(c, PAC_ERR_CUDA, "cudaSetDevice: %s", cudaGetErrorString(e_)); \
    } while (0)

}  // namespace

extern "C" {

pac_status pac_create(pac_ctx** out, int device, void* cuda_stream) {
    if (!out) return PAC_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || count == 0) return PAC_ERR_CUDA;   // no CPU fallback
    if (device < 0 || device >= count) return PAC_ERR_INVALID_ARG;
    if (cudaSetDevice(device) != cudaSuccess) return PAC_ERR_CUDA;
    pac_ctx* c = new (std::nothrow) pac_ctx();
    if (!c) return PAC_ERR_NOMEM;
    c->device = device;
    if (cudaDeviceGetAttribute(&c->sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || c->sms < 1) c->sms = 1;
    if (cuda_stream) {
        c->stream = (cudaStream_t)cuda_stream;
    } else {
        if (cudaStreamCreateWithFlags(&c->stream, cudaStreamNonBlocking) != cudaSuccess) { delete c; return PAC_ERR_CUDA; }
        c->own_stream = true;
    }
    bool ok = cudaMalloc((void**)&c->status, sizeof(unsigned) * ST_WORDS) == cudaSuccess &&
              cudaMemsetAsync(c->status, 0, sizeof(unsigned) * ST_WORDS, c->stream) == cudaSuccess &&
              cudaMallocHost((void**)&c->h_loss, sizeof(float)) == cudaSuccess &&
              cudaMallocHost((void**)&c->h_status, sizeof(unsigned) * ST_WORDS) == cudaSuccess;
    for (auto& e : c->slot_ev) ok = ok && cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) { free_all(c); delete c; return PAC_ERR_CUDA; }
    *out = c;
    return PAC_OK;
}

pac_status pac_destroy(pac_ctx* c) {
    NEED_CTX(c);
    cudaSetDevice(c->device);
    cudaStreamSynchronize(c->stream);
    tensor_plan_destroy(c->tplan);
    free_all(c);
    delete c;
    return PAC_OK;
}

pac_status pac_cache_register(pac_ctx* c, const void* dev_cache, int dtype, long long N, int L, int S, int d,
                              const int* dev_labels, int labels_per_sample) {
    NEED_CTX(c);
    if (c->inited) return fail(c, PAC_ERR_BAD_STATE, "pac_cache_register: adapters already initialised");
    if (!dev_cache || !dev_labels) return fail(c, PAC_ERR_INVALID_ARG, "pac_cache_register: NULL device pointer");
    if (dtype != PAC_F32 && dtype != PAC_BF16) return fail(c, PAC_ERR_INVALID_ARG, "pac_cache_register: bad dtype %d", dtype);
    if (N < 1 || L < 1 || S < 1 || d < 1) return fail(c, PAC_ERR_INVALID_ARG, "pac_cache_register: sizes must be positive");
    if (N > 0x7fffffffLL) return fail(c, PAC_ERR_UNSUPPORTED, "pac_cache_register: N beyond int32 sample ids");
    if ((long long)L * S > 0x7fffffffLL / 4) return fail(c, PAC_ERR_UNSUPPORTED, "pac_cache_register: L*S too large");
    if (labels_per_sample != 1 && labels_per_sample != S)
        return fail(c, PAC_ERR_INVALID_ARG, "pac_cache_register: labels_per_sample must be 1 or S");
    if (((uintptr_t)dev_cache & 15) != 0) return fail(c, PAC_ERR_INVALID_ARG, "pac_cache_register: cache not 16-byte aligned");
    c->cache = dev_cache; c->dtype = dtype;
    c->dm.N = N; c->dm.L = L; c->dm.S = S; c->dm.d = d;
    c->labels = dev_labels; c->labels_per_sample = labels_per_sample;
    c->registered = true;
    return PAC_OK;
}

pac_status pac_cache_register_host(pac_ctx* c, const void* host_cache, int dtype, long long N, int L, int S, int d,
                                   const int* host_labels, int labels_per_sample) {
    NEED_CTX(c);
    // same checks as for a device-resident cache; the pointers are host memory here
    pac_status st = pac_cache_register(c, host_cache, dtype, N, L, S, d, host_labels, labels_per_sample);
    if (st != PAC_OK) return st;
    c->hc.on = true;
    c->hc.host = (const unsigned char*)host_cache;
    c->hc.host_labels = host_labels;
    c->hc.N = N;
    c->hc.sample_bytes = (long long)L * S * d * (dtype == PAC_F32 ? 4 : 2);
    c->cache = nullptr;                  // bound to a staging slot before every use
    c->labels = nullptr;
    return PAC_OK;
}

pac_status pac_cache_register_file(pac_ctx* c, const char* path) {
    NEED_CTX(c);
    if (!path) return fail(c, PAC_ERR_INVALID_ARG, "pac_cache_register_file: path is NULL");
    if (c->inited) return fail(c, PAC_ERR_BAD_STATE, "pac_cache_register_file: adapters already initialised");
    if (c->hc.map_base) return fail(c, PAC_ERR_BAD_STATE, "pac_cache_register_file: a cache file is already registered");
    const int fd = open(path, O_RDONLY);
    if (fd < 0) return fail(c, PAC_ERR_INVALID_ARG, "pac_cache_register_file: cannot open %s", path);
    CacheFileHeader h;
    struct stat sb;
    if (read(fd, &h, sizeof h) != (ssize_t)sizeof h || !cache_file_header_ok(h) || fstat(fd, &sb) != 0 ||
        (size_t)sb.st_size < cache_file_bytes(h)) {
        close(fd);
        return fail(c, PAC_ERR_INVALID_ARG, "pac_cache_register_file: %s is not a complete cache file", path);
    }
    const size_t bytes = cache_file_bytes(h);
    void* base = mmap(nullptr, bytes, PROT_READ, MAP_SHARED, fd, 0);
    close(fd);
    if (base == MAP_FAILED) return fail(c, PAC_ERR_NOMEM, "pac_cache_register_file: mmap of %zu bytes failed", bytes);
    const unsigned char* data = (const unsigned char*)base + sizeof(CacheFileHeader);
    const int* labels = (const int*)((const unsigned char*)base + cache_file_labels_offset(h));
    pac_status st = pac_cache_register_host(c, data, h.dtype, h.N, h.L, h.S, h.d, labels, h.labels_per_sample);
    if (st != PAC_OK) { munmap(base, bytes); return st; }
    c->hc.map_base = base;
    c->hc.map_bytes = bytes;
    return PAC_OK;
}

pac_status pac_adapter_init(pac_ctx* c, const pac_adapter_cfg* cfg, unsigned long long seed) {
    NEED_CTX(c);
    if (!c->registered) return fail(c, PAC_ERR_BAD_STATE, "pac_adapter_init: call pac_cache_register first");
    if (c->inited) return fail(c, PAC_ERR_BAD_STATE, "pac_adapter_init: already initialised");
    if (!cfg) return fail(c, PAC_ERR_INVALID_ARG, "pac_adapter_init: cfg is NULL");
    if (cfg->r < 1 || cfg->n_out < 1 || cfg->max_batch < 1) return fail(c, PAC_ERR_INVALID_ARG, "pac_adapter_init: sizes must be positive");
    if (cfg->act != PAC_ACT_RELU && cfg->act != PAC_ACT_IDENTITY) return fail(c, PAC_ERR_INVALID_ARG, "pac_adapter_init: bad activation");
    if (cfg->head != PAC_HEAD_MEANPOOL_CLS && cfg->head != PAC_HEAD_FROZEN_LM) return fail(c, PAC_ERR_INVALID_ARG, "pac_adapter_init: bad head");
    const bool cls = cfg->head == PAC_HEAD_MEANPOOL_CLS;
    if (cls && c->labels_per_sample != 1) return fail(c, PAC_ERR_INVALID_ARG, "pac_adapter_init: classifier head needs one label per sample");
    if (!cls && c->labels_per_sample != c->dm.S) return fail(c, PAC_ERR_INVALID_ARG, "pac_adapter_init: LM head needs S targets per sample");
    if (!cls && !cfg->lm_head) return fail(c, PAC_ERR_INVALID_ARG, "pac_adapter_init: LM head pointer is NULL");
    if (cls && cfg->n_out > 4096) return fail(c, PAC_ERR_UNSUPPORTED, "pac_adapter_init: classifier head supports up to 4096 classes");
    if ((long long)cfg->max_batch * c->dm.S > 0x7fffffffLL / 8) return fail(c, PAC_ERR_UNSUPPORTED, "pac_adapter_init: max_batch*S too large");
    if (cfg->body != PAC_BODY_POINTWISE && cfg->body != PAC_BODY_TRANSFORMER) return fail(c, PAC_ERR_INVALID_ARG, "pac_adapter_init: bad body");
    if (cfg->body == PAC_BODY_TRANSFORMER) {
        if (!cls) return fail(c, PAC_ERR_UNSUPPORTED, "pac_adapter_init: transformer-body adapters need the classifier head");
        if (cfg->n_heads < 1 || cfg->r % cfg->n_heads != 0 || cfg->ffn_width < 1)
            return fail(c, PAC_ERR_INVALID_ARG, "pac_adapter_init: transformer body needs n_heads dividing r and a positive ffn_width");
        if (c->hc.on) return fail(c, PAC_ERR_UNSUPPORTED, "pac_adapter_init: transformer-body adapters need a device-resident cache");
    }
    CU_OK(c, cudaSetDevice(c->device));
    c->cfg = *cfg;
    c->dm.r = cfg->r; c->dm.C = cfg->n_out;
    c->tb.on = cfg->body == PAC_BODY_TRANSFORMER;
    if (c->hc.on) {
        // the kernels see a staging slot: a cache of max_batch samples
        HostCache& h = c->hc;
        c->dm.N = cfg->max_batch;
        const size_t lab_n = (size_t)cfg->max_batch * c->labels_per_sample;
        CU_OK(c, cudaStreamCreateWithFlags(&h.copy_stream, cudaStreamNonBlocking));
        for (int k = 0; k < 2; ++k) {
            CU_OK(c, cudaMalloc((void**)&h.stage[k], (size_t)cfg->max_batch * h.sample_bytes));
            CU_OK(c, cudaMalloc((void**)&h.lab_stage[k], sizeof(int) * lab_n));
            CU_OK(c, cudaMalloc((void**)&h.hbar_stage[k], sizeof(float) * (size_t)cfg->max_batch * c->dm.d));
            CU_OK(c, cudaMallocHost((void**)&h.h_lab[k], sizeof(int) * lab_n));
            CU_OK(c, cudaEventCreateWithFlags(&h.ready[k], cudaEventDisableTiming));
            CU_OK(c, cudaEventCreateWithFlags(&h.freed[k], cudaEventDisableTiming));
        }
        std::vector<int> iota(cfg->max_batch);
        for (int b = 0; b < cfg->max_batch; ++b) iota[b] = b;
        CU_OK(c, cudaMalloc((void**)&h.iota, sizeof(int) * cfg->max_batch));
        CU_OK(c, cudaMemcpy(h.iota, iota.data(), sizeof(int) * cfg->max_batch, cudaMemcpyHostToDevice));
        c->cache = h.stage[0];
        c->labels = h.lab_stage[0];
    }
    const Dims& dm = c->dm;
    c->lay = ParamLayout::make(dm.L, dm.d, dm.r, dm.C, cls);
    if (c->tb.on) {
        c->tb.H = cfg->n_heads; c->tb.f = cfg->ffn_width;
        c->tb.bl = BodyLayout::make(dm.r, cfg->ffn_width);
        c->lay.body_per = c->tb.bl.per_layer; c->lay.br = dm.r; c->lay.bf = cfg->ffn_width;
        c->lay.total = c->lay.body + (long long)dm.L * c->tb.bl.per_layer;
    }
    c->max_rows = cfg->max_batch * dm.S;
    const long long Mr = (long long)c->max_rows * dm.r;
    c->chain_blocks_max = (int)cdiv(Mr, 256);
    c->mplan = (cls && !c->tb.on) ? mid_plan(dm) : MidPlan{};
    if (c->mplan.ok && cfg->max_batch * 8 > c->chain_blocks_max) c->chain_blocks_max = cfg->max_batch * 8;     // clusters of up to 8
    FusedFwdPlan fwd_plan{};
    if (c->mplan.ok && c->dtype == PAC_BF16 && tensor_shape_supported(dm) && !c->force_simt && c->forward_mode != 2) {
        int max_smem = 0;
        CU_OK(c, cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, c->device));
        fwd_plan = fused_fwd_plan(dm, max_smem);
        if (fwd_plan.ok && cfg->max_batch * fwd_plan.mp.G > c->chain_blocks_max) c->chain_blocks_max = cfg->max_batch * fwd_plan.mp.G;
    }
    c->fplan = FusedFwdPlan{};
    Scratch& s = c->sc;
    pac_status st = PAC_OK;
    auto A = [&](pac_status x) { if (st == PAC_OK) st = x; };
    A(dmalloc(c, &c->params, c->lay.total)); A(dmalloc(c, &c->grads, c->lay.total));
    A(dmalloc(c, &c->m, c->lay.total)); A(dmalloc(c, &c->v, c->lay.total));
    A(dmalloc(c, &s.ids, cfg->max_batch));
    A(dmalloc(c, &s.u, Mr * dm.L)); A(dmalloc(c, &s.a, Mr * dm.L));
    A(dmalloc(c, &s.lam_part, (long long)dm.L * c->chain_blocks_max));
    A(dmalloc(c, &s.loss, 1));
    if (cls) {
        if (c->hc.on) s.hbar = c->hc.hbar_stage[0];
        else A(dmalloc(c, &s.hbar, dm.N * dm.d));
        A(dmalloc(c, &s.pooled_a, (long long)cfg->max_batch * dm.r));
        A(dmalloc(c, &s.pooled_y, (long long)cfg->max_batch * dm.d));
        A(dmalloc(c, &s.logits, (long long)cfg->max_batch * dm.C));
        A(dmalloc(c, &s.dlogits, (long long)cfg->max_batch * dm.C));
        A(dmalloc(c, &s.loss_b, cfg->max_batch));
        A(dmalloc(c, &s.gvec, (long long)cfg->max_batch * dm.d));
        A(dmalloc(c, &s.daL, (long long)cfg->max_batch * dm.r));
        A(dmalloc(c, &s.prodW, (long long)dm.r * dm.C));
    } else {
        A(dmalloc(c, &s.loss_b, c->max_rows));
        A(dmalloc(c, &s.daL, Mr));
        A(dmalloc(c, &s.lm_logits, (long long)c->max_rows * dm.C));
        A(dmalloc(c, &s.dy, (long long)c->max_rows * dm.d));
        A(dmalloc(c, &s.lm_part, LM_MAX_K_SLICES * std::max((long long)dm.r * dm.d, Mr)));
        // the two dense LM-head GEMMs go to the tensor cores for bf16 caches with 16-byte operand rows
        c->lm_tensor = false;
        if (st == PAC_OK && c->dtype == PAC_BF16 && !c->force_simt && dm.d % 8 == 0 && dm.C % 8 == 0) {
            A(dmalloc(c, &s.y16, (long long)c->max_rows * dm.d));
            A(dmalloc(c, &s.dlog16, (long long)c->max_rows * dm.C));
            if (st == PAC_OK) {
                pac_status g1 = gemm_plan_create(c->g_logits, c->device, s.y16, c->max_rows, (const bf16*)cfg->lm_head, dm.C, dm.d, 0, c->forward_mode != 5);
                pac_status g2 = g1 == PAC_OK ? gemm_plan_create(c->g_dy, c->device, s.dlog16, c->max_rows, (const bf16*)cfg->lm_head, dm.d, dm.C, 1, c->forward_mode != 5) : g1;
                if (g1 == PAC_OK && g2 == PAC_OK) {
                    c->lm_tensor = true;
                    int max_smem = 0;
                    c->lm_ce_stream = cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, c->device) == cudaSuccess &&
                                      lm_ce_stream_supported(dm.C, max_smem);
                }
                else if ((g1 != PAC_OK && g1 != PAC_ERR_UNSUPPORTED) || (g2 != PAC_OK && g2 != PAC_ERR_UNSUPPORTED))
                    st = fail(c, PAC_ERR_CUDA, "LM-head GEMM set-up failed: %s", tensor_last_error());
            }
        }
        if (st == PAC_OK && !c->lm_tensor) A(dmalloc(c, &s.y, (long long)c->max_rows * dm.d));
    }
    if (st == PAC_OK && cudaMallocHost((void**)&c->h_ids, sizeof(int) * STAGE_SLOTS * cfg->max_batch) != cudaSuccess)
        st = fail(c, PAC_ERR_NOMEM, "pinned id staging allocation failed");
    if (st == PAC_OK && fwd_plan.ok) {
        // id ring of pac_train_step_async (only the one-launch forward reads ids from host memory)
        if (cudaMallocHost((void**)&c->zc_ids, sizeof(int) * ZC_SLOTS * cfg->max_batch) != cudaSuccess ||
            cudaMallocHost((void**)&c->zc_tags, sizeof(unsigned) * ZC_SLOTS) != cudaSuccess ||
            cudaMalloc((void**)&c->zc_dev_ids, sizeof(int) * 2 * cfg->max_batch) != cudaSuccess ||
            cudaMalloc((void**)&c->zc_dev_tag, sizeof(unsigned) * 2) != cudaSuccess ||
            cudaMemset(c->zc_dev_tag, 0, sizeof(unsigned) * 2) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->zc_ev[0], cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->zc_ev[1], cudaEventDisableTiming) != cudaSuccess)
            st = fail(c, PAC_ERR_NOMEM, "pinned id ring allocation failed");
        else
        {
            std::memset(c->zc_tags, 0, sizeof(unsigned) * ZC_SLOTS);      // sequence numbers start at 1
            std::memset(c->zc_ids, 0, sizeof(int) * ZC_SLOTS * cfg->max_batch);
        }
    }
    // tensor-core path: bf16 cache with TMA/UMMA-compatible sizes
    c->tensor_ok = false;
    if (st == PAC_OK && c->dtype == PAC_BF16 && tensor_shape_supported(dm) && !c->tb.on) {
        A(dmalloc(c, &s.wdT, (long long)dm.L * 2 * dm.r * dm.d));
        A(dmalloc(c, &s.du16, Mr * dm.L));
        long long part_floats = 0;
        if (st == PAC_OK) {
            pac_status ts = tensor_plan_create(c->tplan, c->device, (const bf16*)c->cache, dm, cfg->max_batch, s.wdT,
                                               s.du16, &part_floats);
            if (ts == PAC_OK && c->hc.on) {
                // one set of tensor maps per staging slot
                c->hc.tplan[0] = c->tplan;
                long long pf2 = 0;
                ts = tensor_plan_create(c->hc.tplan[1], c->device, (const bf16*)c->hc.stage[1], dm, cfg->max_batch, s.wdT, s.du16, &pf2);
            }
            if (ts == PAC_OK) {
                A(dmalloc(c, &s.dw_part, part_floats));
                c->chain_ok = false;
                if (st == PAC_OK && cls && c->mplan.ok && chain_fwd_supported(dm) && c->tplan.fp.wide_n) {
                    c->pplan = mid_plan_parked(dm);
                    if (c->pplan.ok) {
                        A(dmalloc(c, &s.gates, Mr));
                        A(dmalloc(c, &s.pool_part, (long long)cfg->max_batch * c->tplan.fp.s_chunks * CF_POOL_PARTS * dm.r));
                        c->chain_ok = (st == PAC_OK);
                        int max_smem = 0;
                        if (c->chain_ok && chain_pair_supported(dm) &&
                            cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, c->device) == cudaSuccess) {
                            const int ps = chain_pair_stages(max_smem);
                            c->chain_pair_stages = ps >= 3 ? ps : 0;
                        }
                    }
                }
                c->tensor_ok = (st == PAC_OK);
                if (c->tensor_ok && fwd_plan.ok) {
                    fwd_plan.max_clusters = fused_fwd_max_clusters(fwd_plan, cfg->act);
                    if (fwd_plan.max_clusters > 0) c->fplan = fwd_plan;
                }
            } else if (ts != PAC_ERR_UNSUPPORTED) {
                st = fail(c, ts, "tensor path set-up failed: %s", tensor_last_error());
            }
        }
    }
    c->lm_skinny_tensor = false;
    if (st == PAC_OK && c->lm_tensor && c->tensor_ok && dm.r % 8 == 0 && dm.r <= 256 && (Mr % 4 == 0) && ((long long)dm.r * dm.d) % 4 == 0) {
        A(dmalloc(c, &s.aL16, Mr)); A(dmalloc(c, &s.wup16, (long long)dm.r * dm.d)); A(dmalloc(c, &s.dy16, (long long)c->max_rows * dm.d));
        if (st == PAC_OK) {
            CU_OK(c, cudaMemsetAsync(s.aL16, 0, sizeof(bf16) * Mr, c->stream));
            CU_OK(c, cudaMemsetAsync(s.dy16, 0, sizeof(bf16) * (size_t)c->max_rows * dm.d, c->stream));
            pac_status g1 = gemm_plan_create(c->g_y, c->device, s.aL16, c->max_rows, s.wup16, dm.d, dm.r, 1, c->forward_mode != 5);
            pac_status g2 = g1 == PAC_OK ? gemm_plan_create(c->g_daL, c->device, s.dy16, c->max_rows, s.wup16, dm.r, dm.d, 0, c->forward_mode != 5) : g1;
            c->lm_skinny_tensor = g1 == PAC_OK && g2 == PAC_OK;
        }
    }
    if (st == PAC_OK && !use_tensor(c)) A(dmalloc(c, &s.du, Mr * dm.L));    // the plain path keeps du in fp32
    if (st == PAC_OK && c->tb.on) {
        TBody& t = c->tb;
        const long long Mx = c->max_rows;
        t.sMr = Mx * dm.r; t.sMf = Mx * t.f; t.sP = (long long)cfg->max_batch * t.H * dm.S * dm.S; t.sM = Mx;
        const long long per_layer = 10 * t.sMr + t.sMf + t.sP + 2 * t.sM;     // x xhat1 n1 qkv(3) o x1 xhat2 n2 | pre | P | rstd1 rstd2
        const long long work = 7 * t.sMr + t.sMf;                             // da dx1 dn dqkv(3) dtmp | dpre
        A(dmalloc(c, &t.buf, per_layer * dm.L + work));
        if (st == PAC_OK) {
            float* q = t.buf;
            auto take = [&](long long k) { float* r_ = q; q += k; return r_; };
            t.x = take(t.sMr * dm.L); t.xhat1 = take(t.sMr * dm.L); t.n1 = take(t.sMr * dm.L); t.qkv = take(3 * t.sMr * dm.L);
            t.o = take(t.sMr * dm.L); t.x1 = take(t.sMr * dm.L); t.xhat2 = take(t.sMr * dm.L); t.n2 = take(t.sMr * dm.L);
            t.pre = take(t.sMf * dm.L); t.P = take(t.sP * dm.L); t.rstd1 = take(t.sM * dm.L); t.rstd2 = take(t.sM * dm.L);
            t.da = take(t.sMr); t.dx1 = take(t.sMr); t.dn = take(t.sMr); t.dqkv = take(3 * t.sMr); t.dtmp = take(t.sMr);
            t.dpre = take(t.sMf);
        }
    }
    if (st != PAC_OK) return st;
    CU_OK(c, cudaMemsetAsync(s.u, 0, sizeof(float) * Mr * dm.L, c->stream));
    CU_OK(c, cudaMemsetAsync(s.a, 0, sizeof(float) * Mr * dm.L, c->stream));
    if (s.du) CU_OK(c, cudaMemsetAsync(s.du, 0, sizeof(float) * Mr * dm.L, c->stream));
    if (s.du16) CU_OK(c, cudaMemsetAsync(s.du16, 0, sizeof(bf16) * Mr * dm.L, c->stream));
    CU_OK(c, cudaMemsetAsync(c->grads, 0, sizeof(float) * c->lay.total, c->stream));
    CU_OK(c, cudaMemsetAsync(c->m, 0, sizeof(float) * c->lay.total, c->stream));
    CU_OK(c, cudaMemsetAsync(c->v, 0, sizeof(float) * c->lay.total, c->stream));
    std::vector<float> init;
    fill_initial_params(c, seed, init);
    CU_OK(c, cudaMemcpyAsync(c->params, init.data(), sizeof(float) * c->lay.total, cudaMemcpyHostToDevice, c->stream));
    CU_OK(c, cudaStreamSynchronize(c->stream));
    c->step = 0;
    if ((st = refresh_shadow(c)) != PAC_OK) return st;
    if (cls && !c->hc.on) {
        if (c->dtype == PAC_F32)
            pool_last_layer_kernel<float><<<(unsigned)dm.N, 256, 0, c->stream>>>((const float*)c->cache, s.hbar, dm.L, dm.S, dm.d);
        else
            pool_last_layer_kernel<bf16><<<(unsigned)dm.N, 256, 0, c->stream>>>((const bf16*)c->cache, s.hbar, dm.L, dm.S, dm.d);
        LAUNCH_CHECK(c);
    }
    CU_OK(c, cudaStreamSynchronize(c->stream));
    c->inited = true;
    return PAC_OK;
}

// ---- out-of-core cache: bring a minibatch's slabs into a staging slot and point the context at it ----
namespace {

// Validates host ids against the host cache, copies their slabs and labels into the next slot on
// the copy stream, makes the compute stream wait for them and binds the slot: afterwards the
// kernels run on ids 0 .. B-1 of a cache of max_batch samples.  *ids_out receives those ids.
pac_status host_cache_stage(pac_ctx* c, const int* ids, int B, const char* who, const int** ids_out) {
    HostCache& h = c->hc;
    if (!ids) return fail(c, PAC_ERR_INVALID_ARG, "%s: sample_ids is NULL", who);
    if (B < 1 || B > c->cfg.max_batch)
        return fail(c, PAC_ERR_INVALID_ARG, "%s: B=%d outside [1, max_batch=%d]", who, B, c->cfg.max_batch);
    for (int b = 0; b < B; ++b)
        if (ids[b] < 0 || ids[b] >= h.N)
            return fail(c, PAC_ERR_SAMPLE_ID_RANGE, "%s: sample_ids[%d]=%d outside [0, %lld)", who, b, ids[b], h.N);
    const int k = h.cur;
    h.cur ^= 1;
    const int lps = c->labels_per_sample;
    // the slot's previous contents: its copies must have run before the label staging is rewritten,
    // its step must have finished before the slabs are overwritten
    CU_OK(c, cudaEventSynchronize(h.ready[k]));
    CU_OK(c, cudaStreamWaitEvent(h.copy_stream, h.freed[k], 0));
    for (int b = 0; b < B; ++b) {
        CU_OK(c, cudaMemcpyAsync(h.stage[k] + (size_t)b * h.sample_bytes, h.host + (size_t)ids[b] * h.sample_bytes,
                                 (size_t)h.sample_bytes, cudaMemcpyHostToDevice, h.copy_stream));
        std::memcpy(h.h_lab[k] + (size_t)b * lps, h.host_labels + (size_t)ids[b] * lps, sizeof(int) * lps);
    }
    CU_OK(c, cudaMemcpyAsync(h.lab_stage[k], h.h_lab[k], sizeof(int) * (size_t)B * lps, cudaMemcpyHostToDevice, h.copy_stream));
    CU_OK(c, cudaEventRecord(h.ready[k], h.copy_stream));
    CU_OK(c, cudaStreamWaitEvent(c->stream, h.ready[k], 0));
    // bind
    c->cache = h.stage[k];
    c->labels = h.lab_stage[k];
    c->sc.hbar = h.hbar_stage[k];
    if (c->tensor_ok) c->tplan = h.tplan[k];
    if (c->cfg.head == PAC_HEAD_MEANPOOL_CLS) {
        // token mean of the last cached layer of the staged samples (computed once at set-up for a resident cache)
        if (c->dtype == PAC_F32)
            pool_last_layer_kernel<float><<<(unsigned)B, 256, 0, c->stream>>>((const float*)c->cache, c->sc.hbar, c->dm.L, c->dm.S, c->dm.d);
        else
            pool_last_layer_kernel<bf16><<<(unsigned)B, 256, 0, c->stream>>>((const bf16*)c->cache, c->sc.hbar, c->dm.L, c->dm.S, c->dm.d);
        LAUNCH_CHECK(c);
    }
    *ids_out = h.iota;
    return PAC_OK;
}

// After the step that uses the bound slot has been enqueued.
pac_status host_cache_release(pac_ctx* c) {
    HostCache& h = c->hc;
    const int k = h.cur ^ 1;               // the slot host_cache_stage bound last
    CU_OK(c, cudaEventRecord(h.freed[k], c->stream));
    return PAC_OK;
}

// Ids of a step, wherever the cache lives: device ids the kernels index the (staged) cache with.
pac_status prepare_ids(pac_ctx* c, const int* sample_ids, int B, const char* who, const int** d_ids) {
    if (c->hc.on) return host_cache_stage(c, sample_ids, B, who, d_ids);
    *d_ids = c->sc.ids;
    return stage_ids(c, sample_ids, B, who);
}
pac_status finish_ids(pac_ctx* c) { return c->hc.on ? host_cache_release(c) : PAC_OK; }

}  // namespace

pac_status pac_train_step(pac_ctx* c, const int* sample_ids, int B, float* loss_out) {
    NEED_INIT(c, "pac_train_step");
    const int* d_ids = nullptr;
    pac_status st = prepare_ids(c, sample_ids, B, "pac_train_step", &d_ids);
    if (st != PAC_OK) return st;
    if ((st = train_enqueue(c, d_ids, B, c->sc.loss, nullptr)) != PAC_OK) return st;
    if ((st = finish_ids(c)) != PAC_OK) return st;
    if (loss_out) {
        CU_OK(c, cudaMemcpyAsync(c->h_loss, c->sc.loss, sizeof(float), cudaMemcpyDeviceToHost, c->stream));
        CU_OK(c, cudaStreamSynchronize(c->stream));
        *loss_out = *c->h_loss;
    }
    return PAC_OK;
}

pac_status pac_train_step_dev_loss(pac_ctx* c, const int* sample_ids, int B, float* dev_loss) {
    NEED_INIT(c, "pac_train_step_dev_loss");
    const int* d_ids = nullptr;
    pac_status st = prepare_ids(c, sample_ids, B, "pac_train_step_dev_loss", &d_ids);
    if (st != PAC_OK) return st;
    if ((st = train_enqueue(c, d_ids, B, dev_loss ? dev_loss : c->sc.loss, nullptr)) != PAC_OK) return st;
    return finish_ids(c);
}

pac_status pac_set_grad_scale(pac_ctx* c, float scale) {
    NEED_CTX(c);
    if (!(scale > 0.f) || !(scale <= 1.f)) return fail(c, PAC_ERR_INVALID_ARG, "pac_set_grad_scale: scale must lie in (0, 1]");
    c->grad_scale = scale;
    return PAC_OK;
}

pac_status pac_train_step_async(pac_ctx* c, const int* sample_ids, int B, const pac_adamw* hp, float* loss_out) {
    NEED_INIT(c, "pac_train_step_async");
    pac_status st = check_hp(c, hp);
    if (st != PAC_OK) return st;
    // where the device can write the loss itself (page-locked host memory): no copy node behind the step
    float* d_loss = c->sc.loss;
    bool copy_loss = loss_out != nullptr;
    if (loss_out) {
        cudaPointerAttributes pa;
        if (cudaPointerGetAttributes(&pa, loss_out) == cudaSuccess && pa.type == cudaMemoryTypeHost && pa.devicePointer) {
            d_loss = (float*)pa.devicePointer;
            copy_loss = false;
        } else {
            cudaGetLastError();
        }
    }
    const int* d_ids = nullptr;
    if (!c->hc.on && c->zc_ids && c->timing == 0 && use_fused_fwd(c, B)) {
        // one-launch forward: it reads the ids straight from a page-locked ring slot, so the step is three
        // kernels back to back with nothing between them and the steps overlap as in pac_train_epoch_dev
        if (!sample_ids) return fail(c, PAC_ERR_INVALID_ARG, "pac_train_step_async: sample_ids is NULL");
        if (B < 1 || B > c->cfg.max_batch)
            return fail(c, PAC_ERR_INVALID_ARG, "pac_train_step_async: B=%d outside [1, max_batch=%d]", B, c->cfg.max_batch);
        for (int b = 0; b < B; ++b)
            if (sample_ids[b] < 0 || sample_ids[b] >= c->dm.N)
                return fail(c, PAC_ERR_SAMPLE_ID_RANGE, "pac_train_step_async: sample_ids[%d]=%d outside [0, %lld)", b, sample_ids[b], c->dm.N);
        const int slot = (int)(c->zc_count % ZC_SLOTS), half = slot / (ZC_SLOTS / 2);
        if (slot % (ZC_SLOTS / 2) == 0) CU_OK(c, cudaEventSynchronize(c->zc_ev[half]));     // the half's previous steps have run
        int* h = c->zc_ids + (size_t)slot * c->cfg.max_batch;
        std::memcpy(h, sample_ids, sizeof(int) * B);
        // publish: ids first, then the step's sequence number (the kernel of the step before may be looking)
        __atomic_store_n(&c->zc_tags[slot], (unsigned)(c->zc_count + 1), __ATOMIC_RELEASE);
        c->step_host_ids = true;
        st = train_enqueue(c, h, B, d_loss, hp);
        c->step_host_ids = false;
        if (st != PAC_OK) return st;
        c->zc_count++;
        if (slot % (ZC_SLOTS / 2) == ZC_SLOTS / 2 - 1) CU_OK(c, cudaEventRecord(c->zc_ev[half], c->stream));
    } else {
        if ((st = prepare_ids(c, sample_ids, B, "pac_train_step_async", &d_ids)) != PAC_OK) return st;
        if ((st = train_enqueue(c, d_ids, B, d_loss, hp)) != PAC_OK) return st;
        if ((st = finish_ids(c)) != PAC_OK) return st;
    }
    if (copy_loss) CU_OK(c, cudaMemcpyAsync(loss_out, d_loss, sizeof(float), cudaMemcpyDeviceToHost, c->stream));
    return PAC_OK;
}

pac_status pac_adam_step(pac_ctx* c, const pac_adamw* hp) {
    NEED_INIT(c, "pac_adam_step");
    pac_status st = check_hp(c, hp);
    if (st != PAC_OK) return st;
    return adam_enqueue(c, hp);
}

pac_status pac_eval_logits(pac_ctx* c, const int* sample_ids, int B, float* dev_out) {
    NEED_INIT(c, "pac_eval_logits");
    if (!dev_out) return fail(c, PAC_ERR_INVALID_ARG, "pac_eval_logits: dev_out is NULL");
    const int* d_ids = nullptr;
    pac_status st = prepare_ids(c, sample_ids, B, "pac_eval_logits", &d_ids);
    if (st != PAC_OK) return st;
    st = c->tb.on ? tb_forward(c, d_ids, B, false, dev_out)
       : use_fused_cls(c) ? cls_forward_enqueue(c, d_ids, B, false, dev_out) : forward(c, d_ids, B, false, dev_out);
    if (st != PAC_OK) return st;
    return finish_ids(c);
}

pac_status pac_gather(pac_ctx* c, const int* sample_ids, int B, void* dev_out) {
    NEED_INIT(c, "pac_gather");
    if (!dev_out) return fail(c, PAC_ERR_INVALID_ARG, "pac_gather: dev_out is NULL");
    const int* d_ids = nullptr;
    pac_status st = prepare_ids(c, sample_ids, B, "pac_gather", &d_ids);
    if (st != PAC_OK) return st;
    const Dims& dm = c->dm;
    const long long slab = (long long)dm.S * dm.d * (c->dtype == PAC_F32 ? 4 : 2);
    const int vec16 = (slab % 16 == 0) && (((uintptr_t)dev_out & 15) == 0);
    unsigned chunks = (unsigned)std::min<long long>(64, std::max<long long>(1, slab / (16 * 256 * 4)));
    dim3 grid((unsigned)(B * dm.L), chunks, 1);
    gather_kernel<<<grid, 256, 0, c->stream>>>((const unsigned char*)c->cache, d_ids, dm.N, dm.L, B, slab,
                                               (unsigned char*)dev_out, vec16, c->status);
    LAUNCH_CHECK(c);
    return finish_ids(c);
}

static pac_status epoch_common(pac_ctx* c, const int* d_perm, long long n, int B, const pac_adamw* hp, float* d_losses) {
    for (long long s = 0; s < n / B; ++s) {
        const int* ids = d_perm + s * B;
        // from the second step on the kernel ahead is this library's own, which does not write ids
        c->step_early_ids = s > 0;
        pac_status st = train_enqueue(c, ids, B, d_losses ? d_losses + s : c->sc.loss, hp);
        c->step_early_ids = false;
        if (st != PAC_OK) return st;
    }
    return PAC_OK;
}

pac_status pac_train_epoch(pac_ctx* c, const int* perm, long long n, int B, const pac_adamw* hp, float* losses_out) {
    NEED_INIT(c, "pac_train_epoch");
    pac_status st = check_hp(c, hp);
    if (st != PAC_OK) return st;
    if (!perm) return fail(c, PAC_ERR_INVALID_ARG, "pac_train_epoch: perm is NULL");
    if (B < 1 || B > c->cfg.max_batch) return fail(c, PAC_ERR_INVALID_ARG, "pac_train_epoch: B=%d outside [1, max_batch]", B);
    if (n < B || n % B != 0) return fail(c, PAC_ERR_INVALID_ARG, "pac_train_epoch: n=%lld is not a positive multiple of B=%d", n, B);
    const long long n_cache = c->hc.on ? c->hc.N : c->dm.N;
    for (long long i = 0; i < n; ++i)
        if (perm[i] < 0 || perm[i] >= n_cache)
            return fail(c, PAC_ERR_SAMPLE_ID_RANGE, "pac_train_epoch: perm[%lld]=%d outside [0, %lld)", i, perm[i], n_cache);
    if (c->hc.on && n / B > c->losses_cap) {
        CU_OK(c, cudaStreamSynchronize(c->stream));
        if (c->d_losses) cudaFree(c->d_losses);
        c->d_losses = nullptr; c->losses_cap = 0;
        if ((st = dmalloc(c, &c->d_losses, n / B)) != PAC_OK) return st;
        c->losses_cap = n / B;
    }
    if (c->hc.on) {
        // host-resident cache: the slabs of step s+1 travel to their staging slot while step s computes
        for (long long s = 0; s < n / B; ++s) {
            const int* d_ids = nullptr;
            if ((st = host_cache_stage(c, perm + s * B, B, "pac_train_epoch", &d_ids)) != PAC_OK) return st;
            if ((st = train_enqueue(c, d_ids, B, c->d_losses + s, hp)) != PAC_OK) return st;
            if ((st = host_cache_release(c)) != PAC_OK) return st;
        }
        if (losses_out)
            CU_OK(c, cudaMemcpyAsync(losses_out, c->d_losses, sizeof(float) * (n / B), cudaMemcpyDeviceToHost, c->stream));
        CU_OK(c, cudaStreamSynchronize(c->stream));
        return PAC_OK;
    }
    if (n > c->perm_cap) {
        CU_OK(c, cudaStreamSynchronize(c->stream));
        if (c->d_perm) cudaFree(c->d_perm);
        c->d_perm = nullptr; c->perm_cap = 0;
        if ((st = dmalloc(c, &c->d_perm, n)) != PAC_OK) return st;
        c->perm_cap = n;
    }
    if (n / B > c->losses_cap) {
        CU_OK(c, cudaStreamSynchronize(c->stream));
        if (c->d_losses) cudaFree(c->d_losses);
        c->d_losses = nullptr; c->losses_cap = 0;
        if ((st = dmalloc(c, &c->d_losses, n / B)) != PAC_OK) return st;
        c->losses_cap = n / B;
    }
    // perm is pageable host memory: cudaMemcpyAsync stages it before returning
    CU_OK(c, cudaMemcpyAsync(c->d_perm, perm, sizeof(int) * n, cudaMemcpyHostToDevice, c->stream));
    if ((st = epoch_common(c, c->d_perm, n, B, hp, c->d_losses)) != PAC_OK) return st;
    if (losses_out)
        CU_OK(c, cudaMemcpyAsync(losses_out, c->d_losses, sizeof(float) * (n / B), cudaMemcpyDeviceToHost, c->stream));
    CU_OK(c, cudaStreamSynchronize(c->stream));
    return PAC_OK;
}

pac_status pac_train_epoch_dev(pac_ctx* c, const int* dev_perm, long long n, int B, const pac_adamw* hp, float* dev_losses) {
    NEED_INIT(c, "pac_train_epoch_dev");
    pac_status st = check_hp(c, hp);
    if (st != PAC_OK) return st;
    if (c->hc.on)
        return fail(c, PAC_ERR_UNSUPPORTED, "pac_train_epoch_dev: a host-resident cache needs the ids on the host (use pac_train_epoch)");
    if (!dev_perm) return fail(c, PAC_ERR_INVALID_ARG, "pac_train_epoch_dev: dev_perm is NULL");
    if (B < 1 || B > c->cfg.max_batch) return fail(c, PAC_ERR_INVALID_ARG, "pac_train_epoch_dev: B=%d outside [1, max_batch]", B);
    if (n < B || n % B != 0) return fail(c, PAC_ERR_INVALID_ARG, "pac_train_epoch_dev: n=%lld is not a positive multiple of B=%d", n, B);
    return epoch_common(c, dev_perm, n, B, hp, dev_losses);
}

pac_status pac_param_count(pac_ctx* c, long long* n) {
    NEED_INIT(c, "pac_param_count");
    if (!n) return fail(c, PAC_ERR_INVALID_ARG, "pac_param_count: n is NULL");
    *n = c->lay.total;
    return PAC_OK;
}

pac_status pac_get_params(pac_ctx* c, float* host) {
    NEED_INIT(c, "pac_get_params");
    if (!host) return fail(c, PAC_ERR_INVALID_ARG, "pac_get_params: host is NULL");
    CU_OK(c, cudaMemcpyAsync(host, c->params, sizeof(float) * c->lay.total, cudaMemcpyDeviceToHost, c->stream));
    CU_OK(c, cudaStreamSynchronize(c->stream));
    return PAC_OK;
}

pac_status pac_set_params(pac_ctx* c, const float* host) {
    NEED_INIT(c, "pac_set_params");
    if (!host) return fail(c, PAC_ERR_INVALID_ARG, "pac_set_params: host is NULL");
    CU_OK(c, cudaMemcpyAsync(c->params, host, sizeof(float) * c->lay.total, cudaMemcpyHostToDevice, c->stream));
    pac_status st = refresh_shadow(c);
    if (st != PAC_OK) return st;
    CU_OK(c, cudaStreamSynchronize(c->stream));
    return PAC_OK;
}

pac_status pac_get_grads(pac_ctx* c, float* host) {
    NEED_INIT(c, "pac_get_grads");
    if (!host) return fail(c, PAC_ERR_INVALID_ARG, "pac_get_grads: host is NULL");
    CU_OK(c, cudaMemcpyAsync(host, c->grads, sizeof(float) * c->lay.total, cudaMemcpyDeviceToHost, c->stream));
    CU_OK(c, cudaStreamSynchronize(c->stream));
    return PAC_OK;
}

pac_status pac_get_opt_state(pac_ctx* c, float* m, float* v, long long* step) {
    NEED_INIT(c, "pac_get_opt_state");
    if (!m || !v || !step) return fail(c, PAC_ERR_INVALID_ARG, "pac_get_opt_state: NULL argument");
    CU_OK(c, cudaMemcpyAsync(m, c->m, sizeof(float) * c->lay.total, cudaMemcpyDeviceToHost, c->stream));
    CU_OK(c, cudaMemcpyAsync(v, c->v, sizeof(float) * c->lay.total, cudaMemcpyDeviceToHost, c->stream));
    CU_OK(c, cudaStreamSynchronize(c->stream));
    *step = c->step;
    return PAC_OK;
}

pac_status pac_set_opt_state(pac_ctx* c, const float* m, const float* v, long long step) {
    NEED_INIT(c, "pac_set_opt_state");
    if (!m || !v || step < 0) return fail(c, PAC_ERR_INVALID_ARG, "pac_set_opt_state: bad argument");
    CU_OK(c, cudaMemcpyAsync(c->m, m, sizeof(float) * c->lay.total, cudaMemcpyHostToDevice, c->stream));
    CU_OK(c, cudaMemcpyAsync(c->v, v, sizeof(float) * c->lay.total, cudaMemcpyHostToDevice, c->stream));
    CU_OK(c, cudaStreamSynchronize(c->stream));
    c->step = step;
    return PAC_OK;
}

pac_status pac_device_buffers(pac_ctx* c, float** dev_params, float** dev_grads) {
    NEED_INIT(c, "pac_device_buffers");
    if (!dev_params || !dev_grads) return fail(c, PAC_ERR_INVALID_ARG, "pac_device_buffers: NULL argument");
    *dev_params = c->params;
    *dev_grads = c->grads;
    return PAC_OK;
}

pac_status pac_params_changed(pac_ctx* c) {
    NEED_INIT(c, "pac_params_changed");
    return refresh_shadow(c);
}

pac_status pac_set_option(pac_ctx* c, int option, int value) {
    NEED_CTX(c);
    if (option == PAC_OPT_KERNEL_PATH) {
        if (value < 0 || value > 5) return fail(c, PAC_ERR_INVALID_ARG, "pac_set_option: kernel path must be 0 ... 5");
        if (c->inited) return fail(c, PAC_ERR_BAD_STATE, "pac_set_option: set the kernel path before pac_adapter_init");
        c->force_simt = value == 1;
        c->forward_mode = value >= 2 ? value : 0;
        return PAC_OK;
    }
    if (option == PAC_OPT_KERNEL_TIMING) {
        if (value < 0 || value > 2) return fail(c, PAC_ERR_INVALID_ARG, "pac_set_option: timing must be 0, 1 or 2");
        if (value == 2) {
            CU_OK(c, cudaSetDevice(c->device));
            pac_status st = reset_stamps(c);
            if (st != PAC_OK) return st;
        }
        c->timing = value;
        return PAC_OK;
    }
    return fail(c, PAC_ERR_INVALID_ARG, "pac_set_option: unknown option %d", option);
}

pac_status pac_stream_phase_times(pac_ctx* c, double* out_ms, long long* out_count) {
    NEED_CTX(c);
    if (!out_ms || !out_count) return fail(c, PAC_ERR_INVALID_ARG, "pac_stream_phase_times: NULL argument");
    out_ms[0] = out_ms[1] = 0.0;
    out_count[0] = out_count[1] = 0;
    if (!c->d_stamps) return PAC_OK;
    CU_OK(c, cudaSetDevice(c->device));
    CU_OK(c, cudaStreamSynchronize(c->stream));
    std::vector<unsigned long long> h(2 * STAMP_SLOTS * 2);
    CU_OK(c, cudaMemcpy(h.data(), c->d_stamps, sizeof(unsigned long long) * h.size(), cudaMemcpyDeviceToHost));
    for (int w = 0; w < 2; ++w)
        for (size_t i = 0; i < c->stamps_used[w]; ++i) {
            const unsigned long long t0 = h[((size_t)w * STAMP_SLOTS + i) * 2], t1 = h[((size_t)w * STAMP_SLOTS + i) * 2 + 1];
            if (t1 > t0) { out_ms[w] += (double)(t1 - t0) * 1e-6; out_count[w]++; }
        }
    return reset_stamps(c);
}

pac_status pac_kernel_times(pac_ctx* c, double* out_ms, long long* out_count) {
    NEED_CTX(c);
    if (!out_ms || !out_count) return fail(c, PAC_ERR_INVALID_ARG, "pac_kernel_times: NULL argument");
    CU_OK(c, cudaSetDevice(c->device));
    CU_OK(c, cudaStreamSynchronize(c->stream));
    for (int w = 0; w < 4; ++w) {
        double tot = 0.0;
        long long cnt = 0;
        for (size_t i = 0; i + 1 < c->tev_used[w]; i += 2) {
            float ms = 0.f;
            if (cudaEventElapsedTime(&ms, c->tev[w][i], c->tev[w][i + 1]) == cudaSuccess) { tot += ms; cnt++; }
        }
        out_ms[w] = tot;
        out_count[w] = cnt;
        c->tev_used[w] = 0;
    }
    return PAC_OK;
}

pac_status pac_launch_count(pac_ctx* c, long long* n) {
    NEED_CTX(c);
    if (!n) return fail(c, PAC_ERR_INVALID_ARG, "pac_launch_count: n is NULL");
    *n = c->launches;
    return PAC_OK;
}

pac_status pac_sync(pac_ctx* c) {
    NEED_CTX(c);
    CU_OK(c, cudaSetDevice(c->device));
    CU_OK(c, cudaMemcpyAsync(c->h_status, c->status, sizeof(unsigned) * ST_WORDS, cudaMemcpyDeviceToHost, c->stream));
    CU_OK(c, cudaMemsetAsync(c->status, 0, sizeof(unsigned) * ST_WORDS, c->stream));
    CU_OK(c, cudaStreamSynchronize(c->stream));
    // optimizer updates that found the timeout flag set were left out: they do not count as steps
    const long long skipped = (long long)c->h_status[ST_SKIPPED_STEPS];
    c->step = c->step > skipped ? c->step - skipped : 0;
    if (c->h_status[ST_TIMEOUT])
        return fail(c, PAC_ERR_TIMEOUT, "a bounded device-side wait ran out (%u); %lld later optimizer updates were skipped",
                    c->h_status[ST_TIMEOUT], skipped);
    if (c->h_status[ST_CLAMPED_IDS])
        return fail(c, PAC_ERR_SAMPLE_ID_RANGE, "%u device-resident sample ids were outside [0, N) and were clamped", c->h_status[ST_CLAMPED_IDS]);
    return PAC_OK;
}

pac_status pac_selftest_wait_expiry(pac_ctx* c, unsigned long long limit_ns) {
    NEED_CTX(c);
    if (limit_ns < 1000ull || limit_ns > 100000000ull)
        return fail(c, PAC_ERR_INVALID_ARG, "pac_selftest_wait_expiry: limit_ns must lie in [1e3, 1e8]");
    CU_OK(c, cudaSetDevice(c->device));
    unsigned* d_res = nullptr;
    CU_OK(c, cudaMalloc((void**)&d_res, 2 * sizeof(unsigned)));
    unsigned h_res[2] = {0u, 0u};
    cudaError_t e = cudaMemsetAsync(d_res, 0, 2 * sizeof(unsigned), c->stream);
    if (e == cudaSuccess) {
        selftest_wait_expiry_kernel<<<1, 64, 0, c->stream>>>(c->status, limit_ns, d_res);
        c->launches++;
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaMemcpyAsync(h_res, d_res, sizeof h_res, cudaMemcpyDeviceToHost, c->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    cudaFree(d_res);
    if (e != cudaSuccess) return fail(c, PAC_ERR_CUDA, "pac_selftest_wait_expiry: %s", cudaGetErrorString(e));
    if (h_res[0] != 1u || h_res[1] != 1u)
        return fail(c, PAC_ERR_BAD_STATE, "pac_selftest_wait_expiry: the wait did not report expiry (expired=%u abort=%u)", h_res[0], h_res[1]);
    return PAC_OK;
}

const char* pac_last_error(const pac_ctx* c) { return c ? c->err.c_str() : "null context"; }

const char* pac_kernel_path(const pac_ctx* c) {
    if (!c || !c->inited || !use_tensor(c)) return "simt";
    if (use_chain_fwd(c, c->cfg.max_batch)) return "tensor+chain_forward";
    return use_fused_fwd(c, c->cfg.max_batch) ? "tensor+fused_forward" : "tensor";
}

}  // extern "C"

// ---------------------------------------------------------------------------
// pac_eval_logits_static: the classifier-head evaluation forward with its scratch in a
// fixed device array instead of context-owned allocations.
// ---------------------------------------------------------------------------
namespace {

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress; the
// device address is looked up once per device below and that pointer is what kernels receive.
static __device__ __align__(256) unsigned char g_static_scratch[PAC_STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
std::mutex g_static_mu;
unsigned char* g_static_ptr[MAX_DEVICES] = {};

// Token mean of the last cached layer for the batch's samples, plus the identity index the
// head kernel uses to address it: hbar_b[b][k] = mean_s cache[ids[b]][L-1][s][k], iota[b] = b.
template <typename T>
__global__ void pool_last_layer_batch_kernel(const T* __restrict__ cache, const int* __restrict__ ids, long long N, int L,
                                             int S, int d, float* __restrict__ hbar_b, int* __restrict__ iota) {
    const int b = blockIdx.x;
    const long long id = safe_id(ids, b, N, nullptr);
    const T* base = cache + ((id * L) + (L - 1)) * (long long)S * d;
    for (int k = threadIdx.x; k < d; k += blockDim.x) {
        float acc = 0.f;
        for (int s = 0; s < S; ++s) acc += to_f32(base[(long long)s * d + k]);
        hbar_b[(long long)b * d + k] = acc / (float)S;
    }
    if (threadIdx.x == 0) iota[b] = b;
}

pac_status static_fail(char* err, int err_len, pac_status st, const char* fmt, ...) {
    if (err && err_len > 0) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(err, (size_t)err_len, fmt, ap);
        va_end(ap);
    }
    return st;
}

inline size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

template <typename T>
cudaError_t static_forward(cudaStream_t st, const T* cache, long long N, int L, int S, int d, const float* params,
                           const ParamLayout& lay, int r, int act, int C, const int* ids, int B, float* out,
                           float* u, float* a, float* pooled_a, float* hbar_b, int* iota) {
    const int M = B * S;
    const long long n = (long long)M * r;
    CacheRows<T> A{cache, ids, N, L, S, d, 0};
    MatB_RowMajor Bm{{params + lay.w_down, (long long)d * r, r}};
    StoreRowMajor E{u, n, r};
    dim3 grid(cdiv(r, SG_BN), cdiv(M, SG_BM), (unsigned)L);
    cudaError_t e;
    // a launch that is rejected ends the call: later kernels would read scratch the earlier one never wrote
    gemm_simt<<<grid, 256, 0, st>>>(M, r, d, A, Bm, E);                                  // u_l = h_l W_down^l
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (act == PAC_ACT_RELU) chain_fwd_kernel<PAC_ACT_RELU><<<cdiv(n, 256), 256, 0, st>>>(u, a, params + lay.lam, L, n, n);
    else chain_fwd_kernel<PAC_ACT_IDENTITY><<<cdiv(n, 256), 256, 0, st>>>(u, a, params + lay.lam, L, n, n);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    pool_tokens_kernel<<<B, 128, 0, st>>>(a + (long long)(L - 1) * n, pooled_a, S, r);     // mean_s a_L
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    pool_last_layer_batch_kernel<T><<<B, 256, 0, st>>>(cache, ids, N, L, S, d, hbar_b, iota);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    cls_head_kernel<<<B, 256, sizeof(float) * (d + C + 32), st>>>(hbar_b, iota, B, nullptr, pooled_a, params + lay.w_up,
                                                                 params + lay.w_head, params + lay.b_head, B, S, d, r, C, 0,
                                                                 nullptr, out, nullptr, nullptr, nullptr, nullptr, nullptr);
    return cudaGetLastError();
}

}  // namespace

extern "C" pac_status pac_eval_logits_static(int device, void* cuda_stream, const void* dev_cache, int dtype, long long N,
                                             int L, int S, int d, const float* dev_params, int r, int act, int n_out,
                                             const int* dev_sample_ids, int B, float* dev_out, char* err, int err_len) {
    if (!dev_cache || !dev_params || !dev_sample_ids || !dev_out)
        return static_fail(err, err_len, PAC_ERR_INVALID_ARG, "pac_eval_logits_static: NULL device pointer");
    if (dtype != PAC_F32 && dtype != PAC_BF16) return static_fail(err, err_len, PAC_ERR_INVALID_ARG, "pac_eval_logits_static: bad dtype %d", dtype);
    if (act != PAC_ACT_RELU && act != PAC_ACT_IDENTITY) return static_fail(err, err_len, PAC_ERR_INVALID_ARG, "pac_eval_logits_static: bad activation %d", act);
    if (N < 1 || L < 1 || S < 1 || d < 1 || r < 1 || n_out < 1 || B < 1)
        return static_fail(err, err_len, PAC_ERR_INVALID_ARG, "pac_eval_logits_static: sizes must be positive");
    if (device < 0 || device >= MAX_DEVICES) return static_fail(err, err_len, PAC_ERR_INVALID_ARG, "pac_eval_logits_static: bad device %d", device);
    if (((size_t)d + (size_t)n_out + 32) * sizeof(float) > 48 * 1024)
        return static_fail(err, err_len, PAC_ERR_UNSUPPORTED, "pac_eval_logits_static: d + C is beyond the head kernel's shared memory");
    // every factor is bounded by the scratch size before any product is formed, so none can wrap:
    // afterwards B*S*r*L*4 <= 8 MiB, B*S fits an int and the grid dimensions (L, B*S/64) are legal
    {
        const size_t cap = (size_t)PAC_STATIC_SCRATCH_BYTES / sizeof(float);
        size_t prod = 1;
        const long long factors[4] = {B, S, r, L};
        for (long long f : factors) {
            if ((size_t)f > cap / prod)
                return static_fail(err, err_len, PAC_ERR_UNSUPPORTED,
                                   "pac_eval_logits_static: L=%d B=%d S=%d r=%d needs more scratch than the fixed array holds (%u bytes)",
                                   L, B, S, r, (unsigned)PAC_STATIC_SCRATCH_BYTES);
            prod *= (size_t)f;
        }
        if (L > 65535 || (size_t)B * (size_t)d > cap)
            return static_fail(err, err_len, PAC_ERR_UNSUPPORTED, "pac_eval_logits_static: L or B*d too large");
    }
    // scratch layout: u | a | pooled_a | hbar_b | iota, each block rounded up to 256 bytes
    const size_t Mr = (size_t)B * S * r;
    const size_t o_u = 0, o_a = o_u + up256(sizeof(float) * Mr * L), o_p = o_a + up256(sizeof(float) * Mr * L);
    const size_t o_h = o_p + up256(sizeof(float) * (size_t)B * r), o_i = o_h + up256(sizeof(float) * (size_t)B * d);
    const size_t need = o_i + up256(sizeof(int) * (size_t)B);
    if (need > (size_t)PAC_STATIC_SCRATCH_BYTES)
        return static_fail(err, err_len, PAC_ERR_UNSUPPORTED,
                           "pac_eval_logits_static: L=%d B=%d S=%d r=%d d=%d needs %zu bytes of scratch, the fixed array holds %u",
                           L, B, S, r, d, need, (unsigned)PAC_STATIC_SCRATCH_BYTES);
    // the caller's current device is put back before returning
    struct DeviceGuard {
        int prev = -1;
        ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
    } guard;
    int cur = -1;
    if (cudaGetDevice(&cur) == cudaSuccess && cur != device) guard.prev = cur;
    cudaError_t e = cudaSetDevice(device);
    if (e != cudaSuccess) return static_fail(err, err_len, PAC_ERR_CUDA, "pac_eval_logits_static: cudaSetDevice: %s", cudaGetErrorString(e));
    unsigned char* base;
    {
        std::lock_guard<std::mutex> lock(g_static_mu);
        if (!g_static_ptr[device]) {
            // once per device, with that device current: the device address of the array
            void* p = nullptr;
            e = cudaGetSymbolAddress(&p, g_static_scratch);
            if (e != cudaSuccess || !p)
                return static_fail(err, err_len, PAC_ERR_CUDA, "pac_eval_logits_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
            g_static_ptr[device] = (unsigned char*)p;
        }
        base = g_static_ptr[device];
    }
    float *u = (float*)(base + o_u), *a = (float*)(base + o_a), *pooled_a = (float*)(base + o_p), *hbar_b = (float*)(base + o_h);
    int* iota = (int*)(base + o_i);
    const ParamLayout lay = ParamLayout::make(L, d, r, n_out, true);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    e = dtype == PAC_F32
            ? static_forward<float>(st, (const float*)dev_cache, N, L, S, d, dev_params, lay, r, act, n_out, dev_sample_ids, B, dev_out, u, a, pooled_a, hbar_b, iota)
            : static_forward<bf16>(st, (const bf16*)dev_cache, N, L, S, d, dev_params, lay, r, act, n_out, dev_sample_ids, B, dev_out, u, a, pooled_a, hbar_b, iota);
    if (e != cudaSuccess) return static_fail(err, err_len, PAC_ERR_CUDA, "pac_eval_logits_static: kernel launch failed: %s", cudaGetErrorString(e));
    return PAC_OK;
}

// ---------------------------------------------------------------------------
// Block-wise absmax INT8 codec (Section IV-D, Eq. 1-2)
// ---------------------------------------------------------------------------
extern "C" pac_status pac_quantize_absmax(int device, void* cuda_stream, const float* dev_x, long long n, int block,
                                          signed char* dev_q, float* dev_c) {
    if (!dev_x || !dev_q || !dev_c || n < 1 || block < 1) return PAC_ERR_INVALID_ARG;
    if (cudaSetDevice(device) != cudaSuccess) return PAC_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const long long n_blocks = (n + block - 1) / block;
    const bool vec = (n % 4 == 0) && (((uintptr_t)dev_x & 15) == 0) && (((uintptr_t)dev_q & 3) == 0);
    if (vec && (block == 16 || block == 32 || block == 64 || block == 128)) {
        const long long n4 = n / 4, want = (n4 + 255) / 256;
        const unsigned grid = (unsigned)(want < 148LL * 32 ? want : 148LL * 32);
        quantize_absmax_subwarp_kernel<<<grid, 256, 0, st>>>((const float4*)dev_x, n4, block / 4, (char4*)dev_q, dev_c);
    } else if (vec && block % 1024 == 0 && block <= 4096 && n_blocks <= 0x7fffffffLL) {
        const long long n4 = n / 4;
        switch (block / 1024) {
            case 1: quantize_absmax_cta_reg_kernel<1><<<(unsigned)n_blocks, 256, 0, st>>>((const float4*)dev_x, n4, (char4*)dev_q, dev_c); break;
            case 2: quantize_absmax_cta_reg_kernel<2><<<(unsigned)n_blocks, 256, 0, st>>>((const float4*)dev_x, n4, (char4*)dev_q, dev_c); break;
            case 3: quantize_absmax_cta_reg_kernel<3><<<(unsigned)n_blocks, 256, 0, st>>>((const float4*)dev_x, n4, (char4*)dev_q, dev_c); break;
            default: quantize_absmax_cta_reg_kernel<4><<<(unsigned)n_blocks, 256, 0, st>>>((const float4*)dev_x, n4, (char4*)dev_q, dev_c); break;
        }
    } else if (block <= QUANT_WARP_MAX) {
        const long long warps = n_blocks < 148LL * 64 ? n_blocks : 148LL * 64;      // up to 8 CTAs of 8 warps per SM
        quantize_absmax_warp_kernel<<<(unsigned)((warps + 7) / 8), 256, 0, st>>>(dev_x, n, block, n_blocks, dev_q, dev_c);
    } else {
        if (n_blocks > 0x7fffffffLL) return PAC_ERR_UNSUPPORTED;
        quantize_absmax_cta_kernel<<<(unsigned)n_blocks, 256, 0, st>>>(dev_x, n, block, dev_q, dev_c);
    }
    return cudaGetLastError() == cudaSuccess ? PAC_OK : PAC_ERR_CUDA;
}

extern "C" pac_status pac_dequantize_absmax(int device, void* cuda_stream, const signed char* dev_q, const float* dev_c,
                                            long long n, int block, float* dev_out) {
    if (!dev_q || !dev_c || !dev_out || n < 1 || block < 1) return PAC_ERR_INVALID_ARG;
    if (cudaSetDevice(device) != cudaSuccess) return PAC_ERR_CUDA;
    if (n % 4 == 0 && block % 4 == 0 && ((uintptr_t)dev_q & 3) == 0 && ((uintptr_t)dev_out & 15) == 0) {
        const long long n4 = n / 4, want = (n4 + 1023) / 1024;
        const unsigned grid = (unsigned)(want < 148LL * 32 ? want : 148LL * 32);
        dequantize_absmax_vec_kernel<<<grid, 256, 0, (cudaStream_t)cuda_stream>>>((const char4*)dev_q, dev_c, n4, block / 4, (float4*)dev_out);
    } else {
        const long long want = (n + 255) / 256;
        const unsigned grid = (unsigned)(want < 148LL * 16 ? want : 148LL * 16);
        dequantize_absmax_kernel<<<grid, 256, 0, (cudaStream_t)cuda_stream>>>(dev_q, dev_c, n, block, dev_out);
    }
    return cudaGetLastError() == cudaSuccess ? PAC_OK : PAC_ERR_CUDA;
}

// ---------------------------------------------------------------------------
// Writer side of a cache file: what the first epoch does (Section IV-B) - every sample's per-layer
// backbone activations are recorded once, as they come out of the caller's backbone forward.
// ---------------------------------------------------------------------------
struct pac_cache_writer {
    int fd = -1;
    void* base = nullptr;
    size_t bytes = 0;
    CacheFileHeader h{};
    unsigned char* bounce = nullptr;       // page-locked, one sample
    size_t sample_bytes = 0;
    long long written = 0;
};

extern "C" pac_status pac_cache_writer_create(pac_cache_writer** out, const char* path, int dtype, long long N, int L, int S, int d,
                                              int labels_per_sample) {
    if (!out || !path) return PAC_ERR_INVALID_ARG;
    *out = nullptr;
    CacheFileHeader h{};
    std::memcpy(h.magic, CACHE_MAGIC, 8);
    h.version = 1u; h.dtype = dtype; h.N = N; h.L = L; h.S = S; h.d = d; h.labels_per_sample = labels_per_sample;
    if (!cache_file_header_ok(h)) return PAC_ERR_INVALID_ARG;
    pac_cache_writer* w = new (std::nothrow) pac_cache_writer();
    if (!w) return PAC_ERR_NOMEM;
    w->h = h;
    w->bytes = cache_file_bytes(h);
    w->sample_bytes = cache_file_data_bytes(h) / (size_t)N;
    w->fd = open(path, O_RDWR | O_CREAT | O_TRUNC, 0644);
    if (w->fd < 0 || ftruncate(w->fd, (off_t)w->bytes) != 0) {
        if (w->fd >= 0) close(w->fd);
        delete w;
        return PAC_ERR_INVALID_ARG;
    }
    w->base = mmap(nullptr, w->bytes, PROT_READ | PROT_WRITE, MAP_SHARED, w->fd, 0);
    if (w->base == MAP_FAILED) { close(w->fd); delete w; return PAC_ERR_NOMEM; }
    std::memcpy(w->base, &h, sizeof h);
    if (cudaMallocHost((void**)&w->bounce, w->sample_bytes) != cudaSuccess) {
        cudaGetLastError();
        w->bounce = nullptr;               // without a device (or page-locked memory) only host sources can be stored
    }
    *out = w;
    return PAC_OK;
}

extern "C" pac_status pac_cache_writer_store(pac_cache_writer* w, long long sample_id, const void* slabs, int slabs_on_device,
                                             const int* host_labels, void* cuda_stream) {
    if (!w || !slabs || !host_labels) return PAC_ERR_INVALID_ARG;
    if (sample_id < 0 || sample_id >= w->h.N) return PAC_ERR_SAMPLE_ID_RANGE;
    unsigned char* data = (unsigned char*)w->base + sizeof(CacheFileHeader);
    unsigned char* dst = data + (size_t)sample_id * w->sample_bytes;
    if (slabs_on_device) {
        if (!w->bounce) return PAC_ERR_CUDA;
        cudaStream_t st = (cudaStream_t)cuda_stream;
        // device -> page-locked bounce buffer -> file mapping (the mapping itself is pageable)
        if (cudaMemcpyAsync(w->bounce, slabs, w->sample_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
            cudaStreamSynchronize(st) != cudaSuccess) {
            cudaGetLastError();
            return PAC_ERR_CUDA;
        }
        std::memcpy(dst, w->bounce, w->sample_bytes);
    } else {
        std::memcpy(dst, slabs, w->sample_bytes);
    }
    int* lab = (int*)((unsigned char*)w->base + cache_file_labels_offset(w->h)) + (size_t)sample_id * w->h.labels_per_sample;
    std::memcpy(lab, host_labels, sizeof(int) * (size_t)w->h.labels_per_sample);
    w->written++;
    return PAC_OK;
}

extern "C" pac_status pac_cache_writer_close(pac_cache_writer* w) {
    if (!w) return PAC_ERR_INVALID_ARG;
    pac_status st = PAC_OK;
    if (w->base && msync(w->base, w->bytes, MS_SYNC) != 0) st = PAC_ERR_CUDA;
    if (w->base) munmap(w->base, w->bytes);
    if (w->fd >= 0) close(w->fd);
    if (w->bounce) cudaFreeHost(w->bounce);
    delete w;
    return st;
}

extern "C" pac_status pac_cache_file_info(const char* path, int* dtype, long long* N, int* L, int* S, int* d, int* labels_per_sample) {
    if (!path) return PAC_ERR_INVALID_ARG;
    const int fd = open(path, O_RDONLY);
    if (fd < 0) return PAC_ERR_INVALID_ARG;
    CacheFileHeader h;
    struct stat sb;
    const bool ok = read(fd, &h, sizeof h) == (ssize_t)sizeof h && cache_file_header_ok(h) && fstat(fd, &sb) == 0 &&
                    (size_t)sb.st_size >= cache_file_bytes(h);
    close(fd);
    if (!ok) return PAC_ERR_INVALID_ARG;
    if (dtype) *dtype = h.dtype;
    if (N) *N = h.N;
    if (L) *L = h.L;
    if (S) *S = h.S;
    if (d) *d = h.d;
    if (labels_per_sample) *labels_per_sample = h.labels_per_sample;
    return PAC_OK;
}
