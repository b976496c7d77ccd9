// Host runtime and C ABI of the rollout-decoding library: context/workspace, paged KV bookkeeping
// (free list, block tables, lengths), per-step launch sequence.  See include/spiral.h for the
// contract of every entry point.
#include "../../include/spiral.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "attn_decode.cuh"
#include "common.cuh"
#include "gemv.cuh"
#include "kernels_small.cuh"
#include "read_ceiling.cuh"
#include "gemm_tc.cuh"
#include "prefill.cuh"

using namespace spiral;
typedef __nv_bfloat16 bf16;

static thread_local std::string g_cuda_error;

#define CU_TRY(expr)                                                                       \
    do {                                                                                   \
        cudaError_t e__ = (expr);                                                          \
        if (e__ != cudaSuccess) {                                                          \
            g_cuda_error = std::string(#expr) + ": " + cudaGetErrorString(e__);            \
            return SPIRAL_ERR_CUDA;                                                        \
        }                                                                                  \
    } while (0)

#define LAUNCH_CHECK(ctx)                                                                  \
    do {                                                                                   \
        (ctx)->launches++;                                                                 \
        cudaError_t e__ = cudaGetLastError();                                              \
        if (e__ != cudaSuccess) {                                                          \
            g_cuda_error = std::string("kernel launch: ") + cudaGetErrorString(e__);       \
            return SPIRAL_ERR_CUDA;                                                        \
        }                                                                                  \
    } while (0)

// Launch on the step's stream with programmatic stream serialization: every kernel orders itself
// with grid_dependency_wait().
#define LAUNCH(ctx, kernel, grid, block, smem, st, ...)                                                    \
    do {                                                                                                   \
        (ctx)->launches++;                                                                                 \
        cudaError_t e__ = launch_kernel(true, kernel, dim3(grid), dim3(block), smem, st, __VA_ARGS__); \
        if (e__ != cudaSuccess) {                                                                          \
            g_cuda_error = std::string("launch of " #kernel ": ") + cudaGetErrorString(e__);               \
            cudaGetLastError();                                                                            \
            return SPIRAL_ERR_CUDA;                                                                        \
        }                                                                                                  \
    } while (0)

namespace {
// byte offset of the StepArgs inside a metadata block (8-byte aligned)
inline size_t meta_args_offset(int max_batch) { return (((size_t)5 * max_batch + 2) * sizeof(int32_t) + 7) & ~(size_t)7; }
constexpr int META_RING = 16;
constexpr int MAX_PIECES = 4;
constexpr int TC_MIN_BATCH = 16;    // below this the batch is no dense contraction: CUDA-core GEMV

// per-kernel timing (spiral_profile): one record = a pair of events around one launch
struct ProfRec { int cls; cudaEvent_t e0, e1; };

// Workspace of the dense context-append path, allocated at the first call that takes it (and grown
// when a later call needs more rows): activations for `cap` token rows, the rows' metadata and the
// attention work list, each with a pinned host mirror.
struct PrefillWs {
    int cap = 0;                        // token rows the buffers hold
    float *x = nullptr, *y = nullptr;
    __half *q = nullptr, *h = nullptr, *attn = nullptr, *act = nullptr;
    int32_t* meta_dev = nullptr;        // [4][cap]: game, position, -1, token index; then [2][max_batch]: rows to
    int32_t* meta_host = nullptr;       // hand to the LM head (source row, destination row)
    size_t meta_elems = 0;
    AppendItem* items_dev = nullptr;
    AppendItem* items_host = nullptr;
    int items_cap = 0;
    cudaEvent_t ev = nullptr;           // the last upload from the pinned mirrors
    bool ev_used = false;
};
constexpr int PREFILL_CHUNK_DEFAULT = 37 * PF_BN;   // 9472 rows: 37 token tiles x (20 | 48 | 152 row tiles) fill
                                                    // 148 SMs in whole waves for the Qwen3-4B matrices
}  // namespace

struct spiral_ctx {
    spiral_model_desc d;
    int device, max_batch, max_ctx;
    int qkv_rows, group;
    const bf16 *embed, *lm_head, *final_norm;
    std::vector<const bf16*> ln1, wqkv, bqkv, q_norm, k_norm, wo, ln2, w_gate_up, w_down;
    // workspace (device)
    float* x = nullptr;            // residual stream [max_batch][d_model]
    __half* h = nullptr;           // normalised activations [max_batch][d_model] (fp16)
    __half* attn_out = nullptr;    // [max_batch][n_q_heads*head_dim]
    __half* act = nullptr;         // [max_batch][d_ff]
    float* q = nullptr;            // [max_batch][n_q_heads][head_dim]
    float* pieces = nullptr;       // split-K pieces of the current GEMM
    size_t pieces_elems = 0;
    float *o_part = nullptr, *m_part = nullptr, *l_part = nullptr;   // attention partials
    int* attn_item_cnt = nullptr;  // [max_batch * n_kv_heads] partials published per item (zero between launches)
    int n_sm = 0;
    float* logits = nullptr;       // [max_batch][vocab] (CUDA-core LM-head path only)
    float *cos_tab = nullptr, *sin_tab = nullptr;
    // step metadata, uploaded once per step: int32 [4][max_batch] (game, position, new page, token
    // index per slot), the attention schedule int32 [max_batch + 2], then one StepArgs
    size_t meta_bytes = 0;
    uint8_t* meta_dev = nullptr;
    uint8_t* meta_host = nullptr;  // pinned ring [META_RING][meta_bytes]
    cudaEvent_t meta_ev[META_RING];
    bool meta_ev_used[META_RING];
    int meta_next = 0;
    cudaStream_t copy_stream = nullptr;    // *_host entry point: carries the noise while the layers run
    cudaEvent_t copy_ev = nullptr;
    int32_t* tok_stage = nullptr;      // device staging of the *_host entry point
    float* gumbel_stage = nullptr;
    int32_t* tokout_stage = nullptr;
    int* status = nullptr;
    int64_t launches = 0;
    std::vector<int> scratch_len;      // host scratch: tokens attended per slot
    std::vector<int> scratch_last;     // host scratch (prefill): game whose last new token a slot carries
    bool use_graph = true;             // replay a recorded CUDA graph of the step when the stream allows it
    bool attn_skip_once = false;       // wait-timeout self-test: the next attention launch leaves a page load out
    unsigned prof_mask = 0;            // bit c set: launches of kernel class c are bracketed by events
    std::vector<ProfRec> prof_recs;
    std::vector<cudaEvent_t> prof_pool;   // events ready for reuse
    TcState tc;
    PrefillWs pf;
    int prefill_chunk = PREFILL_CHUNK_DEFAULT;    // token rows per pass of the dense append path (SPIRAL_PREFILL_CHUNK)
    bool prefill_dense = true;                    // SPIRAL_PREFILL_DENSE=0: always append through decode-shaped steps
    bool pf_ready = false;                        // every layer matrix is registered for the tensor-core path
    bool append_attn_tc = true;                   // SPIRAL_APPEND_ATTN=mma: the mma.sync formulation of the append attention
    int append_tiles = 2;                         // query tiles per CTA of the tcgen05 formulation (SPIRAL_APPEND_ATTN=tc1: one)
};

struct spiral_kv {
    spiral_ctx* ctx;
    uint16_t* pool;
    int kv_f16;                            // 1: fp16 pages, 0: bf16 pages
    int page_size, n_pages, max_games, max_ctx, max_pages;
    std::vector<int32_t> free_list;        // stack; back() is handed out next
    std::vector<int32_t> page_ref;         // games holding each page (> 1: a prefix shared after spiral_kv_fork)
    std::vector<int32_t> seq_len;          // host shadow of every game's cached length
    std::vector<int32_t> n_game_pages;     // pages currently owned by each game
    std::vector<int32_t> table;            // host shadow [max_games][max_pages]
    std::vector<uint32_t> stamp;           // duplicate detection
    uint32_t epoch = 0;
    int32_t* table_dev = nullptr;
    // recorded decode steps, one per batch size (the launch sequence depends on nothing else)
    struct StepGraph { cudaGraphExec_t exec = nullptr; int64_t launches = 0, eager_launches = 0; int uses = 0; bool failed = false; };
    std::map<int, StepGraph> graphs;
    int64_t step_launches = 0;             // kernels in the most recent eagerly launched step
    CUtensorMap pool_map;                  // pool as rows of head_dim elements; box = 32 rows x 64 elements
    CUtensorMap pool_map16;                // the same with a 16-row box (the K or the V rows of one page and head)
};

static inline int32_t* meta_i32(spiral_ctx* c) { return (int32_t*)c->meta_dev; }
static inline const StepArgs* meta_args(spiral_ctx* c) {
    return (const StepArgs*)(c->meta_dev + meta_args_offset(c->max_batch));
}
// attention schedule of the step inside the metadata block (host slot `mh` / device)
static inline int32_t* meta_cum_host(spiral_ctx* c, int32_t* mh) { return mh + (size_t)4 * c->max_batch; }
static inline const int32_t* meta_cum_dev(spiral_ctx* c) { return meta_i32(c) + (size_t)4 * c->max_batch; }

// ------------------------------------------------------------------------------------------------

extern "C" const char* spiral_strerror(int code) {
    switch (code) {
        case SPIRAL_OK: return "ok";
        case SPIRAL_ERR_INVALID: return "invalid argument";
        case SPIRAL_ERR_OOM: return "out of KV pages or memory";
        case SPIRAL_ERR_CUDA: return "CUDA call failed";
        case SPIRAL_ERR_TIMEOUT: return "device-side wait timed out";
        case SPIRAL_ERR_DEVICE_CHECK: return "device-side check failed";
        case SPIRAL_ERR_UNSUPPORTED: return "unsupported shape";
        case SPIRAL_ERR_TOO_LARGE: return "size beyond the fixed capacity of this entry point";
        default: return "unknown error";
    }
}

extern "C" const char* spiral_last_cuda_error(void) { return g_cuda_error.c_str(); }

extern "C" size_t spiral_kv_page_bytes(const spiral_model_desc* d, int page_size) {
    if (!d || page_size <= 0) return 0;
    return (size_t)d->n_layers * d->n_kv_heads * 2 * (size_t)page_size * d->head_dim * sizeof(bf16);
}

static void free_ctx(spiral_ctx* c) {
    if (!c) return;
    cudaSetDevice(c->device);
    cudaDeviceSynchronize();
    cudaFree(c->x); cudaFree(c->h); cudaFree(c->attn_out); cudaFree(c->act); cudaFree(c->q);
    cudaFree(c->pieces); cudaFree(c->o_part); cudaFree(c->m_part); cudaFree(c->l_part);
    cudaFree(c->attn_item_cnt); cudaFree(c->logits); cudaFree(c->cos_tab); cudaFree(c->sin_tab); cudaFree(c->meta_dev);
    cudaFree(c->tok_stage); cudaFree(c->gumbel_stage); cudaFree(c->tokout_stage); cudaFree(c->status);
    if (c->meta_host) cudaFreeHost(c->meta_host);
    if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
    if (c->copy_ev) cudaEventDestroy(c->copy_ev);
    for (int i = 0; i < META_RING; ++i)
        if (c->meta_ev[i]) cudaEventDestroy(c->meta_ev[i]);
    for (auto& r : c->prof_recs) { cudaEventDestroy(r.e0); cudaEventDestroy(r.e1); }
    for (auto e : c->prof_pool) cudaEventDestroy(e);
    cudaFree(c->pf.x); cudaFree(c->pf.y); cudaFree(c->pf.q); cudaFree(c->pf.h); cudaFree(c->pf.attn); cudaFree(c->pf.act);
    cudaFree(c->pf.meta_dev); cudaFree(c->pf.items_dev);
    if (c->pf.meta_host) cudaFreeHost(c->pf.meta_host);
    if (c->pf.items_host) cudaFreeHost(c->pf.items_host);
    if (c->pf.ev) cudaEventDestroy(c->pf.ev);
    tc_destroy(c->tc);
    delete c;
}

extern "C" int spiral_init(spiral_ctx** out, const spiral_model_desc* d, const spiral_weights* w, int device,
                           int max_batch, int max_ctx) {
    if (!out || !d || !w) return SPIRAL_ERR_INVALID;
    if (max_batch < 1 || max_batch > 256 || max_ctx < 1) return SPIRAL_ERR_INVALID;
    if (d->n_layers < 1 || d->vocab < 1 || d->n_kv_heads < 1 || d->n_q_heads < 1) return SPIRAL_ERR_INVALID;
    if (!w->embed || !w->final_norm || !w->ln1 || !w->wqkv || !w->wo || !w->ln2 || !w->w_gate_up || !w->w_down)
        return SPIRAL_ERR_INVALID;
    if (!d->tied_embed && !w->lm_head) return SPIRAL_ERR_INVALID;
    if (d->qkv_bias && !w->bqkv) return SPIRAL_ERR_INVALID;
    if (d->qk_norm && (!w->q_norm || !w->k_norm)) return SPIRAL_ERR_INVALID;
    if (d->head_dim != 64 && d->head_dim != 128) return SPIRAL_ERR_UNSUPPORTED;
    if (d->n_q_heads % d->n_kv_heads != 0 || d->n_q_heads / d->n_kv_heads > 8) return SPIRAL_ERR_UNSUPPORTED;
    if (d->d_model > 4 * RMS_PER_THREAD * RMS_THREADS || d->head_dim > 128) return SPIRAL_ERR_UNSUPPORTED;
    if (d->d_model % 64 != 0 || d->d_ff % 8 != 0 || (d->n_q_heads * d->head_dim) % 64 != 0)
        return SPIRAL_ERR_UNSUPPORTED;
    if (!(d->rope_theta > 0) || !(d->rms_eps >= 0)) return SPIRAL_ERR_INVALID;
    CU_TRY(cudaSetDevice(device));

    spiral_ctx* c = new (std::nothrow) spiral_ctx();
    if (!c) return SPIRAL_ERR_OOM;
    c->d = *d; c->device = device; c->max_batch = max_batch; c->max_ctx = max_ctx;
    {
        const char* off = std::getenv("SPIRAL_NO_GRAPH");
        c->use_graph = !(off && off[0] == '1');
        off = std::getenv("SPIRAL_PREFILL_CHUNK");
        if (off) c->prefill_chunk = std::max(PF_BN, std::min(1 << 16, (atoi(off) + PF_BN - 1) / PF_BN * PF_BN));
        off = std::getenv("SPIRAL_PREFILL_DENSE");
        c->prefill_dense = !(off && off[0] == '0');
        off = std::getenv("SPIRAL_APPEND_ATTN");
        c->append_attn_tc = !(off && off[0] == 'm');
        if (off && off[0] == 't' && off[1] == 'c' && (off[2] == '1' || off[2] == '2')) c->append_tiles = off[2] - '0';
    }
    c->scratch_len.assign(max_batch, 0);
    c->scratch_last.assign(max_batch, -1);
    c->qkv_rows = (d->n_q_heads + 2 * d->n_kv_heads) * d->head_dim;
    c->group = d->n_q_heads / d->n_kv_heads;
    for (int i = 0; i < META_RING; ++i) { c->meta_ev[i] = nullptr; c->meta_ev_used[i] = false; }
    c->embed = (const bf16*)w->embed;
    c->lm_head = d->tied_embed ? (const bf16*)w->embed : (const bf16*)w->lm_head;
    c->final_norm = (const bf16*)w->final_norm;
    const int L = d->n_layers;
    auto copy_ptrs = [&](std::vector<const bf16*>& dst, const void* const* src, bool present) {
        dst.assign(L, nullptr);
        if (present && src)
            for (int l = 0; l < L; ++l) dst[l] = (const bf16*)src[l];
    };
    copy_ptrs(c->ln1, w->ln1, true); copy_ptrs(c->wqkv, w->wqkv, true);
    copy_ptrs(c->bqkv, w->bqkv, d->qkv_bias != 0);
    copy_ptrs(c->q_norm, w->q_norm, d->qk_norm != 0); copy_ptrs(c->k_norm, w->k_norm, d->qk_norm != 0);
    copy_ptrs(c->wo, w->wo, true); copy_ptrs(c->ln2, w->ln2, true);
    copy_ptrs(c->w_gate_up, w->w_gate_up, true); copy_ptrs(c->w_down, w->w_down, true);
    for (int l = 0; l < L; ++l) {
        bool ok = c->ln1[l] && c->wqkv[l] && c->wo[l] && c->ln2[l] && c->w_gate_up[l] && c->w_down[l] &&
                  (!d->qkv_bias || c->bqkv[l]) && (!d->qk_norm || (c->q_norm[l] && c->k_norm[l]));
        ok = ok && ((uintptr_t)c->wqkv[l] % 16 == 0) && ((uintptr_t)c->wo[l] % 16 == 0) &&
             ((uintptr_t)c->w_gate_up[l] % 16 == 0) && ((uintptr_t)c->w_down[l] % 16 == 0);
        if (!ok) { delete c; return SPIRAL_ERR_INVALID; }
    }
    if ((uintptr_t)c->embed % 16 || (uintptr_t)c->lm_head % 16) { delete c; return SPIRAL_ERR_INVALID; }

    const size_t MB = max_batch;
    const int qd = d->n_q_heads * d->head_dim;
    const size_t n_max = std::max<size_t>({(size_t)c->qkv_rows, (size_t)d->d_model, (size_t)2 * d->d_ff});
    c->pieces_elems = (size_t)MAX_PIECES * MB * n_max;
    {
        cudaDeviceProp prop;
        CU_TRY(cudaGetDeviceProperties(&prop, device));
        c->n_sm = prop.multiProcessorCount;
    }
    const size_t parts = ((size_t)c->n_sm * ATTN_WARPS + MB * d->n_kv_heads) * c->group;
    const int half = d->head_dim / 2;
    cudaError_t e = cudaSuccess;
    auto A = [&](void** p, size_t bytes) { if (e == cudaSuccess) e = cudaMalloc(p, bytes); };
    A((void**)&c->x, MB * d->d_model * sizeof(float));
    A((void**)&c->h, MB * d->d_model * sizeof(bf16));
    A((void**)&c->attn_out, MB * qd * sizeof(bf16));
    A((void**)&c->act, MB * d->d_ff * sizeof(bf16));
    A((void**)&c->q, MB * qd * sizeof(float));
    A((void**)&c->o_part, parts * d->head_dim * sizeof(float));
    A((void**)&c->m_part, parts * sizeof(float));
    A((void**)&c->l_part, parts * sizeof(float));
    A((void**)&c->attn_item_cnt, MB * d->n_kv_heads * sizeof(int));
    A((void**)&c->logits, MB * d->vocab * sizeof(float));
    A((void**)&c->cos_tab, (size_t)max_ctx * half * sizeof(float));
    A((void**)&c->sin_tab, (size_t)max_ctx * half * sizeof(float));
    c->meta_bytes = (meta_args_offset(max_batch) + sizeof(StepArgs) + 15) & ~(size_t)15;
    A((void**)&c->meta_dev, c->meta_bytes);
    A((void**)&c->tok_stage, MB * sizeof(int32_t));
    A((void**)&c->tokout_stage, MB * sizeof(int32_t));
    A((void**)&c->gumbel_stage, MB * d->vocab * sizeof(float));
    A((void**)&c->status, sizeof(int));
    if (e == cudaSuccess) e = cudaMallocHost((void**)&c->meta_host, (size_t)META_RING * c->meta_bytes);
    for (int i = 0; i < META_RING && e == cudaSuccess; ++i)
        e = cudaEventCreateWithFlags(&c->meta_ev[i], cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->copy_ev, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaMemset(c->status, 0, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(c->attn_item_cnt, 0, MB * d->n_kv_heads * sizeof(int));
    if (e != cudaSuccess) {
        g_cuda_error = std::string("spiral_init allocation: ") + cudaGetErrorString(e);
        bool oom = e == cudaErrorMemoryAllocation;
        cudaGetLastError();
        free_ctx(c);
        return oom ? SPIRAL_ERR_OOM : SPIRAL_ERR_CUDA;
    }
    size_t tab = (size_t)max_ctx * half;
    rope_table_kernel<<<(unsigned)((tab + 255) / 256), 256>>>(d->rope_theta, d->head_dim, max_ctx, c->cos_tab,
                                                             c->sin_tab);
    c->launches++;
    e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        g_cuda_error = std::string("rope table: ") + cudaGetErrorString(e);
        free_ctx(c);
        return SPIRAL_ERR_CUDA;
    }
    {
        const int attn_smem = ATTN_WARPS * ATTN_STAGES * 2 * 4096 + 1024;
        e = cudaFuncSetAttribute(attn_decode_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_smem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attn_decode_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_smem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attn_decode_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_smem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attn_decode_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_smem);
        if (e != cudaSuccess) {
            g_cuda_error = std::string("attention shared memory: ") + cudaGetErrorString(e);
            free_ctx(c);
            return SPIRAL_ERR_CUDA;
        }
    }
    // tensor-core path: private fp16 copies and TMA descriptors of every matrix, work plans, and
    // the number of split-K pieces they produce (sizes the pieces buffer)
    int rc = tc_init(c->tc, device, max_batch);
    if (rc == SPIRAL_ERR_CUDA) g_cuda_error = tc_last_error();
    if (rc != SPIRAL_OK) { free_ctx(c); return rc; }
    if (c->tc.ready && max_batch >= TC_MIN_BATCH) {
        struct M { const bf16* w; int rows, k; };
        std::vector<M> mats;
        for (int l = 0; l < L; ++l) {
            mats.push_back({c->wqkv[l], c->qkv_rows, d->d_model});
            mats.push_back({c->wo[l], d->d_model, qd});
            mats.push_back({c->w_gate_up[l], 2 * d->d_ff, d->d_model});
            mats.push_back({c->w_down[l], d->d_model, d->d_ff});
        }
        mats.push_back({c->lm_head, d->vocab, d->d_model});
        for (const M& m : mats) {
            if (!tc_usable(c->tc, m.rows, m.k, max_batch, false)) continue;
            rc = tc_register_weight(c->tc, m.w, m.rows, m.k, true, 0, &c->launches, nullptr);
            if (rc == SPIRAL_OK && m.w != c->lm_head) {
                int np = tc_max_pieces(c->tc, m.rows, m.k);
                if (np < 0) rc = SPIRAL_ERR_CUDA;
                else c->pieces_elems = std::max(c->pieces_elems, (size_t)np * MB * m.rows);
            }
            if (rc != SPIRAL_OK) {
                if (rc == SPIRAL_ERR_CUDA) g_cuda_error = tc_last_error();
                free_ctx(c);
                return rc;
            }
        }
        e = cudaDeviceSynchronize();
        if (e != cudaSuccess) {
            g_cuda_error = std::string("weight re-encoding: ") + cudaGetErrorString(e);
            free_ctx(c);
            return SPIRAL_ERR_CUDA;
        }
        // dense append path: needs every layer matrix on the tensor-core path
        c->pf_ready = true;
        for (const M& m : mats)
            if (m.w != c->lm_head && !tc_usable(c->tc, m.rows, m.k, max_batch, false)) c->pf_ready = false;
        if (c->pf_ready) {
            rc = pf_gemm_setup();
            e = cudaSuccess;
            if (rc == SPIRAL_OK) e = cudaFuncSetAttribute(attn_append_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)app_smem_bytes(128));
            if (rc == SPIRAL_OK && e == cudaSuccess) e = cudaFuncSetAttribute(attn_append_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)app_smem_bytes(64));
            if (rc == SPIRAL_OK && e == cudaSuccess) e = cudaFuncSetAttribute((attn_append_tc_kernel<128, 1>), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)apt_smem_bytes(128, 1));
            if (rc == SPIRAL_OK && e == cudaSuccess) e = cudaFuncSetAttribute((attn_append_tc_kernel<128, 2>), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)apt_smem_bytes(128, 2));
            if (rc == SPIRAL_OK && e == cudaSuccess) e = cudaFuncSetAttribute((attn_append_tc_kernel<64, 1>), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)apt_smem_bytes(64, 1));
            if (rc == SPIRAL_OK && e == cudaSuccess) e = cudaFuncSetAttribute((attn_append_tc_kernel<64, 2>), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)apt_smem_bytes(64, 2));
            if (rc != SPIRAL_OK || e != cudaSuccess) {
                g_cuda_error = rc != SPIRAL_OK ? tc_last_error() : std::string("append attention shared memory: ") + cudaGetErrorString(e);
                free_ctx(c);
                return SPIRAL_ERR_CUDA;
            }
        }
    }
    e = cudaMalloc((void**)&c->pieces, c->pieces_elems * sizeof(float));
    if (e != cudaSuccess) {
        g_cuda_error = std::string("pieces buffer: ") + cudaGetErrorString(e);
        cudaGetLastError();
        free_ctx(c);
        return e == cudaErrorMemoryAllocation ? SPIRAL_ERR_OOM : SPIRAL_ERR_CUDA;
    }
    *out = c;
    return SPIRAL_OK;
}

extern "C" int spiral_kv_alloc(spiral_ctx* ctx, void* pool_dev, size_t pool_bytes, int page_size, int kv_dtype,
                               int max_games, int max_ctx, spiral_kv** out) {
    if (!ctx || !pool_dev || !out || max_games < 1 || max_ctx < 1 || max_ctx > ctx->max_ctx)
        return SPIRAL_ERR_INVALID;
    if (page_size != ATTN_PAGE) return SPIRAL_ERR_UNSUPPORTED;
    if (kv_dtype != SPIRAL_KV_F16 && kv_dtype != SPIRAL_KV_BF16) return SPIRAL_ERR_INVALID;
    if ((uintptr_t)pool_dev % 256 != 0) return SPIRAL_ERR_INVALID;
    size_t pb = spiral_kv_page_bytes(&ctx->d, page_size);
    size_t n_pages = pool_bytes / pb;
    if (n_pages < 1 || n_pages > 0x7fffffff) return SPIRAL_ERR_INVALID;
    CU_TRY(cudaSetDevice(ctx->device));
    spiral_kv* kv = new (std::nothrow) spiral_kv();
    if (!kv) return SPIRAL_ERR_OOM;
    kv->ctx = ctx; kv->pool = (uint16_t*)pool_dev; kv->kv_f16 = kv_dtype == SPIRAL_KV_F16; kv->page_size = page_size; kv->n_pages = (int)n_pages;
    kv->max_games = max_games; kv->max_ctx = max_ctx; kv->max_pages = (max_ctx + page_size - 1) / page_size;
    try {
        kv->free_list.resize(n_pages);
        for (size_t i = 0; i < n_pages; ++i) kv->free_list[i] = (int32_t)(n_pages - 1 - i);
        kv->page_ref.assign(n_pages, 0);
        kv->seq_len.assign(max_games, 0);
        kv->n_game_pages.assign(max_games, 0);
        kv->table.assign((size_t)max_games * kv->max_pages, -1);
        kv->stamp.assign(max_games, 0);
    } catch (...) { delete kv; return SPIRAL_ERR_OOM; }
    {
        // the attention kernel fetches (page, head) blocks with tiled TMA: y = pool row, 31 bits
        const size_t pool_rows = n_pages * (size_t)ctx->d.n_layers * ctx->d.n_kv_heads * 2 * page_size;
        if (!ctx->tc.ready || pool_rows > 0x7fffffffull) { delete kv; return SPIRAL_ERR_UNSUPPORTED; }
        int rc = tc_encode(ctx->tc, &kv->pool_map, pool_dev, (uint64_t)ctx->d.head_dim, pool_rows, 32, !kv->kv_f16);
        if (rc == SPIRAL_OK)
            rc = tc_encode(ctx->tc, &kv->pool_map16, pool_dev, (uint64_t)ctx->d.head_dim, pool_rows, 16, !kv->kv_f16);
        if (rc) { g_cuda_error = tc_last_error(); delete kv; return rc; }
    }
    size_t tb = kv->table.size() * sizeof(int32_t);
    cudaError_t e = cudaMalloc((void**)&kv->table_dev, tb);
    if (e == cudaSuccess) e = cudaMemset(kv->table_dev, 0xff, tb);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        g_cuda_error = std::string("spiral_kv_alloc: ") + cudaGetErrorString(e);
        cudaGetLastError();
        cudaFree(kv->table_dev);
        delete kv;
        return e == cudaErrorMemoryAllocation ? SPIRAL_ERR_OOM : SPIRAL_ERR_CUDA;
    }
    *out = kv;
    return SPIRAL_OK;
}

extern "C" int spiral_kv_release(spiral_kv* kv, int n, const int32_t* ids) {
    if (!kv || n < 0 || (n > 0 && !ids)) return SPIRAL_ERR_INVALID;
    for (int i = 0; i < n; ++i)
        if (ids[i] < 0 || ids[i] >= kv->max_games) return SPIRAL_ERR_INVALID;
    for (int i = 0; i < n; ++i) {
        int g = ids[i];
        for (int pgi = kv->n_game_pages[g] - 1; pgi >= 0; --pgi) {
            const int32_t pg = kv->table[(size_t)g * kv->max_pages + pgi];
            if (--kv->page_ref[pg] == 0) kv->free_list.push_back(pg);      // a shared page stays with its other holders
            kv->table[(size_t)g * kv->max_pages + pgi] = -1;
        }
        kv->n_game_pages[g] = 0;
        kv->seq_len[g] = 0;
    }
    return SPIRAL_OK;
}

extern "C" int spiral_kv_truncate(spiral_kv* kv, int n, const int32_t* ids, const int32_t* new_len) {
    if (!kv || n < 0 || (n > 0 && (!ids || !new_len))) return SPIRAL_ERR_INVALID;
    for (int i = 0; i < n; ++i)
        if (ids[i] < 0 || ids[i] >= kv->max_games || new_len[i] < 0 || new_len[i] > kv->seq_len[ids[i]])
            return SPIRAL_ERR_INVALID;
    for (int i = 0; i < n; ++i) {
        // cutting into a shared page would let the game's next token overwrite what other games still read
        const int g = ids[i];
        if (new_len[i] % kv->page_size != 0 && new_len[i] < kv->seq_len[g] &&
            kv->page_ref[kv->table[(size_t)g * kv->max_pages + new_len[i] / kv->page_size]] > 1)
            return SPIRAL_ERR_UNSUPPORTED;
    }
    for (int i = 0; i < n; ++i) {
        int g = ids[i];
        int keep = (new_len[i] + kv->page_size - 1) / kv->page_size;
        while (kv->n_game_pages[g] > keep) {
            int pgi = --kv->n_game_pages[g];
            const int32_t pg = kv->table[(size_t)g * kv->max_pages + pgi];
            if (--kv->page_ref[pg] == 0) kv->free_list.push_back(pg);
            kv->table[(size_t)g * kv->max_pages + pgi] = -1;
        }
        kv->seq_len[g] = new_len[i];
    }
    return SPIRAL_OK;
}

extern "C" int spiral_kv_seq_len(const spiral_kv* kv, int game_id, int32_t* out) {
    if (!kv || !out || game_id < 0 || game_id >= kv->max_games) return SPIRAL_ERR_INVALID;
    *out = kv->seq_len[game_id];
    return SPIRAL_OK;
}

extern "C" int spiral_kv_free_pages(const spiral_kv* kv, int32_t* out) {
    if (!kv || !out) return SPIRAL_ERR_INVALID;
    *out = (int32_t)kv->free_list.size();
    return SPIRAL_OK;
}

// give game g enough pages for `len` tokens; the caller has checked the free count
// one page of every layer: [layer][page][kv_head][K|V][page_size][head_dim] -> the same slot of another page
__global__ void kv_copy_page_kernel(uint16_t* __restrict__ pool, int src_page, int dst_page, int n_pages,
                                    size_t page_layer_elems) {
    const uint4* s = reinterpret_cast<const uint4*>(pool + ((size_t)blockIdx.x * n_pages + src_page) * page_layer_elems);
    uint4* d = reinterpret_cast<uint4*>(pool + ((size_t)blockIdx.x * n_pages + dst_page) * page_layer_elems);
    for (size_t i = threadIdx.x; i < page_layer_elems / 8; i += blockDim.x) d[i] = s[i];
}

static int upload_table_row(spiral_kv* kv, int g, cudaStream_t st);

extern "C" int spiral_kv_fork(spiral_ctx* ctx, spiral_kv* kv, int src_game, int dst_game, int n_tokens, void* stream) {
    if (!ctx || !kv || kv->ctx != ctx) return SPIRAL_ERR_INVALID;
    if (src_game < 0 || src_game >= kv->max_games || dst_game < 0 || dst_game >= kv->max_games || src_game == dst_game)
        return SPIRAL_ERR_INVALID;
    if (n_tokens < 1 || n_tokens > kv->seq_len[src_game]) return SPIRAL_ERR_INVALID;
    if (kv->seq_len[dst_game] != 0 || kv->n_game_pages[dst_game] != 0) return SPIRAL_ERR_INVALID;
    const int full = n_tokens / kv->page_size, part = n_tokens % kv->page_size;
    if (part && kv->free_list.empty()) return SPIRAL_ERR_OOM;
    cudaStream_t st = (cudaStream_t)stream;
    CU_TRY(cudaSetDevice(ctx->device));
    int32_t* src = kv->table.data() + (size_t)src_game * kv->max_pages;
    int32_t* dst = kv->table.data() + (size_t)dst_game * kv->max_pages;
    for (int i = 0; i < full; ++i) {            // whole pages: shared, never written again (appends go to later pages)
        dst[i] = src[i];
        ++kv->page_ref[src[i]];
    }
    kv->n_game_pages[dst_game] = full;
    if (part) {                                 // the partly filled page: a private copy
        const int32_t pg = kv->free_list.back();
        kv->free_list.pop_back();
        kv->page_ref[pg] = 1;
        dst[full] = pg;
        kv->n_game_pages[dst_game] = full + 1;
        const size_t page_layer_elems = (size_t)ctx->d.n_kv_heads * 2 * kv->page_size * ctx->d.head_dim;
        kv_copy_page_kernel<<<ctx->d.n_layers, 256, 0, st>>>(kv->pool, src[full], pg, kv->n_pages, page_layer_elems);
        LAUNCH_CHECK(ctx);
    }
    kv->seq_len[dst_game] = n_tokens;
    return upload_table_row(kv, dst_game, st);
}

static void grow_game(spiral_kv* kv, int g, int len) {
    int need = (len + kv->page_size - 1) / kv->page_size;
    while (kv->n_game_pages[g] < need) {
        int32_t pg = kv->free_list.back();
        kv->free_list.pop_back();
        kv->page_ref[pg] = 1;
        kv->table[(size_t)g * kv->max_pages + kv->n_game_pages[g]] = pg;
        kv->n_game_pages[g]++;
    }
}
static int pages_missing(const spiral_kv* kv, int g, int len) {
    int need = (len + kv->page_size - 1) / kv->page_size;
    return std::max(0, need - kv->n_game_pages[g]);
}
static int upload_table_row(spiral_kv* kv, int g, cudaStream_t st) {
    CU_TRY(cudaMemcpyAsync(kv->table_dev + (size_t)g * kv->max_pages, kv->table.data() + (size_t)g * kv->max_pages,
                           (size_t)kv->max_pages * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    return SPIRAL_OK;
}

extern "C" int spiral_kv_load(spiral_ctx* ctx, spiral_kv* kv, int game_id, int layer, int n_tokens,
                              const void* k_dev, const void* v_dev, void* stream) {
    if (!ctx || !kv || kv->ctx != ctx || !k_dev || !v_dev) return SPIRAL_ERR_INVALID;
    if (game_id < 0 || game_id >= kv->max_games || layer < 0 || layer >= ctx->d.n_layers) return SPIRAL_ERR_INVALID;
    if (n_tokens < 1 || n_tokens > kv->max_ctx) return SPIRAL_ERR_INVALID;
    cudaStream_t st = (cudaStream_t)stream;
    CU_TRY(cudaSetDevice(ctx->device));
    int miss = pages_missing(kv, game_id, n_tokens);
    if (miss > (int)kv->free_list.size()) return SPIRAL_ERR_OOM;
    if (miss > 0) {
        grow_game(kv, game_id, n_tokens);
        int rc = upload_table_row(kv, game_id, st);
        if (rc) return rc;
    }
    kv->seq_len[game_id] = n_tokens;
    kv_load_kernel<<<n_tokens, 128, 0, st>>>((const uint16_t*)k_dev, (const uint16_t*)v_dev, n_tokens,
                                             kv->table_dev + (size_t)game_id * kv->max_pages, kv->page_size,
                                             kv->n_pages, layer, ctx->d.n_kv_heads, ctx->d.head_dim, kv->pool);
    LAUNCH_CHECK(ctx);
    return SPIRAL_OK;
}

// ------------------------------------------------------------------------------------------------
// per-kernel timing
// ------------------------------------------------------------------------------------------------

static cudaEvent_t prof_event(spiral_ctx* c) {
    cudaEvent_t e = nullptr;
    if (!c->prof_pool.empty()) { e = c->prof_pool.back(); c->prof_pool.pop_back(); return e; }
    if (cudaEventCreate(&e) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return e;
}
// returns the record index, or -1 when class `cls` is not being timed
static int prof_begin(spiral_ctx* c, int cls, cudaStream_t st) {
    if (!((c->prof_mask >> cls) & 1u)) return -1;
    ProfRec r{cls, prof_event(c), prof_event(c)};
    if (!r.e0 || !r.e1) return -1;
    cudaEventRecord(r.e0, st);
    c->prof_recs.push_back(r);
    return (int)c->prof_recs.size() - 1;
}
static void prof_end(spiral_ctx* c, int rec, cudaStream_t st) {
    if (rec >= 0) cudaEventRecord(c->prof_recs[rec].e1, st);
}

extern "C" int spiral_profile(spiral_ctx* ctx, uint32_t class_mask) {
    if (!ctx || class_mask >> SPIRAL_KC_COUNT) return SPIRAL_ERR_INVALID;
    CU_TRY(cudaSetDevice(ctx->device));
    CU_TRY(cudaDeviceSynchronize());
    for (auto& r : ctx->prof_recs) { ctx->prof_pool.push_back(r.e0); ctx->prof_pool.push_back(r.e1); }
    ctx->prof_recs.clear();
    ctx->prof_mask = class_mask;
    return SPIRAL_OK;
}

extern "C" int spiral_profile_read(spiral_ctx* ctx, int kernel_class, double* total_ms, int64_t* n_launches) {
    if (!ctx || kernel_class < 0 || kernel_class >= SPIRAL_KC_COUNT || !total_ms || !n_launches)
        return SPIRAL_ERR_INVALID;
    CU_TRY(cudaSetDevice(ctx->device));
    CU_TRY(cudaDeviceSynchronize());
    double tot = 0;
    int64_t n = 0;
    for (auto& r : ctx->prof_recs) {
        if (r.cls != kernel_class) continue;
        float ms = 0.f;
        CU_TRY(cudaEventElapsedTime(&ms, r.e0, r.e1));
        tot += ms;
        ++n;
    }
    *total_ms = tot;
    *n_launches = n;
    return SPIRAL_OK;
}

// ------------------------------------------------------------------------------------------------
// per-step launch sequence
// ------------------------------------------------------------------------------------------------

// y = x W^T as split-K pieces in ctx->pieces (or `y_direct` as a single piece)
static int launch_linear_impl(spiral_ctx* c, const bf16* W, int rows, int K, const __half* X, int n, float* y_direct,
                              int path, Pieces* out, cudaStream_t st);
static int launch_linear(spiral_ctx* c, int cls, const bf16* W, int rows, int K, const __half* X, int n,
                         float* y_direct, int path, Pieces* out, cudaStream_t st) {
    int rec = prof_begin(c, cls, st);
    int rc = launch_linear_impl(c, W, rows, K, X, n, y_direct, path, out, st);
    prof_end(c, rec, st);
    return rc;
}
static int launch_linear_impl(spiral_ctx* c, const bf16* W, int rows, int K, const __half* X, int n, float* y_direct,
                              int path, Pieces* out, cudaStream_t st) {
    float* y = y_direct ? y_direct : c->pieces;
    if (path != 1 && !y_direct && tc_usable(c->tc, rows, K, n, path == 2)) {
        int rc = tc_linear(c->tc, W, rows, K, X, n, c->pieces, c->pieces_elems, out, c->status, st, &c->launches);
        if (rc == SPIRAL_ERR_CUDA) g_cuda_error = tc_last_error();
        if (rc != SPIRAL_ERR_UNSUPPORTED || path == 2) return rc;
    }
    if (path == 2) return SPIRAL_ERR_UNSUPPORTED;
    if (K % 8 != 0) return SPIRAL_ERR_UNSUPPORTED;
    dim3 grid((rows + 2 * GEMV_WARPS - 1) / (2 * GEMV_WARPS), (n + GEMV_BC - 1) / GEMV_BC);
    LAUNCH(c, gemv_kernel, grid, GEMV_WARPS * 32, 0, st, W, rows, K, X, n, y);
    out->base = y; out->stride = (size_t)n * rows; out->ld = rows; out->n_pieces = 1; out->sk_KB = 0; out->sk_G = 0;
    return SPIRAL_OK;
}

static int launch_attention(spiral_ctx* c, spiral_kv* kv, int layer, int n, const int32_t* game_dev,
                            const int32_t* len_dev, int len_add, const float* q, __half* out_f16,
                            float* out_f32, cudaStream_t st) {
    const spiral_model_desc& d = c->d;
    AttnParams p;
    p.q = q; p.block_table = kv->table_dev; p.game = game_dev; p.ctx_len = len_dev; p.cum = meta_cum_dev(c);
    p.len_add = len_add; p.n = n; p.max_pages = kv->max_pages; p.n_pages = kv->n_pages; p.layer = layer;
    p.n_q_heads = d.n_q_heads; p.n_kv_heads = d.n_kv_heads; p.group = c->group;
    p.n_workers = c->n_sm * ATTN_WARPS;
    p.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)d.head_dim));
    p.o_part = c->o_part; p.m_part = c->m_part; p.l_part = c->l_part; p.status = c->status;
    p.item_cnt = c->attn_item_cnt; p.out_f16 = out_f16; p.out_f32 = out_f32;
    p.skip_first_load = c->attn_skip_once ? 1 : 0;
    c->attn_skip_once = false;
    const size_t smem = (size_t)ATTN_WARPS * ATTN_STAGES * (d.head_dim / 64) * 4096 + 1024;
    int rec = prof_begin(c, SPIRAL_KC_ATTN, st);
    auto attn = d.head_dim == 128 ? (kv->kv_f16 ? attn_decode_kernel<128, true> : attn_decode_kernel<128, false>)
                                  : (kv->kv_f16 ? attn_decode_kernel<64, true> : attn_decode_kernel<64, false>);
    LAUNCH(c, attn, c->n_sm, ATTN_WARPS * 32, smem, st, kv->pool_map, p);
    prof_end(c, rec, st);
    return SPIRAL_OK;
}

// Reserve a slot of the pinned metadata ring (waits for the copy that last used it).
static int meta_acquire(spiral_ctx* c, int32_t** host, StepArgs** args) {
    int s = c->meta_next;
    c->meta_next = (s + 1) % META_RING;
    if (c->meta_ev_used[s]) CU_TRY(cudaEventSynchronize(c->meta_ev[s]));
    uint8_t* base = c->meta_host + (size_t)s * c->meta_bytes;
    *host = (int32_t*)base;
    StepArgs* a = (StepArgs*)(base + meta_args_offset(c->max_batch));
    *a = StepArgs{};
    a->temperature = 1.f;
    if (args) *args = a;
    return s;
}
static int meta_upload(spiral_ctx* c, int slot, cudaStream_t st) {
    CU_TRY(cudaMemcpyAsync(c->meta_dev, c->meta_host + (size_t)slot * c->meta_bytes, c->meta_bytes,
                           cudaMemcpyHostToDevice, st));
    CU_TRY(cudaEventRecord(c->meta_ev[slot], st));
    c->meta_ev_used[slot] = true;
    return SPIRAL_OK;
}

// All layers for n batch slots whose metadata is already in ctx->meta_dev.
static int run_layers(spiral_ctx* c, spiral_kv* kv, int n, cudaStream_t st) {
    const spiral_model_desc& d = c->d;
    const int MB = c->max_batch;
    int32_t* mi = meta_i32(c);
    StepMeta meta{mi, mi + MB, mi + 2 * MB, mi + 3 * MB};
    const int qd = d.n_q_heads * d.head_dim;
    const float eps = (float)d.rms_eps;
    LAUNCH(c, embed_kernel, n, 256, 0, st, c->embed, meta_args(c), meta, kv->table_dev, kv->max_pages, kv->page_size,
           d.d_model, d.vocab, c->x, c->status);
    // persistent element-wise kernels: one CTA per SM, fewer when the batch is tiny
    const int small_grid = std::max(1, std::min(c->n_sm, (n * (d.n_q_heads + 2 * d.n_kv_heads) + 43) / 44));
    Pieces pc{};          // pieces of the previous layer's down projection, folded into the next norm
    int has = 0;
    int rc;
    for (int l = 0; l < d.n_layers; ++l) {
        LAUNCH(c, rmsnorm_kernel, n, rms_block(d.d_model), 0, st, c->x, pc, has, c->ln1[l], eps, d.d_model, c->h);
        Pieces pq;
        rc = launch_linear(c, SPIRAL_KC_QKV, c->wqkv[l], c->qkv_rows, d.d_model, c->h, n, nullptr, 0, &pq, st);
        if (rc) return rc;
        LAUNCH(c, qkv_post_kernel, small_grid, QKV_POST_THREADS, 0, st, pq, c->bqkv[l], c->q_norm[l], c->k_norm[l], eps,
               c->cos_tab, c->sin_tab, meta, kv->table_dev, kv->max_pages, kv->page_size, kv->n_pages, l, n,
               d.n_q_heads, d.n_kv_heads, d.head_dim, c->q, kv->pool, kv->kv_f16, c->status);
        rc = launch_attention(c, kv, l, n, meta.game, meta.pos, 1, c->q, c->attn_out, nullptr, st);
        if (rc) return rc;
        Pieces po;
        rc = launch_linear(c, SPIRAL_KC_O, c->wo[l], d.d_model, qd, c->attn_out, n, nullptr, 0, &po, st);
        if (rc) return rc;
        LAUNCH(c, rmsnorm_kernel, n, rms_block(d.d_model), 0, st, c->x, po, 1, c->ln2[l], eps, d.d_model, c->h);
        Pieces pg;
        rc = launch_linear(c, SPIRAL_KC_GATE_UP, c->w_gate_up[l], 2 * d.d_ff, d.d_model, c->h, n, nullptr, 0, &pg, st);
        if (rc) return rc;
        LAUNCH(c, silu_mul_kernel, small_grid, SILU_THREADS, 0, st, pg, n, d.d_ff, c->act);
        rc = launch_linear(c, SPIRAL_KC_DOWN, c->w_down[l], d.d_model, d.d_ff, c->act, n, nullptr, 0, &pc, st);
        if (rc) return rc;
        has = 1;
    }
    // final norm (folds in the last down projection)
    LAUNCH(c, rmsnorm_kernel, n, rms_block(d.d_model), 0, st, c->x, pc, has, c->final_norm, eps, d.d_model, c->h);
    return SPIRAL_OK;
}

// LM head (+ sampling, + logits for the caller) for the n rows of ctx->h, as the step's StepArgs say.
static int run_head_impl(spiral_ctx* c, int n, cudaStream_t st) {
    const spiral_model_desc& d = c->d;
    if (tc_usable(c->tc, d.vocab, d.d_model, n, false)) {
        int rc = tc_lm_head(c->tc, c->lm_head, d.vocab, d.d_model, c->h, n, meta_args(c), c->status, st, &c->launches);
        if (rc == SPIRAL_ERR_CUDA) g_cuda_error = tc_last_error();
        if (rc != SPIRAL_ERR_UNSUPPORTED) return rc;
    }
    Pieces pl;
    int rc = launch_linear_impl(c, c->lm_head, d.vocab, d.d_model, c->h, n, c->logits, 1, &pl, st);
    if (rc) return rc;
    LAUNCH(c, gumbel_argmax_kernel, n, 1024, 0, st, (const float*)c->logits, meta_args(c), d.vocab);
    return SPIRAL_OK;
}
static int run_head(spiral_ctx* c, int n, cudaStream_t st) {
    int rec = prof_begin(c, SPIRAL_KC_LM_HEAD, st);
    int rc = run_head_impl(c, n, st);
    prof_end(c, rec, st);
    return rc;
}

// Launch sequences of a decode step (each with its own recorded graph per batch size)
enum StepVariant { STEP_FUSED_SAMPLER = 0, STEP_NUCLEUS = 1, STEP_LAYERS_ONLY = 2 };

static int run_step_body(spiral_ctx* c, spiral_kv* kv, int n, int variant, cudaStream_t st) {
    const bool nucleus = variant == STEP_NUCLEUS;
    int rc2 = run_layers(c, kv, n, st);
    if (rc2 || variant == STEP_LAYERS_ONLY) return rc2;      // the caller launches the head itself
    rc2 = run_head(c, n, st);
    if (rc2 || !nucleus) return rc2;
    // the LM head left the logits in ctx->logits (StepArgs.defer_sampling): draw from the nucleus
    LAUNCH(c, nucleus_sample_kernel, n, NUCLEUS_THREADS, 0, st, (const float*)c->logits, meta_args(c), c->d.vocab);
    return SPIRAL_OK;
}

// One decode step for n slots whose metadata and StepArgs are already on their way to the device.
// The launch sequence depends on n only, so from its second use on a batch size is replayed from a
// CUDA graph recorded on the caller's stream (not on the legacy default stream, which cannot be
// captured; not while per-kernel timing is on; not inside a capture the caller has begun).
static int run_step(spiral_ctx* c, spiral_kv* kv, int n, int variant, cudaStream_t st) {
    bool graph_ok = c->use_graph && c->prof_mask == 0 && st != nullptr && st != cudaStreamLegacy;
    if (graph_ok) {
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(st, &cs) != cudaSuccess || cs != cudaStreamCaptureStatusNone) {
            cudaGetLastError();
            graph_ok = false;
        }
    }
    if (graph_ok) {
        spiral_kv::StepGraph& g = kv->graphs[n + 1024 * variant];    // one graph per batch size and launch sequence
        if (g.exec) {
            CU_TRY(cudaGraphLaunch(g.exec, st));
            c->launches += g.launches;
            return SPIRAL_OK;
        }
        if (!g.failed && ++g.uses >= 2) {
            // record: the first (eager) use has created every plan and tensor map this size needs
            const int64_t l0 = c->launches;
            CU_TRY(cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
            int rc = run_step_body(c, kv, n, variant, st);
            cudaGraph_t graph = nullptr;
            cudaError_t e = cudaStreamEndCapture(st, &graph);
            c->launches = l0;
            if (rc == SPIRAL_OK && e == cudaSuccess && graph) {
                e = cudaGraphInstantiate(&g.exec, graph, 0);
                if (e != cudaSuccess) g.exec = nullptr;
            }
            if (graph) cudaGraphDestroy(graph);
            if (!g.exec) {
                cudaGetLastError();
                g.failed = true;            // fall back to plain launches for this size
            } else {
                g.launches = g.eager_launches;      // kernels of the same sequence launched eagerly before
            }
        }
        if (g.exec) {
            CU_TRY(cudaGraphLaunch(g.exec, st));
            c->launches += g.launches;
            return SPIRAL_OK;
        }
    }
    const int64_t l0 = c->launches;
    int rc = run_step_body(c, kv, n, variant, st);
    kv->step_launches = c->launches - l0;
    kv->graphs[n + 1024 * variant].eager_launches = kv->step_launches;
    return rc;
}

static int check_ids(spiral_kv* kv, int n, const int32_t* ids) {
    kv->epoch++;
    if (kv->epoch == 0) { std::fill(kv->stamp.begin(), kv->stamp.end(), 0u); kv->epoch = 1; }
    for (int i = 0; i < n; ++i) {
        int g = ids[i];
        if (g < 0 || g >= kv->max_games || kv->stamp[g] == kv->epoch) return SPIRAL_ERR_INVALID;
        kv->stamp[g] = kv->epoch;
    }
    return SPIRAL_OK;
}

static int decode_step_impl(spiral_ctx* ctx, spiral_kv* kv, int n, const int32_t* ids, const int32_t* tok_in,
                            const float* gumbel, float temperature, float top_p, int32_t* tok_out, float* logprob,
                            float* logits_dbg, void* stream, bool tok_by_game = false, cudaEvent_t head_waits_for = nullptr) {
    if (!ctx || !kv || kv->ctx != ctx || !ids || !tok_in || !gumbel || !tok_out) return SPIRAL_ERR_INVALID;
    const bool nucleus = top_p < 1.f;
    if (nucleus && !(top_p > 0.f)) return SPIRAL_ERR_INVALID;
    if (n < 1 || n > ctx->max_batch || !(temperature > 0.f)) return SPIRAL_ERR_INVALID;
    int rc = check_ids(kv, n, ids);
    if (rc) return rc;
    int need = 0;
    for (int i = 0; i < n; ++i) {
        int len = kv->seq_len[ids[i]];
        if (len >= kv->max_ctx) return SPIRAL_ERR_INVALID;
        need += pages_missing(kv, ids[i], len + 1);
    }
    if (need > (int)kv->free_list.size()) return SPIRAL_ERR_OOM;
    cudaStream_t st = (cudaStream_t)stream;
    CU_TRY(cudaSetDevice(ctx->device));
    int32_t* mh;
    StepArgs* sa;
    int slot = meta_acquire(ctx, &mh, &sa);
    if (slot < 0) return slot;
    const int MB = ctx->max_batch;
    int* attended = ctx->scratch_len.data();
    // a failure below (an upload, a launch) must leave the games as they were: their lengths and pages are put back
    auto roll_back = [&]() {
        const int32_t* mhc = mh;
        for (int i = 0; i < n; ++i) {
            const int g = ids[i];
            kv->seq_len[g] = mhc[MB + i];
            if (mhc[2 * MB + i] >= 0) {
                const int pgi = --kv->n_game_pages[g];
                kv->page_ref[mhc[2 * MB + i]] = 0;
                kv->free_list.push_back(mhc[2 * MB + i]);
                kv->table[(size_t)g * kv->max_pages + pgi] = -1;
            }
        }
    };
    for (int i = 0; i < n; ++i) {
        int g = ids[i], len = kv->seq_len[g];
        int before = kv->n_game_pages[g];
        grow_game(kv, g, len + 1);
        mh[i] = g;
        mh[MB + i] = len;
        mh[2 * MB + i] = kv->n_game_pages[g] > before ? kv->table[(size_t)g * kv->max_pages + before] : -1;
        mh[3 * MB + i] = tok_by_game ? g : -1;      // input token of slot i: tok_in[game] or tok_in[i]
        kv->seq_len[g] = len + 1;
        attended[i] = len + 1;
    }
    attn_host_plan(attended, n, ctx->d.n_kv_heads, ctx->n_sm * ATTN_WARPS, meta_cum_host(ctx, mh));
    sa->tokens = tok_in; sa->gumbel = gumbel; sa->tok_out = tok_out; sa->logits = logits_dbg;
    sa->temperature = temperature; sa->logprob = logprob;
    if (nucleus) { sa->logits = ctx->logits; sa->defer_sampling = 1; sa->top_p = top_p; }
    rc = meta_upload(ctx, slot, st);
    if (rc) { roll_back(); return rc; }
    if (head_waits_for && !nucleus) {
        // layers first; the LM head (the first reader of the noise) starts once `head_waits_for` has fired
        rc = run_step(ctx, kv, n, STEP_LAYERS_ONLY, st);
        if (rc) { roll_back(); return rc; }
        CU_TRY(cudaStreamWaitEvent(st, head_waits_for, 0));
        return run_head(ctx, n, st);
    }
    rc = run_step(ctx, kv, n, nucleus ? STEP_NUCLEUS : STEP_FUSED_SAMPLER, st);
    if (rc) { roll_back(); return rc; }
    if (rc == SPIRAL_OK && nucleus && logits_dbg)
        CU_TRY(cudaMemcpyAsync(logits_dbg, ctx->logits, (size_t)n * ctx->d.vocab * sizeof(float), cudaMemcpyDeviceToDevice, st));
    return rc;
}

extern "C" int spiral_decode_step(spiral_ctx* ctx, spiral_kv* kv, int n, const int32_t* ids, const int32_t* tok_in,
                                  const float* gumbel, float temperature, int32_t* tok_out, float* logits_dbg,
                                  void* stream) {
    return decode_step_impl(ctx, kv, n, ids, tok_in, gumbel, temperature, 1.f, tok_out, nullptr, logits_dbg, stream);
}

extern "C" int spiral_decode_step_logprob(spiral_ctx* ctx, spiral_kv* kv, int n, const int32_t* ids,
                                          const int32_t* tok_in, const float* gumbel, float temperature,
                                          int32_t* tok_out, float* logprob, float* logits_dbg, void* stream) {
    if (!logprob) return SPIRAL_ERR_INVALID;
    return decode_step_impl(ctx, kv, n, ids, tok_in, gumbel, temperature, 1.f, tok_out, logprob, logits_dbg, stream);
}

extern "C" int spiral_decode_step_nucleus(spiral_ctx* ctx, spiral_kv* kv, int n, const int32_t* ids,
                                          const int32_t* tok_in, const float* gumbel, float temperature, float top_p,
                                          int32_t* tok_out, float* logits_dbg, void* stream) {
    if (!(top_p > 0.f) || top_p > 1.f) return SPIRAL_ERR_INVALID;
    return decode_step_impl(ctx, kv, n, ids, tok_in, gumbel, temperature, top_p, tok_out, nullptr, logits_dbg, stream);
}

extern "C" int spiral_sample_nucleus(spiral_ctx* ctx, int n, const float* logits_dev, const float* gumbel_dev,
                                     float temperature, float top_p, int32_t* tok_out_dev, void* stream) {
    if (!ctx || !logits_dev || !tok_out_dev || n < 1 || n > ctx->max_batch) return SPIRAL_ERR_INVALID;
    if (!(temperature > 0.f) || !(top_p > 0.f) || top_p > 1.f) return SPIRAL_ERR_INVALID;
    cudaStream_t st = (cudaStream_t)stream;
    CU_TRY(cudaSetDevice(ctx->device));
    int32_t* unused;
    StepArgs* sa;
    int slot = meta_acquire(ctx, &unused, &sa);
    if (slot < 0) return slot;
    sa->gumbel = gumbel_dev; sa->tok_out = tok_out_dev; sa->temperature = temperature; sa->top_p = top_p;
    int rc = meta_upload(ctx, slot, st);
    if (rc) return rc;
    LAUNCH(ctx, nucleus_sample_kernel, n, NUCLEUS_THREADS, 0, st, logits_dev, meta_args(ctx), ctx->d.vocab);
    return SPIRAL_OK;
}

// Role-conditioned advantage estimation: host arithmetic, no device work.
extern "C" int spiral_rae_update(double* baselines, int n_games, double alpha, int n_traj, const int32_t* game_of,
                                 const double* returns, double* advantages) {
    if (!baselines || n_games < 1 || n_traj < 0 || (n_traj > 0 && (!game_of || !returns || !advantages)))
        return SPIRAL_ERR_INVALID;
    if (!(alpha >= 0.0) || !(alpha <= 1.0)) return SPIRAL_ERR_INVALID;
    for (int t = 0; t < n_traj; ++t)
        if (game_of[t] < 0 || game_of[t] >= n_games) return SPIRAL_ERR_INVALID;      // nothing is changed on error
    for (int t = 0; t < n_traj; ++t)
        for (int p = 0; p < 2; ++p) {
            double& b = baselines[2 * (size_t)game_of[t] + p];
            const double r = returns[2 * (size_t)t + p];
            b = alpha * b + (1.0 - alpha) * r;
            advantages[2 * (size_t)t + p] = r - b;
        }
    return SPIRAL_OK;
}

extern "C" int spiral_decode_step_host(spiral_ctx* ctx, spiral_kv* kv, int n, const int32_t* ids,
                                       const int32_t* tok_in_host, const float* gumbel_host, float temperature,
                                       int32_t* tok_out_host, void* stream) {
    if (!ctx || !kv || !tok_in_host || !gumbel_host || !tok_out_host) return SPIRAL_ERR_INVALID;
    if (n < 1 || n > ctx->max_batch) return SPIRAL_ERR_INVALID;
    cudaStream_t st = (cudaStream_t)stream;
    CU_TRY(cudaSetDevice(ctx->device));
    CU_TRY(cudaMemcpyAsync(ctx->tok_stage, tok_in_host, (size_t)n * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    // The noise (n x vocab floats, the bulk of the input) is needed by the LM head only: it travels on a
    // stream of its own while the layers run.  The staging buffer is free: the previous call that used it
    // synchronised before it returned.
    CU_TRY(cudaMemcpyAsync(ctx->gumbel_stage, gumbel_host, (size_t)n * ctx->d.vocab * sizeof(float),
                           cudaMemcpyHostToDevice, ctx->copy_stream));
    CU_TRY(cudaEventRecord(ctx->copy_ev, ctx->copy_stream));
    int rc = decode_step_impl(ctx, kv, n, ids, ctx->tok_stage, ctx->gumbel_stage, temperature, 1.f, ctx->tokout_stage,
                              nullptr, nullptr, stream, false, ctx->copy_ev);
    if (rc) {
        cudaStreamSynchronize(ctx->copy_stream);      // the caller's buffer is not read after an error return
        return rc;
    }
    CU_TRY(cudaMemcpyAsync(tok_out_host, ctx->tokout_stage, (size_t)n * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaStreamSynchronize(st));
    return SPIRAL_OK;
}

// dst[pairs[stride + b]][:] = src[pairs[b]][:]
__global__ void gather_rows_kernel(const float* __restrict__ src, const int32_t* __restrict__ pairs, int stride,
                                   int d_model, float* __restrict__ dst) {
    grid_dependency_sync();
    const int b = blockIdx.x;
    const float4* s = reinterpret_cast<const float4*>(src + (size_t)pairs[b] * d_model);
    float4* d = reinterpret_cast<float4*>(dst + (size_t)pairs[stride + b] * d_model);
    for (int c = threadIdx.x; c < d_model / 4; c += blockDim.x) d[c] = s[c];
}

// h = RMSNorm(x) * gain over T token rows (warp per row while the row fits a warp's registers)
static int launch_rmsnorm_rows(spiral_ctx* c, const float* x, const bf16* gain, int T, __half* h, cudaStream_t st) {
    const spiral_model_desc& d = c->d;
    const float eps = (float)d.rms_eps;
    const int need = (d.d_model / 4 + 31) / 32;
    const int grid = std::max(1, std::min((T + PF_RMS_THREADS / 32 - 1) / (PF_RMS_THREADS / 32), 8 * c->n_sm));
#define PF_RMS_CASE(NV)                                                                                               \
    if (need <= NV) {                                                                                                 \
        LAUNCH(c, pf_rmsnorm_kernel<NV>, grid, PF_RMS_THREADS, 0, st, x, gain, eps, d.d_model, T, h);                 \
        return SPIRAL_OK;                                                                                             \
    }
    PF_RMS_CASE(4) PF_RMS_CASE(8) PF_RMS_CASE(12) PF_RMS_CASE(16) PF_RMS_CASE(20) PF_RMS_CASE(24) PF_RMS_CASE(28)
    PF_RMS_CASE(32)
#undef PF_RMS_CASE
    Pieces none{};
    LAUNCH(c, rmsnorm_kernel, T, rms_block(d.d_model), 0, st, const_cast<float*>(x), none, 0, gain, eps, d.d_model, h);
    return SPIRAL_OK;
}

static int prefill_ws_reserve(spiral_ctx* c, int rows) {
    PrefillWs& w = c->pf;
    if (rows <= w.cap) return SPIRAL_OK;
    CU_TRY(cudaDeviceSynchronize());
    cudaFree(w.x); cudaFree(w.y); cudaFree(w.q); cudaFree(w.h); cudaFree(w.attn); cudaFree(w.act);
    cudaFree(w.meta_dev); cudaFree(w.items_dev);
    if (w.meta_host) cudaFreeHost(w.meta_host);
    if (w.items_host) cudaFreeHost(w.items_host);
    cudaEvent_t ev = w.ev;
    w = PrefillWs{};
    w.ev = ev;
    const spiral_model_desc& d = c->d;
    const size_t R = rows, qd = (size_t)d.n_q_heads * d.head_dim;
    const int per_item = std::min(app_positions_per_item(c->group), apt_positions_per_item(c->group, 1));
    const int items_cap = (rows + per_item - 1) / per_item + c->max_batch + 1;
    const size_t meta_elems = 4 * R + 2 * (size_t)c->max_batch;
    cudaError_t e = cudaSuccess;
    auto A = [&](void** p, size_t bytes) { if (e == cudaSuccess) e = cudaMalloc(p, bytes); };
    A((void**)&w.x, R * d.d_model * sizeof(float));
    A((void**)&w.y, R * c->qkv_rows * sizeof(float));
    A((void**)&w.q, R * qd * sizeof(__half));
    A((void**)&w.h, R * d.d_model * sizeof(__half));
    A((void**)&w.attn, R * qd * sizeof(__half));
    A((void**)&w.act, R * d.d_ff * sizeof(__half));
    A((void**)&w.meta_dev, meta_elems * sizeof(int32_t));
    A((void**)&w.items_dev, (size_t)items_cap * sizeof(AppendItem));
    if (e == cudaSuccess) e = cudaMallocHost((void**)&w.meta_host, meta_elems * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMallocHost((void**)&w.items_host, (size_t)items_cap * sizeof(AppendItem));
    if (e == cudaSuccess && !w.ev) e = cudaEventCreateWithFlags(&w.ev, cudaEventDisableTiming);
    if (e != cudaSuccess) {
        g_cuda_error = std::string("append workspace: ") + cudaGetErrorString(e);
        cudaGetLastError();
        return e == cudaErrorMemoryAllocation ? SPIRAL_ERR_OOM : SPIRAL_ERR_CUDA;    // cap stays 0: freed with the context
    }
    w.cap = rows; w.items_cap = items_cap; w.meta_elems = meta_elems; w.ev_used = false;
    return SPIRAL_OK;
}

// The new tokens of all games as dense passes of up to prefill_chunk token rows: per layer four
// tensor-core GEMMs over all rows and one causal attention over the rows' games.  A game's tokens
// may be cut between two passes: the later pass finds the earlier one's keys and values in the pages.
static int prefill_dense(spiral_ctx* ctx, spiral_kv* kv, int n, const int32_t* ids, const int32_t* tokens_dev,
                         const int32_t* offsets, const std::vector<int>& start, float* last_logits, cudaStream_t st) {
    const spiral_model_desc& d = ctx->d;
    long long total = 0;
    for (int i = 0; i < n; ++i) total += offsets[i + 1] - offsets[i];
    const int chunk = (int)std::min<long long>(ctx->prefill_chunk, (total + PF_BN - 1) / PF_BN * PF_BN);
    int rc = prefill_ws_reserve(ctx, chunk);
    if (rc) return rc;
    PrefillWs& w = ctx->pf;
    const int cap = w.cap, MB = ctx->max_batch;
    const int per_item = ctx->append_attn_tc ? apt_positions_per_item(ctx->group, ctx->append_tiles)
                                             : app_positions_per_item(ctx->group);
    const int qd = d.n_q_heads * d.head_dim;
    const float eps = (float)d.rms_eps;
    int32_t* mdev = w.meta_dev;
    StepMeta meta{mdev, mdev + cap, mdev + 2 * (size_t)cap, mdev + 3 * (size_t)cap};
    const int32_t* pairs_dev = mdev + 4 * (size_t)cap;
    const float q_scale = (float)(1.4426950408889634 / std::sqrt((double)d.head_dim));
    Pieces none{};

    int gi = 0, gt = 0;
    while (gi < n) {
        if (w.ev_used) CU_TRY(cudaEventSynchronize(w.ev));       // the pinned mirrors are free again
        int32_t* mh = w.meta_host;
        int32_t* pairs = mh + 4 * (size_t)cap;
        int nt = 0, n_items = 0, n_pairs = 0;
        while (nt < chunk && gi < n) {
            const int cnt = offsets[gi + 1] - offsets[gi];
            const int take = std::min(cnt - gt, chunk - nt);
            const int pos0 = start[gi] + gt;
            for (int k = 0; k < take; ++k) {
                mh[nt + k] = ids[gi];
                mh[cap + nt + k] = pos0 + k;
                mh[2 * (size_t)cap + nt + k] = -1;
                mh[3 * (size_t)cap + nt + k] = offsets[gi] + gt + k;
            }
            // query blocks of the segment, latest (longest context) first
            for (int b = (take - 1) / per_item; b >= 0; --b) {
                AppendItem it{};
                it.game = ids[gi]; it.pos0 = pos0 + b * per_item; it.n_pos = std::min(per_item, take - b * per_item);
                it.row0 = nt + b * per_item; it.kv_len = pos0 + take;
                w.items_host[n_items++] = it;
            }
            if (gt + take == cnt) {
                pairs[n_pairs] = nt + take - 1;
                pairs[MB + n_pairs] = gi;
                ++n_pairs;
            }
            nt += take;
            gt += take;
            if (gt == cnt) { gt = 0; ++gi; }
        }
        CU_TRY(cudaMemcpyAsync(w.meta_dev, mh, w.meta_elems * sizeof(int32_t), cudaMemcpyHostToDevice, st));
        CU_TRY(cudaMemcpyAsync(w.items_dev, w.items_host, (size_t)n_items * sizeof(AppendItem), cudaMemcpyHostToDevice, st));
        CU_TRY(cudaEventRecord(w.ev, st));
        w.ev_used = true;
        int32_t* unused;
        StepArgs* sa;
        int slot = meta_acquire(ctx, &unused, &sa);
        if (slot < 0) return slot;
        sa->tokens = tokens_dev;
        sa->logits = last_logits;           // read by the LM head after the last pass only
        rc = meta_upload(ctx, slot, st);
        if (rc) return rc;

        LAUNCH(ctx, embed_kernel, nt, 256, 0, st, ctx->embed, meta_args(ctx), meta, kv->table_dev, kv->max_pages,
               kv->page_size, d.d_model, d.vocab, w.x, ctx->status);
        for (int l = 0; l < d.n_layers; ++l) {
            rc = launch_rmsnorm_rows(ctx, w.x, ctx->ln1[l], nt, w.h, st);
            if (rc) return rc;
            int rec = prof_begin(ctx, SPIRAL_KC_QKV, st);
            rc = pf_gemm<PF_EPI_STORE>(ctx->tc, ctx->wqkv[l], ctx->qkv_rows, d.d_model, w.h, nt, w.y, nullptr, ctx->status, st,
                                       &ctx->launches);
            prof_end(ctx, rec, st);
            if (rc == SPIRAL_ERR_CUDA) g_cuda_error = tc_last_error();
            if (rc) return rc;
            {
                const int qgrid = 8 * ctx->n_sm;
                if (d.head_dim == 128)
                    LAUNCH(ctx, pf_qkv_post_kernel<128>, qgrid, PF_QKV_THREADS, 0, st, (const float*)w.y, ctx->bqkv[l],
                           ctx->q_norm[l], ctx->k_norm[l], eps, ctx->cos_tab, ctx->sin_tab, meta.game, meta.pos,
                           kv->table_dev, kv->max_pages, kv->n_pages, l, nt, d.n_q_heads, d.n_kv_heads, q_scale, w.q, kv->pool,
                           ctx->status);
                else
                    LAUNCH(ctx, pf_qkv_post_kernel<64>, qgrid, PF_QKV_THREADS, 0, st, (const float*)w.y, ctx->bqkv[l],
                           ctx->q_norm[l], ctx->k_norm[l], eps, ctx->cos_tab, ctx->sin_tab, meta.game, meta.pos,
                           kv->table_dev, kv->max_pages, kv->n_pages, l, nt, d.n_q_heads, d.n_kv_heads, q_scale, w.q, kv->pool,
                           ctx->status);
            }
            {
                AppendParams ap{};
                ap.q = w.q; ap.items = w.items_dev; ap.block_table = kv->table_dev; ap.max_pages = kv->max_pages;
                ap.n_pages = kv->n_pages; ap.layer = l; ap.n_q_heads = d.n_q_heads; ap.n_kv_heads = d.n_kv_heads;
                ap.group = ctx->group;
                ap.out = w.attn; ap.status = ctx->status;
                rec = prof_begin(ctx, SPIRAL_KC_ATTN, st);
                const int tl = ctx->append_tiles;
                if (ctx->append_attn_tc && d.head_dim == 128 && tl == 2)
                    LAUNCH(ctx, (attn_append_tc_kernel<128, 2>), dim3(n_items, d.n_kv_heads), apt_threads(2), apt_smem_bytes(128, 2),
                           st, kv->pool_map16, ap);
                else if (ctx->append_attn_tc && d.head_dim == 128)
                    LAUNCH(ctx, (attn_append_tc_kernel<128, 1>), dim3(n_items, d.n_kv_heads), apt_threads(1), apt_smem_bytes(128, 1),
                           st, kv->pool_map16, ap);
                else if (ctx->append_attn_tc && tl == 2)
                    LAUNCH(ctx, (attn_append_tc_kernel<64, 2>), dim3(n_items, d.n_kv_heads), apt_threads(2), apt_smem_bytes(64, 2),
                           st, kv->pool_map16, ap);
                else if (ctx->append_attn_tc)
                    LAUNCH(ctx, (attn_append_tc_kernel<64, 1>), dim3(n_items, d.n_kv_heads), apt_threads(1), apt_smem_bytes(64, 1),
                           st, kv->pool_map16, ap);
                else if (d.head_dim == 128)
                    LAUNCH(ctx, attn_append_kernel<128>, dim3(n_items, d.n_kv_heads), APP_THREADS, app_smem_bytes(128), st,
                           kv->pool_map, ap);
                else
                    LAUNCH(ctx, attn_append_kernel<64>, dim3(n_items, d.n_kv_heads), APP_THREADS, app_smem_bytes(64), st,
                           kv->pool_map, ap);
                prof_end(ctx, rec, st);
            }
            rec = prof_begin(ctx, SPIRAL_KC_O, st);
            rc = pf_gemm<PF_EPI_ADD>(ctx->tc, ctx->wo[l], d.d_model, qd, w.attn, nt, w.x, nullptr, ctx->status, st,
                                     &ctx->launches);
            prof_end(ctx, rec, st);
            if (rc == SPIRAL_ERR_CUDA) g_cuda_error = tc_last_error();
            if (rc) return rc;
            rc = launch_rmsnorm_rows(ctx, w.x, ctx->ln2[l], nt, w.h, st);
            if (rc) return rc;
            rec = prof_begin(ctx, SPIRAL_KC_GATE_UP, st);
            rc = pf_gemm<PF_EPI_SILU>(ctx->tc, ctx->w_gate_up[l], 2 * d.d_ff, d.d_model, w.h, nt, nullptr, w.act, ctx->status,
                                      st, &ctx->launches);
            prof_end(ctx, rec, st);
            if (rc == SPIRAL_ERR_CUDA) g_cuda_error = tc_last_error();
            if (rc) return rc;
            rec = prof_begin(ctx, SPIRAL_KC_DOWN, st);
            rc = pf_gemm<PF_EPI_ADD>(ctx->tc, ctx->w_down[l], d.d_model, d.d_ff, w.act, nt, w.x, nullptr, ctx->status, st,
                                     &ctx->launches);
            prof_end(ctx, rec, st);
            if (rc == SPIRAL_ERR_CUDA) g_cuda_error = tc_last_error();
            if (rc) return rc;
        }
        if (last_logits && n_pairs > 0)     // residual rows of the games' last new tokens, in game order
            LAUNCH(ctx, gather_rows_kernel, n_pairs, 256, 0, st, (const float*)w.x, pairs_dev, MB, d.d_model, ctx->x);
    }
    if (last_logits) {
        LAUNCH(ctx, rmsnorm_kernel, n, rms_block(d.d_model), 0, st, ctx->x, none, 0, ctx->final_norm, eps, d.d_model, ctx->h);
        rc = run_head(ctx, n, st);
        if (rc) return rc;
    }
    return SPIRAL_OK;
}

extern "C" int spiral_prefill(spiral_ctx* ctx, spiral_kv* kv, int n, const int32_t* ids, const int32_t* tokens_dev,
                              const int32_t* offsets, float* last_logits, void* stream) {
    if (!ctx || !kv || kv->ctx != ctx || !ids || !tokens_dev || !offsets) return SPIRAL_ERR_INVALID;
    if (n < 1 || n > ctx->max_batch) return SPIRAL_ERR_INVALID;
    int rc = check_ids(kv, n, ids);
    if (rc) return rc;
    int need = 0;
    for (int i = 0; i < n; ++i) {
        int cnt = offsets[i + 1] - offsets[i];
        if (cnt < 1 || offsets[i] < 0) return SPIRAL_ERR_INVALID;
        if (kv->seq_len[ids[i]] + cnt > kv->max_ctx) return SPIRAL_ERR_INVALID;
        need += pages_missing(kv, ids[i], kv->seq_len[ids[i]] + cnt);
    }
    if (need > (int)kv->free_list.size()) return SPIRAL_ERR_OOM;
    cudaStream_t st = (cudaStream_t)stream;
    CU_TRY(cudaSetDevice(ctx->device));
    std::vector<int> start(n);
    // a failure below must leave the games as they were: their pages go back (the lengths are only set at the end)
    auto roll_back = [&](int rc_) {
        std::vector<int32_t> g_ids(ids, ids + n), lens(start.begin(), start.end());
        spiral_kv_truncate(kv, n, g_ids.data(), lens.data());
        return rc_;
    };
    for (int i = 0; i < n; ++i) start[i] = kv->seq_len[ids[i]];
    for (int i = 0; i < n; ++i) {
        int g = ids[i];
        grow_game(kv, g, start[i] + offsets[i + 1] - offsets[i]);
        rc = upload_table_row(kv, g, st);
        if (rc) return roll_back(rc);
    }
    {
        // more new tokens than one decode-shaped step holds: dense passes on the tensor cores
        long long total = 0;
        for (int i = 0; i < n; ++i) total += offsets[i + 1] - offsets[i];
        if (ctx->prefill_dense && ctx->pf_ready && kv->kv_f16 && total > ctx->max_batch) {
            rc = prefill_dense(ctx, kv, n, ids, tokens_dev, offsets, start, last_logits, st);
            if (rc) return roll_back(rc);
            for (int i = 0; i < n; ++i) kv->seq_len[ids[i]] = start[i] + offsets[i + 1] - offsets[i];
            return SPIRAL_OK;
        }
    }
    // Chunked: every step carries up to max_batch (game, position) slots, game after game and in
    // position order.  Slots of the same game may share a step: each slot's keys/values are cached
    // before the step's attention runs and a slot attends to positions up to its own only, so the
    // result is the causal one.
    const int MB = ctx->max_batch;
    const spiral_model_desc& d = ctx->d;
    int gi = 0, gt = 0;                       // next token to schedule: game index, offset in its new tokens
    while (gi < n) {
        int32_t* mh;
        StepArgs* sa;
        int slot = meta_acquire(ctx, &mh, &sa);
        if (slot < 0) return roll_back(slot);
        int* attended = ctx->scratch_len.data();
        int* last_of = ctx->scratch_last.data();      // slot -> game index whose last token it is, or -1
        int nt = 0;
        bool any_last = false;
        while (nt < MB && gi < n) {
            const int cnt = offsets[gi + 1] - offsets[gi];
            mh[nt] = ids[gi];
            mh[MB + nt] = start[gi] + gt;
            mh[2 * MB + nt] = -1;
            mh[3 * MB + nt] = offsets[gi] + gt;
            attended[nt] = start[gi] + gt + 1;
            last_of[nt] = gt + 1 == cnt ? gi : -1;
            any_last = any_last || gt + 1 == cnt;
            ++nt;
            if (++gt == cnt) { gt = 0; ++gi; }
        }
        attn_host_plan(attended, nt, d.n_kv_heads, ctx->n_sm * ATTN_WARPS, meta_cum_host(ctx, mh));
        sa->tokens = tokens_dev;
        sa->logits = (last_logits && any_last) ? ctx->logits : nullptr;     // no sampling: logits only
        rc = meta_upload(ctx, slot, st);
        if (rc) return roll_back(rc);
        rc = run_layers(ctx, kv, nt, st);
        if (rc) return roll_back(rc);
        if (last_logits && any_last) {
            rc = run_head(ctx, nt, st);
            if (rc) return roll_back(rc);
            for (int s = 0; s < nt; ++s)
                if (last_of[s] >= 0)
                    CU_TRY(cudaMemcpyAsync(last_logits + (size_t)last_of[s] * d.vocab, ctx->logits + (size_t)s * d.vocab,
                                           (size_t)d.vocab * sizeof(float), cudaMemcpyDeviceToDevice, st));
        }
    }
    for (int i = 0; i < n; ++i) kv->seq_len[ids[i]] = start[i] + offsets[i + 1] - offsets[i];
    return SPIRAL_OK;
}

// ------------------------------------------------------------------------------------------------
// component entry points
// ------------------------------------------------------------------------------------------------

// fold pieces into a dense fp32 matrix [n][rows]
__global__ void reduce_pieces_kernel(Pieces p, int rows, float* __restrict__ y) {
    grid_dependency_sync();
    int b = blockIdx.y;
    int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r < rows) y[(size_t)b * rows + r] = piece_sum1(p, piece_count(p, r), b, r);
}

extern "C" int spiral_linear(spiral_ctx* ctx, const void* w_dev, int rows, int k_dim, const void* x_dev, int n,
                             float* y_dev, int path, void* stream) {
    if (!ctx || !w_dev || !x_dev || !y_dev || rows < 1 || k_dim < 8 || n < 1 || n > ctx->max_batch)
        return SPIRAL_ERR_INVALID;
    if (path < 0 || path > 2 || (uintptr_t)w_dev % 16 || (uintptr_t)x_dev % 16) return SPIRAL_ERR_INVALID;
    cudaStream_t st = (cudaStream_t)stream;
    CU_TRY(cudaSetDevice(ctx->device));
    if ((size_t)n * rows > ctx->pieces_elems && path != 1) return SPIRAL_ERR_UNSUPPORTED; 
    Pieces pc;
    int rc = launch_linear(ctx, SPIRAL_KC_OTHER, (const bf16*)w_dev, rows, k_dim, (const __half*)x_dev, n, path == 1 ? y_dev : nullptr,
                           path, &pc, st);
    if (rc) return rc;
    if (pc.base != y_dev || pc.n_pieces != 1 || pc.sk_G) {
        dim3 g((rows + 255) / 256, n);
        LAUNCH(ctx, reduce_pieces_kernel, g, 256, 0, st, pc, rows, y_dev);
    }
    return SPIRAL_OK;
}

extern "C" int spiral_attention(spiral_ctx* ctx, spiral_kv* kv, int layer, int n, const int32_t* ids,
                                const int32_t* ctx_len, const float* q_dev, float* out_dev, void* stream) {
    if (!ctx || !kv || kv->ctx != ctx || !ids || !ctx_len || !q_dev || !out_dev) return SPIRAL_ERR_INVALID;
    if (n < 1 || n > ctx->max_batch || layer < 0 || layer >= ctx->d.n_layers) return SPIRAL_ERR_INVALID;
    int rc = check_ids(kv, n, ids);
    if (rc) return rc;
    for (int i = 0; i < n; ++i)
        if (ctx_len[i] < 1 || ctx_len[i] > kv->seq_len[ids[i]]) return SPIRAL_ERR_INVALID;
    cudaStream_t st = (cudaStream_t)stream;
    CU_TRY(cudaSetDevice(ctx->device));
    int32_t* mh;
    int slot = meta_acquire(ctx, &mh, nullptr);
    if (slot < 0) return slot;
    const int MB = ctx->max_batch;
    for (int i = 0; i < n; ++i) { mh[i] = ids[i]; mh[MB + i] = ctx_len[i]; mh[2 * MB + i] = -1; mh[3 * MB + i] = -1; }
    attn_host_plan(ctx_len, n, ctx->d.n_kv_heads, ctx->n_sm * ATTN_WARPS, meta_cum_host(ctx, mh));
    rc = meta_upload(ctx, slot, st);
    if (rc) return rc;
    return launch_attention(ctx, kv, layer, n, meta_i32(ctx), meta_i32(ctx) + MB, 0, q_dev, nullptr, out_dev, st);
}

extern "C" int spiral_kv_block_table(const spiral_kv* kv, int game_id, int32_t* out, int max_entries) {
    if (!kv || !out || game_id < 0 || game_id >= kv->max_games || max_entries < 0) return SPIRAL_ERR_INVALID;
    const int np = kv->n_game_pages[game_id];
    if (np > max_entries) return SPIRAL_ERR_INVALID;
    for (int i = 0; i < np; ++i) out[i] = kv->table[(size_t)game_id * kv->max_pages + i];
    return np;
}

// ------------------------------------------------------------------------------------------------
// attention without any allocation: all scratch lives in one array that is part of the library image
// ------------------------------------------------------------------------------------------------
namespace {
constexpr int NA_MAX_SEQS = SPIRAL_STATIC_ATTN_MAX_SEQS;          // sequences per call
constexpr int NA_MAX_ITEMS = SPIRAL_STATIC_ATTN_MAX_ITEMS;        // sequences x KV heads per call
constexpr int NA_MAX_CTAS = 64;                                    // grid of the attention kernel here
constexpr int NA_WORKERS = NA_MAX_CTAS * ATTN_WARPS;
constexpr int NA_PARTS = NA_WORKERS + NA_MAX_ITEMS;                // partial slots, each <= 8 heads x 128 floats
struct NoAllocScratch {
    float o_part[(size_t)NA_PARTS * 8 * 128];
    float m_part[(size_t)NA_PARTS * 8];
    float l_part[(size_t)NA_PARTS * 8];
    int item_cnt[NA_MAX_ITEMS];            // must be zero when a launch starts
    int32_t game[NA_MAX_SEQS];             // row of the caller's block table per sequence (identity)
    int32_t len[NA_MAX_SEQS];
    int32_t cum[NA_MAX_SEQS + 2];
    int status;
};
}  // namespace
// Held by every GPU that loads the library, until the process exits (about 4.3 MB).
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoAllocScratch)];

namespace {
struct NoAllocDevice {
    bool ready = false;
    NoAllocScratch* scratch = nullptr;     // device address of g_noalloc_scratch on this device
    PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
    int n_sm = 0;
};
NoAllocDevice g_noalloc[64];
std::mutex g_noalloc_mutex;        // two host threads may make a device's first call together

// once per device, with that device current: the device address of the scratch symbol (its name in
// host code is only a handle), the tensor-map encoder and the kernel's shared-memory allowance
int noalloc_setup(int device) {
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    NoAllocDevice& nd = g_noalloc[device];
    if (nd.ready) return SPIRAL_OK;
    void* ptr = nullptr;
    CU_TRY(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
    if (!ptr) { g_cuda_error = "cudaGetSymbolAddress returned no address"; return SPIRAL_ERR_CUDA; }
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    CU_TRY(cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres));
    if (!fn || qres != cudaDriverEntryPointSuccess) { g_cuda_error = "cuTensorMapEncodeTiled not available"; return SPIRAL_ERR_CUDA; }
    int major = 0;
    CU_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device));
    if (major != 10) return SPIRAL_ERR_UNSUPPORTED;
    CU_TRY(cudaDeviceGetAttribute(&nd.n_sm, cudaDevAttrMultiProcessorCount, device));
    const int attn_smem = ATTN_WARPS * ATTN_STAGES * 2 * 4096 + 1024;
    CU_TRY(cudaFuncSetAttribute(attn_decode_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_smem));
    CU_TRY(cudaFuncSetAttribute(attn_decode_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_smem));
    CU_TRY(cudaFuncSetAttribute(attn_decode_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_smem));
    CU_TRY(cudaFuncSetAttribute(attn_decode_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_smem));
    nd.scratch = (NoAllocScratch*)ptr;
    nd.encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
    nd.ready = true;
    return SPIRAL_OK;
}
}  // namespace

extern "C" int spiral_attention_static(int device, const void* pool_dev, int n_pages, int n_layers, int layer,
                                       int kv_dtype, int n_q_heads, int n_kv_heads, int head_dim,
                                       const int32_t* block_table_dev, int max_pages, int n,
                                       const int32_t* ctx_len_host, const float* q_dev, float* out_dev, void* stream) {
    if (!pool_dev || !block_table_dev || !ctx_len_host || !q_dev || !out_dev) return SPIRAL_ERR_INVALID;
    if (device < 0 || device >= 64 || n_pages < 1 || n_layers < 1 || layer < 0 || layer >= n_layers || max_pages < 1)
        return SPIRAL_ERR_INVALID;
    if (kv_dtype != SPIRAL_KV_F16 && kv_dtype != SPIRAL_KV_BF16) return SPIRAL_ERR_INVALID;
    if (head_dim != 64 && head_dim != 128) return SPIRAL_ERR_UNSUPPORTED;
    if (n_kv_heads < 1 || n_q_heads < n_kv_heads || n_q_heads % n_kv_heads != 0 || n_q_heads / n_kv_heads > 8)
        return SPIRAL_ERR_UNSUPPORTED;
    if ((uintptr_t)pool_dev % 256 != 0) return SPIRAL_ERR_INVALID;
    if (n < 1 || n > NA_MAX_SEQS || (long long)n * n_kv_heads > NA_MAX_ITEMS) {
        g_cuda_error = "spiral_attention_static: at most " + std::to_string(NA_MAX_SEQS) + " sequences and " +
                       std::to_string(NA_MAX_ITEMS) + " (sequence, KV head) pairs per call";
        return SPIRAL_ERR_TOO_LARGE;
    }
    for (int i = 0; i < n; ++i)
        if (ctx_len_host[i] < 1 || ctx_len_host[i] > max_pages * ATTN_PAGE) return SPIRAL_ERR_INVALID;
    const size_t pool_rows = (size_t)n_pages * n_layers * n_kv_heads * 2 * ATTN_PAGE;
    if (pool_rows > 0x7fffffffull) return SPIRAL_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    CU_TRY(cudaSetDevice(device));
    {
        // the schedule below is copied from host arrays of this call: a captured copy would replay stale memory
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(st, &cs) != cudaSuccess) { cudaGetLastError(); return SPIRAL_ERR_CUDA; }
        if (cs != cudaStreamCaptureStatusNone) return SPIRAL_ERR_UNSUPPORTED;
    }
    int rc = noalloc_setup(device);
    if (rc) return rc;
    NoAllocDevice& nd = g_noalloc[device];
    NoAllocScratch* sc = nd.scratch;

    TcState enc;                       // only its encoder entry is used
    enc.encode = nd.encode;
    CUtensorMap pool_map;
    rc = tc_encode(enc, &pool_map, pool_dev, (uint64_t)head_dim, pool_rows, 32, kv_dtype == SPIRAL_KV_BF16);
    if (rc) { g_cuda_error = tc_last_error(); return rc; }

    // schedule and per-sequence metadata: small host arrays, copied into the scratch in stream order
    const int grid = std::min(nd.n_sm, NA_MAX_CTAS);
    int32_t game_h[NA_MAX_SEQS], cum_h[NA_MAX_SEQS + 2];
    for (int i = 0; i < n; ++i) game_h[i] = i;
    attn_host_plan(ctx_len_host, n, n_kv_heads, grid * ATTN_WARPS, cum_h);
    CU_TRY(cudaMemcpyAsync(sc->game, game_h, (size_t)n * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    CU_TRY(cudaMemcpyAsync(sc->len, ctx_len_host, (size_t)n * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    CU_TRY(cudaMemcpyAsync(sc->cum, cum_h, (size_t)(n + 2) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    // the array keeps what the last call left: the arrival counters must start at zero (the status word is
    // kept: it holds the first error since spiral_attention_static_status last read it)
    CU_TRY(cudaMemsetAsync(sc->item_cnt, 0, sizeof(sc->item_cnt), st));

    AttnParams p;
    p.q = q_dev; p.block_table = block_table_dev; p.game = sc->game; p.ctx_len = sc->len; p.cum = sc->cum;
    p.len_add = 0; p.n = n; p.max_pages = max_pages; p.n_pages = n_pages; p.layer = layer;
    p.n_q_heads = n_q_heads; p.n_kv_heads = n_kv_heads; p.group = n_q_heads / n_kv_heads;
    p.n_workers = grid * ATTN_WARPS;
    p.scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)head_dim));
    p.o_part = sc->o_part; p.m_part = sc->m_part; p.l_part = sc->l_part; p.item_cnt = sc->item_cnt;
    p.out_f16 = nullptr; p.out_f32 = out_dev; p.status = &sc->status; p.skip_first_load = 0;
    const size_t smem = (size_t)ATTN_WARPS * ATTN_STAGES * (head_dim / 64) * 4096 + 1024;
    const bool f16 = kv_dtype == SPIRAL_KV_F16;
    auto attn = head_dim == 128 ? (f16 ? attn_decode_kernel<128, true> : attn_decode_kernel<128, false>)
                                : (f16 ? attn_decode_kernel<64, true> : attn_decode_kernel<64, false>);
    cudaError_t e = launch_kernel(false, attn, dim3(grid), dim3(ATTN_WARPS * 32), smem, st, pool_map, p);
    if (e != cudaSuccess) {
        g_cuda_error = std::string("launch of the attention kernel: ") + cudaGetErrorString(e);
        cudaGetLastError();
        return SPIRAL_ERR_CUDA;
    }
    return SPIRAL_OK;
}

// ------------------------------------------------------------------------------------------------
// read-only bandwidth probe
// ------------------------------------------------------------------------------------------------
static __device__ int g_read_ceiling_status;

extern "C" int spiral_read_ceiling(int device, const void* buf_dev, size_t bytes, int stage_bytes, int stages,
                                   int ctas_per_sm, int blocked, int tiled, int passes, void* stream, double* gbs_out) {
    if (!buf_dev || !gbs_out || device < 0 || passes < 1 || ctas_per_sm < 1 || ctas_per_sm > 8) return SPIRAL_ERR_INVALID;
    if (stage_bytes < 1024 || stage_bytes % 1024 != 0 || stages < 1 || stages > RC_MAX_STAGES) return SPIRAL_ERR_INVALID;
    if ((uintptr_t)buf_dev % 128 != 0 || bytes < (size_t)stage_bytes) return SPIRAL_ERR_INVALID;
    const size_t smem = (size_t)stages * stage_bytes + 1024;
    if (smem * ctas_per_sm > (size_t)226 * 1024) return SPIRAL_ERR_UNSUPPORTED;
    if (tiled < 0 || tiled > 2) return SPIRAL_ERR_INVALID;
    if (tiled && (stage_bytes > 32768 || (bytes >> 7) > 0x7fffffffull)) return SPIRAL_ERR_UNSUPPORTED;     // box <= 256 rows
    if (tiled == 2 && stage_bytes % 512 != 0) return SPIRAL_ERR_INVALID;
    cudaStream_t st = (cudaStream_t)stream;
    CU_TRY(cudaSetDevice(device));
    int n_sm = 0, major = 0;
    CU_TRY(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, device));
    CU_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device));
    if (major < 9) return SPIRAL_ERR_UNSUPPORTED;
    int* status_dev = nullptr;
    CU_TRY(cudaGetSymbolAddress((void**)&status_dev, g_read_ceiling_status));
    CU_TRY(cudaMemsetAsync(status_dev, 0, sizeof(int), st));
    CU_TRY(cudaFuncSetAttribute(read_ceiling_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    ReadCeilingParams p;
    p.buf = (const uint8_t*)buf_dev; p.chunks = bytes / (size_t)stage_bytes; p.stage_bytes = stage_bytes;
    if (blocked < 0 || blocked > 2) return SPIRAL_ERR_INVALID;
    p.stages = stages; p.passes = passes; p.blocked = blocked; p.status = status_dev;
    if (blocked == 2) {         // the scattered walk visits a power-of-two number of chunks
        unsigned long long c = 1;
        while (c * 2 <= p.chunks) c *= 2;
        p.chunks = c;
    }
    p.scatter_mask = p.chunks - 1;
    const int grid = (int)std::min<unsigned long long>((unsigned long long)n_sm * ctas_per_sm, p.chunks);
    p.chunks = p.chunks / grid * grid;      // every CTA reads the same number of chunks
    CUtensorMap tm;
    std::memset(&tm, 0, sizeof(tm));
    if (tiled) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        CU_TRY(cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres));
        if (!fn || qres != cudaDriverEntryPointSuccess) { g_cuda_error = "cuTensorMapEncodeTiled not available"; return SPIRAL_ERR_CUDA; }
        TcState enc;
        enc.encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
        // tiled = 1: rows of 128 bytes, one box per chunk; tiled = 2: rows of 256 bytes, a chunk = two boxes of
        // (chunk / 256) rows x 128 bytes, the left and the right halves of the rows (how a (page, head) block of keys
        // and values with 128-element rows is fetched)
        int rc = tiled == 2 ? tc_encode(enc, &tm, buf_dev, 128, (uint64_t)(bytes >> 8), (uint32_t)(stage_bytes >> 8))
                            : tc_encode(enc, &tm, buf_dev, 64, (uint64_t)(bytes >> 7), (uint32_t)(stage_bytes >> 7));
        if (rc) { g_cuda_error = tc_last_error(); return rc; }
    }
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    CU_TRY(cudaEventCreate(&e0));
    cudaError_t e = cudaEventCreate(&e1);
    if (e == cudaSuccess) e = cudaEventRecord(e0, st);
    if (e == cudaSuccess) {
        read_ceiling_kernel<<<grid, 32, smem, st>>>(tm, tiled, p);
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaEventRecord(e1, st);
    if (e == cudaSuccess) e = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    int status = 0;
    if (e == cudaSuccess) e = cudaMemcpy(&status, status_dev, sizeof(int), cudaMemcpyDeviceToHost);
    cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    if (e != cudaSuccess) {
        g_cuda_error = std::string("spiral_read_ceiling: ") + cudaGetErrorString(e);
        cudaGetLastError();
        return SPIRAL_ERR_CUDA;
    }
    if (status != STATUS_OK) return SPIRAL_ERR_TIMEOUT;
    *gbs_out = (double)p.chunks * stage_bytes * passes / (ms * 1e-3) / 1e9;
    return SPIRAL_OK;
}

extern "C" int spiral_attention_static_status(int device, int32_t* detail) {
    if (device < 0 || device >= 64) return SPIRAL_ERR_INVALID;
    CU_TRY(cudaSetDevice(device));
    int rc = noalloc_setup(device);
    if (rc) return rc;
    NoAllocScratch* sc = g_noalloc[device].scratch;
    CU_TRY(cudaDeviceSynchronize());
    int s = 0;
    CU_TRY(cudaMemcpy(&s, &sc->status, sizeof(int), cudaMemcpyDeviceToHost));
    if (detail) *detail = s;
    if (s == STATUS_OK) return SPIRAL_OK;
    CU_TRY(cudaMemset(&sc->status, 0, sizeof(int)));
    return s >= STATUS_TIMEOUT_TMA ? SPIRAL_ERR_TIMEOUT : SPIRAL_ERR_DEVICE_CHECK;
}

// ------------------------------------------------------------------------------------------------
// self-test of the bounded waits
// ------------------------------------------------------------------------------------------------
extern "C" int spiral_selftest_wait_timeout(spiral_ctx* ctx, spiral_kv* kv, int which, void* stream) {
    if (!ctx || (which != 0 && which != 1) || (which == 1 && (!kv || kv->ctx != ctx))) return SPIRAL_ERR_INVALID;
    cudaStream_t st = (cudaStream_t)stream;
    CU_TRY(cudaSetDevice(ctx->device));
    const spiral_model_desc& d = ctx->d;
    const int qd = d.n_q_heads * d.head_dim;
    const int n = std::min(ctx->max_batch, 16);
    if (which == 0 && !tc_usable(ctx->tc, d.d_model, qd, n, true)) return SPIRAL_ERR_UNSUPPORTED;
    if (which == 1 && kv->seq_len[0] < 1) return SPIRAL_ERR_INVALID;
    CU_TRY(cudaStreamSynchronize(st));
    const unsigned long long short_ns = 1000000ull, normal_ns = TMA_WAIT_NS;
    CU_TRY(cudaMemcpyToSymbol(g_wait_limit_ns, &short_ns, sizeof(short_ns)));
    int rc;
    if (which == 0) {
        // the output projection of layer 0 on whatever the activation buffer holds, without its activation loads
        Pieces pc;
        ctx->tc.skip_x_once = true;
        rc = tc_linear(ctx->tc, ctx->wo[0], d.d_model, qd, ctx->attn_out, n, ctx->pieces, ctx->pieces_elems, &pc, ctx->status, st,
                       &ctx->launches);
        ctx->tc.skip_x_once = false;
        if (rc == SPIRAL_ERR_CUDA) g_cuda_error = tc_last_error();
    } else {
        // attention of game 0 over its cached context, without the first page load of every range
        int32_t* mh;
        int slot = meta_acquire(ctx, &mh, nullptr);
        rc = slot < 0 ? slot : SPIRAL_OK;
        if (rc == SPIRAL_OK) {
            const int MB = ctx->max_batch;
            const int len = kv->seq_len[0];
            mh[0] = 0; mh[MB] = len; mh[2 * MB] = -1; mh[3 * MB] = -1;
            attn_host_plan(&len, 1, d.n_kv_heads, ctx->n_sm * ATTN_WARPS, meta_cum_host(ctx, mh));
            rc = meta_upload(ctx, slot, st);
        }
        if (rc == SPIRAL_OK) {
            ctx->attn_skip_once = true;
            rc = launch_attention(ctx, kv, 0, 1, meta_i32(ctx), meta_i32(ctx) + ctx->max_batch, 0, ctx->q, ctx->attn_out, nullptr, st);
            ctx->attn_skip_once = false;
        }
    }
    cudaError_t e = cudaStreamSynchronize(st);
    cudaMemcpyToSymbol(g_wait_limit_ns, &normal_ns, sizeof(normal_ns));
    if (rc != SPIRAL_OK) return rc;
    if (e != cudaSuccess) {
        g_cuda_error = std::string("spiral_selftest_wait_timeout: ") + cudaGetErrorString(e);
        return SPIRAL_ERR_CUDA;
    }
    return SPIRAL_OK;
}

#include "scheduler.inl"

#ifdef APT_PROBE
// probe builds only: reads and clears the append attention's phase counters
extern "C" int spiral_apt_probe_read(unsigned long long* out) {
    if (cudaDeviceSynchronize() != cudaSuccess) return -1;
    cudaMemcpyFromSymbol(out, g_apt_probe, 16 * sizeof(unsigned long long));
    unsigned long long zero[16] = {0};
    cudaMemcpyToSymbol(g_apt_probe, zero, sizeof(zero));
    return 0;
}
#endif

#ifdef ATT_PROBE
// probe builds only: copies the attention kernel's per-warp timestamps of its last launch to the host
extern "C" int spiral_att_probe_read(unsigned long long* out) {
    if (cudaDeviceSynchronize() != cudaSuccess) return -1;
    cudaMemcpyFromSymbol(out, g_att_probe, sizeof(unsigned long long) * 2048 * 8);
    return 0;
}
#endif

#ifdef TC_PROBE
// probe builds only: copies the GEMM timestamp ring to the host; returns the number of launches recorded so far
extern "C" int spiral_tc_probe_read(unsigned long long* out) {
    if (cudaDeviceSynchronize() != cudaSuccess) return -1;
    cudaMemcpyFromSymbol(out, g_tc_probe_buf, sizeof(unsigned long long) * TC_PROBE_LAUNCHES * TC_PROBE_CTAS * 8);
    return g_tc_probe_launch;
}
#endif

#ifdef SPIRAL_TRACE
// trace builds only: copies the kernel timeline ring (4 words per record) to the host, returns the
// number of records written since the last call and resets the ring
extern "C" int spiral_trace_read(unsigned long long* out, int max_records) {
    unsigned int n = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return -1;
    cudaMemcpyFromSymbol(&n, g_trace_n, sizeof(n));
    int cnt = (int)std::min<unsigned int>(n, (unsigned)std::min(max_records, 65536));
    cudaMemcpyFromSymbol(out, g_trace, (size_t)cnt * 4 * sizeof(unsigned long long));
    unsigned int zero = 0;
    cudaMemcpyToSymbol(g_trace_n, &zero, sizeof(zero));
    return cnt;
}
#endif

extern "C" int64_t spiral_launch_count(const spiral_ctx* ctx) { return ctx ? ctx->launches : 0; }

extern "C" int spiral_last_status(spiral_ctx* ctx, int32_t* detail) {
    if (!ctx) return SPIRAL_ERR_INVALID;
    CU_TRY(cudaSetDevice(ctx->device));
    CU_TRY(cudaDeviceSynchronize());
    int s = 0;
    CU_TRY(cudaMemcpy(&s, ctx->status, sizeof(int), cudaMemcpyDeviceToHost));
    if (detail) *detail = s;
    if (s == STATUS_OK) return SPIRAL_OK;
    // A kernel that gave up may have left its cross-CTA scratch half used: re-arm what must be zero between launches
    CU_TRY(cudaMemset(ctx->status, 0, sizeof(int)));
    CU_TRY(cudaMemset(ctx->attn_item_cnt, 0, (size_t)ctx->max_batch * ctx->d.n_kv_heads * sizeof(int)));
    if (ctx->tc.best) CU_TRY(cudaMemset(ctx->tc.best, 0, 256 * sizeof(unsigned long long)));
    if (ctx->tc.done) CU_TRY(cudaMemset(ctx->tc.done, 0, sizeof(unsigned int)));
    return s >= STATUS_TIMEOUT_TMA ? SPIRAL_ERR_TIMEOUT : SPIRAL_ERR_DEVICE_CHECK;
}

extern "C" void spiral_free(spiral_ctx* ctx, spiral_kv* kv) {
    if (kv) {
        cudaSetDevice(kv->ctx->device);
        cudaDeviceSynchronize();
        cudaFree(kv->table_dev);
        for (auto& g : kv->graphs)
            if (g.second.exec) cudaGraphExecDestroy(g.second.exec);
        delete kv;
    }
    free_ctx(ctx);
}
