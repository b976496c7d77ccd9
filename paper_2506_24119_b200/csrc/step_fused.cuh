// One persistent cooperative kernel for a whole decode step (one CTA per SM, 8 warps).
//
// The step is a chain of short dependent phases (per layer: RMSNorm, QKV GEMM, q/k-norm + RoPE +
// append, attention, O GEMM, RMSNorm, gate/up GEMM, SwiGLU gate, down GEMM).  As separate kernels
// every phase boundary costs a grid drain, a launch and a pipeline fill; here the boundary is a grid
// barrier (one atomic per CTA + a bounded spin) and the TMA producer already requests the first
// ring-full of the NEXT GEMM's weights while the current GEMM drains and the element-wise phase in
// between runs.  The phases reuse the device code of the stand-alone kernels:
//   warps 0 / 1     TMA producer / tcgen05 MMA issuer (one lane each) in GEMM phases
//   warps 4..7      GEMM epilogue (TMEM lane quadrant = warp % 4)
//   all 8 warps     attention (per-warp TMA rings, attn_warp_work) and the element-wise phases
// mbarrier phases, TMEM and the shared-memory arena persist across phases; the attention rings and
// the GEMM stages share the arena (their phases never overlap; a weight prefetch is only made when
// no attention phase lies before the GEMM it is for).
// Data written by other CTAs in an earlier phase is read through L2 (ld.global.cg / TMA): L1 is not
// coherent across SMs within a kernel.  Every wait is bounded; a timeout records a status code and
// lets every CTA run through the remaining barriers without working.
#pragma once
#include "attn_decode.cuh"
#include "common.cuh"
#include "gemm_tc.cuh"
#include "kernels_small.cuh"
#include "tma.cuh"

namespace spiral {

constexpr int FS_THREADS = 256;
constexpr int FS_ROW_CHUNKS = 8;          // float4 columns per thread of one residual row: d_model <= 8192
constexpr int STATUS_TIMEOUT_GRID = 19;   // bounded wait at a grid barrier ran out

struct FsLayer {                          // per layer, in device memory (64-byte aligned records)
    CUtensorMap w_qkv, w_o, w_gate_up, w_down;
    const __nv_bfloat16 *ln1, *ln2, *bqkv, *q_gain, *k_gain;
    const void* pad[3];
};

struct FsParams {
    int n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ff, vocab, qkv_rows;
    float eps;
    int n, N, stages;
    const FsLayer* layers;
    const __nv_bfloat16 *embed, *final_norm;
    float* x;
    __half *h, *attn_out, *act;
    float *q, *pieces;
    const float *cos_tab, *sin_tab;
    StepMeta meta;
    const int32_t* cum;
    const StepArgs* args;
    int32_t* block_table;
    int max_pages, page_size, n_pages, kv_f16;
    uint16_t* pool;
    float *o_part, *m_part, *l_part;
    int* item_cnt;
    float scale_log2;
    unsigned long long* best;
    unsigned int* done;
    unsigned int* grid_bar;     // zero at launch
    int* status;
};

struct FsShared {
    uint64_t full_bar[TC_MAX_STAGES], empty_bar[TC_MAX_STAGES], acc_full[2], acc_empty[2];
    uint64_t attn_bar[ATTN_WARPS][ATTN_STAGES];
    uint32_t tmem_base;
    int abort_flag, last_flag;
    int cum[ATTN_MAX_SLOTS + 2], len[ATTN_MAX_SLOTS], game[ATTN_MAX_SLOTS];
    unsigned char cnt_tab[PIECE_TABLE];
    float red[FS_THREADS / 32];
    unsigned long long run[4][256];
};

// per-thread pipeline positions that outlive a phase
struct FsRole {
    uint32_t g_it = 0;       // GEMM stages requested (producer lane) / consumed (MMA lane) so far
    uint32_t acc_it = 0;     // accumulators produced (MMA lane) / drained (epilogue threads) so far
    uint32_t pre = 0;        // stages of the next GEMM whose weight tile is already requested (producer lane)
    uint32_t ring_it = 0;    // attention stages this warp has consumed so far
    uint32_t epoch = 0;      // grid barriers passed
};

__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Grid-wide barrier.  Before it, every thread makes its global and shared-memory writes visible to
// the asynchronous proxy (TMA reads of activations / cache rows, TMA writes into reused stages).
__device__ __forceinline__ void fs_grid_sync(const FsParams& p, FsShared& sh, FsRole& r) {
#ifdef SPIRAL_TRACE
    const unsigned long long t_arrive = trace_now();
#endif
    asm volatile("fence.proxy.async;" ::: "memory");
    __syncthreads();
    ++r.epoch;
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(p.grid_bar, 1u);
        const unsigned int target = r.epoch * gridDim.x;
        unsigned long long t0 = global_ns();
        for (uint32_t spin = 1; ld_acquire_u32(p.grid_bar) < target; ++spin) {
            if ((spin & 63u) == 0) {
                if (*(volatile int*)p.status != STATUS_OK) { sh.abort_flag = 1; break; }
                if (global_ns() - t0 > TMA_WAIT_NS) {
                    record_status(p.status, STATUS_TIMEOUT_GRID);
                    sh.abort_flag = 1;
                    break;
                }
            }
        }
        __threadfence();
#ifdef SPIRAL_TRACE
        if (blockIdx.x == 0 || (r.epoch >= 12 && r.epoch <= 21)) {   // (barrier, arrival, CTA-wide sync, opening) of CTA 0; all CTAs for one layer
            unsigned int i = atomicAdd(&g_trace_n, 1u) & 65535u;
            g_trace[4 * i] = (1000ull + r.epoch) * 1000ull + blockIdx.x; g_trace[4 * i + 1] = t_arrive; g_trace[4 * i + 2] = t0;
            g_trace[4 * i + 3] = trace_now();
        }
#endif
    }
    __syncthreads();
}

#ifdef SPIRAL_TRACE
__device__ __forceinline__ void fs_stamp(const FsRole& r, int what) {
    if (blockIdx.x == 0 && r.epoch >= 11 && r.epoch <= 20) {
        unsigned int i = atomicAdd(&g_trace_n, 1u) & 65535u;
        g_trace[4 * i] = 5000000ull + (unsigned long long)r.epoch * 10ull + what; g_trace[4 * i + 1] = trace_now();
        g_trace[4 * i + 2] = 0; g_trace[4 * i + 3] = 0;
    }
}
#define FS_STAMP(r, what) fs_stamp(r, what)
#else
#define FS_STAMP(r, what) do { } while (0)
#endif

__device__ __forceinline__ int fs_gemm_grid(int tiles, int KB, bool whole) {
    const long long U = whole ? tiles : (long long)tiles * KB;
    const long long g = whole ? U : (U / 4 > 1 ? U / 4 : 1);
    return (int)(g < (long long)gridDim.x ? g : (long long)gridDim.x);
}

// One GEMM phase: y = X W^T as stream-K pieces (MODE 0) or LM head + Gumbel-argmax (MODE 1).
// next_w (may be null): weights of the GEMM phase that follows with only element-wise work in
// between; its first ring-full of weight tiles is requested as stages fall free.
template <int MODE>
__device__ __noinline__ void fs_gemm(const FsParams& p, FsShared& sh, FsRole& role, uint32_t arena,
                                        const CUtensorMap* tmW, const CUtensorMap* tmX, int rows, int K,
                                        const CUtensorMap* next_w, int next_rows, int next_K, bool next_whole,
                                        Pieces* out_desc) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    FsRole r = role;                      // positions in registers for the duration of the phase
    // plain locals: stores through float pointers below must not make the compiler re-read the
    // parameter block after every store
    const int S = p.stages, N = p.N, n = p.n;
    float* const pieces = p.pieces;
    int* const status = p.status;
    const uint32_t stage_bytes = TC_W_BYTES + (uint32_t)N * 128u;
    const int tiles = (rows + TC_BM - 1) / TC_BM, KB = (K + TC_BK - 1) / TC_BK;
    const bool whole = MODE == 1;
    const int G = fs_gemm_grid(tiles, KB, whole);
    const bool active = (int)blockIdx.x < G && !sh.abort_flag;
    volatile int* abort_flag = &sh.abort_flag;
    if (out_desc) {
        out_desc->base = pieces; out_desc->stride = (size_t)n * rows; out_desc->ld = rows;
        out_desc->n_pieces = 1; out_desc->sk_KB = KB; out_desc->sk_G = G;
    }
    if (warp == 0) {
        if (lane == 0) {
            const uint64_t pol_w = l2_policy_evict_first(), pol_x = l2_policy_evict_last();
            bool ok = true;
            if (active) {
                TcSchedule sched(tiles, KB, whole, blockIdx.x, G);
                TcSeg sg;
                uint32_t k = 0;
                while (ok && sched.next(sg)) {
                    for (int kb = sg.kb0; kb < sg.kb1; ++kb, ++k, ++r.g_it) {
                        const uint32_t s = r.g_it % S, ph = (r.g_it / S) & 1u;
                        const uint32_t fb = smem_u32(&sh.full_bar[s]);
                        const uint32_t dst = arena + s * stage_bytes;
                        if (k >= r.pre) {
                            if (!mbar_wait(smem_u32(&sh.empty_bar[s]), ph ^ 1u, abort_flag, status, STATUS_TIMEOUT_MMA)) {
                                ok = false;
                                break;
                            }
                            mbar_expect_tx(fb, stage_bytes);
                            tma_load_2d(dst, tmW, 0, (sg.tile * KB + kb) * TC_BM, fb, pol_w);
                        }
                        tma_load_2d(dst + TC_W_BYTES, tmX, kb * TC_BK, 0, fb, pol_x);
                    }
                }
            }
            r.pre = 0;
            FS_STAMP(role, 1);
            if (ok && next_w && !sh.abort_flag) {
                const int nt = (next_rows + TC_BM - 1) / TC_BM, nKB = (next_K + TC_BK - 1) / TC_BK;
                const int nG = fs_gemm_grid(nt, nKB, next_whole);
                if ((int)blockIdx.x < nG) {
                    TcSchedule ns(nt, nKB, next_whole, blockIdx.x, nG);
                    TcSeg sg;
                    uint32_t it2 = r.g_it;
                    while (ok && r.pre < (uint32_t)S && ns.next(sg)) {
                        for (int kb = sg.kb0; kb < sg.kb1 && r.pre < (uint32_t)S; ++kb, ++it2, ++r.pre) {
                            const uint32_t s = it2 % S, ph = (it2 / S) & 1u;
                            if (!mbar_wait(smem_u32(&sh.empty_bar[s]), ph ^ 1u, abort_flag, status, STATUS_TIMEOUT_MMA)) {
                                ok = false;
                                break;
                            }
                            const uint32_t fb = smem_u32(&sh.full_bar[s]);
                            mbar_expect_tx(fb, stage_bytes);
                            tma_load_2d(arena + s * stage_bytes, next_w, 0, (sg.tile * nKB + kb) * TC_BM, fb, pol_w);
                        }
                    }
                }
            }
            FS_STAMP(role, 2);
        }
    } else if (warp == 1) {
        if (lane == 0 && active) {
            const uint32_t idesc = tc_idesc_f16(N);
            bool ok = true;
            TcSchedule sched(tiles, KB, whole, blockIdx.x, G);
            TcSeg sg;
            for (; ok && sched.next(sg); ++r.acc_it) {
                const uint32_t a = r.acc_it & 1u, aph = (r.acc_it >> 1) & 1u;
                if (!mbar_wait(smem_u32(&sh.acc_empty[a]), aph ^ 1u, abort_flag, status, STATUS_TIMEOUT_EPI)) break;
                tc_fence_after();
                const uint32_t d_tmem = sh.tmem_base + a * (uint32_t)N;
                for (int kb = sg.kb0; kb < sg.kb1; ++kb, ++r.g_it) {
                    const uint32_t s = r.g_it % S, ph = (r.g_it / S) & 1u;
                    if (!mbar_wait(smem_u32(&sh.full_bar[s]), ph, abort_flag, status, STATUS_TIMEOUT_TMA)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t w_addr = arena + s * stage_bytes;
                    const uint64_t da = smem_desc_sw128(w_addr), db = smem_desc_sw128(w_addr + TC_W_BYTES);
#pragma unroll
                    for (int k = 0; k < TC_BK / 16; ++k)
                        tc_mma_f16(d_tmem, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc,
                                   (kb > sg.kb0 || k > 0) ? 1u : 0u);
                    tc_commit(smem_u32(&sh.empty_bar[s]));
                }
                if (ok) tc_commit(smem_u32(&sh.acc_full[a]));
                else break;
            }
            FS_STAMP(role, 3);
        }
    } else if (warp >= 4) {
        const int q = warp & 3;
        StepArgs sa{};
        if (MODE == 1) {
            sa = *p.args;
            for (int i = threadIdx.x - 128; i < 4 * 256; i += 128) sh.run[i >> 8][i & 255] = 0ull;
            asm volatile("bar.sync 1, 128;" ::: "memory");
        }
        const bool unit_t = sa.temperature == 1.0f;
        if (active) {
            TcSchedule sched(tiles, KB, whole, blockIdx.x, G);
            TcSeg sg;
            for (; sched.next(sg); ++r.acc_it) {
                const uint32_t a = r.acc_it & 1u, aph = (r.acc_it >> 1) & 1u;
                if (!mbar_wait(smem_u32(&sh.acc_full[a]), aph, abort_flag, status, STATUS_TIMEOUT_MMA)) break;
                tc_fence_after();
                if (threadIdx.x == 128) FS_STAMP(role, 5);
                const int row = sg.tile * TC_BM + q * 32 + lane;
                const bool row_ok = row < rows;
                const uint32_t t_addr = sh.tmem_base + ((uint32_t)(q * 32) << 16) + a * (uint32_t)N;
                if (MODE == 0) {
                    float* dst = pieces + (size_t)sg.piece * ((size_t)n * rows) + row;
                    for (int c0 = 0; c0 < N; c0 += 64) {
                        uint32_t v[4][16];
#pragma unroll
                        for (int h = 0; h < 4; ++h)
                            if (c0 + 16 * h < N) tmem_ld16_async(t_addr + (uint32_t)(c0 + 16 * h), v[h]);
                        tmem_ld_wait();
                        if (threadIdx.x == 128) FS_STAMP(role, 6);
                        if (row_ok) {
#pragma unroll
                            for (int h = 0; h < 4; ++h)
#pragma unroll
                                for (int j = 0; j < 16; ++j)
                                    if (c0 + 16 * h + j < n)
                                        dst[(size_t)(c0 + 16 * h + j) * rows] = __uint_as_float(v[h][j]);
                        }
                        if (threadIdx.x == 128) FS_STAMP(role, 7);
                    }
                } else {
                    for (int c0 = 0; c0 < N; c0 += 64) {
                        uint32_t v[4][16];
                        float gm[4][16];
#pragma unroll
                        for (int h = 0; h < 4; ++h)
                            if (c0 + 16 * h < N) tmem_ld16_async(t_addr + (uint32_t)(c0 + 16 * h), v[h]);
#pragma unroll
                        for (int h = 0; h < 4; ++h)
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                const int b = c0 + 16 * h + j;
                                gm[h][j] = (sa.gumbel && row_ok && b < n) ? __ldg(sa.gumbel + (size_t)b * rows + row) : 0.f;
                            }
                        tmem_ld_wait();
#pragma unroll
                        for (int h = 0; h < 4; ++h) {
                            if (c0 + 16 * h >= N) break;
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                const int b = c0 + 16 * h + j;
                                const bool ok = row_ok && b < n;
                                const float lg = __uint_as_float(v[h][j]);
                                if (ok && sa.logits) sa.logits[(size_t)b * rows + row] = lg;
                                const float z = __fadd_rn(unit_t ? lg : __fdiv_rn(lg, sa.temperature), gm[h][j]);
                                uint32_t u = __float_as_uint(z);
                                u = (!ok || z != z) ? 0u : ((u & 0x80000000u) ? ~u : (u | 0x80000000u));
                                const uint32_t m = __reduce_max_sync(0xffffffffu, u);
                                const uint32_t who = __ballot_sync(0xffffffffu, u == m);
                                if (lane == (b & 31) && b < n) {
                                    const int vbest = sg.tile * TC_BM + q * 32 + (__ffs(who) - 1);
                                    const unsigned long long key =
                                        ((unsigned long long)m << 32) | (uint32_t)(0xffffffffu - (uint32_t)vbest);
                                    if (key > sh.run[q][b]) sh.run[q][b] = key;
                                }
                            }
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&sh.acc_empty[a]));
                if (threadIdx.x == 128) FS_STAMP(role, 4);
            }
        }
        if (MODE == 1) {
            // fold the four warps, publish with an order-independent 64-bit max; the CTA that finishes
            // last turns the keys into tokens and re-arms the scratch for the next launch
            asm volatile("bar.sync 1, 128;" ::: "memory");
            const int t = threadIdx.x - 128;
            if ((int)blockIdx.x < G) {
                for (int b = t; b < n; b += 128) {
                    unsigned long long k = sh.run[0][b];
#pragma unroll
                    for (int w = 1; w < 4; ++w) k = sh.run[w][b] > k ? sh.run[w][b] : k;
                    if (k) atomicMax(p.best + b, k);
                }
                __threadfence();
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (t == 0) sh.last_flag = (atomicAdd(p.done, 1u) == (unsigned)G - 1u) ? 1 : 0;
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (sh.last_flag) {
                    __threadfence();
                    for (int b = t; b < n; b += 128) {
                        const unsigned long long k = atomicExch(p.best + b, 0ull);
                        if (sa.tok_out) sa.tok_out[b] = (int)(0xffffffffu - (uint32_t)(k & 0xffffffffull));
                    }
                    if (t == 0) *p.done = 0u;
                }
            }
        }
    }
    role = r;
}

// ---- element-wise phases (all threads of all CTAs) ----------------------------------------------

// residual row b lives on CTA b % gridDim.x in every phase that touches x
__device__ __noinline__ void fs_embed(const FsParams& params) {
    const FsParams p = params;        // a local copy: stores below must not force re-reads of the parameter block
    const int32_t* tokens = p.args->tokens;
    for (int i = blockIdx.x; i < p.n; i += gridDim.x) {
        const int ti = p.meta.tok_index[i];
        int tok = tokens[ti >= 0 ? ti : i];
        if (tok < 0 || tok >= p.vocab) {
            if (threadIdx.x == 0) record_status(p.status, STATUS_BAD_TOKEN);
            tok = 0;
        }
        if (threadIdx.x == 0) {
            const int np = p.meta.new_page[i];
            if (np >= 0) p.block_table[(size_t)p.meta.game[i] * p.max_pages + p.meta.pos[i] / p.page_size] = np;
        }
        const uint4* row = reinterpret_cast<const uint4*>(p.embed + (size_t)tok * p.d_model);
        float* out = p.x + (size_t)i * p.d_model;
        for (int c = threadIdx.x; c < p.d_model / 8; c += blockDim.x) {
            const uint4 v = ldg_v4(row + c);
            reinterpret_cast<float4*>(out)[2 * c] = make_float4(bf16_lo(v.x), bf16_hi(v.x), bf16_lo(v.y), bf16_hi(v.y));
            reinterpret_cast<float4*>(out)[2 * c + 1] = make_float4(bf16_lo(v.z), bf16_hi(v.z), bf16_lo(v.w), bf16_hi(v.w));
        }
    }
}

__device__ __noinline__ void fs_rmsnorm(const FsParams& params, FsShared& sh, const Pieces& pieces, bool has_pieces,
                                           const __nv_bfloat16* gain) {
    const FsParams p = params;        // a local copy: stores below must not force re-reads of the parameter block
    if ((int)blockIdx.x >= p.n) return;                   // CTA-uniform
    PieceCounts pcnt{sh.cnt_tab};
    if (has_pieces) pcnt = piece_counts_init(pieces, sh.cnt_tab);
    const int nc = p.d_model >> 2;
    for (int b = blockIdx.x; b < p.n; b += gridDim.x) {
        float* xr = p.x + (size_t)b * p.d_model;
        float4 v[FS_ROW_CHUNKS];
        float ss = 0.f;
#pragma unroll
        for (int k = 0; k < FS_ROW_CHUNKS; ++k) {
            const int c = threadIdx.x + k * FS_THREADS;
            v[k] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (c < nc) {
                v[k] = reinterpret_cast<float4*>(xr)[c];
                if (has_pieces) {
                    const float4 a = piece_sum4(pieces, pcnt.of(pieces, 4 * c), b, 4 * c);
                    v[k].x += a.x; v[k].y += a.y; v[k].z += a.z; v[k].w += a.w;
                    reinterpret_cast<float4*>(xr)[c] = v[k];
                }
                ss += v[k].x * v[k].x + v[k].y * v[k].y + v[k].z * v[k].z + v[k].w * v[k].w;
            }
        }
        ss = warp_sum(ss);
        __syncthreads();                                  // sh.red free again (previous row)
        if ((threadIdx.x & 31) == 0) sh.red[threadIdx.x >> 5] = ss;
        __syncthreads();
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < FS_THREADS / 32; ++w) tot += sh.red[w];
        const float inv = rsqrtf(tot / (float)p.d_model + p.eps);
        __half* hr = p.h + (size_t)b * p.d_model;
#pragma unroll
        for (int k = 0; k < FS_ROW_CHUNKS; ++k) {
            const int c = threadIdx.x + k * FS_THREADS;
            if (c < nc) {
                const uint2 g = *reinterpret_cast<const uint2*>(gain + 4 * c);
                uint2 o;
                o.x = pack_f16(v[k].x * inv * bf16_lo(g.x), v[k].y * inv * bf16_hi(g.x));
                o.y = pack_f16(v[k].z * inv * bf16_lo(g.y), v[k].w * inv * bf16_hi(g.y));
                *reinterpret_cast<uint2*>(hr + 4 * c) = o;
            }
        }
    }
}

__device__ __noinline__ void fs_qkv_post(const FsParams& params, FsShared& sh, const Pieces& pieces, const FsLayer& L,
                                            int layer) {
    const FsParams p = params;        // a local copy: stores below must not force re-reads of the parameter block
    const PieceCounts pcnt = piece_counts_init(pieces, sh.cnt_tab);
    const int l16 = threadIdx.x & 15;
    const int n_heads = p.n_q_heads + 2 * p.n_kv_heads;
    const int head_dim = p.head_dim, half = head_dim >> 1, np = head_dim >> 5;
    const int total = p.n * n_heads;
    const int groups = (gridDim.x * blockDim.x) >> 4;
    for (int task = (blockIdx.x * blockDim.x + threadIdx.x) >> 4; task < total; task += groups) {
        const int slot = task / n_heads, head = task - slot * n_heads;
        const int pos = p.meta.pos[slot];
        const int cnt = pcnt.of(pieces, head * head_dim);
        const bool is_q = head < p.n_q_heads;
        const bool is_k = !is_q && head < p.n_q_heads + p.n_kv_heads;
        float cs[4], sn[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            cs[j] = 1.f; sn[j] = 0.f;
            if (j < np && (is_q || is_k)) {
                cs[j] = p.cos_tab[(size_t)pos * half + l16 + 16 * j];
                sn[j] = p.sin_tab[(size_t)pos * half + l16 + 16 * j];
            }
        }
        float lo[4], hi[4];
        float ss = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            lo[j] = 0.f; hi[j] = 0.f;
            if (j < np) {
                const int r0 = head * head_dim + l16 + 16 * j, r1 = r0 + half;
                lo[j] = piece_sum1<4>(pieces, cnt, slot, r0);
                hi[j] = piece_sum1<4>(pieces, cnt, slot, r1);
                if (L.bqkv) {
                    lo[j] += __bfloat162float(L.bqkv[r0]);
                    hi[j] += __bfloat162float(L.bqkv[r1]);
                }
                ss += lo[j] * lo[j] + hi[j] * hi[j];
            }
        }
        if (is_q || is_k) {
            const __nv_bfloat16* gain = is_q ? L.q_gain : L.k_gain;
            if (gain) {
                const unsigned hm = 0xffffu << (threadIdx.x & 16);
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) ss += __shfl_xor_sync(hm, ss, o);
                const float inv = rsqrtf(ss / (float)head_dim + p.eps);
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (j < np) {
                        const int i = l16 + 16 * j;
                        lo[j] = lo[j] * inv * __bfloat162float(gain[i]);
                        hi[j] = hi[j] * inv * __bfloat162float(gain[i + half]);
                    }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (j < np) {
                    const float a = lo[j], b = hi[j];
                    lo[j] = a * cs[j] - b * sn[j];
                    hi[j] = b * cs[j] + a * sn[j];
                }
        }
        if (is_q) {
            float* q = p.q + ((size_t)slot * p.n_q_heads + head) * head_dim;
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (j < np) {
                    q[l16 + 16 * j] = lo[j];
                    q[l16 + 16 * j + half] = hi[j];
                }
            continue;
        }
        const int kvh = is_k ? head - p.n_q_heads : head - p.n_q_heads - p.n_kv_heads;
        const int page = __ldcg(p.block_table + (size_t)p.meta.game[slot] * p.max_pages + pos / p.page_size);
        if (page < 0 || page >= p.n_pages) {
            if (l16 == 0) record_status(p.status, STATUS_BAD_PAGE);
            continue;
        }
        const size_t off = kv_block_offset(layer, page, kvh, p.n_pages, p.n_kv_heads, p.page_size, head_dim) +
                           (is_k ? 0 : (size_t)p.page_size * head_dim) + (size_t)(pos % p.page_size) * head_dim;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (j < np) {
                p.pool[off + l16 + 16 * j] = (uint16_t)(p.kv_f16 ? float_to_f16_bits(lo[j]) : float_to_bf16_bits(lo[j]));
                p.pool[off + l16 + 16 * j + half] = (uint16_t)(p.kv_f16 ? float_to_f16_bits(hi[j]) : float_to_bf16_bits(hi[j]));
            }
    }
}

__device__ __noinline__ void fs_silu(const FsParams& params, FsShared& sh, const Pieces& pieces) {
    const FsParams p = params;        // a local copy: stores below must not force re-reads of the parameter block
    const PieceCounts pcnt = piece_counts_init(pieces, sh.cnt_tab);
    const int per_row = p.d_ff >> 1;
    const int total = p.n * per_row;
    const int stride = gridDim.x * blockDim.x;
    constexpr int T = 6;
    for (int base = blockIdx.x * blockDim.x + threadIdx.x; base < total; base += T * stride) {
        float4 v[T];
        int row[T], col[T];
#pragma unroll
        for (int u = 0; u < T; ++u) {
            const int idx = base + u * stride;
            row[u] = idx / per_row;
            col[u] = idx - row[u] * per_row;
            v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (idx < total) v[u] = piece_sum4<2>(pieces, pcnt.of(pieces, 4 * col[u]), row[u], 4 * col[u]);
        }
#pragma unroll
        for (int u = 0; u < T; ++u) {
            if (base + u * stride < total) {
                const float a0 = v[u].x / (1.f + expf(-v[u].x)) * v[u].y;
                const float a1 = v[u].z / (1.f + expf(-v[u].z)) * v[u].w;
                *reinterpret_cast<uint32_t*>(p.act + (size_t)row[u] * p.d_ff + 2 * col[u]) = pack_f16(a0, a1);
            }
        }
    }
}

template <int HD, bool F16>
__device__ __noinline__ uint32_t fs_attention(const CUtensorMap* tmPool, const AttnParams& params, FsShared& sh, uint32_t ring,
                                              uint32_t ring_it) {
    const int warp = threadIdx.x >> 5;
    const AttnParams ap = params;         // local copy (see above)
    return attn_warp_work<HD, F16>(tmPool, ap, sh.cum, sh.len, sh.game, sh.attn_bar[warp], ring, ring_it, &sh.abort_flag,
                                   warp * (int)gridDim.x + (int)blockIdx.x);
}

// ---- the kernel ----------------------------------------------------------------------------------
template <int HD, bool F16>
__global__ void __launch_bounds__(FS_THREADS, 1) decode_step_fused_kernel(
    const __grid_constant__ CUtensorMap tmH, const __grid_constant__ CUtensorMap tmAttn,
    const __grid_constant__ CUtensorMap tmAct, const __grid_constant__ CUtensorMap tmPool,
    const __grid_constant__ CUtensorMap tmLm, FsParams p) {
    extern __shared__ uint8_t fs_smem_raw[];
    __shared__ __align__(16) FsShared sh;
    const int warp = threadIdx.x >> 5;
    const uint32_t arena = (smem_u32(fs_smem_raw) + 1023u) & ~1023u;
    FsRole r;

    if (threadIdx.x == 0) {
        for (int s = 0; s < TC_MAX_STAGES; ++s) { mbar_init(smem_u32(&sh.full_bar[s]), 1); mbar_init(smem_u32(&sh.empty_bar[s]), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(smem_u32(&sh.acc_full[a]), 1); mbar_init(smem_u32(&sh.acc_empty[a]), 4); }
        for (int w = 0; w < ATTN_WARPS; ++w)
            for (int s = 0; s < ATTN_STAGES; ++s) mbar_init(smem_u32(&sh.attn_bar[w][s]), 1);
        sh.abort_flag = 0;
        sh.last_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = threadIdx.x; i <= p.n + 1; i += blockDim.x) {
        sh.cum[i] = p.cum[i];
        if (i < p.n) { sh.len[i] = p.meta.pos[i] + 1; sh.game[i] = p.meta.game[i]; }
    }
    if (warp == 1) tmem_alloc(smem_u32(&sh.tmem_base), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    fs_embed(p);
    fs_grid_sync(p, sh, r);

    AttnParams ap;
    ap.q = p.q; ap.block_table = p.block_table; ap.game = nullptr; ap.ctx_len = nullptr; ap.cum = nullptr;
    ap.len_add = 0; ap.n = p.n; ap.max_pages = p.max_pages; ap.n_pages = p.n_pages; ap.layer = 0;
    ap.n_q_heads = p.n_q_heads; ap.n_kv_heads = p.n_kv_heads; ap.group = p.n_q_heads / p.n_kv_heads;
    ap.n_workers = gridDim.x * ATTN_WARPS; ap.scale_log2 = p.scale_log2;
    ap.o_part = p.o_part; ap.m_part = p.m_part; ap.l_part = p.l_part; ap.item_cnt = p.item_cnt;
    ap.out_f16 = p.attn_out; ap.out_f32 = nullptr; ap.nx = TcNext{0, 0, 0, 0}; ap.status = p.status;
    const uint32_t attn_ring = arena + (uint32_t)(warp * ATTN_STAGES * (HD / 64) * 4096);
    const int qd = p.n_q_heads * p.head_dim;

    Pieces pc{};
    bool has = false;
    for (int l = 0; l < p.n_layers; ++l) {
        const FsLayer& L = p.layers[l];
        if (!sh.abort_flag) fs_rmsnorm(p, sh, pc, has, L.ln1);
        fs_grid_sync(p, sh, r);
        Pieces pq;
        fs_gemm<0>(p, sh, r, arena, &L.w_qkv, &tmH, p.qkv_rows, p.d_model, nullptr, 0, 0, false, &pq);
        fs_grid_sync(p, sh, r);
        if (!sh.abort_flag) fs_qkv_post(p, sh, pq, L, l);
        fs_grid_sync(p, sh, r);
        if (!sh.abort_flag) {
            ap.layer = l;
            r.ring_it = fs_attention<HD, F16>(&tmPool, ap, sh, attn_ring, r.ring_it);
        }
        fs_grid_sync(p, sh, r);
        Pieces po;
        fs_gemm<0>(p, sh, r, arena, &L.w_o, &tmAttn, p.d_model, qd, &L.w_gate_up, 2 * p.d_ff, p.d_model, false, &po);
        fs_grid_sync(p, sh, r);
        if (!sh.abort_flag) fs_rmsnorm(p, sh, po, true, L.ln2);
        fs_grid_sync(p, sh, r);
        Pieces pg;
        fs_gemm<0>(p, sh, r, arena, &L.w_gate_up, &tmH, 2 * p.d_ff, p.d_model, &L.w_down, p.d_model, p.d_ff, false, &pg);
        fs_grid_sync(p, sh, r);
        if (!sh.abort_flag) fs_silu(p, sh, pg);
        fs_grid_sync(p, sh, r);
        const bool last = l + 1 == p.n_layers;
        fs_gemm<0>(p, sh, r, arena, &L.w_down, &tmAct, p.d_model, p.d_ff, last ? &tmLm : &p.layers[l + 1].w_qkv,
                   last ? p.vocab : p.qkv_rows, p.d_model, last, &pc);
        has = true;
        fs_grid_sync(p, sh, r);
    }
    if (!sh.abort_flag) fs_rmsnorm(p, sh, pc, has, p.final_norm);
    fs_grid_sync(p, sh, r);
    fs_gemm<1>(p, sh, r, arena, &tmLm, &tmH, p.vocab, p.d_model, nullptr, 0, 0, false, nullptr);

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(sh.tmem_base, 512);
}

// ---- host side -----------------------------------------------------------------------------------
template <typename K>
inline cudaError_t fs_launch_kernel(K kernel, int grid, size_t smem, cudaStream_t st, const CUtensorMap& a,
                                    const CUtensorMap& b, const CUtensorMap& c, const CUtensorMap& d, const CUtensorMap& e,
                                    const FsParams& p) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(FS_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;     // all CTAs resident together, or the launch fails
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, a, b, c, d, e, p);
}

inline size_t fs_smem_bytes(int N, int head_dim, int* stages) {
    size_t gemm_smem;
    tc_launch_shape(N, stages, &gemm_smem);
    const size_t attn = (size_t)ATTN_WARPS * ATTN_STAGES * (head_dim / 64) * 4096 + 1024;
    return std::max(gemm_smem, attn);
}

}  // namespace spiral
