// Bandwidth-trivial kernels of the decode step: embedding gather, RMSNorm with the residual /
// split-K reduction folded in, q/k-norm + RoPE + KV append, SwiGLU gating, Gumbel-argmax over
// stored logits, RoPE table construction and the synthetic-cache loader.
#pragma once
#include <algorithm>

#include "common.cuh"

namespace spiral {

// Stream-K bookkeeping shared by the GEMM kernel and the kernels that add its pieces up: work unit
// x of U (flattened (row tile, k block) space, KB units per tile) belongs to CTA c of G when
// floor(U c / G) <= x < floor(U (c+1) / G), i.e. c = ceil((x + 1) G / U) - 1.
__host__ __device__ inline int streamk_cta_of(long long x, int G, long long U) {
    return (int)(((x + 1) * G + U - 1) / U) - 1;
}

// Output of a skinny GEMM before reduction: partial sums ("pieces") per output element, laid out
// [piece][batch row][feature] with feature stride 1.  A stream-K GEMM (sk_G > 0) gives the 128-row
// tile t one piece per CTA whose range touches it; otherwise every element has n_pieces.
struct Pieces {
    const float* base;
    size_t stride;      // elements between pieces
    int ld;             // features per batch row
    int n_pieces;
    int sk_KB, sk_G;    // k blocks per tile and grid of the stream-K GEMM (sk_G == 0: not stream-K)
};

__device__ __forceinline__ int piece_count(const Pieces& P, int r) {
    if (P.sk_G == 0) return P.n_pieces;
    const long long U = (long long)((P.ld + 127) >> 7) * P.sk_KB;
    const long long first = (long long)(r >> 7) * P.sk_KB;
    return streamk_cta_of(first + P.sk_KB - 1, P.sk_G, U) - streamk_cta_of(first, P.sk_G, U) + 1;
}

// The kernels that consume pieces look the count of each 128-feature tile up in a shared-memory
// table filled once per CTA (the divisions above are too slow to repeat per element).
constexpr int PIECE_TABLE = 512;        // tiles covered by the table; beyond it the count is recomputed
struct PieceCounts {
    const unsigned char* tab;
    __device__ __forceinline__ int of(const Pieces& P, int r) const {
        const int t = r >> 7;
        return t < PIECE_TABLE ? (int)tab[t] : piece_count(P, r);
    }
};
// fills `tab` (PIECE_TABLE bytes of shared memory) and synchronises the CTA
__device__ __forceinline__ PieceCounts piece_counts_init(const Pieces& P, unsigned char* tab) {
    const int tiles = min(PIECE_TABLE, (P.ld + 127) >> 7);
    for (int t = threadIdx.x; t < tiles; t += blockDim.x) tab[t] = (unsigned char)piece_count(P, t << 7);
    __syncthreads();
    return PieceCounts{tab};
}

// sums of the pieces of features r..r+3 (r a multiple of 4) / of feature r; the loads of up to eight
// pieces are in flight together (the pieces sit in L2: latency, not bandwidth, is what costs)
template <int DEPTH = 8>       // pieces whose loads are in flight together
__device__ __forceinline__ float4 piece_sum4(const Pieces& P, int c, int b, int r) {
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    const float* p = P.base + (size_t)b * P.ld + r;
    for (int i = 0; i < c; i += DEPTH) {
        float4 v[DEPTH];
#pragma unroll
        for (int u = 0; u < DEPTH; ++u)
            v[u] = i + u < c ? __ldcg(reinterpret_cast<const float4*>(p + (size_t)(i + u) * P.stride))
                             : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int u = 0; u < DEPTH; ++u) { s.x += v[u].x; s.y += v[u].y; s.z += v[u].z; s.w += v[u].w; }
    }
    return s;
}
template <int DEPTH = 8>
__device__ __forceinline__ float piece_sum1(const Pieces& P, int c, int b, int r) {
    float s = 0.f;
    const float* p = P.base + (size_t)b * P.ld + r;
    for (int i = 0; i < c; i += DEPTH) {
        float v[DEPTH];
#pragma unroll
        for (int u = 0; u < DEPTH; ++u) v[u] = i + u < c ? __ldcg(p + (size_t)(i + u) * P.stride) : 0.f;
#pragma unroll
        for (int u = 0; u < DEPTH; ++u) s += v[u];
    }
    return s;
}

// Per-step metadata uploaded by the host: for batch slot i, meta[i] = game id,
// meta[cap + i] = position of the token being appended, meta[2cap + i] = page newly assigned to
// that position (or -1), meta[3cap + i] = index into the token array (prefill) or -1.
struct StepMeta {
    const int32_t* game;
    const int32_t* pos;
    const int32_t* new_page;
    const int32_t* tok_index;
};

// Per-call arguments of a step.  They travel with the step metadata (one host-to-device copy per
// step) instead of being kernel parameters, so that the launch sequence -- and a CUDA graph recorded
// from it -- depends on the batch size only.
struct StepArgs {
    const int32_t* tokens;      // input token ids (indexed by slot, or by meta.tok_index in a prefill)
    const float* gumbel;        // [n][vocab] noise, or null: no sampling
    int32_t* tok_out;           // [n] sampled tokens, or null
    float* logits;              // [n][vocab] logits wanted by the caller, or null
    float temperature;
    int32_t defer_sampling;     // 1: the LM head only writes `logits`; a later kernel (nucleus sampler) draws the tokens
    float* logprob;             // [n] log softmax(logits / T)[sampled token], or null
    float top_p;                // nucleus mass of the deferred sampler
    int32_t pad_;
};

// x[i][:] = E[token_i][:]; also publishes pages newly assigned this step into the block table.
__global__ void embed_kernel(const __nv_bfloat16* __restrict__ embed, const StepArgs* __restrict__ args,
                             StepMeta meta, int32_t* __restrict__ block_table, int max_pages, int page_size,
                             int d_model, int vocab, float* __restrict__ x, int* status) {
    TRACE_BEGIN(1);
    grid_dependency_sync();
    TRACE_WAITED();
    const int32_t* tokens = args->tokens;
    int i = blockIdx.x;
    int ti = meta.tok_index[i];
    int tok = tokens[ti >= 0 ? ti : i];
    if (tok < 0 || tok >= vocab) {
        if (threadIdx.x == 0) record_status(status, STATUS_BAD_TOKEN);
        tok = 0;
    }
    if (threadIdx.x == 0) {
        int np = meta.new_page[i];
        if (np >= 0) block_table[(size_t)meta.game[i] * max_pages + meta.pos[i] / page_size] = np;
    }
    const uint4* row = reinterpret_cast<const uint4*>(embed + (size_t)tok * d_model);
    float* out = x + (size_t)i * d_model;
    for (int c = threadIdx.x; c < d_model / 8; c += blockDim.x) {
        uint4 v = ldg_v4(row + c);
        float4 a = make_float4(bf16_lo(v.x), bf16_hi(v.x), bf16_lo(v.y), bf16_hi(v.y));
        float4 b = make_float4(bf16_lo(v.z), bf16_hi(v.z), bf16_lo(v.w), bf16_hi(v.w));
        reinterpret_cast<float4*>(out)[2 * c] = a;
        reinterpret_cast<float4*>(out)[2 * c + 1] = b;
    }
}

// x <- x + sum(pieces) (when pieces are given), then h = x * rsqrt(mean(x^2) + eps) * gain as fp16.
// One CTA per batch row, one pass: every thread keeps its (up to RMS_PER_THREAD) float4 columns of
// the row in registers between the reduction and the scaling.
constexpr int RMS_THREADS = 1024;       // upper bound; launched with d_model / 4 threads rounded up to a warp
constexpr int RMS_PER_THREAD = 2;       // d_model <= 2 * 4 * 1024 = 8192
inline int rms_block(int d_model) { return std::min(RMS_THREADS, ((d_model / 4 + 31) / 32) * 32); }
__global__ void __launch_bounds__(RMS_THREADS) rmsnorm_kernel(float* __restrict__ x, Pieces pieces, int has_pieces,
                                                              const __nv_bfloat16* __restrict__ gain, float eps,
                                                              int d_model, __half* __restrict__ h) {
    TRACE_BEGIN(2);
    // the table of piece counts depends on the launch's parameters only: it is built while the kernel ahead runs
    grid_launch_dependents();
    __shared__ unsigned char cnt_tab[PIECE_TABLE];
    PieceCounts pcnt{cnt_tab};
    if (has_pieces) pcnt = piece_counts_init(pieces, cnt_tab);
    grid_dependency_wait();
    TRACE_WAITED();
    const int b = blockIdx.x, nc = d_model >> 2;
    float* xr = x + (size_t)b * d_model;
    float4 v[RMS_PER_THREAD];
    float ss = 0.f;
#pragma unroll
    for (int k = 0; k < RMS_PER_THREAD; ++k) {
        const int c = threadIdx.x + k * blockDim.x;
        v[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < nc) {
            v[k] = reinterpret_cast<float4*>(xr)[c];
            if (has_pieces) {
                float4 p = piece_sum4(pieces, pcnt.of(pieces, 4 * c), b, 4 * c);
                v[k].x += p.x; v[k].y += p.y; v[k].z += p.z; v[k].w += p.w;
                reinterpret_cast<float4*>(xr)[c] = v[k];
            }
            ss += v[k].x * v[k].x + v[k].y * v[k].y + v[k].z * v[k].z + v[k].w * v[k].w;
        }
    }
    // the gains are fetched before the reduction's barrier, not after it: one round of latency less
    uint2 g[RMS_PER_THREAD];
#pragma unroll
    for (int k = 0; k < RMS_PER_THREAD; ++k) {
        const int c = threadIdx.x + k * blockDim.x;
        g[k] = c < nc ? *reinterpret_cast<const uint2*>(gain + 4 * c) : make_uint2(0u, 0u);
    }
    __shared__ float red[RMS_THREADS / 32];
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < RMS_THREADS / 32; ++w) tot += w < (int)(blockDim.x >> 5) ? red[w] : 0.f;
    const float inv = rsqrtf(tot / (float)d_model + eps);
    __half* hr = h + (size_t)b * d_model;
#pragma unroll
    for (int k = 0; k < RMS_PER_THREAD; ++k) {
        const int c = threadIdx.x + k * blockDim.x;
        if (c < nc) {
            uint2 o;
            o.x = pack_f16(v[k].x * inv * bf16_lo(g[k].x), v[k].y * inv * bf16_hi(g[k].x));
            o.y = pack_f16(v[k].z * inv * bf16_lo(g[k].y), v[k].w * inv * bf16_hi(g[k].y));
            *reinterpret_cast<uint2*>(hr + 4 * c) = o;
        }
    }
}

// Element offset of the K block of (layer, page, kv head) in the pool
// [layer][page][kv_head][K|V][page_size][head_dim]; the V block follows at + page_size*head_dim.
__device__ __forceinline__ size_t kv_block_offset(int layer, int page, int kvh, int n_pages, int n_kv_heads,
                                                  int page_size, int head_dim) {
    return ((((size_t)layer * n_pages + page) * n_kv_heads + kvh) * 2) * (size_t)page_size * head_dim;
}

// Half a warp per (batch slot, head): reduce the QKV pieces (+bias), per-head RMSNorm of q and k,
// rotate-half RoPE at the token's position, then q -> fp32 buffer, k and v -> their page slot
// (rounded once to the cache's 2-byte type).  Lane l of the 16 holds EPL = head_dim / 32 consecutive
// elements starting at EPL * l and their rotation partners head_dim / 2 further on, as one vector each,
// and fetches them from all (up to four) pieces at once: two rounds of loads per task instead of one
// round per element.  Persistent grid (one CTA per SM) so that the whole grid is resident at once and
// the attention kernel behind it can be launched early.
constexpr int QKV_POST_THREADS = 704;    // 22 warps: fits beside a resident GEMM CTA in the register file
constexpr int QKV_POST_MAX_PIECES = 4;   // pieces fetched together; more are added in further rounds

template <int EPL>
struct QkvVec;                            // EPL floats as one vector load / store
template <>
struct QkvVec<4> {
    float v[4];
    __device__ __forceinline__ void load_cg(const float* p) { const float4 t = __ldcg(reinterpret_cast<const float4*>(p)); v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; }
    __device__ __forceinline__ void load(const float* p) { const float4 t = __ldg(reinterpret_cast<const float4*>(p)); v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; }
    __device__ __forceinline__ void store(float* p) const { *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]); }
};
template <>
struct QkvVec<2> {
    float v[2];
    __device__ __forceinline__ void load_cg(const float* p) { const float2 t = __ldcg(reinterpret_cast<const float2*>(p)); v[0] = t.x; v[1] = t.y; }
    __device__ __forceinline__ void load(const float* p) { const float2 t = __ldg(reinterpret_cast<const float2*>(p)); v[0] = t.x; v[1] = t.y; }
    __device__ __forceinline__ void store(float* p) const { *reinterpret_cast<float2*>(p) = make_float2(v[0], v[1]); }
};

// sum over the pieces of EPL consecutive features starting at r of batch row b
template <int EPL>
__device__ __forceinline__ void qkv_piece_sum(const Pieces& P, int c, int b, int r, float (&out)[EPL]) {
#pragma unroll
    for (int e = 0; e < EPL; ++e) out[e] = 0.f;
    const float* p = P.base + (size_t)b * P.ld + r;
    for (int i = 0; i < c; i += QKV_POST_MAX_PIECES) {
        QkvVec<EPL> t[QKV_POST_MAX_PIECES];
#pragma unroll
        for (int u = 0; u < QKV_POST_MAX_PIECES; ++u) {
            if (i + u < c) t[u].load_cg(p + (size_t)(i + u) * P.stride);
            else {
#pragma unroll
                for (int e = 0; e < EPL; ++e) t[u].v[e] = 0.f;
            }
        }
#pragma unroll
        for (int u = 0; u < QKV_POST_MAX_PIECES; ++u)
#pragma unroll
            for (int e = 0; e < EPL; ++e) out[e] += t[u].v[e];
    }
}

template <int EPL>
__device__ __forceinline__ void qkv_post_task(const Pieces& pieces, const PieceCounts& pcnt, int slot, int head, int l16,
                                              const __nv_bfloat16* bias, const __nv_bfloat16* q_gain,
                                              const __nv_bfloat16* k_gain, float eps, const float* cos_tab,
                                              const float* sin_tab, const StepMeta& meta, const int32_t* block_table,
                                              int max_pages, int page_size, int n_pages, int layer, int n_q_heads,
                                              int n_kv_heads, float* q_out, uint16_t* pool, int kv_f16, int* status) {
    constexpr int HD = 32 * EPL, HALF = HD / 2;
    const int pos = meta.pos[slot];
    const int cnt = pcnt.of(pieces, head * HD);            // head_dim <= 128: a head lies in one 128-row tile
    const int i0 = EPL * l16;                              // this lane's elements i0 .. i0 + EPL - 1 and + HALF
    const bool is_q = head < n_q_heads;
    const bool is_k = !is_q && head < n_q_heads + n_kv_heads;
    QkvVec<EPL> cs, sn;                                    // rotation of this lane's pairs, fetched early
    if (is_q || is_k) {
        cs.load(cos_tab + (size_t)pos * HALF + i0);
        sn.load(sin_tab + (size_t)pos * HALF + i0);
    }
    float lo[EPL], hi[EPL];
    qkv_piece_sum<EPL>(pieces, cnt, slot, head * HD + i0, lo);
    qkv_piece_sum<EPL>(pieces, cnt, slot, head * HD + i0 + HALF, hi);
    if (bias) {
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            lo[e] += __bfloat162float(bias[head * HD + i0 + e]);
            hi[e] += __bfloat162float(bias[head * HD + i0 + e + HALF]);
        }
    }
    if (is_q || is_k) {
        const __nv_bfloat16* gain = is_q ? q_gain : k_gain;
        if (gain) {
            float ss = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) ss += lo[e] * lo[e] + hi[e] * hi[e];
            // sum over the 16 lanes of this head (the other half-warp may be on another branch)
            const unsigned hm = 0xffffu << (threadIdx.x & 16);
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) ss += __shfl_xor_sync(hm, ss, o);
            const float inv = rsqrtf(ss / (float)HD + eps);
#pragma unroll
            for (int e = 0; e < EPL; ++e) {
                lo[e] = lo[e] * inv * __bfloat162float(gain[i0 + e]);
                hi[e] = hi[e] * inv * __bfloat162float(gain[i0 + e + HALF]);
            }
        }
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            const float a = lo[e], b = hi[e];
            lo[e] = a * cs.v[e] - b * sn.v[e];
            hi[e] = b * cs.v[e] + a * sn.v[e];
        }
    }
    if (is_q) {
        float* q = q_out + ((size_t)slot * n_q_heads + head) * HD + i0;
        QkvVec<EPL> o;
#pragma unroll
        for (int e = 0; e < EPL; ++e) o.v[e] = lo[e];
        o.store(q);
#pragma unroll
        for (int e = 0; e < EPL; ++e) o.v[e] = hi[e];
        o.store(q + HALF);
        return;
    }
    const int kvh = is_k ? head - n_q_heads : head - n_q_heads - n_kv_heads;
    const int page = block_table[(size_t)meta.game[slot] * max_pages + pos / page_size];
    if (page < 0 || page >= n_pages) {
        if (l16 == 0) record_status(status, STATUS_BAD_PAGE);
        return;
    }
    const size_t off = kv_block_offset(layer, page, kvh, n_pages, n_kv_heads, page_size, HD) +
                       (is_k ? 0 : (size_t)page_size * HD) + (size_t)(pos % page_size) * HD + i0;
#pragma unroll
    for (int e = 0; e < EPL; e += 2) {
        const uint32_t wl = kv_f16 ? pack_f16(lo[e], lo[e + 1]) : pack_bf16(lo[e], lo[e + 1]);
        const uint32_t wh = kv_f16 ? pack_f16(hi[e], hi[e + 1]) : pack_bf16(hi[e], hi[e + 1]);
        *reinterpret_cast<uint32_t*>(pool + off + e) = wl;
        *reinterpret_cast<uint32_t*>(pool + off + e + HALF) = wh;
    }
}

__global__ void __maxnreg__(56) qkv_post_kernel(      // 56 registers: see QKV_POST_THREADS
    Pieces pieces, const __nv_bfloat16* __restrict__ bias, const __nv_bfloat16* __restrict__ q_gain,
    const __nv_bfloat16* __restrict__ k_gain, float eps, const float* __restrict__ cos_tab,
    const float* __restrict__ sin_tab, StepMeta meta, const int32_t* __restrict__ block_table, int max_pages,
    int page_size, int n_pages, int layer, int n, int n_q_heads, int n_kv_heads, int head_dim,
    float* __restrict__ q_out, uint16_t* __restrict__ pool, int kv_f16, int* status) {
    TRACE_BEGIN(3);
    grid_launch_dependents();
    __shared__ unsigned char cnt_tab[PIECE_TABLE];
    const PieceCounts pcnt = piece_counts_init(pieces, cnt_tab);       // (parameters only: before the wait)
    grid_dependency_wait();
    TRACE_WAITED();
    const int l16 = threadIdx.x & 15;
    const int n_heads = n_q_heads + 2 * n_kv_heads;
    const int total = n * n_heads;
    const int groups = (gridDim.x * blockDim.x) >> 4;
    for (int task = (blockIdx.x * blockDim.x + threadIdx.x) >> 4; task < total; task += groups) {
        const int slot = task / n_heads, head = task - slot * n_heads;
        if (head_dim == 128)
            qkv_post_task<4>(pieces, pcnt, slot, head, l16, bias, q_gain, k_gain, eps, cos_tab, sin_tab, meta, block_table,
                             max_pages, page_size, n_pages, layer, n_q_heads, n_kv_heads, q_out, pool, kv_f16, status);
        else
            qkv_post_task<2>(pieces, pcnt, slot, head, l16, bias, q_gain, k_gain, eps, cos_tab, sin_tab, meta, block_table,
                             max_pages, page_size, n_pages, layer, n_q_heads, n_kv_heads, q_out, pool, kv_f16, status);
    }
}

// act[b][i] = SiLU(gate_i) * up_i with gate_i / up_i the reduced features 2i / 2i+1 of the
// gate-up GEMM (rows interleaved), written as fp16.
// Persistent grid (one CTA per SM): a small grid is resident at once, so the kernel after this one
// can be launched early and prefetch its weights.
constexpr int SILU_THREADS = 1024;
__global__ void __launch_bounds__(SILU_THREADS) silu_mul_kernel(Pieces pieces, int n, int d_ff,
                                                                __half* __restrict__ act) {
    TRACE_BEGIN(4);
    grid_launch_dependents();
    __shared__ unsigned char cnt_tab[PIECE_TABLE];
    const PieceCounts pcnt = piece_counts_init(pieces, cnt_tab);       // (parameters only: before the wait)
    const int per_row = d_ff >> 1;                       // task c of a row: features 4c..4c+3 -> act 2c, 2c+1
    const int total = n * per_row;                       // <= 256 * 2^22: fits
    const int stride = gridDim.x * blockDim.x;
    constexpr int T = 5;        // tasks per pass: all their loads are issued before any is used
    // where the first pass's tasks lie (divisions, table look-ups) is worked out before the wait as well
    const int base0 = blockIdx.x * blockDim.x + threadIdx.x;
    int row[T], col[T], cnt[T];
#pragma unroll
    for (int u = 0; u < T; ++u) {
        const int idx = base0 + u * stride;
        row[u] = idx / per_row;
        col[u] = idx - row[u] * per_row;
        cnt[u] = idx < total ? pcnt.of(pieces, 4 * col[u]) : 0;
    }
    grid_dependency_wait();
    TRACE_WAITED();
    for (int base = base0; base < total; base += T * stride) {
        float4 v[T];
        if (base != base0) {
#pragma unroll
            for (int u = 0; u < T; ++u) {
                const int idx = base + u * stride;
                row[u] = idx / per_row;
                col[u] = idx - row[u] * per_row;
                cnt[u] = idx < total ? pcnt.of(pieces, 4 * col[u]) : 0;
            }
        }
#pragma unroll
        for (int u = 0; u < T; ++u) {
            v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (base + u * stride < total) v[u] = piece_sum4<2>(pieces, cnt[u], row[u], 4 * col[u]);
        }
#pragma unroll
        for (int u = 0; u < T; ++u) {
            if (base + u * stride < total) {
                const float a0 = v[u].x / (1.f + expf(-v[u].x)) * v[u].y;
                const float a1 = v[u].z / (1.f + expf(-v[u].z)) * v[u].w;
                *reinterpret_cast<uint32_t*>(act + (size_t)row[u] * d_ff + 2 * col[u]) = pack_f16(a0, a1);
            }
        }
    }
}

// 64-bit key whose unsigned order is (score ascending, index descending): max key = best score,
// lowest index among equals.  NaN scores rank below everything.
__device__ __forceinline__ unsigned long long argmax_key(float z, int idx) {
    uint32_t u = __float_as_uint(z);
    if (z != z) u = 0u; else u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    return ((unsigned long long)u << 32) | (uint32_t)(0xffffffffu - (uint32_t)idx);
}
__device__ __forceinline__ int argmax_key_index(unsigned long long k) {
    return (int)(0xffffffffu - (uint32_t)(k & 0xffffffffull));
}

// token[b] = argmax_v( logits[b][v] / T + gumbel[b][v] ) from logits stored in memory (the path of
// batches too small for the tensor cores); also hands the logits to the caller when asked.
__global__ void __launch_bounds__(1024) gumbel_argmax_kernel(const float* __restrict__ logits,
                                                            const StepArgs* __restrict__ args, int vocab) {
    TRACE_BEGIN(5);
    grid_dependency_sync();
    TRACE_WAITED();
    StepArgs sa = *args;
    if (sa.defer_sampling) { sa.tok_out = nullptr; sa.gumbel = nullptr; sa.logprob = nullptr; }
    int b = blockIdx.x;
    const float* lg = logits + (size_t)b * vocab;
    if (sa.logits && sa.logits != logits)
        for (int v = threadIdx.x; v < vocab; v += blockDim.x) sa.logits[(size_t)b * vocab + v] = lg[v];
    if (!sa.tok_out) return;
    const float* gm = sa.gumbel ? sa.gumbel + (size_t)b * vocab : nullptr;
    unsigned long long best = 0ull;
    for (int v = threadIdx.x; v < vocab; v += blockDim.x) {
        float z = __fadd_rn(__fdiv_rn(lg[v], sa.temperature), gm ? gm[v] : 0.f);
        unsigned long long k = argmax_key(z, v);
        best = k > best ? k : best;
    }
    __shared__ unsigned long long red[32];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
        best = other > best ? other : best;
    }
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = best;
    __syncthreads();
    if (threadIdx.x < 32) {
        best = red[threadIdx.x];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
            best = other > best ? other : best;
        }
        if (threadIdx.x == 0) { sa.tok_out[b] = argmax_key_index(best); red[0] = best; }
    }
    if (!sa.logprob) return;
    // log-probability of the drawn token: logit/T - logsumexp(logits/T), two block reductions
    __syncthreads();
    const int tok = argmax_key_index(red[0]);
    __shared__ float redf[32];
    float mx = -INFINITY;
    for (int v = threadIdx.x; v < vocab; v += blockDim.x) mx = fmaxf(mx, __fdiv_rn(lg[v], sa.temperature));
    mx = warp_max(mx);
    if ((threadIdx.x & 31) == 0) redf[threadIdx.x >> 5] = mx;
    __syncthreads();
    mx = redf[0];
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w) mx = fmaxf(mx, redf[w]);
    __syncthreads();
    float sum = 0.f;
    for (int v = threadIdx.x; v < vocab; v += blockDim.x) sum += expf(__fdiv_rn(lg[v], sa.temperature) - mx);
    sum = warp_sum(sum);
    if ((threadIdx.x & 31) == 0) redf[threadIdx.x >> 5] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        float tot = 0.f;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) tot += redf[w];
        sa.logprob[b] = __fdiv_rn(lg[tok], sa.temperature) - (mx + logf(tot));
    }
}


// Nucleus (top-p) sampling from stored logits with caller-supplied Gumbel noise -- the evaluation
// setting of the paper (temperature 0.6, top-p 0.95).  With z_v = logit_v / T and p = softmax(z),
// token v is kept when the probability mass of the tokens strictly more probable than v is below
// top_p (the smallest most-probable-first prefix reaching top_p, plus whatever ties its last
// member; the most probable token is always kept), and the draw is argmax over the kept tokens of
// z_v + gumbel_v, lowest index on ties -- a sample from the renormalised kept distribution.
// The kept set is {v : key(z_v) >= K} for a threshold K on the order-preserving 32-bit keys of z,
// found by a 16-way search: 8-9 passes over the row, each with 15 trial thresholds and a deterministic
// block reduction of the mass above every one of them.  One CTA per batch row.
__device__ __forceinline__ uint32_t ordered_key(float z) {          // larger float <=> larger key; NaN -> 0
    const uint32_t u = __float_as_uint(z);
    return z != z ? 0u : ((u & 0x80000000u) ? ~u : (u | 0x80000000u));
}
constexpr int NUCLEUS_THREADS = 1024;
constexpr int NUCLEUS_WAYS = 15;         // thresholds tried per pass of the search
__device__ __forceinline__ float nucleus_block_sum(float v, float* red) {     // fixed order: same result every run
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < NUCLEUS_THREADS / 32; ++w) tot += red[w];
    return tot;
}
__global__ void __launch_bounds__(NUCLEUS_THREADS) nucleus_sample_kernel(const float* __restrict__ logits,
                                                                         const StepArgs* __restrict__ args, int vocab) {
    grid_dependency_sync();
    const StepArgs sa = *args;
    __shared__ float red[NUCLEUS_THREADS / 32];
    __shared__ unsigned long long redk[NUCLEUS_THREADS / 32];
    const int b = blockIdx.x;
    const float* lg = logits + (size_t)b * vocab;
    const float T = sa.temperature;
    float mx = -INFINITY;
    for (int v = threadIdx.x; v < vocab; v += NUCLEUS_THREADS) mx = fmaxf(mx, __fdiv_rn(lg[v], T));
    mx = warp_max(mx);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
    __syncthreads();
    mx = red[0];
#pragma unroll
    for (int w = 1; w < NUCLEUS_THREADS / 32; ++w) mx = fmaxf(mx, red[w]);
    float part = 0.f;
    for (int v = threadIdx.x; v < vocab; v += NUCLEUS_THREADS) {
        const float z = __fdiv_rn(lg[v], T);
        if (z == z) part += __expf(z - mx);
    }
    const float total = nucleus_block_sum(part, red);
    const float target = sa.top_p * total;
    const uint32_t key_max = ordered_key(mx);
    uint32_t lo = 0u, hi = key_max;                  // the mass above key_max is zero: always below a positive target
    if (!(sa.top_p < 1.f)) hi = 0u;                  // top_p >= 1: keep everything
    // Each pass over the row tries 15 thresholds that cut [lo, hi] into 16 parts (four bits of the key per
    // pass: 8-9 passes instead of 32), each threshold with its own fixed-order sum.
    __shared__ float part_sm[NUCLEUS_THREADS / 32][NUCLEUS_WAYS];
    __shared__ float tot_sm[NUCLEUS_WAYS];
    while (lo < hi) {
        const uint32_t span = hi - lo;
        uint32_t cut[NUCLEUS_WAYS];
        float above[NUCLEUS_WAYS];
#pragma unroll
        for (int k = 0; k < NUCLEUS_WAYS; ++k) {
            cut[k] = lo + (uint32_t)(((unsigned long long)span * (unsigned)(k + 1)) >> 4);       // in [lo, hi)
            above[k] = 0.f;
        }
        for (int v = threadIdx.x; v < vocab; v += NUCLEUS_THREADS) {
            const float z = __fdiv_rn(lg[v], T);
            const uint32_t key = ordered_key(z);
            if (key > lo) {                         // below every threshold otherwise (and NaN: key 0)
                const float e = __expf(z - mx);
#pragma unroll
                for (int k = 0; k < NUCLEUS_WAYS; ++k) above[k] += key > cut[k] ? e : 0.f;
            }
        }
#pragma unroll
        for (int k = 0; k < NUCLEUS_WAYS; ++k) above[k] = warp_sum(above[k]);
        __syncthreads();
        if ((threadIdx.x & 31) == 0) {
#pragma unroll
            for (int k = 0; k < NUCLEUS_WAYS; ++k) part_sm[threadIdx.x >> 5][k] = above[k];
        }
        __syncthreads();
        if (threadIdx.x < NUCLEUS_WAYS) {
            float tot = 0.f;
            for (int w = 0; w < NUCLEUS_THREADS / 32; ++w) tot += part_sm[w][threadIdx.x];
            tot_sm[threadIdx.x] = tot;
        }
        __syncthreads();
        // the smallest threshold whose mass above is below the target becomes the new upper end
        int first = NUCLEUS_WAYS;
#pragma unroll
        for (int k = NUCLEUS_WAYS - 1; k >= 0; --k)
            if (tot_sm[k] < target) first = k;
        if (first < NUCLEUS_WAYS) hi = cut[first];
        if (first > 0) lo = cut[first - 1] + 1u;
    }
    const uint32_t K = lo;
    const float* gm = sa.gumbel ? sa.gumbel + (size_t)b * vocab : nullptr;
    unsigned long long best = 0ull;
    for (int v = threadIdx.x; v < vocab; v += NUCLEUS_THREADS) {
        const float z = __fdiv_rn(lg[v], T);
        if (ordered_key(z) >= K && z == z) {
            const unsigned long long k = argmax_key(__fadd_rn(z, gm ? gm[v] : 0.f), v);
            best = k > best ? k : best;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
        best = other > best ? other : best;
    }
    __syncthreads();
    if ((threadIdx.x & 31) == 0) redk[threadIdx.x >> 5] = best;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < NUCLEUS_THREADS / 32; ++w) best = redk[w] > best ? redk[w] : best;
        if (sa.tok_out) sa.tok_out[b] = argmax_key_index(best);
    }
}

// cos/sin of pos * theta^(-2i/head_dim), evaluated in fp64 and stored as fp32 [max_ctx][head_dim/2].
__global__ void rope_table_kernel(double theta, int head_dim, int max_ctx, float* __restrict__ cos_tab,
                                  float* __restrict__ sin_tab) {
    int half = head_dim / 2;
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)max_ctx * half) return;
    int pos = (int)(idx / half), i = (int)(idx % half);
    double phi = (double)pos * pow(theta, -2.0 * (double)i / (double)head_dim);
    cos_tab[idx] = (float)cos(phi);
    sin_tab[idx] = (float)sin(phi);
}

// Scatter 2-byte [n_tokens][kv_head][head_dim] K and V of one game and layer into its pages.
__global__ void kv_load_kernel(const uint16_t* __restrict__ k_src, const uint16_t* __restrict__ v_src,
                               int n_tokens, const int32_t* __restrict__ block_row, int page_size, int n_pages,
                               int layer, int n_kv_heads, int head_dim, uint16_t* __restrict__ pool) {
    int t = blockIdx.x;
    int page = block_row[t / page_size];
    int w = n_kv_heads * head_dim;
    for (int e = threadIdx.x; e < w; e += blockDim.x) {
        int kvh = e / head_dim, i = e % head_dim;
        size_t off = kv_block_offset(layer, page, kvh, n_pages, n_kv_heads, page_size, head_dim) +
                     (size_t)(t % page_size) * head_dim + i;
        pool[off] = k_src[(size_t)t * w + e];
        pool[off + (size_t)page_size * head_dim] = v_src[(size_t)t * w + e];
    }
}

}  // namespace spiral
