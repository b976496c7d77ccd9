// Bandwidth-trivial kernels of the decode step: embedding gather, RMSNorm with the residual /
// split-K reduction folded in, q/k-norm + RoPE + KV append, SwiGLU gating, Gumbel-argmax over
// stored logits, RoPE table construction and the synthetic-cache loader.
#pragma once
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

// sums of the pieces of features r..r+3 (r a multiple of 4) / of feature r, with the loads of four
// pieces in flight at a time
__device__ __forceinline__ float4 piece_sum4(const Pieces& P, int b, int r) {
    const int c = piece_count(P, r);
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    const float* p = P.base + (size_t)b * P.ld + r;
    int i = 0;
    for (; i + 4 <= c; i += 4) {
        float4 v0 = *reinterpret_cast<const float4*>(p + (size_t)i * P.stride);
        float4 v1 = *reinterpret_cast<const float4*>(p + (size_t)(i + 1) * P.stride);
        float4 v2 = *reinterpret_cast<const float4*>(p + (size_t)(i + 2) * P.stride);
        float4 v3 = *reinterpret_cast<const float4*>(p + (size_t)(i + 3) * P.stride);
        s.x += v0.x; s.y += v0.y; s.z += v0.z; s.w += v0.w;
        s.x += v1.x; s.y += v1.y; s.z += v1.z; s.w += v1.w;
        s.x += v2.x; s.y += v2.y; s.z += v2.z; s.w += v2.w;
        s.x += v3.x; s.y += v3.y; s.z += v3.z; s.w += v3.w;
    }
    for (; i < c; ++i) {
        float4 v = *reinterpret_cast<const float4*>(p + (size_t)i * P.stride);
        s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
    }
    return s;
}
__device__ __forceinline__ float piece_sum1(const Pieces& P, int b, int r) {
    const int c = piece_count(P, r);
    float s = 0.f;
    const float* p = P.base + (size_t)b * P.ld + r;
    int i = 0;
    for (; i + 4 <= c; i += 4) {
        float v0 = p[(size_t)i * P.stride], v1 = p[(size_t)(i + 1) * P.stride];
        float v2 = p[(size_t)(i + 2) * P.stride], v3 = p[(size_t)(i + 3) * P.stride];
        s += v0; s += v1; s += v2; s += v3;
    }
    for (; i < c; ++i) s += p[(size_t)i * P.stride];
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
    int32_t reserved;
};

// x[i][:] = E[token_i][:]; also publishes pages newly assigned this step into the block table.
__global__ void embed_kernel(const __nv_bfloat16* __restrict__ embed, const StepArgs* __restrict__ args,
                             StepMeta meta, int32_t* __restrict__ block_table, int max_pages, int page_size,
                             int d_model, int vocab, float* __restrict__ x, int* status) {
    grid_dependency_sync();
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
constexpr int RMS_THREADS = 512;
constexpr int RMS_PER_THREAD = 4;       // d_model <= 4 * 4 * 512 = 8192
__global__ void __launch_bounds__(RMS_THREADS) rmsnorm_kernel(float* __restrict__ x, Pieces pieces, int has_pieces,
                                                              const __nv_bfloat16* __restrict__ gain, float eps,
                                                              int d_model, __half* __restrict__ h) {
    grid_dependency_sync();
    const int b = blockIdx.x, nc = d_model >> 2;
    float* xr = x + (size_t)b * d_model;
    float4 v[RMS_PER_THREAD];
    float ss = 0.f;
#pragma unroll
    for (int k = 0; k < RMS_PER_THREAD; ++k) {
        const int c = threadIdx.x + k * RMS_THREADS;
        v[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < nc) {
            v[k] = reinterpret_cast<float4*>(xr)[c];
            if (has_pieces) {
                float4 p = piece_sum4(pieces, b, 4 * c);
                v[k].x += p.x; v[k].y += p.y; v[k].z += p.z; v[k].w += p.w;
                reinterpret_cast<float4*>(xr)[c] = v[k];
            }
            ss += v[k].x * v[k].x + v[k].y * v[k].y + v[k].z * v[k].z + v[k].w * v[k].w;
        }
    }
    __shared__ float red[RMS_THREADS / 32];
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < RMS_THREADS / 32; ++w) tot += red[w];
    const float inv = rsqrtf(tot / (float)d_model + eps);
    __half* hr = h + (size_t)b * d_model;
#pragma unroll
    for (int k = 0; k < RMS_PER_THREAD; ++k) {
        const int c = threadIdx.x + k * RMS_THREADS;
        if (c < nc) {
            uint2 g = *reinterpret_cast<const uint2*>(gain + 4 * c);
            uint2 o;
            o.x = pack_f16(v[k].x * inv * bf16_lo(g.x), v[k].y * inv * bf16_hi(g.x));
            o.y = pack_f16(v[k].z * inv * bf16_lo(g.y), v[k].w * inv * bf16_hi(g.y));
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

// One warp per (batch slot, head): reduce the QKV pieces (+bias), per-head RMSNorm of q and k,
// rotate-half RoPE at the token's position, then q -> fp32 buffer, k and v -> their page slot
// (rounded once to the cache's 2-byte type).
__global__ void __launch_bounds__(128) qkv_post_kernel(
    Pieces pieces, const __nv_bfloat16* __restrict__ bias, const __nv_bfloat16* __restrict__ q_gain,
    const __nv_bfloat16* __restrict__ k_gain, float eps, const float* __restrict__ cos_tab,
    const float* __restrict__ sin_tab, StepMeta meta, const int32_t* __restrict__ block_table, int max_pages,
    int page_size, int n_pages, int layer, int n_q_heads, int n_kv_heads, int head_dim,
    float* __restrict__ q_out, uint16_t* __restrict__ pool, int kv_f16, int* status) {
    grid_dependency_sync();
    int slot = blockIdx.x;
    int head = blockIdx.y * 4 + (threadIdx.x >> 5);
    int lane = threadIdx.x & 31;
    int n_heads = n_q_heads + 2 * n_kv_heads;
    if (head >= n_heads) return;
    int half = head_dim >> 1;
    int np = head_dim >> 6;                 // rotation pairs per lane (1 or 2)
    int pos = meta.pos[slot];
    float lo[2], hi[2];
    float ss = 0.f;
    for (int j = 0; j < np; ++j) {
        int i = lane + 32 * j;
        int r0 = head * head_dim + i, r1 = r0 + half;
        lo[j] = piece_sum1(pieces, slot, r0);
        hi[j] = piece_sum1(pieces, slot, r1);
        if (bias) {
            lo[j] += __bfloat162float(bias[r0]);
            hi[j] += __bfloat162float(bias[r1]);
        }
        ss += lo[j] * lo[j] + hi[j] * hi[j];
    }
    bool is_q = head < n_q_heads;
    bool is_k = !is_q && head < n_q_heads + n_kv_heads;
    if (is_q || is_k) {
        const __nv_bfloat16* gain = is_q ? q_gain : k_gain;
        if (gain) {
            ss = warp_sum(ss);
            float inv = rsqrtf(ss / (float)head_dim + eps);
            for (int j = 0; j < np; ++j) {
                int i = lane + 32 * j;
                lo[j] = lo[j] * inv * __bfloat162float(gain[i]);
                hi[j] = hi[j] * inv * __bfloat162float(gain[i + half]);
            }
        }
        for (int j = 0; j < np; ++j) {
            int i = lane + 32 * j;
            float c = cos_tab[(size_t)pos * half + i], s = sin_tab[(size_t)pos * half + i];
            float a = lo[j], b = hi[j];
            lo[j] = a * c - b * s;
            hi[j] = b * c + a * s;
        }
    }
    if (is_q) {
        float* q = q_out + ((size_t)slot * n_q_heads + head) * head_dim;
        for (int j = 0; j < np; ++j) {
            q[lane + 32 * j] = lo[j];
            q[lane + 32 * j + half] = hi[j];
        }
        return;
    }
    int kvh = is_k ? head - n_q_heads : head - n_q_heads - n_kv_heads;
    int page = block_table[(size_t)meta.game[slot] * max_pages + pos / page_size];
    if (page < 0 || page >= n_pages) {
        if (lane == 0) record_status(status, STATUS_BAD_PAGE);
        return;
    }
    size_t off = kv_block_offset(layer, page, kvh, n_pages, n_kv_heads, page_size, head_dim) +
                 (is_k ? 0 : (size_t)page_size * head_dim) + (size_t)(pos % page_size) * head_dim;
    for (int j = 0; j < np; ++j) {
        pool[off + lane + 32 * j] = (uint16_t)(kv_f16 ? float_to_f16_bits(lo[j]) : float_to_bf16_bits(lo[j]));
        pool[off + lane + 32 * j + half] = (uint16_t)(kv_f16 ? float_to_f16_bits(hi[j]) : float_to_bf16_bits(hi[j]));
    }
}

// act[b][i] = SiLU(gate_i) * up_i with gate_i / up_i the reduced features 2i / 2i+1 of the
// gate-up GEMM (rows interleaved), written as fp16.
__global__ void silu_mul_kernel(Pieces pieces, int d_ff, __half* __restrict__ act) {
    grid_dependency_sync();
    int b = blockIdx.y;
    int c = blockIdx.x * blockDim.x + threadIdx.x;      // handles features 4c..4c+3 -> act 2c, 2c+1
    if (c >= d_ff / 2) return;
    float4 v = piece_sum4(pieces, b, 4 * c);
    float a0 = v.x / (1.f + expf(-v.x)) * v.y;
    float a1 = v.z / (1.f + expf(-v.z)) * v.w;
    *reinterpret_cast<uint32_t*>(act + (size_t)b * d_ff + 2 * c) = pack_f16(a0, a1);
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
    grid_dependency_sync();
    const StepArgs sa = *args;
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
        if (threadIdx.x == 0) sa.tok_out[b] = argmax_key_index(best);
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
