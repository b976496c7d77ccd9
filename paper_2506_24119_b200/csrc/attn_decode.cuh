// Split-context grouped-query decode attention over a paged 2-byte (fp16 or bf16) KV cache, and the
// merge of the per-chunk partial results.
//
// One CTA (4 warps) handles one (game, KV head, chunk of pages).  The G <= 8 query heads that
// share the KV head are the rows of a 16-row tensor-core tile: rows 0..7 carry the high part of
// (q * scale) in the cache's 2-byte type, rows 8..15 the low part, so that one mma.sync.m16n8k16
// yields the product with a query mantissa twice as long (row g + row g+8).  The same trick is used for the
// softmax weights in P.V.  The op is HBM-bound (G flop per byte), so K and V go straight from
// global memory into the B-operand register layout with coalesced 16-byte loads: the reduction
// index of Q.K^T (head_dim) and of P.V (tokens) may be permuted freely as long as both operands
// use the same permutation, which is chosen so that every thread reads contiguous 16-byte pieces
// of the page rows.  Online softmax runs in the exp2 domain with fp32 running max / sum.
#pragma once
#include "common.cuh"
#include "kernels_small.cuh"

namespace spiral {

constexpr int ATTN_PAGE = 16;          // tokens per page the kernel is built for
constexpr int ATTN_MAX_CHUNKS = 32;    // upper bound on chunks (CTAs) per (game, KV head)
constexpr int ATTN_WARPS = 4;

struct AttnParams {
    const float* q;                 // [n][n_q_heads][head_dim] fp32, normalised and rotated
    const uint16_t* pool;           // 2-byte elements: fp16 or bf16 (template parameter)
    const int32_t* block_table;     // [max_games][max_pages]
    const int32_t* game;            // [n]
    const int32_t* ctx_len;         // [n]; tokens attended = ctx_len[i] + len_add
    int len_add;
    int max_pages, n_pages, layer, n_q_heads, n_kv_heads, group;
    int ppw;                        // pages per warp in one CTA chunk
    float scale_log2;               // log2(e) / sqrt(head_dim)
    float* o_part;                  // [n][n_kv_heads][ATTN_MAX_CHUNKS][group][head_dim]
    float* m_part;                  // [n][n_kv_heads][ATTN_MAX_CHUNKS][group]   (log2 domain)
    float* l_part;
    int* status;
};

template <bool F16>
__device__ __forceinline__ void mma_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1) {
    if (F16)
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    else
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// split v into a high and a low part of the 2-byte type (v ~= hi + lo)
template <bool F16>
__device__ __forceinline__ void split2(float v, uint32_t& hi, uint32_t& lo) {
    if (F16) {
        __half h = __float2half_rn(v);
        hi = (uint32_t)__half_as_ushort(h);
        lo = (uint32_t)__half_as_ushort(__float2half_rn(v - __half2float(h)));
    } else {
        __nv_bfloat16 h = __float2bfloat16_rn(v);
        hi = (uint32_t)__bfloat16_as_ushort(h);
        lo = float_to_bf16_bits(v - __bfloat162float(h));
    }
}

template <int HD, bool F16>
__global__ void __launch_bounds__(ATTN_WARPS * 32, 3) attn_decode_kernel(AttnParams p) {
    constexpr int KSTEPS = HD / 16;    // k-steps of Q.K^T
    constexpr int NT = HD / 8;         // 8-column output tiles of P.V
    constexpr int CH = HD / 32;        // 16-byte pieces of a K row per thread
    constexpr int VH = HD / 64;        // 16-byte pieces of a V row per thread
    const int chunk = blockIdx.x, kvh = blockIdx.y, slot = blockIdx.z;
    const int T = p.ctx_len[slot] + p.len_add;
    const int pages = (T + ATTN_PAGE - 1) / ATTN_PAGE;
    const int pages_per_cta = ATTN_WARPS * p.ppw;
    const int page0 = chunk * pages_per_cta;
    if (page0 >= pages) return;
    const int page_lim = min(pages, page0 + pages_per_cta);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, c = lane & 3;
    const int G = p.group;

    __shared__ uint4 q_frag[KSTEPS][32];
    __shared__ float o_sm[ATTN_WARPS][8][HD];
    __shared__ float ml_sm[ATTN_WARPS][8][2];

    // A-operand fragments of (q * scale * log2 e): hi part in rows 0..7, lo part in rows 8..15
    for (int idx = threadIdx.x; idx < KSTEPS * 32; idx += blockDim.x) {
        int ks = idx >> 5, ln = idx & 31, gg = ln >> 2, cc = ln & 3;
        int e0 = (4 * (ks >> 1) + cc) * 8 + 4 * (ks & 1);
        uint4 f = make_uint4(0u, 0u, 0u, 0u);
        if (gg < G) {
            const float* qp = p.q + ((size_t)slot * p.n_q_heads + kvh * G + gg) * HD + e0;
            float4 v = *reinterpret_cast<const float4*>(qp);
            uint32_t h0, l0, h1, l1, h2, l2, h3, l3;
            split2<F16>(v.x * p.scale_log2, h0, l0);
            split2<F16>(v.y * p.scale_log2, h1, l1);
            split2<F16>(v.z * p.scale_log2, h2, l2);
            split2<F16>(v.w * p.scale_log2, h3, l3);
            f.x = h0 | (h1 << 16); f.y = l0 | (l1 << 16); f.z = h2 | (h3 << 16); f.w = l2 | (l3 << 16);
        }
        q_frag[ks][ln] = f;
    }
    __syncthreads();

    const int32_t* table = p.block_table + (size_t)p.game[slot] * p.max_pages;
    uint32_t kr[2][CH][4];
    uint32_t vr[4][VH][4];

    auto page_base = [&](int pg) -> const uint16_t* {
        int page = table[pg];
        if (page < 0 || page >= p.n_pages) {
            record_status(p.status, STATUS_BAD_PAGE);
            page = 0;
        }
        return p.pool + kv_block_offset(p.layer, page, kvh, p.n_pages, p.n_kv_heads, ATTN_PAGE, HD);
    };
    auto load_k = [&](const uint16_t* kb) {
#pragma unroll
        for (int t = 0; t < 2; ++t)
#pragma unroll
            for (int j = 0; j < CH; ++j) {
                uint4 v = ldg_stream_v4(kb + (8 * t + g) * HD + (4 * j + c) * 8);
                kr[t][j][0] = v.x; kr[t][j][1] = v.y; kr[t][j][2] = v.z; kr[t][j][3] = v.w;
            }
    };
    auto load_v = [&](const uint16_t* kb, int pg) {
        const uint16_t* vb = kb + ATTN_PAGE * HD;
#pragma unroll
        for (int ri = 0; ri < 4; ++ri) {
            int r = 2 * c + (ri & 1) + 8 * (ri >> 1);
            bool valid = pg * ATTN_PAGE + r < T;
#pragma unroll
            for (int h = 0; h < VH; ++h) {
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                if (valid) v = ldg_stream_v4(vb + r * HD + 64 * h + 8 * g);
                vr[ri][h][0] = v.x; vr[ri][h][1] = v.y; vr[ri][h][2] = v.z; vr[ri][h][3] = v.w;
            }
        }
    };

    float m = -INFINITY, l = 0.f;
    float o[NT][4];
#pragma unroll
    for (int i = 0; i < NT; ++i) { o[i][0] = 0.f; o[i][1] = 0.f; o[i][2] = 0.f; o[i][3] = 0.f; }

    int pg = page0 + warp;
    bool have = pg < page_lim;
    if (have) {
        const uint16_t* kb = page_base(pg);
        load_k(kb);
        load_v(kb, pg);
    }
    while (have) {
        float s[2][4];
#pragma unroll
        for (int t = 0; t < 2; ++t) { s[t][0] = 0.f; s[t][1] = 0.f; s[t][2] = 0.f; s[t][3] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
            uint4 a = q_frag[ks][lane];
#pragma unroll
            for (int t = 0; t < 2; ++t)
                mma_16816<F16>(s[t], a.x, a.y, a.z, a.w, kr[t][ks >> 1][2 * (ks & 1)], kr[t][ks >> 1][2 * (ks & 1) + 1]);
        }
        const int npg = pg + ATTN_WARPS;
        const bool nhave = npg < page_lim;
        const uint16_t* nkb = nullptr;
        if (nhave) {
            nkb = page_base(npg);
            load_k(nkb);
        }
        // scores of query row g for tokens pg*16 + 8t + 2c + e  (hi-part row + lo-part row)
        float sc[4];
#pragma unroll
        for (int t = 0; t < 2; ++t)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                float v = s[t][e] + s[t][2 + e];
                int tok = pg * ATTN_PAGE + 8 * t + 2 * c + e;
                sc[2 * t + e] = tok < T ? v : -INFINITY;
            }
        float mx = fmaxf(fmaxf(sc[0], sc[1]), fmaxf(sc[2], sc[3]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m, mx);
        float pr[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) pr[i] = fast_exp2(sc[i] - m_new);
        const float alpha = fast_exp2(m - m_new);
        l = l * alpha + (pr[0] + pr[1]) + (pr[2] + pr[3]);
        if (__any_sync(0xffffffffu, m_new > m)) {
#pragma unroll
            for (int i = 0; i < NT; ++i) { o[i][0] *= alpha; o[i][1] *= alpha; o[i][2] *= alpha; o[i][3] *= alpha; }
        }
        m = m_new;
        uint32_t ph[4], pl[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) split2<F16>(pr[i], ph[i], pl[i]);
        const uint32_t a0 = ph[0] | (ph[1] << 16), a1 = pl[0] | (pl[1] << 16);
        const uint32_t a2 = ph[2] | (ph[3] << 16), a3 = pl[2] | (pl[3] << 16);
#pragma unroll
        for (int h = 0; h < VH; ++h)
#pragma unroll
            for (int jj = 0; jj < 8; ++jj) {
                const uint32_t sel = (jj & 1) ? 0x7632u : 0x5410u;
                uint32_t b0 = __byte_perm(vr[0][h][jj >> 1], vr[1][h][jj >> 1], sel);
                uint32_t b1 = __byte_perm(vr[2][h][jj >> 1], vr[3][h][jj >> 1], sel);
                mma_16816<F16>(o[8 * h + jj], a0, a1, a2, a3, b0, b1);
            }
        if (nhave) load_v(nkb, npg);
        pg = npg;
        have = nhave;
    }
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    if (c == 0) { ml_sm[warp][g][0] = m; ml_sm[warp][g][1] = l; }
#pragma unroll
    for (int h = 0; h < VH; ++h)
#pragma unroll
        for (int jj = 0; jj < 8; ++jj)
#pragma unroll
            for (int e = 0; e < 2; ++e)
                o_sm[warp][g][64 * h + 16 * c + 8 * e + jj] = o[8 * h + jj][e] + o[8 * h + jj][2 + e];
    __syncthreads();
    // combine the four warps and emit this chunk's partial (m, l, o) per query head
    const size_t part = ((size_t)slot * p.n_kv_heads + kvh) * ATTN_MAX_CHUNKS + chunk;
    for (int idx = threadIdx.x; idx < G * HD; idx += blockDim.x) {
        int gg = idx / HD, col = idx % HD;
        float M = ml_sm[0][gg][0];
#pragma unroll
        for (int w = 1; w < ATTN_WARPS; ++w) M = fmaxf(M, ml_sm[w][gg][0]);
        float acc = 0.f, ls = 0.f;
#pragma unroll
        for (int w = 0; w < ATTN_WARPS; ++w) {
            float sc = fast_exp2(ml_sm[w][gg][0] - M);
            acc += sc * o_sm[w][gg][col];
            ls += sc * ml_sm[w][gg][1];
        }
        p.o_part[(part * G + gg) * HD + col] = acc;
        if (col == 0) { p.m_part[part * G + gg] = M; p.l_part[part * G + gg] = ls; }
    }
}

// Combine the chunk partials of each (game, query head): o = sum_i 2^(m_i-M) o_i / sum_i 2^(m_i-M) l_i.
// Writes fp16 [n][n_q_heads*head_dim] (input of the output projection) and/or fp32.
template <int HD>
__global__ void attn_merge_kernel(AttnParams p, __half* __restrict__ out_f16, float* __restrict__ out_f32) {
    const int slot = blockIdx.x, a = blockIdx.y, col = threadIdx.x;
    const int G = p.group, kvh = a / G, gg = a % G;
    const int T = p.ctx_len[slot] + p.len_add;
    const int pages = (T + ATTN_PAGE - 1) / ATTN_PAGE;
    const int n_chunks = (pages + ATTN_WARPS * p.ppw - 1) / (ATTN_WARPS * p.ppw);
    const size_t base = ((size_t)slot * p.n_kv_heads + kvh) * ATTN_MAX_CHUNKS;
    float M = -INFINITY;
    for (int i = 0; i < n_chunks; ++i) M = fmaxf(M, p.m_part[(base + i) * G + gg]);
    float acc = 0.f, ls = 0.f;
    for (int i = 0; i < n_chunks; ++i) {
        float w = fast_exp2(p.m_part[(base + i) * G + gg] - M);
        acc += w * p.o_part[((base + i) * G + gg) * HD + col];
        ls += w * p.l_part[(base + i) * G + gg];
    }
    float r = acc / ls;
    size_t oidx = ((size_t)slot * p.n_q_heads + a) * HD + col;
    if (out_f16) out_f16[oidx] = __ushort_as_half((unsigned short)float_to_f16_bits(r));
    if (out_f32) out_f32[oidx] = r;
}

}  // namespace spiral
