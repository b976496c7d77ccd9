// Split-context grouped-query decode attention over a paged 2-byte (fp16 or bf16) KV cache, and the
// merge of the partial results.
//
// The op reads every cached key and value once and does G (<= 8) multiply-adds per element: it is
// HBM-bound, so the kernel is built around keeping TMA loads in flight.
//
// Work = the flattened list of (game, KV head, page) units of this step, cut into equal contiguous
// ranges, one per warp of a persistent grid (one CTA per SM, 8 warps).  Each warp owns a private
// ring of shared-memory stages; lane 0 issues one tiled TMA load per 64-element half of a
// (page, head) block -- its 16 K rows and 16 V rows are contiguous in the pool, so one box of 32
// rows x 128 bytes fetches both, written with the 128-byte swizzle -- and the whole warp consumes
// the stage with ldmatrix + mma.sync.m16n8k16.  There is no cross-warp synchronisation in the loop.
// The G query heads that share the KV head are the rows of a 16-row tile: rows 0..7 carry the high
// part of (q * scale) in the cache's 2-byte type, rows 8..15 the low part, so one MMA yields the
// product with a query mantissa twice as long (row g + row g+8); the softmax weights in P.V are
// split the same way.  Online softmax runs in the exp2 domain with fp32 running max / sum.
// A range that covers only part of a (game, head) item publishes a partial (m, l, o); the range
// that publishes last folds the item's partials in range order (so the result does not depend on
// which one that is) and emits the normalised output.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "gemm_tc.cuh"
#include "kernels_small.cuh"
#include "tma.cuh"

namespace spiral {

constexpr int ATTN_PAGE = 16;          // tokens per page the kernel is built for
constexpr int ATTN_WARPS = 8;
constexpr int ATTN_STAGES = 2;         // per-warp ring depth (a third stage only adds queueing: 8 warps x 3 x 8 KB oversubscribes the memory system)
constexpr int ATTN_RMIN = 4;           // ranges are never cut shorter than this many pages
constexpr int ATTN_MAX_SLOTS = 256;    // batch slots per launch

struct AttnParams {
    const float* q;                 // [n][n_q_heads][head_dim] fp32, normalised and rotated
    const int32_t* block_table;     // [max_games][max_pages]
    const int32_t* game;            // [n]
    const int32_t* ctx_len;         // [n]; tokens attended = ctx_len[i] + len_add
    const int32_t* cum;             // [n + 1] running count of (head, page) units before each slot, then
                                    // cum[n + 1] = pages per work range (both written by the host per step)
    int len_add;
    int n, max_pages, n_pages, layer, n_q_heads, n_kv_heads, group;
    int n_workers;                  // warps of the attention grid
    float scale_log2;               // log2(e) / sqrt(head_dim)
    float* o_part;                  // [n_workers + n * n_kv_heads][group][head_dim]
    float* m_part;                  // [n_workers + n * n_kv_heads][group]   (log2 domain)
    float* l_part;
    int* item_cnt;                  // [n * n_kv_heads] partials published per item; zero between launches
    __half* out_f16;                // [n][n_q_heads * head_dim] (input of the output projection) and / or
    float* out_f32;                 // the same in fp32; either may be null
    int* status;
    int skip_first_load;            // wait-timeout self-test only: every range leaves its first page load out, so its
                                    // first wait has to run out and the warp has to unwind
};

// Host side of the schedule: unit prefix over the slots and the pages per work range.  The even
// cut is ceil(U / workers); a range length up to a quarter above it is preferred when it makes fewer
// (game, head) items straddle a range boundary, because every straddling item costs a merge of
// partials at the end of the kernel (with equal-length games one item per range avoids them all).
inline void attn_host_plan(const int* tokens, int n, int n_kv_heads, int n_workers, int32_t* cum_out /* n + 2 */) {
    cum_out[0] = 0;
    for (int i = 0; i < n; ++i) cum_out[i + 1] = cum_out[i] + n_kv_heads * ((tokens[i] + ATTN_PAGE - 1) / ATTN_PAGE);
    const long long U = cum_out[n];
    int r0 = (int)((U + n_workers - 1) / n_workers);
    if (r0 < ATTN_RMIN) r0 = ATTN_RMIN;
    int best_r = r0;
    long long best_splits = -1;
    const int r_hi = r0 + (r0 + 3) / 4;
    for (int r = r0; r <= r_hi && best_splits != 0; ++r) {
        long long splits = 0;
        for (int i = 0; i < n; ++i) {
            const int pages = (cum_out[i + 1] - cum_out[i]) / n_kv_heads;
            for (int h = 0; h < n_kv_heads; ++h) {
                const long long ua = cum_out[i] + (long long)h * pages;
                splits += (ua / r) != ((ua + pages - 1) / r);
            }
        }
        if (best_splits < 0 || splits < best_splits) { best_splits = splits; best_r = r; }
    }
    cum_out[n + 1] = best_r;
}

#ifdef ATT_PROBE        // timing-probe builds only: eight timestamps per warp of the last attention launch (entry, schedule in
                        // shared memory, before / after the first requests, first / last page landed, work done)
__device__ unsigned long long g_att_probe[2048 * 8];
#define ATT_STAMP(i) do { if (lane == 0) g_att_probe[(size_t)w * 8 + (i)] = global_ns(); } while (0)
#else
#define ATT_STAMP(i) do { } while (0)
#endif

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
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
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

// The work of one warp: work range w of the step's (game, KV head, page) units.  `bars` are this
// warp's ATTN_STAGES "stage full" mbarriers, `ring` its stages in shared memory, `ring_it0` the
// number of stages the warp has consumed through these barriers before (0 right after their
// initialisation); returns the new count.  cum_sm / len_sm / game_sm: the step's schedule, tokens
// attended and game per slot, in shared memory.
// `dependency_wait` is called once by every thread, at the point from which data written by the kernels ahead (block
// table entries of new pages, queries, appended keys/values) is read; what comes before it uses the schedule only.
template <int HD, bool F16, class WaitFn>
__device__ __forceinline__ uint32_t attn_warp_work(const CUtensorMap* tmKV, const AttnParams& p, const int* cum_sm,
                                                   const int* len_sm, const int* game_sm, uint64_t* bars, uint32_t ring,
                                                   uint32_t ring_it0, volatile int* abort_flag, int w, WaitFn dependency_wait) {
    constexpr int HALVES = HD / 64;                 // TMA boxes (64 elements wide) per stage
    constexpr int STAGE_BYTES = HALVES * 4096;      // 32 rows (16 K + 16 V) x 128 bytes per half
    constexpr int KSTEPS = HD / 16;                 // k-steps of Q.K^T
    constexpr int NT = HD / 8;                      // 8-column output tiles of P.V
    const int lane = threadIdx.x & 31, g = lane >> 2, c = lane & 3;
    const int G = p.group, Hkv = p.n_kv_heads;
    const int U = cum_sm[p.n];
    const int R = cum_sm[p.n + 1];
    const long long u0l = (long long)w * R;
    if (u0l >= U) { dependency_wait(); return ring_it0; }
    const int u0 = (int)u0l;
    const int cnt = min(U, u0 + R) - u0;

    // slot that holds unit u: largest s with cum[s] <= u
    auto slot_of = [&](int u) {
        int lo = 0, hi = p.n - 1;
        while (lo < hi) {
            int mid = (lo + hi + 1) >> 1;
            if (cum_sm[mid] <= u) lo = mid; else hi = mid - 1;
        }
        return lo;
    };
    // where unit u's page id sits in the block table, and its KV head (schedule only)
    auto locate = [&](int u, int& kvh_out) -> size_t {
        int s = slot_of(u);
        int pages = (len_sm[s] + ATTN_PAGE - 1) / ATTN_PAGE;
        int off = u - cum_sm[s];
        int kvh = off / pages, pg = off - kvh * pages;
        kvh_out = kvh;
        return (size_t)game_sm[s] * p.max_pages + pg;
    };
    // first pool row (TMA y coordinate) of the (page, head) block whose page id is table entry `at`
    auto row_of = [&](size_t at, int kvh) -> int {
        int page = __ldcg(p.block_table + at);
        if (page < 0 || page >= p.n_pages) {
            record_status(p.status, STATUS_BAD_PAGE);
            page = 0;
        }
        return (((p.layer * p.n_pages + page) * Hkv) + kvh) * 32;
    };
    auto fetch_row = [&](int u) -> int {
        int kvh;
        const size_t at = locate(u, kvh);
        return row_of(at, kvh);
    };
    // rows of the current and of the next window of 32 units, one unit per lane: located while the kernel ahead may
    // still run, read from the block table once it has finished
    int kvh_c = 0, kvh_n = 0;
    const size_t at_c = lane < cnt ? locate(u0 + lane, kvh_c) : 0;
    const size_t at_n = 32 + lane < cnt ? locate(u0 + 32 + lane, kvh_n) : 0;
    dependency_wait();
    int row_cur = lane < cnt ? row_of(at_c, kvh_c) : 0;
    int row_nxt = 32 + lane < cnt ? row_of(at_n, kvh_n) : 0;
    int win = 0;

    auto issue = [&](int j) {          // unit index j (relative to u0) into stage j % STAGES; all lanes call
        const int y = __shfl_sync(0xffffffffu, row_cur, j & 31);     // j lies in window `win`
        if (lane == 0) {
            const uint32_t bar = smem_u32(&bars[(ring_it0 + (uint32_t)j) % ATTN_STAGES]);
            const uint32_t dst = ring + (uint32_t)(((ring_it0 + (uint32_t)j) % ATTN_STAGES) * STAGE_BYTES);
            mbar_expect_tx(bar, STAGE_BYTES);
            if (p.skip_first_load && j == 0) return;
#pragma unroll
            for (int h = 0; h < HALVES; ++h) tma_load_2d_nohint(dst + h * 4096, tmKV, 64 * h, y, bar);
        }
    };
    ATT_STAMP(2);
    for (int j = 0; j < ATTN_STAGES && j < cnt; ++j) issue(j);
    ATT_STAMP(3);

    // consumer cursor
    int slot = slot_of(u0);
    int T = len_sm[slot];
    int pages = (T + ATTN_PAGE - 1) / ATTN_PAGE;
    int kvh = (u0 - cum_sm[slot]) / pages;
    int pg = (u0 - cum_sm[slot]) - kvh * pages;

    uint32_t qa[KSTEPS][4];
    float m = -INFINITY, l = 0.f;
    float o[NT][4];
    bool fresh = true;                 // the item's query fragments still have to be loaded

    // byte offset of (row r, 16-byte chunk ch) inside one swizzled half box
    const int lr = lane & 7, lm = lane >> 3;
    // ldmatrix row addresses of this lane: K (non-transposed) and V (transposed) variants
    const int k_tok = lr + 8 * (lm >> 1), k_chk = lm & 1;
    const int v_tok = lr + 8 * (lm & 1), v_chk = lm >> 1;
    const uint32_t k_row_off = (uint32_t)(k_tok * 128), v_row_off = (uint32_t)((16 + v_tok) * 128);

    for (int i = 0; i < cnt; ++i) {
        if (fresh) {
            const float* qp = p.q + ((size_t)slot * p.n_q_heads + kvh * G + g) * HD + 2 * c;
#pragma unroll
            for (int ks = 0; ks < KSTEPS; ++ks) {
                float2 a = make_float2(0.f, 0.f), b = make_float2(0.f, 0.f);
                if (g < G) {
                    a = __ldcg(reinterpret_cast<const float2*>(qp + 16 * ks));      // through L2: written by other SMs,
                    b = __ldcg(reinterpret_cast<const float2*>(qp + 16 * ks + 8));  // possibly in this same kernel
                }
                uint32_t h0, l0, h1, l1, h2, l2, h3, l3;
                split2<F16>(a.x * p.scale_log2, h0, l0);
                split2<F16>(a.y * p.scale_log2, h1, l1);
                split2<F16>(b.x * p.scale_log2, h2, l2);
                split2<F16>(b.y * p.scale_log2, h3, l3);
                qa[ks][0] = h0 | (h1 << 16); qa[ks][1] = l0 | (l1 << 16);
                qa[ks][2] = h2 | (h3 << 16); qa[ks][3] = l2 | (l3 << 16);
            }
            m = -INFINITY; l = 0.f;
#pragma unroll
            for (int t = 0; t < NT; ++t) { o[t][0] = 0.f; o[t][1] = 0.f; o[t][2] = 0.f; o[t][3] = 0.f; }
            fresh = false;
        }
        const int st = (int)((ring_it0 + (uint32_t)i) % ATTN_STAGES);
        const uint32_t base = ring + (uint32_t)(st * STAGE_BYTES);
        const bool landed = mbar_wait(smem_u32(&bars[st]), ((ring_it0 + (uint32_t)i) / ATTN_STAGES) & 1u, abort_flag,
                                      p.status, STATUS_TIMEOUT_TMA);
        if (!__all_sync(0xffffffffu, landed)) break;
        if (i == 0) ATT_STAMP(4);
        if (i == cnt - 1) ATT_STAMP(5);
        const int valid = T - pg * ATTN_PAGE;          // tokens of this page that exist (>= 1)
        const bool ragged = valid < ATTN_PAGE;
        if (ragged) {
            // value rows of positions that do not exist yet hold stale pool bytes: zero them so that
            // weight 0 times garbage cannot produce NaN
            for (int idx = lane; idx < (ATTN_PAGE - valid) * 8 * HALVES; idx += 32) {
                int r = valid + idx / (8 * HALVES), rem = idx % (8 * HALVES);
                asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(base + (rem >> 3) * 4096 + (16 + r) * 128 +
                                                                           (rem & 7) * 16), "r"(0u) : "memory");
            }
            __syncwarp();
        }
        // ---- scores: S[16 x 16 tokens] = Q[16 x HD] K^T ----
        float s[2][4];
#pragma unroll
        for (int t = 0; t < 2; ++t) { s[t][0] = 0.f; s[t][1] = 0.f; s[t][2] = 0.f; s[t][3] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
            const int h = ks >> 2, ch = 2 * (ks & 3) + k_chk;
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4(base + h * 4096 + k_row_off + (uint32_t)(((ch ^ (k_tok & 7)) << 4)), b0, b1, b2, b3);
            mma_16816<F16>(s[0], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b0, b1);
            mma_16816<F16>(s[1], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b2, b3);
        }
        // scores of query row g for tokens pg*16 + 8t + 2c + e  (hi-part row + lo-part row)
        float sc[4];
#pragma unroll
        for (int t = 0; t < 2; ++t)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                float v = s[t][e] + s[t][2 + e];
                sc[2 * t + e] = (8 * t + 2 * c + e) < valid ? v : -INFINITY;
            }
        float mx = fmaxf(fmaxf(sc[0], sc[1]), fmaxf(sc[2], sc[3]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m, mx);
        float pr[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) pr[k] = fast_exp2(sc[k] - m_new);
        const float alpha = fast_exp2(m - m_new);
        l = l * alpha + (pr[0] + pr[1]) + (pr[2] + pr[3]);
        if (__any_sync(0xffffffffu, m_new > m)) {
#pragma unroll
            for (int t = 0; t < NT; ++t) { o[t][0] *= alpha; o[t][1] *= alpha; o[t][2] *= alpha; o[t][3] *= alpha; }
        }
        m = m_new;
        uint32_t ph[4], pl[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) split2<F16>(pr[k], ph[k], pl[k]);
        const uint32_t a0 = ph[0] | (ph[1] << 16), a1 = pl[0] | (pl[1] << 16);
        const uint32_t a2 = ph[2] | (ph[3] << 16), a3 = pl[2] | (pl[3] << 16);
        // ---- O[16 x HD] += P[16 x 16 tokens] V ----
#pragma unroll
        for (int np = 0; np < NT / 2; ++np) {
            const int h = np >> 2, ch = 2 * (np & 3) + v_chk;
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4_trans(base + h * 4096 + v_row_off + (uint32_t)(((ch ^ (v_tok & 7)) << 4)), b0, b1, b2, b3);
            mma_16816<F16>(o[2 * np], a0, a1, a2, a3, b0, b1);
            mma_16816<F16>(o[2 * np + 1], a0, a1, a2, a3, b2, b3);
        }
        __syncwarp();
        // refill this stage with the unit ATTN_STAGES ahead
        const int j = i + ATTN_STAGES;
        if (j < cnt) {
            if ((j >> 5) > win) {                  // j entered the next window: look up the one after it
                row_cur = row_nxt;
                ++win;
                row_nxt = (win + 1) * 32 + lane < cnt ? fetch_row(u0 + (win + 1) * 32 + lane) : 0;
            }
            if (ragged && lane == 0) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            issue(j);
        }
        // advance the cursor; close the item when it ends (or the range does)
        ++pg;
        const bool item_end = pg == pages;
        if (item_end || i + 1 == cnt) {
            l += __shfl_xor_sync(0xffffffffu, l, 1);
            l += __shfl_xor_sync(0xffffffffu, l, 2);
            // ranges that touch this item: [w0, w1]
            const int ua = cum_sm[slot] + kvh * pages;
            const int w0 = ua / R, w1 = (ua + pages - 1) / R;
            const size_t item = (size_t)slot * Hkv + kvh;
            if (w0 == w1) {
                // the whole item was in this range: normalise and emit
                if (g < G) {
                    const float inv = 1.f / l;
                    const size_t ob = ((size_t)slot * p.n_q_heads + kvh * G + g) * HD + 2 * c;
#pragma unroll
                    for (int t = 0; t < NT; ++t) {
                        const float r0 = (o[t][0] + o[t][2]) * inv, r1 = (o[t][1] + o[t][3]) * inv;
                        if (p.out_f16) *reinterpret_cast<uint32_t*>(p.out_f16 + ob + 8 * t) = pack_f16(r0, r1);
                        if (p.out_f32) *reinterpret_cast<float2*>(p.out_f32 + ob + 8 * t) = make_float2(r0, r1);
                    }
                }
            } else {
                const size_t part = (size_t)w + item;
                if (g < G) {
                    float* op = p.o_part + (part * G + g) * HD + 2 * c;
#pragma unroll
                    for (int t = 0; t < NT; ++t)
                        *reinterpret_cast<float2*>(op + 8 * t) = make_float2(o[t][0] + o[t][2], o[t][1] + o[t][3]);
                    if (c == 0) { p.m_part[part * G + g] = m; p.l_part[part * G + g] = l; }
                }
                // publish; the range that arrives last folds the partials of the item in range order:
                // o = sum_i 2^(m_i-M) o_i / sum_i 2^(m_i-M) l_i
                __threadfence();
                __syncwarp();
                int last = 0;
                if (lane == 0) last = atomicAdd(p.item_cnt + item, 1) == w1 - w0;
                last = __shfl_sync(0xffffffffu, last, 0);
                if (last) {
                    __threadfence();
                    // lane (partial j, head hh) fetches that partial's m and l; the weights then go
                    // round by shuffle, so the loads of all partials are in flight together
                    const int np = w1 - w0 + 1;
                    for (int gg0 = 0; gg0 < G; gg0 += 4) {              // up to 8 partials x 4 heads per pass
                        const int pj = lane >> 2, ph = gg0 + (lane & 3);
                        float mj = -INFINITY, lj = 0.f;
                        if (pj < np && ph < G && np <= 8) {
                            mj = __ldcg(p.m_part + ((size_t)(w0 + pj) + item) * G + ph);
                            lj = __ldcg(p.l_part + ((size_t)(w0 + pj) + item) * G + ph);
                        }
                        for (int hh = 0; hh < 4 && gg0 + hh < G; ++hh) {
                            const int gg = gg0 + hh;
                            float M = -INFINITY, ls = 0.f, acc[HD / 32];
#pragma unroll
                            for (int k = 0; k < HD / 32; ++k) acc[k] = 0.f;
                            if (np <= 8) {
                                for (int j = 0; j < np; ++j) M = fmaxf(M, __shfl_sync(0xffffffffu, mj, 4 * j + hh));
                                for (int j = 0; j < np; ++j) {
                                    const float wt = fast_exp2(__shfl_sync(0xffffffffu, mj, 4 * j + hh) - M);
                                    ls += wt * __shfl_sync(0xffffffffu, lj, 4 * j + hh);
                                    const float* op = p.o_part + (((size_t)(w0 + j) + item) * G + gg) * HD + lane;
#pragma unroll
                                    for (int k = 0; k < HD / 32; ++k) acc[k] += wt * __ldcg(op + 32 * k);
                                }
                            } else {
                                for (int ww = w0; ww <= w1; ++ww) M = fmaxf(M, __ldcg(p.m_part + (ww + item) * G + gg));
                                for (int ww = w0; ww <= w1; ++ww) {
                                    const float wt = fast_exp2(__ldcg(p.m_part + (ww + item) * G + gg) - M);
                                    ls += wt * __ldcg(p.l_part + (ww + item) * G + gg);
                                    const float* op = p.o_part + ((ww + item) * G + gg) * HD + lane;
#pragma unroll
                                    for (int k = 0; k < HD / 32; ++k) acc[k] += wt * __ldcg(op + 32 * k);
                                }
                            }
                            const float inv = 1.f / ls;
                            const size_t ob = ((size_t)slot * p.n_q_heads + kvh * G + gg) * HD + lane;
#pragma unroll
                            for (int k = 0; k < HD / 32; ++k) {
                                const float r = acc[k] * inv;
                                if (p.out_f16) p.out_f16[ob + 32 * k] = __ushort_as_half((unsigned short)float_to_f16_bits(r));
                                if (p.out_f32) p.out_f32[ob + 32 * k] = r;
                            }
                        }
                    }
                    if (lane == 0) p.item_cnt[item] = 0;
                }
            }
            fresh = true;
        }
        if (item_end) {
            pg = 0;
            if (++kvh == Hkv) {
                kvh = 0;
                ++slot;
                if (slot < p.n) { T = len_sm[slot]; pages = (T + ATTN_PAGE - 1) / ATTN_PAGE; }
            }
        }
    }
    ATT_STAMP(6);
    if (*abort_flag) {
        // loads already issued still land in this warp's ring: give them a bounded time
        for (int s = 0; s < ATTN_STAGES; ++s) {
            unsigned long long t0 = global_ns();
            while (!mbar_try(smem_u32(&bars[s]), 0) && !mbar_try(smem_u32(&bars[s]), 1) &&
                   global_ns() - t0 < g_wait_limit_ns) {}
        }
    }
    return ring_it0 + (uint32_t)cnt;
}

template <int HD, bool F16>
__global__ void __launch_bounds__(ATTN_WARPS * 32, 1) attn_decode_kernel(const __grid_constant__ CUtensorMap tmKV,
                                                                        AttnParams p) {
    constexpr int HALVES = HD / 64;                 // TMA boxes (64 elements wide) per stage
    constexpr int STAGE_BYTES = HALVES * 4096;      // 32 rows (16 K + 16 V) x 128 bytes per half
    extern __shared__ uint8_t attn_smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[ATTN_WARPS][ATTN_STAGES];
    __shared__ int cum_sm[ATTN_MAX_SLOTS + 2];
    __shared__ int len_sm[ATTN_MAX_SLOTS];
    __shared__ int game_sm[ATTN_MAX_SLOTS];
    __shared__ int abort_sm;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    TRACE_BEGIN(7);
#ifdef ATT_PROBE
    const unsigned long long t_entry__ = global_ns();
#endif
    grid_launch_dependents();
    if (lane == 0)
        for (int s = 0; s < ATTN_STAGES; ++s) mbar_init(smem_u32(&full_bar[warp][s]), 1);
    if (threadIdx.x == 0) {
        abort_sm = 0;
        tmap_prefetch(&tmKV);
    }
    // The schedule (range starts, lengths, games) is what the host uploaded before the first kernel of the step: a
    // copy, not a kernel, so it is complete before any kernel of the step starts and can be staged while the kernel
    // ahead still runs.  Queries, the appended keys/values and the block table's new entries come from kernels.
    for (int i = threadIdx.x; i <= p.n + 1; i += blockDim.x) {
        cum_sm[i] = p.cum[i];
        if (i < p.n) { len_sm[i] = p.ctx_len[i] + p.len_add; game_sm[i] = p.game[i]; }
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();

#ifdef ATT_PROBE
    if (lane == 0) { g_att_probe[(size_t)(warp * gridDim.x + blockIdx.x) * 8 + 0] = t_entry__; g_att_probe[(size_t)(warp * gridDim.x + blockIdx.x) * 8 + 1] = global_ns(); }
#endif
    const int w = warp * gridDim.x + blockIdx.x;       // consecutive ranges on different SMs: when fewer
                                                       // ranges than warps have work, every SM still streams
    const uint32_t ring = ((smem_u32(attn_smem_raw) + 1023u) & ~1023u) + (uint32_t)(warp * ATTN_STAGES * STAGE_BYTES);
    attn_warp_work<HD, F16>(&tmKV, p, cum_sm, len_sm, game_sm, full_bar[warp], ring, 0u, &abort_sm, w, [&]() {
        grid_dependency_wait();
        TRACE_WAITED();
    });
}

}  // namespace spiral
