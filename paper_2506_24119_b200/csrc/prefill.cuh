// Context append ("prefill"): the tokens an environment adds to a game's context between two turns
// of Algorithm 1 enter the model many at a time.  With hundreds to thousands of token rows per
// weight matrix the linear layers are dense contractions -- compute-bound on the tensor cores, not
// weight-streaming like the decode step -- and attention reads each cached key once per block of
// queries instead of once per query.  Kernels:
//
//   pf_gemm_kernel<EPI>   Y[t][r] = sum_k X[t][k] W[r][k] over output tiles of 128 weight rows x 256
//                         token rows, tcgen05.mma (M = 128, N = 256, K = 16) with two 256-column
//                         accumulators in tensor memory, a four-stage TMA ring (16 KB of W + 32 KB of
//                         X per stage) and an epilogue that runs under the next tile's mainloop:
//                         plain fp32 store, residual accumulation in place, or SwiGLU gating to fp16.
//   attn_append_tc_kernel causal grouped-query attention of a block of new positions of one game against
//                         everything cached for it (earlier turns and the new tokens up to each query's own
//                         position) on tcgen05: scores and the output accumulator in tensor memory, one
//                         softmax thread per query row, keys/values streamed page by page by TMA.
//   attn_append_kernel    the same attention on mma.sync.m16n8k16 (kept as an option), flash-style with the
//                         fp32 online softmax in registers.
//   pf_rmsnorm_kernel, pf_qkv_post_kernel   the element-wise steps for thousands of token rows.
//
// Every wait is bounded as in the decode kernels.
#pragma once
#include "attn_decode.cuh"
#include "gemm_tc.cuh"

namespace spiral {

// ------------------------------------------------------------------------------------------------
// dense GEMM
// ------------------------------------------------------------------------------------------------
constexpr int PF_BN = 256;                                   // token rows per tile = MMA N
constexpr int PF_STAGES = 4;
constexpr int PF_X_BYTES = PF_BN * TC_BK * 2;                // 32 KB
constexpr int PF_STAGE_BYTES = TC_W_BYTES + PF_X_BYTES;      // 48 KB
constexpr int PF_THREADS = 192;                              // TMA warp, MMA warp, four epilogue warps
constexpr size_t PF_SMEM = (size_t)PF_STAGES * PF_STAGE_BYTES + 1024;
enum { PF_EPI_STORE = 0, PF_EPI_ADD = 1, PF_EPI_SILU = 2 };

struct PfGemmParams {
    int row_tiles, tok_tiles, KB;   // 128-row tiles of W, 256-row tiles of X, 64-wide k blocks
    int rows, T;                    // weight rows (output features) and token rows
    int row_fastest;                // order in which consecutive CTAs take tiles (see pf_tile_of)
    float* out;                     // STORE: y [T][rows] written; ADD: x [T][rows] += result
    __half* act;                    // SILU: [T][rows / 2] = SiLU(y[2i]) * y[2i+1] (gate / up rows interleaved)
    int* status;
};

// Tiles are dealt round-robin.  Token tile fastest: the CTAs running at one time cover a few weight row
// tiles times all token tiles, so every weight tile is fetched from HBM once and shared through L2 while
// the activations are re-read once per wave.  Row tile fastest: the other way round.  The host picks the
// order that re-reads the smaller operand (the activations of the down projection exceed L2).
__device__ __forceinline__ void pf_tile_of(const int L, const int row_tiles, const int tok_tiles, const int row_fastest,
                                           int& rt, int& tt) {
    if (row_fastest) { tt = L / row_tiles; rt = L - tt * row_tiles; }
    else { rt = L / tok_tiles; tt = L - rt * tok_tiles; }
}
template <int EPI>
__global__ void __launch_bounds__(PF_THREADS, 1) pf_gemm_kernel(const __grid_constant__ CUtensorMap tmW,
                                                                const __grid_constant__ CUtensorMap tmX,
                                                                PfGemmParams p) {
    extern __shared__ uint8_t pf_smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[PF_STAGES], empty_bar[PF_STAGES], acc_full[2], acc_empty[2];
    __shared__ uint32_t tmem_base_sm;
    __shared__ int abort_sm;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    grid_launch_dependents();
    const uint32_t tiles_base = (smem_u32(pf_smem_raw) + 1023u) & ~1023u;
    constexpr uint32_t TMEM_COLS = 2 * PF_BN;
    const int n_tiles = p.row_tiles * p.tok_tiles;
    const int G = (int)gridDim.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < PF_STAGES; ++s) { mbar_init(smem_u32(&full_bar[s]), 1); mbar_init(smem_u32(&empty_bar[s]), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(smem_u32(&acc_full[a]), 1); mbar_init(smem_u32(&acc_empty[a]), 4); }
        abort_sm = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tmap_prefetch(&tmW);
        tmap_prefetch(&tmX);
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_sm), TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_sm;
    volatile int* abort_flag = &abort_sm;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            const uint64_t pol_w = l2_policy_evict_last(), pol_x = l2_policy_evict_last();
            // weights are written by nobody: the first ring-full of W tiles goes out before the dependency wait
            int pre = 0;
            for (int L = blockIdx.x, kb = 0; pre < PF_STAGES && L < n_tiles; ++pre) {
                const uint32_t fb = smem_u32(&full_bar[pre]);
                mbar_expect_tx(fb, PF_STAGE_BYTES);
                int rt, tt;
                pf_tile_of(L, p.row_tiles, p.tok_tiles, p.row_fastest, rt, tt);
                tma_load_2d(tiles_base + (uint32_t)pre * PF_STAGE_BYTES, &tmW, 0, (rt * p.KB + kb) * TC_BM, fb, pol_w);
                if (++kb == p.KB) { kb = 0; L += G; }
            }
            grid_dependency_wait();          // X is written by the preceding kernel
            int it = 0;
            bool ok = true;
            for (int L = blockIdx.x; ok && L < n_tiles; L += G) {
                int rt, tt;
                pf_tile_of(L, p.row_tiles, p.tok_tiles, p.row_fastest, rt, tt);
                for (int kb = 0; kb < p.KB; ++kb, ++it) {
                    const int s = it % PF_STAGES;
                    const uint32_t fb = smem_u32(&full_bar[s]);
                    const uint32_t dst = tiles_base + (uint32_t)s * PF_STAGE_BYTES;
                    if (it >= pre) {
                        const uint32_t ph = (uint32_t)(it / PF_STAGES) & 1u;
                        if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_MMA)) {
                            ok = false;
                            break;
                        }
                        mbar_expect_tx(fb, PF_STAGE_BYTES);
                        tma_load_2d(dst, &tmW, 0, (rt * p.KB + kb) * TC_BM, fb, pol_w);
                    }
                    tma_load_2d(dst + TC_W_BYTES, &tmX, kb * TC_BK, tt * PF_BN, fb, pol_x);
                }
            }
            if (!ok) {
                // copies already issued still land in this CTA's shared memory: bounded wait for them
                for (int back = 1; back <= PF_STAGES && back <= it; ++back) {
                    const int j = it - back, s = j % PF_STAGES;
                    const uint32_t ph = (uint32_t)(j / PF_STAGES) & 1u;
                    unsigned long long t0 = global_ns();
                    while (!mbar_try(smem_u32(&full_bar[s]), ph) && global_ns() - t0 < TMA_WAIT_NS) {}
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t idesc = tc_idesc_f16(PF_BN);
            int it = 0, acc_it = 0;
            bool ok = true;
            for (int L = blockIdx.x; ok && L < n_tiles; L += G, ++acc_it) {
                const int a = acc_it & 1;
                const uint32_t aph = (uint32_t)(acc_it >> 1) & 1u;
                if (!mbar_wait(smem_u32(&acc_empty[a]), aph ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_EPI)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(a * PF_BN);
                for (int kb = 0; kb < p.KB; ++kb, ++it) {
                    const int s = it % PF_STAGES;
                    const uint32_t ph = (uint32_t)(it / PF_STAGES) & 1u;
                    if (!mbar_wait(smem_u32(&full_bar[s]), ph, abort_flag, p.status, STATUS_TIMEOUT_TMA)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t w_addr = tiles_base + (uint32_t)s * PF_STAGE_BYTES;
                    const uint64_t da = smem_desc_sw128(w_addr), db = smem_desc_sw128(w_addr + TC_W_BYTES);
#pragma unroll
                    for (int k = 0; k < TC_BK / 16; ++k)
                        tc_mma_f16(d_tmem, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (kb > 0 || k > 0) ? 1u : 0u);
                    tc_commit(smem_u32(&empty_bar[s]));
                }
                if (ok) tc_commit(smem_u32(&acc_full[a]));
            }
        }
    } else {
        // ---------------- epilogue: warp w reads TMEM lanes 32 (w % 4) .. + 31 ----------------
        const int q = warp & 3;
        grid_dependency_wait();              // the output may still be read (or, ADD, written) by earlier kernels
        int acc_it = 0;
        for (int L = blockIdx.x; L < n_tiles; L += G, ++acc_it) {
            int rt, tt;
            pf_tile_of(L, p.row_tiles, p.tok_tiles, p.row_fastest, rt, tt);
            const int a = acc_it & 1;
            const uint32_t aph = (uint32_t)(acc_it >> 1) & 1u;
            if (!mbar_wait(smem_u32(&acc_full[a]), aph, abort_flag, p.status, STATUS_TIMEOUT_MMA)) break;
            tc_fence_after();
            const int row = rt * TC_BM + q * 32 + lane;
            const bool row_ok = row < p.rows;
            const int col0 = tt * PF_BN;
            const int n_cols = min(PF_BN, p.T - col0);                  // token rows of this tile that exist
            const uint32_t t_addr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(a * PF_BN);
            if (EPI == PF_EPI_SILU) {
                const int half_rows = p.rows >> 1;
                const bool odd = lane & 1;
                __half* arow = p.act + (size_t)col0 * half_rows + (row >> 1);
#pragma unroll 1
                for (int c0 = 0; c0 < n_cols; c0 += 32) {
                    uint32_t v[2][16];
                    tmem_ld16_async(t_addr + (uint32_t)c0, v[0]);
                    tmem_ld16_async(t_addr + (uint32_t)(c0 + 16), v[1]);
                    tmem_ld_wait();
                    // even lanes hold gate features, odd lanes the matching up features: per pair of token
                    // columns the even lane finishes the first and the odd lane the second
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int j = 0; j < 16; j += 2) {
                            const float m0 = __uint_as_float(v[h][j]), m1 = __uint_as_float(v[h][j + 1]);
                            const float got = __shfl_xor_sync(0xffffffffu, odd ? m0 : m1, 1);
                            const float gate = odd ? got : m0, up = odd ? m1 : got;
                            const int col = c0 + 16 * h + j + (odd ? 1 : 0);
                            if (row_ok && col < n_cols)
                                arow[(size_t)col * half_rows] = __ushort_as_half(
                                    (unsigned short)float_to_f16_bits(__fdividef(gate, 1.f + __expf(-gate)) * up));
                        }
                }
            } else {
                float* dst = p.out + (size_t)col0 * p.rows + row;
#pragma unroll 1
                for (int c0 = 0; c0 < n_cols; c0 += 16) {
                    uint32_t v[16];
                    float old[16];
                    tmem_ld16_async(t_addr + (uint32_t)c0, v);
                    float* d0 = dst + (size_t)c0 * p.rows;
                    if (EPI == PF_EPI_ADD) {
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            old[j] = (row_ok && c0 + j < n_cols) ? d0[(size_t)j * p.rows] : 0.f;
                    }
                    tmem_ld_wait();
                    if (row_ok) {
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (c0 + j < n_cols)
                                d0[(size_t)j * p.rows] = EPI == PF_EPI_ADD ? old[j] + __uint_as_float(v[j]) : __uint_as_float(v[j]);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&acc_empty[a]));
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, TMEM_COLS);
}

// y (+)= X W^T for T token rows.  W: the caller's bf16 matrix, registered (its fp16 tile-major copy is read).
template <int EPI>
inline int pf_gemm(TcState& tc, const __nv_bfloat16* W, int rows, int K, const __half* X, int T, float* out, __half* act,
                   int* status, cudaStream_t st, int64_t* launches) {
    auto it = tc.weights.find(W);
    if (it == tc.weights.end() || !it->second.resident || it->second.rows != rows || it->second.K != K)
        return SPIRAL_ERR_UNSUPPORTED;
    const CUtensorMap* xm = nullptr;
    int rc = tc_get_xmap(tc, X, K, T, PF_BN, &xm);
    if (rc) return rc;
    PfGemmParams p{};
    p.row_tiles = (rows + TC_BM - 1) / TC_BM;
    p.tok_tiles = (T + PF_BN - 1) / PF_BN;
    p.KB = (K + TC_BK - 1) / TC_BK;
    p.rows = rows; p.T = T; p.out = out; p.act = act; p.status = status;
    // re-read the smaller operand: weights rows x K, activations T x K
    p.row_fastest = (T > rows && p.row_tiles <= tc.n_sm) ? 1 : 0;
    const int grid = std::min(tc.n_sm, p.row_tiles * p.tok_tiles);
    TC_TRY(launch_kernel(true, pf_gemm_kernel<EPI>, dim3(grid), dim3(PF_THREADS), PF_SMEM, st, it->second.map, *xm, p));
    if (launches) ++*launches;
    return SPIRAL_OK;
}

inline int pf_gemm_setup() {
    TC_TRY(cudaFuncSetAttribute(pf_gemm_kernel<PF_EPI_STORE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PF_SMEM));
    TC_TRY(cudaFuncSetAttribute(pf_gemm_kernel<PF_EPI_ADD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PF_SMEM));
    TC_TRY(cudaFuncSetAttribute(pf_gemm_kernel<PF_EPI_SILU>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PF_SMEM));
    return SPIRAL_OK;
}

// ------------------------------------------------------------------------------------------------
// element-wise kernels over thousands of token rows (the decode step's versions are built for a
// few hundred rows at most: one CTA per row, half a warp per head)
// ------------------------------------------------------------------------------------------------

// h[t][:] = x[t][:] * rsqrt(mean(x[t]^2) + eps) * gain as fp16, one warp per token row: the row
// stays in registers between the reduction and the scaling, no block barrier.
constexpr int PF_RMS_MAX_V4 = 32;       // float4 per lane: d_model <= 4096
constexpr int PF_RMS_THREADS = 256;
template <int NV4>                      // float4 per lane the row needs, rounded up to a multiple of 4
__global__ void __launch_bounds__(PF_RMS_THREADS) pf_rmsnorm_kernel(const float* __restrict__ x,
                                                                    const __nv_bfloat16* __restrict__ gain, float eps,
                                                                    int d_model, int T, __half* __restrict__ h) {
    grid_dependency_sync();
    const int lane = threadIdx.x & 31;
    const int warps = (gridDim.x * blockDim.x) >> 5;
    const int nc = d_model >> 2;
    for (int t = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; t < T; t += warps) {
        const float4* xr = reinterpret_cast<const float4*>(x + (size_t)t * d_model);
        float4 v[NV4];
        float ss = 0.f;
#pragma unroll
        for (int k = 0; k < NV4; ++k) {
            const int c = lane + 32 * k;
            v[k] = c < nc ? __ldcs(xr + c) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int k = 0; k < NV4; ++k) ss += v[k].x * v[k].x + v[k].y * v[k].y + v[k].z * v[k].z + v[k].w * v[k].w;
        ss = warp_sum(ss);
        const float inv = rsqrtf(ss / (float)d_model + eps);
        __half* hr = h + (size_t)t * d_model;
#pragma unroll
        for (int k = 0; k < NV4; ++k) {
            const int c = lane + 32 * k;
            if (c < nc) {
                const uint2 g = __ldg(reinterpret_cast<const uint2*>(gain + 4 * c));
                uint2 o;
                o.x = pack_f16(v[k].x * inv * bf16_lo(g.x), v[k].y * inv * bf16_hi(g.x));
                o.y = pack_f16(v[k].z * inv * bf16_lo(g.y), v[k].w * inv * bf16_hi(g.y));
                *reinterpret_cast<uint2*>(hr + 4 * c) = o;
            }
        }
    }
}

// One warp per (token row, head) of the QKV projection y [T][(Hq + 2 Hkv) * HD] (fp32): bias, per-head
// RMSNorm of q and k, rotate-half RoPE at the token's position; then q -> fp16 [T][Hq][HD] already
// multiplied by log2(e) / sqrt(HD) (the attention kernel works in the exp2 domain), k and v -> the
// token's slot in its page, rounded once to fp16.  Lane l holds elements {E l .. E l + E - 1} and
// their rotation partners HD/2 further on (E = HD / 64).
constexpr int PF_QKV_THREADS = 256;
template <int HD>
__global__ void __launch_bounds__(PF_QKV_THREADS) pf_qkv_post_kernel(
    const float* __restrict__ y, const __nv_bfloat16* __restrict__ bias, const __nv_bfloat16* __restrict__ q_gain,
    const __nv_bfloat16* __restrict__ k_gain, float eps, const float* __restrict__ cos_tab,
    const float* __restrict__ sin_tab, const int32_t* __restrict__ game, const int32_t* __restrict__ pos_of,
    const int32_t* __restrict__ block_table, int max_pages, int n_pages, int layer, int T, int n_q_heads,
    int n_kv_heads, float q_scale, __half* __restrict__ q_out, uint16_t* __restrict__ pool, int* status) {
    constexpr int E = HD / 64, HALF = HD / 2;
    grid_dependency_sync();
    const int lane = threadIdx.x & 31;
    const int warps = (gridDim.x * blockDim.x) >> 5;
    const int n_heads = n_q_heads + 2 * n_kv_heads;
    const int ld = n_heads * HD;
    const long long total = (long long)T * n_heads;
    for (long long task = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; task < total; task += warps) {
        const int t = (int)(task / n_heads), head = (int)(task - (long long)t * n_heads);
        const float* yr = y + (size_t)t * ld + head * HD + E * lane;
        float lo[E], hi[E];
        if (E == 2) {
            const float2 a = __ldcs(reinterpret_cast<const float2*>(yr));
            const float2 b = __ldcs(reinterpret_cast<const float2*>(yr + HALF));
            lo[0] = a.x; lo[E - 1] = a.y; hi[0] = b.x; hi[E - 1] = b.y;
        } else {
            lo[0] = __ldcs(yr); hi[0] = __ldcs(yr + HALF);
        }
        const bool is_q = head < n_q_heads, is_k = !is_q && head < n_q_heads + n_kv_heads;
        const int pos = pos_of[t];
        if (bias) {
#pragma unroll
            for (int e = 0; e < E; ++e) {
                lo[e] += __bfloat162float(bias[head * HD + E * lane + e]);
                hi[e] += __bfloat162float(bias[head * HD + E * lane + e + HALF]);
            }
        }
        if (is_q || is_k) {
            const __nv_bfloat16* gain = is_q ? q_gain : k_gain;
            if (gain) {
                float ss = 0.f;
#pragma unroll
                for (int e = 0; e < E; ++e) ss += lo[e] * lo[e] + hi[e] * hi[e];
                ss = warp_sum(ss);
                const float inv = rsqrtf(ss / (float)HD + eps);
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    lo[e] = lo[e] * inv * __bfloat162float(gain[E * lane + e]);
                    hi[e] = hi[e] * inv * __bfloat162float(gain[E * lane + e + HALF]);
                }
            }
#pragma unroll
            for (int e = 0; e < E; ++e) {
                const float cs = __ldg(cos_tab + (size_t)pos * HALF + E * lane + e);
                const float sn = __ldg(sin_tab + (size_t)pos * HALF + E * lane + e);
                const float a = lo[e], b = hi[e];
                lo[e] = a * cs - b * sn;
                hi[e] = b * cs + a * sn;
            }
        }
        if (is_q) {
            __half* q = q_out + ((size_t)t * n_q_heads + head) * HD + E * lane;
            if (E == 2) {
                *reinterpret_cast<uint32_t*>(q) = pack_f16(lo[0] * q_scale, lo[E - 1] * q_scale);
                *reinterpret_cast<uint32_t*>(q + HALF) = pack_f16(hi[0] * q_scale, hi[E - 1] * q_scale);
            } else {
                q[0] = __ushort_as_half((unsigned short)float_to_f16_bits(lo[0] * q_scale));
                q[HALF] = __ushort_as_half((unsigned short)float_to_f16_bits(hi[0] * q_scale));
            }
            continue;
        }
        const int kvh = is_k ? head - n_q_heads : head - n_q_heads - n_kv_heads;
        const int page = __ldg(block_table + (size_t)game[t] * max_pages + pos / ATTN_PAGE);
        if (page < 0 || page >= n_pages) {
            if (lane == 0) record_status(status, STATUS_BAD_PAGE);
            continue;
        }
        uint16_t* dst = pool + kv_block_offset(layer, page, kvh, n_pages, n_kv_heads, ATTN_PAGE, HD) +
                        (is_k ? 0 : (size_t)ATTN_PAGE * HD) + (size_t)(pos % ATTN_PAGE) * HD + E * lane;
        if (E == 2) {
            *reinterpret_cast<uint32_t*>(dst) = pack_f16(lo[0], lo[E - 1]);
            *reinterpret_cast<uint32_t*>(dst + HALF) = pack_f16(hi[0], hi[E - 1]);
        } else {
            dst[0] = (uint16_t)float_to_f16_bits(lo[0]);
            dst[HALF] = (uint16_t)float_to_f16_bits(hi[0]);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// causal append attention
// ------------------------------------------------------------------------------------------------
constexpr int APP_ROWS = 176;              // query rows (position x head of the KV group) per CTA: 11 consumer warps +
                                           // the producer warp = three warps per scheduler, the register file's limit at
                                           // the ~168 registers the consumers need
constexpr int APP_CWARPS = APP_ROWS / 16;  // consumer warps; one more warp issues the TMA loads
constexpr int APP_THREADS = (APP_CWARPS + 1) * 32;
constexpr int APP_BLK_PAGES = 4;           // pages (16 keys each) per ring stage
constexpr int APP_STAGES = 4;

// One block of consecutive new positions of one game: queries at positions pos0 .. pos0 + n_pos - 1
// (rows row0 .. of the chunk's q / output buffers); kv_len = positions of the game whose keys and
// values have been written (everything beyond is stale pool memory).
struct AppendItem { int game, pos0, n_pos, row0, kv_len, pad0, pad1, pad2; };

struct AppendParams {
    const __half* q;                // [T][n_q_heads][head_dim] fp16: normalised, rotated, times log2(e)/sqrt(head_dim)
    const AppendItem* items;
    const int32_t* block_table;     // [max_games][max_pages]
    int max_pages, n_pages, layer, n_q_heads, n_kv_heads, group;
    __half* out;                    // [T][n_q_heads * head_dim]
    int* status;
};

inline int app_positions_per_item(int group) { return APP_ROWS / group; }
__device__ __forceinline__ uint32_t pack_unit_f16(float lo, float hi) {
    const __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}
inline size_t app_smem_bytes(int head_dim) {
    return (size_t)APP_STAGES * APP_BLK_PAGES * (head_dim / 64) * 4096 + 1024;
}

template <int HD>
__global__ void __launch_bounds__(APP_THREADS, 1) attn_append_kernel(const __grid_constant__ CUtensorMap tmKV,
                                                                     AppendParams p) {
    constexpr int HALVES = HD / 64;
    constexpr int PAGE_BYTES = HALVES * 4096;          // 16 K rows + 16 V rows of one (page, head), 128-byte rows
    constexpr int STAGE_BYTES = APP_BLK_PAGES * PAGE_BYTES;
    constexpr int KSTEPS = HD / 16;
    constexpr int NT = HD / 8;
    extern __shared__ uint8_t app_smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[APP_STAGES], empty_bar[APP_STAGES];
    __shared__ int abort_sm;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    grid_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < APP_STAGES; ++s) { mbar_init(smem_u32(&full_bar[s]), 1); mbar_init(smem_u32(&empty_bar[s]), APP_CWARPS); }
        abort_sm = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tmap_prefetch(&tmKV);
    }
    __syncthreads();
    volatile int* abort_flag = &abort_sm;
    grid_dependency_wait();            // items, queries and the new keys/values come from earlier kernels / copies

    const AppendItem item = p.items[blockIdx.x];
    const int kvh = blockIdx.y;
    const int G = p.group;
    const int last_pos = item.pos0 + item.n_pos - 1;
    const int n_pg = last_pos / ATTN_PAGE + 1;                         // pages holding keys 0 .. last_pos
    const int n_blk = (n_pg + APP_BLK_PAGES - 1) / APP_BLK_PAGES;
    const uint32_t ring = (smem_u32(app_smem_raw) + 1023u) & ~1023u;

    if (warp == APP_CWARPS) {
        // ---------------- TMA producer (one warp: lanes look page ids up, lane 0 issues) ----------------
        int my_page = 0;
        for (int j = 0; j < n_blk; ++j) {
            if ((j & 7) == 0) {          // page ids of the next eight blocks, one per lane
                const int pg = APP_BLK_PAGES * j + lane;
                my_page = 0;
                if (pg < n_pg) {
                    my_page = __ldcg(p.block_table + (size_t)item.game * p.max_pages + pg);
                    if (my_page < 0 || my_page >= p.n_pages) {
                        record_status(p.status, STATUS_BAD_PAGE);
                        my_page = 0;
                    }
                }
            }
            const int s = j % APP_STAGES;
            bool ok = true;
            if (j >= APP_STAGES && lane == 0)
                ok = mbar_wait(smem_u32(&empty_bar[s]), (uint32_t)((j / APP_STAGES) - 1) & 1u, abort_flag, p.status,
                               STATUS_TIMEOUT_MMA);
            if (!__shfl_sync(0xffffffffu, ok ? 1 : 0, 0)) break;
            const int npg = min(APP_BLK_PAGES, n_pg - APP_BLK_PAGES * j);
            if (lane == 0) mbar_expect_tx(smem_u32(&full_bar[s]), (uint32_t)(npg * PAGE_BYTES));
#pragma unroll
            for (int k = 0; k < APP_BLK_PAGES; ++k) {
                const int page = __shfl_sync(0xffffffffu, my_page, (j & 7) * APP_BLK_PAGES + k);
                if (lane == 0 && k < npg) {
                    const int y = (((p.layer * p.n_pages + page) * p.n_kv_heads) + kvh) * 32;
#pragma unroll
                    for (int h = 0; h < HALVES; ++h)
                        tma_load_2d_nohint(ring + (uint32_t)(s * STAGE_BYTES + k * PAGE_BYTES + h * 4096), &tmKV, 64 * h, y,
                                           smem_u32(&full_bar[s]));
                }
            }
        }
        // every load issued is waited for by the consumers unless they gave up: then give the copies a bounded time
        if (*abort_flag && lane == 0) {
            for (int s = 0; s < APP_STAGES; ++s) {
                unsigned long long t0 = global_ns();
                while (!mbar_try(smem_u32(&full_bar[s]), 0) && !mbar_try(smem_u32(&full_bar[s]), 1) &&
                       global_ns() - t0 < TMA_WAIT_NS) {}
            }
        }
        return;
    }

    // ---------------- consumers: warp w owns query rows 16 w .. 16 w + 15 ----------------
    const int g = lane >> 2, c = lane & 3;
    const int r0 = 16 * warp + g, r1 = r0 + 8;                   // this thread's two rows
    const int po0 = r0 / G, hh0 = r0 - po0 * G;                  // position offset and head within the group
    const int po1 = r1 / G, hh1 = r1 - po1 * G;
    const bool ok0 = po0 < item.n_pos, ok1 = po1 < item.n_pos;
    const int pos_r0 = item.pos0 + (ok0 ? po0 : 0), pos_r1 = item.pos0 + (ok1 ? po1 : 0);

    uint32_t qa[KSTEPS][4];
    {
        const __half* q0 = p.q + ((size_t)(item.row0 + (ok0 ? po0 : 0)) * p.n_q_heads + kvh * G + hh0) * HD + 2 * c;
        const __half* q1 = p.q + ((size_t)(item.row0 + (ok1 ? po1 : 0)) * p.n_q_heads + kvh * G + hh1) * HD + 2 * c;
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
            qa[ks][0] = __ldcg(reinterpret_cast<const uint32_t*>(q0 + 16 * ks));
            qa[ks][1] = __ldcg(reinterpret_cast<const uint32_t*>(q1 + 16 * ks));
            qa[ks][2] = __ldcg(reinterpret_cast<const uint32_t*>(q0 + 16 * ks + 8));
            qa[ks][3] = __ldcg(reinterpret_cast<const uint32_t*>(q1 + 16 * ks + 8));
        }
    }
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    float o[NT][4];
#pragma unroll
    for (int t = 0; t < NT; ++t) { o[t][0] = 0.f; o[t][1] = 0.f; o[t][2] = 0.f; o[t][3] = 0.f; }

    const int lr = lane & 7, lm = lane >> 3;
    const int k_tok = lr + 8 * (lm >> 1), k_chk = lm & 1;
    const int v_tok = lr + 8 * (lm & 1), v_chk = lm >> 1;
    const uint32_t k_row_off = (uint32_t)(k_tok * 128), v_row_off = (uint32_t)((16 + v_tok) * 128);

    for (int j = 0; j < n_blk; ++j) {
        const int s = j % APP_STAGES;
        const uint32_t base = ring + (uint32_t)(s * STAGE_BYTES);
        const bool landed = mbar_wait(smem_u32(&full_bar[s]), (uint32_t)(j / APP_STAGES) & 1u, abort_flag, p.status,
                                      STATUS_TIMEOUT_TMA);
        if (!__all_sync(0xffffffffu, landed)) break;
        const int npg = min(APP_BLK_PAGES, n_pg - APP_BLK_PAGES * j);
        const int key0 = j * APP_BLK_PAGES * ATTN_PAGE;
        // value rows of positions not written yet hold stale pool bytes (possibly NaN patterns): the
        // weights there are exactly zero, but 0 * NaN is not -- zero those rows (last page only).  Every
        // warp zeroes all of them itself before it reads any: the warps then need no barrier between
        // them (they store the same zeros), and this stage is not refilled afterwards.
        if (j == n_blk - 1 && item.kv_len < n_pg * ATTN_PAGE) {
            const int valid = item.kv_len - (n_pg - 1) * ATTN_PAGE;            // 1 .. 15 rows of the last page exist
            const uint32_t pbase = base + (uint32_t)((npg - 1) * PAGE_BYTES);
            for (int idx = lane; idx < (ATTN_PAGE - valid) * 8 * HALVES; idx += 32) {
                const int r = valid + idx / (8 * HALVES), rem = idx % (8 * HALVES);
                asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(pbase + (rem >> 3) * 4096 + (16 + r) * 128 +
                                                                           (rem & 7) * 16), "r"(0u) : "memory");
            }
            __syncwarp();
        }
        // ---- scores S[16 rows x 64 keys] = Q K^T (already in the log2 domain: q carries the scale) ----
        float sc[2 * APP_BLK_PAGES][4];
#pragma unroll
        for (int t = 0; t < 2 * APP_BLK_PAGES; ++t) { sc[t][0] = 0.f; sc[t][1] = 0.f; sc[t][2] = 0.f; sc[t][3] = 0.f; }
#pragma unroll
        for (int pgi = 0; pgi < APP_BLK_PAGES; ++pgi) {
            if (pgi < npg) {
                const uint32_t pb = base + (uint32_t)(pgi * PAGE_BYTES);
#pragma unroll
                for (int ks = 0; ks < KSTEPS; ++ks) {
                    const int h = ks >> 2, ch = 2 * (ks & 3) + k_chk;
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4(pb + h * 4096 + k_row_off + (uint32_t)(((ch ^ (k_tok & 7)) << 4)), b0, b1, b2, b3);
                    mma_16816<true>(sc[2 * pgi], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b0, b1);
                    mma_16816<true>(sc[2 * pgi + 1], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b2, b3);
                }
            }
        }
        // causal mask: the row at position P sees keys 0 .. P (also hides pages that were not loaded)
        if (key0 + APP_BLK_PAGES * ATTN_PAGE - 1 > item.pos0) {
#pragma unroll
            for (int t = 0; t < 2 * APP_BLK_PAGES; ++t)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int key = key0 + 8 * t + 2 * c + e;
                    if (key > pos_r0) sc[t][e] = -INFINITY;
                    if (key > pos_r1) sc[t][2 + e] = -INFINITY;
                }
        }
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int t = 0; t < 2 * APP_BLK_PAGES; ++t) {
            mx0 = fmaxf(mx0, fmaxf(sc[t][0], sc[t][1]));
            mx1 = fmaxf(mx1, fmaxf(sc[t][2], sc[t][3]));
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        // key 0 is visible to every row and lies in the first block: the running maxima are finite from there on
        const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
        const float al0 = fast_exp2(m0 - mn0), al1 = fast_exp2(m1 - mn1);
        float rs0 = 0.f, rs1 = 0.f;
#pragma unroll
        for (int t = 0; t < 2 * APP_BLK_PAGES; ++t) {
            sc[t][0] = fast_exp2(sc[t][0] - mn0); sc[t][1] = fast_exp2(sc[t][1] - mn0);
            sc[t][2] = fast_exp2(sc[t][2] - mn1); sc[t][3] = fast_exp2(sc[t][3] - mn1);
            rs0 += sc[t][0] + sc[t][1];
            rs1 += sc[t][2] + sc[t][3];
        }
        l0 = l0 * al0 + rs0;
        l1 = l1 * al1 + rs1;
        if (__any_sync(0xffffffffu, mn0 > m0 || mn1 > m1)) {      // a running maximum moved: rescale the accumulators
#pragma unroll
            for (int t = 0; t < NT; ++t) { o[t][0] *= al0; o[t][1] *= al0; o[t][2] *= al1; o[t][3] *= al1; }
        }
        m0 = mn0; m1 = mn1;
        // ---- O[16 x HD] += P[16 x 64 keys] V ----
#pragma unroll
        for (int pgi = 0; pgi < APP_BLK_PAGES; ++pgi) {
            if (pgi < npg) {
                const uint32_t pb = base + (uint32_t)(pgi * PAGE_BYTES);
                // weights lie in [0, 1]: plain round-to-nearest conversion, no saturation needed
                const uint32_t a0 = pack_unit_f16(sc[2 * pgi][0], sc[2 * pgi][1]), a1 = pack_unit_f16(sc[2 * pgi][2], sc[2 * pgi][3]);
                const uint32_t a2 = pack_unit_f16(sc[2 * pgi + 1][0], sc[2 * pgi + 1][1]);
                const uint32_t a3 = pack_unit_f16(sc[2 * pgi + 1][2], sc[2 * pgi + 1][3]);
#pragma unroll
                for (int np = 0; np < NT / 2; ++np) {
                    const int h = np >> 2, ch = 2 * (np & 3) + v_chk;
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4_trans(pb + h * 4096 + v_row_off + (uint32_t)(((ch ^ (v_tok & 7)) << 4)), b0, b1, b2, b3);
                    mma_16816<true>(o[2 * np], a0, a1, a2, a3, b0, b1);
                    mma_16816<true>(o[2 * np + 1], a0, a1, a2, a3, b2, b3);
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&empty_bar[s]));
    }
    if (*abort_flag) return;
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    const float i0 = 1.f / l0, i1 = 1.f / l1;
    __half* o0 = p.out + ((size_t)(item.row0 + po0) * p.n_q_heads + kvh * G + hh0) * HD + 2 * c;
    __half* o1 = p.out + ((size_t)(item.row0 + po1) * p.n_q_heads + kvh * G + hh1) * HD + 2 * c;
#pragma unroll
    for (int t = 0; t < NT; ++t) {
        if (ok0) *reinterpret_cast<uint32_t*>(o0 + 8 * t) = pack_f16(o[t][0] * i0, o[t][1] * i0);
        if (ok1) *reinterpret_cast<uint32_t*>(o1 + 8 * t) = pack_f16(o[t][2] * i1, o[t][3] * i1);
    }
}

// ------------------------------------------------------------------------------------------------
// the same attention on the 5th-generation tensor cores
// ------------------------------------------------------------------------------------------------
// One CTA per (query block, KV head).  The block's query rows (positions x heads of the group) form
// two tiles of 128 rows = 128 TMEM lanes each, which share the keys and values streamed through
// shared memory.  Per block of 64 keys (4 pages) and tile:
//     S = Q K^T      tcgen05.mma M128 N64, Q and K K-major in shared memory        -> TMEM (two S buffers per tile)
//     P = 2^(S - m)  softmax warps, one thread per row (no shuffles), fp16          -> shared memory
//     O += P V       tcgen05.mma M128 N=HD, V as stored ([key][head_dim]: MN-major B), accumulated in TMEM
// m is the row maximum in use; it is only raised (and the row of O in TMEM and the running sum
// rescaled) when a block's maximum exceeds it by more than 2^8, so that P stays within fp16 range and
// the rescaling -- a read-modify-write of tensor memory -- is rare after the first blocks.
// Warp 0 streams K and V pages through a four-stage TMA ring (separate 16-row boxes so that the keys of
// a block are contiguous rows), warps 1 and 10 issue the MMAs of tile 0 and 1 (S of block j+1 is
// computed while the softmax of block j runs), warps 2..5 / 6..9 are the softmax threads of tile 0 / 1.
constexpr int APT_BN = 64;                       // keys per block
constexpr int APT_PAGES = APT_BN / ATTN_PAGE;
// TILES = 2: one CTA per SM holds two query tiles that share the streamed keys and values (four K/V stages).
// TILES = 1: one query tile per CTA, two CTAs per SM (two stages each): the keys and values are fetched
// once per tile, but one CTA's prologue and epilogue run under the other's main loop.
__host__ __device__ constexpr int apt_stages(int tiles) { return tiles == 1 ? 2 : 4; }
__host__ __device__ constexpr int apt_threads(int tiles) { return tiles == 1 ? 192 : 352; }   // TMA warp, MMA warp (tile 0), 4 softmax warps per
                                                                          // tile, and for two tiles the MMA warp of tile 1
constexpr uint32_t APT_QSLAB = 128 * 128;        // 128 query rows of 128 bytes: one 64-element slab of a Q tile / one P tile
constexpr uint32_t APT_KSLAB = APT_BN * 128;     // 64 key rows of 128 bytes: one 64-element slab of a K or V tile
constexpr float APT_RESCALE_LOG2 = 8.f;
// Q tiles, P tiles, the K + V stages, and the slack to reach a 1024-byte boundary.  Two one-tile CTAs of
// head_dim 128 fill an SM to the byte (2 x (112 KB of tiles + 1 KB reserved + the barriers)): their slack is
// what is left, 864 bytes, which suffices where the dynamic region starts 160 bytes past a 1024-byte
// boundary, as it does behind the kernel's static shared memory; the kernel checks and refuses otherwise.
inline size_t apt_smem_bytes(int head_dim, int tiles) {
    const size_t slabs = head_dim / 64;
    return tiles * slabs * APT_QSLAB + tiles * APT_QSLAB + apt_stages(tiles) * 2 * slabs * APT_KSLAB +
           (tiles == 1 && head_dim == 128 ? 864 : 1024);
}
inline int apt_positions_per_item(int group, int tiles) { return tiles * (128 / group); }

// Shared-memory descriptor of an MN-major operand tile with the 128-byte swizzle: rows are k (here: keys)
// of 128 bytes = 64 elements of the N dimension; 8-row groups are `sbo` bytes apart, the next 64 elements
// of N start `lbo` bytes further on.
__device__ __forceinline__ uint64_t smem_desc_sw128_mn(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3ffffu) >> 4);
    d |= (uint64_t)(lbo >> 4) << 16;
    d |= (uint64_t)(sbo >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// 16 consecutive fp32 columns of this warp's 32 TMEM lanes, written from registers
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Timing probe builds (-DAPT_PROBE) only: clock cycles one softmax warp of every CTA's first tile spends in each
// phase of a key block, summed over the launch.
#ifdef APT_PROBE
__device__ unsigned long long g_apt_probe[16];
#define APT_STAMP(i)                                                                         \
    do {                                                                                     \
        if (probe_on) {                                                                      \
            const long long now__ = clock64();                                               \
            atomicAdd(&g_apt_probe[i], (unsigned long long)(now__ - probe_t));               \
            probe_t = now__;                                                                 \
        }                                                                                    \
    } while (0)
#else
#define APT_STAMP(i) do { } while (0)
#endif

template <int HD, int TILES>
__global__ void __launch_bounds__(apt_threads(TILES), TILES == 1 ? 2 : 1) attn_append_tc_kernel(const __grid_constant__ CUtensorMap tmKV16,
                                                                        AppendParams p) {
    constexpr int SLABS = HD / 64;
    constexpr uint32_t Q_TILE = SLABS * APT_QSLAB, P_TILE = APT_QSLAB, KV_BYTES = SLABS * APT_KSLAB;
    constexpr uint32_t STAGE_BYTES = 2 * KV_BYTES;
    constexpr int APT_STAGES = apt_stages(TILES), APT_THREADS = apt_threads(TILES);
    constexpr uint32_t TM_O = 2 * TILES * APT_BN;          // S: (2 tile + buffer) * 64 columns; O: TM_O + tile * HD
    constexpr uint32_t TM_COLS = TILES == 1 ? 256 : 512;
    constexpr uint32_t PAGE_ROWS_BYTES = ATTN_PAGE * 128;  // 16 rows of 128 bytes
    extern __shared__ uint8_t apt_smem_raw[];
    __shared__ __align__(8) uint64_t q_ready, kv_full[APT_STAGES], kv_empty[APT_STAGES], s_full[2][2], s_empty[2][2],
        p_full[2], p_empty[2], o_full[2];
    __shared__ uint32_t tmem_base_sm;
    __shared__ int abort_sm;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    grid_launch_dependents();
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&q_ready), 4 * TILES);
        for (int s = 0; s < APT_STAGES; ++s) { mbar_init(smem_u32(&kv_full[s]), 1); mbar_init(smem_u32(&kv_empty[s]), TILES); }
        for (int t = 0; t < 2; ++t) {
            for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&s_full[t][b]), 1); mbar_init(smem_u32(&s_empty[t][b]), 4); }
            mbar_init(smem_u32(&p_full[t]), 4); mbar_init(smem_u32(&p_empty[t]), 1); mbar_init(smem_u32(&o_full[t]), 1);
        }
        abort_sm = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tmap_prefetch(&tmKV16);
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_sm), TM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_sm;
    volatile int* abort_flag = &abort_sm;
    grid_dependency_wait();            // items, queries and the new keys/values come from earlier kernels / copies

    const AppendItem item = p.items[blockIdx.x];
    const int kvh = blockIdx.y;
    const int G = p.group;
    const int PT = 128 / G;                                       // positions per tile
    const int n_tiles = (TILES == 2 && item.n_pos > PT) ? 2 : 1;  // a second tile without rows to compute stays idle
    const int last_pos = item.pos0 + item.n_pos - 1;
    const int n_pg = last_pos / ATTN_PAGE + 1;
    const int n_blk = (n_pg + APT_PAGES - 1) / APT_PAGES;
    const uint32_t base = (smem_u32(apt_smem_raw) + 1023u) & ~1023u;
    const uint32_t q_base = base, p_base = base + TILES * Q_TILE, ring = base + TILES * Q_TILE + TILES * P_TILE;
    {
        uint32_t dyn_bytes;
        asm volatile("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn_bytes));
        if (ring + APT_STAGES * STAGE_BYTES > smem_u32(apt_smem_raw) + dyn_bytes) {       // CTA-uniform
            if (threadIdx.x == 0) record_status(p.status, STATUS_BAD_SMEM);
            tc_fence_before();
            __syncthreads();
            if (warp == 1) tmem_dealloc(tmem_base, TM_COLS);
            return;
        }
    }

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        int my_page = 0;
        for (int j = 0; j < n_blk; ++j) {
            if ((j & 7) == 0) {          // page ids of the next eight blocks, one per lane
                const int pg = APT_PAGES * j + lane;
                my_page = 0;
                if (pg < n_pg) {
                    my_page = __ldcg(p.block_table + (size_t)item.game * p.max_pages + pg);
                    if (my_page < 0 || my_page >= p.n_pages) {
                        record_status(p.status, STATUS_BAD_PAGE);
                        my_page = 0;
                    }
                }
            }
            const int s = j % APT_STAGES;
            bool ok = true;
            if (j >= APT_STAGES && lane == 0)
                ok = mbar_wait(smem_u32(&kv_empty[s]), (uint32_t)((j / APT_STAGES) - 1) & 1u, abort_flag, p.status,
                               STATUS_TIMEOUT_MMA);
            if (!__shfl_sync(0xffffffffu, ok ? 1 : 0, 0)) break;
            const int npg = min(APT_PAGES, n_pg - APT_PAGES * j);
            const uint32_t stage = ring + (uint32_t)s * STAGE_BYTES;
            if (lane == 0) mbar_expect_tx(smem_u32(&kv_full[s]), (uint32_t)(npg * 2 * SLABS) * PAGE_ROWS_BYTES);
            __syncwarp();
            // lane k fetches page k of the block: its K rows and its V rows, one box per 64-element slab
            const int page = __shfl_sync(0xffffffffu, my_page, (j & 7) * APT_PAGES + (lane & (APT_PAGES - 1)));
            if (lane < npg) {
                const int y = (((p.layer * p.n_pages + page) * p.n_kv_heads) + kvh) * 32;      // K rows; V rows at y + 16
#pragma unroll
                for (int h = 0; h < SLABS; ++h) {
                    tma_load_2d_nohint(stage + h * APT_KSLAB + lane * PAGE_ROWS_BYTES, &tmKV16, 64 * h, y, smem_u32(&kv_full[s]));
                    tma_load_2d_nohint(stage + KV_BYTES + h * APT_KSLAB + lane * PAGE_ROWS_BYTES, &tmKV16, 64 * h, y + 16,
                                       smem_u32(&kv_full[s]));
                }
            }
        }
        if (*abort_flag && lane == 0) {        // the consumers gave up: bounded wait for the copies in flight
            for (int s = 0; s < APT_STAGES; ++s) {
                unsigned long long t0 = global_ns();
                while (!mbar_try(smem_u32(&kv_full[s]), 0) && !mbar_try(smem_u32(&kv_full[s]), 1) &&
                       global_ns() - t0 < TMA_WAIT_NS) {}
            }
        }
    } else if (warp == 1 || (TILES == 2 && warp == APT_THREADS / 32 - 1)) {
        // ---------------- MMA issuers: one thread per tile (issuing is serial work per thread) ----------------
        const int t = warp == 1 ? 0 : 1;
        if (lane == 0 && t < n_tiles) {
            const uint32_t idesc_qk = tc_idesc_f16(APT_BN);
            const uint32_t idesc_pv = tc_idesc_f16(HD) | (1u << 16);          // B (V) is MN-major
#ifdef APT_PROBE
            const bool probe_on = t == 0;
            long long probe_t = clock64();
#endif
            bool ok = mbar_wait(smem_u32(&q_ready), 0u, abort_flag, p.status, STATUS_TIMEOUT_EPI);
            APT_STAMP(6);           // MMA thread: wait for Q
            auto issue_qk = [&](int j) -> bool {
                const int s = j % APT_STAGES, b = j & 1;
                if (!mbar_wait(smem_u32(&kv_full[s]), (uint32_t)(j / APT_STAGES) & 1u, abort_flag, p.status, STATUS_TIMEOUT_TMA))
                    return false;
                APT_STAMP(7);       // MMA thread: wait for K/V
                if (j >= 2 && !mbar_wait(smem_u32(&s_empty[t][b]), (uint32_t)((j >> 1) - 1) & 1u, abort_flag, p.status,
                                         STATUS_TIMEOUT_EPI))
                    return false;
                APT_STAMP(8);       // MMA thread: wait for the S buffer
                tc_fence_after();
                const uint32_t kst = ring + (uint32_t)s * STAGE_BYTES;
#pragma unroll
                for (int h = 0; h < SLABS; ++h) {
                    const uint64_t da = smem_desc_sw128(q_base + (uint32_t)t * Q_TILE + h * APT_QSLAB);
                    const uint64_t db = smem_desc_sw128(kst + h * APT_KSLAB);
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        tc_mma_f16(tmem_base + (uint32_t)((2 * t + b) * APT_BN), da + (uint64_t)(2 * k), db + (uint64_t)(2 * k),
                                   idesc_qk, (h > 0 || k > 0) ? 1u : 0u);
                }
                tc_commit(smem_u32(&s_full[t][b]));
                APT_STAMP(9);       // MMA thread: issue of Q.K
                return true;
            };
            ok = ok && issue_qk(0);
            for (int j = 0; ok && j < n_blk; ++j) {
                if (j + 1 < n_blk && !issue_qk(j + 1)) break;
                const int s = j % APT_STAGES;
                const int npg = min(APT_PAGES, n_pg - APT_PAGES * j);
                const uint32_t vst = ring + (uint32_t)s * STAGE_BYTES + KV_BYTES;
                const uint64_t dv = smem_desc_sw128_mn(vst, APT_KSLAB, 1024u);
                if (!mbar_wait(smem_u32(&p_full[t]), (uint32_t)j & 1u, abort_flag, p.status, STATUS_TIMEOUT_EPI)) break;
                tc_fence_after();
                APT_STAMP(10);      // MMA thread: wait for P
                const uint64_t dp = smem_desc_sw128(p_base + (uint32_t)t * P_TILE);
                for (int ks = 0; ks < npg; ++ks)             // one page = 16 keys = one k step
                    tc_mma_f16(tmem_base + TM_O + (uint32_t)(t * HD), dp + (uint64_t)(2 * ks),
                               dv + (uint64_t)(ks * (PAGE_ROWS_BYTES >> 4)), idesc_pv, (j > 0 || ks > 0) ? 1u : 0u);
                tc_commit(smem_u32(&o_full[t]));
                tc_commit(smem_u32(&p_empty[t]));
                // the stage is free once both tiles' MMAs on it have completed (one tile: it arrives for both)
                tc_commit(smem_u32(&kv_empty[s]));
                if (TILES == 2 && n_tiles == 1) tc_commit(smem_u32(&kv_empty[s]));
                APT_STAMP(11);      // MMA thread: issue of P.V
            }
        }
    } else {
        // ---------------- softmax: thread = query row = TMEM lane of its tile ----------------
        const int t = (warp - 2) >> 2;
        const int qd = warp & 3;
        const int r = 32 * qd + lane;
        const int po_l = r / G;
        const int po = t * PT + po_l;
        const bool row_ok = po_l < PT && po < item.n_pos;
        const int pos_r = item.pos0 + (row_ok ? po : 0);
        const int tile_pos0 = item.pos0 + t * PT;                 // no row of the tile sees less than keys 0 .. tile_pos0
#ifdef APT_PROBE
        const long long probe_t0 = clock64();
#endif
        constexpr int CPR = HD / 8;                 // 16-byte chunks per row
        constexpr int RPI = 32 / CPR;               // rows one warp-wide 16-byte access covers
        {
            // the warp's 32 rows of Q into the swizzled K-major tile, RPI rows per (coalesced) load
#pragma unroll
            for (int i = 0; i < CPR; ++i) {
                const int rr = 32 * qd + i * RPI + lane / CPR, c = lane % CPR;
                const int pl = rr / G, h2 = rr - pl * G;
                const int pp = t * PT + pl;
                const bool okr = pl < PT && pp < item.n_pos;
                const uint4 v = __ldcg(reinterpret_cast<const uint4*>(
                                           p.q + ((size_t)(item.row0 + (okr ? pp : 0)) * p.n_q_heads + kvh * G + h2) * HD) + c);
                const uint32_t dst = q_base + (uint32_t)t * Q_TILE + (uint32_t)(c >> 3) * APT_QSLAB + (uint32_t)rr * 128u +
                                     (uint32_t)(((c & 7) ^ (rr & 7)) << 4);
                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(dst), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&q_ready));
        }
        if (t < n_tiles) {
#ifdef APT_PROBE
            const bool probe_on = warp == 2 && lane == 0;
            long long probe_t = probe_t0;
            APT_STAMP(12);          // softmax warp: Q row into shared memory
#endif
            float m = -INFINITY, l = 0.f;
            const uint32_t t_lane = tmem_base + ((uint32_t)(qd * 32) << 16);
            const uint32_t t_o = t_lane + TM_O + (uint32_t)(t * HD);
            int done_blocks = 0;
            for (int j = 0; j < n_blk; ++j) {
                const int b = j & 1, s = j % APT_STAGES;
                if (!mbar_wait(smem_u32(&s_full[t][b]), (uint32_t)(j >> 1) & 1u, abort_flag, p.status, STATUS_TIMEOUT_MMA)) break;
                tc_fence_after();
                APT_STAMP(0);       // wait for S
                const uint32_t t_s = t_lane + (uint32_t)((2 * t + b) * APT_BN);
                const int key0 = j * APT_BN;
                const int vis = key0 + APT_BN - 1 > tile_pos0 ? pos_r - key0 : APT_BN;      // columns 0 .. vis are visible
                uint32_t v[4][16];
#pragma unroll
                for (int h = 0; h < 4; ++h) tmem_ld16_async(t_s + (uint32_t)(16 * h), v[h]);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&s_empty[t][b]));         // the scores are in registers now
                APT_STAMP(1);       // S into registers
                // (four independent chains each for the maximum and the sum: the row is one thread's work)
                const bool all_vis = vis >= APT_BN - 1;
                float mxs[4];
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    mxs[h] = -INFINITY;
                    if (all_vis) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) mxs[h] = fmaxf(mxs[h], __uint_as_float(v[h][i]));
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            if (16 * h + i <= vis) mxs[h] = fmaxf(mxs[h], __uint_as_float(v[h][i]));
                    }
                }
                const float mx = fmaxf(fmaxf(mxs[0], mxs[1]), fmaxf(mxs[2], mxs[3]));
                if (j == 0) {
                    m = mx;                     // key 0 is visible to every row: finite
                } else {
                    const bool raise = mx > m + APT_RESCALE_LOG2;
                    if (__any_sync(0xffffffffu, raise)) {
                        // rescale this warp's rows of O: the previous block's P.V must have completed
                        if (!mbar_wait(smem_u32(&o_full[t]), (uint32_t)(j - 1) & 1u, abort_flag, p.status, STATUS_TIMEOUT_MMA))
                            break;
                        tc_fence_after();
                        const float alpha = raise ? fast_exp2(m - mx) : 1.f;
#pragma unroll 1
                        for (int c0 = 0; c0 < HD; c0 += 32) {
                            uint32_t w[2][16];
                            tmem_ld16_async(t_o + (uint32_t)c0, w[0]);
                            tmem_ld16_async(t_o + (uint32_t)(c0 + 16), w[1]);
                            tmem_ld_wait();
#pragma unroll
                            for (int h = 0; h < 2; ++h)
#pragma unroll
                                for (int i = 0; i < 16; ++i) w[h][i] = __float_as_uint(__uint_as_float(w[h][i]) * alpha);
                            tmem_st16(t_o + (uint32_t)c0, w[0]);
                            tmem_st16(t_o + (uint32_t)(c0 + 16), w[1]);
                        }
                        tmem_st_wait();
                        tc_fence_before();
                        if (raise) { l *= alpha; m = mx; }
                    }
                }
                APT_STAMP(2);       // maximum (and rescale)
                float sums[4];
                uint32_t w[4][8];               // the row of P as fp16 pairs, ready before the buffer is waited for
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    sums[h] = 0.f;
                    if (all_vis) {
#pragma unroll
                        for (int i = 0; i < 16; i += 2) {
                            const float e0 = fast_exp2(__uint_as_float(v[h][i]) - m);
                            const float e1 = fast_exp2(__uint_as_float(v[h][i + 1]) - m);
                            sums[h] += e0 + e1;
                            w[h][i >> 1] = pack_unit_f16(e0, e1);
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; i += 2) {
                            const int col = 16 * h + i;
                            const float e0 = col <= vis ? fast_exp2(__uint_as_float(v[h][i]) - m) : 0.f;
                            const float e1 = col + 1 <= vis ? fast_exp2(__uint_as_float(v[h][i + 1]) - m) : 0.f;
                            sums[h] += e0 + e1;
                            w[h][i >> 1] = pack_unit_f16(e0, e1);
                        }
                    }
                }
                const float rowsum = (sums[0] + sums[1]) + (sums[2] + sums[3]);
                APT_STAMP(3);       // exponentials
                if (j >= 1 && !mbar_wait(smem_u32(&p_empty[t]), (uint32_t)(j - 1) & 1u, abort_flag, p.status, STATUS_TIMEOUT_MMA))
                    break;
                APT_STAMP(4);       // wait for the P buffer
#pragma unroll
                for (int c = 0; c < 8; ++c) {           // 16-byte chunk (8 keys) of the row
                    const uint32_t dst = p_base + (uint32_t)t * P_TILE + (uint32_t)r * 128u + (uint32_t)((c ^ (r & 7)) << 4);
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(dst), "r"(w[c >> 1][4 * (c & 1)]),
                                 "r"(w[c >> 1][4 * (c & 1) + 1]), "r"(w[c >> 1][4 * (c & 1) + 2]), "r"(w[c >> 1][4 * (c & 1) + 3])
                                 : "memory");
                }
                // value rows of positions not written yet hold stale pool bytes (possibly NaN patterns): their
                // weights are exactly zero, but 0 * NaN is not -- zero them (they lie in the last page loaded).
                // Both tiles do it (the same zeros) before they release their P.V.
                if (j == n_blk - 1 && item.kv_len < n_pg * ATTN_PAGE) {
                    if (!mbar_wait(smem_u32(&kv_full[s]), (uint32_t)(j / APT_STAGES) & 1u, abort_flag, p.status, STATUS_TIMEOUT_TMA))
                        break;
                    const int npg = n_pg - APT_PAGES * j;
                    const int valid = item.kv_len - (n_pg - 1) * ATTN_PAGE;            // rows of the last page that exist
                    const uint32_t vpage = ring + (uint32_t)s * STAGE_BYTES + KV_BYTES + (uint32_t)(npg - 1) * PAGE_ROWS_BYTES;
                    if (qd == 0 && lane < ATTN_PAGE && lane >= valid) {
#pragma unroll
                        for (int h = 0; h < SLABS; ++h)
#pragma unroll
                            for (int c = 0; c < 8; ++c)
                                asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(vpage + h * APT_KSLAB + lane * 128 + c * 16),
                                             "r"(0u) : "memory");
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&p_full[t]));
                APT_STAMP(5);       // P stores, fence, arrive
                l += rowsum;
                ++done_blocks;
                if (*abort_flag) break;
            }
            if (done_blocks == n_blk && !*abort_flag &&
                mbar_wait(smem_u32(&o_full[t]), (uint32_t)(n_blk - 1) & 1u, abort_flag, p.status, STATUS_TIMEOUT_MMA)) {
                tc_fence_after();
                const float inv = 1.f / l;
                const int hh = r - po_l * G;
                uint4* dst = reinterpret_cast<uint4*>(p.out + ((size_t)(item.row0 + po) * p.n_q_heads + kvh * G + hh) * HD);
#pragma unroll 1
                for (int c0 = 0; c0 < HD; c0 += 32) {
                    uint32_t w[2][16];
                    tmem_ld16_async(t_o + (uint32_t)c0, w[0]);
                    tmem_ld16_async(t_o + (uint32_t)(c0 + 16), w[1]);
                    tmem_ld_wait();
                    if (row_ok) {
#pragma unroll
                        for (int h = 0; h < 2; ++h)
#pragma unroll
                            for (int q8 = 0; q8 < 2; ++q8) {
                                uint4 o4;
                                o4.x = pack_f16(__uint_as_float(w[h][8 * q8]) * inv, __uint_as_float(w[h][8 * q8 + 1]) * inv);
                                o4.y = pack_f16(__uint_as_float(w[h][8 * q8 + 2]) * inv, __uint_as_float(w[h][8 * q8 + 3]) * inv);
                                o4.z = pack_f16(__uint_as_float(w[h][8 * q8 + 4]) * inv, __uint_as_float(w[h][8 * q8 + 5]) * inv);
                                o4.w = pack_f16(__uint_as_float(w[h][8 * q8 + 6]) * inv, __uint_as_float(w[h][8 * q8 + 7]) * inv);
                                dst[(c0 >> 3) + 2 * h + q8] = o4;
                            }
                    }
                }
                tc_fence_before();
            }
            APT_STAMP(13);          // softmax warp: wait for the last P.V, normalise, store
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, TM_COLS);
}

}  // namespace spiral
