// Weight-streaming skinny GEMM on the 5th-generation tensor cores (tcgen05, sm_100a):
//     Y[b][r] = sum_k W[r][k] * X[b][k]        W fp16 [rows][K] (a private fp16 re-encoding of the
//     caller's bf16 weights), X fp16 [n][K], fp32 accumulation in tensor memory.
// The weight matrix is the 128-row M operand ("swap-AB"), the batch is the N operand, so one CTA
// reads each weight byte exactly once and the whole batch shares it.  The op is HBM-bound for
// n <= ~200: the kernel is organised around keeping TMA loads in flight, not around the MMAs.
//
// One persistent CTA per SM, seven warps (eleven for the LM head):
//   warp 0      TMA producer: per k block a W tile [128 x 64] (one contiguous 16 KB run of the tile-major
//               fp16 copy) and an X tile [N x 64], 128-byte swizzle; a ring stage holds `bps` k blocks
//   warp 1 and  MMA issuers: four tcgen05.mma (K = 16) per k block, accumulators in TMEM (two buffers).
//   the last    One thread issuing every MMA of the CTA is the bottleneck of the main loop (0.39 us per k
//   warp        block, whatever the batch: instruction issue, not tensor-core time), so two threads in two
//               warps take alternate ring stages, each adding into an accumulator of its own ("chain");
//               the epilogue adds the two chains.  Batches above 128 leave no room in TMEM for four
//               accumulators and run with one issuer.
//   warps 2..5  epilogue: tcgen05.ld of the finished accumulator, then either fp32 partial sums
//               ("pieces") to memory -- transposed through two 16 KB shared-memory buffers and written
//               by TMA stores, 32 batch rows x 128 features at a time -- or, for the LM head,
//               (logit / T + gumbel) and a running argmax
// Work is the flattened (row tile, k block) space cut into equal contiguous ranges, one per CTA
// (stream-K): a tile whose k range spans several CTAs yields several pieces, which the consumer
// kernel adds up in a fixed order.  Every wait is bounded: on a timeout the kernel records a status
// code, all roles leave their loops, TMEM is freed and the kernel returns.
#pragma once
#include <cuda.h>
#include <cudaTypedefs.h>

#include <cstdlib>
#include <map>
#include <string>
#include <tuple>
#include <unordered_map>
#include <vector>

#include "../../include/spiral.h"
#include "common.cuh"
#include "kernels_small.cuh"
#include "tma.cuh"

namespace spiral {

constexpr int TC_BM = 128;            // weight rows per tile = MMA M
constexpr int TC_BK = 64;             // k elements per stage: one 128-byte swizzled row
// Epilogue warps: one per TMEM lane quadrant; the LM head, whose epilogue (noise, running argmax) is as long
// as a tile's mainloop at batch 128, takes two per quadrant, each handling half of the columns.
__host__ __device__ constexpr int tc_epi_warps(int mode) { return mode == 1 ? 8 : 4; }
__host__ __device__ constexpr int tc_threads(int mode) { return 64 + 32 * tc_epi_warps(mode) + 32; }   // + second issuer
constexpr int TC_MAX_STAGES = 8;
constexpr int TC_BPS = 2;             // default number of k blocks per ring stage
constexpr int TC_W_BYTES = TC_BM * TC_BK * 2;
constexpr int TC_OUT_ROWS = 32;                               // batch rows per TMA store of the pieces epilogue
constexpr int TC_OUT_BYTES = TC_OUT_ROWS * TC_BM * 4;         // one staging buffer

struct TcSeg { int tile, kb0, kb1, piece; };

struct TcParams {
    int tiles, KB;              // 128-row tiles and 64-wide k blocks of the weight matrix
    int whole_tiles;            // 1: a CTA's range is whole tiles (LM head); 0: stream-K over (tile, k block)
    int rows, n, N;             // N = n rounded up to 16 (MMA N)
    int stages, bps;            // ring depth and k blocks per stage
    int chains;                 // MMA issuers = accumulators per TMEM buffer: 2 when 4 N columns fit into TMEM, else 1
    int tma_out;                // 1: pieces leave through shared memory and TMA stores (tmOut), 0: plain stores
    int skip_x;                 // wait-timeout self-test only: the producer leaves the activation loads out, so the
                                // "stage full" barriers never complete and every role has to give up and unwind
    float* out;                 // pieces [piece][n][rows]
    size_t piece_stride;
    int* status;
    // LM head mode
    const StepArgs* args;       // noise, temperature, token and logit outputs of this call (device memory)
    unsigned long long* best;   // [256] running argmax keys, zero between launches
    unsigned int* done;         // CTAs finished, zero between launches
    float2* lse_part;           // [grid][256] per-CTA (max, sum exp) of logit/T per batch column (log-prob output)
#ifdef TC_PROBE
    unsigned long long* probe;  // [grid][8] timestamps (timing probe builds only)
#endif
};

#ifdef TC_PROBE
#define TC_STAMP(i) do { if (p.probe) p.probe[(size_t)blockIdx.x * 8 + (i)] = global_ns(); } while (0)
#else
#define TC_STAMP(i) do { } while (0)
#endif

// ------------------------------------------------------------------------------------------------
// tcgen05 wrappers (mbarrier / TMA wrappers: tma.cuh)
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem], M = 128, K = 16, fp16 inputs, fp32 accumulate
__device__ __forceinline__ void tc_mma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                           uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// the same, always accumulating (no predicate to compute)
__device__ __forceinline__ void tc_mma_f16_acc(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.eq.b32 p, 0, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc) : "memory");
}
// the mbarrier receives one arrival when every MMA issued so far by this thread has completed
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 16 consecutive fp32 columns of this warp's 32 TMEM lanes: thread = lane (row), register j = column
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(r[j]);
}
// the same without waiting: several loads may be in flight before one tmem_ld_wait()
__device__ __forceinline__ void tmem_ld16_async(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes (64 fp16) with the
// 128-byte swizzle TMA wrote: 8-row groups are 1024 bytes apart (stride byte offset), the leading
// byte offset is unused for this layout, descriptor version 1, layout type 2 = SWIZZLE_128B.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3ffffu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptor of kind::f16: D fp32, A and B fp16, both K-major, M = 128, N = n_cols
__host__ __device__ inline uint32_t tc_idesc_f16(int n_cols) {
    return (1u << 4) | ((uint32_t)(n_cols >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
}

// The work of CTA c of G: units [U c / G, U (c+1) / G) of the flattened (tile, k block) space
// (U = tiles * KB), or of the tile list (U = tiles) when ranges are whole tiles.  Pieces of a tile
// are numbered in k order: piece = c - (CTA that holds the tile's first unit).  The host plan
// (tc_get_plan) evaluates the same formulas to count the pieces per tile.
struct TcSchedule {
    long long u, u1, U;
    int KB, unit_k, G, c, whole;
    __host__ __device__ TcSchedule(int tiles, int KB_, int whole_, int c_, int G_) {
        KB = KB_; whole = whole_; c = c_; G = G_;
        unit_k = whole ? 1 : KB;
        U = whole ? (long long)tiles : (long long)tiles * KB;
        u = U * c / G;
        u1 = U * (c + 1) / G;
    }
    // pieces of tile `tile` (CTAs whose range touches it)
    __host__ __device__ int pieces_of(int tile) const {
        const long long first = (long long)tile * unit_k;
        return streamk_cta_of(first + unit_k - 1, G, U) - streamk_cta_of(first, G, U) + 1;
    }
    __host__ __device__ bool next(TcSeg& sg) {
        if (u >= u1) return false;
        const int tile = (int)(u / unit_k), off = (int)(u % unit_k);
        const long long left = u1 - u;
        const int len = (int)(left < unit_k - off ? left : unit_k - off);
        sg.tile = tile;
        sg.kb0 = whole ? 0 : off;
        sg.kb1 = whole ? KB : off + len;
        sg.piece = c - streamk_cta_of((long long)tile * unit_k, G, U);
        u += len;
        return true;
    }
};

// A CTA's work as a sequence of k blocks, tile after tile.  In the tile-major weight copy block (tile, kb) sits at
// row (tile KB + kb) 128 of the copy seen as rows of 64 elements (the TMA y coordinate).  A stream-K range starts
// somewhere inside a tile and walks k upwards: consecutive rows of the copy.  CTAs that own whole tiles (LM head)
// would all ask for the same activation block at the same time; each starts its tiles at a k block of its own
// instead (kb0 = KB c / G) and wraps around: the order of a sum changes, who computes it does not.
struct TcRun {
    int y_tile, count, kb0;         // y of the first tile's k block 0, number of blocks, first k block
    int first_tile_blocks;          // blocks of the first tile in the run (KB for whole tiles)
    __device__ TcRun(int tiles, int KB, int whole, int c, int G) {
        const TcSchedule sc(tiles, KB, whole, c, G);
        const long long b0 = whole ? sc.u * KB : sc.u, b1 = whole ? sc.u1 * KB : sc.u1;
        y_tile = (int)(b0 / KB) * KB * TC_BM;
        count = (int)(b1 - b0);
        kb0 = whole ? (int)((long long)KB * c / G) : (int)(b0 % KB);
        first_tile_blocks = whole ? KB : KB - kb0;
    }
};

// ------------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------------
// tmOut (MODE 0 with p.tma_out): the pieces buffer as a tensor [piece][batch row][feature] of floats with a
// box of 1 x 32 x 128
template <int MODE>     // 0: pieces to memory; 1: LM head with fused Gumbel-argmax
// (register cap instead of launch bounds: at 112 registers the seven warps of a layer projection fit into an SM's
// register file beside the CTA of the element-wise kernel before or after it, so that either can start early)
__global__ void __maxnreg__(MODE == 1 ? 168 : 112) tc_gemm_kernel(const __grid_constant__ CUtensorMap tmW,
                                                               const __grid_constant__ CUtensorMap tmX,
                                                               const __grid_constant__ CUtensorMap tmOut, TcParams p) {
    extern __shared__ uint8_t tc_smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[TC_MAX_STAGES], done_bar[TC_MAX_STAGES], acc_full[2], acc_empty[2];
    __shared__ uint32_t tmem_base_sm;
    __shared__ int abort_sm;
    __shared__ int last_sm;
    __shared__ unsigned long long run_sm[MODE == 1 ? 4 : 1][MODE == 1 ? 256 : 1];
    __shared__ float lse_m[MODE == 1 ? 4 : 1][MODE == 1 ? 256 : 1];    // running max / sum of exp(logit/T - max) per
    __shared__ float lse_s[MODE == 1 ? 4 : 1][MODE == 1 ? 256 : 1];    // (lane quadrant, batch column): log-prob output

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    TRACE_BEGIN(MODE == 1 ? 9 : 8);
    grid_launch_dependents();
    if (threadIdx.x == 0) TC_STAMP(0);
    // A stage holds `bps` k blocks, each a W tile [128 x 64] followed by an X tile [N x 64]: one barrier
    // round trip (stage full -> MMAs -> stage free -> next request) per stage, not per block.  The two
    // threads that run the pipeline are serial: their loops keep running counters and contain no division.
    const int S = p.stages, BPS = p.bps, N = p.N;
    const uint32_t blk_bytes = TC_W_BYTES + (uint32_t)N * 128u;
    const uint32_t stage_bytes = (uint32_t)BPS * blk_bytes;
    const uint32_t ring = (smem_u32(tc_smem_raw) + 1023u) & ~1023u;
    const uint32_t out_stage = ring + (uint32_t)S * stage_bytes;      // two staging buffers of the pieces epilogue
    const int CH = p.chains;                    // accumulator (a, c): TMEM columns (a CH + c) N .. + N
    uint32_t tmem_cols = 32;
    while (tmem_cols < 2u * (uint32_t)CH * (uint32_t)N) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(smem_u32(&full_bar[s]), 1); mbar_init(smem_u32(&done_bar[s]), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(smem_u32(&acc_full[a]), (uint32_t)CH); mbar_init(smem_u32(&acc_empty[a]), tc_epi_warps(MODE)); }
        abort_sm = 0;
        last_sm = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tmap_prefetch(&tmW);
        tmap_prefetch(&tmX);
        if (MODE == 0 && p.tma_out) tmap_prefetch(&tmOut);
    }
    if (MODE == 1)
        for (int i = threadIdx.x; i < 4 * 256; i += tc_threads(MODE)) {
            run_sm[i >> 8][i & 255] = 0ull;
            lse_m[i >> 8][i & 255] = -INFINITY;
            lse_s[i >> 8][i & 255] = 0.f;
        }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_sm), tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_sm;
    if (threadIdx.x == 0) TC_STAMP(1);
    volatile int* abort_flag = &abort_sm;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            const uint64_t pol_w = l2_policy_evict_first(), pol_x = l2_policy_evict_last();
            const TcRun run(p.tiles, p.KB, p.whole_tiles, blockIdx.x, gridDim.x);
            const int n_stages = (run.count + BPS - 1) / BPS;
            const uint32_t full0 = smem_u32(&full_bar[0]), done0 = smem_u32(&done_bar[0]);
            // Weights are written by nobody: the W tiles of the first ring-full of stages are requested
            // before the dependency wait, so that they stream in while the preceding kernel finishes.
            int w_tile = run.y_tile, w_kb = run.kb0, w_in_tile = run.first_tile_blocks;     // next W block to request
            auto next_w_row = [&]() {
                const int y = w_tile + w_kb * TC_BM;
                if (++w_kb == p.KB) w_kb = 0;
                if (--w_in_tile == 0) { w_tile += p.KB * TC_BM; w_in_tile = p.KB; }
                return y;
            };
            const int pre = n_stages < S ? n_stages : S;
            for (int st = 0, left = run.count; st < pre; ++st) {
                const int nb = left < BPS ? left : BPS;
                const uint32_t fb = full0 + 8u * (uint32_t)st, dst = ring + (uint32_t)st * stage_bytes;
                mbar_expect_tx(fb, (uint32_t)nb * blk_bytes);
                for (int b = 0; b < nb; ++b) tma_load_2d(dst + (uint32_t)b * blk_bytes, &tmW, 0, next_w_row(), fb, pol_w);
                left -= nb;
            }
            grid_dependency_wait();          // X is written by the preceding kernel
            TC_STAMP(2);
            TRACE_WAITED();
            bool ok = true;
            int x_col = run.kb0 * TC_BK, kb = run.kb0, left = run.count;
            uint32_t s = 0, ph = 0;
            int st = 0;
            for (; st < n_stages; ++st) {
                const int nb = left < BPS ? left : BPS;
                const uint32_t fb = full0 + 8u * s, dst = ring + s * stage_bytes;
                if (st >= S) {
                    if (!mbar_wait(done0 + 8u * s, ph ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_MMA)) {
                        ok = false;
                        break;
                    }
                    mbar_expect_tx(fb, (uint32_t)nb * blk_bytes);
                    for (int b = 0; b < nb; ++b) tma_load_2d(dst + (uint32_t)b * blk_bytes, &tmW, 0, next_w_row(), fb, pol_w);
                }
                for (int b = 0; b < nb; ++b) {
                    if (!p.skip_x) tma_load_2d(dst + (uint32_t)b * blk_bytes + TC_W_BYTES, &tmX, x_col, 0, fb, pol_x);
                    x_col += TC_BK;
                    if (++kb == p.KB) { kb = 0; x_col = 0; }
                }
                left -= nb;
                if (++s == (uint32_t)S) { s = 0; ph ^= 1u; }
            }
            if (!ok) {
                // copies already issued still land in this CTA's shared memory: give them a bounded
                // time to complete before the CTA may exit
                for (int back = 1; back <= S && back <= st; ++back) {
                    const int j = st - back;
                    const uint32_t sj = (uint32_t)(j % S), pj = (uint32_t)(j / S) & 1u;
                    unsigned long long t1 = global_ns();
                    while (!mbar_try(full0 + 8u * sj, pj) && global_ns() - t1 < g_wait_limit_ns) {}
                }
            }
        }
    } else if (warp == 1 || warp == 2 + tc_epi_warps(MODE)) {
        // ---------------- MMA issuers ----------------
        // Issuer `id` owns the ring stages st with st % CH == id and the accumulator chain `id` of either TMEM
        // buffer.  Both walk every stage of the CTA's run, so that both see every tile boundary: at the first block
        // of a segment (a tile, or this CTA's part of one) each waits until the epilogue has released the buffer,
        // at its last block each commits to the buffer's "full" barrier, which counts CH arrivals and therefore
        // completes when the MMAs of both chains have.  Waiting for the release also in segments an issuer adds
        // nothing to keeps it within one phase of the epilogue, which the parity waits rely on.
        const int id = warp == 1 ? 0 : 1;
        if (lane == 0 && id < CH) {
            const uint32_t idesc = tc_idesc_f16(N);
            const TcRun run(p.tiles, p.KB, p.whole_tiles, blockIdx.x, gridDim.x);
            const uint32_t full0 = smem_u32(&full_bar[0]), done0 = smem_u32(&done_bar[0]);
            const uint64_t desc0 = smem_desc_sw128(ring);
            const uint64_t d_blk = (uint64_t)(blk_bytes >> 4), d_stage = (uint64_t)(stage_bytes >> 4);
            int in_tile = run.first_tile_blocks, left = run.count;     // blocks until the tile is complete / until the end
            uint32_t s = 0, ph = 0, a = 0, aph = 0;
            uint64_t d_cur = desc0;                 // descriptor of stage s, block 0 (W tile; the X tile follows it)
            uint32_t d_tmem = tmem_base + (uint32_t)id * (uint32_t)N;   // this issuer's chain of buffer a
            int turn = 0;                           // issuer that owns the stage
            bool seg_open = false;                  // the current segment's buffer has been waited for
            bool mine_open = false;                 // this issuer's chain of it has received an MMA
            bool ok = true;
            // one k block: four MMAs, 32 bytes further along k inside the swizzle atom each
            auto issue_block = [&](uint64_t da, uint32_t first_accumulates) {
                const uint64_t db = da + (uint64_t)(TC_W_BYTES >> 4);
                tc_mma_f16(d_tmem, da, db, idesc, first_accumulates);
#pragma unroll
                for (int k = 1; k < TC_BK / 16; ++k) tc_mma_f16_acc(d_tmem, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc);
            };
            while (left > 0 && ok) {
                const int nb = left < BPS ? left : BPS;
                const bool mine = turn == id;
                // (the other issuer's stages are waited for too: a parity wait is only sound for a thread that has
                // seen every earlier phase of the barrier complete, and tiles need not land in the order requested)
                if (!mbar_wait(full0 + 8u * s, ph, abort_flag, p.status, STATUS_TIMEOUT_TMA)) break;
                if (mine) tc_fence_after();
                if (id == 0 && left == run.count) TC_STAMP(3);
                if (seg_open && nb < in_tile && nb < left) {
                    // the whole stage lies inside the open segment and does not end it (all but one or two stages
                    // of a segment): no per-block bookkeeping
                    if (mine) {
                        uint64_t da = d_cur;
                        for (int b = 0; b < nb; ++b, da += d_blk) issue_block(da, (mine_open || b > 0) ? 1u : 0u);
                        mine_open = true;
                    }
                    in_tile -= nb;
                    left -= nb;
                } else {
                    uint64_t da = d_cur;
                    for (int b = 0; b < nb; ++b, da += d_blk) {
                        if (!seg_open) {
                            if (!mbar_wait(smem_u32(&acc_empty[a]), aph ^ 1u, abort_flag, p.status, STATUS_TIMEOUT_EPI)) {
                                ok = false;
                                break;
                            }
                            tc_fence_after();
                            seg_open = true;
                        }
                        if (mine) {
                            issue_block(da, mine_open ? 1u : 0u);
                            mine_open = true;
                        }
                        --left;
                        if (--in_tile == 0 || left == 0) {        // the tile (or this CTA's part of it) is complete
                            in_tile = p.KB;
                            tc_commit(smem_u32(&acc_full[a]));
                            seg_open = false;
                            mine_open = false;
                            if ((a ^= 1u) == 0) aph ^= 1u;
                            d_tmem = tmem_base + (a * (uint32_t)CH + (uint32_t)id) * (uint32_t)N;
                            if (id == 0) TC_STAMP(4);
                        }
                    }
                    if (!ok) break;
                }
                if (mine) tc_commit(done0 + 8u * s);
                d_cur += d_stage;
                if (++s == (uint32_t)S) { s = 0; ph ^= 1u; d_cur = desc0; }
                if (++turn == CH) turn = 0;
            }
        }
    } else {
        // ---------------- epilogue (warps 2..9: TMEM lanes 32*(warp%4) .. +31; warps 2..5 take the first
        // half of the accumulator columns, warps 6..9 the second) ----------------
        const int q = warp & 3;
        const int ew = warp - 2;
        const int n_half = (((N >> 4) + 1) >> 1) << 4;                 // columns of the first half (multiple of 16)
        const int cb = tc_epi_warps(MODE) == 4 ? 0 : (ew < 4 ? 0 : n_half);   // this warp's columns
        const int ce = tc_epi_warps(MODE) == 4 ? N : (ew < 4 ? n_half : N);
        grid_dependency_wait();              // the pieces buffer may still be read by the preceding kernel
        int acc_it = 0;
        uint32_t out_it = 0;                 // staging buffers filled so far (pieces epilogue with TMA stores)
        StepArgs sa{};
        if (MODE == 1) {
            sa = *p.args;
            if (sa.defer_sampling) { sa.gumbel = nullptr; sa.tok_out = nullptr; sa.logprob = nullptr; }
        }
        const bool unit_t = sa.temperature == 1.0f;
        TcSchedule sched(p.tiles, p.KB, p.whole_tiles, blockIdx.x, gridDim.x);
        TcSeg sg;
        int blocks_before = 0;               // k blocks of this CTA's earlier segments
        for (; sched.next(sg); ++acc_it) {
            const int a = acc_it & 1;
            const uint32_t aph = (uint32_t)(acc_it >> 1) & 1u;
            // the segment's blocks sit in ring stages first_st .. last_st of the run; stage st belongs to chain
            // st % CH: a segment inside one stage has its sum in that chain alone, any other in both
            const int seg_blocks = sg.kb1 - sg.kb0;
            const int first_st = blocks_before / BPS, last_st = (blocks_before + seg_blocks - 1) / BPS;
            blocks_before += seg_blocks;
            const bool both = CH == 2 && last_st > first_st;
            if (!mbar_wait(smem_u32(&acc_full[a]), aph, abort_flag, p.status, STATUS_TIMEOUT_MMA)) break;
            tc_fence_after();
            if (threadIdx.x == 64) TC_STAMP(5);      // last segment's value survives
            const int row = sg.tile * TC_BM + q * 32 + lane;
            const bool row_ok = row < p.rows;
            const uint32_t t_buf = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(a * CH * N);
            const uint32_t t_addr = t_buf + ((CH == 2 && !both && (first_st & 1)) ? (uint32_t)N : 0u);   // the chain read first
            const uint32_t t_add = t_buf + (uint32_t)N;                                                 // the one added when both
            if (MODE == 0 && p.tma_out) {
                // lane = feature, column = batch row.  32 batch rows at a time: every thread puts its feature's 32
                // values into a [32 rows][128 features] buffer (a warp writes 128 contiguous bytes per row), one
                // thread hands the buffer to the TMA unit, which writes whole rows of the piece and leaves out what
                // lies beyond the last batch row or feature.  A buffer is refilled once the store that last used
                // it has read it.
                const uint32_t my_col = (uint32_t)(q * 32 + lane) * 4u;
                for (int c0 = 0; c0 < N && c0 < p.n; c0 += TC_OUT_ROWS, ++out_it) {
                    uint32_t v[2][16], w[2][16];
                    tmem_ld16_async(t_addr + (uint32_t)c0, v[0]);
                    if (c0 + 16 < N) tmem_ld16_async(t_addr + (uint32_t)(c0 + 16), v[1]);      // (rows beyond N are never stored)
                    if (both) {                               // the other chain's columns, added below
                        tmem_ld16_async(t_add + (uint32_t)c0, w[0]);
                        if (c0 + 16 < N) tmem_ld16_async(t_add + (uint32_t)(c0 + 16), w[1]);
                    }
                    const uint32_t buf = out_stage + (out_it & 1u) * TC_OUT_BYTES;
                    if (out_it >= 2) {
                        if (threadIdx.x == 64) tma_store_wait_read<1>();
                        asm volatile("bar.sync 1, 128;" ::: "memory");
                    }
                    tmem_ld_wait();
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const uint32_t val = both ? __float_as_uint(__fadd_rn(__uint_as_float(v[h][j]), __uint_as_float(w[h][j]))) : v[h][j];
                            asm volatile("st.shared.b32 [%0], %1;" ::"r"(buf + (uint32_t)(16 * h + j) * (TC_BM * 4u) + my_col), "r"(val) : "memory");
                        }
                    fence_proxy_async_smem();
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    if (threadIdx.x == 64) {
                        tma_store_3d(&tmOut, buf, sg.tile * TC_BM, c0, sg.piece);
                        tma_store_commit();
                    }
                }
            } else if (MODE == 0) {
                float* dst = p.out + (size_t)sg.piece * p.piece_stride + row;
                for (int c0 = cb; c0 < ce; c0 += 16) {
                    uint32_t v[16], w[16];
                    tmem_ld16_async(t_addr + (uint32_t)c0, v);
                    if (both) tmem_ld16_async(t_add + (uint32_t)c0, w);
                    tmem_ld_wait();
                    if (row_ok) {
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (c0 + j < p.n)
                                dst[(size_t)(c0 + j) * p.rows] =
                                    both ? __fadd_rn(__uint_as_float(v[j]), __uint_as_float(w[j])) : __uint_as_float(v[j]);
                    }
                }
            } else {
                for (int c0 = cb; c0 < ce; c0 += 32) {       // two 16-column loads and 32 noise loads in flight
                    uint32_t km = 0u, kw = 0u;              // column c0 + lane over this warp's 32 rows: best score, rows that have it
                    uint32_t v[2][16], w[2][16];
                    float gm[2][16];
#pragma unroll
                    for (int h = 0; h < 2; ++h)
                        if (c0 + 16 * h < ce) {
                            tmem_ld16_async(t_addr + (uint32_t)(c0 + 16 * h), v[h]);
                            if (both) tmem_ld16_async(t_add + (uint32_t)(c0 + 16 * h), w[h]);
                        }
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const int b = c0 + 16 * h + j;
                            gm[h][j] = (sa.gumbel && row_ok && b < p.n) ? __ldg(sa.gumbel + (size_t)b * p.rows + row) : 0.f;
                        }
                    tmem_ld_wait();
                    if (both) {
#pragma unroll
                        for (int h = 0; h < 2; ++h)
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                if (c0 + 16 * h < ce) v[h][j] = __float_as_uint(__fadd_rn(__uint_as_float(v[h][j]), __uint_as_float(w[h][j])));
                    }
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (c0 + 16 * h >= ce) break;
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const int b = c0 + 16 * h + j;
                            const bool ok = row_ok && b < p.n;
                            const float lg = __uint_as_float(v[h][j]);
                            if (ok && sa.logits) sa.logits[(size_t)b * p.rows + row] = lg;
                            const float z = __fadd_rn(unit_t ? lg : __fdiv_rn(lg, sa.temperature), gm[h][j]);
                            // ordered key of the score: larger float <=> larger unsigned; 0 = absent / NaN
                            uint32_t u = __float_as_uint(z);
                            u = (!ok || z != z) ? 0u : ((u & 0x80000000u) ? ~u : (u | 0x80000000u));
                            const uint32_t m = __reduce_max_sync(0xffffffffu, u);
                            const uint32_t who = __ballot_sync(0xffffffffu, u == m);
                            // lane 16 h + j keeps column b's result; keys are built and the running best in shared
                            // memory is updated once per group, by all lanes together
                            if (lane == 16 * h + j) { km = m; kw = who; }
                            if (sa.logprob) {
                                // running log-sum-exp of logit/T over the rows this warp has seen
                                const float zt = unit_t ? lg : __fdiv_rn(lg, sa.temperature);
                                uint32_t uz = __float_as_uint(zt);
                                uz = (!ok || zt != zt) ? 0u : ((uz & 0x80000000u) ? ~uz : (uz | 0x80000000u));
                                const uint32_t mz = __reduce_max_sync(0xffffffffu, uz);
                                const float mw = __uint_as_float((mz & 0x80000000u) ? (mz ^ 0x80000000u) : ~mz);
                                float e = (ok && zt == zt) ? __expf(zt - mw) : 0.f;
                                e = warp_sum(e);
                                if (lane == (b & 31) && b < p.n && mz != 0u) {
                                    const float m_old = lse_m[q][b], M = fmaxf(m_old, mw);
                                    lse_s[q][b] = lse_s[q][b] * __expf(m_old - M) + e * __expf(mw - M);
                                    lse_m[q][b] = M;
                                }
                            }
                        }
                    }
                    const int bcol = c0 + lane;
                    const int vbest = sg.tile * TC_BM + q * 32 + (__ffs(kw) - 1);       // lowest row among equals
                    const unsigned long long kcol = ((unsigned long long)km << 32) | (uint32_t)(0xffffffffu - (uint32_t)vbest);
                    if (bcol < ce && bcol < p.n && kcol > run_sm[q][bcol]) run_sm[q][bcol] = kcol;
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&acc_empty[a]));
            if (threadIdx.x == 64) TC_STAMP(6);
        }
        if (MODE == 1) {
            // fold the four warps, publish with an order-independent 64-bit max; the CTA that
            // finishes last turns the keys into tokens and re-arms the scratch for the next launch
            asm volatile("bar.sync 1, 256;" ::: "memory");
            const int t = threadIdx.x - 64;
            for (int b = t; b < p.n; b += 32 * tc_epi_warps(MODE)) {
                unsigned long long k = run_sm[0][b];
#pragma unroll
                for (int w = 1; w < 4; ++w) k = run_sm[w][b] > k ? run_sm[w][b] : k;
                if (k) atomicMax(p.best + b, k);
                if (sa.logprob) {           // this CTA's (max, sum) for column b
                    float M = lse_m[0][b];
#pragma unroll
                    for (int w = 1; w < 4; ++w) M = fmaxf(M, lse_m[w][b]);
                    float S = 0.f;
#pragma unroll
                    for (int w = 0; w < 4; ++w) S += lse_m[w][b] == -INFINITY ? 0.f : lse_s[w][b] * __expf(lse_m[w][b] - M);
                    p.lse_part[(size_t)blockIdx.x * 256 + b] = make_float2(M, S);
                }
            }
            __threadfence();
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (t == 0) last_sm = (atomicAdd(p.done, 1u) == gridDim.x - 1) ? 1 : 0;
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (last_sm) {
                __threadfence();
                for (int b = t; b < p.n; b += 32 * tc_epi_warps(MODE)) {
                    const unsigned long long k = atomicExch(p.best + b, 0ull);
                    const int tok = (int)(0xffffffffu - (uint32_t)(k & 0xffffffffull));
                    if (sa.tok_out) sa.tok_out[b] = tok;
                    if (sa.logprob) {
                        // logit/T of the winner = its score minus its noise; logsumexp from the CTAs' partials
                        const uint32_t ub = (uint32_t)(k >> 32);
                        const float zbest = __uint_as_float((ub & 0x80000000u) ? (ub ^ 0x80000000u) : ~ub);
                        const float zt = zbest - (sa.gumbel ? sa.gumbel[(size_t)b * p.rows + tok] : 0.f);
                        float M = -INFINITY;
                        for (unsigned c = 0; c < gridDim.x; ++c) M = fmaxf(M, __ldcg(&p.lse_part[(size_t)c * 256 + b]).x);
                        float S = 0.f;
                        for (unsigned c = 0; c < gridDim.x; ++c) {
                            const float2 ms = __ldcg(&p.lse_part[(size_t)c * 256 + b]);
                            if (ms.x != -INFINITY) S += ms.y * __expf(ms.x - M);
                        }
                        sa.logprob[b] = zt - (M + logf(S));
                    }
                }
                if (t == 0) *p.done = 0u;
            }
        }
    }
    if (MODE == 0 && threadIdx.x == 64) tma_store_wait_all();     // the staging buffers are read, the pieces written
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, tmem_cols);
    if (threadIdx.x == 0) TC_STAMP(7);
}

// fp16 re-encoding of bf16 weights (exact for |w| in [2^-14, 65504]; smaller magnitudes round to
// fp16 subnormals / zero, an absolute error below 2^-25), written TILE-MAJOR: the [128 rows x 64 k]
// tile (row tile t, k block kb) occupies the 16 KB starting at element ((t * KB + kb) * 128) * 64,
// rows of 128 bytes, zero-padded at the ragged edges.  One TMA box is then one contiguous 16 KB run
// of DRAM instead of 128 separate 128-byte row segments.
__global__ void bf16_to_f16_tiled_kernel(const __nv_bfloat16* __restrict__ src, __half* __restrict__ dst, int rows,
                                         int K, int KB, size_t n_chunks) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;       // one 8-element (16-byte) chunk of dst
    if (i >= n_chunks) return;
    const int kc = (int)(i & 7);                     // chunk within the 64-wide row
    const size_t rowi = i >> 3;                      // row of the tiled array
    const int rr = (int)(rowi & 127);
    const size_t tk = rowi >> 7;                     // t * KB + kb
    const int kb = (int)(tk % KB);
    const size_t t = tk / KB;
    const size_t r = t * TC_BM + rr;
    const int k0 = kb * TC_BK + kc * 8;
    uint4 o = make_uint4(0u, 0u, 0u, 0u);
    if (r < (size_t)rows && k0 < K) {                // K is a multiple of 8: a chunk is inside or outside
        uint4 v = *reinterpret_cast<const uint4*>(src + r * K + k0);
        o.x = pack_f16(bf16_lo(v.x), bf16_hi(v.x)); o.y = pack_f16(bf16_lo(v.y), bf16_hi(v.y));
        o.z = pack_f16(bf16_lo(v.z), bf16_hi(v.z)); o.w = pack_f16(bf16_lo(v.w), bf16_hi(v.w));
    }
    *reinterpret_cast<uint4*>(dst + i * 8) = o;
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
struct TcWeight {
    __half* w16 = nullptr;
    CUtensorMap map;
    int rows = 0, K = 0;
    bool resident = false;      // registered at init: the fp16 copy is converted once
};
struct TcPlan {
    int grid = 0, max_pieces = 0;
};
struct TcState {
    int device = 0, max_batch = 0, n_sm = 0;
    bool ready = false;
    int bps = TC_BPS;           // k blocks per ring stage (fewer where the ring would become shallower than 3 stages)
    bool skip_x_once = false;   // wait-timeout self-test: the next tc_linear launch leaves its activation loads out
    PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
    std::unordered_map<const void*, TcWeight> weights;
    std::map<std::tuple<int, int, int>, TcPlan> plans;                  // (rows, K, whole-tile mode)
    std::map<std::tuple<const void*, int, int, int>, CUtensorMap> xmaps;  // (ptr, K, rows of X, N)
    std::map<std::tuple<const void*, int, int, int>, CUtensorMap> omaps;  // pieces buffer as (ptr, rows, n, pieces)
    unsigned long long* best = nullptr;
    unsigned int* done = nullptr;
    float2* lse_part = nullptr;         // [n_sm][256]
};

#ifdef TC_PROBE         // timing-probe builds only: eight timestamps per CTA for each of the last 64 launches
constexpr int TC_PROBE_LAUNCHES = 64, TC_PROBE_CTAS = 160;
__device__ unsigned long long g_tc_probe_buf[TC_PROBE_LAUNCHES * TC_PROBE_CTAS * 8];
static int g_tc_probe_launch = 0;
inline unsigned long long* tc_probe_slot() {
    unsigned long long* base = nullptr;
    if (cudaGetSymbolAddress((void**)&base, g_tc_probe_buf) != cudaSuccess) return nullptr;
    return base + (size_t)(g_tc_probe_launch++ % TC_PROBE_LAUNCHES) * TC_PROBE_CTAS * 8;
}
#endif
static thread_local std::string g_tc_error;
inline const char* tc_last_error() { return g_tc_error.c_str(); }

#define TC_TRY(expr)                                                                 \
    do {                                                                             \
        cudaError_t e__ = (expr);                                                    \
        if (e__ != cudaSuccess) {                                                    \
            g_tc_error = std::string(#expr) + ": " + cudaGetErrorString(e__);        \
            return SPIRAL_ERR_CUDA;                                                  \
        }                                                                            \
    } while (0)

inline int tc_init(TcState& tc, int device, int max_batch) {
    tc.device = device;
    tc.max_batch = max_batch;
    cudaDeviceProp prop;
    TC_TRY(cudaGetDeviceProperties(&prop, device));
    tc.n_sm = prop.multiProcessorCount;
    if (prop.major != 10) {     // tcgen05, TMEM and these TMA forms exist on sm_100 only; there is no other path
        g_tc_error = "device is not sm_100";
        return SPIRAL_ERR_UNSUPPORTED;
    }
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    TC_TRY(cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres));
    if (!fn || qres != cudaDriverEntryPointSuccess) {
        g_tc_error = "cuTensorMapEncodeTiled not available";
        return SPIRAL_ERR_CUDA;
    }
    tc.encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
    TC_TRY(cudaMalloc((void**)&tc.best, 256 * sizeof(unsigned long long)));
    TC_TRY(cudaMalloc((void**)&tc.done, sizeof(unsigned int)));
    TC_TRY(cudaMemset(tc.best, 0, 256 * sizeof(unsigned long long)));
    TC_TRY(cudaMemset(tc.done, 0, sizeof(unsigned int)));
    TC_TRY(cudaMalloc((void**)&tc.lse_part, (size_t)tc.n_sm * 256 * sizeof(float2)));
    TC_TRY(cudaFuncSetAttribute(tc_gemm_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 1024));
    TC_TRY(cudaFuncSetAttribute(tc_gemm_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 18 * 1024));
#ifdef SPIRAL_TUNE      // tuning builds only: ring shape from the environment
    if (const char* v = std::getenv("SPIRAL_TC_BPS")) tc.bps = atoi(v);
#endif
    tc.ready = true;
    return SPIRAL_OK;
}

inline void tc_destroy(TcState& tc) {
    for (auto& kv : tc.weights) cudaFree(kv.second.w16);
    cudaFree(tc.best);
    cudaFree(tc.done);
    cudaFree(tc.lse_part);
    tc.weights.clear(); tc.plans.clear(); tc.xmaps.clear(); tc.omaps.clear();
    tc.best = nullptr; tc.done = nullptr; tc.lse_part = nullptr; tc.ready = false;
}

inline bool tc_usable(const TcState& tc, int rows, int K, int n, bool force) {
    if (!tc.ready) return false;
    if (rows < TC_BM || K < TC_BK || K % 8 != 0 || n < 1 || n > 256) return false;
    return force || n >= 16;
}

// 2-d tensor map [outer][inner] of 2-byte floats with a [box_outer][64] box and 128-byte swizzle
inline int tc_encode(TcState& tc, CUtensorMap* map, const void* base, uint64_t inner, uint64_t outer, uint32_t box_outer,
                     bool bf16 = false) {
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {inner * 2};
    cuuint32_t box[2] = {(cuuint32_t)TC_BK, box_outer};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = tc.encode(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        g_tc_error = "cuTensorMapEncodeTiled failed (" + std::to_string((int)r) + ")";
        return SPIRAL_ERR_CUDA;
    }
    return SPIRAL_OK;
}

inline size_t tc_tiled_elems(int rows, int K) {
    return (size_t)((rows + TC_BM - 1) / TC_BM) * ((K + TC_BK - 1) / TC_BK) * TC_BM * TC_BK;
}
inline int tc_convert(const __nv_bfloat16* W, __half* w16, int rows, int K, cudaStream_t st, int64_t* launches) {
    const size_t chunks = tc_tiled_elems(rows, K) / 8;
    bf16_to_f16_tiled_kernel<<<(unsigned)((chunks + 255) / 256), 256, 0, st>>>(W, w16, rows, K, (K + TC_BK - 1) / TC_BK,
                                                                                chunks);
    if (launches) ++*launches;
    TC_TRY(cudaGetLastError());
    return SPIRAL_OK;
}

// fp16 copy + tensor map of one weight matrix.  resident = converted now, once (model weights).
inline int tc_register_weight(TcState& tc, const __nv_bfloat16* W, int rows, int K, bool resident, cudaStream_t st,
                              int64_t* launches, TcWeight** out) {
    auto it = tc.weights.find(W);
    if (it != tc.weights.end() && (it->second.rows != rows || it->second.K != K)) {
        if (it->second.resident) { g_tc_error = "weight registered with another shape"; return SPIRAL_ERR_INVALID; }
        cudaFree(it->second.w16);
        tc.weights.erase(it);
        it = tc.weights.end();
    }
    if (it == tc.weights.end()) {
        TcWeight w;
        w.rows = rows; w.K = K; w.resident = resident;
        cudaError_t e = cudaMalloc((void**)&w.w16, tc_tiled_elems(rows, K) * sizeof(__half));
        if (e != cudaSuccess) {
            cudaGetLastError();
            g_tc_error = "fp16 weight copy: " + std::string(cudaGetErrorString(e));
            return e == cudaErrorMemoryAllocation ? SPIRAL_ERR_OOM : SPIRAL_ERR_CUDA;
        }
        // tile-major copy seen as rows of 64 elements: tile (t, kb) = rows (t * KB + kb) * 128 ...
        int rc = tc_encode(tc, &w.map, w.w16, (uint64_t)TC_BK, (uint64_t)(tc_tiled_elems(rows, K) / TC_BK), TC_BM);
        if (rc) { cudaFree(w.w16); return rc; }
        if (resident) {
            rc = tc_convert(W, w.w16, rows, K, st, launches);
            if (rc) { cudaFree(w.w16); return rc; }
        }
        it = tc.weights.emplace(W, w).first;
    }
    if (!it->second.resident) {
        int rc = tc_convert(W, it->second.w16, rows, K, st, launches);
        if (rc) return rc;
    }
    if (out) *out = &it->second;
    return SPIRAL_OK;
}

// Grid size of one GEMM and the number of pieces each 128-row tile receives, evaluated with the
// same schedule the kernel walks.
inline int tc_get_plan(TcState& tc, int rows, int K, bool whole_tiles, TcPlan** out) {
    auto key = std::make_tuple(rows, K, whole_tiles ? 1 : 0);
    auto it = tc.plans.find(key);
    if (it != tc.plans.end()) { *out = &it->second; return SPIRAL_OK; }
    const int tiles = (rows + TC_BM - 1) / TC_BM, KB = (K + TC_BK - 1) / TC_BK;
    const long long U = whole_tiles ? tiles : (long long)tiles * KB;
    const long long min_units = whole_tiles ? 1 : 4;            // do not cut ranges shorter than 4 k blocks
    TcPlan pl;
    pl.grid = (int)std::min<long long>(tc.n_sm, std::max<long long>(1, U / min_units));
    // Where a whole number of equal k ranges per tile uses all but at most 3 % of the SMs (48 QKV tiles x 3 = 144 of 148),
    // that cut is taken: no range straddles a tile, so every CTA has one segment and one epilogue (-0.5 % per step);
    // with more SMs left idle (20 tiles x 7 = 140) the even cut over all SMs is faster.
    if (!whole_tiles && tiles <= tc.n_sm) {
        const int aligned = tiles * (tc.n_sm / tiles);
        if (aligned * 100 >= tc.n_sm * 97 && (long long)aligned * min_units <= U) pl.grid = aligned;
    }
    std::vector<int> cnt(tiles, 0);
    for (int c = 0; c < pl.grid; ++c) {
        TcSchedule sched(tiles, KB, whole_tiles ? 1 : 0, c, pl.grid);
        TcSeg sg;
        while (sched.next(sg)) {
            if (sg.piece != cnt[sg.tile]) { g_tc_error = "stream-K plan: piece numbering mismatch"; return SPIRAL_ERR_CUDA; }
            cnt[sg.tile]++;
        }
    }
    pl.max_pieces = 0;
    for (int t = 0; t < tiles; ++t) pl.max_pieces = std::max(pl.max_pieces, cnt[t]);
    for (int t = 0; t < tiles && !whole_tiles; ++t) {      // what the consumers of the pieces will compute
        const long long first = (long long)t * KB;
        if (streamk_cta_of(first + KB - 1, pl.grid, U) - streamk_cta_of(first, pl.grid, U) + 1 != cnt[t]) {
            g_tc_error = "stream-K plan: piece count mismatch";
            return SPIRAL_ERR_CUDA;
        }
    }
    *out = &tc.plans.emplace(key, pl).first->second;
    return SPIRAL_OK;
}

// pieces a [rows][K] GEMM will produce at most per output element (sizes the pieces buffer)
inline int tc_max_pieces(TcState& tc, int rows, int K) {
    TcPlan* pl = nullptr;
    if (tc_get_plan(tc, rows, K, false, &pl) != SPIRAL_OK) return -1;
    return pl->max_pieces;
}

inline int tc_get_xmap(TcState& tc, const void* X, int K, int x_rows, int N, const CUtensorMap** out) {
    auto key = std::make_tuple(X, K, x_rows, N);
    auto it = tc.xmaps.find(key);
    if (it == tc.xmaps.end()) {
        if (tc.xmaps.size() > 4096) tc.xmaps.clear();
        CUtensorMap m;
        int rc = tc_encode(tc, &m, X, (uint64_t)K, (uint64_t)x_rows, (uint32_t)N);
        if (rc) return rc;
        it = tc.xmaps.emplace(key, m).first;
    }
    *out = &it->second;
    return SPIRAL_OK;
}

// Ring shape and dynamic shared memory of one launch: stages of `bps` k blocks (W tile + X tile each),
// as many as the SM's shared memory holds; fewer blocks per stage where that leaves under 3 stages.
inline void tc_launch_shape(const TcState& tc, int N, TcParams* p, size_t* smem, bool lm_head = false) {
    // an SM's 227 KB less the static part (barriers; the LM head's argmax and log-sum-exp scratch), the alignment
    // slack and, for the pieces epilogue, its two staging buffers
    const size_t tail = lm_head ? 0 : 2 * TC_OUT_BYTES;
    const size_t budget = 227 * 1024 - (lm_head ? 18 * 1024 : 1024) - 1024 - tail;
    const size_t blk_bytes = TC_W_BYTES + (size_t)N * 128;
    int bps = std::max(1, std::min(tc.bps, 4));
    while (bps > 1 && budget / (bps * blk_bytes) < 3) --bps;
    p->stages = (int)std::min<size_t>(TC_MAX_STAGES, budget / (bps * blk_bytes));
    p->bps = bps;
    p->chains = 4 * N <= 512 ? 2 : 1;           // TMEM has 512 columns: two buffers of `chains` accumulators of N columns
    *smem = (size_t)p->stages * bps * blk_bytes + 1024 + tail;
}

// the pieces buffer [pieces][n][rows] of floats as a 3-d tensor map with a box of 1 x 32 x 128 (rows % 4 == 0)
inline int tc_get_omap(TcState& tc, const float* base, int rows, int n, int pieces, const CUtensorMap** out) {
    auto key = std::make_tuple((const void*)base, rows, n, pieces);
    auto it = tc.omaps.find(key);
    if (it == tc.omaps.end()) {
        if (tc.omaps.size() > 4096) tc.omaps.clear();
        CUtensorMap m;
        cuuint64_t dims[3] = {(cuuint64_t)rows, (cuuint64_t)n, (cuuint64_t)pieces};
        cuuint64_t strides[2] = {(cuuint64_t)rows * 4, (cuuint64_t)n * rows * 4};
        cuuint32_t box[3] = {(cuuint32_t)TC_BM, (cuuint32_t)TC_OUT_ROWS, 1};
        cuuint32_t estr[3] = {1, 1, 1};
        CUresult r = tc.encode(&m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(base), dims, strides, box, estr,
                               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) {
            g_tc_error = "cuTensorMapEncodeTiled (pieces) failed (" + std::to_string((int)r) + ")";
            return SPIRAL_ERR_CUDA;
        }
        it = tc.omaps.emplace(key, m).first;
    }
    *out = &it->second;
    return SPIRAL_OK;
}

// y pieces = X W^T.  W is the caller's bf16 matrix (its registered fp16 copy is what the kernel reads).
inline int tc_linear(TcState& tc, const __nv_bfloat16* W, int rows, int K, const __half* X, int n, float* pieces,
                     size_t pieces_elems, Pieces* out, int* status, cudaStream_t st, int64_t* launches) {
    TcWeight* w = nullptr;
    int rc = tc_register_weight(tc, W, rows, K, false, st, launches, &w);
    if (rc) return rc;
    TcPlan* pl = nullptr;
    rc = tc_get_plan(tc, rows, K, false, &pl);
    if (rc) return rc;
    if ((size_t)pl->max_pieces * n * rows > pieces_elems) return SPIRAL_ERR_UNSUPPORTED;
    const int N = (n + 15) & ~15;
    const CUtensorMap* xm = nullptr;
    rc = tc_get_xmap(tc, X, K, n, N, &xm);
    if (rc) return rc;
    TcParams p{};
    p.tiles = (rows + TC_BM - 1) / TC_BM; p.KB = (K + TC_BK - 1) / TC_BK; p.whole_tiles = 0;
    p.rows = rows; p.n = n; p.N = N;
    size_t smem;
    tc_launch_shape(tc, N, &p, &smem);
    p.out = pieces; p.piece_stride = (size_t)n * rows; p.status = status;
    p.skip_x = tc.skip_x_once ? 1 : 0;
    tc.skip_x_once = false;
    const CUtensorMap* om = &w->map;        // (unused unless tma_out)
    p.tma_out = (rows % 4 == 0 && ((uintptr_t)pieces & 15) == 0) ? 1 : 0;
    if (p.tma_out) {
        rc = tc_get_omap(tc, pieces, rows, n, pl->max_pieces, &om);
        if (rc) return rc;
    }
#ifdef TC_PROBE
    p.probe = tc_probe_slot();
#endif
    TC_TRY(launch_kernel(true, tc_gemm_kernel<0>, dim3(pl->grid), dim3(tc_threads(0)), smem, st, w->map, *xm, *om, p));
    if (launches) ++*launches;
    out->base = pieces; out->stride = p.piece_stride; out->ld = rows; out->n_pieces = pl->max_pieces;
    out->sk_KB = p.KB; out->sk_G = pl->grid;
    return SPIRAL_OK;
}

// args->tok_out[b] = argmax_v (X W^T)[b][v] / T + gumbel[b][v]; full-vocabulary logits are written
// only when args->logits is set.  args lives in device memory and is read by the kernel.
inline int tc_lm_head(TcState& tc, const __nv_bfloat16* W, int vocab, int K, const __half* X, int n,
                      const StepArgs* args_dev, int* status, cudaStream_t st, int64_t* launches) {
    TcWeight* w = nullptr;
    int rc = tc_register_weight(tc, W, vocab, K, false, st, launches, &w);
    if (rc) return rc;
    TcPlan* pl = nullptr;
    rc = tc_get_plan(tc, vocab, K, true, &pl);
    if (rc) return rc;
    const int N = (n + 15) & ~15;
    const CUtensorMap* xm = nullptr;
    rc = tc_get_xmap(tc, X, K, n, N, &xm);
    if (rc) return rc;
    TcParams p{};
    p.tiles = (vocab + TC_BM - 1) / TC_BM; p.KB = (K + TC_BK - 1) / TC_BK; p.whole_tiles = 1;
    p.rows = vocab; p.n = n; p.N = N;
    size_t smem;
    tc_launch_shape(tc, N, &p, &smem, true);
    p.status = status; p.args = args_dev; p.best = tc.best; p.done = tc.done; p.lse_part = tc.lse_part;
#ifdef TC_PROBE
    p.probe = tc_probe_slot();
#endif
    TC_TRY(launch_kernel(true, tc_gemm_kernel<1>, dim3(pl->grid), dim3(tc_threads(1)), smem, st, w->map, *xm, w->map, p));
    if (launches) ++*launches;
    return SPIRAL_OK;
}

}  // namespace spiral
