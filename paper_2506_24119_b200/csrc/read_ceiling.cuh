// Read-only bandwidth probe: what a kernel that does nothing but stream HBM into shared memory can
// reach on this GPU.  The decode step is a pure read stream (weights and cached keys/values are read
// once per step and nothing comparable is written), so this -- not a read+write copy -- is the
// ceiling its kernels are measured against.
//
// Persistent grid; every CTA owns an interleaved share of the buffer's chunks and pulls them through a
// ring of shared-memory stages with bulk asynchronous copies (cp.async.bulk, the non-tensor form of
// TMA: one contiguous run per request).  One thread per CTA waits for a stage to land and at once
// re-issues the stage for a later chunk; nothing reads the data.  Every wait is bounded.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "tma.cuh"

namespace spiral {

constexpr int RC_MAX_STAGES = 16;

struct ReadCeilingParams {
    const uint8_t* buf;
    unsigned long long chunks;      // chunks of stage_bytes in the buffer
    int stage_bytes, stages, passes;
    int blocked;                    // 0: chunk i of CTA c is chunk c + i * grid (neighbouring CTAs read neighbouring
                                    // chunks at the same time); 1: every CTA streams one contiguous share of the buffer;
                                    // 2: the chunks of pattern 0 scattered over the buffer by a fixed permutation (pages
                                    // of a cache handed out in no particular order)
    unsigned long long scatter_mask;    // pattern 2: chunks rounded down to a power of two, minus one
    int* status;
};

__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// tiled = 1: the same stream fetched as tiled TMA boxes of (stage_bytes / 128) rows x 128 bytes with the
// 128-byte swizzle (the form the GEMM kernels use); tm then maps the buffer as rows of 128 bytes.  tiled = 2: tm
// maps it as rows of 256 bytes and a chunk is fetched as two boxes, the left and the right half of its rows (the
// form the attention kernel uses for blocks with 128-element rows)
__global__ void __launch_bounds__(32, 1) read_ceiling_kernel(const __grid_constant__ CUtensorMap tm, int tiled,
                                                             ReadCeilingParams p) {
    extern __shared__ uint8_t rc_smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[RC_MAX_STAGES];
    __shared__ int abort_sm;
    if (threadIdx.x != 0) return;
    const uint32_t ring = (smem_u32(rc_smem_raw) + 1023u) & ~1023u;
    for (int s = 0; s < p.stages; ++s) mbar_init(smem_u32(&full_bar[s]), 1);
    abort_sm = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // chunks of this CTA per pass (every CTA takes the same number: a ragged tail of the buffer is left out), and
    // the walk over them: running counters only, the loop of the one issuing thread contains no division
    const unsigned int per_pass = (unsigned int)(p.chunks / gridDim.x);
    const unsigned long long step = (unsigned long long)p.stage_bytes * (p.blocked == 1 ? 1u : gridDim.x);
    const uint8_t* const first = p.buf + (unsigned long long)p.stage_bytes *
                                             (p.blocked == 1 ? (unsigned long long)blockIdx.x * per_pass : blockIdx.x);
    const unsigned long long total = (unsigned long long)per_pass * (unsigned long long)p.passes;
    const uint8_t* src = first;
    unsigned int in_pass = 0;
    auto next_src = [&]() {
        const uint8_t* r = src;
        src += step;
        if (++in_pass == per_pass) { in_pass = 0; src = first; }
        if (p.blocked == 2) {       // chunk number -> a scattered chunk number (odd multiplier: a permutation of 0 .. 2^k - 1)
            const unsigned long long c = (unsigned long long)(r - p.buf) / (unsigned int)p.stage_bytes;
            r = p.buf + ((c * 0x9E3779B1ull) & p.scatter_mask) * (unsigned long long)p.stage_bytes;
        }
        return r;
    };
    auto load = [&](uint32_t dst, const uint8_t* from, uint32_t bar) {
        if (tiled == 2) {           // the chunk as two boxes: left and right 128-byte halves of its 256-byte rows
            const int y = (int)((unsigned long long)(from - p.buf) >> 8);
            tma_load_2d_nohint(dst, &tm, 0, y, bar);
            tma_load_2d_nohint(dst + ((uint32_t)p.stage_bytes >> 1), &tm, 64, y, bar);
        } else if (tiled) tma_load_2d_nohint(dst, &tm, 0, (int)((unsigned long long)(from - p.buf) >> 7), bar);
        else bulk_load_1d(dst, from, (uint32_t)p.stage_bytes, bar);
    };
    unsigned long long issued = 0;
    for (; issued < total && issued < (unsigned long long)p.stages; ++issued) {
        const uint32_t bar = smem_u32(&full_bar[issued]);
        mbar_expect_tx(bar, (uint32_t)p.stage_bytes);
        load(ring + (uint32_t)issued * (uint32_t)p.stage_bytes, next_src(), bar);
    }
    unsigned long long done = 0;
    uint32_t s = 0, ph = 0;
    for (; done < total; ++done) {
        if (!mbar_wait(smem_u32(&full_bar[s]), ph, &abort_sm, p.status, STATUS_TIMEOUT_TMA)) break;
        if (issued < total) {
            const uint32_t bar = smem_u32(&full_bar[s]);
            mbar_expect_tx(bar, (uint32_t)p.stage_bytes);
            load(ring + s * (uint32_t)p.stage_bytes, next_src(), bar);
            ++issued;
        }
        if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1u; }
    }
    if (done < total) {
        // copies already issued still land in this CTA's shared memory: give them a bounded time
        for (unsigned long long j = done; j < issued; ++j) {
            const int sj = (int)(j % (unsigned long long)p.stages);
            const uint32_t pj = (uint32_t)(j / (unsigned long long)p.stages) & 1u;
            const unsigned long long t0 = global_ns();
            while (!mbar_try(smem_u32(&full_bar[sj]), pj) && global_ns() - t0 < TMA_WAIT_NS) {}
        }
    }
}

}  // namespace spiral
