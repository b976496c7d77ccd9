// Shared device helpers: status word, bf16 conversions, cache-hinted loads, warp reductions.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace spiral {

// Device status word values (first error wins; see record_status).
enum : int {
    STATUS_OK = 0,
    STATUS_BAD_TOKEN = 1,        // token id outside [0, vocab)
    STATUS_BAD_PAGE = 2,         // page id outside [0, n_pages)
    STATUS_TIMEOUT_TMA = 16,     // bounded wait on a TMA "full" barrier ran out
    STATUS_TIMEOUT_MMA = 17,     // bounded wait on an MMA-completion barrier ran out
    STATUS_TIMEOUT_EPI = 18,     // bounded wait on an accumulator "empty" barrier ran out
    STATUS_BAD_SMEM = 3,         // the dynamic shared memory a kernel was given does not hold its tiles
};

__device__ __forceinline__ void record_status(int* status, int code) {
    atomicCAS(status, STATUS_OK, code);
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t bits16) {
    return __uint_as_float(bits16 << 16);
}
// the two bf16 halves of a packed 32-bit word, widened exactly
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// round-to-nearest-even fp32 -> bf16 bits
__device__ __forceinline__ uint32_t float_to_bf16_bits(float f) {
    return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(f));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    return float_to_bf16_bits(lo) | (float_to_bf16_bits(hi) << 16);
}

// fp32 -> fp16 bits, round to nearest even, saturating at the largest finite value.  Activations
// that feed the GEMMs are carried as fp16 (11-bit mantissa): bf16 weights are exactly
// representable in fp16 over the whole normal range, so weight x activation products are exact and
// the only rounding is the 2^-12 relative one of the activation itself.
__device__ __forceinline__ uint32_t float_to_f16_bits(float f) {
    f = fminf(fmaxf(f, -65504.f), 65504.f);
    return (uint32_t)__half_as_ushort(__float2half_rn(f));
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    return float_to_f16_bits(lo) | (float_to_f16_bits(hi) << 16);
}
__device__ __forceinline__ float2 unpack_f16(uint32_t w) {
    return __half22float2(*reinterpret_cast<const __half2*>(&w));
}

// 16-byte read-only load that does not allocate in L1 (data streamed once per step)
__device__ __forceinline__ uint4 ldg_stream_v4(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}
// 16-byte read-only load through L1 (small, re-read operands such as activations)
__device__ __forceinline__ uint4 ldg_v4(const void* p) {
    return __ldg(reinterpret_cast<const uint4*>(p));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Programmatic dependent launch: launch_dependents lets the next kernel of the stream start its
// prologue (and prefetch data nobody writes, such as weights) while this one runs; wait blocks
// until every kernel this one depends on has completed and its writes are visible.  Both are
// no-ops for a launch without the programmatic-serialization attribute.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
// what every kernel without a prefetchable prologue does first
__device__ __forceinline__ void grid_dependency_sync() {
    grid_launch_dependents();
    grid_dependency_wait();
}

// Timeline tracing (builds with -DSPIRAL_TRACE only; compiled out otherwise): the first CTA of every
// kernel appends (kernel kind, entry time, time its dependency wait returned, exit time) to a ring.
#ifdef SPIRAL_TRACE
__device__ unsigned long long g_trace[4 * 65536];
__device__ unsigned int g_trace_n;
__device__ __forceinline__ unsigned long long trace_now() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
struct TraceRec {
    unsigned long long t0, t1;
    int kind;
    __device__ __forceinline__ TraceRec(int k) : t0(trace_now()), t1(0), kind(k) {}
    __device__ __forceinline__ void waited() { t1 = trace_now(); }
    __device__ __forceinline__ ~TraceRec() {
        if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == 0) {
            unsigned int i = atomicAdd(&g_trace_n, 1u) & 65535u;
            g_trace[4 * i] = (unsigned long long)kind; g_trace[4 * i + 1] = t0; g_trace[4 * i + 2] = t1;
            g_trace[4 * i + 3] = trace_now();
        }
    }
};
#define TRACE_BEGIN(kind) TraceRec trace_rec__(kind)
#define TRACE_WAITED() trace_rec__.waited()
#else
#define TRACE_BEGIN(kind) do { } while (0)
#define TRACE_WAITED() do { } while (0)
#endif

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Launch with the programmatic-serialization attribute (when `pdl`), so that the kernel may begin
// before its predecessor in the stream has finished; the kernel itself orders its reads and writes
// with grid_dependency_wait().
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(bool pdl, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                 cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace spiral
