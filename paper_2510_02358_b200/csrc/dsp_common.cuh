// Shared device/host helpers of the CUDA library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "dsp.h"

namespace dsp {

constexpr int kThreads = 256;                 // threads per CTA of every streaming kernel
constexpr int kWarps = kThreads / 32;
constexpr int kCandCap = 1024;                // candidate buffer entries per CTA (>= 32 slices * DSP_MAX_K)
constexpr int kMaxSlices = 32;                // slices per row a single finaliser merges
constexpr float kLog2e = 1.44269502162933349609375f;      // fp32 nearest to log2(e)
constexpr double kLn2 = 0.693147180559945309417232;
// The streaming sums use 2^(x*kLog2e); kLog2e*ln2 = 1 - kTilt, a known 1.3e-8 tilt that the
// finaliser removes to first order with the row's mean logit.
constexpr double kTilt = 1.0 - (double)kLog2e * kLn2;
constexpr float kRefFloor = -3.0e38f;          // finite stand-in for "no reference exponent yet"

// Host-side record of the last CUDA error seen by an entry point.
extern int32_t g_last_cuda_error;
// Events that bracket a kernel launch while set (see dsp_profile_events).
struct ProfileEvents {
    cudaEvent_t start, stop;
};
extern ProfileEvents g_profile[2];
inline int32_t cuda_fail(cudaError_t e) {
    g_last_cuda_error = (int32_t)e;
    return DSP_ERR_CUDA;
}
#define DSP_CUDA_TRY(expr)                                   \
    do {                                                     \
        cudaError_t e__ = (expr);                            \
        if (e__ != cudaSuccess) return ::dsp::cuda_fail(e__); \
    } while (0)

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---- programmatic dependent launch: a kernel that only consumes what the kernel before it in
// the stream produced is launched with launch_dependent; the device may then place its CTAs as
// soon as every CTA of that kernel has called grid_launch_dependents (or left), and they sit in
// grid_dependency_wait until that kernel has completed and its writes are visible.  The wait is
// the first thing such a kernel does; launched without the attribute, both calls do nothing.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
// `programmatic` false: an ordinary launch (full dependency on the kernel before).
template <typename Arg>
inline cudaError_t launch_dependent(void (*kernel)(Arg), unsigned grid, unsigned block, size_t smem,
                                    cudaStream_t st, const Arg &a, bool programmatic) {
    if (!programmatic) {
        kernel<<<grid, block, smem, st>>>(a);
        return cudaGetLastError();
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, a);
}

// The early placement saves 1 to 2 us per launch between the short kernels of a call, in a stream
// and in a captured graph alike.

// ---- order-preserving 64-bit keys: larger key = better under (logit desc, id asc) ----
__device__ __forceinline__ uint32_t ord_bits(float x) {
    uint32_t b = __float_as_uint(x + 0.0f);                 // -0.0 -> +0.0
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float ord_value(uint32_t o) {
    return __uint_as_float((o & 0x80000000u) ? (o & 0x7FFFFFFFu) : ~o);
}
__device__ __forceinline__ unsigned long long make_key(float x, int id) {
    return ((unsigned long long)ord_bits(x) << 32) | (uint32_t)(0xFFFFFFFFu - (uint32_t)id);
}
__device__ __forceinline__ float key_value(unsigned long long k) { return ord_value((uint32_t)(k >> 32)); }
__device__ __forceinline__ int key_id(unsigned long long k) { return (int)(0xFFFFFFFFu - (uint32_t)k); }

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// 128-bit streaming load: read-only path, do not keep the line in L1.
__device__ __forceinline__ uint4 ldg_stream(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

template <typename T>
__device__ __forceinline__ T warp_max(T v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        T w = __shfl_xor_sync(0xFFFFFFFFu, v, o);
        v = w > v ? w : v;
    }
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// Element type traits: N elements per 128-bit vector, kVpt vectors per thread per tile.
template <typename DT> struct Elem;
template <> struct Elem<__nv_bfloat16> {
    static constexpr int N = 8;
    static constexpr uint32_t kNegInfWord = 0xFF80FF80u;
    static __device__ __forceinline__ float get(const uint4 &v, int e) {
        uint32_t w = e < 2 ? v.x : e < 4 ? v.y : e < 6 ? v.z : v.w;
        return (e & 1) ? bf16_hi(w) : bf16_lo(w);
    }
    static __device__ __forceinline__ float load1(const __nv_bfloat16 *p) {
        return __uint_as_float((uint32_t)(*reinterpret_cast<const unsigned short *>(p)) << 16);
    }
    static __device__ __forceinline__ float vmax(const uint4 &v) {
        __nv_bfloat162 a = __hmax2(*reinterpret_cast<const __nv_bfloat162 *>(&v.x),
                                   *reinterpret_cast<const __nv_bfloat162 *>(&v.y));
        __nv_bfloat162 b = __hmax2(*reinterpret_cast<const __nv_bfloat162 *>(&v.z),
                                   *reinterpret_cast<const __nv_bfloat162 *>(&v.w));
        a = __hmax2(a, b);
        uint32_t w = *reinterpret_cast<uint32_t *>(&a);
        return fmaxf(bf16_lo(w), bf16_hi(w));
    }
};
template <> struct Elem<float> {
    static constexpr int N = 4;
    static constexpr uint32_t kNegInfWord = 0xFF800000u;
    static __device__ __forceinline__ float get(const uint4 &v, int e) {
        return __uint_as_float(e == 0 ? v.x : e == 1 ? v.y : e == 2 ? v.z : v.w);
    }
    static __device__ __forceinline__ float load1(const float *p) { return *p; }
    static __device__ __forceinline__ float vmax(const uint4 &v) {
        return fmaxf(fmaxf(__uint_as_float(v.x), __uint_as_float(v.y)),
                     fmaxf(__uint_as_float(v.z), __uint_as_float(v.w)));
    }
};
// p(v) = 2^(x*kLog2e - c2) with c2 = lse*log2(e) split as hi + lo (lo folded into `corr`).
struct RowProb {
    float nchi;     // -c2_hi
    float corr;     // 2^(-c2_lo)
};
__device__ __forceinline__ RowProb row_prob(double lse) {
    const double c2 = lse / kLn2;
    RowProb r;
    const float hi = (float)c2;
    r.nchi = -hi;
    r.corr = (float)exp2(-(c2 - (double)hi));
    return r;
}
__device__ __forceinline__ float prob(float x, const RowProb &r) {
    return __fmul_rn(ex2_approx(fmaf(x, kLog2e, r.nchi)), r.corr);
}
constexpr int kVpt = 6;                         // vectors per thread per tile

template <typename DT> __host__ __device__ constexpr int tile_elems() { return kThreads * kVpt * Elem<DT>::N; }

}  // namespace dsp
