// Shared device helpers of libgmlp (sm_100a only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace gmlp {

typedef __nv_bfloat16 bf16;

// Device status word: 0, or (kernel id << 16 | site) of the first bounded wait that ran out.
__device__ int g_device_status = 0;

__device__ __forceinline__ void report_timeout(int kernel_id, int site) {
    atomicCAS(&g_device_status, 0, (kernel_id << 16) | (site & 0xFFFF));
}

// Optional timeline of the small-M kernels (builds with -DGMLP_TRACE only; nothing of it exists in the normal
// library): one thread per site stores the global nanosecond timer, the last launch of each kernel wins.
#ifdef GMLP_TRACE
constexpr int kTraceKernels = 4, kTraceCtas = 512, kTraceSites = 16;
__device__ unsigned long long g_trace[kTraceKernels][kTraceCtas][kTraceSites];
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
#define GMLP_TR(kernel, site) do { if (blockIdx.x < gmlp::kTraceCtas) gmlp::g_trace[kernel][blockIdx.x][site] = gmlp::global_timer_ns(); } while (0)
#else
#define GMLP_TR(kernel, site) do { } while (0)
#endif

// silu(g) = g * sigmoid(g), written g / (1 + e^-g): for g -> -inf this tends to -0 and never
// forms 0 * inf.  ex2.approx / fast division are ~2^-21 relative, far below a bf16 ulp.
__device__ __forceinline__ float silu_f32(float g) {
    return __fdividef(g, 1.0f + __expf(-g));
}

// Gate activation of the gated unit, h = act(g) * u (Section 6.1 lists SiLU-, SwiGLU- and GLU-gated forms):
//   SiLU      act(g) = g * sigmoid(g)            beta = 1, glu = 0
//   Swish     act(g) = g * sigmoid(beta * g)     beta free, glu = 0
//   GLU       act(g) = sigmoid(g)                beta = 1, glu = 1
//   GELU      act(g) = g * Phi(g)                glu = 2   (Phi the standard normal distribution function: the exact
//             form, g * erfc(-g / sqrt 2) / 2, not the tanh approximation, whose 5e-4 error would change the bf16 H
//             rounds to far more often than anything else on the path)
// the first three are one expression, numerator g or 1 over 1 + e^(-beta g); with beta = 1, glu = 0 it is silu_f32
// bit for bit.  The choice is uniform over a launch.
struct GateAct {
    float beta;
    int glu;
};
// (The GELU path is a call, not inline code: inlined, the compiler evaluated it under a predicate next to the sigmoid
// form in every epilogue, which cost the SiLU path up to 10 % of a short kernel.)
__device__ __noinline__ float gelu_f32(float g) { return 0.5f * g * erfcf(-0.70710678118654752f * g); }
__device__ __forceinline__ float gate_act_f32(float g, const GateAct a) {
    if (a.glu == 2) return gelu_f32(g);
    return __fdividef(a.glu == 1 ? 1.0f : g, 1.0f + __expf(-(a.beta * g)));
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);   // .x = lo (low half), .y = hi
    return *reinterpret_cast<uint32_t*>(&v);
}

// 16-byte read-only load that does not allocate in L1 (weights are streamed once).
__device__ __forceinline__ uint4 ld_stream_16B(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

}  // namespace gmlp
