// RMSNorm prologue (Eq. 1, Section 2; graph order square -> mean -> add eps -> rsqrt ->
// multiply), with an optional per-column gain:  Xn[m,k] = bf16_rn(X[m,k] * r_m * gamma[k]),
// r_m = rsqrt(mean_k X[m,k]^2 + eps).  One CTA per row; fp32 arithmetic; one rounding.
#pragma once
#include "common.cuh"

namespace gmlp {

constexpr int kRmsThreads = 256;

__global__ void __launch_bounds__(kRmsThreads)
rmsnorm_kernel(const bf16* __restrict__ X, const bf16* __restrict__ gamma, bf16* __restrict__ Xn,
               int64_t M, int d_model, float eps)
{
    // launched with programmatic stream serialization: the GEMM that follows may become resident (barriers, TMEM,
    // tensor-map prefetch) while this kernel runs; X may be the previous kernel's output, so nothing is read
    // before that kernel is complete
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int64_t row = blockIdx.x;
    if (row >= M) return;
    const uint4* x = reinterpret_cast<const uint4*>(X + row * d_model);
    const uint4* g = reinterpret_cast<const uint4*>(gamma);
    uint4* out = reinterpret_cast<uint4*>(Xn + row * d_model);
    const int nvec = d_model >> 3;

    float ss = 0.0f;
    for (int i = threadIdx.x; i < nvec; i += kRmsThreads) {
        const uint4 v = x[i];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float a = bf16_lo(w[j]), b = bf16_hi(w[j]);
            ss = fmaf(a, a, ss);
            ss = fmaf(b, b, ss);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
    __shared__ float warp_sums[kRmsThreads / 32];
    __shared__ float r_shared;
    if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.0f;
#pragma unroll
        for (int w = 0; w < kRmsThreads / 32; ++w) t += warp_sums[w];
        r_shared = rsqrtf(t / (float)d_model + eps);
    }
    __syncthreads();
    const float r = r_shared;

    for (int i = threadIdx.x; i < nvec; i += kRmsThreads) {
        const uint4 v = x[i];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        uint32_t gw[4] = {0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u};   // bf16 ones
        if (gamma != nullptr) {
            const uint4 gv = g[i];
            gw[0] = gv.x; gw[1] = gv.y; gw[2] = gv.z; gw[3] = gv.w;
        }
        uint32_t o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float a = bf16_lo(w[j]) * r * bf16_lo(gw[j]);
            const float b = bf16_hi(w[j]) * r * bf16_hi(gw[j]);
            o[j] = pack_bf16x2(a, b);
        }
        out[i] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// The RMS branch alone: r[m] = rsqrt(mean_k X[m,k]^2 + eps) in fp32, one CTA per row.  Used by the rewritten
// RMSNorm+MatMul, whose GEMM applies r in its epilogue; the kernel lets its dependent start at once, so the
// GEMM's main loop runs while the row scales are being computed.
__global__ void __launch_bounds__(kRmsThreads)
row_rsqrt_kernel(const bf16* __restrict__ X, float* __restrict__ r, int64_t M, int K, float eps)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int64_t row = blockIdx.x;
    if (row >= M) return;
    const uint4* x = reinterpret_cast<const uint4*>(X + row * K);
    const int nvec = K >> 3;
    float ss = 0.0f;
    for (int i = threadIdx.x; i < nvec; i += kRmsThreads) {
        const uint4 v = x[i];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float a = bf16_lo(w[j]), b = bf16_hi(w[j]);
            ss = fmaf(a, a, ss);
            ss = fmaf(b, b, ss);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
    __shared__ float warp_sums[kRmsThreads / 32];
    if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.0f;
#pragma unroll
        for (int w = 0; w < kRmsThreads / 32; ++w) t += warp_sums[w];
        r[row] = rsqrtf(t / (float)K + eps);
    }
}

// Second half of "Matmul+Add+RMSNorm": the GEMM's epilogue has stored S and, per row and column tile, the sum
// of squares of the stored values (sumsq [n_tiles][M]); this kernel adds a row's partials in tile order
// (every thread the same order: deterministic), forms r = rsqrt(sum / N + eps) and writes
// Z[m, n] = bf16_rn(S[m, n] * r * gamma[n]).  One CTA per row, one read of S.
__global__ void __launch_bounds__(kRmsThreads)
rmsnorm_apply_kernel(const bf16* __restrict__ S, const float* __restrict__ sumsq, int n_tiles,
                     const bf16* __restrict__ gamma, bf16* __restrict__ Z, int64_t M, int N, float eps)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");            // S and sumsq come from the previous kernel
    const int64_t row = blockIdx.x;
    if (row >= M) return;
    float t = 0.0f;
    for (int i = 0; i < n_tiles; ++i) t += __ldcg(sumsq + (size_t)i * M + row);
    const float r = rsqrtf(t / (float)N + eps);
    const uint4* x = reinterpret_cast<const uint4*>(S + row * N);
    const uint4* g = reinterpret_cast<const uint4*>(gamma);
    uint4* out = reinterpret_cast<uint4*>(Z + row * N);
    const int nvec = N >> 3;
    for (int i = threadIdx.x; i < nvec; i += kRmsThreads) {
        const uint4 v = __ldcg(x + i);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        uint32_t gw[4] = {0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u};   // bf16 ones
        if (gamma != nullptr) {
            const uint4 gv = g[i];
            gw[0] = gv.x; gw[1] = gv.y; gw[2] = gv.z; gw[3] = gv.w;
        }
        uint32_t o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float a = bf16_lo(w[j]) * r * bf16_lo(gw[j]);
            const float b = bf16_hi(w[j]) * r * bf16_hi(gw[j]);
            o[j] = pack_bf16x2(a, b);
        }
        out[i] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// Unfused schedule of the same chain: S = bf16_rn(T + R) elementwise, T the bf16 product of a plain GEMM.
__global__ void __launch_bounds__(256)
add_bf16_kernel(const bf16* __restrict__ T, const bf16* __restrict__ R, bf16* __restrict__ S, size_t nvec)
{
    const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (i >= nvec) return;
    const uint4 a = reinterpret_cast<const uint4*>(T)[i], b = reinterpret_cast<const uint4*>(R)[i];
    const uint32_t x[4] = {a.x, a.y, a.z, a.w}, y[4] = {b.x, b.y, b.z, b.w};
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) o[j] = pack_bf16x2(bf16_lo(x[j]) + bf16_lo(y[j]), bf16_hi(x[j]) + bf16_hi(y[j]));
    reinterpret_cast<uint4*>(S)[i] = make_uint4(o[0], o[1], o[2], o[3]);
}

// d_ff-sharded Gated MLP: each shard (a slice of d_ff: the matching columns of W_gate / W_up and rows of W_down)
// yields an fp32 partial product of the down projection, Y = sum over shards of H_s W_down,s.  This kernel adds up to
// kMaxPartials partials in the order given (fixed: the result does not depend on scheduling), rounds once and
// stores bf16.  count is a multiple of 4; 16 bytes loaded per partial and thread.
constexpr int kMaxPartials = 8;
struct PartialList {
    const float* p[kMaxPartials];
    int n;
};
__global__ void __launch_bounds__(256)
sum_partials_bf16_kernel(PartialList parts, bf16* __restrict__ Y, size_t nvec4)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");           // the partials may come from the previous kernel
    const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (i >= nvec4) return;
    float4 acc = reinterpret_cast<const float4*>(parts.p[0])[i];
    for (int s = 1; s < parts.n; ++s) {
        const float4 v = reinterpret_cast<const float4*>(parts.p[s])[i];
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    reinterpret_cast<uint2*>(Y)[i] = make_uint2(pack_bf16x2(acc.x, acc.y), pack_bf16x2(acc.z, acc.w));
}

}  // namespace gmlp
