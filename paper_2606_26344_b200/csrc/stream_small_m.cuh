// Small-M schedule: weight-streaming split-K GEMMs on CUDA cores.
//
// For a handful of tokens the Gated MLP is bound by reading the three weight matrices once
// from HBM.  Each CTA owns a slab of 256 output columns and one K-chunk; its four warps walk
// the chunk's weight rows interleaved (row k, k+4, ...), each lane reading 16 bytes (8 bf16
// columns) per row with several rows in flight, and keep MT x 8 fp32 accumulators per lane.
// The four warps' sums are combined through shared memory, the CTA writes one fp32 partial
// tile, and the LAST CTA to arrive on a slab (atomic ticket, no waiting anywhere) adds the
// partials in fixed K-chunk order and applies the epilogue, so results are deterministic.
//   GATEUP: two weight matrices (blockIdx.y parity); epilogue H = bf16_rn(silu(g) * u)
//   else  : one matrix; epilogue Y = bf16_rn(sum)
// SiLU is not linear, so the K-split must be reduced before it: that is why the epilogue
// lives in the last-arriver and not in each CTA.
#pragma once
#include "common.cuh"

namespace gmlp {

constexpr int kStreamThreads = 128;
constexpr int kStreamWarps = kStreamThreads / 32;
constexpr int kStreamSlab = 256;         // output columns per CTA (32 lanes x 8)
constexpr int kStreamMaxChunk = 1024;    // K rows per CTA at most (x tile lives in shared memory)
constexpr int kStreamUnroll = 8;         // weight rows in flight per warp

template <int MT, bool GATEUP>
__global__ void __launch_bounds__(kStreamThreads, 4)
stream_gemm_kernel(const bf16* __restrict__ A, const bf16* __restrict__ W0, const bf16* __restrict__ W1,
                   float* __restrict__ partial, unsigned int* __restrict__ counters, bf16* __restrict__ out,
                   int M, int K, int N, int kchunk, int KS, GateAct act)
{
    constexpr int NMAT = GATEUP ? 2 : 1;
    __shared__ __align__(16) float xs[kStreamMaxChunk][MT];
    __shared__ __align__(16) float red[kStreamWarps][kStreamSlab];
    __shared__ int is_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int slab = blockIdx.x;
    const int mat = GATEUP ? (blockIdx.y & 1) : 0;
    const int ks = GATEUP ? (blockIdx.y >> 1) : blockIdx.y;
    const int m0 = blockIdx.z * MT;
    const int rows = min(MT, M - m0);
    const int k0 = ks * kchunk;
    const int klen = min(kchunk, K - k0);

    // x tile -> shared memory as fp32, [k][m] so that one k's MT values are contiguous
    for (int m = 0; m < MT; ++m) {
        for (int kk = tid; kk < klen; kk += kStreamThreads)
            xs[kk][m] = (m < rows) ? __bfloat162float(A[(size_t)(m0 + m) * K + k0 + kk]) : 0.0f;
    }
    __syncthreads();

    const int n = slab * kStreamSlab + lane * 8;
    const bool active = n < N;
    const bf16* W = (mat ? W1 : W0) + (size_t)k0 * N + n;

    float acc[MT][8];
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[m][j] = 0.0f;

    for (int kk = warp; kk < klen; kk += kStreamWarps * kStreamUnroll) {
        uint4 w[kStreamUnroll];
#pragma unroll
        for (int u = 0; u < kStreamUnroll; ++u) {
            const int k = kk + u * kStreamWarps;
            w[u] = (active && k < klen) ? ld_stream_16B(W + (size_t)k * N) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < kStreamUnroll; ++u) {
            const int k = min(kk + u * kStreamWarps, klen - 1);   // rows past the chunk carry zero weights
            float wf[8];
            wf[0] = bf16_lo(w[u].x); wf[1] = bf16_hi(w[u].x); wf[2] = bf16_lo(w[u].y); wf[3] = bf16_hi(w[u].y);
            wf[4] = bf16_lo(w[u].z); wf[5] = bf16_hi(w[u].z); wf[6] = bf16_lo(w[u].w); wf[7] = bf16_hi(w[u].w);
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                const float xv = xs[k][m];
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[m][j] = fmaf(xv, wf[j], acc[m][j]);
            }
        }
    }

    // combine the four warps through shared memory, one token row at a time, and write the partial tile
    const int c = tid * 2;                                       // this thread's two columns of the slab
    const int nc = slab * kStreamSlab + c;
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        *reinterpret_cast<float4*>(&red[warp][lane * 8]) = make_float4(acc[m][0], acc[m][1], acc[m][2], acc[m][3]);
        *reinterpret_cast<float4*>(&red[warp][lane * 8 + 4]) = make_float4(acc[m][4], acc[m][5], acc[m][6], acc[m][7]);
        __syncthreads();
        if (m < rows && nc < N) {
            float s0 = 0.0f, s1 = 0.0f;
#pragma unroll
            for (int w = 0; w < kStreamWarps; ++w) { s0 += red[w][c]; s1 += red[w][c + 1]; }
            float* p = partial + ((size_t)(mat * KS + ks) * M + (m0 + m)) * N + nc;
            __stcg(reinterpret_cast<float2*>(p), make_float2(s0, s1));
        }
        __syncthreads();
    }

    // arrival ticket: the last CTA of this (row tile, slab) reduces and applies the epilogue
    __threadfence();
    __syncthreads();
    unsigned int* counter = counters + blockIdx.z * gridDim.x + slab;
    if (tid == 0) {
        const unsigned int ticket = atomicAdd(counter, 1u);
        is_last = (ticket == (unsigned int)(NMAT * KS - 1));
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    if (nc < N) {
        // K-chunks are added in ascending order; the MT rows are independent, so each chunk's loads overlap
        float2 g[MT], u[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) { g[m] = make_float2(0.0f, 0.0f); u[m] = make_float2(0.0f, 0.0f); }
        for (int s = 0; s < KS; ++s) {
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                if (m < rows) {
                    const float2 pg = __ldcg(reinterpret_cast<const float2*>(
                        partial + ((size_t)s * M + (m0 + m)) * N + nc));
                    g[m].x += pg.x; g[m].y += pg.y;
                    if (GATEUP) {
                        const float2 pu = __ldcg(reinterpret_cast<const float2*>(
                            partial + ((size_t)(KS + s) * M + (m0 + m)) * N + nc));
                        u[m].x += pu.x; u[m].y += pu.y;
                    }
                }
            }
        }
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            if (m < rows) {
                const float o0 = GATEUP ? gate_act_f32(g[m].x, act) * u[m].x : g[m].x;
                const float o1 = GATEUP ? gate_act_f32(g[m].y, act) * u[m].y : g[m].y;
                *reinterpret_cast<uint32_t*>(out + (size_t)(m0 + m) * N + nc) = pack_bf16x2(o0, o1);
            }
        }
    }
    if (tid == 0) *counter = 0u;     // leave the counter clean for the next call
}

}  // namespace gmlp
