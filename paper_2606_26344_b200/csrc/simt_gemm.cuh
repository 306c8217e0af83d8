// CUDA-core tiled GEMM with the two epilogues of the Gated MLP.  Any shape (K, N multiples
// of 8), fp32 accumulation.  This is the slow, simple schedule used for bring-up, for shapes
// the tensor-core path does not take, and as an on-GPU cross-check of the fast kernels.
//   GATEUP = true :  C = bf16_rn( silu(A*B0) * (A*B1) )      (figure "mlp-example": matmul, matmul, silu, multiply)
//   GATEUP = false:  C = bf16_rn( A*B0 )                      (the down-projection matmul)
// A [M,K], B0/B1 [K,N], C [M,N]: row-major bf16.
#pragma once
#include "common.cuh"

namespace gmlp {

constexpr int kSimtTile = 64;
constexpr int kSimtBK = 16;

template <bool GATEUP>
__global__ void __launch_bounds__(256)
simt_gemm_kernel(const bf16* __restrict__ A, const bf16* __restrict__ B0, const bf16* __restrict__ B1,
                 bf16* __restrict__ C, int64_t M, int K, int N, GateAct act)
{
    __shared__ float As[kSimtBK][kSimtTile + 4];
    __shared__ float Bs0[kSimtBK][kSimtTile];
    __shared__ float Bs1[GATEUP ? kSimtBK : 1][kSimtTile];

    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int64_t m0 = (int64_t)blockIdx.y * kSimtTile;
    const int n0 = blockIdx.x * kSimtTile;

    float acc0[4][4], acc1[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) { acc0[i][j] = 0.0f; acc1[i][j] = 0.0f; }

    const int a_row = tid >> 2, a_k = (tid & 3) * 4;        // A tile: 64 rows x 16 k, 4 elements per thread
    const int b_k = tid >> 4, b_n = (tid & 15) * 4;         // B tile: 16 k x 64 n, 4 elements per thread

    for (int k0 = 0; k0 < K; k0 += kSimtBK) {
        {
            uint2 v = make_uint2(0u, 0u);
            if (m0 + a_row < M && k0 + a_k < K)
                v = *reinterpret_cast<const uint2*>(A + (m0 + a_row) * K + k0 + a_k);
            As[a_k + 0][a_row] = bf16_lo(v.x); As[a_k + 1][a_row] = bf16_hi(v.x);
            As[a_k + 2][a_row] = bf16_lo(v.y); As[a_k + 3][a_row] = bf16_hi(v.y);
        }
        {
            uint2 v = make_uint2(0u, 0u), w = make_uint2(0u, 0u);
            if (k0 + b_k < K && n0 + b_n < N) {
                v = *reinterpret_cast<const uint2*>(B0 + (int64_t)(k0 + b_k) * N + n0 + b_n);
                if (GATEUP) w = *reinterpret_cast<const uint2*>(B1 + (int64_t)(k0 + b_k) * N + n0 + b_n);
            }
            Bs0[b_k][b_n + 0] = bf16_lo(v.x); Bs0[b_k][b_n + 1] = bf16_hi(v.x);
            Bs0[b_k][b_n + 2] = bf16_lo(v.y); Bs0[b_k][b_n + 3] = bf16_hi(v.y);
            if (GATEUP) {
                Bs1[b_k][b_n + 0] = bf16_lo(w.x); Bs1[b_k][b_n + 1] = bf16_hi(w.x);
                Bs1[b_k][b_n + 2] = bf16_lo(w.y); Bs1[b_k][b_n + 3] = bf16_hi(w.y);
            }
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kSimtBK; ++kk) {
            float a[4], b0[4], b1[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) { b0[j] = Bs0[kk][tx * 4 + j]; b1[j] = GATEUP ? Bs1[kk][tx * 4 + j] : 0.0f; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    acc0[i][j] = fmaf(a[i], b0[j], acc0[i][j]);
                    if (GATEUP) acc1[i][j] = fmaf(a[i], b1[j], acc1[i][j]);
                }
        }
        __syncthreads();
    }

    const int n = n0 + tx * 4;
    if (n >= N) return;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t m = m0 + ty * 4 + i;
        if (m >= M) continue;
        float o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) o[j] = GATEUP ? gate_act_f32(acc0[i][j], act) * acc1[i][j] : acc0[i][j];
        *reinterpret_cast<uint2*>(C + m * N + n) = make_uint2(pack_bf16x2(o[0], o[1]), pack_bf16x2(o[2], o[3]));
    }
}

}  // namespace gmlp
