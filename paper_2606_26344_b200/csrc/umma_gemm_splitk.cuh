// Down-projection GEMM for medium M when there are far fewer output tiles than SMs.
//
// With one or two 128-row blocks, Y = H * Wd has only a few dozen 128 x 128 output tiles, and one
// CTA per tile cannot pull its whole weight panel from HBM fast enough (a single SM sustains roughly
// 50 GB/s through a TMA ring).  Here a thread-block cluster of S CTAs shares one output tile: CTA r
// of the cluster runs the tcgen05 main loop over the r-th share of the K range, so S times as many
// SMs stream the weights.  The partial accumulators are then reduced ON CHIP: after a cluster
// barrier (every CTA's MMAs are done, the TMA rings are free) the non-leader CTAs copy their fp32
// accumulators from TMEM into the leader's shared memory through distributed shared memory
// (st.shared::cluster), a second cluster barrier publishes them, and the leader adds them to its own
// accumulator in rank order (deterministic), rounds once and stores Y.  No partial ever touches
// global memory and nothing waits on global flags.
//
// Tile 128 x 128, BK = 64, six stages of 32 KB (A 16 KB + two 64-column weight boxes), one tile per
// cluster (the grid is tiles x S CTAs).  Operand layouts and descriptors as in umma_gemm.cuh.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"
#include "umma_gemm.cuh"
#include "umma_gemm_2cta.cuh"

namespace gmlp {

constexpr int kSplitStages = 6;
constexpr uint32_t kSplitStageBytes = kUmmaABytes + 2 * kUmmaBoxBBytes;          // 32 KB
constexpr uint32_t kSplitSmemBytes = kSplitStages * kSplitStageBytes + 1024 + 256;
constexpr uint32_t kSplitPartialBytes = 128 * 128 * 4;                           // one CTA's fp32 tile: 64 KB

__device__ __forceinline__ void st_cluster_f32x4(uint32_t cluster_addr, float a, float b, float c, float d) {
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "f"(a), "f"(b), "f"(c), "f"(d)
                 : "memory");
}

template <int S>
__global__ void __launch_bounds__(kUmmaThreads, 1)
umma_splitk_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                        bf16* __restrict__ C, int M, int K, int N, int num_m_tiles, int a_box_rows, int w_kmajor, int out_fp32)
{
    static_assert(S >= 2 && (S - 1) * kSplitPartialBytes <= kSplitStages * kSplitStageBytes, "staging must fit the ring");
    constexpr int KERNEL_ID = 9;
    // D = fp32, A = B = bf16, A K-major, B MN-major, M = 128, N = 128
    // (with w_kmajor the weights are stored [N, K] and B is K-major like A: bit 16 clear)
    const uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | ((w_kmajor ? 0u : 1u) << 16) |
                            ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - raw_addr);
    uint64_t* bars = reinterpret_cast<uint64_t*>(base_ptr + kSplitStages * kSplitStageBytes);
    const uint32_t full0 = ptx::smem_addr(bars);
    const uint32_t empty0 = ptx::smem_addr(bars + kSplitStages);
    const uint32_t tfull = ptx::smem_addr(bars + 2 * kSplitStages);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kSplitStages + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();
    const int tile = blockIdx.x / S;
    const int m0 = (tile % num_m_tiles) * 128;
    const int n0 = (tile / num_m_tiles) * 128;
    const int nkb = (K + kUmmaBK - 1) / kUmmaBK;
    const int kb0 = (int)(((long long)rank * nkb) / S), kb1 = (int)(((long long)(rank + 1) * nkb) / S);

    ptx::launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < kSplitStages; ++s) {
            ptx::mbar_init(full0 + 8 * s, 1);
            ptx::mbar_init(empty0 + 8 * s, 1);
        }
        ptx::mbar_init(tfull, 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::fence_proxy_async_smem();
        ptx::prefetch_tensormap(&tmA);
        ptx::prefetch_tensormap(&tmB);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_addr(tmem_slot), 128);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    // producer and MMA issuer run their loops warp-uniformly; the copies and the tensor-core instructions sit under the
    // elected lane (see umma_gemm.cuh)
    if (warp == 0) {
        {
            const bool leader = ptx::elect_one();
            auto load_weights = [&](int kb, uint32_t stage) {      // arms the stage's barrier for the whole stage
                const uint32_t full = full0 + 8 * stage;
                const uint32_t b_dst = base + stage * kSplitStageBytes + kUmmaABytes;
                if (!leader) return;
                ptx::mbar_arrive_expect_tx(full, (uint32_t)a_box_rows * 128u + 2 * kUmmaBoxBBytes);
                if (w_kmajor) {
                    ptx::tma_load_2d(b_dst, &tmB, kb * kUmmaBK, n0, full);
                    ptx::tma_load_2d(b_dst + kUmmaBoxBBytes, &tmB, kb * kUmmaBK, n0 + 64, full);
                } else {
                    ptx::tma_load_2d(b_dst, &tmB, n0, kb * kUmmaBK, full);
                    ptx::tma_load_2d(b_dst + kUmmaBoxBBytes, &tmB, n0 + 64, kb * kUmmaBK, full);
                }
            };
            // The weight tiles of the first ring-full of k-blocks do not depend on the previous kernel: they are requested
            // ahead of the wait (the caller's contract on when weights are read is in gmlp.h, "Stream order")
            const int head = kb1 - kb0 < kSplitStages ? kb1 - kb0 : kSplitStages;
            for (int i = 0; i < head; ++i) load_weights(kb0 + i, (uint32_t)i);
            ptx::grid_dependency_wait();
            uint32_t s = 0, ph = 0;                                // ring position, stepped
            for (int kb = kb0; kb < kb1; ++kb) {
                const bool ahead = kb - kb0 < head;                // this stage's barrier is armed and its weights are on their way
                if (!ahead && !__all_sync(0xFFFFFFFFu, wait_bounded(empty0 + 8 * s, ph ^ 1u, abort_flag, KERNEL_ID, 1))) break;
                if (!ahead) load_weights(kb, s);
                if (leader) ptx::tma_load_2d(base + s * kSplitStageBytes, &tmA, kb * kUmmaBK, m0, full0 + 8 * s);
                __syncwarp();
                if (++s == (uint32_t)kSplitStages) { s = 0; ph ^= 1u; }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        {
            const bool leader = ptx::elect_one();
            // lean issue loop: see umma_gemm.cuh (stepped ring position, one addition per descriptor)
            const uint32_t desc_hi = (uint32_t)(ptx::make_smem_desc_sw128(0, 0, 1024) >> 32);
            const uint32_t a_lo0 = (uint32_t)ptx::make_smem_desc_sw128(base, 16, 1024);
            const uint32_t b_lo0 = w_kmajor ? (uint32_t)ptx::make_smem_desc_sw128(base + kUmmaABytes, 16, 1024)
                                            : (uint32_t)ptx::make_smem_desc_sw128(base + kUmmaABytes, kUmmaBoxBBytes, 1024);
            const uint32_t b_step = w_kmajor ? 2u : 128u;
            uint32_t s = 0, ph = 0;
            bool ok = true;
            for (int kb = kb0; kb < kb1; ++kb) {
                if (!__all_sync(0xFFFFFFFFu, wait_bounded(full0 + 8 * s, ph, abort_flag, KERNEL_ID, 2))) { ok = false; break; }
                ptx::tc_fence_after_sync();
                const uint32_t a_lo = a_lo0 + s * (kSplitStageBytes >> 4), b_lo = b_lo0 + s * (kSplitStageBytes >> 4);
                if (leader) {
                    ptx::umma_bf16_halves(tmem_base, a_lo, b_lo, desc_hi, kIdesc, kb != kb0 ? 1u : 0u);
#pragma unroll
                    for (int k = 1; k < kUmmaBK / 16; ++k)
                        ptx::umma_bf16_halves(tmem_base, a_lo + 2u * (uint32_t)k, b_lo + b_step * (uint32_t)k, desc_hi, kIdesc, 1u);
                    ptx::umma_commit(empty0 + 8 * s);
                }
                __syncwarp();
                if (++s == (uint32_t)kSplitStages) { s = 0; ph ^= 1u; }
            }
            if (ok && leader) ptx::umma_commit(tfull);
            __syncwarp();
        }
        __syncwarp();
    }

    // every thread: wait until this CTA's accumulator is complete (which also means its MMAs no longer read the ring)
    const bool acc_ok = wait_bounded(tfull, 0u, abort_flag, KERNEL_ID, 3);
    ptx::tc_fence_after_sync();
    __syncthreads();
    ptx::cluster_sync();                                   // all rings of the cluster are free from here on

    const int q = warp & 3;
    const int rloc = q * 32 + lane;                        // row within the tile = TMEM lane (epilogue warps 2..5)
    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
    if (warp >= 2 && rank > 0) {
        // copy this CTA's fp32 accumulator into the leader's ring: float4 (c4, row) at index c4 * 128 + row
        const uint32_t remote = ptx::map_to_cta(base, 0) + (rank - 1) * kSplitPartialBytes;
#pragma unroll 1
        for (int c = 0; c < 128; c += 32) {
            uint32_t v[32];
            ptx::tmem_ld_32x32(taddr + c, v);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const bool z = !acc_ok;
                st_cluster_f32x4(remote + (uint32_t)(((c >> 2) + j) * 128 + rloc) * 16u,
                                 z ? 0.f : __uint_as_float(v[4 * j]), z ? 0.f : __uint_as_float(v[4 * j + 1]),
                                 z ? 0.f : __uint_as_float(v[4 * j + 2]), z ? 0.f : __uint_as_float(v[4 * j + 3]));
            }
        }
    }
    __syncthreads();
    ptx::cluster_sync();                                   // the partials are in the leader's shared memory
    if (warp >= 2 && rank == 0) {
        ptx::grid_dependency_wait();                       // C may still be read by the previous kernel
        const int row = m0 + rloc;
        bf16* crow = C + (size_t)row * N + n0;
        const float4* stage = reinterpret_cast<const float4*>(base_ptr);
#pragma unroll 1
        for (int c = 0; c < 128; c += 32) {
            uint32_t v[32];
            ptx::tmem_ld_32x32(taddr + c, v);
            ptx::tmem_ld_wait();
            uint32_t packed[16];
            float* frow = reinterpret_cast<float*>(C) + (size_t)row * N + n0 + c;     // used when Y is kept in fp32
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                float4 acc = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                         __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
#pragma unroll
                for (int s = 1; s < S; ++s) {                // fixed rank order
                    const float4 p = stage[(size_t)(s - 1) * (kSplitPartialBytes / 16) + ((c >> 2) + j) * 128 + rloc];
                    acc.x += p.x; acc.y += p.y; acc.z += p.z; acc.w += p.w;
                }
                packed[2 * j] = pack_bf16x2(acc.x, acc.y);
                packed[2 * j + 1] = pack_bf16x2(acc.z, acc.w);
                if (out_fp32 && row < M && acc_ok && n0 + c + j * 4 < N) *reinterpret_cast<float4*>(frow + j * 4) = acc;
            }
            if (!out_fp32 && row < M && acc_ok) {
#pragma unroll
                for (int v4 = 0; v4 < 4; ++v4) {
                    if (n0 + c + v4 * 8 < N)
                        *reinterpret_cast<uint4*>(crow + c + v4 * 8) =
                            make_uint4(packed[4 * v4], packed[4 * v4 + 1], packed[4 * v4 + 2], packed[4 * v4 + 3]);
                }
            }
        }
    }

    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, 128);
    }
}

}  // namespace gmlp
