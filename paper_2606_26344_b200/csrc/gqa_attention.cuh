// Group Query Attention (one of the paper's multi-operator kernels, Section 6.1), forward, no mask:
//     O_h = softmax( Q_h K_g^T / sqrt(D) ) V_g,      g = h / (Hq / Hkv),      D = 128,
// Q [M, Hq*D], K and V [S, Hkv*D], O [M, Hq*D] row-major bf16.  One CTA per (128 query rows, query head); the
// key/value sequence is walked in blocks of 128 with the running-maximum (online) softmax, so the scores never
// leave the SM: both matmuls run on tcgen05 with their accumulators in TMEM and the probabilities go from
// registers to shared memory as the second matmul's A operand.
//
//   warp 0      TMA producer: Q tile once, then K blocks and V blocks into two two-stage rings of their own
//   warp 1      MMA issuer:   S = Q K^T into one of two TMEM score buffers (columns [0,128) / [128,256)), so the
//                             scores of block j+1 are computed while block j is in the softmax; then
//                             O += P V (TMEM columns [256,384))
//   warps 2..5  softmax:      thread t owns query row t (its TMEM lane), so row maxima and sums need no shuffles;
//                             reads its 128 scores once into registers, writes P (bf16) into the
//                             128-byte-swizzled K-major layout the MMA expects, and at the end stores O / l.
//                             The exponent base is a running maximum that is only moved when a block's maximum
//                             exceeds it by more than 8 (probabilities stay below 2^8), so O in TMEM is rescaled
//                             rarely instead of once per block.
//
// Operand forms: Q and P are K-major A operands (rows of 128 B, two 64-wide swizzle atoms side by side); a K block
// [128 keys, D] is a K-major B operand (keys are the N dimension); a V block [128 keys, D] is an MN-major B
// operand (keys are the K dimension, D the N dimension) read as it lies in memory - no transposed copy of K or V.
// Every wait is bounded (see umma_gemm.cuh).
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"
#include "umma_gemm.cuh"

namespace gmlp {

constexpr int kGqaD = 128;                       // head dimension
constexpr int kGqaBM = 128;                      // query rows per CTA
constexpr int kGqaBS = 128;                      // keys per block
constexpr uint32_t kGqaTileBytes = 128 * 128 * 2;                         // one 128 x 128 bf16 tile: 32 KB
constexpr int kGqaStages = 2;                                             // per ring (K blocks, V blocks)
constexpr uint32_t kGqaSmemBytes = (2 + 2 * kGqaStages) * kGqaTileBytes + 1024 + 256;   // Q, P, K ring, V ring
constexpr float kGqaLazyLog2 = 8.0f;                                      // move the exponent base only beyond this

__device__ __forceinline__ void tmem_st_32x32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__global__ void __launch_bounds__(kUmmaThreads, 1)
gqa_attention_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                     const __grid_constant__ CUtensorMap tmV, bf16* __restrict__ O,
                     int M, int S, int n_q_heads, int group, float scale_log2)
{
    constexpr int KERNEL_ID = 10;
    // S = Q K^T: A and B K-major;  O += P V: A K-major, B MN-major;  both M = 128, N = 128, fp32 accumulate
    constexpr uint32_t kIdescQK = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (0u << 16) |
                                  ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
    constexpr uint32_t kIdescPV = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) |
                                  ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - raw_addr);
    const uint32_t q_smem = base, p_smem = base + kGqaTileBytes;
    const uint32_t k_ring = base + 2 * kGqaTileBytes, v_ring = k_ring + kGqaStages * kGqaTileBytes;
    uint8_t* p_ptr = base_ptr + kGqaTileBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(base_ptr + (2 + 2 * kGqaStages) * kGqaTileBytes);
    const uint32_t k_full0 = ptx::smem_addr(bars);                   // [2]
    const uint32_t k_empty0 = ptx::smem_addr(bars + 2);              // [2]
    const uint32_t v_full0 = ptx::smem_addr(bars + 4);               // [2]
    const uint32_t v_empty0 = ptx::smem_addr(bars + 6);              // [2]
    const uint32_t s_full0 = ptx::smem_addr(bars + 8);               // [2] the scores of a block are in TMEM buffer b
    const uint32_t q_full = ptx::smem_addr(bars + 10);
    const uint32_t p_full = ptx::smem_addr(bars + 11);               // P is in shared memory (and O rescaled if need be)
    const uint32_t o_full = ptx::smem_addr(bars + 12);               // O += P V of a block is done
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 13);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * kGqaBM;
    const int h = blockIdx.y;
    const int g = h / group;
    const int n_blocks = (S + kGqaBS - 1) / kGqaBS;

    ptx::launch_dependents();
    if (threadIdx.x == 0) {
        for (int i = 0; i < 10; ++i) ptx::mbar_init(k_full0 + 8 * i, 1);      // the five two-entry barrier arrays
        ptx::mbar_init(q_full, 1);
        ptx::mbar_init(p_full, 4);                                   // one arrival per softmax warp
        ptx::mbar_init(o_full, 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::fence_proxy_async_smem();
        ptx::prefetch_tensormap(&tmQ);
        ptx::prefetch_tensormap(&tmK);
        ptx::prefetch_tensormap(&tmV);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_addr(tmem_slot), 512);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_o = tmem_base + 256;                         // scores: tmem_base + 128 * (block & 1)

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            ptx::grid_dependency_wait();                             // Q, K, V may come from the previous kernel
            ptx::mbar_arrive_expect_tx(q_full, kGqaTileBytes);
            ptx::tma_load_2d(q_smem, &tmQ, h * kGqaD, m0, q_full);
            ptx::tma_load_2d(q_smem + 16384, &tmQ, h * kGqaD + 64, m0, q_full);
            for (int j = 0; j < n_blocks; ++j) {
                const int s = j % kGqaStages;
                const uint32_t ph = (uint32_t)(j / kGqaStages) & 1u;
                const int s0 = j * kGqaBS;
                // K block: two boxes of 64 d x 128 keys (K-major: a key's d values are contiguous)
                if (!wait_bounded(k_empty0 + 8 * s, ph ^ 1u, abort_flag, KERNEL_ID, 1)) break;
                const uint32_t k_dst = k_ring + s * kGqaTileBytes;
                ptx::mbar_arrive_expect_tx(k_full0 + 8 * s, kGqaTileBytes);
                ptx::tma_load_2d(k_dst, &tmK, g * kGqaD, s0, k_full0 + 8 * s);
                ptx::tma_load_2d(k_dst + 16384, &tmK, g * kGqaD + 64, s0, k_full0 + 8 * s);
                // V block: four boxes of 64 d x 64 keys; (key half, d half) at (2 * key half + d half) * 8 KB
                if (!wait_bounded(v_empty0 + 8 * s, ph ^ 1u, abort_flag, KERNEL_ID, 8)) break;
                const uint32_t v_dst = v_ring + s * kGqaTileBytes;
                ptx::mbar_arrive_expect_tx(v_full0 + 8 * s, kGqaTileBytes);
#pragma unroll
                for (int sh = 0; sh < 2; ++sh)
#pragma unroll
                    for (int nh = 0; nh < 2; ++nh)
                        ptx::tma_load_2d(v_dst + (sh * 2 + nh) * 8192, &tmV, g * kGqaD + nh * 64, s0 + sh * 64,
                                         v_full0 + 8 * s);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            // S(j) = Q K(j)^T over D = 128: eight K = 16 steps, four per 64-wide swizzle atom
            auto issue_scores = [&](int j) -> bool {
                const int s = j % kGqaStages;
                if (!wait_bounded(k_full0 + 8 * s, (uint32_t)(j / kGqaStages) & 1u, abort_flag, KERNEL_ID, 2)) return false;
                ptx::tc_fence_after_sync();
                const uint32_t k_smem = k_ring + s * kGqaTileBytes;
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const uint32_t off = (uint32_t)(k >> 2) * 16384u + (uint32_t)(k & 3) * 32u;
                    ptx::umma_bf16(tmem_base + 128u * (uint32_t)(j & 1), ptx::make_smem_desc_sw128(q_smem + off, 16, 1024),
                                   ptx::make_smem_desc_sw128(k_smem + off, 16, 1024), kIdescQK, k != 0 ? 1u : 0u);
                }
                ptx::umma_commit(s_full0 + 8 * (j & 1));
                ptx::umma_commit(k_empty0 + 8 * s);
                return true;
            };
            bool ok = wait_bounded(q_full, 0u, abort_flag, KERNEL_ID, 5);
            ok = ok && issue_scores(0);
            for (int j = 0; j < n_blocks && ok; ++j) {
                // the scores of the next block are computed while this block is in the softmax: its score buffer
                // was last read for block j-1, whose probabilities the wait below (one iteration ago) has seen
                if (j + 1 < n_blocks && !issue_scores(j + 1)) break;
                const int s = j % kGqaStages;
                if (!wait_bounded(p_full, (uint32_t)j & 1u, abort_flag, KERNEL_ID, 6)) break;
                if (!wait_bounded(v_full0 + 8 * s, (uint32_t)(j / kGqaStages) & 1u, abort_flag, KERNEL_ID, 9)) break;
                ptx::tc_fence_after_sync();
                const uint32_t v_smem = v_ring + s * kGqaTileBytes;
                // O += P V over the block's 128 keys
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const uint64_t a_desc = ptx::make_smem_desc_sw128(
                        p_smem + (uint32_t)(k >> 2) * 16384u + (uint32_t)(k & 3) * 32u, 16, 1024);
                    const uint64_t b_desc = ptx::make_smem_desc_sw128(
                        v_smem + (uint32_t)(k >> 2) * 16384u + (uint32_t)(k & 3) * 2048u, 8192, 1024);
                    ptx::umma_bf16(tmem_o, a_desc, b_desc, kIdescPV, (j | k) != 0 ? 1u : 0u);
                }
                ptx::umma_commit(v_empty0 + 8 * s);
                ptx::umma_commit(o_full);
            }
        }
        __syncwarp();
    } else {
        // ---------------- softmax and epilogue: thread = query row ----------------
        const int q = warp & 3;
        const int r = q * 32 + lane;                                 // row within the tile = TMEM lane
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        float m_use = 0.0f, l_run = 0.0f;                            // exponent base (set on the first block), row sum
        bool ok = true;
        for (int j = 0; j < n_blocks && ok; ++j) {
            if (!wait_bounded(s_full0 + 8 * (j & 1), (uint32_t)(j >> 1) & 1u, abort_flag, KERNEL_ID, 3)) { ok = false; break; }
            ptx::tc_fence_after_sync();
            const int valid = min(kGqaBS, S - j * kGqaBS);           // keys of this block that exist
            const uint32_t s_addr = tmem_base + 128u * (uint32_t)(j & 1) + lane_addr;
            uint32_t sv[4][32];                                      // this row's 128 scores
#pragma unroll
            for (int c = 0; c < 4; ++c) ptx::tmem_ld_32x32(s_addr + 32 * c, sv[c]);
            ptx::tmem_ld_wait();
            float m_blk = -INFINITY;
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (32 * c + i < valid) m_blk = fmaxf(m_blk, __uint_as_float(sv[c][i]) * scale_log2);
            // P of the previous block must have been consumed (and O complete) before P is overwritten
            if (j > 0) {
                if (!wait_bounded(o_full, (uint32_t)(j - 1) & 1u, abort_flag, KERNEL_ID, 4)) { ok = false; break; }
                ptx::tc_fence_after_sync();
            }
            if (j == 0) {
                m_use = m_blk;                                       // finite: the first block has at least one key
            } else if (__any_sync(0xFFFFFFFFu, m_blk > m_use + kGqaLazyLog2)) {
                // some row's maximum moved far: rescale this warp's rows of O (and l) to the new base
                const float m_new = fmaxf(m_use, m_blk);
                const float alpha = ex2_approx(m_use - m_new);
                m_use = m_new;
                l_run *= alpha;
#pragma unroll 1
                for (int c = 0; c < kGqaD; c += 32) {
                    uint32_t v[32];
                    ptx::tmem_ld_32x32(tmem_o + lane_addr + c, v);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
                    tmem_st_32x32(tmem_o + lane_addr + c, v);
                }
                tmem_st_wait();
            }
            // p = 2^(x - base), row sum, P as bf16 into the swizzled K-major tile
            float l_blk = 0.0f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t packed[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float p0 = (32 * c + 2 * i < valid) ? ex2_approx(__uint_as_float(sv[c][2 * i]) * scale_log2 - m_use) : 0.0f;
                    const float p1 = (32 * c + 2 * i + 1 < valid) ? ex2_approx(__uint_as_float(sv[c][2 * i + 1]) * scale_log2 - m_use) : 0.0f;
                    l_blk += p0 + p1;
                    packed[i] = pack_bf16x2(p0, p1);
                }
                // columns 32c .. 32c+31 of row r: four 16-byte chunks of the 64-wide atom (c / 2)
                uint8_t* atom = p_ptr + (size_t)(c >> 1) * 16384 + (size_t)r * 128;
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    const int chunk = (c & 1) * 4 + ch;                              // 0..7 within the 128-byte row
                    *reinterpret_cast<uint4*>(atom + ((chunk ^ (r & 7)) << 4)) =
                        make_uint4(packed[4 * ch], packed[4 * ch + 1], packed[4 * ch + 2], packed[4 * ch + 3]);
                }
            }
            l_run += l_blk;
            ptx::fence_proxy_async_smem();                           // P (generic writes) -> visible to the MMA
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(p_full);
        }
        // epilogue: O / l, one rounding, 256 contiguous bytes per row
        if (ok && wait_bounded(o_full, (uint32_t)(n_blocks - 1) & 1u, abort_flag, KERNEL_ID, 7)) {
            ptx::tc_fence_after_sync();
            const float inv_l = 1.0f / l_run;
            const int row = m0 + r;
            bf16* orow = O + (size_t)row * ((size_t)n_q_heads * kGqaD) + (size_t)h * kGqaD;
#pragma unroll 1
            for (int c = 0; c < kGqaD; c += 32) {
                uint32_t v[32];
                ptx::tmem_ld_32x32(tmem_o + lane_addr + c, v);
                ptx::tmem_ld_wait();
                if (row < M) {
#pragma unroll
                    for (int v4 = 0; v4 < 4; ++v4) {
                        uint32_t pk[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            pk[i] = pack_bf16x2(__uint_as_float(v[8 * v4 + 2 * i]) * inv_l, __uint_as_float(v[8 * v4 + 2 * i + 1]) * inv_l);
                        *reinterpret_cast<uint4*>(orow + c + v4 * 8) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
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
        ptx::tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace gmlp
