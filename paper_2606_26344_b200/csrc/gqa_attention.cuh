// Group Query Attention (one of the paper's multi-operator kernels, Section 6.1), forward, no mask:
//     O_h = softmax( Q_h K_g^T / sqrt(D) ) V_g,      g = h / (Hq / Hkv),      D = 128,
// Q [M, Hq*D], K and V [S, Hkv*D], O [M, Hq*D] row-major bf16.  One CTA per (256 query rows, query head), as TWO
// query tiles of 128 rows that take turns on the tensor pipe: while one tile's scores are in the softmax, the
// other tile's matmuls run.  The key/value sequence is walked in blocks of 128 with the running-maximum (online)
// softmax, so the scores never leave the SM: both matmuls run on tcgen05 with their accumulators in TMEM, and the
// probabilities go from registers back to TMEM, where the second matmul reads them as its A operand.
//
//   warp 0      TMA producer: both Q tiles once, then K(0), V(0), K(1), V(1), ... through one five-slot FIFO
//   warp 1      MMA issuer:   per tile t, S_t = Q_t K^T (TMEM columns 128 t) and O_t += P_t V (columns 256 + 128 t),
//                             in the order PV_A(j), S_A(j+1), PV_B(j), S_B(j+1)
//   warps 2, 3  idle (they fill warp group 0, which gives most of its registers to the softmax groups)
//   warps 4..7  softmax of tile A, warps 8..11 of tile B: thread = query row (its TMEM lane), so row maxima and sums
//                             need no shuffles.  A block's 128 scores are read into registers once and go
//                             through ONE pass of exponentials with the current base (scale folded into the
//                             exponent's FMA, packed fp32 pairs, a quarter of the exponentials as a cubic on the
//                             FMA pipe).  The base is a running maximum that is only moved when some row's sum of
//                             a block exceeds 2^10: only then is the block's row maximum taken, O in TMEM and l
//                             rescaled and the pass repeated (in the first block the maximum comes first).  P (bf16
//                             pairs) overwrites the first 64 columns of the tile's own score buffer; at the end
//                             O / l is stored.
//
// Operand forms: Q is a K-major A operand in shared memory (rows of 128 B, two 64-wide swizzle atoms side by side),
// P an A operand in TMEM (lane = query row, 8 columns of packed pairs per K step of 16 keys); a K block
// [128 keys, D] is a K-major B operand (keys are the N dimension); a V block [128 keys, D] is an MN-major B
// operand (keys are the K dimension, D the N dimension) read as it lies in memory - no transposed copy of K or V.
// Every wait is bounded (see umma_gemm.cuh).
#pragma once
#include <type_traits>
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"
#include "umma_gemm.cuh"

namespace gmlp {

constexpr int kGqaD = 128;                       // head dimension
constexpr int kGqaBM = 256;                      // query rows per CTA (two tiles of 128)
constexpr int kGqaBS = 128;                      // keys per block
constexpr int kGqaThreads = 384;                 // warp group 0: producer warp, MMA warp, two idle; groups 1, 2: softmax
constexpr int kGqaRegsLight = 72, kGqaRegsSoftmax = 216;   // registers per thread after the groups trade (sum kept)
constexpr uint32_t kGqaTileBytes = 128 * 128 * 2;                         // one 128 x 128 bf16 tile: 32 KB
constexpr int kGqaSlots = 5;                                              // K/V FIFO slots
constexpr uint32_t kGqaSmemBytes = (2 + kGqaSlots) * kGqaTileBytes + 1024 + 256;   // Q_A Q_B, FIFO
constexpr float kGqaLazySum = 1024.0f;          // move the exponent base only when a row of a block sums to more

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
// D[tmem] (+)= A[tmem] * B[smem desc]: the A operand (M = 128 rows = lanes, K = 16 per instruction as 8 columns of
// packed 16-bit pairs) is read from tensor memory.
__device__ __forceinline__ void umma_bf16_tmem_a(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// The TMEM-operand form with the shared-memory descriptor given as its two 32-bit words (see ptx::umma_bf16_halves).
__device__ __forceinline__ void umma_bf16_tmem_a_halves(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t desc_hi,
                                                        uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Two fp32 values in one 64-bit register pair: sm_100 adds, multiplies and fuses them two at a time, which halves
// the instruction count of the softmax's scaling and summing (the softmax warps are bound by instruction issue
// and by the special-function unit, not by arithmetic).
__device__ __forceinline__ uint64_t pack_f32x2(float a, float b) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& a, float& b) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.ftz.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.ftz.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float max3_f32(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// 2^x on the FMA pipe for part of the exponentials: x is split into the nearest integer n (taken from the mantissa
// of x + 1.5 * 2^23) and f in [-1/2, 1/2]; 2^f is a cubic fitted for minimum relative error (7.5e-5, a twenty-fifth
// of the bf16 rounding that P gets next); n is added to the exponent field.  Both values of a pair at once.
__device__ __forceinline__ void ex2_poly_x2(float x0, float x1, float& p0, float& p1) {
    const uint64_t x = pack_f32x2(fmaxf(x0, -125.0f), fmaxf(x1, -125.0f));
    const uint64_t t = add_f32x2(x, pack_f32x2(12582912.0f, 12582912.0f));
    const uint64_t n = add_f32x2(t, pack_f32x2(-12582912.0f, -12582912.0f));
    const uint64_t f = fma_f32x2(n, pack_f32x2(-1.0f, -1.0f), x);
    uint64_t p = fma_f32x2(pack_f32x2(0.0551716685f, 0.0551716685f), f, pack_f32x2(0.2426111400f, 0.2426111400f));
    p = fma_f32x2(p, f, pack_f32x2(0.6932609677f, 0.6932609677f));
    p = fma_f32x2(p, f, pack_f32x2(0.9999280572f, 0.9999280572f));
    float q0, q1, t0, t1;
    unpack_f32x2(p, q0, q1);
    unpack_f32x2(t, t0, t1);
    p0 = __int_as_float(__float_as_int(q0) + (__float_as_int(t0) << 23));
    p1 = __int_as_float(__float_as_int(q1) + (__float_as_int(t1) << 23));
}
// Which column pairs take the polynomial: bit (i & 7) for pair i of a 32-column chunk, i.e. two pairs in eight, a
// quarter of the exponentials (measured at 8K tokens: none 1278, an eighth 1294, a quarter 1318, three eighths
// 1250-1269, a half 1152 TFLOP/s - the softmax warps are bound by instruction issue as much as by the
// special-function unit, and a polynomial pair costs five times the instructions of a hardware pair).
#ifndef GMLP_GQA_POLY_MASK
#define GMLP_GQA_POLY_MASK 0x11
#endif

__global__ void __launch_bounds__(kGqaThreads, 1)
gqa_attention_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                     const __grid_constant__ CUtensorMap tmV, bf16* __restrict__ O,
                     int M, int S, int n_q_heads, int group, float scale_log2, int causal_off)
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
    const uint32_t q_smem = base;                                    // + tile * 32 KB
    const uint32_t fifo = base + 2 * kGqaTileBytes;                  // + slot * 32 KB
    uint64_t* bars = reinterpret_cast<uint64_t*>(base_ptr + (2 + kGqaSlots) * kGqaTileBytes);
    const uint32_t kv_full0 = ptx::smem_addr(bars);                  // [slots]
    const uint32_t kv_empty0 = ptx::smem_addr(bars + kGqaSlots);     // [slots]
    const uint32_t s_full0 = ptx::smem_addr(bars + 2 * kGqaSlots);   // [2] tile t: the scores of a block are in TMEM
    const uint32_t p_full0 = ptx::smem_addr(bars + 2 * kGqaSlots + 2);   // [2] tile t: P is in TMEM
    const uint32_t o_full0 = ptx::smem_addr(bars + 2 * kGqaSlots + 4);   // [2] tile t: O += P V of a block is done
    const uint32_t q_full = ptx::smem_addr(bars + 2 * kGqaSlots + 6);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kGqaSlots + 7);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // causal: the query tiles with the longest horizons (the most key blocks) are started first
    const int m0 = (causal_off >= 0 ? (int)(gridDim.x - 1 - blockIdx.x) : (int)blockIdx.x) * kGqaBM;
    const int h = blockIdx.y;
    const int g = h / group;
    // causal_off >= 0: causal attention, query row m sees keys s <= m + causal_off (causal_off = S - M: the queries
    // are the last M positions); blocks entirely beyond the horizon of this CTA's last row are not visited
    int n_blocks = (S + kGqaBS - 1) / kGqaBS;
    if (causal_off >= 0) n_blocks = min(n_blocks, (m0 + kGqaBM - 1 + causal_off) / kGqaBS + 1);

    ptx::launch_dependents();
    if (threadIdx.x == 0) {
        for (int i = 0; i < 2 * kGqaSlots + 2; ++i) ptx::mbar_init(kv_full0 + 8 * i, 1);   // kv_full, kv_empty, s_full
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(p_full0 + 8 * i, 4);                      // one arrival per softmax warp of the tile
            ptx::mbar_init(o_full0 + 8 * i, 1);
        }
        ptx::mbar_init(q_full, 1);
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
    const uint32_t tmem_base = *tmem_slot;                           // S_t at + 128 t, O_t at + 256 + 128 t

    // The launch gives every thread 168 registers (65536 / 384); the softmax threads hold a block's 128 scores and
    // want more, the producer, the MMA issuer and the two idle warps need few: warp group 0 hands registers back
    // and the two softmax groups take them (72 * 128 + 216 * 256 = 168 * 384).  Each form of the instruction sits
    // inside its own branch, so that the compiler knows the budget of the code that follows it.
    if (warp < 4) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kGqaRegsLight));
      if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            ptx::grid_dependency_wait();                             // Q, K, V may come from the previous kernel
            ptx::mbar_arrive_expect_tx(q_full, 2 * kGqaTileBytes);
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                ptx::tma_load_2d(q_smem + t * kGqaTileBytes, &tmQ, h * kGqaD, m0 + 128 * t, q_full);
                ptx::tma_load_2d(q_smem + t * kGqaTileBytes + 16384, &tmQ, h * kGqaD + 64, m0 + 128 * t, q_full);
            }
            for (int i = 0; i < 2 * n_blocks; ++i) {                 // item 2j = K(j), item 2j+1 = V(j)
                const int slot = i % kGqaSlots;
                if (!wait_bounded(kv_empty0 + 8 * slot, ((uint32_t)(i / kGqaSlots) & 1u) ^ 1u, abort_flag, KERNEL_ID, 1)) break;
                const uint32_t full = kv_full0 + 8 * slot;
                const uint32_t dst = fifo + slot * kGqaTileBytes;
                const int s0 = (i >> 1) * kGqaBS;
                ptx::mbar_arrive_expect_tx(full, kGqaTileBytes);
                if ((i & 1) == 0) {
                    // K block: two boxes of 64 d x 128 keys (K-major: a key's d values are contiguous)
                    ptx::tma_load_2d(dst, &tmK, g * kGqaD, s0, full);
                    ptx::tma_load_2d(dst + 16384, &tmK, g * kGqaD + 64, s0, full);
                } else {
                    // V block: four boxes of 64 d x 64 keys; (key half, d half) at (2 * key half + d half) * 8 KB
#pragma unroll
                    for (int sh = 0; sh < 2; ++sh)
#pragma unroll
                        for (int nh = 0; nh < 2; ++nh)
                            ptx::tma_load_2d(dst + (sh * 2 + nh) * 8192, &tmV, g * kGqaD + nh * 64, s0 + sh * 64, full);
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        // All 32 lanes run the loop, its waits and its arithmetic, so that everything the MMAs take is warp-uniform
        // (the tensor-core instructions read their operands from uniform registers; inside a one-lane branch every
        // operand has to be moved there per MMA); only the instructions themselves sit under the elected lane.
        {
            const bool leader = ptx::elect_one();
            // The issuing thread is a single dependent instruction stream with a budget of 64 cycles per MMA, so
            // nothing is derived per MMA: the FIFO position is stepped, not divided, and the descriptors of a group
            // of eight K = 16 steps are formed (base + constant, independent of one another) before its first MMA.
            // In 16-byte units a step advances a K-major operand by 2 within a 64-wide swizzle atom and by 1024 to
            // the next atom of 128 rows; the MN-major V operand by 128 per 16 keys and by 1024 per 64 keys.
            uint32_t it_slot = 0, it_phase = 0;                      // next K/V item (K(0), V(0), K(1), ...) to wait for
            auto wait_next = [&](int site, uint32_t& slot_out) -> bool {
                const bool ok = __all_sync(0xFFFFFFFFu, wait_bounded(kv_full0 + 8 * it_slot, it_phase, abort_flag, KERNEL_ID, site));
                ptx::tc_fence_after_sync();
                slot_out = it_slot;
                if (++it_slot == (uint32_t)kGqaSlots) { it_slot = 0; it_phase ^= 1u; }
                return ok;
            };
            // (the upper word of every descriptor here is the same: stride 1024 B, version 1, 128-byte swizzle; only
            // the lower words, start address and leading offset, are kept per step)
            const uint32_t desc_hi = (uint32_t)(ptx::make_smem_desc_sw128(0, 0, 1024) >> 32);
            const uint32_t q_lo0 = (uint32_t)ptx::make_smem_desc_sw128(q_smem, 16, 1024);
            const uint32_t q_lo1 = (uint32_t)ptx::make_smem_desc_sw128(q_smem + kGqaTileBytes, 16, 1024);
            const uint32_t k_lo_base = (uint32_t)ptx::make_smem_desc_sw128(fifo, 16, 1024);
            const uint32_t v_lo_base = (uint32_t)ptx::make_smem_desc_sw128(fifo, 8192, 1024);
            // S_t = Q_t K^T over D = 128 with the K block in FIFO slot `slot`
            auto issue_scores = [&](int t, uint32_t slot) {
                const uint32_t a0 = t ? q_lo1 : q_lo0;
                const uint32_t b0 = k_lo_base + slot * (kGqaTileBytes >> 4);
                uint32_t ad[8], bd[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    ad[k] = a0 + (uint32_t)((k >> 2) * 1024 + (k & 3) * 2);
                    bd[k] = b0 + (uint32_t)((k >> 2) * 1024 + (k & 3) * 2);
                }
                if (leader) {
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        ptx::umma_bf16_halves(tmem_base + 128u * (uint32_t)t, ad[k], bd[k], desc_hi, kIdescQK, k != 0 ? 1u : 0u);
                    ptx::umma_commit(s_full0 + 8 * t);
                    if (t == 1) ptx::umma_commit(kv_empty0 + 8 * slot);          // both tiles have used this K block
                }
                __syncwarp();
            };
            uint32_t k_slot = 0, v_slot = 0;
            bool ok = __all_sync(0xFFFFFFFFu, wait_bounded(q_full, 0u, abort_flag, KERNEL_ID, 5)) && wait_next(2, k_slot);
            if (ok) {
                issue_scores(0, k_slot);
                issue_scores(1, k_slot);
            }
            for (int j = 0; j < n_blocks && ok; ++j) {
                for (int t = 0; t < 2 && ok; ++t) {
                    // tile t's probabilities of block j are in TMEM; V(j) has landed
                    if (!__all_sync(0xFFFFFFFFu, wait_bounded(p_full0 + 8 * t, (uint32_t)j & 1u, abort_flag, KERNEL_ID, 6))) { ok = false; break; }
                    if (t == 0 && !wait_next(9, v_slot)) { ok = false; break; }
                    ptx::tc_fence_after_sync();
                    {
                        // A = P_t from TMEM: 16 keys of a K step are 8 columns of packed bf16 pairs
                        const uint32_t v0 = v_lo_base + v_slot * (kGqaTileBytes >> 4);
                        const uint32_t d_tmem = tmem_base + 256u + 128u * (uint32_t)t, p_tmem = tmem_base + 128u * (uint32_t)t;
                        uint32_t bd[8];
#pragma unroll
                        for (int k = 0; k < 8; ++k) bd[k] = v0 + (uint32_t)((k >> 2) * 1024 + (k & 3) * 128);
                        if (leader) {
                            umma_bf16_tmem_a_halves(d_tmem, p_tmem, bd[0], desc_hi, kIdescPV, j != 0 ? 1u : 0u);
#pragma unroll
                            for (int k = 1; k < 8; ++k)
                                umma_bf16_tmem_a_halves(d_tmem, p_tmem + 8u * (uint32_t)k, bd[k], desc_hi, kIdescPV, 1u);
                            ptx::umma_commit(o_full0 + 8 * t);
                            if (t == 1) ptx::umma_commit(kv_empty0 + 8 * v_slot);    // both tiles have used V(j)
                        }
                        __syncwarp();
                    }
                    // the tile's next scores follow at once: its score buffer was consumed before p_full
                    if (j + 1 < n_blocks) {
                        if (t == 0 && !wait_next(2, k_slot)) { ok = false; break; }
                        issue_scores(t, k_slot);
                    }
                }
            }
        }
        __syncwarp();
      }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kGqaRegsSoftmax));
        // ---------------- softmax and epilogue: one group of four warps per tile, thread = query row ----------------
        const int t = (warp - 4) >> 2;                               // tile
        const int q = warp & 3;
        const int r = q * 32 + lane;                                 // row within the tile = TMEM lane
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        const uint32_t s_addr = tmem_base + 128u * (uint32_t)t + lane_addr;
        const uint32_t o_addr = tmem_base + 256u + 128u * (uint32_t)t + lane_addr;
        float m_use = -INFINITY, l_run = 0.0f;                       // exponent base, row sum
        bool ok = true;
        // last key this row may see (causal), or none of that
        const int horizon = causal_off >= 0 ? m0 + 128 * t + r + causal_off : 0x7FFFFFFF - kGqaBS;

        // One block: the scores come from TMEM into registers once; P goes back to TMEM as packed bf16 pairs over
        // the first 64 columns of the tile's own score buffer (its scores are in registers by then): the second
        // matmul reads its A operand from there, so P never crosses shared memory.  Only a block with keys a row
        // may not see (the last one, or the diagonal under a causal mask) pays for the masking.
        auto block_pass = [&](auto masked_tag, int j, int valid) {
            constexpr bool masked = decltype(masked_tag)::value;
            uint32_t v[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) ptx::tmem_ld_32x32(s_addr + 32 * c, v[c]);
            ptx::tmem_ld_wait();
            if constexpr (masked) {
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (32 * c + i >= valid) v[c][i] = 0xFF800000u;                  // -inf
            }
            // exponentials of the block with the current base: P to TMEM, returns the row's sum
            auto exp_pass = [&]() -> float {
                const uint64_t scale2 = pack_f32x2(scale_log2, scale_log2), neg_base2 = pack_f32x2(-m_use, -m_use);
                uint64_t l_acc2 = pack_f32x2(0.0f, 0.0f);
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    uint32_t packed[32];
#pragma unroll
                    for (int ci = 0; ci < 32; ++ci) {
                        const int c = 2 * hh + (ci >> 4), i = ci & 15;
                        float e0, e1;
                        unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(v[c][2 * i]), __uint_as_float(v[c][2 * i + 1])),
                                               scale2, neg_base2), e0, e1);
                        float p0, p1;
                        if ((GMLP_GQA_POLY_MASK >> (i & 7)) & 1) {
                            ex2_poly_x2(e0, e1, p0, p1);
                        } else {
                            p0 = ex2_approx(e0);
                            p1 = ex2_approx(e1);
                        }
                        l_acc2 = add_f32x2(l_acc2, pack_f32x2(p0, p1));
                        packed[ci] = pack_bf16x2(p0, p1);
                    }
                    tmem_st_32x32(s_addr + 32 * hh, packed);         // P columns 64 hh .. 64 hh + 63 as 32 pairs
                }
                float l0, l1;
                unpack_f32x2(l_acc2, l0, l1);
                return l0 + l1;
            };
            // The row maximum (64 three-input maxima, 290 cycles of a half-rate pipe, on the critical path of the
            // tile) is only taken when it is needed: in the first block, and when some row's sum of exponentials
            // with the current base says that the base is far too low.  The sum bounds every term: below
            // kGqaLazySum nothing can overflow and P keeps its relative precision, whatever the base.
            float l_blk = 0.0f;
            bool moved = j == 0;
            if (j > 0) {
                l_blk = exp_pass();
                moved = __any_sync(0xFFFFFFFFu, !(l_blk <= kGqaLazySum));        // also catches inf and NaN
            }
            if (moved) {
                float m_raw = -INFINITY;
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        m_raw = max3_f32(m_raw, __uint_as_float(v[c][2 * i]), __uint_as_float(v[c][2 * i + 1]));
                const float m_new = fmaxf(m_use, m_raw * scale_log2);            // the scale is positive
                if (j > 0) {
                    // O of the blocks so far is complete: this block's scores were issued after their matmuls
                    const float alpha = ex2_approx(m_use - m_new);
                    l_run *= alpha;
#pragma unroll 1
                    for (int c = 0; c < kGqaD; c += 32) {
                        uint32_t o[32];
                        ptx::tmem_ld_32x32(o_addr + c, o);
                        ptx::tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                        tmem_st_32x32(o_addr + c, o);
                    }
                }
                m_use = m_new;
                l_blk = exp_pass();
            }
            l_run += l_blk;
            tmem_st_wait();
        };

        for (int j = 0; j < n_blocks && ok; ++j) {
            // the scores of block j are complete, and with them every matmul issued before them: O += P V of block
            // j - 1 is done and has read its P
            // (the outcome is made warp-uniform: a warp must not split around the warp-wide instructions below)
            if (!__all_sync(0xFFFFFFFFu, wait_bounded(s_full0 + 8 * t, (uint32_t)j & 1u, abort_flag, KERNEL_ID, 3))) { ok = false; break; }
            ptx::tc_fence_after_sync();
            // keys of this block that exist and that this row may see (0 when the whole block is beyond its horizon)
            const int valid = max(0, min(min(kGqaBS, S - j * kGqaBS), horizon - j * kGqaBS + 1));
            if (__any_sync(0xFFFFFFFFu, valid < kGqaBS)) block_pass(std::true_type{}, j, valid);
            else block_pass(std::false_type{}, j, valid);
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(p_full0 + 8 * t);
        }
        // epilogue: O / l, one rounding, 256 contiguous bytes per row
        if (ok && __all_sync(0xFFFFFFFFu, wait_bounded(o_full0 + 8 * t, (uint32_t)(n_blocks - 1) & 1u, abort_flag, KERNEL_ID, 7))) {
            ptx::tc_fence_after_sync();
            const float inv_l = 1.0f / l_run;
            const int row = m0 + 128 * t + r;
            bf16* orow = O + (size_t)row * ((size_t)n_q_heads * kGqaD) + (size_t)h * kGqaD;
#pragma unroll 1
            for (int c = 0; c < kGqaD; c += 32) {
                uint32_t v[32];
                ptx::tmem_ld_32x32(o_addr + c, v);
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
