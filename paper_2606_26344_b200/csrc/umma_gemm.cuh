// Large-M schedule: tcgen05 tensor-core GEMMs with the Gated-MLP epilogues.
//
//   GATEUP = true :  H[m, n] = bf16_rn( silu(sum_k A[m,k] Wg[k,n]) * (sum_k A[m,k] Wu[k,n]) )
//                    one CTA tile = 128 rows x 128 H-columns; a single N = 256 MMA holds the
//                    gate columns in TMEM columns [0,128) and the up columns in [128,256),
//                    so an epilogue thread owns g and u of the same element: SiLU and the
//                    product happen in registers and H is written once
//   GATEUP = false:  Y[m, c] = bf16_rn( sum_n H[m,n] Wd[n,c] ),  tile = 128 rows x 256 columns
//
// Operands: A is row-major [M, K] = K-major for the MMA; the weights are row-major [K, N]
// ("[in, out]"), i.e. MN-major B operands, which tcgen05 consumes directly (no transpose is
// ever materialised).  TMA (128-byte swizzle) fills a ring of shared-memory stages; one
// thread issues tcgen05.mma; fp32 accumulators live in TMEM; four epilogue warps read them
// back with tcgen05.ld.  Ragged M / N / K come from TMA's zero fill and predicated stores.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer,
// warps 2..5 = epilogue (warp w reads TMEM lanes 32*(w%4) .. +31).
// CTAs are persistent (one per SM, tiles taken round-robin) and TMEM holds two accumulator
// buffers, so the epilogue of one tile runs while the MMAs of the next tile are issued.
// Every mbarrier wait is bounded; a wait that runs out records a status word, raises a
// CTA-wide abort flag and the CTA leaves through the normal teardown (TMEM freed).
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"

namespace gmlp {

constexpr int kUmmaBM = 128;
constexpr int kUmmaBK = 64;
constexpr int kUmmaN = 256;                 // MMA N: 128 gate + 128 up, or 256 plain columns
constexpr int kUmmaStages = 4;
constexpr uint32_t kUmmaTmemCols = 512;      // two accumulator buffers of 256 columns
constexpr int kUmmaThreads = 192;
constexpr uint32_t kUmmaABytes = kUmmaBM * kUmmaBK * 2;          // 16 KB: 128 rows x 128 B
constexpr uint32_t kUmmaBoxBBytes = 64 * kUmmaBK * 2;            // 8 KB: 64 k-rows x 128 B (64 columns)
constexpr uint32_t kUmmaBBytes = 4 * kUmmaBoxBBytes;             // 32 KB
constexpr uint32_t kUmmaStageBytes = kUmmaABytes + kUmmaBBytes;  // 48 KB
constexpr uint32_t kUmmaSmemBytes = kUmmaStages * kUmmaStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
// stages for a kernel with NB weight boxes per stage: the ring fills the same shared-memory budget
__host__ __device__ constexpr int umma_stages(int nb) {
    return (int)((kUmmaStages * kUmmaStageBytes) / (kUmmaABytes + nb * kUmmaBoxBBytes));
}
constexpr long long kWaitLimitCycles = 2000000000LL;             // about a second

__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                             int kernel_id, int site, long long limit_cycles = kWaitLimitCycles) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long start = clock64();
    while (!ptx::mbar_try_wait(bar, parity)) {
        if (*abort_flag) return false;
        if (clock64() - start > limit_cycles) {
            *abort_flag = 1;
            report_timeout(kernel_id, site);
            return false;
        }
    }
    return true;
}

// Self-test of the bounded wait: one warp waits on an mbarrier that nothing will ever complete, with a
// short limit.  The wait gives up, records (kernel id 99, site 1) in the device status word and the kernel
// returns normally; nothing traps, faults or spins without bound.
__global__ void wait_timeout_probe_kernel(long long limit_cycles)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_addr(&bar), 1);
        abort_flag = 0;
        ptx::fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x == 0)
        (void)wait_bounded(ptx::smem_addr(&bar), 0u, &abort_flag, 99, 1, limit_cycles);
    __syncthreads();
}

// Several weight matrices behind one A operand in ONE launch (the QKV projection of Section 6.1: three matmuls
// that share X).  The column tiles of the matrices are laid end to end: tiles [0, tiles0) belong to the first
// matrix (tensor map tmB0, output C, N columns), [tiles0, tiles0 + tiles1) to the second (tmB1, C1, N1), the rest
// to the third (tmB2, C2, N2).  Row tiles vary fastest, so a round of CTAs shares A panels in L2.
struct alignas(64) MultiB {
    CUtensorMap tmB2;
    bf16* C1;
    bf16* C2;
    int N1, N2;
    int tiles0, tiles1;
};
// which matrix a column tile belongs to (0, 1, 2) and its tile index inside that matrix
__device__ __forceinline__ int multi_segment(const MultiB& m, int n_tile, int* local) {
    if (n_tile < m.tiles0) { *local = n_tile; return 0; }
    if (n_tile < m.tiles0 + m.tiles1) { *local = n_tile - m.tiles0; return 1; }
    *local = n_tile - m.tiles0 - m.tiles1;
    return 2;
}

// Residual epilogue of "Matmul+Add+RMSNorm" (Section 6.1) for 32 accumulator columns of one row:
// s = acc + R, stored value = bf16_rn(s), and ss += (stored value)^2 - the statistic of Eq. (1) is taken over
// what is stored.  rrow points at the row's residual for the chunk's first column; columns at or beyond
// cols_left do not exist (their accumulators are zero and they add nothing).
__device__ __forceinline__ void add_residual_chunk(const uint32_t (&acc)[32], uint32_t (&packed)[16],
                                                   const bf16* rrow, int cols_left, bool row_ok, float& ss) {
#pragma unroll
    for (int v = 0; v < 4; ++v) {
        uint4 rr = make_uint4(0u, 0u, 0u, 0u);
        if (row_ok && v * 8 < cols_left) rr = __ldcg(reinterpret_cast<const uint4*>(rrow + v * 8));   // R may be the buffer S is written to
        const uint32_t w[4] = {rr.x, rr.y, rr.z, rr.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t p = pack_bf16x2(__uint_as_float(acc[v * 8 + 2 * j]) + bf16_lo(w[j]),
                                           __uint_as_float(acc[v * 8 + 2 * j + 1]) + bf16_hi(w[j]));
            packed[4 * v + j] = p;
            const float a = bf16_lo(p), b = bf16_hi(p);
            ss = fmaf(a, a, ss);
            ss = fmaf(b, b, ss);
        }
    }
}

// NB = 64-column weight boxes per stage: 4 -> MMA N = 256 (the default), 2 -> MMA N = 128 (smaller tiles for
// shapes that would otherwise leave most SMs without a tile; more stages, lower arithmetic intensity).
//
// ROWSCALE = true turns the plain GEMM into the paper's rewritten RMSNorm+MatMul (Section 2):
// Z = (X * W) (.) r with r_m = 1/sqrt(mean_k X[m,k]^2 + eps) applied in the epilogue (legal because r does
// not depend on k).  r comes from row_rsqrt_kernel, the kernel launched just before this one: the two
// are chained by programmatic dependent launch and ONLY the epilogue warps wait for it, so the main loop
// (which reads the raw X) runs in parallel with the RMS branch.
template <bool GATEUP, int NB, bool ROWSCALE = false, bool ADDSS = false, bool MULTI = false>
__global__ void __launch_bounds__(kUmmaThreads, 1)
umma_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
                 const __grid_constant__ CUtensorMap tmB1, bf16* __restrict__ C,
                 int M, int K, int N, int num_m_tiles, int num_tiles, const float* __restrict__ row_scale, int a_box_rows, GateAct act,
                 const bf16* residual, float* __restrict__ sumsq, const __grid_constant__ MultiB multi,
                 int w_kmajor, int out_fp32)
{
    static_assert(!(ROWSCALE && GATEUP), "row scaling is for the plain GEMM");
    static_assert(!(ADDSS && (GATEUP || ROWSCALE)), "the residual epilogue is for the plain GEMM");
    static_assert(!(MULTI && (GATEUP || ROWSCALE || ADDSS)), "several weight matrices: plain GEMM only");
    constexpr int KERNEL_ID = GATEUP ? 1 : 2;
    constexpr int N_MMA = 64 * NB;
    constexpr int BN_OUT = GATEUP ? N_MMA / 2 : N_MMA;
    constexpr int kStages = umma_stages(NB);
    constexpr uint32_t kStageBytes = kUmmaABytes + NB * kUmmaBoxBBytes;
    // kind::f16 instruction descriptor: D = fp32, A = B = bf16, A K-major, B MN-major, M = 128, N = N_MMA
    // (bit 16 = B is MN-major: weights stored [K, N]; with w_kmajor they are stored [N, K] and B is K-major like A)
    const uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | ((w_kmajor ? 0u : 1u) << 16) |
                            ((uint32_t)(N_MMA >> 3) << 17) | ((uint32_t)(kUmmaBM >> 4) << 24);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;            // swizzle atoms need 1024-byte alignment
    uint8_t* base_ptr = smem_raw + (base - raw_addr);
    uint64_t* bars = reinterpret_cast<uint64_t*>(base_ptr + kStages * kStageBytes);
    const uint32_t full0 = ptx::smem_addr(bars);
    const uint32_t empty0 = ptx::smem_addr(bars + kStages);
    const uint32_t tfull0 = ptx::smem_addr(bars + 2 * kStages);          // accumulator buffer b is complete
    const uint32_t tempty0 = ptx::smem_addr(bars + 2 * kStages + 2);     // accumulator buffer b has been read out
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_kb = (K + kUmmaBK - 1) / kUmmaBK;

    ptx::launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(full0 + 8 * s, 1);
            ptx::mbar_init(empty0 + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(tfull0 + 8 * b, 1);
            ptx::mbar_init(tempty0 + 8 * b, 4);                   // one arrival per epilogue warp
        }
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::fence_proxy_async_smem();
        ptx::prefetch_tensormap(&tmA);
        ptx::prefetch_tensormap(&tmB0);
        if (GATEUP || MULTI) ptx::prefetch_tensormap(&tmB1);
        if (MULTI) ptx::prefetch_tensormap(&multi.tmB2);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_addr(tmem_slot), kUmmaTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    // Persistent CTA: tiles blockIdx.x, blockIdx.x + gridDim.x, ...; row tiles vary fastest, so the CTAs of
    // one round work on the same few weight panels (L2 reuse).
    if (warp == 0) {
        // ---------------- TMA producer ----------------
        // (warp-uniform like the MMA issuer: coordinates and addresses by all lanes, the copies by the elected one)
        {
            const bool leader = ptx::elect_one();
            // the A box holds a_box_rows rows of 128 B (fewer than 128 only when the whole problem has fewer rows:
            // the rest of the 128-row operand tile is never written and feeds accumulator rows nobody stores)
            const uint32_t a_tx_bytes = (uint32_t)a_box_rows * 128u;
            auto tile_operands = [&](int tile, int& m0, int& n0, const CUtensorMap*& plain_map) {
                m0 = (tile % num_m_tiles) * kUmmaBM;
                n0 = (tile / num_m_tiles) * BN_OUT;
                plain_map = &tmB0;
                if (MULTI) {
                    int local;
                    const int seg = multi_segment(multi, tile / num_m_tiles, &local);
                    n0 = local * BN_OUT;
                    plain_map = seg == 0 ? &tmB0 : (seg == 1 ? &tmB1 : &multi.tmB2);
                }
            };
            auto load_weights = [&](int kb, uint32_t stage, int n0, const CUtensorMap* plain_map) {   // arms the barrier for the whole stage
                const uint32_t full = full0 + 8 * stage;
                const uint32_t b_dst = base + stage * kStageBytes + kUmmaABytes;
                if (!leader) return;
                ptx::mbar_arrive_expect_tx(full, a_tx_bytes + NB * kUmmaBoxBBytes);
#pragma unroll
                for (int i = 0; i < NB; ++i) {
                    // gate/up: the first NB/2 boxes are gate columns, the rest the same columns of up
                    const CUtensorMap* map = (GATEUP && i >= NB / 2) ? &tmB1 : plain_map;
                    const int x = GATEUP ? n0 + (i % (NB / 2)) * 64 : n0 + i * 64;
                    // [K, N] weights: box of 64 columns x 64 k; [N, K] weights: box of 64 k x 64 rows of N
                    if (w_kmajor) ptx::tma_load_2d(b_dst + i * kUmmaBoxBBytes, map, kb * kUmmaBK, x, full);
                    else ptx::tma_load_2d(b_dst + i * kUmmaBoxBBytes, map, x, kb * kUmmaBK, full);
                }
            };
            // The weight tiles of the first ring-full of k-blocks of this CTA's first tile do not depend on the previous
            // kernel: they are requested ahead of the wait (the caller's contract on when weights are read is in gmlp.h,
            // "Stream order"); A (Xn or H) may come from the previous kernel
            int head = 0;
            if (!ROWSCALE) {
                if ((int)blockIdx.x < num_tiles) {
                    int m0, n0;
                    const CUtensorMap* plain_map;
                    tile_operands(blockIdx.x, m0, n0, plain_map);
                    head = num_kb < kStages ? num_kb : kStages;
                    for (int i = 0; i < head; ++i) load_weights(i, (uint32_t)i, n0, plain_map);
                }
                ptx::grid_dependency_wait();
            }
            uint32_t s = 0, ph = 0;                                // ring position of the next k-block (stepped, not divided)
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                int m0, n0;
                const CUtensorMap* plain_map;
                tile_operands(tile, m0, n0, plain_map);
                for (int kb = 0; kb < num_kb; ++kb) {
                    const bool ahead = tile == (int)blockIdx.x && kb < head;     // barrier armed, weights on their way
                    if (!ahead && !__all_sync(0xFFFFFFFFu, wait_bounded(empty0 + 8 * s, ph ^ 1u, abort_flag, KERNEL_ID, 1))) { ok = false; break; }
                    if (!ahead) load_weights(kb, s, n0, plain_map);
                    if (leader) ptx::tma_load_2d(base + s * kStageBytes, &tmA, kb * kUmmaBK, m0, full0 + 8 * s);
                    __syncwarp();
                    if (++s == (uint32_t)kStages) { s = 0; ph ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        // All 32 lanes run the loop, its waits and its arithmetic, so that everything the MMAs take is warp-uniform
        // (the tensor-core instructions read their operands from uniform registers; inside a one-lane branch every
        // operand would have to be moved there per MMA); only the instructions themselves sit under the elected lane.
        {
            const bool leader = ptx::elect_one();
            // Nothing is derived per MMA: the ring position is stepped, not divided, and a step's descriptors are the
            // stage's first ones plus a constant, added to the lower descriptor word only (the single issuing thread
            // is a dependent instruction stream; with everything derived per MMA it ran at about ten cycles per
            // instruction and bounded the kernel).  In 16-byte units a K = 16 step advances
            //   A, K-major (rows of 128 B, 8-row groups 1024 B apart): 2;
            //   B, MN-major (64-column chunks 8 KB apart (LBO), 8-row k-groups 1024 B apart (SBO); K = 16 is two
            //      k-groups): 128;  B, K-major ([N, K] weights: the boxes stack to N_MMA rows of 128 B, like A): 2.
            const uint32_t desc_hi = (uint32_t)(ptx::make_smem_desc_sw128(0, 0, 1024) >> 32);
            const uint32_t a_lo0 = (uint32_t)ptx::make_smem_desc_sw128(base, 16, 1024);
            const uint32_t b_lo0 = w_kmajor ? (uint32_t)ptx::make_smem_desc_sw128(base + kUmmaABytes, 16, 1024)
                                            : (uint32_t)ptx::make_smem_desc_sw128(base + kUmmaABytes, kUmmaBoxBBytes, 1024);
            const uint32_t b_step = w_kmajor ? 2u : 128u;
            uint32_t s = 0, ph = 0;
            int t = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++t) {
                const int buf = t & 1;
                // the epilogue must have drained this accumulator buffer (two tiles ago)
                if (!__all_sync(0xFFFFFFFFu, wait_bounded(tempty0 + 8 * buf, (((uint32_t)t >> 1) & 1u) ^ 1u, abort_flag, KERNEL_ID, 4))) break;
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * kUmmaN);
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!__all_sync(0xFFFFFFFFu, wait_bounded(full0 + 8 * s, ph, abort_flag, KERNEL_ID, 2))) { ok = false; break; }
                    ptx::tc_fence_after_sync();
                    const uint32_t a_lo = a_lo0 + s * (kStageBytes >> 4), b_lo = b_lo0 + s * (kStageBytes >> 4);
                    if (leader) {
                        ptx::umma_bf16_halves(d_tmem, a_lo, b_lo, desc_hi, kIdesc, kb != 0 ? 1u : 0u);
#pragma unroll
                        for (int k = 1; k < kUmmaBK / 16; ++k)
                            ptx::umma_bf16_halves(d_tmem, a_lo + 2u * (uint32_t)k, b_lo + b_step * (uint32_t)k, desc_hi, kIdesc, 1u);
                        ptx::umma_commit(empty0 + 8 * s);  // stage is free once these MMAs have read it
                    }
                    __syncwarp();
                    if (++s == (uint32_t)kStages) { s = 0; ph ^= 1u; }
                }
                if (ok && leader) ptx::umma_commit(tfull0 + 8 * buf);   // accumulator complete
                __syncwarp();
            }
        }
        __syncwarp();
    } else {
        // ---------------- epilogue ----------------
        const int q = warp & 3;
        ptx::grid_dependency_wait();                              // C may still be read by the previous kernel
        int t = 0;
        for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++t) {
            const int buf = t & 1;
            const int m0 = (tile % num_m_tiles) * kUmmaBM;
            int n0 = (tile / num_m_tiles) * BN_OUT;
            const int row = m0 + q * 32 + lane;
            // (warp-uniform outcome: a warp must not split around the warp-wide TMEM loads and __syncwarp below)
            if (!__all_sync(0xFFFFFFFFu, wait_bounded(tfull0 + 8 * buf, ((uint32_t)t >> 1) & 1u, abort_flag, KERNEL_ID, 3))) break;
            ptx::tc_fence_after_sync();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * kUmmaN);
            bf16* Cseg = C;
            int Nseg = N;
            if (MULTI) {                                           // this tile's matrix: its output and width
                int local;
                const int seg = multi_segment(multi, tile / num_m_tiles, &local);
                n0 = local * BN_OUT;
                if (seg == 1) { Cseg = multi.C1; Nseg = multi.N1; }
                else if (seg == 2) { Cseg = multi.C2; Nseg = multi.N2; }
            }
            bf16* crow = Cseg + (size_t)row * Nseg + n0;
            const float rscale = (ROWSCALE && row < M) ? __ldcg(row_scale + row) : 1.0f;
            float ss = 0.0f;                                       // ADDSS: sum of squares of this row's stored values
#pragma unroll 1
            for (int c = 0; c < BN_OUT; c += 32) {
                uint32_t g[32];
                uint32_t packed[16];
                if (GATEUP) {
                    uint32_t u[32];
                    ptx::tmem_ld_32x32(taddr + c, g);
                    ptx::tmem_ld_32x32(taddr + N_MMA / 2 + c, u);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float h0 = gate_act_f32(__uint_as_float(g[2 * j]), act) * __uint_as_float(u[2 * j]);
                        const float h1 = gate_act_f32(__uint_as_float(g[2 * j + 1]), act) * __uint_as_float(u[2 * j + 1]);
                        packed[j] = pack_bf16x2(h0, h1);
                    }
                } else if (ADDSS) {
                    ptx::tmem_ld_32x32(taddr + c, g);
                    ptx::tmem_ld_wait();
                    add_residual_chunk(g, packed, residual + (size_t)row * N + n0 + c, N - (n0 + c), row < M, ss);
                } else {
                    ptx::tmem_ld_32x32(taddr + c, g);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        packed[j] = pack_bf16x2(__uint_as_float(g[2 * j]) * rscale, __uint_as_float(g[2 * j + 1]) * rscale);
                }
                if (!GATEUP && !ADDSS && !MULTI && out_fp32) {
                    // the plain product left in fp32 (C is a float matrix): 128 bytes of this row per chunk
                    if (row < M) {
                        float* frow = reinterpret_cast<float*>(C) + (size_t)row * N + n0 + c;
#pragma unroll
                        for (int v = 0; v < 8; ++v)
                            if (n0 + c + v * 4 < N)
                                *reinterpret_cast<float4*>(frow + v * 4) =
                                    make_float4(__uint_as_float(g[4 * v]) * rscale, __uint_as_float(g[4 * v + 1]) * rscale,
                                                __uint_as_float(g[4 * v + 2]) * rscale, __uint_as_float(g[4 * v + 3]) * rscale);
                    }
                } else if (row < M) {
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        if (n0 + c + v * 8 < Nseg)
                            *reinterpret_cast<uint4*>(crow + c + v * 8) =
                                make_uint4(packed[4 * v], packed[4 * v + 1], packed[4 * v + 2], packed[4 * v + 3]);
                    }
                }
            }
            if (ADDSS && row < M) sumsq[(size_t)(tile / num_m_tiles) * M + row] = ss;
            // all of this warp's TMEM reads of the buffer are done: hand it back to the MMA issuer
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(tempty0 + 8 * buf);
        }
    }

    if (*abort_flag) {
        // A wait ran out: give copies that may still be in flight time to land before the
        // shared memory is handed back, then leave through the same teardown.
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kUmmaTmemCols);
    }
}

}  // namespace gmlp
