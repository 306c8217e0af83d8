// Large-M schedule on CTA pairs: the same two GEMMs as umma_gemm.cuh, issued as
// tcgen05.mma.cta_group::2 by thread-block clusters of two CTAs (the two SMs of a TPC).
//
// One pair tile = 256 rows x 256 MMA columns (gate/up: 128 gate + 128 up columns of H; down: 256
// columns of Y).  CTA r of the pair holds rows [128 r, 128 r + 128) of A and HALF of the B columns
// (gate/up: CTA 0 the gate columns, CTA 1 the up columns; down: columns [128 r, 128 r + 128)), so a
// stage is 16 KB of A + 16 KB of B per CTA instead of 16 + 32: the ring is six stages deep and the
// shared-memory fill per MMA cycle drops from 96 to 64 bytes.  No TMA multicast is involved: each
// CTA loads its own halves; the tensor cores of the pair read B from both CTAs' shared memory.
//
// Only the leader (cluster rank 0) issues MMAs.  Barriers:
//   full[s]   (leader's)  two arrivals: each CTA's producer arms its own 32 KB; both CTAs' TMA loads
//                         complete on it (the peer's through .cta_group::2 addressing)
//   empty[s]  (per CTA)   tcgen05.commit to each CTA's barrier when the stage's MMAs are done
//   tfull[b]  (per CTA)   tcgen05.commit to each CTA's barrier: accumulator buffer b is complete
//   tempty[b] (leader's)  eight arrivals: the four epilogue warps of both CTAs have drained buffer b
// Each CTA's TMEM holds its 128 rows x 256 columns, two buffers; the epilogue is the one of
// umma_gemm.cuh.  Every wait is bounded; the pair leaves through a cluster barrier so that neither
// CTA's shared memory or TMEM disappears under the other.
//
// CHUNKED = true (the Gated MLP's two GEMMs): the K loop is cut into chunks of `chunk_kb` k-blocks.  Each chunk
// starts a fresh accumulation in one of the two TMEM buffers, and eight epilogue warps (two per TMEM lane
// quarter, half of the columns each) add the finished chunk into fp32 REGISTERS with round-to-nearest while the
// tensor cores fill the other buffer.  Reason: the tensor core adds into its fp32 accumulator by truncation, a
// small bias toward zero per MMA that grows linearly with the length of the accumulation chain (measured: the
// share of H values that round to another bf16 than the fp64 reference does is 1.8 % on rows scaled by 20 for one
// chain of 512 MMAs, and falls in proportion to the chain length down to the 0.05 % of sequential fp32 FMA);
// rows with |h| in the thousands then miss an absolute output tolerance.  Chains of 32 MMAs (8 k-blocks) joined
// by ordinary fp32 additions behave like sequential fp32.  The per-tile epilogue then works from registers.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"
#include "umma_gemm.cuh"

namespace gmlp {

constexpr int kPairStages = 6;
constexpr uint32_t kPairABytes = 128 * kUmmaBK * 2;               // 16 KB: this CTA's 128 rows
constexpr uint32_t kPairBBytes = 2 * kUmmaBoxBBytes;              // 16 KB: this CTA's 128 columns
constexpr uint32_t kPairStageBytes = kPairABytes + kPairBBytes;   // 32 KB per CTA
constexpr uint32_t kPairSmemBytes = kPairStages * kPairStageBytes + 1024 + 256;
constexpr int kPairChunkThreads = 64 + 8 * 32;                    // CHUNKED: producer, issuer and eight epilogue warps
constexpr int kPairChunkKb = 8;                                   // k-blocks (of 64) per accumulation chain

namespace ptx {
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr_local, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr_local), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx_cluster(uint32_t bar_cluster_addr, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(bar_cluster_addr), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
// TMA load whose completion is counted on a barrier that may live in the pair's other CTA (no multicast)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst_smem, const void* tmap, int x, int y, uint32_t bar_cluster_addr) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst_smem), "l"(tmap), "r"(x), "r"(y), "r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// descriptors as 32-bit halves (see umma_bf16_halves)
__device__ __forceinline__ void umma_bf16_pair_halves(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi,
                                                      uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 da, {%1, %3};\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate) : "memory");
}
// One arrival on the barrier at this shared-memory offset in BOTH CTAs of the pair once the MMAs issued so far are
// done: two commits, one to the leader's own barrier and one to the peer's (its shared::cluster address, from mapa).
// peer_delta = map_to_cta(x, 1) - x, the same for every offset, is computed once by the caller.  (Measured against the
// single instruction that signals both CTAs at once: the same time on every large-M workload, within 0.3 %.)
__device__ __forceinline__ void umma_commit_pair(uint32_t bar, uint32_t peer_delta) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar + peer_delta) : "memory");
}
}  // namespace ptx

// ROWSCALE: see umma_gemm.cuh (epilogue row scale from row_rsqrt_kernel; only the epilogue waits for it).
template <bool GATEUP, bool ROWSCALE = false, bool ADDSS = false, bool MULTI = false, bool CHUNKED = false>
__global__ void __launch_bounds__(CHUNKED ? kPairChunkThreads : kUmmaThreads, 1)
umma_pair_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
                      const __grid_constant__ CUtensorMap tmB1, bf16* __restrict__ C,
                      int M, int K, int N, int num_m_tiles, int num_tiles, const float* __restrict__ row_scale, GateAct act,
                      const bf16* residual, float* __restrict__ sumsq, const __grid_constant__ MultiB multi,
                      int w_kmajor, int out_fp32, int chunk_kb, int group_m)
{
    static_assert(!(CHUNKED && (ROWSCALE || ADDSS || MULTI)), "chunked accumulation: the Gated MLP's two GEMMs only");
    static_assert(!(ROWSCALE && GATEUP), "row scaling is for the plain GEMM");
    static_assert(!(ADDSS && (GATEUP || ROWSCALE)), "the residual epilogue is for the plain GEMM");
    static_assert(!(MULTI && (GATEUP || ROWSCALE || ADDSS)), "several weight matrices: plain GEMM only");
    constexpr int KERNEL_ID = GATEUP ? 6 : 7;
    constexpr int BN_OUT = GATEUP ? 128 : 256;
    // D = fp32, A = B = bf16, A K-major, B MN-major, M = 256 (128 per CTA), N = 256
    // (with w_kmajor the weights are stored [N, K] and B is K-major like A: bit 16 clear)
    const uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | ((w_kmajor ? 0u : 1u) << 16) |
                            ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;            // identical in both CTAs of the pair
    uint8_t* base_ptr = smem_raw + (base - raw_addr);
    uint64_t* bars = reinterpret_cast<uint64_t*>(base_ptr + kPairStages * kPairStageBytes);
    const uint32_t full0 = ptx::smem_addr(bars);
    const uint32_t empty0 = ptx::smem_addr(bars + kPairStages);
    const uint32_t tfull0 = ptx::smem_addr(bars + 2 * kPairStages);
    const uint32_t tempty0 = ptx::smem_addr(bars + 2 * kPairStages + 2);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kPairStages + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();                 // 0 = leader
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int num_kb = (K + kUmmaBK - 1) / kUmmaBK;
    // Order of the tiles: row tiles fastest, so that the pairs of one round work on few weight panels.  With
    // 0 < group_m < num_m_tiles the row tiles are taken in groups of group_m: all column tiles of a group before the
    // next group, so that the A rows of a group stay in L2 while the weights stream past (each weight panel is then
    // read once per group instead of A once per round).
    const int num_n_tiles = num_tiles / num_m_tiles;
    auto tile_coords = [&](int tile, int& mt, int& nt) {
        if (group_m <= 0 || group_m >= num_m_tiles) { mt = tile % num_m_tiles; nt = tile / num_m_tiles; return; }
        const int per = group_m * num_n_tiles, g = tile / per, r = tile - g * per;
        const int gs = num_m_tiles - g * group_m < group_m ? num_m_tiles - g * group_m : group_m;
        mt = g * group_m + r % gs;
        nt = r / gs;
    };

    ptx::launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < kPairStages; ++s) {
            ptx::mbar_init(full0 + 8 * s, 2);                     // one arming arrival per CTA (used in the leader)
            ptx::mbar_init(empty0 + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(tfull0 + 8 * b, 1);
            ptx::mbar_init(tempty0 + 8 * b, CHUNKED ? 16 : 8);    // the epilogue warps of both CTAs (used in the leader)
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
        ptx::tmem_alloc_pair(ptx::smem_addr(tmem_slot), kUmmaTmemCols);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();                                          // the peer's barriers exist before anyone signals them
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer (both CTAs) ----------------
        // (warp-uniform like the MMA issuer: coordinates and addresses by all lanes, the copies by the elected one)
        {
            const bool leader = ptx::elect_one();
            const uint32_t leader_full0 = ptx::map_to_cta(full0, 0);
            auto tile_operands = [&](int tile, int& m0, int& bx, const CUtensorMap*& bmap) {
                int mt, nt;
                tile_coords(tile, mt, nt);
                m0 = mt * 256 + (int)rank * 128;
                int n0 = nt * BN_OUT;
                // this CTA's half of the B columns: gate/up -> gate (rank 0) or up (rank 1) columns n0..n0+127
                bmap = (GATEUP && rank == 1) ? &tmB1 : &tmB0;
                if (MULTI) {
                    int local;
                    const int seg = multi_segment(multi, nt, &local);
                    n0 = local * BN_OUT;
                    bmap = seg == 0 ? &tmB0 : (seg == 1 ? &tmB1 : &multi.tmB2);
                }
                bx = GATEUP ? n0 : n0 + (int)rank * 128;
            };
            auto load_weights = [&](int kb, uint32_t stage, int bx, const CUtensorMap* bmap) {   // arms the leader's barrier for this CTA's whole stage
                const uint32_t full = leader_full0 + 8 * stage;
                const uint32_t b_dst = base + stage * kPairStageBytes + kPairABytes;
                if (!leader) return;
                ptx::mbar_arrive_expect_tx_cluster(full, kPairStageBytes);
                if (w_kmajor) {                    // [N, K] weights: boxes of 64 k x 64 rows of N
                    ptx::tma_load_2d_pair(b_dst, bmap, kb * kUmmaBK, bx, full);
                    ptx::tma_load_2d_pair(b_dst + kUmmaBoxBBytes, bmap, kb * kUmmaBK, bx + 64, full);
                } else {                           // [K, N] weights: boxes of 64 columns x 64 k
                    ptx::tma_load_2d_pair(b_dst, bmap, bx, kb * kUmmaBK, full);
                    ptx::tma_load_2d_pair(b_dst + kUmmaBoxBBytes, bmap, bx + 64, kb * kUmmaBK, full);
                }
            };
            // The weight tiles of the first ring-full of k-blocks of this pair's first tile do not depend on the previous
            // kernel: they are requested ahead of the wait (the caller's contract on when weights are read is in gmlp.h,
            // "Stream order")
            int head = 0;
            if (!ROWSCALE) {
                if (pair < num_tiles) {
                    int m0, bx;
                    const CUtensorMap* bmap;
                    tile_operands(pair, m0, bx, bmap);
                    head = num_kb < kPairStages ? num_kb : kPairStages;
                    for (int i = 0; i < head; ++i) load_weights(i, (uint32_t)i, bx, bmap);
                }
                ptx::grid_dependency_wait();
            }
            uint32_t s = 0, ph = 0;                              // ring position of the next k-block
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
                int m0, bx;
                const CUtensorMap* bmap;
                tile_operands(tile, m0, bx, bmap);
                for (int kb = 0; kb < num_kb; ++kb) {
                    const bool ahead = tile == pair && kb < head;       // barrier armed, weights on their way
                    if (!ahead && !__all_sync(0xFFFFFFFFu, wait_bounded(empty0 + 8 * s, ph ^ 1u, abort_flag, KERNEL_ID, 1))) { ok = false; break; }
                    if (!ahead) load_weights(kb, s, bx, bmap);
                    if (leader) ptx::tma_load_2d_pair(base + s * kPairStageBytes, &tmA, kb * kUmmaBK, m0, leader_full0 + 8 * s);
                    __syncwarp();
                    if (++s == (uint32_t)kPairStages) { s = 0; ph ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA only) ----------------
        // All 32 lanes run the loop, its waits and its arithmetic, so that everything the MMAs take is warp-uniform
        // (the tensor-core instructions read their operands from uniform registers; inside a one-lane branch every
        // operand would have to be moved there per MMA); only the instructions themselves sit under the elected lane.
        if (rank == 0) {
            const bool leader = ptx::elect_one();
            // Nothing is derived per MMA: the ring position is stepped, not divided, and a step's descriptors are
            // the stage's first ones plus a constant (in 16-byte units: 2 per K = 16 step of a K-major operand,
            // 128 of the MN-major weights); only the lower descriptor word changes.
            const uint32_t desc_hi = (uint32_t)(ptx::make_smem_desc_sw128(0, 0, 1024) >> 32);
            const uint32_t a_lo0 = (uint32_t)ptx::make_smem_desc_sw128(base, 16, 1024);
            const uint32_t b_lo0 = w_kmajor ? (uint32_t)ptx::make_smem_desc_sw128(base + kPairABytes, 16, 1024)
                                            : (uint32_t)ptx::make_smem_desc_sw128(base + kPairABytes, kUmmaBoxBBytes, 1024);
            const uint32_t b_step = w_kmajor ? 2u : 128u;
            // a shared::cta address is the executing CTA's own window of the shared::cluster space; the peer's window
            // lies a constant distance away
            const uint32_t peer_delta = ptx::map_to_cta(empty0, 1) - empty0;
            uint32_t s = 0, ph = 0;                              // ring position of the next k-block
            bool ok = true;
            if (CHUNKED) {
                // every chunk of chunk_kb k-blocks is an accumulation of its own, in the TMEM buffer its number selects
                uint32_t n = 0;                                   // chunks issued so far (all tiles)
                for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
                    int left = 0;                                 // k-blocks left in the current chunk
                    uint32_t d_tmem = tmem_base;
                    for (int kb = 0; kb < num_kb; ++kb) {
                        const bool fresh = left == 0;
                        if (fresh) {
                            left = chunk_kb;
                            if (!__all_sync(0xFFFFFFFFu, wait_bounded(tempty0 + 8 * (n & 1u), ((n >> 1) & 1u) ^ 1u, abort_flag, KERNEL_ID, 4))) { ok = false; break; }
                            ptx::tc_fence_after_sync();
                            d_tmem = tmem_base + (n & 1u) * 256u;
                        }
                        if (!__all_sync(0xFFFFFFFFu, wait_bounded(full0 + 8 * s, ph, abort_flag, KERNEL_ID, 2))) { ok = false; break; }
                        ptx::tc_fence_after_sync();
                        const uint32_t a_lo = a_lo0 + s * (kPairStageBytes >> 4), b_lo = b_lo0 + s * (kPairStageBytes >> 4);
                        --left;
                        const bool closes = left == 0 || kb == num_kb - 1;
                        if (leader) {
                            ptx::umma_bf16_pair_halves(d_tmem, a_lo, b_lo, desc_hi, kIdesc, fresh ? 0u : 1u);
#pragma unroll
                            for (int k = 1; k < kUmmaBK / 16; ++k)
                                ptx::umma_bf16_pair_halves(d_tmem, a_lo + 2u * (uint32_t)k, b_lo + b_step * (uint32_t)k, desc_hi, kIdesc, 1u);
                            ptx::umma_commit_pair(empty0 + 8 * s, peer_delta);
                            if (closes) ptx::umma_commit_pair(tfull0 + 8 * (n & 1u), peer_delta);
                        }
                        __syncwarp();
                        if (closes) { ++n; left = 0; }
                        if (++s == (uint32_t)kPairStages) { s = 0; ph ^= 1u; }
                    }
                }
            } else {
            int t = 0;
            for (int tile = pair; tile < num_tiles && ok; tile += num_pairs, ++t) {
                const int buf = t & 1;
                if (!__all_sync(0xFFFFFFFFu, wait_bounded(tempty0 + 8 * buf, (((uint32_t)t >> 1) & 1u) ^ 1u, abort_flag, KERNEL_ID, 4))) break;
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * 256);
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!__all_sync(0xFFFFFFFFu, wait_bounded(full0 + 8 * s, ph, abort_flag, KERNEL_ID, 2))) { ok = false; break; }
                    ptx::tc_fence_after_sync();
                    const uint32_t a_lo = a_lo0 + s * (kPairStageBytes >> 4), b_lo = b_lo0 + s * (kPairStageBytes >> 4);
                    if (leader) {
                        ptx::umma_bf16_pair_halves(d_tmem, a_lo, b_lo, desc_hi, kIdesc, kb != 0 ? 1u : 0u);
#pragma unroll
                        for (int k = 1; k < kUmmaBK / 16; ++k)
                            ptx::umma_bf16_pair_halves(d_tmem, a_lo + 2u * (uint32_t)k, b_lo + b_step * (uint32_t)k, desc_hi, kIdesc, 1u);
                        ptx::umma_commit_pair(empty0 + 8 * s, peer_delta);
                    }
                    __syncwarp();
                    if (++s == (uint32_t)kPairStages) { s = 0; ph ^= 1u; }
                }
                if (ok && leader) ptx::umma_commit_pair(tfull0 + 8 * buf, peer_delta);
                __syncwarp();
            }
            }
        }
        __syncwarp();
    } else {
        // ---------------- epilogue (both CTAs, own 128 rows) ----------------
        const int q = warp & 3;
        ptx::grid_dependency_wait();
        const uint32_t leader_tempty0 = ptx::map_to_cta(tempty0, 0);
        if (CHUNKED) {
            // Warps 2..9: warp w reads TMEM lanes 32 (w % 4) .. +31 (its row) and half `hsel` of the tile's columns:
            // gate/up: 64 gate accumulators (TMEM columns 64 hsel .. +63) and the 64 up accumulators of the same H
            // columns (128 + 64 hsel ..); plain: 128 accumulators (columns 128 hsel ..).  The running sums of a
            // tile live in registers; TMEM only ever holds one chunk per buffer.
            const int hsel = (warp - 2) >> 2;
            const int num_chunks = (num_kb + chunk_kb - 1) / chunk_kb;
            uint32_t n = 0;                                       // chunks drained so far (all tiles)
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
                float acc[128];
#pragma unroll
                for (int i = 0; i < 128; ++i) acc[i] = 0.0f;
                for (int c = 0; c < num_chunks; ++c, ++n) {
                    const uint32_t buf = n & 1u;
                    if (!__all_sync(0xFFFFFFFFu, wait_bounded(tfull0 + 8 * buf, (n >> 1) & 1u, abort_flag, KERNEL_ID, 3))) { ok = false; break; }
                    ptx::tc_fence_after_sync();
                    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * 256u;
#pragma unroll
                    for (int p = 0; p < 4; ++p) {
                        uint32_t r[32];
                        const uint32_t col = GATEUP ? (uint32_t)((p >> 1) * 128 + hsel * 64 + (p & 1) * 32)
                                                    : (uint32_t)(hsel * 128 + p * 32);
                        ptx::tmem_ld_32x32(taddr + col, r);
                        ptx::tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 32; ++i) acc[p * 32 + i] += __uint_as_float(r[i]);
                    }
                    // this warp's reads of the buffer are done: hand it back to the MMA issuer
                    ptx::tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive_cluster(leader_tempty0 + 8 * buf);
                }
                if (!ok) break;
                int mt, nt;
                tile_coords(tile, mt, nt);
                const int m0 = mt * 256 + (int)rank * 128;
                const int row = m0 + q * 32 + lane;
                if (row >= M) continue;
                if (GATEUP) {
                    const int col0 = nt * BN_OUT + hsel * 64;
                    bf16* crow = C + (size_t)row * N + col0;
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        uint32_t w[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const int i = v * 8 + 2 * j;
                            w[j] = pack_bf16x2(gate_act_f32(acc[i], act) * acc[64 + i], gate_act_f32(acc[i + 1], act) * acc[64 + i + 1]);
                        }
                        if (col0 + v * 8 < N) *reinterpret_cast<uint4*>(crow + v * 8) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                } else {
                    const int col0 = nt * BN_OUT + hsel * 128;
                    if (out_fp32) {
                        float* frow = reinterpret_cast<float*>(C) + (size_t)row * N + col0;
#pragma unroll
                        for (int v = 0; v < 32; ++v)
                            if (col0 + v * 4 < N)
                                *reinterpret_cast<float4*>(frow + v * 4) = make_float4(acc[4 * v], acc[4 * v + 1], acc[4 * v + 2], acc[4 * v + 3]);
                    } else {
                        bf16* crow = C + (size_t)row * N + col0;
#pragma unroll
                        for (int v = 0; v < 16; ++v)
                            if (col0 + v * 8 < N)
                                *reinterpret_cast<uint4*>(crow + v * 8) =
                                    make_uint4(pack_bf16x2(acc[8 * v], acc[8 * v + 1]), pack_bf16x2(acc[8 * v + 2], acc[8 * v + 3]),
                                               pack_bf16x2(acc[8 * v + 4], acc[8 * v + 5]), pack_bf16x2(acc[8 * v + 6], acc[8 * v + 7]));
                    }
                }
            }
        } else {
        int t = 0;
        for (int tile = pair; tile < num_tiles; tile += num_pairs, ++t) {
            const int buf = t & 1;
            int mt, nt;
            tile_coords(tile, mt, nt);
            const int m0 = mt * 256 + (int)rank * 128;
            int n0 = nt * BN_OUT;
            const int row = m0 + q * 32 + lane;
            if (!__all_sync(0xFFFFFFFFu, wait_bounded(tfull0 + 8 * buf, ((uint32_t)t >> 1) & 1u, abort_flag, KERNEL_ID, 3))) break;
            ptx::tc_fence_after_sync();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * 256);
            bf16* Cseg = C;
            int Nseg = N;
            if (MULTI) {                                           // this tile's matrix: its output and width
                int local;
                const int seg = multi_segment(multi, nt, &local);
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
                    ptx::tmem_ld_32x32(taddr + 128 + c, u);
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
            if (ADDSS && row < M) sumsq[(size_t)nt * M + row] = ss;
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(leader_tempty0 + 8 * buf);
        }
        }
    }

    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();                       // the peer may still be reading this CTA's shared memory through the MMA
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem_base, kUmmaTmemCols);
    }
}

}  // namespace gmlp
