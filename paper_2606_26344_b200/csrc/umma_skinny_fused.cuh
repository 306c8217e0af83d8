// Small-M schedule, fused form: the whole Gated MLP of a few tokens in ONE kernel, one thread-block cluster per
// 128-wide slice of d_ff (the composition of Section 5's operation table carried out inside a kernel: gate and up
// matmuls, the gated activation and the down matmul without H ever leaving the chip).
//
// Two dependent kernels cost a small layer two hand-overs (last MMA -> reduction -> stores -> grid completion -> release
// of the dependent -> its token tile), during which HBM idles; on 2048 x 5632 (69 MB, 10.6 us of streaming) they add up
// to as much as the streaming itself.  Cutting the work along d_ff removes the dependency between the GEMMs:
//   cluster s (C CTAs) owns the columns f in [128 s, 128 s + 128) of W_gate / W_up and the same ROWS of W_down.
//   phase A  CTA r multiplies the k-blocks [r KB / C, (r + 1) KB / C) of the two weight tiles with the tokens
//            (operand-swapped tcgen05 MMAs as in umma_skinny.cuh: weights are the 128-row operand, tokens the N);
//            the partial sums are ALL-REDUCED over the cluster through distributed shared memory (each CTA copies its
//            accumulators into every other CTA's staging area, one cluster barrier, every CTA adds the C shares in rank
//            order), and every CTA forms the slice of H = bf16(act(g) * u) in its own shared memory, laid out as the
//            K-major B operand of the next MMAs.
//   phase B  CTA r multiplies that slice of H with its share of the 128-column tiles of W_down[128 s .. 128 s + 128, :]
//            (tiles [r NT / C, (r + 1) NT / C)), which gives a PARTIAL Y (the sum over this slice's f only) in TMEM.
//   reduce   the partial Y of the d_ff / 128 slices go to fp32 scratch ([slice][token][d_model]), and a second, tiny kernel
//            (sum_slices_kernel, launched as this kernel's programmatic dependent: resident early, it waits for this
//            grid to complete) adds them in slice order and writes Y.  Nothing in either kernel waits for another CTA of
//            its grid through global memory, so no residency assumption and no counter is involved, and the sum is
//            bitwise deterministic.
// The weight ring does not know about the phases: the producer streams W_gate / W_up k-blocks and then W_down tiles
// through the same stages as fast as the MMAs free them, so HBM stays busy across the exchange in the middle.
#pragma once
#include <cuda.h>

#include "umma_skinny_cluster.cuh"

namespace gmlp {

namespace ptx {
__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_acquire() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
}  // namespace ptx

constexpr int kFusedMaxTokens = 16;
// (224 KB, not the 227 KB a CTA can have: the sixth stage that the last 3 KB buy at seven tokens made a step slower,
// 19.6 against 18.2 us)
constexpr uint32_t kFusedSmemBudget = kSkinnySmemBudget;
constexpr uint32_t kFusedWeightBytes = 4 * kSkinnyBoxBytes;      // per stage: gate and up k-block (2 x 2 boxes), or one W_down tile (2 k-blocks x 2 boxes)

// bytes of a CTA's staging area: the other CTAs' gate and up partial sums (fp32, 128 columns) for the real tokens
__host__ __device__ constexpr uint32_t skinny_fused_staging_bytes(int cluster, int M) {
    return (uint32_t)(cluster - 1) * 2u * (uint32_t)((M + 3) / 4) * 128u * 16u;
}

__global__ void __launch_bounds__(kSkinnyThreads, 1)
skinny_fused_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmWg,
                    const __grid_constant__ CUtensorMap tmWu, const __grid_constant__ CUtensorMap tmWd,
                    float* __restrict__ partial, int M, int Mpad, int d_model, int stages, uint32_t tmem_cols, int evict_first,
                    GateAct act, uint32_t hbuf_off, uint32_t staging_off, uint32_t bars_off, int w_kmajor)
{
    constexpr int KERNEL_ID = 12;
    constexpr int TRK = 2;                                            // timeline slot (GMLP_TRACE builds)
    (void)TRK;
    const uint32_t x_bytes = (uint32_t)Mpad * 128u;
    const uint32_t stage_bytes = kFusedWeightBytes + x_bytes;
    const int KB = (d_model + 63) >> 6, NT = (d_model + 127) >> 7;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;                // identical in every CTA of the cluster
    uint8_t* base_ptr = smem_raw + (base - raw_addr);
    uint64_t* bars = reinterpret_cast<uint64_t*>(base_ptr + bars_off);
    const uint32_t full0 = ptx::smem_addr(bars);
    const uint32_t empty0 = ptx::smem_addr(bars + kSkinnyMaxStages);
    const uint32_t tfull_a = ptx::smem_addr(bars + 2 * kSkinnyMaxStages);
    const uint32_t hready = ptx::smem_addr(bars + 2 * kSkinnyMaxStages + 1);
    const uint32_t tfull_b = ptx::smem_addr(bars + 2 * kSkinnyMaxStages + 2);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kSkinnyMaxStages + 3);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* ok_flag = reinterpret_cast<volatile int*>(tmem_slot + 2);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank(), csize = ptx::cluster_nctarank();
    const int slice = (int)(blockIdx.x / csize);
    const int kb0 = (int)(((long long)rank * KB) / csize), kb1 = (int)(((long long)(rank + 1) * KB) / csize);
    // (Tile ranges that run against the k-block ranges would give every CTA the same number of units; measured, that
    // form is much slower in back-to-back steps - 24.0 against 18.3 us on 2048 x 5632 - because one cluster of the next
    // launch then finds no free SMs until the first clusters of its own launch exit.)
    const int t0 = (int)((rank * (uint32_t)NT) / csize), t1 = (int)(((rank + 1) * (uint32_t)NT) / csize);
    const int n_a = kb1 - kb0, n_b = t1 - t0, n_units = n_a + n_b;

    ptx::launch_dependents();
    if (threadIdx.x == 0) {
        GMLP_TR(TRK, 0);
        for (int s = 0; s < stages; ++s) {
            ptx::mbar_init(full0 + 8 * s, 1);
            ptx::mbar_init(empty0 + 8 * s, 1);
        }
        ptx::mbar_init(tfull_a, 1);
        ptx::mbar_init(hready, 128);
        ptx::mbar_init(tfull_b, 1);
        *abort_flag = 0;
        *ok_flag = 0;
        ptx::fence_mbar_init();
        ptx::fence_proxy_async_smem();
        ptx::prefetch_tensormap(&tmX);
        ptx::prefetch_tensormap(&tmWg);
        ptx::prefetch_tensormap(&tmWu);
        ptx::prefetch_tensormap(&tmWd);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_addr(tmem_slot), tmem_cols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    if (threadIdx.x == 0) GMLP_TR(TRK, 1);

    if (warp == 0) {
        // ---------------- TMA producer (warp-uniform; the copies are issued by the elected lane) ----------------
        // The cluster barrier is used once, by the epilogue threads in the middle of the kernel; this warp has nothing to
        // publish or to receive, so it arrives right away and collects the (long completed) phase at the very end.
        if (csize > 1) ptx::cluster_arrive_release();
        const bool leader = ptx::elect_one();
        const uint64_t policy = ptx::l2_policy_evict_first();
        auto load_box = [&](uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t full) {
            if (evict_first) ptx::tma_load_2d_hint(dst, map, x, y, full, policy);
            else ptx::tma_load_2d(dst, map, x, y, full);
        };
        // unit u < n_a: k-block kb0 + u of the gate and up tiles (and of the tokens); else W_down tile t0 + u - n_a
        auto load_weights = [&](int u, int s) {
            const uint32_t full = full0 + 8 * s;
            const uint32_t st = base + s * stage_bytes;
            if (!leader) return;
            if (u < n_a) {
                const int kb = kb0 + u;
                ptx::mbar_arrive_expect_tx(full, stage_bytes);
#pragma unroll
                for (int j = 0; j < 2; ++j)
#pragma unroll
                    for (int hb = 0; hb < 2; ++hb) {
                        // [K, N] weights: box of 64 columns x 64 k at (n, k); [N, K] weights: 64 k x 64 rows at (k, n)
                        const int n = slice * 128 + hb * 64;
                        load_box(st + (j * 2 + hb) * kSkinnyBoxBytes, j ? &tmWu : &tmWg, w_kmajor ? kb * 64 : n, w_kmajor ? n : kb * 64, full);
                    }
            } else {
                const int t = t0 + (u - n_a);
                ptx::mbar_arrive_expect_tx(full, kFusedWeightBytes);
#pragma unroll
                for (int kbi = 0; kbi < 2; ++kbi)
#pragma unroll
                    for (int hb = 0; hb < 2; ++hb) {
                        const int n = t * 128 + hb * 64, f = slice * 128 + kbi * 64;
                        load_box(st + (kbi * 2 + hb) * kSkinnyBoxBytes, &tmWd, w_kmajor ? f : n, w_kmajor ? n : f, full);
                    }
            }
        };
        auto load_tokens = [&](int u, int s) {
            if (leader && u < n_a) ptx::tma_load_2d(base + s * stage_bytes + kFusedWeightBytes, &tmX, (kb0 + u) * 64, 0, full0 + 8 * s);
        };
        // the weights of the first ring-full of units do not depend on the previous kernel
        const int head = n_units < stages ? n_units : stages;
        for (int i = 0; i < head; ++i) load_weights(i, i);
        if (leader) GMLP_TR(TRK, 2);
        ptx::grid_dependency_wait();
        if (leader) GMLP_TR(TRK, 3);
        for (int i = 0; i < head; ++i) load_tokens(i, i);
        int s = head == stages ? 0 : head;
        uint32_t ph = head == stages ? 1u : 0u;
        for (int u = head; u < n_units; ++u) {
            if (!__all_sync(0xFFFFFFFFu, wait_bounded(empty0 + 8 * s, ph ^ 1u, abort_flag, KERNEL_ID, 1))) break;
            load_weights(u, s);
            load_tokens(u, s);
            __syncwarp();
            if (++s == stages) { s = 0; ph ^= 1u; }
        }
        if (leader) GMLP_TR(TRK, 4);
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer (warp-uniform; the instructions are issued by the elected lane) ----------------
        if (csize > 1) ptx::cluster_arrive_release();
        const bool leader = ptx::elect_one();
        // D = fp32, A = B = bf16, A (weights) MN-major, B (tokens, then H) K-major, M = 128, N = Mpad
        // (weights stored [N, K]: A is K-major too, bit 15 clear, and the two boxes of a tile stack to 128 rows of 128 bytes)
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((w_kmajor ? 0u : 1u) << 15) | (0u << 16) |
                               ((uint32_t)(Mpad >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        const uint32_t desc_hi = (uint32_t)(ptx::make_smem_desc_sw128(0, 0, 1024) >> 32);
        const uint32_t tok_lo0 = (uint32_t)ptx::make_smem_desc_sw128(base + kFusedWeightBytes, 16, 1024);
        const uint32_t h_lo0 = (uint32_t)ptx::make_smem_desc_sw128(base + hbuf_off, 16, 1024);
        const uint32_t w_lo0 = w_kmajor ? (uint32_t)ptx::make_smem_desc_sw128(base, 16, 1024)
                                        : (uint32_t)ptx::make_smem_desc_sw128(base, kSkinnyBoxBytes, 1024);
        const uint32_t w_step = w_kmajor ? 2u : 128u;                 // 16-byte units per K = 16 step
        const uint32_t half16 = (2 * kSkinnyBoxBytes) >> 4;           // one matrix's (phase A) or one k-block's (phase B) two boxes
        const uint32_t stage16 = stage_bytes >> 4;
        int s = 0;
        uint32_t ph = 0u;
        bool ok = true;
        for (int u = 0; u < n_a; ++u) {
            if (!__all_sync(0xFFFFFFFFu, wait_bounded(full0 + 8 * s, ph, abort_flag, KERNEL_ID, 2))) { ok = false; break; }
            ptx::tc_fence_after_sync();
            if (leader && u == 0) GMLP_TR(TRK, 5);
            const uint32_t tok_lo = tok_lo0 + (uint32_t)s * stage16, w_lo = w_lo0 + (uint32_t)s * stage16;
            if (leader) {
#pragma unroll
                for (int k = 0; k < 4; ++k)
#pragma unroll
                    for (int j = 0; j < 2; ++j)
                        ptx::umma_bf16_halves(tmem_base + (uint32_t)(j * Mpad), w_lo + (uint32_t)j * half16 + w_step * (uint32_t)k,
                                              tok_lo + 2u * (uint32_t)k, desc_hi, idesc, (u == 0 && k == 0) ? 0u : 1u);
                ptx::umma_commit(empty0 + 8 * s);
            }
            __syncwarp();
            if (++s == stages) { s = 0; ph ^= 1u; }
        }
        if (ok && leader) { ptx::umma_commit(tfull_a); GMLP_TR(TRK, 6); }
        __syncwarp();
        // the slice of H is in shared memory once all 128 epilogue threads have arrived
        if (ok && !__all_sync(0xFFFFFFFFu, wait_bounded(hready, 0u, abort_flag, KERNEL_ID, 5))) ok = false;
        ptx::tc_fence_after_sync();
        if (ok && leader) GMLP_TR(TRK, 7);
        const uint32_t hblock16 = x_bytes >> 4;                       // one 64-deep k-block of H: Mpad rows of 128 bytes
        for (int i = 0; ok && i < n_b; ++i) {
            if (!__all_sync(0xFFFFFFFFu, wait_bounded(full0 + 8 * s, ph, abort_flag, KERNEL_ID, 6))) { ok = false; break; }
            ptx::tc_fence_after_sync();
            const uint32_t w_lo = w_lo0 + (uint32_t)s * stage16;
            if (leader) {
#pragma unroll
                for (int kbi = 0; kbi < 2; ++kbi)
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        ptx::umma_bf16_halves(tmem_base + (uint32_t)((2 + i) * Mpad), w_lo + (uint32_t)kbi * half16 + w_step * (uint32_t)k,
                                              h_lo0 + (uint32_t)kbi * hblock16 + 2u * (uint32_t)k, desc_hi, idesc, (kbi == 0 && k == 0) ? 0u : 1u);
                ptx::umma_commit(empty0 + 8 * s);
            }
            __syncwarp();
            if (++s == stages) { s = 0; ph ^= 1u; }
        }
        if (ok && leader) { ptx::umma_commit(tfull_b); GMLP_TR(TRK, 8); }
        __syncwarp();
    } else {
        // ---------------- epilogue (128 threads: one weight column = one TMEM lane each) ----------------
        const int q = warp & 3;
        const int nl = q * 32 + lane;
        const int et = threadIdx.x - 64;
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
        const int rq = (M + 3) >> 2;                                  // groups of four tokens ("quads") that hold real tokens
        constexpr int kMaxQuads = kFusedMaxTokens / 4;
        // every wait has ended; whoever gave up raised the flag first.  One thread reads it for all 128, which must agree
        // (the code below contains barriers over them)
        auto all_ok = [&]() {
            epi_bar_sync();
            if (et == 0) *ok_flag = (*abort_flag == 0) ? 1 : 0;
            epi_bar_sync();
            return *ok_flag != 0;
        };
        // ---- phase A: all-reduce of the gate / up partial sums over the cluster, then H into shared memory ----
        (void)wait_bounded(tfull_a, 0u, abort_flag, KERNEL_ID, 3);
        ptx::tc_fence_after_sync();
        bool ok = all_ok();
        if (et == 0) GMLP_TR(TRK, 9);
        // (at most 16 tokens: Mpad == 16, so the gate and the up accumulator are one 16-column load each)
        uint32_t own_g[16], own_u[16];                                // this CTA's partial sums, one token per element
        tmem_ld_32x16(taddr, own_g);
        tmem_ld_32x16(taddr + 16u, own_u);
        ptx::tmem_ld_wait();
        if (csize > 1) {
            if (ok) {
                // staging in the receiver: float4 ((slot * 2 + j) * rq + quad) * 128 + column, slot = the sender's place
                // among the receiver's other ranks
                for (uint32_t p = 0; p < csize; ++p) {
                    if (p == rank) continue;
                    const uint32_t slot = rank < p ? rank : rank - 1u;
                    const uint32_t remote = ptx::map_to_cta(base + staging_off, p) + (uint32_t)(slot * 2 * rq * 128 + nl) * 16u;
#pragma unroll
                    for (int quad = 0; quad < kMaxQuads; ++quad)
                        if (quad < rq) {
                            st_cluster_f32x4(remote + (uint32_t)(quad * 128) * 16u, __uint_as_float(own_g[4 * quad]), __uint_as_float(own_g[4 * quad + 1]),
                                             __uint_as_float(own_g[4 * quad + 2]), __uint_as_float(own_g[4 * quad + 3]));
                            st_cluster_f32x4(remote + (uint32_t)((rq + quad) * 128) * 16u, __uint_as_float(own_u[4 * quad]), __uint_as_float(own_u[4 * quad + 1]),
                                             __uint_as_float(own_u[4 * quad + 2]), __uint_as_float(own_u[4 * quad + 3]));
                        }
                }
            }
            // (also after a failed wait: the other CTAs of the cluster are waiting for this arrival)
            ptx::cluster_arrive_release();
            ptx::cluster_wait_acquire();
        }
        if (et == 0) GMLP_TR(TRK, 10);
        {
            // the C shares in rank order, this CTA's own in its place: ranks below, own, ranks above
            const float4* stage = reinterpret_cast<const float4*>(base_ptr + staging_off) + nl;
            float g[16], u[16];
            auto add_share = [&](uint32_t slot, bool first) {
#pragma unroll
                for (int quad = 0; quad < kMaxQuads; ++quad)
                    if (quad < rq) {
                        const float4 a = stage[((slot * 2 + 0) * rq + quad) * 128], b = stage[((slot * 2 + 1) * rq + quad) * 128];
                        if (first) {
                            g[4 * quad] = a.x; g[4 * quad + 1] = a.y; g[4 * quad + 2] = a.z; g[4 * quad + 3] = a.w;
                            u[4 * quad] = b.x; u[4 * quad + 1] = b.y; u[4 * quad + 2] = b.z; u[4 * quad + 3] = b.w;
                        } else {
                            g[4 * quad] += a.x; g[4 * quad + 1] += a.y; g[4 * quad + 2] += a.z; g[4 * quad + 3] += a.w;
                            u[4 * quad] += b.x; u[4 * quad + 1] += b.y; u[4 * quad + 2] += b.z; u[4 * quad + 3] += b.w;
                        }
                    }
            };
            if (rank == 0) {
#pragma unroll
                for (int i = 0; i < 16; ++i) { g[i] = __uint_as_float(own_g[i]); u[i] = __uint_as_float(own_u[i]); }
            } else {
                add_share(0u, true);
                for (uint32_t r = 1; r < rank; ++r) add_share(r, false);
#pragma unroll
                for (int i = 0; i < 16; ++i) { g[i] += __uint_as_float(own_g[i]); u[i] += __uint_as_float(own_u[i]); }
            }
            for (uint32_t r = rank + 1; r < csize; ++r) add_share(r - 1u, false);
            // K-major operand with the 128-byte swizzle: token m is row m (128 bytes), the 16-byte chunk index of a row is
            // XORed with (m mod 8); rows of padding tokens are zero
            uint8_t* hrow = base_ptr + hbuf_off + (size_t)(nl >> 6) * x_bytes;       // this column's k-block of H
            const uint32_t kk = (uint32_t)(nl & 63);
            const uint32_t chunk = kk >> 3, within = (kk & 7u) << 1;
            // (the activation is chosen once, outside the loop: the GELU form is a call, and a possible call per element would
            // keep the compiler from overlapping the sixteen independent evaluations)
            float hv[16];
            if (act.glu == 2) {
#pragma unroll
                for (int m = 0; m < 16; ++m) hv[m] = m < M ? gelu_f32(g[m]) * u[m] : 0.f;
            } else {
                const float beta = act.beta;
                const bool glu = act.glu == 1;
#pragma unroll
                for (int m = 0; m < 16; ++m) hv[m] = __fdividef(glu ? 1.0f : g[m], 1.0f + __expf(-(beta * g[m]))) * u[m];
#pragma unroll
                for (int m = 0; m < 16; ++m) hv[m] = m < M ? hv[m] : 0.f;
            }
#pragma unroll
            for (int m = 0; m < 16; ++m)
                *reinterpret_cast<bf16*>(hrow + (uint32_t)m * 128u + (((chunk ^ ((uint32_t)m & 7u)) << 4) | within)) = __float2bfloat16_rn(hv[m]);
            ptx::fence_proxy_async_smem();                            // generic-proxy stores before the MMAs' reads
            if (ok) ptx::mbar_arrive(hready);
        }
        if (et == 0) GMLP_TR(TRK, 11);
        // ---- phase B: this CTA's partial Y tiles ([slice][token][d_model], fp32) for the kernel that adds the slices ----
        (void)wait_bounded(tfull_b, 0u, abort_flag, KERNEL_ID, 4);
        ptx::tc_fence_after_sync();
        ok = all_ok();
        if (et == 0) GMLP_TR(TRK, 12);
        if (ok) {
            // (no griddepcontrol.wait of its own: the producer's returned before the first token tile was loaded, and
            // everything here follows that through the barriers, so the previous kernel no longer reads the partial sums)
            float* dst = partial + (size_t)slice * M * d_model + nl;
            for (int i0 = 0; i0 < n_b; i0 += 3) {                     // three tiles' loads in flight
                uint32_t v[3][16];
#pragma unroll
                for (int t = 0; t < 3; ++t)
                    if (i0 + t < n_b) tmem_ld_32x16(taddr + (uint32_t)((2 + i0 + t) * 16), v[t]);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int t = 0; t < 3; ++t) {
                    const int n0 = (t0 + i0 + t) * 128;
                    if (i0 + t < n_b && n0 + nl < d_model) {
#pragma unroll
                        for (int m = 0; m < 16; ++m)
                            if (m < M) __stcg(dst + (size_t)m * d_model + n0, __uint_as_float(v[t][m]));
                    }
                }
            }
        }
        if (et == 0) GMLP_TR(TRK, 13);
    }

    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
    if (warp < 2 && csize > 1) ptx::cluster_wait_acquire();           // the phase these warps arrived on at the start
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, tmem_cols);
    }
    if (threadIdx.x == 0) GMLP_TR(TRK, 14);
}

// Y[m, n] = sum over the slices s (in order) of partial[s][m][n], rounded once (or left in fp32).  kSumLanes consecutive
// threads share one group of four columns: thread j adds the slices [j S / L, (j + 1) S / L) with all its loads in flight
// at once, and the L partial sums are added in lane order through shuffles - a fixed association, so the result does not
// depend on anything but the inputs.
constexpr int kSumLanes = 8;
constexpr int kSumMaxPerLane = 8;                                     // slices per lane held in registers at once
__global__ void __launch_bounds__(256)
sum_slices_kernel(const float* __restrict__ partial, bf16* __restrict__ Y, int M, int d_model, int S, int out_fp32)
{
    ptx::launch_dependents();
    if (threadIdx.x == 0) GMLP_TR(3, 0);
    const int row4 = d_model >> 2;
    const int P = M * row4;
    const int gid = blockIdx.x * 256 + threadIdx.x;
    const int pos = gid / kSumLanes, j = gid % kSumLanes;
    const bool live = pos < P;
    const int m = live ? pos / row4 : 0, c4 = live ? pos - m * row4 : 0;
    const int s0 = (j * S) / kSumLanes, s1 = ((j + 1) * S) / kSumLanes;
    const size_t slice_stride = (size_t)M * d_model;
    const float* src = partial + (size_t)m * d_model + 4 * c4;
    ptx::grid_dependency_wait();                                      // the partial sums are complete and visible
    if (threadIdx.x == 0) GMLP_TR(3, 3);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (live) {
        for (int sb = s0; sb < s1; sb += kSumMaxPerLane) {
            float4 a[kSumMaxPerLane];
#pragma unroll
            for (int t = 0; t < kSumMaxPerLane; ++t)
                if (sb + t < s1) a[t] = __ldcg(reinterpret_cast<const float4*>(src + (size_t)(sb + t) * slice_stride));
#pragma unroll
            for (int t = 0; t < kSumMaxPerLane; ++t)
                if (sb + t < s1) { acc.x += a[t].x; acc.y += a[t].y; acc.z += a[t].z; acc.w += a[t].w; }
        }
    }
    // lane 0 of the group adds the others' sums in lane order (all 32 lanes take part in the shuffles)
    float4 total = acc;
#pragma unroll
    for (int k = 1; k < kSumLanes; ++k) {
        const int from = (threadIdx.x & 31 & ~(kSumLanes - 1)) + k;
        const float x = __shfl_sync(0xFFFFFFFFu, acc.x, from), y = __shfl_sync(0xFFFFFFFFu, acc.y, from);
        const float z = __shfl_sync(0xFFFFFFFFu, acc.z, from), w = __shfl_sync(0xFFFFFFFFu, acc.w, from);
        total.x += x; total.y += y; total.z += z; total.w += w;
    }
    if (live && j == 0) {
        if (out_fp32) *reinterpret_cast<float4*>(reinterpret_cast<float*>(Y) + (size_t)m * d_model + 4 * c4) = total;
        else *reinterpret_cast<uint2*>(Y + (size_t)m * d_model + 4 * c4) = make_uint2(pack_bf16x2(total.x, total.y), pack_bf16x2(total.z, total.w));
    }
    if (threadIdx.x == 0) GMLP_TR(3, 10);
}

}  // namespace gmlp
