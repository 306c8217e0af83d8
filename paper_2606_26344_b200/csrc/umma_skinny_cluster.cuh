// Small-M schedule, cluster form: the operand-swapped tcgen05 GEMMs of umma_skinny.cuh with the K range of a
// column tile split over the CTAs of ONE thread-block cluster and reduced on chip.
//
// The stream-K form of umma_skinny.cuh hands a tile's partial sums from CTA to CTA through global memory: partial
// stores, a fence, an atomic ticket, and the last arriver's loads of the other partials - four dependent trips to L2
// at the end of each kernel.  On a layer whose weights stream in about ten microseconds (2048 x 5632: 69 MB) those
// trips cost as much as the streaming itself (timeline: 4 to 4.5 us from a kernel's last MMA to its last store, in
// both kernels).  Here a cluster of C CTAs owns one 128-column tile: CTA r runs the k-blocks [r KB / C, (r + 1) KB / C),
// then the partial sums are reduce-scattered: the tokens are dealt out over the C CTAs, every CTA copies the others'
// shares of its fp32 accumulators from TMEM into their shared memory (st.shared::cluster, 16-byte stores,
// conflict-free; into a staging region of its own for few tokens, else into the ring once a first cluster barrier has
// shown that every ring of the cluster is free), a cluster barrier publishes them, and
// every CTA adds what it received to its own accumulator in rank order (bitwise deterministic), applies the epilogue and
// stores its tokens.  Nothing of the reduction touches global memory, nobody polls a global flag, and there is no
// scratch buffer or counter to keep clean; the epilogue's work is spread over the cluster.
//
// The grid is tiles x C CTAs; tile width (128 columns, or 64) and C are chosen on the host so that the clusters fill most
// of the SMs in one wave (2048 x 5632: gate/up 44 tiles of 128 x 3 CTAs, down 32 tiles of 64 x 4; a B200 holds 45 clusters of
// three CTAs at once, 33 of four, 15 of eight).  Shapes with more tiles than SMs keep the stream-K form.
// A 64-column tile is one TMA box per matrix and stage; the MMA still has 128 rows, the upper 64 of which read whatever
// follows the box in shared memory and fill TMEM lanes 64..127, which nobody reads.
// Operands, descriptors, the weight ring filled ahead of griddepcontrol.wait and the bounded waits are those of
// umma_skinny.cuh.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"
#include "umma_gemm.cuh"
#include "umma_gemm_2cta.cuh"
#include "umma_gemm_splitk.cuh"
#include "umma_skinny.cuh"

namespace gmlp {

namespace ptx {
__device__ __forceinline__ uint32_t cluster_nctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
}  // namespace ptx

constexpr int kSkinnyClusterMaxTokens = 256;                    // MMA N <= 256; gate + up accumulators: 512 TMEM columns

__device__ __forceinline__ void tmem_ld_32x4(uint32_t taddr, uint32_t (&r)[4]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr) : "memory");
}

// bytes of a CTA's staging area: the other CTAs' partial sums (fp32, 128 columns) for this CTA's share of the M tokens
__host__ __device__ constexpr uint32_t skinny_cluster_staging_bytes(int cluster, int nmat, int M) {
    return (uint32_t)(cluster - 1) * (uint32_t)nmat * (uint32_t)(((M + 3) / 4 + cluster - 1) / cluster) * 128u * 16u;
}

template <bool GATEUP>
__global__ void __launch_bounds__(kSkinnyThreads, 1)
skinny_cluster_gemm_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW0,
                           const __grid_constant__ CUtensorMap tmW1, bf16* __restrict__ out,
                           int M, int Mpad, int N, int KB, int stages, uint32_t tmem_cols, int evict_first,
                           GateAct act, int w_kmajor, int out_fp32, int boxes, uint32_t staging_off)
{
    constexpr int KERNEL_ID = GATEUP ? 10 : 11;
    constexpr int NMAT = GATEUP ? 2 : 1;
    const uint32_t W_BYTES = (uint32_t)(NMAT * boxes) * kSkinnyBoxBytes;   // weight bytes per stage: `boxes` boxes of 64 columns x 64 k per matrix
    const int TW = 64 * boxes;                                        // tile width in columns
    constexpr int TRK = GATEUP ? 2 : 3;                               // timeline slot (GMLP_TRACE builds)
    (void)TRK;
    const uint32_t x_bytes = (uint32_t)Mpad * 128u;
    const uint32_t stage_bytes = W_BYTES + x_bytes;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;                // identical in every CTA of the cluster
    uint8_t* base_ptr = smem_raw + (base - raw_addr);
    uint64_t* bars = reinterpret_cast<uint64_t*>(base_ptr + (size_t)stages * stage_bytes);
    const uint32_t full0 = ptx::smem_addr(bars);
    const uint32_t empty0 = ptx::smem_addr(bars + kSkinnyMaxStages);
    const uint32_t tfull = ptx::smem_addr(bars + 2 * kSkinnyMaxStages);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kSkinnyMaxStages + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank(), csize = ptx::cluster_nctarank();
    const int tile = (int)(blockIdx.x / csize);
    const int kb0 = (int)(((long long)rank * KB) / csize), kb1 = (int)(((long long)(rank + 1) * KB) / csize);
    const int n_units = kb1 - kb0;

    ptx::launch_dependents();
    if (threadIdx.x == 0) {
        GMLP_TR(TRK, 0);
        for (int s = 0; s < stages; ++s) {
            ptx::mbar_init(full0 + 8 * s, 1);
            ptx::mbar_init(empty0 + 8 * s, 1);
        }
        ptx::mbar_init(tfull, 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::fence_proxy_async_smem();
        ptx::prefetch_tensormap(&tmX);
        ptx::prefetch_tensormap(&tmW0);
        if (GATEUP) ptx::prefetch_tensormap(&tmW1);
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
        const bool leader = ptx::elect_one();
        const uint64_t policy = ptx::l2_policy_evict_first();
        auto load_weights = [&](int kb, int s) {
            const uint32_t full = full0 + 8 * s;
            const uint32_t st = base + s * stage_bytes;
            if (!leader) return;
            ptx::mbar_arrive_expect_tx(full, stage_bytes);
#pragma unroll
            for (int j = 0; j < NMAT; ++j)
#pragma unroll
                for (int hb = 0; hb < 2; ++hb) {
                    if (hb >= boxes) break;
                    // [K, N] weights: box of 64 columns x 64 k at (n, k); [N, K] weights: 64 k x 64 rows at (k, n)
                    const int n = tile * TW + hb * 64;
                    const int cx = w_kmajor ? kb * 64 : n, cy = w_kmajor ? n : kb * 64;
                    if (evict_first) ptx::tma_load_2d_hint(st + (j * boxes + hb) * kSkinnyBoxBytes, j ? &tmW1 : &tmW0, cx, cy, full, policy);
                    else ptx::tma_load_2d(st + (j * boxes + hb) * kSkinnyBoxBytes, j ? &tmW1 : &tmW0, cx, cy, full);
                }
        };
        auto load_tokens = [&](int kb, int s) {
            if (leader) ptx::tma_load_2d(base + s * stage_bytes + W_BYTES, &tmX, kb * 64, 0, full0 + 8 * s);
        };
        // the weights of the first ring-full of k-blocks do not depend on the previous kernel
        const int head = n_units < stages ? n_units : stages;
        for (int i = 0; i < head; ++i) load_weights(kb0 + i, i);
        if (leader) GMLP_TR(TRK, 2);
        ptx::grid_dependency_wait();
        if (leader) GMLP_TR(TRK, 3);
        for (int i = 0; i < head; ++i) load_tokens(kb0 + i, i);
        int s = head == stages ? 0 : head;
        uint32_t ph = head == stages ? 1u : 0u;
        for (int kb = kb0 + head; kb < kb1; ++kb) {
            if (!__all_sync(0xFFFFFFFFu, wait_bounded(empty0 + 8 * s, ph ^ 1u, abort_flag, KERNEL_ID, 1))) break;
            load_weights(kb, s);
            load_tokens(kb, s);
            __syncwarp();
            if (++s == stages) { s = 0; ph ^= 1u; }
        }
        if (leader) GMLP_TR(TRK, 4);
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer (warp-uniform; the instructions are issued by the elected lane) ----------------
        const bool leader = ptx::elect_one();
        // D = fp32, A = B = bf16, A (weights) MN-major, B (tokens) K-major, M = 128, N = Mpad
        // (weights stored [N, K]: A is K-major too, bit 15 clear)
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((w_kmajor ? 0u : 1u) << 15) | (0u << 16) |
                               ((uint32_t)(Mpad >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        const uint32_t desc_hi = (uint32_t)(ptx::make_smem_desc_sw128(0, 0, 1024) >> 32);
        const uint32_t tok_lo0 = (uint32_t)ptx::make_smem_desc_sw128(base + W_BYTES, 16, 1024);
        const uint32_t w_lo0 = w_kmajor ? (uint32_t)ptx::make_smem_desc_sw128(base, 16, 1024)
                                        : (uint32_t)ptx::make_smem_desc_sw128(base, kSkinnyBoxBytes, 1024);
        const uint32_t w_step = w_kmajor ? 2u : 128u;                 // 16-byte units per K = 16 step
        const uint32_t stage16 = stage_bytes >> 4;
        int s = 0;
        uint32_t ph = 0u;
        bool ok = true;
        for (int kb = kb0; kb < kb1; ++kb) {
            if (!__all_sync(0xFFFFFFFFu, wait_bounded(full0 + 8 * s, ph, abort_flag, KERNEL_ID, 2))) { ok = false; break; }
            ptx::tc_fence_after_sync();
            if (leader && kb == kb0) GMLP_TR(TRK, 5);
            const uint32_t tok_lo = tok_lo0 + (uint32_t)s * stage16, w_lo = w_lo0 + (uint32_t)s * stage16;
            if (leader) {
#pragma unroll
                for (int k = 0; k < 4; ++k)
#pragma unroll
                    for (int j = 0; j < NMAT; ++j)
                        ptx::umma_bf16_halves(tmem_base + (uint32_t)(j * Mpad), w_lo + (uint32_t)(j * boxes) * (kSkinnyBoxBytes >> 4) + w_step * (uint32_t)k,
                                              tok_lo + 2u * (uint32_t)k, desc_hi, idesc, (kb == kb0 && k == 0) ? 0u : 1u);
                ptx::umma_commit(empty0 + 8 * s);
            }
            __syncwarp();
            if (++s == stages) { s = 0; ph ^= 1u; }
        }
        if (ok && leader) { ptx::umma_commit(tfull); GMLP_TR(TRK, 6); }
        __syncwarp();
    }

    // every thread: this CTA's accumulator is complete, which also means that its MMAs no longer read the ring and that
    // no copy into the ring is in flight (every stage that was loaded has been consumed)
    (void)wait_bounded(tfull, 0u, abort_flag, KERNEL_ID, 3);
    ptx::tc_fence_after_sync();
    if (threadIdx.x == 64) GMLP_TR(TRK, 8);
    // The partial sums travel to a staging area in the receiver: its own region behind the ring when the host found
    // room for one (staging_off != 0; few tokens) - then a CTA sends as soon as its own accumulator is complete - or
    // else the ring itself, which needs a cluster barrier first (every ring of the cluster must be free).
    if (csize > 1 && staging_off == 0) {
        __syncthreads();
        ptx::cluster_sync();
    }
    if (threadIdx.x == 64) GMLP_TR(TRK, 12);

    const int q = warp & 3;
    const int nl = q * 32 + lane;                                     // column within the tile = TMEM lane (warps 2..5)
    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
    const bool has_columns = warp >= 2 && q * 32 < TW;                // a 64-column tile leaves the warps of TMEM lanes 64..127 without columns
    // Reduce-scatter over the cluster: the tokens are dealt out in groups of four ("quads", one float4 per column);
    // CTA r owns quads [r rq / C, (r + 1) rq / C) of the rq quads that hold real tokens, receives the other CTAs' partial
    // sums for them, adds them to its own in rank order and writes those tokens' outputs.  Staging in the owner:
    // float4 ((slot * NMAT + j) * own quads + quad) * 128 + column, slot = the sender's position among the other ranks.
    const int rq = (M + 3) >> 2;
    auto quad_begin = [&](uint32_t r) { return (int)((r * (uint32_t)rq) / csize); };
    const int myq0 = quad_begin(rank), myq1 = quad_begin(rank + 1), mynq = myq1 - myq0;
    if (csize > 1) {
        if (has_columns) {
            // peer by peer, the quads that peer owns (nothing is divided per quad: the bounds are stepped)
            int pq0 = 0;
            for (uint32_t p = 0; p < csize; ++p) {
                const int pq1 = quad_begin(p + 1), pnq = pq1 - pq0;
                if (p != rank && pnq > 0) {
                    const uint32_t slot = rank < p ? rank : rank - 1u;
                    const uint32_t remote = ptx::map_to_cta(base + staging_off, p) + (uint32_t)nl * 16u;
                    // (eight, four or one quad per TMEM load: with many tokens a wait per quad was most of this loop)
#pragma unroll
                    for (int j = 0; j < NMAT; ++j) {
                        const uint32_t dst = remote + (uint32_t)(((slot * NMAT + j) * pnq) * 128) * 16u;
                        const uint32_t tcol = taddr + (uint32_t)(j * Mpad);
                        int quad = pq0;
                        for (; quad + 8 <= pq1; quad += 8) {
                            uint32_t v[32];
                            ptx::tmem_ld_32x32(tcol + (uint32_t)(4 * quad), v);
                            ptx::tmem_ld_wait();
#pragma unroll
                            for (int k = 0; k < 8; ++k)
                                st_cluster_f32x4(dst + (uint32_t)((quad - pq0 + k) * 128) * 16u, __uint_as_float(v[4 * k]), __uint_as_float(v[4 * k + 1]),
                                                 __uint_as_float(v[4 * k + 2]), __uint_as_float(v[4 * k + 3]));
                        }
                        if (quad + 4 <= pq1) {
                            uint32_t v[16];
                            tmem_ld_32x16(tcol + (uint32_t)(4 * quad), v);
                            ptx::tmem_ld_wait();
#pragma unroll
                            for (int k = 0; k < 4; ++k)
                                st_cluster_f32x4(dst + (uint32_t)((quad - pq0 + k) * 128) * 16u, __uint_as_float(v[4 * k]), __uint_as_float(v[4 * k + 1]),
                                                 __uint_as_float(v[4 * k + 2]), __uint_as_float(v[4 * k + 3]));
                            quad += 4;
                        }
                        for (; quad < pq1; ++quad) {
                            uint32_t v[4];
                            tmem_ld_32x4(tcol + (uint32_t)(4 * quad), v);
                            ptx::tmem_ld_wait();
                            st_cluster_f32x4(dst + (uint32_t)((quad - pq0) * 128) * 16u,
                                             __uint_as_float(v[0]), __uint_as_float(v[1]), __uint_as_float(v[2]), __uint_as_float(v[3]));
                        }
                    }
                }
                pq0 = pq1;
            }
        }
        if (threadIdx.x == 64) GMLP_TR(TRK, 13);
        __syncthreads();
        ptx::cluster_sync();                                          // every CTA holds the partial sums of its own tokens
        if (threadIdx.x == 64) GMLP_TR(TRK, 14);
    }
    if (has_columns && mynq > 0) {
        ptx::grid_dependency_wait();                                  // `out` may still be read by the previous kernel
        const float4* stage = reinterpret_cast<const float4*>(base_ptr + staging_off);
        const int n = tile * TW + nl;
        const bool gelu = act.glu == 2, glu = act.glu == 1;
        const float beta = act.beta;
        // Four quads (sixteen tokens) per round when this CTA has four or more; the last round then starts at the fourth quad
        // from the end and repeats what the round before it has done of those (same values, same stores).
        int q0 = myq0;
        for (bool more = mynq >= 4; more; ) {
            uint32_t g[16], uu[16];
            tmem_ld_32x16(taddr + (uint32_t)(4 * q0), g);
            if (GATEUP) tmem_ld_32x16(taddr + (uint32_t)(Mpad + 4 * q0), uu);
            ptx::tmem_ld_wait();
            // the C shares in rank order, this CTA's own in its place
            float ga[16], ua[16];
            for (uint32_t r = 0; r < csize; ++r) {
                if (r != rank) {
                    const uint32_t slot = r < rank ? r : r - 1u;
                    const float4* sg = stage + ((size_t)(slot * NMAT) * mynq + (q0 - myq0)) * 128 + nl;
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const float4 a = sg[(size_t)k * 128];
                        const float4 b = GATEUP ? sg[((size_t)mynq + k) * 128] : make_float4(0.f, 0.f, 0.f, 0.f);
                        if (r == 0) {
                            ga[4 * k] = a.x; ga[4 * k + 1] = a.y; ga[4 * k + 2] = a.z; ga[4 * k + 3] = a.w;
                            ua[4 * k] = b.x; ua[4 * k + 1] = b.y; ua[4 * k + 2] = b.z; ua[4 * k + 3] = b.w;
                        } else {
                            ga[4 * k] += a.x; ga[4 * k + 1] += a.y; ga[4 * k + 2] += a.z; ga[4 * k + 3] += a.w;
                            if (GATEUP) { ua[4 * k] += b.x; ua[4 * k + 1] += b.y; ua[4 * k + 2] += b.z; ua[4 * k + 3] += b.w; }
                        }
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float og = __uint_as_float(g[i]), ou = GATEUP ? __uint_as_float(uu[i]) : 0.f;
                        ga[i] = r == 0 ? og : ga[i] + og;
                        ua[i] = r == 0 ? ou : ua[i] + ou;
                    }
                }
            }
            // (the activation is chosen outside the loops: the GELU form is a call, and a possible call per element would
            // keep the sixteen independent evaluations from overlapping)
            float v[16];
            if (!GATEUP) {
#pragma unroll
                for (int i = 0; i < 16; ++i) v[i] = ga[i];
            } else if (gelu) {
#pragma unroll
                for (int i = 0; i < 16; ++i) v[i] = gelu_f32(ga[i]) * ua[i];
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i) v[i] = __fdividef(glu ? 1.0f : ga[i], 1.0f + __expf(-(beta * ga[i]))) * ua[i];
            }
            if (n < N) {
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int m = 4 * q0 + i;
                    if (m < M) {
                        if (!GATEUP && out_fp32) reinterpret_cast<float*>(out)[(size_t)m * N + n] = v[i];
                        else out[(size_t)m * N + n] = __float2bfloat16_rn(v[i]);
                    }
                }
            }
            more = q0 + 4 < myq1;
            q0 = q0 + 8 <= myq1 ? q0 + 4 : myq1 - 4;
        }
        for (int quad = myq0; mynq < 4 && quad < myq1; ++quad) {      // fewer than four quads: one at a time
            uint32_t g[4], uu[4];
            tmem_ld_32x4(taddr + (uint32_t)(4 * quad), g);
            if (GATEUP) tmem_ld_32x4(taddr + (uint32_t)(Mpad + 4 * quad), uu);
            ptx::tmem_ld_wait();
            const float4 own_g = make_float4(__uint_as_float(g[0]), __uint_as_float(g[1]), __uint_as_float(g[2]), __uint_as_float(g[3]));
            const float4 own_u = GATEUP ? make_float4(__uint_as_float(uu[0]), __uint_as_float(uu[1]), __uint_as_float(uu[2]), __uint_as_float(uu[3]))
                                        : make_float4(0.f, 0.f, 0.f, 0.f);
            float4 ga = make_float4(0.f, 0.f, 0.f, 0.f), ua = ga;
            for (uint32_t r = 0; r < csize; ++r) {                    // fixed rank order, this CTA's own share in its place
                float4 pg = own_g, pu = own_u;
                if (r != rank) {
                    const uint32_t slot = r < rank ? r : r - 1u;
                    const size_t at = ((size_t)(slot * NMAT) * mynq + (quad - myq0)) * 128 + nl;
                    pg = stage[at];
                    if (GATEUP) pu = stage[at + (size_t)mynq * 128];
                }
                if (r == 0) { ga = pg; ua = pu; }
                else {
                    ga.x += pg.x; ga.y += pg.y; ga.z += pg.z; ga.w += pg.w;
                    if (GATEUP) { ua.x += pu.x; ua.y += pu.y; ua.z += pu.z; ua.w += pu.w; }
                }
            }
            const float gv[4] = {ga.x, ga.y, ga.z, ga.w}, uv[4] = {ua.x, ua.y, ua.z, ua.w};
            if (n < N) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int m = 4 * quad + i;
                    if (m < M) {
                        const float v = GATEUP ? gate_act_f32(gv[i], act) * uv[i] : gv[i];
                        if (!GATEUP && out_fp32) reinterpret_cast<float*>(out)[(size_t)m * N + n] = v;
                        else out[(size_t)m * N + n] = __float2bfloat16_rn(v);
                    }
                }
            }
        }
        if (lane == 0 && q == 0) GMLP_TR(TRK, 10);
    }

    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0) GMLP_TR(TRK, 11);
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, tmem_cols);
    }
}

}  // namespace gmlp
