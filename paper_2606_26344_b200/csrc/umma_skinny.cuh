// Small-M schedule on the tensor cores: operand-swapped ("swap-AB") tcgen05 GEMMs that
// stream each weight matrix once from HBM.
//
// For M <= 128 tokens the Gated MLP is bound by reading the weights, and CUDA cores cannot
// keep up with HBM beyond a few tokens.  Here the WEIGHT tile is the MMA's 128-row operand
// and the tokens are its N dimension (16..128): D[n, m] = sum_k W[k, n] * X[m, k].  With
// row-major [K, N] weights the weight tile is an MN-major A operand, which tcgen05 reads
// directly from the TMA-swizzled tile, and X (row-major [M, K]) is a K-major B operand: no
// transpose exists anywhere.  This is the B200 image of the paper's instruction fusion
// transpose(nc_matmul(X^T, W)) -> nc_matmul(W, X^T) (Section 4.5).
//
// Work split ("stream-K"): the (column tile, 64-deep k-block) pairs form one flat sequence
// that is cut into gridDim.x equal contiguous ranges, one per persistent CTA (one CTA per
// SM), so every SM streams the same number of bytes.  A CTA that covers only part of a
// column tile's K range writes its fp32 partial accumulators to scratch; the last CTA to
// arrive on that tile (atomic ticket, nobody waits) adds the partials in fixed CTA order and
// applies the epilogue.  SiLU is not linear, so it must come after this K reduction.
//   GATEUP: two weight matrices share the X tile; epilogue H = bf16_rn(silu(g) * u)
//   else  : one matrix; epilogue Y = bf16_rn(sum)
// NH = number of 128-column halves per tile (2 -> 512-byte contiguous weight rows per stage).
//
// Overlap between the two phases (and between calls): the kernels are launched with
// programmatic stream serialization.  Weight tiles do not depend on the previous kernel, so the
// producer fills its whole shared-memory ring with weights BEFORE griddepcontrol.wait and only
// then loads the token tile (X, or the H written by the previous kernel); every other access
// to global memory comes after the wait.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"
#include "umma_gemm.cuh"

namespace gmlp {

constexpr int kSkinnyThreads = 192;
constexpr int kSkinnyMaxStages = 12;
constexpr uint32_t kSkinnyBoxBytes = 64 * 64 * 2;            // 64 k-rows x 128 B
constexpr uint32_t kSkinnySmemBudget = 229376;               // dynamic shared memory requested (224 KB)
constexpr int kSkinnyMaxContrib = 256;                       // CTAs that can share one column tile (>= grid size)

__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}

__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Flat work sequence of `total` units cut into `parts` ranges: range c = [c*total/parts, (c+1)*total/parts).
// (64-bit division is a long instruction sequence on the GPU; the products fit 32 bits for every realistic shape)
__device__ __forceinline__ long long div_fast(long long a, int b) {          // a >= 0, b > 0
    if (((unsigned long long)a >> 32) == 0) return (long long)((uint32_t)a / (uint32_t)b);
    return a / b;
}
__device__ __forceinline__ long long range_start(long long c, long long total, long long parts) {
    const unsigned long long num = (unsigned long long)c * (unsigned long long)total;
    if ((num >> 32) == 0 && ((unsigned long long)parts >> 32) == 0) return (long long)((uint32_t)num / (uint32_t)parts);
    return (long long)(num / (unsigned long long)parts);
}
__device__ __forceinline__ int range_owner(long long unit, long long total, long long parts) {
    const unsigned long long num = (unsigned long long)(unit + 1) * (unsigned long long)parts - 1;
    if ((num >> 32) == 0 && ((unsigned long long)total >> 32) == 0) return (int)((uint32_t)num / (uint32_t)total);
    return (int)(num / (unsigned long long)total);
}

// One segment (this CTA's share of one column tile's K range) as seen by the 128 epilogue threads:
// either the CTA owns the tile's whole K range and applies the epilogue straight from TMEM, or it parks its
// fp32 partial in scratch, draws an arrival ticket, and - if it is the last contributor - adds all partials
// in CTA order and applies the epilogue.  Returns true when this CTA wrote the tile's final output.
//   acc0        TMEM address (lane quarter and first column) of the accumulator buffer; accumulator (j, h)
//               starts at column (j * NH + h) * Mpad
//   total/parts/KB  the flat work sequence (see range_start / range_owner) this phase was cut from
template <bool GATEUP, int NH>
__device__ __forceinline__ bool skinny_epilogue_segment(
    uint32_t acc0, uint32_t tempty_bar, int tile, int first_c, int last_c, bool first_segment_of_cta, int cta,
    long long total, long long parts,
    int KB, int M, int Mpad, int N, float* __restrict__ scratch, unsigned int* __restrict__ counters,
    bf16* __restrict__ out, unsigned long long* slot_off, volatile int* last_flag, int et, int nl, int lane,
    const GateAct act, const int out_fp32)
{
    constexpr int NMAT = GATEUP ? 2 : 1;
    constexpr int TILE_N = 128 * NH;
    const size_t slot_floats = (size_t)NMAT * NH * Mpad * 128;
    const int n_base = tile * TILE_N;

    if (first_c == last_c) {
        // this CTA owns the whole K range of the tile: epilogue straight from TMEM
#pragma unroll
        for (int h = 0; h < NH; ++h) {
            const int n = n_base + h * 128 + nl;
            for (int c0 = 0; c0 < Mpad; c0 += 16) {
                uint32_t g[16], uu[16];
                tmem_ld_32x16(acc0 + (uint32_t)((0 * NH + h) * Mpad + c0), g);
                if (GATEUP) tmem_ld_32x16(acc0 + (uint32_t)((1 * NH + h) * Mpad + c0), uu);
                ptx::tmem_ld_wait();
                if (n < N) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int m = c0 + i;
                        if (m < M) {
                            const float v = GATEUP ? gate_act_f32(__uint_as_float(g[i]), act) * __uint_as_float(uu[i])
                                                   : __uint_as_float(g[i]);
                            if (!GATEUP && out_fp32) reinterpret_cast<float*>(out)[(size_t)m * N + n] = v;
                            else out[(size_t)m * N + n] = __float2bfloat16_rn(v);
                        }
                    }
                }
            }
        }
        ptx::tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(tempty_bar);
        return true;
    }

    // partial K range: park the fp32 accumulators in this CTA's scratch slot
    const int slot = first_segment_of_cta ? 0 : 1;
    float* mine = scratch + ((size_t)cta * 2 + slot) * slot_floats;
#pragma unroll
    for (int j = 0; j < NMAT; ++j)
#pragma unroll
        for (int h = 0; h < NH; ++h)
            for (int c0 = 0; c0 < Mpad; c0 += 16) {
                uint32_t v[16];
                tmem_ld_32x16(acc0 + (uint32_t)((j * NH + h) * Mpad + c0), v);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    if (c0 + i < M)      // rows past M are padding: never read back
                        __stcg(mine + ((size_t)(j * NH + h) * Mpad + c0 + i) * 128 + nl, __uint_as_float(v[i]));
            }
    ptx::tc_fence_before_sync();
    __syncwarp();
    if (lane == 0) ptx::mbar_arrive(tempty_bar);
    __threadfence();
    epi_bar_sync();
    if (et == 0) {
        const unsigned int ticket = atomicAdd(counters + tile, 1u);
        *last_flag = (ticket == (unsigned int)(last_c - first_c)) ? 1 : 0;
    }
    epi_bar_sync();
    if (*last_flag == 0) return false;

    __threadfence();
    // Sum the contributors' partials in CTA order.  Thread mapping: 32 column groups of 4 columns x 4 row
    // groups; float4 loads, several contributors and two token rows per round, so that many loads are in
    // flight while the additions keep their fixed order.
    const int ncontrib = last_c - first_c + 1;
    for (int i = et; i < ncontrib; i += 128) {
        const int c = first_c + i;
        const int cslot = ((int)div_fast(range_start(c, total, parts), KB) == tile) ? 0 : 1;
        slot_off[i] = ((unsigned long long)c * 2 + cslot) * slot_floats;
    }
    epi_bar_sync();
    const int cg = et & 31, rg = et >> 5;
    auto add4 = [](float4& a, const float4& b) { a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w; };
#pragma unroll
    for (int h = 0; h < NH; ++h) {
        const int n = n_base + h * 128 + cg * 4;
        if (n >= N) continue;
        for (int m = rg; m < M; m += 8) {
            constexpr int CB = GATEUP ? 4 : 8;
            const bool two = (m + 4) < M;
            const size_t og0 = ((size_t)h * Mpad + m) * 128 + cg * 4;
            const size_t og1 = two ? og0 + 4 * 128 : og0;
            const size_t du = (size_t)NH * Mpad * 128;      // gate -> up offset inside a slot
            float4 g0 = make_float4(0.f, 0.f, 0.f, 0.f), g1 = g0, u0 = g0, u1 = g0;
            int i = 0;
            for (; i + CB <= ncontrib; i += CB) {
                float4 a0[CB], a1[CB], b0[CB], b1[CB];
#pragma unroll
                for (int t = 0; t < CB; ++t) {
                    const float* p = scratch + slot_off[i + t];
                    a0[t] = __ldcg(reinterpret_cast<const float4*>(p + og0));
                    a1[t] = __ldcg(reinterpret_cast<const float4*>(p + og1));
                    if (GATEUP) {
                        b0[t] = __ldcg(reinterpret_cast<const float4*>(p + og0 + du));
                        b1[t] = __ldcg(reinterpret_cast<const float4*>(p + og1 + du));
                    }
                }
#pragma unroll
                for (int t = 0; t < CB; ++t) {
                    add4(g0, a0[t]); add4(g1, a1[t]);
                    if (GATEUP) { add4(u0, b0[t]); add4(u1, b1[t]); }
                }
            }
            for (; i < ncontrib; ++i) {
                const float* p = scratch + slot_off[i];
                add4(g0, __ldcg(reinterpret_cast<const float4*>(p + og0)));
                add4(g1, __ldcg(reinterpret_cast<const float4*>(p + og1)));
                if (GATEUP) {
                    add4(u0, __ldcg(reinterpret_cast<const float4*>(p + og0 + du)));
                    add4(u1, __ldcg(reinterpret_cast<const float4*>(p + og1 + du)));
                }
            }
            auto finish = [&](const float4& g, const float4& uu, int mm) {
                float v[4] = {g.x, g.y, g.z, g.w};
                if (GATEUP) {
                    v[0] = gate_act_f32(g.x, act) * uu.x; v[1] = gate_act_f32(g.y, act) * uu.y;
                    v[2] = gate_act_f32(g.z, act) * uu.z; v[3] = gate_act_f32(g.w, act) * uu.w;
                }
                // N is a multiple of 8 and n of 4: the four columns are all inside or all outside
                if (!GATEUP && out_fp32)
                    *reinterpret_cast<float4*>(reinterpret_cast<float*>(out) + (size_t)mm * N + n) = make_float4(v[0], v[1], v[2], v[3]);
                else
                    *reinterpret_cast<uint2*>(out + (size_t)mm * N + n) =
                        make_uint2(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]));
            };
            finish(g0, u0, m);
            if (two) finish(g1, u1, m + 4);
        }
    }
    if (et == 0) counters[tile] = 0u;        // clean for the next call
    return true;
}

template <bool GATEUP, int NH>
__global__ void __launch_bounds__(kSkinnyThreads, 1)
skinny_gemm_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW0,
                   const __grid_constant__ CUtensorMap tmW1, float* __restrict__ scratch,
                   unsigned int* __restrict__ counters, bf16* __restrict__ out,
                   int M, int Mpad, int N, int num_tiles, int KB, int stages, uint32_t tmem_cols, int evict_first,
                   GateAct act, int w_kmajor, int out_fp32)
{
    constexpr int KERNEL_ID = GATEUP ? 3 : 4;
    constexpr int NMAT = GATEUP ? 2 : 1;
    constexpr int TILE_N = 128 * NH;
    constexpr uint32_t W_BYTES = NMAT * NH * 2 * kSkinnyBoxBytes;     // weight bytes per stage
    const uint32_t x_bytes = (uint32_t)Mpad * 128u;
    const uint32_t stage_bytes = W_BYTES + x_bytes;

    extern __shared__ uint8_t smem_raw[];
    __shared__ unsigned long long slot_off[kSkinnyMaxContrib];     // scratch offsets of a tile's contributors
    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    const uint32_t base = (raw_addr + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - raw_addr);
    uint64_t* bars = reinterpret_cast<uint64_t*>(base_ptr + (size_t)stages * stage_bytes);
    const uint32_t full0 = ptx::smem_addr(bars);
    const uint32_t empty0 = ptx::smem_addr(bars + kSkinnyMaxStages);
    const uint32_t tfull0 = ptx::smem_addr(bars + 2 * kSkinnyMaxStages);
    const uint32_t tempty0 = ptx::smem_addr(bars + 2 * kSkinnyMaxStages + 2);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kSkinnyMaxStages + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* last_flag = reinterpret_cast<volatile int*>(tmem_slot + 2);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long total = (long long)num_tiles * KB;
    const long long parts = gridDim.x;
    const long long u_begin = range_start(blockIdx.x, total, parts);
    const long long u_end = range_start(blockIdx.x + 1, total, parts);

    constexpr int TRK = GATEUP ? 0 : 1;                  // timeline slot (GMLP_TRACE builds)
    (void)TRK;
    ptx::launch_dependents();
    if (threadIdx.x == 0) {
        GMLP_TR(TRK, 0);
        for (int s = 0; s < stages; ++s) {
            ptx::mbar_init(full0 + 8 * s, 1);
            ptx::mbar_init(empty0 + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(tfull0 + 8 * b, 1);
            ptx::mbar_init(tempty0 + 8 * b, 4);          // one arrival per epilogue warp
        }
        *abort_flag = 0;
        *last_flag = 0;
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
    // TMEM column of accumulator (buffer b, matrix j, half h): Mpad fp32 columns each
    auto acc_col = [&](int b, int j, int h) -> uint32_t { return (uint32_t)(((b * NMAT + j) * NH + h) * Mpad); };

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        // (warp-uniform like the MMA issuer: coordinates and addresses are computed by all lanes, the copies are
        // issued by the elected one)
        {
            const bool leader = ptx::elect_one();
            const uint64_t policy = ptx::l2_policy_evict_first();
            // (tile, k-block) of a unit are carried along and stepped, never recomputed: 64-bit divisions by a
            // run-time KB cost this single thread hundreds of cycles per unit, as much as the unit's share of time
            auto load_weights = [&](int tile, int kb, int s) {
                const uint32_t full = full0 + 8 * s;
                const uint32_t st = base + s * stage_bytes;
                if (!leader) return;
                ptx::mbar_arrive_expect_tx(full, stage_bytes);
#pragma unroll
                for (int j = 0; j < NMAT; ++j)
#pragma unroll
                    for (int hb = 0; hb < NH * 2; ++hb)
                    {
                        // [K, N] weights: box of 64 columns x 64 k at (n, k); [N, K] weights: 64 k x 64 rows at (k, n)
                        const int n = tile * TILE_N + hb * 64;
                        const int cx = w_kmajor ? kb * 64 : n, cy = w_kmajor ? n : kb * 64;
                        if (evict_first)
                            ptx::tma_load_2d_hint(st + (j * NH * 2 + hb) * kSkinnyBoxBytes, j ? &tmW1 : &tmW0, cx, cy, full,
                                                  policy);
                        else
                            ptx::tma_load_2d(st + (j * NH * 2 + hb) * kSkinnyBoxBytes, j ? &tmW1 : &tmW0, cx, cy, full);
                    }
            };
            auto load_tokens = [&](int kb, int s) {
                if (leader) ptx::tma_load_2d(base + s * stage_bytes + W_BYTES, &tmX, kb * 64, 0, full0 + 8 * s);
            };
            auto step = [&](int& tile, int& kb) { if (++kb == KB) { kb = 0; ++tile; } };
            const int tile0 = (int)div_fast(u_begin, KB), kb0 = (int)(u_begin - (long long)tile0 * KB);
            // weights of the first ring-full of units do not depend on the previous kernel
            const long long n_units = u_end - u_begin;
            const int head = (int)(n_units < stages ? n_units : stages);
            int tile = tile0, kb = kb0;
            for (int i = 0; i < head; ++i) { load_weights(tile, kb, i); step(tile, kb); }
            if (leader) GMLP_TR(TRK, 2);
            ptx::grid_dependency_wait();
            if (leader) GMLP_TR(TRK, 3);
            { int t2 = tile0, k2 = kb0; for (int i = 0; i < head; ++i) { load_tokens(k2, i); step(t2, k2); } }
            int s = head == stages ? 0 : head;                     // ring slot and its phase, stepped as well
            uint32_t ph = head == stages ? 1u : 0u;
            for (long long u = u_begin + head; u < u_end; ++u) {
                if (!__all_sync(0xFFFFFFFFu, wait_bounded(empty0 + 8 * s, ph ^ 1u, abort_flag, KERNEL_ID, 1))) break;
                load_weights(tile, kb, s);
                load_tokens(kb, s);
                __syncwarp();
                step(tile, kb);
                if (++s == stages) { s = 0; ph ^= 1u; }
            }
            if (leader) GMLP_TR(TRK, 4);
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        // All 32 lanes run the loop, its waits and its arithmetic, so that everything the MMAs take is warp-uniform
        // (the tensor-core instructions read their operands from uniform registers); only the instructions
        // themselves sit under the elected lane.  Nothing is derived per MMA: a descriptor is the stage's first one
        // plus a constant, added to the lower descriptor word (the upper word is the same for all).
        {
            const bool leader = ptx::elect_one();
            // D = fp32, A = B = bf16, A (weights) MN-major, B (tokens) K-major, M = 128, N = Mpad
            // (weights stored [N, K]: A is K-major too, bit 15 clear)
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((w_kmajor ? 0u : 1u) << 15) | (0u << 16) |
                                   ((uint32_t)(Mpad >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
            const uint32_t desc_hi = (uint32_t)(ptx::make_smem_desc_sw128(0, 0, 1024) >> 32);
            const uint32_t tok_lo0 = (uint32_t)ptx::make_smem_desc_sw128(base + W_BYTES, 16, 1024);
            // weights stored [N, K]: the two boxes stack to 128 rows of 128 B, K-major like the tokens
            const uint32_t w_lo0 = w_kmajor ? (uint32_t)ptx::make_smem_desc_sw128(base, 16, 1024)
                                            : (uint32_t)ptx::make_smem_desc_sw128(base, kSkinnyBoxBytes, 1024);
            const uint32_t w_step = w_kmajor ? 2u : 128u;            // 16-byte units per K = 16 step
            const uint32_t stage16 = stage_bytes >> 4;
            int seg = 0, s = 0, kb = (int)(u_begin - div_fast(u_begin, KB) * KB);   // ring slot, its phase and the k-block are stepped
            uint32_t ph = 0u;
            bool fresh = true;
            for (long long u = u_begin; u < u_end; ++u) {
                const int buf = seg & 1;
                if (fresh) {
                    // the accumulator buffer must have been drained by the epilogue two segments ago
                    if (!__all_sync(0xFFFFFFFFu, wait_bounded(tempty0 + 8 * buf, (((uint32_t)seg >> 1) & 1u) ^ 1u, abort_flag, KERNEL_ID, 4))) break;
                    ptx::tc_fence_after_sync();
                }
                if (!__all_sync(0xFFFFFFFFu, wait_bounded(full0 + 8 * s, ph, abort_flag, KERNEL_ID, 2))) break;
                ptx::tc_fence_after_sync();
                if (leader && u == u_begin) GMLP_TR(TRK, 5);
                const uint32_t tok_lo = tok_lo0 + (uint32_t)s * stage16, w_lo = w_lo0 + (uint32_t)s * stage16;
                const bool last_of_segment = kb == KB - 1 || u == u_end - 1;
                if (leader) {
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
#pragma unroll
                        for (int j = 0; j < NMAT; ++j)
#pragma unroll
                            for (int h = 0; h < NH; ++h)
                                ptx::umma_bf16_halves(tmem_base + acc_col(buf, j, h),
                                                      w_lo + (uint32_t)((j * NH + h) * ((2 * kSkinnyBoxBytes) >> 4)) + w_step * (uint32_t)k,
                                                      tok_lo + 2u * (uint32_t)k, desc_hi, idesc, (fresh && k == 0) ? 0u : 1u);
                    }
                    ptx::umma_commit(empty0 + 8 * s);
                    if (last_of_segment) ptx::umma_commit(tfull0 + 8 * buf);
                    if (u == u_end - 1) GMLP_TR(TRK, 6);
                }
                __syncwarp();
                fresh = false;
                if (last_of_segment) {
                    ++seg;
                    fresh = true;
                }
                if (++kb == KB) kb = 0;
                if (++s == stages) { s = 0; ph ^= 1u; }
            }
        }
        __syncwarp();
    } else {
        // ---------------- epilogue (128 threads: one weight column each) ----------------
        const int q = warp & 3;
        const int nl = q * 32 + lane;                       // column within a 128-column half = TMEM lane
        const int et = threadIdx.x - 64;
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        int seg = 0;
        int tile = (int)div_fast(u_begin, KB);
        const int first_tile = tile;
        ptx::grid_dependency_wait();          // scratch, counters and `out` may still be in use by the previous kernel
        for (long long u = u_begin; u < u_end; ++seg, ++tile) {
            const long long tile_first = (long long)tile * KB;
            const long long seg_end = (tile_first + KB < u_end) ? tile_first + KB : u_end;
            // who shares this tile: worked out while the accumulator is still being produced
            const int first_c = range_owner(tile_first, total, parts);
            const int last_c = range_owner(tile_first + KB - 1, total, parts);
            const int buf = seg & 1;
            (void)wait_bounded(tfull0 + 8 * buf, ((uint32_t)seg >> 1) & 1u, abort_flag, KERNEL_ID, 3);
            ptx::tc_fence_after_sync();
            // The segment's code contains barriers over all 128 epilogue threads, so they must all take the same
            // branch: every wait above has ended (each is bounded); whoever gave up raised the abort flag first,
            // and after this barrier every thread sees it.
            epi_bar_sync();
            if (*abort_flag) break;
            if (et == 0) { if (seg == 0) GMLP_TR(TRK, 7); GMLP_TR(TRK, 8); }
            const bool wrote = skinny_epilogue_segment<GATEUP, NH>(tmem_base + lane_base + acc_col(buf, 0, 0), tempty0 + 8 * buf, tile,
                                                first_c, last_c, tile == first_tile, blockIdx.x, total, parts, KB, M, Mpad, N,
                                                scratch, counters, out, slot_off, last_flag, et, nl, lane, act, out_fp32);
            if (et == 0) { GMLP_TR(TRK, 9); if (wrote) GMLP_TR(TRK, 10); }
            (void)wrote;
            u = seg_end;
        }
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
