// libgmlp: C-ABI entry points, argument checks, schedule selection, workspace layout and
// kernel launches.  See include/gmlp.h for the contract of each call.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <atomic>
#include <cstring>
#include <mutex>
#include <string>
#include <vector>
#include <new>

#include "../../include/gmlp.h"
#include "common.cuh"
#include "rmsnorm.cuh"
#include "simt_gemm.cuh"
#include "stream_small_m.cuh"
#include "umma_gemm.cuh"
#include "umma_gemm_2cta.cuh"
#include "umma_gemm_splitk.cuh"
#include "umma_skinny.cuh"
#include "umma_skinny_cluster.cuh"
#include "umma_skinny_fused.cuh"
#include "gqa_attention.cuh"

namespace {

using gmlp::bf16;

constexpr int kVersion = 101;            // 101: one-kernel small-M form, tuned small-M forms in the tune file, GMLP_FLAG_WEIGHTS_IN_STREAM_ORDER
constexpr int kMaxDevices = 64;
constexpr int64_t kMaxDim = (int64_t)1 << 30;      // per-dimension limit (TMA coordinates are int32)
constexpr uint32_t kKnownFlags = GMLP_FLAG_RMSNORM | GMLP_FLAG_CHECKED | GMLP_FLAG_ACT_SWISH | GMLP_FLAG_ACT_GLU |
                                 GMLP_FLAG_ACT_GELU | GMLP_FLAG_WEIGHTS_OUT_IN | GMLP_FLAG_Y_FP32 | GMLP_FLAG_WEIGHTS_IN_STREAM_ORDER;
constexpr gmlp::GateAct kSilu = {1.0f, 0};
// weights of the call in flight are stored [out, in] (set by the entry points around their launches)
thread_local bool t_w_out_in = false;
// the down projection of the call in flight leaves Y in fp32 (set by gmlp_forward_ex around its second GEMM)
thread_local bool t_y_fp32 = false;
struct OutputTypeScope {
    bool prev;
    explicit OutputTypeScope(bool fp32) : prev(t_y_fp32) { t_y_fp32 = fp32; }
    ~OutputTypeScope() { t_y_fp32 = prev; }
};
struct WeightLayoutScope {                       // sets the switch for one call, restores it on every exit path
    bool prev;
    explicit WeightLayoutScope(bool out_in) : prev(t_w_out_in) { t_w_out_in = out_in; }
    ~WeightLayoutScope() { t_w_out_in = prev; }
};
// GMLP_FLAG_WEIGHTS_IN_STREAM_ORDER: the FIRST kernel of the call in flight is launched without programmatic stream
// serialization, so it starts only when everything enqueued before the call is complete; the call's later kernels
// cannot start before all CTAs of the first one are running, so nothing of the call - in particular none of the weight
// tiles that the small-M kernels fetch ahead of their griddepcontrol.wait - is read earlier than stream order allows.
thread_local bool t_first_launch_ordered = false;
struct StreamOrderScope {
    bool prev;
    explicit StreamOrderScope(bool ordered) : prev(t_first_launch_ordered) { t_first_launch_ordered = ordered; }
    ~StreamOrderScope() { t_first_launch_ordered = prev; }
};
// value of programmaticStreamSerializationAllowed for the next launch (GMLP_CHECK_LAUNCH, which follows every launch that
// went through, ends the "first kernel" state: a launch that is only prepared and then not made does not)
inline int pdl_allowed() { return t_first_launch_ordered ? 0 : 1; }
// tensor map of a weight matrix with `n` output columns and `k` input rows, 64 x 64 boxes either way
#define GMLP_ENCODE_W(map, ptr, n, k) \
    (t_w_out_in ? encode_2d(map, ptr, (uint64_t)(k), (uint64_t)(n), 64, 64) : encode_2d(map, ptr, (uint64_t)(n), (uint64_t)(k), 64, 64))
const gmlp::MultiB kNoMulti = {};

// Gate activation named by the flags (SiLU when none is set); false for a contradictory or non-finite request.
bool gate_act_from(uint32_t flags, float beta, gmlp::GateAct* out) {
    const bool swish = flags & GMLP_FLAG_ACT_SWISH, glu = flags & GMLP_FLAG_ACT_GLU, gelu = flags & GMLP_FLAG_ACT_GELU;
    if ((swish ? 1 : 0) + (glu ? 1 : 0) + (gelu ? 1 : 0) > 1) return false;
    *out = kSilu;
    if (swish) {
        if (!(beta == beta) || beta - beta != 0.0f) return false;      // NaN or infinite
        out->beta = beta;
    }
    if (glu) out->glu = 1;
    if (gelu) out->glu = 2;
    return true;
}

thread_local cudaStream_t t_stream = nullptr;
thread_local float t_default_eps = 1e-5f;
thread_local uint64_t t_launches = 0;

// Optional per-kernel event timing (benchmarks only): a ring of the most recent calls, so that a
// benchmark can enqueue many calls back to back and read the averages afterwards.
constexpr int kMaxProfKernels = 4;
constexpr int kProfRing = 64;
struct ProfCall {
    cudaEvent_t ev[kMaxProfKernels + 1] = {};
    int n = 0;
    const char* names[kMaxProfKernels] = {};
};
struct Profile {
    bool on = false;
    bool created = false;
    ProfCall calls[kProfRing];
    int recorded = 0;                           // calls recorded since profiling was enabled
    ProfCall* cur = nullptr;
};
thread_local Profile t_prof;

void prof_begin(cudaStream_t st) {
    if (!t_prof.on) return;
    if (!t_prof.created) {
        for (auto& c : t_prof.calls)
            for (auto& e : c.ev)
                if (cudaEventCreate(&e) != cudaSuccess) { t_prof.on = false; return; }
        t_prof.created = true;
    }
    t_prof.cur = &t_prof.calls[t_prof.recorded % kProfRing];
    ++t_prof.recorded;
    t_prof.cur->n = 0;
    (void)cudaEventRecord(t_prof.cur->ev[0], st);
}
void prof_mark(const char* name, cudaStream_t st) {
    if (!t_prof.on || t_prof.cur == nullptr || t_prof.cur->n >= kMaxProfKernels) return;
    ProfCall* c = t_prof.cur;
    c->names[c->n] = name;
    ++c->n;
    (void)cudaEventRecord(c->ev[c->n], st);
}

struct DeviceState {
    bool probed = false;
    bool is_sm100 = false;
    int sm_count = 0;
    void* workspace = nullptr;
    uint64_t workspace_bytes = 0;
    bool splitk_attr_set = false;
    bool addss_attr_set = false;
    bool multi_attr_set = false;
    bool gqa_attr_set = false;
    bool umma_attr_set = false;
    bool pair_attr_set = false;
    bool rowscale_attr_set = false;
    bool skinny_attr_set = false;
    bool skinny_cluster_attr_set = false;
    bool skinny_fused_attr_set = false;
    int fused_capacity[9] = {};                  // the same for the fused small-M kernel
    int cluster_capacity[2][9] = {};             // clusters of C CTAs of the cluster-form kernels resident at once (0 = not asked yet)
    // arrival-counter regions zeroed by the library (the kernels leave them zero after every call); a few are
    // remembered so that callers alternating between workspaces (one per stream) do not pay a memset per call
    static constexpr int kCleanSlots = 4;
    const void* clean_counters[kCleanSlots] = {};
    uint64_t clean_counters_bytes[kCleanSlots] = {};
    int clean_next = 0;
};
std::mutex g_mutex;
DeviceState g_dev[kMaxDevices];

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode_tiled = nullptr;

inline uint64_t align256(uint64_t v) { return (v + 255u) & ~(uint64_t)255u; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int tune_cache_load(const char* path, const char* device_name);
int tune_cache_save(const char* path);

// Returns the state of the current device, probing it on first use; nullptr if there is none.
DeviceState* current_device(int* status) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        *status = GMLP_ERR_ARCH;
        return nullptr;
    }
    bool load_cache = false;                     // first touch of this device: read the tuned choices kept in a file
    std::unique_lock<std::mutex> lock(g_mutex);
    DeviceState& d = g_dev[dev];
    if (!d.probed) {
        int major = 0, sms = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            (void)cudaGetLastError();
            *status = GMLP_ERR_ARCH;
            return nullptr;
        }
        d.is_sm100 = (major == 10);
        d.sm_count = sms;
        d.probed = true;
        load_cache = d.is_sm100;
    }
    if (!d.is_sm100) {
        *status = GMLP_ERR_ARCH;
        return nullptr;
    }
    if (g_encode_tiled == nullptr) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess || fn == nullptr) {
            (void)cudaGetLastError();
            *status = GMLP_ERR_ARCH;
            return nullptr;
        }
        g_encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
    }
    lock.unlock();
    if (load_cache)
        if (const char* cache = getenv("GMLP_TUNE_CACHE")) (void)tune_cache_load(cache, nullptr);
    *status = GMLP_OK;
    return &d;
}

// ------------------------------------------------------------------ small-M plan
struct StreamPlan {
    int MT, row_tiles, slabs, KS, kchunk;
};

StreamPlan make_stream_plan(int64_t M, int64_t K, int64_t N, int nmat, int sm_count) {
    StreamPlan p;
    p.MT = M <= 1 ? 1 : (M <= 2 ? 2 : (M <= 4 ? 4 : 8));
    p.row_tiles = (int)((M + p.MT - 1) / p.MT);
    if (p.row_tiles < 1) p.row_tiles = 1;
    p.slabs = (int)((N + gmlp::kStreamSlab - 1) / gmlp::kStreamSlab);
    const int64_t resident = (int64_t)(sm_count > 0 ? sm_count : 148) * 4;      // 4 CTAs of 128 threads per SM
    int64_t ks = resident / ((int64_t)p.slabs * nmat * p.row_tiles);
    const int64_t ks_min = (K + gmlp::kStreamMaxChunk - 1) / gmlp::kStreamMaxChunk;
    const int64_t ks_max = (K + 31) / 32;
    if (ks < ks_min) ks = ks_min;
    if (ks > ks_max) ks = ks_max;
    if (ks < 1) ks = 1;
    int64_t chunk = (K + ks - 1) / ks;
    chunk = (chunk + gmlp::kStreamWarps - 1) / gmlp::kStreamWarps * gmlp::kStreamWarps;
    if (chunk > gmlp::kStreamMaxChunk) chunk = gmlp::kStreamMaxChunk;
    p.kchunk = (int)chunk;
    p.KS = (int)((K + chunk - 1) / chunk);
    return p;
}

// Clusters of C CTAs (one CTA per SM, about half of an SM's shared memory each) that a device with `sms` SMs holds at
// once.  A cluster lives inside one GPC, and the GPCs do not all have a multiple of C SMs: measured on B200 (148 SMs;
// cudaOccupancyMaxActiveClusters) 74 / 45 / 33 / 26 / 22 / 15 / 15 for C = 2 .. 8.  Elsewhere a cautious guess; the launch
// asks the runtime and falls back to the stream-K form if the plan's clusters do not fit one wave.
int cluster_capacity_estimate(int C, int sms) {
    static const int b200[9] = {0, 148, 74, 45, 33, 26, 22, 15, 15};
    if (C < 1 || C > 8) return 0;
    if (sms == 148) return b200[C];
    return C == 1 ? sms : (sms / C) * 85 / 100;
}

// Forms of the SKINNY schedule for a shape, as gmlp_autotune measured them or as it is forcing them right now
// (0 = by the built-in rule): *fused 1 = the one-kernel form wherever its plan applies, 2 = two kernels; *ring
// 1 = half-size weight rings (up to 32 tokens), 2 = full-size rings.  Defined with the tuned choices below.
void skinny_forms(int64_t M, int64_t d_model, int64_t d_ff, int* fused, int* ring);

// ------------------------------------------------------------------ skinny (swap-AB tcgen05) plan
struct SkinnyPlan {
    int Mpad, NH, num_tiles, KB, stages, grid;
    uint32_t smem_bytes;
    uint32_t tmem_cols;
    uint64_t scratch_bytes;
    // cluster form (umma_skinny_cluster.cuh): CTAs per 128-column tile, 0 = not applicable (the stream-K form runs)
    int cluster, c_boxes, c_tiles, c_stages;     // c_boxes: 64-column boxes per tile (2 = 128-column tiles, 1 = 64)
    uint32_t c_smem_bytes, c_tmem_cols, c_staging_off;    // c_staging_off: the partial sums' own region (0 = they reuse the ring)
};

SkinnyPlan make_skinny_plan(int64_t M, int64_t K, int64_t N, int nmat, int sm_count) {
    SkinnyPlan p;
    p.Mpad = (int)((M + 15) / 16 * 16);
    if (p.Mpad < 16) p.Mpad = 16;
    // Few tokens: half-size shared-memory rings (112 KB), so that the next kernel on the stream - launched with
    // programmatic stream serialization - is co-resident on every SM and has its weight ring full by the time
    // this one drains.  Both kernels then use 128-column tiles (more, smaller units balance better: measured
    // 1-17 % faster than 256-column tiles for the down projection on nine layer shapes).
    int small_max = 32;
    if (const char* e = getenv("GMLP_SKINNY_SMALL_MPAD")) small_max = atoi(e);                      // tuning override
    int tuned_fused = 0, tuned_ring = 0;         // what gmlp_autotune found for this layer, if it ran
    skinny_forms(M, nmat == 2 ? K : N, nmat == 2 ? N : K, &tuned_fused, &tuned_ring);
    (void)tuned_fused;
    if (p.Mpad > 32 && tuned_ring == 1) tuned_ring = 0;          // half-size rings exist for up to 32 tokens only
    const bool small = tuned_ring == 0 ? p.Mpad <= small_max : tuned_ring == 1;
    p.NH = (N >= 256 && 2 * nmat * 2 * p.Mpad <= 512 && !small) ? 2 : 1;
    if (const char* e = getenv(nmat == 2 ? "GMLP_SKINNY_NH1" : "GMLP_SKINNY_NH2")) {      // tuning override
        if (e[0] == '1') p.NH = 1;
        if (e[0] == '2' && N >= 256 && 2 * nmat * 2 * p.Mpad <= 512) p.NH = 2;
    }
    const int tile_n = 128 * p.NH;
    p.num_tiles = (int)((N + tile_n - 1) / tile_n);
    p.KB = (int)((K + 63) / 64);
    const uint32_t stage_bytes = (uint32_t)nmat * p.NH * 2 * gmlp::kSkinnyBoxBytes + (uint32_t)p.Mpad * 128u;
    uint32_t budget = small ? gmlp::kSkinnySmemBudget / 2 : gmlp::kSkinnySmemBudget;
    if (const char* e = getenv("GMLP_SKINNY_SMEM_KB")) { int v = atoi(e); if (v >= 48 && v <= 224) budget = (uint32_t)v * 1024u; }  // tuning override
    int st = (int)((budget - 1024 - 256) / stage_bytes);
    p.stages = st > gmlp::kSkinnyMaxStages ? gmlp::kSkinnyMaxStages : st;
    p.smem_bytes = (uint32_t)p.stages * stage_bytes + 1024 + 256;
    if (const char* e = getenv("GMLP_SKINNY_STAGES")) { int v = atoi(e); if (v >= 2 && v < p.stages) p.stages = v; }   // tuning override
    uint32_t cols = (uint32_t)(2 * nmat * p.NH * p.Mpad);
    uint32_t pow2 = 32;
    while (pow2 < cols) pow2 <<= 1;
    p.tmem_cols = pow2;
    const int64_t total = (int64_t)p.num_tiles * p.KB;
    const int sms = sm_count > 0 ? sm_count : 148;
    p.grid = (int)(total < sms ? total : sms);
    // gate/up with half-size rings: two CTAs per SM keep more loads in flight (about 2 % on a large layer), as
    // long as every CTA still gets 16 or more units, which also bounds the contributors of a tile
    if (small && nmat == 2 && total >= (int64_t)32 * sms && p.KB / 16 + 2 <= gmlp::kSkinnyMaxContrib) p.grid = 2 * sms;
    if (const char* e = getenv(nmat == 2 ? "GMLP_SKINNY_GRID1" : "GMLP_SKINNY_GRID2")) {   // tuning override
        const int v = atoi(e);
        if (v == -1) p.grid = (int)(p.num_tiles < total ? p.num_tiles : total);          // one CTA per tile
        else if (v >= 1 && v <= total) p.grid = v;
    }
    // a column tile is shared by at most min(grid, KB / (units per CTA) + 2) consecutive CTAs; the kernel keeps one
    // scratch offset per contributor in a fixed shared array
    {
        const int64_t per_cta = total / p.grid > 0 ? total / p.grid : 1;
        const int64_t contrib = p.KB / per_cta + 2 < p.grid ? p.KB / per_cta + 2 : p.grid;
        if (contrib > gmlp::kSkinnyMaxContrib) p.stages = 0;               // launch_skinny refuses the plan
    }
    // (beyond 128 tokens only the cluster form below can run, and it needs no scratch)
    p.scratch_bytes = M > 128 ? 0 : (uint64_t)p.grid * 2 * nmat * p.NH * p.Mpad * 128 * 4;
    // Cluster form: one cluster of C CTAs per column tile (128 columns, or 64), K split C ways and reduced in distributed
    // shared memory.  Taken for few tokens when the tiles are fewer than the SMs and tiles x C - with C <= 8, two k-blocks
    // or more per CTA, the non-leaders' partial sums fitting the leader's ring, and all clusters resident at once - fill at
    // least 80 % of the SMs; otherwise (8B and 70B gate/up: 112 and 224 tiles) the stream-K form keeps every SM streaming.
    p.cluster = 0;
    p.c_boxes = 2;
    p.c_tiles = 0;
    p.c_stages = 0;
    p.c_smem_bytes = 0;
    p.c_staging_off = 0;
    {
        uint32_t c_cols = (uint32_t)(nmat * p.Mpad), c_pow2 = 32;
        while (c_pow2 < c_cols) c_pow2 <<= 1;
        p.c_tmem_cols = c_pow2;
        // Half-size rings (co-residency with the next kernel, see above) in the cluster form: only with at most 16 tokens and a
        // matrix of at most 28 MB.  A deep ring is worth more than the early start of the successor once the stream is long
        // (us per step, half / full: 2048 x 5632 20.4 / 22.3 at M = 8, but 22.7 / 21.2 at M = 17; 2048 x 8192 25.2 / 23.7;
        // 3072 x 8192 30.8 / 29.5; 8B layer 60.0 / 55.7; 5120 x 13824 71.8 / 66.0).
        bool c_small = p.Mpad <= 16 && K * N * 2 <= (int64_t)28 << 20;
        if (tuned_ring != 0) c_small = tuned_ring == 1;
        if (const char* e = getenv("GMLP_SKINNY_CLUSTER_SMALL")) { const int v = atoi(e); if (v == 0 || v == 1) c_small = v == 1; }   // tuning override
        int forced = -1;
        if (const char* e = getenv(nmat == 2 ? "GMLP_SKINNY_CLUSTER1" : "GMLP_SKINNY_CLUSTER2")) forced = atoi(e);   // tuning override: 0 = stream-K, 1..8 = that cluster size
        int forced_boxes = 0;
        if (const char* e = getenv("GMLP_SKINNY_CLUSTER_BOXES")) forced_boxes = atoi(e);                              // tuning override: 1 or 2
        int64_t best_ctas = 0;
        for (int boxes = 2; boxes >= 1 && p.Mpad <= gmlp::kSkinnyClusterMaxTokens && forced != 0; --boxes) {
            if (forced_boxes != 0 && forced_boxes != boxes) continue;
            if (boxes == 1 && p.cluster >= 1 && forced_boxes == 0) break;        // the wide tiles qualified
            const int tiles = (int)((N + 64 * boxes - 1) / (64 * boxes));
            const uint32_t c_stage_bytes = (uint32_t)(nmat * boxes) * gmlp::kSkinnyBoxBytes + (uint32_t)p.Mpad * 128u;
            // (a 64-column tile's MMA reads one box length past its box: keep that inside the allocation)
            const uint32_t tail = 1024 + 256 + (boxes == 1 ? gmlp::kSkinnyBoxBytes : 0);
            // few tokens: half of the shared memory, so that the next kernel on the stream is co-resident (see above)
            int cst = (int)(((c_small ? gmlp::kSkinnySmemBudget / 2 : gmlp::kSkinnySmemBudget) - tail) / c_stage_bytes);
            if (cst > gmlp::kSkinnyMaxStages) cst = gmlp::kSkinnyMaxStages;
            if (tiles > sms || cst < 2) continue;
            int C = forced > 0 ? forced : sms / tiles;
            if (C > 8) C = 8;
            if (C > p.KB / 2) C = p.KB / 2 > 0 ? p.KB / 2 : 1;
            while (C > 1 && (gmlp::skinny_cluster_staging_bytes(C, nmat, (int)M) > (uint32_t)cst * c_stage_bytes ||
                             cluster_capacity_estimate(C, sms) < tiles))
                --C;
            if (forced > 0 && C != forced) continue;
            const int64_t ctas = (int64_t)tiles * C;
            // 128-column tiles read 256 contiguous bytes per weight row, 64-column tiles 128: the narrow rows use DRAM
            // so much worse (8B down projection, 128 CTAs either way: 34.8 against 26.9 us) that the wide tiles are
            // taken from a quarter of the SMs on, the narrow ones only if they alone reach 80 %.  (The cluster form beats
            // stream-K, whose partial sums go through global memory, long before it fills the GPU: one SM pulls about 85 GB/s
            // through a full-size ring, so 77 of them keep up with HBM, and on small layers the hand-over counts for more
            // than the stream.  us per step, cluster form / stream-K for that GEMM: 4096 x 11008, 86 gate/up tiles with one
            // CTA each 45.6 / 47.3 at M = 8, 46.4 / 54.7 at 24, 49.2 / 78.5 at 64; 4096 x 9600, 75 tiles 40.0 / 43.1,
            // 41.5 / 49.8, 44.5 / 69.7; 1024 x 4096 down projection, 8 tiles x 8 CTAs 14.2 / 15.7, 14.7 / 19.9, 17.5 / 62.1.)
            if (ctas > best_ctas && (forced > 0 || ctas * 100 >= (int64_t)sms * (boxes == 2 ? 25 : 80))) {
                best_ctas = ctas;
                p.cluster = C;
                p.c_boxes = boxes;
                p.c_tiles = tiles;
                // partial sums of at most 24 KB get a region of their own behind the ring and its barriers (a stage less
                // if need be): the senders then do not have to wait for the receiver's ring to be free
                const uint32_t staging = gmlp::skinny_cluster_staging_bytes(C, nmat, (int)M);
                const uint32_t limit = c_small ? gmlp::kSkinnySmemBudget / 2 : gmlp::kSkinnySmemBudget;
                p.c_staging_off = 0;
                if (C > 1 && staging <= 24 * 1024) {
                    while (cst > 2 && (uint32_t)cst * c_stage_bytes + tail + staging > limit) --cst;
                    if ((uint32_t)cst * c_stage_bytes + tail + staging <= limit) p.c_staging_off = (uint32_t)cst * c_stage_bytes + tail;
                }
                p.c_stages = cst;
                p.c_smem_bytes = (uint32_t)cst * c_stage_bytes + tail + (p.c_staging_off ? staging : 0);
            }
        }
    }
    return p;
}

// ------------------------------------------------------------------ fused small-M plan (umma_skinny_fused.cuh)
// One cluster of C CTAs per 128-wide slice of d_ff; both GEMMs and the activation in one kernel, partial Y summed over
// the slices through scratch by a second, tiny kernel.  Applicable when the slices x C fill at least 60 % of the SMs in
// one wave, the accumulators fit TMEM - gate, up and this CTA's share of the d_model / 128
// partial-Y tiles, each Mpad columns - and every CTA has two k-blocks or more.  cluster == 0: not applicable.
struct FusedPlan {
    int cluster, slices, Mpad, stages;
    bool preferred;                             // faster than the two-kernel forms by measurement (see make_fused_plan)
    uint32_t smem_bytes, tmem_cols, hbuf_off, staging_off, bars_off;
    uint64_t scratch_bytes;
};

FusedPlan make_fused_plan(int64_t M, int64_t d_model, int64_t d_ff, int sm_count) {
    FusedPlan p{};
    if (M < 1 || M > gmlp::kFusedMaxTokens) return p;
    const int sms = sm_count > 0 ? sm_count : 148;
    p.Mpad = (int)((M + 15) / 16 * 16);
    const int64_t S = (d_ff + 127) / 128, NT = (d_model + 127) / 128, KB = (d_model + 63) / 64;
    if (S > sms) return p;
    int forced = -1;
    if (const char* e = getenv("GMLP_FUSED_CLUSTER")) forced = atoi(e);          // tuning override: that cluster size (0: none)
    if (forced == 0) return p;
    int best = 0;
    for (int C = 1; C <= 8; ++C) {
        if (forced > 0 && C != forced) continue;
        if (S * C > sms || cluster_capacity_estimate(C, sms) < S) continue;
        if (C > 1 && (KB / C < 2 || C > NT)) continue;
        if ((2 + (NT + C - 1) / C) * p.Mpad > 512) continue;
        best = C;                                                                 // the largest that fits: most SMs streaming
    }
    if (best == 0 || (forced <= 0 && S * best * 10 < (int64_t)sms * 6)) return p;
    const uint32_t stage_bytes = gmlp::kFusedWeightBytes + (uint32_t)p.Mpad * 128u;
    const uint32_t hbuf = 2u * (uint32_t)p.Mpad * 128u;
    const uint32_t staging = gmlp::skinny_fused_staging_bytes(best, (int)M);
    // all of the shared memory: a deep ring keeps W_down streaming through the exchange in the middle of the kernel, which
    // is worth more than having the next kernel on the stream co-resident (2048 x 5632, M = 7: 18.8 against 22.6 us per step)
    uint32_t budget = gmlp::kFusedSmemBudget;
    if (const char* e = getenv("GMLP_FUSED_SMEM_KB")) { int v = atoi(e); if (v >= 48 && v <= 224) budget = (uint32_t)v * 1024u; }   // tuning override
    const uint32_t fixed = 1024 + hbuf + staging + 256;
    if (budget < fixed + 2 * stage_bytes) return p;
    int st = (int)((budget - fixed) / stage_bytes);
    if (st > gmlp::kSkinnyMaxStages) st = gmlp::kSkinnyMaxStages;
    p.stages = st;
    p.hbuf_off = (uint32_t)st * stage_bytes;
    p.staging_off = p.hbuf_off + hbuf;
    p.bars_off = p.staging_off + staging;
    p.smem_bytes = p.bars_off + 256 + 1024;
    uint32_t cols = (uint32_t)((2 + (NT + best - 1) / best) * p.Mpad), pow2 = 32;
    while (pow2 < cols) pow2 <<= 1;
    p.tmem_cols = pow2;
    p.slices = (int)S;
    p.cluster = best;
    p.scratch_bytes = (uint64_t)S * (uint64_t)M * (uint64_t)d_model * 4u;
    // Where it pays (B200, cold weights, steps back to back, us per step fused / two kernels, M = 1 and M = 16):
    // 1024 x 4096 10.0 / 15.5 and 12.5 / 18.5; 1536 x 6144 15.2 / 18.9 and 16.1 / 20.4; 2048 x 5632 16.4 / 18.6 and 20.7 / 21.7;
    // 2048 x 6144 18.1 / 21.6 and 22.0 / 22.7; 1536 x 8960 19.8 / 22.2 and 22.8 / 23.3; from about 100 MB of weights on the
    // two forms are within a few percent of each other either way (2048 x 8192 22.1 / 23.5 and 26.7 / 24.6; 2560 x 6912
    // 22.9 / 23.8 and 27.8 / 25.2), and with more than six down-projection tiles per CTA, whose MMAs all come after the
    // exchange, the fused form loses (4096 x 5632: 35.5 / 26.9; 3072 x 8192 at M = 8: 33.4 / 29.5).
    p.preferred = 3 * d_model * d_ff * 2 <= (int64_t)90 << 20 && (NT + best - 1) / best <= 6;
    return p;
}

// ------------------------------------------------------------------ workspace layout
struct Layout {
    uint64_t xn_off, h_off, partial_off, counters_off, total;
    uint64_t counters_bytes;
    StreamPlan p1, p2;
    SkinnyPlan s1, s2;
    FusedPlan sf;
};

// Schedule choice for AUTO, from A/B timings on B200 (resolve_variant below has the table).  The operand-swapped SKINNY
// schedule streams every weight once with all SMs whatever the token count, where the 128-row tiles of TENSOR have too few
// tiles to fill the GPU on small and medium layers; SKINNY's epilogue work and, in its stream-K form, its partial-sum
// traffic grow with M, so TENSOR takes over from a token count that depends on the form.  TENSOR then picks, per GEMM,
// between single-CTA tiles and CTA pairs.  gmlp_autotune replaces this rule by a measurement for a given shape.
int check_shape_values(int64_t M, int64_t d_model, int64_t d_ff);
constexpr int kDownForms[6] = {0, 2, 3, 4, 12, 14};   // forms of the single-CTA down projection (see t_force_down_form)
struct TunedShape {
    int device;
    int64_t M, d_model, d_ff;
    int variant;
    int gu_pair, down_pair;                      // TENSOR: kernel of each GEMM (1 = CTA pairs, 0 = single CTAs)
    int gu_nb, down_form;                        // single-CTA kernels: tile form (see t_force_gu_nb / t_force_down_form)
    char device_name[64];                        // for the cache file: a choice belongs to the GPU model it was measured on
};
std::vector<TunedShape> g_tuned;                 // written by gmlp_autotune, under g_mutex
std::atomic<int> g_tuned_count{0};               // lets untuned processes skip the lock

// ---- the tuned choices as a text file (format: include/gmlp.h) ----
void device_name_of(int device, char (&name)[64]) {
    name[0] = 0;
    cudaDeviceProp prop;
    if (device >= 0 && cudaGetDeviceProperties(&prop, device) == cudaSuccess) {
        snprintf(name, sizeof(name), "%.63s", prop.name);
        for (char* c = name; *c; ++c)
            if (*c == '\t' || *c == '\n') *c = ' ';
    } else {
        (void)cudaGetLastError();
    }
}

bool tuned_values_valid(const TunedShape& t) {
    if (t.M <= 0 || check_shape_values(t.M, t.d_model, t.d_ff) != GMLP_OK) return false;
    if (t.variant != GMLP_VARIANT_SKINNY && t.variant != GMLP_VARIANT_TENSOR) return false;
    if (t.gu_pair < -1 || t.gu_pair > 1 || t.down_pair < -1 || t.down_pair > 1) return false;
    // (a SKINNY choice keeps its own two forms in the same fields: gu_nb = one-kernel form 0 rule / 1 on / 2 off, down_form =
    // ring size 0 rule / 1 half / 2 full)
    if (t.variant == GMLP_VARIANT_SKINNY) return t.gu_nb >= 0 && t.gu_nb <= 2 && t.down_form >= 0 && t.down_form <= 2;
    if (t.gu_nb != 0 && t.gu_nb != 2 && t.gu_nb != 4) return false;
    bool form_ok = false;
    for (int f : kDownForms) form_ok = form_ok || f == t.down_form;
    return form_ok;
}

int tune_cache_save(const char* path) {
    if (path == nullptr) return GMLP_ERR_NULL;
    const std::string tmp = std::string(path) + ".tmp";
    FILE* f = fopen(tmp.c_str(), "w");
    if (f == nullptr) return GMLP_ERR_LAUNCH;
    int n = 0;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        fprintf(f, "# libgmlp tuned schedule choices: version, device, M, d_model, d_ff, variant, gate_up_pair, down_pair, gate_up_form, down_form\n");
        for (const TunedShape& t : g_tuned) {
            fprintf(f, "gmlp-tune-v1\t%d\t%s\t%lld\t%lld\t%lld\t%d\t%d\t%d\t%d\t%d\n", kVersion, t.device_name, (long long)t.M,
                    (long long)t.d_model, (long long)t.d_ff, t.variant, t.gu_pair, t.down_pair, t.gu_nb, t.down_form);
            ++n;
        }
    }
    if (fclose(f) != 0 || rename(tmp.c_str(), path) != 0) {
        (void)remove(tmp.c_str());
        return GMLP_ERR_LAUNCH;
    }
    return n;
}

int tune_cache_load(const char* path, const char* device_name) {
    if (path == nullptr) return GMLP_ERR_NULL;
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0) { (void)cudaGetLastError(); device = 0; }
    char own_name[64];
    if (device_name == nullptr) {
        device_name_of(device, own_name);
        device_name = own_name;
    }
    FILE* f = fopen(path, "r");
    if (f == nullptr) return GMLP_ERR_LAUNCH;
    char line[512];
    int taken = 0;
    while (fgets(line, sizeof(line), f) != nullptr) {
        if (line[0] == '#' || line[0] == '\n' || line[0] == 0) continue;
        // tab-separated fields; the device name may contain spaces
        char* field[11];
        int nf = 0;
        for (char* p = line; nf < 11; ++nf) {
            field[nf] = p;
            char* tab = strchr(p, '\t');
            if (tab == nullptr) { ++nf; break; }
            *tab = 0;
            p = tab + 1;
        }
        if (nf != 11 || strcmp(field[0], "gmlp-tune-v1") != 0) continue;
        if (char* nl = strchr(field[10], '\n')) *nl = 0;
        char* end = nullptr;
        long long v[10] = {};
        bool ok = true;
        for (int i = 1; i < 11 && ok; ++i) {
            if (i == 2) continue;
            v[i - 1] = strtoll(field[i], &end, 10);
            ok = end != field[i] && *end == 0;
        }
        if (!ok || v[0] != kVersion || strcmp(field[2], device_name) != 0) continue;
        TunedShape t = {device, v[2], v[3], v[4], (int)v[5], (int)v[6], (int)v[7], (int)v[8], (int)v[9], {0}};
        snprintf(t.device_name, sizeof(t.device_name), "%s", device_name);
        if (!tuned_values_valid(t)) continue;
        std::lock_guard<std::mutex> lock(g_mutex);
        bool found = false;
        for (TunedShape& o : g_tuned)
            if (o.device == device && o.M == t.M && o.d_model == t.d_model && o.d_ff == t.d_ff) { o = t; found = true; }
        if (!found) g_tuned.push_back(t);
        g_tuned_count.store((int)g_tuned.size(), std::memory_order_release);
        ++taken;
    }
    fclose(f);
    return taken;
}

bool tuned_lookup(int64_t M, int64_t d_model, int64_t d_ff, TunedShape* out) {
    if (g_tuned_count.load(std::memory_order_acquire) == 0) return false;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return false; }
    std::lock_guard<std::mutex> lock(g_mutex);
    for (const TunedShape& t : g_tuned)
        if (t.device == dev && t.M == M && t.d_model == d_model && t.d_ff == d_ff) { *out = t; return true; }
    return false;
}

int tuned_variant(int64_t M, int64_t d_model, int64_t d_ff) {
    TunedShape t;
    return tuned_lookup(M, d_model, d_ff, &t) ? t.variant : GMLP_VARIANT_AUTO;
}

// gmlp_autotune forces the forms of the SKINNY schedule while it measures them (t_skinny_forced: also "by the rule", 0 / 0)
thread_local bool t_skinny_forced = false;
thread_local int t_force_skinny_fused = 0, t_force_skinny_ring = 0;
void skinny_forms(int64_t M, int64_t d_model, int64_t d_ff, int* fused, int* ring) {
    *fused = 0;
    *ring = 0;
    if (t_skinny_forced) {
        *fused = t_force_skinny_fused;
        *ring = t_force_skinny_ring;
        return;
    }
    TunedShape t;
    if (tuned_lookup(M, d_model, d_ff, &t) && t.variant == GMLP_VARIANT_SKINNY) {
        *fused = t.gu_nb;
        *ring = t.down_form;
    }
}

bool skinny_both_cluster(int64_t M, int64_t d_model, int64_t d_ff);

int resolve_variant(int64_t M, int64_t d_model, int64_t d_ff, int32_t variant) {
    if (variant != GMLP_VARIANT_AUTO) return variant;
    const int tuned = tuned_variant(M, d_model, d_ff);
    if (tuned != GMLP_VARIANT_AUTO) return tuned;
    // Measured, cold weights, us per step, operand-swapped / 128-row tiles:
    //   2048 x 5632:   M = 33 21.5 / 28.8, 64 24.0 / 29.2, 96 28.2 / 29.8, 128 31.8 / 30.5, 160 33.9 / 30.9, 256 46.5 / 31.5
    //   2048 x 8192:   M = 33 26.0 / 32.9, 96 29.9 / 33.9, 128 33.7 / 34.4, 160 36.2 / 34.6, 256 48.0 / 35.0
    //   3072 x 8192:   M = 33 32.0 / 39.0, 128 39.7 / 40.8, 129 40.4 / 53.5, 200 49.0 / 53.7, 256 55.6 / 54.3
    //   4096 x 14336:  M = 33 57.7 / 70.2, 128 66.1 / 72.1, 129 67.6 / 84.8, 200 81.2 / 87.7, 256 91.8 / 89.6
    //   5120 x 13824:  M = 33 67.5 / 78.9, 128 78.2 / 81.9, 129 79.7 / 109.1, 200 96.1 / 112.1, 256 109.1 / 115.1
    //   4096 x 11008:  M = 33 65.0 / 60.5, 64 79.3 / 61.2 (gate/up as stream-K: 86 tiles)
    //   8192 x 28672:  M = 8 211 / 232, 33 230 / 229, 64 248 / 230, 128 257 / 240 (gate/up as stream-K)
    // The operand-swapped schedule wins up to 32 tokens everywhere.  Where both of its GEMMs have the cluster form (no
    // partial sums through global memory) it wins up to 96 tokens on the narrow layers and - because the 128-row tiles pay
    // for a second row block from 129 tokens on - up to 200 on layers with d_model of 3072 or more.
    if (M <= 32) return GMLP_VARIANT_SKINNY;
    if (M <= (d_model >= 3072 ? 200 : 96) && skinny_both_cluster(M, d_model, d_ff)) return GMLP_VARIANT_SKINNY;
    return GMLP_VARIANT_TENSOR;
}

// TENSOR: which kernel each GEMM takes.  Both kernels are persistent, so a GEMM costs (rounds of tiles over the SMs)
// x (cost of a tile).  A CTA pair works on 256 rows at 0.94 of the cost of two single-CTA tiles (measured), but an
// odd number of 128-row blocks leaves half a pair idle in the last row tile and a pair tile count just above a
// multiple of 74 pays a whole extra round; the single-CTA kernel can narrow its tiles (128 columns at 0.75 of the
// cost) or split K over a cluster when its tiles are few.  The counts decide; this model reproduces the measured
// winner of all four combinations on 41 shapes (128-row blocks 2..32 on the 2048x5632, 8B and 70B layers), e.g.
// gate/up 8B: pairs for even block counts, single CTAs for odd ones up to 23; 2048x5632: pairs from 4 blocks on;
// down 8B: single CTAs up to 4 blocks and at 9 (307 vs 382 us), pairs otherwise.
// gmlp_autotune measures the four combinations for a given shape and overrides this rule.
int pick_split_k(int num_m, int64_t K, int64_t N, int sms);
static double rounds_of(int64_t tiles, int64_t units) { return (double)((tiles + units - 1) / units); }
constexpr double kPairTileCost = 0.94;
bool gate_up_uses_pair(int64_t M, int64_t d_ff, int sms) {
    const int64_t mt = (M + 127) / 128, ct = (d_ff + 127) / 128;
    if (mt < 2) return false;
    return kPairTileCost * rounds_of(((mt + 1) / 2) * ct, sms / 2) < rounds_of(mt * ct, sms);
}
bool down_uses_pair(int64_t M, int64_t d_ff, int64_t d_model, int sms) {
    const int64_t mt = (M + 127) / 128;
    if (mt < 2) return false;
    const int64_t t256 = mt * ((d_model + 255) / 256), t128 = mt * ((d_model + 127) / 128);
    double single = rounds_of(t256, sms);
    if (0.75 * rounds_of(t128, sms) < single) single = 0.75 * rounds_of(t128, sms);
    const int S = pick_split_k((int)mt, d_ff, d_model, sms);
    if (S >= 2) single = 0.75 / S + 0.1;                                // K split over a cluster, reduced on chip
    return kPairTileCost * rounds_of(((mt + 1) / 2) * ((d_model + 255) / 256), sms / 2) < single;
}

// The TENSOR plan of a shape: the rule above, unless gmlp_autotune measured the four combinations for this
// shape and kept another one; t_force_* is how the tuner runs a combination of its choosing.
struct TensorPlan {
    bool gu_pair, down_pair;
    int gu_nb, down_form;
};
thread_local int t_force_gu = -1, t_force_down = -1;
// Form of the single-CTA kernels, 0 = the library's own choice (pick_split_k / pick_umma_boxes / one-wave rule):
//   gate/up: 2 = 64-column tiles, 4 = 128-column tiles;
//   down:    2, 3, 4 = K split over a cluster of that many CTAs; 12 = 128-column tiles, 14 = 256-column tiles, no split.
// Set by gmlp_autotune while it measures, and from its result around the launches of a tuned shape.
thread_local int t_force_gu_nb = 0, t_force_down_form = 0;
struct UmmaFormScope {
    int prev_gu, prev_down;
    UmmaFormScope(int gu_nb, int down_form) : prev_gu(t_force_gu_nb), prev_down(t_force_down_form) {
        t_force_gu_nb = gu_nb;
        t_force_down_form = down_form;
    }
    ~UmmaFormScope() {
        t_force_gu_nb = prev_gu;
        t_force_down_form = prev_down;
    }
};
TensorPlan tensor_plan(int64_t M, int64_t d_model, int64_t d_ff, int sms) {
    if (sms <= 0) sms = 148;
    TensorPlan p = {gate_up_uses_pair(M, d_ff, sms), down_uses_pair(M, d_ff, d_model, sms), t_force_gu_nb, t_force_down_form};
    TunedShape t;
    if (tuned_lookup(M, d_model, d_ff, &t) && t.variant == GMLP_VARIANT_TENSOR) {
        p.gu_pair = t.gu_pair != 0;
        p.down_pair = t.down_pair != 0;
        if (t_force_gu_nb == 0) p.gu_nb = t.gu_nb;
        if (t_force_down_form == 0) p.down_form = t.down_form;
    }
    if (t_force_gu >= 0) p.gu_pair = t_force_gu != 0;
    if (t_force_down >= 0) p.down_pair = t_force_down != 0;
    return p;
}

Layout make_layout(int64_t M, int64_t d_model, int64_t d_ff, uint32_t flags, int variant, int sm_count) {
    Layout L{};
    uint64_t off = 0;
    L.xn_off = off;
    if (flags & GMLP_FLAG_RMSNORM) off += align256((uint64_t)M * d_model * 2);
    L.h_off = off;
    off += align256((uint64_t)M * d_ff * 2);
    L.partial_off = off;
    L.counters_off = off;
    if (variant == GMLP_VARIANT_STREAM) {
        L.p1 = make_stream_plan(M, d_model, d_ff, 2, sm_count);
        L.p2 = make_stream_plan(M, d_ff, d_model, 1, sm_count);
        const uint64_t b1 = (uint64_t)2 * L.p1.KS * M * d_ff * 4;
        const uint64_t b2 = (uint64_t)L.p2.KS * M * d_model * 4;
        off += align256(b1 > b2 ? b1 : b2);      // the two phases run one after the other and share it
        L.counters_off = off;
        L.counters_bytes = align256((uint64_t)(L.p1.row_tiles * L.p1.slabs + L.p2.row_tiles * L.p2.slabs) * 4);
        off += L.counters_bytes;
    } else if (variant == GMLP_VARIANT_SKINNY) {
        L.s1 = make_skinny_plan(M, d_model, d_ff, 2, sm_count);
        L.s2 = make_skinny_plan(M, d_ff, d_model, 1, sm_count);
        L.sf = make_fused_plan(M, d_model, d_ff, sm_count);
        uint64_t scratch = L.s1.scratch_bytes > L.s2.scratch_bytes ? L.s1.scratch_bytes : L.s2.scratch_bytes;
        if (L.sf.cluster >= 1 && L.sf.scratch_bytes > scratch) scratch = L.sf.scratch_bytes;
        off += align256(scratch);
        L.counters_off = off;
        L.counters_bytes = align256((uint64_t)(L.s1.num_tiles + L.s2.num_tiles) * 4);
        off += L.counters_bytes;
    }
    L.total = off;
    return L;
}

// The operand-swapped schedule takes up to 128 tokens in its stream-K form, and up to kSkinnyClusterMaxTokens when both
// GEMMs of the shape have a cluster form.
bool skinny_can_run(int64_t M, int64_t d_model, int64_t d_ff, int sm_count) {
    if (M <= 128) return true;
    if (M > gmlp::kSkinnyClusterMaxTokens) return false;
    return make_skinny_plan(M, d_model, d_ff, 2, sm_count).cluster >= 1 && make_skinny_plan(M, d_ff, d_model, 1, sm_count).cluster >= 1;
}

int current_sm_count() {
    int dev = -1, sms = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < kMaxDevices &&
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
        return sms;
    (void)cudaGetLastError();
    return 148;
}
bool skinny_both_cluster(int64_t M, int64_t d_model, int64_t d_ff) {
    const int sms = current_sm_count();
    return make_skinny_plan(M, d_model, d_ff, 2, sms).cluster >= 1 && make_skinny_plan(M, d_ff, d_model, 1, sms).cluster >= 1;
}

int check_shape(int64_t M, int64_t d_model, int64_t d_ff) {
    if (M < 0 || d_model <= 0 || d_ff <= 0 || (d_model & 7) || (d_ff & 7)) return GMLP_ERR_SHAPE;
    if (M > kMaxDim || d_model > kMaxDim || d_ff > kMaxDim) return GMLP_ERR_SHAPE;
    return GMLP_OK;
}
int check_shape_values(int64_t M, int64_t d_model, int64_t d_ff) { return check_shape(M, d_model, d_ff); }

// ------------------------------------------------------------------ TMA descriptors
// 2-D bf16 tensor, row-major [outer, inner]; box = box_outer rows x box_inner elements, 128-byte swizzle,
// out-of-bounds elements read as zero.
bool encode_2d(CUtensorMap* map, const void* ptr, uint64_t inner, uint64_t outer, uint32_t box_inner, uint32_t box_outer) {
    const cuuint64_t gdim[2] = {inner, outer};
    const cuuint64_t gstride[1] = {inner * 2};
    const cuuint32_t box[2] = {box_inner, box_outer};
    const cuuint32_t estride[2] = {1, 1};
    return g_encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), gdim, gstride, box, estride,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The split-K kernels leave their arrival counters at zero when they finish, so the counters only
// need clearing the first time a given counter region is used (or after a failed call).
int ensure_counters_zero(DeviceState* dev, void* ptr, uint64_t bytes, cudaStream_t st) {
    std::lock_guard<std::mutex> lock(g_mutex);
    for (int i = 0; i < DeviceState::kCleanSlots; ++i)
        if (dev->clean_counters[i] == ptr && dev->clean_counters_bytes[i] == bytes) return GMLP_OK;
    if (cudaMemsetAsync(ptr, 0, bytes, st) != cudaSuccess) return GMLP_ERR_LAUNCH;
    dev->clean_counters[dev->clean_next] = ptr;
    dev->clean_counters_bytes[dev->clean_next] = bytes;
    dev->clean_next = (dev->clean_next + 1) % DeviceState::kCleanSlots;
    return GMLP_OK;
}

// A call is about to use [ws, ws + total) as its workspace.  Counter regions remembered as zero that lie in that
// range were put there by calls with another layout (another shape or schedule in the same buffer) and are about to
// be overwritten by this call's intermediates - except the region this call itself keeps its counters in.
void claim_workspace(DeviceState* dev, const uint8_t* ws, uint64_t total, const void* keep_ptr, uint64_t keep_bytes) {
    std::lock_guard<std::mutex> lock(g_mutex);
    for (int i = 0; i < DeviceState::kCleanSlots; ++i) {
        const uint8_t* c = static_cast<const uint8_t*>(dev->clean_counters[i]);
        if (c == nullptr) continue;
        const bool same = dev->clean_counters[i] == keep_ptr && dev->clean_counters_bytes[i] == keep_bytes;
        const bool overlaps = c < ws + total && c + dev->clean_counters_bytes[i] > ws;
        if (overlaps && !same) {
            dev->clean_counters[i] = nullptr;
            dev->clean_counters_bytes[i] = 0;
        }
    }
}

void forget_counters_locked(DeviceState* dev) {
    for (int i = 0; i < DeviceState::kCleanSlots; ++i) {
        dev->clean_counters[i] = nullptr;
        dev->clean_counters_bytes[i] = 0;
    }
}

void forget_counters(DeviceState* dev) {
    std::lock_guard<std::mutex> lock(g_mutex);
    forget_counters_locked(dev);
}

// ------------------------------------------------------------------ launches
#define GMLP_CHECK_LAUNCH()                                   \
    do {                                                      \
        if (cudaPeekAtLastError() != cudaSuccess) return GMLP_ERR_LAUNCH; \
        ++t_launches;                                         \
        t_first_launch_ordered = false;                       \
    } while (0)

int launch_rmsnorm(const bf16* X, const bf16* gain, bf16* Xn, int64_t M, int64_t d_model, float eps, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)M);
    cfg.blockDim = dim3(gmlp::kRmsThreads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl_allowed();
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int dm = (int)d_model;
    if (cudaLaunchKernelEx(&cfg, gmlp::rmsnorm_kernel, X, gain, Xn, M, dm, eps) != cudaSuccess) return GMLP_ERR_LAUNCH;
    GMLP_CHECK_LAUNCH();
    return GMLP_OK;
}

int run_simt(const bf16* A, const bf16* Wg, const bf16* Wu, const bf16* Wd, bf16* H, bf16* Y,
             int64_t M, int64_t d_model, int64_t d_ff, cudaStream_t st, gmlp::GateAct act) {
    const int T = gmlp::kSimtTile;
    dim3 g1((unsigned)((d_ff + T - 1) / T), (unsigned)((M + T - 1) / T));
    gmlp::simt_gemm_kernel<true><<<g1, 256, 0, st>>>(A, Wg, Wu, H, M, (int)d_model, (int)d_ff, act);
    GMLP_CHECK_LAUNCH();
    prof_mark("gate_up", st);
    dim3 g2((unsigned)((d_model + T - 1) / T), (unsigned)((M + T - 1) / T));
    gmlp::simt_gemm_kernel<false><<<g2, 256, 0, st>>>(H, Wd, nullptr, Y, M, (int)d_ff, (int)d_model, kSilu);
    GMLP_CHECK_LAUNCH();
    prof_mark("down", st);
    return GMLP_OK;
}

template <bool GATEUP>
int launch_stream(const StreamPlan& p, const bf16* A, const bf16* W0, const bf16* W1, float* partial,
                  unsigned int* counters, bf16* out, int64_t M, int64_t K, int64_t N, cudaStream_t st,
                  gmlp::GateAct act = kSilu) {
    dim3 grid((unsigned)p.slabs, (unsigned)(p.KS * (GATEUP ? 2 : 1)), (unsigned)p.row_tiles);
    const int Mi = (int)M, Ki = (int)K, Ni = (int)N;
    switch (p.MT) {
        case 1: gmlp::stream_gemm_kernel<1, GATEUP><<<grid, gmlp::kStreamThreads, 0, st>>>(A, W0, W1, partial, counters, out, Mi, Ki, Ni, p.kchunk, p.KS, act); break;
        case 2: gmlp::stream_gemm_kernel<2, GATEUP><<<grid, gmlp::kStreamThreads, 0, st>>>(A, W0, W1, partial, counters, out, Mi, Ki, Ni, p.kchunk, p.KS, act); break;
        case 4: gmlp::stream_gemm_kernel<4, GATEUP><<<grid, gmlp::kStreamThreads, 0, st>>>(A, W0, W1, partial, counters, out, Mi, Ki, Ni, p.kchunk, p.KS, act); break;
        default: gmlp::stream_gemm_kernel<8, GATEUP><<<grid, gmlp::kStreamThreads, 0, st>>>(A, W0, W1, partial, counters, out, Mi, Ki, Ni, p.kchunk, p.KS, act); break;
    }
    GMLP_CHECK_LAUNCH();
    return GMLP_OK;
}

int run_stream(DeviceState* dev, const Layout& L, uint8_t* ws, const bf16* A, const bf16* Wg, const bf16* Wu, const bf16* Wd, bf16* H,
               bf16* Y, int64_t M, int64_t d_model, int64_t d_ff, cudaStream_t st, gmlp::GateAct act) {
    float* partial = reinterpret_cast<float*>(ws + L.partial_off);
    unsigned int* c1 = reinterpret_cast<unsigned int*>(ws + L.counters_off);
    unsigned int* c2 = c1 + L.p1.row_tiles * L.p1.slabs;
    int rc = ensure_counters_zero(dev, c1, L.counters_bytes, st);
    if (rc != GMLP_OK) return rc;
    rc = launch_stream<true>(L.p1, A, Wg, Wu, partial, c1, H, M, d_model, d_ff, st, act);
    if (rc != GMLP_OK) return rc;
    prof_mark("gate_up", st);
    rc = launch_stream<false>(L.p2, H, Wd, nullptr, partial, c2, Y, M, d_ff, d_model, st);
    if (rc == GMLP_OK) prof_mark("down", st);
    return rc;
}

// Tile width for the plain (down) GEMM: 256 columns unless the grid would be so small, or the last round so
// empty, that 128-column tiles (about 0.75 of the cost each, measured) finish sooner.
int pick_umma_boxes(int64_t num_m, int64_t N, int sms) {
    const int64_t t256 = num_m * ((N + 255) / 256), t128 = num_m * ((N + 127) / 128);
    const double c256 = (double)((t256 + sms - 1) / sms), c128 = 0.75 * (double)((t128 + sms - 1) / sms);
    int nb = c128 < c256 ? 2 : 4;
    if (const char* e = getenv("GMLP_UMMA_NB")) { if (e[0] == '2') nb = 2; if (e[0] == '4') nb = 4; }   // tuning override
    return nb;
}

// Length of an accumulation chain (in k-blocks of 64) of the Gated MLP's CTA-pair GEMMs; 0 = one chain per tile.
// Gate/up: the tensor core's truncating accumulation biases g and u in proportion to the chain length, and H is
// rounded to bf16 right after, so a long chain changes which bf16 many H values round to (measured on rows scaled
// by 20, K = 8192: 1.8 % of them with one chain, 0.24 % with chains of 16 k-blocks, 0.12 % with 8, 0.05 % for
// sequential fp32 FMA; elements beyond the absolute output tolerance on three such rows: 274 / 134 / 19 / 15).
// Chains of 8 cost 3.5 % of the kernel's cycles (about one MMA time per chain switch), chains of 16 nothing
// measurable: 8 from K = 8192 on, 16 below.  Down projection: its output is rounded once at the end and the
// chain length made no difference to any compared element (one chain of 448 k-blocks: 18 elements, chains of 8: 19),
// so it keeps one chain.
int pair_chunk_kb(bool gate_up, int64_t K) {
    int v = gate_up ? (K >= 8192 ? gmlp::kPairChunkKb : 2 * gmlp::kPairChunkKb) : 0;
    if (const char* e = getenv("GMLP_PAIR_CHUNK_KB")) v = atoi(e);                                   // tuning override
    if (const char* e = getenv(gate_up ? "GMLP_PAIR_CHUNK_KB_GU" : "GMLP_PAIR_CHUNK_KB_DOWN")) v = atoi(e);
    return v > 0 ? v : 0;
}

// chunk_kb > 0: the kernel form that accumulates K in chains of that many k-blocks (the Gated MLP's own GEMMs);
// the other operators' plain products keep one chain per tile.
template <bool GATEUP>
int launch_umma_pair(DeviceState* dev, const bf16* A, const bf16* W0, const bf16* W1, bf16* C,
                     int64_t M, int64_t K, int64_t N, cudaStream_t st, gmlp::GateAct act = kSilu, int chunk_kb = 0) {
    const int wkm = t_w_out_in ? 1 : 0;
    const int yf32 = (!GATEUP && t_y_fp32) ? 1 : 0;
    CUtensorMap tmA, tmB0, tmB1;
    if (!encode_2d(&tmA, A, (uint64_t)K, (uint64_t)M, gmlp::kUmmaBK, 128)) return GMLP_ERR_LAUNCH;
    if (!GMLP_ENCODE_W(&tmB0, W0, N, K)) return GMLP_ERR_LAUNCH;
    if (GATEUP) {
        if (!GMLP_ENCODE_W(&tmB1, W1, N, K)) return GMLP_ERR_LAUNCH;
    } else {
        tmB1 = tmB0;
    }
    if (!dev->pair_attr_set) {
        const int b = (int)gmlp::kPairSmemBytes;
        if (cudaFuncSetAttribute(gmlp::umma_pair_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, b) != cudaSuccess ||
            cudaFuncSetAttribute(gmlp::umma_pair_gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, b) != cudaSuccess ||
            cudaFuncSetAttribute(gmlp::umma_pair_gemm_kernel<true, false, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, b) != cudaSuccess ||
            cudaFuncSetAttribute(gmlp::umma_pair_gemm_kernel<false, false, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, b) != cudaSuccess)
            return GMLP_ERR_LAUNCH;
        dev->pair_attr_set = true;
    }
    const int sms = dev->sm_count > 0 ? dev->sm_count : 148;
    const int num_m = (int)((M + 255) / 256);
    const int bn = GATEUP ? 128 : 256;
    const int num_tiles = num_m * (int)((N + bn - 1) / bn);
    const int pairs = num_tiles < sms / 2 ? num_tiles : sms / 2;
    const bool chunked = chunk_kb > 0;
    // Row tiles in groups of eight when there are two groups or more (70B prefill, 16 row tiles: 4.33 -> 4.22 ms;
    // 2048 x 5632 at M = 8192: 0.441 -> 0.432 ms; on 8 row tiles groups of four cost 3 %)
    int group_m = num_m >= 16 ? 8 : 0;
    if (const char* e = getenv(GATEUP ? "GMLP_PAIR_GROUP_M_GU" : "GMLP_PAIR_GROUP_M_DOWN")) group_m = atoi(e);   // tuning override
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * pairs));
    cfg.blockDim = dim3(chunked ? gmlp::kPairChunkThreads : gmlp::kUmmaThreads);
    cfg.dynamicSmemBytes = gmlp::kPairSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = pdl_allowed();
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    const int Mi = (int)M, Ki = (int)K, Ni = (int)N;
    const cudaError_t err = chunked
        ? cudaLaunchKernelEx(&cfg, gmlp::umma_pair_gemm_kernel<GATEUP, false, false, false, true>, tmA, tmB0, tmB1, C, Mi, Ki, Ni,
                             num_m, num_tiles, (const float*)nullptr, act, (const bf16*)nullptr, (float*)nullptr, kNoMulti, wkm,
                             yf32, chunk_kb, group_m)
        : cudaLaunchKernelEx(&cfg, gmlp::umma_pair_gemm_kernel<GATEUP, false>, tmA, tmB0, tmB1, C, Mi, Ki, Ni, num_m,
                             num_tiles, (const float*)nullptr, act, (const bf16*)nullptr, (float*)nullptr, kNoMulti, wkm, yf32, 0,
                             group_m);
    if (err != cudaSuccess) return GMLP_ERR_LAUNCH;
    GMLP_CHECK_LAUNCH();
    return GMLP_OK;
}

// Cluster size of the split-K schedule for a plain GEMM with num_m x ceil(N/128) output tiles, or 0 when the
// ordinary one-CTA-per-tile schedule is to be used: the largest S in {4, 3, 2} whose tiles x S CTAs still fit
// the SMs in one wave, provided every CTA keeps at least 8 k-blocks.
int pick_split_k(int num_m, int64_t K, int64_t N, int sms) {
    if (const char* e = getenv("GMLP_UMMA_SPLITK")) {               // tuning override: 0 disables, 2..4 forces
        const int v = atoi(e);
        if (v == 0) return 0;
        if (v >= 2 && v <= 4 && (K + 63) / 64 >= v) return v;
    }
    const int64_t tiles = (int64_t)num_m * ((N + 127) / 128);
    const int64_t nkb = (K + gmlp::kUmmaBK - 1) / gmlp::kUmmaBK;
    for (int S = 4; S >= 2; --S)
        if (tiles * S <= sms && nkb / S >= 8) return S;
    return 0;
}

int launch_umma_splitk(DeviceState* dev, int S, const CUtensorMap& tmA, const CUtensorMap& tmB, bf16* C,
                       int64_t M, int64_t K, int64_t N, int num_m, int a_box_rows, cudaStream_t st) {
    const int wkm = t_w_out_in ? 1 : 0;
    const int yf32 = t_y_fp32 ? 1 : 0;
    if (!dev->splitk_attr_set) {
        const int b = (int)gmlp::kSplitSmemBytes;
        if (cudaFuncSetAttribute(gmlp::umma_splitk_gemm_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, b) != cudaSuccess ||
            cudaFuncSetAttribute(gmlp::umma_splitk_gemm_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, b) != cudaSuccess ||
            cudaFuncSetAttribute(gmlp::umma_splitk_gemm_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, b) != cudaSuccess)
            return GMLP_ERR_LAUNCH;
        dev->splitk_attr_set = true;
    }
    const int num_tiles = num_m * (int)((N + 127) / 128);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(num_tiles * S));
    cfg.blockDim = dim3(gmlp::kUmmaThreads);
    cfg.dynamicSmemBytes = gmlp::kSplitSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)S;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = pdl_allowed();
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    const int Mi = (int)M, Ki = (int)K, Ni = (int)N;
    cudaError_t err;
    if (S == 4) err = cudaLaunchKernelEx(&cfg, gmlp::umma_splitk_gemm_kernel<4>, tmA, tmB, C, Mi, Ki, Ni, num_m, a_box_rows, wkm, yf32);
    else if (S == 3) err = cudaLaunchKernelEx(&cfg, gmlp::umma_splitk_gemm_kernel<3>, tmA, tmB, C, Mi, Ki, Ni, num_m, a_box_rows, wkm, yf32);
    else err = cudaLaunchKernelEx(&cfg, gmlp::umma_splitk_gemm_kernel<2>, tmA, tmB, C, Mi, Ki, Ni, num_m, a_box_rows, wkm, yf32);
    if (err != cudaSuccess) return GMLP_ERR_LAUNCH;
    GMLP_CHECK_LAUNCH();
    return GMLP_OK;
}

template <bool GATEUP>
int launch_umma(DeviceState* dev, const bf16* A, const bf16* W0, const bf16* W1, bf16* C,
                int64_t M, int64_t K, int64_t N, cudaStream_t st, gmlp::GateAct act = kSilu) {
    const int wkm = t_w_out_in ? 1 : 0;
    const int yf32 = (!GATEUP && t_y_fp32) ? 1 : 0;
    CUtensorMap tmA, tmB0, tmB1;
    // TMA is markedly slower when a box has fewer than 16 rows inside the tensor; with so few rows in all, the
    // box is made exactly M rows high instead (no out-of-range rows to fill)
    int exact_below = 16;
    if (const char* e = getenv("GMLP_UMMA_EXACT_BOX_BELOW")) exact_below = atoi(e);      // tuning override
    const int a_box_rows = (M < exact_below && M < gmlp::kUmmaBM) ? (int)M : gmlp::kUmmaBM;
    if (!encode_2d(&tmA, A, (uint64_t)K, (uint64_t)M, gmlp::kUmmaBK, (uint32_t)a_box_rows)) return GMLP_ERR_LAUNCH;
    if (!GMLP_ENCODE_W(&tmB0, W0, N, K)) return GMLP_ERR_LAUNCH;
    if (GATEUP) {
        if (!GMLP_ENCODE_W(&tmB1, W1, N, K)) return GMLP_ERR_LAUNCH;
    } else {
        tmB1 = tmB0;
    }
    if (!dev->umma_attr_set) {
        const int b = (int)gmlp::kUmmaSmemBytes;
        if (cudaFuncSetAttribute(gmlp::umma_gemm_kernel<true, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, b) != cudaSuccess ||
            cudaFuncSetAttribute(gmlp::umma_gemm_kernel<true, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, b) != cudaSuccess ||
            cudaFuncSetAttribute(gmlp::umma_gemm_kernel<false, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, b) != cudaSuccess ||
            cudaFuncSetAttribute(gmlp::umma_gemm_kernel<false, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, b) != cudaSuccess)
            return GMLP_ERR_LAUNCH;
        dev->umma_attr_set = true;
    }
    const int sms = dev->sm_count > 0 ? dev->sm_count : 148;
    const int num_m = (int)((M + gmlp::kUmmaBM - 1) / gmlp::kUmmaBM);
    if (!GATEUP) {
        // few output tiles: a cluster of S CTAs per tile splits K and reduces through distributed shared memory
        int S = pick_split_k(num_m, K, N, sms);
        const int form = t_force_down_form;
        if (form >= 2 && form <= 4 && (K + gmlp::kUmmaBK - 1) / gmlp::kUmmaBK >= form) S = form;
        else if (form == 12 || form == 14) S = 0;
        if (S >= 2) return launch_umma_splitk(dev, S, tmA, tmB0, C, M, K, N, num_m, a_box_rows, st);
    }
    // gate/up: 128 output columns per tile (two boxes of gate + two of up), or 64 when that still fits one wave
    int gu_nb = (int64_t)num_m * ((N + 63) / 64) <= sms ? 2 : 4;
    if (const char* e = getenv("GMLP_UMMA_GATEUP_NB")) gu_nb = atoi(e) == 2 ? 2 : 4;    // tuning override
    if (t_force_gu_nb == 2 || t_force_gu_nb == 4) gu_nb = t_force_gu_nb;
    int down_nb = pick_umma_boxes(num_m, N, sms);
    if (t_force_down_form == 12) down_nb = 2;
    if (t_force_down_form == 14) down_nb = 4;
    const int nb = GATEUP ? gu_nb : down_nb;
    const int bn = GATEUP ? 32 * nb : 64 * nb;
    const int num_n = (int)((N + bn - 1) / bn);
    const int num_tiles = num_m * num_n;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(num_tiles < sms ? num_tiles : sms));     // persistent: one CTA per SM
    cfg.blockDim = dim3(gmlp::kUmmaThreads);
    cfg.dynamicSmemBytes = gmlp::kUmmaSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl_allowed();
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int Mi = (int)M, Ki = (int)K, Ni = (int)N;
    cudaError_t err;
    if (GATEUP && nb == 4)
        err = cudaLaunchKernelEx(&cfg, gmlp::umma_gemm_kernel<true, 4>, tmA, tmB0, tmB1, C, Mi, Ki, Ni, num_m, num_tiles,
                                 (const float*)nullptr, a_box_rows, act, (const bf16*)nullptr, (float*)nullptr, kNoMulti, wkm, yf32);
    else if (GATEUP)
        err = cudaLaunchKernelEx(&cfg, gmlp::umma_gemm_kernel<true, 2>, tmA, tmB0, tmB1, C, Mi, Ki, Ni, num_m, num_tiles,
                                 (const float*)nullptr, a_box_rows, act, (const bf16*)nullptr, (float*)nullptr, kNoMulti, wkm, yf32);
    else if (nb == 4)
        err = cudaLaunchKernelEx(&cfg, gmlp::umma_gemm_kernel<false, 4>, tmA, tmB0, tmB1, C, Mi, Ki, Ni, num_m, num_tiles,
                                 (const float*)nullptr, a_box_rows, act, (const bf16*)nullptr, (float*)nullptr, kNoMulti, wkm, yf32);
    else
        err = cudaLaunchKernelEx(&cfg, gmlp::umma_gemm_kernel<false, 2>, tmA, tmB0, tmB1, C, Mi, Ki, Ni, num_m, num_tiles,
                                 (const float*)nullptr, a_box_rows, act, (const bf16*)nullptr, (float*)nullptr, kNoMulti, wkm, yf32);
    if (err != cudaSuccess) return GMLP_ERR_LAUNCH;
    GMLP_CHECK_LAUNCH();
    return GMLP_OK;
}

// The cluster form of a small-M GEMM (umma_skinny_cluster.cuh).  Returns GMLP_ERR_UNSUPPORTED when the device cannot
// hold the plan's clusters in one wave (the caller then runs the stream-K form).
template <bool GATEUP>
int launch_skinny_cluster(DeviceState* dev, const SkinnyPlan& p, const CUtensorMap& tmX, const CUtensorMap& tmW0,
                          const CUtensorMap& tmW1, bf16* out, int64_t M, int64_t N, cudaStream_t st, gmlp::GateAct act,
                          int wkm, int yf32) {
    if (!dev->skinny_cluster_attr_set) {
        const int b = (int)gmlp::kSkinnySmemBudget;
        if (cudaFuncSetAttribute(gmlp::skinny_cluster_gemm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, b) != cudaSuccess ||
            cudaFuncSetAttribute(gmlp::skinny_cluster_gemm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, b) != cudaSuccess)
            return GMLP_ERR_LAUNCH;
        dev->skinny_cluster_attr_set = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.c_tiles * p.cluster));
    cfg.blockDim = dim3(gmlp::kSkinnyThreads);
    cfg.dynamicSmemBytes = p.c_smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)p.cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = pdl_allowed();
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    int& capacity = dev->cluster_capacity[GATEUP ? 0 : 1][p.cluster];
    if (capacity == 0) {
        int n = 0;
        cfg.numAttrs = 1;                                   // the occupancy query takes the cluster shape only
        if (cudaOccupancyMaxActiveClusters(&n, gmlp::skinny_cluster_gemm_kernel<GATEUP>, &cfg) != cudaSuccess) {
            (void)cudaGetLastError();
            n = -1;
        }
        cfg.numAttrs = 2;
        capacity = n > 0 ? n : -1;
        if (getenv("GMLP_TUNE_VERBOSE"))
            fprintf(stderr, "gmlp: clusters of %d CTAs (%s, %u B shared memory) resident at once: %d\n", p.cluster,
                    GATEUP ? "gate/up" : "down", p.c_smem_bytes, n);
    }
    if (capacity < p.c_tiles) return GMLP_ERR_UNSUPPORTED;
    const int Mi = (int)M, Ni = (int)N;
    int evict_first = 1;
    if (const char* e = getenv("GMLP_SKINNY_EVICT_FIRST")) evict_first = atoi(e);      // tuning override
    if (cudaLaunchKernelEx(&cfg, gmlp::skinny_cluster_gemm_kernel<GATEUP>, tmX, tmW0, tmW1, out, Mi, p.Mpad, Ni, p.KB, p.c_stages,
                           p.c_tmem_cols, evict_first, act, wkm, yf32, p.c_boxes, p.c_staging_off) != cudaSuccess)
        return GMLP_ERR_LAUNCH;
    GMLP_CHECK_LAUNCH();
    return GMLP_OK;
}

template <bool GATEUP>
int launch_skinny(DeviceState* dev, const SkinnyPlan& p, const bf16* X, const bf16* W0, const bf16* W1, float* scratch,
                  unsigned int* counters, bf16* out, int64_t M, int64_t K, int64_t N, cudaStream_t st,
                  gmlp::GateAct act = kSilu) {
    const int wkm = t_w_out_in ? 1 : 0;
    const int yf32 = (!GATEUP && t_y_fp32) ? 1 : 0;
    if (p.cluster < 1 && (p.stages < 2 || p.tmem_cols > 512)) return GMLP_ERR_UNSUPPORTED;
    CUtensorMap tmX, tmW0, tmW1;
    if (!encode_2d(&tmX, X, (uint64_t)K, (uint64_t)M, 64, (uint32_t)p.Mpad)) return GMLP_ERR_LAUNCH;
    if (!GMLP_ENCODE_W(&tmW0, W0, N, K)) return GMLP_ERR_LAUNCH;
    if (GATEUP) {
        if (!GMLP_ENCODE_W(&tmW1, W1, N, K)) return GMLP_ERR_LAUNCH;
    } else {
        tmW1 = tmW0;
    }
    if (p.cluster >= 1) {
        const int rc = launch_skinny_cluster<GATEUP>(dev, p, tmX, tmW0, tmW1, out, M, N, st, act, wkm, yf32);
        if (rc != GMLP_ERR_UNSUPPORTED) return rc;          // clusters that do not fit one wave: the stream-K form below
        if (M > 128 || p.stages < 2 || p.tmem_cols > 512) return GMLP_ERR_UNSUPPORTED;
    }
    if (!dev->skinny_attr_set) {
        const int b = (int)gmlp::kSkinnySmemBudget;
        if (cudaFuncSetAttribute(gmlp::skinny_gemm_kernel<true, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, b) != cudaSuccess ||
            cudaFuncSetAttribute(gmlp::skinny_gemm_kernel<true, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, b) != cudaSuccess ||
            cudaFuncSetAttribute(gmlp::skinny_gemm_kernel<false, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, b) != cudaSuccess ||
            cudaFuncSetAttribute(gmlp::skinny_gemm_kernel<false, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, b) != cudaSuccess)
            return GMLP_ERR_LAUNCH;
        dev->skinny_attr_set = true;
    }
    // programmatic stream serialization: this kernel may become resident while the previous kernel on
    // the stream drains; it orders itself with griddepcontrol.wait
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.grid);
    cfg.blockDim = dim3(gmlp::kSkinnyThreads);
    cfg.dynamicSmemBytes = p.smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl_allowed();
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int Mi = (int)M, Ni = (int)N;
    int evict_first = 1;                                // weights are read once: let L2 drop them first
    if (const char* e = getenv("GMLP_SKINNY_EVICT_FIRST")) evict_first = atoi(e);      // tuning override
    cudaError_t err;
    if (p.NH == 2)
        err = cudaLaunchKernelEx(&cfg, gmlp::skinny_gemm_kernel<GATEUP, 2>, tmX, tmW0, tmW1, scratch, counters, out,
                                 Mi, p.Mpad, Ni, p.num_tiles, p.KB, p.stages, p.tmem_cols, evict_first, act, wkm, yf32);
    else
        err = cudaLaunchKernelEx(&cfg, gmlp::skinny_gemm_kernel<GATEUP, 1>, tmX, tmW0, tmW1, scratch, counters, out,
                                 Mi, p.Mpad, Ni, p.num_tiles, p.KB, p.stages, p.tmem_cols, evict_first, act, wkm, yf32);
    if (err != cudaSuccess) return GMLP_ERR_LAUNCH;
    GMLP_CHECK_LAUNCH();
    return GMLP_OK;
}

// The fused form of the small-M schedule (umma_skinny_fused.cuh): one launch for the whole layer.  Returns
// GMLP_ERR_UNSUPPORTED when the device cannot hold all clusters at once (the caller then runs the two-kernel forms).
int launch_skinny_fused(DeviceState* dev, const FusedPlan& p, const bf16* X, const bf16* Wg, const bf16* Wu, const bf16* Wd,
                        float* scratch, bf16* Y, int64_t M, int64_t d_model, int64_t d_ff, cudaStream_t st, gmlp::GateAct act) {
    if (p.Mpad != 16) return GMLP_ERR_UNSUPPORTED;          // the kernel's epilogue is written for one 16-token accumulator per matrix
    if (!dev->skinny_fused_attr_set) {
        if (cudaFuncSetAttribute(gmlp::skinny_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gmlp::kFusedSmemBudget) != cudaSuccess)
            return GMLP_ERR_LAUNCH;
        dev->skinny_fused_attr_set = true;
    }
    CUtensorMap tmX, tmWg, tmWu, tmWd;
    if (!encode_2d(&tmX, X, (uint64_t)d_model, (uint64_t)M, 64, (uint32_t)p.Mpad)) return GMLP_ERR_LAUNCH;
    if (!GMLP_ENCODE_W(&tmWg, Wg, d_ff, d_model)) return GMLP_ERR_LAUNCH;
    if (!GMLP_ENCODE_W(&tmWu, Wu, d_ff, d_model)) return GMLP_ERR_LAUNCH;
    if (!GMLP_ENCODE_W(&tmWd, Wd, d_model, d_ff)) return GMLP_ERR_LAUNCH;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.slices * p.cluster));
    cfg.blockDim = dim3(gmlp::kSkinnyThreads);
    cfg.dynamicSmemBytes = p.smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)p.cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = pdl_allowed();
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    int& capacity = dev->fused_capacity[p.cluster];
    if (capacity == 0) {
        int n = 0;
        cfg.numAttrs = 1;                                   // the occupancy query takes the cluster shape only
        if (cudaOccupancyMaxActiveClusters(&n, gmlp::skinny_fused_kernel, &cfg) != cudaSuccess) {
            (void)cudaGetLastError();
            n = -1;
        }
        cfg.numAttrs = 2;
        capacity = n > 0 ? n : -1;
        if (getenv("GMLP_TUNE_VERBOSE"))
            fprintf(stderr, "gmlp: clusters of %d CTAs (fused small-M kernel, %u B shared memory) resident at once: %d\n", p.cluster, p.smem_bytes, n);
    }
    if (capacity < p.slices) return GMLP_ERR_UNSUPPORTED;
    int evict_first = 1;
    if (const char* e = getenv("GMLP_SKINNY_EVICT_FIRST")) evict_first = atoi(e);      // tuning override
    if (cudaLaunchKernelEx(&cfg, gmlp::skinny_fused_kernel, tmX, tmWg, tmWu, tmWd, scratch, (int)M, p.Mpad, (int)d_model,
                           p.stages, p.tmem_cols, evict_first, act, p.hbuf_off, p.staging_off, p.bars_off, t_w_out_in ? 1 : 0) != cudaSuccess)
        return GMLP_ERR_LAUNCH;
    GMLP_CHECK_LAUNCH();
    prof_mark("fused", st);
    // the sum over the slices: a programmatic dependent of the kernel above
    cudaLaunchConfig_t sum = {};
    const int64_t threads = M * (d_model / 4) * gmlp::kSumLanes;
    sum.gridDim = dim3((unsigned)((threads + 255) / 256));
    sum.blockDim = dim3(256);
    sum.stream = st;
    sum.attrs = attr + 1;
    sum.numAttrs = 1;
    if (cudaLaunchKernelEx(&sum, gmlp::sum_slices_kernel, (const float*)scratch, Y, (int)M, (int)d_model, p.slices, t_y_fp32 ? 1 : 0) != cudaSuccess)
        return GMLP_ERR_LAUNCH;
    GMLP_CHECK_LAUNCH();
    prof_mark("sum", st);
    return GMLP_OK;
}

// Whether the SKINNY schedule runs this layer as one fused kernel: where the plan applies and was measured to pay.
// Tuning override GMLP_SKINNY_FUSED: 0 never, 1 wherever the plan applies.
bool skinny_use_fused(const FusedPlan& f, int64_t M, int64_t d_model, int64_t d_ff) {
    if (f.cluster < 1) return false;
    if (const char* e = getenv("GMLP_SKINNY_FUSED")) return atoi(e) != 0;
    int tuned_fused = 0, tuned_ring = 0;
    skinny_forms(M, d_model, d_ff, &tuned_fused, &tuned_ring);
    if (tuned_fused != 0) return tuned_fused == 1;
    return f.preferred;
}

int run_skinny(DeviceState* dev, const Layout& L, uint8_t* ws, const bf16* A, const bf16* Wg, const bf16* Wu,
               const bf16* Wd, bf16* H, bf16* Y, int64_t M, int64_t d_model, int64_t d_ff, cudaStream_t st,
               gmlp::GateAct act) {
    float* scratch = reinterpret_cast<float*>(ws + L.partial_off);
    unsigned int* c1 = reinterpret_cast<unsigned int*>(ws + L.counters_off);
    unsigned int* c2 = c1 + L.s1.num_tiles;
    int rc = ensure_counters_zero(dev, c1, L.counters_bytes, st);
    if (rc != GMLP_OK) return rc;
    if (skinny_use_fused(L.sf, M, d_model, d_ff)) {
        rc = launch_skinny_fused(dev, L.sf, A, Wg, Wu, Wd, scratch, Y, M, d_model, d_ff, st, act);
        if (rc != GMLP_ERR_UNSUPPORTED) return rc;          // clusters that do not fit one wave: the two-kernel forms below
    }
    rc = launch_skinny<true>(dev, L.s1, A, Wg, Wu, scratch, c1, H, M, d_model, d_ff, st, act);
    if (rc != GMLP_OK) return rc;
    prof_mark("gate_up", st);
    rc = launch_skinny<false>(dev, L.s2, H, Wd, nullptr, scratch, c2, Y, M, d_ff, d_model, st);
    if (rc == GMLP_OK) prof_mark("down", st);
    return rc;
}

int read_device_status() {
    if (cudaDeviceSynchronize() != cudaSuccess) return GMLP_ERR_LAUNCH;
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, gmlp::g_device_status, sizeof(int)) != cudaSuccess) return GMLP_ERR_LAUNCH;
    if (v != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbol(gmlp::g_device_status, &zero, sizeof(int)) != cudaSuccess) return GMLP_ERR_LAUNCH;
    }
    return v;
}

int forward_impl(const gmlp_args* a) {
    if (a == nullptr) return GMLP_ERR_NULL;
    if (a->struct_bytes != sizeof(gmlp_args)) return GMLP_ERR_FLAGS;
    if (a->flags & ~kKnownFlags) return GMLP_ERR_FLAGS;
    gmlp::GateAct act;
    if (a->reserved != 0 || !gate_act_from(a->flags, a->act_beta, &act)) return GMLP_ERR_FLAGS;
    if (a->variant < GMLP_VARIANT_AUTO || a->variant > GMLP_VARIANT_TENSOR) return GMLP_ERR_FLAGS;
    int rc = check_shape(a->M, a->d_model, a->d_ff);
    if (rc != GMLP_OK) return rc;
    if (a->M == 0) return GMLP_OK;              // nothing to compute; pointers may be NULL
    if (!a->X || !a->Wg || !a->Wu || !a->Wd || !a->Y) return GMLP_ERR_NULL;
    if (!aligned16(a->X) || !aligned16(a->Wg) || !aligned16(a->Wu) || !aligned16(a->Wd) || !aligned16(a->Y) ||
        !aligned16(a->rms_gain))
        return GMLP_ERR_ALIGN;
    if (a->workspace != nullptr && (reinterpret_cast<uintptr_t>(a->workspace) & 255u)) return GMLP_ERR_ALIGN;
    const bool norm = (a->flags & GMLP_FLAG_RMSNORM) != 0;

    DeviceState* dev = current_device(&rc);
    if (dev == nullptr) return rc;

    const int variant = resolve_variant(a->M, a->d_model, a->d_ff, a->variant);
    if (variant == GMLP_VARIANT_SKINNY && !skinny_can_run(a->M, a->d_model, a->d_ff, dev->sm_count)) return GMLP_ERR_UNSUPPORTED;
    const bool w_out_in = (a->flags & GMLP_FLAG_WEIGHTS_OUT_IN) != 0;
    const bool y_fp32 = (a->flags & GMLP_FLAG_Y_FP32) != 0;
    if ((w_out_in || y_fp32) && (variant == GMLP_VARIANT_SIMT || variant == GMLP_VARIANT_STREAM)) return GMLP_ERR_UNSUPPORTED;
    const WeightLayoutScope layout_scope(w_out_in);
    const OutputTypeScope output_scope(y_fp32);
    const StreamOrderScope order_scope((a->flags & GMLP_FLAG_WEIGHTS_IN_STREAM_ORDER) != 0);
    const Layout L = make_layout(a->M, a->d_model, a->d_ff, a->flags, variant, dev->sm_count);

    uint8_t* ws = static_cast<uint8_t*>(a->workspace);
    if (ws == nullptr) {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (dev->workspace_bytes < L.total) {
            // grow the library-owned buffer; work queued on the old one must finish first
            if (dev->workspace != nullptr) {
                if (cudaDeviceSynchronize() != cudaSuccess || cudaFree(dev->workspace) != cudaSuccess) return GMLP_ERR_LAUNCH;
                dev->workspace = nullptr;
                dev->workspace_bytes = 0;
                forget_counters_locked(dev);
            }
            void* p = nullptr;
            if (cudaMalloc(&p, L.total) != cudaSuccess) {
                (void)cudaGetLastError();
                return GMLP_ERR_WORKSPACE;
            }
            dev->workspace = p;
            dev->workspace_bytes = L.total;
        }
        ws = static_cast<uint8_t*>(dev->workspace);
    } else if (a->workspace_bytes < L.total) {
        return GMLP_ERR_WORKSPACE;
    }
    claim_workspace(dev, ws, L.total, L.counters_bytes ? ws + L.counters_off : nullptr, L.counters_bytes);

    cudaStream_t st = static_cast<cudaStream_t>(a->stream);
    const bf16* X = static_cast<const bf16*>(a->X);
    const bf16* Wg = static_cast<const bf16*>(a->Wg);
    const bf16* Wu = static_cast<const bf16*>(a->Wu);
    const bf16* Wd = static_cast<const bf16*>(a->Wd);
    bf16* Y = static_cast<bf16*>(a->Y);
    bf16* H = reinterpret_cast<bf16*>(ws + L.h_off);

    prof_begin(st);
    const bf16* A = X;
    if (norm) {
        bf16* Xn = reinterpret_cast<bf16*>(ws + L.xn_off);
        rc = launch_rmsnorm(X, static_cast<const bf16*>(a->rms_gain), Xn, a->M, a->d_model, a->rms_eps, st);
        if (rc != GMLP_OK) return rc;
        prof_mark("rmsnorm", st);
        A = Xn;
    }

    switch (variant) {
        case GMLP_VARIANT_SIMT:
            rc = run_simt(A, Wg, Wu, Wd, H, Y, a->M, a->d_model, a->d_ff, st, act);
            break;
        case GMLP_VARIANT_STREAM:
            rc = run_stream(dev, L, ws, A, Wg, Wu, Wd, H, Y, a->M, a->d_model, a->d_ff, st, act);
            break;
        case GMLP_VARIANT_SKINNY:
            rc = run_skinny(dev, L, ws, A, Wg, Wu, Wd, H, Y, a->M, a->d_model, a->d_ff, st, act);
            break;
        case GMLP_VARIANT_PAIR:
            rc = launch_umma_pair<true>(dev, A, Wg, Wu, H, a->M, a->d_model, a->d_ff, st, act, pair_chunk_kb(true, a->d_model));
            if (rc == GMLP_OK) {
                prof_mark("gate_up", st);
                rc = launch_umma_pair<false>(dev, H, Wd, nullptr, Y, a->M, a->d_ff, a->d_model, st, kSilu, pair_chunk_kb(false, a->d_ff));
                if (rc == GMLP_OK) prof_mark("down", st);
            }
            break;
        case GMLP_VARIANT_TENSOR: {
            const TensorPlan plan = tensor_plan(a->M, a->d_model, a->d_ff, dev->sm_count);
            UmmaFormScope forms(plan.gu_nb, plan.down_form);
            rc = plan.gu_pair ? launch_umma_pair<true>(dev, A, Wg, Wu, H, a->M, a->d_model, a->d_ff, st, act, pair_chunk_kb(true, a->d_model))
                              : launch_umma<true>(dev, A, Wg, Wu, H, a->M, a->d_model, a->d_ff, st, act);
            if (rc == GMLP_OK) {
                prof_mark("gate_up", st);
                rc = plan.down_pair ? launch_umma_pair<false>(dev, H, Wd, nullptr, Y, a->M, a->d_ff, a->d_model, st, kSilu, pair_chunk_kb(false, a->d_ff))
                                    : launch_umma<false>(dev, H, Wd, nullptr, Y, a->M, a->d_ff, a->d_model, st);
                if (rc == GMLP_OK) prof_mark("down", st);
            }
            break;
        }
        default:
            rc = launch_umma<true>(dev, A, Wg, Wu, H, a->M, a->d_model, a->d_ff, st, act);
            if (rc == GMLP_OK) {
                prof_mark("gate_up", st);
                rc = launch_umma<false>(dev, H, Wd, nullptr, Y, a->M, a->d_ff, a->d_model, st);
                if (rc == GMLP_OK) prof_mark("down", st);
            }
            break;
    }
    if (rc != GMLP_OK) {
        forget_counters(dev);
        return rc;
    }

    if (a->flags & GMLP_FLAG_CHECKED) {
        if (cudaStreamSynchronize(st) != cudaSuccess) { forget_counters(dev); return GMLP_ERR_LAUNCH; }
        const int s = read_device_status();
        if (s != 0) forget_counters(dev);
        if (s < 0) return s;
        if (s != 0) return GMLP_ERR_TIMEOUT;
    }
    return GMLP_OK;
}

// ------------------------------------------------------------------ allocation-free entry point
// Scratch of gmlp_forward_static: part of the library image, one copy per GPU that loads it.  In host
// code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[GMLP_STATIC_SCRATCH_BYTES];

struct StaticScratch {
    bool ready = false;
    uint8_t* ptr = nullptr;          // device address of g_static_scratch on this device
};
StaticScratch g_static[kMaxDevices];

int forward_static_impl(const void* Xp, const void* Wgp, const void* Wup, const void* Wdp, void* Yp,
                        int64_t M, int64_t d_model, int64_t d_ff, cudaStream_t st) {
    int rc = check_shape(M, d_model, d_ff);
    if (rc != GMLP_OK) return rc;
    if (M > GMLP_STATIC_MAX_M) return GMLP_ERR_STATIC_LIMIT;
    if (M == 0) return GMLP_OK;
    if (!Xp || !Wgp || !Wup || !Wdp || !Yp) return GMLP_ERR_NULL;
    if (!aligned16(Xp) || !aligned16(Wgp) || !aligned16(Wup) || !aligned16(Wdp) || !aligned16(Yp)) return GMLP_ERR_ALIGN;

    DeviceState* dev = current_device(&rc);
    if (dev == nullptr) return rc;
    const Layout L = make_layout(M, d_model, d_ff, 0, GMLP_VARIANT_SKINNY, dev->sm_count);
    if (L.total > (uint64_t)GMLP_STATIC_SCRATCH_BYTES) return GMLP_ERR_STATIC_LIMIT;

    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess) return GMLP_ERR_ARCH;
    uint8_t* ws = nullptr;
    {
        // once per device, with that device current: the array's device address
        std::lock_guard<std::mutex> lock(g_mutex);
        StaticScratch& s = g_static[device];
        if (!s.ready) {
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) {
                (void)cudaGetLastError();
                return GMLP_ERR_LAUNCH;
            }
            s.ptr = static_cast<uint8_t*>(p);
            s.ready = true;
        }
        ws = s.ptr;
    }

    const bf16* X = static_cast<const bf16*>(Xp);
    bf16* H = reinterpret_cast<bf16*>(ws + L.h_off);
    float* scratch = reinterpret_cast<float*>(ws + L.partial_off);
    unsigned int* c1 = reinterpret_cast<unsigned int*>(ws + L.counters_off);
    unsigned int* c2 = c1 + L.s1.num_tiles;
    // the array keeps the previous call's contents: the arrival counters must start at zero
    if (cudaMemsetAsync(c1, 0, L.counters_bytes, st) != cudaSuccess) return GMLP_ERR_LAUNCH;
    rc = launch_skinny<true>(dev, L.s1, X, static_cast<const bf16*>(Wgp), static_cast<const bf16*>(Wup), scratch, c1, H,
                             M, d_model, d_ff, st);
    if (rc != GMLP_OK) return rc;
    return launch_skinny<false>(dev, L.s2, H, static_cast<const bf16*>(Wdp), nullptr, scratch, c2,
                                static_cast<bf16*>(Yp), M, d_ff, d_model, st);
}

// The gate/up half alone: same checks and schedules as forward_impl, output H to args->Y.
int gate_up_impl(const gmlp_args* a) {
    if (a == nullptr) return GMLP_ERR_NULL;
    if (a->struct_bytes != sizeof(gmlp_args)) return GMLP_ERR_FLAGS;
    if (a->flags & ~kKnownFlags) return GMLP_ERR_FLAGS;
    gmlp::GateAct act;
    if (a->reserved != 0 || !gate_act_from(a->flags, a->act_beta, &act)) return GMLP_ERR_FLAGS;
    if (a->variant < GMLP_VARIANT_AUTO || a->variant > GMLP_VARIANT_TENSOR) return GMLP_ERR_FLAGS;
    int rc = check_shape(a->M, a->d_model, a->d_ff);
    if (rc != GMLP_OK) return rc;
    if (a->M == 0) return GMLP_OK;
    if (!a->X || !a->Wg || !a->Wu || !a->Y) return GMLP_ERR_NULL;
    if (!aligned16(a->X) || !aligned16(a->Wg) || !aligned16(a->Wu) || !aligned16(a->Y) || !aligned16(a->rms_gain))
        return GMLP_ERR_ALIGN;
    if (a->workspace != nullptr && (reinterpret_cast<uintptr_t>(a->workspace) & 255u)) return GMLP_ERR_ALIGN;
    const int variant = resolve_variant(a->M, a->d_model, a->d_ff, a->variant);
    if (variant == GMLP_VARIANT_SIMT || variant == GMLP_VARIANT_STREAM) return GMLP_ERR_UNSUPPORTED;
    if (a->flags & GMLP_FLAG_Y_FP32) return GMLP_ERR_FLAGS;          // H is the bf16 operand of the next GEMM
    const WeightLayoutScope layout_scope((a->flags & GMLP_FLAG_WEIGHTS_OUT_IN) != 0);
    const StreamOrderScope order_scope((a->flags & GMLP_FLAG_WEIGHTS_IN_STREAM_ORDER) != 0);
    DeviceState* dev = current_device(&rc);
    if (dev == nullptr) return rc;
    if (variant == GMLP_VARIANT_SKINNY && !skinny_can_run(a->M, a->d_model, a->d_ff, dev->sm_count)) return GMLP_ERR_UNSUPPORTED;
    const Layout L = make_layout(a->M, a->d_model, a->d_ff, a->flags, variant, dev->sm_count);
    uint8_t* ws = static_cast<uint8_t*>(a->workspace);
    if (ws == nullptr) {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (dev->workspace_bytes < L.total) {
            if (dev->workspace != nullptr) {
                if (cudaDeviceSynchronize() != cudaSuccess || cudaFree(dev->workspace) != cudaSuccess) return GMLP_ERR_LAUNCH;
                dev->workspace = nullptr;
                dev->workspace_bytes = 0;
                forget_counters_locked(dev);
            }
            void* p = nullptr;
            if (cudaMalloc(&p, L.total) != cudaSuccess) {
                (void)cudaGetLastError();
                return GMLP_ERR_WORKSPACE;
            }
            dev->workspace = p;
            dev->workspace_bytes = L.total;
        }
        ws = static_cast<uint8_t*>(dev->workspace);
    } else if (a->workspace_bytes < L.total) {
        return GMLP_ERR_WORKSPACE;
    }
    claim_workspace(dev, ws, L.total, L.counters_bytes ? ws + L.counters_off : nullptr, L.counters_bytes);
    cudaStream_t st = static_cast<cudaStream_t>(a->stream);
    const bf16* A = static_cast<const bf16*>(a->X);
    const bf16* Wg = static_cast<const bf16*>(a->Wg);
    const bf16* Wu = static_cast<const bf16*>(a->Wu);
    bf16* Hout = static_cast<bf16*>(a->Y);
    prof_begin(st);
    if (a->flags & GMLP_FLAG_RMSNORM) {
        bf16* Xn = reinterpret_cast<bf16*>(ws + L.xn_off);
        rc = launch_rmsnorm(A, static_cast<const bf16*>(a->rms_gain), Xn, a->M, a->d_model, a->rms_eps, st);
        if (rc != GMLP_OK) return rc;
        prof_mark("rmsnorm", st);
        A = Xn;
    }
    if (variant == GMLP_VARIANT_SKINNY) {
        float* scratch = reinterpret_cast<float*>(ws + L.partial_off);
        unsigned int* c1 = reinterpret_cast<unsigned int*>(ws + L.counters_off);
        rc = ensure_counters_zero(dev, c1, L.counters_bytes, st);
        if (rc == GMLP_OK) rc = launch_skinny<true>(dev, L.s1, A, Wg, Wu, scratch, c1, Hout, a->M, a->d_model, a->d_ff, st, act);
    } else if (variant == GMLP_VARIANT_PAIR ||
               (variant == GMLP_VARIANT_TENSOR && tensor_plan(a->M, a->d_model, a->d_ff, dev->sm_count).gu_pair)) {
        rc = launch_umma_pair<true>(dev, A, Wg, Wu, Hout, a->M, a->d_model, a->d_ff, st, act, pair_chunk_kb(true, a->d_model));
    } else {
        // (a tuned shape's tile form applies to the gate/up half alone as well)
        UmmaFormScope forms(variant == GMLP_VARIANT_TENSOR ? tensor_plan(a->M, a->d_model, a->d_ff, dev->sm_count).gu_nb : 0, 0);
        rc = launch_umma<true>(dev, A, Wg, Wu, Hout, a->M, a->d_model, a->d_ff, st, act);
    }
    if (rc != GMLP_OK) {
        forget_counters(dev);
        return rc;
    }
    prof_mark("gate_up", st);
    if (a->flags & GMLP_FLAG_CHECKED) {
        if (cudaStreamSynchronize(st) != cudaSuccess) { forget_counters(dev); return GMLP_ERR_LAUNCH; }
        const int s = read_device_status();
        if (s != 0) forget_counters(dev);
        if (s < 0) return s;
        if (s != 0) return GMLP_ERR_TIMEOUT;
    }
    return GMLP_OK;
}

// RMSNorm+MatMul.  Rewritten schedule: one GEMM kernel with row-square reducer warps and an epilogue row scale.
int rmsnorm_matmul_impl(const gmlp_rmsmm_args* a) {
    if (a == nullptr) return GMLP_ERR_NULL;
    if (a->struct_bytes != sizeof(gmlp_rmsmm_args)) return GMLP_ERR_FLAGS;
    if ((a->flags & ~(uint32_t)(GMLP_FLAG_CHECKED | GMLP_RMSMM_UNFUSED)) || a->reserved != 0) return GMLP_ERR_FLAGS;
    int rc = check_shape(a->M, a->K, a->N);
    if (rc != GMLP_OK) return rc;
    if (a->M == 0) return GMLP_OK;
    if (!a->X || !a->W || !a->Z) return GMLP_ERR_NULL;
    if (!aligned16(a->X) || !aligned16(a->W) || !aligned16(a->Z) || !aligned16(a->rms_gain)) return GMLP_ERR_ALIGN;
    if (a->workspace != nullptr && (reinterpret_cast<uintptr_t>(a->workspace) & 255u)) return GMLP_ERR_ALIGN;
    DeviceState* dev = current_device(&rc);
    if (dev == nullptr) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(a->stream);
    const bf16* X = static_cast<const bf16*>(a->X);
    const bf16* W = static_cast<const bf16*>(a->W);
    bf16* Z = static_cast<bf16*>(a->Z);
    const bool unfused = (a->flags & GMLP_RMSMM_UNFUSED) != 0 || a->rms_gain != nullptr;
    prof_begin(st);
    if (unfused) {
        const uint64_t need = align256((uint64_t)a->M * a->K * 2);
        if (a->workspace == nullptr || a->workspace_bytes < need) return GMLP_ERR_WORKSPACE;
        claim_workspace(dev, static_cast<const uint8_t*>(a->workspace), need, nullptr, 0);
        bf16* Xn = static_cast<bf16*>(a->workspace);
        rc = launch_rmsnorm(X, static_cast<const bf16*>(a->rms_gain), Xn, a->M, a->K, a->rms_eps, st);
        if (rc != GMLP_OK) return rc;
        prof_mark("rmsnorm", st);
        rc = a->M >= 1024 ? launch_umma_pair<false>(dev, Xn, W, nullptr, Z, a->M, a->K, a->N, st)
                          : launch_umma<false>(dev, Xn, W, nullptr, Z, a->M, a->K, a->N, st);
        if (rc != GMLP_OK) return rc;
        prof_mark("matmul", st);
    } else {
        // rewritten: r = rsqrt(mean(x^2) + eps) per row (tiny kernel), then the GEMM on the raw X with the row scale
        // in its epilogue; programmatic dependent launch lets the GEMM's main loop overlap the RMS branch
        const uint64_t need = align256((uint64_t)a->M * 4);
        if (a->workspace == nullptr || a->workspace_bytes < need) return GMLP_ERR_WORKSPACE;
        claim_workspace(dev, static_cast<const uint8_t*>(a->workspace), need, nullptr, 0);
        float* r = static_cast<float*>(a->workspace);
        gmlp::row_rsqrt_kernel<<<(unsigned)a->M, gmlp::kRmsThreads, 0, st>>>(X, r, a->M, (int)a->K, a->rms_eps);
        GMLP_CHECK_LAUNCH();
        prof_mark("row_rsqrt", st);
        const bool pair = a->M >= 1024;
        CUtensorMap tmA, tmB;
        if (!encode_2d(&tmA, X, (uint64_t)a->K, (uint64_t)a->M, gmlp::kUmmaBK, 128) ||
            !encode_2d(&tmB, W, (uint64_t)a->N, (uint64_t)a->K, 64, gmlp::kUmmaBK))
            return GMLP_ERR_LAUNCH;
        if (!dev->rowscale_attr_set) {
            if (cudaFuncSetAttribute(gmlp::umma_gemm_kernel<false, 4, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)gmlp::kUmmaSmemBytes) != cudaSuccess ||
                cudaFuncSetAttribute(gmlp::umma_pair_gemm_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)gmlp::kPairSmemBytes) != cudaSuccess)
                return GMLP_ERR_LAUNCH;
            dev->rowscale_attr_set = true;
        }
        const int sms = dev->sm_count > 0 ? dev->sm_count : 148;
        const int num_m = (int)((a->M + (pair ? 255 : 127)) / (pair ? 256 : 128));
        const int num_tiles = num_m * (int)((a->N + 255) / 256);
        const int ctas = pair ? 2 * (num_tiles < sms / 2 ? num_tiles : sms / 2) : (num_tiles < sms ? num_tiles : sms);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)ctas);
        cfg.blockDim = dim3(gmlp::kUmmaThreads);
        cfg.dynamicSmemBytes = pair ? gmlp::kPairSmemBytes : gmlp::kUmmaSmemBytes;
        cfg.stream = st;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = pdl_allowed();
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = 2;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = pair ? 2 : 1;
        const int Mi = (int)a->M, Ki = (int)a->K, Ni = (int)a->N;
        const float* rc_ptr = r;
        cudaError_t err = pair
            ? cudaLaunchKernelEx(&cfg, gmlp::umma_pair_gemm_kernel<false, true>, tmA, tmB, tmB, Z, Mi, Ki, Ni, num_m, num_tiles, rc_ptr, kSilu, (const bf16*)nullptr, (float*)nullptr, kNoMulti, 0, 0, 0, 0)
            : cudaLaunchKernelEx(&cfg, gmlp::umma_gemm_kernel<false, 4, true>, tmA, tmB, tmB, Z, Mi, Ki, Ni, num_m, num_tiles, rc_ptr, 128, kSilu, (const bf16*)nullptr, (float*)nullptr, kNoMulti, 0, 0);
        if (err != cudaSuccess) return GMLP_ERR_LAUNCH;
        GMLP_CHECK_LAUNCH();
        prof_mark("matmul_rowscale", st);
    }
    if (a->flags & GMLP_FLAG_CHECKED) {
        if (cudaStreamSynchronize(st) != cudaSuccess) return GMLP_ERR_LAUNCH;
        const int s = read_device_status();
        if (s < 0) return s;
        if (s != 0) return GMLP_ERR_TIMEOUT;
    }
    return GMLP_OK;
}

// "Matmul+Add+RMSNorm" (Section 6.1): S = X W + R, Z = RMSNorm(S).
int matmul_add_rmsnorm_impl(const gmlp_mmaddnorm_args* a) {
    if (a == nullptr) return GMLP_ERR_NULL;
    if (a->struct_bytes != sizeof(gmlp_mmaddnorm_args)) return GMLP_ERR_FLAGS;
    if ((a->flags & ~(uint32_t)(GMLP_FLAG_CHECKED | GMLP_MMADDNORM_UNFUSED)) || a->reserved != 0) return GMLP_ERR_FLAGS;
    int rc = check_shape(a->M, a->K, a->N);
    if (rc != GMLP_OK) return rc;
    if (a->M == 0) return GMLP_OK;
    if (!a->X || !a->W || !a->R || !a->S || !a->Z) return GMLP_ERR_NULL;
    if (!aligned16(a->X) || !aligned16(a->W) || !aligned16(a->R) || !aligned16(a->S) || !aligned16(a->Z) ||
        !aligned16(a->rms_gain))
        return GMLP_ERR_ALIGN;
    if (a->workspace != nullptr && (reinterpret_cast<uintptr_t>(a->workspace) & 255u)) return GMLP_ERR_ALIGN;
    DeviceState* dev = current_device(&rc);
    if (dev == nullptr) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(a->stream);
    const bf16* X = static_cast<const bf16*>(a->X);
    const bf16* W = static_cast<const bf16*>(a->W);
    const bf16* R = static_cast<const bf16*>(a->R);
    const bf16* gain = static_cast<const bf16*>(a->rms_gain);
    bf16* S = static_cast<bf16*>(a->S);
    bf16* Z = static_cast<bf16*>(a->Z);
    const bool pair = a->M >= 1024;
    prof_begin(st);
    if (a->flags & GMLP_MMADDNORM_UNFUSED) {
        // three separate operators: T = X W (bf16), S = T + R, Z = RMSNorm(S)
        const uint64_t need = align256((uint64_t)a->M * a->N * 2);
        if (a->workspace == nullptr || a->workspace_bytes < need) return GMLP_ERR_WORKSPACE;
        claim_workspace(dev, static_cast<const uint8_t*>(a->workspace), need, nullptr, 0);
        bf16* T = static_cast<bf16*>(a->workspace);
        rc = pair ? launch_umma_pair<false>(dev, X, W, nullptr, T, a->M, a->K, a->N, st)
                  : launch_umma<false>(dev, X, W, nullptr, T, a->M, a->K, a->N, st);
        if (rc != GMLP_OK) return rc;
        prof_mark("matmul", st);
        const size_t nvec = (size_t)a->M * (size_t)a->N / 8;
        gmlp::add_bf16_kernel<<<(unsigned)((nvec + 255) / 256), 256, 0, st>>>(T, R, S, nvec);
        GMLP_CHECK_LAUNCH();
        prof_mark("add", st);
        rc = launch_rmsnorm(S, gain, Z, a->M, a->N, a->rms_eps, st);
        if (rc != GMLP_OK) return rc;
        prof_mark("rmsnorm", st);
    } else {
        // fused: the GEMM's epilogue adds R, stores S and leaves per-tile sums of squares; one light pass normalises
        const int n_tiles = (int)((a->N + 255) / 256);
        const uint64_t need = align256((uint64_t)n_tiles * a->M * 4);
        if (a->workspace == nullptr || a->workspace_bytes < need) return GMLP_ERR_WORKSPACE;
        claim_workspace(dev, static_cast<const uint8_t*>(a->workspace), need, nullptr, 0);
        float* sumsq = static_cast<float*>(a->workspace);
        CUtensorMap tmA, tmB;
        if (!encode_2d(&tmA, X, (uint64_t)a->K, (uint64_t)a->M, gmlp::kUmmaBK, 128) ||
            !encode_2d(&tmB, W, (uint64_t)a->N, (uint64_t)a->K, 64, gmlp::kUmmaBK))
            return GMLP_ERR_LAUNCH;
        if (!dev->addss_attr_set) {
            if (cudaFuncSetAttribute(gmlp::umma_gemm_kernel<false, 4, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)gmlp::kUmmaSmemBytes) != cudaSuccess ||
                cudaFuncSetAttribute(gmlp::umma_pair_gemm_kernel<false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)gmlp::kPairSmemBytes) != cudaSuccess)
                return GMLP_ERR_LAUNCH;
            dev->addss_attr_set = true;
        }
        const int sms = dev->sm_count > 0 ? dev->sm_count : 148;
        const int num_m = (int)((a->M + (pair ? 255 : 127)) / (pair ? 256 : 128));
        const int num_tiles = num_m * n_tiles;
        const int ctas = pair ? 2 * (num_tiles < sms / 2 ? num_tiles : sms / 2) : (num_tiles < sms ? num_tiles : sms);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)ctas);
        cfg.blockDim = dim3(gmlp::kUmmaThreads);
        cfg.dynamicSmemBytes = pair ? gmlp::kPairSmemBytes : gmlp::kUmmaSmemBytes;
        cfg.stream = st;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = pdl_allowed();
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = 2;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = pair ? 2 : 1;
        const int Mi = (int)a->M, Ki = (int)a->K, Ni = (int)a->N;
        cudaError_t err = pair
            ? cudaLaunchKernelEx(&cfg, gmlp::umma_pair_gemm_kernel<false, false, true>, tmA, tmB, tmB, S, Mi, Ki, Ni, num_m,
                                 num_tiles, (const float*)nullptr, kSilu, R, sumsq, kNoMulti, 0, 0, 0, 0)
            : cudaLaunchKernelEx(&cfg, gmlp::umma_gemm_kernel<false, 4, false, true>, tmA, tmB, tmB, S, Mi, Ki, Ni, num_m,
                                 num_tiles, (const float*)nullptr, 128, kSilu, R, sumsq, kNoMulti, 0, 0);
        if (err != cudaSuccess) return GMLP_ERR_LAUNCH;
        GMLP_CHECK_LAUNCH();
        prof_mark("matmul_add", st);
        cudaLaunchConfig_t c2 = {};
        c2.gridDim = dim3((unsigned)a->M);
        c2.blockDim = dim3(gmlp::kRmsThreads);
        c2.stream = st;
        c2.attrs = attr;                                   // programmatic stream serialization only
        c2.numAttrs = 1;
        const int64_t M64 = a->M;
        const float eps = a->rms_eps;
        const bf16* Sc = S;
        const float* ssc = sumsq;
        if (cudaLaunchKernelEx(&c2, gmlp::rmsnorm_apply_kernel, Sc, ssc, n_tiles, gain, Z, M64, Ni, eps) != cudaSuccess)
            return GMLP_ERR_LAUNCH;
        GMLP_CHECK_LAUNCH();
        prof_mark("rmsnorm_apply", st);
    }
    if (a->flags & GMLP_FLAG_CHECKED) {
        if (cudaStreamSynchronize(st) != cudaSuccess) return GMLP_ERR_LAUNCH;
        const int s = read_device_status();
        if (s < 0) return s;
        if (s != 0) return GMLP_ERR_TIMEOUT;
    }
    return GMLP_OK;
}

// QKV projection (Section 6.1): Q = X Wq, K = X Wk, V = X Wv in one launch of the multi-matrix GEMM.
int qkv_proj_impl(const gmlp_qkv_args* a) {
    if (a == nullptr) return GMLP_ERR_NULL;
    if (a->struct_bytes != sizeof(gmlp_qkv_args)) return GMLP_ERR_FLAGS;
    if ((a->flags & ~(uint32_t)(GMLP_FLAG_CHECKED | GMLP_QKV_SEPARATE)) || a->reserved != 0) return GMLP_ERR_FLAGS;
    int rc = check_shape(a->M, a->K, a->Nq);
    if (rc == GMLP_OK) rc = check_shape(a->M, a->K, a->Nkv);
    if (rc != GMLP_OK) return rc;
    if (a->M == 0) return GMLP_OK;
    if (!a->X || !a->Wq || !a->Wk || !a->Wv || !a->Q || !a->Kout || !a->V) return GMLP_ERR_NULL;
    if (!aligned16(a->X) || !aligned16(a->Wq) || !aligned16(a->Wk) || !aligned16(a->Wv) || !aligned16(a->Q) ||
        !aligned16(a->Kout) || !aligned16(a->V))
        return GMLP_ERR_ALIGN;
    DeviceState* dev = current_device(&rc);
    if (dev == nullptr) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(a->stream);
    const bf16* X = static_cast<const bf16*>(a->X);
    const bf16* Wq = static_cast<const bf16*>(a->Wq);
    const bf16* Wk = static_cast<const bf16*>(a->Wk);
    const bf16* Wv = static_cast<const bf16*>(a->Wv);
    bf16* Q = static_cast<bf16*>(a->Q);
    bf16* Ko = static_cast<bf16*>(a->Kout);
    bf16* V = static_cast<bf16*>(a->V);
    const int64_t mt = (a->M + 127) / 128;
    const bool pair = mt >= 24 || (mt >= 2 && mt % 2 == 0);          // as for the gate/up GEMM
    prof_begin(st);
    if (a->flags & GMLP_QKV_SEPARATE) {
        // three plain GEMMs, one after the other
        const bf16* Ws[3] = {Wq, Wk, Wv};
        bf16* Os[3] = {Q, Ko, V};
        const int64_t Ns[3] = {a->Nq, a->Nkv, a->Nkv};
        const char* names[3] = {"q", "k", "v"};
        for (int i = 0; i < 3; ++i) {
            rc = pair ? launch_umma_pair<false>(dev, X, Ws[i], nullptr, Os[i], a->M, a->K, Ns[i], st)
                      : launch_umma<false>(dev, X, Ws[i], nullptr, Os[i], a->M, a->K, Ns[i], st);
            if (rc != GMLP_OK) return rc;
            prof_mark(names[i], st);
        }
    } else {
        CUtensorMap tmA, tmB0, tmB1;
        gmlp::MultiB multi = {};
        if (!encode_2d(&tmA, X, (uint64_t)a->K, (uint64_t)a->M, gmlp::kUmmaBK, 128) ||
            !encode_2d(&tmB0, Wq, (uint64_t)a->Nq, (uint64_t)a->K, 64, gmlp::kUmmaBK) ||
            !encode_2d(&tmB1, Wk, (uint64_t)a->Nkv, (uint64_t)a->K, 64, gmlp::kUmmaBK) ||
            !encode_2d(&multi.tmB2, Wv, (uint64_t)a->Nkv, (uint64_t)a->K, 64, gmlp::kUmmaBK))
            return GMLP_ERR_LAUNCH;
        multi.C1 = Ko;
        multi.C2 = V;
        multi.N1 = multi.N2 = (int)a->Nkv;
        multi.tiles0 = (int)((a->Nq + 255) / 256);
        multi.tiles1 = (int)((a->Nkv + 255) / 256);
        if (!dev->multi_attr_set) {
            if (cudaFuncSetAttribute(gmlp::umma_gemm_kernel<false, 4, false, false, true>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gmlp::kUmmaSmemBytes) != cudaSuccess ||
                cudaFuncSetAttribute(gmlp::umma_pair_gemm_kernel<false, false, false, true>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gmlp::kPairSmemBytes) != cudaSuccess)
                return GMLP_ERR_LAUNCH;
            dev->multi_attr_set = true;
        }
        const int sms = dev->sm_count > 0 ? dev->sm_count : 148;
        const int num_m = (int)((a->M + (pair ? 255 : 127)) / (pair ? 256 : 128));
        const int num_tiles = num_m * (multi.tiles0 + 2 * multi.tiles1);
        const int ctas = pair ? 2 * (num_tiles < sms / 2 ? num_tiles : sms / 2) : (num_tiles < sms ? num_tiles : sms);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)ctas);
        cfg.blockDim = dim3(gmlp::kUmmaThreads);
        cfg.dynamicSmemBytes = pair ? gmlp::kPairSmemBytes : gmlp::kUmmaSmemBytes;
        cfg.stream = st;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = pdl_allowed();
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = 2;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = pair ? 2 : 1;
        const int Mi = (int)a->M, Ki = (int)a->K, Ni = (int)a->Nq;
        cudaError_t err = pair
            ? cudaLaunchKernelEx(&cfg, gmlp::umma_pair_gemm_kernel<false, false, false, true>, tmA, tmB0, tmB1, Q, Mi, Ki, Ni,
                                 num_m, num_tiles, (const float*)nullptr, kSilu, (const bf16*)nullptr, (float*)nullptr, multi, 0, 0, 0, 0)
            : cudaLaunchKernelEx(&cfg, gmlp::umma_gemm_kernel<false, 4, false, false, true>, tmA, tmB0, tmB1, Q, Mi, Ki, Ni,
                                 num_m, num_tiles, (const float*)nullptr, 128, kSilu, (const bf16*)nullptr, (float*)nullptr,
                                 multi, 0, 0);
        if (err != cudaSuccess) return GMLP_ERR_LAUNCH;
        GMLP_CHECK_LAUNCH();
        prof_mark("qkv", st);
    }
    if (a->flags & GMLP_FLAG_CHECKED) {
        if (cudaStreamSynchronize(st) != cudaSuccess) return GMLP_ERR_LAUNCH;
        const int s = read_device_status();
        if (s < 0) return s;
        if (s != 0) return GMLP_ERR_TIMEOUT;
    }
    return GMLP_OK;
}

// Group Query Attention forward (Section 6.1), no mask, head dimension 128.
int gqa_attention_impl(const gmlp_gqa_args* a) {
    if (a == nullptr) return GMLP_ERR_NULL;
    if (a->struct_bytes != sizeof(gmlp_gqa_args)) return GMLP_ERR_FLAGS;
    if ((a->flags & ~(uint32_t)(GMLP_FLAG_CHECKED | GMLP_GQA_CAUSAL)) || a->reserved != 0) return GMLP_ERR_FLAGS;
    if ((a->flags & GMLP_GQA_CAUSAL) && a->S < a->M) return GMLP_ERR_SHAPE;
    if (a->M < 0 || a->S <= 0 || a->n_q_heads <= 0 || a->n_kv_heads <= 0 || a->n_q_heads % a->n_kv_heads != 0 ||
        a->M > (1 << 30) || a->S > (1 << 30) || a->n_q_heads > 65535)
        return GMLP_ERR_SHAPE;
    if (a->head_dim != gmlp::kGqaD) return GMLP_ERR_UNSUPPORTED;
    if (a->M == 0) return GMLP_OK;
    if (!a->Q || !a->K || !a->V || !a->O) return GMLP_ERR_NULL;
    if (!aligned16(a->Q) || !aligned16(a->K) || !aligned16(a->V) || !aligned16(a->O)) return GMLP_ERR_ALIGN;
    int rc = GMLP_OK;
    DeviceState* dev = current_device(&rc);
    if (dev == nullptr) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(a->stream);
    const uint64_t qw = (uint64_t)a->n_q_heads * gmlp::kGqaD, kvw = (uint64_t)a->n_kv_heads * gmlp::kGqaD;
    CUtensorMap tmQ, tmK, tmV;
    if (!encode_2d(&tmQ, a->Q, qw, (uint64_t)a->M, 64, 128) || !encode_2d(&tmK, a->K, kvw, (uint64_t)a->S, 64, 128) ||
        !encode_2d(&tmV, a->V, kvw, (uint64_t)a->S, 64, 64))
        return GMLP_ERR_LAUNCH;
    if (!dev->gqa_attr_set) {
        if (cudaFuncSetAttribute(gmlp::gqa_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)gmlp::kGqaSmemBytes) != cudaSuccess)
            return GMLP_ERR_LAUNCH;
        dev->gqa_attr_set = true;
    }
    prof_begin(st);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((a->M + gmlp::kGqaBM - 1) / gmlp::kGqaBM), (unsigned)a->n_q_heads);
    cfg.blockDim = dim3(gmlp::kGqaThreads);
    cfg.dynamicSmemBytes = gmlp::kGqaSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl_allowed();
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int Mi = (int)a->M, Si = (int)a->S, Hq = (int)a->n_q_heads, group = (int)(a->n_q_heads / a->n_kv_heads);
    const float scale_log2 = 1.4426950408889634f / sqrtf((float)gmlp::kGqaD);      // log2(e) / sqrt(D)
    bf16* O = static_cast<bf16*>(a->O);
    const int causal_off = (a->flags & GMLP_GQA_CAUSAL) ? (int)(a->S - a->M) : -1;
    if (cudaLaunchKernelEx(&cfg, gmlp::gqa_attention_kernel, tmQ, tmK, tmV, O, Mi, Si, Hq, group, scale_log2, causal_off) !=
        cudaSuccess)
        return GMLP_ERR_LAUNCH;
    GMLP_CHECK_LAUNCH();
    prof_mark("gqa", st);
    if (a->flags & GMLP_FLAG_CHECKED) {
        if (cudaStreamSynchronize(st) != cudaSuccess) return GMLP_ERR_LAUNCH;
        const int s = read_device_status();
        if (s < 0) return s;
        if (s != 0) return GMLP_ERR_TIMEOUT;
    }
    return GMLP_OK;
}

// Empirical schedule selection for one shape: time every tensor-core schedule that can run it, keep the fastest.
int autotune_impl(const gmlp_args* a, int iters, int32_t* best_variant, float* best_us) {
    if (a == nullptr) return GMLP_ERR_NULL;
    if (a->struct_bytes != sizeof(gmlp_args)) return GMLP_ERR_FLAGS;
    if (iters < 1 || iters > 10000) return GMLP_ERR_FLAGS;
    int rc = check_shape(a->M, a->d_model, a->d_ff);
    if (rc != GMLP_OK) return rc;
    if (a->M == 0) return GMLP_ERR_SHAPE;
    DeviceState* dev = current_device(&rc);
    if (dev == nullptr) return rc;
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) return GMLP_ERR_LAUNCH;
    cudaStream_t st = static_cast<cudaStream_t>(a->stream);
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) {
        if (e0) (void)cudaEventDestroy(e0);
        return GMLP_ERR_LAUNCH;
    }
    // candidates: SKINNY, and TENSOR with each of the four (gate/up kernel, down kernel) combinations
    struct Cand { int variant, gu, down; };
    const Cand candidates[5] = {{GMLP_VARIANT_SKINNY, -1, -1}, {GMLP_VARIANT_TENSOR, 0, 0}, {GMLP_VARIANT_TENSOR, 0, 1},
                                {GMLP_VARIANT_TENSOR, 1, 0}, {GMLP_VARIANT_TENSOR, 1, 1}};
    // The candidates are timed in interleaved rounds (each round runs every candidate for a share of the
    // iterations; the first round is a warm-up and is not counted), so that clock and power drift over the
    // tuning run falls on all of them alike instead of favouring whoever runs first.
    constexpr int kRounds = 4;
    const int per_round = (iters + kRounds - 1) / kRounds;
    bool usable[5];
    float total_ms[5] = {0, 0, 0, 0, 0};
    int n_usable = 0;
    for (int c = 0; c < 5; ++c) {
        const int v = candidates[c].variant;
        usable[c] = !(v == GMLP_VARIANT_SKINNY && !skinny_can_run(a->M, a->d_model, a->d_ff, dev->sm_count)) &&
                    !(a->workspace != nullptr &&      // the caller's workspace must hold the schedule
                      make_layout(a->M, a->d_model, a->d_ff, a->flags, v, dev->sm_count).total > a->workspace_bytes);
        n_usable += usable[c] ? 1 : 0;
    }
    rc = GMLP_OK;
    for (int round = 0; round <= kRounds && rc == GMLP_OK && n_usable > 0; ++round) {
        for (int c = 0; c < 5 && rc == GMLP_OK; ++c) {
            if (!usable[c]) continue;
            gmlp_args t = *a;
            t.variant = candidates[c].variant;
            t.flags &= ~(uint32_t)GMLP_FLAG_CHECKED;
            t_force_gu = candidates[c].gu;
            t_force_down = candidates[c].down;
            rc = forward_impl(&t);                          // not timed: the switch of schedule itself
            float ms = 0.0f;
            if (rc == GMLP_OK && cudaEventRecord(e0, st) != cudaSuccess) rc = GMLP_ERR_LAUNCH;
            for (int i = 0; i < per_round && rc == GMLP_OK; ++i) rc = forward_impl(&t);
            t_force_gu = t_force_down = -1;
            if (rc != GMLP_OK) break;
            if (cudaEventRecord(e1, st) != cudaSuccess || cudaEventSynchronize(e1) != cudaSuccess ||
                cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) { rc = GMLP_ERR_LAUNCH; break; }
            if (round > 0) total_ms[c] += ms;
        }
    }
    if (rc == GMLP_OK) {
        const int s = read_device_status();
        if (s < 0) rc = s;
        else if (s != 0) rc = GMLP_ERR_TIMEOUT;
    }
    int best = -1;
    for (int c = 0; c < 5; ++c)
        if (usable[c] && (best < 0 || total_ms[c] < total_ms[best])) best = c;
    const float best_ms = best >= 0 ? total_ms[best] : 0.0f;
    const int timed_calls = kRounds * per_round;
    if (getenv("GMLP_TUNE_VERBOSE")) {                       // the measurements behind the choice, on stderr
        fprintf(stderr, "gmlp_autotune M=%lld d_model=%lld d_ff=%lld:", (long long)a->M, (long long)a->d_model, (long long)a->d_ff);
        for (int c = 0; c < 5; ++c)
            if (usable[c])
                fprintf(stderr, " [variant %d gate_up_pair %d down_pair %d: %.1f us]%s", candidates[c].variant, candidates[c].gu,
                        candidates[c].down, total_ms[c] * 1000.0f / (float)timed_calls, c == best ? "*" : "");
        fprintf(stderr, "\n");
    }
    if (rc != GMLP_OK || best < 0) {
        (void)cudaEventDestroy(e0);
        (void)cudaEventDestroy(e1);
    }
    if (rc != GMLP_OK) return rc;
    if (best < 0) return GMLP_ERR_WORKSPACE;                        // no candidate fitted the workspace
    const Cand w = candidates[best];
    // Second stage, for the single-CTA kernels of a TENSOR winner: their tile form (gate/up: 64- or 128-column
    // tiles; down: K split over a cluster of 2 to 4 CTAs, or 128- or 256-column tiles without a split) is otherwise
    // picked by rule.  One GEMM at a time, the other left as chosen so far; the same interleaved rounds.
    int best_gu_nb = 0, best_down_form = 0;
    if (w.variant == GMLP_VARIANT_TENSOR && (w.gu == 0 || w.down == 0)) {
        const int64_t mt = (a->M + 127) / 128, nkb = (a->d_ff + 63) / 64;
        for (int which = 0; which < 2 && rc == GMLP_OK; ++which) {       // 0: gate/up forms, 1: down forms
            if ((which == 0 ? w.gu : w.down) != 0) continue;
            int forms[6], n_forms = 0;
            if (which == 0) { forms[0] = 0; forms[1] = 2; forms[2] = 4; n_forms = 3; }
            else
                for (int f : kDownForms) {
                    const bool split = f >= 2 && f <= 4;
                    if (split && (nkb / f < 8 || mt * ((a->d_model + 127) / 128) * f > 2 * (int64_t)dev->sm_count)) continue;
                    forms[n_forms++] = f;
                }
            float form_ms[6] = {0, 0, 0, 0, 0, 0};
            for (int round = 0; round <= kRounds && rc == GMLP_OK; ++round)
                for (int c = 0; c < n_forms && rc == GMLP_OK; ++c) {
                    gmlp_args t = *a;
                    t.variant = GMLP_VARIANT_TENSOR;
                    t.flags &= ~(uint32_t)GMLP_FLAG_CHECKED;
                    t_force_gu = w.gu;
                    t_force_down = w.down;
                    t_force_gu_nb = which == 0 ? forms[c] : best_gu_nb;
                    t_force_down_form = which == 1 ? forms[c] : 0;
                    rc = forward_impl(&t);
                    float ms = 0.0f;
                    if (rc == GMLP_OK && cudaEventRecord(e0, st) != cudaSuccess) rc = GMLP_ERR_LAUNCH;
                    for (int i = 0; i < per_round && rc == GMLP_OK; ++i) rc = forward_impl(&t);
                    t_force_gu = t_force_down = -1;
                    t_force_gu_nb = t_force_down_form = 0;
                    if (rc != GMLP_OK) break;
                    if (cudaEventRecord(e1, st) != cudaSuccess || cudaEventSynchronize(e1) != cudaSuccess ||
                        cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) { rc = GMLP_ERR_LAUNCH; break; }
                    if (round > 0) form_ms[c] += ms;
                }
            if (rc != GMLP_OK) break;
            int bf = 0;
            for (int c = 1; c < n_forms; ++c)
                if (form_ms[c] < form_ms[bf]) bf = c;
            // the rule's own choice (form 0) is kept unless another form is measurably (1 %) faster
            if (form_ms[bf] < 0.99f * form_ms[0]) (which == 0 ? best_gu_nb : best_down_form) = forms[bf];
            if (getenv("GMLP_TUNE_VERBOSE")) {
                fprintf(stderr, "gmlp_autotune   %s forms:", which == 0 ? "gate/up" : "down");
                for (int c = 0; c < n_forms; ++c)
                    fprintf(stderr, " [%d: %.1f us]%s", forms[c], form_ms[c] * 1000.0f / (float)timed_calls,
                            forms[c] == (which == 0 ? best_gu_nb : best_down_form) ? "*" : "");
                fprintf(stderr, "\n");
            }
        }
        if (rc == GMLP_OK) {
            const int s2 = read_device_status();
            if (s2 < 0) rc = s2;
            else if (s2 != 0) rc = GMLP_ERR_TIMEOUT;
        }
        if (rc != GMLP_OK) { (void)0; }
    }
    // The same for a SKINNY winner: the one-kernel form against the two-kernel forms where its plan applies, and half-size
    // against full-size weight rings (up to 32 tokens), each against what the built-in rule takes.
    if (w.variant == GMLP_VARIANT_SKINNY && rc == GMLP_OK) {
        struct Form { int fused, ring; };
        Form forms[4] = {{0, 0}, {0, 0}, {0, 0}, {0, 0}};
        int n_forms = 1;
        const FusedPlan fp = make_fused_plan(a->M, a->d_model, a->d_ff, dev->sm_count);
        if (fp.cluster >= 1) forms[n_forms++] = {fp.preferred ? 2 : 1, 0};
        if (a->M <= 32) { forms[n_forms++] = {0, 1}; forms[n_forms++] = {0, 2}; }
        float form_ms[4] = {0, 0, 0, 0};
        bool form_fits[4] = {true, true, true, true};
        t_skinny_forced = true;
        for (int c = 0; c < n_forms; ++c) {
            t_force_skinny_fused = forms[c].fused;
            t_force_skinny_ring = forms[c].ring;
            form_fits[c] = a->workspace == nullptr ||
                           make_layout(a->M, a->d_model, a->d_ff, a->flags, GMLP_VARIANT_SKINNY, dev->sm_count).total <= a->workspace_bytes;
        }
        for (int round = 0; round <= kRounds && rc == GMLP_OK && n_forms > 1; ++round)
            for (int c = 0; c < n_forms && rc == GMLP_OK; ++c) {
                if (!form_fits[c]) continue;
                gmlp_args t = *a;
                t.variant = GMLP_VARIANT_SKINNY;
                t.flags &= ~(uint32_t)GMLP_FLAG_CHECKED;
                t_force_skinny_fused = forms[c].fused;
                t_force_skinny_ring = forms[c].ring;
                rc = forward_impl(&t);
                float ms = 0.0f;
                if (rc == GMLP_OK && cudaEventRecord(e0, st) != cudaSuccess) rc = GMLP_ERR_LAUNCH;
                for (int i = 0; i < per_round && rc == GMLP_OK; ++i) rc = forward_impl(&t);
                if (rc != GMLP_OK) break;
                if (cudaEventRecord(e1, st) != cudaSuccess || cudaEventSynchronize(e1) != cudaSuccess ||
                    cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) { rc = GMLP_ERR_LAUNCH; break; }
                if (round > 0) form_ms[c] += ms;
            }
        t_skinny_forced = false;
        t_force_skinny_fused = t_force_skinny_ring = 0;
        if (rc == GMLP_OK) {
            const int s3 = read_device_status();
            if (s3 < 0) rc = s3;
            else if (s3 != 0) rc = GMLP_ERR_TIMEOUT;
        }
        if (rc == GMLP_OK && n_forms > 1 && form_fits[0]) {
            int bf = 0;
            for (int c = 1; c < n_forms; ++c)
                if (form_fits[c] && form_ms[c] < form_ms[bf]) bf = c;
            // the rule's own choice is kept unless another form is measurably (1 %) faster
            if (form_ms[bf] < 0.99f * form_ms[0]) { best_gu_nb = forms[bf].fused; best_down_form = forms[bf].ring; }
            if (getenv("GMLP_TUNE_VERBOSE")) {
                fprintf(stderr, "gmlp_autotune   small-M forms (one-kernel form 0 rule / 1 on / 2 off, rings 0 rule / 1 half / 2 full):");
                for (int c = 0; c < n_forms; ++c)
                    if (form_fits[c])
                        fprintf(stderr, " [%d %d: %.1f us]%s", forms[c].fused, forms[c].ring, form_ms[c] * 1000.0f / (float)timed_calls,
                                (forms[c].fused == best_gu_nb && forms[c].ring == best_down_form) ? "*" : "");
                fprintf(stderr, "\n");
            }
        }
    }
    (void)cudaEventDestroy(e0);
    (void)cudaEventDestroy(e1);
    if (rc != GMLP_OK) return rc;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        bool found = false;
        for (TunedShape& t : g_tuned)
            if (t.device == device && t.M == a->M && t.d_model == a->d_model && t.d_ff == a->d_ff) {
                t.variant = w.variant; t.gu_pair = w.gu; t.down_pair = w.down;
                t.gu_nb = best_gu_nb; t.down_form = best_down_form;
                found = true;
            }
        if (!found) {
            TunedShape t = {device, a->M, a->d_model, a->d_ff, w.variant, w.gu, w.down, best_gu_nb, best_down_form, {0}};
            device_name_of(device, t.device_name);
            g_tuned.push_back(t);
        }
        g_tuned_count.store((int)g_tuned.size(), std::memory_order_release);
    }
    if (const char* cache = getenv("GMLP_TUNE_CACHE")) (void)tune_cache_save(cache);
    if (best_variant) *best_variant = w.variant;
    if (best_us) *best_us = best_ms * 1000.0f / (float)timed_calls;
    return GMLP_OK;
}

}  // namespace

extern "C" {

int gmlp_gqa_attention(const gmlp_gqa_args* args) {
    try {
        return gqa_attention_impl(args);
    } catch (...) {
        return GMLP_ERR_LAUNCH;
    }
}

int gmlp_qkv_proj(const gmlp_qkv_args* args) {
    try {
        return qkv_proj_impl(args);
    } catch (...) {
        return GMLP_ERR_LAUNCH;
    }
}

int gmlp_autotune(const gmlp_args* args, int iters, int32_t* best_variant, float* best_us) {
    try {
        return autotune_impl(args, iters, best_variant, best_us);
    } catch (...) {
        return GMLP_ERR_LAUNCH;
    }
}

int gmlp_autotune_query(int64_t M, int64_t d_model, int64_t d_ff, int32_t* variant, int32_t* gate_up_pair,
                        int32_t* down_pair) {
    TunedShape t;
    if (!tuned_lookup(M, d_model, d_ff, &t)) return 0;
    if (variant) *variant = t.variant;
    if (gate_up_pair) *gate_up_pair = t.gu_pair;
    if (down_pair) *down_pair = t.down_pair;
    return 1;
}

int gmlp_sum_partials(const void* const* partials, int32_t n_partials, void* Y, uint64_t count, void* stream) {
    if (partials == nullptr || Y == nullptr) return GMLP_ERR_NULL;
    if (n_partials < 1 || n_partials > gmlp::kMaxPartials) return GMLP_ERR_SHAPE;
    if (count % 8 != 0) return GMLP_ERR_SHAPE;
    if (!aligned16(Y)) return GMLP_ERR_ALIGN;
    gmlp::PartialList list = {};
    list.n = n_partials;
    for (int i = 0; i < n_partials; ++i) {
        if (partials[i] == nullptr) return GMLP_ERR_NULL;
        if (!aligned16(partials[i])) return GMLP_ERR_ALIGN;
        list.p[i] = static_cast<const float*>(partials[i]);
    }
    int rc = GMLP_OK;
    DeviceState* dev = current_device(&rc);
    if (dev == nullptr) return rc;
    if (count == 0) return GMLP_OK;
    const size_t nvec4 = (size_t)(count / 4);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((nvec4 + 255) / 256));
    cfg.blockDim = dim3(256);
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = pdl_allowed();
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, gmlp::sum_partials_bf16_kernel, list, static_cast<bf16*>(Y), nvec4) != cudaSuccess)
        return GMLP_ERR_LAUNCH;
    GMLP_CHECK_LAUNCH();
    return GMLP_OK;
}

int gmlp_workspace_forget(const void* workspace, uint64_t bytes) {
    int rc = GMLP_OK;
    DeviceState* dev = current_device(&rc);
    if (dev == nullptr) return rc;
    std::lock_guard<std::mutex> lock(g_mutex);
    const uint8_t* w = static_cast<const uint8_t*>(workspace);
    for (int i = 0; i < DeviceState::kCleanSlots; ++i) {
        const uint8_t* c = static_cast<const uint8_t*>(dev->clean_counters[i]);
        if (c != nullptr && (w == nullptr || (c >= w && (uint64_t)(c - w) < bytes))) {
            dev->clean_counters[i] = nullptr;
            dev->clean_counters_bytes[i] = 0;
        }
    }
    return GMLP_OK;
}

int gmlp_autotune_save(const char* path) {
    try {
        return tune_cache_save(path);
    } catch (...) {
        return GMLP_ERR_LAUNCH;
    }
}

int gmlp_autotune_load(const char* path, const char* device_name) {
    try {
        return tune_cache_load(path, device_name);
    } catch (...) {
        return GMLP_ERR_LAUNCH;
    }
}

void gmlp_autotune_clear(void) {
    std::lock_guard<std::mutex> lock(g_mutex);
    g_tuned.clear();
    g_tuned_count.store(0, std::memory_order_release);
}

int gmlp_matmul_add_rmsnorm(const gmlp_mmaddnorm_args* args) {
    try {
        return matmul_add_rmsnorm_impl(args);
    } catch (...) {
        return GMLP_ERR_LAUNCH;
    }
}

int gmlp_rmsnorm_matmul(const gmlp_rmsmm_args* args) {
    try {
        return rmsnorm_matmul_impl(args);
    } catch (...) {
        return GMLP_ERR_LAUNCH;
    }
}

int gmlp_gate_up(const gmlp_args* args) {
    try {
        return gate_up_impl(args);
    } catch (...) {
        return GMLP_ERR_LAUNCH;
    }
}

int gmlp_forward_static(const void* X, const void* Wg, const void* Wu, const void* Wd, void* Y,
                        int64_t M, int64_t d_model, int64_t d_ff, void* stream) {
    try {
        return forward_static_impl(X, Wg, Wu, Wd, Y, M, d_model, d_ff, static_cast<cudaStream_t>(stream));
    } catch (...) {
        return GMLP_ERR_LAUNCH;
    }
}

int gmlp_forward_ex(const gmlp_args* args) {
    try {
        return forward_impl(args);
    } catch (...) {
        return GMLP_ERR_LAUNCH;
    }
}

int gmlp_forward(const void* X, const void* Wg, const void* Wu, const void* Wd, void* Y,
                 int64_t M, int64_t d_model, int64_t d_ff, uint32_t flags) {
    gmlp_args a{};
    a.struct_bytes = sizeof(gmlp_args);
    a.flags = flags;
    a.X = X; a.Wg = Wg; a.Wu = Wu; a.Wd = Wd; a.Y = Y;
    a.M = M; a.d_model = d_model; a.d_ff = d_ff;
    a.rms_gain = nullptr;
    a.rms_eps = t_default_eps;
    a.variant = GMLP_VARIANT_AUTO;
    a.stream = t_stream;
    a.workspace = nullptr;
    a.workspace_bytes = 0;
    a.act_beta = 1.0f;
    return gmlp_forward_ex(&a);
}

int gmlp_forward_host(const gmlp_args* args, const void* X_host, void* Y_host) {
    if (args == nullptr || X_host == nullptr || Y_host == nullptr) return GMLP_ERR_NULL;
    if (args->struct_bytes != sizeof(gmlp_args)) return GMLP_ERR_FLAGS;
    int rc = check_shape(args->M, args->d_model, args->d_ff);
    if (rc != GMLP_OK) return rc;
    if (args->M == 0) return gmlp_forward_ex(args);
    if (!args->X || !args->Y) return GMLP_ERR_NULL;
    const size_t bytes = (size_t)args->M * (size_t)args->d_model * 2;
    const size_t y_bytes = (args->flags & GMLP_FLAG_Y_FP32) ? 2 * bytes : bytes;
    cudaStream_t st = static_cast<cudaStream_t>(args->stream);
    if (cudaMemcpyAsync(const_cast<void*>(args->X), X_host, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return GMLP_ERR_LAUNCH;
    rc = gmlp_forward_ex(args);
    if (rc != GMLP_OK) return rc;
    if (cudaMemcpyAsync(Y_host, args->Y, y_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return GMLP_ERR_LAUNCH;
    return GMLP_OK;
}

uint64_t gmlp_workspace_bytes(int64_t M, int64_t d_model, int64_t d_ff, uint32_t flags, int32_t variant) {
    if (check_shape(M, d_model, d_ff) != GMLP_OK) return 0;
    if (variant < GMLP_VARIANT_AUTO || variant > GMLP_VARIANT_TENSOR) return 0;
    int sm_count = 148;
    int dev = -1;
    if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < kMaxDevices) {
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0) sm_count = sms;
    }
    (void)cudaGetLastError();
    const Layout L = make_layout(M, d_model, d_ff, flags, resolve_variant(M, d_model, d_ff, variant), sm_count);
    return L.total > 256 ? L.total : 256;
}

int gmlp_small_m_plan(int64_t M, int64_t d_model, int64_t d_ff, int32_t sm_count, int32_t plan[6]) {
    if (plan == nullptr) return GMLP_ERR_NULL;
    if (check_shape(M, d_model, d_ff) != GMLP_OK || M < 1) return GMLP_ERR_SHAPE;
    const int sms = sm_count > 0 ? sm_count : current_sm_count();
    const SkinnyPlan a = make_skinny_plan(M, d_model, d_ff, 2, sms), b = make_skinny_plan(M, d_ff, d_model, 1, sms);
    const SkinnyPlan* p[2] = {&a, &b};
    for (int i = 0; i < 2; ++i) {
        plan[3 * i] = p[i]->cluster;
        plan[3 * i + 1] = p[i]->cluster >= 1 ? 64 * p[i]->c_boxes : 128 * p[i]->NH;
        plan[3 * i + 2] = p[i]->cluster >= 1 ? p[i]->c_tiles : p[i]->num_tiles;
    }
    return GMLP_OK;
}

int gmlp_small_m_fused_plan(int64_t M, int64_t d_model, int64_t d_ff, int32_t sm_count, int32_t plan[5]) {
    if (plan == nullptr) return GMLP_ERR_NULL;
    if (check_shape(M, d_model, d_ff) != GMLP_OK || M < 1) return GMLP_ERR_SHAPE;
    const FusedPlan f = make_fused_plan(M, d_model, d_ff, sm_count > 0 ? sm_count : current_sm_count());
    plan[0] = f.cluster;
    plan[1] = f.cluster >= 1 ? f.slices : 0;
    plan[2] = f.cluster >= 1 ? f.stages : 0;
    plan[3] = f.cluster >= 1 ? (int32_t)f.tmem_cols : 0;
    plan[4] = f.cluster >= 1 && f.preferred ? 1 : 0;
    return GMLP_OK;
}

int gmlp_pick_variant(int64_t M, int64_t d_model, int64_t d_ff, uint32_t flags) {
    (void)flags;
    if (check_shape(M, d_model, d_ff) != GMLP_OK) return GMLP_ERR_SHAPE;
    return resolve_variant(M, d_model, d_ff, GMLP_VARIANT_AUTO);
}

int gmlp_device_status(void) {
    int rc = GMLP_OK;
    DeviceState* dev = current_device(&rc);
    if (dev == nullptr) return rc;
    const int s = read_device_status();
    if (s != 0) forget_counters(dev);
    return s;
}

int gmlp_profile_enable(int on) {
    t_prof.on = (on != 0);
    t_prof.recorded = 0;
    t_prof.cur = nullptr;
    return GMLP_OK;
}

int gmlp_profile_read(float* ms, int max_count, int* count) {
    if (ms == nullptr || count == nullptr) return GMLP_ERR_NULL;
    *count = 0;
    if (!t_prof.created || t_prof.recorded == 0) return GMLP_OK;
    const int ncalls = t_prof.recorded < kProfRing ? t_prof.recorded : kProfRing;
    const ProfCall& last = t_prof.calls[(t_prof.recorded - 1) % kProfRing];
    const int nk = last.n;
    double sum[kMaxProfKernels] = {};
    int used = 0;
    for (int i = 0; i < ncalls; ++i) {
        const ProfCall& c = t_prof.calls[i];
        if (c.n != nk) continue;                 // a call of another shape/schedule: not averaged in
        if (cudaEventSynchronize(c.ev[c.n]) != cudaSuccess) return GMLP_ERR_LAUNCH;
        for (int k = 0; k < nk; ++k) {
            float t = 0.0f;
            if (cudaEventElapsedTime(&t, c.ev[k], c.ev[k + 1]) != cudaSuccess) return GMLP_ERR_LAUNCH;
            sum[k] += t;
        }
        ++used;
    }
    for (int k = 0; k < nk && k < max_count && used > 0; ++k) {
        ms[k] = (float)(sum[k] / used);
        *count = k + 1;
    }
    return GMLP_OK;
}

const char* gmlp_profile_kernel_name(int index) {
    if (t_prof.recorded == 0) return "";
    const ProfCall& last = t_prof.calls[(t_prof.recorded - 1) % kProfRing];
    if (index < 0 || index >= last.n) return "";
    return last.names[index];
}

int gmlp_selftest_wait_timeout(void* stream) {
    int rc = GMLP_OK;
    DeviceState* dev = current_device(&rc);
    if (dev == nullptr) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(st) != cudaSuccess) return GMLP_ERR_LAUNCH;
    int s = read_device_status();                       // start from a clean status word
    if (s < 0) return s;
    gmlp::wait_timeout_probe_kernel<<<1, 32, 0, st>>>(2000000LL);      // about a millisecond
    if (cudaPeekAtLastError() != cudaSuccess) return GMLP_ERR_LAUNCH;
    if (cudaStreamSynchronize(st) != cudaSuccess) return GMLP_ERR_LAUNCH;
    s = read_device_status();
    if (s < 0) return s;
    return s == ((99 << 16) | 1) ? GMLP_ERR_TIMEOUT : (s == 0 ? GMLP_OK : GMLP_ERR_LAUNCH);
}

#ifdef GMLP_TRACE
// GMLP_TRACE builds only: copies the timeline (kernels x CTAs x sites, nanoseconds) to `dst` after a device synchronize
int gmlp_trace_read(unsigned long long* dst, uint64_t bytes) {
    if (cudaDeviceSynchronize() != cudaSuccess) return GMLP_ERR_LAUNCH;
    if (bytes > sizeof(gmlp::g_trace)) bytes = sizeof(gmlp::g_trace);
    return cudaMemcpyFromSymbol(dst, gmlp::g_trace, bytes) == cudaSuccess ? GMLP_OK : GMLP_ERR_LAUNCH;
}
#endif

uint64_t gmlp_launch_count(void) { return t_launches; }
void gmlp_reset_launch_count(void) { t_launches = 0; }

const char* gmlp_status_string(int status) {
    switch (status) {
        case GMLP_OK: return "ok";
        case GMLP_ERR_NULL: return "a required pointer is NULL";
        case GMLP_ERR_SHAPE: return "bad shape: M < 0, or d_model/d_ff not a positive multiple of 8, or too large";
        case GMLP_ERR_ALIGN: return "a pointer is not sufficiently aligned (16 bytes; workspace 256)";
        case GMLP_ERR_FLAGS: return "unknown flag bit, unknown variant or wrong struct_bytes";
        case GMLP_ERR_WORKSPACE: return "workspace too small or could not be allocated";
        case GMLP_ERR_ARCH: return "no CUDA device, or the current device is not sm_100";
        case GMLP_ERR_LAUNCH: return "a CUDA runtime call failed";
        case GMLP_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case GMLP_ERR_UNSUPPORTED: return "the forced variant cannot run this shape";
        case GMLP_ERR_STATIC_LIMIT:
            return "gmlp_forward_static: shape exceeds its fixed scratch (M <= 16, no RMSNorm, scratch <= 12 MiB)";
        default: return "unknown status";
    }
}

int gmlp_version(void) { return kVersion; }

int gmlp_set_stream(void* cuda_stream) {
    t_stream = static_cast<cudaStream_t>(cuda_stream);
    return GMLP_OK;
}

int gmlp_set_default_eps(float eps) {
    if (!(eps >= 0.0f)) return GMLP_ERR_FLAGS;
    t_default_eps = eps;
    return GMLP_OK;
}

void gmlp_shutdown(void) {
    std::lock_guard<std::mutex> lock(g_mutex);
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) { (void)cudaGetLastError(); return; }
    for (int d = 0; d < kMaxDevices; ++d) {
        if (g_dev[d].workspace != nullptr) {
            if (cudaSetDevice(d) == cudaSuccess) {
                (void)cudaDeviceSynchronize();
                (void)cudaFree(g_dev[d].workspace);
            }
            g_dev[d].workspace = nullptr;
            g_dev[d].workspace_bytes = 0;
        }
    }
    (void)cudaSetDevice(prev);
    (void)cudaGetLastError();
}

}  // extern "C"
