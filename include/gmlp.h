/*
 * libgmlp — the fused Gated MLP for NVIDIA B200 (sm_100a), C ABI.
 *
 *     Y = ( SiLU(Xn * W_gate)  (.)  (Xn * W_up) ) * W_down,      Xn = X  or  RMSNorm(X)
 *
 * The operator is the five-node dataflow graph of the paper's Gated-MLP example (figure
 * "mlp-example" (a): matmul, matmul, silu, multiply, matmul; W1 = gate, W2 = up,
 * W3 = down) with the element-level meanings of its granular-operation table (Section 5:
 * matmul(x,y) = sum_k x[i,k]*y[k,j]; silu(x) = x*sigmoid(x)).  The optional prologue is
 * RMSNorm as in Eq. (1) of Section 2, Xn = X (.) 1/sqrt(mean_k(X^2) + eps), followed by an
 * optional per-column gain (an extension; no gain = the paper's form).
 *
 * Data: bf16 in, bf16 out, fp32 accumulation.  The gated product H = silu(G)*U is rounded
 * once to bf16 (round-to-nearest-even); so is Xn when the prologue is on; so is Y.
 *
 * Layout (operand convention of the paper's matmul, a[..., i0, i1] * b[..., i1, i2]):
 *   X  [M, d_model]      row-major bf16
 *   Wg [d_model, d_ff]   row-major bf16   ("[in, out]")
 *   Wu [d_model, d_ff]   row-major bf16
 *   Wd [d_ff, d_model]   row-major bf16
 *   Y  [M, d_model]      row-major bf16
 * All pointers are DEVICE pointers unless a parameter says "host".  Every pointer must be
 * 16-byte aligned; d_model and d_ff must be positive multiples of 8; M >= 0 (M == 0 is a
 * successful no-op that looks at no pointer).  Y must not overlap any input.  Inputs are only read.
 *
 * Ownership: the caller owns every buffer.  The library allocates nothing per call when a
 * workspace is passed; with workspace == NULL it uses a library-owned buffer that grows on
 * demand (cudaMalloc on the calling thread's current device) and is freed by
 * gmlp_shutdown().
 * A caller-made workspace belongs to the library between calls: the small-M schedules keep arrival
 * counters in it, which the library zeroes the first time it sees a (pointer, size) and which its kernels
 * leave zero after every call, so later calls with the same workspace start without a memset (calls of other
 * shapes or schedules through the same buffer are noticed: what they overwrite is forgotten by itself).  If
 * anything else writes to that memory between two calls (the buffer was freed and handed out again by an
 * allocator, reused as scratch, ...), tell the library with gmlp_workspace_forget() before the next call.
 *
 * Stream order: X, the outputs and the workspace are used in stream order, like any kernel's operands.  The WEIGHT
 * MATRICES (Wg, Wu, Wd here; W, Wq, Wk, Wv of the other operators below) may be read EARLIER: the kernels of a call are
 * chained by programmatic dependent launch, and the GEMM kernels request their first weight tiles before they wait for
 * the work that precedes the call on the stream (a call's start overlaps its predecessor's tail; for a few tokens that
 * is a tenth of the step).  Weights that are complete
 * when the call is made - the normal case - need nothing.  If a kernel enqueued shortly before the call on the SAME
 * stream produces them (dequantisation on the fly, an optimiser step), pass GMLP_FLAG_WEIGHTS_IN_STREAM_ORDER: the
 * call's first kernel is then launched in plain stream order, nothing of the call starts before that work is
 * complete, and the call loses the overlap with its predecessor (a few microseconds).  gmlp_forward_static and the
 * other operators have no such flag: their weights must be complete before the call is made (or be produced on another
 * stream and handed over with an event, which orders everything).
 *
 * Errors: every entry point returns a gmlp_status code; nothing throws, aborts or prints.
 * Calls are asynchronous on the given stream: device-side problems (a bounded wait that
 * ran out) surface after the stream is synchronised, through gmlp_device_status(), or at
 * once with GMLP_FLAG_CHECKED.  On a device that is not sm_100 the calls return
 * GMLP_ERR_ARCH: there is no fallback of any kind.
 */
#ifndef GMLP_H_
#define GMLP_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum gmlp_status {
    GMLP_OK = 0,
    GMLP_ERR_NULL = -1,       /* a required pointer is NULL */
    GMLP_ERR_SHAPE = -2,      /* M < 0, or d_model / d_ff not a positive multiple of 8, or too large */
    GMLP_ERR_ALIGN = -3,      /* a pointer is not 16-byte aligned */
    GMLP_ERR_FLAGS = -4,      /* unknown flag bit, unknown variant, or bad struct_bytes */
    GMLP_ERR_WORKSPACE = -5,  /* workspace too small (or could not be grown) */
    GMLP_ERR_ARCH = -6,       /* no CUDA device, or the current device is not sm_100 */
    GMLP_ERR_LAUNCH = -7,     /* a CUDA runtime call failed (cudaGetLastError is left readable) */
    GMLP_ERR_TIMEOUT = -8,    /* a bounded device-side wait ran out (see gmlp_device_status) */
    GMLP_ERR_UNSUPPORTED = -9,/* the forced variant cannot run this shape (SKINNY: M <= 128, or <= 256 on layers whose
                                 two GEMMs both have its cluster form) */
    GMLP_ERR_STATIC_LIMIT = -10 /* gmlp_forward_static: the shape needs more than its fixed built-in scratch */
} gmlp_status;

enum {
    GMLP_FLAG_RMSNORM = 1u << 0, /* apply the RMSNorm prologue to X */
    GMLP_FLAG_CHECKED = 1u << 2, /* synchronise the stream and report the device status before returning */
    /* Gate activation of the gated unit H = act(G) (.) U.  The paper's operator uses SiLU (no flag); its
     * benchmark list (Section 6.1) also names SwiGLU- and GLU-gated forms, which differ only in act:
     *   none             act(g) = g * sigmoid(g)              (SiLU)
     *   ACT_SWISH        act(g) = g * sigmoid(act_beta * g)   (Swish-beta; beta = 1 is SiLU bit for bit)
     *   ACT_GLU          act(g) = sigmoid(g)                  (GLU)
     *   ACT_GELU         act(g) = g * Phi(g)                  (GELU gate; Phi the standard normal distribution function,
     *                                                          the exact erf form, not the tanh approximation)
     * Setting more than one is GMLP_ERR_FLAGS, and so is a NaN or infinite act_beta with ACT_SWISH. */
    GMLP_FLAG_ACT_SWISH = 1u << 5,
    GMLP_FLAG_ACT_GLU = 1u << 6,
    GMLP_FLAG_ACT_GELU = 1u << 9,
    /* The three weight matrices are stored [out, in] (the layout of a linear layer's weight in the common
     * frameworks): Wg, Wu [d_ff, d_model], Wd [d_model, d_ff], row-major.  The operator is unchanged
     * (Y = (act(X Wg^T) (.) (X Wu^T)) Wd^T in that storage); the tensor-core kernels read such a matrix as a
     * K-major operand straight from its TMA tile, so no transposed copy is made and the results are the same
     * bit for bit as with the [in, out] storage.  gmlp_forward_ex and gmlp_gate_up with the tensor-core
     * schedules only (GMLP_VARIANT_SIMT / _STREAM: GMLP_ERR_UNSUPPORTED); gmlp_forward_static and the other
     * operators take [in, out] weights. */
    GMLP_FLAG_WEIGHTS_OUT_IN = 1u << 7,
    /* Y is left in fp32: args->Y is a float matrix [M, d_model] and receives the down projection's fp32
     * accumulator without the final rounding (rounding it to bf16 gives the default output bit for bit).
     * gmlp_forward_ex / gmlp_forward_host with the tensor-core schedules only (SIMT / STREAM:
     * GMLP_ERR_UNSUPPORTED); gmlp_gate_up rejects it (GMLP_ERR_FLAGS). */
    GMLP_FLAG_Y_FP32 = 1u << 8,
    /* The weights (or the gain) may still be written by work enqueued earlier on the same stream: see "Stream order"
     * above.  gmlp_forward_ex, gmlp_forward_host and gmlp_gate_up. */
    GMLP_FLAG_WEIGHTS_IN_STREAM_ORDER = 1u << 10
};

/* Kernel schedule.  AUTO picks by shape; the others force one schedule (tests, benchmarks). */
enum {
    GMLP_VARIANT_AUTO = 0,
    GMLP_VARIANT_SIMT = 1,   /* CUDA-core tiled GEMMs: any shape, slow; bring-up and cross-check */
    GMLP_VARIANT_STREAM = 2, /* small M: weight-streaming split-K kernels on CUDA cores (HBM-bound regime) */
    GMLP_VARIANT_UMMA = 3,   /* medium M: tcgen05 tensor-core GEMMs fed by TMA, accumulators in TMEM, one CTA per tile */
    GMLP_VARIANT_SKINNY = 4, /* few tokens (HBM-bound regime): operand-swapped tcgen05 GEMMs that stream the weights once; per
                                GEMM either K split over a thread-block cluster per column tile and reduced on chip (layers
                                with fewer column tiles than SMs; up to 256 tokens) or stream-K over all SMs with partial
                                sums through the workspace (up to 128 tokens); on small layers with at most 16 tokens
                                both GEMMs and the activation run in ONE kernel per 128-wide slice of d_ff (see
                                gmlp_small_m_fused_plan).  AUTO takes it up to 32 tokens; where both GEMMs have the cluster
                                form up to 96, and up to 200 on layers with d_model >= 3072. */
    GMLP_VARIANT_PAIR = 5,   /* large M: the same GEMMs on CTA pairs (tcgen05 cta_group::2, 256-row tiles) */
    GMLP_VARIANT_TENSOR = 6  /* what AUTO takes outside SKINNY: each of the two GEMMs picks, by its number of
                                128-row blocks, the CTA-pair kernel or the single-CTA kernel (whose down projection
                                splits K over a thread-block cluster when there are few output tiles) */
};

typedef struct gmlp_args {
    uint32_t struct_bytes;    /* sizeof(gmlp_args); guards against ABI drift */
    uint32_t flags;           /* GMLP_FLAG_* */
    const void* X;            /* device, [M, d_model] bf16 */
    const void* Wg;           /* device, [d_model, d_ff] bf16 */
    const void* Wu;           /* device, [d_model, d_ff] bf16 */
    const void* Wd;           /* device, [d_ff, d_model] bf16 */
    void* Y;                  /* device, [M, d_model] bf16, written */
    int64_t M, d_model, d_ff;
    const void* rms_gain;     /* device, [d_model] bf16, or NULL for no gain; read only with GMLP_FLAG_RMSNORM */
    float rms_eps;            /* eps of Eq. (1); used only with GMLP_FLAG_RMSNORM */
    int32_t variant;          /* GMLP_VARIANT_* */
    void* stream;             /* cudaStream_t; NULL = the legacy default stream */
    void* workspace;          /* device scratch of >= gmlp_workspace_bytes(...) bytes, 256-byte aligned, or NULL */
    uint64_t workspace_bytes;
    float act_beta;           /* beta of GMLP_FLAG_ACT_SWISH; ignored without that flag */
    uint32_t reserved;        /* must be 0 */
} gmlp_args;

/*
 * The operator as the paper states it: Y = (silu(X Wg) (.) (X Wu)) Wd.
 * Runs on the stream set by gmlp_set_stream (default: legacy default stream) with the
 * library-owned workspace.  With GMLP_FLAG_RMSNORM the prologue has no gain and uses the eps
 * set by gmlp_set_default_eps (default 1e-5); GMLP_FLAG_ACT_SWISH here means beta = 1 (use
 * gmlp_forward_ex for another beta).  Asynchronous; returns a gmlp_status.
 */
int gmlp_forward(const void* X, const void* Wg, const void* Wu, const void* Wd, void* Y,
                 int64_t M, int64_t d_model, int64_t d_ff, uint32_t flags);

/* Same operator with every option explicit (gain, eps, stream, workspace, variant). */
int gmlp_forward_ex(const gmlp_args* args);

/*
 * The gate/up half on its own: H = bf16( silu(Xn Wg) (.) (Xn Wu) ), the four-operator kernel
 * "Matmul+Matmul+SiLU+Mul" of the paper's benchmark list (Section 6.1).  Uses args->X, Wg, Wu, the
 * prologue options, stream, workspace and variant exactly as gmlp_forward_ex does; args->Wd is ignored
 * (may be NULL) and args->Y receives H, row-major [M, d_ff] bf16 (d_ff columns, not d_model).
 * Workspace: gmlp_workspace_bytes() of the same shape is sufficient.  GMLP_VARIANT_SIMT and _STREAM are
 * not offered for this call (GMLP_ERR_UNSUPPORTED).
 */
int gmlp_gate_up(const gmlp_args* args);

/*
 * RMSNorm followed by a matrix multiplication, the paper's running example (Section 2):
 *     Z = RMSNorm(X) * W,     X [M, K], W [K, N], Z [M, N], row-major bf16, K and N multiples of 8.
 * Default schedule = the paper's algebraic rewrite (X*W) (.) r: the row scale r = 1/sqrt(mean(X^2)+eps)
 * does not depend on k, so the GEMM runs on the raw X and applies r in its epilogue, while a small
 * kernel computes r; the two are chained by programmatic dependent launch and only the GEMM's epilogue
 * waits for r, so the RMS branch runs in parallel with the matmul's main loop.  No normalised copy of X
 * is stored.  A gain (rms_gain != NULL, along K) does not commute with the matmul: such calls, and calls
 * with GMLP_RMSMM_UNFUSED, run the RMSNorm kernel into the workspace and then the plain GEMM.
 * workspace (256-byte aligned, required): M*4 bytes for the rewritten schedule, M*K*2 for the unfused one.
 */
enum { GMLP_RMSMM_UNFUSED = 1u << 4 };   /* flag for gmlp_rmsmm_args.flags, next to GMLP_FLAG_CHECKED */
typedef struct gmlp_rmsmm_args {
    uint32_t struct_bytes;    /* sizeof(gmlp_rmsmm_args) */
    uint32_t flags;           /* GMLP_FLAG_CHECKED | GMLP_RMSMM_UNFUSED */
    const void* X;            /* device, [M, K] bf16 */
    const void* W;            /* device, [K, N] bf16 */
    void* Z;                  /* device, [M, N] bf16, written */
    int64_t M, K, N;
    const void* rms_gain;     /* device, [K] bf16, or NULL (the paper's form) */
    float rms_eps;
    int32_t reserved;         /* must be 0 */
    void* stream;
    void* workspace;
    uint64_t workspace_bytes;
} gmlp_rmsmm_args;
int gmlp_rmsnorm_matmul(const gmlp_rmsmm_args* args);

/*
 * A matrix multiplication, a residual addition and RMSNorm, "Matmul+Add+RMSNorm" of the paper's benchmark
 * list (Section 6.1; the paper names the chain, the graph below is the reading taken):
 *     S = bf16( X * W + R ),     Z = bf16( RMSNorm(S) ) = bf16( S * rsqrt(mean_n S^2 + eps) * gain ),
 * X [M, K], W [K, N], R, S, Z [M, N] row-major bf16, gain [N] bf16 or NULL; K and N multiples of 8.  S (the
 * updated residual stream) is an output too and is rounded once from the fp32 sum; the statistic of Eq. (1)
 * is taken over the stored S.  R and S may be the same buffer (in-place residual update); Z must not alias.
 * Default schedule: the GEMM's epilogue adds R, stores S and leaves one sum of squares per row and column
 * tile; a light second kernel (chained by programmatic dependent launch) adds those in fixed order and
 * writes Z with one read of S.  GMLP_MMADDNORM_UNFUSED runs the three operators one after the other
 * (GEMM -> T, T + R -> S, RMSNorm(S) -> Z; T is rounded to bf16 on the way, so S may differ by an ulp).
 * workspace (256-byte aligned, required): ceil(N/256)*M*4 bytes fused, M*N*2 bytes unfused.
 */
enum { GMLP_MMADDNORM_UNFUSED = 1u << 4 };
typedef struct gmlp_mmaddnorm_args {
    uint32_t struct_bytes;    /* sizeof(gmlp_mmaddnorm_args) */
    uint32_t flags;           /* GMLP_FLAG_CHECKED | GMLP_MMADDNORM_UNFUSED */
    const void* X;            /* device, [M, K] bf16 */
    const void* W;            /* device, [K, N] bf16 */
    const void* R;            /* device, [M, N] bf16 residual */
    void* S;                  /* device, [M, N] bf16, written */
    void* Z;                  /* device, [M, N] bf16, written */
    int64_t M, K, N;
    const void* rms_gain;     /* device, [N] bf16, or NULL */
    float rms_eps;
    int32_t reserved;         /* must be 0 */
    void* stream;             /* cudaStream_t */
    void* workspace;
    uint64_t workspace_bytes;
} gmlp_mmaddnorm_args;
int gmlp_matmul_add_rmsnorm(const gmlp_mmaddnorm_args* args);

/*
 * QKV projection, one of the paper's multi-operator kernels (Section 6.1): three matmuls that share X,
 *     Q = X * Wq  [M, Nq],     K = X * Wk  [M, Nkv],     V = X * Wv  [M, Nkv]       (grouped-query shapes: Nkv <= Nq),
 * X [M, K], W* [K, N*], outputs row-major bf16, fp32 accumulation, one rounding; K, Nq, Nkv multiples of 8.
 * Default: ONE launch of the tensor-core GEMM whose column tiles run through the three weight matrices end to end
 * (the same sharing of the X strip that fuses the gate and up matmuls), each tile written to its own output.
 * GMLP_QKV_SEPARATE runs three GEMMs one after the other (for comparison).  No workspace.  The attention that
 * follows is gmlp_gqa_attention below.
 */
enum { GMLP_QKV_SEPARATE = 1u << 4 };
typedef struct gmlp_qkv_args {
    uint32_t struct_bytes;    /* sizeof(gmlp_qkv_args) */
    uint32_t flags;           /* GMLP_FLAG_CHECKED | GMLP_QKV_SEPARATE */
    const void* X;            /* device, [M, K] bf16 */
    const void* Wq;           /* device, [K, Nq] bf16 */
    const void* Wk;           /* device, [K, Nkv] bf16 */
    const void* Wv;           /* device, [K, Nkv] bf16 */
    void* Q;                  /* device, [M, Nq] bf16, written */
    void* Kout;               /* device, [M, Nkv] bf16, written */
    void* V;                  /* device, [M, Nkv] bf16, written */
    int64_t M, K, Nq, Nkv;
    void* stream;             /* cudaStream_t */
    uint64_t reserved;        /* must be 0 */
} gmlp_qkv_args;
int gmlp_qkv_proj(const gmlp_qkv_args* args);

/*
 * Group Query Attention, forward, no mask - the kernel that follows the QKV projection in the paper's benchmark
 * list (Section 6.1; the paper names it, the definition below is the standard one):
 *     for query head h, with key/value head g = h / (n_q_heads / n_kv_heads):
 *         O_h = softmax( Q_h K_g^T / sqrt(head_dim) ) V_g
 * Q [M, n_q_heads*head_dim], K and V [S, n_kv_heads*head_dim], O [M, n_q_heads*head_dim], row-major bf16 (head h in
 * columns [h*head_dim, (h+1)*head_dim) - the layout gmlp_qkv_proj writes); fp32 scores and accumulation, the
 * probabilities are rounded to bf16 for the second matmul, O is rounded once.  head_dim must be 128
 * (GMLP_ERR_UNSUPPORTED otherwise); n_q_heads a multiple of n_kv_heads.  One tcgen05 kernel, online softmax, the
 * scores never leave the SM.  No workspace.
 * GMLP_GQA_CAUSAL (an extension; the paper's kernel has no mask): query row m sees keys s <= m + (S - M) only -
 * the queries are the last M positions of the S-long sequence; needs S >= M (GMLP_ERR_SHAPE otherwise).  Key
 * blocks beyond a query tile's horizon are skipped.
 */
enum { GMLP_GQA_CAUSAL = 1u << 4 };
typedef struct gmlp_gqa_args {
    uint32_t struct_bytes;    /* sizeof(gmlp_gqa_args) */
    uint32_t flags;           /* GMLP_FLAG_CHECKED | GMLP_GQA_CAUSAL */
    const void* Q;            /* device, [M, n_q_heads*head_dim] bf16 */
    const void* K;            /* device, [S, n_kv_heads*head_dim] bf16 */
    const void* V;            /* device, [S, n_kv_heads*head_dim] bf16 */
    void* O;                  /* device, [M, n_q_heads*head_dim] bf16, written */
    int64_t M, S;             /* query rows, key/value rows */
    int32_t n_q_heads, n_kv_heads, head_dim;
    int32_t reserved;         /* must be 0 */
    void* stream;             /* cudaStream_t */
} gmlp_gqa_args;
int gmlp_gqa_attention(const gmlp_gqa_args* args);

/*
 * The same call for a caller whose activations live in HOST memory: copies X_host
 * (M*d_model bf16, ideally pinned) to args->X, runs gmlp_forward_ex, and copies args->Y
 * to Y_host, all asynchronously on args->stream.  args->X and args->Y are device staging
 * buffers owned by the caller; weights, gain and workspace are device-resident as usual.
 * Y_host is valid once the stream has been synchronised.
 */
int gmlp_forward_host(const gmlp_args* args, const void* X_host, void* Y_host);

/*
 * The same operator for callers that must not allocate device memory.  (The paper has no
 * counterpart of this call; it exists for deployment reasons only.)
 *
 * Who needs it: code that runs after an application has frozen its memory plan, e.g. a
 * serving loop that handed the whole device to its own pool at start-up, a process under a
 * memory manager that forbids further cudaMalloc, or a real-time path where an allocation's
 * implicit synchronisation is not acceptable.  gmlp_forward may grow a library-owned buffer
 * with cudaMalloc and gmlp_forward_ex wants a caller-made workspace; this call wants
 * neither.  Its scratch (the bf16 intermediate H, the split-K partial sums and the arrival
 * counters of the small-M schedule) lives in a fixed array of GMLP_STATIC_SCRATCH_BYTES that
 * is part of the library image: every GPU that loads the library holds that much memory
 * until the process exits, whether or not this call is ever used.
 *
 * Limits: M <= GMLP_STATIC_MAX_M tokens, no RMSNorm prologue, and a shape whose scratch fits
 * the array (any Llama-sized layer does at M <= 16).  Anything larger is refused with
 * GMLP_ERR_STATIC_LIMIT before any device work.  X, Wg, Wu, Wd, Y: device pointers as for
 * gmlp_forward; stream: cudaStream_t (NULL = legacy default stream).  Asynchronous.
 *
 * It calls no cudaMalloc, cudaFree or allocating library routine.  The FIRST call on each
 * device looks up the device address of the built-in array (cudaGetSymbolAddress, with that
 * device current) and sets kernel attributes; make that first call outside any stream
 * capture.  That first call is also what makes the CUDA runtime load the library's code and
 * the array onto the device (module loading is lazy), so make one call with M >= 1 per
 * device BEFORE the application freezes its memory plan: a caller that has already handed
 * every byte to its own pool gets GMLP_ERR_LAUNCH from that first call instead (the lookup
 * fails for lack of memory), and a call with M == 0 returns before the lookup and does not
 * serve as the warm-up.  After it, a call leaves the device's free memory as it found it.
 * All calls on a device share the one array, and it keeps whatever the previous
 * call left: each call clears the counters it needs itself, so back-to-back calls on one
 * stream are fine, but two calls that can overlap on the GPU (different streams, no
 * ordering) race on the scratch and give wrong results.
 */
#define GMLP_STATIC_SCRATCH_BYTES (12u << 20)
#define GMLP_STATIC_MAX_M 16
int gmlp_forward_static(const void* X, const void* Wg, const void* Wu, const void* Wd, void* Y,
                        int64_t M, int64_t d_model, int64_t d_ff, void* stream);

/*
 * Bytes of scratch gmlp_forward_ex needs for this shape, for the schedule `variant` would
 * run (AUTO = the one the library would pick): the bf16 intermediate H [M, d_ff], Xn
 * [M, d_model] when the prologue is on, and split-K partial sums and arrival counters for
 * the small-M schedule.  Returns 0 for invalid shapes.
 */
uint64_t gmlp_workspace_bytes(int64_t M, int64_t d_model, int64_t d_ff, uint32_t flags, int32_t variant);

/*
 * The last step of a d_ff-sharded Gated MLP.  Y = H W_down sums over d_ff (Section 2), so the layer may be cut into
 * shards of d_ff - the matching columns of W_gate and W_up and rows of W_down - each of which is a complete call of
 * this library with GMLP_FLAG_Y_FP32 that leaves an fp32 partial product [M, d_model] (H, and with it the rounding
 * of H, is per element of d_ff and does not depend on the cut).  gmlp_sum_partials adds n_partials (1..8) such
 * buffers in the order given - fixed, so the result does not depend on scheduling - rounds once and stores bf16:
 *   Y[i] = bf16_rn(partials[0][i] + partials[1][i] + ...),   i < count.
 * partials is a HOST array of DEVICE pointers (fp32, 16-byte aligned, count elements each); Y is a device pointer
 * (bf16, 16-byte aligned); count must be a multiple of 8.  With one process per GPU the partials are first summed
 * across ranks by the caller's collective (one all-reduce of M * d_model floats) and n_partials is 1.
 * Asynchronous on `stream` (a cudaStream_t, NULL = the default stream).  Returns GMLP_OK, GMLP_ERR_NULL,
 * GMLP_ERR_SHAPE (n_partials or count), GMLP_ERR_ALIGN, GMLP_ERR_ARCH or GMLP_ERR_LAUNCH.
 */
int gmlp_sum_partials(const void* const* partials, int32_t n_partials, void* Y, uint64_t count, void* stream);

/*
 * Drop what the library remembers about the contents of caller-made workspaces on the current device (the
 * arrival counters it believes to be zero; see "Ownership" above): those inside [workspace, workspace + bytes),
 * or all of them when `workspace` is NULL.  The next call that uses such a workspace zeroes its counters again
 * (one cudaMemsetAsync on the call's stream).  Host-side bookkeeping only; returns GMLP_OK or GMLP_ERR_ARCH.
 */
int gmlp_workspace_forget(const void* workspace, uint64_t bytes);

/*
 * Empirical schedule selection for one shape (the paper's extraction phase keeps, among the candidate kernels
 * its search produced, the one that measures fastest, Sections 3 and 6): runs args (a complete, valid
 * gmlp_forward_ex call; Y is overwritten with the correct result) with each tensor-core schedule that can run
 * the shape (SKINNY where it can run, and TENSOR with each of the four combinations of single-CTA or CTA-pair
 * kernel for the gate/up and for the down GEMM; those that do not fit a caller-supplied workspace are
 * skipped), about `iters` (1..10000) timed back-to-back calls each, in four interleaved rounds after a warm-up
 * round so that clock drift falls on all candidates alike, CUDA events on args->stream, and
 * remembers the fastest for (current device, M, d_model, d_ff): GMLP_VARIANT_AUTO, gmlp_pick_variant and
 * gmlp_workspace_bytes use it from then on (size workspaces after tuning).  When a single-CTA kernel is part of
 * the winner, a second stage measures its tile forms the same way (gate/up: 64- or 128-column tiles; down: K split
 * over a cluster of 2, 3 or 4 CTAs, or 128- or 256-column tiles without a split) and keeps a form that beats the
 * library's own rule by more than 1 %.  When SKINNY wins, the second stage measures ITS forms instead: the one-kernel
 * form against the two-kernel forms where gmlp_small_m_fused_plan applies, and, up to 32 tokens, half-size against
 * full-size weight rings (a half-size ring lets the next kernel on the stream become resident early, a full-size one
 * keeps more of the weight stream in flight), again keeping what beats the rule by more than 1 %.  Synchronises the stream.
 * best_variant (GMLP_VARIANT_SKINNY or _TENSOR) / best_us (microseconds per call) may be NULL.
 * gmlp_autotune_query returns 1 and the kept choice if the shape was tuned on the current device (gate_up_pair /
 * down_pair: 1 = CTA pairs, 0 = single CTAs, -1 = not applicable), else 0.  gmlp_autotune_clear forgets every
 * tuned shape.
 */
int gmlp_autotune(const gmlp_args* args, int iters, int32_t* best_variant, float* best_us);
int gmlp_autotune_query(int64_t M, int64_t d_model, int64_t d_ff, int32_t* variant, int32_t* gate_up_pair,
                        int32_t* down_pair);
void gmlp_autotune_clear(void);

/*
 * The tuned choices as a file (the scaled-down image of the paper's per-shape kernel cache, Section 6.5: a
 * search result is kept and reused, not recomputed).  One text line per tuned shape, tab-separated:
 *     gmlp-tune-v1  <library version>  <device name>  M  d_model  d_ff  variant  gate_up_pair  down_pair  gate_up_form  down_form
 * (gate_up_form / down_form, TENSOR: tile form of the single-CTA kernels, 0 = by rule; SKINNY: gate_up_form = one-kernel
 * form 0 by rule / 1 on / 2 off, down_form = weight rings 0 by rule / 1 half-size / 2 full-size.)
 * Lines that start with '#' and empty lines are ignored.
 * gmlp_autotune_save writes every choice the process holds (all devices) to `path`, through a temporary file that is
 * renamed over it; returns the number of lines written or a negative status.
 * gmlp_autotune_load reads `path` and keeps the lines whose library version is this library's and whose device name
 * is `device_name` (NULL: the name of the current CUDA device), attached to the current device (device 0 when there is
 * no CUDA device: loading and saving then still work, which is how the file format is tested on a machine without a
 * GPU); malformed lines and lines with values no schedule has are skipped.  Returns the number of shapes taken, or
 * GMLP_ERR_NULL / GMLP_ERR_LAUNCH (the file cannot be opened).  A shape loaded twice keeps the later line.
 * With the environment variable GMLP_TUNE_CACHE set to a path, the file is loaded the first time the library touches a
 * device and rewritten after every gmlp_autotune.
 */
int gmlp_autotune_save(const char* path);
int gmlp_autotune_load(const char* path, const char* device_name);

/*
 * How GMLP_VARIANT_SKINNY would run this shape on a device with `sm_count` SMs (0: the current device, 148 if there is
 * none): for the gate/up GEMM in plan[0..2] and the down projection in plan[3..5], the CTAs per thread-block cluster
 * that share a column tile (0: that GEMM runs as stream-K over all SMs, with partial sums through the workspace),
 * the tile width in columns and the number of tiles.  Returns GMLP_OK, or GMLP_ERR_SHAPE / GMLP_ERR_NULL.
 * Pure host arithmetic (the launch still asks the device whether the clusters fit one wave).
 */
int gmlp_small_m_plan(int64_t M, int64_t d_model, int64_t d_ff, int32_t sm_count, int32_t plan[6]);

/*
 * The one-kernel ("fused") form of GMLP_VARIANT_SKINNY for this shape on a device with `sm_count` SMs (0: the current
 * device, 148 if there is none).  In that form a thread-block cluster per 128-wide slice of d_ff computes its slice of
 * H = act(X Wg) * (X Wu) on chip and multiplies it with its rows of W_down at once; the partial Y of the slices go
 * through the workspace and a second, tiny kernel adds them in slice order.  plan[0] = CTAs per cluster (0: the form
 * does not apply and the two kernels of gmlp_small_m_plan run), plan[1] = number of slices (= clusters), plan[2] =
 * stages of the weight ring, plan[3] = TMEM columns per CTA, plan[4] = 1 if GMLP_VARIANT_SKINNY takes this form by
 * default (small layers, where the hand-over between two kernels costs more than it; by measurement), else 0.
 * The form needs at most 16 tokens, all clusters resident in one wave and the accumulators of gate, up
 * and a CTA's share of the d_model / 128 partial-Y tiles in TMEM.  Returns GMLP_OK, or GMLP_ERR_SHAPE / GMLP_ERR_NULL.
 * Pure host arithmetic.
 */
int gmlp_small_m_fused_plan(int64_t M, int64_t d_model, int64_t d_ff, int32_t sm_count, int32_t plan[5]);

/* The schedule AUTO resolves to for this shape (GMLP_VARIANT_SKINNY or _TENSOR, or what gmlp_autotune kept). */
int gmlp_pick_variant(int64_t M, int64_t d_model, int64_t d_ff, uint32_t flags);

/*
 * Reads and clears the device status word of the current device (synchronises the device).
 * 0 = no device-side problem since the last read; otherwise a code naming the wait that ran
 * out (high 16 bits: kernel id, low 16 bits: site).  Returns GMLP_ERR_* (< 0) on failure.
 */
int gmlp_device_status(void);

/*
 * Self-test of the device-side failure path: launches one tiny kernel whose bounded wait is bound to run
 * out (it waits, for about a millisecond at most, on a barrier that nothing completes), synchronises, and
 * checks that the device status word names that wait.  Nothing faults, traps or hangs; the context stays
 * usable.  Returns GMLP_ERR_TIMEOUT when the time-out was detected and reported as designed (the
 * expected outcome), GMLP_OK if the wait unexpectedly did not run out, or another GMLP_ERR_*.
 */
int gmlp_selftest_wait_timeout(void* stream);

/* Number of kernels the library launched on this host thread since the last reset. */
uint64_t gmlp_launch_count(void);
void gmlp_reset_launch_count(void);

/*
 * Per-kernel timing for benchmarks (per host thread, off by default).  While enabled, every
 * gmlp_forward_ex call records a CUDA event on its stream before its first kernel and after
 * each kernel; the library keeps the events of the 64 most recent calls, so calls can be
 * enqueued back to back.  gmlp_profile_read synchronises on those events and writes the
 * AVERAGE duration of each kernel over the recorded calls, in launch order, in milliseconds;
 * *count gets the number of kernels (at most max_count are written).
 * gmlp_profile_kernel_name(i) names the i-th kernel ("rmsnorm", "gate_up", "down"; "fused", "sum" for the one-kernel small-M form).  An event
 * between two kernels keeps the second from overlapping the first's tail, so these are
 * stand-alone kernel durations; do not leave profiling on in a timed region.
 */
int gmlp_profile_enable(int on);
int gmlp_profile_read(float* ms, int max_count, int* count);
const char* gmlp_profile_kernel_name(int index);

const char* gmlp_status_string(int status);
int gmlp_version(void);

/* Per-host-thread defaults for the 9-argument call. */
int gmlp_set_stream(void* cuda_stream);
int gmlp_set_default_eps(float eps);

/* Frees the library-owned workspace of every device.  Safe to call more than once. */
void gmlp_shutdown(void);

#ifdef __cplusplus
}
#endif
#endif /* GMLP_H_ */
