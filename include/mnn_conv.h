/*
 * mnn_conv.h — C ABI of the B200 (sm_100a) convolution library.
 *
 * The library computes y = act(conv2d(x, w) + bias) on NCHW fp32 tensors through
 * one of three schemes chosen ahead of inference (the paper's "pre-inference",
 * Section 3.2): Winograd F(m x m, k x k) (Eq. 6), a GEMM over gathered patches
 * (k = 1 "is just a matrix multiplication", Section 3.2 item 1; k > 1 strided or
 * dilated layers gather patches first) and a direct "sliding window" kernel
 * (Section 3.2 item 3, Eq. 3).
 *
 * Conventions for every entry point
 *   - x, w, bias, y and the workspace are DEVICE pointers owned by the caller,
 *     dense and contiguous: x [N][Cin][H][W], w [Cout][Cin/groups][k][k],
 *     bias [Cout] (NULL = zeros), y [N][Cout][OH][OW], all fp32 and 16-byte aligned.
 *   - OH = floor((H + 2 pad - dilation (k-1) - 1)/stride) + 1, same for OW.
 *     Cross-correlation (no kernel flip).
 *   - Matrices and info structs are HOST pointers.
 *   - `stream` is a cudaStream_t passed as void*.  Runs are asynchronous on it;
 *     the library never synchronises and never allocates device memory in a run.
 *   - Functions returning int give MNN_OK (0) or a negative mnn_status; the reason
 *     is kept in a thread-local string read with mnn_last_error().
 *   - A plan is immutable after creation and may be used from one stream at a
 *     time (its workspace is per plan).  y must not alias x.
 *   - There is no CPU fallback: without a CUDA device runs fail with MNN_ECUDA.
 */
#ifndef MNN_CONV_H_
#define MNN_CONV_H_

#if defined(__GNUC__)
#define MNN_API __attribute__((visibility("default")))
#else
#define MNN_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mnn_conv_plan_s* mnn_conv_plan_t;   /* opaque host object */

typedef enum {
    MNN_OK = 0,
    MNN_EINVAL = -1,         /* argument outside the definition (NULL, non-positive size, ...) */
    MNN_EUNSUPPORTED = -2,   /* valid but not implemented (e.g. forced Winograd with stride 2) */
    MNN_EWORKSPACE = -3,     /* workspace missing or too small */
    MNN_EALIGN = -4,         /* a device pointer is not 16-byte aligned */
    MNN_ECUDA = -5,          /* a CUDA call failed, or a kernel reported a bounded wait that ran out */
    MNN_ENOTCALIBRATED = -6
} mnn_status;

enum { MNN_ALGO_AUTO = 0, MNN_ALGO_WINOGRAD = 1, MNN_ALGO_GEMM = 2, MNN_ALGO_DIRECT = 3 };
enum { MNN_PREC_TF32 = 0, MNN_PREC_BF16 = 1 };             /* accuracy class */
enum { MNN_OPERAND_AUTO = 0, MNN_OPERAND_TF32 = 1, MNN_OPERAND_BF16 = 2, MNN_OPERAND_FP32_REF = 3 };
enum { MNN_POINTS_AUTO = 0, MNN_POINTS_PAPER = 1, MNN_POINTS_UNIT = 2, MNN_POINTS_MIXED = 3 };
enum { MNN_GEMM_LHS_AUTO = 0, MNN_GEMM_LHS_PATCHES = 1, MNN_GEMM_LHS_X = 2, MNN_GEMM_LHS_IMPLICIT = 3 };
enum { MNN_STAGE_WEIGHT = 1, MNN_STAGE_INPUT = 2, MNN_STAGE_CONTRACT = 4, MNN_STAGE_OUTPUT = 8,
       MNN_STAGE_ALL = 15 };

#define MNN_N_CANDIDATES 16
#define MNN_N_CONSTS 16
#define MNN_COST_INADMISSIBLE 0xFFFFFFFFFFFFFFFFull

/*
 * Options of mnn_conv_plan_ex.  Zero-initialise for the defaults of mnn_conv_plan
 * except `relu`, which mnn_conv_plan sets to 1.
 *   groups     any divisor of Cin and Cout (w is [Cout][Cin/groups][k][k]).  1: all schemes; Cin = Cout = groups
 *              (depthwise 3x3, padding 1, stride 1 or 2): the depthwise kernels; every other grouped layer runs the
 *              generic sliding-window kernel.  0 means 1.
 *   relu       0/1: y = max(0, .) after the bias.
 *   precision  accuracy class the result must meet against an exact evaluation:
 *              MNN_PREC_TF32: relative L2 error <= 1e-3; MNN_PREC_BF16: <= 1e-2.
 *   operand    tensor-core operand format of the contraction; AUTO lets the
 *              planner pick any format/pass count admissible for the class.
 *              FP32_REF runs the contraction on CUDA cores in fp32 (a slow
 *              checking path, never chosen by the planner).
 *   passes     0 = planner; 1 = operands rounded once; 3 = each operand split
 *              into hi + lo of the operand format and hi*hi + lo*hi + hi*lo
 *              accumulated (near-fp32 accuracy at 3x the tensor work).
 *   force_algo MNN_ALGO_*; AUTO = planner.
 *   force_m    0 = planner, else the Winograd output tile size m (2..8).
 *   points_id  interpolation point set of the generator (Eq. 8): PAPER = 0, +-1/2,
 *              +-1, ... (the paper's f = 1/2); UNIT = 0, +-1, +-2, ...; MIXED = 0, +-1,
 *              +-1/2, +-2, +-1/4, +-4; AUTO = the set with the lowest predicted error.
 *   chunk_images  0 = planner; else images per pipeline chunk.  The planner cuts the
 *              batch only when the transformed tensors of the whole batch would
 *              exceed 4 GiB.
 *   gemm_lhs   left operand of the GEMM scheme.  PATCHES: the gathered patch matrix
 *              V [N*OH*OW][Cin*k*k] in the operand format.  X: the input itself, read as
 *              the pixel-contiguous matrix [Cin][H*W] of each image (no gather, no V);
 *              only for 1x1 stride-1 unpadded ungrouped layers with H*W >= 32 and a
 *              multiple of 4 and single-pass TF32 operands, where the tensor core drops
 *              the low 13 mantissa bits of x (truncation) instead of a rounded copy being
 *              stored.  IMPLICIT: no patch matrix either, for any k / stride / padding /
 *              dilation: producer warps of the GEMM kernel gather the patches into the
 *              shared-memory operand tile themselves (single-pass TF32 operands, rounded
 *              to nearest).  AUTO = the planner takes the cheapest that applies.  Asking
 *              for X or IMPLICIT where it does not apply fails the plan.
 *   fused      Winograd F(2x2, 3x3) as ONE kernel (input transform, contraction and output
 *              transform fused; the transformed tensors V and M never reach device memory):
 *              0 = the planner weighs it against the other candidates, 1 = never,
 *              2 = this kernel or fail.  It applies to 3x3 stride-1 undilated ungrouped layers with
 *              pad <= 2, accuracy class permitting single-pass TF32 at m = 2.
 *   strassen   1 = run a 1x1 stride-1 unpadded layer's matrix product through ONE recursion level of
 *              Strassen's algorithm (Section 3.3.2): seven half-size products in one batched contraction,
 *              the additions folded into one pass before and one after it.  Needs even N, Cin and Cout.
 *              Unless operand/passes are given, the operands are BF16 hi + lo (3 passes) under the TF32
 *              accuracy class (the sums and differences of products lose about a factor three of
 *              accuracy) and single-pass TF32 under the BF16 class.  0 = plain product (the planner
 *              never chooses Strassen by itself: on this GPU it loses at every size a layer produces).
 */
typedef struct {
    int groups;
    int relu;
    int precision;
    int operand;
    int passes;
    int force_algo;
    int force_m;
    int points_id;
    int chunk_images;
    int gemm_lhs;
    int fused;
    int strassen;
    int reserved[4];
} mnn_conv_opts;

/*
 * What the planner decided (Eq. 1-5 re-stated for this GPU: per candidate
 * cost = sum over its kernels of max(bytes * c_byte, tensor flops * c_tensor,
 * ALU flops * c_alu) + launch cost, in integer picoseconds).
 * cost_ps[] order: 0 DIRECT; 1 GEMM tf32; 2 GEMM bf16; 3..5 Winograd m=2,4,6 tf32x1;
 * 6..8 tf32x3; 9..11 bf16x1; 12..14 bf16x3; 15 Winograd F(2x2,3x3) tf32x1 as one fused kernel.
 * Candidates that are not applicable or fail the accuracy gate hold MNN_COST_INADMISSIBLE; every
 * other figure saturates at MNN_COST_INADMISSIBLE - 1.
 * paper_mul[] is the paper's own multiplication count (Eq. 2) for output tile sizes n = 1, 2, 4, 6,
 * read as a count per tile (so multiplied by the number of tiles) with the output-channel factor
 * its third term lacks as printed; paper_n_hat is its argmin (1 = sliding window, Eq. 3).  It is
 * reported for comparison only and does not enter the choice.
 * Workspace layout (byte offsets from the workspace base, each 1024-aligned):
 *   u_offset  transformed weights  U [alpha^2][Cout][cin_pad]  (operand format; hi then lo when passes = 3)
 *   v_offset  transformed inputs   V [alpha^2][chunk_tiles][cin_pad] of one chunk (same format)
 *   m_offset  contraction results  M [alpha^2][Cout][m_row_stride] fp32 of one chunk
 * For the GEMM scheme alpha = 1, cin_pad covers Cin*k*k and M is unused.
 */
typedef struct {
    int algo, m, alpha, precision, operand, passes, points_id;
    int OH, OW, groups, relu;
    int chunk_images, n_chunks, launches_per_run;
    int cin_pad, m_row_stride;
    long long chunk_tiles;           /* Winograd tiles (or GEMM columns) per full chunk */
    long long workspace_bytes;       /* total the caller must provide (0 for DIRECT) */
    long long u_offset, u_bytes, v_offset, v_bytes, m_offset, m_bytes;
    long long predicted_error_ppm;   /* accuracy model's relative L2 error x 1e6 for the choice */
    int chosen_candidate;            /* index into cost_ps, -1 when the choice was forced outside the list */
    int gemm_lhs;                    /* GEMM scheme: MNN_GEMM_LHS_PATCHES, _X or _IMPLICIT as planned, else 0 */
    unsigned long long cost_ps[MNN_N_CANDIDATES];
    int fused;                       /* 1 when the plan is the single fused Winograd kernel (no V, no M) */
    int paper_n_hat;
    unsigned long long paper_mul[4];
    int strassen;                    /* 1 when the plan runs one Strassen level (alpha = 1, seven products) */
    int rect;                        /* plans of mnn_conv_plan_rect: 1 = kernel 1 x k, 2 = kernel k x 1; else 0 */
} mnn_conv_info;

/* Plan one layer with groups = 1, relu = 1, accuracy class TF32, everything else
 * decided by the planner (Section 3.2 "computation scheme selection").  Host only;
 * needs no GPU.  Returns NULL on error. */
MNN_API mnn_conv_plan_t mnn_conv_plan(int N, int Cin, int Cout, int H, int W, int k,
                              int stride, int pad, int dilation);

/* Same with explicit options (opts may be NULL = all defaults incl. relu = 0). */
MNN_API mnn_conv_plan_t mnn_conv_plan_ex(int N, int Cin, int Cout, int H, int W, int k,
                                 int stride, int pad, int dilation, const mnn_conv_opts* opts);

/* Rectangular kernels 1 x k and k x 1 (the paper's Section 4.2 names the 1 x 7 and 7 x 1 layers of Inception-v3
 * as a case other engines handle badly): w is [Cout][Cin][kh][kw] with kh = 1 or kw = 1 and the other one k in
 * {2, 3, 5, 7}; stride 1, no dilation, one group, padding given per axis; OH = H + 2 pad_h - kh + 1, OW likewise.
 * The layer runs as a ONE-dimensional Winograd F(m, k) along the kernel's long axis (Eq. 6 with the identity on
 * the other axis: alpha = m + k - 1 transform positions) through the same tensor-core contraction.  opts as for
 * mnn_conv_plan_ex (relu, precision, operand, passes, force_m, points_id are read; force_m = 0 takes m = 4,
 * or 2 where m + k - 1 would pass 10; operand AUTO takes BF16 hi + lo under the TF32 accuracy class).
 * The plan is used with the same mnn_conv_* calls as any other; info.alpha is the number of transform positions. */
MNN_API mnn_conv_plan_t mnn_conv_plan_rect(int N, int Cin, int Cout, int H, int W, int kh, int kw, int pad_h, int pad_w,
                                           const mnn_conv_opts* opts);

/* Copy the plan's decisions into *info (host). */
MNN_API int mnn_conv_plan_query(mnn_conv_plan_t plan, mnn_conv_info* info);

/* Hand the plan its device workspace (>= info.workspace_bytes, 1024-byte aligned).
 * The caller keeps ownership and must keep it alive while the plan is used
 * (memory pre-allocation ahead of inference, Section 3.2 "preparation-execution
 * decoupling").  Invalidates prepared weights. */
MNN_API int mnn_conv_set_workspace(mnn_conv_plan_t plan, void* workspace, long long bytes);

/* Transform the weights into the workspace now (U = G w G^T of Eq. 6, or the
 * rounded copy the GEMM scheme uses).  Optional: mnn_conv_run does it on first
 * use of a given w pointer.  Asynchronous on stream. */
MNN_API int mnn_conv_prepare_weights(mnn_conv_plan_t plan, const float* w, void* stream);

/* One forward pass of the layer: y = act(conv(x, w) + bias).  If w differs from
 * the pointer last prepared, the weight transform runs first on the stream. */
MNN_API int mnn_conv_run(mnn_conv_plan_t plan, const float* x, const float* w, const float* bias,
                 float* y, void* stream);

/* The same pass restricted to the stages in stage_mask (MNN_STAGE_*), for checking
 * and timing the stages one by one: INPUT writes V (Eq. 6, B^T X B), CONTRACT reads
 * U, V and writes M (Section 3.3.1 (2): the Hadamard product summed over channels as
 * one matrix product per transform position), OUTPUT reads M and writes y (A^T . A,
 * plus bias and ReLU).  Each selected stage runs for every chunk.  For GEMM plans
 * INPUT is the patch gather and CONTRACT writes y; DIRECT plans have one stage
 * (MNN_STAGE_CONTRACT). */
MNN_API int mnn_conv_run_stages(mnn_conv_plan_t plan, const float* x, const float* w, const float* bias,
                        float* y, void* stream, unsigned stage_mask);

/* Read and clear the device-side status word of the plan (synchronises the
 * stream): 0 = no kernel reported a problem; otherwise a code naming the bounded
 * wait that ran out.  Returns MNN_OK and stores the code in *code. */
MNN_API int mnn_conv_device_status(mnn_conv_plan_t plan, void* stream, int* code);

/* Per-stage device timing.  mnn_conv_profile(plan, 1) makes every later run bracket
 * each of its kernel launches with CUDA events on the run's stream (a small
 * perturbation: keep it off for headline timings); 0 switches it off and frees the
 * events.  mnn_conv_profile_read waits for the events of the LAST run and returns,
 * per stage index (0 weight, 1 input, 2 contraction, 3 output), the summed kernel
 * time in milliseconds and the number of launches.  Host arrays of 4. */
MNN_API int mnn_conv_profile(mnn_conv_plan_t plan, int enable);
MNN_API int mnn_conv_profile_read(mnn_conv_plan_t plan, float stage_ms[4], int stage_launches[4]);

MNN_API void mnn_conv_destroy(mnn_conv_plan_t plan);

/* The same forward pass as mnn_conv_run for callers that have no way to provide a
 * workspace.  (The paper has no counterpart: its engine owns a memory pool.)
 *
 * Who needs it: code that is handed x, w, bias and y by somebody else and is not
 * allowed to create device memory itself -- a plug-in running inside another
 * framework's memory budget, a real-time loop whose rules forbid calls that may
 * block on the driver (cudaMalloc and cudaFree synchronise the device), a process
 * whose allocator is locked after start-up.  For them the library carries its own
 * workspace: a fixed array of MNN_STATIC_WORKSPACE_BYTES that is part of the
 * library image, so every GPU on which the library is loaded holds that much memory
 * until the process exits.
 *
 * The plan is used for its decisions only; its own workspace (if any), prepared
 * weights and profiling state are neither needed nor touched, and
 * mnn_conv_set_workspace need not have been called.  The call makes no cudaMalloc,
 * cudaFree or other allocating call.  The weights are transformed on every call
 * (the array is shared, so nothing can be assumed to survive between calls).
 *
 * Limits and rules:
 *   - plans whose info.workspace_bytes exceed MNN_STATIC_WORKSPACE_BYTES are
 *     rejected with MNN_EWORKSPACE (nothing is launched); plan with a smaller
 *     batch, or a smaller tile size, to fit.
 *   - the first call on each device looks up the array's device address (with
 *     that device current); make that first call outside any stream capture.
 *     The current device must be the device of `stream` in every call.
 *   - every call on a device uses the same array, which keeps the previous
 *     call's contents; the call clears the one word that must start at zero.
 *     Two calls that overlap on the GPU (different streams, or different
 *     threads) race on it: serialise them.
 *   - a bounded wait that runs out inside a kernel is recorded in the array's
 *     status word, which this entry point does not read back.
 * Same argument conventions, asynchrony and return codes as mnn_conv_run. */
#define MNN_STATIC_WORKSPACE_BYTES (32u << 20)
MNN_API int mnn_conv_run_static(mnn_conv_plan_t plan, const float* x, const float* w, const float* bias,
                                float* y, void* stream);

/* Winograd generator (Eq. 8): transform matrices of F(m, k) from the chosen
 * interpolation points plus the point at infinity, computed in exact rational
 * arithmetic and rounded once to fp32.  Host arrays, row-major:
 * At [m][alpha], G [alpha][k], Bt [alpha][alpha], alpha = m + k - 1 <= 16.
 * Any may be NULL.  points_id must not be AUTO. */
MNN_API int mnn_winograd_matrices(int m, int k, int points_id, float* At, float* G, float* Bt);

/* Predicted relative L2 error x 1e6 of Winograd F(m,k) with the given point set,
 * operand format (MNN_OPERAND_TF32/BF16) and passes (1/3): a deterministic host
 * simulation with rounded operands; the planner's accuracy gate.  m = 1 with
 * points_id = 0 gives the figure of the GEMM scheme (no transforms).  < 0 on error. */
MNN_API long long mnn_accuracy_ppm(int m, int k, int points_id, int operand, int passes);

/* The paper's stopping rule for the Strassen recursion (Eq. 9) for a product [n x k] times [k x m]:
 * 1 when m n k - 7 (m/2)(n/2)(k/2) > 4 (m/2)(k/2) + 4 (n/2)(k/2) + 7 (m/2)(n/2), i.e. when the multiplications
 * saved outnumber the additions added, counting both alike; else 0.  Reported for comparison: it weighs a
 * multiplication like an addition, which does not hold where the multiplications run on tensor cores. */
MNN_API int mnn_strassen_rule(long long m, long long n, long long k);

/* Cost-model constants (Eq. 5's FLOPS and t_schedule, re-stated for this GPU).
 * consts[0] attoseconds per HBM byte          consts[1] attoseconds per L2-resident byte
 * consts[2] attoseconds per TF32 tensor flop  consts[3] attoseconds per BF16 tensor flop
 * consts[4] attoseconds per fp32 ALU flop     consts[5] picoseconds of fixed cost per kernel (launch, ramp-up, tail)
 * consts[6] L2 bytes usable for one chunk     consts[7] number of SMs
 * consts[8] attoseconds per flop of the direct kernel
 * consts[9] attoseconds per flop of the direct kernel for layers with at most 4 input channels
 *            (measured on 3 -> 32, 3x3, stride 2, padding 1, which has a kernel of its own; the other shapes
 *            with at most 4 input channels are booked at twice this figure)
 *           (0 = use consts[8])
 * consts[10] attoseconds per byte of transformed weights delivered from L2 to ONE SM (fused Winograd kernel)
 * consts[11] picoseconds the fused kernel's tensor work takes per block of 32 input channels of one work item
 * consts[12] picoseconds of epilogue per work item of the fused kernel
 *            (consts[10] or [11] = 0: the fused kernel is never chosen by the planner)
 * consts[13] attoseconds per patch element gathered by the implicit GEMM's producer warps, per SM
 *            (0 = the planner never takes the implicit left operand by itself)
 * consts[14..15] reserved (0).
 * mnn_calibrate measures them on the current device (launches micro-benchmarks and
 * synchronises; allocates and frees its own scratch) and installs them;
 * mnn_set_calibration installs a frozen record so that plans are reproducible;
 * mnn_get_calibration reads the record in force (built-in defaults if none was set). */
MNN_API int mnn_calibrate(int device, void* stream, long long consts[MNN_N_CONSTS]);
MNN_API int mnn_set_calibration(const long long consts[MNN_N_CONSTS]);
MNN_API int mnn_get_calibration(long long consts[MNN_N_CONSTS]);

/*
 * Network-level pre-inference (Section 3.2, "preparation-execution decoupling": the
 * engine walks the graph once, decides every scheme and lays out all memory before the
 * first inference).  A network here is a sequential stack of convolution layers on one
 * input of shape [N][layers[0].Cin][H][W]; layer i consumes layer i-1's output.
 *
 * mnn_net_plan plans every layer (same options as mnn_conv_plan_ex: accuracy class
 * `precision`; groups / relu per layer) and lays out ONE workspace by a virtual walk:
 *   - a persistent part per layer (status word and transformed weights U),
 *   - one transient part shared by all layers (V and M of the largest layer),
 *   - two activation buffers used in turn, each as large as the largest intermediate tensor.
 * mnn_net_query reports the layout and each layer's plan; mnn_net_set_workspace hands over
 * the caller-owned workspace (1024-byte aligned, >= info.workspace_bytes);
 * mnn_net_prepare transforms all weights; mnn_net_run enqueues the whole forward pass
 * on `stream` (x -> y; w[i], bias[i] are the layers' device tensors, bias[i] may be NULL)
 * with no allocation, no synchronisation and no host work beyond the kernel launches, so
 * that it can also be recorded once (e.g. into a CUDA graph) and replayed.
 * Layers run in order on one stream: the shared transient part is safe by stream order.
 */
typedef struct mnn_net_s* mnn_net_t;

typedef struct {
    int Cin, Cout, k, stride, pad, dilation;
    int groups;        /* 0 or 1, Cin (= Cout) for depthwise, or any divisor of Cin and Cout */
    int relu;
} mnn_layer_desc;

#define MNN_NET_MAX_LAYERS 128
typedef struct {
    int n_layers;
    int N, H, W;                       /* input */
    int out_C, out_H, out_W;           /* output of the last layer */
    int launches_per_run;
    long long workspace_bytes;         /* total the caller must provide */
    long long persistent_bytes, transient_bytes, activation_bytes;   /* activation_bytes = one of the two buffers */
    long long sum_of_layer_workspaces; /* what per-layer workspaces would need without sharing */
    int algo[MNN_NET_MAX_LAYERS], m[MNN_NET_MAX_LAYERS], operand[MNN_NET_MAX_LAYERS], passes[MNN_NET_MAX_LAYERS];
    int OH[MNN_NET_MAX_LAYERS], OW[MNN_NET_MAX_LAYERS];
} mnn_net_info;

MNN_API mnn_net_t mnn_net_plan(int N, int H, int W, int n_layers, const mnn_layer_desc* layers, int precision);
MNN_API int mnn_net_query(mnn_net_t net, mnn_net_info* info);
MNN_API int mnn_net_set_workspace(mnn_net_t net, void* workspace, long long bytes);
MNN_API int mnn_net_prepare(mnn_net_t net, const float* const* w, void* stream);
MNN_API int mnn_net_run(mnn_net_t net, const float* x, const float* const* w, const float* const* bias, float* y,
                        void* stream);
/* Reads and clears the status words of all layers (synchronises the stream); *code gets the first
 * non-zero code, *layer its index (-1 if none). */
MNN_API int mnn_net_device_status(mnn_net_t net, void* stream, int* code, int* layer);
MNN_API void mnn_net_destroy(mnn_net_t net);

/* Self-test of the bounded waits every persistent kernel of the library relies on (no counterpart in the paper).
 * Launches one tiny kernel on `stream` that initialises a shared-memory barrier nobody ever arrives on and waits
 * on it with the library's bounded wait; the wait gives up after its limit (about one second) and the
 * kernel returns normally.  `device_word` (device memory, 4 bytes, caller-owned) receives 1 when the kernel has
 * started, then 2 when the wait gave up as it must, or 3 if it reported completion.  Asynchronous; no fault, trap
 * or endless loop is involved, and the context stays usable. */
MNN_API int mnn_wait_probe(int* device_word, void* stream);

MNN_API const char* mnn_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* MNN_CONV_H_ */
