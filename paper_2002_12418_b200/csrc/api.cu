// C ABI of the library: plan objects, run entry points, generator and planner access.
#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "../../include/mnn_conv.h"
#include "generator.h"
#include "implicit_gemm.h"
#include "contract_pair.h"
#include "contract_umma.h"
#include "kernels.h"
#include "planner.h"
#include "strassen.h"
#include "wino_fused.h"
#include "wino_rect.h"

using namespace mnnb;

namespace {

thread_local std::string g_last_error;

int fail(int code, const std::string& why)
{
    g_last_error = why;
    return code;
}

int fail_cuda(cudaError_t e, const char* where)
{
    g_last_error = std::string(where) + ": " + cudaGetErrorString(e);
    return MNN_ECUDA;
}

long long align_up(long long v, long long a) { return (v + a - 1) / a * a; }

constexpr long long kStatusBytes = 1024;   // head of the workspace: device status word

}  // namespace

struct mnn_conv_plan_s {
    LayerShape s;
    mnn_conv_opts o;
    Decision d;
    int store_mode = STORE_TF32;
    int cin_pad = 0;                 // row length of U and V (Winograd: padded Cin; GEMM: padded Cin*k*k)
    long long chunk_tiles = 0;       // capacity of V / M in tiles (or GEMM columns)
    int m_row_stride = 0;
    long long u_offset = 0, u_bytes = 0, v_offset = 0, v_bytes = 0, m_offset = 0, m_bytes = 0, workspace_bytes = 0;
    int launches_per_run = 1;
    bool gemm_x = false;             // GEMM scheme with x itself as the left operand: no V, one launch
    bool gemm_implicit = false;      // GEMM scheme with the patches gathered inside the GEMM kernel: no V, one launch
    ImplicitGemm ig;
    TransformMatrices mats;
    // run-time state
    char* ws = nullptr;              // status word and U (persistent part), and V, M unless tws is set
    char* tws = nullptr;             // optional separate transient part: V at tws, M at tws + (m_offset - v_offset)
    long long ws_bytes = 0;
    const float* prepared_w = nullptr;
    UmmaContract uc;
    PairContract pc;           // the Winograd contraction on pairs of SMs, when use_pair
    bool use_pair = false;
    bool strassen = false;           // GEMM scheme through one Strassen level: seven half-size products
    int rect = 0;                    // 1: kernel 1 x k, 2: kernel k x 1 (one-dimensional Winograd along the long axis)
    int pad_h = 0, pad_w = 0;        // rectangular plans: padding per axis (s.pad is unused there)
    bool fused = false;              // Winograd F(2x2,3x3) as the single fused kernel: the workspace holds U only
    FusedWino fw;
    // optional per-launch timing
    bool profiling = false;
    std::vector<cudaEvent_t> events;     // pairs (before, after)
    std::vector<int> event_stage;        // stage index of each pair used by the last run
};

namespace {

void* u_hi(mnn_conv_plan_t p) { return p->ws + p->u_offset; }
void* u_lo(mnn_conv_plan_t p) { return store_is_split(p->store_mode) ? p->ws + p->u_offset + p->u_bytes / 2 : nullptr; }
char* transient_base(mnn_conv_plan_t p) { return p->tws ? p->tws - p->v_offset : p->ws; }
void* v_hi(mnn_conv_plan_t p) { return transient_base(p) + p->v_offset; }
void* v_lo(mnn_conv_plan_t p)
{
    return store_is_split(p->store_mode) ? transient_base(p) + p->v_offset + p->v_bytes / 2 : nullptr;
}
float* m_buf(mnn_conv_plan_t p) { return reinterpret_cast<float*>(transient_base(p) + p->m_offset); }
int* status_word(mnn_conv_plan_t p) { return reinterpret_cast<int*>(p->ws); }

int store_mode_of(int operand, int passes)
{
    if (operand == MNN_OPERAND_FP32_REF) return STORE_FP32;
    if (operand == MNN_OPERAND_BF16) return passes == 3 ? STORE_BF16_SPLIT : STORE_BF16;
    return passes == 3 ? STORE_TF32_SPLIT : STORE_TF32;
}

void layout_workspace(mnn_conv_plan_t p)
{
    const LayerShape& s = p->s;
    const Decision& d = p->d;
    p->store_mode = store_mode_of(d.operand, d.passes);
    const long long eb = store_elem_bytes(p->store_mode) * (store_is_split(p->store_mode) ? 2 : 1);
    if (d.algo == MNN_ALGO_DIRECT) {
        p->workspace_bytes = 0;
        p->launches_per_run = 1;
        return;
    }
    long long off = kStatusBytes;
    if (p->rect) {
        const long long n_seg = p->rect == 1 ? (s.OW + d.m - 1) / d.m : (s.OH + d.m - 1) / d.m;
        p->cin_pad = (int)align_up(s.Cin, 8);
        p->chunk_tiles = p->rect == 1 ? (long long)s.N * s.OH * n_seg : (long long)s.N * n_seg * s.OW;
        p->m_row_stride = (int)align_up(p->chunk_tiles, 32);
        p->u_bytes = align_up((long long)d.alpha * s.Cout * p->cin_pad * eb, 2048);
        p->v_bytes = align_up((long long)d.alpha * p->chunk_tiles * p->cin_pad * eb, 2048);
        p->m_bytes = align_up((long long)d.alpha * s.Cout * p->m_row_stride * 4, 1024);
        p->launches_per_run = 3;
    } else if (d.algo == MNN_ALGO_WINOGRAD) {
        const long long a2 = (long long)d.alpha * d.alpha;
        const long long th = (s.OH + d.m - 1) / d.m, tw = (s.OW + d.m - 1) / d.m;
        p->cin_pad = (int)align_up(s.Cin, 8);
        p->chunk_tiles = (long long)d.chunk_images * th * tw;
        p->m_row_stride = (int)align_up(p->chunk_tiles, 32);
        p->fused = d.fused != 0;
        p->u_bytes = p->fused ? align_up(fused_wino_weight_bytes(s.Cout, s.Cin), 2048) : align_up(a2 * s.Cout * p->cin_pad * eb, 2048);
        p->v_bytes = p->fused ? 0 : align_up(a2 * p->chunk_tiles * p->cin_pad * eb, 2048);
        p->m_bytes = p->fused ? 0 : align_up(a2 * s.Cout * p->m_row_stride * 4, 1024);
        p->launches_per_run = p->fused ? 1 : 3 * d.n_chunks;
    } else if (p->strassen) {
        const long long Mh = s.Cout / 2;
        p->cin_pad = (int)align_up(s.Cin / 2, 8);
        p->chunk_tiles = (long long)(s.N / 2) * s.OH * s.OW;
        p->m_row_stride = (int)align_up(p->chunk_tiles, 32);
        p->u_bytes = align_up(7 * Mh * p->cin_pad * eb, 2048);
        p->v_bytes = align_up(7 * p->chunk_tiles * p->cin_pad * eb, 2048);
        p->m_bytes = align_up(7 * Mh * p->m_row_stride * 4, 1024);
        p->launches_per_run = 3;
    } else {
        p->cin_pad = (int)align_up((long long)s.Cin * s.k * s.k, 8);
        p->chunk_tiles = (long long)s.N * s.OH * s.OW;
        p->m_row_stride = 0;
        p->u_bytes = align_up((long long)s.Cout * p->cin_pad * eb, 2048);
        p->gemm_x = d.gemm_lhs == MNN_GEMM_LHS_X;
        p->gemm_implicit = d.gemm_lhs == MNN_GEMM_LHS_IMPLICIT;
        const bool no_v = p->gemm_x || p->gemm_implicit;
        p->v_bytes = no_v ? 0 : align_up(p->chunk_tiles * p->cin_pad * eb, 2048);
        p->m_bytes = 0;
        p->launches_per_run = no_v ? 1 : 2;
    }
    p->u_offset = off;
    off += p->u_bytes;
    p->v_offset = off;
    off += p->v_bytes;
    p->m_offset = off;
    off += p->m_bytes;
    p->workspace_bytes = off;
}

bool aligned16(const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15u) == 0; }

// Brackets one launch with events when profiling is on.
struct LaunchTimer {
    mnn_conv_plan_t p;
    cudaStream_t st;
    int slot = -1;
    LaunchTimer(mnn_conv_plan_t plan, cudaStream_t stream, int stage) : p(plan), st(stream)
    {
        if (!p->profiling) return;
        const size_t used = p->event_stage.size();
        if (2 * used + 1 >= p->events.size()) return;
        slot = (int)used;
        p->event_stage.push_back(stage);
        cudaEventRecord(p->events[2 * slot], st);
    }
    ~LaunchTimer()
    {
        if (slot >= 0) cudaEventRecord(p->events[2 * slot + 1], st);
    }
};

void free_events(mnn_conv_plan_t p)
{
    for (cudaEvent_t e : p->events) cudaEventDestroy(e);
    p->events.clear();
    p->event_stage.clear();
}

}  // namespace

extern "C" {

const char* mnn_last_error(void) { return g_last_error.c_str(); }

mnn_conv_plan_t mnn_conv_plan_ex(int N, int Cin, int Cout, int H, int W, int k, int stride, int pad, int dilation,
                                 const mnn_conv_opts* opts)
{
    mnn_conv_opts o;
    std::memset(&o, 0, sizeof(o));
    if (opts) o = *opts;
    if (o.groups == 0) o.groups = 1;
    if (N <= 0 || Cin <= 0 || Cout <= 0 || H <= 0 || W <= 0 || k <= 0 || stride <= 0 || pad < 0 || dilation <= 0) {
        fail(MNN_EINVAL, "sizes, k, stride and dilation must be positive and pad non-negative");
        return nullptr;
    }
    if (o.groups < 1 || Cin % o.groups || Cout % o.groups) {
        fail(MNN_EINVAL, "groups must divide Cin and Cout");
        return nullptr;
    }
    if (o.precision != MNN_PREC_TF32 && o.precision != MNN_PREC_BF16) {
        fail(MNN_EINVAL, "precision must be MNN_PREC_TF32 or MNN_PREC_BF16");
        return nullptr;
    }
    if (o.operand < 0 || o.operand > MNN_OPERAND_FP32_REF || !(o.passes == 0 || o.passes == 1 || o.passes == 3) ||
        o.force_algo < 0 || o.force_algo > MNN_ALGO_DIRECT || o.points_id < 0 || o.points_id > MNN_POINTS_MIXED ||
        o.force_m < 0 || o.chunk_images < 0 || o.gemm_lhs < 0 || o.gemm_lhs > MNN_GEMM_LHS_IMPLICIT || o.fused < 0 || o.fused > 2 || o.strassen < 0 || o.strassen > 1) {
        fail(MNN_EINVAL, "an option is outside its range");
        return nullptr;
    }
    if (k > 11) {
        fail(MNN_EUNSUPPORTED, "kernel sizes above 11 are not supported");
        return nullptr;
    }
    LayerShape s;
    s.N = N; s.Cin = Cin; s.Cout = Cout; s.H = H; s.W = W; s.k = k; s.stride = stride; s.pad = pad; s.dil = dilation;
    s.groups = o.groups; s.relu = o.relu ? 1 : 0;
    s.OH = conv_out_extent(H, k, stride, pad, dilation);
    s.OW = conv_out_extent(W, k, stride, pad, dilation);
    if (s.OH <= 0 || s.OW <= 0) {
        fail(MNN_EINVAL, "the dilated kernel does not fit the padded input");
        return nullptr;
    }
    if ((long long)N * Cin * H * W >= (1ll << 40) || (long long)N * Cout * s.OH * s.OW >= (1ll << 40)) {
        fail(MNN_EUNSUPPORTED, "tensor too large");
        return nullptr;
    }
    if (o.strassen) {
        if (!strassen_applies(N, Cin, Cout, k, stride, pad, dilation, o.groups) || o.force_algo == MNN_ALGO_WINOGRAD ||
            o.force_algo == MNN_ALGO_DIRECT || o.operand == MNN_OPERAND_FP32_REF || o.gemm_lhs == MNN_GEMM_LHS_X || o.gemm_lhs == MNN_GEMM_LHS_IMPLICIT) {
            fail(MNN_EUNSUPPORTED, "Strassen needs a 1x1 stride-1 unpadded ungrouped layer with even N, Cin and Cout on the GEMM scheme");
            return nullptr;
        }
        // the sums and differences of the seven products lose about a factor three of accuracy
        o.force_algo = MNN_ALGO_GEMM;
        o.gemm_lhs = MNN_GEMM_LHS_PATCHES;
        if (o.operand == MNN_OPERAND_AUTO) {
            o.operand = o.precision == MNN_PREC_TF32 ? MNN_OPERAND_BF16 : MNN_OPERAND_TF32;
            o.passes = o.precision == MNN_PREC_TF32 ? 3 : 1;
        } else if (o.passes == 0) {
            o.passes = 1;
        }
    }
    mnn_conv_plan_t p = new (std::nothrow) mnn_conv_plan_s();
    if (!p) {
        fail(MNN_EINVAL, "out of host memory");
        return nullptr;
    }
    p->s = s;
    p->o = o;
    p->strassen = o.strassen != 0;
    const char* why = "";
    mnn_conv_opts o_plan = o;
    if (p->strassen) o_plan.passes = 1;      // the candidate list holds single-pass GEMMs; the pass count is set below
    int rc = plan_layer(s, o_plan, current_calibration(), &p->d, &why);
    if (rc != MNN_OK) {
        fail(rc, why);
        delete p;
        return nullptr;
    }
    if (p->strassen) {
        p->d.passes = o.passes;
        p->d.chosen = -1;
        p->d.gemm_lhs = MNN_GEMM_LHS_PATCHES;
        p->d.error_ppm = accuracy_ppm(1, 1, 0, p->d.operand, p->d.passes);
    }
    if (p->d.algo == MNN_ALGO_WINOGRAD) {
        WinogradMatrices wm;
        if (!generate_winograd(p->d.m, k, p->d.points_id, &wm) || p->d.alpha > 12 || p->d.m > 6 || k > 7) {
            fail(MNN_EUNSUPPORTED, "no transform matrices for this (m, k, points)");
            delete p;
            return nullptr;
        }
        std::memset(&p->mats, 0, sizeof(p->mats));
        std::memcpy(p->mats.At, wm.At32.data(), wm.At32.size() * sizeof(float));
        std::memcpy(p->mats.G, wm.G32.data(), wm.G32.size() * sizeof(float));
        std::memcpy(p->mats.Bt, wm.Bt32.data(), wm.Bt32.size() * sizeof(float));
    }
    layout_workspace(p);
    return p;
}

mnn_conv_plan_t mnn_conv_plan_rect(int N, int Cin, int Cout, int H, int W, int kh, int kw, int pad_h, int pad_w,
                                   const mnn_conv_opts* opts)
{
    mnn_conv_opts o;
    std::memset(&o, 0, sizeof(o));
    if (opts) o = *opts;
    if (N <= 0 || Cin <= 0 || Cout <= 0 || H <= 0 || W <= 0 || kh <= 0 || kw <= 0 || pad_h < 0 || pad_w < 0) {
        fail(MNN_EINVAL, "sizes must be positive and paddings non-negative");
        return nullptr;
    }
    const int k = kh > kw ? kh : kw;
    if ((kh != 1 && kw != 1) || k == 1 || !(k == 2 || k == 3 || k == 5 || k == 7) || (o.groups != 0 && o.groups != 1)) {
        fail(MNN_EUNSUPPORTED, "rectangular plans take 1 x k or k x 1 kernels with k in {2,3,5,7} and one group; "
                               "square kernels go through mnn_conv_plan_ex");
        return nullptr;
    }
    if (o.precision != MNN_PREC_TF32 && o.precision != MNN_PREC_BF16) {
        fail(MNN_EINVAL, "precision must be MNN_PREC_TF32 or MNN_PREC_BF16");
        return nullptr;
    }
    const int OH = H + 2 * pad_h - kh + 1, OW = W + 2 * pad_w - kw + 1;
    if (OH <= 0 || OW <= 0) {
        fail(MNN_EINVAL, "the kernel does not fit the padded input");
        return nullptr;
    }
    int m = o.force_m ? o.force_m : (4 + k - 1 <= kRectMaxAlpha ? 4 : 2);
    if (!(m == 2 || m == 4 || m == 6) || m + k - 1 > kRectMaxAlpha) {
        fail(MNN_EUNSUPPORTED, "rectangular plans take m in {2,4,6} with m + k - 1 <= 10");
        return nullptr;
    }
    if (o.operand == MNN_OPERAND_FP32_REF || o.operand < 0 || o.operand > MNN_OPERAND_FP32_REF ||
        !(o.passes == 0 || o.passes == 1 || o.passes == 3) || o.points_id < 0 || o.points_id > MNN_POINTS_MIXED) {
        fail(MNN_EINVAL, "an option is outside its range");
        return nullptr;
    }
    // The accuracy model is the two-dimensional one (an upper bound for one dimension): single-pass operands where
    // it admits them for the class, else the hi + lo split.
    const long long gate = (o.precision == MNN_PREC_BF16 ? 10000 : 1000) * kGateNumerator / kGateDenominator;
    int operand = o.operand, passes = o.passes;
    if (operand == MNN_OPERAND_AUTO) {
        operand = MNN_OPERAND_BF16;
        if (passes == 0) {
            long long ppm1 = 0;
            best_points(m, k, operand, 1, &ppm1);
            passes = (ppm1 >= 0 && ppm1 <= gate) ? 1 : 3;
        }
    } else if (passes == 0) {
        passes = 1;
    }
    long long ppm = 0;
    const int pid = o.points_id ? o.points_id : best_points(m, k, operand, passes, &ppm);
    if (o.points_id) ppm = accuracy_ppm(m, k, pid, operand, passes);
    WinogradMatrices wm;
    if (pid == 0 || !generate_winograd(m, k, pid, &wm)) {
        fail(MNN_EUNSUPPORTED, "no transform matrices for this (m, k, points)");
        return nullptr;
    }
    mnn_conv_plan_t p = new (std::nothrow) mnn_conv_plan_s();
    if (!p) {
        fail(MNN_EINVAL, "out of host memory");
        return nullptr;
    }
    LayerShape s;
    s.N = N; s.Cin = Cin; s.Cout = Cout; s.H = H; s.W = W; s.k = k; s.stride = 1; s.pad = 0; s.dil = 1;
    s.groups = 1; s.relu = o.relu ? 1 : 0; s.OH = OH; s.OW = OW;
    o.groups = 1;
    p->s = s;
    p->o = o;
    p->rect = kh == 1 ? 1 : 2;
    p->pad_h = pad_h;
    p->pad_w = pad_w;
    for (int i = 0; i < MNN_N_CANDIDATES; ++i) p->d.cost_ps[i] = MNN_COST_INADMISSIBLE;
    p->d.algo = MNN_ALGO_WINOGRAD;
    p->d.m = m;
    p->d.alpha = m + k - 1;
    p->d.operand = operand;
    p->d.passes = passes;
    p->d.points_id = pid;
    p->d.chunk_images = N;
    p->d.n_chunks = 1;
    p->d.chosen = -1;
    p->d.error_ppm = ppm;
    std::memset(&p->mats, 0, sizeof(p->mats));
    std::memcpy(p->mats.At, wm.At32.data(), wm.At32.size() * sizeof(float));
    std::memcpy(p->mats.G, wm.G32.data(), wm.G32.size() * sizeof(float));
    std::memcpy(p->mats.Bt, wm.Bt32.data(), wm.Bt32.size() * sizeof(float));
    layout_workspace(p);
    if (p->v_bytes + p->m_bytes > (4ll << 30) || (long long)N * Cin * H * W >= (1ll << 40) ||
        (long long)N * Cout * OH * OW >= (1ll << 40)) {
        fail(MNN_EUNSUPPORTED, "layer too large for one pass of the rectangular path: split the batch");
        delete p;
        return nullptr;
    }
    return p;
}

mnn_conv_plan_t mnn_conv_plan(int N, int Cin, int Cout, int H, int W, int k, int stride, int pad, int dilation)
{
    mnn_conv_opts o;
    std::memset(&o, 0, sizeof(o));
    o.groups = 1;
    o.relu = 1;
    o.precision = MNN_PREC_TF32;
    return mnn_conv_plan_ex(N, Cin, Cout, H, W, k, stride, pad, dilation, &o);
}

int mnn_conv_plan_query(mnn_conv_plan_t p, mnn_conv_info* info)
{
    if (!p || !info) return fail(MNN_EINVAL, "NULL plan or info");
    std::memset(info, 0, sizeof(*info));
    info->algo = p->d.algo;
    info->m = p->d.m;
    info->alpha = p->d.alpha;
    info->precision = p->o.precision;
    info->operand = p->d.operand;
    info->passes = p->d.passes;
    info->points_id = p->d.points_id;
    info->OH = p->s.OH;
    info->OW = p->s.OW;
    info->groups = p->s.groups;
    info->relu = p->s.relu;
    info->chunk_images = p->d.chunk_images;
    info->n_chunks = p->d.n_chunks;
    info->launches_per_run = p->launches_per_run;
    info->cin_pad = p->cin_pad;
    info->m_row_stride = p->m_row_stride;
    info->chunk_tiles = p->chunk_tiles;
    info->workspace_bytes = p->workspace_bytes;
    info->u_offset = p->u_offset;
    info->u_bytes = p->u_bytes;
    info->v_offset = p->v_offset;
    info->v_bytes = p->v_bytes;
    info->m_offset = p->m_offset;
    info->m_bytes = p->m_bytes;
    info->predicted_error_ppm = p->d.error_ppm;
    info->chosen_candidate = p->d.chosen;
    info->gemm_lhs = p->d.algo == MNN_ALGO_GEMM ? p->d.gemm_lhs : 0;
    for (int i = 0; i < MNN_N_CANDIDATES; ++i) info->cost_ps[i] = p->d.cost_ps[i];
    info->fused = p->fused ? 1 : 0;
    info->strassen = p->strassen ? 1 : 0;
    info->rect = p->rect;
    if (p->strassen) info->predicted_error_ppm = 3 * p->d.error_ppm;
    info->paper_n_hat = p->d.paper_n_hat;
    for (int i = 0; i < 4; ++i) info->paper_mul[i] = p->d.paper_mul[i];
    return MNN_OK;
}

// Whether the Winograd contraction of a layer runs on pairs of SMs (256 tiles x 256 channels per work item): at least 256
// output channels and at least two work items per SM pair, so that the coarser items still fill the machine.
// MNN_CONV_PAIR=0 in the environment keeps the single-SM kernel (for comparisons).
static bool pair_contraction_wanted(int Cout, long long tiles, int alpha2)
{
    static const bool off = [] {
        const char* v = std::getenv("MNN_CONV_PAIR");
        return v && v[0] == '0';
    }();
    if (off || Cout < 256) return false;     // narrower layers measured slower on pairs (128 channels: 44 -> 63 us)
    const long long items = ((tiles + 255) / 256) * ((Cout + 255) / 256) * alpha2;
    return items >= 148;
}

// Tensor maps and launch parameters of the plan's tensor-core kernel for the workspace now in p->ws / p->tws.
static cudaError_t setup_tensor_kernels(mnn_conv_plan_t p, const char** why)
{
    const int alpha2 = p->d.algo == MNN_ALGO_WINOGRAD ? p->d.alpha * p->d.alpha : 1;
    if (p->fused) return fused_wino_setup(&p->fw, p->s.Cout, p->s.Cin, u_hi(p), why);
    if (p->rect)
        return umma_contract_setup(&p->uc, p->store_mode, p->d.alpha, p->s.Cout, p->cin_pad, p->chunk_tiles, u_hi(p), u_lo(p),
                                   v_hi(p), v_lo(p), why);
    if (p->strassen)
        return umma_contract_setup(&p->uc, p->store_mode, 7, p->s.Cout / 2, p->cin_pad, p->chunk_tiles, u_hi(p), u_lo(p), v_hi(p),
                                   v_lo(p), why);
    if (p->gemm_implicit) {
        const LayerShape& s = p->s;
        GatherGeom g = {s.N, s.Cin, s.H, s.W, s.OH, s.OW, s.k, s.stride, s.pad, s.dil, p->cin_pad};
        return implicit_gemm_setup(&p->ig, g, s.Cout, u_hi(p), why);
    }
    if (p->gemm_x) return umma_contract_setup_x(&p->uc, p->s.Cout, p->s.Cin, p->cin_pad, p->s.N, p->s.H * p->s.W, u_hi(p), why);
    cudaError_t e = umma_contract_setup(&p->uc, p->store_mode, alpha2, p->s.Cout, p->cin_pad, p->chunk_tiles, u_hi(p), u_lo(p),
                                        v_hi(p), v_lo(p), why);
    p->use_pair = false;
    if (e == cudaSuccess && alpha2 > 1 && pair_contraction_wanted(p->s.Cout, p->chunk_tiles, alpha2)) {
        const char* why_not = nullptr;
        if (pair_contract_setup(&p->pc, p->store_mode, alpha2, p->s.Cout, p->cin_pad, p->chunk_tiles, u_hi(p), u_lo(p), v_hi(p),
                                v_lo(p), &why_not) == cudaSuccess)
            p->use_pair = true;
    }
    return e;
}

// Workspace in two parts (used by the network plan): `persistent` holds the status word and U
// (the first v_offset bytes of the single-workspace layout), `transient` holds V and M and may be shared
// with other plans that run on the same stream.
static int set_workspace_split(mnn_conv_plan_t p, void* persistent, long long persistent_bytes, void* transient,
                               long long transient_bytes);

int mnn_conv_set_workspace(mnn_conv_plan_t p, void* workspace, long long bytes)
{
    if (!p) return fail(MNN_EINVAL, "NULL plan");
    if (p->workspace_bytes == 0) {
        p->prepared_w = nullptr;
        p->uc.ready = false;
        p->ws = p->tws = nullptr;
        p->ws_bytes = 0;
        return MNN_OK;
    }
    if (!workspace) {
        p->ws = p->tws = nullptr;
        return fail(MNN_EWORKSPACE, "this plan needs a workspace");
    }
    if (bytes < p->workspace_bytes) {
        p->ws = p->tws = nullptr;
        return fail(MNN_EWORKSPACE, "workspace smaller than info.workspace_bytes");
    }
    return set_workspace_split(p, workspace, bytes, nullptr, 0);
}

static int set_workspace_split(mnn_conv_plan_t p, void* persistent, long long persistent_bytes, void* transient,
                               long long transient_bytes)
{
    p->prepared_w = nullptr;
    p->uc.ready = false;
    p->ws = p->tws = nullptr;
    p->ws_bytes = 0;
    if (p->workspace_bytes == 0) return MNN_OK;
    void* workspace = persistent;
    long long bytes = persistent_bytes;
    if (!persistent) return fail(MNN_EWORKSPACE, "this plan needs a workspace");
    if (transient) {
        if (persistent_bytes < p->v_offset || transient_bytes < p->workspace_bytes - p->v_offset)
            return fail(MNN_EWORKSPACE, "workspace part too small");
        if (reinterpret_cast<uintptr_t>(transient) & 1023u) return fail(MNN_EALIGN, "workspace must be 1024-byte aligned");
    }
    if (reinterpret_cast<uintptr_t>(workspace) & 1023u) return fail(MNN_EALIGN, "workspace must be 1024-byte aligned");
    p->ws = static_cast<char*>(workspace);
    p->tws = static_cast<char*>(transient);
    p->ws_bytes = bytes;
    cudaError_t e = cudaMemset(p->ws, 0, kStatusBytes);
    if (e != cudaSuccess) return fail_cuda(e, "clearing the status word");
    if (p->d.operand != MNN_OPERAND_FP32_REF) {
        const char* why = "";
        e = setup_tensor_kernels(p, &why);
        if (e != cudaSuccess) {
            p->ws = nullptr;
            return fail(MNN_ECUDA, std::string("tensor-core contraction setup: ") + why + " (" + cudaGetErrorString(e) + ")");
        }
    }
    return MNN_OK;
}

static int check_run_args(mnn_conv_plan_t p, const float* x, const float* w, const float* y, unsigned mask)
{
    if (!p) return fail(MNN_EINVAL, "NULL plan");
    if ((mask & ~(unsigned)MNN_STAGE_ALL) || mask == 0) return fail(MNN_EINVAL, "bad stage mask");
    if (p->workspace_bytes > 0 && !p->ws) return fail(MNN_EWORKSPACE, "call mnn_conv_set_workspace first");
    const bool direct = p->d.algo == MNN_ALGO_DIRECT;
    const bool one_kernel = p->gemm_x || p->gemm_implicit || p->fused;       // x in, y out in the contraction stage
    const bool need_x = direct || (!one_kernel && (mask & MNN_STAGE_INPUT)) || (one_kernel && (mask & MNN_STAGE_CONTRACT));
    const bool need_w = direct || (mask & MNN_STAGE_WEIGHT);
    const bool need_y = direct || (!p->fused && (mask & MNN_STAGE_OUTPUT)) ||
                        (((p->d.algo == MNN_ALGO_GEMM && !p->strassen) || p->fused) && (mask & MNN_STAGE_CONTRACT));
    if ((need_x && !x) || (need_w && !w) || (need_y && !y)) return fail(MNN_EINVAL, "NULL tensor pointer");
    if ((x && !aligned16(x)) || (w && !aligned16(w)) || (y && !aligned16(y)))
        return fail(MNN_EALIGN, "x, w and y must be 16-byte aligned");
    if (x && y) {
        // the tensors may not overlap anywhere: a kernel reads x while another block already writes y
        const uintptr_t x0 = reinterpret_cast<uintptr_t>(x), y0 = reinterpret_cast<uintptr_t>(y);
        const uintptr_t x1 = x0 + 4ull * p->s.N * p->s.Cin * p->s.H * p->s.W;
        const uintptr_t y1 = y0 + 4ull * p->s.N * p->s.Cout * p->s.OH * p->s.OW;
        if (x0 < y1 && y0 < x1) return fail(MNN_EINVAL, "y must not overlap x");
    }
    return MNN_OK;
}

static StrassenGeom strassen_geom(mnn_conv_plan_t p)
{
    StrassenGeom g;
    g.N = p->s.N; g.Cin = p->s.Cin; g.Cout = p->s.Cout; g.HW = p->s.H * p->s.W;
    g.k_pad = p->cin_pad;
    g.t_half = p->chunk_tiles;
    g.m_row_stride = p->m_row_stride;
    return g;
}

static RectGeom rect_geom(mnn_conv_plan_t p)
{
    RectGeom g;
    g.N = p->s.N; g.Cin = p->s.Cin; g.Cout = p->s.Cout; g.H = p->s.H; g.W = p->s.W; g.OH = p->s.OH; g.OW = p->s.OW;
    g.k = p->s.k; g.along_w = p->rect == 1 ? 1 : 0; g.pad_h = p->pad_h; g.pad_w = p->pad_w;
    g.m = p->d.m; g.alpha = p->d.alpha;
    g.n_seg = p->rect == 1 ? (p->s.OW + g.m - 1) / g.m : (p->s.OH + g.m - 1) / g.m;
    g.cin_pad = p->cin_pad;
    g.tiles = p->chunk_tiles;
    g.m_row_stride = p->m_row_stride;
    return g;
}

static int do_weights(mnn_conv_plan_t p, const float* w, cudaStream_t st)
{
    cudaError_t e;
    LaunchTimer lt(p, st, 0);
    if (p->gemm_implicit)
        e = launch_implicit_weights(w, u_hi(p), p->s.Cout, p->s.Cin, p->s.k, p->cin_pad, st);
    else if (p->rect)
        e = launch_rect_weights(w, u_hi(p), u_lo(p), rect_geom(p), p->store_mode, p->mats, st);
    else if (p->strassen)
        e = launch_strassen_weights(w, u_hi(p), u_lo(p), strassen_geom(p), p->store_mode, st);
    else if (p->fused)
        e = launch_fused_wino_weights(w, u_hi(p), p->s.Cout, p->s.Cin, p->mats, st);
    else if (p->d.algo == MNN_ALGO_WINOGRAD)
        e = launch_weight_transform(w, u_hi(p), u_lo(p), p->s.Cout, p->s.Cin, p->s.k, p->d.m, p->cin_pad, p->store_mode,
                                    p->mats, st);
    else
        e = launch_weight_round(w, u_hi(p), u_lo(p), p->s.Cout, p->s.Cin * p->s.k * p->s.k, p->cin_pad, p->store_mode, st);
    if (e != cudaSuccess) return fail_cuda(e, "weight transform");
    p->prepared_w = w;
    return MNN_OK;
}

int mnn_conv_prepare_weights(mnn_conv_plan_t p, const float* w, void* stream)
{
    if (!p || !w) return fail(MNN_EINVAL, "NULL plan or weights");
    if (p->d.algo == MNN_ALGO_DIRECT) {
        p->prepared_w = w;
        return MNN_OK;
    }
    if (!p->ws) return fail(MNN_EWORKSPACE, "call mnn_conv_set_workspace first");
    if (!aligned16(w)) return fail(MNN_EALIGN, "w must be 16-byte aligned");
    return do_weights(p, w, static_cast<cudaStream_t>(stream));
}

int mnn_conv_run_stages(mnn_conv_plan_t p, const float* x, const float* w, const float* bias, float* y, void* stream,
                        unsigned mask)
{
    int rc = check_run_args(p, x, w, y, mask);
    if (rc != MNN_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const LayerShape& s = p->s;
    const Decision& d = p->d;
    cudaError_t e;
    p->event_stage.clear();

    if (d.algo == MNN_ALGO_DIRECT) {
        if (!(mask & MNN_STAGE_CONTRACT)) return MNN_OK;
        DirectGeom g = {s.N, s.Cin, s.Cout, s.H, s.W, s.OH, s.OW, s.k, s.stride, s.pad, s.dil, s.groups, s.relu};
        {
            LaunchTimer lt(p, st, 2);
            e = launch_direct(x, w, bias, y, g, st);
        }
        if (e != cudaSuccess) return fail_cuda(e, "direct convolution");
        return MNN_OK;
    }

    if (mask & MNN_STAGE_WEIGHT) {
        rc = do_weights(p, w, st);
        if (rc != MNN_OK) return rc;
    }
    const bool reference = d.operand == MNN_OPERAND_FP32_REF;

    if (p->rect) {
        const RectGeom g = rect_geom(p);
        if (reference) return fail(MNN_EUNSUPPORTED, "rectangular kernels run on the tensor-core contraction only");
        if (mask & MNN_STAGE_INPUT) {
            LaunchTimer lt(p, st, 1);
            e = launch_rect_input(x, v_hi(p), v_lo(p), g, p->store_mode, p->mats, st);
            if (e != cudaSuccess) return fail_cuda(e, "one-dimensional input transform");
        }
        if (mask & MNN_STAGE_CONTRACT) {
            ContractEpilogue epi = {0, m_buf(p), p->m_row_stride, nullptr, nullptr, 0, 1};
            LaunchTimer lt(p, st, 2);
            e = launch_contract_umma(p->uc, g.tiles, epi, status_word(p), st);
            if (e != cudaSuccess) return fail_cuda(e, "Winograd contraction");
        }
        if (mask & MNN_STAGE_OUTPUT) {
            LaunchTimer lt(p, st, 3);
            e = launch_rect_output(m_buf(p), bias, y, g, s.relu, p->mats, st);
            if (e != cudaSuccess) return fail_cuda(e, "one-dimensional output transform");
        }
        return MNN_OK;
    }
    if (p->strassen) {
        const StrassenGeom g = strassen_geom(p);
        if (reference) return fail(MNN_EUNSUPPORTED, "Strassen runs on the tensor-core contraction only");
        if (mask & MNN_STAGE_INPUT) {
            LaunchTimer lt(p, st, 1);
            e = launch_strassen_input(x, v_hi(p), v_lo(p), g, p->store_mode, st);
            if (e != cudaSuccess) return fail_cuda(e, "Strassen operand pass");
        }
        if (mask & MNN_STAGE_CONTRACT) {
            ContractEpilogue epi = {0, m_buf(p), p->m_row_stride, nullptr, nullptr, 0, 1};
            LaunchTimer lt(p, st, 2);
            e = launch_contract_umma(p->uc, g.t_half, epi, status_word(p), st);
            if (e != cudaSuccess) return fail_cuda(e, "Strassen products");
        }
        if (mask & MNN_STAGE_OUTPUT) {
            LaunchTimer lt(p, st, 3);
            e = launch_strassen_output(m_buf(p), bias, y, g, s.relu, st);
            if (e != cudaSuccess) return fail_cuda(e, "Strassen result pass");
        }
        return MNN_OK;
    }
    if (d.algo == MNN_ALGO_GEMM) {
        const long long T = (long long)s.N * s.OH * s.OW;
        if ((mask & MNN_STAGE_INPUT) && !p->gemm_x && !p->gemm_implicit) {
            GatherGeom g = {s.N, s.Cin, s.H, s.W, s.OH, s.OW, s.k, s.stride, s.pad, s.dil, p->cin_pad};
            LaunchTimer lt(p, st, 1);
            e = launch_gather(x, v_hi(p), v_lo(p), g, p->store_mode, st);
            if (e != cudaSuccess) return fail_cuda(e, "patch gather");
        }
        if (mask & MNN_STAGE_CONTRACT) {
            ContractEpilogue epi = {1, nullptr, 0, y, bias, s.relu, s.OH * s.OW};
            LaunchTimer lt(p, st, 2);
            if (reference)
                e = launch_contract_reference(u_hi(p), u_lo(p), v_hi(p), v_lo(p), p->store_mode, 1, s.Cout, T, p->cin_pad,
                                              (long long)s.Cout * p->cin_pad, T * p->cin_pad, epi, st);
            else if (p->gemm_implicit) {
                GatherGeom g = {s.N, s.Cin, s.H, s.W, s.OH, s.OW, s.k, s.stride, s.pad, s.dil, p->cin_pad};
                e = launch_implicit_gemm(p->ig, x, bias, y, g, s.relu, status_word(p), st);
            } else if (p->gemm_x)
                e = launch_contract_umma_x(p->uc, x, epi, status_word(p), st);
            else
                e = launch_contract_umma(p->uc, T, epi, status_word(p), st);
            if (e != cudaSuccess) return fail_cuda(e, "GEMM contraction");
        }
        return MNN_OK;
    }

    const int th = (s.OH + d.m - 1) / d.m, tw = (s.OW + d.m - 1) / d.m;
    const int alpha2 = d.alpha * d.alpha;
    if (p->fused) {
        // one kernel does the three stages; it is booked as the contraction stage
        if (!(mask & MNN_STAGE_CONTRACT)) return MNN_OK;
        WinoGeom g;
        g.images = s.N;
        g.Cin = s.Cin; g.Cout = s.Cout; g.H = s.H; g.W = s.W; g.OH = s.OH; g.OW = s.OW; g.k = s.k; g.pad = s.pad;
        g.m = d.m; g.alpha = d.alpha; g.th = th; g.tw = tw; g.cin_pad = p->cin_pad;
        g.tiles = (long long)s.N * th * tw;
        g.v_plane = 0;
        g.m_row_stride = 0;
        LaunchTimer lt(p, st, 2);
        e = launch_fused_wino(p->fw, x, bias, y, g, s.relu, p->mats, status_word(p), st);
        if (e != cudaSuccess) return fail_cuda(e, "fused Winograd kernel");
        return MNN_OK;
    }
    // Winograd: the three stages chunk by chunk, so that one chunk's V and M stay in L2.
    for (int n0 = 0; n0 < s.N; n0 += d.chunk_images) {
        const int n_img = (s.N - n0) < d.chunk_images ? (s.N - n0) : d.chunk_images;
        WinoGeom g;
        g.images = n_img;
        g.Cin = s.Cin; g.Cout = s.Cout; g.H = s.H; g.W = s.W; g.OH = s.OH; g.OW = s.OW; g.k = s.k; g.pad = s.pad;
        g.m = d.m; g.alpha = d.alpha; g.th = th; g.tw = tw; g.cin_pad = p->cin_pad;
        g.tiles = (long long)n_img * th * tw;
        g.v_plane = p->chunk_tiles * p->cin_pad;
        g.m_row_stride = p->m_row_stride;
        if (mask & MNN_STAGE_INPUT) {
            LaunchTimer lt(p, st, 1);
            e = launch_input_transform(x + (size_t)n0 * s.Cin * s.H * s.W, v_hi(p), v_lo(p), g, p->store_mode, p->mats,
                                       status_word(p), st);
            if (e != cudaSuccess) return fail_cuda(e, "input transform");
        }
        if (mask & MNN_STAGE_CONTRACT) {
            ContractEpilogue epi = {0, m_buf(p), p->m_row_stride, nullptr, nullptr, 0, 1};
            LaunchTimer lt(p, st, 2);
            if (reference)
                e = launch_contract_reference(u_hi(p), u_lo(p), v_hi(p), v_lo(p), p->store_mode, alpha2, s.Cout, g.tiles,
                                              p->cin_pad, (long long)s.Cout * p->cin_pad, g.v_plane, epi, st);
            else if (p->use_pair)
                e = launch_contract_pair(p->pc, g.tiles, m_buf(p), p->m_row_stride, status_word(p), st);
            else
                e = launch_contract_umma(p->uc, g.tiles, epi, status_word(p), st);
            if (e != cudaSuccess) return fail_cuda(e, "Winograd contraction");
        }
        if (mask & MNN_STAGE_OUTPUT) {
            LaunchTimer lt(p, st, 3);
            e = launch_output_transform(m_buf(p), bias, y + (size_t)n0 * s.Cout * s.OH * s.OW, g, s.relu, p->mats, st);
            if (e != cudaSuccess) return fail_cuda(e, "output transform");
        }
    }
    return MNN_OK;
}

int mnn_conv_run(mnn_conv_plan_t p, const float* x, const float* w, const float* bias, float* y, void* stream)
{
    if (!p) return fail(MNN_EINVAL, "NULL plan");
    if (!x || !w || !y) return fail(MNN_EINVAL, "NULL tensor pointer");
    unsigned mask = MNN_STAGE_INPUT | MNN_STAGE_CONTRACT | MNN_STAGE_OUTPUT;
    if (p->d.algo != MNN_ALGO_DIRECT && p->prepared_w != w) mask |= MNN_STAGE_WEIGHT;
    return mnn_conv_run_stages(p, x, w, bias, y, stream, mask);
}

int mnn_conv_device_status(mnn_conv_plan_t p, void* stream, int* code)
{
    if (!p || !code) return fail(MNN_EINVAL, "NULL plan or code");
    *code = 0;
    if (!p->ws) return MNN_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(code, status_word(p), sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return fail_cuda(e, "reading the status word");
    if (*code != 0) {
        e = cudaMemsetAsync(status_word(p), 0, sizeof(int), st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) return fail_cuda(e, "clearing the status word");
    }
    return MNN_OK;
}

int mnn_conv_profile(mnn_conv_plan_t p, int enable)
{
    if (!p) return fail(MNN_EINVAL, "NULL plan");
    free_events(p);
    p->profiling = false;
    if (!enable) return MNN_OK;
    const int pairs = p->launches_per_run + 2;
    for (int i = 0; i < 2 * pairs; ++i) {
        cudaEvent_t ev;
        cudaError_t e = cudaEventCreate(&ev);
        if (e != cudaSuccess) {
            free_events(p);
            return fail_cuda(e, "creating profiling events");
        }
        p->events.push_back(ev);
    }
    p->profiling = true;
    return MNN_OK;
}

int mnn_conv_profile_read(mnn_conv_plan_t p, float stage_ms[4], int stage_launches[4])
{
    if (!p || !stage_ms || !stage_launches) return fail(MNN_EINVAL, "NULL argument");
    if (!p->profiling) return fail(MNN_EINVAL, "profiling is off");
    for (int i = 0; i < 4; ++i) {
        stage_ms[i] = 0.0f;
        stage_launches[i] = 0;
    }
    for (size_t i = 0; i < p->event_stage.size(); ++i) {
        cudaError_t e = cudaEventSynchronize(p->events[2 * i + 1]);
        float ms = 0.0f;
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, p->events[2 * i], p->events[2 * i + 1]);
        if (e != cudaSuccess) return fail_cuda(e, "reading profiling events");
        stage_ms[p->event_stage[i]] += ms;
        stage_launches[p->event_stage[i]] += 1;
    }
    return MNN_OK;
}

void mnn_conv_destroy(mnn_conv_plan_t p)
{
    if (!p) return;
    free_events(p);
    delete p;
}

int mnn_winograd_matrices(int m, int k, int points_id, float* At, float* G, float* Bt)
{
    WinogradMatrices wm;
    if (points_id < 1 || points_id > 3) return fail(MNN_EINVAL, "points_id must be 1, 2 or 3");
    if (!generate_winograd(m, k, points_id, &wm)) return fail(MNN_EINVAL, "need m, k >= 1 and m + k - 1 <= 16 within the point set");
    if (At) std::memcpy(At, wm.At32.data(), wm.At32.size() * sizeof(float));
    if (G) std::memcpy(G, wm.G32.data(), wm.G32.size() * sizeof(float));
    if (Bt) std::memcpy(Bt, wm.Bt32.data(), wm.Bt32.size() * sizeof(float));
    return MNN_OK;
}

long long mnn_accuracy_ppm(int m, int k, int points_id, int operand, int passes)
{
    long long v = accuracy_ppm(m, k, points_id, operand, passes);
    if (v < 0) fail(MNN_EINVAL, "invalid (m, k, points_id, operand, passes)");
    return v;
}

int mnn_wait_probe(int* device_word, void* stream)
{
    if (!device_word) return fail(MNN_EINVAL, "NULL device word");
    cudaError_t e = launch_wait_probe(device_word, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return fail_cuda(e, "wait probe");
    return MNN_OK;
}

int mnn_strassen_rule(long long m, long long n, long long k)
{
    if (m < 2 || n < 2 || k < 2) return 0;
    const __int128 mh = m / 2, nh = n / 2, kh = k / 2;
    const __int128 saved = (__int128)m * n * k - 7 * mh * nh * kh;
    const __int128 added = 4 * mh * kh + 4 * nh * kh + 7 * mh * nh;
    return saved > added ? 1 : 0;
}

int mnn_set_calibration(const long long consts[MNN_N_CONSTS])
{
    if (!consts) return fail(MNN_EINVAL, "NULL constants");
    Calibration c;
    for (int i = 0; i < MNN_N_CONSTS; ++i) c.c[i] = consts[i];
    for (int i = 0; i <= 8; ++i)
        if (c.c[i] <= 0) return fail(MNN_EINVAL, "constants 0..8 must be positive");
    install_calibration(c);
    return MNN_OK;
}

int mnn_get_calibration(long long consts[MNN_N_CONSTS])
{
    if (!consts) return fail(MNN_EINVAL, "NULL constants");
    Calibration c = current_calibration();
    for (int i = 0; i < MNN_N_CONSTS; ++i) consts[i] = c.c[i];
    return MNN_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------
// Network-level plan: a sequential stack of layers, one workspace laid out by a virtual walk.
// ---------------------------------------------------------------------------
struct mnn_net_s {
    int N = 0, H = 0, W = 0;
    std::vector<mnn_conv_plan_t> plans;
    std::vector<long long> persistent_offset;      // per layer, from the workspace base
    long long persistent_bytes = 0, transient_bytes = 0, activation_bytes = 0, workspace_bytes = 0;
    long long sum_of_layer_workspaces = 0;
    long long transient_offset = 0, act_offset[2] = {0, 0};
    char* ws = nullptr;
    ~mnn_net_s()
    {
        for (mnn_conv_plan_t p : plans) mnn_conv_destroy(p);
    }
};

extern "C" {

mnn_net_t mnn_net_plan(int N, int H, int W, int n_layers, const mnn_layer_desc* layers, int precision)
{
    if (n_layers < 1 || n_layers > MNN_NET_MAX_LAYERS || !layers) {
        fail(MNN_EINVAL, "a network needs 1..MNN_NET_MAX_LAYERS layers");
        return nullptr;
    }
    mnn_net_t net = new (std::nothrow) mnn_net_s();
    if (!net) {
        fail(MNN_EINVAL, "out of host memory");
        return nullptr;
    }
    net->N = N; net->H = H; net->W = W;
    int c = layers[0].Cin, h = H, w = W;
    long long off = 0;
    for (int i = 0; i < n_layers; ++i) {
        const mnn_layer_desc& L = layers[i];
        if (L.Cin != c) {
            fail(MNN_EINVAL, "layer " + std::to_string(i) + ": Cin does not match the previous layer's Cout");
            delete net;
            return nullptr;
        }
        mnn_conv_opts o;
        std::memset(&o, 0, sizeof(o));
        o.groups = L.groups ? L.groups : 1;
        o.relu = L.relu;
        o.precision = precision;
        mnn_conv_plan_t p = mnn_conv_plan_ex(N, L.Cin, L.Cout, h, w, L.k, L.stride, L.pad, L.dilation, &o);
        if (!p) {
            g_last_error = "layer " + std::to_string(i) + ": " + g_last_error;
            delete net;
            return nullptr;
        }
        net->plans.push_back(p);
        // virtual walk: the persistent part (status word + U) gets its own place, the transient part
        // (V + M) only counts towards the maximum, the output towards the activation buffers
        const long long persistent = p->workspace_bytes > 0 ? align_up(p->v_offset, 1024) : 0;
        const long long transient = p->workspace_bytes > 0 ? p->workspace_bytes - p->v_offset : 0;
        net->persistent_offset.push_back(off);
        off += persistent;
        if (transient > net->transient_bytes) net->transient_bytes = transient;
        net->sum_of_layer_workspaces += p->workspace_bytes;
        if (i + 1 < n_layers) {
            const long long act = 4ll * N * L.Cout * p->s.OH * p->s.OW;
            if (act > net->activation_bytes) net->activation_bytes = act;
        }
        c = L.Cout; h = p->s.OH; w = p->s.OW;
    }
    net->persistent_bytes = off;
    net->transient_bytes = align_up(net->transient_bytes, 1024);
    net->activation_bytes = align_up(net->activation_bytes, 1024);
    net->transient_offset = net->persistent_bytes;
    net->act_offset[0] = net->transient_offset + net->transient_bytes;
    net->act_offset[1] = net->act_offset[0] + net->activation_bytes;
    net->workspace_bytes = net->act_offset[1] + net->activation_bytes;
    return net;
}

int mnn_net_query(mnn_net_t net, mnn_net_info* info)
{
    if (!net || !info) return fail(MNN_EINVAL, "NULL network or info");
    std::memset(info, 0, sizeof(*info));
    info->n_layers = (int)net->plans.size();
    info->N = net->N; info->H = net->H; info->W = net->W;
    info->workspace_bytes = net->workspace_bytes;
    info->persistent_bytes = net->persistent_bytes;
    info->transient_bytes = net->transient_bytes;
    info->activation_bytes = net->activation_bytes;
    info->sum_of_layer_workspaces = net->sum_of_layer_workspaces;
    for (size_t i = 0; i < net->plans.size(); ++i) {
        mnn_conv_plan_t p = net->plans[i];
        info->algo[i] = p->d.algo; info->m[i] = p->d.m; info->operand[i] = p->d.operand; info->passes[i] = p->d.passes;
        info->OH[i] = p->s.OH; info->OW[i] = p->s.OW;
        info->launches_per_run += p->launches_per_run;
    }
    mnn_conv_plan_t last = net->plans.back();
    info->out_C = last->s.Cout; info->out_H = last->s.OH; info->out_W = last->s.OW;
    return MNN_OK;
}

int mnn_net_set_workspace(mnn_net_t net, void* workspace, long long bytes)
{
    if (!net) return fail(MNN_EINVAL, "NULL network");
    net->ws = nullptr;
    if (!workspace) return fail(MNN_EWORKSPACE, "the network needs a workspace");
    if (bytes < net->workspace_bytes) return fail(MNN_EWORKSPACE, "workspace smaller than info.workspace_bytes");
    if (reinterpret_cast<uintptr_t>(workspace) & 1023u) return fail(MNN_EALIGN, "workspace must be 1024-byte aligned");
    char* base = static_cast<char*>(workspace);
    for (size_t i = 0; i < net->plans.size(); ++i) {
        mnn_conv_plan_t p = net->plans[i];
        if (p->workspace_bytes == 0) continue;
        int rc = set_workspace_split(p, base + net->persistent_offset[i], align_up(p->v_offset, 1024),
                                     base + net->transient_offset, net->transient_bytes);
        if (rc != MNN_OK) return rc;
    }
    net->ws = base;
    return MNN_OK;
}

int mnn_net_prepare(mnn_net_t net, const float* const* w, void* stream)
{
    if (!net || !w) return fail(MNN_EINVAL, "NULL network or weights");
    if (!net->ws) return fail(MNN_EWORKSPACE, "call mnn_net_set_workspace first");
    for (size_t i = 0; i < net->plans.size(); ++i) {
        int rc = mnn_conv_prepare_weights(net->plans[i], w[i], stream);
        if (rc != MNN_OK) return rc;
    }
    return MNN_OK;
}

int mnn_net_run(mnn_net_t net, const float* x, const float* const* w, const float* const* bias, float* y, void* stream)
{
    if (!net || !x || !w || !y) return fail(MNN_EINVAL, "NULL argument");
    if (!net->ws) return fail(MNN_EWORKSPACE, "call mnn_net_set_workspace first");
    const size_t n = net->plans.size();
    const float* in = x;
    for (size_t i = 0; i < n; ++i) {
        float* out = i + 1 == n ? y : reinterpret_cast<float*>(net->ws + net->act_offset[i & 1]);
        int rc = mnn_conv_run(net->plans[i], in, w[i], bias ? bias[i] : nullptr, out, stream);
        if (rc != MNN_OK) {
            g_last_error = "layer " + std::to_string(i) + ": " + g_last_error;
            return rc;
        }
        in = out;
    }
    return MNN_OK;
}

int mnn_net_device_status(mnn_net_t net, void* stream, int* code, int* layer)
{
    if (!net || !code || !layer) return fail(MNN_EINVAL, "NULL argument");
    *code = 0;
    *layer = -1;
    for (size_t i = 0; i < net->plans.size(); ++i) {
        int c = 0;
        int rc = mnn_conv_device_status(net->plans[i], stream, &c);
        if (rc != MNN_OK) return rc;
        if (c != 0 && *code == 0) {
            *code = c;
            *layer = (int)i;
        }
    }
    return MNN_OK;
}

void mnn_net_destroy(mnn_net_t net) { delete net; }

}  // extern "C"

// ---------------------------------------------------------------------------
// A run that allocates nothing: the plan's workspace is a fixed array that is
// part of the library image on every GPU that loads it.
// ---------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_workspace[MNN_STATIC_WORKSPACE_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void* g_static_workspace_ptr[kMaxDevices] = {nullptr};

// Device address of the array on the current device.  In host code the array's
// name is only a handle for the runtime, so the address is asked for once per
// device, with that device current.
int static_workspace_of_current_device(void** out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail_cuda(e, "cudaGetDevice");
    if (dev < 0 || dev >= kMaxDevices) return fail(MNN_EUNSUPPORTED, "device index above 63");
    std::lock_guard<std::mutex> lk(g_static_mutex);
    if (!g_static_workspace_ptr[dev]) {
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_static_workspace);
        if (e != cudaSuccess) return fail_cuda(e, "cudaGetSymbolAddress of the built-in workspace");
        if (!ptr || (reinterpret_cast<uintptr_t>(ptr) & 255u))
            return fail(MNN_ECUDA, "the built-in workspace has no usable device address");
        g_static_workspace_ptr[dev] = ptr;
    }
    *out = g_static_workspace_ptr[dev];
    return MNN_OK;
}

}  // namespace

extern "C" int mnn_conv_run_static(mnn_conv_plan_t p, const float* x, const float* w, const float* bias, float* y,
                                   void* stream)
{
    if (!p) return fail(MNN_EINVAL, "NULL plan");
    if (!x || !w || !y) return fail(MNN_EINVAL, "NULL tensor pointer");
    if (p->workspace_bytes > (long long)MNN_STATIC_WORKSPACE_BYTES)
        return fail(MNN_EWORKSPACE, "this plan needs " + std::to_string(p->workspace_bytes) +
                                        " workspace bytes; the built-in workspace holds " +
                                        std::to_string((long long)MNN_STATIC_WORKSPACE_BYTES));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // A private copy of the host-side plan whose workspace is the built-in array: the caller's
    // plan (its own workspace, prepared weights, profiling state) is left untouched.
    mnn_conv_plan_s local = *p;
    local.profiling = false;
    local.events.clear();
    local.event_stage.clear();
    local.prepared_w = nullptr;
    local.uc.ready = false;
    local.ws = nullptr;
    local.tws = nullptr;
    local.ws_bytes = 0;
    if (local.workspace_bytes > 0) {
        void* ptr = nullptr;
        int rc = static_workspace_of_current_device(&ptr);
        if (rc != MNN_OK) return rc;
        local.ws = static_cast<char*>(ptr);
        local.ws_bytes = (long long)MNN_STATIC_WORKSPACE_BYTES;
        // The array keeps whatever the previous call left: the status word must start at zero.
        cudaError_t e = cudaMemsetAsync(local.ws, 0, kStatusBytes, st);
        if (e != cudaSuccess) return fail_cuda(e, "clearing the status word");
        if (local.d.operand != MNN_OPERAND_FP32_REF) {
            const char* why = "";
            e = setup_tensor_kernels(&local, &why);
            if (e != cudaSuccess)
                return fail(MNN_ECUDA, std::string("tensor-core contraction setup: ") + why + " (" + cudaGetErrorString(e) + ")");
        }
    }
    // Transformed weights are rebuilt on every call: another call may have overwritten them.
    return mnn_conv_run_stages(&local, x, w, bias, y, stream, MNN_STAGE_ALL);
}
