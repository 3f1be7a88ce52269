// Pre-inference planner (Section 3.2): choose the computation scheme of one
// convolution layer by minimising a cost, Eq. 1.  The paper's arithmetic count
// (Eq. 2) and its backend term MUL/FLOPS + t_schedule (Eq. 5) are re-stated for a
// GPU whose kernels are bound by memory traffic, tensor throughput or ALU
// throughput, whichever is largest:
//     cost(candidate) = sum over its kernels of
//         max(bytes x c_byte, tensor flops x c_tensor, ALU flops x c_alu) / 1e6 + c_launch
// in integer picoseconds (the constants are attoseconds per unit).  Everything
// below the accuracy model is integer arithmetic, so that a choice can be
// reproduced bit for bit from the nine layer integers and the constant record.
#include "planner.h"

#include <cmath>
#include <cstring>
#include <map>
#include <mutex>
#include <tuple>
#include <vector>

#include "generator.h"

namespace mnnb {

namespace {
std::mutex g_cal_mutex;
Calibration g_cal;
bool g_cal_set = false;

uint64_t ceil_div(uint64_t a, uint64_t b) { return (a + b - 1) / b; }
constexpr uint64_t kMaxChunkBytes = 4ull << 30;   // V + M of one chunk
uint64_t round_up(uint64_t a, uint64_t b) { return ceil_div(a, b) * b; }
// Attosecond products of byte or flop counts and rate constants can pass 2^64 for very large layers; they
// are formed in 128 bits and every picosecond figure saturates just below the "inadmissible" marker, so a
// huge layer can never wrap around into a small cost.
typedef unsigned __int128 u128;
constexpr uint64_t kCostSaturated = MNN_COST_INADMISSIBLE - 1;
uint64_t saturate(u128 v) { return v > (u128)kCostSaturated ? kCostSaturated : (uint64_t)v; }
u128 max3(u128 a, u128 b, u128 c) { return a > b ? (a > c ? a : c) : (b > c ? b : c); }
}  // namespace

Calibration default_calibration()
{
    Calibration c;
    std::memset(&c, 0, sizeof(c));
    // one calibration record measured on a B200 (mnn_calibrate), rounded
    c.c[0] = 173000;      // as per HBM byte          (~5.8 TB/s with a plain copy kernel)
    c.c[1] = 84000;       // as per L2-resident byte  (~12 TB/s)
    c.c[2] = 1930;        // as per TF32 tensor flop  (~520 TFLOP/s achieved by the contraction kernel)
    c.c[3] = 1050;        // as per BF16 tensor flop  (~950 TFLOP/s achieved)
    c.c[4] = 28000;       // as per fp32 ALU flop in the transform kernels (~36 TFLOP/s)
    c.c[5] = 3530000;     // ps of fixed cost per kernel: launch, ramp-up and tail (the t_schedule of Eq. 5)
    c.c[6] = 80ll << 20;  // L2 bytes one chunk's V + M may occupy
    c.c[7] = 148;         // SMs
    c.c[8] = 571000;      // as per flop of the direct kernel (~3.5 TFLOP/s)
    c.c[9] = 31000;       // as per flop of the 3 -> Cout 3x3 stride-2 kernel (~32 TFLOP/s); other Cin <= 4 shapes: twice that
    c.c[10] = 23000000;   // as per byte of U delivered to one SM by the fused kernel's weight stream (~43 GB/s per SM)
    c.c[11] = 6000000;    // ps per 32-channel block of a fused work item (64 MMAs of 128 x 32 x 8 at ~90 ns each)
    c.c[12] = 4300000;    // ps of epilogue per fused work item
    c.c[13] = 400000000;  // as per patch element gathered by the implicit GEMM's producer warps, per SM (~1.6 us per 128 x 32 tile)
    return c;
}

Calibration current_calibration()
{
    std::lock_guard<std::mutex> lk(g_cal_mutex);
    return g_cal_set ? g_cal : default_calibration();
}

void install_calibration(const Calibration& c)
{
    std::lock_guard<std::mutex> lk(g_cal_mutex);
    g_cal = c;
    g_cal_set = true;
}

int conv_out_extent(int in, int k, int stride, int pad, int dil)
{
    if (stride <= 0) return 0;
    long long span = (long long)in + 2ll * pad - (long long)dil * (k - 1) - 1;
    if (span < 0) return 0;
    return (int)(span / stride) + 1;
}

bool winograd_supported(int m, int k)
{
    if (!(m == 2 || m == 4 || m == 6)) return false;
    if (!(k == 2 || k == 3 || k == 5 || k == 7)) return false;
    return m + k - 1 <= 12;
}

// ---------------------------------------------------------------------------
// Accuracy model: simulate F(m,k) on a fixed pseudo-random problem in fp64 with
// U and V rounded to the operand format (optionally split into hi + lo), and
// report the relative L2 error against the plain correlation.
// ---------------------------------------------------------------------------
namespace {

struct Lcg {
    uint64_t s;
    explicit Lcg(uint64_t seed) : s(seed) {}
    double uniform()
    {
        s = s * 6364136223846793005ull + 1442695040888963407ull;
        return (double)(s >> 11) * (1.0 / 9007199254740992.0);
    }
    // sum of twelve uniforms minus six: mean 0, variance 1, additions only
    double normalish()
    {
        double a = 0.0;
        for (int i = 0; i < 12; ++i) a += uniform();
        return a - 6.0;
    }
};

double round_mantissa(double v, int bits)
{
    // nearest-even rounding of fp32(v) to `bits` explicit mantissa bits
    float f = (float)v;
    uint32_t u;
    std::memcpy(&u, &f, 4);
    const int drop = 23 - bits;
    if (drop > 0) {
        uint32_t lsb = (u >> drop) & 1u;
        u += (1u << (drop - 1)) - 1u + lsb;
        u &= ~((1u << drop) - 1u);
    }
    std::memcpy(&f, &u, 4);
    return (double)f;
}

void split_operand(double v, int bits, int passes, double* hi, double* lo)
{
    *hi = round_mantissa(v, bits);
    *lo = passes == 3 ? round_mantissa((double)(float)v - *hi, bits) : 0.0;
}

std::mutex g_acc_mutex;
std::map<std::tuple<int, int, int, int, int>, long long> g_acc_cache;

long long simulate_ppm(int m, int k, int points_id, int bits, int passes)
{
    const int C = 64, CO = 4, TILES = 16;
    Lcg rng(0x9E3779B97F4A7C15ull ^ (uint64_t)(m * 1000 + k * 10));   // same data for every point set
    const bool gemm = (m == 1 && points_id == 0);
    WinogradMatrices wm;
    if (!gemm && !generate_winograd(m, k, points_id, &wm)) return -1;
    const int alpha = m + k - 1;
    const int a2 = alpha * alpha;

    std::vector<double> w((size_t)CO * C * k * k), x((size_t)TILES * C * a2);
    const double wscale = 1.0 / std::sqrt((double)(C * k * k));
    for (auto& v : w) v = (double)(float)(rng.normalish() * wscale);
    for (auto& v : x) v = (double)(float)rng.normalish();

    double num = 0.0, den = 0.0;
    if (gemm) {
        // one dot product of length C*k*k per output, operands rounded directly
        for (int t = 0; t < TILES; ++t)
            for (int co = 0; co < CO; ++co) {
                double ref = 0.0, got = 0.0;
                for (int c = 0; c < C; ++c)
                    for (int e = 0; e < k * k; ++e) {
                        const double wv = w[((size_t)co * C + c) * k * k + e];
                        const double xv = x[((size_t)t * C + c) * a2 + e];
                        double wh, wl, xh, xl;
                        split_operand(wv, bits, passes, &wh, &wl);
                        split_operand(xv, bits, passes, &xh, &xl);
                        ref += wv * xv;
                        got += wh * xh + wl * xh + wh * xl;
                    }
                num += (got - ref) * (got - ref);
                den += ref * ref;
            }
    } else {
        const std::vector<double>&G = wm.G64, &Bt = wm.Bt64, &At = wm.At64;
        // U hi/lo [co][c][a2], V hi/lo [t][c][a2]
        std::vector<double> Uh((size_t)CO * C * a2), Ul(Uh.size()), Vh((size_t)TILES * C * a2), Vl(Vh.size());
        std::vector<double> tmp((size_t)alpha * alpha);
        for (int co = 0; co < CO; ++co)
            for (int c = 0; c < C; ++c) {
                const double* g = &w[((size_t)co * C + c) * k * k];
                for (int i = 0; i < alpha; ++i)
                    for (int b = 0; b < k; ++b) {
                        double s = 0.0;
                        for (int a = 0; a < k; ++a) s += G[i * k + a] * g[a * k + b];
                        tmp[i * k + b] = s;
                    }
                for (int i = 0; i < alpha; ++i)
                    for (int j = 0; j < alpha; ++j) {
                        double s = 0.0;
                        for (int b = 0; b < k; ++b) s += tmp[i * k + b] * G[j * k + b];
                        split_operand(s, bits, passes, &Uh[((size_t)co * C + c) * a2 + i * alpha + j],
                                      &Ul[((size_t)co * C + c) * a2 + i * alpha + j]);
                    }
            }
        for (int t = 0; t < TILES; ++t)
            for (int c = 0; c < C; ++c) {
                const double* d = &x[((size_t)t * C + c) * a2];
                for (int i = 0; i < alpha; ++i)
                    for (int b = 0; b < alpha; ++b) {
                        double s = 0.0;
                        for (int a = 0; a < alpha; ++a) s += Bt[i * alpha + a] * d[a * alpha + b];
                        tmp[i * alpha + b] = s;
                    }
                for (int i = 0; i < alpha; ++i)
                    for (int j = 0; j < alpha; ++j) {
                        double s = 0.0;
                        for (int b = 0; b < alpha; ++b) s += tmp[i * alpha + b] * Bt[j * alpha + b];
                        split_operand(s, bits, passes, &Vh[((size_t)t * C + c) * a2 + i * alpha + j],
                                      &Vl[((size_t)t * C + c) * a2 + i * alpha + j]);
                    }
            }
        std::vector<double> Mx((size_t)a2), t2((size_t)m * alpha);
        for (int t = 0; t < TILES; ++t)
            for (int co = 0; co < CO; ++co) {
                for (int e = 0; e < a2; ++e) {
                    double s = 0.0;
                    for (int c = 0; c < C; ++c) {
                        const size_t ui = ((size_t)co * C + c) * a2 + e, vi = ((size_t)t * C + c) * a2 + e;
                        s += Uh[ui] * Vh[vi] + Ul[ui] * Vh[vi] + Uh[ui] * Vl[vi];
                    }
                    Mx[e] = (double)(float)s;
                }
                for (int a = 0; a < m; ++a)
                    for (int j = 0; j < alpha; ++j) {
                        double s = 0.0;
                        for (int i = 0; i < alpha; ++i) s += At[a * alpha + i] * Mx[i * alpha + j];
                        t2[a * alpha + j] = s;
                    }
                for (int a = 0; a < m; ++a)
                    for (int b = 0; b < m; ++b) {
                        double got = 0.0;
                        for (int j = 0; j < alpha; ++j) got += t2[a * alpha + j] * At[b * alpha + j];
                        double ref = 0.0;
                        for (int c = 0; c < C; ++c)
                            for (int i = 0; i < k; ++i)
                                for (int j = 0; j < k; ++j)
                                    ref += w[((size_t)co * C + c) * k * k + i * k + j] *
                                           x[((size_t)t * C + c) * a2 + (a + i) * alpha + (b + j)];
                        num += (got - ref) * (got - ref);
                        den += ref * ref;
                    }
            }
    }
    if (!(den > 0.0)) return -1;
    const double rel = std::sqrt(num / den);
    double ppm = std::ceil(rel * 1e6);
    if (ppm > 4e18) ppm = 4e18;
    return (long long)ppm;
}

}  // namespace

long long accuracy_ppm(int m, int k, int points_id, int operand, int passes)
{
    if (m < 1 || k < 1 || m + k - 1 > kMaxAlpha) return -1;
    if (!(operand == MNN_OPERAND_TF32 || operand == MNN_OPERAND_BF16 || operand == MNN_OPERAND_FP32_REF)) return -1;
    if (!(passes == 1 || passes == 3)) return -1;
    const bool gemm = (m == 1 && points_id == 0);
    if (!gemm && (points_id < 1 || points_id > 3)) return -1;
    const int bits = operand == MNN_OPERAND_TF32 ? 10 : (operand == MNN_OPERAND_BF16 ? 7 : 23);
    auto key = std::make_tuple(m, k, points_id, bits, passes);
    {
        std::lock_guard<std::mutex> lk(g_acc_mutex);
        auto it = g_acc_cache.find(key);
        if (it != g_acc_cache.end()) return it->second;
    }
    long long v = simulate_ppm(m, k, points_id, bits, passes);
    std::lock_guard<std::mutex> lk(g_acc_mutex);
    g_acc_cache[key] = v;
    return v;
}

int best_points(int m, int k, int operand, int passes, long long* ppm_out)
{
    int best = 0;
    long long best_ppm = -1;
    for (int pid = 1; pid <= 3; ++pid) {
        long long p = accuracy_ppm(m, k, pid, operand, passes);
        if (p < 0) continue;
        if (best == 0 || p < best_ppm) {
            best = pid;
            best_ppm = p;
        }
    }
    if (ppm_out) *ppm_out = best_ppm;
    return best;
}

// ---------------------------------------------------------------------------
// Cost model (integers only).
// ---------------------------------------------------------------------------
namespace {

uint64_t kernel_ps(u128 as_mem, u128 as_tensor, u128 as_alu, const Calibration& cal)
{
    return saturate(max3(as_mem, as_tensor, as_alu) / 1000000u + (u128)cal.c[5]);
}

uint64_t operand_bytes(int operand) { return operand == MNN_OPERAND_BF16 ? 2 : 4; }
uint64_t tensor_as(int operand, const Calibration& cal) { return (uint64_t)(operand == MNN_OPERAND_BF16 ? cal.c[3] : cal.c[2]); }

uint64_t direct_cost(const LayerShape& s, const Calibration& cal)
{
    const uint64_t x_bytes = 4ull * s.N * s.Cin * s.H * s.W;
    const uint64_t y_bytes = 4ull * s.N * s.Cout * s.OH * s.OW;
    const uint64_t w_bytes = 4ull * s.Cout * (s.Cin / s.groups) * s.k * s.k;
    const uint64_t flops = 2ull * s.N * s.Cout * (s.Cin / s.groups) * s.OH * s.OW * s.k * s.k;
    // layers with at most 4 input channels (groups 1) run a dedicated kernel with its own rate (consts[9])
    const bool stem = s.groups == 1 && s.Cin <= 4 && cal.c[9] > 0 &&
                      (long long)s.Cin * s.k * s.k * ((s.Cout + 31) / 32 * 32) * 4 <= 160 * 1024 && s.N <= 65535;
    // consts[9] is measured on the 3 -> 32, 3x3, stride 2 layer, which has a kernel of its own (blocks of output
    // pixels per thread); the other few-channel shapes run the one-pixel kernel at half that rate
    const bool pixel_blocks = s.Cin == 3 && s.k == 3 && s.stride == 2 && s.pad == 1 && s.dil == 1 && s.H % 2 == 0 &&
                              s.W % 4 == 0 && (long long)27 * ((s.Cout + 31) / 32 * 32) * 4 <= 48 * 1024;
    const uint64_t rate = (uint64_t)(stem ? (pixel_blocks ? cal.c[9] : 2 * cal.c[9]) : cal.c[8]);
    return kernel_ps((u128)(x_bytes + y_bytes + w_bytes) * (uint64_t)cal.c[0], 0, (u128)flops * rate, cal);
}

}  // namespace

void contract_tiling(long long tile_blocks, int alpha2, int Cout, int num_sms, int* bn_out, int* n_co_blocks)
{
    const int co16 = (Cout + 15) / 16 * 16;
    const int min_blocks = (co16 + 255) / 256;
    long long best_cost = -1;
    for (int mult = 1; mult <= 4; mult *= 2) {
        const int blocks = min_blocks * mult;
        const int bn = ((co16 / 16 + blocks - 1) / blocks) * 16;
        if (bn < 32 && mult > 1) break;
        const int real_blocks = (co16 + bn - 1) / bn;
        const long long items = tile_blocks * real_blocks * alpha2;
        const long long rounds = (items + num_sms - 1) / num_sms;
        const long long cost = rounds * (128 + bn);
        if (best_cost < 0 || cost < best_cost) {
            best_cost = cost;
            *bn_out = bn;
            *n_co_blocks = real_blocks;
        }
    }
}

bool gemm_reads_x(const LayerShape& s, int operand, int passes)
{
    return s.k == 1 && s.stride == 1 && s.pad == 0 && s.groups == 1 && operand == MNN_OPERAND_TF32 && passes == 1 &&
           s.H * s.W >= 32 && (s.H * s.W) % 4 == 0;
}

namespace {

// lhs: MNN_GEMM_LHS_PATCHES (gather kernel + GEMM), MNN_GEMM_LHS_X (the GEMM reads x itself) or
// MNN_GEMM_LHS_IMPLICIT (producer warps gather the patches inside the GEMM kernel)
uint64_t gemm_cost(const LayerShape& s, int operand, int lhs, const Calibration& cal)
{
    const bool lhs_x = lhs == MNN_GEMM_LHS_X;
    const uint64_t b = operand_bytes(operand);
    const uint64_t Kp = round_up((uint64_t)s.Cin * s.k * s.k, 8);
    const uint64_t T = (uint64_t)s.N * s.OH * s.OW;
    const uint64_t x_bytes = 4ull * s.N * s.Cin * s.H * s.W;
    const uint64_t y_bytes = 4ull * s.N * s.Cout * s.OH * s.OW;
    const uint64_t v_bytes = T * Kp * b, u_bytes = (uint64_t)s.Cout * Kp * b;
    // the patch gather (measured rates): a transposition at about two thirds of the copy rate for 1x1 stride-1
    // layers, the gather staged through shared memory at about a third of it for k > 1, the element-wise gather
    // at about a fifth of it for strided 1x1 layers
    const bool transposer = s.k == 1 && s.stride == 1 && s.pad == 0 && (s.H * s.W) % 4 == 0;
    const uint64_t gather = kernel_ps((u128)(x_bytes + v_bytes) * (uint64_t)cal.c[0] * (transposer ? 3u : (s.k > 1 ? 6u : 10u)) / 2u, 0, 0, cal);
    // The contraction as the kernel schedules it: rounds of work items over the SMs, each item a serial loop
    // over blocks of K whose pace is the slower of the tensor core and the delivery of the two operand tiles
    // from L2 to one SM (about 63 GB/s measured, for either left operand).  With x as the left operand a work
    // item covers up to four 32-pixel atoms of one image, so images whose atom count is not a multiple of four
    // leave part of their last item empty.
    const int sms = cal.c[7] > 0 ? (int)cal.c[7] : 148;
    const uint64_t tile_blocks = lhs_x ? (uint64_t)s.N * ceil_div(ceil_div((uint64_t)s.H * s.W, 32), 4) : ceil_div(T, 128);
    int bn = 256, n_co_blocks = 1;
    contract_tiling((long long)tile_blocks, 1, s.Cout, sms, &bn, &n_co_blocks);
    const uint64_t rounds = ceil_div(tile_blocks * (uint64_t)n_co_blocks, (uint64_t)sms);
    const uint64_t k_elems = 128 / b, k_blocks = ceil_div(Kp, k_elems);
    const uint64_t deliver_ps = (128ull * 128 + (uint64_t)bn * 128) * 16;
    const uint64_t mma_ps = saturate((u128)(2ull * 128 * bn * k_elems) * tensor_as(operand, cal) * (uint64_t)sms / 1000000u);
    // an item's accumulator (128 x bn fp32) is drained at about 22 GB/s per SM while the next item's loop runs
    // (two accumulators), with about half a microsecond of hand-over per item; the last drain is exposed
    const uint64_t drain_ps = 128ull * bn * 4 * 45;
    const uint64_t loop_ps = k_blocks * (deliver_ps > mma_ps ? deliver_ps : mma_ps);
    if (lhs == MNN_GEMM_LHS_IMPLICIT) {
        // only the weight tile is delivered; the producers' gather of 128 x 32 patch elements paces a block too
        const uint64_t deliver_b = (uint64_t)bn * 128 * 16;
        // (consts[13] is measured on the tap-major gather, Cin a multiple of 32; the element-wise gather of other
        // channel counts takes about twice as long)
        const uint64_t gather_ps = saturate((u128)128 * 32 * (uint64_t)cal.c[13] * (s.Cin % 32 == 0 ? 1u : 2u) / 1000000u);
        uint64_t block_ps = deliver_b > mma_ps ? deliver_b : mma_ps;
        if (gather_ps > block_ps) block_ps = gather_ps;
        const uint64_t loop_i = k_blocks * block_ps;
        const uint64_t item_i = loop_i > drain_ps + 500000 ? loop_i : drain_ps + 500000;
        const u128 serial_i = ((u128)rounds * item_i + drain_ps) * 1000000u;
        return kernel_ps((u128)(x_bytes + u_bytes + y_bytes) * (uint64_t)cal.c[0], serial_i, 0, cal);
    }
    const uint64_t item_ps = loop_ps > drain_ps + 500000 ? loop_ps : drain_ps + 500000;
    const u128 serial_as = ((u128)rounds * item_ps + drain_ps) * 1000000u;
    if (lhs_x) return kernel_ps((u128)(x_bytes + u_bytes + y_bytes) * (uint64_t)cal.c[0], serial_as, 0, cal);
    const uint64_t contract = kernel_ps((u128)(v_bytes + u_bytes + y_bytes) * (uint64_t)cal.c[0], serial_as, 0, cal);
    return saturate((u128)gather + contract);
}

uint64_t winograd_chunk_cost(const LayerShape& s, int m, int operand, int passes, uint64_t n, bool resident,
                             const Calibration& cal)
{
    const uint64_t alpha = (uint64_t)(m + s.k - 1), a2 = alpha * alpha;
    const uint64_t tiles_img = ceil_div(s.OH, m) * ceil_div(s.OW, m);
    const uint64_t Cp = round_up(s.Cin, 8);
    const uint64_t b_el = operand_bytes(operand) * (passes == 3 ? 2 : 1);
    const uint64_t v_bytes = n * a2 * tiles_img * Cp * b_el;
    const uint64_t m_bytes = n * a2 * (uint64_t)s.Cout * tiles_img * 4;
    const uint64_t u_bytes = a2 * (uint64_t)s.Cout * Cp * b_el;
    const uint64_t x_bytes = 4ull * n * s.Cin * s.H * s.W;
    const uint64_t y_bytes = 4ull * n * s.Cout * s.OH * s.OW;
    const uint64_t cV = (uint64_t)(resident ? cal.c[1] : cal.c[0]);
    const uint64_t c0 = (uint64_t)cal.c[0], cA = (uint64_t)cal.c[4];
    // from alpha = 8 on a lane of the input transform holds one channel instead of a packed pair (twice the ALU
    // time) and does the tile in sweeps of columns; measured against the pair form: x 2 at alpha = 8, x 2.25 at
    // alpha = 10, x 4 at alpha = 12 (quarters: 8, 9, 16)
    const u128 tile_channels_in = (u128)n * tiles_img * (uint64_t)s.Cin, tile_channels_out = (u128)n * tiles_img * (uint64_t)s.Cout;
    const u128 in_alu = (alpha >= 12 ? 16u : (alpha >= 10 ? 9u : (alpha >= 8 ? 8u : 4u))) * alpha * a2 * tile_channels_in * cA;
    const uint64_t in = kernel_ps((u128)x_bytes * c0 + (u128)v_bytes * cV, 0, in_alu, cal);
    // the contraction's work items (128 tiles x bn channels x one position) run in rounds over the SMs: its
    // tensor time is that of full rounds
    const uint64_t sms = cal.c[7] > 0 ? (uint64_t)cal.c[7] : 148;
    const uint64_t tile_blocks = ceil_div(n * tiles_img, 128);
    int bn = 0, co_blocks = 1;
    contract_tiling((long long)tile_blocks, (int)a2, s.Cout, (int)sms, &bn, &co_blocks);
    const uint64_t items = tile_blocks * (uint64_t)co_blocks * a2, rounds = ceil_div(items, sms);
    // (per item first: the product with rounds x SMs then stays below twice the plain tensor time)
    const u128 con_tensor = 2u * a2 * Cp * tile_channels_out * (uint64_t)passes * tensor_as(operand, cal) / items * (rounds * sms);
    const uint64_t con = kernel_ps((u128)(v_bytes + m_bytes) * cV + (u128)u_bytes * c0, con_tensor, 0, cal);
    const uint64_t out = kernel_ps((u128)m_bytes * cV + (u128)y_bytes * c0, 0,
                                   2u * (uint64_t)m * alpha * (alpha + m) * tile_channels_out * cA, cal);
    return saturate((u128)in + con + out);
}

// Winograd F(2x2, 3x3) as one kernel: HBM sees x, y and U only.  A work item (32 tiles x 128 output channels)
// is a serial loop over blocks of 32 input channels; a block costs the delivery of sixteen 128 x 32 weight tiles
// from L2 to the SM or its sixty-four small MMAs, whichever is larger; the item's epilogue is not overlapped
// (the sixteen accumulators fill tensor memory).
uint64_t fused_cost(const LayerShape& s, const Calibration& cal)
{
    const uint64_t tiles = (uint64_t)s.N * ceil_div(s.OH, 2) * ceil_div(s.OW, 2);
    const uint64_t sms = cal.c[7] > 0 ? (uint64_t)cal.c[7] : 148;
    const uint64_t x_bytes = 4ull * s.N * s.Cin * s.H * s.W;
    const uint64_t y_bytes = 4ull * s.N * s.Cout * s.OH * s.OW;
    const uint64_t u_bytes = 16ull * s.Cout * s.Cin * 4;
    const uint64_t co_blocks = ceil_div(s.Cout, 128);
    const uint64_t rounds = ceil_div(ceil_div(tiles, 32) * co_blocks, sms);
    const uint64_t k_blocks = ceil_div(s.Cin, 32);
    const uint64_t deliver_ps = 16ull * 128 * 32 * 4 * (uint64_t)cal.c[10] / 1000000ull;
    const uint64_t block_ps = deliver_ps > (uint64_t)cal.c[11] ? deliver_ps : (uint64_t)cal.c[11];
    const u128 item_ps = (u128)k_blocks * block_ps + (uint64_t)cal.c[12];
    const u128 serial_as = (u128)rounds * item_ps * 1000000u;
    // x comes from HBM once; the other channel blocks find it in L2
    return kernel_ps((u128)(x_bytes + y_bytes + u_bytes) * (uint64_t)cal.c[0] + (u128)(co_blocks - 1) * x_bytes * (uint64_t)cal.c[1],
                     serial_as, 0, cal);
}

}  // namespace

bool fused_shape_ok(const LayerShape& s)
{
    return s.k == 3 && s.stride == 1 && s.dil == 1 && s.groups == 1 && s.pad <= 2;
}

// Eq. 2, made comparable across tile sizes: a per-tile count, so multiplied by the number of tiles; its third
// term (the output transform) with the output-channel factor it lacks as printed.
uint64_t paper_multiplications(const LayerShape& s, int n)
{
    const uint64_t a = (uint64_t)(n + s.k - 1);
    const u128 tiles = (u128)s.N * ceil_div(s.OH, n) * ceil_div(s.OW, n);
    const u128 per_tile = (u128)2 * s.Cin * a * a * a + (u128)s.Cin * s.Cout * a * a + (u128)s.Cout * n * a * (2 * n + s.k - 1);
    return saturate(tiles * per_tile);
}

void winograd_chunking(const LayerShape& s, int m, int operand, int passes, const Calibration& cal,
                       int* chunk_images, int* n_chunks, uint64_t* cost_ps)
{
    const uint64_t alpha = (uint64_t)(m + s.k - 1), a2 = alpha * alpha;
    const uint64_t tiles_img = ceil_div(s.OH, m) * ceil_div(s.OW, m);
    const uint64_t Cp = round_up(s.Cin, 8);
    const uint64_t b_el = operand_bytes(operand) * (passes == 3 ? 2 : 1);
    const uint64_t per_img = a2 * tiles_img * Cp * b_el + a2 * (uint64_t)s.Cout * tiles_img * 4;
    const uint64_t N = (uint64_t)s.N;
    const uint64_t n_fit = per_img ? (uint64_t)cal.c[6] / per_img : N;
    // the transformed tensors of one chunk may not exceed kMaxChunkBytes, whatever the cost says
    uint64_t n_cap = per_img ? kMaxChunkBytes / per_img : N;
    if (n_cap < 1) n_cap = 1;

    // option A: the largest chunk the cap allows (the whole batch if it fits)
    const uint64_t chunkA = N < n_cap ? N : ceil_div(N, ceil_div(N, n_cap));
    const uint64_t nA = ceil_div(N, chunkA);
    const uint64_t costA = saturate((u128)nA * winograd_chunk_cost(s, m, operand, passes, chunkA, n_fit >= chunkA, cal));
    uint64_t best_cost = costA;
    uint64_t best_chunk = chunkA, best_n = nA;
    // Cutting the batch further so that a chunk's V and M stay in L2 was measured on B200 and never paid:
    // the fixed cost of three more kernels per chunk outweighs what the kernels gain from L2-resident
    // operands.  The L2 rate is still used for the byte cost when a whole chunk fits.
    *chunk_images = (int)best_chunk;
    *n_chunks = (int)best_n;
    *cost_ps = best_cost;
}

int plan_layer(const LayerShape& s, const mnn_conv_opts& o, const Calibration& cal, Decision* d, const char** err)
{
    static const int kM[3] = {2, 4, 6};
    for (int i = 0; i < MNN_N_CANDIDATES; ++i) d->cost_ps[i] = MNN_COST_INADMISSIBLE;

    const uint64_t tol_ppm = o.precision == MNN_PREC_BF16 ? 10000 : 1000;
    const uint64_t gate_ppm = tol_ppm * kGateNumerator / kGateDenominator;
    const bool fully_forced = o.force_m != 0 && o.operand != 0 && o.passes != 0;
    const bool wino_shape_ok = s.stride == 1 && s.dil == 1 && s.groups == 1 && s.k >= 2 && s.k <= 7;

    struct Cand { int algo, m, operand, passes; };
    Cand cands[MNN_N_CANDIDATES];
    cands[0] = {MNN_ALGO_DIRECT, 0, 0, 0};
    cands[1] = {MNN_ALGO_GEMM, 0, MNN_OPERAND_TF32, 1};
    cands[2] = {MNN_ALGO_GEMM, 0, MNN_OPERAND_BF16, 1};
    for (int g = 0; g < 4; ++g)
        for (int i = 0; i < 3; ++i)
            cands[3 + g * 3 + i] = {MNN_ALGO_WINOGRAD, kM[i], g < 2 ? MNN_OPERAND_TF32 : MNN_OPERAND_BF16, (g & 1) ? 3 : 1};
    cands[15] = {MNN_ALGO_WINOGRAD, 2, MNN_OPERAND_TF32, 1};      // the fused kernel
    {
        static const int kN[4] = {1, 2, 4, 6};
        int arg = 0;
        for (int i = 0; i < 4; ++i) {
            d->paper_mul[i] = paper_multiplications(s, kN[i]);
            if (d->paper_mul[i] < d->paper_mul[arg]) arg = i;
        }
        d->paper_n_hat = kN[arg];
    }

    int chunk_of[MNN_N_CANDIDATES] = {0}, nch_of[MNN_N_CANDIDATES] = {0}, pts_of[MNN_N_CANDIDATES] = {0};
    int lhs_of[MNN_N_CANDIDATES] = {0};
    long long ppm_of[MNN_N_CANDIDATES] = {0};

    for (int i = 0; i < MNN_N_CANDIDATES; ++i) {
        const Cand& c = cands[i];
        if (o.fused == 2 && i != 15) continue;                     // the fused kernel or nothing
        if (o.force_algo != MNN_ALGO_AUTO && o.force_algo != c.algo) continue;
        if (c.algo == MNN_ALGO_DIRECT) {
            if (o.operand == MNN_OPERAND_FP32_REF || o.operand == MNN_OPERAND_AUTO || o.force_algo == MNN_ALGO_DIRECT)
                d->cost_ps[i] = direct_cost(s, cal);
            continue;
        }
        if (o.operand != MNN_OPERAND_AUTO && o.operand != c.operand) continue;
        if (o.passes != 0 && o.passes != c.passes) continue;
        if (c.algo == MNN_ALGO_GEMM) {
            if (s.groups != 1) continue;
            if (o.force_m != 0) continue;
            long long ppm = accuracy_ppm(1, s.k, 0, c.operand, c.passes);
            if (ppm < 0) continue;
            if ((uint64_t)ppm > gate_ppm && !(o.operand != 0 && o.force_algo == MNN_ALGO_GEMM)) continue;
            // left operand: the patch matrix, or x itself where that applies (whichever is cheaper)
            const bool x_ok = gemm_reads_x(s, c.operand, c.passes);
            const bool implicit_ok = c.operand == MNN_OPERAND_TF32 && c.passes == 1;
            if (o.gemm_lhs == MNN_GEMM_LHS_X && !x_ok) continue;
            if (o.gemm_lhs == MNN_GEMM_LHS_IMPLICIT && !implicit_ok) continue;
            const uint64_t cost_patches = gemm_cost(s, c.operand, MNN_GEMM_LHS_PATCHES, cal);
            const uint64_t cost_x = x_ok ? gemm_cost(s, c.operand, MNN_GEMM_LHS_X, cal) : MNN_COST_INADMISSIBLE;
            const uint64_t cost_i = implicit_ok ? gemm_cost(s, c.operand, MNN_GEMM_LHS_IMPLICIT, cal) : MNN_COST_INADMISSIBLE;
            // left operand: as asked for, else the cheapest that applies (patch matrix, x itself, implicit gather;
            // earlier in this order on ties; the implicit gather only once its rate constant is known)
            int lhs = o.gemm_lhs;
            if (lhs == MNN_GEMM_LHS_AUTO) {
                lhs = MNN_GEMM_LHS_PATCHES;
                uint64_t best_lhs = cost_patches;
                if (x_ok && cost_x < best_lhs) {
                    lhs = MNN_GEMM_LHS_X;
                    best_lhs = cost_x;
                }
                // (plain pointwise layers keep the tuned paths: measured, the implicit gather never beat them there)
                const bool pointwise = s.k == 1 && s.stride == 1;
                if (implicit_ok && !pointwise && cal.c[13] > 0 && cost_i < best_lhs) lhs = MNN_GEMM_LHS_IMPLICIT;
            }
            const bool take_x = lhs == MNN_GEMM_LHS_X;
            if (take_x && ppm < kGemmLhsXErrorPpm) ppm = kGemmLhsXErrorPpm;
            lhs_of[i] = lhs;
            ppm_of[i] = ppm;
            d->cost_ps[i] = lhs == MNN_GEMM_LHS_X ? cost_x : (lhs == MNN_GEMM_LHS_IMPLICIT ? cost_i : cost_patches);
            continue;
        }
        // Winograd
        const bool fused = i == 15;
        if (fused && (o.fused == 1 || !fused_shape_ok(s) || cal.c[10] <= 0 || cal.c[11] <= 0)) continue;
        if (!wino_shape_ok || !winograd_supported(c.m, s.k)) continue;
        if (o.force_m != 0 && o.force_m != c.m) continue;
        long long ppm = 0;
        int pid = o.points_id;
        if (pid == MNN_POINTS_AUTO) pid = best_points(c.m, s.k, c.operand, c.passes, &ppm);
        else ppm = accuracy_ppm(c.m, s.k, pid, c.operand, c.passes);
        if (pid == 0 || ppm < 0) continue;
        if ((uint64_t)ppm > gate_ppm && !fully_forced) continue;
        pts_of[i] = pid;
        ppm_of[i] = ppm;
        uint64_t cost;
        if (fused) {
            chunk_of[i] = s.N;
            nch_of[i] = 1;
            cost = fused_cost(s, cal);
        } else {
            winograd_chunking(s, c.m, c.operand, c.passes, cal, &chunk_of[i], &nch_of[i], &cost);
        }
        d->cost_ps[i] = cost;
    }

    int best = -1;
    for (int i = 0; i < MNN_N_CANDIDATES; ++i)
        if (d->cost_ps[i] != MNN_COST_INADMISSIBLE && (best < 0 || d->cost_ps[i] < d->cost_ps[best])) best = i;

    // A forced combination outside the candidate list (other m, fp32 checking contraction).
    const bool off_list = o.force_algo == MNN_ALGO_WINOGRAD && o.force_m != 0 &&
                          (o.operand == MNN_OPERAND_FP32_REF || !(o.force_m == 2 || o.force_m == 4 || o.force_m == 6));
    if (off_list || (best < 0 && o.force_algo == MNN_ALGO_GEMM && o.operand == MNN_OPERAND_FP32_REF)) {
        if (o.force_algo == MNN_ALGO_WINOGRAD) {
            if (!wino_shape_ok || !winograd_supported(o.force_m, s.k)) {
                *err = "Winograd needs stride 1, dilation 1, groups 1, k in {2,3,5,7}, m in {2,4,6}";
                return MNN_EUNSUPPORTED;
            }
            const int operand = o.operand == 0 ? MNN_OPERAND_TF32 : o.operand;
            const int passes = o.passes == 0 ? 1 : o.passes;
            d->algo = MNN_ALGO_WINOGRAD;
            d->m = o.force_m;
            d->alpha = o.force_m + s.k - 1;
            d->operand = operand;
            d->passes = operand == MNN_OPERAND_FP32_REF ? 1 : passes;
            long long ppm = 0;
            d->points_id = o.points_id ? o.points_id : best_points(d->m, s.k, operand, d->passes, &ppm);
            d->error_ppm = accuracy_ppm(d->m, s.k, d->points_id, operand, d->passes);
            uint64_t cost;
            winograd_chunking(s, d->m, operand == MNN_OPERAND_FP32_REF ? MNN_OPERAND_TF32 : operand, d->passes, cal,
                              &d->chunk_images, &d->n_chunks, &cost);
        } else {
            if (s.groups != 1) {
                *err = "the GEMM scheme needs groups = 1";
                return MNN_EUNSUPPORTED;
            }
            d->algo = MNN_ALGO_GEMM;
            d->gemm_lhs = MNN_GEMM_LHS_PATCHES;
            d->m = 1;
            d->alpha = 1;
            d->operand = MNN_OPERAND_FP32_REF;
            d->passes = 1;
            d->points_id = 0;
            d->error_ppm = accuracy_ppm(1, s.k, 0, MNN_OPERAND_FP32_REF, 1);
            d->chunk_images = s.N;
            d->n_chunks = 1;
        }
        d->chosen = -1;
        if (o.chunk_images > 0 && d->algo == MNN_ALGO_WINOGRAD) {
            d->chunk_images = o.chunk_images < s.N ? o.chunk_images : s.N;
            d->n_chunks = (s.N + d->chunk_images - 1) / d->chunk_images;
        }
        return MNN_OK;
    }

    if (best < 0) {
        *err = "no scheme satisfies the forced options and the accuracy gate for this layer";
        return MNN_EUNSUPPORTED;
    }
    const Cand& c = cands[best];
    d->chosen = best;
    d->algo = c.algo;
    d->operand = c.operand;
    d->passes = c.passes;
    d->error_ppm = ppm_of[best];
    if (c.algo == MNN_ALGO_WINOGRAD) {
        d->m = c.m;
        d->alpha = c.m + s.k - 1;
        d->points_id = pts_of[best];
        d->chunk_images = chunk_of[best];
        d->n_chunks = nch_of[best];
        d->fused = best == 15 ? 1 : 0;
        if (o.chunk_images > 0 && !d->fused) {
            d->chunk_images = o.chunk_images < s.N ? o.chunk_images : s.N;
            d->n_chunks = (s.N + d->chunk_images - 1) / d->chunk_images;
        }
    } else {
        d->m = 1;
        d->alpha = 1;
        d->points_id = 0;
        d->chunk_images = s.N;
        d->n_chunks = 1;
        d->gemm_lhs = c.algo == MNN_ALGO_GEMM ? lhs_of[best] : 0;
    }
    return MNN_OK;
}

}  // namespace mnnb
