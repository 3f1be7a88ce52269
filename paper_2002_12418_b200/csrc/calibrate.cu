// One-time calibration of the planner's cost constants (the FLOPS and t_schedule
// of Eq. 5, which the paper's appendix "Backend cost evaluation" obtains by running
// a network 100 times on each GPU): micro-benchmarks of this library's own kernels
// on the current device.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstring>
#include <string>
#include <vector>

#include "../../include/mnn_conv.h"
#include "generator.h"
#include "implicit_gemm.h"
#include "contract_umma.h"
#include "kernels.h"
#include "planner.h"
#include "wino_fused.h"

using namespace mnnb;

namespace {

__global__ void copy_kernel(const float4* __restrict__ src, float4* __restrict__ dst, size_t n)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        dst[i] = src[i];
}

__global__ void empty_kernel() {}

__global__ void fill_kernel(float* p, size_t n, float scale)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        p[i] = scale * (float)((i * 2654435761u) & 1023u) * (1.0f / 1024.0f) - 0.5f * scale;
}

struct Timer {
    cudaEvent_t a = nullptr, b = nullptr;
    cudaStream_t st;
    explicit Timer(cudaStream_t s) : st(s)
    {
        cudaEventCreate(&a);
        cudaEventCreate(&b);
    }
    ~Timer()
    {
        if (a) cudaEventDestroy(a);
        if (b) cudaEventDestroy(b);
    }
    void start() { cudaEventRecord(a, st); }
    // milliseconds
    double stop()
    {
        cudaEventRecord(b, st);
        cudaEventSynchronize(b);
        float ms = 0.0f;
        cudaEventElapsedTime(&ms, a, b);
        return (double)ms;
    }
};

long long to_ll(double v) { return v < 1.0 ? 1 : (long long)(v + 0.5); }

}  // namespace

extern "C" int mnn_calibrate(int device, void* stream, long long consts[MNN_N_CONSTS])
{
    // reported through mnn_last_error by the callers in api.cu; keep the reason local here
    if (!consts) return MNN_EINVAL;
    cudaError_t e = cudaSetDevice(device);
    if (e != cudaSuccess) return MNN_ECUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    Calibration cal = default_calibration();
    int sms = 0, l2 = 0;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
    cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, device);
    if (sms > 0) cal.c[7] = sms;
    if (l2 > 0) cal.c[6] = (long long)l2 / 8 * 5;       // five eighths of L2 for one chunk's V + M

    const size_t big = 512ull << 20, small = 16ull << 20;
    char* buf = nullptr;
    e = cudaMalloc(&buf, 2 * big);
    if (e != cudaSuccess) return MNN_ECUDA;
    Timer tm(st);
    const int blocks = (sms > 0 ? sms : 148) * 8;

    fill_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<float*>(buf), 2 * big / 4, 1.0f);
    // HBM: stream 512 MB -> 512 MB
    for (int i = 0; i < 2; ++i)
        copy_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<float4*>(buf), reinterpret_cast<float4*>(buf + big), big / 16);
    tm.start();
    const int hbm_reps = 5;
    for (int i = 0; i < hbm_reps; ++i)
        copy_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<float4*>(buf), reinterpret_cast<float4*>(buf + big), big / 16);
    double ms = tm.stop();
    cal.c[0] = to_ll(ms * 1e15 / ((double)hbm_reps * 2.0 * (double)big));
    // L2: 16 MB -> 16 MB, resident
    for (int i = 0; i < 3; ++i)
        copy_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<float4*>(buf), reinterpret_cast<float4*>(buf + small), small / 16);
    tm.start();
    const int l2_reps = 50;
    for (int i = 0; i < l2_reps; ++i)
        copy_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<float4*>(buf), reinterpret_cast<float4*>(buf + small), small / 16);
    ms = tm.stop();
    // includes the launch gaps: subtract them below once the launch cost is known
    const double l2_ms_per = ms / l2_reps;
    // launch cost
    for (int i = 0; i < 20; ++i) empty_kernel<<<1, 32, 0, st>>>();
    tm.start();
    const int launch_reps = 500;
    for (int i = 0; i < launch_reps; ++i) empty_kernel<<<1, 32, 0, st>>>();
    ms = tm.stop();
    const double launch_ms = ms / launch_reps;
    cal.c[5] = to_ll(launch_ms * 1e9);
    {
        double t = l2_ms_per - launch_ms;
        if (t < l2_ms_per * 0.25) t = l2_ms_per * 0.25;
        cal.c[1] = to_ll(t * 1e15 / (2.0 * (double)small));
        if (cal.c[1] > cal.c[0]) cal.c[1] = cal.c[0];
    }

    // tensor rates: the contraction kernel on an L2-friendly problem
    for (int kind = 0; kind < 2; ++kind) {
        const int mode = kind == 0 ? STORE_TF32 : STORE_BF16;
        const int eb = kind == 0 ? 4 : 2;
        const int alpha2 = 4, Cout = 256, cin = 1024;
        const long long tiles = 4096;
        const size_t u_bytes = (size_t)alpha2 * Cout * cin * eb, v_bytes = (size_t)alpha2 * tiles * cin * eb;
        const size_t m_bytes = (size_t)alpha2 * Cout * tiles * 4;
        char* U = buf + 1024;
        char* V = U + ((u_bytes + 1023) / 1024) * 1024;
        char* M = V + ((v_bytes + 1023) / 1024) * 1024;
        if ((size_t)(M - buf) + m_bytes > 2 * big) continue;
        cudaMemsetAsync(buf, 0, 1024, st);                 // status word
        UmmaContract uc;
        const char* why = "";
        if (umma_contract_setup(&uc, mode, alpha2, Cout, cin, tiles, U, nullptr, V, nullptr, &why) != cudaSuccess) continue;
        ContractEpilogue epi = {0, reinterpret_cast<float*>(M), tiles, nullptr, nullptr, 0, 1};
        int* status = reinterpret_cast<int*>(buf);
        for (int i = 0; i < 3; ++i) launch_contract_umma(uc, tiles, epi, status, st);
        tm.start();
        const int reps = 10;
        for (int i = 0; i < reps; ++i) launch_contract_umma(uc, tiles, epi, status, st);
        ms = tm.stop();
        int code = 0;
        cudaMemcpy(&code, status, sizeof(int), cudaMemcpyDeviceToHost);
        if (code != 0) continue;
        double t = ms / reps - launch_ms;
        if (t < ms / reps * 0.25) t = ms / reps * 0.25;
        const double flops = 2.0 * alpha2 * (double)tiles * Cout * cin;
        cal.c[2 + kind] = to_ll(t * 1e15 / flops);
    }

    // fixed cost of one kernel of the pipeline (launch, ramp-up, tail): the contraction on a problem of four work items
    {
        const int alpha2 = 4, Cout = 128, cin = 64;
        const long long tiles = 128;
        char* U = buf + 1024;
        char* V = U + (1 << 20);
        char* M = V + (1 << 20);
        cudaMemsetAsync(buf, 0, 1024, st);
        UmmaContract uc;
        const char* why = "";
        if (umma_contract_setup(&uc, STORE_BF16, alpha2, Cout, cin, tiles, U, nullptr, V, nullptr, &why) == cudaSuccess) {
            ContractEpilogue epi = {0, reinterpret_cast<float*>(M), tiles, nullptr, nullptr, 0, 1};
            int* status = reinterpret_cast<int*>(buf);
            for (int i = 0; i < 5; ++i) launch_contract_umma(uc, tiles, epi, status, st);
            tm.start();
            const int reps = 50;
            for (int i = 0; i < reps; ++i) launch_contract_umma(uc, tiles, epi, status, st);
            ms = tm.stop();
            int code = 0;
            cudaMemcpy(&code, status, sizeof(int), cudaMemcpyDeviceToHost);
            if (code == 0 && ms > 0.0) cal.c[5] = to_ll(ms / reps * 1e9);
        }
    }

    // direct kernel rate: 3x3, 64 -> 64 channels, 56 x 56, 4 images
    {
        DirectGeom g = {4, 64, 64, 56, 56, 56, 56, 3, 1, 1, 1, 1, 1};
        float* x = reinterpret_cast<float*>(buf);
        float* w = x + (size_t)4 * 64 * 56 * 56;
        float* y = w + 64 * 64 * 9 + 64;
        fill_kernel<<<blocks, 256, 0, st>>>(x, (size_t)(y - x), 1.0f);
        for (int i = 0; i < 2; ++i) launch_direct(x, w, nullptr, y, g, st);
        tm.start();
        const int reps = 5;
        for (int i = 0; i < reps; ++i) launch_direct(x, w, nullptr, y, g, st);
        ms = tm.stop();
        const double flops = 2.0 * 4 * 64 * 64 * 56 * 56 * 9;
        double t = ms / reps - launch_ms;
        if (t < ms / reps * 0.25) t = ms / reps * 0.25;
        cal.c[8] = to_ll(t * 1e15 / flops);
    }

    // rate of the direct kernel for very few input channels: 3x3 stride 2, 3 -> 32 channels, 224 x 224, 32 images
    // (several waves of CTAs: a handful of images would measure the ramp-up instead of the rate)
    {
        DirectGeom g = {32, 3, 32, 224, 224, 112, 112, 3, 2, 1, 1, 1, 1};
        float* x = reinterpret_cast<float*>(buf);
        float* w = x + (size_t)32 * 3 * 224 * 224;
        float* y = w + 32 * 27 + 32;
        if (direct_stem_applies(g)) {
            for (int i = 0; i < 2; ++i) launch_direct(x, w, nullptr, y, g, st);
            tm.start();
            const int reps = 5;
            for (int i = 0; i < reps; ++i) launch_direct(x, w, nullptr, y, g, st);
            ms = tm.stop();
            const double flops = 2.0 * 32 * 32 * 3 * 112 * 112 * 9;
            double t = ms / reps - launch_ms;
            if (t < ms / reps * 0.25) t = ms / reps * 0.25;
            cal.c[9] = to_ll(t * 1e15 / flops);
        }
    }

    // transform ALU rate: the alpha = 8 input transform on L2-resident data
    {
        WinogradMatrices wm;
        if (generate_winograd(6, 3, 3, &wm)) {
            TransformMatrices mats;
            std::memset(&mats, 0, sizeof(mats));
            std::memcpy(mats.Bt, wm.Bt32.data(), wm.Bt32.size() * sizeof(float));
            WinoGeom g;
            g.images = 4; g.Cin = 64; g.Cout = 64; g.H = 56; g.W = 56; g.OH = 56; g.OW = 56; g.k = 3; g.pad = 1;
            g.m = 6; g.alpha = 8; g.th = 10; g.tw = 10; g.cin_pad = 64;
            g.tiles = 400; g.v_plane = 400 * 64; g.m_row_stride = 416;
            float* x = reinterpret_cast<float*>(buf);
            float* V = x + (size_t)4 * 64 * 56 * 56;
            for (int i = 0; i < 2; ++i) launch_input_transform(x, V, nullptr, g, STORE_TF32, mats, nullptr, st);
            tm.start();
            const int reps = 10;
            for (int i = 0; i < reps; ++i) launch_input_transform(x, V, nullptr, g, STORE_TF32, mats, nullptr, st);
            ms = tm.stop();
            double t = ms / reps - launch_ms;
            if (t < ms / reps * 0.25) t = ms / reps * 0.25;
            const double flops = 4.0 * 8 * 64 * (double)g.tiles * 64;
            const long long measured = to_ll(t * 1e15 / flops);
            // the run is partly memory-bound, so this is an upper bound on the ALU cost
            if (measured < cal.c[4]) cal.c[4] = measured;
        }
    }

    // fused F(2x2,3x3) kernel: one work item (32 tiles x 128 output channels) with 32 and with 256 input channels;
    // the difference is seven blocks of 32 input channels, the rest of the short run is launch and epilogue
    {
        WinogradMatrices wm;
        if (generate_winograd(2, 3, 2, &wm)) {
            TransformMatrices mats;
            std::memset(&mats, 0, sizeof(mats));
            std::memcpy(mats.At, wm.At32.data(), wm.At32.size() * sizeof(float));
            std::memcpy(mats.G, wm.G32.data(), wm.G32.size() * sizeof(float));
            std::memcpy(mats.Bt, wm.Bt32.data(), wm.Bt32.size() * sizeof(float));
            double t_of[2] = {0.0, 0.0};
            bool ok = true;
            for (int v = 0; v < 2 && ok; ++v) {
                const int cin = v == 0 ? 32 : 256, cout = 128;
                WinoGeom g;
                g.images = 2; g.Cin = cin; g.Cout = cout; g.H = 8; g.W = 8; g.OH = 8; g.OW = 8; g.k = 3; g.pad = 1;
                g.m = 2; g.alpha = 4; g.th = 4; g.tw = 4; g.cin_pad = cin;
                g.tiles = 32; g.v_plane = 0; g.m_row_stride = 0;
                int* status = reinterpret_cast<int*>(buf);
                float* x = reinterpret_cast<float*>(buf + 1024);
                float* w = x + (size_t)2 * 256 * 64;
                float* y = w + (size_t)128 * 256 * 9;
                char* U = buf + (8 << 20);
                cudaMemsetAsync(buf, 0, 1024, st);
                FusedWino fw;
                const char* why = "";
                if (fused_wino_setup(&fw, cout, cin, U, &why) != cudaSuccess ||
                    launch_fused_wino_weights(w, U, cout, cin, mats, st) != cudaSuccess) {
                    ok = false;
                    break;
                }
                for (int i = 0; i < 3; ++i) launch_fused_wino(fw, x, nullptr, y, g, 0, mats, status, st);
                tm.start();
                const int reps = 20;
                for (int i = 0; i < reps; ++i) launch_fused_wino(fw, x, nullptr, y, g, 0, mats, status, st);
                t_of[v] = tm.stop() / reps;
                int code = 0;
                cudaMemcpy(&code, status, sizeof(int), cudaMemcpyDeviceToHost);
                if (code != 0 || !(t_of[v] > 0.0)) ok = false;
            }
            if (ok && t_of[1] > t_of[0]) {
                const double block_ms = (t_of[1] - t_of[0]) / 7.0;
                cal.c[11] = to_ll(block_ms * 1e9);
                cal.c[10] = to_ll(block_ms * 1e15 / (16.0 * 128 * 32 * 4));
                double epi_ms = t_of[0] - block_ms - (double)cal.c[5] * 1e-9;
                if (epi_ms < block_ms * 0.25) epi_ms = block_ms * 0.25;
                cal.c[12] = to_ll(epi_ms * 1e9);
            }
        }
    }

    // implicit GEMM: pace of the producer warps' gather.  3x3 stride 2, 64 -> 64 channels, 56 x 56, 4 images: 25
    // work items of 18 blocks of 32 patch elements each, one item per SM, so the run is launch + 18 blocks + drain
    {
        GatherGeom g = {4, 64, 56, 56, 28, 28, 3, 2, 1, 1, 576};
        int* status = reinterpret_cast<int*>(buf);
        float* x = reinterpret_cast<float*>(buf + 1024);
        float* U = x + (size_t)4 * 64 * 56 * 56;
        float* y = U + (size_t)64 * 576;
        cudaMemsetAsync(buf, 0, 1024, st);
        ImplicitGemm ig;
        const char* why = "";
        if (implicit_gemm_setup(&ig, g, 64, U, &why) == cudaSuccess) {
            for (int i = 0; i < 3; ++i) launch_implicit_gemm(ig, x, nullptr, y, g, 0, status, st);
            tm.start();
            const int reps = 20;
            for (int i = 0; i < reps; ++i) launch_implicit_gemm(ig, x, nullptr, y, g, 0, status, st);
            ms = tm.stop() / reps;
            int code = 0;
            cudaMemcpy(&code, status, sizeof(int), cudaMemcpyDeviceToHost);
            double t = ms - (double)cal.c[5] * 1e-9;
            if (t < ms * 0.25) t = ms * 0.25;
            if (code == 0 && ms > 0.0) cal.c[13] = to_ll(t * 1e15 / (18.0 * 128 * 32));
        }
    }

    e = cudaStreamSynchronize(st);
    cudaFree(buf);
    if (e != cudaSuccess) return MNN_ECUDA;
    install_calibration(cal);
    for (int i = 0; i < MNN_N_CONSTS; ++i) consts[i] = cal.c[i];
    return MNN_OK;
}
