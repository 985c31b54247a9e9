// Measurement helper (not part of the method): the rate at which this GPU's CUDA cores retire
// the instruction mixes the distance kernels are made of, measured with register-resident
// operands so that nothing but instruction issue limits it.  The benchmark divides a kernel's
// algorithmic instruction count by these rates to get its roofline fraction.
#include "kge_common.cuh"

namespace kge {
namespace {

constexpr int MB_THREADS = 256;
// A thread keeps MB_ACC independent accumulators and takes MB_ROUNDS rounds per trip of the measuring loop.  How the
// registers of a shape fall on the register file's banks changes the rate by a few per cent, so several shapes are
// timed and the best one counts: the question is what the pipes can retire, not what one register allocation does.

// mix 0: one fused multiply-add per element (the dot-product kinds)
// mix 1: subtract, then add the absolute value (p = 1 distance forward): 2 instructions
// mix 2: compare, then a predicated add (p = 1 backward, see add_if_gt): 2 instructions
// mix 3: one special-function exponential (ex2.approx) and one add per element; counted as 1 special-function instruction
template <int MIX, int MB_ACC, int MB_ROUNDS>
__global__ void __launch_bounds__(MB_THREADS) alu_mix_kernel(float* out, float seed, int iters) {
    float acc[MB_ACC], q[MB_ACC];
#pragma unroll
    for (int j = 0; j < MB_ACC; ++j) { acc[j] = 0.f; q[j] = seed * (float)(j + 1) + (float)threadIdx.x * 1e-3f; }
    float t[MB_ROUNDS], w = seed + 1.f;
#pragma unroll
    for (int r = 0; r < MB_ROUNDS; ++r) t[r] = seed * 0.5f + 0.01f * (float)r;
    for (int i = 0; i < iters; i += MB_ROUNDS) {
        // every round of a trip has its own value of the other operand (as a new tail row would bring), so that no
        // two rounds share a subtraction or a comparison; the trip's own instructions (MB_ROUNDS adds that move those
        // values, the counter, the branch) are a few per MB_ROUNDS * MB_ACC measured elements
#pragma unroll
        for (int r = 0; r < MB_ROUNDS; ++r) {
#pragma unroll
            for (int j = 0; j < MB_ACC; ++j) {
                if (MIX == 0) {
                    acc[j] = fmaf(t[r], w, acc[j]);      // (two of the three operands are shared by the round: no register-bank stalls)
                } else if (MIX == 1) {
                    asm volatile("{\n .reg .f32 x;\n sub.f32 x, %1, %2;\n abs.f32 x, x;\n add.f32 %0, %0, x;\n}\n" : "+f"(acc[j]) : "f"(q[j]), "f"(t[r]));
                } else if (MIX == 2) {
                    asm volatile("{\n .reg .pred p;\n setp.gt.f32 p, %1, %2;\n @p add.f32 %0, %0, %3;\n}\n" : "+f"(acc[j]) : "f"(q[j]), "f"(t[r]), "f"(w));
                } else {
                    float e;
                    asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(q[j] - t[r]));
                    acc[j] += e;
                }
            }
            t[r] += 1e-3f;
        }
    }
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < MB_ACC; ++j) s += acc[j];
    if (s == 12345.678f) out[0] = s;   // keeps the loop alive; practically never true
}

}  // namespace
}  // namespace kge

extern "C" int kge_measure_alu(int32_t mix, int32_t iters, double* per_second, void* stream) {
    using namespace kge;
    if (mix < 0 || mix > 3 || iters <= 0 || !per_second) return KGE_ERR_BAD_ARG;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return KGE_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    float* out = nullptr;
    if (cudaMalloc(&out, 256) != cudaSuccess) return KGE_ERR_CUDA;
    cudaEvent_t a, b;
    cudaEventCreate(&a); cudaEventCreate(&b);
    const int grid = sms * 8;                       // 8 resident blocks of 256 threads per SM: every scheduler has 16 warps
    double best_rate = 0.0;
    bool failed = false;
    auto time_shape = [&](auto launch, int acc, int rounds) {
        const int n = (iters + rounds - 1) / rounds * rounds;
        launch(n / 8 + rounds);                     // warm-up
        float best = 1e30f;
        for (int rep = 0; rep < 3; ++rep) {
            cudaEventRecord(a, s);
            launch(n);
            cudaEventRecord(b, s);
            if (cudaEventSynchronize(b) != cudaSuccess) { failed = true; return; }
            float ms = 0.f;
            cudaEventElapsedTime(&ms, a, b);
            best = ms < best ? ms : best;
        }
        const double per_element = (mix == 1 || mix == 2) ? 2.0 : 1.0;      // instructions counted per element of the mix
        const double rate = (double)grid * MB_THREADS * acc * (double)n * per_element / ((double)best * 1e-3);
        best_rate = rate > best_rate ? rate : best_rate;
    };
#define KGE_MB_SHAPE(ACC, ROUNDS)                                                                                     \
    time_shape([&](int n) {                                                                                           \
        switch (mix) {                                                                                                \
            case 0: alu_mix_kernel<0, ACC, ROUNDS><<<grid, MB_THREADS, 0, s>>>(out, 0.37f, n); break;                  \
            case 1: alu_mix_kernel<1, ACC, ROUNDS><<<grid, MB_THREADS, 0, s>>>(out, 0.37f, n); break;                  \
            case 2: alu_mix_kernel<2, ACC, ROUNDS><<<grid, MB_THREADS, 0, s>>>(out, 0.37f, n); break;                  \
            default: alu_mix_kernel<3, ACC, ROUNDS><<<grid, MB_THREADS, 0, s>>>(out, 0.37f, n); break;                 \
        }                                                                                                             \
    }, ACC, ROUNDS)
    KGE_MB_SHAPE(16, 8);
    KGE_MB_SHAPE(8, 8);
    KGE_MB_SHAPE(16, 4);
    KGE_MB_SHAPE(12, 8);
    KGE_MB_SHAPE(8, 16);
#undef KGE_MB_SHAPE
    cudaEventDestroy(a); cudaEventDestroy(b);
    cudaFree(out);
    if (failed || cudaGetLastError() != cudaSuccess) return KGE_ERR_CUDA;
    *per_second = best_rate;
    return KGE_OK;
}
