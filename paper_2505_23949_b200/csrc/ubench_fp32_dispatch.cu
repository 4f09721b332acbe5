// Micro-benchmark behind the roofline of the Dykstra loop: how many fp32 lane operations a
// B200 SM sub-partition retires per clock for the instruction mix of one iteration.
//   part 1: throughput of single instruction kinds (scalar fma, packed fp32x2 fma/add/mul,
//           exp2 and log2 on the SFU, warp shuffle), in clocks per warp instruction;
//   part 2: the element-wise core of one iteration on a 4 x 8 sub-tile per lane (clip, row-sum
//           add, column fma, two scalings; no shuffles), packed and scalar, with and without
//           the clip's min, at 1, 2 and 4 warps per sub-partition.
// Build: nvcc -gencode arch=compute_100a,code=sm_100a -O3 -o ubench_fp32_dispatch ubench_fp32_dispatch.cu
#include <cstdio>
#include <cuda_runtime.h>

#define ITER 4096
template <int KIND> __global__ void single_kind(float* out, float a, float b) {
    float2 v[8];
    for (int i = 0; i < 8; ++i) v[i] = make_float2(threadIdx.x * 1e-3f + i, threadIdx.x * 2e-3f - i);
    const float2 A = make_float2(a, a), B = make_float2(b, b);
    for (int it = 0; it < ITER; ++it) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (KIND == 0) { v[i].x = fmaf(v[i].x, a, b); v[i].y = fmaf(v[i].y, a, b); }
            if (KIND == 1) v[i] = __ffma2_rn(v[i], A, B);
            if (KIND == 2) v[i] = __fadd2_rn(v[i], A);
            if (KIND == 3) v[i] = __fmul2_rn(v[i], A);
            if (KIND == 4) { float y; asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(v[i].x)); v[i].x = y; }
            if (KIND == 5) { float y; asm volatile("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(v[i].x)); v[i].x = y; }
            if (KIND == 6) v[i].x = __shfl_xor_sync(0xffffffffu, v[i].x, 1 + (i & 7));
        }
    }
    float s = 0;
    for (int i = 0; i < 8; ++i) s += v[i].x + v[i].y;
    out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}

#define BODY_ITER 3000
template <int KIND> __global__ void __launch_bounds__(128, 4) iteration_core(float* out, const float* in) {
    float2 U[4][4];
    float rho[4], kap[8];
    for (int a = 0; a < 4; ++a)
        for (int b = 0; b < 4; ++b)
            U[a][b] = make_float2(in[threadIdx.x + a * 8 + 2 * b], in[threadIdx.x + a * 8 + 2 * b + 1]);
    float acc = 0.f;
    for (int it = 0; it < BODY_ITER; ++it) {
        float2 e[4][4];
        float rp[4], cp[8];
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            float2 s2;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                if (KIND != 2) e[a][b] = make_float2(fminf(U[a][b].x, 1.0f), fminf(U[a][b].y, 1.0f));
                else e[a][b] = U[a][b];
                if (KIND == 1) { if (b == 0) s2 = e[a][b]; else { s2.x += e[a][b].x; s2.y += e[a][b].y; } }
                else s2 = (b == 0) ? e[a][b] : __fadd2_rn(s2, e[a][b]);
            }
            rp[a] = s2.x + s2.y;
        }
#pragma unroll
        for (int a = 0; a < 4; ++a) rho[a] = 2.0f - rp[a] * 0.03f;   // stands in for N / r
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            float2 c2;
            if (KIND == 1) {
                c2.x = e[0][b].x * rho[0]; c2.y = e[0][b].y * rho[0];
#pragma unroll
                for (int a = 1; a < 4; ++a) { c2.x = fmaf(e[a][b].x, rho[a], c2.x); c2.y = fmaf(e[a][b].y, rho[a], c2.y); }
            } else {
                c2 = __fmul2_rn(e[0][b], make_float2(rho[0], rho[0]));
#pragma unroll
                for (int a = 1; a < 4; ++a) c2 = __ffma2_rn(e[a][b], make_float2(rho[a], rho[a]), c2);
            }
            cp[2 * b] = c2.x; cp[2 * b + 1] = c2.y;
        }
#pragma unroll
        for (int b = 0; b < 8; ++b) kap[b] = 2.0f - cp[b] * 0.03f;
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                if (KIND == 1) { U[a][b].x = U[a][b].x * rho[a] * kap[2 * b]; U[a][b].y = U[a][b].y * rho[a] * kap[2 * b + 1]; }
                else U[a][b] = __fmul2_rn(__fmul2_rn(U[a][b], make_float2(rho[a], rho[a])), make_float2(kap[2 * b], kap[2 * b + 1]));
            }
        acc += rp[0];
    }
    float s = acc;
    for (int a = 0; a < 4; ++a) for (int b = 0; b < 4; ++b) s += U[a][b].x + U[a][b].y;
    out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}

static double sm_clock_hz() {
    int khz = 0;
    cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, 0);
    return khz * 1e3;
}

template <int KIND> void run_single(const char* name, int per_step, float* out) {
    cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
    int sms = 0; cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0);
    const int blocks = sms * 4, threads = 512;
    single_kind<KIND><<<blocks, threads>>>(out, 0.999f, 1e-3f);
    cudaEventRecord(e0);
    single_kind<KIND><<<blocks, threads>>>(out, 0.999f, 1e-3f);
    cudaEventRecord(e1); cudaEventSynchronize(e1);
    float ms; cudaEventElapsedTime(&ms, e0, e1);
    const double warps_per_smsp = (double)blocks * threads / 32 / sms / 4;
    const double instr = warps_per_smsp * ITER * 8.0 * per_step, clk = ms * 1e-3 * sm_clock_hz();
    printf("%-28s %7.3f ms  %5.2f clocks per warp instruction per sub-partition\n", name, ms, clk / instr);
}

template <int KIND> void run_core(const char* name, float* out, float* in, int ctas_per_sm) {
    cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
    int sms = 0; cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0);
    iteration_core<KIND><<<sms * ctas_per_sm, 128>>>(out, in);
    cudaEventRecord(e0);
    iteration_core<KIND><<<sms * ctas_per_sm, 128>>>(out, in);
    cudaEventRecord(e1); cudaEventSynchronize(e1);
    float ms; cudaEventElapsedTime(&ms, e0, e1);
    const double clk = ms * 1e-3 * sm_clock_hz();
    printf("%-30s warps/sub-partition=%d  %7.3f ms  %6.1f clocks per warp-iteration (32 elements per lane)\n",
           name, ctas_per_sm, ms, clk / ((double)ctas_per_sm * BODY_ITER));
}

int main() {
    float *out, *in;
    cudaMalloc(&out, 160 * 8 * 512 * 4); cudaMalloc(&in, 4096); cudaMemset(in, 0, 4096);
    run_single<0>("scalar fma x2", 2, out);
    run_single<1>("packed fma.f32x2", 1, out);
    run_single<2>("packed add.f32x2", 1, out);
    run_single<3>("packed mul.f32x2", 1, out);
    run_single<4>("ex2.approx (SFU)", 1, out);
    run_single<5>("lg2.approx (SFU)", 1, out);
    run_single<6>("shfl.xor", 1, out);
    for (int c : {1, 2, 4}) {
        run_core<0>("core, packed fp32x2", out, in, c);
        run_core<1>("core, scalar", out, in, c);
        run_core<2>("core, packed, without the min", out, in, c);
    }
    printf("%s\n", cudaGetErrorString(cudaDeviceSynchronize()));
    return 0;
}
