// C ABI of the TSENOR hot path (see include/tsenor.h): argument checks on the
// host, then kernel launches on the caller's stream.  No allocation, no
// synchronisation, no CPU fallback.
#include "tsenor.h"
#include "tsenor_device.cuh"

#include <atomic>
#include <cmath>

namespace {

thread_local int g_last_cuda_error = 0;
std::atomic<long long> g_launches{0};

inline bool valid_M(int M) { return M == 4 || M == 8 || M == 16 || M == 32; }

int check_matrix(int64_t rows, int64_t cols, int64_t ld, int M) {
    if (rows < 0 || cols < 0 || ld < cols) return TSENOR_ERR_SHAPE;
    if (rows % M || cols % M) return TSENOR_ERR_SHAPE;
    return TSENOR_OK;
}

int finish_launch() {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        return TSENOR_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return TSENOR_OK;
}

inline bool aligned16(const void* p, int64_t ld) {
    return (reinterpret_cast<uintptr_t>(p) % 16 == 0) && (ld % 4 == 0);
}

template <int M, int MODE>
int launch(const tsenor::Params& P, cudaStream_t st) {
    using G = tsenor::Geom<M>;
    const int64_t npc = (P.cols + G::PANEL - 1) / G::PANEL;
    const int64_t panels = (P.rows / M) * npc;
    if (panels == 0) return TSENOR_OK;
    if (panels > 0x7fffffffLL) return TSENOR_ERR_SHAPE;
    tsenor::Params Q = P;
    Q.npc = (int)npc;
    const size_t smem = sizeof(tsenor::SmemLayout<M, MODE>);
    static thread_local int configured_device = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (configured_device != dev) {
        cudaError_t e = cudaFuncSetAttribute(tsenor::tsenor_kernel<M, MODE>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) {
            g_last_cuda_error = (int)e;
            return TSENOR_ERR_CUDA;
        }
        configured_device = dev;
    }
    tsenor::tsenor_kernel<M, MODE><<<(unsigned)panels, tsenor::WARPS * 32, smem, st>>>(Q);
    return finish_launch();
}

template <int MODE>
int dispatch(const tsenor::Params& P, int M, cudaStream_t st) {
    switch (M) {
        case 4: return launch<4, MODE>(P, st);
        case 8: return launch<8, MODE>(P, st);
        case 16: return launch<16, MODE>(P, st);
        default: return launch<32, MODE>(P, st);
    }
}

void set_tau(tsenor::Params& P, float tau) {
    const double c = (double)tau * 1.4426950408889634074;  // tau * log2(e)
    P.c_hi = (float)c;
    P.c_lo = (float)(c - (double)P.c_hi);
}

// ------------------------------------------------------------ small kernels

__global__ void fill_mask_kernel(uint32_t* bits, int64_t rows, int64_t wpr, int64_t cols, uint32_t value) {
    const int64_t n = rows * wpr;
    for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < n;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t wd = idx % wpr;
        uint32_t v = value;
        const int64_t left = cols - wd * 32;
        if (left < 32) v &= (left <= 0) ? 0u : ((1u << left) - 1u);
        bits[idx] = v;
    }
}

__global__ void objective_kernel(const float* __restrict__ scores, int64_t ld, const uint32_t* __restrict__ bits,
                                 int64_t rows, int64_t cols, int64_t wpr, double* out) {
    double acc = 0.0;
    const int64_t nwords = rows * wpr;
    for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < nwords;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = idx / wpr, wd = idx % wpr;
        uint32_t m = bits[idx];
        while (m) {
            const int b = __ffs(m) - 1;
            m &= m - 1;
            const int64_t c = wd * 32 + b;
            if (c < cols) acc += (double)fabsf(scores[r * ld + c]);
        }
    }
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    __shared__ double part[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) part[warp] = acc;
    __syncthreads();
    if (warp == 0) {
        acc = (lane < (int)(blockDim.x >> 5)) ? part[lane] : 0.0;
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (lane == 0) atomicAdd(out, acc);
    }
}

// One thread per block of the mask.
__global__ void check_kernel(const uint32_t* __restrict__ bits, int64_t rows, int64_t cols, int64_t wpr, int N,
                             int M, unsigned long long* bad_out) {
    const int64_t nbc = cols / M, nblk = (rows / M) * nbc;
    unsigned long long bad = 0;
    for (int64_t b = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; b < nblk;
         b += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r0 = (b / nbc) * M, c0 = (b % nbc) * M;
        const uint32_t gm = (M == 32) ? 0xffffffffu : ((1u << M) - 1u);
        bool ok = true;
        uint32_t colcnt[5] = {0, 0, 0, 0, 0};  // bit-sliced column counters (counts up to 31)
        uint32_t over = 0;
        for (int i = 0; i < M; ++i) {
            const uint32_t row = (bits[(r0 + i) * wpr + c0 / 32] >> (c0 % 32)) & gm;
            ok = ok && (__popc(row) == N);
            uint32_t carry = row;
            for (int k = 0; k < 5; ++k) {
                const uint32_t t = colcnt[k] & carry;
                colcnt[k] ^= carry;
                carry = t;
            }
            over |= carry;  // a column reached 32
        }
        uint32_t eq = gm;
        for (int k = 0; k < 5; ++k) eq &= ((N >> k) & 1) ? colcnt[k] : ~colcnt[k];
        if (N == 32) ok = ok && (over == gm); else ok = ok && (over == 0) && (eq == gm);
        bad += ok ? 0 : 1;
    }
    for (int off = 16; off > 0; off >>= 1) bad += __shfl_xor_sync(0xffffffffu, bad, off);
    if ((threadIdx.x & 31) == 0 && bad) atomicAdd(bad_out, bad);
}

__global__ void max_abs_kernel(const float* __restrict__ scores, int64_t rows, int64_t cols, int64_t ld,
                               unsigned int* out_bits) {
    float m = 0.f;
    const int64_t n = rows * cols;
    for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < n;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const float v = fabsf(scores[(idx / cols) * ld + idx % cols]);
        m = fmaxf(m, v);  // fmaxf drops NaN
    }
    for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    // non-negative floats order like their bit patterns
    if ((threadIdx.x & 31) == 0) atomicMax(out_bits, __float_as_uint(m));
}

int grid_for(int64_t work, int threads) {
    int64_t g = (work + threads - 1) / threads;
    if (g < 1) g = 1;
    if (g > 148 * 16) g = 148 * 16;
    return (int)g;
}

int trivial_mask(uint32_t* bits, int64_t rows, int64_t cols, bool ones, cudaStream_t st) {
    const int64_t wpr = (cols + 31) / 32;
    if (rows * wpr == 0) return TSENOR_OK;
    fill_mask_kernel<<<grid_for(rows * wpr, 256), 256, 0, st>>>(bits, rows, wpr, cols, ones ? 0xffffffffu : 0u);
    return finish_launch();
}

}  // namespace

extern "C" {

int tsenor_solve(const float* scores, int64_t rows, int64_t cols, int64_t ld, int N, int M, float tau, int iters,
                 int ls_steps, uint32_t* mask_bits_out, int32_t* dev_status, tsenor_stream_t stream) {
    if (!valid_M(M) || N < 0 || N > M) return TSENOR_ERR_NM;
    if (int rc = check_matrix(rows, cols, ld, M)) return rc;
    if (iters < 0 || !(tau >= 0.0f) || !std::isfinite(tau)) return TSENOR_ERR_ARG;
    if (rows == 0 || cols == 0) return TSENOR_OK;
    if (!scores || !mask_bits_out) return TSENOR_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    if (N == 0 || N == M) return trivial_mask(mask_bits_out, rows, cols, N == M, st);
    tsenor::Params P{};
    P.scores = scores; P.ld = ld;
    P.bits = mask_bits_out; P.wpr = (cols + 31) / 32;
    P.rows = rows; P.cols = cols;
    P.N = N; P.Nf = (float)N; P.log2N = (float)std::log2((double)N);
    set_tau(P, tau);
    P.iters = iters; P.ls_steps = ls_steps;
    P.status = dev_status;
    P.vec_scores = aligned16(scores, ld);
    return dispatch<0>(P, M, st);
}

int tsenor_dykstra(const float* scores, int64_t rows, int64_t cols, int64_t ld, int N, int M, float tau, int iters,
                   float* plan_out, int64_t ld_plan, int plan_is_log, int32_t* dev_status, tsenor_stream_t stream) {
    if (!valid_M(M) || N < 1 || N >= M) return TSENOR_ERR_NM;
    if (int rc = check_matrix(rows, cols, ld, M)) return rc;
    if (ld_plan < cols) return TSENOR_ERR_SHAPE;
    if (iters < 0 || !(tau >= 0.0f) || !std::isfinite(tau)) return TSENOR_ERR_ARG;
    if (rows == 0 || cols == 0) return TSENOR_OK;
    if (!scores || !plan_out) return TSENOR_ERR_NULL;
    tsenor::Params P{};
    P.scores = scores; P.ld = ld;
    P.plan = plan_out; P.ld_plan = ld_plan; P.plan_is_log = plan_is_log;
    P.rows = rows; P.cols = cols;
    P.N = N; P.Nf = (float)N; P.log2N = (float)std::log2((double)N);
    set_tau(P, tau);
    P.iters = iters; P.ls_steps = -1;
    P.status = dev_status;
    P.vec_scores = aligned16(scores, ld);
    return dispatch<1>(P, M, (cudaStream_t)stream);
}

int tsenor_round(const float* plan_key, int64_t ld_plan, const float* scores, int64_t ld, int64_t rows,
                 int64_t cols, int N, int M, int ls_steps, uint32_t* mask_bits_out, int32_t* dev_status,
                 tsenor_stream_t stream) {
    if (!valid_M(M) || N < 0 || N > M) return TSENOR_ERR_NM;
    if (int rc = check_matrix(rows, cols, ld, M)) return rc;
    if (ld_plan < cols) return TSENOR_ERR_SHAPE;
    if (rows == 0 || cols == 0) return TSENOR_OK;
    if (!plan_key || !scores || !mask_bits_out) return TSENOR_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    if (N == 0 || N == M) return trivial_mask(mask_bits_out, rows, cols, N == M, st);
    tsenor::Params P{};
    P.scores = scores; P.ld = ld;
    P.keys = plan_key; P.ld_keys = ld_plan;
    P.bits = mask_bits_out; P.wpr = (cols + 31) / 32;
    P.rows = rows; P.cols = cols;
    P.N = N; P.Nf = (float)N; P.log2N = 0.f;
    P.iters = 0; P.ls_steps = ls_steps;
    P.status = dev_status;
    P.vec_scores = aligned16(scores, ld);
    P.vec_keys = aligned16(plan_key, ld_plan);
    return dispatch<2>(P, M, st);
}

int tsenor_objective(const float* scores, int64_t ld, const uint32_t* mask_bits, int64_t rows, int64_t cols,
                     double* dev_sum_out, tsenor_stream_t stream) {
    if (rows < 0 || cols < 0 || ld < cols) return TSENOR_ERR_SHAPE;
    if (!dev_sum_out) return TSENOR_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(dev_sum_out, 0, sizeof(double), st) != cudaSuccess) return finish_launch(), TSENOR_ERR_CUDA;
    if (rows == 0 || cols == 0) return TSENOR_OK;
    if (!scores || !mask_bits) return TSENOR_ERR_NULL;
    const int64_t wpr = (cols + 31) / 32;
    objective_kernel<<<grid_for(rows * wpr, 256), 256, 0, st>>>(scores, ld, mask_bits, rows, cols, wpr, dev_sum_out);
    return finish_launch();
}

int tsenor_check(const uint32_t* mask_bits, int64_t rows, int64_t cols, int N, int M, int64_t* dev_bad_blocks_out,
                 tsenor_stream_t stream) {
    if (!valid_M(M) || N < 0 || N > M) return TSENOR_ERR_NM;
    if (int rc = check_matrix(rows, cols, cols, M)) return rc;
    if (!dev_bad_blocks_out) return TSENOR_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(dev_bad_blocks_out, 0, sizeof(int64_t), st) != cudaSuccess)
        return finish_launch(), TSENOR_ERR_CUDA;
    if (rows == 0 || cols == 0) return TSENOR_OK;
    if (!mask_bits) return TSENOR_ERR_NULL;
    const int64_t nblk = (rows / M) * (cols / M), wpr = (cols + 31) / 32;
    check_kernel<<<grid_for(nblk, 128), 128, 0, st>>>(mask_bits, rows, cols, wpr, N, M,
                                                     reinterpret_cast<unsigned long long*>(dev_bad_blocks_out));
    return finish_launch();
}

int tsenor_max_abs(const float* scores, int64_t rows, int64_t cols, int64_t ld, float* dev_max_out,
                   tsenor_stream_t stream) {
    if (rows < 0 || cols < 0 || ld < cols) return TSENOR_ERR_SHAPE;
    if (!dev_max_out) return TSENOR_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(dev_max_out, 0, sizeof(float), st) != cudaSuccess) return finish_launch(), TSENOR_ERR_CUDA;
    if (rows == 0 || cols == 0) return TSENOR_OK;
    if (!scores) return TSENOR_ERR_NULL;
    max_abs_kernel<<<grid_for(rows * cols, 256 * 8), 256, 0, st>>>(scores, rows, cols, ld,
                                                                   reinterpret_cast<unsigned int*>(dev_max_out));
    return finish_launch();
}

int64_t tsenor_mask_words_per_row(int64_t cols) { return cols <= 0 ? 0 : (cols + 31) / 32; }

const char* tsenor_strerror(int status) {
    switch (status) {
        case TSENOR_OK: return "ok";
        case TSENOR_ERR_NULL: return "a required pointer is NULL";
        case TSENOR_ERR_SHAPE: return "bad shape: negative size, ld < cols, or rows/cols not a multiple of M";
        case TSENOR_ERR_NM: return "bad N:M: M must be 4, 8, 16 or 32 and N within range";
        case TSENOR_ERR_ARG: return "bad argument: iters < 0 or tau negative / not finite";
        case TSENOR_ERR_CUDA: return "CUDA launch failed: see tsenor_last_cuda_error()";
        default: return "unknown status";
    }
}

int tsenor_last_cuda_error(void) { return g_last_cuda_error; }

int64_t tsenor_launch_count(void) { return (int64_t)g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
