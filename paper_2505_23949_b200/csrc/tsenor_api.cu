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

tsenor::ScoreSrc abs_source(const float* scores, int64_t ld) {
    tsenor::ScoreSrc S{};
    S.kind = tsenor::SC_ABS;
    S.w = scores; S.ld = ld;
    S.vec_w = aligned16(scores, ld);
    return S;
}

// Validates a caller's descriptor and turns it into the device-side form.
int make_source(const tsenor_scores_t* d, int64_t cols, tsenor::ScoreSrc* out) {
    if (!d) return TSENOR_ERR_NULL;
    if (d->kind < TSENOR_SCORES_ABS || d->kind > TSENOR_SCORES_COLMUL) return TSENOR_ERR_ARG;
    if (d->ld < cols) return TSENOR_ERR_SHAPE;
    if (!d->w) return TSENOR_ERR_NULL;
    tsenor::ScoreSrc S{};
    S.kind = d->kind;
    S.w_is_bf16 = d->w_is_bf16 ? 1 : 0;
    S.w = d->w; S.ld = d->ld;
    S.vec_w = d->w_is_bf16 ? ((reinterpret_cast<uintptr_t>(d->w) % 8 == 0) && (d->ld % 4 == 0))
                           : aligned16(d->w, d->ld);
    if (d->kind == TSENOR_SCORES_ADMM) {
        if (!d->v) return TSENOR_ERR_NULL;
        if (d->ld_v < cols) return TSENOR_ERR_SHAPE;
        if (!std::isfinite(d->scalar)) return TSENOR_ERR_ARG;
        S.v = d->v; S.ld_v = d->ld_v; S.scalar = d->scalar;
        S.vec_v = aligned16(d->v, d->ld_v);
    }
    if (d->kind == TSENOR_SCORES_COLDIV || d->kind == TSENOR_SCORES_COLMUL) {
        if (!d->colvec) return TSENOR_ERR_NULL;
        S.colvec = d->colvec;
        S.vec_c = (reinterpret_cast<uintptr_t>(d->colvec) % 16 == 0);
    }
    *out = S;
    return TSENOR_OK;
}

std::atomic<int> g_layout{TSENOR_LAYOUT_AUTO};

// Panels (= CTAs) a matrix is cut into under layout V.
template <int M, int V>
int64_t panel_count(const tsenor::Params& P, bool tall, int64_t* npc_out) {
    using G = tsenor::Geom<M, V>;
    constexpr int NB = G::PANEL / M;
    const int64_t npc = (P.cols + G::PANEL - 1) / G::PANEL;
    *npc_out = npc;
    return tall ? (P.rows / M + NB - 1) / NB : (P.rows / M) * npc;
}

int sm_count() {
    static thread_local int cached_dev = -1, cached = 148;
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev != cached_dev) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) cached = n;
        cached_dev = dev;
    }
    return cached;
}

template <int M, int MODE, int V>
int launch_layout(const tsenor::Params& P, bool tall, cudaStream_t st) {
    using G = tsenor::Geom<M, V>;
    int64_t npc = 0;
    const int64_t panels = panel_count<M, V>(P, tall, &npc);
    if (panels == 0) return TSENOR_OK;
    if (panels > 0x7fffffffLL) return TSENOR_ERR_SHAPE;
    tsenor::Params Q = P;
    Q.npc = (int)npc;
    Q.tall = tall ? 1 : 0;
    const size_t smem = sizeof(tsenor::SmemLayout<G, MODE>);
    static thread_local int configured_device = -1;
    int dev = 0;
    cudaGetDevice(&dev);
    if (configured_device != dev) {
        cudaError_t e = cudaFuncSetAttribute(tsenor::tsenor_kernel<M, MODE, V>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) {
            g_last_cuda_error = (int)e;
            return TSENOR_ERR_CUDA;
        }
        configured_device = dev;
    }
    tsenor::tsenor_kernel<M, MODE, V><<<(unsigned)panels, tsenor::WARPS * 32, smem, st>>>(Q);
    return finish_launch();
}

// Chooses the register layout: the latency layout (a block over M lanes) when even its
// finer panels leave the GPU with no more than four CTAs per SM, i.e. when the run time is
// the chain of dependent iterations of a single warp rather than instruction throughput.
template <int M, int MODE>
int launch(const tsenor::Params& P, cudaStream_t st) {
    // a slab (single block column) is cut into panels of vertically stacked blocks
    const bool tall = (P.cols == M) && (P.rows > M);
    if constexpr (M < 32) {   // a 32 x 32 block takes a whole warp in either layout
        const int policy = g_layout.load(std::memory_order_relaxed);
        bool fine = (policy == TSENOR_LAYOUT_LATENCY);
        if (policy == TSENOR_LAYOUT_AUTO) {
            int64_t npc = 0;
            fine = panel_count<M, 1>(P, tall, &npc) <= 4LL * sm_count();
        }
        if (fine) return launch_layout<M, MODE, 1>(P, tall, st);
    }
    return launch_layout<M, MODE, 0>(P, tall, st);
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

// Retained score of up to two masks under one score source (quads of 4 columns).
__global__ void objective_kernel(const tsenor::ScoreSrc S, const uint32_t* __restrict__ bits_a,
                                 const uint32_t* __restrict__ bits_b, int64_t rows, int64_t cols, int64_t wpr,
                                 double* out) {
    double acc_a = 0.0, acc_b = 0.0;
    const int64_t qpr = cols / 4, nq = rows * qpr;
    for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < nq;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = idx / qpr, c = (idx % qpr) * 4;
        const uint32_t ma = (bits_a[r * wpr + c / 32] >> (c % 32)) & 15u;
        const uint32_t mb = bits_b ? (bits_b[r * wpr + c / 32] >> (c % 32)) & 15u : 0u;
        if ((ma | mb) == 0u) continue;
        const float4 v = tsenor::load_score_quad(S, r, c);
        const float e[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if ((ma >> k) & 1u) acc_a += (double)e[k];
            if ((mb >> k) & 1u) acc_b += (double)e[k];
        }
    }
    for (int off = 16; off > 0; off >>= 1) {
        acc_a += __shfl_xor_sync(0xffffffffu, acc_a, off);
        acc_b += __shfl_xor_sync(0xffffffffu, acc_b, off);
    }
    __shared__ double part[2][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { part[0][warp] = acc_a; part[1][warp] = acc_b; }
    __syncthreads();
    if (warp == 0) {
        acc_a = (lane < (int)(blockDim.x >> 5)) ? part[0][lane] : 0.0;
        acc_b = (lane < (int)(blockDim.x >> 5)) ? part[1][lane] : 0.0;
        for (int off = 16; off > 0; off >>= 1) {
            acc_a += __shfl_xor_sync(0xffffffffu, acc_a, off);
            acc_b += __shfl_xor_sync(0xffffffffu, acc_b, off);
        }
        if (lane == 0) {
            atomicAdd(out, acc_a);
            if (bits_b) atomicAdd(out + 1, acc_b);
        }
    }
}

// mask_inout <- prev wherever the previous mask retained more score (obj2 = {new, prev}).
__global__ void keep_better_kernel(const double* __restrict__ obj2, const uint32_t* __restrict__ prev,
                                   uint32_t* __restrict__ mask_inout, int64_t nwords) {
    if (!(obj2[0] < obj2[1])) return;
    for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < nwords;
         idx += (int64_t)gridDim.x * blockDim.x)
        mask_inout[idx] = prev[idx];
}

__global__ void scores_max_kernel(const tsenor::ScoreSrc S, int64_t rows, int64_t cols, unsigned int* out_bits) {
    float m = 0.f;
    const int64_t qpr = cols / 4, nq = rows * qpr;
    for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < nq;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const float4 v = tsenor::load_score_quad(S, idx / qpr, (idx % qpr) * 4);
        m = fmaxf(fmaxf(m, fmaxf(v.x, v.y)), fmaxf(v.z, v.w));  // fmaxf drops NaN
    }
    for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    // non-negative floats order like their bit patterns
    if ((threadIdx.x & 31) == 0) atomicMax(out_bits, __float_as_uint(m));
}

__global__ void materialize_kernel(const tsenor::ScoreSrc S, int64_t rows, int64_t cols, float* out,
                                   int64_t ld_out) {
    const int64_t qpr = cols / 4, nq = rows * qpr;
    for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < nq;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = idx / qpr, c = (idx % qpr) * 4;
        const float4 v = tsenor::load_score_quad(S, r, c);
        float* p = out + r * ld_out + c;
        p[0] = v.x; p[1] = v.y; p[2] = v.z; p[3] = v.w;
    }
}

// "Simple" rounding: one warp per block; lane i is row i in the first pass and column i in
// the second.  Ranks by counting under the strict order (key descending, index ascending).
__device__ __forceinline__ bool key_before(float ka, int ia, float kb, int ib) {
    return ka > kb || (ka == kb && ia < ib);
}
__global__ void simple_round_kernel(const float* __restrict__ key, int64_t ld, int64_t rows, int64_t cols,
                                    int64_t wpr, int N, int M, uint32_t* bits) {
    __shared__ float ks[4][32][33];
    __shared__ unsigned rowmask[4][32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t nbc = cols / M, nblk = (rows / M) * nbc;
    for (int64_t b = blockIdx.x * 4LL + warp; b < nblk; b += gridDim.x * 4LL) {
        const int64_t r0 = (b / nbc) * M, c0 = (b % nbc) * M;
        for (int i = 0; i < M; ++i)
            if (lane < M) {
                float k = key[(r0 + i) * ld + c0 + lane];
                if (!(k == k)) k = __int_as_float(0xff800000);
                ks[warp][i][lane] = k + 0.0f;
            }
        __syncwarp();
        unsigned keep = 0u;
        if (lane < M) {   // row pass: the N best of my row
            for (int j = 0; j < M; ++j) {
                int rank = 0;
                for (int j2 = 0; j2 < M; ++j2) rank += key_before(ks[warp][lane][j2], j2, ks[warp][lane][j], j) ? 1 : 0;
                if (rank < N) keep |= 1u << j;
            }
        }
        rowmask[warp][lane] = keep;
        __syncwarp();
        unsigned colkeep = 0u;   // bits over rows, for my column
        if (lane < M) {
            unsigned surv = 0u;
            for (int i = 0; i < M; ++i) surv |= ((rowmask[warp][i] >> lane) & 1u) << i;
            for (int i = 0; i < M; ++i) {
                if (!((surv >> i) & 1u)) continue;
                int rank = 0;
                for (int i2 = 0; i2 < M; ++i2)
                    if ((surv >> i2) & 1u) rank += key_before(ks[warp][i2][lane], i2, ks[warp][i][lane], i) ? 1 : 0;
                if (rank < N) colkeep |= 1u << i;
            }
        }
        __syncwarp();
        rowmask[warp][lane] = colkeep;   // now indexed by column
        __syncwarp();
        if (lane < M) {
            unsigned row = 0u;
            for (int j = 0; j < M; ++j) row |= ((rowmask[warp][j] >> lane) & 1u) << j;
            if (row) atomicOr(&bits[(r0 + lane) * wpr + c0 / 32], row << (c0 % 32));
        }
        __syncwarp();
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

struct Extras {   // optional settings carried by tsenor_scores_t
    int per_block_tau = 0;
    float ee_eps = 0.0f;
    unsigned long long* iter_sum = nullptr;
};

static int extras_of(const tsenor_scores_t* s, Extras* x) {
    x->per_block_tau = s->per_block_tau ? 1 : 0;
    if (!(s->early_exit_eps >= 0.0f) || !std::isfinite(s->early_exit_eps)) return TSENOR_ERR_ARG;
    x->ee_eps = s->early_exit_eps;
    x->iter_sum = reinterpret_cast<unsigned long long*>(s->dev_iters_out);
    return TSENOR_OK;
}

static int solve_on(const tsenor::ScoreSrc& src, const Extras& x, int64_t rows, int64_t cols, int N, int M,
                    float tau, int iters, int ls_steps, uint32_t* mask_bits_out, int32_t* dev_status,
                    cudaStream_t st) {
    if (N == 0 || N == M) return trivial_mask(mask_bits_out, rows, cols, N == M, st);
    tsenor::Params P{};
    P.src = src;
    P.bits = mask_bits_out; P.wpr = (cols + 31) / 32;
    P.rows = rows; P.cols = cols;
    P.N = N; P.Nf = (float)N; P.log2N = (float)std::log2((double)N);
    set_tau(P, tau);
    P.per_block_tau = x.per_block_tau;
    P.ee_eps = x.ee_eps; P.iter_sum = x.iter_sum;
    P.iters = iters; P.ls_steps = ls_steps;
    P.status = dev_status;
    return dispatch<0>(P, M, st);
}

int tsenor_solve(const float* scores, int64_t rows, int64_t cols, int64_t ld, int N, int M, float tau, int iters,
                 int ls_steps, uint32_t* mask_bits_out, int32_t* dev_status, tsenor_stream_t stream) {
    if (!valid_M(M) || N < 0 || N > M) return TSENOR_ERR_NM;
    if (int rc = check_matrix(rows, cols, ld, M)) return rc;
    if (iters < 0 || !(tau >= 0.0f) || !std::isfinite(tau)) return TSENOR_ERR_ARG;
    if (rows == 0 || cols == 0) return TSENOR_OK;
    if (!scores || !mask_bits_out) return TSENOR_ERR_NULL;
    return solve_on(abs_source(scores, ld), Extras{}, rows, cols, N, M, tau, iters, ls_steps, mask_bits_out,
                    dev_status, (cudaStream_t)stream);
}

int tsenor_solve_scores(const tsenor_scores_t* s, int64_t rows, int64_t cols, int N, int M, float tau, int iters,
                        int ls_steps, uint32_t* mask_bits_out, int32_t* dev_status, tsenor_stream_t stream) {
    if (!valid_M(M) || N < 0 || N > M) return TSENOR_ERR_NM;
    if (int rc = check_matrix(rows, cols, cols, M)) return rc;
    if (iters < 0 || !(tau >= 0.0f) || !std::isfinite(tau)) return TSENOR_ERR_ARG;
    tsenor::ScoreSrc src{};
    if (int rc = make_source(s, cols, &src)) return rc;
    if (rows == 0 || cols == 0) return TSENOR_OK;
    if (!mask_bits_out) return TSENOR_ERR_NULL;
    Extras x;
    if (int rc = extras_of(s, &x)) return rc;
    return solve_on(src, x, rows, cols, N, M, tau, iters, ls_steps, mask_bits_out, dev_status,
                    (cudaStream_t)stream);
}

static int max_on(const tsenor::ScoreSrc& src, int64_t rows, int64_t cols, float* dev_max_out, cudaStream_t st) {
    if (cudaMemsetAsync(dev_max_out, 0, sizeof(float), st) != cudaSuccess) return finish_launch(), TSENOR_ERR_CUDA;
    if (rows == 0 || cols == 0) return TSENOR_OK;
    scores_max_kernel<<<grid_for(rows * (cols / 4), 256 * 2), 256, 0, st>>>(
        src, rows, cols, reinterpret_cast<unsigned int*>(dev_max_out));
    return finish_launch();
}

int tsenor_scores_max(const tsenor_scores_t* s, int64_t rows, int64_t cols, float* dev_max_out,
                      tsenor_stream_t stream) {
    if (rows < 0 || cols < 0 || cols % 4) return TSENOR_ERR_SHAPE;
    tsenor::ScoreSrc src{};
    if (int rc = make_source(s, cols, &src)) return rc;
    if (!dev_max_out) return TSENOR_ERR_NULL;
    return max_on(src, rows, cols, dev_max_out, (cudaStream_t)stream);
}

int tsenor_scores_materialize(const tsenor_scores_t* s, int64_t rows, int64_t cols, float* scores_out,
                              int64_t ld_out, tsenor_stream_t stream) {
    if (rows < 0 || cols < 0 || cols % 4 || ld_out < cols) return TSENOR_ERR_SHAPE;
    tsenor::ScoreSrc src{};
    if (int rc = make_source(s, cols, &src)) return rc;
    if (rows == 0 || cols == 0) return TSENOR_OK;
    if (!scores_out) return TSENOR_ERR_NULL;
    materialize_kernel<<<grid_for(rows * (cols / 4), 256), 256, 0, (cudaStream_t)stream>>>(src, rows, cols,
                                                                                          scores_out, ld_out);
    return finish_launch();
}

int tsenor_keep_better(const tsenor_scores_t* s, int64_t rows, int64_t cols, const uint32_t* prev_mask,
                       uint32_t* mask_inout, double* dev_obj2_out, tsenor_stream_t stream) {
    if (rows < 0 || cols < 0 || cols % 4) return TSENOR_ERR_SHAPE;
    tsenor::ScoreSrc src{};
    if (int rc = make_source(s, cols, &src)) return rc;
    if (!dev_obj2_out) return TSENOR_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(dev_obj2_out, 0, 2 * sizeof(double), st) != cudaSuccess)
        return finish_launch(), TSENOR_ERR_CUDA;
    if (rows == 0 || cols == 0) return TSENOR_OK;
    if (!prev_mask || !mask_inout) return TSENOR_ERR_NULL;
    const int64_t wpr = (cols + 31) / 32;
    objective_kernel<<<grid_for(rows * (cols / 4), 256), 256, 0, st>>>(src, mask_inout, prev_mask, rows, cols, wpr,
                                                                      dev_obj2_out);
    if (int rc = finish_launch()) return rc;
    keep_better_kernel<<<grid_for(rows * wpr, 256), 256, 0, st>>>(dev_obj2_out, prev_mask, mask_inout, rows * wpr);
    return finish_launch();
}

int tsenor_simple_round(const float* plan_key, int64_t ld_plan, int64_t rows, int64_t cols, int N, int M,
                        uint32_t* mask_bits_out, tsenor_stream_t stream) {
    if (!valid_M(M) || N < 1 || N >= M) return TSENOR_ERR_NM;
    if (int rc = check_matrix(rows, cols, ld_plan, M)) return rc;
    if (rows == 0 || cols == 0) return TSENOR_OK;
    if (!plan_key || !mask_bits_out) return TSENOR_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    const int64_t wpr = (cols + 31) / 32, nblk = (rows / M) * (cols / M);
    if (cudaMemsetAsync(mask_bits_out, 0, sizeof(uint32_t) * (size_t)(rows * wpr), st) != cudaSuccess)
        return finish_launch(), TSENOR_ERR_CUDA;
    simple_round_kernel<<<grid_for(nblk, 4), 128, 0, st>>>(plan_key, ld_plan, rows, cols, wpr, N, M, mask_bits_out);
    return finish_launch();
}

static int dykstra_on(const tsenor::ScoreSrc& src, const Extras& x, int64_t rows, int64_t cols, int N, int M,
                      float tau, int iters, float* plan_out, int64_t ld_plan, int plan_is_log,
                      int32_t* dev_status, cudaStream_t st) {
    tsenor::Params P{};
    P.src = src;
    P.plan = plan_out; P.ld_plan = ld_plan; P.plan_is_log = plan_is_log;
    P.rows = rows; P.cols = cols;
    P.N = N; P.Nf = (float)N; P.log2N = (float)std::log2((double)N);
    set_tau(P, tau);
    P.per_block_tau = x.per_block_tau;
    P.ee_eps = x.ee_eps; P.iter_sum = x.iter_sum;
    P.iters = iters; P.ls_steps = -1;
    P.status = dev_status;
    return dispatch<1>(P, M, st);
}

int tsenor_dykstra(const float* scores, int64_t rows, int64_t cols, int64_t ld, int N, int M, float tau, int iters,
                   float* plan_out, int64_t ld_plan, int plan_is_log, int32_t* dev_status, tsenor_stream_t stream) {
    if (!valid_M(M) || N < 1 || N >= M) return TSENOR_ERR_NM;
    if (int rc = check_matrix(rows, cols, ld, M)) return rc;
    if (ld_plan < cols) return TSENOR_ERR_SHAPE;
    if (iters < 0 || !(tau >= 0.0f) || !std::isfinite(tau)) return TSENOR_ERR_ARG;
    if (rows == 0 || cols == 0) return TSENOR_OK;
    if (!scores || !plan_out) return TSENOR_ERR_NULL;
    return dykstra_on(abs_source(scores, ld), Extras{}, rows, cols, N, M, tau, iters, plan_out, ld_plan, plan_is_log,
                      dev_status, (cudaStream_t)stream);
}

int tsenor_dykstra_scores(const tsenor_scores_t* s, int64_t rows, int64_t cols, int N, int M, float tau, int iters,
                          float* plan_out, int64_t ld_plan, int plan_is_log, int32_t* dev_status,
                          tsenor_stream_t stream) {
    if (!valid_M(M) || N < 1 || N >= M) return TSENOR_ERR_NM;
    if (int rc = check_matrix(rows, cols, cols, M)) return rc;
    if (ld_plan < cols) return TSENOR_ERR_SHAPE;
    if (iters < 0 || !(tau >= 0.0f) || !std::isfinite(tau)) return TSENOR_ERR_ARG;
    tsenor::ScoreSrc src{};
    if (int rc = make_source(s, cols, &src)) return rc;
    if (rows == 0 || cols == 0) return TSENOR_OK;
    if (!plan_out) return TSENOR_ERR_NULL;
    Extras x;
    if (int rc = extras_of(s, &x)) return rc;
    return dykstra_on(src, x, rows, cols, N, M, tau, iters, plan_out, ld_plan, plan_is_log,
                      dev_status, (cudaStream_t)stream);
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
    P.src = abs_source(scores, ld);
    P.keys = plan_key; P.ld_keys = ld_plan;
    P.bits = mask_bits_out; P.wpr = (cols + 31) / 32;
    P.rows = rows; P.cols = cols;
    P.N = N; P.Nf = (float)N; P.log2N = 0.f;
    P.iters = 0; P.ls_steps = ls_steps;
    P.status = dev_status;
    P.vec_keys = aligned16(plan_key, ld_plan);
    return dispatch<2>(P, M, st);
}

int tsenor_objective(const float* scores, int64_t ld, const uint32_t* mask_bits, int64_t rows, int64_t cols,
                     double* dev_sum_out, tsenor_stream_t stream) {
    if (rows < 0 || cols < 0 || ld < cols || cols % 4) return TSENOR_ERR_SHAPE;
    if (!dev_sum_out) return TSENOR_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(dev_sum_out, 0, sizeof(double), st) != cudaSuccess) return finish_launch(), TSENOR_ERR_CUDA;
    if (rows == 0 || cols == 0) return TSENOR_OK;
    if (!scores || !mask_bits) return TSENOR_ERR_NULL;
    const int64_t wpr = (cols + 31) / 32;
    objective_kernel<<<grid_for(rows * (cols / 4), 256), 256, 0, st>>>(abs_source(scores, ld), mask_bits, nullptr,
                                                                      rows, cols, wpr, dev_sum_out);
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
    if (rows < 0 || cols < 0 || ld < cols || cols % 4) return TSENOR_ERR_SHAPE;
    if (!dev_max_out) return TSENOR_ERR_NULL;
    if (rows > 0 && cols > 0 && !scores) return TSENOR_ERR_NULL;
    return max_on(abs_source(scores, ld), rows, cols, dev_max_out, (cudaStream_t)stream);
}

int64_t tsenor_mask_words_per_row(int64_t cols) { return cols <= 0 ? 0 : (cols + 31) / 32; }

const char* tsenor_strerror(int status) {
    switch (status) {
        case TSENOR_OK: return "ok";
        case TSENOR_ERR_NULL: return "a required pointer is NULL";
        case TSENOR_ERR_SHAPE: return "bad shape: negative size, ld < cols, or rows/cols not a multiple of M (of 4)";
        case TSENOR_ERR_NM: return "bad N:M: M must be 4, 8, 16 or 32 and N within range";
        case TSENOR_ERR_ARG: return "bad argument: iters < 0 or tau negative / not finite";
        case TSENOR_ERR_CUDA: return "CUDA launch failed: see tsenor_last_cuda_error()";
        default: return "unknown status";
    }
}

int tsenor_last_cuda_error(void) { return g_last_cuda_error; }

int64_t tsenor_launch_count(void) { return (int64_t)g_launches.load(std::memory_order_relaxed); }

int tsenor_set_layout(int layout) {
    if (layout < TSENOR_LAYOUT_AUTO || layout > TSENOR_LAYOUT_LATENCY) return TSENOR_ERR_ARG;
    return g_layout.exchange(layout, std::memory_order_relaxed);
}

}  // extern "C"
