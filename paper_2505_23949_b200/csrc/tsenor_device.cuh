// Device code of the TSENOR hot path for sm_100a: block loader, log-domain
// Dykstra iterations (Algorithm 1), greedy selection and local search
// (Algorithm 2, Eq. 6), bit-packed mask writer.
//
// Layout in one sentence: a CTA owns a panel of M rows x PANEL columns of the
// score matrix (PANEL = WARPS * BPW * M), stages it in shared memory with
// coalesced loads, every warp runs Dykstra for its BPW blocks entirely in
// registers, hands the log-plan to the rounding stage through shared memory,
// and the CTA writes whole 32-bit mask words back.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace tsenor {

constexpr unsigned FULL = 0xffffffffu;
constexpr int WARPS = 4;  // warps per CTA

enum : int { DEV_NONFINITE = 1, DEV_UNDERFILLED = 2, DEV_INTERNAL = 4 };

// Checked build flavour (-DTSENOR_BOUNDS, a second library built from the same sources): every
// data-dependent or computed index of the loaders, the rounding tables, the local search and the
// writers is tested against the extent of its array before the access; a bad one ORs
// DEV_INTERNAL into the status word and the access is skipped (nothing traps, nothing faults).
// It stands in for a memory checker on machines where none can be run.  In the normal build
// TS_CHECK(x) is the constant true and costs nothing.
#ifdef TSENOR_BOUNDS
__shared__ int g_bounds_flags;
#define TS_CHECK(cond) ((cond) ? true : (atomicOr(&tsenor::g_bounds_flags, tsenor::DEV_INTERNAL), false))
#else
#define TS_CHECK(cond) true
#endif

// ---------------------------------------------------------------------------
// Dykstra register layout.  A block is spread over LPB = PR*PC lanes arranged
// as PR x PC; each lane keeps an MR x MC sub-tile.  Row sums are reduced over
// the PC lanes that share rows, column sums over the PR lanes that share
// columns.  Two layouts per block size:
//   V = 0  throughput: 4 x 8 sub-tiles (4 x 4 for M = 4), the fewest exchanges per
//          element; used whenever the matrix has enough blocks to fill the GPU;
//   V = 1  latency (M < 32): a block over M lanes (the most the exchange scheme allows:
//          every lane must end up owning one row sum and one column sum), i.e. the
//          shortest chain of dependent work per iteration and 2-4 times as many
//          warps for the same matrix; used for matrices too small to fill the GPU.
//          (Butterfly all-reduces in place of reduce-scatter + all-gather halve the
//          exchange hops but measured no faster: the chain is then bound by the two
//          reciprocals and the arithmetic between the hops.)
// ---------------------------------------------------------------------------
template <int M, int V> struct Tile;
template <> struct Tile<32, 0> { static constexpr int PR = 8, PC = 4, MR = 4, MC = 8; };
template <> struct Tile<16, 0> { static constexpr int PR = 4, PC = 2, MR = 4, MC = 8; };
template <> struct Tile<8, 0>  { static constexpr int PR = 2, PC = 1, MR = 4, MC = 8; };
template <> struct Tile<4, 0>  { static constexpr int PR = 1, PC = 1, MR = 4, MC = 4; };
template <> struct Tile<16, 1> { static constexpr int PR = 4, PC = 4, MR = 4, MC = 4; };
template <> struct Tile<8, 1>  { static constexpr int PR = 4, PC = 2, MR = 2, MC = 4; };
template <> struct Tile<4, 1>  { static constexpr int PR = 2, PC = 2, MR = 2, MC = 2; };

template <int M_, int V_> struct Geom {
    static constexpr int M = M_, V = V_;
    using T = Tile<M, V>;
    static constexpr int LPB = T::PR * T::PC;        // lanes per block (Dykstra)
    static constexpr int BPW = 32 / LPB;             // blocks per warp
    static constexpr int PANEL = WARPS * BPW * M;    // panel width in columns
    static constexpr int WS = PANEL + 1;             // shared row stride (floats)
    static constexpr int GPW = 32 / M;               // rounding groups per warp
    static constexpr int PASSES = (BPW + GPW - 1) / GPW;   // rounding passes per warp
    static constexpr int WORDS = PANEL / 32;         // mask words per panel row
    static_assert(T::MR >= T::PC && T::MC >= T::PR && T::MC % 2 == 0 && (T::MR * T::MC) % 4 == 0, "tile shape");
    static_assert(T::PR * T::MR == M && T::PC * T::MC == M, "tile covers the block");
    static_assert(WARPS * 32 * T::MR * T::MC <= M * WS, "the per-warp stashes of t0 fit in the key panel");
};

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float lg2_approx(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float rcp_approx(float x) {
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Register r of a lane holds line (r ^ perm) of its sub-tile, where perm is
// built from the lane's coordinate along the reduction direction.  With that
// permutation the recursive-halving exchange below needs no selects: every
// lane always sends its upper half and keeps its lower half.
template <int K, int P> __device__ __forceinline__ int xor_perm(int l) {
    int g = 0;
#pragma unroll
    for (int s = 0; (1 << s) < P; ++s) g |= ((l >> s) & 1) * (K >> (s + 1));
    return g;
}

struct OpAdd { __device__ __forceinline__ float operator()(float a, float b) const { return a + b; } };
struct OpMax { __device__ __forceinline__ float operator()(float a, float b) const { return fmaxf(a, b); } };

// After the call v[0 .. K/P) hold the reduction over the P lanes (lane stride
// `base`) of the lines those registers stand for.
template <int K, int P, class Op>
__device__ __forceinline__ void reduce_scatter(float (&v)[K], int base, Op op) {
#pragma unroll
    for (int s = 0; (1 << s) < P; ++s) {
        const int h = K >> (s + 1);
#pragma unroll
        for (int k = 0; k < h; ++k)
            v[k] = op(v[k], __shfl_xor_sync(FULL, v[k + h], base << s));
    }
}
// Inverse exchange: v[0 .. K/P) valid on entry, all K valid on return.
template <int K, int P>
__device__ __forceinline__ void all_gather(float (&v)[K], int base) {
    constexpr int S = (P == 1) ? 0 : (P == 2) ? 1 : (P == 4) ? 2 : 3;
#pragma unroll
    for (int s = S - 1; s >= 0; --s) {
        const int h = K >> (s + 1);
#pragma unroll
        for (int k = 0; k < h; ++k)
            v[k + h] = __shfl_xor_sync(FULL, v[k], base << s);
    }
}

// Kahan-compensated running sum for the few potentials a lane owns.
struct Comp {
    float hi, lo;
    __device__ __forceinline__ void add(float a) {
        float y = a - lo;
        float t = hi + y;
        lo = (t - hi) - y;
        hi = t;
    }
};

// ---------------------------------------------------------------------------
// Algorithm 1 in potential form, with stabilised linear-domain steps.
//
// In the log domain the three projections only ever add a row term and a
// column term to x + q, and after the clip x = min(t, 0), q = max(t, 0) for
// t = x + q.  So the whole state is t_ij = t0_ij + F_i + G_j with
// t0 = tau |w| (base-2 units here), and with U = 2^t (the unclipped S .* Q)
// one iteration is
//     e_ij   = min(U_ij, 1)                        (S after the previous clip)
//     rho_i  = N / sum_j e_ij                      (projection on C1)
//     kap_j  = N / sum_i e_ij rho_i                (projection on C2)
//     U_ij  <- U_ij rho_i kap_j ,  F_i += log2 rho_i ,  G_j += log2 kap_j
// with the clip (C3) and the dual update implicit in the next e.  U is the
// linear-domain iterate of Algorithm 1 (kept as U / R_i in the registers, see
// the loop below).  It is trusted only while the scalings
// applied since it was last rebuilt stay small, and is then rebuilt as
// 2^(t0 + F + G) from the log-domain potentials; that is what keeps large
// tau |w| safe in fp32.  Every CHECK iterations the products of rho_i and of
// kap_j since the last rebuild are tested against [2^-16, 2^17), and U is
// rebuilt when one of them has left that range or after MAXRUN iterations.
// From iteration 1 on every rho*kap lies in [N/M^3, N M^2], below 2^15 in
// magnitude (row sums of e are in [1/M, M], column sums of e*rho in
// [N/M, N M^2]), so between two rebuilds no entry moves by more than
// 2^(34 + 15 CHECK) = 2^94 relative to its value at the last rebuild: an
// entry that overflowed to +inf is still above the cap, and one that flushed
// to zero (below 2^-126) is still below 2^-32, when the rebuild restores it
// (in practice the scalings are within a few percent of 1 after the first
// dozen iterations and the runs reach MAXRUN).  Iteration 0 has no clip yet and is done
// entirely in the log domain with the column maximum subtracted, because
// 2^t0 of a whole column can underflow against a large entry elsewhere in
// its rows.
//
// On entry t holds t0 with its row maximum subtracted (exact no-op for the
// method: the first row projection removes any row constant); on return t
// holds the final t = x + q.  stash: 32 * MR * MC floats of shared memory
// private to the warp (keeps t0 while the registers hold U).
// ---------------------------------------------------------------------------
constexpr int CHECK = 4;     // iterations between range tests of the accumulated scalings
constexpr int MAXRUN = 48;   // longest run of linear-domain iterations (multiple of CHECK)

__device__ __forceinline__ bool out_of_window(float p) {
    const unsigned e = (__float_as_uint(p) >> 23) & 0xffu;
    return (e - 111u) > 32u && e != 255u;
}

// One iteration t >= 1 on the linear-domain iterate.  Element-wise work runs on
// pairs of columns with the packed fp32x2 add / mul / fma of sm_100 (half the
// issue slots).  The row scalings are never applied to the tile: the registers
// hold V = U / R_i with R_i the product of the rho_i since the last rebuild, and
// one multiply per element (by kap_j) is left.  Four fp32 operations per element
// and iteration, in one of two forms:
//   SAT  (M >= 16)  rs[a] = R_i:    e = sat(V R_i) = min(U, 1) by a saturating multiply
//                   (FMA pipe), row sums of e give rho_i = N / sum, column sums are
//                   sum_i e_ij rho_i, R_i <- R_i rho_i in every lane of the row;
//   !SAT (M <= 8)   rs[a] = 1/R_i:  m = min(V, 1/R_i) (the clip threshold moves
//                   instead of the tile), the new R_i is simply N / sum_j m_ij and
//                   the column sums are sum_i m_ij R_i(new).
// Both compute the same iterate; which one is faster depends on how the ALU pipe
// (fp32 min) and the FMA pipe are loaded at that block size (measured).
template <int M> struct UseSat { static constexpr bool value = (M >= 16); };

// DELTA: also returns this lane's share of the marginal violation seen by the iteration,
// max over the lines it owns of |row sum of e - N| and |column sum of e rho - N|.
template <class G, bool DELTA = false>
__device__ __forceinline__ float dykstra_step(float2 (&V)[G::T::MR][G::T::MC / 2], float (&rs)[G::T::MR],
                                              float (&Pr)[G::T::MR / G::T::PC],
                                              float (&Pc)[G::T::MC / G::T::PR], float Nf, float invN) {
    using T = typename G::T;
    constexpr int M = G::M;
    constexpr int MR = T::MR, MC = T::MC, PR = T::PR, PC = T::PC;
    constexpr int RO = MR / PC, CO = MC / PR, MP = MC / 2;
    constexpr bool SAT = UseSat<M>::value;
    float2 m[MR][MP];
    float rp[MR], sc[MR], thr[MR], cp[MC], kap[MC];
#pragma unroll
    for (int a = 0; a < MR; ++a) {
        float2 s2;
#pragma unroll
        for (int b = 0; b < MP; ++b) {
            if (SAT) m[a][b] = make_float2(__saturatef(V[a][b].x * rs[a]), __saturatef(V[a][b].y * rs[a]));
            else m[a][b] = make_float2(fminf(V[a][b].x, rs[a]), fminf(V[a][b].y, rs[a]));
            s2 = (b == 0) ? m[a][b] : __fadd2_rn(s2, m[a][b]);
        }
        rp[a] = s2.x + s2.y;
    }
    reduce_scatter<MR, PC>(rp, 1, OpAdd());
    float delta = 0.0f;
    if (DELTA) {   // row sums of e: rp itself (SAT), rp R_i(old) otherwise
#pragma unroll
        for (int k = 0; k < RO; ++k) delta = fmaxf(delta, fabsf((SAT ? rp[k] : rp[k] * Pr[k]) - Nf));
    }
#pragma unroll
    for (int k = 0; k < RO; ++k) {
        sc[k] = Nf * rcp_approx(rp[k]);          // SAT: rho_i; !SAT: the new R_i
        if (SAT) Pr[k] *= sc[k];
        else { Pr[k] = sc[k]; thr[k] = rp[k] * invN; }
    }
    all_gather<MR, PC>(sc, 1);
    if (!SAT) all_gather<MR, PC>(thr, 1);
#pragma unroll
    for (int b = 0; b < MP; ++b) {
        float2 c2 = __fmul2_rn(m[0][b], make_float2(sc[0], sc[0]));
#pragma unroll
        for (int a = 1; a < MR; ++a) c2 = __ffma2_rn(m[a][b], make_float2(sc[a], sc[a]), c2);
        cp[2 * b] = c2.x;
        cp[2 * b + 1] = c2.y;
    }
    reduce_scatter<MC, PR>(cp, PC, OpAdd());
    if (DELTA) {
#pragma unroll
        for (int k = 0; k < CO; ++k) delta = fmaxf(delta, fabsf(cp[k] - Nf));
    }
#pragma unroll
    for (int k = 0; k < CO; ++k) {
        kap[k] = Nf * rcp_approx(cp[k]);
        Pc[k] *= kap[k];
    }
    all_gather<MC, PR>(kap, PC);
#pragma unroll
    for (int a = 0; a < MR; ++a) {
        if (SAT) rs[a] *= sc[a];
        else rs[a] = thr[a];
#pragma unroll
        for (int b = 0; b < MP; ++b) V[a][b] = __fmul2_rn(V[a][b], make_float2(kap[2 * b], kap[2 * b + 1]));
    }
    return delta;
}

// Returns the number of iterations run: iters, or fewer in the stopping-test mode (ee_eps > 0):
// after every group of CHECK iterations, i.e. at iterations 5, 9, 13, ... of Algorithm 1, the
// warp stops once the marginal violation of every block it holds is below ee_eps.
template <class G>
__device__ __forceinline__ int dykstra_iterate(float (&t)[G::T::MR][G::T::MC], float* stash, int lane,
                                               float Nf, float log2N, int iters, float ee_eps) {
    using T = typename G::T;
    constexpr int MR = T::MR, MC = T::MC, PR = T::PR, PC = T::PC;
    constexpr int RO = MR / PC, CO = MC / PR;  // lines whose sums this lane finishes
    constexpr int MP = MC / 2, NQ = MR * MC / 4;
    float F[MR], Gc[MC];
    Comp Fo[RO], Go[CO];
    float Pr[RO], Pc[CO];                      // products of rho / kap since the last rebuild
    if (iters <= 0) return 0;
    float4* const st4 = reinterpret_cast<float4*>(stash) + lane;
#pragma unroll
    for (int q = 0; q < NQ; ++q) {   // sub-tile in row-major order, four elements per slot
        const int e = 4 * q;
        st4[q * 32] = make_float4(t[e / MC][e % MC], t[(e + 1) / MC][(e + 1) % MC], t[(e + 2) / MC][(e + 2) % MC],
                                  t[(e + 3) / MC][(e + 3) % MC]);
    }
    {   // iteration 0, log domain
        float rp[MR];
#pragma unroll
        for (int a = 0; a < MR; ++a) {
            float s = 0.f;
#pragma unroll
            for (int b = 0; b < MC; ++b) s += ex2_approx(t[a][b]);
            rp[a] = s;
        }
        reduce_scatter<MR, PC>(rp, 1, OpAdd());
#pragma unroll
        for (int k = 0; k < RO; ++k) {
            Fo[k].hi = log2N - lg2_approx(rp[k]);
            Fo[k].lo = 0.f;
            F[k] = Fo[k].hi;
            Pr[k] = 1.0f;
        }
        all_gather<MR, PC>(F, 1);
        float cm[MC];
#pragma unroll
        for (int b = 0; b < MC; ++b) {
            float m = t[0][b] + F[0];
#pragma unroll
            for (int a = 1; a < MR; ++a) m = fmaxf(m, t[a][b] + F[a]);
            cm[b] = m;
        }
        reduce_scatter<MC, PR>(cm, PC, OpMax());
        all_gather<MC, PR>(cm, PC);
        float cp[MC];
#pragma unroll
        for (int b = 0; b < MC; ++b) {
            float s = 0.f;
#pragma unroll
            for (int a = 0; a < MR; ++a) s += ex2_approx((t[a][b] + F[a]) - cm[b]);
            cp[b] = s;
        }
        reduce_scatter<MC, PR>(cp, PC, OpAdd());
#pragma unroll
        for (int k = 0; k < CO; ++k) {
            Go[k].hi = (log2N - cm[k]) - lg2_approx(cp[k]);
            Go[k].lo = 0.f;
            Pc[k] = 1.0f;
        }
    }
    // Iterations 1 .. iters-1 in runs: rebuild U from the potentials, then groups of
    // CHECK iterations with the range test of the accumulated scalings between groups.
    float2 V[MR][MP];
    float rs[MR];
    const float invN = 1.0f / Nf;
    int it = 1;
#pragma unroll 1
    while (it < iters) {
#pragma unroll
        for (int k = 0; k < RO; ++k) { Fo[k].add(lg2_approx(Pr[k])); Pr[k] = 1.0f; F[k] = Fo[k].hi; }
#pragma unroll
        for (int k = 0; k < CO; ++k) { Go[k].add(lg2_approx(Pc[k])); Pc[k] = 1.0f; Gc[k] = Go[k].hi; }
        all_gather<MR, PC>(F, 1);
        all_gather<MC, PR>(Gc, PC);
#pragma unroll
        for (int q = 0; q < NQ; ++q) {   // pairs never straddle a row (MC is even)
            const int a0 = (4 * q) / MC, b0 = (4 * q) % MC, a1 = (4 * q + 2) / MC, b1 = (4 * q + 2) % MC;
            const float4 v = st4[q * 32];
            const float2 x0 = __fadd2_rn(__fadd2_rn(make_float2(v.x, v.y), make_float2(F[a0], F[a0])),
                                         make_float2(Gc[b0], Gc[b0 + 1]));
            const float2 x1 = __fadd2_rn(__fadd2_rn(make_float2(v.z, v.w), make_float2(F[a1], F[a1])),
                                         make_float2(Gc[b1], Gc[b1 + 1]));
            V[a0][b0 / 2] = make_float2(ex2_approx(x0.x), ex2_approx(x0.y));
            V[a1][b1 / 2] = make_float2(ex2_approx(x1.x), ex2_approx(x1.y));
        }
#pragma unroll
        for (int a = 0; a < MR; ++a) rs[a] = 1.0f;     // R_i = 1 (and 1/R_i = 1)
        const int run_end = (iters - it > MAXRUN) ? it + MAXRUN : iters;
        bool wide = false;
#pragma unroll 1
        while (!wide && it + CHECK <= run_end) {
#pragma unroll(G::M == 8 ? 1 : CHECK)   // measured: unrolling the group helps every size but M = 8
            for (int u = 0; u < CHECK - 1; ++u) dykstra_step<G>(V, rs, Pr, Pc, Nf, invN);
            if (ee_eps > 0.0f) {
                const float delta = dykstra_step<G, true>(V, rs, Pr, Pc, Nf, invN);
                if (__all_sync(FULL, delta < ee_eps)) {   // every block of the warp has converged
                    it += CHECK;
                    iters = it;
                    wide = true;                          // skips the remainder loop as well
                    break;
                }
            } else {
                dykstra_step<G>(V, rs, Pr, Pc, Nf, invN);
            }
            it += CHECK;
            // exponent field in [127-16, 127+16] <=> product in [2^-16, 2^17).  A product that
            // is inf or NaN (exponent field 255: a block poisoned by a non-finite score) does
            // not vote, so that it cannot change when the other blocks of its warp rebuild.
            bool w = false;
#pragma unroll
            for (int k = 0; k < RO; ++k) w |= out_of_window(Pr[k]);
#pragma unroll
            for (int k = 0; k < CO; ++k) w |= out_of_window(Pc[k]);
            wide = __any_sync(FULL, w);
        }
        if (!wide) {   // fewer than CHECK iterations left (end of the last run only)
#pragma unroll 1
            for (; it < run_end; ++it) dykstra_step<G>(V, rs, Pr, Pc, Nf, invN);
        }
    }
    // final potentials and t = t0 + F + G
#pragma unroll
    for (int k = 0; k < RO; ++k) { Fo[k].add(lg2_approx(Pr[k])); F[k] = Fo[k].hi; }
#pragma unroll
    for (int k = 0; k < CO; ++k) { Go[k].add(lg2_approx(Pc[k])); Gc[k] = Go[k].hi; }
    all_gather<MR, PC>(F, 1);
    all_gather<MC, PR>(Gc, PC);
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
        const int e = 4 * q;
        const float4 v = st4[q * 32];
        t[e / MC][e % MC] = (v.x + F[e / MC]) + Gc[e % MC];
        t[(e + 1) / MC][(e + 1) % MC] = (v.y + F[(e + 1) / MC]) + Gc[(e + 1) % MC];
        t[(e + 2) / MC][(e + 2) % MC] = (v.z + F[(e + 2) / MC]) + Gc[(e + 2) % MC];
        t[(e + 3) / MC][(e + 3) % MC] = (v.w + F[(e + 3) / MC]) + Gc[(e + 3) % MC];
    }
    return iters;
}

// ---------------------------------------------------------------------------
// Score source: the matrix the solver works on, described rather than
// materialised (Section 4: magnitude, ADMM D-update, SparseGPT group, Wanda).
// One fp32 rounding per operation, no fused multiply-add.
// ---------------------------------------------------------------------------
enum : int { SC_ABS = 0, SC_ADMM = 1, SC_COLDIV = 2, SC_COLMUL = 3 };

struct ScoreSrc {
    int kind, w_is_bf16;
    const void* w; int64_t ld;
    const float* v; int64_t ld_v;
    float scalar;
    const float* colvec;
    int vec_w, vec_v, vec_c;       // 16-byte (8-byte for bf16) vector loads allowed
};

__device__ __forceinline__ float score_of(int kind, float w, float v, float scalar, float cv) {
    switch (kind) {
        case SC_ADMM: { const float s = __fadd_rn(w, __fmul_rn(v, scalar)); return __fmul_rn(s, s); }
        case SC_COLDIV: return fabsf(__fdiv_rn(w, cv));
        case SC_COLMUL: return __fmul_rn(fabsf(w), cv);
        default: return fabsf(w);
    }
}

// Scores of the four consecutive elements (r, c .. c+3); c is a multiple of 4.
__device__ __forceinline__ float4 load_score_quad(const ScoreSrc& S, int64_t r, int64_t c) {
    float4 w;
    if (S.w_is_bf16) {
        const unsigned short* p = static_cast<const unsigned short*>(S.w) + r * S.ld + c;
        unsigned lo, hi;
        if (S.vec_w) {
            const uint2 q = __ldg(reinterpret_cast<const uint2*>(p));
            lo = q.x; hi = q.y;
        } else {
            lo = __ldg(p) | ((unsigned)__ldg(p + 1) << 16);
            hi = __ldg(p + 2) | ((unsigned)__ldg(p + 3) << 16);
        }
        w = make_float4(__uint_as_float(lo << 16), __uint_as_float(lo & 0xffff0000u),
                        __uint_as_float(hi << 16), __uint_as_float(hi & 0xffff0000u));
    } else {
        const float* p = static_cast<const float*>(S.w) + r * S.ld + c;
        if (S.vec_w) w = __ldg(reinterpret_cast<const float4*>(p));
        else w = make_float4(__ldg(p), __ldg(p + 1), __ldg(p + 2), __ldg(p + 3));
    }
    if (S.kind == SC_ABS) return make_float4(fabsf(w.x), fabsf(w.y), fabsf(w.z), fabsf(w.w));
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f), cv = make_float4(1.f, 1.f, 1.f, 1.f);
    if (S.kind == SC_ADMM) {
        const float* p = S.v + r * S.ld_v + c;
        if (S.vec_v) v = __ldg(reinterpret_cast<const float4*>(p));
        else v = make_float4(__ldg(p), __ldg(p + 1), __ldg(p + 2), __ldg(p + 3));
    } else {
        const float* p = S.colvec + c;
        if (S.vec_c) cv = __ldg(reinterpret_cast<const float4*>(p));
        else cv = make_float4(__ldg(p), __ldg(p + 1), __ldg(p + 2), __ldg(p + 3));
    }
    return make_float4(score_of(S.kind, w.x, v.x, S.scalar, cv.x), score_of(S.kind, w.y, v.y, S.scalar, cv.y),
                       score_of(S.kind, w.z, v.z, S.scalar, cv.z), score_of(S.kind, w.w, v.w, S.scalar, cv.w));
}

__device__ __forceinline__ int any_nan(const float4& v) {
    return !(v.x == v.x) | !(v.y == v.y) | !(v.z == v.z) | !(v.w == v.w);
}
__device__ __forceinline__ int any_nonfinite(const float4& v) {
    return !(fabsf(v.x) <= 3.4028234e38f) | !(fabsf(v.y) <= 3.4028234e38f) |
           !(fabsf(v.z) <= 3.4028234e38f) | !(fabsf(v.w) <= 3.4028234e38f);
}

// ---------------------------------------------------------------------------
// Where a panel's cells live in the matrix.  Wide matrices: the panel is M rows
// x PANEL columns at (r0, c0).  Slabs (a single block column, cols == M, as in
// the column groups of SparseGPT): the panel's blocks are stacked vertically,
// block b of the panel being rows [(first + b) M, (first + b + 1) M), so that a
// CTA still gets a full set of blocks and the whole slab is one wave of CTAs.
// In shared memory both look the same: block b occupies columns [b M, b M + M).
// ---------------------------------------------------------------------------
template <int M> struct PanelMap {
    int tall;
    int64_t r0, c0;        // wide: origin of the panel
    int64_t first;         // tall: first block (= block row) of the panel
    int valid_cols;        // columns of the shared-memory panel that hold blocks
    int64_t rows, cols;    // extent of the matrix
    __device__ __forceinline__ bool holds_quad(int64_t r, int64_t c) const {
        return r >= 0 && r < rows && c >= 0 && c + 4 <= cols;
    }
    __device__ __forceinline__ int64_t row(int r, int c) const { return tall ? (first + c / M) * M + r : r0 + r; }
    __device__ __forceinline__ int64_t col(int c) const { return tall ? (int64_t)(c % M) : c0 + c; }
};

// ---------------------------------------------------------------------------
// Panel loaders: an M x PANEL panel into shared memory, coalesced, vector
// loads when the addresses allow it.  Return non-zero if this thread saw a
// non-finite score, respectively a NaN key.
// ---------------------------------------------------------------------------
template <class G>
__device__ __forceinline__ int load_score_panel(const ScoreSrc& S, const PanelMap<G::M>& pm,
                                                float* __restrict__ dst) {
    constexpr int M = G::M;
    constexpr int V = G::PANEL / 4;
    int bad = 0;
    for (int idx = threadIdx.x; idx < M * V; idx += WARPS * 32) {
        const int r = idx / V, c = (idx % V) * 4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < pm.valid_cols && TS_CHECK(pm.holds_quad(pm.row(r, c), pm.col(c))))
            v = load_score_quad(S, pm.row(r, c), pm.col(c));  // a quad is all in or all out
        bad |= any_nonfinite(v);
        if (TS_CHECK(r < M && c + 4 <= G::PANEL)) {
            float* d = dst + r * G::WS + c;
            d[0] = v.x; d[1] = v.y; d[2] = v.z; d[3] = v.w;
        }
    }
    return bad;
}

template <class G>
__device__ __forceinline__ int load_key_panel(const float* __restrict__ src, int64_t ld, const PanelMap<G::M>& pm,
                                              bool vec_ok, float* __restrict__ dst) {
    constexpr int M = G::M;
    constexpr int V = G::PANEL / 4;
    int bad = 0;
    for (int idx = threadIdx.x; idx < M * V; idx += WARPS * 32) {
        const int r = idx / V, c = (idx % V) * 4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < pm.valid_cols && TS_CHECK(pm.holds_quad(pm.row(r, c), pm.col(c)))) {
            const float* p = src + pm.row(r, c) * ld + pm.col(c);
            if (vec_ok) v = __ldg(reinterpret_cast<const float4*>(p));
            else v = make_float4(__ldg(p), __ldg(p + 1), __ldg(p + 2), __ldg(p + 3));
        }
        bad |= any_nan(v);          // infinite keys have a place in the order; NaN keys are flagged
        if (TS_CHECK(r < M && c + 4 <= G::PANEL)) {
            float* d = dst + r * G::WS + c;
            d[0] = v.x; d[1] = v.y; d[2] = v.z; d[3] = v.w;
        }
    }
    return bad;
}

// ---------------------------------------------------------------------------
// Rounding stage (Algorithm 2).  A group of M lanes owns one block; lane i of
// the group plays row i and column i at once.
// ---------------------------------------------------------------------------
// Tables of the rounding stage: for every line (row or column) of a block the
// M prefix sets of its sorted order, prefix p = bit mask of the positions of its
// p+1 best entries (uint32 words for M = 32, uint16 otherwise).  Each lane only
// ever reads the two tables of its own row and column.  The row tables (and for
// M <= 16 the column tables too) are written over the block's own key cells once
// both sorts have consumed the keys: key row i (M floats = 4M bytes) becomes
//   M = 32 :  [0,4M) row prefixes of row i          (column prefixes: SmemLayout::cpre)
//   M <= 16:  [0,2M) row prefixes of row i, [2M,4M) column prefixes of column i
constexpr int CPRE_STRIDE = 33;   // words per column-prefix table at M = 32 (odd: conflict-free)

// Strict order "key descending, index ascending" as one ascending u64.
__device__ __forceinline__ unsigned long long sort_word(float key, int idx) {
    if (!(key == key)) key = __int_as_float(0xff800000);  // NaN orders as -inf
    key += 0.0f;                                          // -0 -> +0
    unsigned u = __float_as_uint(key);
    u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);       // ascending uint == ascending float
    return ((unsigned long long)(~u) << 32) | (unsigned)idx;
}

// The same order packed into one ascending 32-bit word: the high word of sort_word with its
// five low bits replaced by the index.  Dropping those bits is harmless unless two keys of
// the line agree in the 27 bits kept ("same bucket"): then their order may depend on the
// bits dropped, and the caller falls back to the 64-bit words.  Keys that are exactly zero
// (the capped entries of a plan: up to half of a line) are the one common case of equal
// keys; each of them gets a bucket of its own, ZERO_BUCKET + index (zeros order among
// themselves by index), and the positive keys are shifted down by the 32 buckets this takes.
constexpr unsigned ZERO_BUCKET = 0x03ffffe0u;
__device__ __forceinline__ unsigned sort_word_packed(float key, unsigned idx) {
    if (!(key == key)) key = __int_as_float(0xff800000);
    key += 0.0f;
    const unsigned b = __float_as_uint(key);
    unsigned hi;
    if (b & 0x80000000u) hi = b;                               // negative: larger magnitude later
    else if (b == 0u) hi = (ZERO_BUCKET + idx) << 5;
    else hi = 0x7fffffffu - b - (32u * 32u + 31u);             // positive: larger first, all before the zeros
    return (hi & ~31u) | idx;
}

// Batcher's odd-even merge sort as a fully unrolled network (191 compare-exchanges for 32
// keys, 63 for 16, 19 for 8, 5 for 4), ascending.  Indices are template constants so that the
// keys stay in registers.  A compare-exchange costs two instructions on 32-bit words (min,
// max) and six on 64-bit words.
template <int I, int J, int M> __device__ __forceinline__ void cmp_swap(unsigned long long (&v)[M]) {
    const unsigned long long a = v[I], b = v[J];
    const bool sw = a > b;
    v[I] = sw ? b : a;
    v[J] = sw ? a : b;
}
template <int I, int J, int M> __device__ __forceinline__ void cmp_swap(unsigned (&v)[M]) {
    const unsigned a = v[I], b = v[J];
    v[I] = min(a, b);
    v[J] = max(a, b);
}
template <int LO, int N, int R, int I, class T, int M> __device__ __forceinline__ void oem_chain(T (&v)[M]) {
    if constexpr (I + R < LO + N) {
        cmp_swap<I, I + R, M>(v);
        oem_chain<LO, N, R, I + 2 * R, T, M>(v);
    }
}
// merges the two sorted halves of the subsequence LO, LO+R, LO+2R, ... of v[LO .. LO+N)
template <int LO, int N, int R, class T, int M> __device__ __forceinline__ void oem_merge(T (&v)[M]) {
    if constexpr (2 * R < N) {
        oem_merge<LO, N, 2 * R, T, M>(v);
        oem_merge<LO + R, N, 2 * R, T, M>(v);
        oem_chain<LO, N, R, LO + R, T, M>(v);
    } else {
        cmp_swap<LO, LO + R, M>(v);
    }
}
template <int LO, int N, class T, int M> __device__ __forceinline__ void oem_sort(T (&v)[M]) {
    if constexpr (N > 1) {
        oem_sort<LO, N / 2, T, M>(v);
        oem_sort<LO + N / 2, N / 2, T, M>(v);
        oem_merge<LO, N, 1, T, M>(v);
    }
}
template <class T, int M> __device__ __forceinline__ void sort_regs(T (&v)[M]) { oem_sort<0, M, T, M>(v); }

// Sorts one line (stride `st` floats in shared memory) and returns the prefix sets of the
// sorted order: pre[p] = positions of the p+1 best entries, packed two per word (16 bits
// each) for M <= 16.
template <int M> struct PreWords { static constexpr int value = (M == 32) ? 32 : M / 2; };
template <int M, class T>
__device__ __forceinline__ void prefix_sets(const T (&v)[M], unsigned (&pre)[PreWords<M>::value]) {
    unsigned acc = 0u;
#pragma unroll
    for (int p = 0; p < M; ++p) {
        acc |= 1u << ((unsigned)v[p] & 31u);
        if (M == 32) pre[p] = acc;
        else if (p % 2 == 0) pre[p / 2] = acc;
        else pre[p / 2] |= acc << 16;
    }
}
template <int M>
__device__ __forceinline__ void sort_line(const float* line, int st, unsigned (&pre)[PreWords<M>::value]) {
    bool same_bucket;
    {   // fast path: packed 32-bit words
        unsigned w[M];
#pragma unroll
        for (int k = 0; k < M; ++k) w[k] = sort_word_packed(line[k * st], k);
        sort_regs(w);
        unsigned closest = 0xffffffffu;     // smallest difference pattern of two neighbours
#pragma unroll
        for (int p = 0; p + 1 < M; ++p) closest = min(closest, w[p] ^ w[p + 1]);
        same_bucket = closest < 32u;
        prefix_sets<M>(w, pre);
    }
    if (__any_sync(FULL, same_bucket)) {   // rare: two non-zero keys of a line within 2^-18 of each other
        unsigned long long v[M];
#pragma unroll
        for (int k = 0; k < M; ++k) v[k] = sort_word(line[k * st], k);
        sort_regs(v);
        prefix_sets<M>(v, pre);
    }
}

// Prefix p of a stored table (tab points to the table's first byte).
template <int M> __device__ __forceinline__ unsigned prefix_at(const void* tab, int p) {
    if (!TS_CHECK(p >= 0 && p < M)) return 0u;
    if (M == 32) return static_cast<const unsigned*>(tab)[p];
    return static_cast<const unsigned short*>(tab)[p];
}

// The first `cap` entries of `avail` (a set of positions of one line) in the line's sorted
// order, or all of them if there are no more than `cap`: binary search for the shortest
// prefix of the order that holds `cap` available entries.
template <int M>
__device__ __forceinline__ unsigned first_available(unsigned avail, int cap, const void* tab) {
    if (__popc(avail) <= cap) return avail;
    int p = 0;
#pragma unroll
    for (int b = M / 2; b > 0; b >>= 1)
        if (__popc(avail & prefix_at<M>(tab, p + b - 1)) < cap) p += b;
    return avail & prefix_at<M>(tab, p);
}

// Transpose of the M x M bit matrix whose row i is held by lane i of a group of M lanes
// (bit j of x = element (i, j)): recursive exchange of the off-diagonal blocks.
template <int M> __device__ __forceinline__ unsigned transpose_bits(unsigned x, int i) {
#pragma unroll
    for (int s = M / 2; s > 0; s >>= 1) {
        // positions whose bit s is clear
        const unsigned lo = (s == 16) ? 0x0000ffffu : (s == 8) ? 0x00ff00ffu : (s == 4) ? 0x0f0f0f0fu
                          : (s == 2) ? 0x33333333u : 0x55555555u;
        const unsigned y = __shfl_xor_sync(FULL, x, s);
        const bool up = (i & s) != 0;
        const unsigned keep = up ? ~lo : lo;
        const unsigned z = up ? (y >> s) : (y << s);
        x = (x & keep) | (z & ~keep);
    }
    return x;
}

// Greedy selection + local search for the block of this lane's group.
//   ks, ws: shared-memory pointers to element (0,0) of the block's keys and
//   |scores| (row stride WS); the key cells are overwritten.  cpre: this
//   lane's column-prefix table when it does not fit in the key cells (M = 32).
//   active: group has a block.
// Returns this lane's row of the mask (M bits).  flags accumulates DEV_* bits.
template <class G>
__device__ __forceinline__ unsigned round_block(float* ks, const float* ws, unsigned* cpre, int lane, bool active,
                                                int N, int ls_steps, int& flags) {
    constexpr int M = G::M;
    constexpr int WS = G::WS;
    constexpr unsigned GM = (M == 32) ? 0xffffffffu : ((1u << (M & 31)) - 1u);
    const int i = lane % M;            // my row, and my column
    const int gsh = (lane / M) * M;    // first lane of my group

    // ---- sorted orders of my row and of my column (Algorithm 2 line 2), kept as prefix sets
    unsigned char* const rtab = reinterpret_cast<unsigned char*>(ks + i * WS);
    unsigned char* const ctab = (M == 32) ? reinterpret_cast<unsigned char*>(cpre) : rtab + 2 * M;
    {
        constexpr int PW = PreWords<M>::value;
        unsigned pc[PW];
        sort_line<M>(ks + i, WS, pc);
        if (M == 32) {                      // not aliased with the keys: store at once
#pragma unroll
            for (int w = 0; w < PW; ++w) reinterpret_cast<unsigned*>(ctab)[w] = pc[w];
        }
        unsigned pr[PW];
        sort_line<M>(ks + i * WS, 1, pr);
        __syncwarp();                       // every lane is done reading keys
#pragma unroll
        for (int w = 0; w < PW; ++w) reinterpret_cast<unsigned*>(rtab)[w] = pr[w];
        if (M != 32) {
#pragma unroll
            for (int w = 0; w < PW; ++w) reinterpret_cast<unsigned*>(ctab)[w] = pc[w];
        }
    }
    __syncwarp();

    // ---- greedy selection (lines 3-6) in synchronous rounds.  An available
    // entry (not taken, row and column not full) that is among the first
    // capR available entries of its row and the first capC of its column
    // (cap = remaining capacity) is taken by the sequential scan whatever
    // happens elsewhere, so all such entries are taken at once; the first
    // available entry in the global order always qualifies, hence every round
    // makes progress and the fixed point is the sequential result.  availR:
    // available columns of my row; availC: available rows of my column.
    unsigned availR = active ? GM : 0u, availC = availR;
    int capR = active ? N : 0, capC = capR;
    unsigned sel = 0u, selC = 0u;
    for (int round = 0; round < M * M; ++round) {
        if (!__any_sync(FULL, availR != 0u)) break;
        if (round == M * M - 1) flags |= DEV_INTERNAL;
        const unsigned pickR = first_available<M>(availR, capR, rtab);
        const unsigned pickC = first_available<M>(availC, capC, ctab);
        // an entry picked from both sides is taken
        const unsigned takenR = pickR & transpose_bits<M>(pickC, i);   // columns taken in my row
        const unsigned takenC = transpose_bits<M>(takenR, i);          // rows taken in my column
        sel |= takenR;
        selC |= takenC;
        capR -= __popc(takenR);
        capC -= __popc(takenC);
        // lines that just filled up drop out, and so do their entries
        const unsigned fullR = (__ballot_sync(FULL, capR == 0) >> gsh) & GM;
        const unsigned fullC = (__ballot_sync(FULL, capC == 0) >> gsh) & GM;
        availR = (capR == 0) ? 0u : (availR & ~takenR & ~fullC);
        availC = (capC == 0) ? 0u : (availC & ~takenC & ~fullR);
    }

    // ---- local search (lines 7-13, Eq. 6).  sel: my row of the mask (bits over columns);
    // selC: my column (bits over rows).  Lane j' scans the rows i' that can form a valid
    // triple with it: S[i'][j'] = 1 and S[i'][j] = 0, provided S[i][j'] = 0.
    bool stopped = !active;
    int steps = 0;
    for (int it = 0; it <= M * N; ++it) {
        const unsigned rdef = (__ballot_sync(FULL, capR > 0) >> gsh) & GM;
        const unsigned cdef = (__ballot_sync(FULL, capC > 0) >> gsh) & GM;
        const bool work = !stopped && rdef != 0u && cdef != 0u && (ls_steps < 0 || steps < ls_steps);
        if (!__any_sync(FULL, work)) break;
        if (it == M * N) { flags |= DEV_INTERNAL; break; }
        const int di = work ? __ffs(rdef) - 1 : 0;   // lowest unsaturated row
        const int dj = work ? __ffs(cdef) - 1 : 0;   // lowest unsaturated column
        const int jp = i;                            // my candidate column j'
        const bool lines_ok = TS_CHECK(di >= 0 && di < M && dj >= 0 && dj < M);
        const unsigned col_dj = __shfl_sync(FULL, selC, lines_ok ? dj : 0, M);   // rows that hold column j
        unsigned cand = (work && lines_ok && !((selC >> di) & 1u)) ? (selC & ~col_dj & GM) : 0u;
        float best = __int_as_float(0xff800000);
        int bi = 0x7fffffff;
        const float w_ijp = lines_ok ? ws[di * WS + jp] : 0.0f;
        while (cand) {                               // ascending i': ties keep the smallest
            const int ip = __ffs(cand) - 1;
            cand &= cand - 1u;
            if (!TS_CHECK(ip < M)) continue;
            const float sc = __fsub_rn(__fadd_rn(w_ijp, ws[ip * WS + dj]), ws[ip * WS + jp]);
            if (sc > best) { best = sc; bi = ip; }
        }
        int bflat = (bi == 0x7fffffff) ? 0x7fffffff : bi * M + jp;
#pragma unroll
        for (int off = M / 2; off > 0; off >>= 1) {
            const float ob = __shfl_xor_sync(FULL, best, off, M);
            const int of = __shfl_xor_sync(FULL, bflat, off, M);
            if (ob > best || (ob == best && of < bflat)) { best = ob; bflat = of; }
        }
        if (work) {
            if (bflat == 0x7fffffff) {            // no valid triple: only with non-finite scores
                stopped = true;
            } else if (ls_steps >= 0 && !(best > 0.0f)) {
                stopped = true;                   // paper-strict loop: improving swaps only
            } else if (!TS_CHECK(bflat >= 0 && bflat < M * M)) {
                stopped = true;
            } else {
                const int ip = bflat / M, jq = bflat % M;
                if (i == ip) sel = (sel & ~(1u << jq)) | (1u << dj);
                if (i == di) { sel |= 1u << jq; --capR; }
                if (i == jq) selC = (selC & ~(1u << ip)) | (1u << di);
                if (i == dj) { selC |= 1u << ip; --capC; }
                ++steps;
            }
        }
    }
    if (active && (capR != 0 || capC != 0)) flags |= DEV_UNDERFILLED;
    return sel;
}

// ---------------------------------------------------------------------------
// Fused kernel.  MODE 0: whole method; 1: Algorithm 1 only (plan to global);
// 2: Algorithm 2 only (keys from global).
// ---------------------------------------------------------------------------
struct Params {
    ScoreSrc src;
    const float* keys;   int64_t ld_keys;
    float* plan;         int64_t ld_plan; int plan_is_log;
    uint32_t* bits;      int64_t wpr;
    int64_t rows, cols;
    int npc;                       // panels per block row
    int tall;                      // slab: one block column, panels stacked vertically
    int N; float Nf, log2N;
    float c_hi, c_lo;              // tau * log2(e), split in two floats
    int per_block_tau;             // tau is divided by each block's own largest score
    int iters, ls_steps;
    float ee_eps;                  // > 0: stopping test of Algorithm 1 (non-parity mode)
    unsigned long long* iter_sum;  // optional: iterations run, summed over the blocks
    int32_t* status;
    int vec_keys;
};

template <class G, int MODE> struct SmemLayout {
    static constexpr int M = G::M;
    float w[M * G::WS];
    float k[M * G::WS];
    unsigned int bits[M * G::WORDS];
    unsigned int cpre[(M == 32) ? WARPS * 32 * CPRE_STRIDE : 1];   // column-prefix tables (M = 32)
};
template <class G> struct SmemLayout<G, 1> {   // Algorithm 1 alone: score panel and the t0 stash
    static constexpr int M = G::M;
    float w[M * G::WS];
    float k[WARPS * 32 * G::T::MR * G::T::MC];
    unsigned int bits[1];
    unsigned int cpre[1];
};
// Resident CTAs per SM the register allocation aims for.
template <int M, int V> struct MinBlocks { static constexpr int value = (V == 1) ? 4 : (M == 4) ? 5 : 4; };

template <int M, int MODE, int V>
__global__ void __launch_bounds__(WARPS * 32, MinBlocks<M, V>::value) tsenor_kernel(const Params P) {
    using G = Geom<M, V>;
    using T = typename G::T;
    constexpr int MR = T::MR, MC = T::MC, PR = T::PR, PC = T::PC;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SmemLayout<G, MODE>& sm = *reinterpret_cast<SmemLayout<G, MODE>*>(smem_raw);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t panel = blockIdx.x;
    PanelMap<M> pm;
    pm.tall = P.tall;
    pm.rows = P.rows; pm.cols = P.cols;
#ifdef TSENOR_BOUNDS
    if (threadIdx.x == 0) g_bounds_flags = 0;
    __syncthreads();
#endif
    if (P.tall) {
        constexpr int NB = G::PANEL / M;
        const int64_t left = P.rows / M - panel * NB;
        pm.first = panel * NB; pm.r0 = 0; pm.c0 = 0;
        pm.valid_cols = (int)(left < NB ? left : NB) * M;
    } else {
        pm.r0 = (panel / P.npc) * M;
        pm.c0 = (panel % P.npc) * (int64_t)G::PANEL;
        pm.first = 0;
        pm.valid_cols = (int)((P.cols - pm.c0 < G::PANEL) ? (P.cols - pm.c0) : G::PANEL);
    }
    const int valid_cols = pm.valid_cols;
    int flags = 0;

    // ---- block loader
    if (load_score_panel<G>(P.src, pm, sm.w)) flags |= DEV_NONFINITE;
    if (MODE == 2)
        if (load_key_panel<G>(P.keys, P.ld_keys, pm, P.vec_keys != 0, sm.k)) flags |= DEV_NONFINITE;
    if (MODE != 1)
        for (int idx = threadIdx.x; idx < M * G::WORDS; idx += WARPS * 32) sm.bits[idx] = 0u;
    __syncthreads();

    // ---- Algorithm 1
    if (MODE != 2) {
        const int g = lane % G::LPB;                          // lane inside its block
        const int blk = warp * G::BPW + lane / G::LPB;        // block inside the panel
        const int lr = g / PC, lc = g % PC;
        const int gr = xor_perm<MR, PC>(lc), gc = xor_perm<MC, PR>(lr);
        const bool active = blk * M < valid_cols;
        float t[MR][MC];
        float mx[MR];
#pragma unroll
        for (int a = 0; a < MR; ++a) {
            const int row = lr * MR + (a ^ gr);
            float m = 0.f;
#pragma unroll
            for (int b = 0; b < MC; ++b) {
                const int col = blk * M + lc * MC + (b ^ gc);
                t[a][b] = TS_CHECK(row < M && col < G::PANEL) ? sm.w[row * G::WS + col] : 0.0f;
                m = fmaxf(m, t[a][b]);
            }
            mx[a] = m;
        }
        float c_hi = P.c_hi, c_lo = P.c_lo;
        if (P.iters > 0 || P.per_block_tau) {
            reduce_scatter<MR, PC>(mx, 1, OpMax());
            all_gather<MR, PC>(mx, 1);
        }
        if (P.per_block_tau) {   // tau of this block = tau_rel / its largest score
            float bm = mx[0];
#pragma unroll
            for (int a = 1; a < MR; ++a) bm = fmaxf(bm, mx[a]);
#pragma unroll
            for (int s = 0; (1 << s) < PR; ++s) bm = fmaxf(bm, __shfl_xor_sync(FULL, bm, PC << s));
            if (bm > 0.0f) {
                c_hi = __fdiv_rn(P.c_hi, bm);
                c_lo = __fdiv_rn(fmaf(-c_hi, bm, P.c_hi) + P.c_lo, bm);
            } else {
                c_hi = 0.0f; c_lo = 0.0f;
            }
        }
        if (P.iters > 0) {
#pragma unroll
            for (int a = 0; a < MR; ++a) {
                const float sh = mx[a] * c_hi;
#pragma unroll
                for (int b = 0; b < MC; ++b) t[a][b] = fmaf(t[a][b], c_lo, fmaf(t[a][b], c_hi, -sh));
            }
            const int ran =
                dykstra_iterate<G>(t, sm.k + warp * (32 * MR * MC), lane, P.Nf, P.log2N, P.iters, P.ee_eps);
            if (P.iter_sum) {   // one add per warp: iterations x blocks of the warp that exist
                const int nact = __popc(__ballot_sync(FULL, active && g == 0));
                if (lane == 0 && nact) atomicAdd(P.iter_sum, (unsigned long long)ran * nact);
            }
#pragma unroll
            for (int a = 0; a < MR; ++a)
#pragma unroll
                for (int b = 0; b < MC; ++b) t[a][b] = fminf(t[a][b], 0.0f);   // x = min(x + q, 0)
        } else {
#pragma unroll
            for (int a = 0; a < MR; ++a)
#pragma unroll
                for (int b = 0; b < MC; ++b) t[a][b] = fmaf(t[a][b], c_lo, t[a][b] * c_hi);
        }
        if (MODE == 1) {
            if (active) {
#pragma unroll
                for (int a = 0; a < MR; ++a)
#pragma unroll
                    for (int b = 0; b < MC; ++b) {
                        const int pc = blk * M + lc * MC + (b ^ gc);
                        const int64_t row = pm.row(lr * MR + (a ^ gr), pc), col = pm.col(pc);
                        if (TS_CHECK(row >= 0 && row < P.rows && col >= 0 && col < P.cols))
                            P.plan[row * P.ld_plan + col] =
                                P.plan_is_log ? t[a][b] * 0.6931471805599453f : exp2f(t[a][b]);
                    }
            }
        } else {
            __syncthreads();   // sm.k served as per-warp stash until here; now it takes the keys
#pragma unroll
            for (int a = 0; a < MR; ++a)
#pragma unroll
                for (int b = 0; b < MC; ++b)
                    if (TS_CHECK(lr * MR + (a ^ gr) < M && blk * M + lc * MC + (b ^ gc) < G::PANEL))
                        sm.k[(lr * MR + (a ^ gr)) * G::WS + blk * M + lc * MC + (b ^ gc)] = t[a][b];
        }
        __syncwarp();
    }

    // ---- Algorithm 2 and the mask writer
    if (MODE != 1) {
        const int grp = lane / M;
#pragma unroll 1
        for (int pass = 0; pass < G::PASSES; ++pass) {
            const int blk = warp * G::BPW + pass * G::GPW + grp;
            const bool active = (pass * G::GPW + grp < G::BPW) && blk * M < valid_cols;
            if (!TS_CHECK(blk * M + M <= G::PANEL)) continue;     // warp-uniform up to the group
            const unsigned row_bits =
                round_block<G>(sm.k + blk * M, sm.w + blk * M, sm.cpre + (warp * 32 + lane) * CPRE_STRIDE, lane,
                               active, P.N, P.ls_steps, flags);
            if (active && TS_CHECK(blk * M / 32 < G::WORDS)) {
                const int off = blk * M;
                if (M == 32) sm.bits[(lane % M) * G::WORDS + off / 32] = row_bits;
                else atomicOr(&sm.bits[(lane % M) * G::WORDS + off / 32], row_bits << (off % 32));
            }
            __syncwarp();
        }
        __syncthreads();
        if (P.tall) {   // one word (M bits) per matrix row
            constexpr unsigned GM = (M == 32) ? 0xffffffffu : ((1u << (M & 31)) - 1u);
            for (int idx = threadIdx.x; idx < valid_cols; idx += WARPS * 32) {
                const int blk = idx / M, r = idx % M;
                if (TS_CHECK((pm.first + blk) * M + r < P.rows && (blk * M) / 32 < G::WORDS))
                    P.bits[((pm.first + blk) * M + r) * P.wpr] =
                        (sm.bits[r * G::WORDS + (blk * M) / 32] >> ((blk * M) % 32)) & GM;
            }
        } else {
            const int nwords = (valid_cols + 31) / 32;
            for (int idx = threadIdx.x; idx < M * G::WORDS; idx += WARPS * 32) {
                const int r = idx / G::WORDS, wd = idx % G::WORDS;
                if (wd < nwords && TS_CHECK(pm.r0 + r < P.rows && pm.c0 / 32 + wd < P.wpr))
                    P.bits[(pm.r0 + r) * P.wpr + pm.c0 / 32 + wd] = sm.bits[idx];
            }
        }
    }
#ifdef TSENOR_BOUNDS
    __syncthreads();
    flags |= g_bounds_flags;
#endif
    flags = __reduce_or_sync(FULL, flags);
    if (flags && lane == 0 && P.status) atomicOr(P.status, flags);
}

}  // namespace tsenor
