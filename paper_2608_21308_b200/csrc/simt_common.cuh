// Building blocks of the any-shape kernels (scans, layer norm, reductions, phase barrier, the FMA GEMM).
// Real = double for fp32 I/O, float for bf16 I/O.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace e2ttt {

constexpr int kSimtThreads = 256;
constexpr int kMaxC = 512;  // the paper trains with chunks of 512 tokens
constexpr int kMaxMat = 3;
constexpr int kBM = 64, kBN = 64, kBK = 16;

// ---- I/O conversion -------------------------------------------------------------------------
template <typename Real> __device__ __forceinline__ Real ld_io(const float* p, size_t i) { return (Real)p[i]; }
template <typename Real> __device__ __forceinline__ Real ld_io(const __nv_bfloat16* p, size_t i) {
    return (Real)__bfloat162float(p[i]);
}
template <typename Real> __device__ __forceinline__ void st_io(float* p, size_t i, Real v) { p[i] = (float)v; }
template <typename Real> __device__ __forceinline__ void st_io(__nv_bfloat16* p, size_t i, Real v) {
    p[i] = __float2bfloat16_rn((float)v);
}

// ---- scalar nonlinearities (exact erf GELU; Section 4 "Fast-weight Network") -------------------
__device__ __forceinline__ float r_erf(float x) { return erff(x); }
__device__ __forceinline__ double r_erf(double x) { return erf(x); }
__device__ __forceinline__ float r_exp(float x) { return expf(x); }
__device__ __forceinline__ double r_exp(double x) { return exp(x); }
__device__ __forceinline__ float r_rsqrt(float x) { return 1.0f / sqrtf(x); }
__device__ __forceinline__ double r_rsqrt(double x) { return 1.0 / sqrt(x); }

template <typename Real> __device__ __forceinline__ Real norm_cdf(Real z) {
    return (Real)0.5 * ((Real)1 + r_erf(z * (Real)0.70710678118654752440));
}
template <typename Real> __device__ __forceinline__ Real norm_pdf(Real z) {
    return (Real)0.39894228040143267794 * r_exp((Real)-0.5 * z * z);
}
template <typename Real> __device__ __forceinline__ Real gelu_f(Real z) { return z * norm_cdf(z); }
template <typename Real> __device__ __forceinline__ Real gelu_d1(Real z) { return norm_cdf(z) + z * norm_pdf(z); }
template <typename Real> __device__ __forceinline__ Real gelu_d2(Real z) { return norm_pdf(z) * ((Real)2 - z * z); }
template <typename Real> __device__ __forceinline__ Real sigmoid_f(Real z) { return (Real)1 / ((Real)1 + r_exp(-z)); }
template <typename Real> __device__ __forceinline__ Real silu_f(Real z) { return z * sigmoid_f(z); }
template <typename Real> __device__ __forceinline__ Real silu_d1(Real z) {
    Real s = sigmoid_f(z);
    return s * ((Real)1 + z * ((Real)1 - s));
}

// ---- warp helpers ------------------------------------------------------------------------------
__device__ __forceinline__ float shfl_down_r(float v, int off) { return __shfl_down_sync(0xffffffffu, v, off); }
__device__ __forceinline__ double shfl_down_r(double v, int off) { return __shfl_down_sync(0xffffffffu, v, off); }
__device__ __forceinline__ float shfl_xor_r(float v, int off) { return __shfl_xor_sync(0xffffffffu, v, off); }
__device__ __forceinline__ double shfl_xor_r(double v, int off) { return __shfl_xor_sync(0xffffffffu, v, off); }
template <typename Real> __device__ __forceinline__ Real warp_sum(Real v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += shfl_xor_r(v, off);
    return v;
}

// Deterministic CTA-wide sum (fixed tree); every thread gets the result. red: >= 16 Reals of shared memory.
template <typename Real> __device__ Real block_sum(Real v, Real* red) {
    v = warp_sum(v);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    Real s = 0;
    const int nw = (int)blockDim.x >> 5;
    for (int w = 0; w < nw; ++w) s += red[w];
    return s;
}

// ---- scalar kernels of a chunk -----------------------------------------------------------------
// Suffix scans over the gates of one chunk (Eq. "scalar_aux"), in the division-free form
//   gt_t = gamma_{t+1} gt_{t+1},  bt_t = beta_{t+1} bt_{t+1},  S_t = beta_{t+1} S_{t+1} + gt_t,   S_C = bt_C = gt_C = 1,
// where S_t = bt_t R_t is the weight of G_t in W_C (the inner sum of Eq. "unroll_recurrence").  A step is the
// linear map (bt, gt, S) -> (B bt, G gt, B S + X gt); maps compose associatively, so the suffix composites come
// from a warp-shuffle scan: each lane folds its own consecutive tokens, then five shuffle rounds fold the lanes.
template <typename Real> struct ScanMap { Real B, G, X; };
template <typename Real>
__device__ __forceinline__ ScanMap<Real> compose(const ScanMap<Real>& outer, const ScanMap<Real>& inner) {
    // inner acts first (it is nearer the chunk end), outer second
    ScanMap<Real> r;
    r.B = outer.B * inner.B;
    r.G = outer.G * inner.G;
    r.X = outer.B * inner.X + outer.X * inner.G;
    return r;
}

template <typename Real> struct ChunkScalars {
    Real kW[kMaxC];     // K^W_t = eta_t S_t          (token t at index t-1)
    Real kM[kMaxC];     // K^M_t = eta_t bt_t
    Real bt[kMaxC + 1]; // bt_t, t = 0..len
    Real gt[kMaxC + 1];
    Real S[kMaxC + 1];
    Real cw, cm, cb;    // gt_0, bt_0 R_1 = beta_1 S_1, bt_0
};

// Executed by warp 0 only.  eta/beta/gamma point at the chunk's first token; len <= kMaxC tokens.
template <typename Real>
__device__ void chunk_scalars_warp(const float* eta, const float* beta, const float* gamma, int len,
                                   ChunkScalars<Real>* out) {
    constexpr int EPL = kMaxC / 32; // tokens per lane
    const int lane = threadIdx.x & 31;
    ScanMap<Real> local[EPL + 1];
    local[EPL].B = 1; local[EPL].G = 1; local[EPL].X = 0;
#pragma unroll
    for (int e = EPL - 1; e >= 0; --e) {
        const int i = lane * EPL + e;
        ScanMap<Real> m;
        if (i < len) { m.B = (Real)beta[i]; m.G = (Real)gamma[i]; m.X = m.G; }
        else { m.B = 1; m.G = 1; m.X = 0; }
        local[e] = compose(m, local[e + 1]);
    }
    ScanMap<Real> incl = local[0];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        ScanMap<Real> other;
        other.B = shfl_down_r(incl.B, off);
        other.G = shfl_down_r(incl.G, off);
        other.X = shfl_down_r(incl.X, off);
        if (lane + off < 32) incl = compose(incl, other);
    }
    ScanMap<Real> excl;
    excl.B = shfl_down_r(incl.B, 1);
    excl.G = shfl_down_r(incl.G, 1);
    excl.X = shfl_down_r(incl.X, 1);
    if (lane == 31) { excl.B = 1; excl.G = 1; excl.X = 0; }
#pragma unroll
    for (int e = 0; e <= EPL; ++e) {
        const int t = lane * EPL + e; // state index t = composite of tokens t+1..len
        if (e == EPL && lane != 31) continue; // same index as the next lane's e = 0
        if (t > len) continue;
        ScanMap<Real> f = compose(local[e], excl);
        out->bt[t] = f.B;
        out->gt[t] = f.G;
        out->S[t] = f.B + f.X;
    }
    __syncwarp();
    for (int i = lane; i < len; i += 32) {
        const Real e = (Real)eta[i];
        out->kW[i] = e * out->S[i + 1];
        out->kM[i] = e * out->bt[i + 1];
    }
    if (lane == 0) {
        out->cw = out->gt[0];
        out->cb = out->bt[0];
        out->cm = (Real)beta[0] * out->S[1];
    }
}

// ---- elementwise pass with batched loads ---------------------------------------------------------
// for e = begin, begin + stride, ... < end:  store(e, load(e)).  `load` returns everything element e needs from
// memory (a value or a small struct), `store` computes and writes.  U loads are issued before the U stores that
// follow them; written as one loop body, every load would wait for the previous element's store (the compiler must
// assume they alias) and the pass would take one memory round trip per element.
template <int U, typename FL, typename FS>
__device__ __forceinline__ void batched_for(size_t begin, size_t end, size_t stride, FL load, FS store) {
    using P = decltype(load((size_t)0));
    for (size_t e0 = begin; e0 < end; e0 += stride * U) {
        P p[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t e = e0 + (size_t)u * stride;
            if (e < end) p[u] = load(e);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t e = e0 + (size_t)u * stride;
            if (e < end) store(e, p[u]);
        }
    }
}

// ---- phase barrier ---------------------------------------------------------------------------------
// A sequence may be worked on by a cluster of `nranks` CTAs that split every phase (GEMM tiles, rows, elements)
// and share all intermediates through global memory.  The hardware cluster barrier (release / acquire at cluster
// scope) orders one phase's global writes before the next phase's reads; with one CTA it is the CTA barrier.
__device__ __forceinline__ void phase_sync(int nranks) {
    if (nranks == 1) {
        __syncthreads();
    } else {
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    }
}

// ---- generic CTA GEMM --------------------------------------------------------------------------
// out(m, n) = sum_k a(m, k) * b(n, k), m < M, n < N, k < K, for NACC (1 or 2) A operands sharing one B.
//   fa(m, k, a0, a1) writes the A value(s); fb(n, k) returns the B value; pre(m, n) loads what a result combines
//   with; epi(m, n, acc0, acc1, loaded) consumes a result.
// A_KFAST / B_KFAST say which index is contiguous in memory, so that neighbouring threads read neighbouring words.
// 64x64 output tiles (dealt round-robin to the `nranks` CTAs of the sequence's cluster), 16-deep k slices through
// shared memory, 4x4 results per thread.  Ends with phase_sync().
template <typename Real> struct GemmSmem {
    Real A[2][kBK][kBM + 4];
    Real B[kBK][kBN + 4];
};

template <typename Real, int NACC, bool A_KFAST, bool B_KFAST, typename FA, typename FB, typename FP, typename FE>
__device__ void block_gemm(int M, int N, int K, FA fa, FB fb, FP pre, FE epi, GemmSmem<Real>* sm, int rank, int nranks) {
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    int tile = 0;
    for (int m0 = 0; m0 < M; m0 += kBM) {
        for (int n0 = 0; n0 < N; n0 += kBN, ++tile) {
            if (tile % nranks != rank) continue;
            Real acc[NACC][4][4];
#pragma unroll
            for (int a = 0; a < NACC; ++a)
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[a][i][j] = 0;
            for (int k0 = 0; k0 < K; k0 += kBK) {
                __syncthreads();
#pragma unroll
                for (int r = 0; r < (kBM * kBK) / kSimtThreads; ++r) {
                    const int idx = tid + r * kSimtThreads;
                    const int mm = A_KFAST ? idx / kBK : idx % kBM;
                    const int kk = A_KFAST ? idx % kBK : idx / kBM;
                    Real a0 = 0, a1 = 0;
                    if (m0 + mm < M && k0 + kk < K) fa(m0 + mm, k0 + kk, a0, a1);
                    sm->A[0][kk][mm] = a0;
                    if (NACC == 2) sm->A[1][kk][mm] = a1;
                }
#pragma unroll
                for (int r = 0; r < (kBN * kBK) / kSimtThreads; ++r) {
                    const int idx = tid + r * kSimtThreads;
                    const int nn = B_KFAST ? idx / kBK : idx % kBN;
                    const int kk = B_KFAST ? idx % kBK : idx / kBN;
                    Real b = 0;
                    if (n0 + nn < N && k0 + kk < K) b = fb(n0 + nn, k0 + kk);
                    sm->B[kk][nn] = b;
                }
                __syncthreads();
#pragma unroll
                for (int kk = 0; kk < kBK; ++kk) {
                    Real bv[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) bv[j] = sm->B[kk][tx * 4 + j];
#pragma unroll
                    for (int a = 0; a < NACC; ++a) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const Real av = sm->A[a][kk][ty * 4 + i];
#pragma unroll
                            for (int j = 0; j < 4; ++j) acc[a][i][j] += av * bv[j];
                        }
                    }
                }
            }
            // what the results combine with is loaded for the whole 4x4 block first (loads in flight together)
            using P = decltype(pre(0, 0));
            P p[4][4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int m = m0 + ty * 4 + i, n = n0 + tx * 4 + j;
                    if (m < M && n < N) p[i][j] = pre(m, n);
                }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int m = m0 + ty * 4 + i, n = n0 + tx * 4 + j;
                    if (m < M && n < N) epi(m, n, acc[0][i][j], NACC == 2 ? acc[NACC - 1][i][j] : (Real)0, p[i][j]);
                }
        }
    }
    phase_sync(nranks);
}

// ---- layer norm of one row by one warp -----------------------------------------------------------
// Returns r = (var + eps)^(-1/2); writes y (may alias u).  d values, strided over the 32 lanes.
template <typename Real>
__device__ __forceinline__ Real warp_layernorm(const Real* u, Real* y, int d, Real eps) {
    const int lane = threadIdx.x & 31;
    Real s = 0;
    for (int i = lane; i < d; i += 32) s += u[i];
    const Real mu = warp_sum(s) / (Real)d;
    Real v = 0;
    for (int i = lane; i < d; i += 32) { const Real c = u[i] - mu; v += c * c; }
    const Real r = r_rsqrt(warp_sum(v) / (Real)d + eps);
    for (int i = lane; i < d; i += 32) y[i] = (u[i] - mu) * r;
    return r;
}

}  // namespace e2ttt
