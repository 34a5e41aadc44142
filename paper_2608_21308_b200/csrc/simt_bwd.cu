// Any-shape backward: the adjoint of the chunk program, chunks in reverse order, a cluster of 1-8 CTAs per sequence,
// for both fast-weight networks, on the same two GEMM engines as the forward (tc_gemm.cuh).  Per chunk it re-runs the chunk's forward from the saved chunk-start state, then reverses,
// in matrix form over the whole chunk,
//   (i)   the outputs o = f_{W0}(q),
//   (ii)  the closed-form state transition of Proposition 1 (carries cw, cm, cb and kernels K^W, K^M),
//   (iii) the per-token gradients G_t(W0, k_t, v_t) - a second-order pass through LN and the activation,
//   (iv)  the suffix scans that made the scalar kernels.
// Notation: T, S = adjoints of the chunk-end (W, M); a trailing "b" marks an adjoint.  "Wl" is the last matrix
// [d x h] (W2 of the GELU MLP, W3 of SwiGLU); the first matrices are [h x d].
//   GELU MLP : hidden a = gelu(z1)                 pz1 = ph gelu'(z1)
//   SwiGLU   : hidden a = silu(z1) z2              pz1 = ph z2 silu'(z1),  pz2 = ph silu(z1)
#include <type_traits>

#include "simt_common.cuh"
#include "simt_layout.h"
#include "tc_gemm.cuh"

namespace e2ttt {

#ifdef SIMT_PROFILE
// Debug build only: cycles thread 0 of CTA 0 spends between consecutive stamps, summed over the chunks of a launch.
__device__ long long g_simt_bwd_prof[32];
#define BPROF(i)                                            \
    do {                                                    \
        if (threadIdx.x == 0 && blockIdx.x == 0) {          \
            const long long now_ = clock64();               \
            g_simt_bwd_prof[i] += now_ - bp_;               \
            bp_ = now_;                                     \
        }                                                   \
    } while (0)
extern "C" __attribute__((visibility("default"))) int e2ttt_debug_read_simt_bwd_profile(long long* host, int reset) {
    const cudaError_t e = cudaMemcpyFromSymbol(host, g_simt_bwd_prof, sizeof(long long) * 32);
    if (reset) {
        long long z[32] = {0};
        cudaMemcpyToSymbol(g_simt_bwd_prof, z, sizeof(z));
    }
    return (int)e;
}
#else
#define BPROF(i)
#endif

template <typename Real> __device__ __forceinline__ Real silu_d2(Real z) {
    const Real s = sigmoid_f(z);
    return s * ((Real)1 - s) * ((Real)2 + z * ((Real)1 - (Real)2 * s));
}

// out = r ( x - mean(x) - y mean(x*y) ) for one row held by one warp (the LN Jacobian is symmetric)
template <typename Real>
__device__ __forceinline__ void warp_ln_jac(const Real* x, const Real* y, Real r, int d, Real* out) {
    const int lane = threadIdx.x & 31;
    Real sx = 0, sxy = 0;
    for (int i = lane; i < d; i += 32) { sx += x[i]; sxy += x[i] * y[i]; }
    sx = warp_sum(sx) / (Real)d;
    sxy = warp_sum(sxy) / (Real)d;
    for (int i = lane; i < d; i += 32) out[i] = r * (x[i] - sx - y[i] * sxy);
}

// TC = true (bf16 I/O only): every GEMM runs on the tensor cores with bf16 operands; everything else is unchanged.
template <typename Real, typename IO, int KIND, bool TC>
__global__ void __launch_bounds__(TC ? kTgThreads : kSimtThreads, 1) simt_bwd_kernel(const SimtBwdArgs a) {
    constexpr int NMAT = (KIND == 0) ? 2 : 3;
    constexpr int LAST = NMAT - 1;
    constexpr bool SW = (KIND == 1);
    using Engine = typename std::conditional<TC, TcGemmT<true>, FmaGemm<Real>>::type;
    constexpr int NT = Engine::kThreads;  // threads per CTA
    extern __shared__ __align__(16) unsigned char simt_smem_raw[];
    unsigned char* smem_base = Engine::align(simt_smem_raw);
    ChunkScalars<Real>& sc = *reinterpret_cast<ChunkScalars<Real>*>(smem_base + Engine::kBytes);
    Real* red = reinterpret_cast<Real*>(smem_base + Engine::kBytes + sizeof(ChunkScalars<Real>));
    Real* rev = red + 16;  // [8][kMaxC] operands and results of the reverse scan

    const int CL = a.cl;                 // CTAs working on this sequence (one cluster)
    const int seq = blockIdx.x / CL, rank = blockIdx.x % CL;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr int NW = NT / 32;
    Engine G;
    G.setup(smem_base, a.status, rank, CL);
    const int d = a.d, h = a.h, C = a.C, L = a.L;
    const size_t dh = (size_t)d * h;
    const SimtLayout& lay = a.lay;
    Real* ws = reinterpret_cast<Real*>(a.ws) + (size_t)seq * lay.per_seq;
    G.set_scratch(ws + lay.splitk);
    const IO* q = reinterpret_cast<const IO*>(a.q) + (size_t)seq * a.Ls * d;
    const IO* k = reinterpret_cast<const IO*>(a.k) + (size_t)seq * a.Ls * d;
    const IO* v = reinterpret_cast<const IO*>(a.v) + (size_t)seq * a.Ls * d;
    const IO* d_o = reinterpret_cast<const IO*>(a.d_o) + (size_t)seq * a.Ls * d;
    IO* dq = reinterpret_cast<IO*>(a.dq) + (size_t)seq * a.Ls * d;
    IO* dk = reinterpret_cast<IO*>(a.dk) + (size_t)seq * a.Ls * d;
    IO* dv = reinterpret_cast<IO*>(a.dv) + (size_t)seq * a.Ls * d;
    const float* eta = a.eta + (size_t)seq * a.Ls;
    const float* beta = a.beta + (size_t)seq * a.Ls;
    const float* gamma = a.gamma + (size_t)seq * a.Ls;
    float* d_eta = a.d_eta + (size_t)seq * a.Ls;
    float* d_beta = a.d_beta + (size_t)seq * a.Ls;
    float* d_gamma = a.d_gamma + (size_t)seq * a.Ls;
    const Real eps = (Real)a.eps;

    Real *T[NMAT], *S[NMAT], *Wb[NMAT];
#pragma unroll
    for (int i = 0; i < NMAT; ++i) {
        T[i] = ws + lay.T[i]; S[i] = ws + lay.S[i]; Wb[i] = ws + lay.Wb[i];
        const float* tf = a.dW_final[i] ? a.dW_final[i] + (size_t)seq * dh : nullptr;
        const float* sf = a.dM_final[i] ? a.dM_final[i] + (size_t)seq * dh : nullptr;
        if (a.carry_in) continue;  // a later segment's launch left them in place
        for (size_t e = tid + (size_t)rank * NT; e < dh; e += (size_t)NT * CL) {
            T[i][e] = tf ? (Real)tf[e] : (Real)0;
            S[i][e] = sf ? (Real)sf[e] : (Real)0;
        }
    }
    Real* Z1 = ws + lay.Z1;    // [2len x h]  pre-activations of matrix 1, key rows then query rows
    Real* Z2 = ws + lay.Z2;    // [2len x h]  SwiGLU: pre-activations of matrix 2
    Real* A = ws + lay.A;      // [2len x h]  hidden activation fed to the last matrix
    Real* U = ws + lay.U;      // [2len x d]  normalised rows y (after the LN step)
    Real* Pu = ws + lay.Pu;    // [len x d]
    Real* Pz1 = ws + lay.Pz1;  // [len x h]
    Real* Pz2 = ws + lay.Pz2;  // [len x h]   SwiGLU
    Real* Pa = ws + lay.Pa;    // [len x h]   ph = dL/d(hidden activation)
    Real* E = ws + lay.E;      // [len x d]
    Real* XY2 = ws + lay.XY2;  // [len x 2d]  (Ak Tl^T | Ak Sl^T)
    Real* XY1 = ws + lay.XY1;  // [len x 2h]  (K T1^T | K S1^T)
    Real* XY1b = ws + lay.XY1b;// [len x 2h]  SwiGLU: (K T2^T | K S2^T)
    Real* Pub = ws + lay.Pub;
    Real* Pzb = ws + lay.Pzb;  // adjoint of pz1; MLP: becomes the adjoint of ph in place
    Real* Pzb2 = ws + lay.Pzb2;
    Real* Zkb = ws + lay.Zkb;  // adjoint of z1 (key rows)
    Real* Zkb2 = ws + lay.Zkb2;
    Real* Akb = ws + lay.Akb;  // adjoint of the hidden activation (key rows)
    Real* Kb = ws + lay.Kb;
    Real* Eb = ws + lay.Eb;
    Real* Ukb = ws + lay.Ukb;
    Real* Uqb = ws + lay.Uqb;
    Real* Zqb = ws + lay.Zqb;
    Real* Zqb2 = ws + lay.Zqb2;
    Real* rk = ws + lay.rk;
    Real* rq = ws + lay.rq;
    Real* kWb_g = ws + lay.kWb;  // adjoints of K^W_t, K^M_t (rows are produced by different CTAs)
    Real* kMb_g = ws + lay.kMb;
    phase_sync(CL);

    for (int c = a.nchunks - 1; c >= 0; --c) {
#ifdef SIMT_PROFILE
        long long bp_ = clock64();
#endif
        const int s = c * C;
        const int len = min(C, L - s);
        const IO* kc = k + (size_t)s * d;
        const IO* qc = q + (size_t)s * d;
        const IO* vc = v + (size_t)s * d;
        const IO* doc = d_o + (size_t)s * d;
        const Real* ck = ws + lay.ckpt + (size_t)c * 2 * NMAT * dh;
        const Real* W1 = ck;                        // [h x d]
        const Real* W2 = ck + dh;                   // SwiGLU: [h x d]
        const Real* Wl = ck + (size_t)LAST * dh;    // [d x h]
        const Real* M0[NMAT];
#pragma unroll
        for (int i = 0; i < NMAT; ++i) M0[i] = ck + (size_t)(NMAT + i) * dh;

        if (warp == 0) chunk_scalars_warp<Real>(eta + s, beta + s, gamma + s, len, &sc);
#pragma unroll
        for (int i = 0; i < NMAT; ++i)
            for (size_t e = tid + (size_t)rank * NT; e < dh; e += (size_t)NT * CL) Wb[i][e] = 0;

        // post-chunk normalisation (optional): T arrives as the adjoint of the normalised chunk-end weights
        // y = n w / (s + eps_n), s = ||w||.  With y itself (the next chunk's saved start state) and the saved s:
        //   w_bar = n/(s + eps_n) y_bar - y <y_bar, y> / (n s),      n_bar = <y_bar, y> / n
        if (a.row_norm[0]) {
            const int maxdim = d > h ? d : h;
            const Real* nxt = ck + (size_t)2 * NMAT * dh;  // state after this chunk: W part
#pragma unroll
            for (int i = 0; i < NMAT; ++i) {
                const int rows = (i == LAST) ? d : h, cols = (i == LAST) ? h : d;
                const float* target = a.row_norm[i] + (size_t)seq * rows;
                float* tb = a.d_row_norm[i] ? a.d_row_norm[i] + (size_t)seq * rows : nullptr;
                for (int r = warp + rank * (NT / 32); r < rows; r += (NT / 32) * CL) {
                    Real* t = T[i] + (size_t)r * cols;
                    const Real* y = nxt + (size_t)i * dh + (size_t)r * cols;
                    Real ty = 0;
                    for (int j = lane; j < cols; j += 32) ty += t[j] * y[j];
                    ty = warp_sum(ty);
                    const Real n = (Real)target[r], nrm = ws[lay.rown + ((size_t)c * 3 + i) * maxdim + r];
                    const Real f = n / (nrm + (Real)a.norm_eps);
                    const Real g = (n != (Real)0 && nrm > (Real)0) ? ty / (n * nrm) : (Real)0;
                    for (int j = lane; j < cols; j += 32) t[j] = f * t[j] - y[j] * g;
                    if (tb && lane == 0) {
                        const Real nb = (n != (Real)0) ? ty / n : (Real)0;
                        tb[r] = (c == a.nchunks - 1) ? (float)nb : tb[r] + (float)nb;
                    }
                }
            }
            phase_sync(CL);
        }

        auto load_x = [&](int m, int kk, Real& a0, Real& a1) {
            a0 = (m < len) ? ld_io<Real>(kc, (size_t)m * d + kk) : ld_io<Real>(qc, (size_t)(m - len) * d + kk);
        };
        auto load_k = [&](int m, int kk, Real& a0, Real& a1) { a0 = ld_io<Real>(kc, (size_t)m * d + kk); };

        BPROF(0);
        // ---------------- forward of the chunk, recomputed ----------------
        BPROF(1);
        G.template run<1, true, true>(
            2 * len, h, d, load_x, [&](int n, int kk) { return W1[(size_t)n * d + kk]; },
            [&](int m, int n, Real acc, Real) {
                Z1[(size_t)m * h + n] = acc;
                if (!SW) A[(size_t)m * h + n] = gelu_f(acc);
            });
        if (SW) {
            G.template run<1, true, true>(
                2 * len, h, d, load_x, [&](int n, int kk) { return W2[(size_t)n * d + kk]; },
                [&](int m, int n, Real acc, Real) {
                    const size_t e = (size_t)m * h + n;
                    Z2[e] = acc;
                    A[e] = silu_f(Z1[e]) * acc;
                });
        }
        BPROF(2);
        G.template run<1, true, true>(
            2 * len, d, h, [&](int m, int kk, Real& a0, Real& a1) { a0 = A[(size_t)m * h + kk]; },
            [&](int n, int kk) { return Wl[(size_t)n * h + kk]; },
            [&](int m, int n, Real acc, Real) { U[(size_t)m * d + n] = acc; });
        BPROF(3);
        for (int m = warp + rank * (NT / 32); m < 2 * len; m += (NT / 32) * CL) {
            Real* u = U + (size_t)m * d;
            const Real r = warp_layernorm(u, u, d, eps);
            if (m >= len) {
                if (lane == 0) rq[m - len] = r;
                // adjoint of the output's LN: Uqb = J_q d_o
                const size_t row = (size_t)(m - len) * d;
                Real sx = 0, sxy = 0;
                for (int i = lane; i < d; i += 32) {
                    const Real x = ld_io<Real>(doc, row + i);
                    sx += x; sxy += x * u[i];
                }
                sx = warp_sum(sx) / (Real)d;
                sxy = warp_sum(sxy) / (Real)d;
                for (int i = lane; i < d; i += 32)
                    Uqb[row + i] = r * (ld_io<Real>(doc, row + i) - sx - u[i] * sxy);
            } else {
                if (lane == 0) rk[m] = r;
                const size_t row = (size_t)m * d;
                for (int i = lane; i < d; i += 32)
                    E[row + i] = ld_io<Real>(kc, row + i) + u[i] - ld_io<Real>(vc, row + i);
                __syncwarp();
                warp_ln_jac(E + row, u, r, d, Pu + row);
            }
        }
        phase_sync(CL);
        BPROF(4);
        G.template run<1, true, false>(
            len, h, d, [&](int m, int kk, Real& a0, Real& a1) { a0 = Pu[(size_t)m * d + kk]; },
            [&](int n, int kk) { return Wl[(size_t)kk * h + n]; },
            [&](int m, int n, Real acc, Real) {
                const size_t e = (size_t)m * h + n;
                Pa[e] = acc;
                if (!SW) {
                    Pz1[e] = acc * gelu_d1(Z1[e]);
                } else {
                    Pz1[e] = acc * Z2[e] * silu_d1(Z1[e]);
                    Pz2[e] = acc * silu_f(Z1[e]);
                }
            });

        BPROF(5);
        // ---------------- (i) outputs o = q + LN(Wl a(q)) ----------------
        const Real* Z1q = Z1 + (size_t)len * h;
        const Real* Z2q = Z2 + (size_t)len * h;
        const Real* Aq = A + (size_t)len * h;
        BPROF(6);
        G.template run<1, true, false>(
            len, h, d, [&](int m, int kk, Real& a0, Real& a1) { a0 = Uqb[(size_t)m * d + kk]; },
            [&](int n, int kk) { return Wl[(size_t)kk * h + n]; },
            [&](int m, int n, Real acc, Real) {
                const size_t e = (size_t)m * h + n;
                if (!SW) {
                    Zqb[e] = acc * gelu_d1(Z1q[e]);
                } else {
                    Zqb[e] = acc * Z2q[e] * silu_d1(Z1q[e]);
                    Zqb2[e] = acc * silu_f(Z1q[e]);
                }
            });
        BPROF(7);
        G.template run<1, true, false>(
            len, d, SW ? 2 * h : h,
            [&](int m, int kk, Real& a0, Real& a1) {
                a0 = kk < h ? Zqb[(size_t)m * h + kk] : Zqb2[(size_t)m * h + kk - h];
            },
            [&](int n, int kk) { return kk < h ? W1[(size_t)kk * d + n] : W2[(size_t)(kk - h) * d + n]; },
            [&](int m, int n, Real acc, Real) {
                const size_t e = (size_t)m * d + n;
                st_io(dq + (size_t)s * d, e, ld_io<Real>(doc, e) + acc);
            });
        BPROF(8);
        G.template run<1, false, false>( // Wbl += Uqb^T Aq
            d, h, len, [&](int m, int t, Real& a0, Real& a1) { a0 = Uqb[(size_t)t * d + m]; },
            [&](int n, int t) { return Aq[(size_t)t * h + n]; },
            [&](int m, int n, Real acc, Real) { Wb[LAST][(size_t)m * h + n] += acc; });
        BPROF(9);
        G.template run<1, false, false>( // Wb1 += Zqb^T Q
            h, d, len, [&](int m, int t, Real& a0, Real& a1) { a0 = Zqb[(size_t)t * h + m]; },
            [&](int n, int t) { return ld_io<Real>(qc, (size_t)t * d + n); },
            [&](int m, int n, Real acc, Real) { Wb[0][(size_t)m * d + n] += acc; });
        BPROF(10);
        if (SW)
            G.template run<1, false, false>( // Wb2 += Zqb2^T Q
                h, d, len, [&](int m, int t, Real& a0, Real& a1) { a0 = Zqb2[(size_t)t * h + m]; },
                [&](int n, int t) { return ld_io<Real>(qc, (size_t)t * d + n); },
                [&](int m, int n, Real acc, Real) { Wb[1][(size_t)m * d + n] += acc; });

        BPROF(11);
        // ---------------- (ii) state transition: carries ----------------
        Real cwb, cmb, cbb;
        {
            Real pw = 0, pm = 0, pb = 0;
#pragma unroll
            for (int i = 0; i < NMAT; ++i) {
                const Real* Wi = ck + (size_t)i * dh;
                for (size_t e = tid + (size_t)rank * NT; e < dh; e += (size_t)NT * CL) {  // this CTA's share
                    pw += T[i][e] * Wi[e];
                    pm += T[i][e] * M0[i][e];
                    pb += S[i][e] * M0[i][e];
                }
            }
            pw = block_sum(pw, red);
            pm = block_sum(pm, red);
            pb = block_sum(pb, red);
            // the shares meet in the workspace; every CTA adds them in rank order: same value everywhere
            Real* shares = ws + lay.red;
            if (tid == 0) { shares[3 * rank] = pw; shares[3 * rank + 1] = pm; shares[3 * rank + 2] = pb; }
            phase_sync(CL);
            cwb = 0; cmb = 0; cbb = 0;
            for (int r = 0; r < CL; ++r) { cwb += shares[3 * r]; cmb += shares[3 * r + 1]; cbb += shares[3 * r + 2]; }
        }
        // G_t enters W_C with K^W_t and M_C with K^M_t: its adjoint is K^W_t T + K^M_t S.
        BPROF(12);
        G.template run<1, true, true>( // XY2 = Ak [Tl; Sl]^T
            len, 2 * d, h, [&](int m, int kk, Real& a0, Real& a1) { a0 = A[(size_t)m * h + kk]; },
            [&](int n, int kk) { return n < d ? T[LAST][(size_t)n * h + kk] : S[LAST][(size_t)(n - d) * h + kk]; },
            [&](int m, int n, Real acc, Real) { XY2[(size_t)m * 2 * d + n] = acc; });
        BPROF(13);
        G.template run<1, true, true>( // XY1 = K [T1; S1]^T
            len, 2 * h, d, load_k,
            [&](int n, int kk) { return n < h ? T[0][(size_t)n * d + kk] : S[0][(size_t)(n - h) * d + kk]; },
            [&](int m, int n, Real acc, Real) { XY1[(size_t)m * 2 * h + n] = acc; });
        BPROF(14);
        if (SW)
            G.template run<1, true, true>( // XY1b = K [T2; S2]^T
                len, 2 * h, d, load_k,
                [&](int n, int kk) { return n < h ? T[1][(size_t)n * d + kk] : S[1][(size_t)(n - h) * d + kk]; },
                [&](int m, int n, Real acc, Real) { XY1b[(size_t)m * 2 * h + n] = acc; });
        BPROF(15);
        for (int t = warp + rank * (NT / 32); t < len; t += (NT / 32) * CL) {
            const Real* x2 = XY2 + (size_t)t * 2 * d;
            const Real* x1 = XY1 + (size_t)t * 2 * h;
            const Real* x1b = XY1b + (size_t)t * 2 * h;
            Real sw = 0, sm = 0;
            for (int i = lane; i < d; i += 32) {
                const Real p = Pu[(size_t)t * d + i];
                sw += p * x2[i]; sm += p * x2[d + i];
            }
            for (int j = lane; j < h; j += 32) {
                const Real p = Pz1[(size_t)t * h + j];
                sw += p * x1[j]; sm += p * x1[h + j];
                if (SW) {
                    const Real p2 = Pz2[(size_t)t * h + j];
                    sw += p2 * x1b[j]; sm += p2 * x1b[h + j];
                }
            }
            sw = warp_sum(sw); sm = warp_sum(sm);
            if (lane == 0) { kWb_g[t] = -sw; kMb_g[t] = -sm; }
            const Real kw = sc.kW[t], km = sc.kM[t];
            for (int i = lane; i < d; i += 32) Pub[(size_t)t * d + i] = -(kw * x2[i] + km * x2[d + i]);
            for (int j = lane; j < h; j += 32) {
                Pzb[(size_t)t * h + j] = -(kw * x1[j] + km * x1[h + j]);
                if (SW) Pzb2[(size_t)t * h + j] = -(kw * x1b[j] + km * x1b[h + j]);
            }
        }
        phase_sync(CL);
        BPROF(16);
        // ---------------- (iii) per-token gradients G_t = -(pz1 k^T, [pz2 k^T,] pu a^T) ----------------
        BPROF(17);
        G.template run<1, true, false>( // Akb = -[kW Pu | kM Pu] [Tl; Sl]
            len, h, 2 * d,
            [&](int m, int kk, Real& a0, Real& a1) {
                a0 = kk < d ? sc.kW[m] * Pu[(size_t)m * d + kk] : sc.kM[m] * Pu[(size_t)m * d + kk - d];
            },
            [&](int n, int kk) { return kk < d ? T[LAST][(size_t)kk * h + n] : S[LAST][(size_t)(kk - d) * h + n]; },
            [&](int m, int n, Real acc, Real) { Akb[(size_t)m * h + n] = -acc; });
        BPROF(18);
        G.template run<1, true, false>( // Kb = -[kW Pz1 | kM Pz1] [T1; S1]
            len, d, 2 * h,
            [&](int m, int kk, Real& a0, Real& a1) {
                a0 = kk < h ? sc.kW[m] * Pz1[(size_t)m * h + kk] : sc.kM[m] * Pz1[(size_t)m * h + kk - h];
            },
            [&](int n, int kk) { return kk < h ? T[0][(size_t)kk * d + n] : S[0][(size_t)(kk - h) * d + n]; },
            [&](int m, int n, Real acc, Real) { Kb[(size_t)m * d + n] = -acc; });
        BPROF(19);
        if (SW)
            G.template run<1, true, false>( // Kb -= [kW Pz2 | kM Pz2] [T2; S2]
                len, d, 2 * h,
                [&](int m, int kk, Real& a0, Real& a1) {
                    a0 = kk < h ? sc.kW[m] * Pz2[(size_t)m * h + kk] : sc.kM[m] * Pz2[(size_t)m * h + kk - h];
                },
                [&](int n, int kk) { return kk < h ? T[1][(size_t)kk * d + n] : S[1][(size_t)(kk - h) * d + n]; },
                [&](int m, int n, Real acc, Real) { Kb[(size_t)m * d + n] -= acc; });
        // back through pz: Pzb becomes the adjoint of ph; Zkb (Zkb2) start with the second-order terms
        BPROF(20);
        for (size_t e = tid + (size_t)rank * NT; e < (size_t)len * h; e += (size_t)NT * CL) {
            const Real z1 = Z1[e], ph = Pa[e];
            if (!SW) {
                const Real pzb = Pzb[e];
                Zkb[e] = pzb * ph * gelu_d2(z1);
                Pzb[e] = pzb * gelu_d1(z1);
            } else {
                const Real b1 = Pzb[e], b2 = Pzb2[e], z2 = Z2[e], g1 = silu_d1(z1);
                Pzb[e] = b1 * z2 * g1 + b2 * silu_f(z1);
                Zkb2[e] = b1 * ph * g1;
                Zkb[e] = b1 * ph * z2 * silu_d2(z1) + b2 * ph * g1;
            }
        }
        phase_sync(CL);
        const Real* Phb = Pzb;
        // ph = Wl^T pu
        BPROF(21);
        G.template run<1, true, true>(
            len, d, h, [&](int m, int kk, Real& a0, Real& a1) { a0 = Phb[(size_t)m * h + kk]; },
            [&](int n, int kk) { return Wl[(size_t)n * h + kk]; },
            [&](int m, int n, Real acc, Real) { Pub[(size_t)m * d + n] += acc; });
        BPROF(22);
        G.template run<1, false, false>( // Wbl += Pu^T Phb
            d, h, len, [&](int m, int t, Real& a0, Real& a1) { a0 = Pu[(size_t)t * d + m]; },
            [&](int n, int t) { return Phb[(size_t)t * h + n]; },
            [&](int m, int n, Real acc, Real) { Wb[LAST][(size_t)m * h + n] += acc; });
        // pu = J(u) e, e = k + y - v, y = LN(u)
        BPROF(23);
        for (int t = warp + rank * (NT / 32); t < len; t += (NT / 32) * CL) {
            const size_t row = (size_t)t * d;
            const Real* y = U + row;
            const Real r = rk[t];
            warp_ln_jac(Pub + row, y, r, d, Eb + row);
            __syncwarp();
            Real spp = 0, mpy = 0, mey = 0;
            for (int i = lane; i < d; i += 32) {
                spp += Pub[row + i] * Pu[row + i];
                mpy += Pub[row + i] * y[i];
                mey += E[row + i] * y[i];
            }
            spp = warp_sum(spp);
            mpy = warp_sum(mpy) / (Real)d;
            mey = warp_sum(mey) / (Real)d;
            // second-order term of the LN Jacobian, then dy -> du for the y inside e
            warp_ln_jac(Eb + row, y, r, d, Ukb + row);
            __syncwarp();
            for (int i = lane; i < d; i += 32) {
                Ukb[row + i] += -(r / (Real)d) * spp * y[i] - r * (mpy * Pu[row + i] + mey * Eb[row + i]);
                Kb[row + i] += Eb[row + i];
                st_io(dv + (size_t)s * d, row + i, -Eb[row + i]);
            }
        }
        phase_sync(CL);
        // u = Wl a ; a = gelu(z1)  or  silu(z1) z2
        BPROF(24);
        G.template run<1, true, false>(
            len, h, d, [&](int m, int kk, Real& a0, Real& a1) { a0 = Ukb[(size_t)m * d + kk]; },
            [&](int n, int kk) { return Wl[(size_t)kk * h + n]; },
            [&](int m, int n, Real acc, Real) {
                const size_t e = (size_t)m * h + n;
                const Real ab = Akb[e] + acc;
                if (!SW) {
                    Zkb[e] += ab * gelu_d1(Z1[e]);
                } else {
                    Zkb[e] += ab * Z2[e] * silu_d1(Z1[e]);
                    Zkb2[e] += ab * silu_f(Z1[e]);
                }
            });
        BPROF(25);
        G.template run<1, false, false>( // Wbl += Ukb^T Ak
            d, h, len, [&](int m, int t, Real& a0, Real& a1) { a0 = Ukb[(size_t)t * d + m]; },
            [&](int n, int t) { return A[(size_t)t * h + n]; },
            [&](int m, int n, Real acc, Real) { Wb[LAST][(size_t)m * h + n] += acc; });
        // z1 = W1 k (, z2 = W2 k)
        BPROF(26);
        G.template run<1, true, false>(
            len, d, SW ? 2 * h : h,
            [&](int m, int kk, Real& a0, Real& a1) {
                a0 = kk < h ? Zkb[(size_t)m * h + kk] : Zkb2[(size_t)m * h + kk - h];
            },
            [&](int n, int kk) { return kk < h ? W1[(size_t)kk * d + n] : W2[(size_t)(kk - h) * d + n]; },
            [&](int m, int n, Real acc, Real) {
                const size_t e = (size_t)m * d + n;
                st_io(dk + (size_t)s * d, e, Kb[e] + acc);
            });
        BPROF(27);
        G.template run<1, false, false>( // Wb1 += Zkb^T K
            h, d, len, [&](int m, int t, Real& a0, Real& a1) { a0 = Zkb[(size_t)t * h + m]; },
            [&](int n, int t) { return ld_io<Real>(kc, (size_t)t * d + n); },
            [&](int m, int n, Real acc, Real) { Wb[0][(size_t)m * d + n] += acc; });
        BPROF(28);
        if (SW)
            G.template run<1, false, false>( // Wb2 += Zkb2^T K
                h, d, len, [&](int m, int t, Real& a0, Real& a1) { a0 = Zkb2[(size_t)t * h + m]; },
                [&](int n, int t) { return ld_io<Real>(kc, (size_t)t * d + n); },
                [&](int m, int n, Real acc, Real) { Wb[1][(size_t)m * d + n] += acc; });

        BPROF(29);
        // ---------------- adjoints of the chunk-start state ----------------
        {
            const Real cw = sc.cw, cm = sc.cm, cb = sc.cb;
#pragma unroll
            for (int i = 0; i < NMAT; ++i)
                for (size_t e = tid + (size_t)rank * NT; e < dh; e += (size_t)NT * CL) {
                    const Real t = T[i][e], sv = S[i][e];
                    T[i][e] = cw * t + Wb[i][e];
                    S[i][e] = cm * t + cb * sv;
                }
        }
        BPROF(30);
        // ---------------- (iv) reverse of the suffix scans ----------------
        // One thread walks the chunk (a 3-term linear recurrence, ~10 flop per token); its operands are brought into
        // shared memory by the whole CTA first and its results leave the same way, so the walk itself never waits
        // for global memory.
        if (rank == 0) {
            Real* r_beta = rev, *r_gamma = rev + kMaxC, *r_eta = rev + 2 * kMaxC, *r_kWb = rev + 3 * kMaxC,
                 *r_kMb = rev + 4 * kMaxC, *r_de = rev + 5 * kMaxC, *r_db = rev + 6 * kMaxC, *r_dg = rev + 7 * kMaxC;
            for (int t = tid; t < len; t += NT) {
                r_beta[t] = (Real)beta[s + t];
                r_gamma[t] = (Real)gamma[s + t];
                r_eta[t] = (Real)eta[s + t];
                r_kWb[t] = kWb_g[t];
                r_kMb[t] = kMb_g[t];
            }
            __syncthreads();
            if (tid == 0) {
                Real Sb = 0, btb = cbb, gtb = cwb; // adjoints of S_0 (unused), bt_0, gt_0
                for (int t = 0; t < len; ++t) {
                    // index t: state t; token t+1 lives at array index t
                    const Real b1 = r_beta[t], g1 = r_gamma[t], e1 = r_eta[t];
                    const Real kWb = r_kWb[t], kMb = r_kMb[t];
                    // S_t = beta_{t+1} S_{t+1} + gt_t ; bt_t = beta_{t+1} bt_{t+1} ; gt_t = gamma_{t+1} gt_{t+1}
                    gtb += Sb;
                    Real bb = Sb * sc.S[t + 1] + btb * sc.bt[t + 1];
                    Real Sb_next = Sb * b1;
                    Real btb_next = btb * b1;
                    const Real gb = gtb * sc.gt[t + 1];
                    Real gtb_next = gtb * g1;
                    if (t == 0) { // cm = beta_1 S_1
                        bb += cmb * sc.S[1];
                        Sb_next += cmb * b1;
                    }
                    // K^M_{t+1} = eta bt_{t+1}, K^W_{t+1} = eta S_{t+1}
                    r_de[t] = kMb * sc.bt[t + 1] + kWb * sc.S[t + 1];
                    btb_next += kMb * e1;
                    Sb_next += kWb * e1;
                    r_db[t] = bb;
                    r_dg[t] = gb;
                    Sb = Sb_next; btb = btb_next; gtb = gtb_next;
                }
            }
            __syncthreads();
            for (int t = tid; t < len; t += NT) {
                d_eta[s + t] = (float)r_de[t];
                d_beta[s + t] = (float)r_db[t];
                d_gamma[s + t] = (float)r_dg[t];
            }
        }
        phase_sync(CL);
    }

#pragma unroll
    for (int i = 0; i < NMAT; ++i) {
        if (a.carry_out) break;  // the launch for the segment before this one picks T, S up from the workspace
        float* wf = a.dW_init[i] + (size_t)seq * dh;
        float* mf = a.dM_init[i] + (size_t)seq * dh;
        for (size_t e = tid + (size_t)rank * NT; e < dh; e += (size_t)NT * CL) {
            wf[e] = (float)T[i][e];
            mf[e] = (float)S[i][e];
        }
    }
    G.teardown();
}

template <typename Real, typename IO, int KIND, bool TC>
static int launch_bwd(const SimtBwdArgs& a, cudaStream_t st) {
    using Engine = typename std::conditional<TC, TcGemmT<true>, FmaGemm<Real>>::type;
    constexpr size_t smem = Engine::kBytes + sizeof(ChunkScalars<Real>) + (16 + 8 * kMaxC) * sizeof(Real) + (TC ? 1024 : 0);
    static bool attr_done[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return (int)cudaGetLastError();
    if (dev < 0 || dev >= 64 || !attr_done[dev]) {
        cudaError_t e =
            cudaFuncSetAttribute(simt_bwd_kernel<Real, IO, KIND, TC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return (int)e;
        if (dev >= 0 && dev < 64) attr_done[dev] = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(a.N * a.cl));
    cfg.blockDim = dim3(Engine::kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)a.cl;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, simt_bwd_kernel<Real, IO, KIND, TC>, a);
    if (e != cudaSuccess) return (int)e;
    return (int)cudaGetLastError();
}

int simt_bwd_launch(const SimtBwdArgs& a, int kind, int io_dtype, void* stream) {
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (io_dtype == 0)
        return kind == 0 ? launch_bwd<double, float, 0, false>(a, st) : launch_bwd<double, float, 1, false>(a, st);
    if (a.tc)
        return kind == 0 ? launch_bwd<float, __nv_bfloat16, 0, true>(a, st) : launch_bwd<float, __nv_bfloat16, 1, true>(a, st);
    return kind == 0 ? launch_bwd<float, __nv_bfloat16, 0, false>(a, st) : launch_bwd<float, __nv_bfloat16, 1, false>(a, st);
}

}  // namespace e2ttt
