// Any-shape forward: Algorithm 1 applied chunk after chunk for any d, h, C and both networks.  A cluster of 1-8 CTAs
// works on one sequence; the CTAs split every phase and share state and intermediates through the workspace, meeting
// at the cluster barrier between phases.  The matrix products run on one of two engines (tc_gemm.cuh): CUDA-core FMAs
// (fp64 for fp32 I/O - the GPU-side reference of the tensor-core paths - or fp32), or tcgen05 MMAs for bf16 I/O.
#include <type_traits>

#include "simt_common.cuh"
#include "simt_layout.h"
#include "tc_gemm.cuh"

namespace e2ttt {

#ifdef SIMT_PROFILE
// Debug build only: cycle stamps of thread 0 of CTA 0 at the phase boundaries of the first 32 chunks.
__device__ long long g_simt_fwd_prof[32 * 16];
#define SPROF(i)                                                                                      \
    do {                                                                                              \
        if (threadIdx.x == 0 && blockIdx.x == 0 && c < 32) g_simt_fwd_prof[c * 16 + (i)] = clock64(); \
    } while (0)
extern "C" __attribute__((visibility("default"))) int e2ttt_debug_read_simt_fwd_profile(long long* host, int n) {
    return (int)cudaMemcpyFromSymbol(host, g_simt_fwd_prof, sizeof(long long) * (size_t)n);
}
extern "C" __attribute__((visibility("default"))) int e2ttt_debug_read_gemm_profile(long long* host, int reset) {
    const cudaError_t e = cudaMemcpyFromSymbol(host, g_tg_prof, sizeof(long long) * 16);
    if (reset) {
        long long z[16] = {0};
        cudaMemcpyToSymbol(g_tg_prof, z, sizeof(z));
    }
    return (int)e;
}
#else
#define SPROF(i)
#endif

// TC = true (bf16 I/O only): every GEMM runs on the tensor cores with bf16 operands; everything else is unchanged.
template <typename Real, typename IO, int KIND, bool TC>
__global__ void __launch_bounds__(TC ? kTgThreads : kSimtThreads, 1) simt_fwd_kernel(const SimtFwdArgs a) {
    constexpr int NMAT = (KIND == 0) ? 2 : 3;
    constexpr int LAST = NMAT - 1;
    using Engine = typename std::conditional<TC, TcGemmT<false>, FmaGemm<Real>>::type;
    constexpr int NT = Engine::kThreads;  // threads per CTA
    extern __shared__ __align__(16) unsigned char simt_smem_raw[];
    unsigned char* smem_base = Engine::align(simt_smem_raw);
    ChunkScalars<Real>& sc = *reinterpret_cast<ChunkScalars<Real>*>(smem_base + Engine::kBytes);

    const int CL = a.cl;                 // CTAs working on this sequence (one cluster)
    const int seq = blockIdx.x / CL, rank = blockIdx.x % CL;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
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
    IO* o = reinterpret_cast<IO*>(a.o) + (size_t)seq * a.Ls * d;
    const float* eta = a.eta + (size_t)seq * a.Ls;
    const float* beta = a.beta + (size_t)seq * a.Ls;
    const float* gamma = a.gamma + (size_t)seq * a.Ls;
    const Real eps = (Real)a.eps;

    Real* W[NMAT];
    Real* M[NMAT];
#pragma unroll
    for (int i = 0; i < NMAT; ++i) {
        W[i] = ws + lay.W[i];
        M[i] = ws + lay.M[i];
        struct WM { Real w, m; };
        if (a.init_slot >= 0) {  // a segment of the backward's recomputation: start from a checkpoint
            const Real* ck = ws + lay.cck + (size_t)a.init_slot * 2 * NMAT * dh;
            batched_for<8>(tid + (size_t)rank * NT, dh, (size_t)NT * CL,
                           [&](size_t e) { return WM{ck[(size_t)i * dh + e], ck[(size_t)(NMAT + i) * dh + e]}; },
                           [&](size_t e, const WM& x) { W[i][e] = x.w; M[i][e] = x.m; });
        } else {
            const float* wi = a.W_init[i] + (size_t)seq * dh;
            const float* mi = a.M_init[i] ? a.M_init[i] + (size_t)seq * dh : nullptr;
            batched_for<8>(tid + (size_t)rank * NT, dh, (size_t)NT * CL,
                           [&](size_t e) { return WM{(Real)wi[e], mi ? (Real)mi[e] : (Real)0}; },
                           [&](size_t e, const WM& x) { W[i][e] = x.w; M[i][e] = x.m; });
        }
    }
    Real* Z1 = ws + lay.Z1;
    Real* Z2 = ws + lay.Z2;
    Real* A = ws + lay.A;
    Real* U = ws + lay.U;
    Real* Pu = ws + lay.Pu;
    Real* Pz1 = ws + lay.Pz1;
    Real* Pz2 = ws + lay.Pz2;
    phase_sync(CL);

    for (int c = 0; c < a.nchunks; ++c) {
        const int s = c * C;
        const int len = min(C, L - s);
        const IO* kc = k + (size_t)s * d;
        const IO* qc = q + (size_t)s * d;
        const IO* vc = v + (size_t)s * d;

        SPROF(0);
        // Algorithm 1 line 2: scalar kernels and carries
        if (warp == 0) chunk_scalars_warp<Real>(eta + s, beta + s, gamma + s, len, &sc);
        if (a.save_states == 1 || (a.save_states == 2 && c % lay.seg == 0)) {
            Real* ck = a.save_states == 1 ? ws + lay.ckpt + (size_t)c * 2 * NMAT * dh
                                          : ws + lay.cck + (size_t)(c / lay.seg) * 2 * NMAT * dh;
#pragma unroll
            for (int i = 0; i < NMAT; ++i) {
                struct WM { Real w, m; };
                batched_for<8>(tid + (size_t)rank * NT, dh, (size_t)NT * CL,
                               [&](size_t e) { return WM{W[i][e], M[i][e]}; },
                               [&](size_t e, const WM& x) {
                                   ck[(size_t)i * dh + e] = x.w;
                                   ck[(size_t)(NMAT + i) * dh + e] = x.m;
                               });
            }
        }

        SPROF(1);
        // Algorithm 1 line 1: the network on the chunk's keys (rows 0..len-1) and queries (rows len..2len-1)
        auto load_x = [&](int m, int kk, Real& a0, Real& a1) {
            a0 = (m < len) ? ld_io<Real>(kc, (size_t)m * d + kk) : ld_io<Real>(qc, (size_t)(m - len) * d + kk);
        };
        G.template run<1, true, true>(
            2 * len, h, d, load_x, [&](int n, int kk) { return W[0][(size_t)n * d + kk]; },
            [&](int m, int n, Real acc, Real) { Z1[(size_t)m * h + n] = acc; });
        SPROF(2);
        if (KIND == 1)
            G.template run<1, true, true>(
                2 * len, h, d, load_x, [&](int n, int kk) { return W[1][(size_t)n * d + kk]; },
                [&](int m, int n, Real acc, Real) { Z2[(size_t)m * h + n] = acc; });
        SPROF(3);
        struct ZZ { Real z1, z2; };
        batched_for<8>(tid + (size_t)rank * NT, (size_t)2 * len * h, (size_t)NT * CL,
                       [&](size_t e) { return ZZ{Z1[e], KIND == 0 ? (Real)0 : Z2[e]}; },
                       [&](size_t e, const ZZ& z) { A[e] = (KIND == 0) ? gelu_f(z.z1) : silu_f(z.z1) * z.z2; });
        phase_sync(CL);
        SPROF(4);
        G.template run<1, true, true>(
            2 * len, d, h, [&](int m, int kk, Real& a0, Real& a1) { a0 = A[(size_t)m * h + kk]; },
            [&](int n, int kk) { return W[LAST][(size_t)n * h + kk]; },
            [&](int m, int n, Real acc, Real) { U[(size_t)m * d + n] = acc; });

        SPROF(5);
        // layer norm; outputs for the query rows; e = f(k) - v and pu = dL/du for the key rows (Algorithm 1 line 3)
        for (int m = warp + rank * (NT / 32); m < 2 * len; m += (NT / 32) * CL) {
            Real* u = U + (size_t)m * d;
            const Real r = warp_layernorm(u, u, d, eps);
            if (m >= len) {
                const size_t row = (size_t)(m - len) * d;
                if (a.o)
                    for (int i = lane; i < d; i += 32)
                        st_io(o + (size_t)s * d, row + i, ld_io<Real>(qc, row + i) + u[i]);
            } else {
                const size_t row = (size_t)m * d;
                Real se = 0, sey = 0;
                for (int i = lane; i < d; i += 32) {
                    const Real e = ld_io<Real>(kc, row + i) + u[i] - ld_io<Real>(vc, row + i);
                    se += e;
                    sey += e * u[i];
                }
                se = warp_sum(se) / (Real)d;
                sey = warp_sum(sey) / (Real)d;
                for (int i = lane; i < d; i += 32) {
                    const Real e = ld_io<Real>(kc, row + i) + u[i] - ld_io<Real>(vc, row + i);
                    Pu[row + i] = r * (e - se - u[i] * sey);
                }
            }
        }
        phase_sync(CL);

        SPROF(6);
        // back through the last matrix and the activation
        G.template run_rmw<1, true, false>(
            len, h, d, [&](int m, int kk, Real& a0, Real& a1) { a0 = Pu[(size_t)m * d + kk]; },
            [&](int n, int kk) { return W[LAST][(size_t)kk * h + n]; },
            [&](int m, int n) {
                const size_t e = (size_t)m * h + n;
                return ZZ{Z1[e], KIND == 0 ? (Real)0 : Z2[e]};
            },
            [&](int m, int n, Real acc, Real, const ZZ& z) {
                const size_t e = (size_t)m * h + n;
                if (KIND == 0) {
                    Pz1[e] = acc * gelu_d1(z.z1);
                } else {
                    Pz1[e] = acc * z.z2 * silu_d1(z.z1);
                    Pz2[e] = acc * silu_f(z.z1);
                }
            });

        SPROF(7);
        // Algorithm 1 lines 4-7: both weighted aggregations of every matrix, fused with the state transition
        const Real cw = sc.cw, cm = sc.cm, cb = sc.cb;
        auto update = [&](Real* Wm, Real* Mm, int rows, int cols, const Real* P, auto load_xcol) {
            G.template run_rmw<2, false, false>(
                rows, cols, len,
                [&](int m, int t, Real& a0, Real& a1) {
                    const Real p = P[(size_t)t * rows + m];
                    a0 = sc.kW[t] * p;
                    a1 = sc.kM[t] * p;
                },
                load_xcol,
                [&](int m, int n) {
                    const size_t e = (size_t)m * cols + n;
                    return ZZ{Wm[e], Mm[e]};
                },
                [&](int m, int n, Real aW, Real aM, const ZZ& wm) {
                    const size_t e = (size_t)m * cols + n;
                    Wm[e] = cw * wm.z1 + cm * wm.z2 - aW; // G_t = -grad: the aggregations enter with a minus sign
                    Mm[e] = cb * wm.z2 - aM;
                });
        };
        auto key_col = [&](int n, int t) { return ld_io<Real>(kc, (size_t)t * d + n); };
        auto act_col = [&](int n, int t) { return A[(size_t)t * h + n]; };
        update(W[0], M[0], h, d, Pz1, key_col);
        SPROF(8);
        if (KIND == 1) update(W[1], M[1], h, d, Pz2, key_col);
        SPROF(9);
        update(W[LAST], M[LAST], d, h, Pu, act_col);
        SPROF(10);

        // post-chunk normalisation (optional): every row w of every W_i becomes n w / (||w|| + eps_n); one warp per row
        if (a.row_norm[0]) {
            const int maxdim = d > h ? d : h;
#pragma unroll
            for (int i = 0; i < NMAT; ++i) {
                const int rows = (i == LAST) ? d : h, cols = (i == LAST) ? h : d;
                const float* target = a.row_norm[i] + (size_t)seq * rows;
                for (int r = warp + rank * (NT / 32); r < rows; r += (NT / 32) * CL) {
                    Real* w = W[i] + (size_t)r * cols;
                    Real ss = 0;
                    for (int j = lane; j < cols; j += 32) ss += w[j] * w[j];
                    const Real nrm = sqrt(warp_sum(ss));
                    const Real f = (Real)target[r] / (nrm + (Real)a.norm_eps);
                    for (int j = lane; j < cols; j += 32) w[j] *= f;
                    if (a.save_states && lane == 0) ws[lay.rown + ((size_t)c * 3 + i) * maxdim + r] = nrm;
                }
            }
            phase_sync(CL);
        }
    }
    if (a.save_states && a.row_norm[0]) {  // the reverse pass needs the normalised end state of the last chunk too
        Real* ck = ws + lay.ckpt + (size_t)a.nchunks * 2 * NMAT * dh;
#pragma unroll
        for (int i = 0; i < NMAT; ++i) {
            struct WM { Real w, m; };
            batched_for<8>(tid + (size_t)rank * NT, dh, (size_t)NT * CL,
                           [&](size_t e) { return WM{W[i][e], M[i][e]}; },
                           [&](size_t e, const WM& x) {
                               ck[(size_t)i * dh + e] = x.w;
                               ck[(size_t)(NMAT + i) * dh + e] = x.m;
                           });
        }
    }

#pragma unroll
    for (int i = 0; i < NMAT; ++i) {
        if (!a.W_final[i]) continue; // state-recompute run of the backward: only the saved chunk states matter
        float* wf = a.W_final[i] + (size_t)seq * dh;
        float* mf = a.M_final[i] + (size_t)seq * dh;
        struct WM { Real w, m; };
        batched_for<8>(tid + (size_t)rank * NT, dh, (size_t)NT * CL,
                       [&](size_t e) { return WM{W[i][e], M[i][e]}; },
                       [&](size_t e, const WM& x) { wf[e] = (float)x.w; mf[e] = (float)x.m; });
    }
    G.teardown();
}

template <typename Real, typename IO, int KIND, bool TC>
static int launch_fwd(const SimtFwdArgs& a, cudaStream_t st) {
    using Engine = typename std::conditional<TC, TcGemmT<false>, FmaGemm<Real>>::type;
    constexpr size_t smem = Engine::kBytes + sizeof(ChunkScalars<Real>) + (TC ? 1024 : 0);
    static bool attr_done[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return (int)cudaGetLastError();
    if (dev < 0 || dev >= 64 || !attr_done[dev]) {
        cudaError_t e = cudaFuncSetAttribute(simt_fwd_kernel<Real, IO, KIND, TC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
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
    cudaError_t e = cudaLaunchKernelEx(&cfg, simt_fwd_kernel<Real, IO, KIND, TC>, a);
    if (e != cudaSuccess) return (int)e;
    return (int)cudaGetLastError();
}

int simt_fwd_launch(const SimtFwdArgs& a, int kind, int io_dtype, void* stream) {
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (io_dtype == 0)
        return kind == 0 ? launch_fwd<double, float, 0, false>(a, st) : launch_fwd<double, float, 1, false>(a, st);
    if (a.tc)
        return kind == 0 ? launch_fwd<float, __nv_bfloat16, 0, true>(a, st) : launch_fwd<float, __nv_bfloat16, 1, true>(a, st);
    return kind == 0 ? launch_fwd<float, __nv_bfloat16, 0, false>(a, st) : launch_fwd<float, __nv_bfloat16, 1, false>(a, st);
}

}  // namespace e2ttt
