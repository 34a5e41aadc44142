// SIMT forward: Algorithm 1 applied chunk after chunk, one CTA per sequence, for any shape.
// The fp32-I/O instantiation computes in fp64 and is the GPU-side reference for the tensor-core path.
#include "simt_common.cuh"
#include "simt_layout.h"

namespace e2ttt {

template <typename Real, typename IO, int KIND>
__global__ void __launch_bounds__(kSimtThreads) simt_fwd_kernel(const SimtFwdArgs a) {
    constexpr int NMAT = (KIND == 0) ? 2 : 3;
    constexpr int LAST = NMAT - 1;
    extern __shared__ __align__(16) unsigned char simt_smem_raw[];
    GemmSmem<Real>& gsm = *reinterpret_cast<GemmSmem<Real>*>(simt_smem_raw);
    ChunkScalars<Real>& sc = *reinterpret_cast<ChunkScalars<Real>*>(simt_smem_raw + sizeof(GemmSmem<Real>));

    const int CL = a.cl;                 // CTAs working on this sequence (one cluster)
    const int seq = blockIdx.x / CL, rank = blockIdx.x % CL;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int d = a.d, h = a.h, C = a.C, L = a.L;
    const size_t dh = (size_t)d * h;
    const SimtLayout& lay = a.lay;
    Real* ws = reinterpret_cast<Real*>(a.ws) + (size_t)seq * lay.per_seq;
    const IO* q = reinterpret_cast<const IO*>(a.q) + (size_t)seq * L * d;
    const IO* k = reinterpret_cast<const IO*>(a.k) + (size_t)seq * L * d;
    const IO* v = reinterpret_cast<const IO*>(a.v) + (size_t)seq * L * d;
    IO* o = reinterpret_cast<IO*>(a.o) + (size_t)seq * L * d;
    const float* eta = a.eta + (size_t)seq * L;
    const float* beta = a.beta + (size_t)seq * L;
    const float* gamma = a.gamma + (size_t)seq * L;
    const Real eps = (Real)a.eps;

    Real* W[NMAT];
    Real* M[NMAT];
#pragma unroll
    for (int i = 0; i < NMAT; ++i) {
        W[i] = ws + lay.W[i];
        M[i] = ws + lay.M[i];
        const float* wi = a.W_init[i] + (size_t)seq * dh;
        const float* mi = a.M_init[i] ? a.M_init[i] + (size_t)seq * dh : nullptr;
        for (size_t e = tid + (size_t)rank * kSimtThreads; e < dh; e += (size_t)kSimtThreads * CL) {
            W[i][e] = (Real)wi[e];
            M[i][e] = mi ? (Real)mi[e] : (Real)0;
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

        // Algorithm 1 line 2: scalar kernels and carries
        if (warp == 0) chunk_scalars_warp<Real>(eta + s, beta + s, gamma + s, len, &sc);
        if (a.save_states) {
            Real* ck = ws + lay.ckpt + (size_t)c * 2 * NMAT * dh;
#pragma unroll
            for (int i = 0; i < NMAT; ++i)
                for (size_t e = tid + (size_t)rank * kSimtThreads; e < dh; e += (size_t)kSimtThreads * CL) {
                    ck[(size_t)i * dh + e] = W[i][e];
                    ck[(size_t)(NMAT + i) * dh + e] = M[i][e];
                }
        }

        // Algorithm 1 line 1: the network on the chunk's keys (rows 0..len-1) and queries (rows len..2len-1)
        auto load_x = [&](int m, int kk, Real& a0, Real& a1) {
            a0 = (m < len) ? ld_io<Real>(kc, (size_t)m * d + kk) : ld_io<Real>(qc, (size_t)(m - len) * d + kk);
        };
        block_gemm<Real, 1, true, true>(
            2 * len, h, d, load_x, [&](int n, int kk) { return W[0][(size_t)n * d + kk]; },
            [&](int m, int n, Real acc, Real) { Z1[(size_t)m * h + n] = acc; }, &gsm, rank, CL);
        if (KIND == 1)
            block_gemm<Real, 1, true, true>(
                2 * len, h, d, load_x, [&](int n, int kk) { return W[1][(size_t)n * d + kk]; },
                [&](int m, int n, Real acc, Real) { Z2[(size_t)m * h + n] = acc; }, &gsm, rank, CL);
        for (size_t e = tid + (size_t)rank * kSimtThreads; e < (size_t)2 * len * h; e += (size_t)kSimtThreads * CL)
            A[e] = (KIND == 0) ? gelu_f(Z1[e]) : silu_f(Z1[e]) * Z2[e];
        phase_sync(CL);
        block_gemm<Real, 1, true, true>(
            2 * len, d, h, [&](int m, int kk, Real& a0, Real& a1) { a0 = A[(size_t)m * h + kk]; },
            [&](int n, int kk) { return W[LAST][(size_t)n * h + kk]; },
            [&](int m, int n, Real acc, Real) { U[(size_t)m * d + n] = acc; }, &gsm, rank, CL);

        // layer norm; outputs for the query rows; e = f(k) - v and pu = dL/du for the key rows (Algorithm 1 line 3)
        for (int m = warp + rank * (kSimtThreads / 32); m < 2 * len; m += (kSimtThreads / 32) * CL) {
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

        // back through the last matrix and the activation
        block_gemm<Real, 1, true, false>(
            len, h, d, [&](int m, int kk, Real& a0, Real& a1) { a0 = Pu[(size_t)m * d + kk]; },
            [&](int n, int kk) { return W[LAST][(size_t)kk * h + n]; },
            [&](int m, int n, Real acc, Real) {
                const size_t e = (size_t)m * h + n;
                if (KIND == 0) {
                    Pz1[e] = acc * gelu_d1(Z1[e]);
                } else {
                    Pz1[e] = acc * Z2[e] * silu_d1(Z1[e]);
                    Pz2[e] = acc * silu_f(Z1[e]);
                }
            },
            &gsm, rank, CL);

        // Algorithm 1 lines 4-7: both weighted aggregations of every matrix, fused with the state transition
        const Real cw = sc.cw, cm = sc.cm, cb = sc.cb;
        auto update = [&](Real* Wm, Real* Mm, int rows, int cols, const Real* P, auto load_xcol) {
            block_gemm<Real, 2, false, false>(
                rows, cols, len,
                [&](int m, int t, Real& a0, Real& a1) {
                    const Real p = P[(size_t)t * rows + m];
                    a0 = sc.kW[t] * p;
                    a1 = sc.kM[t] * p;
                },
                load_xcol,
                [&](int m, int n, Real aW, Real aM) {
                    const size_t e = (size_t)m * cols + n;
                    const Real w = Wm[e], mm = Mm[e];
                    Wm[e] = cw * w + cm * mm - aW; // G_t = -grad: the aggregations enter with a minus sign
                    Mm[e] = cb * mm - aM;
                },
                &gsm, rank, CL);
        };
        auto key_col = [&](int n, int t) { return ld_io<Real>(kc, (size_t)t * d + n); };
        auto act_col = [&](int n, int t) { return A[(size_t)t * h + n]; };
        update(W[0], M[0], h, d, Pz1, key_col);
        if (KIND == 1) update(W[1], M[1], h, d, Pz2, key_col);
        update(W[LAST], M[LAST], d, h, Pu, act_col);
    }

#pragma unroll
    for (int i = 0; i < NMAT; ++i) {
        if (!a.W_final[i]) continue; // state-recompute run of the backward: only the saved chunk states matter
        float* wf = a.W_final[i] + (size_t)seq * dh;
        float* mf = a.M_final[i] + (size_t)seq * dh;
        for (size_t e = tid + (size_t)rank * kSimtThreads; e < dh; e += (size_t)kSimtThreads * CL) {
            wf[e] = (float)W[i][e];
            mf[e] = (float)M[i][e];
        }
    }
}

template <typename Real, typename IO, int KIND>
static int launch_fwd(const SimtFwdArgs& a, cudaStream_t st) {
    constexpr size_t smem = sizeof(GemmSmem<Real>) + sizeof(ChunkScalars<Real>);
    static bool attr_done[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return (int)cudaGetLastError();
    if (dev < 0 || dev >= 64 || !attr_done[dev]) {
        cudaError_t e = cudaFuncSetAttribute(simt_fwd_kernel<Real, IO, KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return (int)e;
        if (dev >= 0 && dev < 64) attr_done[dev] = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(a.N * a.cl));
    cfg.blockDim = dim3(kSimtThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)a.cl;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, simt_fwd_kernel<Real, IO, KIND>, a);
    if (e != cudaSuccess) return (int)e;
    return (int)cudaGetLastError();
}

int simt_fwd_launch(const SimtFwdArgs& a, int kind, int io_dtype, void* stream) {
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (io_dtype == 0) return kind == 0 ? launch_fwd<double, float, 0>(a, st) : launch_fwd<double, float, 1>(a, st);
    return kind == 0 ? launch_fwd<float, __nv_bfloat16, 0>(a, st) : launch_fwd<float, __nv_bfloat16, 1>(a, st);
}

}  // namespace e2ttt
