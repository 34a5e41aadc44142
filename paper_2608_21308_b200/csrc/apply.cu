// Outputs of fixed fast weights: o_t = f_W(q_t) = q_t + LN(W_last act(W_first q_t)) for T tokens per sequence, no update.
// This is the decode path between chunk boundaries (Algorithm 1 line 1 with the chunk-start weights; the state only
// changes once a whole chunk of keys and values has accumulated, and that step is e2ttt_chunk_fwd on those tokens).
//
// For a handful of tokens the work is a matrix-vector product over the whole state, so the kernel is bound by reading
// W once from HBM: 4 * nmat * d * h bytes per sequence.  A cluster of up to 8 CTAs serves one sequence; CTA c streams
// the hidden units [h0, h1) of every matrix - rows of the first matrices, a column slice of the last - with 8
// independent 16-byte loads per lane in flight, keeps the activations of its slice in shared memory, and produces a
// partial sum of the d outputs.  The slice of the last matrix does not depend on the activations, so its copy into
// shared memory (cp.async, no registers) is started before the first matrices are read: all of a CTA's bytes are in
// flight together.  The partial sums meet in the shared memory of the cluster's first CTA (distributed
// shared memory, fixed summation order), which applies the layer norm and the residual and stores o.
#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "apply.h"
#include "simt_common.cuh"

namespace cg = cooperative_groups;

namespace e2ttt {
namespace {

constexpr int kApThreads = 256;
constexpr int kApWarps = kApThreads / 32;
constexpr int kApHB = 256;   // hidden units per pass through shared memory
constexpr int kApRows = 8;   // rows a warp streams at once (independent loads in flight)
constexpr int kApStageBytes = 64 * 1024;  // shared-memory staging of the last matrix's block (asynchronous copies)

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src)
                 : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
}

template <typename T> __device__ __forceinline__ float ap_ld(const T* p, size_t i);
template <> __device__ __forceinline__ float ap_ld<float>(const float* p, size_t i) { return p[i]; }
template <> __device__ __forceinline__ float ap_ld<__nv_bfloat16>(const __nv_bfloat16* p, size_t i) { return __bfloat162float(p[i]); }
__device__ __forceinline__ void ap_st(float* p, size_t i, float v) { p[i] = v; }
__device__ __forceinline__ void ap_st(__nv_bfloat16* p, size_t i, float v) { p[i] = __float2bfloat16(v); }

// dot products of R rows of a row-major matrix (row stride ld, columns [c0, c0 + n)) with TB vectors held in shared
// memory (x[t][0..n)); one warp, result valid in every lane.  VEC: 16-byte loads (n % 4 == 0, aligned rows).
template <int R, int TB, bool VEC>
__device__ __forceinline__ void warp_dots(const float* __restrict__ w, size_t ld, int rows_valid, int n,
                                          const float* x, int xld, float (&acc)[R][TB]) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int t = 0; t < TB; ++t) acc[r][t] = 0.0f;
    if (VEC) {
        for (int c = 4 * lane; c < n; c += 128) {
            float4 wv[R];
#pragma unroll
            for (int r = 0; r < R; ++r)
                wv[r] = (r < rows_valid) ? *reinterpret_cast<const float4*>(w + (size_t)r * ld + c) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int t = 0; t < TB; ++t) {
                const float4 xv = *reinterpret_cast<const float4*>(x + (size_t)t * xld + c);
#pragma unroll
                for (int r = 0; r < R; ++r)
                    acc[r][t] += wv[r].x * xv.x + wv[r].y * xv.y + wv[r].z * xv.z + wv[r].w * xv.w;
            }
        }
    } else {
        for (int c = lane; c < n; c += 32) {
            float wv[R];
#pragma unroll
            for (int r = 0; r < R; ++r) wv[r] = (r < rows_valid) ? w[(size_t)r * ld + c] : 0.0f;
#pragma unroll
            for (int t = 0; t < TB; ++t) {
                const float xv = x[(size_t)t * xld + c];
#pragma unroll
                for (int r = 0; r < R; ++r) acc[r][t] += wv[r] * xv;
            }
        }
    }
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int t = 0; t < TB; ++t) acc[r][t] = warp_sum(acc[r][t]);
}

template <typename IO, int KIND, int TB, bool VEC>
__global__ void __launch_bounds__(kApThreads, 2) apply_kernel(const ApplyArgs a) {
    constexpr int NMAT = (KIND == 0) ? 2 : 3;
    extern __shared__ __align__(16) float ap_smem[];
    cg::cluster_group cluster = cg::this_cluster();
    const int CL = a.cl;
    const int seq = blockIdx.x / CL, rank = blockIdx.x % CL;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int d = a.d, h = a.h, T = a.T;
    const size_t dh = (size_t)d * h;

    float* qs = ap_smem;                       // [TB][d]   the tokens
    float* as = qs + (size_t)TB * d;           // [TB][HB]  activations of the current hidden block
    float* up = as + (size_t)TB * kApHB;       // [TB][d]   this CTA's partial sums
    float* slots = up + (size_t)TB * d;        // [CL][TB][d] on the first CTA: every CTA's partial sums
    float* wls = slots + (size_t)CL * TB * d;  // [d][nh] staged block of the last matrix (when a.stage)

    const IO* q = reinterpret_cast<const IO*>(a.q) + (size_t)seq * T * d;
    IO* o = reinterpret_cast<IO*>(a.o) + (size_t)seq * T * d;
    const float* W1 = a.W[0] + (size_t)seq * dh;                                 // [h, d]
    const float* W2 = (KIND == 1) ? a.W[1] + (size_t)seq * dh : nullptr;         // [h, d] (SwiGLU gate partner)
    const float* Wl = a.W[NMAT - 1] + (size_t)seq * dh;                          // [d, h]

    // this CTA's hidden units: an even split in multiples of 4 (keeps 16-byte alignment of the column slices)
    const int per = ((h + CL - 1) / CL + 3) & ~3;
    const int h0 = min(h, rank * per), h1 = min(h, h0 + per);
    float* slot0 = cluster.map_shared_rank(slots, 0);

    // Programmatic dependent launch: this grid may start while the previous kernel of the stream is still running.
    // Nothing it produces may be touched before griddepcontrol.wait - but the fast weights of this CTA can already be
    // pulled from HBM into L2 (a prefetch has no effect on memory contents), so that the next layer's weights stream
    // in under the tail of the previous kernel.  Without a programmatic predecessor the wait returns at once.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (h0 < h1) {
        const int nrows = h1 - h0;
        // rows [h0, h1) of the first matrices are contiguous; the last matrix contributes d row segments
        const size_t bytes1 = (size_t)nrows * d * sizeof(float);
        for (size_t off = (size_t)tid * 128; off < bytes1; off += (size_t)kApThreads * 128) {
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(W1 + (size_t)h0 * d) + off));
            if (KIND == 1) asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(W2 + (size_t)h0 * d) + off));
        }
        const int seg = (nrows * (int)sizeof(float) + 127) / 128;  // 128-byte lines per row segment
        for (int e = tid; e < d * seg; e += kApThreads) {
            const int i = e / seg, c = e - i * seg;
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(Wl + (size_t)i * h + h0) + (size_t)c * 128));
        }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");

    for (int t0 = 0; t0 < T; t0 += TB) {
        const int tb = min(TB, T - t0);
        for (int e = tid; e < TB * d; e += kApThreads) {
            const int t = e / d, i = e - t * d;
            qs[e] = (t < tb) ? ap_ld<IO>(q, (size_t)(t0 + t) * d + i) : 0.0f;
            up[e] = 0.0f;
        }
        __syncthreads();
        for (int hb = h0; hb < h1; hb += kApHB) {
            const int nh = min(kApHB, h1 - hb);
            if (VEC && a.stage) {  // start the copy of the last matrix's block; it lands while the activations are computed
                const int n4 = nh >> 2;
                for (int e = tid; e < d * n4; e += kApThreads) {
                    const int i = e / n4, c4 = e - i * n4;
                    cp_async16(wls + (size_t)i * nh + 4 * c4, Wl + (size_t)i * h + hb + 4 * c4);
                }
            }
            // hidden activations of the block: one warp per group of rows
            for (int j0 = warp * kApRows; j0 < nh; j0 += kApWarps * kApRows) {
                const int rv = min(kApRows, nh - j0);
                float z1[kApRows][TB];
                warp_dots<kApRows, TB, VEC>(W1 + (size_t)(hb + j0) * d, d, rv, d, qs, d, z1);
                if (KIND == 1) {
                    float z2[kApRows][TB];
                    warp_dots<kApRows, TB, VEC>(W2 + (size_t)(hb + j0) * d, d, rv, d, qs, d, z2);
#pragma unroll
                    for (int r = 0; r < kApRows; ++r)
#pragma unroll
                        for (int t = 0; t < TB; ++t) z1[r][t] = silu_f(z1[r][t]) * z2[r][t];
                } else {
#pragma unroll
                    for (int r = 0; r < kApRows; ++r)
#pragma unroll
                        for (int t = 0; t < TB; ++t) z1[r][t] = gelu_f(z1[r][t]);
                }
                if (lane == 0) {
#pragma unroll
                    for (int r = 0; r < kApRows; ++r)
                        if (r < rv)
#pragma unroll
                            for (int t = 0; t < TB; ++t) as[(size_t)t * kApHB + j0 + r] = z1[r][t];
                }
            }
            // zero the tail so that the vector loop below may run over a multiple of 4
            for (int e = tid; e < TB * 4; e += kApThreads) {
                const int t = e >> 2, j = nh + (e & 3);
                if (j < kApHB) as[(size_t)t * kApHB + j] = 0.0f;
            }
            if (VEC && a.stage) cp_async_wait_all();
            __syncthreads();
            // partial outputs: row i of the last matrix, columns of this block (the same warp owns row i in every block)
            for (int i0 = warp * kApRows; i0 < d; i0 += kApWarps * kApRows) {
                const int rv = min(kApRows, d - i0);
                float u[kApRows][TB];
                if (VEC && a.stage)
                    warp_dots<kApRows, TB, VEC>(wls + (size_t)i0 * nh, nh, rv, nh, as, kApHB, u);
                else
                    warp_dots<kApRows, TB, VEC>(Wl + (size_t)i0 * h + hb, h, rv, nh, as, kApHB, u);
                if (lane == 0) {
#pragma unroll
                    for (int r = 0; r < kApRows; ++r)
                        if (r < rv)
#pragma unroll
                            for (int t = 0; t < TB; ++t) up[(size_t)t * d + i0 + r] += u[r][t];
                }
            }
            __syncthreads();
        }
        // hand the partial sums to the first CTA of the cluster
        for (int e = tid; e < TB * d; e += kApThreads) slot0[(size_t)rank * TB * d + e] = up[e];
        cluster.sync();
        if (rank == 0) {
            for (int e = tid; e < TB * d; e += kApThreads) {
                float s = 0.0f;
                for (int c = 0; c < CL; ++c) s += slots[(size_t)c * TB * d + e];  // fixed order
                up[e] = s;
            }
            __syncthreads();
            for (int t = warp; t < tb; t += kApWarps) {
                float* u = up + (size_t)t * d;
                warp_layernorm(u, u, d, a.eps);
                for (int i = lane; i < d; i += 32) ap_st(o, (size_t)(t0 + t) * d + i, qs[(size_t)t * d + i] + u[i]);
            }
        }
        if (t0 + TB < T) cluster.sync();  // the slots are free again (after the last pass nobody writes them any more)
    }
}

}  // namespace

size_t apply_smem_bytes(int d, int cl, int tb) { return ((size_t)tb * d * (2 + cl) + (size_t)tb * kApHB) * sizeof(float); }

namespace {

template <typename IO, int KIND, int TB, bool VEC>
int launch_apply(const ApplyArgs& a, cudaStream_t st) {
    const size_t smem = apply_smem_bytes(a.d, a.cl, TB) + (a.stage ? (size_t)kApStageBytes : 0);
    static size_t attr_bytes[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return (int)cudaGetLastError();
    if (dev < 0 || dev >= 64 || attr_bytes[dev] < smem) {
        cudaError_t e = cudaFuncSetAttribute(apply_kernel<IO, KIND, TB, VEC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return (int)e;
        if (dev >= 0 && dev < 64) attr_bytes[dev] = smem;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(a.N * a.cl));
    cfg.blockDim = dim3(kApThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)a.cl;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // see griddepcontrol in the kernel
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 2;
    cudaError_t e = cudaLaunchKernelEx(&cfg, apply_kernel<IO, KIND, TB, VEC>, a);
    if (e != cudaSuccess) return (int)e;
    return (int)cudaGetLastError();
}

template <typename IO, int KIND>
int dispatch_apply(const ApplyArgs& a, bool vec, cudaStream_t st) {
    if (a.tb == 1) return vec ? launch_apply<IO, KIND, 1, true>(a, st) : launch_apply<IO, KIND, 1, false>(a, st);
    return vec ? launch_apply<IO, KIND, 4, true>(a, st) : launch_apply<IO, KIND, 4, false>(a, st);
}

}  // namespace

int apply_token_block(int T) { return T == 1 ? 1 : 4; }

// The last matrix's block [d][min(256, hidden units per CTA)] is staged when it fits the staging buffer.
int apply_can_stage(int d, int h, int cl) {
    const int per = ((h + cl - 1) / cl + 3) & ~3;
    const int nh = per < kApHB ? per : kApHB;
    return (size_t)d * nh * sizeof(float) <= (size_t)kApStageBytes;
}

int apply_launch(const ApplyArgs& a, int kind, int io_dtype, void* stream) {
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    // 16-byte loads need rows that start on 16-byte boundaries: d and h multiples of 4, 16-byte aligned bases
    bool vec = (a.d % 4 == 0) && (a.h % 4 == 0);
    const int nmat = kind == 0 ? 2 : 3;
    for (int i = 0; i < nmat; ++i) vec = vec && (reinterpret_cast<uintptr_t>(a.W[i]) % 16 == 0);
    if (io_dtype == 0)
        return kind == 0 ? dispatch_apply<float, 0>(a, vec, st) : dispatch_apply<float, 1>(a, vec, st);
    return kind == 0 ? dispatch_apply<__nv_bfloat16, 0>(a, vec, st) : dispatch_apply<__nv_bfloat16, 1>(a, vec, st);
}

}  // namespace e2ttt
