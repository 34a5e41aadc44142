// Token preparation upstream of the chunk update (Section 4, "Overall Architecture" and the gate parameterisation):
//   q, k <- silu(x) / max(||silu(x)||_2, eps) per token and head;
//   eta = eta_base sigmoid(a),  beta = sigmoid(b)^(1/tau),  gamma = 1 - eta alpha_base sigmoid(c)
// and the reverse pass.  Pure streaming work: every byte is read once and written once, so the kernels are bound by
// HBM.  One warp owns a token-head row of d elements: lane l holds the V-element pieces (p * 32 + l) of the row in
// registers between the norm reduction and the scaled store (V and the piece count are compile-time, so nothing
// spills to local memory), and works on the query and the key rows of two tokens at once so that four rows' loads
// are in flight per lane.  Grid: one wave of 8-warp CTAs with a grid-stride loop over the token-heads.
// The forward of rows that allow it (row bytes a multiple of 16, aligned bases, d <= 256) runs as a bulk-copy pipeline
// instead: tiles of 32 tokens travel global -> shared memory -> global with `cp.async.bulk` (mbarrier transaction
// counts on the way in, bulk groups on the way out), four tiles deep per CTA, so the bytes in flight do not depend
// on registers or occupancy; the warps only touch shared memory.  The reverse pass has the same form (four tiles in,
// two out, three deep).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <type_traits>

#include "prepare.h"
#include "simt_common.cuh"
#include "sm100.cuh"

namespace e2ttt {
namespace {

constexpr int kPrThreads = 256;
constexpr int kPrTokens = 2;  // tokens a warp works on at once

// sigmoid with the hardware exp2 and reciprocal: the IEEE division alone costs more instructions than the rest of
// an element's work, and the kernels are meant to be bound by memory, not by issue slots
__device__ __forceinline__ float pr_sigmoid(float z) { return __fdividef(1.0f, 1.0f + __expf(-z)); }

// silu(x) = x sigmoid(x).  With bf16 I/O the result is rounded to 2^-9 relative right after, so the hardware tanh
// serves: x sigmoid(x) = hx + hx tanh(hx), hx = x / 2 (one MUFU and two FMA-pipe instructions; tanh.approx is good to
// about 2^-11).  fp32 I/O keeps the exp form.
template <typename IO> __device__ __forceinline__ float pr_silu(float x) {
    if (sizeof(IO) == 2) {
        const float hx = 0.5f * x;
        float t;
        asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(hx));
        return fmaf(hx, t, hx);
    }
    return x * pr_sigmoid(x);
}

// V consecutive elements <-> registers, one memory access of V * sizeof(IO) bytes (V = 1, 2 or 4)
template <typename IO, int V> __device__ __forceinline__ void ld_piece(const IO* p, float* v) {
    if (sizeof(IO) == 4) {
        if (V == 4) { const float4 x = *reinterpret_cast<const float4*>(p); v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w; }
        else if (V == 2) { const float2 x = *reinterpret_cast<const float2*>(p); v[0] = x.x; v[1] = x.y; }
        else v[0] = ld_io<float>(p, (size_t)0);
    } else {
        if (V == 4) {
            const uint2 raw = *reinterpret_cast<const uint2*>(p);
            const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
            const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
            v[0] = a.x; v[1] = a.y; v[2] = b.x; v[3] = b.y;
        } else if (V == 2) {
            const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(p));
            v[0] = a.x; v[1] = a.y;
        } else v[0] = ld_io<float>(p, (size_t)0);
    }
}
template <typename IO, int V> __device__ __forceinline__ void st_piece(IO* p, const float* v) {
    if (sizeof(IO) == 4) {
        if (V == 4) *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
        else if (V == 2) *reinterpret_cast<float2*>(p) = make_float2(v[0], v[1]);
        else st_io(p, (size_t)0, v[0]);
    } else {
        if (V == 4) {
            uint2 raw;
            *reinterpret_cast<__nv_bfloat162*>(&raw.x) = __floats2bfloat162_rn(v[0], v[1]);
            *reinterpret_cast<__nv_bfloat162*>(&raw.y) = __floats2bfloat162_rn(v[2], v[3]);
            *reinterpret_cast<uint2*>(p) = raw;
        } else if (V == 2) {
            *reinterpret_cast<__nv_bfloat162*>(p) = __floats2bfloat162_rn(v[0], v[1]);
        } else st_io(p, (size_t)0, v[0]);
    }
}

// a row in registers: NP pieces of V elements per lane
template <typename IO, int V, int NP> __device__ __forceinline__ void ld_row(const IO* p, int d, float (&v)[NP * V]) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int pc = 0; pc < NP; ++pc) {
        const int c = (pc * 32 + lane) * V;
        if (c < d) ld_piece<IO, V>(p + c, &v[pc * V]);
        else
#pragma unroll
            for (int j = 0; j < V; ++j) v[pc * V + j] = 0.0f;
    }
}
template <typename IO, int V, int NP> __device__ __forceinline__ void st_row(IO* p, int d, const float (&v)[NP * V]) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int pc = 0; pc < NP; ++pc) {
        const int c = (pc * 32 + lane) * V;
        if (c < d) st_piece<IO, V>(p + c, &v[pc * V]);
    }
}

template <typename IO, int V, int NP>
__global__ void __launch_bounds__(kPrThreads) prepare_fwd_kernel(const PrepareArgs a) {
    const long long warp = (long long)((blockIdx.x * (size_t)kPrThreads + threadIdx.x) >> 5);
    const long long nwarps = (long long)((gridDim.x * (size_t)kPrThreads) >> 5);
    const int lane = threadIdx.x & 31;
    const int d = a.d;
    const IO* q_raw = reinterpret_cast<const IO*>(a.q_raw);
    const IO* k_raw = reinterpret_cast<const IO*>(a.k_raw);
    IO* q = reinterpret_cast<IO*>(a.q);
    IO* k = reinterpret_cast<IO*>(a.k);
    for (long long t0 = warp * kPrTokens; t0 < a.rows; t0 += nwarps * kPrTokens) {
        float x[2 * kPrTokens][NP * V];  // query and key rows of the warp's tokens
#pragma unroll
        for (int u = 0; u < kPrTokens; ++u) {
            const long long t = t0 + u;
            if (t < a.rows) {
                ld_row<IO, V, NP>(q_raw + (size_t)t * d, d, x[2 * u]);
                ld_row<IO, V, NP>(k_raw + (size_t)t * d, d, x[2 * u + 1]);
            }
        }
#pragma unroll
        for (int r = 0; r < 2 * kPrTokens; ++r) {
            const long long t = t0 + (r >> 1);
            if (t >= a.rows) continue;
            float ss = 0.0f;
#pragma unroll
            for (int j = 0; j < NP * V; ++j) {
                x[r][j] = pr_silu<IO>(x[r][j]);
                ss = fmaf(x[r][j], x[r][j], ss);
            }
            const float f = 1.0f / fmaxf(sqrtf(warp_sum(ss)), a.norm_eps);
#pragma unroll
            for (int j = 0; j < NP * V; ++j) x[r][j] *= f;
            st_row<IO, V, NP>(((r & 1) ? k : q) + (size_t)t * d, d, x[r]);
        }
        if (lane < kPrTokens && t0 + lane < a.rows) {
            const long long t = t0 + lane;
            const float eta = a.eta_base * pr_sigmoid(a.a_eta[t]);
            const float beta = __powf(pr_sigmoid(a.a_beta[t]), 1.0f / a.tau);
            const float alpha = a.alpha_base * pr_sigmoid(a.a_alpha[t]);
            a.eta[t] = eta;
            a.beta[t] = beta;
            a.gamma[t] = 1.0f - eta * alpha;
        }
    }
}

// reverse of a normalised row: y = s / m, m = max(||s||, eps), s = silu(x):  x_bar = silu'(x) (y_bar - y <y_bar, y>) / m
template <typename IO, int V, int NP>
__global__ void __launch_bounds__(kPrThreads) prepare_bwd_kernel(const PrepareBwdArgs a) {
    const long long warp = (long long)((blockIdx.x * (size_t)kPrThreads + threadIdx.x) >> 5);
    const long long nwarps = (long long)((gridDim.x * (size_t)kPrThreads) >> 5);
    const int lane = threadIdx.x & 31;
    const int d = a.f.d;
    for (long long t = warp; t < a.f.rows; t += nwarps) {
        const size_t off = (size_t)t * d;
        float x[2][NP * V], g[2][NP * V];
        ld_row<IO, V, NP>(reinterpret_cast<const IO*>(a.f.q_raw) + off, d, x[0]);
        ld_row<IO, V, NP>(reinterpret_cast<const IO*>(a.f.k_raw) + off, d, x[1]);
        ld_row<IO, V, NP>(reinterpret_cast<const IO*>(a.dq) + off, d, g[0]);
        ld_row<IO, V, NP>(reinterpret_cast<const IO*>(a.dk) + off, d, g[1]);
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            float ss = 0.0f, sg = 0.0f;
#pragma unroll
            for (int j = 0; j < NP * V; ++j) {
                const float sig = pr_sigmoid(x[r][j]);
                const float s = x[r][j] * sig;
                ss = fmaf(s, s, ss);
                sg = fmaf(s, g[r][j], sg);
                g[r][j] *= sig * (1.0f + x[r][j] * (1.0f - sig));  // y_bar silu'(x)
                x[r][j] = s * sig * (1.0f + x[r][j] * (1.0f - sig));  // s silu'(x)
            }
            const float nrm = sqrtf(warp_sum(ss));
            sg = warp_sum(sg);
            const float m = fmaxf(nrm, a.f.norm_eps);
            const float proj = (nrm > a.f.norm_eps) ? sg / (m * m) : 0.0f;  // <y_bar, y> / m
            const float inv = 1.0f / m;
#pragma unroll
            for (int j = 0; j < NP * V; ++j) g[r][j] = (g[r][j] - x[r][j] * proj) * inv;
            st_row<IO, V, NP>(reinterpret_cast<IO*>(r ? a.dk_raw : a.dq_raw) + off, d, g[r]);
        }
        if (lane == 0) {
            const float sa = pr_sigmoid(a.f.a_eta[t]), sb = pr_sigmoid(a.f.a_beta[t]), sc = pr_sigmoid(a.f.a_alpha[t]);
            const float eta = a.f.eta_base * sa, alpha = a.f.alpha_base * sc;
            const float beta = __powf(sb, 1.0f / a.f.tau);
            const float eta_bar = a.d_eta[t] - a.d_gamma[t] * alpha;
            a.da_eta[t] = eta_bar * a.f.eta_base * sa * (1.0f - sa);
            a.da_beta[t] = a.d_beta[t] * beta * (1.0f - sb) / a.f.tau;
            a.da_alpha[t] = -a.d_gamma[t] * eta * a.f.alpha_base * sc * (1.0f - sc);
        }
    }
}

// ---- forward as a bulk-copy pipeline ------------------------------------------------------------------------
constexpr int kBkTok = 32;     // tokens per tile
constexpr int kBkStages = 4;   // tiles in flight per CTA

__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(sm100::smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(sm100::smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void bulk_store(void* gdst, const void* smem_src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(gdst), "r"(sm100::smem_u32(smem_src)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
template <int N> __device__ __forceinline__ void bulk_wait_all() {
    asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}
// Bounded wait for a tile (about a second), every lane polling so that the warp stays converged.  A wait that runs out
// raises the CTA-wide `dead` flag; later waits then return at once and the CTA runs through its remaining tiles (and all
// of its barriers) without meaning.  These two kernels have no status word to report it through: the bulk loads they
// wait for cannot fail short of a device fault, which the next runtime call reports.
__device__ __forceinline__ void bulk_wait_tile(uint64_t* bar, uint32_t parity, volatile int* dead) {
    if (!sm100::mbar_try_wait<false>(bar, parity) && !*dead) {
        const long long t0 = clock64();
        int spins = 0;
        while (!sm100::mbar_try_wait<false>(bar, parity)) {
            if ((++spins & 255) == 0 && (*dead || clock64() - t0 > sm100::kWaitCycles)) { *dead = 1; break; }
        }
    }
    __syncwarp();
}

// LPR = lanes per row: a row is LPR pieces of 16 bytes (d = LPR * 16 / sizeof(IO)), one piece per lane, so a warp works on
// 32 / LPR rows at once and the norm reduction runs over LPR lanes only.
template <typename IO, int LPR>
__global__ void __launch_bounds__(kPrThreads) prepare_fwd_bulk_kernel(const PrepareArgs a) {
    extern __shared__ __align__(128) unsigned char pr_smem[];
    const int d = a.d;
    const uint32_t row_bytes = (uint32_t)d * sizeof(IO);
    const uint32_t tile_bytes = kBkTok * row_bytes;          // one of q / k
    uint64_t* full = reinterpret_cast<uint64_t*>(pr_smem);   // [kBkStages]
    volatile int* dead = reinterpret_cast<volatile int*>(pr_smem + 64);
    unsigned char* tiles = pr_smem + 128;                    // [kBkStages][2][tile_bytes]
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long ntiles = (a.rows + kBkTok - 1) / kBkTok;
    const IO* q_raw = reinterpret_cast<const IO*>(a.q_raw);
    const IO* k_raw = reinterpret_cast<const IO*>(a.k_raw);
    IO* q = reinterpret_cast<IO*>(a.q);
    IO* k = reinterpret_cast<IO*>(a.k);

    if (tid == 0) {
        for (int s = 0; s < kBkStages; ++s) sm100::mbar_init(&full[s], 1);
        *dead = 0;
        sm100::fence_mbar_init();
    }
    __syncthreads();
    auto tokens_of = [&](long long tile) { return (int)min((long long)kBkTok, a.rows - tile * kBkTok); };
    auto issue = [&](long long tile, int s) {  // thread 0
        const uint32_t bytes = (uint32_t)tokens_of(tile) * row_bytes;
        sm100::mbar_expect_tx(&full[s], 2 * bytes);
        bulk_load(tiles + (size_t)(2 * s) * tile_bytes, q_raw + (size_t)tile * kBkTok * d, bytes, &full[s]);
        bulk_load(tiles + (size_t)(2 * s + 1) * tile_bytes, k_raw + (size_t)tile * kBkTok * d, bytes, &full[s]);
    };
    if (tid == 0)
        for (int i = 0; i < kBkStages; ++i) {
            const long long tile = blockIdx.x + (long long)i * gridDim.x;
            if (tile < ntiles) issue(tile, i);
        }

    long long it = 0;
    for (long long tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++it) {
        const int s = (int)(it % kBkStages);
        const uint32_t parity = (uint32_t)((it / kBkStages) & 1);
        const int ntok = tokens_of(tile);
        bulk_wait_tile(&full[s], parity, dead);
        IO* tq = reinterpret_cast<IO*>(tiles + (size_t)(2 * s) * tile_bytes);
        IO* tk = reinterpret_cast<IO*>(tiles + (size_t)(2 * s + 1) * tile_bytes);
        // gates of the tile's tokens (plain coalesced accesses)
        if (tid < ntok) {
            const long long t = tile * kBkTok + tid;
            const float eta = a.eta_base * pr_sigmoid(a.a_eta[t]);
            const float beta = __powf(pr_sigmoid(a.a_beta[t]), 1.0f / a.tau);
            const float alpha = a.alpha_base * pr_sigmoid(a.a_alpha[t]);
            a.eta[t] = eta;
            a.beta[t] = beta;
            a.gamma[t] = 1.0f - eta * alpha;
        }
        // rows 0..31 of the tile pair are the query rows, 32..63 the key rows; a warp pass covers 32 / LPR of them, in place
        {
            constexpr int E = 16 / (int)sizeof(IO), RPP = 32 / LPR;
            const int sub = lane / LPR, li = lane % LPR;
            for (int base = warp * RPP; base < 2 * kBkTok; base += (kPrThreads / 32) * RPP) {
                const int r = base + sub;
                const int u = r & (kBkTok - 1);
                const bool valid = u < ntok;
                IO* piece = ((r >= kBkTok) ? tk : tq) + (size_t)u * d + li * E;
                float x[E];
                if (valid) {
                    const uint4 raw = *reinterpret_cast<const uint4*>(piece);
                    if (sizeof(IO) == 2) {
                        const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
                        for (int j = 0; j < E / 2; ++j) {
                            const float2 f2 = __bfloat1622float2(h2[j]);
                            x[2 * j] = f2.x;
                            x[2 * j + 1] = f2.y;
                        }
                    } else {
                        const float* f4 = reinterpret_cast<const float*>(&raw);
#pragma unroll
                        for (int j = 0; j < E; ++j) x[j] = f4[j];
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < E; ++j) x[j] = 0.0f;
                }
                float ss = 0.0f;
#pragma unroll
                for (int j = 0; j < E; ++j) {
                    x[j] = pr_silu<IO>(x[j]);
                    ss = fmaf(x[j], x[j], ss);
                }
#pragma unroll
                for (int off = LPR / 2; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
                // 1 / max(||s||, eps)
                const float f = (ss > a.norm_eps * a.norm_eps) ? rsqrtf(ss) : __fdividef(1.0f, a.norm_eps);
                if (valid) {
                    uint4 raw;
                    if (sizeof(IO) == 2) {
                        __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&raw);
#pragma unroll
                        for (int j = 0; j < E / 2; ++j) h2[j] = __floats2bfloat162_rn(x[2 * j] * f, x[2 * j + 1] * f);
                    } else {
                        float* f4 = reinterpret_cast<float*>(&raw);
#pragma unroll
                        for (int j = 0; j < E; ++j) f4[j] = x[j] * f;
                    }
                    *reinterpret_cast<uint4*>(piece) = raw;
                }
            }
        }
        sm100::fence_proxy_async_smem();  // the normalised rows -> visible to the bulk store
        __syncthreads();
        if (tid == 0) {
            const uint32_t bytes = (uint32_t)ntok * row_bytes;
            bulk_store(q + (size_t)tile * kBkTok * d, tq, bytes);
            bulk_store(k + (size_t)tile * kBkTok * d, tk, bytes);
            bulk_commit();
            // the stage used one tile ago is free once its store has read shared memory: refill it
            if (it >= 1) {
                bulk_wait_read<1>();
                const long long next = tile + (long long)(kBkStages - 1) * gridDim.x;
                if (next < ntiles) issue(next, (int)((it - 1) % kBkStages));
            }
        }
    }
    if (tid == 0) bulk_wait_all<0>();  // the CTA's shared memory must outlive its stores
    __syncthreads();
}

int grid_for(long long rows, int rows_per_warp) {
    const long long warps = (rows + rows_per_warp - 1) / rows_per_warp;
    const long long want = (warps + (kPrThreads / 32) - 1) / (kPrThreads / 32);
    const long long cap = 148LL * 8;  // one wave at 8 CTAs of 256 threads per SM
    return (int)(want < cap ? (want < 1 ? 1 : want) : cap);
}

// piece width and count: 4-element pieces when the rows allow aligned 8-/16-byte accesses, else scalar
struct Shape { int v, np; };
Shape pick_shape(int d, int io_bytes, const void* const* ptrs, int nptrs) {
    bool al = true;
    for (int i = 0; i < nptrs; ++i) al = al && (reinterpret_cast<uintptr_t>(ptrs[i]) % 16 == 0);
    (void)io_bytes;
    if (al && d % 4 == 0 && d >= 128) return {4, d <= 128 ? 1 : d <= 256 ? 2 : d <= 512 ? 4 : 8};
    if (al && d % 2 == 0 && d <= 64) return {2, 1};
    return {1, 32};
}

template <typename IO, typename Args, typename F> int dispatch(const Shape& s, F launch) {
    if (s.v == 4 && s.np == 1) return launch(std::integral_constant<int, 4>(), std::integral_constant<int, 1>());
    if (s.v == 4 && s.np == 2) return launch(std::integral_constant<int, 4>(), std::integral_constant<int, 2>());
    if (s.v == 4 && s.np == 4) return launch(std::integral_constant<int, 4>(), std::integral_constant<int, 4>());
    if (s.v == 4 && s.np == 8) return launch(std::integral_constant<int, 4>(), std::integral_constant<int, 8>());
    if (s.v == 2) return launch(std::integral_constant<int, 2>(), std::integral_constant<int, 1>());
    return launch(std::integral_constant<int, 1>(), std::integral_constant<int, 32>());
}

// ---- reverse pass as the same kind of pipeline: four tiles in (x of q and k, y_bar of q and k), two out (in place) ----
constexpr int kBkStagesBwd = 3;

template <typename IO> __device__ __forceinline__ float pr_sig(float x) {
    if (sizeof(IO) == 2) {  // bf16 I/O: hardware tanh, sigmoid(x) = 0.5 + 0.5 tanh(x / 2)
        float t;
        asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(0.5f * x));
        return fmaf(0.5f, t, 0.5f);
    }
    return pr_sigmoid(x);
}

template <typename IO, int LPR>
__global__ void __launch_bounds__(kPrThreads) prepare_bwd_bulk_kernel(const PrepareBwdArgs a) {
    extern __shared__ __align__(128) unsigned char pr_smem[];
    const int d = a.f.d;
    const uint32_t row_bytes = (uint32_t)d * sizeof(IO);
    const uint32_t tile_bytes = kBkTok * row_bytes;
    uint64_t* full = reinterpret_cast<uint64_t*>(pr_smem);
    volatile int* dead = reinterpret_cast<volatile int*>(pr_smem + 64);
    unsigned char* tiles = pr_smem + 128;  // [stages][4][tile_bytes]: x_q, x_k, g_q, g_k
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long ntiles = (a.f.rows + kBkTok - 1) / kBkTok;
    const IO* src[4] = {reinterpret_cast<const IO*>(a.f.q_raw), reinterpret_cast<const IO*>(a.f.k_raw),
                        reinterpret_cast<const IO*>(a.dq), reinterpret_cast<const IO*>(a.dk)};
    IO* dst[2] = {reinterpret_cast<IO*>(a.dq_raw), reinterpret_cast<IO*>(a.dk_raw)};

    if (tid == 0) {
        for (int s = 0; s < kBkStagesBwd; ++s) sm100::mbar_init(&full[s], 1);
        *dead = 0;
        sm100::fence_mbar_init();
    }
    __syncthreads();
    auto tokens_of = [&](long long tile) { return (int)min((long long)kBkTok, a.f.rows - tile * kBkTok); };
    auto issue = [&](long long tile, int s) {  // thread 0
        const uint32_t bytes = (uint32_t)tokens_of(tile) * row_bytes;
        sm100::mbar_expect_tx(&full[s], 4 * bytes);
#pragma unroll
        for (int i = 0; i < 4; ++i)
            bulk_load(tiles + (size_t)(4 * s + i) * tile_bytes, src[i] + (size_t)tile * kBkTok * d, bytes, &full[s]);
    };
    if (tid == 0)
        for (int i = 0; i < kBkStagesBwd; ++i) {
            const long long tile = blockIdx.x + (long long)i * gridDim.x;
            if (tile < ntiles) issue(tile, i);
        }

    long long it = 0;
    for (long long tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++it) {
        const int s = (int)(it % kBkStagesBwd);
        const uint32_t parity = (uint32_t)((it / kBkStagesBwd) & 1);
        const int ntok = tokens_of(tile);
        bulk_wait_tile(&full[s], parity, dead);
        unsigned char* st = tiles + (size_t)(4 * s) * tile_bytes;
        if (tid < ntok) {  // adjoints of the gate logits
            const long long t = tile * kBkTok + tid;
            const float sa = pr_sigmoid(a.f.a_eta[t]), sb = pr_sigmoid(a.f.a_beta[t]), sc = pr_sigmoid(a.f.a_alpha[t]);
            const float eta = a.f.eta_base * sa, alpha = a.f.alpha_base * sc;
            const float beta = __powf(sb, 1.0f / a.f.tau);
            const float eta_bar = a.d_eta[t] - a.d_gamma[t] * alpha;
            a.da_eta[t] = eta_bar * a.f.eta_base * sa * (1.0f - sa);
            a.da_beta[t] = a.d_beta[t] * beta * (1.0f - sb) / a.f.tau;
            a.da_alpha[t] = -a.d_gamma[t] * eta * a.f.alpha_base * sc * (1.0f - sc);
        }
        {
            constexpr int E = 16 / (int)sizeof(IO), RPP = 32 / LPR;
            const int sub = lane / LPR, li = lane % LPR;
            for (int base = warp * RPP; base < 2 * kBkTok; base += (kPrThreads / 32) * RPP) {
                const int r = base + sub;
                const int u = r & (kBkTok - 1), which = r >= kBkTok ? 1 : 0;
                const bool valid = u < ntok;
                const IO* xp = reinterpret_cast<const IO*>(st + (size_t)which * tile_bytes) + (size_t)u * d + li * E;
                IO* gp = reinterpret_cast<IO*>(st + (size_t)(2 + which) * tile_bytes) + (size_t)u * d + li * E;
                float x[E], g[E];
#pragma unroll
                for (int j = 0; j < E; ++j) { x[j] = 0.0f; g[j] = 0.0f; }
                if (valid) {
                    const uint4 rx = *reinterpret_cast<const uint4*>(xp), rg = *reinterpret_cast<const uint4*>(gp);
                    if (sizeof(IO) == 2) {
                        const __nv_bfloat162* hx = reinterpret_cast<const __nv_bfloat162*>(&rx);
                        const __nv_bfloat162* hg = reinterpret_cast<const __nv_bfloat162*>(&rg);
#pragma unroll
                        for (int j = 0; j < E / 2; ++j) {
                            const float2 fx = __bfloat1622float2(hx[j]), fg = __bfloat1622float2(hg[j]);
                            x[2 * j] = fx.x; x[2 * j + 1] = fx.y;
                            g[2 * j] = fg.x; g[2 * j + 1] = fg.y;
                        }
                    } else {
                        const float* fx = reinterpret_cast<const float*>(&rx);
                        const float* fg = reinterpret_cast<const float*>(&rg);
#pragma unroll
                        for (int j = 0; j < E; ++j) { x[j] = fx[j]; g[j] = fg[j]; }
                    }
                }
                float ss = 0.0f, sg = 0.0f;
#pragma unroll
                for (int j = 0; j < E; ++j) {
                    const float sig = pr_sig<IO>(x[j]);
                    const float sv = x[j] * sig;
                    const float dsl = sig * (1.0f + x[j] * (1.0f - sig));  // silu'(x)
                    ss = fmaf(sv, sv, ss);
                    sg = fmaf(sv, g[j], sg);
                    g[j] *= dsl;       // y_bar silu'(x)
                    x[j] = sv * dsl;   // s silu'(x)
                }
#pragma unroll
                for (int off = LPR / 2; off > 0; off >>= 1) {
                    ss += __shfl_xor_sync(0xffffffffu, ss, off);
                    sg += __shfl_xor_sync(0xffffffffu, sg, off);
                }
                const float eps = a.f.norm_eps;
                const bool big = ss > eps * eps;
                const float inv = big ? rsqrtf(ss) : __fdividef(1.0f, eps);   // 1 / max(||s||, eps)
                const float proj = big ? sg * inv * inv : 0.0f;                // <y_bar, y> / m
                if (valid) {
                    uint4 raw;
                    if (sizeof(IO) == 2) {
                        __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&raw);
#pragma unroll
                        for (int j = 0; j < E / 2; ++j)
                            h2[j] = __floats2bfloat162_rn((g[2 * j] - x[2 * j] * proj) * inv, (g[2 * j + 1] - x[2 * j + 1] * proj) * inv);
                    } else {
                        float* f4 = reinterpret_cast<float*>(&raw);
#pragma unroll
                        for (int j = 0; j < E; ++j) f4[j] = (g[j] - x[j] * proj) * inv;
                    }
                    *reinterpret_cast<uint4*>(gp) = raw;  // the adjoint replaces y_bar in its tile
                }
            }
        }
        sm100::fence_proxy_async_smem();
        __syncthreads();
        if (tid == 0) {
            const uint32_t bytes = (uint32_t)ntok * row_bytes;
            bulk_store(dst[0] + (size_t)tile * kBkTok * d, st + (size_t)2 * tile_bytes, bytes);
            bulk_store(dst[1] + (size_t)tile * kBkTok * d, st + (size_t)3 * tile_bytes, bytes);
            bulk_commit();
            if (it >= 1) {
                bulk_wait_read<1>();
                const long long next = tile + (long long)(kBkStagesBwd - 1) * gridDim.x;
                if (next < ntiles) issue(next, (int)((it - 1) % kBkStagesBwd));
            }
        }
    }
    if (tid == 0) bulk_wait_all<0>();
    __syncthreads();
}

template <typename IO, int LPR> int bwd_bulk(const PrepareBwdArgs& a, cudaStream_t st) {
    const size_t smem = 128 + (size_t)kBkStagesBwd * 4 * kBkTok * a.f.d * sizeof(IO);
    static size_t attr_bytes[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return (int)cudaGetLastError();
    if (dev < 0 || dev >= 64 || attr_bytes[dev] < smem) {
        cudaError_t e = cudaFuncSetAttribute(prepare_bwd_bulk_kernel<IO, LPR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return (int)e;
        if (dev >= 0 && dev < 64) attr_bytes[dev] = smem;
    }
    const long long ntiles = (a.f.rows + kBkTok - 1) / kBkTok;
    const int per_sm = (int)(220 * 1024 / smem);
    const long long cap = 148LL * (per_sm > 4 ? 4 : per_sm);
    const int grid = (int)(ntiles < cap ? ntiles : cap);
    prepare_bwd_bulk_kernel<IO, LPR><<<grid, kPrThreads, smem, st>>>(a);
    return (int)cudaGetLastError();
}

size_t bulk_smem_bytes(int d, size_t io_bytes) { return 128 + (size_t)kBkStages * 2 * kBkTok * d * io_bytes; }

template <typename IO, int LPR> int fwd_bulk(const PrepareArgs& a, cudaStream_t st) {
    const size_t smem = bulk_smem_bytes(a.d, sizeof(IO));
    static size_t attr_bytes[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return (int)cudaGetLastError();
    if (dev < 0 || dev >= 64 || attr_bytes[dev] < smem) {
        cudaError_t e = cudaFuncSetAttribute(prepare_fwd_bulk_kernel<IO, LPR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return (int)e;
        if (dev >= 0 && dev < 64) attr_bytes[dev] = smem;
    }
    const long long ntiles = (a.rows + kBkTok - 1) / kBkTok;
    const int per_sm = (int)(220 * 1024 / smem);
    const long long cap = 148LL * (per_sm > 4 ? 4 : per_sm);
    const int grid = (int)(ntiles < cap ? ntiles : cap);
    prepare_fwd_bulk_kernel<IO, LPR><<<grid, kPrThreads, smem, st>>>(a);
    return (int)cudaGetLastError();
}

template <typename IO> int fwd_io(const PrepareArgs& a, cudaStream_t st) {
    const void* ptrs[4] = {a.q_raw, a.k_raw, a.q, a.k};
    const Shape s = pick_shape(a.d, (int)sizeof(IO), ptrs, 4);
    // the bulk-copy pipeline: rows of 8, 16 or 32 pieces of 16 bytes, aligned bases, enough rows to fill the stages
    // (in-place use, q == q_raw, is fine: a tile is read before it is written)
    bool al = true;
    for (int i = 0; i < 4; ++i) al = al && (reinterpret_cast<uintptr_t>(ptrs[i]) % 16 == 0);
    const int lpr = (int)(a.d * sizeof(IO) / 16);
    if (al && (size_t)lpr * 16 == a.d * sizeof(IO) && (lpr == 8 || lpr == 16 || lpr == 32) && a.rows >= 4 * kBkTok) {
        if (lpr == 8) return fwd_bulk<IO, 8>(a, st);
        if (lpr == 16) return fwd_bulk<IO, 16>(a, st);
        return fwd_bulk<IO, 32>(a, st);
    }
    const int grid = grid_for(a.rows, kPrTokens);
    return dispatch<IO, PrepareArgs>(s, [&](auto v, auto np) {
        prepare_fwd_kernel<IO, decltype(v)::value, decltype(np)::value><<<grid, kPrThreads, 0, st>>>(a);
        return (int)cudaGetLastError();
    });
}
template <typename IO> int bwd_io(const PrepareBwdArgs& a, cudaStream_t st) {
    const void* ptrs[6] = {a.f.q_raw, a.f.k_raw, a.dq, a.dk, a.dq_raw, a.dk_raw};
    const Shape s = pick_shape(a.f.d, (int)sizeof(IO), ptrs, 6);
    bool al = true;
    for (int i = 0; i < 6; ++i) al = al && (reinterpret_cast<uintptr_t>(ptrs[i]) % 16 == 0);
    const int lpr = (int)(a.f.d * sizeof(IO) / 16);
    if (al && (size_t)lpr * 16 == a.f.d * sizeof(IO) && (lpr == 8 || lpr == 16 || lpr == 32) && a.f.rows >= 4 * kBkTok) {
        if (lpr == 8) return bwd_bulk<IO, 8>(a, st);
        if (lpr == 16) return bwd_bulk<IO, 16>(a, st);
        return bwd_bulk<IO, 32>(a, st);
    }
    const int grid = grid_for(a.f.rows, 1);
    return dispatch<IO, PrepareBwdArgs>(s, [&](auto v, auto np) {
        prepare_bwd_kernel<IO, decltype(v)::value, decltype(np)::value><<<grid, kPrThreads, 0, st>>>(a);
        return (int)cudaGetLastError();
    });
}

}  // namespace

int prepare_fwd_launch(const PrepareArgs& a, int io_dtype, void* stream) {
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    return io_dtype == 0 ? fwd_io<float>(a, st) : fwd_io<__nv_bfloat16>(a, st);
}

int prepare_bwd_launch(const PrepareBwdArgs& a, int io_dtype, void* stream) {
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    return io_dtype == 0 ? bwd_io<float>(a, st) : bwd_io<__nv_bfloat16>(a, st);
}

}  // namespace e2ttt
