// Tensor-core forward for GELU-MLP fast weights, d = 128, h = 512, C = 64, bf16 I/O (sm_100a).
//
// One cluster of 4 CTAs per sequence; CTA c owns hidden units [128c, 128c+128): rows of W1, columns of W2.
// Everything that carries over from chunk to chunk stays on chip for the whole sequence:
//   - fp32 master copy of the CTA's W1/W2 slices: tensor memory columns [0,256).  The aggregation MMAs
//     accumulate -sum_t K^W_t grad_t straight into it (it is pre-scaled by the decay carry cw beforehand).
//   - fp32 master copy of the momentum slices: registers (each thread keeps the 2 x 128/NG elements it owns).
//   - bf16 operand copy of W1/W2: shared memory, refreshed once per chunk from the fp32 master.
// Per chunk (Algorithm 1), rows = tokens (64 keys then 64 queries), all GEMMs on tcgen05 with TMEM accumulators:
//   G1  Z = [K;Q] W1c^T          G2  Upart = gelu(Z) W2c^T      -> cross-CTA sum of Upart through DSMEM (each CTA
//   owns 32 token rows: LN, output rows o = q + LN(u), or e = k + LN(u) - v and pu = dL/du), pu rows broadcast
//   G3  Pa = Pu W2c, Pz = Pa * gelu'(Z)
//   aggregations (contraction over the 64 tokens, MN-major operands):
//       W1c -= (kW*Pz)^T K    M1acc = -(kM*Pz)^T K    W2c -= Pu^T (kW*Ak)    M2acc = -Pu^T (kM*Ak)
//   state pass: W = Wacc + cm M0;  M = cb M0 + Macc;  bf16(W) -> shared;  cw_next W -> TMEM.
// Every wait on an mbarrier is bounded (sm100.cuh); a wait that gives up is reported through the status word.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "simt_common.cuh"
#include "sm100.cuh"
#include "tc_fwd.h"

namespace e2ttt {
using namespace sm100;

#ifdef TC_PROFILE
// Debug build only: cycle stamps of thread 0 of CTA 0 at the phase boundaries of the first 64 chunks.
__device__ long long g_tc_prof[4 * 32 * 16];
#define PROF(i)                                                                                          \
    do {                                                                                                 \
        if ((threadIdx.x == 0 || threadIdx.x == 64) && (blockIdx.x == 0 || blockIdx.x == 2) && r < 32)    \
            g_tc_prof[(((blockIdx.x >> 1) * 2 + (threadIdx.x >> 6)) * 32 + r) * 16 + (i)] = clock64();    \
    } while (0)
#else
#define PROF(i)
#endif

namespace {

constexpr int D = 128, HC = 128, C = 64, NC = 4;
constexpr int NG = TC_NG;                // column groups per TMEM lane quadrant
constexpr int NTHREADS = 128 * NG;
constexpr int CW = 128 / NG;             // accumulator columns a thread owns in a 128-column region
constexpr int NB = CW / 16;              // 16-column batches per thread

// TMEM columns
constexpr uint32_t T_W1 = 0, T_W2 = 128, T_R0 = 256, T_R1 = 384;

struct Scalars {
    float kW[C], kM[C];
    float cw, cm, cb, pad;
};

struct __align__(1024) Smem {
    uint8_t W1[2][16384];  // bf16 W1c  [128 j][64 i] per slab (i = 64 s ..)         K-major B of G1
    uint8_t W2[2][16384];  // bf16 W2c  [128 i][64 j] per slab (j = 64 s ..)         K-major B of G2, MN-major B of G3
    uint8_t X[2][16384];   // [128 tokens][64 i] per slab; rows 0..63 keys, 64..127 queries (TMA)
    uint8_t A[2][16384];   // bf16 gelu(Z) [128 tokens][64 j] per slab               K-major A of G2
    uint8_t AkW[2][8192];  // kW_t gelu(Zk) [64 t][64 j] per slab                    MN-major B of the W2 aggregation
    uint8_t AkM[2][8192];  // kM_t gelu(Zk)
    uint8_t Pu[2][8192];   // bf16 pu [64 t][64 i] per slab                          K-major A of G3, MN-major A of the W2 aggregations
    uint8_t PzW[2][8192];  // kW_t pz [64 t][64 j] per slab                          MN-major A of the W1 aggregation; staging slot 0
    uint8_t PzM[2][8192];  // kM_t pz                                                 staging slot 1
    uint8_t Stage2[16384]; // staging slot 2
    Scalars sc[2];
    uint64_t bar_x, bar_g1, bar_g2, bar_g3, bar_agg, bar_agg2, bar_ak, bar_v, bar_ksent, bar_partK, bar_partQ, bar_pu, bar_credit, bar_rs;
    uint32_t tmem_base;
    int dead;
};

__device__ __forceinline__ uint64_t desc_k(uint32_t base, uint32_t slab_stride, int k) {
    return make_smem_desc(base + (uint32_t)(k >> 2) * slab_stride + (uint32_t)(k & 3) * 32u, 16, 1024);
}
__device__ __forceinline__ uint64_t desc_mn(uint32_t base, uint32_t slab_stride, int k) {
    return make_smem_desc(base + (uint32_t)k * 2048u, slab_stride, 1024);
}

// Suffix scans of one 64-token chunk by one warp (two tokens per lane), same recurrences as the SIMT path:
// a step is the map (bt, gt, S) -> (beta bt, gamma gt, beta S + gamma gt); suffix composites by warp shuffles.
__device__ void tc_chunk_scalars(const float* eta, const float* beta, const float* gamma, Scalars* out) {
    const int lane = threadIdx.x & 31;
    ScanMap<float> e0, e1, id;
    id.B = 1.0f; id.G = 1.0f; id.X = 0.0f;
    e0.B = beta[2 * lane]; e0.G = gamma[2 * lane]; e0.X = e0.G;
    e1.B = beta[2 * lane + 1]; e1.G = gamma[2 * lane + 1]; e1.X = e1.G;
    const ScanMap<float> loc1 = e1;                 // tokens 2l+1 .. of this lane
    const ScanMap<float> loc0 = compose(e0, loc1);  // tokens 2l ..   of this lane
    ScanMap<float> incl = loc0;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        ScanMap<float> o;
        o.B = __shfl_down_sync(0xffffffffu, incl.B, off);
        o.G = __shfl_down_sync(0xffffffffu, incl.G, off);
        o.X = __shfl_down_sync(0xffffffffu, incl.X, off);
        if (lane + off < 32) incl = compose(incl, o);
    }
    ScanMap<float> excl;
    excl.B = __shfl_down_sync(0xffffffffu, incl.B, 1);
    excl.G = __shfl_down_sync(0xffffffffu, incl.G, 1);
    excl.X = __shfl_down_sync(0xffffffffu, incl.X, 1);
    if (lane == 31) excl = id;
    // token index 2l sees the state after tokens 2l+1.., token 2l+1 the state after the later lanes' tokens
    const ScanMap<float> f1 = compose(loc1, excl);
    const float et0 = eta[2 * lane], et1 = eta[2 * lane + 1];
    out->kW[2 * lane] = et0 * (f1.B + f1.X);
    out->kM[2 * lane] = et0 * f1.B;
    out->kW[2 * lane + 1] = et1 * (excl.B + excl.X);
    out->kM[2 * lane + 1] = et1 * excl.B;
    if (lane == 0) {
        const ScanMap<float> f0 = compose(loc0, excl);
        out->cw = f0.G;
        out->cb = f0.B;
        out->cm = e0.B * (f1.B + f1.X);  // beta_1 S_1
    }
}

// GELU on the bf16 path: the tanh form g(z) = 0.5 z (1 + tanh(u)), u = sqrt(2/pi) (z + 0.044715 z^3), with the
// hardware tanh (6 FMA-pipe instructions and one MUFU), and its exact derivative
// g'(z) = 0.5 (1 + T) + 0.5 z (1 - T^2) u'(z).  g differs from z Phi(z) by at most 4.7e-4 absolute and g' from
// Phi(z) + z phi(z) by at most 8.7e-4 (plus 2^-11 relative from tanh.approx); both values are rounded to bf16 right
// after (half an ulp = 2^-9 relative).  The fp32/fp64 SIMT path keeps the exact erf form.
__device__ __forceinline__ float fast_tanh(float x) {
    float t;
    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(x));
    return t;
}
__device__ __forceinline__ float gelu_only(float z) {
    const float z2 = z * z;
    const float t = fast_tanh(z * fmaf(0.0356774081f, z2, 0.7978845608f));
    const float hz = 0.5f * z;
    return fmaf(hz, t, hz);
}
__device__ __forceinline__ float gelu_fast(float z, float& dgelu) {
    const float z2 = z * z;
    const float t = fast_tanh(z * fmaf(0.0356774081f, z2, 0.7978845608f));
    const float hz = 0.5f * z;
    const float du = fmaf(0.1070322243f, z2, 0.7978845608f);  // u'(z)
    dgelu = fmaf(hz * fmaf(-t, t, 1.0f), du, fmaf(0.5f, t, 0.5f));
    return fmaf(hz, t, hz);
}

// Staging slot for partial sums: 32 rows x 128 fp32, kept as 16-byte pieces.  Piece c4 (4 columns) of row r sits at
// piece index c4 * 32 + (r ^ ((c4 >> 1) & 15)): the 16 lanes that send one piece of 16 neighbouring rows write 256
// contiguous bytes (DSMEM moves whole segments; scattered 16-byte stores cost several times the bandwidth), and the
// layer-norm readers (16 threads per row, pieces 2cg and 2cg+1) spread over all banks.
__device__ __forceinline__ uint32_t stage_offset(uint32_t c4, uint32_t r) {
    return (c4 * 32u + (r ^ ((c4 >> 1) & 15u))) << 4;
}

// 16 bf16 (32 bytes) = two 16-byte chunks into a swizzled slab row
__device__ __forceinline__ void st_slab16(uint8_t* slab, int row, int col0, const float (&v)[16]) {
    const int c = col0 >> 3;
    uint4 a, b;
    a.x = pack_bf16(v[0], v[1]); a.y = pack_bf16(v[2], v[3]); a.z = pack_bf16(v[4], v[5]); a.w = pack_bf16(v[6], v[7]);
    b.x = pack_bf16(v[8], v[9]); b.y = pack_bf16(v[10], v[11]); b.z = pack_bf16(v[12], v[13]); b.w = pack_bf16(v[14], v[15]);
    *reinterpret_cast<uint4*>(slab + row * 128 + (((c) ^ (row & 7)) << 4)) = a;
    *reinterpret_cast<uint4*>(slab + row * 128 + (((c + 1) ^ (row & 7)) << 4)) = b;
}

// PAD = false: the native 128 x 512 shape, every mask folds away.  PAD = true: d and h come from the arguments.
// NORM = true: post-chunk normalisation - after the state transition every row of W1 and of W2 is rescaled to its
// target norm.  A row of W1c lives in one CTA (its 128 columns spread over the 4 column-group warps); a row of W2
// spans the 4 CTAs, so its sum of squares crosses the cluster once per chunk.
template <bool PAD, bool NORM>
__global__ void __launch_bounds__(NTHREADS, 1)
tc_fwd_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ,
              const __grid_constant__ CUtensorMap tmV, const TcFwdArgs a) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    Smem& s = *reinterpret_cast<Smem*>(smem_raw);
    if ((smem_u32(smem_raw) & 1023u) != 0u) {  // the swizzled tiles need a 1024-byte aligned base: refuse to run otherwise
        if (threadIdx.x == 0) atomicCAS(a.status, 0, 99);
        return;
    }

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int q = warp & 3;          // TMEM lane quadrant
    const int g = warp >> 2;         // column group
    const int row = 32 * q + lane;   // TMEM lane this thread reads
    const int c0 = CW * g;           // first of its columns inside a 128-column region
    const uint32_t me = cluster_ctarank();
    const int seq = blockIdx.x / NC;
    const int issuer_warp = 2;  // a warp of quadrant 2: free while quadrants 0/1 produce the backward-only operands
    const bool is_issuer = (warp == issuer_warp) && (lane == 0);
    const int L = a.L, nchunks = L / C;
    WaitCtx wc{&s.dead, a.status};

    // Real shape: de x he.  Columns >= de of every token tile and hidden units >= he are zero padding: they stay
    // exactly zero through every product, so only the layer norm (divisor, masks) and the global I/O know about them.
    const int de = PAD ? a.d : D, he = PAD ? a.h : NC * HC;
    const size_t dh = (size_t)de * he;
    const bool cta_real = HC * (int)me < he;  // this CTA's 128 hidden units exist
    const float inv_d = 1.0f / (float)de;
    // normalisation targets of this thread's rows: hidden unit 128 me + row of W1, output row `row` of W2
    const float tgt1 = (NORM && cta_real) ? a.norm1[(size_t)seq * he + HC * me + row] : 0.0f;
    const float tgt2 = (NORM && row < de) ? a.norm2[(size_t)seq * de + row] : 0.0f;
    __nv_bfloat16* go = a.o + (size_t)seq * L * de;
    const float* eta = a.eta + (size_t)seq * L;
    const float* beta = a.beta + (size_t)seq * L;
    const float* gamma = a.gamma + (size_t)seq * L;

    if (tid == 0) {
        s.dead = 0;
        mbar_init(&s.bar_x, 1);
        mbar_init(&s.bar_g1, 1);
        mbar_init(&s.bar_g2, 1);
        mbar_init(&s.bar_g3, 1);
        mbar_init(&s.bar_agg, 1);
        mbar_init(&s.bar_agg2, 1);
        mbar_init(&s.bar_ak, 2 * NG);
        mbar_init(&s.bar_v, 1);
        mbar_init(&s.bar_partK, 1);  // + 3 x 8 KB of peer partial sums (key rows) per chunk
        mbar_init(&s.bar_partQ, 1);  // + 3 x 8 KB (query rows)
        mbar_init(&s.bar_ksent, 2 * NG);
        mbar_init(&s.bar_pu, 1);    // + 16 KB of pu rows per chunk
        mbar_init(&s.bar_credit, 3);
        mbar_init(&s.bar_rs, 1);    // + 3 x 512 B of peer row sums per chunk (normalisation only)
        fence_mbar_init();
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmV);
    }
    if (warp == 0) { tmem_alloc(&s.tmem_base, 512); tmem_relinquish(); }
    if (warp == 1) tc_chunk_scalars(eta, beta, gamma, &s.sc[0]);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tb = s.tmem_base;
    const uint32_t lane_addr = tb + ((uint32_t)(32 * q) << 16);

    // ---- load the state: fp32 master of W -> TMEM (pre-scaled by the first decay carry) and bf16 -> shared; M -> registers
    float M1[CW], M2[CW];
    {
        const float cw0 = s.sc[0].cw;
        const size_t head = (size_t)seq * dh;
        // W1c[j][i]: global W1 [h][d], row 128 me + j
        const float* w1 = a.W1_init + head + ((size_t)(HC * me) + row) * de + c0;
        const float* m1 = a.M1_init ? a.M1_init + head + ((size_t)(HC * me) + row) * de + c0 : nullptr;
        // W2c[i][j]: global W2 [d][h], row i, column 128 me + j
        const float* w2 = a.W2_init + head + (size_t)row * he + HC * me + c0;
        const float* m2 = a.M2_init ? a.M2_init + head + (size_t)row * he + HC * me + c0 : nullptr;
        const bool real2 = cta_real && row < de;  // this thread's W2 row exists
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            float w[16];
            uint32_t st[16];
            const bool real1 = cta_real && c0 + 16 * b < de;  // these 16 columns of W1 exist
#pragma unroll
            for (int j = 0; j < 16; j += 4) {
                const float4 x = real1 ? *reinterpret_cast<const float4*>(w1 + 16 * b + j) : make_float4(0.f, 0.f, 0.f, 0.f);
                w[j] = x.x; w[j + 1] = x.y; w[j + 2] = x.z; w[j + 3] = x.w;
            }
#pragma unroll
            for (int j = 0; j < 16; ++j) { st[j] = __float_as_uint(cw0 * w[j]); M1[16 * b + j] = (m1 && real1) ? m1[16 * b + j] : 0.0f; }
            tmem_st16(lane_addr + T_W1 + c0 + 16 * b, st);
            st_slab16(s.W1[(c0 + 16 * b) >> 6], row, (c0 + 16 * b) & 63, w);
            float* ck = a.ckpt ? a.ckpt + (size_t)seq * a.ckpt_seq_stride : nullptr;  // chunk-start state of chunk 0
            if (ck && real1) {
                const size_t o1 = ((size_t)(HC * me) + row) * de + c0 + 16 * b;
#pragma unroll
                for (int j = 0; j < 16; j += 4) {
                    *reinterpret_cast<float4*>(ck + o1 + j) = make_float4(w[j], w[j + 1], w[j + 2], w[j + 3]);
                    *reinterpret_cast<float4*>(ck + 2 * dh + o1 + j) =
                        make_float4(M1[16 * b + j], M1[16 * b + j + 1], M1[16 * b + j + 2], M1[16 * b + j + 3]);
                }
            }
#pragma unroll
            for (int j = 0; j < 16; j += 4) {
                const float4 x = real2 ? *reinterpret_cast<const float4*>(w2 + 16 * b + j) : make_float4(0.f, 0.f, 0.f, 0.f);
                w[j] = x.x; w[j + 1] = x.y; w[j + 2] = x.z; w[j + 3] = x.w;
            }
#pragma unroll
            for (int j = 0; j < 16; ++j) { st[j] = __float_as_uint(cw0 * w[j]); M2[16 * b + j] = (m2 && real2) ? m2[16 * b + j] : 0.0f; }
            tmem_st16(lane_addr + T_W2 + c0 + 16 * b, st);
            st_slab16(s.W2[(c0 + 16 * b) >> 6], row, (c0 + 16 * b) & 63, w);
            if (ck && real2) {
                const size_t o2 = (size_t)row * he + HC * me + c0 + 16 * b;
#pragma unroll
                for (int j = 0; j < 16; j += 4) {
                    *reinterpret_cast<float4*>(ck + dh + o2 + j) = make_float4(w[j], w[j + 1], w[j + 2], w[j + 3]);
                    *reinterpret_cast<float4*>(ck + 3 * dh + o2 + j) =
                        make_float4(M2[16 * b + j], M2[16 * b + j + 1], M2[16 * b + j + 2], M2[16 * b + j + 3]);
                }
            }
        }
        tmem_wait_st();
    }
    // token tile of the chunk that starts at global row y: keys into rows 0..63, queries into rows 64..127
    auto load_tokens = [&](int y) {
        mbar_expect_tx(&s.bar_x, de == 128 ? 32768u : 16384u);
        tma_load_2d(s.X[0], &tmK, 0, y, &s.bar_x);
        tma_load_2d(s.X[0] + 8192, &tmQ, 0, y, &s.bar_x);
        if (de == 128) {
            tma_load_2d(s.X[1], &tmK, 64, y, &s.bar_x);
            tma_load_2d(s.X[1] + 8192, &tmQ, 64, y, &s.bar_x);
        }
    };
    if (de < 128)  // the padded half of the token tile is never loaded: zero it once
        for (int i = tid; i < 16384 / 16; i += NTHREADS) reinterpret_cast<uint4*>(s.X[1])[i] = make_uint4(0u, 0u, 0u, 0u);
    if (is_issuer) load_tokens(seq * L);
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    // every CTA's barriers are initialised before any peer may arrive on them
    cluster_sync();
    tc_fence_after_sync();

    const uint32_t id_kk = make_idesc(128, 128, false, false);
    const uint32_t id_kmn = make_idesc(128, 128, false, true);
    const uint32_t id_agg = make_idesc(128, 128, true, true) | (1u << 13);  // negate A: G_t is minus the gradient

    // G1 of chunk `chunk` (issuer thread only): needs that chunk's tokens in X and the refreshed bf16 W1
    auto issue_g1 = [&](int chunk) {
        mbar_wait_one(&s.bar_x, (uint32_t)(chunk & 1), wc, 100 + 1);
        tc_fence_after_sync();
#pragma unroll
        for (int k = 0; k < 8; ++k)
            umma_bf16(tb + T_R0, desc_k(smem_u32(s.X[0]), 16384, k), desc_k(smem_u32(s.W1[0]), 16384, k), id_kk, k > 0);
        umma_commit(&s.bar_g1);
    };
    if (is_issuer) issue_g1(0);
    __syncwarp();

    for (int r = 0; r < nchunks; ++r) {
        const uint32_t ph = (uint32_t)(r & 1);
        const Scalars& sc = s.sc[r & 1];
        const int tok0 = r * C;

        // scalars of the next chunk (suffix scans over its gates), by a warp that is not the issuer
        if (warp == 3 + 4 * (NG - 1) && r + 1 < nchunks) {
            tc_chunk_scalars(eta + tok0 + C, beta + tok0 + C, gamma + tok0 + C, &s.sc[(r + 1) & 1]);
        }
        PROF(0);
        // ---------------- G1: Z = X W1c^T -> R0 (issued at the end of the previous iteration / before the loop)
        if (is_issuer) {
            if (r + 1 < nchunks) {
                // the next chunk's tokens: into L2 now, so that the loads issued at the end of this chunk are short
                const int y = seq * L + tok0 + C;
                tma_prefetch_l2_2d(&tmK, 0, y);
                tma_prefetch_l2_2d(&tmQ, 0, y);
                tma_prefetch_l2_2d(&tmV, 0, y + 16 * (int)me);
                if (de == 128) {
                    tma_prefetch_l2_2d(&tmK, 64, y);
                    tma_prefetch_l2_2d(&tmQ, 64, y);
                    tma_prefetch_l2_2d(&tmV, 64, y + 16 * (int)me);
                }
            }
            mbar_expect_tx(&s.bar_partK, 3 * 8192);  // this chunk's incoming partial sums and pu rows
            mbar_expect_tx(&s.bar_partQ, 3 * 8192);
            mbar_expect_tx(&s.bar_pu, 16384);
            if (NORM) mbar_expect_tx(&s.bar_rs, 3 * 512);
        }
        mbar_wait(&s.bar_g1, ph, wc, 100 + 2);
        PROF(1);
        __syncwarp();
        tc_fence_after_sync();
        // epilogue: a = gelu(z) -> A (bf16); for key rows also kW a, kM a and gelu'(z) (kept in TMEM over z)
        // a = gelu(z) -> A (bf16) for all 128 rows: all that G2 needs
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            uint32_t z[16];
            tmem_ld16(lane_addr + T_R0 + c0 + 16 * b, z);
            tmem_wait_ld();
            float av[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) av[j] = gelu_only(__uint_as_float(z[j]));
            const int col = c0 + 16 * b;
            st_slab16(s.A[col >> 6], row, col & 63, av);
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        __syncthreads();
        PROF(2);
        // ---------------- G2: Upart = A W2c^T -> R1
        if (is_issuer) {
            tc_fence_after_sync();
#pragma unroll
            for (int k = 0; k < 8; ++k)
                umma_bf16(tb + T_R1, desc_k(smem_u32(s.A[0]), 16384, k), desc_k(smem_u32(s.W2[0]), 16384, k), id_kk, k > 0);
            umma_commit(&s.bar_g2);
        }
        __syncwarp();
        mbar_wait(&s.bar_g2, ph, wc, 100 + 3);
        if (is_issuer) {
            // the 16 value rows this CTA needs for its key rows: into the gelu tile's first slab, dead once G2 is done
            mbar_expect_tx(&s.bar_v, de == 128 ? 4096u : 2048u);
            const int y = seq * L + tok0 + 16 * (int)me;
            tma_load_2d(s.A[0], &tmV, 0, y, &s.bar_v);
            if (de == 128) tma_load_2d(s.A[0] + 2048, &tmV, 64, y, &s.bar_v);
        }
        __syncwarp();
        PROF(3);
        __syncwarp();
        tc_fence_after_sync();
        // Row ownership: CTA c normalises key tokens 16c..16c+15 and query tokens 16c..16c+15, so every CTA carries
        // the same mix of work.  TMEM lane 32q+l holds key token 32q+l (q < 2) or query token 32(q-2)+l.
        auto send_rows = [&](uint64_t* bar_local) {
            const uint32_t owner = 2u * ((uint32_t)q & 1u) + ((uint32_t)lane >> 4);
            const uint32_t srow = ((q < 2) ? 0u : 16u) + ((uint32_t)lane & 15u);  // row inside the owner's staging slot
            const bool mine = owner == me;
            uint32_t dst_base, dst_bar = 0;
            if (mine) {
                dst_base = smem_u32(s.A[1]);  // own rows: the gelu tile is dead once G2 has completed
            } else {
                const uint32_t slot = (me - owner - 1u) & 3u;  // where the owner keeps what comes from me
                const uint8_t* p = (slot == 0) ? s.PzW[0] : (slot == 1) ? s.PzM[0] : s.Stage2;
                dst_base = map_to_cta(smem_u32(p), owner);
                dst_bar = map_to_cta(smem_u32(bar_local), owner);
            }
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                uint32_t u[16];
                tmem_ld16(lane_addr + T_R1 + c0 + 16 * b, u);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 16; j += 4) {
                    const uint32_t c4 = (uint32_t)((c0 + 16 * b + j) >> 2);
                    const uint32_t dst = dst_base + stage_offset(c4, srow);
                    if (mine) st_cluster_v4_b32(dst, u[j], u[j + 1], u[j + 2], u[j + 3]);
                    else st_async_v4(dst, u[j], u[j + 1], u[j + 2], u[j + 3], dst_bar);
                }
            }
        };

        // What only the inner backward needs, for the key rows (the warps of TMEM quadrants 0 and 1): kW a, kM a
        // (operands of the W2 aggregations) and gelu'(z), which replaces z in TMEM.  Runs while pu travels.
        auto backward_extras = [&]() {
            const float kw = sc.kW[row], km = sc.kM[row];
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                uint32_t z[16];
                tmem_ld16(lane_addr + T_R0 + c0 + 16 * b, z);
                tmem_wait_ld();
                float aw[16], am[16];
                uint32_t dg[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    float d1;
                    const float av = gelu_fast(__uint_as_float(z[j]), d1);
                    dg[j] = __float_as_uint(d1);
                    aw[j] = kw * av;
                    am[j] = km * av;
                }
                const int col = c0 + 16 * b;
                st_slab16(s.AkW[col >> 6], row, col & 63, aw);
                st_slab16(s.AkM[col >> 6], row, col & 63, am);
                tmem_st16(lane_addr + T_R0 + col, dg);
            }
            tmem_wait_st();
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(&s.bar_ak);
        };

        // Layer norm on the 16 key rows (warps of quadrants 0/1) or the 16 query rows (quadrants 2/3) this CTA owns:
        // 16 threads per row, 8 columns each.
        auto layer_norm = [&](const bool key_rows) {
            constexpr int TPR = NTHREADS / 32, CPT = 128 / TPR;  // threads per row, columns per thread
            static_assert(TPR == 16, "row mapping below assumes two rows per warp");
            // staging rows 0..15: key tokens, 16..31: query tokens
            const int lrow = (key_rows ? 0 : 16) + 2 * ((q & 1) + 2 * g) + (lane >> 4);
            const int cg = lane & 15;
            const int t = 16 * (int)me + (lrow & 15);    // token inside the chunk
            const int xrow = key_rows ? t : 64 + t;      // its row in the X tile
            const int col0 = CPT * cg;
            const size_t off = (size_t)(tok0 + t) * de + col0;
            const bool real = col0 < de;  // this thread's 8 columns exist (padding columns carry exact zeros)
            uint4 vraw[CPT / 8], xraw[CPT / 8];
#pragma unroll
            for (int ch = 0; ch < CPT / 8; ++ch) {
                const int c = ((col0 & 63) >> 3) + ch;
                xraw[ch] = *reinterpret_cast<const uint4*>(s.X[col0 >> 6] + xrow * 128 + ((c ^ (xrow & 7)) << 4));
            }
            mbar_wait<true>(key_rows ? &s.bar_partK : &s.bar_partQ, ph, wc, 100 + 5);
            if (key_rows) {
                mbar_wait(&s.bar_v, ph, wc, 100 + 11);
                const int lr = lrow & 15;
#pragma unroll
                for (int ch = 0; ch < CPT / 8; ++ch) {
                    const int c = ((col0 & 63) >> 3) + ch;
                    vraw[ch] = real ? *reinterpret_cast<const uint4*>(s.A[0] + (col0 >> 6) * 2048 + lr * 128 + ((c ^ (lr & 7)) << 4))
                                    : make_uint4(0u, 0u, 0u, 0u);
                }
            }
            float u[CPT];
#pragma unroll
            for (int j = 0; j < CPT; ++j) u[j] = 0.0f;
#pragma unroll
            for (int src = 0; src < NC; ++src) {  // fixed order: the sum does not depend on arrival order
                const uint32_t slot = ((uint32_t)src - me - 1u) & 3u;
                const uint8_t* p = (src == (int)me) ? s.A[1] : (slot == 0) ? s.PzW[0] : (slot == 1) ? s.PzM[0] : s.Stage2;
#pragma unroll
                for (int j = 0; j < CPT; j += 4) {
                    const int c4 = (col0 + j) >> 2;
                    const float4 x = *reinterpret_cast<const float4*>(p + stage_offset((uint32_t)c4, (uint32_t)lrow));
                    u[j] += x.x; u[j + 1] += x.y; u[j + 2] += x.z; u[j + 3] += x.w;
                }
            }
            auto row_sum = [&](float v) -> float {  // over the TPR lanes that share a row
#pragma unroll
                for (int o = TPR / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                return v;
            };
            float sum = 0.0f;
#pragma unroll
            for (int j = 0; j < CPT; ++j) sum += u[j];
            const float mu = row_sum(sum) * inv_d;
            float sq = 0.0f;
#pragma unroll
            for (int j = 0; j < CPT; ++j) { u[j] = real ? u[j] - mu : 0.0f; sq = fmaf(u[j], u[j], sq); }
            const float rstd = rsqrtf(row_sum(sq) * inv_d + a.eps);
#pragma unroll
            for (int j = 0; j < CPT; ++j) u[j] *= rstd;  // y (zero in the padding)
            if (key_rows) {
                // key rows: e = k + y - v, pu = rstd (e - mean(e) - y mean(e y))
                float e[CPT];
                float se = 0.0f, sey = 0.0f;
#pragma unroll
                for (int ch = 0; ch < CPT / 8; ++ch) {
                    const __nv_bfloat162* k2 = reinterpret_cast<const __nv_bfloat162*>(&xraw[ch]);
                    const __nv_bfloat162* v2 = reinterpret_cast<const __nv_bfloat162*>(&vraw[ch]);
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        const float2 kf = __bfloat1622float2(k2[x]), vf = __bfloat1622float2(v2[x]);
                        const int j = 8 * ch + 2 * x;
                        e[j] = kf.x + u[j] - vf.x;
                        e[j + 1] = kf.y + u[j + 1] - vf.y;
                    }
                }
#pragma unroll
                for (int j = 0; j < CPT; ++j) { se += e[j]; sey = fmaf(e[j], u[j], sey); }
                const float me_ = real ? row_sum(se) * inv_d : (row_sum(se), 0.0f);
                const float mey = row_sum(sey) * inv_d;
                    // broadcast the bf16 pu row piece to every CTA of the cluster
                uint32_t pk[CPT / 2];
#pragma unroll
                for (int j = 0; j < CPT; j += 2)
                    pk[j / 2] = pack_bf16(rstd * (e[j] - me_ - u[j] * mey), rstd * (e[j + 1] - me_ - u[j + 1] * mey));  // 0 in the padding
                const uint32_t pu_local = smem_u32(s.Pu[col0 >> 6]);
#pragma unroll
                for (uint32_t dst = 0; dst < NC; ++dst) {
                    const uint32_t base = map_to_cta(pu_local, dst) + (uint32_t)t * 128u;
                    const uint32_t bar = map_to_cta(smem_u32(&s.bar_pu), dst);
#pragma unroll
                    for (int ch = 0; ch < CPT / 8; ++ch) {
                        const uint32_t c = (uint32_t)(((col0 & 63) >> 3) + ch);
                        st_async_v4(base + ((c ^ ((uint32_t)t & 7u)) << 4), pk[4 * ch], pk[4 * ch + 1], pk[4 * ch + 2],
                                    pk[4 * ch + 3], bar);
                    }
                }
            } else {
                // query rows: o = q + y
#pragma unroll
                for (int ch = 0; ch < CPT / 8; ++ch) {
                    const __nv_bfloat162* q2 = reinterpret_cast<const __nv_bfloat162*>(&xraw[ch]);
                    uint4 ov;
                    uint32_t* o32 = reinterpret_cast<uint32_t*>(&ov);
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        const float2 qf = __bfloat1622float2(q2[x]);
                        o32[x] = pack_bf16(qf.x + u[8 * ch + 2 * x], qf.y + u[8 * ch + 2 * x + 1]);
                    }
                    if (real) *reinterpret_cast<uint4*>(go + off + 8 * ch) = ov;
                }
            }
        };

        // ---------------- cross-CTA sum of Upart, layer norm, pu broadcast
        // The key rows are on the critical path of the whole cluster, the query rows are not.  So the warps holding
        // key rows (quadrants 0/1) hand them to the network first, normalise this CTA's key rows as soon as the
        // peers' pieces are in, broadcast pu, and only then produce the backward-only operands; the warps holding
        // query rows (quadrants 2/3) send after the key rows have gone out, normalise the query rows, write o.
        if (r > 0) mbar_wait<true>(&s.bar_credit, (uint32_t)((r - 1) & 1), wc, 100 + 4);
        if (q < 2) {
            send_rows(&s.bar_partK);
            __syncwarp();
            if (lane == 0) mbar_arrive(&s.bar_ksent);
            asm volatile("bar.sync 4, %0;" ::"r"(64 * NG) : "memory");  // this CTA's own key rows are staged
            PROF(4);
            layer_norm(true);
            PROF(5);
            backward_extras();
            PROF(6);
            // the Pz tiles (G3 epilogue, below) overlay staging slots: wait until the query-row readers are done too
            asm volatile("bar.sync 3, %0;" ::"r"(128 * NG) : "memory");
        } else {
            mbar_wait(&s.bar_ksent, ph, wc, 100 + 12);
            send_rows(&s.bar_partQ);
            asm volatile("bar.sync 5, %0;" ::"r"(64 * NG) : "memory");  // own query rows staged; R1 fully read
            PROF(4);
            layer_norm(false);
            PROF(5);
            asm volatile("bar.arrive 3, %0;" ::"r"(128 * NG) : "memory");
            PROF(6);
        }
        PROF(7);
        // ---------------- G3: Pa = Pu W2c -> R1 ; then the W2 aggregation that needs nothing else
        if (is_issuer) {
            mbar_wait_one<true>(&s.bar_pu, ph, wc, 100 + 6);
            asm volatile("fence.proxy.async;" ::: "memory");
            tc_fence_after_sync();
#pragma unroll
            for (int k = 0; k < 8; ++k)
                umma_bf16(tb + T_R1, desc_k(smem_u32(s.Pu[0]), 8192, k), desc_mn(smem_u32(s.W2[0]), 16384, k), id_kmn, k > 0);
            umma_commit(&s.bar_g3);
            mbar_wait_one(&s.bar_ak, ph, wc, 100 + 10);  // kW a / kM a written by the quadrant-0/1 warps
            tc_fence_after_sync();
#pragma unroll
            for (int k = 0; k < 4; ++k)
                umma_bf16(tb + T_W2, desc_mn(smem_u32(s.Pu[0]), 8192, k), desc_mn(smem_u32(s.AkW[0]), 8192, k), id_agg, true);
        }
        mbar_wait(&s.bar_g3, ph, wc, 100 + 7);
        PROF(8);
        __syncwarp();
        tc_fence_after_sync();
        if (row < C) {
            const float kw = sc.kW[row], km = sc.kM[row];
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                uint32_t pa[16], dg[16];
                tmem_ld16(lane_addr + T_R1 + c0 + 16 * b, pa);
                tmem_ld16(lane_addr + T_R0 + c0 + 16 * b, dg);
                tmem_wait_ld();
                float pw[16], pm[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float pz = __uint_as_float(pa[j]) * __uint_as_float(dg[j]);
                    pw[j] = kw * pz;
                    pm[j] = km * pz;
                }
                const int col = c0 + 16 * b;
                st_slab16(s.PzW[col >> 6], row, col & 63, pw);
                st_slab16(s.PzM[col >> 6], row, col & 63, pm);
            }
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        __syncthreads();
        PROF(9);
        // ---------------- remaining aggregations, in two groups so that the state pass can start on W1 early
        if (is_issuer) {
            tc_fence_after_sync();
#pragma unroll
            for (int k = 0; k < 4; ++k)
                umma_bf16(tb + T_W1, desc_mn(smem_u32(s.PzW[0]), 8192, k), desc_mn(smem_u32(s.X[0]), 16384, k), id_agg, true);
#pragma unroll
            for (int k = 0; k < 4; ++k)
                umma_bf16(tb + T_R0, desc_mn(smem_u32(s.PzM[0]), 8192, k), desc_mn(smem_u32(s.X[0]), 16384, k), id_agg, k > 0);
            umma_commit(&s.bar_agg);
            PROF(14);
#pragma unroll
            for (int k = 0; k < 4; ++k)
                umma_bf16(tb + T_R1, desc_mn(smem_u32(s.Pu[0]), 8192, k), desc_mn(smem_u32(s.AkM[0]), 8192, k), id_agg, k > 0);
            umma_commit(&s.bar_agg2);
            PROF(15);
        }
        const bool last = (r + 1 == nchunks);
        const float cm = sc.cm, cb = sc.cb;
        const float cwn = last ? 1.0f : s.sc[(r + 1) & 1].cw;
        const size_t head = (size_t)seq * dh;

        mbar_wait(&s.bar_agg, ph, wc, 100 + 8);
        PROF(10);
        tc_fence_after_sync();
        if (is_issuer && !last) {
            // the W1 aggregations were the last readers of the key tile: the next chunk's tokens may land in X
            load_tokens(seq * L + tok0 + C);
        }
        __syncwarp();
        // ---------------- state pass, W1 half (Algorithm 1 lines 6-7), while the M2 aggregation still runs
        float ss1 = 0.0f;
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            const int col = c0 + 16 * b;
            uint32_t wa[16], ma[16], st[16];
            float wn[16];
            tmem_ld16(lane_addr + T_W1 + col, wa);
            tmem_ld16(lane_addr + T_R0 + col, ma);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const float m0 = M1[16 * b + j];
                wn[j] = __uint_as_float(wa[j]) + cm * m0;
                M1[16 * b + j] = cb * m0 + __uint_as_float(ma[j]);
                st[j] = __float_as_uint(NORM ? wn[j] : cwn * wn[j]);
                if (NORM) ss1 = fmaf(wn[j], wn[j], ss1);
            }
            tmem_st16(lane_addr + T_W1 + col, st);
            if (!NORM) {
                st_slab16(s.W1[col >> 6], row, col & 63, wn);
                if ((last || a.ckpt) && cta_real && col < de) {  // final state, or the next chunk's start state for the backward
                    const size_t off = ((size_t)(HC * me) + row) * de + col;
                    float* ck = last ? nullptr : a.ckpt + (size_t)seq * a.ckpt_seq_stride + (size_t)(r + 1) * 4 * dh;
                    float* wf = last ? a.W1_final + head + off : ck + off;
                    float* mf = last ? a.M1_final + head + off : ck + 2 * dh + off;
#pragma unroll
                    for (int j = 0; j < 16; j += 4) {
                        *reinterpret_cast<float4*>(wf + j) = make_float4(wn[j], wn[j + 1], wn[j + 2], wn[j + 3]);
                        *reinterpret_cast<float4*>(mf + j) =
                            make_float4(M1[16 * b + j], M1[16 * b + j + 1], M1[16 * b + j + 2], M1[16 * b + j + 3]);
                    }
                }
            }
        }
        if (NORM) {
            // row sums of squares: the four column-group warps of a row meet in shared memory (the Pz tile is dead)
            float* rs = reinterpret_cast<float*>(s.PzW[0]);  // [NG][128]
            rs[g * 128 + row] = ss1;
            tmem_wait_st();
            tc_fence_before_sync();
            __syncthreads();
            tc_fence_after_sync();
            float tot = 0.0f;
#pragma unroll
            for (int gg = 0; gg < NG; ++gg) tot += rs[gg * 128 + row];
            const float f = tgt1 / (sqrtf(tot) + a.norm_eps);
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                const int col = c0 + 16 * b;
                uint32_t wa[16], st[16];
                float wn[16];
                tmem_ld16(lane_addr + T_W1 + col, wa);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    wn[j] = __uint_as_float(wa[j]) * f;
                    st[j] = __float_as_uint(cwn * wn[j]);
                }
                tmem_st16(lane_addr + T_W1 + col, st);
                st_slab16(s.W1[col >> 6], row, col & 63, wn);
                if (cta_real && col < de) {
                    const size_t off = ((size_t)(HC * me) + row) * de + col;
                    if (last) {
#pragma unroll
                        for (int j = 0; j < 16; j += 4) {
                            *reinterpret_cast<float4*>(a.W1_final + head + off + j) = make_float4(wn[j], wn[j + 1], wn[j + 2], wn[j + 3]);
                            *reinterpret_cast<float4*>(a.M1_final + head + off + j) =
                                make_float4(M1[16 * b + j], M1[16 * b + j + 1], M1[16 * b + j + 2], M1[16 * b + j + 3]);
                        }
                    }
                    if (a.ckpt) {  // the state after this chunk: slot r + 1 (the last slot is the final state)
                        float* ck = a.ckpt + (size_t)seq * a.ckpt_seq_stride + (size_t)(r + 1) * 4 * dh;
#pragma unroll
                        for (int j = 0; j < 16; j += 4) {
                            *reinterpret_cast<float4*>(ck + off + j) = make_float4(wn[j], wn[j + 1], wn[j + 2], wn[j + 3]);
                            *reinterpret_cast<float4*>(ck + 2 * dh + off + j) =
                                make_float4(M1[16 * b + j], M1[16 * b + j + 1], M1[16 * b + j + 2], M1[16 * b + j + 3]);
                        }
                    }
                }
            }
            if (a.ckpt && g == 0 && cta_real)  // row norm before the normalisation, for the reverse pass
                a.rown[(size_t)seq * a.ckpt_seq_stride + ((size_t)r * 3 + 0) * (size_t)max(de, he) + HC * me + row] = sqrtf(tot);
        }
        tmem_wait_st();
        fence_proxy_async_smem();
        tc_fence_before_sync();
        __syncthreads();  // bf16 W1 is complete and R0 is free: the next chunk's G1 may run under the W2 half
        PROF(11);
        if (is_issuer && !last) issue_g1(r + 1);
        __syncwarp();

        mbar_wait(&s.bar_agg2, ph, wc, 100 + 9);
        PROF(12);
        tc_fence_after_sync();
        if (is_issuer) {
            // every reader of this chunk's staging / pu / scaled-activation buffers is done: peers may overwrite them
#pragma unroll
            for (uint32_t dst = 0; dst < NC; ++dst)
                if (dst != me) mbar_arrive_remote(map_to_cta(smem_u32(&s.bar_credit), dst));
        }
        __syncwarp();
        // ---------------- state pass, W2 half
        float ss2 = 0.0f;
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            const int col = c0 + 16 * b;
            uint32_t wa[16], ma[16], st[16];
            float wn[16];
            tmem_ld16(lane_addr + T_W2 + col, wa);
            tmem_ld16(lane_addr + T_R1 + col, ma);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const float m0 = M2[16 * b + j];
                wn[j] = __uint_as_float(wa[j]) + cm * m0;
                M2[16 * b + j] = cb * m0 + __uint_as_float(ma[j]);
                st[j] = __float_as_uint(NORM ? wn[j] : cwn * wn[j]);
                if (NORM) ss2 = fmaf(wn[j], wn[j], ss2);
            }
            tmem_st16(lane_addr + T_W2 + col, st);
            if (!NORM) {
                st_slab16(s.W2[col >> 6], row, col & 63, wn);
                if ((last || a.ckpt) && cta_real && row < de) {
                    const size_t off = (size_t)row * he + HC * me + col;
                    float* ck = last ? nullptr : a.ckpt + (size_t)seq * a.ckpt_seq_stride + (size_t)(r + 1) * 4 * dh;
                    float* wf = last ? a.W2_final + head + off : ck + dh + off;
                    float* mf = last ? a.M2_final + head + off : ck + 3 * dh + off;
#pragma unroll
                    for (int j = 0; j < 16; j += 4) {
                        *reinterpret_cast<float4*>(wf + j) = make_float4(wn[j], wn[j + 1], wn[j + 2], wn[j + 3]);
                        *reinterpret_cast<float4*>(mf + j) =
                            make_float4(M2[16 * b + j], M2[16 * b + j + 1], M2[16 * b + j + 2], M2[16 * b + j + 3]);
                    }
                }
            }
        }
        if (NORM) {
            // A row of W2 spans the cluster: the CTA's own sum of squares (over its four column-group warps) goes to
            // every CTA, each adds the four pieces in CTA order (the same number everywhere).  The kW a tile is dead.
            float* rs = reinterpret_cast<float*>(s.AkW[0]);          // [NG][128] this CTA's pieces
            float* got = reinterpret_cast<float*>(s.AkW[0]) + 1024;  // [NC][128] one row-sum vector per CTA
            rs[g * 128 + row] = ss2;
            tmem_wait_st();
            tc_fence_before_sync();
            __syncthreads();
            tc_fence_after_sync();
            if (warp == 0) {  // 32 lanes x 4 rows
                // a peer's receive area overlays an operand tile of its W2 aggregations: it is free once that peer
                // has seen them finish, which is what its credit of this chunk says
                mbar_wait<true>(&s.bar_credit, ph, wc, 100 + 14);
                float4 v;
                float* pv = reinterpret_cast<float*>(&v);
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    float t = 0.0f;
#pragma unroll
                    for (int gg = 0; gg < NG; ++gg) t += rs[gg * 128 + 4 * lane + x];
                    pv[x] = t;
                }
                const uint32_t local = smem_u32(got + me * 128 + 4 * lane);
                *reinterpret_cast<float4*>(got + me * 128 + 4 * lane) = v;
#pragma unroll
                for (uint32_t dst = 0; dst < NC; ++dst)
                    if (dst != me)
                        st_async_v4(map_to_cta(local, dst), __float_as_uint(v.x), __float_as_uint(v.y), __float_as_uint(v.z),
                                    __float_as_uint(v.w), map_to_cta(smem_u32(&s.bar_rs), dst));
            }
            __syncthreads();  // the CTA's own vector is in place
            mbar_wait<true>(&s.bar_rs, ph, wc, 100 + 13);
            float tot = 0.0f;
#pragma unroll
            for (uint32_t c = 0; c < NC; ++c) tot += got[c * 128 + row];
            const float f = tgt2 / (sqrtf(tot) + a.norm_eps);
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                const int col = c0 + 16 * b;
                uint32_t wa[16], st[16];
                float wn[16];
                tmem_ld16(lane_addr + T_W2 + col, wa);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    wn[j] = __uint_as_float(wa[j]) * f;
                    st[j] = __float_as_uint(cwn * wn[j]);
                }
                tmem_st16(lane_addr + T_W2 + col, st);
                st_slab16(s.W2[col >> 6], row, col & 63, wn);
                if (cta_real && row < de) {
                    const size_t off = (size_t)row * he + HC * me + col;
                    if (last) {
#pragma unroll
                        for (int j = 0; j < 16; j += 4) {
                            *reinterpret_cast<float4*>(a.W2_final + head + off + j) = make_float4(wn[j], wn[j + 1], wn[j + 2], wn[j + 3]);
                            *reinterpret_cast<float4*>(a.M2_final + head + off + j) =
                                make_float4(M2[16 * b + j], M2[16 * b + j + 1], M2[16 * b + j + 2], M2[16 * b + j + 3]);
                        }
                    }
                    if (a.ckpt) {
                        float* ck = a.ckpt + (size_t)seq * a.ckpt_seq_stride + (size_t)(r + 1) * 4 * dh;
#pragma unroll
                        for (int j = 0; j < 16; j += 4) {
                            *reinterpret_cast<float4*>(ck + dh + off + j) = make_float4(wn[j], wn[j + 1], wn[j + 2], wn[j + 3]);
                            *reinterpret_cast<float4*>(ck + 3 * dh + off + j) =
                                make_float4(M2[16 * b + j], M2[16 * b + j + 1], M2[16 * b + j + 2], M2[16 * b + j + 3]);
                        }
                    }
                }
            }
            if (a.ckpt && g == 0 && me == 0 && row < de)
                a.rown[(size_t)seq * a.ckpt_seq_stride + ((size_t)r * 3 + 1) * (size_t)max(de, he) + row] = sqrtf(tot);
        }
        tmem_wait_st();
        fence_proxy_async_smem();
        tc_fence_before_sync();
        __syncthreads();
        tc_fence_after_sync();
        PROF(13);
    }

    // no CTA leaves while a peer may still write into its shared memory or arrive on its barriers
    tc_fence_before_sync();
    cluster_sync();
    if (warp == 0) tmem_dealloc(tb, 512);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) != cudaSuccess ||
            qr != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// [rows][d] bf16 row-major, tiles of box_rows rows x 64 columns, 128-byte swizzle
bool make_token_map(CUtensorMap* tm, const void* base, size_t rows, unsigned box_rows, int d) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)d * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t es[2] = {1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

size_t tc_fwd_smem_bytes() { return sizeof(Smem); }

#ifdef TC_PROFILE
extern "C" __attribute__((visibility("default"))) int e2ttt_debug_read_profile(long long* host, int n) {
    return (int)cudaMemcpyFromSymbol(host, g_tc_prof, sizeof(long long) * (size_t)n);
}
#endif

int tc_fwd_launch(const TcFwdArgs& a, void* stream) {
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    CUtensorMap tmK, tmQ, tmV;
    const size_t rows = (size_t)a.N * a.L;
    if (!make_token_map(&tmK, a.k, rows, 64, a.d) || !make_token_map(&tmQ, a.q, rows, 64, a.d) ||
        !make_token_map(&tmV, a.v, rows, 16, a.d))
        return (int)cudaErrorInvalidValue;
    static bool attr_done[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return (int)cudaGetLastError();
    const int smem = (int)tc_fwd_smem_bytes();
    if (dev < 0 || dev >= 64 || !attr_done[dev]) {
        cudaError_t e = cudaFuncSetAttribute(tc_fwd_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_fwd_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_fwd_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_fwd_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return (int)e;
        if (dev >= 0 && dev < 64) attr_done[dev] = true;
    }
    cudaError_t e = cudaMemsetAsync(a.status, 0, sizeof(int), st);
    if (e != cudaSuccess) return (int)e;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(a.N * NC));
    cfg.blockDim = dim3(NTHREADS);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = NC;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    const bool native = a.d == D && a.h == NC * HC;
    if (a.norm1 && a.norm2) {
        if (a.ckpt && !a.rown) return (int)cudaErrorInvalidValue;
        e = native ? cudaLaunchKernelEx(&cfg, tc_fwd_kernel<false, true>, tmK, tmQ, tmV, a)
                   : cudaLaunchKernelEx(&cfg, tc_fwd_kernel<true, true>, tmK, tmQ, tmV, a);
    } else {
        e = native ? cudaLaunchKernelEx(&cfg, tc_fwd_kernel<false, false>, tmK, tmQ, tmV, a)
                   : cudaLaunchKernelEx(&cfg, tc_fwd_kernel<true, false>, tmK, tmQ, tmV, a);
    }
    if (e != cudaSuccess) return (int)e;
    return (int)cudaGetLastError();
}

}  // namespace e2ttt
