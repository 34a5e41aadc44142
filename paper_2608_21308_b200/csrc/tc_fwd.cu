// Tensor-core forward for GELU-MLP fast weights, d = 128, h = 512, C = 64, bf16 I/O (sm_100a).
//
// One cluster of 4 CTAs per sequence; CTA c owns hidden units [128c, 128c+128): rows of W1, columns of W2.
// Everything that carries over from chunk to chunk stays on chip for the whole sequence:
//   - fp32 master copy of the CTA's W1/W2 slices: tensor memory columns [0,256).  The aggregation MMAs
//     accumulate -sum_t K^W_t grad_t straight into it (it is pre-scaled by the decay carry cw beforehand).
//   - fp32 master copy of the momentum slices: registers (each epilogue thread keeps the 2 x 32 elements it owns).
//   - bf16 operand copy of W1/W2: shared memory, refreshed once per chunk from the fp32 master.
// Per chunk (Algorithm 1), rows = tokens (64 keys then 64 queries), all GEMMs on tcgen05 with TMEM accumulators:
//   G1  Z = [K;Q] W1c^T          G2  Upart = gelu(Z) W2c^T      -> cross-CTA sum of Upart through DSMEM (each CTA
//   owns 32 token rows: LN, output rows o = q + LN(u), or e = k + LN(u) - v and pu = dL/du), pu rows broadcast
//   G3  Pa = Pu W2c, Pz = Pa * gelu'(Z)
//   aggregations (contraction over the 64 tokens, MN-major operands):
//       W1c -= (kW*Pz)^T K    M1acc = -(kM*Pz)^T K    W2c -= Pu^T (kW*Ak)    M2acc = -Pu^T (kM*Ak)
//   state pass: W = Wacc + cm M0;  M = cb M0 + Macc;  bf16(W) -> shared;  cw_next W -> TMEM.
//
// Warp roles (640 threads): warps 0-15 are epilogue warps (warp w reads TMEM lanes 32 (w & 3) .., columns
// 32 (w >> 2) ..; quadrants 0/1 hold the key rows, 2/3 the query rows); warp 18 is the MMA issuer (one lane issues,
// descriptors are compile-time offsets from one base); warp 19 loads tokens by TMA and runs the gate scans of the
// next chunk.  Nothing is CTA-wide inside the chunk loop: producers and consumers meet on mbarriers (one per
// buffer), the issuer never touches an epilogue.  setmaxnreg moves registers from the control warps to the epilogue warps.
// Every wait on an mbarrier is bounded (sm100.cuh); a wait that gives up is reported through the status word.
#include "tc_common.cuh"
#include "tc_fwd.h"

namespace e2ttt {
using namespace sm100;
using namespace tc;

#ifdef TC_PROFILE
#ifndef TC_PROF_CTAS
#define TC_PROF_CTAS 1
#endif
#ifndef TC_PROF_MASK
#define TC_PROF_MASK 15
#endif
// Debug build only: cycle stamps at the phase boundaries of the first 32 chunks, CTA 0 of the grid, for one
// key-row warp (thread 0), one query-row warp (thread 64), the issuer (thread 576) and the loader (thread 608).
__device__ long long g_tc_prof[16 * 32 * 24];
#define PROF(i)                                                                                      \
    do {                                                                                             \
        const int t_ = threadIdx.x;                                                                  \
        if (blockIdx.x < TC_PROF_CTAS && r < 32 && (t_ == 0 || t_ == 64 || t_ == 576 || t_ == 608) && (blockIdx.x == 0 || ((TC_PROF_MASK >> ((t_ == 0) ? 0 : (t_ == 64) ? 1 : (t_ == 576) ? 2 : 3)) & 1)))            \
            g_tc_prof[(((blockIdx.x * 4) + ((t_ == 0) ? 0 : (t_ == 64) ? 1 : (t_ == 576) ? 2 : 3)) * 32 + r) * 24 + (i)] = clock64(); \
    } while (0)
#else
#define PROF(i)
#endif


namespace {

constexpr int D = 128, HC = 128, NC = 4;
constexpr int NG = 4;                    // column groups per TMEM lane quadrant
constexpr int NEPI = 128 * NG;           // epilogue threads
constexpr int NTHREADS = NEPI + 128;     // + one control warpgroup (issuer warp, loader warp, two idle warps)
constexpr int NEW = NEPI / 32;           // epilogue warps
constexpr int CW = 128 / NG;             // accumulator columns a thread owns in a 128-column region
constexpr int NB = CW / 16;              // 16-column batches per thread
// The kernel starts with 96 registers per thread (640 threads).  The control warpgroup drops to 32 and its 64 x 128
// registers go to the 512 epilogue threads (+16 each): a warp can only take what its own CTA released.
constexpr int EPI_REGS = 112, CTRL_REGS = 32;

// TMEM columns
constexpr uint32_t T_W1 = 0, T_W2 = 128, T_R0 = 256, T_R1 = 384;

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
    ScanMap<float> tails[8];  // chunks of several blocks: composite gate map of the chunk's tokens behind each block
    // TMA / loader
    uint64_t bar_x, bar_v, bar_sc;
    // MMA completions (tcgen05.commit)
    uint64_t bar_g1, bar_g2, bar_g3, bar_aw1, bar_am1, bar_am2;
    // epilogue warps -> issuer: operand tiles written / accumulator regions read
    uint64_t bar_a, bar_ak, bar_pz, bar_r1, bar_w1, bar_w2;
    // cluster traffic
    uint64_t bar_go, bar_ksent, bar_partK, bar_partQ, bar_pu, bar_credit, bar_rs;
    uint32_t tmem_base;
    int dead;
};

// GELU on the bf16 path: the tanh form g(z) = 0.5 z (1 + tanh(u)), u = sqrt(2/pi) (z + 0.044715 z^3), with the
// hardware tanh (6 FMA-pipe instructions and one MUFU), and its exact derivative
// g'(z) = 0.5 (1 + T) + 0.5 z (1 - T^2) u'(z).  g differs from z Phi(z) by at most 4.7e-4 absolute and g' from
// Phi(z) + z phi(z) by at most 8.7e-4 (plus 2^-11 relative from tanh.approx); both values are rounded to bf16 right
// after (half an ulp = 2^-9 relative).  The fp32/fp64 SIMT path keeps the exact erf form.
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

// g'(z) alone
__device__ __forceinline__ float gelu_d1_fast(float z) {
    const float z2 = z * z;
    const float t = fast_tanh(z * fmaf(0.0356774081f, z2, 0.7978845608f));
    const float du = fmaf(0.1070322243f, z2, 0.7978845608f);
    return fmaf((0.5f * z) * fmaf(-t, t, 1.0f), du, fmaf(0.5f, t, 0.5f));
}

// PAD = false: the native 128 x 512 shape, every mask folds away.  PAD = true: d and h come from the arguments.
// NORM = true: post-chunk normalisation - after the state transition every row of W1 and of W2 is rescaled to its
// target norm.  A row of W1c lives in one CTA (its 128 columns spread over the 4 column-group warps); a row of W2
// spans the 4 CTAs, so its sum of squares crosses the cluster once per chunk.
// MULTI: chunks of several 64-token blocks (128, 256, 512 tokens); a compile-time switch, so that the single-block
// instantiations are exactly the code they were without it
template <bool PAD, bool NORM, bool MULTI = false>
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
    const uint32_t me = cluster_ctarank();
    const int seq = blockIdx.x / NC;
    const int Cc = a.C;                     // chunk size
    const int Cr = min(Cc, C);              // tokens per block (<= C = 64, the tile's rows)
    const int m = MULTI ? Cc / C : 1;       // 64-token blocks per chunk
    constexpr bool multi = MULTI;
    // `nchunks` counts the blocks (= chunks unless a chunk has several); the last one may be shorter: its unused rows
    // get zero scalar kernels
    const int L = a.L, nchunks = (L + Cr - 1) / Cr;
    const int Ls = a.Ls;  // sequence stride in tokens
    WaitCtx wc{&s.dead, a.status};

    // Real shape: de x he.  Columns >= de of every token tile and hidden units >= he are zero padding: they stay
    // exactly zero through every product, so only the layer norm (divisor, masks) and the global I/O know about them.
    const int de = PAD ? a.d : D, he = PAD ? a.h : NC * HC;
    const float* eta = a.eta + (size_t)seq * Ls;
    const float* beta = a.beta + (size_t)seq * Ls;
    const float* gamma = a.gamma + (size_t)seq * Ls;

    if (tid == 0) {
        s.dead = 0;
        mbar_init(&s.bar_x, 1);
        mbar_init(&s.bar_v, 1);
        mbar_init(&s.bar_sc, 1);
        mbar_init(&s.bar_g1, 1);
        mbar_init(&s.bar_g2, 1);
        mbar_init(&s.bar_g3, 1);
        mbar_init(&s.bar_aw1, 1);
        mbar_init(&s.bar_am1, 1);
        mbar_init(&s.bar_am2, 1);
        mbar_init(&s.bar_a, NEW);
        mbar_init(&s.bar_ak, NEW / 2);
        mbar_init(&s.bar_pz, NEW / 2);
        mbar_init(&s.bar_r1, NEW);
        mbar_init(&s.bar_w1, NEW);
        mbar_init(&s.bar_w2, NEW);
        mbar_init(&s.bar_ksent, NEW / 2);
        mbar_init(&s.bar_go, 1);
        mbar_init(&s.bar_partK, 1);  // + 3 x 8 KB of peer partial sums (key rows) per chunk
        mbar_init(&s.bar_partQ, 1);  // + 3 x 4 KB (query rows, bf16)
        mbar_init(&s.bar_pu, 2);     // + 12 KB of pu rows from the peers per chunk, one arrival for the own rows
        mbar_init(&s.bar_credit, 3);
        mbar_init(&s.bar_rs, 1);     // + 3 x 512 B of peer row sums per chunk (normalisation only)
        fence_mbar_init();
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmV);
    }
    if (warp == 0) { tmem_alloc(&s.tmem_base, 512); tmem_relinquish(); }
    if (warp == 1) {
        if (multi) tc_chunk_tails(beta, gamma, min(Cc, L), min(m, nchunks), s.tails);
        tc_chunk_scalars(eta, beta, gamma, &s.sc[0], min(Cr, L), multi ? &s.tails[0] : nullptr);
    }
    if (de < 128)  // the padded half of the token tile is never loaded: zero it once
        for (int i = tid; i < 16384 / 16; i += NTHREADS) reinterpret_cast<uint4*>(s.X[1])[i] = make_uint4(0u, 0u, 0u, 0u);
    if (Cr < C)    // short chunks: the key and query rows past the chunk are never loaded either (128-byte rows, 8 pieces each)
        for (int i = tid; i < 32768 / 16; i += NTHREADS)
            if (((i >> 3) & 63) >= Cr) reinterpret_cast<uint4*>(s.X[0])[i] = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    // every CTA's barriers are initialised before any peer may arrive on them
    cluster_sync();
    tc_fence_after_sync();
    const uint32_t tb = s.tmem_base;

    if (warp >= NEW) {
        // =====================================================================================================
        // control warpgroup
        // =====================================================================================================
#ifndef TC_NO_SETMAXNREG
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(CTRL_REGS));
#endif
        if (warp == NEW + 2) {
            // the whole warp runs the loop converged (every lane polls the barriers); lane 0 issues
            // ------------------------------------------------------------------------------------- MMA issuer
            // the descriptor's address field has 14 bits; a shared::cta address of a CTA of a cluster carries more above them
            const uint32_t sb = (smem_u32(smem_raw) >> 4) & 0x3FFFu;
            constexpr uint32_t oW1 = offsetof(Smem, W1) >> 4, oW2 = offsetof(Smem, W2) >> 4, oX = offsetof(Smem, X) >> 4,
                               oA = offsetof(Smem, A) >> 4, oAkW = offsetof(Smem, AkW) >> 4, oAkM = offsetof(Smem, AkM) >> 4,
                               oPu = offsetof(Smem, Pu) >> 4, oPzW = offsetof(Smem, PzW) >> 4, oPzM = offsetof(Smem, PzM) >> 4;
            const uint32_t id_kk = make_idesc(128, 128, false, false);
            const uint32_t id_kmn = make_idesc(128, 128, false, true);
            const uint32_t id_agg = make_idesc(128, 128, true, true) | (1u << 13);  // negate A: G_t is minus the gradient
            const bool el = lane == 0;  // the lane whose MMA / commit instructions are not predicated off
            for (int r = 0; r < nchunks; ++r) {
                const uint32_t ph = (uint32_t)(r & 1);
                // G1: Z = X W1c^T -> R0.  Needs the chunk's tokens, the refreshed bf16 W1 and R0 read out (M1 aggregate).
                mbar_wait(&s.bar_x, ph, wc, 100 + 1);
                mbar_wait(&s.bar_w1, ph, wc, 100 + 2);
                tc_fence_after_sync();
                PROF(0);
#pragma unroll
                for (int k = 0; k < 8; ++k) umma_bf16_elect(tb + T_R0, dk(sb + oX, 16384, k), dk(sb + oW1, 16384, k), id_kk, k > 0, el);
                umma_commit_elect(&s.bar_g1, el);
                PROF(1);
                // G2: Upart = A W2c^T -> R1.  Needs gelu(Z) in A, the refreshed bf16 W2 and R1 read out (M2 aggregate).
                mbar_wait(&s.bar_a, ph, wc, 100 + 3);
                mbar_wait(&s.bar_w2, ph, wc, 100 + 4);
                tc_fence_after_sync();
                PROF(2);
#pragma unroll
                for (int k = 0; k < 8; ++k) umma_bf16_elect(tb + T_R1, dk(sb + oA, 16384, k), dk(sb + oW2, 16384, k), id_kk, k > 0, el);
                umma_commit_elect(&s.bar_g2, el);
                PROF(3);
                // G3: Pa = Pu W2c -> R1.  Needs every CTA's pu rows (bulk copies: async proxy, no proxy fence needed here) and
                // the partial sums read out of R1 by all warps.  The instruction is M = 128 although pu has 64 token rows: an
                // M = 64 instruction costs the same, so rows 64..127 of the A descriptor run on into whatever lies behind the
                // pu slab, and lanes 64..127 of R1 receive values that nobody reads (the next writer of R1 starts afresh).
                mbar_wait<true>(&s.bar_pu, ph, wc, 100 + 5);
                PROF(13);
                mbar_wait(&s.bar_r1, ph, wc, 100 + 6);
                tc_fence_after_sync();
                PROF(4);
#pragma unroll
                for (int k = 0; k < 8; ++k) umma_bf16_elect(tb + T_R1, dk(sb + oPu, 8192, k), dmn(sb + oW2, 16384, k), id_kmn, k > 0, el);
                umma_commit_elect(&s.bar_g3, el);
                PROF(5);
                // W2 aggregation on top of the master
                mbar_wait(&s.bar_ak, ph, wc, 100 + 7);
                tc_fence_after_sync();
#pragma unroll
                for (int k = 0; k < 4; ++k) umma_bf16_elect(tb + T_W2, dmn(sb + oPu, 8192, k), dmn(sb + oAkW, 8192, k), id_agg, true, el);
                PROF(14);
                // W1 aggregation first (the next chunk's G1 hangs on it), then the two momentum aggregates
                mbar_wait(&s.bar_pz, ph, wc, 100 + 8);
                tc_fence_after_sync();
                PROF(6);
                if (multi) {  // several blocks per chunk: the momentum aggregate is read out after every block, the weights' is not
#pragma unroll
                    for (int k = 0; k < 4; ++k) umma_bf16_elect(tb + T_R0, dmn(sb + oPzM, 8192, k), dmn(sb + oX, 16384, k), id_agg, k > 0, el);
                    umma_commit_elect(&s.bar_am1, el);
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) umma_bf16_elect(tb + T_W1, dmn(sb + oPzW, 8192, k), dmn(sb + oX, 16384, k), id_agg, true, el);
                umma_commit_elect(&s.bar_aw1, el);
                if (!multi) {
#pragma unroll
                    for (int k = 0; k < 4; ++k) umma_bf16_elect(tb + T_R0, dmn(sb + oPzM, 8192, k), dmn(sb + oX, 16384, k), id_agg, k > 0, el);
                    umma_commit_elect(&s.bar_am1, el);
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) umma_bf16_elect(tb + T_R1, dmn(sb + oPu, 8192, k), dmn(sb + oAkM, 8192, k), id_agg, k > 0, el);
                umma_commit_elect(&s.bar_am2, el);
                PROF(7);
            }
        } else if (warp == NEW + 3) {
            // ------------------------------------------------------------------- token loads and gate scans
            for (int r = 0; r < nchunks; ++r) {
                const uint32_t ph = (uint32_t)(r & 1);
                const int tok0 = r * Cr;
                if (r == 0) {
                    if (lane == 0) {
                        mbar_expect_tx(&s.bar_x, (uint32_t)Cr * (de == 128 ? 512u : 256u));
                        const int y = seq * Ls;
                        tma_load_2d(s.X[0], &tmK, 0, y, &s.bar_x);
                        tma_load_2d(s.X[0] + 8192, &tmQ, 0, y, &s.bar_x);
                        if (de == 128) {
                            tma_load_2d(s.X[1], &tmK, 64, y, &s.bar_x);
                            tma_load_2d(s.X[1] + 8192, &tmQ, 64, y, &s.bar_x);
                        }
                    }
                } else {
                    // the previous chunk is over in this CTA: its scalars, barriers' phases and staging are history
                    mbar_wait(&s.bar_w2, ph, wc, 100 + 20);
                }
                if (lane == 0) {
                    mbar_expect_tx(&s.bar_partK, 3 * 8192);  // this chunk's incoming partial sums and pu rows
                    mbar_expect_tx(&s.bar_partQ, 3 * 4096);
                    mbar_expect_tx(&s.bar_pu, 12288);
                    if (NORM) mbar_expect_tx(&s.bar_rs, 3 * 512);
                    if (r + 1 < nchunks) {
                        // the next chunk's tokens: into L2 now, so that the loads issued at the end of this chunk are short
                        const int y = seq * Ls + tok0 + Cr;
                        tma_prefetch_l2_2d(&tmK, 0, y);
                        tma_prefetch_l2_2d(&tmQ, 0, y);
                        tma_prefetch_l2_2d(&tmV, 0, y + 16 * (int)me);
                        if (de == 128) {
                            tma_prefetch_l2_2d(&tmK, 64, y);
                            tma_prefetch_l2_2d(&tmQ, 64, y);
                            tma_prefetch_l2_2d(&tmV, 64, y + 16 * (int)me);
                        }
                    }
                }
                __syncwarp();
                if (r + 1 < nchunks) {
                    // scalars of the next chunk (suffix scans over its gates)
                    const int tokn = tok0 + Cr;
                    const ScanMap<float>* tl = nullptr;
                    if (multi) {
                        const int bn = (r + 1) % m;  // a chunk's first block: the tails of all its blocks first
                        if (bn == 0) tc_chunk_tails(beta + tokn, gamma + tokn, min(Cc, L - tokn), min(m, nchunks - r - 1), s.tails);
                        tl = &s.tails[bn];
                    }
                    tc_chunk_scalars(eta + tokn, beta + tokn, gamma + tokn, &s.sc[(r + 1) & 1], min(Cr, L - tokn), tl);
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&s.bar_sc);
                }
                // the 16 value rows this CTA needs for its key rows: into the gelu tile's first slab, dead once G2 is done
                mbar_wait(&s.bar_g2, ph, wc, 100 + 21);
                if (lane == 0) {
                    mbar_expect_tx(&s.bar_v, de == 128 ? 4096u : 2048u);
                    const int y = seq * Ls + tok0 + 16 * (int)me;
                    tma_load_2d(s.A[0], &tmV, 0, y, &s.bar_v);
                    if (de == 128) tma_load_2d(s.A[0] + 2048, &tmV, 64, y, &s.bar_v);
                }
                if (r + 1 < nchunks) {
                    // the W1 / M1 aggregations were the last readers of the key tile: the next chunk's tokens may land in X
                    mbar_wait(multi ? &s.bar_aw1 : &s.bar_am1, ph, wc, 100 + 22);  // whichever was issued last
                    if (lane == 0) {
                        mbar_expect_tx(&s.bar_x, (uint32_t)Cr * (de == 128 ? 512u : 256u));
                        const int y2 = seq * Ls + tok0 + Cr;
                        tma_load_2d(s.X[0], &tmK, 0, y2, &s.bar_x);
                        tma_load_2d(s.X[0] + 8192, &tmQ, 0, y2, &s.bar_x);
                        if (de == 128) {
                            tma_load_2d(s.X[1], &tmK, 64, y2, &s.bar_x);
                            tma_load_2d(s.X[1] + 8192, &tmQ, 64, y2, &s.bar_x);
                        }
                    }
                }
                if (NORM || r + 1 < nchunks) {
                    // Every reader of this chunk's staging / pu / scaled-activation buffers is done once the aggregations
                    // have completed and every epilogue warp has left its layer norm (it has then released W1): tell the
                    // peers they may overwrite them.  (With normalisation the last chunk's row sums still need it.)
                    mbar_wait(&s.bar_am2, ph, wc, 100 + 23);
                    mbar_wait(&s.bar_w1, ph ^ 1u, wc, 100 + 24);
                    if (lane < NC && lane != (int)me) mbar_arrive_remote(map_to_cta(smem_u32(&s.bar_credit), (uint32_t)lane));
                    __syncwarp();
                }
                if (r + 1 < nchunks) {
                    // ... and pass the peers' credits on to the epilogue warps (a local barrier is cheaper to wait on)
                    mbar_wait<true>(&s.bar_credit, ph, wc, 100 + 25);
                    if (lane == 0) mbar_arrive(&s.bar_go);
                    __syncwarp();
                }
            }
        }
    } else {
        // =====================================================================================================
        // epilogue warps
        // =====================================================================================================
#ifndef TC_NO_SETMAXNREG
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(EPI_REGS));
#endif
        const int q = warp & 3;          // TMEM lane quadrant
        const int g = warp >> 2;         // column group
        const int row = 32 * q + lane;   // TMEM lane this thread reads
        const int c0 = CW * g;           // first of its columns inside a 128-column region
        const uint32_t lane_addr = tb + ((uint32_t)(32 * q) << 16);
        const size_t dh = (size_t)de * he;
        const bool cta_real = HC * (int)me < he;  // this CTA's 128 hidden units exist
        const float inv_d = 1.0f / (float)de;
        // normalisation targets of this thread's rows: hidden unit 128 me + row of W1, output row `row` of W2
        const float tgt1 = (NORM && cta_real) ? a.norm1[(size_t)seq * he + HC * me + row] : 0.0f;
        const float tgt2 = (NORM && row < de) ? a.norm2[(size_t)seq * de + row] : 0.0f;
        __nv_bfloat16* go = a.o ? a.o + (size_t)seq * Ls * de : nullptr;

        // ---- load the state: fp32 master of W -> TMEM (pre-scaled by the first decay carry) and bf16 -> shared; M -> registers
        float M1[CW], M2[CW];
        {
            const float cw0 = s.sc[0].cw, cm0 = s.sc[0].cm;
            const size_t head = (size_t)seq * a.init_seq_stride;
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
                for (int j = 0; j < 16; ++j) {
                    M1[16 * b + j] = (m1 && real1) ? m1[16 * b + j] : 0.0f;
                    st[j] = __float_as_uint(multi ? fmaf(cm0, M1[16 * b + j], cw0 * w[j]) : cw0 * w[j]);
                }
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
                for (int j = 0; j < 16; ++j) {
                    M2[16 * b + j] = (m2 && real2) ? m2[16 * b + j] : 0.0f;
                    st[j] = __float_as_uint(multi ? fmaf(cm0, M2[16 * b + j], cw0 * w[j]) : cw0 * w[j]);
                }
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
            warp_release(&s.bar_w1);
            if (lane == 0) mbar_arrive(&s.bar_w2);
        }

        for (int r = 0; r < nchunks; ++r) {
            const uint32_t ph = (uint32_t)(r & 1);
            const Scalars& sc = s.sc[r & 1];
            const int tok0 = r * Cr;
            const bool last = (r + 1 == nchunks);
            PROF(0);
            // ---------------- G1 epilogue: a = gelu(z) -> A (bf16), all that G2 needs.  The key rows' a also goes, unscaled,
            // (as fp16) into the kW a tile: the query-row warps turn it into bf16 kW a and kM a while G2 runs.
            mbar_wait(&s.bar_g1, ph, wc, 100 + 30);
            tc_fence_after_sync();
            PROF(1);
            {
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    uint32_t z[16];
                    tmem_ld16(lane_addr + T_R0 + c0 + 16 * b, z);
                    tmem_wait_ld();
                    uint32_t p[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float a0 = gelu_only(__uint_as_float(z[2 * i])), a1 = gelu_only(__uint_as_float(z[2 * i + 1]));
                        p[i] = pack_bf16(a0, a1);
                        z[i] = pack_f16(a0, a1);  // fp16 keeps 3 more bits: no visible second rounding in kW a, kM a
                    }
                    const int col = c0 + 16 * b;
                    st_slab16p(s.A[col >> 6], row, col & 63, p);
                    if (q < 2) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) p[i] = z[i];
                        st_slab16p(s.AkW[col >> 6], row, col & 63, p);
                    }
                }
                warp_release(&s.bar_a);
                PROF(2);
                if (q < 2) {
                    // key rows: gelu'(z) replaces z in TMEM (the G3 epilogue multiplies by it), in the shadow of G2
#pragma unroll
                    for (int b = 0; b < NB; ++b) {
                        uint32_t z[16];
                        tmem_ld16(lane_addr + T_R0 + c0 + 16 * b, z);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 16; ++j) z[j] = __float_as_uint(gelu_d1_fast(__uint_as_float(z[j])));
                        tmem_st16(lane_addr + T_R0 + c0 + 16 * b, z);
                    }
                    tmem_wait_st();
                } else {
                    // query-row warps: scale the key rows' a by kW and kM (operands of the W2 aggregations).  256 threads over
                    // the [64 x 128] tile: 4 threads per row, 32 columns each; kW a overwrites a in place.
                    mbar_wait(&s.bar_a, ph, wc, 100 + 38);
                    const int tq = 32 * (2 * g + (q & 1)) + lane;
                    const int ar = tq >> 2, ac = 32 * (tq & 3);
                    const float kw = sc.kW[ar], km = sc.kM[ar];
                    uint8_t* rw = s.AkW[ac >> 6] + ar * 128;
                    uint8_t* rm = s.AkM[ac >> 6] + ar * 128;
                    uint4 v[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) v[i] = *reinterpret_cast<const uint4*>(rw + (((((ac & 63) >> 3) + i) ^ (ar & 7)) << 4));
                    auto scale2 = [](uint32_t x, float k) {  // two packed fp16 times k -> two packed bf16
                        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&x));
                        return pack_bf16(k * f.x, k * f.y);
                    };
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int off = ((((ac & 63) >> 3) + i) ^ (ar & 7)) << 4;
                        *reinterpret_cast<uint4*>(rw + off) = make_uint4(scale2(v[i].x, kw), scale2(v[i].y, kw), scale2(v[i].z, kw), scale2(v[i].w, kw));
                        *reinterpret_cast<uint4*>(rm + off) = make_uint4(scale2(v[i].x, km), scale2(v[i].y, km), scale2(v[i].z, km), scale2(v[i].w, km));
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&s.bar_ak);
                }
            }
            PROF(3);

            // Row ownership: CTA c normalises key tokens 16c..16c+15 and query tokens 16c..16c+15, so every CTA carries
            // the same mix of work.  TMEM lane 32q+l holds key token 32q+l (q < 2) or query token 32(q-2)+l.
            // Partial sums of the key rows travel as fp32 (they feed the state), those of the query rows as bf16 (they
            // only feed o, which is rounded to bf16 anyway).  The sender's own rows stay fp32 in the dead gelu tile.
            const uint32_t owner = 2u * ((uint32_t)q & 1u) + ((uint32_t)lane >> 4);
            const uint32_t srow = (uint32_t)lane & 15u;                 // row inside the owner's slot
            const uint32_t slot = (me - owner - 1u) & 3u;               // where the owner keeps what comes from this CTA
            auto send_k = [&]() {
                const bool mine = owner == me;
                uint32_t dst_base, dst_bar = 0;
                if (mine) {
                    dst_base = smem_u32(s.A[1]);  // the gelu tile is dead once G2 has completed
                } else {
                    const uint8_t* p = (slot == 0) ? s.PzW[0] : (slot == 1) ? s.PzW[1] : s.PzM[0];
                    dst_base = map_to_cta(smem_u32(p), owner);
                    dst_bar = map_to_cta(smem_u32(&s.bar_partK), owner);
                }
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    uint32_t u[16];
                    tmem_ld16(lane_addr + T_R1 + c0 + 16 * b, u);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 16; j += 4) {
                        const uint32_t dst = dst_base + stage_offset((uint32_t)((c0 + 16 * b + j) >> 2), srow);
                        if (mine) st_cluster_v4_b32(dst, u[j], u[j + 1], u[j + 2], u[j + 3]);
                        else st_async_v4(dst, u[j], u[j + 1], u[j + 2], u[j + 3], dst_bar);
                    }
                }
                // R1 may be overwritten by G3 once every warp has taken its rows
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) { mbar_arrive(&s.bar_r1); mbar_arrive(&s.bar_ksent); }
            };
            auto send_q = [&]() {
                const bool mine = owner == me;
                const uint32_t own_base = smem_u32(s.A[1]) + 8192u;
                const uint32_t dst_base = map_to_cta(smem_u32(s.Stage2) + slot * 4096u, owner);
                const uint32_t dst_bar = map_to_cta(smem_u32(&s.bar_partQ), owner);
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    uint32_t u[16];
                    tmem_ld16(lane_addr + T_R1 + c0 + 16 * b, u);
                    tmem_wait_ld();
                    if (mine) {
#pragma unroll
                        for (int j = 0; j < 16; j += 4)
                            st_cluster_v4_b32(own_base + stage_offset((uint32_t)((c0 + 16 * b + j) >> 2), srow), u[j], u[j + 1], u[j + 2], u[j + 3]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; j += 8)
                            st_async_v4(dst_base + stage_offset_q((uint32_t)((c0 + 16 * b + j) >> 3), srow),
                                        pack_bf16(__uint_as_float(u[j]), __uint_as_float(u[j + 1])),
                                        pack_bf16(__uint_as_float(u[j + 2]), __uint_as_float(u[j + 3])),
                                        pack_bf16(__uint_as_float(u[j + 4]), __uint_as_float(u[j + 5])),
                                        pack_bf16(__uint_as_float(u[j + 6]), __uint_as_float(u[j + 7])), dst_bar);
                    }
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&s.bar_r1);
            };

            // Layer norm on the 16 key rows (warps of quadrants 0/1) or the 16 query rows (quadrants 2/3) this CTA owns:
            // 16 threads per row, 8 columns each.
            auto layer_norm = [&](const bool key_rows) {
                constexpr int TPR = NEPI / 32, CPT = 128 / TPR;  // threads per row, columns per thread
                static_assert(TPR == 16 && CPT == 8, "row mapping below assumes two rows per warp, one 16-byte piece per thread");
                const int lrow = 2 * ((q & 1) + 2 * g) + (lane >> 4);   // row of the slot (0..15)
                const int cg = lane & 15;
                const int t = 16 * (int)me + lrow;           // token inside the chunk
                const int xrow = key_rows ? t : 64 + t;      // its row in the X tile
                const int col0 = CPT * cg;
                const size_t off = (size_t)(tok0 + t) * de + col0;
                const bool real = col0 < de;  // this thread's 8 columns exist (padding columns carry exact zeros)
                const int c = (col0 & 63) >> 3;
                const uint4 xraw = *reinterpret_cast<const uint4*>(s.X[col0 >> 6] + xrow * 128 + ((c ^ (xrow & 7)) << 4));
                float u[CPT];
                {   // own rows, fp32
                    const uint8_t* p = s.A[1] + (key_rows ? 0 : 8192);
                    const float4 x0 = *reinterpret_cast<const float4*>(p + stage_offset((uint32_t)(2 * cg), (uint32_t)lrow));
                    const float4 x1 = *reinterpret_cast<const float4*>(p + stage_offset((uint32_t)(2 * cg + 1), (uint32_t)lrow));
                    u[0] = x0.x; u[1] = x0.y; u[2] = x0.z; u[3] = x0.w; u[4] = x1.x; u[5] = x1.y; u[6] = x1.z; u[7] = x1.w;
                }
                mbar_wait<true>(key_rows ? &s.bar_partK : &s.bar_partQ, ph, wc, 100 + 35);
                PROF(15);
                // the peers' pieces, added in a fixed order (slot 0, 1, 2 = the CTAs me+1, me+2, me+3): the sum does not
                // depend on arrival order, and each CTA adds its four pieces in its own fixed order
                if (key_rows) {
#pragma unroll
                    for (int sl = 0; sl < 3; ++sl) {
                        const uint8_t* p = (sl == 0) ? s.PzW[0] : (sl == 1) ? s.PzW[1] : s.PzM[0];
                        const float4 x0 = *reinterpret_cast<const float4*>(p + stage_offset((uint32_t)(2 * cg), (uint32_t)lrow));
                        const float4 x1 = *reinterpret_cast<const float4*>(p + stage_offset((uint32_t)(2 * cg + 1), (uint32_t)lrow));
                        u[0] += x0.x; u[1] += x0.y; u[2] += x0.z; u[3] += x0.w; u[4] += x1.x; u[5] += x1.y; u[6] += x1.z; u[7] += x1.w;
                    }
                } else {
#pragma unroll
                    for (int sl = 0; sl < 3; ++sl) {
                        const uint4 x = *reinterpret_cast<const uint4*>(s.Stage2 + sl * 4096 + stage_offset_q((uint32_t)cg, (uint32_t)lrow));
                        const __nv_bfloat162* x2 = reinterpret_cast<const __nv_bfloat162*>(&x);
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const float2 f = __bfloat1622float2(x2[i]);
                            u[2 * i] += f.x;
                            u[2 * i + 1] += f.y;
                        }
                    }
                }
                auto row_sum = [&](float v) -> float {  // over the TPR lanes that share a row
#pragma unroll
                    for (int o = TPR / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                    return v;
                };
                if (key_rows) {
                    // Key rows (the critical path of the whole cluster): e = k + y - v, pu = rstd (e - mean(e) - y mean(e y)).
                    // All four row sums the two statistics need are taken in ONE pass of shuffles (the shuffles share the
                    // shared-memory data path with the cluster traffic, a dependent round costs ~60 cycles here):
                    //   s1 = sum u, s2 = sum u^2, s3 = sum (k - v), s4 = sum (k - v) u
                    //   mu = s1/d, var = s2/d - mu^2, mean(e) = s3/d (the mean of y is 0),
                    //   mean(e y) = rstd (s4 - mu s3)/d + var rstd^2
                    mbar_wait(&s.bar_v, ph, wc, 100 + 36);
                    PROF(16);
                    const uint4 vraw = real ? *reinterpret_cast<const uint4*>(s.A[0] + (col0 >> 6) * 2048 + lrow * 128 + ((c ^ (lrow & 7)) << 4))
                                            : make_uint4(0u, 0u, 0u, 0u);
                    const __nv_bfloat162* k2 = reinterpret_cast<const __nv_bfloat162*>(&xraw);
                    const __nv_bfloat162* v2 = reinterpret_cast<const __nv_bfloat162*>(&vraw);
                    float kv[CPT];
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        const float2 kf = __bfloat1622float2(k2[x]), vf = __bfloat1622float2(v2[x]);
                        kv[2 * x] = kf.x - vf.x;
                        kv[2 * x + 1] = kf.y - vf.y;
                    }
                    float s1 = 0.0f, s2 = 0.0f, s3 = 0.0f, s4 = 0.0f;
#pragma unroll
                    for (int j = 0; j < CPT; ++j) {
                        if (!real) u[j] = 0.0f;
                        s1 += u[j]; s2 = fmaf(u[j], u[j], s2); s3 += kv[j]; s4 = fmaf(kv[j], u[j], s4);
                    }
#pragma unroll
                    for (int o = TPR / 2; o > 0; o >>= 1) {
                        const float t1 = __shfl_xor_sync(0xffffffffu, s1, o), t2 = __shfl_xor_sync(0xffffffffu, s2, o);
                        const float t3 = __shfl_xor_sync(0xffffffffu, s3, o), t4 = __shfl_xor_sync(0xffffffffu, s4, o);
                        s1 += t1; s2 += t2; s3 += t3; s4 += t4;
                    }
                    const float mu = s1 * inv_d;
                    const float var = fmaxf(fmaf(-mu, mu, s2 * inv_d), 0.0f);
                    const float rstd = rsqrtf(var + a.eps);
                    const float me_ = s3 * inv_d;
                    const float mey = fmaf(rstd * inv_d, fmaf(-mu, s3, s4), var * rstd * rstd);
                    float e[CPT];
#pragma unroll
                    for (int j = 0; j < CPT; ++j) {
                        u[j] = real ? (u[j] - mu) * rstd : 0.0f;  // y (zero in the padding)
                        e[j] = kv[j] + u[j];
                    }
                    uint32_t pk[CPT / 2];
#pragma unroll
                    for (int j = 0; j < CPT; j += 2)
                        pk[j / 2] = real ? pack_bf16(rstd * (e[j] - me_ - u[j] * mey), rstd * (e[j + 1] - me_ - u[j + 1] * mey)) : 0u;  // 0 in the padding
                    // The bf16 pu rows go into this CTA's own pu tile; one bulk copy per peer and slab (2 KB: the 16 rows of a
                    // slab are contiguous) then carries them to the peers' tiles.  Bulk copies write through the async proxy,
                    // the one the MMAs read through, so the receivers need no proxy fence.
                    *reinterpret_cast<uint4*>(s.Pu[col0 >> 6] + t * 128 + ((c ^ (t & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    fence_proxy_async_smem();
                    named_sync(BAR_KOWN, NEPI / 2);
                    if (warp == 0) {
                        if (lane < 6) {
                            const uint32_t dst = (me + 1u + (uint32_t)(lane >> 1)) & 3u;
                            const uint32_t src = smem_u32(s.Pu[lane & 1]) + 2048u * me;
                            bulk_copy_to_cta(map_to_cta(src, dst), src, 2048u, map_to_cta(smem_u32(&s.bar_pu), dst));
                        }
                        if (lane == 0) mbar_arrive(&s.bar_pu);  // the own rows are in place
                    }
                } else {
                    // query rows (not on the critical path): two-pass statistics, o = q + y
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
                    const __nv_bfloat162* q2 = reinterpret_cast<const __nv_bfloat162*>(&xraw);
                    uint4 ov;
                    uint32_t* o32 = reinterpret_cast<uint32_t*>(&ov);
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        const float2 qf = __bfloat1622float2(q2[x]);
                        o32[x] = pack_bf16(qf.x + u[2 * x], qf.y + u[2 * x + 1]);
                    }
                    if (real && go && t < min(Cr, L - tok0)) *reinterpret_cast<uint4*>(go + off) = ov;
                }
            };

            // ---------------- cross-CTA sum of Upart, layer norm, pu broadcast
            // The key rows are on the critical path of the whole cluster, the query rows are not.  So the warps holding
            // key rows (quadrants 0/1) hand them to the network first, normalise this CTA's key rows as soon as the
            // peers' pieces are in and broadcast pu; the warps holding query rows (quadrants 2/3) send after the key
            // rows have gone out, normalise the query rows, write o.
            mbar_wait(&s.bar_g2, ph, wc, 100 + 31);
            tc_fence_after_sync();
            PROF(4);
            // the peers' staging slots, pu tile and scaled-activation tiles are free again: every peer has finished the
            // previous chunk (the loader warp collects the peers' credits)
            if (r > 0) mbar_wait(&s.bar_go, (uint32_t)((r - 1) & 1), wc, 100 + 32);
            PROF(13);
            if (q < 2) {
                send_k();
                PROF(14);
                named_sync(BAR_KOWN, NEPI / 2);  // this CTA's own key rows are staged
                PROF(5);
                layer_norm(true);
                PROF(6);
                PROF(17);
                // ---------------- G3 epilogue: Pz = Pa * gelu'(Zk), scaled by kW and kM into two bf16 tiles
                mbar_wait(&s.bar_g3, ph, wc, 100 + 33);
                tc_fence_after_sync();
                PROF(7);
                {
                    const float kw = sc.kW[row], km = sc.kM[row];
#pragma unroll
                    for (int b = 0; b < NB; ++b) {
                        uint32_t pa[16], dg[16];
                        tmem_ld16(lane_addr + T_R1 + c0 + 16 * b, pa);
                        tmem_ld16(lane_addr + T_R0 + c0 + 16 * b, dg);
                        tmem_wait_ld();
                        uint32_t p[8];
#pragma unroll
                        for (int j = 0; j < 16; ++j) pa[j] = __float_as_uint(__uint_as_float(pa[j]) * __uint_as_float(dg[j]));  // pz
                        const int col = c0 + 16 * b;
#pragma unroll
                        for (int i = 0; i < 8; ++i) p[i] = pack_bf16(kw * __uint_as_float(pa[2 * i]), kw * __uint_as_float(pa[2 * i + 1]));
                        st_slab16p(s.PzW[col >> 6], row, col & 63, p);
#pragma unroll
                        for (int i = 0; i < 8; ++i) p[i] = pack_bf16(km * __uint_as_float(pa[2 * i]), km * __uint_as_float(pa[2 * i + 1]));
                        st_slab16p(s.PzM[col >> 6], row, col & 63, p);
                    }
                }
                warp_release(&s.bar_pz);
                PROF(8);
            } else {
                mbar_wait(&s.bar_ksent, ph, wc, 100 + 34);
                send_q();
                PROF(14);
                named_sync(BAR_QOWN, NEPI / 2);  // own query rows staged
                PROF(5);
                layer_norm(false);
                PROF(6);
            }

            // ---------------- state pass (Algorithm 1 lines 6-7)
            if (!last) mbar_wait(&s.bar_sc, ph, wc, 100 + 37);  // the next chunk's scalars (its decay carry pre-scales the master)
            PROF(18);
            const float cm = sc.cm, cb = sc.cb;
            const float cwn = last ? 1.0f : s.sc[(r + 1) & 1].cw;
            const size_t head = (size_t)seq * a.final_seq_stride;
            // slot of the state after this chunk in the saved states (the slot after the last chunk is the final state)
            const int ce = NORM ? 1 : max(a.ckpt_every, 1);
            float* ckn = a.ckpt ? a.ckpt + (size_t)seq * a.ckpt_seq_stride + (size_t)((r + 1) / ce) * 4 * dh : nullptr;
            const bool save_ck = a.ckpt && (NORM || !last) && (r + 1) % ce == 0;

            if constexpr (!NORM && MULTI) {
                // ---- chunks of several 64-token blocks.  Every block's products read the chunk-start weights: the bf16
                // copies and the pre-scaling of the masters are refreshed after the chunk's last block only.  The master
                // already holds cw W_0 + cm M_0 (the momentum term was added when it was pre-scaled), so the momentum
                // registers can follow the blocks: M = cb M_0 + aggregate on the first block, M += aggregate afterwards.
                const int bidx = r % m;
                const bool final_block = bidx == m - 1 || last;
                const float cbk = bidx == 0 ? cb : 1.0f;
                const float cwn2 = last ? 1.0f : s.sc[(r + 1) & 1].cw, cmn2 = last ? 0.0f : s.sc[(r + 1) & 1].cm;
                const int cdone = r / m + 1;  // chunks completed after this block (if it is a final one)
                const bool save2 = a.ckpt && final_block && !last && cdone % ce == 0;
                float* ck2 = a.ckpt ? a.ckpt + (size_t)seq * a.ckpt_seq_stride + (size_t)(cdone / ce) * 4 * dh : nullptr;
                const bool wr = final_block && (last || save2);
                {
                    const bool real1 = cta_real;
                    const size_t off0 = ((size_t)(HC * me) + row) * de;
                    mbar_wait(&s.bar_am1, ph, wc, 100 + 39);
                    tc_fence_after_sync();
#pragma unroll
                    for (int b = 0; b < NB; ++b) {
                        const int col = c0 + 16 * b;
                        uint32_t ma[16];
                        tmem_ld16(lane_addr + T_R0 + col, ma);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 16; ++j) M1[16 * b + j] = fmaf(cbk, M1[16 * b + j], __uint_as_float(ma[j]));
                        if (wr && real1 && col < de) {
                            float* dst = (last ? a.M1_final + head : ck2 + 2 * dh) + off0 + col;
#pragma unroll
                            for (int j = 0; j < 16; j += 4)
                                *reinterpret_cast<float4*>(dst + j) = make_float4(M1[16 * b + j], M1[16 * b + j + 1], M1[16 * b + j + 2], M1[16 * b + j + 3]);
                        }
                    }
                    if (final_block) {
                        mbar_wait(&s.bar_aw1, ph, wc, 100 + 38);
                        tc_fence_after_sync();
#pragma unroll
                        for (int b = 0; b < NB; ++b) {
                            const int col = c0 + 16 * b;
                            uint32_t wa[16];
                            tmem_ld16(lane_addr + T_W1 + col, wa);
                            tmem_wait_ld();
                            uint32_t p[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) p[i] = pack_bf16(__uint_as_float(wa[2 * i]), __uint_as_float(wa[2 * i + 1]));
                            st_slab16p(s.W1[col >> 6], row, col & 63, p);
                            if (wr && real1 && col < de) {
                                float* dst = (last ? a.W1_final + head : ck2) + off0 + col;
#pragma unroll
                                for (int j = 0; j < 16; j += 4)
                                    *reinterpret_cast<uint4*>(dst + j) = make_uint4(wa[j], wa[j + 1], wa[j + 2], wa[j + 3]);
                            }
#pragma unroll
                            for (int j = 0; j < 16; ++j) wa[j] = __float_as_uint(fmaf(cmn2, M1[16 * b + j], cwn2 * __uint_as_float(wa[j])));
                            tmem_st16(lane_addr + T_W1 + col, wa);
                        }
                    }
                    tmem_wait_st();
                    warp_release(&s.bar_w1);  // R0 free (and, after a final block, W1 refreshed): the next block's G1 may run
                }
                {
                    const bool real2 = cta_real && row < de;
                    const size_t off0 = (size_t)row * he + HC * me;
                    mbar_wait(&s.bar_am2, ph, wc, 100 + 40);
                    tc_fence_after_sync();
#pragma unroll
                    for (int b = 0; b < NB; ++b) {
                        const int col = c0 + 16 * b;
                        uint32_t ma[16];
                        tmem_ld16(lane_addr + T_R1 + col, ma);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 16; ++j) M2[16 * b + j] = fmaf(cbk, M2[16 * b + j], __uint_as_float(ma[j]));
                        if (wr && real2) {
                            float* dst = (last ? a.M2_final + head : ck2 + 3 * dh) + off0 + col;
#pragma unroll
                            for (int j = 0; j < 16; j += 4)
                                *reinterpret_cast<float4*>(dst + j) = make_float4(M2[16 * b + j], M2[16 * b + j + 1], M2[16 * b + j + 2], M2[16 * b + j + 3]);
                        }
                        if (final_block) {
                            uint32_t wa[16];
                            tmem_ld16(lane_addr + T_W2 + col, wa);
                            tmem_wait_ld();
                            uint32_t p[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) p[i] = pack_bf16(__uint_as_float(wa[2 * i]), __uint_as_float(wa[2 * i + 1]));
                            st_slab16p(s.W2[col >> 6], row, col & 63, p);
                            if (wr && real2) {
                                float* dst = (last ? a.W2_final + head : ck2 + dh) + off0 + col;
#pragma unroll
                                for (int j = 0; j < 16; j += 4)
                                    *reinterpret_cast<uint4*>(dst + j) = make_uint4(wa[j], wa[j + 1], wa[j + 2], wa[j + 3]);
                            }
#pragma unroll
                            for (int j = 0; j < 16; ++j) wa[j] = __float_as_uint(fmaf(cmn2, M2[16 * b + j], cwn2 * __uint_as_float(wa[j])));
                            tmem_st16(lane_addr + T_W2 + col, wa);
                        }
                    }
                    tmem_wait_st();
                    warp_release(&s.bar_w2);  // R1 free (and, after a final block, W2 refreshed)
                }
            } else {
            // W1 half, as soon as the W1 aggregation is in (the momentum aggregate follows right behind it)
            mbar_wait(&s.bar_aw1, ph, wc, 100 + 38);
            tc_fence_after_sync();
            PROF(9);
            {
                const bool real1 = cta_real;
                const size_t off0 = ((size_t)(HC * me) + row) * de;
                float ss1 = 0.0f;
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    const int col = c0 + 16 * b;
                    uint32_t wa[16];  // the new weights, in place: unscaled first, then pre-scaled for the next chunk
                    tmem_ld16(lane_addr + T_W1 + col, wa);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float wn = fmaf(cm, M1[16 * b + j], __uint_as_float(wa[j]));
                        wa[j] = __float_as_uint(wn);
                        if (NORM) ss1 = fmaf(wn, wn, ss1);
                    }
                    if (!NORM) {
                        uint32_t p[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) p[i] = pack_bf16(__uint_as_float(wa[2 * i]), __uint_as_float(wa[2 * i + 1]));
                        st_slab16p(s.W1[col >> 6], row, col & 63, p);
                        if (real1 && col < de && (last || save_ck)) {
                            float* dst = (last ? a.W1_final + head : ckn) + off0 + col;
#pragma unroll
                            for (int j = 0; j < 16; j += 4)
                                *reinterpret_cast<uint4*>(dst + j) = make_uint4(wa[j], wa[j + 1], wa[j + 2], wa[j + 3]);
                        }
#pragma unroll
                        for (int j = 0; j < 16; ++j) wa[j] = __float_as_uint(cwn * __uint_as_float(wa[j]));
                    }
                    tmem_st16(lane_addr + T_W1 + col, wa);
                }
                if (NORM) {
                    // row sums of squares: the four column-group warps of a row meet in shared memory (the kW pz tile is dead)
                    float* rs = reinterpret_cast<float*>(s.PzW[0]);  // [NG][128]
                    rs[g * 128 + row] = ss1;
                    tmem_wait_st();
                    named_sync(BAR_EPI, NEPI);
                    float tot = 0.0f;
#pragma unroll
                    for (int gg = 0; gg < NG; ++gg) tot += rs[gg * 128 + row];
                    // padded hidden units have target 0 and norm 0: keep them at exactly 0 whatever norm_eps is
                    const float f = cta_real ? tgt1 / (sqrtf(tot) + a.norm_eps) : 0.0f;
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
                        if (real1 && col < de) {
                            if (last) {
#pragma unroll
                                for (int j = 0; j < 16; j += 4)
                                    *reinterpret_cast<float4*>(a.W1_final + head + off0 + col + j) = make_float4(wn[j], wn[j + 1], wn[j + 2], wn[j + 3]);
                            }
                            if (save_ck) {
#pragma unroll
                                for (int j = 0; j < 16; j += 4)
                                    *reinterpret_cast<float4*>(ckn + off0 + col + j) = make_float4(wn[j], wn[j + 1], wn[j + 2], wn[j + 3]);
                            }
                        }
                    }
                    if (a.ckpt && g == 0 && cta_real)  // row norm before the normalisation, for the reverse pass
                        a.rown[(size_t)seq * a.ckpt_seq_stride + ((size_t)r * 3 + 0) * (size_t)max(de, he) + HC * me + row] = sqrtf(tot);
                }
                // momentum half of W1: M1 = cb M1 + aggregate (R0)
                PROF(19);
                mbar_wait(&s.bar_am1, ph, wc, 100 + 39);
                PROF(20);
                tc_fence_after_sync();
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    const int col = c0 + 16 * b;
                    uint32_t ma[16];
                    tmem_ld16(lane_addr + T_R0 + col, ma);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 16; ++j) M1[16 * b + j] = fmaf(cb, M1[16 * b + j], __uint_as_float(ma[j]));
                    if (real1 && col < de) {
                        if (last) {
#pragma unroll
                            for (int j = 0; j < 16; j += 4)
                                *reinterpret_cast<float4*>(a.M1_final + head + off0 + col + j) =
                                    make_float4(M1[16 * b + j], M1[16 * b + j + 1], M1[16 * b + j + 2], M1[16 * b + j + 3]);
                        }
                        if (save_ck) {
#pragma unroll
                            for (int j = 0; j < 16; j += 4)
                                *reinterpret_cast<float4*>(ckn + 2 * dh + off0 + col + j) =
                                    make_float4(M1[16 * b + j], M1[16 * b + j + 1], M1[16 * b + j + 2], M1[16 * b + j + 3]);
                        }
                    }
                }
                tmem_wait_st();
                warp_release(&s.bar_w1);  // bf16 W1 complete, master rescaled, R0 free: the next chunk's G1 may run
            }
            PROF(10);

            // W2 half
            mbar_wait(&s.bar_am2, ph, wc, 100 + 40);
            tc_fence_after_sync();
            PROF(11);
            {
                const bool real2 = cta_real && row < de;
                const size_t off0 = (size_t)row * he + HC * me;
                float ss2 = 0.0f;
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    const int col = c0 + 16 * b;
                    {
                        uint32_t wa[16];  // the new weights, in place: unscaled first, then pre-scaled for the next chunk
                        tmem_ld16(lane_addr + T_W2 + col, wa);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const float wn = fmaf(cm, M2[16 * b + j], __uint_as_float(wa[j]));
                            wa[j] = __float_as_uint(wn);
                            if (NORM) ss2 = fmaf(wn, wn, ss2);
                        }
                        if (!NORM) {
                            uint32_t p[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) p[i] = pack_bf16(__uint_as_float(wa[2 * i]), __uint_as_float(wa[2 * i + 1]));
                            st_slab16p(s.W2[col >> 6], row, col & 63, p);
                            if (real2 && (last || save_ck)) {
                                float* dst = (last ? a.W2_final + head : ckn + dh) + off0 + col;
#pragma unroll
                                for (int j = 0; j < 16; j += 4)
                                    *reinterpret_cast<uint4*>(dst + j) = make_uint4(wa[j], wa[j + 1], wa[j + 2], wa[j + 3]);
                            }
#pragma unroll
                            for (int j = 0; j < 16; ++j) wa[j] = __float_as_uint(cwn * __uint_as_float(wa[j]));
                        }
                        tmem_st16(lane_addr + T_W2 + col, wa);
                    }
                    {
                        uint32_t ma[16];
                        tmem_ld16(lane_addr + T_R1 + col, ma);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 16; ++j) M2[16 * b + j] = fmaf(cb, M2[16 * b + j], __uint_as_float(ma[j]));
                    }
                    if (real2) {
                        if (last) {
#pragma unroll
                            for (int j = 0; j < 16; j += 4)
                                *reinterpret_cast<float4*>(a.M2_final + head + off0 + col + j) =
                                    make_float4(M2[16 * b + j], M2[16 * b + j + 1], M2[16 * b + j + 2], M2[16 * b + j + 3]);
                        }
                        if (save_ck) {
#pragma unroll
                            for (int j = 0; j < 16; j += 4)
                                *reinterpret_cast<float4*>(ckn + 3 * dh + off0 + col + j) =
                                    make_float4(M2[16 * b + j], M2[16 * b + j + 1], M2[16 * b + j + 2], M2[16 * b + j + 3]);
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
                    named_sync(BAR_EPI, NEPI);
                    if (warp == 0) {  // 32 lanes x 4 rows
                        // a peer's receive area overlays an operand tile of its W2 aggregations: it is free once that peer
                        // has seen them finish, which is what its credit of this chunk says
                        mbar_wait<true>(&s.bar_credit, ph, wc, 100 + 41);
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
                    named_sync(BAR_EPI, NEPI);  // the CTA's own vector is in place
                    mbar_wait<true>(&s.bar_rs, ph, wc, 100 + 42);
                    float tot = 0.0f;
#pragma unroll
                    for (uint32_t c = 0; c < NC; ++c) tot += got[c * 128 + row];
                    // padded rows have target 0 and norm 0: keep them at exactly 0 whatever norm_eps is
                    const float f = row < de ? tgt2 / (sqrtf(tot) + a.norm_eps) : 0.0f;
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
                        if (real2) {
                            if (last) {
#pragma unroll
                                for (int j = 0; j < 16; j += 4)
                                    *reinterpret_cast<float4*>(a.W2_final + head + off0 + col + j) = make_float4(wn[j], wn[j + 1], wn[j + 2], wn[j + 3]);
                            }
                            if (save_ck) {
#pragma unroll
                                for (int j = 0; j < 16; j += 4)
                                    *reinterpret_cast<float4*>(ckn + dh + off0 + col + j) = make_float4(wn[j], wn[j + 1], wn[j + 2], wn[j + 3]);
                            }
                        }
                    }
                    if (a.ckpt && g == 0 && me == 0 && row < de)
                        a.rown[(size_t)seq * a.ckpt_seq_stride + ((size_t)r * 3 + 1) * (size_t)max(de, he) + row] = sqrtf(tot);
                }
                tmem_wait_st();
                warp_release(&s.bar_w2);  // bf16 W2 complete, master rescaled, R1 free: the next chunk's G2 may run
            }
            }  // single-block chunks
            PROF(12);
        }
    }

    // no CTA leaves while a peer may still write into its shared memory or arrive on its barriers
    tc_fence_before_sync();
    __syncwarp();
    cluster_sync();
    if (warp == 0) tmem_dealloc(tb, 512);
}

}  // namespace

size_t tc_fwd_smem_bytes() { return sizeof(Smem); }

#ifdef TC_PROFILE
extern "C" __attribute__((visibility("default"))) int e2ttt_debug_read_profile(long long* host, int n) {
    return (int)cudaMemcpyFromSymbol(host, g_tc_prof, sizeof(long long) * (size_t)n);
}
#endif

int tc_fwd_launch(const TcFwdArgs& a_in, void* stream) {
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    TcFwdArgs a = a_in;
    if (a.Ls == 0) a.Ls = a.L;
    if (a.C == 0) a.C = C;
    if ((a.C != 512 && a.C != 256 && a.C != 128 && a.C != 64 && a.C != 32 && a.C != 16) || a.L <= 0) return (int)cudaErrorInvalidValue;
    if (a.C > 64 && a.norm1) return (int)cudaErrorInvalidValue;
    if (a.init_seq_stride == 0) a.init_seq_stride = (size_t)a.d * a.h;
    if (a.final_seq_stride == 0) a.final_seq_stride = (size_t)a.d * a.h;
    if (a.Ls < a.L) return (int)cudaErrorInvalidValue;
    CUtensorMap tmK, tmQ, tmV;
    // token rows the maps cover: up to the end of the last sequence's range
    const size_t rows = (size_t)(a.N - 1) * a.Ls + a.L;
    const unsigned box_rows = (unsigned)(a.C < 64 ? a.C : 64);
    if (!make_token_map(&tmK, a.k, rows, box_rows, a.d) || !make_token_map(&tmQ, a.q, rows, box_rows, a.d) ||
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
        if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_fwd_kernel<false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_fwd_kernel<true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return (int)e;
        if (dev >= 0 && dev < 64) attr_done[dev] = true;
    }
    cudaError_t e = a.keep_status ? cudaSuccess : cudaMemsetAsync(a.status, 0, sizeof(int), st);
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
        if (a.ckpt_every > 1) return (int)cudaErrorInvalidValue;
        e = native ? cudaLaunchKernelEx(&cfg, tc_fwd_kernel<false, true>, tmK, tmQ, tmV, a)
                   : cudaLaunchKernelEx(&cfg, tc_fwd_kernel<true, true>, tmK, tmQ, tmV, a);
    } else {
        if (a.C > 64)
            e = native ? cudaLaunchKernelEx(&cfg, tc_fwd_kernel<false, false, true>, tmK, tmQ, tmV, a)
                       : cudaLaunchKernelEx(&cfg, tc_fwd_kernel<true, false, true>, tmK, tmQ, tmV, a);
        else
            e = native ? cudaLaunchKernelEx(&cfg, tc_fwd_kernel<false, false>, tmK, tmQ, tmV, a)
                       : cudaLaunchKernelEx(&cfg, tc_fwd_kernel<true, false>, tmK, tmQ, tmV, a);
    }
    if (e != cudaSuccess) return (int)e;
    return (int)cudaGetLastError();
}

}  // namespace e2ttt
