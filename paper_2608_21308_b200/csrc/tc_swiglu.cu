// Tensor-core forward for SwiGLU fast weights, d = 128, h = 384, C = 64, bf16 I/O (sm_100a).
//   f_W(x) = x + LN(W3 (silu(W1 x) * (W2 x)))                         (Section 4, "Fast-weight Network")
//
// Same design as the GELU-MLP kernel (tc_fwd.cu): the state of a sequence stays on chip for all of its chunks, every
// product runs on tcgen05 with TMEM accumulators, warps are specialised (16 epilogue warps, an MMA issuer, a loader)
// and meet on per-buffer mbarriers.  What differs:
//   - three fp32 matrices of 128 hidden units would fill 384 of the 512 TMEM columns, so a CTA owns 64 hidden units and
//     a sequence is a cluster of 6 CTAs (h = 384);
//   - the gate and up projections of the CTA's hidden units are stacked into one 128-row matrix W12 = [W1c; W2c], so the
//     first product Z12 = [K;Q] W12^T (columns 0..63: z1, 64..127: z2), its aggregation W12 -= (kW*[pz1|pz2])^T K and its
//     state pass are the full-width 128 x 128 ones of the MLP kernel; W3c is [128 d][64 hidden];
//   - 64 tokens do not divide by 6: CTA c normalises the key (and query) tokens [ (64 c + 5) / 6, (64 (c+1) + 5) / 6 ),
//     11 or 10 of them;
//   - the staging slots of the exchange are buffers of their own (no overlay with operand tiles).
// Per chunk (Algorithm 1 with the SwiGLU network; s = sigmoid(z1)):
//   G1  Z12 = [K;Q] W12^T      hd = silu(z1) z2                 G2  Upart = Hd W3c^T -> cluster sum, LN, o / pu
//   G3  Ph = Pu W3c            pz1 = Ph z2 s (1 + z1 (1 - s)),  pz2 = Ph silu(z1)
//   aggregations   W12 -= (kW*Pz12)^T K   M12acc = -(kM*Pz12)^T K   W3c -= Pu^T (kW*Hd_k)   M3acc = -Pu^T (kM*Hd_k)
//   state pass     W = Wacc + cm M0;  M = cb M0 + Macc;  bf16(W) -> shared;  cw_next W -> TMEM.
// Every wait on an mbarrier is bounded (sm100.cuh); a wait that gives up is reported through the status word.
#include "tc_common.cuh"
#include "tc_swiglu.h"

namespace e2ttt {
using namespace sm100;
using namespace tc;

namespace {
// The issuer's MMA loops stay rolled: unrolled, the 76 descriptor words of a chunk are hoisted out of the chunk loop
// and spilled (the control warps run with 32 registers), and every MMA then waits for reloads (2.28 ms instead of
// 1.73 ms on the 4 x 16 x 4096 workload).
constexpr int kIssueUnroll = 1;

constexpr int D = 128, HS = 64, NC = 6;
constexpr int NG = 4;                    // column groups per TMEM lane quadrant
constexpr int NEPI = 128 * NG;           // epilogue threads
constexpr int NTHREADS = NEPI + 128;     // + one control warpgroup (issuer warp, loader warp, two idle warps)
constexpr int NEW = NEPI / 32;           // epilogue warps
constexpr int EPI_REGS = 112, CTRL_REGS = 32;

// TMEM columns: W12 master, W3c master, Z12 / gate derivatives / M12 aggregate, Upart / Ph / M3 aggregate
constexpr uint32_t T_W12 = 0, T_W3 = 128, T_R0 = 256, T_R1 = 384;

__host__ __device__ constexpr int tok_begin(int c) { return (64 * c + 5) / 6; }   // 0 11 22 32 43 54 64
__device__ __forceinline__ uint32_t tok_owner(int t) {
    return (uint32_t)((t >= 11) + (t >= 22) + (t >= 32) + (t >= 43) + (t >= 54));
}

struct __align__(1024) Smem {
    uint8_t W12[2][16384];   // bf16 [W1c; W2c]  [128 rows][64 i] per slab                 K-major B of G1
    uint8_t W12lo[2][16384]; // bf16 of what the first copy leaves of the fp32 master      second K-major B of G1
    uint8_t W3[16384];       // bf16 W3c  [128 i][64 j]                                    K-major B of G2, MN-major B of G3
    uint8_t X[2][16384];     // [128 tokens][64 i] per slab; rows 0..63 keys, 64..127 queries (TMA)
    uint8_t Hd[16384];       // bf16 hd [128 tokens][64 j]                                 K-major A of G2; then the CTA's own partial rows
    uint8_t HdW[8192];       // kW_t hd_k [64 t][64 j]  (first an fp16 copy of hd_k)       MN-major B of the W3 aggregation
    uint8_t HdM[8192];       // kM_t hd_k
    uint8_t Pu[2][8192];     // bf16 pu [64 t][64 i] per slab                              K-major A of G3, MN-major A of the W3 aggregations
    uint8_t PzW[2][8192];    // kW_t [pz1 | pz2]  [64 t][64 j] per slab                    MN-major A of the W12 aggregation
    uint8_t PzM[2][8192];    // kM_t [pz1 | pz2]
    // The peers' fp32 partial sums of the owned key rows, one 8 KB slot per peer: slots 0..3 lie over the four pz tiles
    // (written after G3, when the layer norm has consumed the slots; a peer sends a chunk's sums only after this CTA's
    // aggregations of the chunk before have completed: the credits), slot 4 has a place of its own.
    uint8_t StageK4[8192];
    uint8_t StageQ[NC - 1][4096];  // the peers' bf16 partial sums of the owned query rows
    uint8_t Vrows[4096];     // value rows of the owned key tokens (TMA, 16 rows)
    Scalars sc[2];
    ScanMap<float> tails[8];  // chunks of several blocks: composite gate map of the chunk's tokens behind each block
    uint64_t bar_x, bar_v, bar_sc;
    uint64_t bar_g1, bar_g2, bar_g3, bar_aw12, bar_am12, bar_am3;
    uint64_t bar_a, bar_ak, bar_pz, bar_r1, bar_w12, bar_w3;
    uint64_t bar_go, bar_ksent, bar_partK, bar_partQ, bar_pu, bar_credit;
    uint32_t tmem_base;
    int dead;
};

// Two-term bf16 form of 16 fp32 values: hi = bf16(w) and lo = bf16(w - hi) into the same place of two slabs
// (w - hi is exact in fp32; what hi + lo leaves of w is below 2^-16 |w|).
__device__ __forceinline__ void st_two_term(uint8_t* hi_slab, uint8_t* lo_slab, int row, int col0, const uint32_t (&w)[16]) {
    uint32_t ph[8], pl[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float w0 = __uint_as_float(w[2 * i]), w1 = __uint_as_float(w[2 * i + 1]);
        ph[i] = pack_bf16(w0, w1);
        // a bf16 is the upper half of the fp32 with the same value
        pl[i] = pack_bf16(w0 - __uint_as_float(ph[i] << 16), w1 - __uint_as_float(ph[i] & 0xFFFF0000u));
    }
    st_slab16p(hi_slab, row, col0, ph);
    st_slab16p(lo_slab, row, col0, pl);
}

// sigmoid by the hardware tanh: s(z) = 0.5 + 0.5 tanh(z / 2)
__device__ __forceinline__ float fast_sigmoid(float z) { return fmaf(0.5f, fast_tanh(0.5f * z), 0.5f); }

// MULTI: chunks of several 64-token blocks (128, 256, 512 tokens), a compile-time switch
template <bool MULTI>
__global__ void __launch_bounds__(NTHREADS, 1)
tc_swiglu_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ,
                 const __grid_constant__ CUtensorMap tmV, const TcSwigluArgs a) {
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
    // `nchunks` counts the blocks (= chunks unless a chunk has several); the last one may be shorter
    const int L = a.L, nchunks = (L + Cr - 1) / Cr;
    const int Ls = a.Ls;  // sequence stride in tokens
    const int h = NC * HS;
    WaitCtx wc{&s.dead, a.status};
    const int t0 = tok_begin((int)me), nown = tok_begin((int)me + 1) - t0;   // the key / query tokens this CTA normalises
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
        mbar_init(&s.bar_aw12, 1);
        mbar_init(&s.bar_am12, 1);
        mbar_init(&s.bar_am3, 1);
        mbar_init(&s.bar_a, NEW);
        mbar_init(&s.bar_ak, NEW / 2);
        mbar_init(&s.bar_pz, NEW / 2);
        mbar_init(&s.bar_r1, NEW);
        mbar_init(&s.bar_w12, NEW);
        mbar_init(&s.bar_w3, NEW);
        mbar_init(&s.bar_ksent, NEW / 2);
        mbar_init(&s.bar_go, 1);
        mbar_init(&s.bar_partK, 1);  // + 5 x nown x 512 B of peer partial sums (key rows) per chunk
        mbar_init(&s.bar_partQ, 1);  // + 5 x nown x 256 B (query rows, bf16)
        mbar_init(&s.bar_pu, 2);     // + (64 - nown) x 256 B of pu rows from the peers per chunk, one arrival for the own rows
        mbar_init(&s.bar_credit, NC - 1);
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
    if (Cr < C)    // short chunks: the key and query rows past the chunk are never loaded (128-byte rows, 8 pieces each)
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
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(CTRL_REGS));
        if (warp == NEW + 2) {
            // ------------------------------------------------------------------------------------- MMA issuer
            // The whole warp runs the loop converged (every lane polls the barriers); the MMA and commit instructions are
            // predicated to lane 0.  The descriptor's address field has 14 bits; a shared::cta address carries more above.
            const uint32_t sb = (smem_u32(smem_raw) >> 4) & 0x3FFFu;
            constexpr uint32_t oW12 = offsetof(Smem, W12) >> 4, oW12lo = offsetof(Smem, W12lo) >> 4, oW3 = offsetof(Smem, W3) >> 4, oX = offsetof(Smem, X) >> 4,
                               oHd = offsetof(Smem, Hd) >> 4, oHdW = offsetof(Smem, HdW) >> 4, oHdM = offsetof(Smem, HdM) >> 4,
                               oPu = offsetof(Smem, Pu) >> 4, oPzW = offsetof(Smem, PzW) >> 4, oPzM = offsetof(Smem, PzM) >> 4;
            const uint32_t id_kk = make_idesc(128, 128, false, false);
            const uint32_t id_kmn64 = make_idesc(128, 64, false, true);
            const uint32_t id_agg = make_idesc(128, 128, true, true) | (1u << 13);   // negate A: G_t is minus the gradient
            const uint32_t id_agg64 = make_idesc(128, 64, true, true) | (1u << 13);
            const bool el = lane == 0;
            for (int r = 0; r < nchunks; ++r) {
                const uint32_t ph = (uint32_t)(r & 1);
                // G1: Z12 = X W12^T -> R0
                mbar_wait(&s.bar_x, ph, wc, 300 + 1);
                mbar_wait(&s.bar_w12, ph, wc, 300 + 2);
                tc_fence_after_sync();
#pragma unroll kIssueUnroll
                for (int k = 0; k < 8; ++k) umma_bf16_elect(tb + T_R0, dk(sb + oX, 16384, k), dk(sb + oW12, 16384, k), id_kk, k > 0, el);
                // second term of the two-term bf16 form of W12: z1 z2 multiplies the rounding of a plain bf16 copy up
#pragma unroll kIssueUnroll
                for (int k = 0; k < 8; ++k) umma_bf16_elect(tb + T_R0, dk(sb + oX, 16384, k), dk(sb + oW12lo, 16384, k), id_kk, true, el);
                umma_commit_elect(&s.bar_g1, el);
                // G2: Upart = Hd W3c^T -> R1 (contraction over the CTA's 64 hidden units)
                mbar_wait(&s.bar_a, ph, wc, 300 + 3);
                mbar_wait(&s.bar_w3, ph, wc, 300 + 4);
                tc_fence_after_sync();
#pragma unroll kIssueUnroll
                for (int k = 0; k < 4; ++k) umma_bf16_elect(tb + T_R1, dk(sb + oHd, 16384, k), dk(sb + oW3, 16384, k), id_kk, k > 0, el);
                umma_commit_elect(&s.bar_g2, el);
                // G3: Ph = Pu W3c -> R1 columns 0..63 (M = 128 costs what M = 64 costs: lanes 64..127 get values nobody reads)
                mbar_wait<true>(&s.bar_pu, ph, wc, 300 + 5);
                mbar_wait(&s.bar_r1, ph, wc, 300 + 6);
                tc_fence_after_sync();
#pragma unroll kIssueUnroll
                for (int k = 0; k < 8; ++k) umma_bf16_elect(tb + T_R1, dk(sb + oPu, 8192, k), dmn(sb + oW3, 16384, k), id_kmn64, k > 0, el);
                umma_commit_elect(&s.bar_g3, el);
                // W3 aggregation on top of the master
                mbar_wait(&s.bar_ak, ph, wc, 300 + 7);
                tc_fence_after_sync();
#pragma unroll kIssueUnroll
                for (int k = 0; k < 4; ++k) umma_bf16_elect(tb + T_W3, dmn(sb + oPu, 8192, k), dmn(sb + oHdW, 8192, k), id_agg64, true, el);
                // W12 aggregation first (the next chunk's G1 hangs on it), then the two momentum aggregates
                mbar_wait(&s.bar_pz, ph, wc, 300 + 8);
                tc_fence_after_sync();
                if (multi) {  // the momentum aggregate is read out after every block, the weights' only after the chunk's last
#pragma unroll kIssueUnroll
                    for (int k = 0; k < 4; ++k) umma_bf16_elect(tb + T_R0, dmn(sb + oPzM, 8192, k), dmn(sb + oX, 16384, k), id_agg, k > 0, el);
                    umma_commit_elect(&s.bar_am12, el);
                }
#pragma unroll kIssueUnroll
                for (int k = 0; k < 4; ++k) umma_bf16_elect(tb + T_W12, dmn(sb + oPzW, 8192, k), dmn(sb + oX, 16384, k), id_agg, true, el);
                umma_commit_elect(&s.bar_aw12, el);
                if (!multi) {
#pragma unroll kIssueUnroll
                    for (int k = 0; k < 4; ++k) umma_bf16_elect(tb + T_R0, dmn(sb + oPzM, 8192, k), dmn(sb + oX, 16384, k), id_agg, k > 0, el);
                    umma_commit_elect(&s.bar_am12, el);
                }
#pragma unroll kIssueUnroll
                for (int k = 0; k < 4; ++k) umma_bf16_elect(tb + T_R1, dmn(sb + oPu, 8192, k), dmn(sb + oHdM, 8192, k), id_agg64, k > 0, el);
                umma_commit_elect(&s.bar_am3, el);
            }
        } else if (warp == NEW + 3) {
            // ------------------------------------------------------------------- token loads, gate scans, credits
            auto load_tokens = [&](int y) {
                mbar_expect_tx(&s.bar_x, (uint32_t)Cr * 512u);
                tma_load_2d(s.X[0], &tmK, 0, y, &s.bar_x);
                tma_load_2d(s.X[0] + 8192, &tmQ, 0, y, &s.bar_x);
                tma_load_2d(s.X[1], &tmK, 64, y, &s.bar_x);
                tma_load_2d(s.X[1] + 8192, &tmQ, 64, y, &s.bar_x);
            };
            for (int r = 0; r < nchunks; ++r) {
                const uint32_t ph = (uint32_t)(r & 1);
                const int tok0 = r * Cr;
                if (r == 0) {
                    if (lane == 0) load_tokens(seq * Ls);
                } else {
                    mbar_wait(&s.bar_w3, ph, wc, 300 + 20);  // the previous chunk is over in this CTA
                }
                if (lane == 0) {
                    mbar_expect_tx(&s.bar_partK, (uint32_t)((NC - 1) * nown * 512));
                    mbar_expect_tx(&s.bar_partQ, (uint32_t)((NC - 1) * nown * 256));
                    mbar_expect_tx(&s.bar_pu, (uint32_t)((C - nown) * 256));
                    if (r + 1 < nchunks) {
                        const int y = seq * Ls + tok0 + Cr;
                        tma_prefetch_l2_2d(&tmK, 0, y);
                        tma_prefetch_l2_2d(&tmQ, 0, y);
                        tma_prefetch_l2_2d(&tmK, 64, y);
                        tma_prefetch_l2_2d(&tmQ, 64, y);
                        tma_prefetch_l2_2d(&tmV, 0, y + t0);
                        tma_prefetch_l2_2d(&tmV, 64, y + t0);
                    }
                }
                __syncwarp();
                if (r + 1 < nchunks) {
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
                if (lane == 0) {
                    // the value rows of the owned key tokens (a box of 16 rows: the rows past the owned ones are not read)
                    mbar_expect_tx(&s.bar_v, 4096u);
                    const int y = seq * Ls + tok0 + t0;
                    tma_load_2d(s.Vrows, &tmV, 0, y, &s.bar_v);
                    tma_load_2d(s.Vrows + 2048, &tmV, 64, y, &s.bar_v);
                }
                if (r + 1 < nchunks) {
                    // the W12 / M12 aggregations were the last readers of the key tile: the next chunk's tokens may land in X
                    mbar_wait(multi ? &s.bar_aw12 : &s.bar_am12, ph, wc, 300 + 22);  // whichever was issued last
                    if (lane == 0) load_tokens(seq * Ls + tok0 + Cr);
                    // every reader of this chunk's staging / pu / scaled tiles is done once the aggregations have completed and
                    // every epilogue warp has left its layer norm (it has then released W12): credits to and from the peers
                    mbar_wait(&s.bar_am3, ph, wc, 300 + 23);
                    mbar_wait(&s.bar_w12, ph ^ 1u, wc, 300 + 24);
                    if (lane < NC && lane != (int)me) mbar_arrive_remote(map_to_cta(smem_u32(&s.bar_credit), (uint32_t)lane));
                    __syncwarp();
                    mbar_wait<true>(&s.bar_credit, ph, wc, 300 + 25);
                    if (lane == 0) mbar_arrive(&s.bar_go);
                    __syncwarp();
                }
            }
        }
    } else {
        // =====================================================================================================
        // epilogue warps
        // =====================================================================================================
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(EPI_REGS));
        const int q = warp & 3;          // TMEM lane quadrant
        const int g = warp >> 2;         // column group
        const int row = 32 * q + lane;   // TMEM lane this thread reads
        const uint32_t lane_addr = tb + ((uint32_t)(32 * q) << 16);
        const size_t dh = (size_t)D * h;
        const float inv_d = 1.0f / (float)D;
        __nv_bfloat16* go = a.o ? a.o + (size_t)seq * Ls * D : nullptr;
        const size_t head = (size_t)seq * a.final_seq_stride, head0 = (size_t)seq * a.init_seq_stride;
        float* const ck0 = a.ckpt ? a.ckpt + (size_t)seq * a.ckpt_seq_stride : nullptr;  // slot 0: the initial state
        // W12 row `row`: W1 (row < 64) or W2 row of hidden unit 64 me + (row & 63); this thread's columns 32 g ..
        const size_t off12 = ((size_t)(HS * me) + (row & 63)) * D + 32 * g;
        // W3c[i = row][j]: global W3 [d][h], this thread's columns 64 me + 16 g ..
        const size_t off3 = (size_t)row * h + HS * me + 16 * g;

        // ---- load the state: fp32 masters -> TMEM (pre-scaled by the first decay carry), bf16 copies -> shared, M -> registers
        float M12[32], M3[16];
        {
            const float cw0 = s.sc[0].cw, cm0 = s.sc[0].cm;
            const float* w12 = (row < 64 ? a.W1_init : a.W2_init) + head0 + off12;
            const float* m12p = row < 64 ? a.M1_init : a.M2_init;
            const float* m12 = m12p ? m12p + head0 + off12 : nullptr;
#pragma unroll
            for (int b = 0; b < 2; ++b) {
                float w[16];
                uint32_t st[16];
#pragma unroll
                for (int j = 0; j < 16; j += 4) {
                    const float4 x = *reinterpret_cast<const float4*>(w12 + 16 * b + j);
                    w[j] = x.x; w[j + 1] = x.y; w[j + 2] = x.z; w[j + 3] = x.w;
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    M12[16 * b + j] = m12 ? m12[16 * b + j] : 0.0f;
                    st[j] = __float_as_uint(multi ? fmaf(cm0, M12[16 * b + j], cw0 * w[j]) : cw0 * w[j]);
                }
                const int col = 32 * g + 16 * b;
                tmem_st16(lane_addr + T_W12 + col, st);
                uint32_t wu[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) wu[j] = __float_as_uint(w[j]);
                st_two_term(s.W12[col >> 6], s.W12lo[col >> 6], row, col & 63, wu);
                if (ck0) {
                    float* cw = ck0 + (row < 64 ? 0 : dh) + off12 + 16 * b;       // W1 | W2
                    float* cm_ = ck0 + (row < 64 ? 3 : 4) * dh + off12 + 16 * b;   // M1 | M2
#pragma unroll
                    for (int j = 0; j < 16; j += 4) {
                        *reinterpret_cast<float4*>(cw + j) = make_float4(w[j], w[j + 1], w[j + 2], w[j + 3]);
                        *reinterpret_cast<float4*>(cm_ + j) = make_float4(M12[16 * b + j], M12[16 * b + j + 1], M12[16 * b + j + 2], M12[16 * b + j + 3]);
                    }
                }
            }
            {
                const float* w3 = a.W3_init + head0 + off3;
                const float* m3 = a.M3_init ? a.M3_init + head0 + off3 : nullptr;
                float w[16];
                uint32_t st[16];
#pragma unroll
                for (int j = 0; j < 16; j += 4) {
                    const float4 x = *reinterpret_cast<const float4*>(w3 + j);
                    w[j] = x.x; w[j + 1] = x.y; w[j + 2] = x.z; w[j + 3] = x.w;
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    M3[j] = m3 ? m3[j] : 0.0f;
                    st[j] = __float_as_uint(multi ? fmaf(cm0, M3[j], cw0 * w[j]) : cw0 * w[j]);
                }
                tmem_st16(lane_addr + T_W3 + 16 * g, st);
                st_slab16(s.W3, row, 16 * g, w);
                if (ck0) {
#pragma unroll
                    for (int j = 0; j < 16; j += 4) {
                        *reinterpret_cast<float4*>(ck0 + 2 * dh + off3 + j) = make_float4(w[j], w[j + 1], w[j + 2], w[j + 3]);
                        *reinterpret_cast<float4*>(ck0 + 5 * dh + off3 + j) = make_float4(M3[j], M3[j + 1], M3[j + 2], M3[j + 3]);
                    }
                }
            }
            tmem_wait_st();
            warp_release(&s.bar_w12);
            if (lane == 0) mbar_arrive(&s.bar_w3);
        }

        for (int r = 0; r < nchunks; ++r) {
            const uint32_t ph = (uint32_t)(r & 1);
            const Scalars& sc = s.sc[r & 1];
            const int tok0 = r * Cr;
            const bool last = (r + 1 == nchunks);
            // ---------------- G1 epilogue: hd = silu(z1) z2 -> Hd (bf16), all that G2 needs.  The key rows' hd also goes, as
            // fp16, into the kW hd tile: the query-row warps turn it into bf16 kW hd and kM hd while G2 runs.
            mbar_wait(&s.bar_g1, ph, wc, 300 + 30);
            tc_fence_after_sync();
            {
                uint32_t z1[16], z2[16];
                tmem_ld16(lane_addr + T_R0 + 16 * g, z1);
                tmem_ld16(lane_addr + T_R0 + 64 + 16 * g, z2);
                tmem_wait_ld();
                uint32_t p[8], p16[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float za = __uint_as_float(z1[2 * i]), zb = __uint_as_float(z1[2 * i + 1]);
                    const float h0 = za * fast_sigmoid(za) * __uint_as_float(z2[2 * i]);
                    const float h1 = zb * fast_sigmoid(zb) * __uint_as_float(z2[2 * i + 1]);
                    p[i] = pack_bf16(h0, h1);
                    p16[i] = pack_f16(h0, h1);
                }
                st_slab16p(s.Hd, row, 16 * g, p);
                if (q < 2) st_slab16p(s.HdW, row, 16 * g, p16);
                warp_release(&s.bar_a);
                if (q < 2) {
                    // key rows: what the G3 epilogue multiplies by replaces z1, z2 in TMEM, in the shadow of G2:
                    //   d1 = z2 silu'(z1) = z2 s (1 + z1 (1 - s))   (pz1 = ph d1)      d2 = silu(z1)   (pz2 = ph d2)
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float z = __uint_as_float(z1[j]);
                        const float sg = fast_sigmoid(z);
                        z1[j] = __float_as_uint(__uint_as_float(z2[j]) * sg * fmaf(z, 1.0f - sg, 1.0f));
                        z2[j] = __float_as_uint(z * sg);
                    }
                    tmem_st16(lane_addr + T_R0 + 16 * g, z1);
                    tmem_st16(lane_addr + T_R0 + 64 + 16 * g, z2);
                    tmem_wait_st();
                } else {
                    // query-row warps: scale the key rows' hd by kW and kM (operands of the W3 aggregations).  256 threads over
                    // the [64 x 64] tile: 4 threads per row, 16 columns each; kW hd overwrites the fp16 copy in place.
                    mbar_wait(&s.bar_a, ph, wc, 300 + 38);
                    const int tq = 32 * (2 * g + (q & 1)) + lane;
                    const int ar = tq >> 2, ac = 16 * (tq & 3);
                    const float kw = sc.kW[ar], km = sc.kM[ar];
                    uint8_t* rw = s.HdW + ar * 128;
                    uint8_t* rm = s.HdM + ar * 128;
                    auto scale2 = [](uint32_t x, float k) {  // two packed fp16 times k -> two packed bf16
                        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&x));
                        return pack_bf16(k * f.x, k * f.y);
                    };
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        const int off = (((ac >> 3) + i) ^ (ar & 7)) << 4;
                        const uint4 v = *reinterpret_cast<const uint4*>(rw + off);
                        *reinterpret_cast<uint4*>(rw + off) = make_uint4(scale2(v.x, kw), scale2(v.y, kw), scale2(v.z, kw), scale2(v.w, kw));
                        *reinterpret_cast<uint4*>(rm + off) = make_uint4(scale2(v.x, km), scale2(v.y, km), scale2(v.z, km), scale2(v.w, km));
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&s.bar_ak);
                }
            }

            // ---------------- cross-CTA sum of Upart
            // TMEM lane 32q+l holds key token 32q+l (q < 2) or query token 32(q-2)+l; its owner normalises it.  Key rows
            // travel as fp32 (they feed the state), query rows as bf16 (they only feed o).  The sender's own rows stay
            // fp32 in the dead hd tile.  This thread's columns of U: 32 g ..
            const int tkn = 32 * (q & 1) + lane;
            const uint32_t owner = tok_owner(tkn);
            const uint32_t srow = (uint32_t)(tkn - tok_begin((int)owner));
            const uint32_t slot = (me + (uint32_t)NC - owner - 1u) % (uint32_t)NC;   // where the owner keeps what comes from this CTA
            const bool mine = owner == me;
            mbar_wait(&s.bar_g2, ph, wc, 300 + 31);
            tc_fence_after_sync();
            if (r > 0) mbar_wait(&s.bar_go, (uint32_t)((r - 1) & 1), wc, 300 + 32);

            auto layer_norm = [&](const bool key_rows) {
                // 16 threads per row, 8 columns each; 16 row slots per CTA of which nown are in use
                const int lrow = 2 * ((q & 1) + 2 * g) + (lane >> 4);
                const bool act = lrow < nown;
                const int cg = lane & 15;
                const int t = t0 + (act ? lrow : 0);         // token inside the chunk
                const int xrow = key_rows ? t : 64 + t;      // its row in the X tile
                const int col0 = 8 * cg;
                const int c = (col0 & 63) >> 3;
                const uint4 xraw = *reinterpret_cast<const uint4*>(s.X[col0 >> 6] + xrow * 128 + ((c ^ (xrow & 7)) << 4));
                float u[8];
                {   // own rows, fp32
                    const uint8_t* p = s.Hd + (key_rows ? 0 : 8192);
                    const float4 x0 = *reinterpret_cast<const float4*>(p + stage_offset((uint32_t)(2 * cg), (uint32_t)lrow));
                    const float4 x1 = *reinterpret_cast<const float4*>(p + stage_offset((uint32_t)(2 * cg + 1), (uint32_t)lrow));
                    u[0] = x0.x; u[1] = x0.y; u[2] = x0.z; u[3] = x0.w; u[4] = x1.x; u[5] = x1.y; u[6] = x1.z; u[7] = x1.w;
                }
                mbar_wait<true>(key_rows ? &s.bar_partK : &s.bar_partQ, ph, wc, 300 + 35);
                // the peers' pieces in a fixed order (slot 0..4 = the CTAs me+1 .. me+5): the sum does not depend on arrival order
                if (key_rows) {
#pragma unroll
                    for (int sl = 0; sl < NC - 1; ++sl) {
                        const uint8_t* sk = sl < 4 ? s.PzW[0] + sl * 8192 : s.StageK4;
                        const float4 x0 = *reinterpret_cast<const float4*>(sk + stage_offset((uint32_t)(2 * cg), (uint32_t)lrow));
                        const float4 x1 = *reinterpret_cast<const float4*>(sk + stage_offset((uint32_t)(2 * cg + 1), (uint32_t)lrow));
                        u[0] += x0.x; u[1] += x0.y; u[2] += x0.z; u[3] += x0.w; u[4] += x1.x; u[5] += x1.y; u[6] += x1.z; u[7] += x1.w;
                    }
                } else {
#pragma unroll
                    for (int sl = 0; sl < NC - 1; ++sl) {
                        const uint4 x = *reinterpret_cast<const uint4*>(s.StageQ[sl] + stage_offset_q((uint32_t)cg, (uint32_t)lrow));
                        const float2 f0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&x.x));
                        const float2 f1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&x.y));
                        const float2 f2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&x.z));
                        const float2 f3 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&x.w));
                        u[0] += f0.x; u[1] += f0.y; u[2] += f1.x; u[3] += f1.y; u[4] += f2.x; u[5] += f2.y; u[6] += f3.x; u[7] += f3.y;
                    }
                }
                if (!act) {  // rows past the owned ones hold stale data: keep them finite
#pragma unroll
                    for (int j = 0; j < 8; ++j) u[j] = 0.0f;
                }
                auto row_sum = [&](float v) -> float {  // over the 16 lanes that share a row
#pragma unroll
                    for (int o = 8; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                    return v;
                };
                float sum = 0.0f;
#pragma unroll
                for (int j = 0; j < 8; ++j) sum += u[j];
                const float mu = row_sum(sum) * inv_d;
                float sq = 0.0f;
#pragma unroll
                for (int j = 0; j < 8; ++j) { u[j] -= mu; sq = fmaf(u[j], u[j], sq); }
                const float rstd = rsqrtf(row_sum(sq) * inv_d + a.eps);
#pragma unroll
                for (int j = 0; j < 8; ++j) u[j] *= rstd;  // y
                const __nv_bfloat162* x2 = reinterpret_cast<const __nv_bfloat162*>(&xraw);
                if (key_rows) {
                    // key rows: e = k + y - v, pu = rstd (e - mean(e) - y mean(e y))
                    mbar_wait(&s.bar_v, ph, wc, 300 + 36);
                    const int lr = act ? lrow : 0;
                    const uint4 vraw = *reinterpret_cast<const uint4*>(s.Vrows + (col0 >> 6) * 2048 + lr * 128 + ((c ^ (lr & 7)) << 4));
                    const __nv_bfloat162* v2 = reinterpret_cast<const __nv_bfloat162*>(&vraw);
                    float e[8];
                    float se = 0.0f, sey = 0.0f;
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        const float2 kf = __bfloat1622float2(x2[x]), vf = __bfloat1622float2(v2[x]);
                        e[2 * x] = kf.x + u[2 * x] - vf.x;
                        e[2 * x + 1] = kf.y + u[2 * x + 1] - vf.y;
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) { se += e[j]; sey = fmaf(e[j], u[j], sey); }
                    const float me_ = row_sum(se) * inv_d;
                    const float mey = row_sum(sey) * inv_d;
                    if (act) {
                        *reinterpret_cast<uint4*>(s.Pu[col0 >> 6] + t * 128 + ((c ^ (t & 7)) << 4)) =
                            make_uint4(pack_bf16(rstd * (e[0] - me_ - u[0] * mey), rstd * (e[1] - me_ - u[1] * mey)),
                                       pack_bf16(rstd * (e[2] - me_ - u[2] * mey), rstd * (e[3] - me_ - u[3] * mey)),
                                       pack_bf16(rstd * (e[4] - me_ - u[4] * mey), rstd * (e[5] - me_ - u[5] * mey)),
                                       pack_bf16(rstd * (e[6] - me_ - u[6] * mey), rstd * (e[7] - me_ - u[7] * mey)));
                    }
                    // the owned pu rows are contiguous in each slab: one bulk copy per peer and slab carries them over
                    fence_proxy_async_smem();
                    named_sync(BAR_KOWN, NEPI / 2);
                    if (warp == 0) {
                        if (lane < 2 * (NC - 1)) {
                            const uint32_t dst = (me + 1u + (uint32_t)(lane >> 1)) % (uint32_t)NC;
                            const uint32_t src = smem_u32(s.Pu[lane & 1]) + 128u * (uint32_t)t0;
                            bulk_copy_to_cta(map_to_cta(src, dst), src, 128u * (uint32_t)nown, map_to_cta(smem_u32(&s.bar_pu), dst));
                        }
                        if (lane == 0) mbar_arrive(&s.bar_pu);  // the own rows are in place
                    }
                } else if (act && t < min(Cr, L - tok0) && go) {
                    // query rows: o = q + y
                    uint4 ov;
                    const float2 q0 = __bfloat1622float2(x2[0]), q1 = __bfloat1622float2(x2[1]), q2 = __bfloat1622float2(x2[2]),
                                 q3 = __bfloat1622float2(x2[3]);
                    ov.x = pack_bf16(q0.x + u[0], q0.y + u[1]);
                    ov.y = pack_bf16(q1.x + u[2], q1.y + u[3]);
                    ov.z = pack_bf16(q2.x + u[4], q2.y + u[5]);
                    ov.w = pack_bf16(q3.x + u[6], q3.y + u[7]);
                    *reinterpret_cast<uint4*>(go + (size_t)(tok0 + t) * D + col0) = ov;
                }
            };

            if (q < 2) {
                // key rows out first
                {
                    uint32_t dst_base, dst_bar = 0;
                    if (mine) {
                        dst_base = smem_u32(s.Hd);  // the hd tile is dead once G2 has completed
                    } else {
                        dst_base = map_to_cta(slot < 4u ? smem_u32(s.PzW[0]) + slot * 8192u : smem_u32(s.StageK4), owner);
                        dst_bar = map_to_cta(smem_u32(&s.bar_partK), owner);
                    }
#pragma unroll
                    for (int b = 0; b < 2; ++b) {
                        uint32_t u[16];
                        tmem_ld16(lane_addr + T_R1 + 32 * g + 16 * b, u);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 16; j += 4) {
                            const uint32_t dst = dst_base + stage_offset((uint32_t)((32 * g + 16 * b + j) >> 2), srow);
                            if (mine) st_cluster_v4_b32(dst, u[j], u[j + 1], u[j + 2], u[j + 3]);
                            else st_async_v4(dst, u[j], u[j + 1], u[j + 2], u[j + 3], dst_bar);
                        }
                    }
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) { mbar_arrive(&s.bar_r1); mbar_arrive(&s.bar_ksent); }
                }
                named_sync(BAR_KOWN, NEPI / 2);  // this CTA's own key rows are staged
                layer_norm(true);
                // ---------------- G3 epilogue: pz1 = ph d1, pz2 = ph d2, scaled by kW and kM into two bf16 tiles each
                mbar_wait(&s.bar_g3, ph, wc, 300 + 33);
                tc_fence_after_sync();
                {
                    const float kw = sc.kW[row], km = sc.kM[row];
                    uint32_t phv[16], d1[16], d2[16];
                    tmem_ld16(lane_addr + T_R1 + 16 * g, phv);
                    tmem_ld16(lane_addr + T_R0 + 16 * g, d1);
                    tmem_ld16(lane_addr + T_R0 + 64 + 16 * g, d2);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        d1[j] = __float_as_uint(__uint_as_float(phv[j]) * __uint_as_float(d1[j]));  // pz1
                        d2[j] = __float_as_uint(__uint_as_float(phv[j]) * __uint_as_float(d2[j]));  // pz2
                    }
                    uint32_t p[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) p[i] = pack_bf16(kw * __uint_as_float(d1[2 * i]), kw * __uint_as_float(d1[2 * i + 1]));
                    st_slab16p(s.PzW[0], row, 16 * g, p);
#pragma unroll
                    for (int i = 0; i < 8; ++i) p[i] = pack_bf16(kw * __uint_as_float(d2[2 * i]), kw * __uint_as_float(d2[2 * i + 1]));
                    st_slab16p(s.PzW[1], row, 16 * g, p);
#pragma unroll
                    for (int i = 0; i < 8; ++i) p[i] = pack_bf16(km * __uint_as_float(d1[2 * i]), km * __uint_as_float(d1[2 * i + 1]));
                    st_slab16p(s.PzM[0], row, 16 * g, p);
#pragma unroll
                    for (int i = 0; i < 8; ++i) p[i] = pack_bf16(km * __uint_as_float(d2[2 * i]), km * __uint_as_float(d2[2 * i + 1]));
                    st_slab16p(s.PzM[1], row, 16 * g, p);
                }
                warp_release(&s.bar_pz);
            } else {
                mbar_wait(&s.bar_ksent, ph, wc, 300 + 34);
                {
                    const uint32_t own_base = smem_u32(s.Hd) + 8192u;
                    const uint32_t dst_base = map_to_cta(smem_u32(s.StageQ[0]) + slot * 4096u, owner);
                    const uint32_t dst_bar = map_to_cta(smem_u32(&s.bar_partQ), owner);
#pragma unroll
                    for (int b = 0; b < 2; ++b) {
                        uint32_t u[16];
                        tmem_ld16(lane_addr + T_R1 + 32 * g + 16 * b, u);
                        tmem_wait_ld();
                        if (mine) {
#pragma unroll
                            for (int j = 0; j < 16; j += 4)
                                st_cluster_v4_b32(own_base + stage_offset((uint32_t)((32 * g + 16 * b + j) >> 2), srow), u[j], u[j + 1], u[j + 2], u[j + 3]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 16; j += 8)
                                st_async_v4(dst_base + stage_offset_q((uint32_t)((32 * g + 16 * b + j) >> 3), srow),
                                            pack_bf16(__uint_as_float(u[j]), __uint_as_float(u[j + 1])),
                                            pack_bf16(__uint_as_float(u[j + 2]), __uint_as_float(u[j + 3])),
                                            pack_bf16(__uint_as_float(u[j + 4]), __uint_as_float(u[j + 5])),
                                            pack_bf16(__uint_as_float(u[j + 6]), __uint_as_float(u[j + 7])), dst_bar);
                        }
                    }
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&s.bar_r1);
                }
                named_sync(BAR_QOWN, NEPI / 2);  // own query rows staged
                layer_norm(false);
            }

            // ---------------- state pass (Algorithm 1 lines 6-7)
            if (!last) mbar_wait(&s.bar_sc, ph, wc, 300 + 37);  // the next chunk's scalars (its decay carry pre-scales the masters)
            const float cm = sc.cm, cb = sc.cb;
            const float cwn = last ? 1.0f : s.sc[(r + 1) & 1].cw;
            // slot of the state after this chunk in the saved states (every chunk's, or every ckpt_every-th)
            const int ce = max(a.ckpt_every, 1);
            float* const ckn = ck0 ? ck0 + (size_t)((r + 1) / ce) * 6 * dh : nullptr;
            const bool save_ck = ck0 && !last && (r + 1) % ce == 0;
            if constexpr (MULTI) {
                // ---- chunks of several 64-token blocks (see the GELU-MLP kernel): the bf16 copies and the masters' pre-scaling
                // are refreshed after the chunk's last block only; the master carries cw W_0 + cm M_0, so the momentum
                // registers follow the blocks (M = cb M_0 + aggregate on the first block, M += aggregate afterwards).
                const int bidx = r % m;
                const bool final_block = bidx == m - 1 || last;
                const float cbk = bidx == 0 ? cb : 1.0f;
                const float cwn2 = last ? 1.0f : s.sc[(r + 1) & 1].cw, cmn2 = last ? 0.0f : s.sc[(r + 1) & 1].cm;
                const int cdone = r / m + 1;
                const bool save2 = ck0 && final_block && !last && cdone % ce == 0;
                float* const ck2 = ck0 ? ck0 + (size_t)(cdone / ce) * 6 * dh : nullptr;
                const bool wr = final_block && (last || save2);
                mbar_wait(&s.bar_am12, ph, wc, 300 + 39);
                tc_fence_after_sync();
#pragma unroll
                for (int b = 0; b < 2; ++b) {
                    uint32_t ma[16];
                    tmem_ld16(lane_addr + T_R0 + 32 * g + 16 * b, ma);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 16; ++j) M12[16 * b + j] = fmaf(cbk, M12[16 * b + j], __uint_as_float(ma[j]));
                    if (wr) {
                        float* dst = (last ? (row < 64 ? a.M1_final : a.M2_final) + head : ck2 + (row < 64 ? 3 : 4) * dh) + off12 + 16 * b;
#pragma unroll
                        for (int j = 0; j < 16; j += 4)
                            *reinterpret_cast<float4*>(dst + j) = make_float4(M12[16 * b + j], M12[16 * b + j + 1], M12[16 * b + j + 2], M12[16 * b + j + 3]);
                    }
                }
                if (final_block) {
                    mbar_wait(&s.bar_aw12, ph, wc, 300 + 38);
                    tc_fence_after_sync();
#pragma unroll
                    for (int b = 0; b < 2; ++b) {
                        const int col = 32 * g + 16 * b;
                        uint32_t wa[16];
                        tmem_ld16(lane_addr + T_W12 + col, wa);
                        tmem_wait_ld();
                        st_two_term(s.W12[col >> 6], s.W12lo[col >> 6], row, col & 63, wa);
                        if (wr) {
                            float* dst = (last ? (row < 64 ? a.W1_final : a.W2_final) + head : ck2 + (row < 64 ? 0 : dh)) + off12 + 16 * b;
#pragma unroll
                            for (int j = 0; j < 16; j += 4) *reinterpret_cast<uint4*>(dst + j) = make_uint4(wa[j], wa[j + 1], wa[j + 2], wa[j + 3]);
                        }
#pragma unroll
                        for (int j = 0; j < 16; ++j) wa[j] = __float_as_uint(fmaf(cmn2, M12[16 * b + j], cwn2 * __uint_as_float(wa[j])));
                        tmem_st16(lane_addr + T_W12 + col, wa);
                    }
                }
                tmem_wait_st();
                warp_release(&s.bar_w12);  // R0 free (and, after a final block, W12 refreshed)
                mbar_wait(&s.bar_am3, ph, wc, 300 + 40);
                tc_fence_after_sync();
                {
                    uint32_t ma[16];
                    tmem_ld16(lane_addr + T_R1 + 16 * g, ma);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 16; ++j) M3[j] = fmaf(cbk, M3[j], __uint_as_float(ma[j]));
                    if (wr) {
                        float* dst = (last ? a.M3_final + head : ck2 + 5 * dh) + off3;
#pragma unroll
                        for (int j = 0; j < 16; j += 4) *reinterpret_cast<float4*>(dst + j) = make_float4(M3[j], M3[j + 1], M3[j + 2], M3[j + 3]);
                    }
                    if (final_block) {
                        uint32_t wa[16];
                        tmem_ld16(lane_addr + T_W3 + 16 * g, wa);
                        tmem_wait_ld();
                        uint32_t p[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) p[i] = pack_bf16(__uint_as_float(wa[2 * i]), __uint_as_float(wa[2 * i + 1]));
                        st_slab16p(s.W3, row, 16 * g, p);
                        if (wr) {
                            float* dst = (last ? a.W3_final + head : ck2 + 2 * dh) + off3;
#pragma unroll
                            for (int j = 0; j < 16; j += 4) *reinterpret_cast<uint4*>(dst + j) = make_uint4(wa[j], wa[j + 1], wa[j + 2], wa[j + 3]);
                        }
#pragma unroll
                        for (int j = 0; j < 16; ++j) wa[j] = __float_as_uint(fmaf(cmn2, M3[j], cwn2 * __uint_as_float(wa[j])));
                        tmem_st16(lane_addr + T_W3 + 16 * g, wa);
                    }
                }
                tmem_wait_st();
                warp_release(&s.bar_w3);  // R1 free (and, after a final block, W3 refreshed)
            } else {
            // W12 half, as soon as its aggregation is in (the momentum aggregate follows right behind it)
            mbar_wait(&s.bar_aw12, ph, wc, 300 + 38);
            tc_fence_after_sync();
#pragma unroll
            for (int b = 0; b < 2; ++b) {
                const int col = 32 * g + 16 * b;
                uint32_t wa[16];  // the new weights, in place: unscaled first, then pre-scaled for the next chunk
                tmem_ld16(lane_addr + T_W12 + col, wa);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 16; ++j) wa[j] = __float_as_uint(fmaf(cm, M12[16 * b + j], __uint_as_float(wa[j])));
                st_two_term(s.W12[col >> 6], s.W12lo[col >> 6], row, col & 63, wa);
                if (last || save_ck) {
                    float* dst = (last ? (row < 64 ? a.W1_final : a.W2_final) + head : ckn + (row < 64 ? 0 : dh)) + off12 + 16 * b;
#pragma unroll
                    for (int j = 0; j < 16; j += 4) *reinterpret_cast<uint4*>(dst + j) = make_uint4(wa[j], wa[j + 1], wa[j + 2], wa[j + 3]);
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) wa[j] = __float_as_uint(cwn * __uint_as_float(wa[j]));
                tmem_st16(lane_addr + T_W12 + col, wa);
            }
            mbar_wait(&s.bar_am12, ph, wc, 300 + 39);
            tc_fence_after_sync();
#pragma unroll
            for (int b = 0; b < 2; ++b) {
                uint32_t ma[16];
                tmem_ld16(lane_addr + T_R0 + 32 * g + 16 * b, ma);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 16; ++j) M12[16 * b + j] = fmaf(cb, M12[16 * b + j], __uint_as_float(ma[j]));
                if (last || save_ck) {
                    float* dst = (last ? (row < 64 ? a.M1_final : a.M2_final) + head : ckn + (row < 64 ? 3 : 4) * dh) + off12 + 16 * b;
#pragma unroll
                    for (int j = 0; j < 16; j += 4)
                        *reinterpret_cast<float4*>(dst + j) = make_float4(M12[16 * b + j], M12[16 * b + j + 1], M12[16 * b + j + 2], M12[16 * b + j + 3]);
                }
            }
            tmem_wait_st();
            warp_release(&s.bar_w12);  // bf16 W12 complete, master rescaled, R0 free: the next chunk's G1 may run

            // W3 half
            mbar_wait(&s.bar_am3, ph, wc, 300 + 40);
            tc_fence_after_sync();
            {
                uint32_t wa[16];
                tmem_ld16(lane_addr + T_W3 + 16 * g, wa);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 16; ++j) wa[j] = __float_as_uint(fmaf(cm, M3[j], __uint_as_float(wa[j])));
                uint32_t p[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) p[i] = pack_bf16(__uint_as_float(wa[2 * i]), __uint_as_float(wa[2 * i + 1]));
                st_slab16p(s.W3, row, 16 * g, p);
                if (last || save_ck) {
                    float* dst = (last ? a.W3_final + head : ckn + 2 * dh) + off3;
#pragma unroll
                    for (int j = 0; j < 16; j += 4) *reinterpret_cast<uint4*>(dst + j) = make_uint4(wa[j], wa[j + 1], wa[j + 2], wa[j + 3]);
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) wa[j] = __float_as_uint(cwn * __uint_as_float(wa[j]));
                tmem_st16(lane_addr + T_W3 + 16 * g, wa);
                uint32_t ma[16];
                tmem_ld16(lane_addr + T_R1 + 16 * g, ma);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 16; ++j) M3[j] = fmaf(cb, M3[j], __uint_as_float(ma[j]));
                if (last || save_ck) {
                    float* dst = (last ? a.M3_final + head : ckn + 5 * dh) + off3;
#pragma unroll
                    for (int j = 0; j < 16; j += 4) *reinterpret_cast<float4*>(dst + j) = make_float4(M3[j], M3[j + 1], M3[j + 2], M3[j + 3]);
                }
            }
            tmem_wait_st();
            warp_release(&s.bar_w3);  // bf16 W3 complete, master rescaled, R1 free: the next chunk's G2 may run
            }  // single-block chunks
        }
    }

    // no CTA leaves while a peer may still write into its shared memory or arrive on its barriers
    tc_fence_before_sync();
    __syncwarp();
    cluster_sync();
    if (warp == 0) tmem_dealloc(tb, 512);
}

}  // namespace

size_t tc_swiglu_smem_bytes() { return sizeof(Smem); }

int tc_swiglu_launch(const TcSwigluArgs& a_in, void* stream) {
    TcSwigluArgs a = a_in;
    if (a.C == 0) a.C = C;
    if (a.Ls == 0) a.Ls = a.L;
    if (a.init_seq_stride == 0) a.init_seq_stride = (size_t)D * NC * HS;
    if (a.final_seq_stride == 0) a.final_seq_stride = (size_t)D * NC * HS;
    if (a.Ls < a.L) return (int)cudaErrorInvalidValue;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    CUtensorMap tmK, tmQ, tmV;
    const size_t rows = (size_t)(a.N - 1) * a.Ls + a.L;  // token rows the maps cover: up to the end of the last sequence's range
    const int Cc = a.C;
    if ((Cc != 512 && Cc != 256 && Cc != 128 && Cc != 64 && Cc != 32 && Cc != 16) || a.L <= 0) return (int)cudaErrorInvalidValue;
    const unsigned box_rows = (unsigned)(Cc < 64 ? Cc : 64);
    if (!make_token_map(&tmK, a.k, rows, box_rows, D) || !make_token_map(&tmQ, a.q, rows, box_rows, D) || !make_token_map(&tmV, a.v, rows, 16, D))
        return (int)cudaErrorInvalidValue;
    static bool attr_done[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return (int)cudaGetLastError();
    const int smem = (int)tc_swiglu_smem_bytes();
    if (dev < 0 || dev >= 64 || !attr_done[dev]) {
        cudaError_t e = cudaFuncSetAttribute(tc_swiglu_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_swiglu_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
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
    e = a.C > 64 ? cudaLaunchKernelEx(&cfg, tc_swiglu_kernel<true>, tmK, tmQ, tmV, a)
                 : cudaLaunchKernelEx(&cfg, tc_swiglu_kernel<false>, tmK, tmQ, tmV, a);
    if (e != cudaSuccess) return (int)e;
    return (int)cudaGetLastError();
}

}  // namespace e2ttt
