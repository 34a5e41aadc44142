// CTA-level GEMM engines of the any-shape kernels.
//
// Both engines compute   out(m, n) = sum_k a(m, k) * b(n, k),  m < M, n < N, k < K,
// for NACC (1 or 2) A operands that share one B, through callables:
//   fa(m, k, a0, a1) writes the A value(s); fb(n, k) returns the B value;
//   run    : epi(m, n, acc0, acc1) consumes a result;
//   run_rmw: pre(m, n) returns what the result has to be combined with (anything loaded from memory), and
//            epi(m, n, acc0, acc1, loaded) consumes it.  The engine calls pre for a batch of results before the
//            batch's epi calls, so that the loads are in flight together instead of one memory round trip per result
//            (the compiler cannot move a load of epi above the previous result's store: they may alias).
// Output tiles are dealt round-robin to the `nranks` CTAs of the sequence's cluster; run() ends with phase_sync().
//
//   FmaGemm<Real> : CUDA-core FMAs in the kernel's own precision (fp64 for fp32 I/O, fp32 for bf16 I/O).
//   TcGemm        : the 5th-generation tensor cores (tcgen05.mma, fp32 accumulation in tensor memory).  Every fp32
//                   operand x is staged as two bf16 numbers, hi = bf16(x) and lo = bf16(x - hi), and a product is
//                   three MMAs, hi*hi + hi*lo + lo*hi: the dropped lo*lo term and the residual of the split are
//                   ~2^-16 relative, so the result matches an fp32 FMA chain to a few 1e-5.  (Plain bf16 operands
//                   put the SwiGLU momentum of a single chunk outside the 2e-2 parity bound; the staging from L2,
//                   not the MMA count, bounds this engine.)
#pragma once
#include "simt_common.cuh"
#include "sm100.cuh"

namespace e2ttt {

template <typename Real> struct FmaGemm {
    static constexpr int kThreads = kSimtThreads;
    static constexpr size_t kBytes = sizeof(GemmSmem<Real>);
    GemmSmem<Real>* sm;
    int rank, nranks;
    __device__ static unsigned char* align(unsigned char* raw) { return raw; }
    __device__ void setup(unsigned char* base, int* /*status*/, int rank_, int nranks_) {
        sm = reinterpret_cast<GemmSmem<Real>*>(base);
        rank = rank_;
        nranks = nranks_;
    }
    __device__ void teardown() {}
    __device__ void set_scratch(Real*) {}
    template <int NACC, bool A_KFAST, bool B_KFAST, typename FA, typename FB, typename FP, typename FE>
    __device__ void run_rmw(int M, int N, int K, FA fa, FB fb, FP pre, FE epi) {
        block_gemm<Real, NACC, A_KFAST, B_KFAST>(M, N, K, fa, fb, pre, epi, sm, rank, nranks);
    }
    template <int NACC, bool A_KFAST, bool B_KFAST, typename FA, typename FB, typename FE>
    __device__ void run(int M, int N, int K, FA fa, FB fb, FE epi) {
        run_rmw<NACC, A_KFAST, B_KFAST>(M, N, K, fa, fb, [](int, int) { return 0; },
                                        [&](int m, int n, Real a0, Real a1, int) { epi(m, n, a0, a1); });
    }
};

// ---- tensor-core engine ---------------------------------------------------------------------------------------
// A tile is 128 output columns n (one per tensor-memory lane) by 64 output rows m (tensor-memory columns): the
// accumulator is held transposed, so that in the epilogue the 32 lanes of a warp own 32 consecutive n - the
// contiguous index of every result matrix - and global accesses of `epi` coalesce.
// In MMA terms: A operand = the fb rows (128 x k), B operand = the fa rows (64 x k), D[n][m] in tensor memory.
// The contraction runs in slices of 64 k.  A slice of an operand is one "slab": rows of 128 bytes (64 bf16),
// 16-byte chunk c of row r stored at chunk position c ^ (r & 7) (the 128-byte swizzle of the MMA descriptors).
// Two stages: while the tensor core works on one slice, all threads stage the next.
// Split-K: a product with fewer output tiles than CTAs in the cluster (a [tokens x d] result with a long contraction)
// is cut along k into as many parts as there are idle CTAs; every part writes its raw accumulators to a scratch area
// of the workspace, and after a phase barrier all CTAs sum the parts in a fixed order (so the result does not depend
// on timing) and run the epilogue elementwise.
constexpr int kTgStages = 2;
constexpr int kTgBN = 128;
constexpr int kTgBM = 64;
constexpr int kTgBK = 64;
constexpr uint32_t kTgTmemCols = 128;  // two accumulators of 64 columns
constexpr int kTgThreads = 512;        // 16 warps: four per tensor-memory lane quadrant, 16 accumulator columns each
constexpr int kTgMaxParts = 8;         // split-K: parts x tiles <= 8 (the largest cluster)
constexpr size_t kTgScratchElems = (size_t)2 * kTgMaxParts * kTgBN * kTgBM;  // floats per sequence

struct __align__(1024) TcGemmSmem {
    uint8_t R[kTgStages][2][kTgBN * 128];      // fb operand, row = n; [hi, lo]
    uint8_t Cc[kTgStages][2][2][kTgBM * 128];  // fa operand(s), row = m; [accumulator][hi, lo]
    uint64_t bar[kTgStages];                // "the MMAs that read this stage are done"
    uint32_t tmem_base;
    int dead;
};

// Stage ROWS x (8 * nchunk) values into one slab pair (hi, lo) - two pairs when NOUT == 2, from one call of `get`.
// KFAST says that k is the contiguous index of the source: then neighbouring threads take neighbouring k chunks
// of one row, else neighbouring rows of one k chunk, so that the source reads coalesce either way.
// A thread first loads all of its values, then converts and stores them: the loads are in flight together.
__device__ __forceinline__ void tg_split_store(uint8_t* hi, uint8_t* lo, uint32_t off, const float (&v)[8]) {
    uint32_t h[4], l[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const __nv_bfloat162 hh = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
        const float2 hf = __bfloat1622float2(hh);
        h[j] = *reinterpret_cast<const uint32_t*>(&hh);
        l[j] = sm100::pack_bf16(v[2 * j] - hf.x, v[2 * j + 1] - hf.y);
    }
    *reinterpret_cast<uint4*>(hi + off) = make_uint4(h[0], h[1], h[2], h[3]);
    *reinterpret_cast<uint4*>(lo + off) = make_uint4(l[0], l[1], l[2], l[3]);
}

template <int ROWS, bool KFAST, int NOUT, typename G>
__device__ __forceinline__ void tg_fill(uint8_t* hi0, uint8_t* lo0, uint8_t* hi1, uint8_t* lo1, int nchunk, G get) {
    constexpr int T = ROWS * 8 / kTgThreads;  // tasks (16-byte chunks) per thread when the slice is full
    const int tasks = ROWS * nchunk;
    float v0[T][8], v1[NOUT == 2 ? T : 1][8];
    uint32_t off[T];
#pragma unroll
    for (int t = 0; t < T; ++t) {
        const int idx = threadIdx.x + t * kTgThreads;
        int row, ch;
        if (KFAST) {
            ch = idx % nchunk;
            row = idx / nchunk;
        } else {
            row = idx % ROWS;
            ch = idx / ROWS;
        }
        off[t] = (uint32_t)row * 128u + ((uint32_t)(ch ^ (row & 7)) << 4);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            v0[t][j] = 0.0f;
            float w = 0.0f;
            if (idx < tasks) get(row, ch * 8 + j, v0[t][j], w);
            if (NOUT == 2) v1[t][j] = w;
        }
    }
#pragma unroll
    for (int t = 0; t < T; ++t) {
        if (threadIdx.x + t * kTgThreads < tasks) {
            tg_split_store(hi0, lo0, off[t], v0[t]);
            if (NOUT == 2) tg_split_store(hi1, lo1, off[t], v1[t]);
        }
    }
}

#ifdef SIMT_PROFILE
// Debug build only: cycles thread 0 of CTA 0 spends in each section of TcGemm::run_rmw, summed over the launch.
__device__ long long g_tg_prof[16];
#define TGPROF(i)                                                          \
    do {                                                                   \
        if (threadIdx.x == 0 && blockIdx.x == 0) {                         \
            const long long now_ = clock64();                              \
            g_tg_prof[i] += now_ - tgp_;                                   \
            tgp_ = now_;                                                   \
        }                                                                  \
    } while (0)
#define TGPROF_START() long long tgp_ = clock64()
#else
#define TGPROF(i)
#define TGPROF_START()
#endif

// SPLITK = false compiles the split-K path out (the forward kernel: its clusters are small and its code size matters).
template <bool SPLITK> struct TcGemmT {
    static constexpr int kThreads = kTgThreads;
    static constexpr size_t kBytes = sizeof(TcGemmSmem);
    TcGemmSmem* sm;
    uint32_t tmem;
    uint32_t it;  // slices issued so far by this CTA: slice `it` uses stage it & 1 and is that stage's (it >> 1)-th use
    sm100::WaitCtx wc;
    int rank, nranks;
    float* scratch;  // split-K partial sums of this sequence (kTgScratchElems floats), or nullptr: no split-K

    __device__ void set_scratch(float* p) { scratch = p; }

    // the slabs need 1024-byte alignment; the dynamic shared memory carries 1024 bytes of slack for it
    __device__ static unsigned char* align(unsigned char* raw) {
        const uint32_t a = sm100::smem_u32(raw);
        return raw + ((1024u - (a & 1023u)) & 1023u);
    }
    __device__ void setup(unsigned char* base, int* status, int rank_, int nranks_) {
        sm = reinterpret_cast<TcGemmSmem*>(base);
        rank = rank_;
        nranks = nranks_;
        it = 0;
        scratch = nullptr;
        if (threadIdx.x == 0) {
            for (int s = 0; s < kTgStages; ++s) sm100::mbar_init(&sm->bar[s], 1);
            sm->dead = 0;
            sm100::fence_mbar_init();
        }
        if (threadIdx.x < 32) {
            sm100::tmem_alloc(&sm->tmem_base, kTgTmemCols);
            sm100::tmem_relinquish();
        }
        sm100::tc_fence_before_sync();
        __syncthreads();
        sm100::tc_fence_after_sync();
        tmem = sm->tmem_base;
        wc.dead = &sm->dead;
        wc.status = status;
    }
    __device__ void teardown() {
        sm100::tc_fence_before_sync();
        __syncthreads();
        if (threadIdx.x < 32) sm100::tmem_dealloc(tmem, kTgTmemCols);
    }

    template <int NACC, bool A_KFAST, bool B_KFAST, typename FA, typename FB, typename FE>
    __device__ void run(int M, int N, int K, FA fa, FB fb, FE epi) {
        run_rmw<NACC, A_KFAST, B_KFAST>(M, N, K, fa, fb, [](int, int) { return 0; },
                                        [&](int m, int n, float a0, float a1, int) { epi(m, n, a0, a1); });
    }

    template <int NACC, bool A_KFAST, bool B_KFAST, typename FA, typename FB, typename FP, typename FE>
    __device__ void run_rmw(int M, int N, int K, FA fa, FB fb, FP pre, FE epi) {
        using namespace sm100;
        const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
        const uint32_t idesc = make_idesc(kTgBN, kTgBM, false, false);
        const int tiles_m = (M + kTgBM - 1) / kTgBM, tiles = ((N + kTgBN - 1) / kTgBN) * tiles_m;
        const int nslab = (K + kTgBK - 1) / kTgBK;
        int parts = 1;
        if (SPLITK && scratch && tiles < nranks && nslab >= 2) parts = min(min(nranks / tiles, nslab), kTgMaxParts / tiles);
        if (parts < 1) parts = 1;
        const int slabs_per_part = (nslab + parts - 1) / parts;
        TGPROF_START();
        for (int w = rank; w < tiles * parts; w += nranks) {  // work item = (tile, k part)
            const int tile = w / parts, part = w - tile * parts;
            const int n0 = (tile / tiles_m) * kTgBN, m0 = (tile % tiles_m) * kTgBM;
            const int kbeg = part * slabs_per_part * kTgBK, kend = min(K, kbeg + slabs_per_part * kTgBK);
            if (SPLITK && kbeg >= kend) {  // an empty part (more parts than slices): its partial sum is zero
                for (int e = tid; e < NACC * kTgBM * kTgBN; e += kTgThreads) {
                    const int acc = e / (kTgBM * kTgBN), r = e - acc * (kTgBM * kTgBN);
                    scratch[((size_t)(acc * kTgMaxParts + part * tiles + tile)) * (kTgBM * kTgBN) + r] = 0.0f;
                }
                continue;
            }
            {
                uint32_t last_it = 0;
                for (int k0 = kbeg; k0 < kend; k0 += kTgBK) {
                    const uint32_t s = it & 1u;
                    // the MMAs of the slice that used this stage two slices ago have read it
                    if (it >= 2) mbar_wait(&sm->bar[s], ((it >> 1) - 1u) & 1u, wc, 200 + 1);
                    TGPROF(0);
                    const int kc16 = (min(kTgBK, K - k0) + 15) >> 4;  // MMAs (16 k each) in this slice
                    tg_fill<kTgBN, B_KFAST, 1>(sm->R[s][0], sm->R[s][1], nullptr, nullptr, 2 * kc16,
                                               [&](int r, int kk, float& v0, float&) {
                                                   if (n0 + r < N && k0 + kk < K) v0 = (float)fb(n0 + r, k0 + kk);
                                               });
                    TGPROF(1);
                    tg_fill<kTgBM, A_KFAST, NACC>(sm->Cc[s][0][0], sm->Cc[s][0][1], sm->Cc[s][1][0], sm->Cc[s][1][1], 2 * kc16,
                                                  [&](int r, int kk, float& v0, float& v1) {
                                                      if (m0 + r < M && k0 + kk < K) {
                                                          float a0 = 0.0f, a1 = 0.0f;
                                                          fa(m0 + r, k0 + kk, a0, a1);
                                                          v0 = a0;
                                                          v1 = a1;
                                                      }
                                                  });
                    TGPROF(2);
                    fence_proxy_async_smem();
                    __syncthreads();
                    TGPROF(3);
                    if (tid == 0) {
                        tc_fence_after_sync();
                        for (int k = 0; k < kc16; ++k) {
                            const uint64_t da_hi = make_smem_desc(smem_u32(sm->R[s][0]) + 32u * k, 16, 1024);
                            const uint64_t da_lo = make_smem_desc(smem_u32(sm->R[s][1]) + 32u * k, 16, 1024);
#pragma unroll
                            for (int acc = 0; acc < NACC; ++acc) {
                                const uint64_t db_hi = make_smem_desc(smem_u32(sm->Cc[s][acc][0]) + 32u * k, 16, 1024);
                                const uint64_t db_lo = make_smem_desc(smem_u32(sm->Cc[s][acc][1]) + 32u * k, 16, 1024);
                                const uint32_t dst = tmem + (uint32_t)(acc * kTgBM);
                                umma_bf16(dst, da_lo, db_hi, idesc, k0 > kbeg || k > 0);  // small terms first
                                umma_bf16(dst, da_hi, db_lo, idesc, true);
                                umma_bf16(dst, da_hi, db_hi, idesc, true);
                            }
                        }
                        umma_commit(&sm->bar[s]);
                    }
                    last_it = it;
                    ++it;
                    TGPROF(4);
                }
                // all MMAs of the tile are done when the last slice's are (they complete in order)
                mbar_wait(&sm->bar[last_it & 1u], (last_it >> 1) & 1u, wc, 200 + 2);
                tc_fence_after_sync();
                TGPROF(5);
                {
                    const int qd = warp & 3, grp = warp >> 2;  // lane quadrant of this warp; which 16 of the 64 columns
                    const uint32_t taddr = tmem + ((uint32_t)(32 * qd) << 16) + (uint32_t)(16 * grp);
                    uint32_t acc0[16], acc1[16];
                    tmem_ld16(taddr, acc0);
                    if (NACC == 2) tmem_ld16(taddr + kTgBM, acc1);
                    tmem_wait_ld();
                    const int nl = 32 * qd + lane;
                    const int n = n0 + nl;
                    if (SPLITK && parts > 1) {
                        // raw partial sums: [accumulator][part x tile][m (64)][n (128)], coalesced over the lanes
                        float* dst = scratch + ((size_t)(part * tiles + tile)) * (kTgBM * kTgBN) + (size_t)(16 * grp) * kTgBN + nl;
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            dst[(size_t)j * kTgBN] = __uint_as_float(acc0[j]);
                            if (NACC == 2) dst[(size_t)kTgMaxParts * (kTgBM * kTgBN) + (size_t)j * kTgBN] = __uint_as_float(acc1[j]);
                        }
                    } else if (n < N) {
                        using P = decltype(pre(0, 0));
                        constexpr int kBatch = 8;
#pragma unroll
                        for (int j0 = 0; j0 < 16; j0 += kBatch) {
                            P p[kBatch];
#pragma unroll
                            for (int j = 0; j < kBatch; ++j) {
                                const int m = m0 + 16 * grp + j0 + j;
                                if (m < M) p[j] = pre(m, n);
                            }
#pragma unroll
                            for (int j = 0; j < kBatch; ++j) {
                                const int m = m0 + 16 * grp + j0 + j;
                                if (m < M)
                                    epi(m, n, __uint_as_float(acc0[j0 + j]), NACC == 2 ? __uint_as_float(acc1[j0 + j]) : 0.0f,
                                        p[j]);
                            }
                        }
                    }
                }
                TGPROF(6);
                tc_fence_before_sync();
                __syncthreads();  // the accumulators may be overwritten by the next tile
                tc_fence_after_sync();
                TGPROF(7);
            }
        }
        if (SPLITK && parts > 1) {
            // every part is in the scratch area: sum them in part order and run the epilogue, elementwise over all CTAs
            phase_sync(nranks);
            using P = decltype(pre(0, 0));
            constexpr int kBatch = 4;
            const int total = tiles * kTgBM * kTgBN;
            const int stride = kTgThreads * nranks;
            for (int e0 = tid + rank * kTgThreads; e0 < total; e0 += stride * kBatch) {
                P p[kBatch];
                float s0[kBatch], s1[kBatch];
#pragma unroll
                for (int u = 0; u < kBatch; ++u) {
                    const int e = e0 + u * stride;
                    s0[u] = 0.0f;
                    s1[u] = 0.0f;
                    if (e < total) {
                        const int tile = e / (kTgBM * kTgBN), r = e - tile * (kTgBM * kTgBN);
                        const int m = (tile % tiles_m) * kTgBM + r / kTgBN, n = (tile / tiles_m) * kTgBN + r % kTgBN;
                        if (m < M && n < N) {
                            for (int part = 0; part < parts; ++part) {
                                const float* src = scratch + ((size_t)(part * tiles + tile)) * (kTgBM * kTgBN) + r;
                                s0[u] += src[0];
                                if (NACC == 2) s1[u] += src[(size_t)kTgMaxParts * (kTgBM * kTgBN)];
                            }
                            p[u] = pre(m, n);
                        }
                    }
                }
#pragma unroll
                for (int u = 0; u < kBatch; ++u) {
                    const int e = e0 + u * stride;
                    if (e < total) {
                        const int tile = e / (kTgBM * kTgBN), r = e - tile * (kTgBM * kTgBN);
                        const int m = (tile % tiles_m) * kTgBM + r / kTgBN, n = (tile / tiles_m) * kTgBN + r % kTgBN;
                        if (m < M && n < N) epi(m, n, s0[u], s1[u], p[u]);
                    }
                }
            }
        }
        phase_sync(nranks);
        TGPROF(8);
    }
};

}  // namespace e2ttt
