// Pieces shared by the fused tensor-core kernels (tc_fwd.cu: GELU-MLP, tc_swiglu.cu: SwiGLU): the per-chunk scalar
// kernels by warp-shuffle scans, shared-memory matrix descriptors as immediates, staging-slot layouts of the cluster
// exchange, swizzled slab stores, the warp -> issuer hand-over, TMA map creation.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "simt_common.cuh"
#include "sm100.cuh"

namespace e2ttt {
namespace tc {
using namespace sm100;

constexpr int C = 64;  // chunk size the fused kernels are built for

struct Scalars {
    float kW[C], kM[C];
    float cw, cm, cb, pad;
};

// Shared-memory matrix descriptors as compile-time offsets from one run-time value: base16 = (address of the tile) >> 4.
// High word: SBO = 1024 B, descriptor version 1, 128-byte swizzle.  Low word: start address >> 4 | LBO >> 4 << 16.
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
// K-major operand: k-step k covers columns 16k..16k+15 of slab (k >> 2); LBO is unused (16 B).
__device__ __forceinline__ uint64_t dk(uint32_t base16, uint32_t slab_stride, int k) {
    return ((uint64_t)kDescHi << 32) | (uint64_t)(base16 + (((uint32_t)(k >> 2) * slab_stride + (uint32_t)(k & 3) * 32u) >> 4) + (1u << 16));
}
// MN-major operand: k-step k covers rows 16k..16k+15; LBO = distance between the slabs of 64 M/N indices.
__device__ __forceinline__ uint64_t dmn(uint32_t base16, uint32_t slab_stride, int k) {
    return ((uint64_t)kDescHi << 32) | (uint64_t)(base16 + (((uint32_t)k * 2048u) >> 4) + ((slab_stride >> 4) << 16));
}

__device__ __forceinline__ void named_sync(int id, int nthreads) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory"); }
__device__ __forceinline__ void named_arrive(int id, int nthreads) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(nthreads) : "memory"); }
// barrier ids (0 is __syncthreads)
constexpr int BAR_EPI = 1, BAR_STAGE = 3, BAR_KOWN = 4, BAR_QOWN = 5;

// Suffix scans of one chunk of len <= 64 tokens by one warp (two tokens per lane), same recurrences as the SIMT path:
// a step is the map (bt, gt, S) -> (beta bt, gamma gt, beta S + gamma gt); suffix composites by warp shuffles.
// Positions at and beyond len (the unused rows of a 64-row tile) are the identity map with a zero learning rate: their
// kW, kM come out as 0 and the carries are those of the len real tokens.
// The composition of two scan maps with the rounding pinned (one fused multiply-add), so that the scalars do not depend
// on how the compiler contracts the expression at a given call site.
__device__ __forceinline__ ScanMap<float> compose_pinned(const ScanMap<float>& outer, const ScanMap<float>& inner) {
    ScanMap<float> r;
    r.B = outer.B * inner.B;
    r.G = outer.G * inner.G;
    r.X = __fmaf_rn(outer.B, inner.X, __fmul_rn(outer.X, inner.G));
    return r;
}
// `tail` (optional): the composite map of the chunk's tokens behind this block, for chunks of several 64-token blocks;
// the scalars and, for the chunk's first block, the carries are then those of the whole chunk.
static __device__ void tc_chunk_scalars(const float* eta, const float* beta, const float* gamma, Scalars* out, int len = 64,
                                        const ScanMap<float>* tail = nullptr) {
    const int lane = threadIdx.x & 31;
    ScanMap<float> e0, e1, id;
    id.B = 1.0f; id.G = 1.0f; id.X = 0.0f;
    const bool in0 = 2 * lane < len, in1 = 2 * lane + 1 < len;
    e0 = id; e1 = id;
    if (in0) { e0.B = beta[2 * lane]; e0.G = gamma[2 * lane]; e0.X = e0.G; }
    if (in1) { e1.B = beta[2 * lane + 1]; e1.G = gamma[2 * lane + 1]; e1.X = e1.G; }
    const ScanMap<float> loc1 = e1;                 // tokens 2l+1 .. of this lane
    const ScanMap<float> loc0 = compose_pinned(e0, loc1);  // tokens 2l ..   of this lane
    ScanMap<float> incl = loc0;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        ScanMap<float> o;
        o.B = __shfl_down_sync(0xffffffffu, incl.B, off);
        o.G = __shfl_down_sync(0xffffffffu, incl.G, off);
        o.X = __shfl_down_sync(0xffffffffu, incl.X, off);
        if (lane + off < 32) incl = compose_pinned(incl, o);
    }
    ScanMap<float> excl;
    excl.B = __shfl_down_sync(0xffffffffu, incl.B, 1);
    excl.G = __shfl_down_sync(0xffffffffu, incl.G, 1);
    excl.X = __shfl_down_sync(0xffffffffu, incl.X, 1);
    if (lane == 31) excl = id;
    if (tail) excl = compose_pinned(excl, *tail);
    // token index 2l sees the state after tokens 2l+1.., token 2l+1 the state after the later lanes' tokens
    const ScanMap<float> f1 = compose_pinned(loc1, excl);
    const float et0 = in0 ? eta[2 * lane] : 0.0f, et1 = in1 ? eta[2 * lane + 1] : 0.0f;
    out->kW[2 * lane] = __fmul_rn(et0, __fadd_rn(f1.B, f1.X));
    out->kM[2 * lane] = et0 * f1.B;
    out->kW[2 * lane + 1] = __fmul_rn(et1, __fadd_rn(excl.B, excl.X));
    out->kM[2 * lane + 1] = et1 * excl.B;
    if (lane == 0) {
        const ScanMap<float> f0 = compose_pinned(loc0, excl);
        out->cw = f0.G;
        out->cb = f0.B;
        out->cm = __fmul_rn(e0.B, __fadd_rn(f1.B, f1.X));  // beta_1 S_1
    }
}

// Composite map of a block of len <= 64 tokens (all of them, first token outermost), the same in every lane.
static __device__ ScanMap<float> tc_block_composite(const float* beta, const float* gamma, int len) {
    const int lane = threadIdx.x & 31;
    ScanMap<float> e0, e1, id;
    id.B = 1.0f; id.G = 1.0f; id.X = 0.0f;
    e0 = id; e1 = id;
    if (2 * lane < len) { e0.B = beta[2 * lane]; e0.G = gamma[2 * lane]; e0.X = e0.G; }
    if (2 * lane + 1 < len) { e1.B = beta[2 * lane + 1]; e1.G = gamma[2 * lane + 1]; e1.X = e1.G; }
    ScanMap<float> incl = compose_pinned(e0, e1);
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        ScanMap<float> o;
        o.B = __shfl_down_sync(0xffffffffu, incl.B, off);
        o.G = __shfl_down_sync(0xffffffffu, incl.G, off);
        o.X = __shfl_down_sync(0xffffffffu, incl.X, off);
        if (lane + off < 32) incl = compose_pinned(incl, o);
    }
    ScanMap<float> r;
    r.B = __shfl_sync(0xffffffffu, incl.B, 0);
    r.G = __shfl_sync(0xffffffffu, incl.G, 0);
    r.X = __shfl_sync(0xffffffffu, incl.X, 0);
    return r;
}
// Tails of the blocks of one chunk: tails[j] = composite of the blocks behind block j (identity for the last one).
// tokens: the chunk's real tokens (<= 64 * nblk).  Called by one converged warp.
static __device__ void tc_chunk_tails(const float* beta, const float* gamma, int tokens, int nblk, ScanMap<float>* tails) {
    ScanMap<float> tail;
    tail.B = 1.0f; tail.G = 1.0f; tail.X = 0.0f;
    for (int j = nblk - 1; j >= 0; --j) {
        if ((threadIdx.x & 31) == 0) tails[j] = tail;
        if (j > 0) {
            const ScanMap<float> comp = tc_block_composite(beta + 64 * j, gamma + 64 * j, min(64, tokens - 64 * j));
            tail = compose_pinned(comp, tail);
        }
    }
    __syncwarp();
}

__device__ __forceinline__ float fast_tanh(float x) {
    float t;
    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(x));
    return t;
}
// Staging slot for fp32 partial sums: 16 rows x 128 fp32 = 8 KB, kept as 16-byte pieces.  Piece c4 (4 columns) of row r
// sits at piece index c4 * 16 + (r ^ ((c4 >> 1) & 15)): the 16 lanes that send one piece of 16 neighbouring rows write 256
// contiguous bytes (DSMEM moves whole segments; scattered 16-byte stores cost several times the bandwidth), and the
// layer-norm readers (16 threads per row, pieces 2cg and 2cg+1) spread over all banks.
__device__ __forceinline__ uint32_t stage_offset(uint32_t c4, uint32_t r) {
    return (c4 * 16u + (r ^ ((c4 >> 1) & 15u))) << 4;
}
// The same for bf16 partial sums: 16 rows x 128 bf16 = 4 KB, piece c8 (8 columns) of row r at c8 * 16 + (r ^ c8).
__device__ __forceinline__ uint32_t stage_offset_q(uint32_t c8, uint32_t r) {
    return (c8 * 16u + (r ^ c8)) << 4;
}
// Bulk copy of `bytes` (a multiple of 16) from this CTA's shared memory into a peer's; the peer's mbarrier gets the bytes.
__device__ __forceinline__ void bulk_copy_to_cta(uint32_t dst_cluster_addr, uint32_t src_addr, uint32_t bytes, uint32_t dst_cluster_mbar) {
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_cluster_addr), "r"(src_addr), "r"(bytes), "r"(dst_cluster_mbar) : "memory");
}

// 16 bf16 (32 bytes, already packed in pairs) = two 16-byte chunks into a swizzled slab row
__device__ __forceinline__ void st_slab16p(uint8_t* slab, int row, int col0, const uint32_t (&p)[8]) {
    const int c = col0 >> 3;
    *reinterpret_cast<uint4*>(slab + row * 128 + (((c) ^ (row & 7)) << 4)) = make_uint4(p[0], p[1], p[2], p[3]);
    *reinterpret_cast<uint4*>(slab + row * 128 + (((c + 1) ^ (row & 7)) << 4)) = make_uint4(p[4], p[5], p[6], p[7]);
}
__device__ __forceinline__ void st_slab16(uint8_t* slab, int row, int col0, const float (&v)[16]) {
    uint32_t p[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) p[i] = pack_bf16(v[2 * i], v[2 * i + 1]);
    st_slab16p(slab, row, col0, p);
}

__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    const __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// A warp has finished writing operand tiles in shared memory (generic proxy) and / or reading or writing tensor
// memory: make that visible to the MMA issuer, then one lane arrives.
__device__ __forceinline__ void warp_release(uint64_t* bar) {
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static inline EncodeTiledFn encode_fn() {
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
static inline bool make_token_map(CUtensorMap* tm, const void* base, size_t rows, unsigned box_rows, int d) {
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


}  // namespace tc
}  // namespace e2ttt
