// C ABI of the library: argument validation, workspace sizing, kernel-family dispatch.
#include <cuda_runtime.h>

#include "../../include/e2ttt.h"
#include "apply.h"
#include "prepare.h"
#include "simt_layout.h"
#include "tc_fwd.h"
#include "tc_swiglu.h"

using namespace e2ttt;

namespace e2ttt {
const void* noalloc_scratch_if_known();  // noalloc.cu
}

namespace {

constexpr int kMaxD = 1024;
constexpr int kMaxH = 8192;
constexpr int kMaxChunk = 512;

int nmat_of(int kind) { return kind == E2TTT_MLP_GELU ? 2 : (kind == E2TTT_SWIGLU ? 3 : 0); }

int check_params(const e2ttt_params* p) {
    if (!p) return E2TTT_ERR_NULL;
    if (p->kind != E2TTT_MLP_GELU && p->kind != E2TTT_SWIGLU) return E2TTT_ERR_SHAPE;
    if (p->io_dtype != E2TTT_F32 && p->io_dtype != E2TTT_BF16) return E2TTT_ERR_DTYPE;
    if (p->impl != E2TTT_IMPL_AUTO && p->impl != E2TTT_IMPL_SIMT && p->impl != E2TTT_IMPL_TCGEN05 &&
        p->impl != E2TTT_IMPL_TILED)
        return E2TTT_ERR_DTYPE;
    if (p->B <= 0 || p->H <= 0 || p->L <= 0 || p->d <= 0 || p->h <= 0 || p->C <= 0) return E2TTT_ERR_SHAPE;
    if (p->C > kMaxChunk || p->d > kMaxD || p->h > kMaxH) return E2TTT_ERR_SHAPE;
    if ((int64_t)p->B * p->H > (int64_t)1 << 24) return E2TTT_ERR_SHAPE;
    if (!(p->ln_eps >= 0.0f)) return E2TTT_ERR_SHAPE;
    if (p->ckpt_every < 0) return E2TTT_ERR_SHAPE;
    return E2TTT_OK;
}

// chunks per recomputed segment of the backward; 0 = every chunk's state is kept
int segment_chunks(const e2ttt_params* p) { return p->ckpt_every >= 2 ? p->ckpt_every : 0; }

// Every workspace starts with a status block: word 0 is the device status of the last launch that used it.
constexpr size_t kStatusBytes = 256;

// 1 = a tensor-core specialisation exists for these parameters (the forward; with save_states it also writes the
// chunk-start states in the layout the SIMT backward reads)
int has_tcgen05(const e2ttt_params* p, bool save_states) {
    // chunks of 32 or 16 tokens run in the same 64-row tiles (unused rows zero): half / a quarter of the tile's work is useful;
    // both kernels also run chunks of 128, 256 or 512 tokens as 2, 4 or 8 blocks of 64 (on request, see pick_impl)
    if (p->io_dtype != E2TTT_BF16) return 0;
    const bool small = p->C == 64 || p->C == 32 || p->C == 16;
    const bool large = p->C == 128 || p->C == 256 || p->C == 512;
    if (p->kind == E2TTT_MLP_GELU) return (small || large) && (p->d == 128 || p->d == 64) && p->h % 128 == 0 && p->h <= 512;
    // SwiGLU: the fused kernel is built for d = 128, h = 384
    (void)save_states;
    return (small || large) && p->kind == E2TTT_SWIGLU && p->d == 128 && p->h == 384;
}

int pick_impl(const e2ttt_params* p, bool save_states, int* impl) {
    if (p->impl == E2TTT_IMPL_TCGEN05) {
        if (!has_tcgen05(p, save_states)) return E2TTT_ERR_SHAPE;
        *impl = E2TTT_IMPL_TCGEN05;
    } else if (p->impl == E2TTT_IMPL_TILED) {
        if (p->io_dtype != E2TTT_BF16) return E2TTT_ERR_SHAPE;
        *impl = E2TTT_IMPL_TILED;
    } else if (p->impl == E2TTT_IMPL_AUTO) {
        // Chunks above 64 tokens run on the fused kernels when asked for (TCGEN05), not by default: their plain bf16
        // operands leave the W1 momentum of long chunks outside the 2e-2 bound when the chunk's gradients cancel
        // (measured 3-4e-2 at C = 512 under the paper's gates; the any-shape kernels' two-term operands do not).
        *impl = (has_tcgen05(p, save_states) && p->C <= 64)
                    ? E2TTT_IMPL_TCGEN05
                    : (p->io_dtype == E2TTT_BF16 ? E2TTT_IMPL_TILED : E2TTT_IMPL_SIMT);
    } else {
        *impl = E2TTT_IMPL_SIMT;
    }
    return E2TTT_OK;
}

size_t simt_bytes(const e2ttt_params* p, bool save_states, bool backward, bool normed) {
    const int nchunks = (p->L + p->C - 1) / p->C;
    SimtLayout l = simt_layout(p->d, p->h, p->C, nmat_of(p->kind), nchunks, save_states, backward, normed ? 0 : segment_chunks(p));
    const size_t elem = (p->io_dtype == E2TTT_F32) ? sizeof(double) : sizeof(float);
    return kStatusBytes + l.per_seq * elem * (size_t)p->B * p->H;
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

int check_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return E2TTT_ERR_ARCH; }
    static int cached_major[64];
    static bool known[64];
    int major = 0;
    if (dev >= 0 && dev < 64 && known[dev]) {
        major = cached_major[dev];
    } else {
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
            (void)cudaGetLastError();
            return E2TTT_ERR_ARCH;
        }
        if (dev >= 0 && dev < 64) { cached_major[dev] = major; known[dev] = true; }
    }
    return major == 10 ? E2TTT_OK : E2TTT_ERR_ARCH;
}

}  // namespace

extern "C" {

int e2ttt_num_matrices(int kind) { return nmat_of(kind); }

int e2ttt_matrix_shape(int kind, int d, int h, int i, int* rows, int* cols) {
    const int n = nmat_of(kind);
    if (n == 0 || i < 0 || i >= n || !rows || !cols) return E2TTT_ERR_SHAPE;
    const bool last = (i == n - 1);
    *rows = last ? d : h;
    *cols = last ? h : d;
    return E2TTT_OK;
}

int e2ttt_workspace_bytes(const e2ttt_params* p, int save_states, size_t* bytes) {
    if (!bytes) return E2TTT_ERR_NULL;
    int rc = check_params(p);
    if (rc) return rc;
    int impl = 0;
    rc = pick_impl(p, save_states != 0, &impl);
    if (rc) return rc;
    // fused tensor-core path: all state lives on chip, only the status block is needed.
    // any-shape kernels: with saved states the same buffer serves the backward, which needs the larger layout.
    *bytes = (impl == E2TTT_IMPL_TCGEN05 && !save_states) ? kStatusBytes : simt_bytes(p, save_states != 0, save_states != 0, false);
    return E2TTT_OK;
}

int e2ttt_workspace_bytes_normed(const e2ttt_params* p, int save_states, size_t* bytes) {
    if (!bytes) return E2TTT_ERR_NULL;
    int rc = check_params(p);
    if (rc) return rc;
    if (p->impl == E2TTT_IMPL_TCGEN05 && !(has_tcgen05(p, false) && p->kind == E2TTT_MLP_GELU && p->C <= 64)) return E2TTT_ERR_SHAPE;
    if (segment_chunks(p)) return E2TTT_ERR_SHAPE;
    *bytes = simt_bytes(p, save_states != 0, save_states != 0, true);
    return E2TTT_OK;
}

static int fwd_common(const e2ttt_params* p, const void* q, const void* k, const void* v, const float* eta,
                      const float* beta, const float* gamma, const float* const* W_init, const float* const* M_init,
                      const float* const* row_norm, float norm_eps,
                      void* o, float* const* W_final, float* const* M_final, void* workspace, size_t workspace_bytes,
                      int save_states, void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    if (!q || !k || !v || !eta || !beta || !gamma || !W_init || !o || !W_final || !M_final) return E2TTT_ERR_NULL;
    const int nmat = nmat_of(p->kind);
    for (int i = 0; i < nmat; ++i) {
        if (!W_init[i] || !W_final[i] || !M_final[i]) return E2TTT_ERR_NULL;
        if (M_init && !M_init[i]) return E2TTT_ERR_NULL;
    }
    int impl = 0;
    rc = pick_impl(p, save_states != 0, &impl);
    if (rc) return rc;
    if (!aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(o, 16)) return E2TTT_ERR_ALIGN;
    size_t need = 0;
    if (row_norm) {
        if (!(norm_eps >= 0.0f) || segment_chunks(p)) return E2TTT_ERR_SHAPE;
        for (int i = 0; i < nmat; ++i)
            if (!row_norm[i]) return E2TTT_ERR_NULL;
        need = simt_bytes(p, save_states != 0, save_states != 0, true);  // the size e2ttt_workspace_bytes_normed reports
    } else {
        rc = e2ttt_workspace_bytes(p, save_states, &need);
        if (rc) return rc;
    }
    if (!workspace || workspace_bytes < need) return E2TTT_ERR_WORKSPACE;
    if (!aligned(workspace, 256)) return E2TTT_ERR_ALIGN;
    rc = check_device();
    if (rc) return rc;

    if (impl == E2TTT_IMPL_TCGEN05 && row_norm && (p->kind == E2TTT_SWIGLU || p->C > 64)) {
        // no fused kernel with post-chunk normalisation for SwiGLU or for chunks of several blocks: the any-shape kernels serve it
        if (p->impl == E2TTT_IMPL_TCGEN05) return E2TTT_ERR_SHAPE;
        impl = E2TTT_IMPL_TILED;
    }
    if (impl == E2TTT_IMPL_TCGEN05 && p->kind == E2TTT_SWIGLU) {
        TcSwigluArgs t{};
        t.N = p->B * p->H; t.L = p->L; t.C = p->C; t.eps = p->ln_eps;
        t.q = static_cast<const __nv_bfloat16*>(q); t.k = static_cast<const __nv_bfloat16*>(k);
        t.v = static_cast<const __nv_bfloat16*>(v); t.o = static_cast<__nv_bfloat16*>(o);
        t.eta = eta; t.beta = beta; t.gamma = gamma;
        t.W1_init = W_init[0]; t.W2_init = W_init[1]; t.W3_init = W_init[2];
        t.M1_init = M_init ? M_init[0] : nullptr; t.M2_init = M_init ? M_init[1] : nullptr; t.M3_init = M_init ? M_init[2] : nullptr;
        t.W1_final = W_final[0]; t.W2_final = W_final[1]; t.W3_final = W_final[2];
        t.M1_final = M_final[0]; t.M2_final = M_final[1]; t.M3_final = M_final[2];
        t.status = static_cast<int*>(workspace);
        if (save_states) {
            const int seg = segment_chunks(p);
            const SimtLayout lay = simt_layout(p->d, p->h, p->C, nmat, (p->L + p->C - 1) / p->C, true, true, seg);
            t.ckpt = reinterpret_cast<float*>(static_cast<char*>(workspace) + kStatusBytes) + (seg ? lay.cck : lay.ckpt);
            t.ckpt_seq_stride = lay.per_seq;
            t.ckpt_every = seg;
        }
        return tc_swiglu_launch(t, stream) == 0 ? E2TTT_OK : E2TTT_ERR_CUDA;
    }
    if (impl == E2TTT_IMPL_TCGEN05) {
        TcFwdArgs t{};
        t.N = p->B * p->H; t.L = p->L; t.C = p->C; t.d = p->d; t.h = p->h; t.eps = p->ln_eps;
        t.q = static_cast<const __nv_bfloat16*>(q); t.k = static_cast<const __nv_bfloat16*>(k);
        t.v = static_cast<const __nv_bfloat16*>(v); t.o = static_cast<__nv_bfloat16*>(o);
        t.eta = eta; t.beta = beta; t.gamma = gamma;
        t.W1_init = W_init[0]; t.W2_init = W_init[1];
        t.M1_init = M_init ? M_init[0] : nullptr; t.M2_init = M_init ? M_init[1] : nullptr;
        t.W1_final = W_final[0]; t.W2_final = W_final[1]; t.M1_final = M_final[0]; t.M2_final = M_final[1];
        t.status = static_cast<int*>(workspace);
        if (row_norm) { t.norm1 = row_norm[0]; t.norm2 = row_norm[1]; t.norm_eps = norm_eps; }
        if (save_states) {
            const int seg = row_norm ? 0 : segment_chunks(p);
            const SimtLayout lay = simt_layout(p->d, p->h, p->C, nmat, (p->L + p->C - 1) / p->C, true, true, seg);
            t.ckpt = reinterpret_cast<float*>(static_cast<char*>(workspace) + kStatusBytes) + (seg ? lay.cck : lay.ckpt);
            t.ckpt_seq_stride = lay.per_seq;
            t.ckpt_every = seg;
            t.rown = reinterpret_cast<float*>(static_cast<char*>(workspace) + kStatusBytes) + lay.rown;
        }
        return tc_fwd_launch(t, stream) == 0 ? E2TTT_OK : E2TTT_ERR_CUDA;
    }
    if (cudaMemsetAsync(workspace, 0, sizeof(int), reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) {
        (void)cudaGetLastError();
        return E2TTT_ERR_CUDA;
    }

    SimtFwdArgs a{};
    a.N = p->B * p->H; a.L = p->L; a.d = p->d; a.h = p->h; a.C = p->C;
    a.nchunks = (p->L + p->C - 1) / p->C;
    a.cl = simt_cluster_size(a.N);
    a.tc = impl == E2TTT_IMPL_TILED;
    a.status = static_cast<int*>(workspace);
    const int seg = row_norm ? 0 : segment_chunks(p);
    a.save_states = save_states ? (seg ? 2 : 1) : 0;
    a.Ls = p->L; a.init_slot = -1;
    a.eps = p->ln_eps;
    a.q = q; a.k = k; a.v = v; a.eta = eta; a.beta = beta; a.gamma = gamma; a.o = o;
    a.ws = static_cast<char*>(workspace) + kStatusBytes;
    for (int i = 0; i < nmat; ++i) {
        a.W_init[i] = W_init[i];
        a.M_init[i] = M_init ? M_init[i] : nullptr;
        a.W_final[i] = W_final[i];
        a.M_final[i] = M_final[i];
        a.row_norm[i] = row_norm ? row_norm[i] : nullptr;
    }
    a.norm_eps = norm_eps;
    a.lay = simt_layout(p->d, p->h, p->C, nmat, a.nchunks, save_states != 0, save_states != 0, seg);
    return simt_fwd_launch(a, p->kind, p->io_dtype, stream) == 0 ? E2TTT_OK : E2TTT_ERR_CUDA;
}

int e2ttt_chunk_fwd(const e2ttt_params* p, const void* q, const void* k, const void* v, const float* eta,
                    const float* beta, const float* gamma, const float* const* W_init, const float* const* M_init,
                    void* o, float* const* W_final, float* const* M_final, void* workspace, size_t workspace_bytes,
                    int save_states, void* stream) {
    return fwd_common(p, q, k, v, eta, beta, gamma, W_init, M_init, nullptr, 0.0f, o, W_final, M_final, workspace,
                      workspace_bytes, save_states, stream);
}

int e2ttt_chunk_fwd_normed(const e2ttt_params* p, const void* q, const void* k, const void* v, const float* eta,
                           const float* beta, const float* gamma, const float* const* W_init,
                           const float* const* M_init, const float* const* row_norm, float norm_eps, void* o,
                           float* const* W_final, float* const* M_final, void* workspace, size_t workspace_bytes,
                           int save_states, void* stream) {
    if (!row_norm) return E2TTT_ERR_NULL;
    return fwd_common(p, q, k, v, eta, beta, gamma, W_init, M_init, row_norm, norm_eps, o, W_final, M_final, workspace,
                      workspace_bytes, save_states, stream);
}

static int bwd_common(const e2ttt_params* p, const void* q, const void* k, const void* v, const float* eta,
                      const float* beta, const float* gamma, const float* const* W_init, const float* const* M_init,
                      const float* const* row_norm, float norm_eps,
                      const void* d_o, const float* const* dW_final, const float* const* dM_final, void* dq, void* dk,
                      void* dv, float* d_eta, float* d_beta, float* d_gamma, float* const* dW_init,
                      float* const* dM_init, float* const* d_row_norm, void* workspace, size_t workspace_bytes,
                      int states_saved, void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    if (!q || !k || !v || !eta || !beta || !gamma || !W_init || !d_o || !dq || !dk || !dv || !d_eta || !d_beta ||
        !d_gamma || !dW_init || !dM_init)
        return E2TTT_ERR_NULL;
    const int nmat = nmat_of(p->kind);
    for (int i = 0; i < nmat; ++i) {
        if (!W_init[i] || !dW_init[i] || !dM_init[i]) return E2TTT_ERR_NULL;
        if (M_init && !M_init[i]) return E2TTT_ERR_NULL;
        if (dW_final && !dW_final[i]) return E2TTT_ERR_NULL;
        if (dM_final && !dM_final[i]) return E2TTT_ERR_NULL;
    }
    int impl = 0;
    rc = pick_impl(p, true, &impl);
    if (rc) return rc;
    if (row_norm) {
        if (!(norm_eps >= 0.0f) || segment_chunks(p)) return E2TTT_ERR_SHAPE;
        for (int i = 0; i < nmat; ++i)
            if (!row_norm[i]) return E2TTT_ERR_NULL;
    }
    if (!aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(d_o, 16) || !aligned(dq, 16) ||
        !aligned(dk, 16) || !aligned(dv, 16))
        return E2TTT_ERR_ALIGN;
    const size_t need = simt_bytes(p, true, true, row_norm != nullptr);
    if (!workspace || workspace_bytes < need) return E2TTT_ERR_WORKSPACE;
    if (!aligned(workspace, 256)) return E2TTT_ERR_ALIGN;
    rc = check_device();
    if (rc) return rc;

    const int nchunks = (p->L + p->C - 1) / p->C;
    const int seg = row_norm ? 0 : segment_chunks(p);
    const SimtLayout lay = simt_layout(p->d, p->h, p->C, nmat, nchunks, true, true, seg);
    void* ws_data = static_cast<char*>(workspace) + kStatusBytes;
    if (cudaMemsetAsync(workspace, 0, sizeof(int), reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) {
        (void)cudaGetLastError();
        return E2TTT_ERR_CUDA;
    }
    // A forward that only records chunk-start states: outputs and final states are not written.
    //   first_chunk, n  : the chunks it covers;  mode 1: every chunk's state -> lay.ckpt, 2: checkpoints -> lay.cck
    //   init_slot       : -1 = start from W_init / M_init, else from checkpoint init_slot
    // The fused tensor-core forward serves the recomputation where it serves the shape (bit-identical to the states a
    // fused forward with save_states wrote, since it is the same kernel restarted from its own fp32 state).
    const bool fused_recompute = impl == E2TTT_IMPL_TCGEN05 && !row_norm;
    auto recompute = [&](int first_chunk, int n, int mode, int init_slot) -> int {
        const size_t t0 = (size_t)first_chunk * p->C;
        const size_t esz = p->io_dtype == E2TTT_F32 ? 4 : 2;
        if (fused_recompute && p->kind == E2TTT_SWIGLU) {
            const size_t dh = (size_t)p->d * p->h;
            float* wsf = static_cast<float*>(ws_data);
            TcSwigluArgs t{};
            t.N = p->B * p->H; t.L = (int)((size_t)p->L - t0 < (size_t)n * p->C ? (size_t)p->L - t0 : (size_t)n * p->C); t.C = p->C; t.Ls = p->L; t.eps = p->ln_eps;
            t.q = static_cast<const __nv_bfloat16*>(q) + t0 * p->d; t.k = static_cast<const __nv_bfloat16*>(k) + t0 * p->d;
            t.v = static_cast<const __nv_bfloat16*>(v) + t0 * p->d; t.o = nullptr;
            t.eta = eta + t0; t.beta = beta + t0; t.gamma = gamma + t0;
            if (init_slot >= 0) {
                const float* ck = wsf + lay.cck + (size_t)init_slot * 6 * dh;
                t.W1_init = ck; t.W2_init = ck + dh; t.W3_init = ck + 2 * dh;
                t.M1_init = ck + 3 * dh; t.M2_init = ck + 4 * dh; t.M3_init = ck + 5 * dh;
                t.init_seq_stride = lay.per_seq;
            } else {
                t.W1_init = W_init[0]; t.W2_init = W_init[1]; t.W3_init = W_init[2];
                t.M1_init = M_init ? M_init[0] : nullptr; t.M2_init = M_init ? M_init[1] : nullptr;
                t.M3_init = M_init ? M_init[2] : nullptr;
            }
            float* fin = wsf + (mode == 1 ? lay.ckpt + (size_t)n * 6 * dh : lay.cck + (size_t)((n + seg - 1) / seg) * 6 * dh);
            t.W1_final = fin; t.W2_final = fin + dh; t.W3_final = fin + 2 * dh;
            t.M1_final = fin + 3 * dh; t.M2_final = fin + 4 * dh; t.M3_final = fin + 5 * dh;
            t.final_seq_stride = lay.per_seq;
            t.status = static_cast<int*>(workspace); t.keep_status = 1;
            t.ckpt = wsf + (mode == 1 ? lay.ckpt : lay.cck);
            t.ckpt_seq_stride = lay.per_seq;
            t.ckpt_every = mode == 1 ? 0 : seg;
            return tc_swiglu_launch(t, stream);
        }
        if (fused_recompute) {
            const size_t dh = (size_t)p->d * p->h;
            float* wsf = static_cast<float*>(ws_data);
            TcFwdArgs t{};
            t.N = p->B * p->H; t.L = (int)((size_t)p->L - t0 < (size_t)n * p->C ? (size_t)p->L - t0 : (size_t)n * p->C); t.C = p->C; t.Ls = p->L; t.d = p->d; t.h = p->h; t.eps = p->ln_eps;
            t.q = static_cast<const __nv_bfloat16*>(q) + t0 * p->d; t.k = static_cast<const __nv_bfloat16*>(k) + t0 * p->d;
            t.v = static_cast<const __nv_bfloat16*>(v) + t0 * p->d; t.o = nullptr;
            t.eta = eta + t0; t.beta = beta + t0; t.gamma = gamma + t0;
            if (init_slot >= 0) {
                const float* ck = wsf + lay.cck + (size_t)init_slot * 4 * dh;
                t.W1_init = ck; t.W2_init = ck + dh; t.M1_init = ck + 2 * dh; t.M2_init = ck + 3 * dh;
                t.init_seq_stride = lay.per_seq;
            } else {
                t.W1_init = W_init[0]; t.W2_init = W_init[1];
                t.M1_init = M_init ? M_init[0] : nullptr; t.M2_init = M_init ? M_init[1] : nullptr;
            }
            // the state after the call is not wanted: it lands in the slot behind the last one the reverse sweep reads
            // (mode 1: slot n of the per-chunk states; mode 2: the slot behind the last checkpoint)
            float* fin = wsf + (mode == 1 ? lay.ckpt + (size_t)n * 4 * dh : lay.cck + (size_t)((n + seg - 1) / seg) * 4 * dh);
            t.W1_final = fin; t.W2_final = fin + dh; t.M1_final = fin + 2 * dh; t.M2_final = fin + 3 * dh;
            t.final_seq_stride = lay.per_seq;
            t.status = static_cast<int*>(workspace); t.keep_status = 1;
            t.ckpt = wsf + (mode == 1 ? lay.ckpt : lay.cck);
            t.ckpt_seq_stride = lay.per_seq;
            t.ckpt_every = mode == 1 ? 0 : seg;
            return tc_fwd_launch(t, stream);
        }
        SimtFwdArgs f{};
        f.N = p->B * p->H; f.d = p->d; f.h = p->h; f.C = p->C; f.nchunks = n;
        f.L = (int)((size_t)p->L - t0 < (size_t)n * p->C ? (size_t)p->L - t0 : (size_t)n * p->C);
        f.Ls = p->L; f.init_slot = init_slot;
        f.save_states = mode; f.eps = p->ln_eps; f.cl = simt_cluster_size(f.N);
        f.tc = impl != E2TTT_IMPL_SIMT; f.status = static_cast<int*>(workspace);
        f.q = static_cast<const char*>(q) + t0 * p->d * esz;
        f.k = static_cast<const char*>(k) + t0 * p->d * esz;
        f.v = static_cast<const char*>(v) + t0 * p->d * esz;
        f.eta = eta + t0; f.beta = beta + t0; f.gamma = gamma + t0; f.ws = ws_data; f.lay = lay;
        f.o = nullptr;
        for (int i = 0; i < nmat; ++i) {
            f.W_init[i] = W_init[i];
            f.M_init[i] = M_init ? M_init[i] : nullptr;
            f.W_final[i] = nullptr;
            f.M_final[i] = nullptr;
            f.row_norm[i] = row_norm ? row_norm[i] : nullptr;
        }
        f.norm_eps = norm_eps;
        return simt_fwd_launch(f, p->kind, p->io_dtype, stream);
    };
    // The reverse sweep over chunks [first_chunk, first_chunk + n), whose start states sit in lay.ckpt slots 0 .. n-1.
    auto reverse = [&](int first_chunk, int n, bool carry_in, bool carry_out) -> int {
        const size_t t0 = (size_t)first_chunk * p->C;
        const size_t esz = p->io_dtype == E2TTT_F32 ? 4 : 2;
        const size_t tok = t0 * p->d * esz;
        SimtBwdArgs b{};
        b.N = p->B * p->H; b.d = p->d; b.h = p->h; b.C = p->C; b.nchunks = n; b.eps = p->ln_eps;
        b.L = (int)((size_t)p->L - t0 < (size_t)n * p->C ? (size_t)p->L - t0 : (size_t)n * p->C);
        b.Ls = p->L; b.carry_in = carry_in; b.carry_out = carry_out;
        b.cl = simt_cluster_size(b.N);
        b.tc = impl != E2TTT_IMPL_SIMT; b.status = static_cast<int*>(workspace);
        b.q = static_cast<const char*>(q) + tok; b.k = static_cast<const char*>(k) + tok;
        b.v = static_cast<const char*>(v) + tok; b.d_o = static_cast<const char*>(d_o) + tok;
        b.eta = eta + t0; b.beta = beta + t0; b.gamma = gamma + t0;
        b.dq = static_cast<char*>(dq) + tok; b.dk = static_cast<char*>(dk) + tok; b.dv = static_cast<char*>(dv) + tok;
        b.d_eta = d_eta + t0; b.d_beta = d_beta + t0; b.d_gamma = d_gamma + t0;
        b.ws = ws_data; b.lay = lay;
        for (int i = 0; i < nmat; ++i) {
            b.dW_final[i] = dW_final ? dW_final[i] : nullptr;
            b.dM_final[i] = dM_final ? dM_final[i] : nullptr;
            b.dW_init[i] = dW_init[i];
            b.dM_init[i] = dM_init[i];
            b.row_norm[i] = row_norm ? row_norm[i] : nullptr;
            b.d_row_norm[i] = (row_norm && d_row_norm) ? d_row_norm[i] : nullptr;
        }
        b.norm_eps = norm_eps;
        return simt_bwd_launch(b, p->kind, p->io_dtype, stream);
    };

    if (seg == 0) {
        // every chunk's start state is in the workspace, or is recomputed into it by one forward
        if (!states_saved && recompute(0, nchunks, 1, -1) != 0) return E2TTT_ERR_CUDA;
        return reverse(0, nchunks, false, false) == 0 ? E2TTT_OK : E2TTT_ERR_CUDA;
    }
    // checkpoints every seg chunks: the segments are walked from the last to the first; each one gets the start
    // states of its chunks recomputed from its checkpoint, then its reverse sweep.  The adjoints of the state
    // (and nothing else) pass from one launch to the next, in the workspace.
    if (!states_saved && recompute(0, nchunks, 2, -1) != 0) return E2TTT_ERR_CUDA;
    const int nseg = (nchunks + seg - 1) / seg;
    for (int sgi = nseg - 1; sgi >= 0; --sgi) {
        const int first = sgi * seg;
        const int n = nchunks - first < seg ? nchunks - first : seg;
        if (recompute(first, n, 1, sgi) != 0) return E2TTT_ERR_CUDA;
        if (reverse(first, n, sgi != nseg - 1, sgi != 0) != 0) return E2TTT_ERR_CUDA;
    }
    return E2TTT_OK;
}

int e2ttt_chunk_bwd(const e2ttt_params* p, const void* q, const void* k, const void* v, const float* eta,
                    const float* beta, const float* gamma, const float* const* W_init, const float* const* M_init,
                    const void* d_o, const float* const* dW_final, const float* const* dM_final, void* dq, void* dk,
                    void* dv, float* d_eta, float* d_beta, float* d_gamma, float* const* dW_init,
                    float* const* dM_init, void* workspace, size_t workspace_bytes, int states_saved, void* stream) {
    return bwd_common(p, q, k, v, eta, beta, gamma, W_init, M_init, nullptr, 0.0f, d_o, dW_final, dM_final, dq, dk, dv,
                      d_eta, d_beta, d_gamma, dW_init, dM_init, nullptr, workspace, workspace_bytes, states_saved, stream);
}

int e2ttt_chunk_bwd_normed(const e2ttt_params* p, const void* q, const void* k, const void* v, const float* eta,
                           const float* beta, const float* gamma, const float* const* W_init,
                           const float* const* M_init, const float* const* row_norm, float norm_eps, const void* d_o,
                           const float* const* dW_final, const float* const* dM_final, void* dq, void* dk, void* dv,
                           float* d_eta, float* d_beta, float* d_gamma, float* const* dW_init, float* const* dM_init,
                           float* const* d_row_norm, void* workspace, size_t workspace_bytes, int states_saved,
                           void* stream) {
    if (!row_norm) return E2TTT_ERR_NULL;
    return bwd_common(p, q, k, v, eta, beta, gamma, W_init, M_init, row_norm, norm_eps, d_o, dW_final, dM_final, dq, dk,
                      dv, d_eta, d_beta, d_gamma, dW_init, dM_init, d_row_norm, workspace, workspace_bytes, states_saved,
                      stream);
}

int e2ttt_apply(const e2ttt_params* p, const void* q, const float* const* W, void* o, void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    if (!q || !W || !o) return E2TTT_ERR_NULL;
    const int nmat = nmat_of(p->kind);
    for (int i = 0; i < nmat; ++i)
        if (!W[i]) return E2TTT_ERR_NULL;
    if (!aligned(q, 16) || !aligned(o, 16)) return E2TTT_ERR_ALIGN;
    rc = check_device();
    if (rc) return rc;
    ApplyArgs a{};
    a.N = p->B * p->H; a.T = p->L; a.d = p->d; a.h = p->h; a.eps = p->ln_eps;
    a.cl = apply_cluster_size(a.N);
    a.tb = apply_token_block(a.T);
    while (a.cl > 1 && apply_smem_bytes(a.d, a.cl, a.tb) > 40 * 1024) a.cl /= 2;  // room for two CTAs per SM
    if (apply_smem_bytes(a.d, a.cl, a.tb) > 200 * 1024) return E2TTT_ERR_SHAPE;
    a.stage = apply_smem_bytes(a.d, a.cl, a.tb) <= 40 * 1024 && apply_can_stage(a.d, a.h, a.cl);
    a.q = q; a.o = o;
    for (int i = 0; i < nmat; ++i) a.W[i] = W[i];
    return apply_launch(a, p->kind, p->io_dtype, stream) == 0 ? E2TTT_OK : E2TTT_ERR_CUDA;
}

static int check_gates(const e2ttt_gate_params* g) {
    if (!g) return E2TTT_ERR_NULL;
    if (!(g->eta_base > 0.0f) || !(g->tau > 0.0f) || !(g->alpha_base >= 0.0f) || !(g->norm_eps >= 0.0f)) return E2TTT_ERR_SHAPE;
    return E2TTT_OK;
}

int e2ttt_prepare_fwd(const e2ttt_params* p, const e2ttt_gate_params* g, const void* q_raw, const void* k_raw,
                      const float* a_eta, const float* a_beta, const float* a_alpha, void* q, void* k, float* eta,
                      float* beta, float* gamma, void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    rc = check_gates(g);
    if (rc) return rc;
    if (!q_raw || !k_raw || !a_eta || !a_beta || !a_alpha || !q || !k || !eta || !beta || !gamma) return E2TTT_ERR_NULL;
    rc = check_device();
    if (rc) return rc;
    PrepareArgs a{};
    a.rows = (long long)p->B * p->H * p->L; a.d = p->d;
    a.eta_base = g->eta_base; a.tau = g->tau; a.alpha_base = g->alpha_base; a.norm_eps = g->norm_eps;
    a.q_raw = q_raw; a.k_raw = k_raw; a.a_eta = a_eta; a.a_beta = a_beta; a.a_alpha = a_alpha;
    a.q = q; a.k = k; a.eta = eta; a.beta = beta; a.gamma = gamma;
    return prepare_fwd_launch(a, p->io_dtype, stream) == 0 ? E2TTT_OK : E2TTT_ERR_CUDA;
}

int e2ttt_prepare_bwd(const e2ttt_params* p, const e2ttt_gate_params* g, const void* q_raw, const void* k_raw,
                      const float* a_eta, const float* a_beta, const float* a_alpha, const void* dq, const void* dk,
                      const float* d_eta, const float* d_beta, const float* d_gamma, void* dq_raw, void* dk_raw,
                      float* da_eta, float* da_beta, float* da_alpha, void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    rc = check_gates(g);
    if (rc) return rc;
    if (!q_raw || !k_raw || !a_eta || !a_beta || !a_alpha || !dq || !dk || !d_eta || !d_beta || !d_gamma || !dq_raw ||
        !dk_raw || !da_eta || !da_beta || !da_alpha)
        return E2TTT_ERR_NULL;
    rc = check_device();
    if (rc) return rc;
    PrepareBwdArgs b{};
    b.f.rows = (long long)p->B * p->H * p->L; b.f.d = p->d;
    b.f.eta_base = g->eta_base; b.f.tau = g->tau; b.f.alpha_base = g->alpha_base; b.f.norm_eps = g->norm_eps;
    b.f.q_raw = q_raw; b.f.k_raw = k_raw; b.f.a_eta = a_eta; b.f.a_beta = a_beta; b.f.a_alpha = a_alpha;
    b.dq = dq; b.dk = dk; b.d_eta = d_eta; b.d_beta = d_beta; b.d_gamma = d_gamma;
    b.dq_raw = dq_raw; b.dk_raw = dk_raw; b.da_eta = da_eta; b.da_beta = da_beta; b.da_alpha = da_alpha;
    return prepare_bwd_launch(b, p->io_dtype, stream) == 0 ? E2TTT_OK : E2TTT_ERR_CUDA;
}

int e2ttt_device_status(const void* workspace, void* stream, int* status) {
    if (!status) return E2TTT_ERR_NULL;
    if (!workspace) {  // the scratch array of e2ttt_chunk_fwd_noalloc on this device
        workspace = noalloc_scratch_if_known();
        if (!workspace) { *status = 0; return E2TTT_OK; }
    }
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    int word = 0;
    if (cudaMemcpyAsync(&word, workspace, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        (void)cudaGetLastError();
        return E2TTT_ERR_CUDA;
    }
    *status = word;
    return word == 0 ? E2TTT_OK : E2TTT_ERR_TIMEOUT;
}

const char* e2ttt_status_string(int status) {
    switch (status) {
        case E2TTT_OK: return "ok";
        case E2TTT_ERR_NULL: return "a required pointer is NULL";
        case E2TTT_ERR_SHAPE: return "unsupported shape, kind or chunk size";
        case E2TTT_ERR_DTYPE: return "unknown io_dtype or impl";
        case E2TTT_ERR_ALIGN: return "a buffer is not aligned as required";
        case E2TTT_ERR_WORKSPACE: return "workspace missing or too small";
        case E2TTT_ERR_ARCH: return "current device is not compute capability 10.x (B200)";
        case E2TTT_ERR_CUDA: return "the CUDA runtime reported an error at launch";
        case E2TTT_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        default: return "unknown status";
    }
}

int e2ttt_version(void) { return 101; }

}  // extern "C"
