// Workspace layout of the SIMT kernels (host and device).  Offsets are in elements of the kernel's
// internal type (double for fp32 I/O, float for bf16 I/O), relative to the sequence's own slice.
#pragma once
#include <stddef.h>
#include <stdint.h>

namespace e2ttt {

struct SimtLayout {
    // running state
    size_t W[3], M[3];
    // forward intermediates of one chunk ([2C x .] buffers hold the k-path rows first, then the q-path rows)
    size_t Z1, Z2, A, U, Pu, Pz1, Pz2;
    // backward only
    size_t T[3], S[3];   // adjoints of the chunk-end state (W, M)
    size_t Wb[3];        // adjoint accumulators of the chunk-start weights
    size_t Pa, E, XY2, XY1, Pub, Pzb, Zkb, Akb, Kb, Eb, Ukb, Uqb, Zqb;
    size_t XY1b, Pzb2, Zkb2, Zqb2;  // SwiGLU only: the second [h x d] matrix
    size_t rk, rq, red;  // per-row 1/std of the two LN calls; small reduction scratch
    size_t kWb, kMb;     // adjoints of the scalar kernels, one per token of the chunk
    size_t splitk;       // split-K partial sums of the tensor-core GEMM engine (2 * 8 * 128 * 64 elements)
    size_t rown;         // [nchunks][3][max(d,h)] row norms of the chunk-end weights before their normalisation
    size_t ckpt;         // [nchunks + 1][2][nmat][d*h] chunk-start (W, M) and, last, the final state; when states are saved.
                         // With seg > 0: [seg + 1] slots, the chunk-start states of ONE segment (recomputed by the backward)
    size_t cck;          // seg > 0: [nseg + 1][2][nmat][d*h] chunk-start states of every seg-th chunk (the checkpoints)
    int seg;             // chunks per segment (e2ttt_params.ckpt_every >= 2); 0 = the state of every chunk is kept
    size_t per_seq;      // elements per sequence
};

inline SimtLayout simt_layout(int d, int h, int C, int nmat, int nchunks, bool save_states, bool backward, int seg = 0) {
    SimtLayout l{};
    size_t o = 0;
    const size_t dh = (size_t)d * h;
    auto take = [&](size_t n) { size_t r = o; o += (n + 31) / 32 * 32; return r; };
    for (int i = 0; i < 3; ++i) { l.W[i] = take(i < nmat ? dh : 0); l.M[i] = take(i < nmat ? dh : 0); }
    l.Z1 = take((size_t)2 * C * h); l.Z2 = take((size_t)2 * C * h); l.A = take((size_t)2 * C * h);
    l.U = take((size_t)2 * C * d); l.Pu = take((size_t)C * d);
    l.Pz1 = take((size_t)C * h); l.Pz2 = take((size_t)C * h);
    if (backward) {
        for (int i = 0; i < 3; ++i) {
            l.T[i] = take(i < nmat ? dh : 0); l.S[i] = take(i < nmat ? dh : 0); l.Wb[i] = take(i < nmat ? dh : 0);
        }
        l.Pa = take((size_t)C * h); l.E = take((size_t)C * d);
        l.XY2 = take((size_t)C * 2 * d); l.XY1 = take((size_t)C * 2 * h);
        l.Pub = take((size_t)C * d); l.Pzb = take((size_t)C * h); l.Zkb = take((size_t)C * h);
        l.Akb = take((size_t)C * h); l.Kb = take((size_t)C * d); l.Eb = take((size_t)C * d);
        l.Ukb = take((size_t)C * d); l.Uqb = take((size_t)C * d); l.Zqb = take((size_t)C * h);
        const size_t sw = (nmat == 3) ? 1 : 0;
        l.XY1b = take(sw * C * 2 * h); l.Pzb2 = take(sw * C * h); l.Zkb2 = take(sw * C * h); l.Zqb2 = take(sw * C * h);
        l.rk = take(C); l.rq = take(C); l.red = take(64);
        l.kWb = take(C); l.kMb = take(C);
    }
    l.splitk = take((size_t)2 * 8 * 128 * 64);
    l.rown = take(save_states ? (size_t)nchunks * 3 * (size_t)(d > h ? d : h) : 0);
    l.seg = save_states ? seg : 0;
    if (l.seg > 0) {
        l.ckpt = take((size_t)(l.seg + 1) * 2 * nmat * dh);
        l.cck = take((size_t)((nchunks + l.seg - 1) / l.seg + 1) * 2 * nmat * dh);
    } else {
        l.ckpt = take(save_states ? (size_t)(nchunks + 1) * 2 * nmat * dh : 0);
        l.cck = 0;
    }
    l.per_seq = o;
    return l;
}

struct SimtFwdArgs {
    int N, L, d, h, C, nchunks;
    int save_states;  // 0: none; 1: the start state of every chunk -> lay.ckpt; 2: of every lay.seg-th chunk -> lay.cck
    int Ls;           // tokens between two sequences in q, k, v, o and the gates (L for a whole-sequence call; a segment
                      // call passes pointers to its first token and the full length here)
    int init_slot;    // >= 0: start from checkpoint slot init_slot of lay.cck instead of W_init / M_init; -1 otherwise
    int cl;  // CTAs per sequence (cluster size), chosen by the launcher
    int tc;  // GEMMs on the tensor cores with bf16 operands (bf16 I/O only) instead of fp32 FMAs
    int* status;  // device status word of the call (bounded waits report here)
    float eps;
    const void *q, *k, *v;
    const float *eta, *beta, *gamma;
    const float* W_init[3];
    const float* M_init[3]; // nullptr entries = zeros
    void* o;
    float* W_final[3];
    float* M_final[3];
    const float* row_norm[3];  // post-chunk normalisation targets [N, rows_i]; row_norm[0] == nullptr: none
    float norm_eps;
    void* ws;
    SimtLayout lay;
};

struct SimtBwdArgs {
    int N, L, d, h, C, nchunks;
    int Ls;           // tokens between two sequences in the token tensors (see SimtFwdArgs)
    int carry_in;     // 1: the adjoints T, S of the chunk-end state are already in the workspace (left there by the launch
                      // for the next segment); 0: read them from dW_final / dM_final
    int carry_out;    // 1: leave T, S in the workspace for the previous segment's launch; 0: write dW_init / dM_init
    int cl;  // CTAs per sequence (cluster size), chosen by the launcher
    int tc;  // GEMMs on the tensor cores with bf16 operands (bf16 I/O only) instead of fp32 FMAs
    int* status;  // device status word of the call (bounded waits report here)
    float eps;
    const void *q, *k, *v, *d_o;
    const float *eta, *beta, *gamma;
    const float* dW_final[3]; // nullptr entries = zeros
    const float* dM_final[3];
    void *dq, *dk, *dv;
    float *d_eta, *d_beta, *d_gamma;
    float* dW_init[3];
    float* dM_init[3];
    const float* row_norm[3];  // post-chunk normalisation targets [N, rows_i]; row_norm[0] == nullptr: none
    float* d_row_norm[3];      // adjoints of the targets (nullptr entries: not wanted)
    float norm_eps;
    void* ws;
    SimtLayout lay;
};

// CTAs per sequence: the largest power of two <= 8 that keeps N * cl within one wave of the GPU's SMs
inline int simt_cluster_size(int N) {
    int cl = 1;
    while (cl < 8 && (long long)N * (cl * 2) <= 148) cl *= 2;
    return cl;
}

// launchers (simt_fwd.cu / simt_bwd.cu); return a cudaError_t value as int
int simt_fwd_launch(const SimtFwdArgs& a, int kind, int io_dtype, void* stream);
int simt_bwd_launch(const SimtBwdArgs& a, int kind, int io_dtype, void* stream);

}  // namespace e2ttt
