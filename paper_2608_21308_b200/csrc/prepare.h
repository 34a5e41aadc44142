// Launchers of the token-preparation kernels (prepare.cu).
#pragma once
#include <stddef.h>
#include <stdint.h>

namespace e2ttt {

struct PrepareArgs {
    long long rows;  // B * H * L token-heads
    int d;
    float eta_base, tau, alpha_base, norm_eps;
    const void *q_raw, *k_raw;                  // [rows, d] io dtype
    const float *a_eta, *a_beta, *a_alpha;      // [rows] gate logits
    void *q, *k;                                // [rows, d] io dtype
    float *eta, *beta, *gamma;                  // [rows]
};

struct PrepareBwdArgs {
    PrepareArgs f;                              // the forward's inputs (its outputs are not needed)
    const void *dq, *dk;                        // [rows, d] io dtype
    const float *d_eta, *d_beta, *d_gamma;      // [rows]
    void *dq_raw, *dk_raw;                      // [rows, d] io dtype
    float *da_eta, *da_beta, *da_alpha;         // [rows]
};

// return a cudaError_t value as int
int prepare_fwd_launch(const PrepareArgs& a, int io_dtype, void* stream);
int prepare_bwd_launch(const PrepareBwdArgs& a, int io_dtype, void* stream);

}  // namespace e2ttt
