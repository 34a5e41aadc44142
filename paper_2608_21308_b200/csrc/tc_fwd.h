// Host interface of the tensor-core forward (tc_fwd.cu).
#pragma once
#include <cuda_bf16.h>
#include <stddef.h>

namespace e2ttt {

struct TcFwdArgs {
    int N, L;  // sequences, tokens per sequence (L a multiple of the chunk size)
    int C;     // chunk size: 64, or 32 / 16 (a short chunk runs in the 64-row tiles with the unused rows zero and their
               // scalar kernels zero); 0 = 64
    int Ls;    // tokens between two sequences in q, k, v, o and the gates; 0 = L.  A call on a token sub-range of longer
               // sequences (the backward's recomputation) passes pointers to its first token and the full length here
    size_t init_seq_stride, final_seq_stride;  // floats between two sequences in *_init / *_final; 0 = d * h
    int keep_status;  // 1: one launch of several that share the status word: do not clear it
    int d, h;  // head dimension (64 or 128) and hidden width (a multiple of 128, at most 512): smaller shapes run
               // zero-padded inside the 128 x 512 tiles the kernel is built for
    float eps;
    const __nv_bfloat16 *q, *k, *v;
    const float *eta, *beta, *gamma;
    const float *W1_init, *W2_init, *M1_init, *M2_init;  // M*_init may be nullptr (zeros)
    __nv_bfloat16* o;  // nullptr: the outputs are not wanted
    float *W1_final, *W2_final, *M1_final, *M2_final;
    int* status;  // device word, 0 after a clean run
    // optional: chunk-start states for the backward, fp32, [N][nchunks][W1 | W2 | M1 | M2] (nullptr = do not save)
    float* ckpt;
    size_t ckpt_seq_stride;  // floats between two sequences
    int ckpt_every;          // >= 2: only the start states of chunks 0, n, 2n, .. are saved, in slots 0, 1, 2, .. (not with norm1)
    // optional post-chunk normalisation: per-row target norms of W1 [N, h] and W2 [N, d] (nullptr = none).  With ckpt
    // the kernel also writes what the normalised reverse pass reads: the final state as one more ckpt slot and the
    // row norms before normalisation, rown[N (stride ckpt_seq_stride)][nchunks][3][max(d, h)]
    const float *norm1, *norm2;
    float norm_eps;
    float* rown;
};

size_t tc_fwd_smem_bytes();
// returns a cudaError_t value as int (0 = launched)
int tc_fwd_launch(const TcFwdArgs& a, void* stream);

}  // namespace e2ttt
