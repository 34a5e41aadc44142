// Host interface of the tensor-core forward for SwiGLU fast weights (tc_swiglu.cu).
#pragma once
#include <cuda_bf16.h>
#include <stddef.h>

namespace e2ttt {

struct TcSwigluArgs {
    int N, L;  // sequences, tokens per sequence (L a multiple of the chunk size); d = 128, h = 384 are compiled in
    int C;     // chunk size: 64, or 32 / 16 (short chunks run in the 64-row tiles, unused rows zero); 0 = 64
    int Ls;    // tokens between two sequences in q, k, v, o and the gates; 0 = L (a call on a token sub-range of longer
               // sequences passes pointers to its first token and the full length here)
    size_t init_seq_stride, final_seq_stride;  // floats between two sequences in *_init / *_final; 0 = d * h
    int keep_status;  // 1: one launch of several that share the status word: do not clear it
    float eps;
    const __nv_bfloat16 *q, *k, *v;
    const float *eta, *beta, *gamma;
    const float *W1_init, *W2_init, *W3_init, *M1_init, *M2_init, *M3_init;  // M*_init may be nullptr (zeros)
    __nv_bfloat16* o;  // nullptr: the outputs are not wanted
    float *W1_final, *W2_final, *W3_final, *M1_final, *M2_final, *M3_final;
    int* status;  // device word, 0 after a clean run
    // optional: chunk-start states for the backward, fp32, slot c = [W1 | W2 | W3 | M1 | M2 | M3] at the start of chunk
    // c (nullptr = do not save); ckpt_every >= 2: only chunks 0, n, 2n, .. in slots 0, 1, 2, ..
    float* ckpt;
    size_t ckpt_seq_stride;  // floats between two sequences
    int ckpt_every;
};

size_t tc_swiglu_smem_bytes();
// returns a cudaError_t value as int (0 = launched)
int tc_swiglu_launch(const TcSwigluArgs& a, void* stream);

}  // namespace e2ttt
