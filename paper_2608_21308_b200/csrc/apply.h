// Launcher of the apply kernel (outputs of fixed fast weights, no update).
#pragma once
#include <stddef.h>
#include <stdint.h>

namespace e2ttt {

struct ApplyArgs {
    int N, T, d, h;  // sequences, tokens per sequence, head dimension, hidden width
    int cl;          // CTAs per sequence (cluster size)
    int tb;          // tokens per pass (1 or 4): apply_token_block(T)
    int stage;       // stage the last matrix's block in shared memory with asynchronous copies (apply_can_stage)
    float eps;
    const void* q;   // [N, T, d] io dtype
    const float* W[3];
    void* o;         // [N, T, d] io dtype
};

int apply_token_block(int T);
// CTAs per sequence: the largest power of two <= 8 that keeps all N * cl CTAs resident at two per SM
inline int apply_cluster_size(int N) {
    int cl = 1;
    while (cl < 8 && (long long)N * (cl * 2) <= 2 * 148) cl *= 2;
    return cl;
}
size_t apply_smem_bytes(int d, int cl, int tb);  // without the 64 KB staging buffer
int apply_can_stage(int d, int h, int cl);
int apply_launch(const ApplyArgs& a, int kind, int io_dtype, void* stream);  // returns a cudaError_t value

}  // namespace e2ttt
