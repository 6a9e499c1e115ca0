// Internal launch interface between the C ABI (api.cu) and the kernel files.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>

namespace mgn {

struct Problem {
    int BH, S, D, causal;
    float scale;
};

// Tensor maps (host side).  rank-3 view (D, S, BH) of a dense [BH,S,D] tensor with
// a (box_d, box_rows, 1) box and the 128-byte swizzle.  Returns 0 on success.
int make_tmap_3d(CUtensorMap* out, const void* base, int elem_bytes, int is_bf16,
                 int BH, int S, int D, int box_d, int box_rows);

// Strict (f32 FFMA) kernels.
cudaError_t launch_strict_fwd(const Problem& p, const float* q, const float* k, const float* v,
                              float* o, float* lse, unsigned* status, cudaStream_t st);
cudaError_t launch_strict_bwd(const Problem& p, const float* q, const float* k, const float* v,
                              const float* d_o, const float* lse, const float* delta,
                              float* dq, float* dk, float* dv, unsigned* status, cudaStream_t st);

// delta_i = sum_d dO[i,d] O[i,d]  (f32 or bf16 inputs, f32 output), HBM-bound; also clears the
// f32 dQ accumulation target `zero` ([rows][D] floats).
cudaError_t launch_bwd_preprocess(const void* o, const void* d_o, float* delta, float* zero,
                                  size_t rows, int D, int is_bf16, cudaStream_t st);

// Fast (bf16 tcgen05) kernels.
cudaError_t launch_fast_fwd(const Problem& p, const void* q, const void* k, const void* v,
                            void* o, float* lse, unsigned* status, cudaStream_t st);
cudaError_t launch_fast_bwd(const Problem& p, const void* q, const void* k, const void* v,
                            const void* d_o, const float* lse, const float* delta,
                            float* dq_acc, void* dq, void* dk, void* dv,
                            unsigned* status, cudaStream_t st);

}  // namespace mgn
