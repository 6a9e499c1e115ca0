// Backward preprocess: delta_i = sum_d dO[i,d] * O[i,d] for every (b,h,i) row.
// HBM-bound streaming kernel: 128-bit loads, D/4 (f32) or D/8 (bf16) lanes per row,
// shuffle reduction inside the lane group.  The same pass clears the f32 dQ accumulation target
// (row r of `zero`, D floats), which saves a separate memset launch.  (The paper's backward kernels need this
// row statistic; it is the "backward preprocess" step of the attention path.)
#include <cuda_bf16.h>

#include "kernels.h"
#include "ptx.cuh"

namespace mgn {
namespace {

// L2 eviction hints: the accumulator that the next kernel reduces into should stay in L2, the
// streamed inputs should not push it out.
__device__ __forceinline__ uint64_t l2_policy_keep() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_stream() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void st_hint(float4* a, float4 v, uint64_t pol) {
    asm volatile("st.global.L2::cache_hint.v4.f32 [%0], {%1,%2,%3,%4}, %5;" ::"l"(a), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "l"(pol) : "memory");
}
__device__ __forceinline__ uint4 ld_hint(const uint4* a, uint64_t pol) {
    uint4 v;
    asm volatile("ld.global.nc.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(a), "l"(pol));
    return v;
}

template <int LANES, bool BF16>
__global__ void __launch_bounds__(256)
bwd_preprocess_kernel(const uint4* __restrict__ o, const uint4* __restrict__ d_o, float* __restrict__ delta,
                      float4* __restrict__ zero, unsigned* __restrict__ counter, size_t rows)
{
    pdl_launch_dependents();   // the backward main kernel may set itself up while this one streams
    if (counter && blockIdx.x == 0 && threadIdx.x == 0) *counter = 0u;
    constexpr int ROWS_PER_BLOCK = 256 / LANES;
    const int lane = threadIdx.x % LANES;
    const int sub = threadIdx.x / LANES;
    const uint64_t keep = l2_policy_keep(), stream = l2_policy_stream();
    for (size_t r0 = static_cast<size_t>(blockIdx.x) * ROWS_PER_BLOCK; r0 < rows;
         r0 += static_cast<size_t>(gridDim.x) * ROWS_PER_BLOCK) {
        const size_t r = r0 + sub;
        float acc = 0.f;
        if (r < rows) {
            constexpr int ZPL = BF16 ? 2 : 1;      // float4 stores per lane to cover a row of D floats
#pragma unroll
            for (int t = 0; t < ZPL; ++t)
                if (zero) st_hint(&zero[(r * LANES + lane) * ZPL + t], make_float4(0.f, 0.f, 0.f, 0.f), keep);
            const uint4 a = ld_hint(o + r * LANES + lane, stream);
            const uint4 b = ld_hint(d_o + r * LANES + lane, stream);
            if constexpr (BF16) {
                const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
                const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&b);
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const float2 fa = __bfloat1622float2(pa[t]), fb = __bfloat1622float2(pb[t]);
                    acc = fmaf(fa.x, fb.x, acc);
                    acc = fmaf(fa.y, fb.y, acc);
                }
            } else {
                acc = fmaf(__uint_as_float(a.x), __uint_as_float(b.x), acc);
                acc = fmaf(__uint_as_float(a.y), __uint_as_float(b.y), acc);
                acc = fmaf(__uint_as_float(a.z), __uint_as_float(b.z), acc);
                acc = fmaf(__uint_as_float(a.w), __uint_as_float(b.w), acc);
            }
        }
#pragma unroll
        for (int off = LANES / 2; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (r < rows && lane == 0) delta[r] = acc;
    }
}

// Clears the dQ accumulation target and the work-item counter: what is left of the preprocess pass
// when delta comes from elsewhere (the dO producer of the output projection).
__global__ void __launch_bounds__(256)
bwd_clear_kernel(float4* __restrict__ zero, size_t n4, unsigned* __restrict__ counter)
{
    pdl_launch_dependents();
    if (counter && blockIdx.x == 0 && threadIdx.x == 0) *counter = 0u;
    if (!zero) return;
    const uint64_t keep = l2_policy_keep();
    for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n4;
         i += static_cast<size_t>(gridDim.x) * blockDim.x)
        st_hint(&zero[i], make_float4(0.f, 0.f, 0.f, 0.f), keep);
}

template <int LANES, bool BF16>
cudaError_t run(const void* o, const void* d_o, float* delta, float* zero, unsigned* counter, size_t rows, cudaStream_t st)
{
    constexpr int ROWS_PER_BLOCK = 256 / LANES;
    size_t blocks = (rows + ROWS_PER_BLOCK - 1) / ROWS_PER_BLOCK;
    const size_t cap = 148u * 8u * 4u;
    if (blocks > cap) blocks = cap;
    bwd_preprocess_kernel<LANES, BF16><<<static_cast<unsigned>(blocks), 256, 0, st>>>(
        static_cast<const uint4*>(o), static_cast<const uint4*>(d_o), delta, reinterpret_cast<float4*>(zero), counter, rows);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_bwd_clear(float* zero, size_t n_floats, unsigned* counter, cudaStream_t st)
{
    const size_t n4 = n_floats / 4;
    const size_t cap = 148u * 16u;
    const size_t blocks = n4 / 256 + 1 < cap ? n4 / 256 + 1 : cap;
    bwd_clear_kernel<<<static_cast<unsigned>(blocks), 256, 0, st>>>(reinterpret_cast<float4*>(zero), n4, counter);
    return cudaGetLastError();
}

cudaError_t launch_bwd_preprocess(const void* o, const void* d_o, float* delta, float* zero, unsigned* counter,
                                  size_t rows, int D, int is_bf16, cudaStream_t st)
{
    if (is_bf16) {
        switch (D) {
            case 32:  return run<4, true>(o, d_o, delta, zero, counter, rows, st);
            case 64:  return run<8, true>(o, d_o, delta, zero, counter, rows, st);
            case 128: return run<16, true>(o, d_o, delta, zero, counter, rows, st);
        }
    } else {
        switch (D) {
            case 32:  return run<8, false>(o, d_o, delta, zero, counter, rows, st);
            case 64:  return run<16, false>(o, d_o, delta, zero, counter, rows, st);
            case 128: return run<32, false>(o, d_o, delta, zero, counter, rows, st);
        }
    }
    return cudaErrorInvalidValue;
}

}  // namespace mgn
