// Shared-memory tile access shared by the strict (FFMA) backward kernels.  Tiles arrive by TMA in
// the 128-byte-swizzled layout described in strict_fwd.cu.
#pragma once
#include "ptx.cuh"

namespace mgn {

// d columns owned by column group tc: D=32 -> {2tc, 2tc+1}; else {4tc + 64e + 0..3}.
template <int D, int R>
__device__ __forceinline__ void load_row_cols(uint32_t tile, int r, int r7, int tc, float (&out)[D / 16]) {
    if constexpr (D == 32) {
        const float2 t = lds64(tile + r * 128 + (((tc >> 1) ^ r7) << 4) + (tc & 1) * 8);
        out[0] = t.x; out[1] = t.y;
    } else {
#pragma unroll
        for (int e = 0; e < D / 64; ++e) {
            const int piece = tc + 16 * e;
            const float4 t = lds128(tile + (piece >> 3) * (R * 128) + r * 128 + (((piece & 7) ^ r7) << 4));
            out[4 * e + 0] = t.x; out[4 * e + 1] = t.y; out[4 * e + 2] = t.z; out[4 * e + 3] = t.w;
        }
    }
}

__device__ __forceinline__ float f4_get(const float4& v, int u) {
    return u == 0 ? v.x : u == 1 ? v.y : u == 2 ? v.z : v.w;
}

}  // namespace mgn
