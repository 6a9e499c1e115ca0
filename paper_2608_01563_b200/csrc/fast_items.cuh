// Shapes and work-item dealing shared by the persistent fast (tcgen05) kernels.
#pragma once

namespace mgn {

// Shapes: q, o, d_o, dq [BH = B*H, Sq, D]; k, v, dk, dv [B*H/G, Sk, D]; query head h reads
// key/value head h / G; causal: key j is visible to query i iff j <= i + off, off = Sk - Sq >= 0.
struct Dims {
    int Sq, Sk, BH, H, G, off;
};

// k-th item of CTA c out of G, -1 past the end (then also for every larger k).
//   order 0 (block-major): tiers of G items, odd tiers dealt backwards (snake);
//   order 1 (head-major):  CTA c takes the consecutive item pairs c, c+G, c+2G, ...
__device__ __forceinline__ int item_index(int c, int k, int G, int n_items, int order) {
    const int it = order == 0 ? k * G + ((k & 1) ? (G - 1 - c) : c) : 2 * (c + G * (k >> 1)) + (k & 1);
    return it < n_items ? it : -1;
}

}  // namespace mgn
