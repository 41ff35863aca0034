// fp8 (e4m3) expert stacks on the tensor cores: the kernels that feed dense_group.cuh's fp8
// operand format.  tcgen05.mma.kind::f8f6f4 multiplies the e4m3 weight tiles as TMA lands them
// (no widening pass, no extra shared-memory round trip) against activations held as three e5m2
// planes: plane 0 is the activation rounded to e5m2 (f16's exponent range, so no scale has to be
// found first), plane 1 the rounded residue, plane 2 the residue of that; their sum differs from
// the activation by at most 2^-9 of its magnitude, the precision of a bf16 operand.  The hidden
// state's planes are written here, the gated activations' planes by the gate/up epilogue.
#pragma once
#include "dense_group.cuh"

namespace stmoe_dev {

// planes of the hidden state: x8[p][t][c], p < 3, t < 64 (kDenseMaxTokens rows per plane)
__device__ __forceinline__ void store_e5m2_planes(uint8_t *x8, size_t plane_elems, size_t i, float v)
{
    uint8_t tp[3];
    split_e5m2x3(v, tp);
#pragma unroll
    for (int p = 0; p < 3; ++p) x8[p * plane_elems + i] = tp[p];
}

// h_out[b][c] = h[b][c] + r * (weighted sum of the partial sums); the e5m2 planes are the next
// layer's gate/up operand
__global__ void __launch_bounds__(256) dense8_combine_kernel(FfnArgs a, int S, uint8_t *x8)
{
    const size_t plane = (size_t)kDenseMaxTokens * a.H;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < a.B * a.H; i += gridDim.x * blockDim.x) {
        const float v = finish_value(a, i / a.H, i % a.H, S);
        a.h_out[i] = v;
        store_e5m2_planes(x8, plane, (size_t)i, v);
    }
}

__global__ void __launch_bounds__(256) dense8_cast_kernel(const float *__restrict__ h, int n, int H, uint8_t *__restrict__ x8)
{
    const size_t plane = (size_t)kDenseMaxTokens * H;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x)
        store_e5m2_planes(x8, plane, (size_t)i, h[i]);
}

}  // namespace stmoe_dev
