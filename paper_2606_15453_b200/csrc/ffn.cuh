// Routed SwiGLU expert FFN (Section 2: experts are feed-forward networks whose outputs are
// summed with the gating probabilities as weights), written as weight-streaming GEMVs: the
// step is bound by reading every routed expert's weights once from HBM.
//
// Work unit: one warp streams R rows (gate/up: R rows of both matrices) of one expert for the
// <= MT tokens of a work-list entry, 16 bytes per lane per load, U loads per row in flight,
// and reduces the split-K partial sums with warp shuffles.  Activations are re-read from L1.
// Partial outputs go to fixed places and are summed in a fixed order, so results are
// reproducible run to run (no floating-point atomics).
#pragma once
#include "device_utils.cuh"
#include "router.cuh"

namespace stmoe_dev {

constexpr int kFfnThreads = 256;

struct FfnArgs {
    const float *h;          // [B][H] layer input (un-normalised)
    const float *inv_rms;    // [B] or nullptr (x = h)
    WorkList wl;
    const uint8_t *const *blob;  // [E + n_shared] expert image of each expert for this layer
    float *act;              // [B*(K+n_shared)][I]
    float *part;             // [B*(K+n_shared)][H]
    int H, I, E;
};

// Layout of one expert image.
__host__ __device__ inline size_t image_gate(int, int, int) { return 0; }
__host__ __device__ inline size_t image_up(int H, int I, int wb) { return (size_t)H * I * wb; }
__host__ __device__ inline size_t image_down(int H, int I, int wb) { return 2 * (size_t)H * I * wb; }
__host__ __device__ inline size_t image_scales(int H, int I, int wb) { return 3 * (size_t)H * I * wb; }

// acc[m][r][t] += sum over this lane's columns of W_m[row r][col] * x_t[col]
template <int DT, int NMAT, int R, int MT, int U>
__device__ __forceinline__ void gemv_rows(const uint8_t *(&rowp)[NMAT][R], const float *(&xp)[MT],
                                          int cols, int lane, float (&acc)[NMAT][R][MT])
{
    constexpr int EPL = Fmt<DT>::kEpl, BYTES = Fmt<DT>::kBytes, STEP = kWarp * EPL;
    for (int k0 = lane * EPL; k0 < cols; k0 += STEP * U) {
        uint4 wv[U][NMAT][R];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int k = k0 + u * STEP;
            if (k < cols) {
#pragma unroll
                for (int m = 0; m < NMAT; ++m)
#pragma unroll
                    for (int r = 0; r < R; ++r) wv[u][m][r] = ld_stream16(rowp[m][r] + (size_t)k * BYTES);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int k = k0 + u * STEP;
            if (k < cols) {
                float xv[MT][EPL];
#pragma unroll
                for (int t = 0; t < MT; ++t)
#pragma unroll
                    for (int e = 0; e < EPL; e += 4) {
                        const float4 v = ld_f4(xp[t] + k + e);
                        xv[t][e] = v.x, xv[t][e + 1] = v.y, xv[t][e + 2] = v.z, xv[t][e + 3] = v.w;
                    }
#pragma unroll
                for (int m = 0; m < NMAT; ++m)
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        float wf[EPL];
                        Fmt<DT>::unpack(wv[u][m][r], wf);
#pragma unroll
                        for (int t = 0; t < MT; ++t)
#pragma unroll
                            for (int e = 0; e < EPL; ++e) acc[m][r][t] = fmaf(wf[e], xv[t][e], acc[m][r][t]);
                    }
            }
        }
    }
}

// act[slot][i] = silu(g_i) * u_i,  g = W_g x, u = W_u x,  x = h * inv_rms  (folded into g, u)
template <int DT, int R, int MT, int U>
__global__ void __launch_bounds__(kFfnThreads) gate_up_kernel(FfnArgs a)
{
    constexpr int BYTES = Fmt<DT>::kBytes;
    const int lane = threadIdx.x % kWarp;
    const int wid = (blockIdx.x * kFfnThreads + threadIdx.x) / kWarp;
    const int nwarps = gridDim.x * (kFfnThreads / kWarp);
    const int H = a.H, I = a.I;
    const int blocks = (I + R - 1) / R;
    const int items = *a.wl.n_groups * blocks;
    const size_t row_bytes = (size_t)H * BYTES;

    for (int it = wid; it < items; it += nwarps) {
        const int g = it / blocks, r0 = (it % blocks) * R;
        const int ex = a.wl.g_expert[g], start = a.wl.g_start[g], cnt = a.wl.g_count[g];
        const uint8_t *img = a.blob[ex];
        const uint8_t *rowp[2][R];
        const float *xp[MT];
        int tok[MT], slot[MT];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int row = min(r0 + r, I - 1);
            rowp[0][r] = img + image_gate(H, I, BYTES) + row * row_bytes;
            rowp[1][r] = img + image_up(H, I, BYTES) + row * row_bytes;
        }
#pragma unroll
        for (int t = 0; t < MT; ++t) {
            const int p = start + min(t, cnt - 1);
            tok[t] = a.wl.pair_token[p], slot[t] = a.wl.pair_slot[p];
            xp[t] = a.h + (size_t)tok[t] * H;
        }
        float acc[2][R][MT];
#pragma unroll
        for (int m = 0; m < 2; ++m)
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int t = 0; t < MT; ++t) acc[m][r][t] = 0.f;
        gemv_rows<DT, 2, R, MT, U>(rowp, xp, H, lane, acc);

        const uint16_t *sc = reinterpret_cast<const uint16_t *>(img + image_scales(H, I, BYTES));
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int t = 0; t < MT; ++t) {
                float gv = warp_sum(acc[0][r][t]), uv = warp_sum(acc[1][r][t]);
                if (lane == (r * MT + t) % kWarp && r0 + r < I && t < cnt) {
                    const float inv = a.inv_rms ? a.inv_rms[tok[t]] : 1.f;
                    gv *= inv, uv *= inv;
                    if (DT == 2) {
                        gv *= bf16_to_f32(sc[r0 + r]);
                        uv *= bf16_to_f32(sc[I + r0 + r]);
                    }
                    a.act[(size_t)slot[t] * I + r0 + r] = gv / (1.f + expf(-gv)) * uv;
                }
            }
    }
}

// part[slot][h] = (W_d act[slot])[h]
template <int DT, int R, int MT, int U>
__global__ void __launch_bounds__(kFfnThreads) down_kernel(FfnArgs a)
{
    constexpr int BYTES = Fmt<DT>::kBytes;
    const int lane = threadIdx.x % kWarp;
    const int wid = (blockIdx.x * kFfnThreads + threadIdx.x) / kWarp;
    const int nwarps = gridDim.x * (kFfnThreads / kWarp);
    const int H = a.H, I = a.I;
    const int blocks = (H + R - 1) / R;
    const int items = *a.wl.n_groups * blocks;
    const size_t row_bytes = (size_t)I * BYTES;

    for (int it = wid; it < items; it += nwarps) {
        const int g = it / blocks, r0 = (it % blocks) * R;
        const int ex = a.wl.g_expert[g], start = a.wl.g_start[g], cnt = a.wl.g_count[g];
        const uint8_t *img = a.blob[ex];
        const uint8_t *rowp[1][R];
        const float *xp[MT];
        int slot[MT];
#pragma unroll
        for (int r = 0; r < R; ++r)
            rowp[0][r] = img + image_down(H, I, BYTES) + min(r0 + r, H - 1) * row_bytes;
#pragma unroll
        for (int t = 0; t < MT; ++t) {
            slot[t] = a.wl.pair_slot[start + min(t, cnt - 1)];
            xp[t] = a.act + (size_t)slot[t] * I;
        }
        float acc[1][R][MT];
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int t = 0; t < MT; ++t) acc[0][r][t] = 0.f;
        gemv_rows<DT, 1, R, MT, U>(rowp, xp, I, lane, acc);

        const uint16_t *sc = reinterpret_cast<const uint16_t *>(img + image_scales(H, I, BYTES));
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int t = 0; t < MT; ++t) {
                float v = warp_sum(acc[0][r][t]);
                if (lane == (r * MT + t) % kWarp && r0 + r < H && t < cnt) {
                    if (DT == 2) v *= bf16_to_f32(sc[2 * I + r0 + r]);
                    a.part[(size_t)slot[t] * H + r0 + r] = v;
                }
            }
    }
}

// h_out[b][i] = h[b][i] + r * ( sum_shared part + sum_k w[b][k] * part ), fixed order
__global__ void __launch_bounds__(256)
combine_kernel(const float *__restrict__ h, const float *__restrict__ part, const float *__restrict__ w,
               int B, int H, int K, int n_shared, float residual_scale, float *__restrict__ h_out)
{
    const int KS = K + n_shared;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < (size_t)B * H;
         i += (size_t)gridDim.x * blockDim.x) {
        const int b = (int)(i / H), c = (int)(i % H);
        float y = 0.f;
        for (int s = 0; s < n_shared; ++s) y += part[((size_t)b * KS + K + s) * H + c];
        for (int k = 0; k < K; ++k) y = fmaf(w[b * K + k], part[((size_t)b * KS + k) * H + c], y);
        h_out[i] = fmaf(residual_scale, y, h[i]);
    }
}

}  // namespace stmoe_dev
