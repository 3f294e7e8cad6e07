// Multi-scale structural similarity between two decodes of a record (the paper's diagnostic for
// choosing a scan group: MSSIM of fidelity k against full fidelity, Section 4.3).
//
// Definition used (Wang, Simoncelli and Bovik's multi-scale SSIM in its common form):
//   luminance Y = 0.299 R + 0.587 G + 0.114 B, range L = 255, C1 = (0.01 L)^2, C2 = (0.03 L)^2;
//   per scale: Gaussian 11x11 window (sigma 1.5, normalised), positions where it fits only;
//   cs = (2 s_xy + C2) / (s_x^2 + s_y^2 + C2), l = (2 m_x m_y + C1) / (m_x^2 + m_y^2 + C1),
//   averaged over the scale's positions; next scale = 2x2 block averages (odd edge dropped);
//   score = prod_j max(mean cs_j, 0)^w_j * max(mean l_M, 0)^w_M, weights 0.0448, 0.2856, 0.3001,
//   0.2363, 0.1333; with fewer than five scales (a side below 11 * 2^(M-1)) the first M weights
//   rescaled to sum to one; no scale at all (a side below 11): NaN.
// Single precision per window (on luminance minus 128, which leaves variances unchanged and
// keeps the squares small), double precision for the sums over a scale.
#pragma once
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

namespace pcr {

constexpr int kMsWin = 11;
constexpr int kMsMaxScales = 5;
constexpr int kMsTile = 16;                       // output positions per CTA side

struct MsDesc {
    uint32_t W, H, M, rsvd;
    uint64_t rgb_off;        // first byte of the image in a decode's output buffer
    uint64_t plane_off;      // first float of the image's pyramid (plane A; plane B follows it)
    uint64_t plane_len;      // floats in one pyramid
};

__device__ __forceinline__ uint64_t ms_level_off(uint32_t W, uint32_t H, int j) {
    uint64_t o = 0;
    for (int i = 0; i < j; ++i) o += (uint64_t)(W >> i) * (H >> i);
    return o;
}

struct MsWindow { float g[kMsWin]; };

// level 0 of both pyramids: luminance minus 128
__global__ void __launch_bounds__(256) ms_luma_kernel(const MsDesc* __restrict__ desc, const uint8_t* __restrict__ a,
                                                      const uint8_t* __restrict__ b, float* __restrict__ planes) {
    const MsDesc d = desc[blockIdx.y];
    if (d.M == 0) return;
    const uint64_t n = (uint64_t)d.W * d.H;
    float* pa = planes + d.plane_off;
    float* pb = pa + d.plane_len;
    for (uint64_t p = (uint64_t)blockIdx.x * 256 + threadIdx.x; p < n; p += (uint64_t)gridDim.x * 256) {
        const uint8_t* qa = a + d.rgb_off + 3 * p;
        const uint8_t* qb = b + d.rgb_off + 3 * p;
        pa[p] = 0.299f * (float)qa[0] + 0.587f * (float)qa[1] + 0.114f * (float)qa[2] - 128.f;
        pb[p] = 0.299f * (float)qb[0] + 0.587f * (float)qb[1] + 0.114f * (float)qb[2] - 128.f;
    }
}

// sums of cs and l over the positions of scale j: sums[(img * kMsMaxScales + j) * 2 + {0, 1}]
__global__ void __launch_bounds__(kMsTile * kMsTile) ms_scale_kernel(const MsDesc* __restrict__ desc, const float* __restrict__ planes,
                                                                      double* __restrict__ sums, int j, MsWindow win) {
    constexpr int kIn = kMsTile + kMsWin - 1;                      // 26 input rows / columns per tile
    __shared__ float s_x[kIn][kIn + 1], s_y[kIn][kIn + 1];
    __shared__ float s_h[5][kIn][kMsTile + 1];
    __shared__ double s_red[2][kMsTile * kMsTile / 32];
    const MsDesc d = desc[blockIdx.y];
    if ((int)d.M <= j) return;
    const int W = (int)(d.W >> j), H = (int)(d.H >> j);
    const int Wv = W - kMsWin + 1, Hv = H - kMsWin + 1;            // positions where the window fits
    const int tx = (Wv + kMsTile - 1) / kMsTile, ty = (Hv + kMsTile - 1) / kMsTile;
    const float* pa = planes + d.plane_off + ms_level_off(d.W, d.H, j);
    const float* pb = pa + d.plane_len;
    const float C1 = 6.5025f, C2 = 58.5225f;
    const int tid = threadIdx.x, lx = tid % kMsTile, ly = tid / kMsTile;
    double acc_cs = 0.0, acc_l = 0.0;
    for (int t = blockIdx.x; t < tx * ty; t += gridDim.x) {
        const int x0 = (t % tx) * kMsTile, y0 = (t / tx) * kMsTile;
        __syncthreads();
        for (int i = tid; i < kIn * kIn; i += kMsTile * kMsTile) {
            const int r = i / kIn, c = i % kIn;
            const int gx = x0 + c, gy = y0 + r;
            const bool in = gx < W && gy < H;
            s_x[r][c] = in ? pa[(size_t)gy * W + gx] : 0.f;
            s_y[r][c] = in ? pb[(size_t)gy * W + gx] : 0.f;
        }
        __syncthreads();
        for (int i = tid; i < kIn * kMsTile; i += kMsTile * kMsTile) {       // horizontal pass
            const int r = i / kMsTile, c = i % kMsTile;
            float mx = 0.f, my = 0.f, xx = 0.f, yy = 0.f, xy = 0.f;
#pragma unroll
            for (int k = 0; k < kMsWin; ++k) {
                const float g = win.g[k], vx = s_x[r][c + k], vy = s_y[r][c + k];
                mx += g * vx; my += g * vy; xx += g * vx * vx; yy += g * vy * vy; xy += g * vx * vy;
            }
            s_h[0][r][c] = mx; s_h[1][r][c] = my; s_h[2][r][c] = xx; s_h[3][r][c] = yy; s_h[4][r][c] = xy;
        }
        __syncthreads();
        if (x0 + lx < Wv && y0 + ly < Hv) {                                  // vertical pass, one position per thread
            float mx = 0.f, my = 0.f, xx = 0.f, yy = 0.f, xy = 0.f;
#pragma unroll
            for (int k = 0; k < kMsWin; ++k) {
                const float g = win.g[k];
                mx += g * s_h[0][ly + k][lx]; my += g * s_h[1][ly + k][lx];
                xx += g * s_h[2][ly + k][lx]; yy += g * s_h[3][ly + k][lx]; xy += g * s_h[4][ly + k][lx];
            }
            const float sxx = xx - mx * mx, syy = yy - my * my, sxy = xy - mx * my;
            const float ux = mx + 128.f, uy = my + 128.f;
            acc_cs += (double)((2.f * sxy + C2) / (sxx + syy + C2));
            acc_l += (double)((2.f * ux * uy + C1) / (ux * ux + uy * uy + C1));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        acc_cs += __shfl_down_sync(0xffffffffu, acc_cs, o);
        acc_l += __shfl_down_sync(0xffffffffu, acc_l, o);
    }
    __syncthreads();
    if ((tid & 31) == 0) { s_red[0][tid >> 5] = acc_cs; s_red[1][tid >> 5] = acc_l; }
    __syncthreads();
    if (tid == 0) {
        double c = 0.0, l = 0.0;
        for (int w = 0; w < kMsTile * kMsTile / 32; ++w) { c += s_red[0][w]; l += s_red[1][w]; }
        double* out = sums + ((size_t)blockIdx.y * kMsMaxScales + j) * 2;
        atomicAdd(out, c);
        atomicAdd(out + 1, l);
    }
}

// scale j -> j + 1: 2x2 block averages of both planes
__global__ void __launch_bounds__(256) ms_pool_kernel(const MsDesc* __restrict__ desc, float* __restrict__ planes, int j) {
    const MsDesc d = desc[blockIdx.y];
    if ((int)d.M <= j + 1) return;
    const uint32_t W = d.W >> j, W2 = d.W >> (j + 1), H2 = d.H >> (j + 1);
    const uint64_t n = (uint64_t)W2 * H2;
    float* src = planes + d.plane_off + ms_level_off(d.W, d.H, j);
    float* dst = planes + d.plane_off + ms_level_off(d.W, d.H, j + 1);
    for (uint64_t p = (uint64_t)blockIdx.x * 256 + threadIdx.x; p < 2 * n; p += (uint64_t)gridDim.x * 256) {
        const uint64_t q = p < n ? p : p - n;
        const uint64_t shift = p < n ? 0 : d.plane_len;                    // plane A, then plane B
        const uint32_t y = (uint32_t)(q / W2), x = (uint32_t)(q % W2);
        const float* s = src + shift + (size_t)(2 * y) * W + 2 * x;
        dst[shift + q] = 0.25f * ((s[0] + s[1]) + (s[W] + s[W + 1]));
    }
}

__global__ void __launch_bounds__(256) ms_final_kernel(const MsDesc* __restrict__ desc, const double* __restrict__ sums,
                                                       float* __restrict__ scores, int n) {
    const int i = blockIdx.x * 256 + threadIdx.x;
    if (i >= n) return;
    const MsDesc d = desc[i];
    if (d.M == 0) { scores[i] = nanf(""); return; }
    const double w5[kMsMaxScales] = {0.0448, 0.2856, 0.3001, 0.2363, 0.1333};
    double wsum = 0.0;
    for (uint32_t j = 0; j < d.M; ++j) wsum += w5[j];
    if (d.M == kMsMaxScales) wsum = 1.0;                                   // the published weights as printed
    double r = 1.0;
    for (uint32_t j = 0; j < d.M; ++j) {
        const double cnt = (double)((d.W >> j) - kMsWin + 1) * (double)((d.H >> j) - kMsWin + 1);
        const double cs = fmax(sums[((size_t)i * kMsMaxScales + j) * 2] / cnt, 0.0);
        r *= pow(cs, w5[j] / wsum);
        if (j == d.M - 1) r *= pow(fmax(sums[((size_t)i * kMsMaxScales + j) * 2 + 1] / cnt, 0.0), w5[j] / wsum);
    }
    scores[i] = (float)r;
}

}  // namespace pcr
