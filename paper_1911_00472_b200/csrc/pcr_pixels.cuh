// Pixel stage of the PCR decoder: dequantise -> 8x8 inverse DCT -> 2x2 chroma replication ->
// YCbCr to RGB -> crop -> packed uint8 store, fused in one kernel.
//
// Integer specification (the CPU oracle implements the same function from its definition):
//   F = coef * Q                                              (int32)
//   pass 1, columns:  T(y,u) = (sum_v M[y][v] F(v,u) + 2^11) >> 12
//   pass 2, rows:     s(y,x) = (sum_u M[x][u] T(y,u) + 2^15) >> 16,  sample = clamp(s + 128)
//   M[n][k] = round(8192 * c_k * cos((2n+1) k pi / 16)), c_0 = 1/sqrt 2, i.e. +-K_j with
//   K_j = round(8192 cos(j pi / 16)); all sums modulo 2^32, shifts arithmetic.
//   The sums are evaluated here by an even/odd butterfly, which is exact integer algebra on
//   the same matrix, so the result is identical to the plain matrix product.
//   R = clamp(Y + ((91881 cr + 32768) >> 16)), G = clamp(Y + ((-22553 cb - 46802 cr + 32768) >> 16)),
//   B = clamp(Y + ((116130 cb + 32768) >> 16)) with cb, cr = sample - 128 of chroma (x>>1, y>>1).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "pcr_types.h"

namespace pcr {

constexpr int kPixMcus = 8;                   // MCUs per CTA
constexpr int kPixBlocks = 6 * kPixMcus;      // 32 Y + 8 Cb + 8 Cr
constexpr int kPixThreads = 8 * kPixBlocks;   // one thread per block column / row
constexpr int kBlkPitch = 72;                 // words per block in shared memory: 8 rows of 9
constexpr int kStagePitch = 3 * 16 * kPixMcus + 4;   // bytes per staged RGB row (+ one spare word)

// zigzag position -> natural index, by walking the anti-diagonals
struct ZigzagTable {
    uint8_t nat[64];
    uint8_t pad[64];   // position inside a 9-word-pitch block
    constexpr ZigzagTable() : nat(), pad() {
        int r = 0, c = 0;
        for (int k = 0; k < 64; ++k) {
            nat[k] = (uint8_t)(r * 8 + c);
            pad[k] = (uint8_t)(r * 9 + c);
            if (((r + c) & 1) == 0) {
                if (c == 7) ++r; else if (r == 0) ++c; else { --r; ++c; }
            } else {
                if (r == 7) ++c; else if (c == 0) ++r; else { ++r; --c; }
            }
        }
    }
};
__device__ constexpr ZigzagTable kZigzag{};

__device__ __forceinline__ void idct8(const uint32_t x[8], int out[8], uint32_t rnd, int shift) {
    constexpr uint32_t K1 = 8035, K2 = 7568, K3 = 6811, K4 = 5793, K5 = 4551, K6 = 3135, K7 = 1598;
    uint32_t a0 = K4 * (x[0] + x[4]), a1 = K4 * (x[0] - x[4]);
    uint32_t b0 = K2 * x[2] + K6 * x[6], b1 = K6 * x[2] - K2 * x[6];
    uint32_t e0 = a0 + b0 + rnd, e3 = a0 - b0 + rnd, e1 = a1 + b1 + rnd, e2 = a1 - b1 + rnd;
    uint32_t o0 = K1 * x[1] + K3 * x[3] + K5 * x[5] + K7 * x[7];
    uint32_t o1 = K3 * x[1] - K7 * x[3] - K1 * x[5] - K5 * x[7];
    uint32_t o2 = K5 * x[1] - K1 * x[3] + K7 * x[5] + K3 * x[7];
    uint32_t o3 = K7 * x[1] - K5 * x[3] + K3 * x[5] - K1 * x[7];
    out[0] = (int)(e0 + o0) >> shift; out[7] = (int)(e0 - o0) >> shift;
    out[1] = (int)(e1 + o1) >> shift; out[6] = (int)(e1 - o1) >> shift;
    out[2] = (int)(e2 + o2) >> shift; out[5] = (int)(e2 - o2) >> shift;
    out[3] = (int)(e3 + o3) >> shift; out[4] = (int)(e3 - o3) >> shift;
}

__device__ __forceinline__ uint32_t clamp255(int v) { return (uint32_t)min(max(v, 0), 255); }

__global__ void __launch_bounds__(kPixThreads) pixel_kernel(Params P, uint8_t* __restrict__ out) {
    __shared__ __align__(16) uint32_t s_coef[kPixBlocks * kBlkPitch];
    __shared__ __align__(16) uint8_t s_y[16][16 * kPixMcus];
    __shared__ __align__(16) uint8_t s_c[2][8][8 * kPixMcus];
    __shared__ uint8_t s_zpad[64];

    const int tid = threadIdx.x;
    const Unit un = P.units[blockIdx.x];
    const ImgDesc im = P.imgs[un.img];
    const int nm = min((int)kPixMcus, (int)im.mx - (int)un.mcol0);   // MCUs in this unit
    if (tid < 64) s_zpad[tid] = kZigzag.pad[tid];
    __syncthreads();

    // ---- load + dequantise: shared block order is Y row 0 (16), Y row 1 (16), Cb (8), Cr (8)
    const uint64_t ybase = im.blk_base, cbbase = im.blk_base + 4ull * im.mx * im.my, crbase = cbbase + (uint64_t)im.mx * im.my;
    const uint16_t* q = P.qtab + (size_t)un.img * 192;
    for (int idx = tid; idx < kPixBlocks * 32; idx += kPixThreads) {
        int j = idx >> 5, w = idx & 31;
        int comp, valid;
        uint64_t blk;
        if (j < 32) {
            int r = j >> 4, c = j & 15;
            comp = 0; valid = c < 2 * nm;
            blk = ybase + (uint64_t)(2 * un.mrow + r) * (2 * im.mx) + 2 * un.mcol0 + c;
        } else {
            int c = (j - 32) & 7;
            comp = 1 + ((j - 32) >> 3); valid = c < nm;
            blk = (comp == 1 ? cbbase : crbase) + (uint64_t)un.mrow * im.mx + un.mcol0 + c;
        }
        if (valid) {
            uint32_t v = __ldg(reinterpret_cast<const uint32_t*>(P.planes + blk * 64) + w);
            uint32_t qq = __ldg(reinterpret_cast<const uint32_t*>(q + comp * 64) + w);
            int c0 = (int)(int16_t)(v & 0xFFFFu), c1 = (int)v >> 16;
            s_coef[j * kBlkPitch + s_zpad[2 * w]] = (uint32_t)(c0 * (int)(qq & 0xFFFFu));
            s_coef[j * kBlkPitch + s_zpad[2 * w + 1]] = (uint32_t)(c1 * (int)(qq >> 16));
        }
    }
    __syncthreads();

    const int j = tid >> 3, t8 = tid & 7;
    bool valid;
    if (j < 32) valid = (j & 15) < 2 * nm; else valid = ((j - 32) & 7) < nm;
    uint32_t* blkp = s_coef + j * kBlkPitch;
    // ---- pass 1: column t8
    if (valid) {
        uint32_t x[8]; int o[8];
#pragma unroll
        for (int v = 0; v < 8; ++v) x[v] = blkp[v * 9 + t8];
        idct8(x, o, 1u << 11, 12);
#pragma unroll
        for (int v = 0; v < 8; ++v) blkp[v * 9 + t8] = (uint32_t)o[v];
    }
    __syncthreads();
    // ---- pass 2: row t8
    if (valid) {
        uint32_t x[8]; int o[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) x[u] = blkp[t8 * 9 + u];
        idct8(x, o, 1u << 15, 16);
        uint32_t lo = clamp255(o[0] + 128) | (clamp255(o[1] + 128) << 8) | (clamp255(o[2] + 128) << 16) | (clamp255(o[3] + 128) << 24);
        uint32_t hi = clamp255(o[4] + 128) | (clamp255(o[5] + 128) << 8) | (clamp255(o[6] + 128) << 16) | (clamp255(o[7] + 128) << 24);
        uint2* dst;
        if (j < 32) dst = reinterpret_cast<uint2*>(&s_y[(j >> 4) * 8 + t8][(j & 15) * 8]);
        else dst = reinterpret_cast<uint2*>(&s_c[(j - 32) >> 3][t8][((j - 32) & 7) * 8]);
        *dst = make_uint2(lo, hi);
    }
    __syncthreads();

    // ---- colour: 4 pixels per step, staged as the output's byte layout (aliases s_coef)
    uint8_t* stage = reinterpret_cast<uint8_t*>(s_coef);
    for (int gi = tid; gi < 16 * 4 * kPixMcus; gi += kPixThreads) {
        int row = gi / (4 * kPixMcus), gx = gi % (4 * kPixMcus);
        if (gx >= 4 * nm) continue;
        uint32_t yw = *reinterpret_cast<const uint32_t*>(&s_y[row][4 * gx]);
        uint32_t cbw = *reinterpret_cast<const uint16_t*>(&s_c[0][row >> 1][2 * gx]);
        uint32_t crw = *reinterpret_cast<const uint16_t*>(&s_c[1][row >> 1][2 * gx]);
        uint32_t px[12];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            int cb = (int)((cbw >> (8 * h)) & 255u) - 128, cr = (int)((crw >> (8 * h)) & 255u) - 128;
            int dr = (91881 * cr + 32768) >> 16;
            int dg = (-22553 * cb - 46802 * cr + 32768) >> 16;
            int db = (116130 * cb + 32768) >> 16;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                int Y = (int)((yw >> (8 * (2 * h + e))) & 255u);
                px[(2 * h + e) * 3 + 0] = clamp255(Y + dr);
                px[(2 * h + e) * 3 + 1] = clamp255(Y + dg);
                px[(2 * h + e) * 3 + 2] = clamp255(Y + db);
            }
        }
        uint32_t* d = reinterpret_cast<uint32_t*>(stage + row * kStagePitch + 12 * gx);
        d[0] = px[0] | (px[1] << 8) | (px[2] << 16) | (px[3] << 24);
        d[1] = px[4] | (px[5] << 8) | (px[6] << 16) | (px[7] << 24);
        d[2] = px[8] | (px[9] << 8) | (px[10] << 16) | (px[11] << 24);
    }
    __syncthreads();

    // ---- store: each staged row is a contiguous byte run of the output; write aligned words
    const int x0 = 16 * (int)un.mcol0;
    const int npx = min(16 * nm, (int)im.W - x0);
    const int nrows = min(16, (int)im.H - 16 * (int)un.mrow);
    const int nbytes = 3 * npx;
    const int wid = tid >> 5, lane = tid & 31;
    for (int row = wid; row < nrows; row += kPixThreads / 32) {
        uint64_t g0 = im.out_off + ((uint64_t)(16 * un.mrow + row) * im.W + x0) * 3;
        uint8_t* gp = out + g0;
        const int a = (int)(reinterpret_cast<uintptr_t>(gp) & 3u);
        const uint8_t* srow = stage + row * kStagePitch;
        const uint32_t* sw = reinterpret_cast<const uint32_t*>(srow);
        const int nw = (a + nbytes + 3) >> 2;
        for (int i = lane; i < nw; i += 32) {
            int sb = 4 * i - a;                     // first staged byte of this output word
            if (sb >= 0 && sb + 4 <= nbytes) {
                uint32_t lo = sw[sb >> 2], hi = sw[(sb >> 2) + 1];   // the spare word keeps hi in bounds
                uint32_t v = a ? __funnelshift_r(lo, hi, 8 * (sb & 3)) : lo;
                *reinterpret_cast<uint32_t*>(gp + sb) = v;
            } else {
                for (int b = max(sb, 0); b < min(sb + 4, nbytes); ++b) gp[b] = srow[b];
            }
        }
    }
}

}  // namespace pcr
