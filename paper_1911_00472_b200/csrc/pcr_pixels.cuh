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
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "pcr_types.h"

namespace pcr {

#ifndef PCR_PIX_MIN_CTAS
#define PCR_PIX_MIN_CTAS 10                   // CTAs per SM the compiler must leave registers for (1: 13 % slower, 14: 8 % slower)
#endif
constexpr int kPixMcus = 8;                   // MCUs per CTA (4:2:0)
constexpr int kPixThreads = 64;               // one thread per block for the transform
constexpr int kStagePitch = 3 * 128 + 16;     // bytes per staged RGB row (+ spare, keeps rows 16-byte aligned)

// Chroma sampling of a record as a template code: luminance blocks per MCU (horizontal, vertical),
// components, and the MCUs of one work unit, chosen so that a unit is 128 pixels wide and has at
// most 64 blocks: 4:2:0 -> 8 MCUs (32 Y + 8 Cb + 8 Cr), 4:2:2 -> 8 (16 + 8 + 8), 4:4:0 -> 16
// (32 + 16 + 16), 4:4:4 -> 16 (16 + 16 + 16), greyscale -> 16 (16 Y).
enum { kSamp420 = 0, kSamp422 = 1, kSamp440 = 2, kSamp444 = 3, kSampGrey = 4 };
template <int kSamp> struct Sampling;
template <> struct Sampling<kSamp420> { static constexpr int HS = 2, VS = 2, NC = 3, U = 8; };
template <> struct Sampling<kSamp422> { static constexpr int HS = 2, VS = 1, NC = 3, U = 8; };
template <> struct Sampling<kSamp440> { static constexpr int HS = 1, VS = 2, NC = 3, U = 16; };
template <> struct Sampling<kSamp444> { static constexpr int HS = 1, VS = 1, NC = 3, U = 16; };
template <> struct Sampling<kSampGrey> { static constexpr int HS = 1, VS = 1, NC = 1, U = 16; };

// zigzag position -> natural index, by walking the anti-diagonals
struct ZigzagTable {
    uint8_t nat[64];
    constexpr ZigzagTable() : nat() {
        int r = 0, c = 0;
        for (int k = 0; k < 64; ++k) {
            nat[k] = (uint8_t)(r * 8 + c);
            if (((r + c) & 1) == 0) {
                if (c == 7) ++r; else if (r == 0) ++c; else { --r; ++c; }
            } else {
                if (r == 7) ++c; else if (c == 0) ++r; else { ++r; --c; }
            }
        }
    }
};
__device__ constexpr ZigzagTable kZigzag{};

// One 8-point pass on the integer matrix M (see the header comment): out[n] = (sum_k M[n][k] x[k] + rnd) >> shift
__device__ __forceinline__ void idct8(uint32_t& x0, uint32_t& x1, uint32_t& x2, uint32_t& x3, uint32_t& x4, uint32_t& x5,
                                      uint32_t& x6, uint32_t& x7, uint32_t rnd, int shift) {
    constexpr uint32_t K1 = 8035, K2 = 7568, K3 = 6811, K4 = 5793, K5 = 4551, K6 = 3135, K7 = 1598;
    const uint32_t a0 = K4 * (x0 + x4) + rnd, a1 = K4 * (x0 - x4) + rnd;
    const uint32_t b0 = K2 * x2 + K6 * x6, b1 = K6 * x2 - K2 * x6;
    const uint32_t e0 = a0 + b0, e3 = a0 - b0, e1 = a1 + b1, e2 = a1 - b1;
    const uint32_t o0 = K1 * x1 + K3 * x3 + K5 * x5 + K7 * x7;
    const uint32_t o1 = K3 * x1 - K7 * x3 - K1 * x5 - K5 * x7;
    const uint32_t o2 = K5 * x1 - K1 * x3 + K7 * x5 + K3 * x7;
    const uint32_t o3 = K7 * x1 - K5 * x3 + K3 * x5 - K1 * x7;
    x0 = (uint32_t)((int)(e0 + o0) >> shift); x7 = (uint32_t)((int)(e0 - o0) >> shift);
    x1 = (uint32_t)((int)(e1 + o1) >> shift); x6 = (uint32_t)((int)(e1 - o1) >> shift);
    x2 = (uint32_t)((int)(e2 + o2) >> shift); x5 = (uint32_t)((int)(e2 - o2) >> shift);
    x3 = (uint32_t)((int)(e3 + o3) >> shift); x4 = (uint32_t)((int)(e3 - o3) >> shift);
}

// bytes {clamp(v0), clamp(v1), clamp(v2), clamp(v3)} of a little-endian word, clamp to 0..255
__device__ __forceinline__ uint32_t pack4_sat(int v0, int v1, int v2, int v3) {
    uint32_t hi, w;
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(v3), "r"(v2), "r"(0));
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(v1), "r"(v0), "r"(hi));
    return w;
}

// bytes {clamp(v0 + 128), ..., clamp(v3 + 128)}, clamp to 0..255, for any 32-bit v: clamping v to
// -128..127 and flipping the byte's top bit is the same as adding 128 and clamping to 0..255, and it
// needs no addition that could overflow for v near the ends of the 32-bit range
__device__ __forceinline__ uint32_t pack4_sat_plus128(int v0, int v1, int v2, int v3) {
    uint32_t hi, w;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(v3), "r"(v2), "r"(0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(w) : "r"(v1), "r"(v0), "r"(hi));
    return w ^ 0x80808080u;
}

// kRefine: first fold the side data of the AC refinement scans (see ScanAux) into the block, in
// scan order, and write the updated 128-byte line back, so the planes in device memory hold the
// final coefficients.  The thread parks its line in shared memory for that (word w of thread t
// at [w][t]): the walk over the set bits of the masks addresses coefficients by position, which
// registers cannot do.  A correction moves a non-zero coefficient away from zero by 2^Al if its
// bit Al is still clear; a new coefficient is +-2^Al.
//
// kDcMode: 0 = all 64 coefficients sit in the block's line; 1 = positions 0..7 come from the dense
// head plane (the line's first 16 bytes are ignored); 2 = the block has nothing but its DC
// coefficient (no AC scan decoded): only the head plane is read and the transform collapses to
// one value; 3 = no decoded scan reaches beyond position 7: the lines are not read at all.
// kRoi: only work units that touch their image's crop rectangle (P.roi) are processed.
//
// kStage serves triangle chroma upsampling, which needs chroma samples of neighbouring work
// units: 0 = everything in one launch (2x2 replication); 1 = chroma pass: the chroma blocks are
// folded, written back, transformed and their samples stored in P.chroma, nothing else; 2 = pixel
// pass: luminance blocks as in 0, chroma samples with a one-sample border read back from
// P.chroma, every pixel's chroma = (9 own + 3 horizontally nearer + 3 vertically nearer +
// 1 diagonal + 8) >> 4, neighbours clamped to the MCU-padded planes.
// kSamp: the record's chroma sampling (see Sampling); the triangle filter (kStage 1, 2) exists for
// 4:2:0 only.  A greyscale record has no chroma: every pixel is (Y, Y, Y).
template <bool kRefine, int kDcMode, bool kRoi = false, int kStage = 0, int kSamp = kSamp420>
__global__ void __launch_bounds__(kPixThreads, PCR_PIX_MIN_CTAS) pixel_kernel(Params P, FinalizeList fl, uint8_t* __restrict__ out) {
    using S = Sampling<kSamp>;
    constexpr int HS = S::HS, VS = S::VS, NC = S::NC, U = S::U;
    constexpr int kYCols = HS * U;                            // luminance blocks per block row of a unit
    constexpr int kYBlocks = VS * kYCols;                      // luminance blocks of a unit
    constexpr int kBlocks = kYBlocks + (NC == 3 ? 2 * U : 0);
    constexpr int kBpm = HS * VS + (NC == 3 ? 2 : 0);          // blocks per MCU
    constexpr int kPxW = 8 * HS, kPxH = 8 * VS;                // pixels per MCU
    static_assert(kBlocks <= kPixThreads && kPxW * U == 128, "a unit is 128 pixels wide and has at most 64 blocks");
    static_assert(kStage == 0 || kSamp == kSamp420, "triangle upsampling is built for 4:2:0");
    __shared__ __align__(16) uint32_t s_line[kRefine ? 32 * kPixThreads : 1];
    __shared__ __align__(16) uint8_t s_y[kPxH][128];
    __shared__ __align__(16) uint8_t s_c[2][8][8 * U];
    __shared__ __align__(16) uint8_t s_stage[kPxH * kStagePitch];
    __shared__ __align__(16) uint16_t s_q[3][64];
    __shared__ uint8_t s_ct[kStage == 2 ? 2 : 1][kStage == 2 ? 10 : 1][kStage == 2 ? 8 * kPixMcus + 2 : 1];   // chroma tile + border

    const int tid = threadIdx.x;
    const Unit un = P.units[blockIdx.x];
    const ImgDesc im = P.imgs[un.img];
    const int nm = min(U, (int)im.mx - (int)un.mcol0);                // MCUs in this unit
    if (kRoi) {                                                       // whole CTA: nothing of this unit is wanted
        const CropRect r = P.roi[un.img];
        const uint32_t ux0 = (uint32_t)kPxW * un.mcol0, uy0 = (uint32_t)kPxH * un.mrow;
        if (ux0 >= r.x0 + r.w || ux0 + (uint32_t)(kPxW * nm) <= r.x0 || uy0 >= r.y0 + r.h || uy0 + (uint32_t)kPxH <= r.y0) return;
    }
    for (int i = tid; i < 96; i += kPixThreads)
        reinterpret_cast<uint32_t*>(&s_q[0][0])[i] = __ldg(reinterpret_cast<const uint32_t*>(P.qtab + (size_t)un.img * 192) + i);
    __syncthreads();

    // ---- transform: thread j owns block j; block order: the unit's luminance block rows, then Cb, then Cr
    {
        const int j = tid;
        int comp = 0;
        bool valid = false;
        uint64_t blk = 0, local = 0;      // block number in the planes / inside its component
        int yr = 0, yc = 0;               // block row / column inside the unit
        if (j < kYBlocks) {
            yr = j / kYCols; yc = j % kYCols;
            valid = yc < HS * nm;
            local = (uint64_t)(VS * un.mrow + yr) * (HS * im.mx) + HS * un.mcol0 + yc;
            blk = im.blk_base + local;
            local += (uint64_t)(HS * VS) * (im.blk_base / kBpm);
        } else if (j < kBlocks) {
            yc = (j - kYBlocks) % U;
            comp = 1 + (j - kYBlocks) / U;
            valid = yc < nm;
            local = (uint64_t)un.mrow * im.mx + un.mcol0 + yc;
            blk = im.blk_base + (uint64_t)(HS * VS + comp - 1) * im.mx * im.my + local;
            local += im.blk_base / kBpm;
        }
        if (kStage == 1 && comp == 0) valid = false;          // chroma pass
        if (kStage == 2 && comp != 0) valid = false;          // pixel pass: chroma comes from the sample planes
        uint8_t* cplane = nullptr;                            // chroma pass: where this block's samples go
        if (kStage == 1 && comp != 0)
            cplane = P.chroma + (im.blk_base / 6) * 128 + (comp == 2 ? 64ull * im.mx * im.my : 0ull) +
                     (size_t)(8 * un.mrow) * (8 * im.mx) + 8 * (un.mcol0 + yc);
        if (valid && kDcMode == 2) {
            // all AC zero: both passes keep only the k = 0 term, every sample of the block is equal
            constexpr uint32_t K4 = 5793;
            const int F = (int)P.head[blk * 8] * (int)s_q[comp][0];
            const int T = (int)(K4 * (uint32_t)F + (1u << 11)) >> 12;
            const int smp = (int)(K4 * (uint32_t)T + (1u << 15)) >> 16;
            const uint32_t w = pack4_sat_plus128(smp, smp, smp, smp);
            uint8_t* dst;
            int pitch;
            if (comp == 0) { dst = &s_y[yr * 8][yc * 8]; pitch = 128; }
            else { dst = &s_c[comp - 1][0][yc * 8]; pitch = 8 * U; }
#pragma unroll
            for (int y = 0; y < 8; ++y) *reinterpret_cast<uint2*>(dst + y * pitch) = make_uint2(w, w);
        } else if (valid) {
            uint4* line = reinterpret_cast<uint4*>(P.planes + blk * 64);
            uint4 raw[8];
            const uint4* headv = reinterpret_cast<const uint4*>(P.head + blk * 8);
            if (kRefine && fl.n[comp] > 0) {
                // the side data of the first two refinement scans is requested before the lines: all of the
                // block's loads are then in flight together
                const int nref = fl.n[comp];
                const ulonglong2 zero2 = make_ulonglong2(0ull, 0ull);
                ulonglong2 a0 = zero2, b0 = zero2, a1 = zero2, b1 = zero2;
                {
                    const ulonglong2* o = reinterpret_cast<const ulonglong2*>(P.aux + fl.base[comp][0] + local * 4);
                    a0 = __ldg(o); b0 = __ldg(o + 1);                        // {mask, corrections}, {new, signs}
                    if (nref > 1) {
                        const ulonglong2* o1 = reinterpret_cast<const ulonglong2*>(P.aux + fl.base[comp][1] + local * 4);
                        a1 = __ldg(o1); b1 = __ldg(o1 + 1);
                    }
                }
                if (kDcMode == 3) {
#pragma unroll
                    for (int q = 1; q < 8; ++q) raw[q] = make_uint4(0, 0, 0, 0);
                } else {
#pragma unroll
                    for (int q = (kDcMode == 0 ? 0 : 1); q < 8; ++q) raw[q] = line[q];
                }
                if (kDcMode != 0) raw[0] = *headv;
                uint32_t* col = s_line + tid;
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    col[(4 * q) * kPixThreads] = raw[q].x; col[(4 * q + 1) * kPixThreads] = raw[q].y;
                    col[(4 * q + 2) * kPixThreads] = raw[q].z; col[(4 * q + 3) * kPixThreads] = raw[q].w;
                }
                uint32_t dirty = 0;                                         // 16-byte chunks of the line that changed
                for (int i = 0; i < nref; ++i) {
                    const int p1 = fl.p1[comp][i];
                    ulonglong2 a = i == 0 ? a0 : a1, b = i == 0 ? b0 : b1;
                    if (i > 1) {
                        const ulonglong2* o = reinterpret_cast<const ulonglong2*>(P.aux + fl.base[comp][i] + local * 4);
                        a = __ldg(o); b = __ldg(o + 1);
                    }
                    // corrections: the coefficients that were non-zero before the scan, in zigzag order, take the
                    // correction bits in reading order (from bit 63 down); the walk ends with the last set bit.
                    // Positions 0..31 and 32..63 are walked as 32-bit masks.
                    const uint64_t hist = a.x & ~b.x;
                    uint64_t cc = a.y;
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        uint32_t h32 = half ? (uint32_t)(hist >> 32) : (uint32_t)hist;
                        uint32_t* hb = col + half * 16 * kPixThreads;
                        while (h32 && cc) {
                            const int pos = __ffs((int)h32) - 1;
                            h32 &= h32 - 1u;
                            if ((long long)cc < 0) {
                                int16_t* e = reinterpret_cast<int16_t*>(hb + (pos >> 1) * kPixThreads) + (pos & 1);
                                const int v = *e;
                                if ((v & p1) == 0) { *e = (int16_t)(v >= 0 ? v + p1 : v - p1); dirty |= 1u << ((pos >> 3) + 4 * half); }
                            }
                            cc <<= 1;
                        }
                    }
                    // new coefficients: +-2^Al at positions that were zero
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        uint32_t nw = half ? (uint32_t)(b.x >> 32) : (uint32_t)b.x;
                        const uint32_t sg = half ? (uint32_t)(b.y >> 32) : (uint32_t)b.y;
                        uint32_t* hb = col + half * 16 * kPixThreads;
                        while (nw) {
                            const int pos = __ffs((int)nw) - 1;
                            nw &= nw - 1u;
                            *(reinterpret_cast<int16_t*>(hb + (pos >> 1) * kPixThreads) + (pos & 1)) = (int16_t)(((sg >> pos) & 1u) ? p1 : -p1);
                            dirty |= 1u << ((pos >> 3) + 4 * half);
                        }
                    }
                }
                // only the chunks that changed are read back and written to the planes
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    if ((dirty >> q) & 1u) {
                        raw[q] = make_uint4(col[(4 * q) * kPixThreads], col[(4 * q + 1) * kPixThreads],
                                            col[(4 * q + 2) * kPixThreads], col[(4 * q + 3) * kPixThreads]);
                        if (q == 0 && kDcMode != 0) *reinterpret_cast<uint4*>(P.head + blk * 8) = raw[0];
                        else if (kDcMode != 3) line[q] = raw[q];
                    }
                }
            } else {
                if (kDcMode == 3) {
#pragma unroll
                    for (int q = 1; q < 8; ++q) raw[q] = make_uint4(0, 0, 0, 0);
                } else {
#pragma unroll
                    for (int q = (kDcMode == 0 ? 0 : 1); q < 8; ++q) raw[q] = __ldg(line + q);
                }
                if (kDcMode != 0) raw[0] = __ldg(headv);
            }
            const uint32_t* qw = reinterpret_cast<const uint32_t*>(&s_q[comp][0]);
            uint32_t v[64];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const uint32_t w4[4] = {raw[q].x, raw[q].y, raw[q].z, raw[q].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int k = 8 * q + 2 * e;                 // zigzag positions k, k + 1
                    const uint32_t qq = qw[k >> 1];
                    const int c0 = (int)(short)(w4[e] & 0xFFFFu), c1 = (int)w4[e] >> 16;
                    v[kZigzag.nat[k]] = (uint32_t)(c0 * (int)(qq & 0xFFFFu));
                    v[kZigzag.nat[k + 1]] = (uint32_t)(c1 * (int)(qq >> 16));
                }
            }
            // pass 1: columns (two fraction bits kept)
#pragma unroll
            for (int u = 0; u < 8; ++u)
                idct8(v[u], v[8 + u], v[16 + u], v[24 + u], v[32 + u], v[40 + u], v[48 + u], v[56 + u], 1u << 11, 12);
            // pass 2: rows; the +128 level shift is part of the packing
            uint8_t* dst;
            int pitch;
            if (kStage == 1) { dst = cplane; pitch = 8 * (int)im.mx; }
            else if (comp == 0) { dst = &s_y[yr * 8][yc * 8]; pitch = 128; }
            else { dst = &s_c[comp - 1][0][yc * 8]; pitch = 8 * U; }
#pragma unroll
            for (int y = 0; y < 8; ++y) {
                idct8(v[8 * y], v[8 * y + 1], v[8 * y + 2], v[8 * y + 3], v[8 * y + 4], v[8 * y + 5], v[8 * y + 6], v[8 * y + 7],
                      1u << 15, 16);
                const uint32_t lo = pack4_sat_plus128((int)v[8 * y], (int)v[8 * y + 1], (int)v[8 * y + 2], (int)v[8 * y + 3]);
                const uint32_t hi = pack4_sat_plus128((int)v[8 * y + 4], (int)v[8 * y + 5], (int)v[8 * y + 6], (int)v[8 * y + 7]);
                *reinterpret_cast<uint2*>(dst + y * pitch) = make_uint2(lo, hi);
            }
        }
    }
    if (kStage == 1) return;                                // chroma pass: no pixels
    if (kStage == 2) {
        // chroma tile of the unit with a one-sample border, clamped to the padded planes
        const int cw = 8 * (int)im.mx, chh = 8 * (int)im.my, tw = 8 * nm + 2;
        const uint8_t* cbase = P.chroma + (im.blk_base / 6) * 128;
        for (int i = tid; i < 2 * 10 * tw; i += kPixThreads) {
            const int c = i / (10 * tw), rem2 = i - c * 10 * tw, r = rem2 / tw, x = rem2 - r * tw;
            const int gy = min(max(8 * (int)un.mrow + r - 1, 0), chh - 1), gx2 = min(max(8 * (int)un.mcol0 + x - 1, 0), cw - 1);
            s_ct[c][r][x] = cbase[(size_t)c * cw * chh + (size_t)gy * cw + gx2];
        }
    }
    __syncthreads();

    // ---- colour: 4 pixels per step, staged as the output's byte layout
    for (int gi = tid; gi < kPxH * 32; gi += kPixThreads) {
        const int row = gi / 32, gx = gi % 32;                  // 32 groups of four pixels per row
        if (4 * gx >= kPxW * nm) continue;
        const uint32_t yw = *reinterpret_cast<const uint32_t*>(&s_y[row][4 * gx]);
        int px[12];
        if (kStage == 2) {
            const int ry = 1 + (row >> 1), rn = ry + ((row & 1) ? 1 : -1);       // own / vertically nearer tile row
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int x = 4 * gx + e, cx = 1 + (x >> 1), cn = cx + ((x & 1) ? 1 : -1);
                const int cb = ((9 * s_ct[0][ry][cx] + 3 * s_ct[0][ry][cn] + 3 * s_ct[0][rn][cx] + s_ct[0][rn][cn] + 8) >> 4) - 128;
                const int cr = ((9 * s_ct[1][ry][cx] + 3 * s_ct[1][ry][cn] + 3 * s_ct[1][rn][cx] + s_ct[1][rn][cn] + 8) >> 4) - 128;
                const int Y = (int)((yw >> (8 * e)) & 255u);
                px[e * 3 + 0] = Y + ((91881 * cr + 32768) >> 16);
                px[e * 3 + 1] = Y + ((-22553 * cb - 46802 * cr + 32768) >> 16);
                px[e * 3 + 2] = Y + ((116130 * cb + 32768) >> 16);
            }
        } else if (NC == 1) {
#pragma unroll
            for (int e = 0; e < 4; ++e) px[3 * e] = px[3 * e + 1] = px[3 * e + 2] = (int)((yw >> (8 * e)) & 255u);
        } else if (HS == 1) {
            // every pixel its own chroma sample of row (row / VS)
            const uint32_t cbw = *reinterpret_cast<const uint32_t*>(&s_c[0][row / VS][4 * gx]);
            const uint32_t crw = *reinterpret_cast<const uint32_t*>(&s_c[1][row / VS][4 * gx]);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int cb = (int)((cbw >> (8 * e)) & 255u) - 128, cr = (int)((crw >> (8 * e)) & 255u) - 128;
                const int Y = (int)((yw >> (8 * e)) & 255u);
                px[e * 3 + 0] = Y + ((91881 * cr + 32768) >> 16);
                px[e * 3 + 1] = Y + ((-22553 * cb - 46802 * cr + 32768) >> 16);
                px[e * 3 + 2] = Y + ((116130 * cb + 32768) >> 16);
            }
        } else {
        const uint32_t cbw = *reinterpret_cast<const uint16_t*>(&s_c[0][row / VS][2 * gx]);
        const uint32_t crw = *reinterpret_cast<const uint16_t*>(&s_c[1][row / VS][2 * gx]);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int cb = (int)((cbw >> (8 * h)) & 255u) - 128, cr = (int)((crw >> (8 * h)) & 255u) - 128;
            const int dr = (91881 * cr + 32768) >> 16;
            const int dg = (-22553 * cb - 46802 * cr + 32768) >> 16;
            const int db = (116130 * cb + 32768) >> 16;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int Y = (int)((yw >> (8 * (2 * h + e))) & 255u);
                px[(2 * h + e) * 3 + 0] = Y + dr;
                px[(2 * h + e) * 3 + 1] = Y + dg;
                px[(2 * h + e) * 3 + 2] = Y + db;
            }
        }
        }
        uint32_t* d = reinterpret_cast<uint32_t*>(s_stage + row * kStagePitch + 12 * gx);
        d[0] = pack4_sat(px[0], px[1], px[2], px[3]);
        d[1] = pack4_sat(px[4], px[5], px[6], px[7]);
        d[2] = pack4_sat(px[8], px[9], px[10], px[11]);
    }
    __syncthreads();

    // ---- store: each staged row is a contiguous byte run of the output
    const int x0 = kPxW * (int)un.mcol0;
    const int npx = min(kPxW * nm, (int)im.W - x0);
    const int nrows = min(kPxH, (int)im.H - kPxH * (int)un.mrow);
    const int nbytes = 3 * npx;
    uint8_t* gbase = out + im.out_off + ((uint64_t)(kPxH * un.mrow) * im.W + x0) * 3;
    const size_t gpitch = (size_t)im.W * 3;
    if (((reinterpret_cast<uintptr_t>(gbase) | gpitch | (uintptr_t)nbytes) & 15u) == 0) {
        // rows start and end on 16-byte boundaries: whole 16-byte vectors
        const int vec = nbytes >> 4;
        for (int i = tid; i < nrows * vec; i += kPixThreads) {
            const int row = i / vec, c = i % vec;
            *reinterpret_cast<uint4*>(gbase + row * gpitch + 16 * c) = *reinterpret_cast<const uint4*>(s_stage + row * kStagePitch + 16 * c);
        }
    } else {
        // rows at any byte address.  The 16-byte-aligned chunks of global memory that lie inside a row:
        // five staged words shifted into place, one 16-byte store
        constexpr int kInner = (3 * 128) / 16 - 1;
        for (int i = tid; i < nrows * kInner; i += kPixThreads) {
            const int row = i / kInner, slot = 1 + (i - row * kInner);
            uint8_t* gp = gbase + row * gpitch;
            const int lead = (int)(reinterpret_cast<uintptr_t>(gp) & 15u);
            if (16 * slot + 16 > lead + nbytes) continue;     // the row's last chunk, or behind it
            const int o0 = 16 * slot - lead;                  // the chunk's first byte, counted from the row's first
            const uint32_t* q = reinterpret_cast<const uint32_t*>(s_stage + row * kStagePitch) + (o0 >> 2);
            const int sh = 8 * (o0 & 3);
            const uint32_t p0 = q[0], p1 = q[1], p2 = q[2], p3 = q[3], p4 = q[4];   // (the spare bytes keep p4 in bounds)
            *reinterpret_cast<uint4*>(gp + o0) = make_uint4(__funnelshift_r(p0, p1, sh), __funnelshift_r(p1, p2, sh),
                                                            __funnelshift_r(p2, p3, sh), __funnelshift_r(p3, p4, sh));
        }
        // the first and the last chunk of every row: whole words where they lie inside the row, else bytes
        if (tid < 2 * nrows) {
            const int row = tid >> 1;
            uint8_t* gp = gbase + row * gpitch;
            const int lead = (int)(reinterpret_cast<uintptr_t>(gp) & 15u);
            const int nch = (lead + nbytes + 15) >> 4;
            if (!(tid & 1) || nch > 1) {
                const int o0 = 16 * ((tid & 1) ? nch - 1 : 0) - lead;
                const uint8_t* srow = s_stage + row * kStagePitch;
                const uint32_t* sw = reinterpret_cast<const uint32_t*>(srow);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int sb = o0 + 4 * j;                // first staged byte of this output word
                    if (sb >= 0 && sb + 4 <= nbytes) {
                        const uint32_t lo = sw[sb >> 2], hi = sw[(sb >> 2) + 1];   // the spare bytes keep hi in bounds
                        *reinterpret_cast<uint32_t*>(gp + sb) = __funnelshift_r(lo, hi, 8 * (sb & 3));
                    } else {
                        for (int b = max(sb, 0); b < min(sb + 4, nbytes); ++b) gp[b] = srow[b];
                    }
                }
            }
        }
    }
}

// Pixel stage when nothing but DC coefficients has been decoded and every image is a multiple of
// 16 pixels wide: each 8x8 luminance block is one constant sample, each MCU one chroma pair, so
// an MCU row of the output is runs of eight equal pixels.  A CTA takes one work unit (8 MCUs of
// one MCU row): 32 threads turn the unit's 32 luminance blocks into RGB triples (the same
// arithmetic as the general kernel: the transform collapses to its k = 0 term, samples clamp to
// 0..255), then every thread writes 16-byte vectors whose bytes are picked from the two triples
// of the vector's MCU half-row.  48 bytes per MCU row = 3 vectors, so a vector never leaves its MCU.
// kAligned = false: images of any width.  A row of the unit then starts at any byte address: every
// thread takes one 16-byte-aligned chunk of global memory that the row touches, builds its four
// words from the triples of the (at most two) pixels each word covers, and stores the chunk whole
// when it lies inside the row, byte by byte at the row's two ends.
template <bool kRoi, bool kAligned = true>
__global__ void __launch_bounds__(128) dc_pixel_kernel(Params P, uint8_t* __restrict__ out) {
    __shared__ uint32_t s_tri[2][2 * kPixMcus];        // [block row of the MCU row][block column]: R | G << 8 | B << 16
    const int tid = threadIdx.x;
    const Unit un = P.units[blockIdx.x];
    const ImgDesc im = P.imgs[un.img];
    const int nm = min((int)kPixMcus, (int)im.mx - (int)un.mcol0);
    if (kRoi) {
        const CropRect r = P.roi[un.img];
        const uint32_t ux0 = 16u * un.mcol0, uy0 = 16u * un.mrow;
        if (ux0 >= r.x0 + r.w || ux0 + 16u * (uint32_t)nm <= r.x0 || uy0 >= r.y0 + r.h || uy0 + 16u <= r.y0) return;
    }
    if (tid < 4 * nm) {
        constexpr uint32_t K4 = 5793;
        const int brow = tid / (2 * nm), bcol = tid % (2 * nm);
        const uint16_t* q = P.qtab + (size_t)un.img * 192;
        auto sample = [&](uint64_t blk, int comp) {
            const int F = (int)P.head[blk * 8] * (int)q[64 * comp];
            const int T = (int)(K4 * (uint32_t)F + (1u << 11)) >> 12;
            const int smp = ((int)(K4 * (uint32_t)T + (1u << 15)) >> 16) + 128;
            return min(max(smp, 0), 255);
        };
        const uint64_t mcus = (uint64_t)im.mx * im.my;
        const uint64_t yb = im.blk_base + (uint64_t)(2 * un.mrow + brow) * (2 * im.mx) + 2 * un.mcol0 + bcol;
        const uint64_t cbk = im.blk_base + 4 * mcus + (uint64_t)un.mrow * im.mx + un.mcol0 + (bcol >> 1);
        const int Y = sample(yb, 0), cb = sample(cbk, 1) - 128, cr = sample(cbk + mcus, 2) - 128;
        const int R = Y + ((91881 * cr + 32768) >> 16);
        const int G = Y + ((-22553 * cb - 46802 * cr + 32768) >> 16);
        const int B = Y + ((116130 * cb + 32768) >> 16);
        s_tri[brow][bcol] = (uint32_t)min(max(R, 0), 255) | ((uint32_t)min(max(G, 0), 255) << 8) | ((uint32_t)min(max(B, 0), 255) << 16);
    }
    __syncthreads();
    const int nrows = min(16, (int)im.H - 16 * (int)un.mrow);
    const size_t gpitch = (size_t)im.W * 3;
    uint8_t* gbase = out + im.out_off + ((uint64_t)(16 * un.mrow) * im.W + 16 * (uint64_t)un.mcol0) * 3;
    if (!kAligned) {
        const int len = 3 * min(16 * nm, (int)im.W - 16 * (int)un.mcol0);      // bytes of the unit in one output row
        // the four bytes at offset o of a row (o may lie up to 15 bytes before the row or behind its end:
        // those bytes are not stored, their pixels are clamped into the unit): pixel px from channel ph
        // on, then pixel px + 1
        auto word_at = [&](const uint32_t* tri, int o) {
            const int oo = o + 24;
            const int px = (int)(((uint32_t)oo * 0xAAABu) >> 17) - 8, ph = oo - 3 * (px + 8);
            const uint32_t A = tri[min(max(px, 0), 16 * nm - 1) >> 3], Bt = tri[min(max(px + 1, 0), 16 * nm - 1) >> 3];
            return __byte_perm(A, Bt, ph == 0 ? 0x4210u : (ph == 1 ? 0x5421u : 0x6542u));
        };
        // the bytes of one output row of the unit, once per block row (the eight pixel rows of a block row are
        // equal), with 16 bytes of margin on either side so that a chunk may begin before the row or end behind it
        constexpr int kPatWords = (16 + 3 * 16 * kPixMcus + 16) / 4;
        __shared__ __align__(16) uint32_t s_pat[2][kPatWords];
        for (int i = tid; i < 2 * kPatWords; i += 128) {
            const int br = i / kPatWords, wi = i - br * kPatWords;
            s_pat[br][wi] = word_at(s_tri[br], 4 * wi - 16);
        }
        __syncthreads();
        // the 16 bytes of a row from offset o on (o >= -16): five pattern words, shifted into place
        auto chunk_at = [&](const uint32_t* pat, int o) {
            const int sb = o + 16, a = 8 * (sb & 3);
            const uint32_t* q = pat + (sb >> 2);
            const uint32_t p0 = q[0], p1 = q[1], p2 = q[2], p3 = q[3], p4 = q[4];
            return make_uint4(__funnelshift_r(p0, p1, a), __funnelshift_r(p1, p2, a), __funnelshift_r(p2, p3, a), __funnelshift_r(p3, p4, a));
        };
        // chunks that lie inside the row: whole 16-byte stores
        constexpr int kInner = (3 * 16 * kPixMcus) / 16 - 1;
        for (int i = tid; i < nrows * kInner; i += 128) {
            const int row = i / kInner, slot = 1 + (i - row * kInner);
            uint8_t* g = gbase + row * gpitch;                                  // first byte of the row
            const int lead = (int)(reinterpret_cast<uintptr_t>(g) & 15u);
            if (16 * slot + 16 > lead + len) continue;                          // the row's last chunk, or behind it
            const int o0 = 16 * slot - lead;                                    // the chunk's first byte, counted from g
            *reinterpret_cast<uint4*>(g + o0) = chunk_at(s_pat[row >> 3], o0);
        }
        // the first and the last chunk of every row: whole words where they lie inside, else bytes
        if (tid < 2 * nrows) {
            const int row = tid >> 1;
            uint8_t* g = gbase + row * gpitch;
            const int lead = (int)(reinterpret_cast<uintptr_t>(g) & 15u);
            const int nch = (lead + len + 15) >> 4;
            const int slot = (tid & 1) ? nch - 1 : 0;
            if (!(tid & 1) || nch > 1) {
                const int o0 = 16 * slot - lead;
                const uint4 v = chunk_at(s_pat[row >> 3], o0);
                const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int o = o0 + 4 * j;
                    if (o >= 0 && o + 4 <= len) {
                        *reinterpret_cast<uint32_t*>(g + o) = w4[j];
                    } else {
#pragma unroll
                        for (int b = 0; b < 4; ++b)
                            if (o + b >= 0 && o + b < len) g[o + b] = (uint8_t)(w4[j] >> (8 * b));
                    }
                }
            }
        }
        return;
    }
    const int vec = 3 * nm;                                 // 16-byte vectors per output row of this unit
    for (int i = tid; i < nrows * vec; i += 128) {
        const int row = i / vec, v = i - row * vec, mcu = v / 3, kk = v - 3 * mcu;
        const uint32_t A = s_tri[row >> 3][2 * mcu], Bt = s_tri[row >> 3][2 * mcu + 1];
        // four-byte words of a run of equal pixels repeat with period three: RGBR GBRG BRGB
        const uint32_t aw0 = __byte_perm(A, 0, 0x0210), aw1 = __byte_perm(A, 0, 0x1021), aw2 = __byte_perm(A, 0, 0x2102);
        const uint32_t bw0 = __byte_perm(Bt, 0, 0x0210), bw1 = __byte_perm(Bt, 0, 0x1021), bw2 = __byte_perm(Bt, 0, 0x2102);
        uint4 o;
        if (kk == 0) o = make_uint4(aw0, aw1, aw2, aw0);           // bytes 0..15: left pixels
        else if (kk == 1) o = make_uint4(aw1, aw2, bw0, bw1);      // bytes 16..23 left, 24..31 right
        else o = make_uint4(bw2, bw0, bw1, bw2);                   // bytes 32..47: right pixels
        *reinterpret_cast<uint4*>(gbase + row * gpitch + 16 * v) = o;
    }
}

// Training-tensor epilogue: crop, optional mirror, bilinear resize to size x size with half-pixel
// centres (the crop's edge pixels repeated, no low-pass filter), (v / 255 - mean) / std, planar
// output [image][channel][row][column].  Images pos0 .. pos0 + gridDim.y - 1 of the processing order.
struct TensorArgs {
    const CropRect* crops;     // [N], by image index
    void* out;                 // [N][3][size][size]
    int32_t size;
    int32_t f32;               // output type: 0 half precision, 1 single precision, 2 bfloat16
    float mean[3], inv_std[3];
};

__device__ __forceinline__ void tensor_store(float* p, float v) { *p = v; }
__device__ __forceinline__ void tensor_store(__half* p, float v) { *p = __float2half_rn(v); }
__device__ __forceinline__ void tensor_store(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// Two horizontally adjacent RGB pixels (six bytes at any alignment) as floats, read as aligned
// words: the word holding the first byte, the next one, and a third only when the six bytes reach
// into it.  `same`: the right neighbour is the pixel itself (clamped at the crop's edge).
__device__ __forceinline__ void load_rgb_pair(const uint8_t* p, bool same, float& r0, float& g0, float& b0,
                                              float& r1, float& g1, float& b1) {
    const uint32_t a = (uint32_t)(reinterpret_cast<uintptr_t>(p) & 3u);
    const uint32_t* w = reinterpret_cast<const uint32_t*>(p - a);
    const uint32_t w0 = __ldg(w), w1 = __ldg(w + 1);
    const uint32_t w2 = (a == 3u && !same) ? __ldg(w + 2) : 0u;
    const uint32_t lo = __funnelshift_r(w0, w1, 8 * a), hi = __funnelshift_r(w1, w2, 8 * a);   // bytes 0..3, 4..7
    r0 = __uint_as_float(__byte_perm(lo, 0x4B000000u, 0x7540)) - 8388608.f;      // byte into the mantissa of 2^23
    g0 = __uint_as_float(__byte_perm(lo, 0x4B000000u, 0x7541)) - 8388608.f;
    b0 = __uint_as_float(__byte_perm(lo, 0x4B000000u, 0x7542)) - 8388608.f;
    r1 = same ? r0 : __uint_as_float(__byte_perm(lo, 0x4B000000u, 0x7543)) - 8388608.f;
    g1 = same ? g0 : __uint_as_float(__byte_perm(hi, 0x4B000000u, 0x7540)) - 8388608.f;
    b1 = same ? b0 : __uint_as_float(__byte_perm(hi, 0x4B000000u, 0x7541)) - 8388608.f;
}

#ifndef PCR_TENSOR_ROWS
#define PCR_TENSOR_ROWS 16
#endif
constexpr int kTensorRows = PCR_TENSOR_ROWS;      // output rows per CTA

// One CTA per band of kTensorRows output rows of one image, one output column per thread (the
// column's horizontal taps and weights are computed once for the band).  The taps are read from
// global memory through the read-only path: neighbouring threads and rows hit the same cache
// lines (staging the band's source rows in shared memory first was 40 % slower: it costs the
// L1 capacity that these reads live on).
template <typename OutT>
__global__ void __launch_bounds__(256) tensor_kernel(Params P, TensorArgs T, const uint8_t* __restrict__ rgb, uint32_t pos0) {
    __shared__ int s_off0[kTensorRows], s_off1[kTensorRows];       // byte offsets of a row's upper / lower source row in the crop
    __shared__ float s_ay[kTensorRows];
    const uint32_t img = P.order[pos0 + blockIdx.y];
    const int S = T.size;
    const int oy0 = blockIdx.x * kTensorRows;
    const int nrows = min(kTensorRows, S - oy0);
    const ImgDesc im = P.imgs[img];
    const CropRect r = T.crops[img];
    const float sx = (float)r.w / (float)S, sy = (float)r.h / (float)S;
    const uint32_t pitch = im.W * 3u;
    const uint8_t* crop0 = rgb + im.out_off + (size_t)r.y0 * pitch + (size_t)r.x0 * 3;   // first byte of the crop
    if ((int)threadIdx.x < nrows) {
        float fy = ((float)(oy0 + (int)threadIdx.x) + 0.5f) * sy - 0.5f;
        fy = fminf(fmaxf(fy, 0.f), (float)(r.h - 1));
        const int iy = (int)floorf(fy), iy1 = min(iy + 1, (int)r.h - 1);
        s_ay[threadIdx.x] = fy - (float)iy;
        s_off0[threadIdx.x] = iy * (int)pitch; s_off1[threadIdx.x] = iy1 * (int)pitch;   // an image stays below 2 GiB
    }
    __syncthreads();
    const uint32_t plane = (uint32_t)S * (uint32_t)S;
    const float k255 = 1.f / 255.f;
    const float m0 = T.mean[0], m1 = T.mean[1], m2 = T.mean[2], i0 = T.inv_std[0], i1 = T.inv_std[1], i2 = T.inv_std[2];
    OutT* const obase = static_cast<OutT*>(T.out) + (size_t)img * 3 * plane + (size_t)oy0 * S;
    for (int ox = threadIdx.x; ox < S; ox += 256) {
        const int u = r.flip ? S - 1 - ox : ox;
        float fx = ((float)u + 0.5f) * sx - 0.5f;
        fx = fminf(fmaxf(fx, 0.f), (float)(r.w - 1));
        const int ix = (int)floorf(fx);
        const float ax = fx - (float)ix, bx = 1.f - ax;
        const uint8_t* p0 = crop0 + 3 * ix;
        const bool same = ix + 1 > (int)r.w - 1;            // the right tap is clamped onto the left one
        OutT* o = obase + ox;
        for (int dy = 0; dy < nrows; ++dy, o += S) {
            const int q0 = s_off0[dy], q1 = s_off1[dy];
            const float ay = s_ay[dy], by = 1.f - ay;
            float r00, g00, b00, r01, g01, b01, r10, g10, b10, r11, g11, b11;
            load_rgb_pair(p0 + q0, same, r00, g00, b00, r01, g01, b01);
            load_rgb_pair(p0 + q1, same, r10, g10, b10, r11, g11, b11);
            const float tr = bx * r00 + ax * r01, tg = bx * g00 + ax * g01, tb = bx * b00 + ax * b01;
            const float hr = bx * r10 + ax * r11, hg = bx * g10 + ax * g11, hb = bx * b10 + ax * b11;
            tensor_store(o, ((by * tr + ay * hr) * k255 - m0) * i0);
            tensor_store(o + plane, ((by * tg + ay * hg) * k255 - m1) * i1);
            tensor_store(o + 2 * plane, ((by * tb + ay * hb) * k255 - m2) * i2);
        }
    }
}

// Copies the head plane into positions 0..7 of every block (for readers of the full planes).
__global__ void __launch_bounds__(256) merge_head_kernel(Params P, uint64_t n_blocks) {
    const uint64_t b = (uint64_t)blockIdx.x * 256 + threadIdx.x;
    if (b < n_blocks) *reinterpret_cast<uint4*>(P.planes + b * 64) = *reinterpret_cast<const uint4*>(P.head + b * 8);
}

}  // namespace pcr
