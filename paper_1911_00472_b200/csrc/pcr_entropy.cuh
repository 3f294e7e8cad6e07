// Entropy stage of the PCR decoder: restart-interval index, progressive Huffman decode of one
// wave of scans, and the pass that folds the refinement scans into the coefficient planes.
//
// Parallel decomposition: one LANE per restart interval.  A warp takes up to 32 consecutive
// restart intervals of one (scan, image) pair, so its lanes share the scan's Huffman tables
// (lookup tables in shared memory).  Every lane runs ONE flat loop whose iteration decodes one
// Huffman symbol (or one block of an end-of-band run); block changes are a few predicated
// instructions inside that loop, so lanes that sit in different blocks stay converged.
//
// First passes write coefficients straight into the (pre-zeroed) planes.  An AC refinement
// needs, per block, only WHICH band positions are already non-zero: a 64-bit mask.  First-pass
// AC scans leave that mask as side data; a refinement lane reads it, decodes with bit
// operations (skipping r zero positions = dropping r set bits of the inverted mask; one
// correction bit per set bit of the mask passed over) and leaves {new mask, correction bits,
// new positions, their signs} as side data.  The pixel kernel folds that side data into each
// block before it transforms it and writes the updated block back, so the planes in device
// memory end up holding the final coefficients.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "pcr_types.h"

namespace pcr {

constexpr int kErrCorrupt = -3;

#ifndef PCR_LUT_BITS
#define PCR_LUT_BITS 11
#endif
#ifndef PCR_ENTROPY_WARPS
#define PCR_ENTROPY_WARPS 3
#endif
constexpr int kLutBits = PCR_LUT_BITS;
constexpr int kEntropyWarps = PCR_ENTROPY_WARPS;

// Decoder tables of one Huffman table: a direct lookup on the next kBits bits for short
// codes, and the canonical first-code / count / index triple per length for the rest.
template <int kBits>
struct HuffTabT {
    uint16_t lut[1 << kBits];  // (length << 8) | symbol, 0 = longer than kBits (or undefined)
    uint32_t first[17];
    uint16_t cnt[17];
    uint16_t idx[17];
    uint8_t vals[256];
};
using HuffTab = HuffTabT<kLutBits>;

template <int kBits>
__device__ __forceinline__ void build_hufftab(HuffTabT<kBits>& t, const uint8_t* __restrict__ dht, int lane) {
    // dht: 16 length counts, then the symbol values in code order
    uint32_t code = 0, p = 0;
    for (int l = 1; l <= 16; ++l) {
        uint32_t c = dht[l - 1];
        if (lane == 0) { t.first[l] = code; t.cnt[l] = (uint16_t)c; t.idx[l] = (uint16_t)p; }
        code = (code + c) << 1;
        p += c;
    }
    const uint32_t nvals = min(p, 256u);
    for (uint32_t j = lane; j < nvals; j += 32) t.vals[j] = dht[16 + j];
    uint32_t* lw = reinterpret_cast<uint32_t*>(t.lut);
    for (int e = lane; e < (1 << kBits) / 2; e += 32) lw[e] = 0;
    __syncwarp();
    // every symbol with a short code fills its 2^(kBits - length) entries, all lanes together
    uint32_t j = 0;
    for (int l = 1; l <= kBits; ++l) {
        const uint32_t c = t.cnt[l], f = t.first[l], span = 1u << (kBits - l);
        for (uint32_t i = 0; i < c && j < nvals; ++i, ++j) {
            const uint32_t base = (f + i) << (kBits - l);
            const uint16_t entry = (uint16_t)(((uint32_t)l << 8) | t.vals[j]);
            if (base + span <= (1u << kBits))
                for (uint32_t e = lane; e < span; e += 32) t.lut[base + e] = entry;
        }
    }
    __syncwarp();
}

// MSB-first bit reader over the unstuffed copy of the entropy-coded bytes (see
// unstuff_index_kernel), which holds big-endian 32-bit words.  Each lane owns one column of a
// 16-word ring in shared memory.  All lanes of the warp top their rings up together
// (16-byte global loads), then decode for a while reading single words from the ring: the
// serial decode chain only ever waits on shared memory, and the latency of global memory is
// paid once per top-up for the whole warp instead of once per lane and load.
constexpr int kRingWords = 16;

struct BitReader {
    uint32_t* col;        // this lane's ring column: word j lives at col[(j & 15) * 32]
    const uint4* g4;      // the unstuffed copy as 16-byte groups
    uint32_t rd, wr;      // next word to consume / to fetch (absolute word indices, wr a multiple of 4)
    uint32_t rd0;         // first word of the restart interval
    uint64_t buf;         // left-aligned bit buffer
    int nbits;            // bits held in buf
    uint32_t lead;        // bits of the first word that precede the interval
    uint32_t limit;       // bits in the restart interval

    __device__ __forceinline__ void init(uint32_t* ring_col, const uint8_t* ubuf, uint32_t bstart, uint32_t bend) {
        col = ring_col;
        g4 = reinterpret_cast<const uint4*>(ubuf);
        rd = rd0 = bstart >> 2;
        wr = rd & ~3u;
        buf = 0; nbits = 0;
        lead = 8u * (bstart & 3u);
        limit = (bend - bstart) * 8u;
    }
    // fetch as many 16-byte groups as the ring has room for (all lanes call this together)
    __device__ __forceinline__ void topup(bool on) {
        const int room = on ? (int)(kRingWords - (wr - rd)) >> 2 : 0;
        uint4 v0, v1, v2, v3;
        if (room > 0) v0 = __ldg(g4 + (wr >> 2));
        if (room > 1) v1 = __ldg(g4 + (wr >> 2) + 1);
        if (room > 2) v2 = __ldg(g4 + (wr >> 2) + 2);
        if (room > 3) v3 = __ldg(g4 + (wr >> 2) + 3);
        if (room > 0) put(wr, v0);
        if (room > 1) put(wr + 4, v1);
        if (room > 2) put(wr + 8, v2);
        if (room > 3) put(wr + 12, v3);
        wr += 4u * (uint32_t)max(room, 0);
    }
    __device__ __forceinline__ void put(uint32_t w, const uint4& v) {
        uint32_t* p = col + (w & (kRingWords - 1)) * 32;
        p[0] = v.x; p[32] = v.y; p[64] = v.z; p[96] = v.w;
    }
    // enough words in the ring for one whole decode step (a code, its extra bits, 63 raw bits)
    __device__ __forceinline__ bool ready() const { return wr - rd >= 3u; }
    // once, after the first top-up: take the first word without the bytes that precede the interval
    __device__ __forceinline__ void prime() {
        const uint32_t w = col[(rd & (kRingWords - 1)) * 32] << lead;
        buf = (uint64_t)w << 32;
        nbits = 32 - (int)lead;
        ++rd;
    }
    // afterwards at least 33 bits are held
    __device__ __forceinline__ void refill() {
        if (nbits <= 32) {
            const uint32_t w = col[(rd & (kRingWords - 1)) * 32];
            buf |= (uint64_t)w << (32 - nbits);
            nbits += 32;
            ++rd;
        }
    }
    __device__ __forceinline__ uint32_t top32() const { return (uint32_t)(buf >> 32); }
    __device__ __forceinline__ void skip(int n) { buf <<= n; nbits -= n; }
    __device__ __forceinline__ bool overran() const { return (int)((rd - rd0) * 32u - lead) - nbits > (int)limit; }
};

// Huffman symbol at the top of the 32-bit window; returns (length << 8) | symbol, 0 if undefined
template <int kBits>
__device__ __forceinline__ uint32_t huff_lookup(const HuffTabT<kBits>& t, uint32_t win) {
    uint32_t e = t.lut[win >> (32 - kBits)];
    if (e) return e;
    const uint32_t w16 = win >> 16;
    for (int l = kBits + 1; l <= 16; ++l) {
        uint32_t d = (w16 >> (16 - l)) - t.first[l];
        if (d < t.cnt[l]) return ((uint32_t)l << 8) | t.vals[(t.idx[l] + d) & 255u];   // (index masked: damaged tables stay in bounds)
    }
    return 0;
}

__device__ __forceinline__ int extend_bits(uint32_t v, int s) {
    // value of an s-bit magnitude field: the top bit clear means negative
    return s == 0 ? 0 : ((v >> (s - 1)) ? (int)v : (int)v - (1 << s) + 1);
}
// the top n bits of x (n in 0..32)
__device__ __forceinline__ uint32_t top_bits(uint32_t x, int n) { return n ? x >> (32 - n) : 0u; }

// ---------------------------------------------------------------------------------------
// Restart-interval index and unstuffing, one warp per (listed scan, image).
// Copies the pair's entropy-coded bytes into P.ubuf with the zero byte after every 0xFF
// removed, bytes of each aligned group of four stored in reverse (big-endian words), at the
// same start offset as in the record.  Records, in offsets of that copy, the first byte of every
// restart interval (the byte after each RSTn marker) plus one final entry = end of data + 2, so
// interval j spans [seg[j], seg[j+1] - 2).  Lanes take 16-byte slices; positions come from a
// warp prefix sum of the bytes each slice keeps.
// ---------------------------------------------------------------------------------------
struct ScanList { int32_t n; int32_t s[64]; };      // the scans one launch covers

__global__ void __launch_bounds__(256) unstuff_index_kernel(Params P, ScanList sl, int img0, int nimg) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= sl.n * nimg) return;
    const int img = (int)P.order[img0 + warp % nimg];      // img0, nimg: a run of the processing order
    const ScanDesc sd = P.scans[sl.s[warp / nimg] * P.N + img];
    uint32_t* seg = P.seg_start + sd.seg_base;
    const uint32_t a = sd.data_off, b = sd.data_end;
    if (lane == 0) seg[0] = a;
    uint32_t found = 0;      // markers seen so far (warp uniform)
    uint32_t kept = 0;       // bytes written so far (warp uniform)
    // the next tile's 16 bytes are loaded while the current tile is processed; the byte before
    // and the byte after a lane's slice come from its neighbours by shuffle
    const uint4 zero4 = make_uint4(0, 0, 0, 0);
    uint4 ahead = zero4;
    {
        const uint32_t p = (a & ~15u) + 16u * lane;
        if (p < b) ahead = __ldg(reinterpret_cast<const uint4*>(P.rec + p));   // chunks are padded to 16 bytes
    }
    uint32_t carry = 0;      // last byte of the previous tile
    __shared__ __align__(16) uint8_t s_stage[8][528];
    uint8_t* stage = s_stage[threadIdx.x >> 5];
    uint32_t* out32 = reinterpret_cast<uint32_t*>(P.ubuf);
    uint32_t gpos = a & ~3u;                 // position in the copy of stage[0]
    uint32_t pend = a & 3u;                  // bytes already staged in front of the next tile's
    if (lane < 4) stage[lane] = 0;
    __syncwarp();
    for (uint32_t p0 = a & ~15u; p0 < b; p0 += 512) {
        const uint32_t p = p0 + 16u * lane;
        const uint4 v = ahead;
        ahead = zero4;
        if (p + 512 < b) ahead = __ldg(reinterpret_cast<const uint4*>(P.rec + p + 512));
        const uint32_t first_next_tile = __shfl_sync(0xffffffffu, ahead.x & 255u, 0);
        uint32_t nxt = __shfl_down_sync(0xffffffffu, v.x & 255u, 1);
        if (lane == 31) nxt = first_next_tile;
        uint32_t prev = __shfl_up_sync(0xffffffffu, v.w >> 24, 1);
        if (lane == 0) prev = carry;
        carry = __shfl_sync(0xffffffffu, v.w >> 24, 31);
        const uint32_t w[5] = {v.x, v.y, v.z, v.w, nxt};
        uint32_t keep = 0, mark = 0;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            const uint32_t c0 = (w[j >> 2] >> (8 * (j & 3))) & 255u;
            const uint32_t c1 = (w[(j + 1) >> 2] >> (8 * ((j + 1) & 3))) & 255u;
            const uint32_t cp = j ? (w[(j - 1) >> 2] >> (8 * ((j - 1) & 3))) & 255u : prev;
            const uint32_t q = p + j;
            const bool in = q >= a && q < b;
            if (in && !(c0 == 0u && cp == 0xFFu && q > a)) keep |= 1u << j;
            if (in && q + 1 < b && c0 == 0xFFu && (c1 & 0xF8u) == 0xD0u) mark |= 1u << j;
        }
        // exclusive prefix sums over lanes of kept bytes and of markers
        uint32_t kc = __popc(keep), mc = __popc(mark), kin = kc, min_ = mc;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t ok = __shfl_up_sync(0xffffffffu, kin, d), om = __shfl_up_sync(0xffffffffu, min_, d);
            if (lane >= d) { kin += ok; min_ += om; }
        }
        // kept bytes go to the warp's staging row (after the bytes left over from the last tile),
        // from there to the copy as whole byte-reversed words
        const uint32_t obase = a + kept + kin - kc;
        const uint32_t sbase = pend + kin - kc;
        uint32_t ord = found + min_ - mc;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            if ((keep >> j) & 1u) {
                const uint32_t off = __popc(keep & ((1u << j) - 1u));
                stage[sbase + off] = (uint8_t)((w[j >> 2] >> (8 * (j & 3))) & 255u);
                if ((mark >> j) & 1u) {
                    ++ord;
                    if (ord < sd.nseg) seg[ord] = obase + off + 2;
                }
            }
        }
        const uint32_t tile_kept = __shfl_sync(0xffffffffu, kin, 31);
        __syncwarp();
        const uint32_t total = pend + tile_kept, nwords = total >> 2;
        for (uint32_t i = lane; i < nwords; i += 32)
            out32[(gpos >> 2) + i] = __byte_perm(reinterpret_cast<const uint32_t*>(stage)[i], 0, 0x0123);
        __syncwarp();
        const uint32_t left = total & 3u;
        uint32_t lb = 0;
        if (lane < left) lb = stage[4 * nwords + lane];
        __syncwarp();
        if (lane < left) stage[lane] = (uint8_t)lb;
        __syncwarp();
        gpos += 4 * nwords;
        pend = left;
        kept += tile_kept;
        found += __shfl_sync(0xffffffffu, min_, 31);
    }
    if (pend && lane == 0) {                // the last, incomplete word (zero padded)
        uint32_t wlast = 0;
        for (uint32_t i = 0; i < pend; ++i) wlast |= (uint32_t)stage[i] << (8 * i);
        out32[gpos >> 2] = __byte_perm(wlast, 0, 0x0123);
    }
    if (lane == 0) {
        seg[sd.nseg] = a + kept + 2;
        if (found != sd.nseg - 1) atomicMin(&P.status[img], kErrCorrupt);
    }
}

// ---------------------------------------------------------------------------------------
// One wave of scans.  Each warp takes one item; each lane one restart interval.
// ---------------------------------------------------------------------------------------
struct Geometry {
    uint32_t mx, my;          // MCU grid
    uint32_t bw[3], ubw[3], ubh[3];
    uint64_t coff[3];         // first block of each component (global block index)
    uint64_t loff[3];         // first block of each component counted inside its component
};

__device__ __forceinline__ Geometry make_geometry(const ImgDesc& im, const Params& P) {
    Geometry g;
    const uint32_t hs = (uint32_t)P.hs, vs = (uint32_t)P.vs, ny = hs * vs;      // luminance blocks per MCU
    g.mx = im.mx; g.my = im.my;
    g.bw[0] = hs * im.mx; g.bw[1] = g.bw[2] = im.mx;
    g.ubw[0] = (im.W + 7) / 8; g.ubh[0] = (im.H + 7) / 8;
    uint32_t cw = (im.W + hs - 1) / hs, ch = (im.H + vs - 1) / vs;
    g.ubw[1] = g.ubw[2] = (cw + 7) / 8; g.ubh[1] = g.ubh[2] = (ch + 7) / 8;
    g.coff[0] = im.blk_base;
    g.coff[1] = im.blk_base + (uint64_t)ny * im.mx * im.my;
    g.coff[2] = g.coff[1] + (uint64_t)im.mx * im.my;
    const uint64_t mcus_before = im.blk_base / (ny + (P.nc == 3 ? 2u : 0u));   // every image holds the same blocks per MCU
    g.loff[0] = ny * mcus_before; g.loff[1] = g.loff[2] = mcus_before;
    return g;
}

// Block number (in the planes) of block j of MCU (mrow, mcol) in an interleaved scan: the luminance
// blocks of the MCU row by row, then Cb, then Cr.  *comp = its component.
__device__ __forceinline__ uint64_t mcu_block(const Geometry& g, const Params& P, uint32_t mrow, uint32_t mcol, int j, int* comp) {
    const int ny = P.hs * P.vs;
    if (j < ny) {
        const uint32_t r = (uint32_t)j >> (P.hs - 1), c = (uint32_t)j & (uint32_t)(P.hs - 1);
        *comp = 0;
        return g.coff[0] + (uint64_t)((uint32_t)P.vs * mrow + r) * g.bw[0] + (uint32_t)P.hs * mcol + c;
    }
    const int cc = j - ny + 1;
    *comp = cc;
    return g.coff[cc] + (uint64_t)mrow * g.bw[cc] + mcol;
}

__device__ __forceinline__ uint64_t low_mask(int p) { return p >= 64 ? ~0ull : ((1ull << p) - 1ull); }

// position of the (r+1)-th set bit of z, or 64 if z has fewer: a fixed five-step search on
// population counts, so lanes with different r stay converged
__device__ __forceinline__ int select_bit(uint64_t z, int r) {
    const uint32_t lo = (uint32_t)z, hi = (uint32_t)(z >> 32);
    int c = __popc(lo), base = 0;
    uint32_t x = lo;
    if (r >= c) { r -= c; x = hi; base = 32; }
    const bool none = r >= __popc(x);
    c = __popc(x & 0xFFFFu); if (r >= c) { r -= c; x >>= 16; base += 16; }
    c = __popc(x & 0xFFu);   if (r >= c) { r -= c; x >>= 8;  base += 8; }
    c = __popc(x & 0xFu);    if (r >= c) { r -= c; x >>= 4;  base += 4; }
    c = __popc(x & 0x3u);    if (r >= c) { r -= c; x >>= 2;  base += 2; }
    if (r >= (int)(x & 1u)) base += 1;
    return none ? 64 : base;
}

constexpr int kDecodeSteps = 16;     // decode steps between two top-ups of the rings

// kRoi: restart intervals whose MCU rows lie wholly outside the MCU rows that the image's crop
// rectangle (P.roi) touches are not decoded (their blocks are never transformed).
template <bool kRoi>
__global__ void __launch_bounds__(32 * kEntropyWarps) entropy_kernel(Params P, uint32_t item_begin, uint32_t item_count) {
    __shared__ HuffTab tabs[kEntropyWarps][2];
    __shared__ uint32_t s_ring[kEntropyWarps][kRingWords][32];
    __shared__ uint64_t s_hq[kEntropyWarps][4][32];          // masks of the next blocks (AC refinement)
    const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t it = blockIdx.x * kEntropyWarps + wid;
    if (it >= item_count) return;                             // whole warp
    const Item item = P.items[item_begin + it];
    const ScanDesc sd0 = P.scans[item.si];
    const int s = item.si / P.N;
    const ScanScript sc = P.script[s];
    const bool dc = sc.Ss == 0;              // a DC first pass (DC refinement scans go to dc_refine_kernel)
    // tables: a DC scan may use two tables of one image; an AC item may span two images
    const bool two_images = item.next != 0;
    const uint32_t si1 = two_images ? item.next - 1u : item.si;
    // From here on no lane leaves before the warp does: lanes without work just stay `done`.
    bool done = (uint32_t)lane >= item.count;
    const uint32_t rem0 = sd0.nseg - item.seg0;               // restart intervals left in the first image
    const int which = (two_images && (uint32_t)lane >= rem0) ? 1 : 0;
    uint32_t seg = which ? (uint32_t)lane - rem0 : item.seg0 + lane;
    const ScanDesc sd = which ? P.scans[si1] : sd0;
    const int img = (int)((which ? si1 : item.si) % (uint32_t)P.N);
    if (seg >= sd.nseg) { done = true; seg = 0; }
    const ImgDesc im = P.imgs[img];
    const Geometry g = make_geometry(im, P);

    const bool inter = sc.ncomp > 1;
    const int c0 = sc.comp[0];
    const uint32_t mcu_w = inter ? g.mx : g.ubw[c0];
    const uint32_t mcu_h = inter ? g.my : g.ubh[c0];
    const uint32_t total = mcu_w * mcu_h;
    const uint32_t m0 = sd.ri ? seg * sd.ri : 0;
    const uint32_t m1 = sd.ri ? min(m0 + sd.ri, total) : total;
    const unsigned full = 0xffffffffu;
    if (kRoi) {
        if (!done && m1 > m0) {
            const CropRect rc = P.roi[img];
            const uint32_t mh = 8u * (uint32_t)P.vs;                       // pixel rows of an MCU row
            const uint32_t ph = (inter || c0 != 0) ? mh : 8u;              // pixel rows per MCU row of this scan
            const uint32_t lo = mh * (rc.y0 / mh), hi = mh * ((rc.y0 + rc.h + mh - 1u) / mh);
            const uint32_t r0 = m0 / mcu_w, r1 = (m1 - 1u) / mcu_w;
            if ((r1 + 1u) * ph <= lo || r0 * ph >= hi) done = true;
        }
        if (__all_sync(full, done)) return;                               // nothing of this item is wanted
    }
    build_hufftab(tabs[wid][0], P.rec + sd0.tab_off[0], lane);
    if (two_images) build_hufftab(tabs[wid][1], P.rec + P.scans[si1].tab_off[0], lane);
    else if (sd0.tab_off[1]) build_hufftab(tabs[wid][1], P.rec + sd0.tab_off[1], lane);
    const uint32_t* segtab = P.seg_start + sd.seg_base;
    uint32_t bstart = segtab[seg];
    uint32_t bend = segtab[seg + 1] - 2;
    bool bad = false;
    if (!done && (bstart < sd.data_off || bend > sd.data_end || bend < bstart)) {   // a missing marker left a hole
        bad = true; done = true;
    }
    if (done) { bstart = sd.data_off; bend = sd.data_off; }
    BitReader br;
    br.init(&s_ring[wid][0][lane], P.ubuf, bstart, bend);
    br.topup(!done);
    br.prime();
    const int Al = sc.Al, p1 = 1 << sc.Al;

    if (dc) {
        // ---- DC first pass: one block per step
        const int bpm = inter ? P.hs * P.vs + 2 : 1;       // blocks per MCU
        uint32_t m = m0, mrow = m0 / mcu_w, mcol = m0 % mcu_w;
        int j = 0;                                         // block inside the MCU: the luminance blocks, Cb, Cr
        int pred0 = 0, pred1 = 0, pred2 = 0;
        if (m >= m1) done = true;
        for (;;) {
            br.topup(!done);
            __syncwarp(full);
            if (__all_sync(full, done)) break;
#pragma unroll 1
            for (int t = 0; t < kDecodeSteps; ++t) {
                if (done || !br.ready()) continue;
                br.refill();
                const uint32_t win = br.top32();
                int ci = 0;
                uint64_t blk;
                if (inter) blk = mcu_block(g, P, mrow, mcol, j, &ci);
                else blk = g.coff[c0] + (uint64_t)mrow * g.bw[c0] + mcol;
                const int c = inter ? ci : c0;
                int16_t* dcv = P.head + blk * 8;
                {
                    const HuffTab& tab = tabs[wid][(sd.slots >> (2 * ci)) & 1u];
                    const uint32_t e = huff_lookup(tab, win);
                    const int len = (int)(e >> 8), sz = (int)(e & 255u);
                    if (e == 0 || sz > 15) { bad = true; done = true; continue; }
                    const int d = extend_bits(top_bits(win << len, sz), sz);
                    br.skip(len + sz);
                    const int pv = (c == 0 ? pred0 : (c == 1 ? pred1 : pred2)) + d;
                    if (c == 0) pred0 = pv; else if (c == 1) pred1 = pv; else pred2 = pv;
                    *dcv = (int16_t)(pv << Al);
                }
                if (++j == bpm) {
                    j = 0; ++m;
                    if (++mcol == mcu_w) { mcol = 0; ++mrow; }
                }
                if (br.overran()) { bad = true; done = true; }
                if (m >= m1) done = true;
            }
            __syncwarp(full);
        }
    } else {
        const HuffTab& tab = tabs[wid][which];
        const int c = c0, Ss = sc.Ss, Se = sc.Se;
        const ScanAux ax = P.saux[s];
        const uint32_t bw = g.bw[c];
        const uint32_t wrap = bw - mcu_w + 1;              // step of the block index at the end of a block row
        uint32_t m = m0, bcol = m0 % mcu_w;
        uint32_t bi = (m0 / mcu_w) * bw + bcol;            // block index inside the image's component
        uint32_t eobrun = 0;
        if (m >= m1) done = true;
        if (sc.Ah == 0) {
            // ---- AC first pass: one Huffman symbol per step
            uint64_t* maskp = P.aux + ax.base + g.loff[c];
            int16_t* plane = P.planes + g.coff[c] * 64;
            int16_t* headp = P.head + g.coff[c] * 8;
            uint64_t M = 0;
            int k = Ss;
            for (;;) {
                br.topup(!done);
                __syncwarp(full);
                if (__all_sync(full, done)) break;
#pragma unroll 1
                for (int t = 0; t < kDecodeSteps; ++t) {
                    if (done || !br.ready()) continue;
                    br.refill();
                    const uint32_t win = br.top32();
                    uint32_t e = tab.lut[win >> (32 - kLutBits)];
                    if (e == 0) e = huff_lookup(tab, win);
                    const int len = (int)(e >> 8), r = (int)(e >> 4) & 15, sz = (int)(e & 15u);
                    const bool is_coef = sz != 0, is_eob = sz == 0 && r < 15;
                    const int kk = k + r;                                  // position of the coefficient
                    const bool fail = e == 0 || (is_coef && kk > Se);
                    const int extra = is_coef ? sz : (is_eob ? r : 0);
                    const uint32_t xb = top_bits(win << len, extra);       // magnitude bits / run length bits
                    br.skip(len + extra);
                    if (is_coef && !fail) {
                        const int16_t val = (int16_t)(extend_bits(xb, sz) * p1);
                        if (kk < 8) headp[(uint64_t)bi * 8 + kk] = val;
                        else plane[(uint64_t)bi * 64 + kk] = val;
                        M |= 1ull << kk;
                    }
                    k = is_coef ? kk + 1 : (is_eob ? k : k + 16);
                    if (is_eob) eobrun = (1u << r) + xb - 1u;
                    const bool fin = is_eob || k > Se;
                    if (fail) { bad = true; done = true; continue; }
                    if (fin) {
                        if (M) maskp[bi] = M;
                        uint32_t adv = 1;
                        if (eobrun) {                      // the following blocks of the run are empty
                            const uint32_t more = min(eobrun, m1 - (m + 1));
                            eobrun -= more;
                            adv += more;
                        }
                        m += adv;
                        if (adv == 1) { if (++bcol == mcu_w) { bcol = 0; bi += wrap; } else ++bi; }
                        else { bcol = m % mcu_w; bi = (m / mcu_w) * bw + bcol; }
                        k = Ss; M = 0;
                    }
                    if (br.overran()) { bad = true; done = true; }
                    if (m >= m1) done = true;
                }
                __syncwarp(full);
            }
        } else {
            // ---- AC refinement: one Huffman symbol, or one block of an end-of-band run, per step.
            // Hs holds the already-non-zero positions of the band from the current position k on
            // (bit 0 = position k), rem the positions left.  Skipping r zero positions: the target
            // sits at distance t = r + (non-zero positions up to t), found by iterating from t = r;
            // the count reached is also the number of correction bits that follow the symbol.
            const uint64_t band = low_mask(Se + 1) & ~low_mask(Ss);
            const uint64_t* src0 = nullptr; const uint64_t* src1 = nullptr; const uint64_t* src2 = nullptr; const uint64_t* src3 = nullptr;
            uint32_t st0 = 0, st1 = 0, st2 = 0, st3 = 0;
            {
                const ScanAux x0 = P.saux[ax.src[0]];
                src0 = P.aux + x0.base + g.loff[c] * x0.stride; st0 = x0.stride;
                if (ax.nsrc > 1) { const ScanAux x = P.saux[ax.src[1]]; src1 = P.aux + x.base + g.loff[c] * x.stride; st1 = x.stride; }
                if (ax.nsrc > 2) { const ScanAux x = P.saux[ax.src[2]]; src2 = P.aux + x.base + g.loff[c] * x.stride; st2 = x.stride; }
                if (ax.nsrc > 3) { const ScanAux x = P.saux[ax.src[3]]; src3 = P.aux + x.base + g.loff[c] * x.stride; st3 = x.stride; }
            }
            uint64_t* outp = P.aux + ax.base + g.loff[c] * 4ull;
            uint64_t* hq = &s_hq[wid][0][lane];                       // slot j at hq[j * 32]
            uint32_t hm = m, hcol = bcol, hbi = bi;                    // fetch cursor of the mask queue
            uint64_t H = 0, Hs = 0, cstr = 0, Nw = 0, NS = 0;
            int k = Ss, cn = 0;
            uint32_t rem = 0;
            bool newblk = true;
            for (;;) {
                br.topup(!done);
                // masks of the next blocks, up to four ahead
                {
                    uint64_t h[4];
                    const int want = done ? 0 : (int)min(4u - (hm - m), m1 - hm);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        if (q < want) {
                            uint64_t v = src0[(uint64_t)hbi * st0];
                            if (src1) v |= src1[(uint64_t)hbi * st1];
                            if (src2) v |= src2[(uint64_t)hbi * st2];
                            if (src3) v |= src3[(uint64_t)hbi * st3];
                            h[q] = v & band;
                            hq[((hm + q) & 3u) * 32] = h[q];
                            if (++hcol == mcu_w) { hcol = 0; hbi += wrap; } else ++hbi;
                        }
                    }
                    hm += (uint32_t)max(want, 0);
                }
                __syncwarp(full);
                if (__all_sync(full, done)) break;
#pragma unroll 1
                for (int t = 0; t < kDecodeSteps; ++t) {
                    if (done || !br.ready() || m >= hm) continue;
                    if (newblk) {
                        H = hq[(m & 3u) * 32];
                        Hs = H >> Ss;
                        k = Ss; rem = (uint32_t)(Se - Ss + 1);
                        cstr = 0; Nw = 0; NS = 0; cn = 0;
                        newblk = false;
                    }
                    br.refill();
                    const uint32_t win = br.top32();
                    const bool run = eobrun > 0;                       // this block lies inside an end-of-band run
                    uint32_t e = tab.lut[win >> (32 - kLutBits)];
                    if (e == 0 && !run) e = huff_lookup(tab, win);
                    const int len = (int)(e >> 8), r = (int)(e >> 4) & 15, sz = (int)(e & 15u);
                    const bool is_new = !run && sz != 0;
                    const bool is_eob = !run && sz == 0 && r < 15;
                    bool fail = !run && (e == 0 || sz > 1);
                    const int extra = is_new ? 1 : (is_eob ? r : 0);
                    const uint32_t xbits = top_bits(win << len, extra);    // sign of a new coefficient / run length bits
                    br.skip(run ? 0 : len + extra);
                    if (is_eob) eobrun = (1u << r) + xbits;
                    bool beyond = run || is_eob;                       // the rest of the band is passed over
                    // three rounds of dist = r + (non-zero positions up to dist) settle all but rare
                    // cases; those (and targets past bit 31) take the general search
                    const uint32_t lo = (uint32_t)Hs;
                    const uint32_t ur = (uint32_t)r;
                    uint32_t dist, cnt;
                    {
                        const uint32_t c1 = __popc(lo & ((2u << ur) - 1u));                  // ur <= 15
                        const uint32_t t1 = ur + c1;                                          // <= 31
                        const uint32_t c2 = __popc(lo & ((2u << t1) - 1u));
                        const uint32_t t2 = min(ur + c2, 31u);
                        const uint32_t c3 = __popc(lo & ((2u << t2) - 1u));
                        dist = ur + c3; cnt = c3;
                        if (!beyond && (dist != ur + c2 || dist >= 32u) && dist < rem) {     // not settled
                            const int sel = select_bit(~Hs & low_mask((int)rem), r);
                            if (sel >= 64) dist = rem;
                            else { dist = (uint32_t)sel; cnt = (uint32_t)__popcll(Hs & low_mask(sel)); }
                        }
                    }
                    beyond = beyond || dist >= rem;
                    const int n = beyond ? __popcll(Hs) : (int)cnt;    // correction bits that follow
                    const uint32_t adv = beyond ? rem : dist + 1u;
                    fail = fail || cn + n > 64;
                    if (n > 32) {                                      // rare: more than a word of correction bits
                        br.refill();
                        uint64_t bits = br.top32();
                        br.skip(32);
                        br.refill();
                        bits = (bits << (n - 32)) | top_bits(br.top32(), n - 32);
                        br.skip(n - 32);
                        if (!fail) cstr |= bits << (64 - cn - n);
                    } else {
                        if (br.nbits < n) br.refill();
                        const uint64_t bits = top_bits(br.top32(), n);
                        br.skip(n);
                        if (!fail && n) cstr |= bits << (64 - cn - n);
                    }
                    cn += n;
                    if (fail) { bad = true; done = true; continue; }
                    {
                        const uint64_t bit = (uint64_t)(is_new && !beyond) << ((k + (int)dist) & 63);
                        Nw |= bit;
                        NS |= xbits ? bit : 0ull;
                    }
                    k += (int)adv;
                    rem -= adv;
                    Hs = adv >= 64u ? 0ull : Hs >> adv;
                    eobrun -= (run || is_eob) ? 1u : 0u;
                    fail = br.overran();
                    if (rem == 0) {                                    // block finished
                        uint64_t* o = outp + (uint64_t)bi * 4;
                        *reinterpret_cast<ulonglong2*>(o) = make_ulonglong2(H | Nw, cstr);
                        *reinterpret_cast<ulonglong2*>(o + 2) = make_ulonglong2(Nw, NS);
                        ++m;
                        if (++bcol == mcu_w) { bcol = 0; bi += wrap; } else ++bi;
                        // the next block's mask is usually queued already
                        newblk = m >= hm;
                        H = hq[(m & 3u) * 32];
                        Hs = H >> Ss;
                        k = Ss; rem = (uint32_t)(Se - Ss + 1);
                        cstr = 0; Nw = 0; NS = 0; cn = 0;
                    }
                    bad = bad || fail;
                    done = fail || m >= m1;
                }
                __syncwarp(full);
            }

        }
    }
    if (bad) atomicMin(&P.status[img], kErrCorrupt);
}

// ---------------------------------------------------------------------------------------
// Sequential (baseline) scans: one interleaved scan carries, block after block, the DC difference
// and then the AC coefficients up to an end-of-block symbol.  Same decomposition as above (one
// lane per restart interval, one Huffman symbol per step), four tables per warp (DC and AC,
// luminance and chrominance).  Coefficients go where the progressive first passes put them:
// zigzag positions 0..7 into the dense head plane, the rest into the block's line.
// ---------------------------------------------------------------------------------------
constexpr int kSeqWarps = 2;

template <bool kRoi>
__global__ void __launch_bounds__(32 * kSeqWarps) sequential_kernel(Params P, uint32_t item_begin, uint32_t item_count) {
    __shared__ HuffTab tabs[kSeqWarps][4];                    // DC 0, DC 1, AC 0, AC 1
    __shared__ uint32_t s_ring[kSeqWarps][kRingWords][32];
    const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t it = blockIdx.x * kSeqWarps + wid;
    if (it >= item_count) return;                             // whole warp
    const Item item = P.items[item_begin + it];
    const ScanDesc sd = P.scans[item.si];
    const int img = (int)(item.si % (uint32_t)P.N);
    bool done = (uint32_t)lane >= item.count;
    uint32_t seg = item.seg0 + lane;
    if (seg >= sd.nseg) { done = true; seg = 0; }
    const ImgDesc im = P.imgs[img];
    const Geometry g = make_geometry(im, P);
    const uint32_t mcu_w = g.mx, total = g.mx * g.my;
    const uint32_t m0 = sd.ri ? seg * sd.ri : 0;
    const uint32_t m1 = sd.ri ? min(m0 + sd.ri, total) : total;
    const unsigned full = 0xffffffffu;
    if (kRoi) {
        if (!done && m1 > m0) {
            const CropRect rc = P.roi[img];
            const uint32_t mh = 8u * (uint32_t)P.vs;                       // pixel rows of an MCU row
            const uint32_t lo = mh * (rc.y0 / mh), hi = mh * ((rc.y0 + rc.h + mh - 1u) / mh);
            const uint32_t r0 = m0 / mcu_w, r1 = (m1 - 1u) / mcu_w;
            if ((r1 + 1u) * mh <= lo || r0 * mh >= hi) done = true;
        }
        if (__all_sync(full, done)) return;
    }
    build_hufftab(tabs[wid][0], P.rec + sd.tab_off[0], lane);
    if (sd.tab_off[1]) build_hufftab(tabs[wid][1], P.rec + sd.tab_off[1], lane);
    build_hufftab(tabs[wid][2], P.rec + sd.tab_ac[0], lane);
    if (sd.tab_ac[1]) build_hufftab(tabs[wid][3], P.rec + sd.tab_ac[1], lane);
    const uint32_t* segtab = P.seg_start + sd.seg_base;
    uint32_t bstart = segtab[seg];
    uint32_t bend = segtab[seg + 1] - 2;
    bool bad = false;
    if (!done && (bstart < sd.data_off || bend > sd.data_end || bend < bstart)) { bad = true; done = true; }
    if (done) { bstart = sd.data_off; bend = sd.data_off; }
    BitReader br;
    br.init(&s_ring[wid][0][lane], P.ubuf, bstart, bend);
    br.topup(!done);
    br.prime();

    uint32_t m = m0, mrow = m0 / mcu_w, mcol = m0 % mcu_w;
    const int bpm = P.nc == 3 ? P.hs * P.vs + 2 : 1;      // blocks per MCU (a lone component: one block, no padding)
    int j = 0;                                            // block inside the MCU: the luminance blocks, Cb, Cr
    int k = 0;                                            // 0: the block's DC symbol comes next
    int pred0 = 0, pred1 = 0, pred2 = 0;
    if (m >= m1) done = true;
    for (;;) {
        br.topup(!done);
        __syncwarp(full);
        if (__all_sync(full, done)) break;
#pragma unroll 1
        for (int t = 0; t < kDecodeSteps; ++t) {
            if (done || !br.ready()) continue;
            br.refill();
            const uint32_t win = br.top32();
            int c = 0;
            const uint64_t blk = P.nc == 3 ? mcu_block(g, P, mrow, mcol, j, &c) : g.coff[0] + (uint64_t)mrow * g.bw[0] + mcol;
            const bool is_dc = k == 0;
            const int ti = is_dc ? (int)((sd.slots >> (2 * c)) & 1u) : 2 + (int)((sd.slots_ac >> (2 * c)) & 1u);
            const HuffTab& tab = tabs[wid][ti];
            uint32_t e = tab.lut[win >> (32 - kLutBits)];
            if (e == 0) e = huff_lookup(tab, win);
            const int len = (int)(e >> 8), r = is_dc ? 0 : (int)(e >> 4) & 15, sz = is_dc ? (int)(e & 255u) : (int)(e & 15u);
            const bool is_coef = sz != 0, is_zrl = !is_dc && sz == 0 && r == 15, is_eob = !is_dc && sz == 0 && r == 0;
            const int kk = k + r;
            const bool fail = e == 0 || sz > 15 || (!is_dc && !is_coef && !is_zrl && !is_eob) || (is_coef && kk > 63);
            if (fail) { bad = true; done = true; continue; }
            const int extra = is_coef ? sz : 0;
            const int v = extend_bits(top_bits(win << len, extra), extra);
            br.skip(len + extra);
            if (is_dc) {
                const int pv = (c == 0 ? pred0 : (c == 1 ? pred1 : pred2)) + v;
                if (c == 0) pred0 = pv; else if (c == 1) pred1 = pv; else pred2 = pv;
                P.head[blk * 8] = (int16_t)pv;
                k = 1;
            } else if (is_coef) {
                if (kk < 8) P.head[blk * 8 + kk] = (int16_t)v;
                else P.planes[blk * 64 + kk] = (int16_t)v;
                k = kk + 1;
            } else if (is_zrl) {
                k += 16;
            }
            if (is_eob || k > 63) {                       // block finished
                k = 0;
                if (++j == bpm) {
                    j = 0; ++m;
                    if (++mcol == mcu_w) { mcol = 0; ++mrow; }
                }
            }
            if (br.overran()) { bad = true; done = true; }
            if (m >= m1) done = true;
        }
        __syncwarp(full);
    }
    if (bad) atomicMin(&P.status[img], kErrCorrupt);
}

}  // namespace pcr
