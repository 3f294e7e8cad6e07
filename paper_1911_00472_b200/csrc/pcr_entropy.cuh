// Entropy stage of the PCR decoder: restart-interval index and progressive Huffman decode
// of one wave of scans into the int16 coefficient planes.
//
// Parallel decomposition: one LANE per restart interval.  A warp takes up to 32 consecutive
// restart intervals of one (scan, image) pair, so its lanes share the scan's Huffman tables
// (held as lookup tables in shared memory) and run the same scan kind in lock step.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "pcr_types.h"

namespace pcr {

constexpr int kErrCorrupt = -3;

constexpr int kLutBits = 9;
constexpr int kEntropyWarps = 8;

// Decoder tables of one Huffman table: a direct lookup on the next kLutBits bits for short
// codes, and the canonical first-code / count / index triple per length for the rest.
struct HuffTab {
    uint16_t lut[1 << kLutBits];  // (length << 8) | symbol, 0 = longer than kLutBits (or undefined)
    uint32_t first[17];
    uint16_t cnt[17];
    uint16_t idx[17];
    uint8_t vals[256];
};

__device__ __forceinline__ void build_hufftab(HuffTab& t, const uint8_t* __restrict__ dht, int lane) {
    // dht: 16 length counts, then the symbol values in code order
    uint32_t code = 0, p = 0;
    for (int l = 1; l <= 16; ++l) {
        uint32_t c = dht[l - 1];
        if (lane == 0) { t.first[l] = code; t.cnt[l] = (uint16_t)c; t.idx[l] = (uint16_t)p; }
        code = (code + c) << 1;
        p += c;
    }
    if (p > 256) p = 256;
    for (uint32_t j = lane; j < p; j += 32) t.vals[j] = dht[16 + j];
    __syncwarp();
    for (int e = lane; e < (1 << kLutBits); e += 32) {
        uint32_t entry = 0;
        for (int l = 1; l <= kLutBits; ++l) {
            uint32_t d = ((uint32_t)e >> (kLutBits - l)) - t.first[l];
            if (d < t.cnt[l]) { entry = ((uint32_t)l << 8) | t.vals[t.idx[l] + d]; break; }
        }
        t.lut[e] = (uint16_t)entry;
    }
    __syncwarp();
}

// MSB-first bit reader over one restart interval, removing the stuffed zero byte after 0xFF.
// Past the end of the interval it feeds zero bits and counts them, so that over-reading is
// detected at the end instead of touching bytes of another interval.
struct BitReader {
    const uint8_t* base;
    uint32_t pos, end;
    uint64_t buf;     // left aligned
    int nbits;        // bits held in buf
    int fake;         // zero bits appended past the end

    __device__ __forceinline__ void init(const uint8_t* b, uint32_t p, uint32_t e) {
        base = b; pos = p; end = e; buf = 0; nbits = 0; fake = 0;
    }
    // afterwards at least 33 bits are held
    __device__ __forceinline__ void refill() {
        while (nbits <= 32) {
            if ((pos & 3u) == 0 && pos + 4 <= end) {
                uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(base + pos));
                uint32_t ff = ((w & 0x7F7F7F7Fu) + 0x01010101u) & w & 0x80808080u;
                if (ff == 0) {
                    buf |= (uint64_t)__byte_perm(w, 0, 0x0123) << (32 - nbits);
                    nbits += 32;
                    pos += 4;
                    continue;
                }
            }
            uint32_t b = 0;
            if (pos < end) {
                b = __ldg(base + pos);
                pos += (b == 0xFF) ? 2 : 1;
            } else {
                fake += 8;
            }
            buf |= (uint64_t)b << (56 - nbits);
            nbits += 8;
        }
    }
    __device__ __forceinline__ uint32_t peek16() const { return (uint32_t)(buf >> 48); }
    __device__ __forceinline__ void skip(int n) { buf <<= n; nbits -= n; }
    // n in 0..32, bits must be held
    __device__ __forceinline__ uint32_t take(int n) {
        uint32_t v = n ? (uint32_t)(buf >> (64 - n)) : 0u;
        skip(n);
        return v;
    }
    __device__ __forceinline__ bool overran() const { return nbits < fake; }
};

__device__ __forceinline__ int huff_decode(const HuffTab& t, BitReader& br, bool& bad) {
    uint32_t w = br.peek16();
    uint32_t e = t.lut[w >> (16 - kLutBits)];
    if (e) { br.skip((int)(e >> 8)); return (int)(e & 255u); }
    for (int l = kLutBits + 1; l <= 16; ++l) {
        uint32_t d = (w >> (16 - l)) - t.first[l];
        if (d < t.cnt[l]) { br.skip(l); return t.vals[t.idx[l] + d]; }
    }
    bad = true;
    return 0;
}

__device__ __forceinline__ int extend_bits(uint32_t v, int s) {
    // value of an s-bit magnitude field: the top bit clear means negative
    return s == 0 ? 0 : ((v >> (s - 1)) ? (int)v : (int)v - (1 << s) + 1);
}

// ---------------------------------------------------------------------------------------
// Restart-interval index: for every (scan < nscans, image), the first byte of each restart
// interval.  One warp per pair; markers found per 16-byte lane slice, ordinals by a warp
// prefix sum.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) seg_index_kernel(Params P, int nscans) {
    int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (warp >= nscans * P.N) return;
    const ScanDesc sd = P.scans[warp];
    int img = warp % P.N;
    uint32_t* seg = P.seg_start + sd.seg_base;
    if (lane == 0) seg[0] = sd.data_off;
    if (sd.nseg <= 1) return;
    uint32_t a = sd.data_off, b = sd.data_end;
    uint32_t found = 0;  // markers seen so far (warp uniform)
    for (uint32_t p0 = a & ~15u; p0 < b; p0 += 512) {
        uint32_t p = p0 + 16u * lane;
        uint4 v = make_uint4(0, 0, 0, 0);
        uint32_t nxt = 0;
        if (p < b) v = __ldg(reinterpret_cast<const uint4*>(P.rec + p));   // chunks are padded to 16 bytes
        if (p + 16 < b) nxt = __ldg(P.rec + p + 16);
        uint32_t w[5] = {v.x, v.y, v.z, v.w, nxt};
        uint32_t mask = 0;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            uint32_t c0 = (w[j >> 2] >> (8 * (j & 3))) & 255u;
            uint32_t c1 = (w[(j + 1) >> 2] >> (8 * ((j + 1) & 3))) & 255u;
            uint32_t q = p + j;
            if (c0 == 0xFFu && (c1 & 0xF8u) == 0xD0u && q >= a && q + 1 < b) mask |= 1u << j;
        }
        uint32_t cnt = __popc(mask), incl = cnt;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            uint32_t o = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += o;
        }
        uint32_t ord = found + incl - cnt;
        while (mask) {
            int j = __ffs(mask) - 1;
            mask &= mask - 1;
            ++ord;
            if (ord < sd.nseg) seg[ord] = p + j + 2;
        }
        found += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0 && found != sd.nseg - 1) atomicMin(&P.status[img], kErrCorrupt);
}

// ---------------------------------------------------------------------------------------
// One wave of scans.  Each warp takes one item; each lane one restart interval.
// ---------------------------------------------------------------------------------------
struct Geometry {
    uint32_t mx, my;          // MCU grid
    uint32_t bw[3], ubw[3], ubh[3];
    uint64_t coff[3];         // first block of each component (global block index)
};

__device__ __forceinline__ Geometry make_geometry(const ImgDesc& im) {
    Geometry g;
    g.mx = im.mx; g.my = im.my;
    g.bw[0] = 2 * im.mx; g.bw[1] = g.bw[2] = im.mx;
    g.ubw[0] = (im.W + 7) / 8; g.ubh[0] = (im.H + 7) / 8;
    uint32_t cw = (im.W + 1) / 2, ch = (im.H + 1) / 2;
    g.ubw[1] = g.ubw[2] = (cw + 7) / 8; g.ubh[1] = g.ubh[2] = (ch + 7) / 8;
    g.coff[0] = im.blk_base;
    g.coff[1] = im.blk_base + 4ull * im.mx * im.my;
    g.coff[2] = im.blk_base + 5ull * im.mx * im.my;
    return g;
}

__global__ void __launch_bounds__(32 * kEntropyWarps) entropy_kernel(Params P, uint32_t item_begin, uint32_t item_count) {
    __shared__ HuffTab tabs[kEntropyWarps][2];
    int wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint32_t it = blockIdx.x * kEntropyWarps + wid;
    if (it >= item_count) return;
    const Item item = P.items[item_begin + it];
    const ScanDesc sd = P.scans[item.si];
    int s = item.si / P.N, img = item.si % P.N;
    const ScanScript sc = P.script[s];
    const ImgDesc im = P.imgs[img];
    const Geometry g = make_geometry(im);
    const bool dc = sc.Ss == 0;
    const bool huff = !(dc && sc.Ah != 0);
    if (huff) {
        build_hufftab(tabs[wid][0], P.rec + sd.tab_off[0], lane);
        if (sd.tab_off[1]) build_hufftab(tabs[wid][1], P.rec + sd.tab_off[1], lane);
    }
    uint32_t seg = item.seg0 + lane;
    if (seg >= sd.nseg) return;

    const bool inter = sc.ncomp > 1;
    const int c0 = sc.comp[0];
    uint32_t mcu_w = inter ? g.mx : g.ubw[c0];
    uint32_t mcu_h = inter ? g.my : g.ubh[c0];
    uint32_t total = mcu_w * mcu_h;
    uint32_t m0 = sd.ri ? seg * sd.ri : 0;
    uint32_t m1 = sd.ri ? min(m0 + sd.ri, total) : total;
    const uint32_t* segtab = P.seg_start + sd.seg_base;
    uint32_t bstart = segtab[seg];
    uint32_t bend = (seg + 1 < sd.nseg) ? segtab[seg + 1] - 2 : sd.data_end;
    if (bstart < sd.data_off || bend > sd.data_end || bend < bstart) {   // a missing marker left a hole
        atomicMin(&P.status[img], kErrCorrupt);
        return;
    }
    BitReader br;
    br.init(P.rec, bstart, bend);
    bool bad = false;
    const int Al = sc.Al, p1 = 1 << sc.Al;
    uint32_t mrow = m0 / mcu_w, mcol = m0 % mcu_w;

    if (dc) {
        int pred[3] = {0, 0, 0};
        for (uint32_t m = m0; m < m1 && !bad; ++m) {
            for (int ci = 0; ci < sc.ncomp; ++ci) {
                int c = sc.comp[ci];
                int hv = (inter && c == 0) ? 2 : 1;
                const HuffTab& tab = tabs[wid][(sd.slots >> (2 * ci)) & 3u];
                for (int sub = 0; sub < hv * hv; ++sub) {
                    uint64_t blk = g.coff[c] + (uint64_t)(mrow * hv + (sub >> (hv - 1))) * g.bw[c] + mcol * hv + (sub & (hv - 1));
                    int16_t* cf = P.planes + blk * 64;
                    br.refill();
                    if (sc.Ah == 0) {
                        int sz = huff_decode(tab, br, bad);
                        if (sz > 15) bad = true;
                        if (bad) break;
                        int d = extend_bits(br.take(sz), sz);
                        pred[c] += d;
                        cf[0] = (int16_t)(pred[c] << Al);
                    } else {
                        if (br.take(1)) cf[0] = (int16_t)(cf[0] | p1);
                    }
                }
                if (bad) break;
            }
            if (++mcol == mcu_w) { mcol = 0; ++mrow; }
        }
    } else {
        const HuffTab& tab = tabs[wid][sd.slots & 3u];
        const int c = c0, Ss = sc.Ss, Se = sc.Se;
        uint32_t eobrun = 0;
        if (sc.Ah == 0) {
            uint32_t m = m0;
            while (m < m1 && !bad) {
                if (eobrun > 0) {                       // whole blocks inside an end-of-band run
                    uint32_t sk = min(eobrun, m1 - m);
                    eobrun -= sk; m += sk;
                    continue;
                }
                uint32_t brow = m / mcu_w, bcol = m % mcu_w;
                int16_t* cf = P.planes + (g.coff[c] + (uint64_t)brow * g.bw[c] + bcol) * 64;
                int k = Ss;
                while (k <= Se) {
                    br.refill();
                    int rs = huff_decode(tab, br, bad);
                    if (bad) break;
                    int r = rs >> 4, sz = rs & 15;
                    if (sz) {
                        k += r;
                        if (k > Se) { bad = true; break; }
                        cf[k] = (int16_t)(extend_bits(br.take(sz), sz) * p1);
                        ++k;
                    } else if (r == 15) {
                        k += 16;
                    } else {
                        eobrun = (1u << r) + (r ? br.take(r) : 0u) - 1u;
                        break;
                    }
                }
                ++m;
            }
        } else {
            for (uint32_t m = m0; m < m1 && !bad; ++m) {
                uint32_t brow = m / mcu_w, bcol = m % mcu_w;
                int16_t* cf = P.planes + (g.coff[c] + (uint64_t)brow * g.bw[c] + bcol) * 64;
                int k = Ss;
                if (eobrun == 0) {
                    while (k <= Se) {
                        br.refill();
                        int rs = huff_decode(tab, br, bad);
                        if (bad) break;
                        int r = rs >> 4, sz = rs & 15, newval = 0;
                        if (sz) {
                            if (sz != 1) { bad = true; break; }
                            newval = br.take(1) ? p1 : -p1;
                        } else if (r < 15) {
                            eobrun = (1u << r) + (r ? br.take(r) : 0u);
                            break;
                        }
                        while (k <= Se) {
                            int v = cf[k];
                            if (v != 0) {
                                br.refill();
                                if (br.take(1) && (v & p1) == 0) cf[k] = (int16_t)(v >= 0 ? v + p1 : v - p1);
                            } else {
                                if (r == 0) break;
                                --r;
                            }
                            ++k;
                        }
                        if (sz && k <= Se) cf[k] = (int16_t)newval;
                        ++k;
                    }
                }
                if (eobrun > 0 && !bad) {
                    for (; k <= Se; ++k) {
                        int v = cf[k];
                        if (v != 0) {
                            br.refill();
                            if (br.take(1) && (v & p1) == 0) cf[k] = (int16_t)(v >= 0 ? v + p1 : v - p1);
                        }
                    }
                    --eobrun;
                }
            }
        }
    }
    if (bad || br.overran()) atomicMin(&P.status[img], kErrCorrupt);
}

}  // namespace pcr
