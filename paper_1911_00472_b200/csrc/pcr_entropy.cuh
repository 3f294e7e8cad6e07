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
// new positions, their signs} as side data.  finalize_kernel then updates the planes in place,
// one lane per coefficient pair, fully coalesced.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "pcr_types.h"

namespace pcr {

constexpr int kErrCorrupt = -3;

constexpr int kLutBits = 11;
constexpr int kEntropyWarps = 4;

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
    const uint32_t nvals = min(p, 256u);
    for (uint32_t j = lane; j < nvals; j += 32) t.vals[j] = dht[16 + j];
    uint32_t* lw = reinterpret_cast<uint32_t*>(t.lut);
    for (int e = lane; e < (1 << kLutBits) / 2; e += 32) lw[e] = 0;
    __syncwarp();
    // every symbol with a short code fills its 2^(kLutBits - length) entries, all lanes together
    uint32_t j = 0;
    for (int l = 1; l <= kLutBits; ++l) {
        const uint32_t c = t.cnt[l], f = t.first[l], span = 1u << (kLutBits - l);
        for (uint32_t i = 0; i < c && j < nvals; ++i, ++j) {
            const uint32_t base = (f + i) << (kLutBits - l);
            const uint16_t entry = (uint16_t)(((uint32_t)l << 8) | t.vals[j]);
            if (base + span <= (1u << kLutBits))
                for (uint32_t e = lane; e < span; e += 32) t.lut[base + e] = entry;
        }
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
    uint64_t loff[3];         // first block of each component counted inside its component
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
    const uint64_t mcus_before = im.blk_base / 6;      // every image holds 6 blocks per MCU
    g.loff[0] = 4 * mcus_before; g.loff[1] = g.loff[2] = mcus_before;
    return g;
}

__device__ __forceinline__ uint64_t low_mask(int p) { return p >= 64 ? ~0ull : ((1ull << p) - 1ull); }

__global__ void __launch_bounds__(32 * kEntropyWarps) entropy_kernel(Params P, uint32_t item_begin, uint32_t item_count) {
    __shared__ HuffTab tabs[kEntropyWarps][2];
    const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t it = blockIdx.x * kEntropyWarps + wid;
    if (it >= item_count) return;
    const Item item = P.items[item_begin + it];
    const ScanDesc sd = P.scans[item.si];
    const int s = item.si / P.N, img = item.si % P.N;
    const ScanScript sc = P.script[s];
    const ImgDesc im = P.imgs[img];
    const Geometry g = make_geometry(im);
    const bool dc = sc.Ss == 0;
    const bool huff = !(dc && sc.Ah != 0);
    if (huff) {
        build_hufftab(tabs[wid][0], P.rec + sd.tab_off[0], lane);
        if (sd.tab_off[1]) build_hufftab(tabs[wid][1], P.rec + sd.tab_off[1], lane);
    }
    const uint32_t seg = item.seg0 + lane;
    if ((uint32_t)lane >= item.count || seg >= sd.nseg) return;

    const bool inter = sc.ncomp > 1;
    const int c0 = sc.comp[0];
    const uint32_t mcu_w = inter ? g.mx : g.ubw[c0];
    const uint32_t mcu_h = inter ? g.my : g.ubh[c0];
    const uint32_t total = mcu_w * mcu_h;
    const uint32_t m0 = sd.ri ? seg * sd.ri : 0;
    const uint32_t m1 = sd.ri ? min(m0 + sd.ri, total) : total;
    const uint32_t* segtab = P.seg_start + sd.seg_base;
    const uint32_t bstart = segtab[seg];
    const uint32_t bend = (seg + 1 < sd.nseg) ? segtab[seg + 1] - 2 : sd.data_end;
    if (bstart < sd.data_off || bend > sd.data_end || bend < bstart) {   // a missing marker left a hole
        atomicMin(&P.status[img], kErrCorrupt);
        return;
    }
    BitReader br;
    br.init(P.rec, bstart, bend);
    bool bad = false;
    const int Al = sc.Al, p1 = 1 << sc.Al;

    if (dc) {
        // DC scans: every lane walks the same MCU structure, so the loop nest stays converged.
        uint32_t mrow = m0 / mcu_w, mcol = m0 % mcu_w;
        int pred0 = 0, pred1 = 0, pred2 = 0;
        for (uint32_t m = m0; m < m1 && !bad; ++m) {
            for (int ci = 0; ci < sc.ncomp; ++ci) {
                const int c = sc.comp[ci];
                const int hv = (inter && c == 0) ? 2 : 1;
                const HuffTab& tab = tabs[wid][(sd.slots >> (2 * ci)) & 1u];
                for (int sub = 0; sub < hv * hv; ++sub) {
                    const uint64_t blk = g.coff[c] + (uint64_t)(mrow * hv + (sub >> (hv - 1))) * g.bw[c] + mcol * hv + (sub & (hv - 1));
                    int16_t* cf = P.planes + blk * 64;
                    br.refill();
                    if (sc.Ah == 0) {
                        const int sz = huff_decode(tab, br, bad);
                        if (sz > 15) bad = true;
                        if (bad) break;
                        const int d = extend_bits(br.take(sz), sz);
                        int pv = (c == 0 ? pred0 : (c == 1 ? pred1 : pred2)) + d;
                        if (c == 0) pred0 = pv; else if (c == 1) pred1 = pv; else pred2 = pv;
                        cf[0] = (int16_t)(pv << Al);
                    } else {
                        if (br.take(1)) cf[0] = (int16_t)(cf[0] | p1);
                    }
                }
                if (bad) break;
            }
            if (++mcol == mcu_w) { mcol = 0; ++mrow; }
        }
    } else {
        const HuffTab& tab = tabs[wid][0];
        const int c = c0, Ss = sc.Ss, Se = sc.Se;
        const ScanAux ax = P.saux[s];
        const uint32_t bw = g.bw[c];
        uint32_t m = m0, brow = m0 / mcu_w, bcol = m0 % mcu_w;
        uint32_t eobrun = 0;
        int k = Ss;
        if (sc.Ah == 0) {
            // ---- AC first pass: one Huffman symbol per iteration
            uint64_t* maskp = P.aux + ax.base + g.loff[c];
            uint64_t M = 0;
            while (m < m1 && !bad) {
                br.refill();
                const int rs = huff_decode(tab, br, bad);
                if (bad) break;
                const int r = rs >> 4, sz = rs & 15;
                bool done;
                if (sz) {
                    k += r;
                    if (k > Se) { bad = true; break; }
                    const int v = extend_bits(br.take(sz), sz) * p1;
                    P.planes[(g.coff[c] + (uint64_t)brow * bw + bcol) * 64 + k] = (int16_t)v;
                    M |= 1ull << k;
                    ++k;
                    done = k > Se;
                } else if (r == 15) {
                    k += 16;
                    done = k > Se;
                } else {
                    eobrun = (1u << r) + (r ? br.take(r) : 0u) - 1u;
                    done = true;
                }
                if (done) {
                    if (M) maskp[(uint64_t)brow * bw + bcol] = M;
                    uint32_t adv = 1;
                    if (eobrun) {                      // the following blocks of the run are empty
                        const uint32_t extra = min(eobrun, m1 - (m + 1));
                        eobrun -= extra;
                        adv += extra;
                    }
                    m += adv;
                    if (adv == 1) { if (++bcol == mcu_w) { bcol = 0; ++brow; } }
                    else { brow = m / mcu_w; bcol = m % mcu_w; }
                    k = Ss; M = 0;
                }
            }
        } else {
            // ---- AC refinement: one Huffman symbol, or one block of an end-of-band run, per iteration
            const uint64_t band = low_mask(Se + 1) & ~low_mask(Ss);
            const uint64_t* srcp[4];
            uint32_t srcs[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const ScanAux sx = P.saux[ax.src[i < ax.nsrc ? i : 0]];
                srcp[i] = P.aux + sx.base + (uint64_t)g.loff[c] * sx.stride;
                srcs[i] = sx.stride;
            }
            uint64_t* outp = P.aux + ax.base + g.loff[c] * 4ull;
            auto load_hist = [&](uint32_t row, uint32_t col) -> uint64_t {
                const uint64_t bi = (uint64_t)row * bw + col;
                uint64_t h = srcp[0][bi * srcs[0]];
                if (ax.nsrc > 1) h |= srcp[1][bi * srcs[1]];
                if (ax.nsrc > 2) h |= srcp[2][bi * srcs[2]];
                if (ax.nsrc > 3) h |= srcp[3][bi * srcs[3]];
                return h & band;
            };
            uint64_t H = load_hist(brow, bcol);
            uint32_t nrow = brow, ncol = bcol + 1;
            if (ncol == mcu_w) { ncol = 0; ++nrow; }
            uint64_t Hn = (m + 1 < m1) ? load_hist(nrow, ncol) : 0ull;      // the next block's mask is already in flight
            uint64_t cstr = 0, Nw = 0, NS = 0;
            int cn = 0;
            while (m < m1 && !bad) {
                bool eob = eobrun > 0;
                int r = 0, sz = 0;
                uint32_t sign = 0;
                if (!eob) {
                    br.refill();
                    const int rs = huff_decode(tab, br, bad);
                    if (bad) break;
                    r = rs >> 4; sz = rs & 15;
                    if (sz) {
                        if (sz != 1) { bad = true; break; }
                        sign = br.take(1);
                    } else if (r < 15) {
                        eobrun = (1u << r) + (r ? br.take(r) : 0u);
                        eob = true;
                    }
                }
                const uint64_t from = ~0ull << k;                      // k <= Se <= 63 here
                int pos = Se + 1;
                if (!eob) {
                    uint64_t Z = ~H & band & from;                     // zero-valued positions still ahead
                    for (; r > 0 && Z; --r) Z &= Z - 1;                // pass over r of them
                    if (Z) pos = __ffsll((long long)Z) - 1;
                }
                const uint64_t hist = H & from & low_mask(pos);        // non-zero positions passed: one correction bit each
                const int n = __popcll(hist);
                if (n) {
                    if (cn + n > 64) { bad = true; break; }
                    br.refill();
                    uint64_t bits = br.take(min(n, 32));
                    if (n > 32) { br.refill(); bits = (bits << (n - 32)) | br.take(n - 32); }
                    cstr |= bits << (64 - cn - n);
                    cn += n;
                }
                if (sz && pos <= Se) { Nw |= 1ull << pos; NS |= (uint64_t)sign << pos; }
                k = pos + 1;
                if (eob) --eobrun;
                if (k > Se) {                                          // block finished
                    uint64_t* o = outp + ((uint64_t)brow * bw + bcol) * 4;
                    *reinterpret_cast<ulonglong2*>(o) = make_ulonglong2(H | Nw, cstr);
                    *reinterpret_cast<ulonglong2*>(o + 2) = make_ulonglong2(Nw, NS);
                    ++m;
                    brow = nrow; bcol = ncol;
                    H = Hn;
                    if (++ncol == mcu_w) { ncol = 0; ++nrow; }
                    if (m + 1 < m1) Hn = load_hist(nrow, ncol);
                    k = Ss; cstr = 0; Nw = 0; NS = 0; cn = 0;
                }
            }
        }
    }
    if (bad || br.overran()) atomicMin(&P.status[img], kErrCorrupt);
}

// ---------------------------------------------------------------------------------------
// Fold the side data of the AC refinement scans into the coefficient planes, in scan order.
// One thread per block; the work is proportional to the coefficients that actually change:
// the thread walks the set bits of the "already non-zero" mask while correction bits equal to 1
// remain (a correction moves the coefficient away from zero by 2^Al if its bit Al is still
// clear), then the set bits of the "newly non-zero" mask (value +-2^Al).
// ---------------------------------------------------------------------------------------
constexpr int kFinalizeThreads = 192;      // four units of 48 blocks

__global__ void __launch_bounds__(kFinalizeThreads) finalize_kernel(Params P, FinalizeList fl, uint32_t n_units) {
    const uint32_t t = blockIdx.x * kFinalizeThreads + threadIdx.x;
    const uint32_t unit = t / 48;
    const int j = (int)(t % 48);
    if (unit >= n_units) return;
    const Unit un = P.units[unit];
    const ImgDesc im = P.imgs[un.img];
    const int nm = min(8, (int)im.mx - (int)un.mcol0);
    const uint64_t mcus_before = im.blk_base / 6;
    // same block order as the pixel kernel: Y row 0 (16), Y row 1 (16), Cb (8), Cr (8)
    int c;
    uint64_t local, blk;
    if (j < 32) {
        const int r = j >> 4, col = j & 15;
        if (col >= 2 * nm) return;
        c = 0;
        local = (uint64_t)(2 * un.mrow + r) * (2 * im.mx) + 2 * un.mcol0 + col;
        blk = im.blk_base + local;
        local += 4 * mcus_before;
    } else {
        const int col = (j - 32) & 7;
        if (col >= nm) return;
        c = 1 + ((j - 32) >> 3);
        local = (uint64_t)un.mrow * im.mx + un.mcol0 + col;
        blk = im.blk_base + (c == 1 ? 4ull : 5ull) * im.mx * im.my + local;
        local += mcus_before;
    }
    int16_t* cf = P.planes + blk * 64;
    for (int i = 0; i < fl.n[c]; ++i) {
        const int s = fl.scan[c][i];
        const int p1 = fl.p1[c][i];
        const ulonglong2* o = reinterpret_cast<const ulonglong2*>(P.aux + fl.base[c][i] + local * 4);
        const ulonglong2 a = __ldg(o), b = __ldg(o + 1);       // {mask, corrections}, {new, signs}
        (void)s;
        uint64_t h = a.x & ~b.x, cc = a.y;
        while (cc) {
            const int pos = __ffsll((long long)h) - 1;
            if (pos < 0) break;
            h &= h - 1;
            if (cc >> 63) {
                const int v = cf[pos];
                if ((v & p1) == 0) cf[pos] = (int16_t)(v >= 0 ? v + p1 : v - p1);
            }
            cc <<= 1;
        }
        uint64_t nw = b.x;
        while (nw) {
            const int pos = __ffsll((long long)nw) - 1;
            nw &= nw - 1;
            cf[pos] = (int16_t)(((b.y >> pos) & 1ull) ? p1 : -p1);
        }
    }
}

}  // namespace pcr
