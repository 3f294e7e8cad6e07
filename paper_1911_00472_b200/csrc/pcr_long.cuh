// Entropy stage for scans that are ONE long restart interval (records written without restart
// markers: one entropy-coded segment per image and scan), and the DC refinement scans of any record.
//
// A Huffman stream is a serial chain, so a whole scan on one lane takes tens of thousands of
// dependent steps.  These kernels shorten or remove that chain:
//
//  * dc_refine_kernel: a DC refinement scan carries exactly one raw bit per block, so after
//    unstuffing bit j of a restart interval is block j of the interval in scan order: one thread
//    per MCU, no chain at all.  Used for every record.
//  * first_pass_long_kernel: DC and AC first passes.  One small CTA per (scan, image); the segment is
//    cut into one subsequence of equal bit length per thread and every thread decodes its own.  A
//    thread that starts in the middle of the stream does not know where a code begins nor which
//    coefficient (or which block of the MCU) it is at; it starts anyway, and because Huffman streams
//    re-synchronise, its state at the end of its subsequence is often right.  The threads then hand
//    their end states on: a thread whose predecessor ended in a state other than the one it started
//    from decodes again from there; the rounds stop when nothing changes (thread 0 starts at the
//    true beginning, so after round r threads 0..r are exact).  A prefix sum of the blocks each
//    thread finished (and of the DC differences per component) gives every thread its first block
//    and its predictors, and a last pass decodes once more and writes.
//  * sequential_long_kernel: the same scheme for the one scan of a baseline JPEG.
//  * ac_refine_group_kernel: an AC refinement cannot be entered in the middle (how many correction
//    bits follow a symbol depends on which coefficients of the block are already non-zero, i.e. on
//    the block number).  A scan is one chain: one thread follows it with ordinary branches, a
//    helper warp fetches the bitstream into a shared-memory ring, prepares the masks of the next 32
//    blocks and turns the thread's symbol records into side data.  All chains of a record run in
//    one persistent launch that deals them to the SMs' schedulers evenly; the refinements of one
//    component run behind one another, block by block.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "pcr_entropy.cuh"
#include "pcr_types.h"

namespace pcr {

// ---------------------------------------------------------------------------------------
// DC refinement: thread per MCU of the scan.  grid = (chunks of MCUs, images of the run).
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) dc_refine_kernel(Params P, int s, uint32_t pos0) {
    const int img = (int)P.order[pos0 + blockIdx.y];
    const ScanDesc sd = P.scans[(size_t)s * P.N + img];
    const ScanScript sc = P.script[s];
    const ImgDesc im = P.imgs[img];
    const Geometry g = make_geometry(im, P);
    const bool inter = sc.ncomp > 1;
    const int c0 = sc.comp[0];
    const uint32_t mcu_w = inter ? g.mx : g.ubw[c0];
    const uint32_t mcu_h = inter ? g.my : g.ubh[c0];
    const uint32_t total = mcu_w * mcu_h;
    const uint32_t bpm = inter ? (uint32_t)(P.hs * P.vs + 2) : 1u;   // blocks (= bits) per MCU
    const uint32_t* segtab = P.seg_start + sd.seg_base;
    const uint32_t* words = reinterpret_cast<const uint32_t*>(P.ubuf);
    const int p1 = 1 << sc.Al;
    bool bad = false;
    for (uint32_t m = blockIdx.x * 256u + threadIdx.x; m < total; m += gridDim.x * 256u) {
        const uint32_t seg = sd.ri ? m / sd.ri : 0u;
        if (seg >= sd.nseg) { bad = true; continue; }
        const uint32_t m0 = seg * sd.ri;                       // 0 without restart markers
        const uint32_t bstart = segtab[seg], bend = segtab[seg + 1] - 2u;
        if (bstart < sd.data_off || bend > sd.data_end || bend < bstart) { bad = true; continue; }   // a missing marker left a hole
        const uint32_t bit = bpm * (m - m0);
        if (bit + bpm > 8u * (bend - bstart)) { bad = true; continue; }                             // the interval is too short
        const uint32_t p = 8u * (bstart & 3u) + bit;           // from the first bit of word bstart >> 2
        const uint32_t wi = (bstart >> 2) + (p >> 5);
        const uint32_t w0 = __ldg(words + wi), w1 = __ldg(words + wi + 1);   // the copy has spare bytes behind its end
        const uint32_t v = __funnelshift_l(w1, w0, p & 31u) >> (32u - bpm);  // the MCU's bits, first block in the top bit
        const uint32_t mrow = m / mcu_w, mcol = m - mrow * mcu_w;
#pragma unroll
        for (uint32_t j = 0; j < 6; ++j) {
            if (j >= bpm) break;
            if (!((v >> (bpm - 1u - j)) & 1u)) continue;
            uint64_t blk;
            int comp;
            if (!inter) blk = g.coff[c0] + (uint64_t)mrow * g.bw[c0] + mcol;
            else blk = mcu_block(g, P, mrow, mcol, (int)j, &comp);
            // coefficient 0 is the first int16 of the block's head entry; no other scan of the wave writes it
            int16_t* dcv = P.head + blk * 8;
            *dcv = (int16_t)(*dcv | p1);
        }
    }
    if (bad) atomicMin(&P.status[img], kErrCorrupt);
}

// ---------------------------------------------------------------------------------------
// Bit reader of one lane over the unstuffed big-endian words: a 64-bit window, the next word
// already requested while the current bits are consumed.  Positions are bits counted from the
// first bit of a base word.
// ---------------------------------------------------------------------------------------
struct WordReader {
    const uint32_t* w;     // base word
    uint32_t rd;           // index of the word held in `ahead`
    uint64_t buf;          // left-aligned window
    int nbits;
    uint32_t ahead;
    __device__ __forceinline__ void init(const uint32_t* base, uint32_t pos) {
        w = base;
        rd = pos >> 5;
        const uint32_t first = __ldg(w + rd) << (pos & 31u);
        buf = (uint64_t)first << 32;
        nbits = 32 - (int)(pos & 31u);
        ++rd;
        ahead = __ldg(w + rd);
    }
    __device__ __forceinline__ void refill() {                 // afterwards at least 33 bits are held
        if (nbits <= 32) {
            buf |= (uint64_t)ahead << (32 - nbits);
            nbits += 32;
            ++rd;
            ahead = __ldg(w + rd);
        }
    }
    __device__ __forceinline__ uint32_t top32() const { return (uint32_t)(buf >> 32); }
    __device__ __forceinline__ void skip(int n) { buf <<= n; nbits -= n; }
    __device__ __forceinline__ uint32_t pos() const { return rd * 32u - (uint32_t)nbits; }
};

#ifndef PCR_LONG_WARPS
#define PCR_LONG_WARPS 2
#endif
constexpr int kLongWarps = PCR_LONG_WARPS;   // warps per scan in first_pass_long_kernel: 32 subsequences each

// ---------------------------------------------------------------------------------------
// The search passes of first_pass_long_kernel (a thread decodes its subsequence only to learn in which
// state it ends and how many blocks it finishes) are the serial part of that kernel: when a stream
// does not re-synchronise (a stretch of equally long symbols, in which a shifted reading stays shifted)
// the true state moves on by one subsequence per round.  So they are kept short: a lookup table that
// already holds what the search needs of a symbol, and a reader of three words in registers.
// ---------------------------------------------------------------------------------------
struct GlobalBits {
    const uint32_t* w;     // base word (global memory; the neighbouring threads share its cache lines)
    uint32_t w0, w1, w2;   // the word the next bit lies in and the two after it
    uint32_t bits;         // position of the next bit, counted from the first bit of the base word
    __device__ __forceinline__ void init(const uint32_t* base, uint32_t pos) {
        w = base;
        bits = pos;
        const uint32_t i = pos >> 5;
        w0 = __ldg(w + i); w1 = __ldg(w + i + 1); w2 = __ldg(w + i + 2);
    }
    __device__ __forceinline__ uint32_t win() const { return __funnelshift_l(w1, w0, bits); }   // the next 32 bits (shift taken mod 32)
    __device__ __forceinline__ void skip(uint32_t n) {        // n < 32: at most one word further
        const uint32_t nb = bits + n;
        if ((nb ^ bits) >> 5) { w0 = w1; w1 = w2; w2 = __ldg(w + (nb >> 5) + 2); }
        bits = nb;
    }
};

// What the search of an AC first pass needs of a symbol (a HuffTab entry (length << 8) | (run << 4 | size)):
// bits 0..4 bits to skip (code and extra bits), 5..8 positions the symbol moves on minus one (run + 1 for
// a coefficient, 16 for sixteen zeros), 9 end of band, 10..13 its run-length exponent.
constexpr uint32_t kSearchEob = 0x200u;
__device__ __forceinline__ uint32_t ac_search_entry(uint32_t t) {
    if (t == 0) return 0;
    const uint32_t len = t >> 8, r = (t >> 4) & 15u, sz = t & 15u;
    if (sz) return (len + sz) | (r << 5);
    if (r == 15u) return len | (15u << 5);
    return (len + r) | kSearchEob | (r << 10);
}

// Search pass of an AC first pass: the symbols that START in [pos, pos_end), from zigzag position k.
// An undefined code is skipped by one bit and a coefficient beyond the band ends the block (the thread
// is then reading from a wrong entry point and only has to arrive somewhere).
__device__ __forceinline__ void ac_search_span(const HuffTab& tab, const uint16_t* slut, const uint32_t* base, uint32_t pos, int k,
                                               uint32_t pos_end, int Ss, int Se, uint32_t& pos_out, int& k_out, uint32_t& nblk) {
    GlobalBits B;
    B.init(base, pos);
    uint32_t nb = 0;
    while (B.bits < pos_end) {
        const uint32_t win = B.win();
        uint32_t e = slut[win >> (32 - kLutBits)];
        if (e == 0) {                                          // a code longer than the table's index, or none
            e = ac_search_entry(huff_lookup(tab, win));
            if (e == 0) { B.skip(1); continue; }
        }
        if (e & kSearchEob) {
            const uint32_t r = e >> 10;
            nb += r ? (1u << r) + ((win << ((e & 31u) - r)) >> (32u - r)) : 1u;
            k = Ss;
        } else {
            const int nk = k + (int)((e >> 5) & 15u) + 1;
            if (nk > Se) { ++nb; k = Ss; } else k = nk;
        }
        B.skip(e & 31u);
    }
    pos_out = B.bits;
    k_out = k;
    nblk = nb;
}

// Search pass of a DC first pass.  dlut: per table, (length << 4) | size of the codes of at most kLutBits
// bits; tbits: bit j = the table of the j-th block of an MCU; cpack: two bits per j = its component.
__device__ __forceinline__ void dc_search_span(const HuffTab* tabs2, const uint8_t* dlut, uint32_t tbits, uint32_t cpack, int bpm,
                                               const uint32_t* base, uint32_t pos, int j, uint32_t pos_end, uint32_t& pos_out,
                                               int& j_out, uint32_t& nblk, int& sum0, int& sum1, int& sum2) {
    GlobalBits B;
    B.init(base, pos);
    uint32_t nb = 0;
    int s0 = 0, s1 = 0, s2 = 0;
    while (B.bits < pos_end) {
        const uint32_t win = B.win();
        const uint32_t tsel = (tbits >> j) & 1u;
        const uint32_t e = dlut[(tsel << kLutBits) + (win >> (32 - kLutBits))];
        int len = (int)(e >> 4), sz = (int)(e & 15u);
        if (e == 0) {
            const uint32_t t = huff_lookup(tabs2[tsel], win);
            len = (int)(t >> 8); sz = (int)(t & 255u);
            if (t == 0 || sz > 15) { B.skip(1); continue; }
        }
        const int d = extend_bits(top_bits(win << len, sz), sz);
        const uint32_t c = (cpack >> (2 * j)) & 3u;
        s0 += c == 0u ? d : 0; s1 += c == 1u ? d : 0; s2 += c == 2u ? d : 0;
        B.skip((uint32_t)(len + sz));
        ++nb;
        if (++j == bpm) j = 0;
    }
    pos_out = B.bits;
    j_out = j;
    nblk = nb;
    sum0 = s0; sum1 = s1; sum2 = s2;
}

// What one lane needs to write the coefficients of an AC first pass.
struct AcWrite {
    int16_t* plane;        // the component's lines
    int16_t* headp;        // the component's head entries
    unsigned long long* maskp;   // the scan's non-zero masks, by block number inside the component
    uint32_t mcu_w, bw;    // blocks per row of the scan's (unpadded) grid / of the padded grid
    uint32_t m, m1;        // next block of the scan, one past its last
    int p1;
};

// Decodes the symbols of an AC first pass that START in [pos, pos_end), from zigzag position k of the
// current block.  Every step consumes at least one bit, so the loop ends.  Without kWrite (search
// for the true entry state) an undefined code is skipped by one bit and a coefficient beyond the
// band ends the block: the lane is then reading from a wrong entry point and only has to arrive
// somewhere.  With kWrite the entry state is the true one, such events mean a corrupt stream.
template <bool kWrite>
__device__ __forceinline__ void ac_first_span(const HuffTab& tab, const uint32_t* base, uint32_t pos, int k, uint32_t pos_end,
                                              int Ss, int Se, uint32_t& pos_out, int& k_out, uint32_t& nblk, AcWrite& W, bool& bad) {
    WordReader br;
    br.init(base, pos);
    uint32_t nb = 0;
    unsigned long long M = 0;
    uint32_t bcol = 0, bi = 0;
    if (kWrite) { bcol = W.m % W.mcu_w; bi = (W.m / W.mcu_w) * W.bw + bcol; }
    bool stop = kWrite && W.m >= W.m1;
    while (!stop && br.pos() < pos_end) {
        br.refill();
        const uint32_t win = br.top32();
        uint32_t e = tab.lut[win >> (32 - kLutBits)];
        if (e == 0) e = huff_lookup(tab, win);
        if (e == 0) {
            if (kWrite) { bad = true; break; }
            br.skip(1);
            continue;
        }
        const int len = (int)(e >> 8), r = (int)(e >> 4) & 15, sz = (int)(e & 15u);
        const bool is_coef = sz != 0, is_eob = sz == 0 && r < 15;
        const int kk = k + r;
        const bool over = is_coef && kk > Se;
        if (kWrite && over) { bad = true; break; }
        const int extra = is_coef ? sz : (is_eob ? r : 0);
        const uint32_t xb = top_bits(win << len, extra);
        br.skip(len + extra);
        if (kWrite && is_coef) {
            const int16_t val = (int16_t)(extend_bits(xb, sz) * W.p1);
            if (kk < 8) W.headp[(uint64_t)bi * 8 + kk] = val;
            else W.plane[(uint64_t)bi * 64 + kk] = val;
            M |= 1ull << kk;
        }
        k = is_coef ? kk + 1 : (is_eob ? k : k + 16);
        if (is_eob || over || k > Se) {                        // the block ends, an end-of-band run skips more
            const uint32_t adv = 1u + (is_eob ? (1u << r) + xb - 1u : 0u);
            nb += adv;
            k = Ss;
            if (kWrite) {
                if (M) atomicOr(W.maskp + bi, M);              // a block may be shared with the neighbouring lane
                M = 0;
                W.m += adv;
                if (W.m >= W.m1) stop = true;
                else if (adv == 1u) { if (++bcol == W.mcu_w) { bcol = 0; bi += W.bw - W.mcu_w + 1u; } else ++bi; }
                else { bcol = W.m % W.mcu_w; bi = (W.m / W.mcu_w) * W.bw + bcol; }
            }
        }
    }
    if (kWrite && M) atomicOr(W.maskp + bi, M);                // the part of a block that ends in the next lane's span
    pos_out = br.pos();
    k_out = k;
    nblk = nb;
}

// The same for a DC first pass: one symbol (size category, then that many difference bits) per block;
// j = the block's place in its MCU (Y00 Y01 Y10 Y11 Cb Cr, or always 0 in a one-component scan).
struct DcWrite {
    int16_t* head;
    uint64_t coff[3];
    uint32_t bw[3];
    uint32_t mcu_w;
    uint32_t hs, vs;       // luminance blocks per MCU
    uint32_t n, n1;        // next block of the scan in scan order, one past its last
    int pred[3];
    int Al;
};

template <bool kWrite>
__device__ __forceinline__ void dc_first_span(const HuffTab* tabs2, uint32_t slots, bool inter, int c0, const uint32_t* base,
                                              uint32_t pos, int j, uint32_t pos_end, uint32_t& pos_out, int& j_out, uint32_t& nblk,
                                              int& sum0, int& sum1, int& sum2, DcWrite& W, bool& bad) {
    WordReader br;
    br.init(base, pos);
    const int ny = (int)(W.hs * W.vs), bpm = inter ? ny + 2 : 1;
    uint32_t nb = 0;
    int s0 = 0, s1 = 0, s2 = 0;
    uint32_t mrow = 0, mcol = 0;
    if (kWrite) { const uint32_t m = W.n / (uint32_t)bpm; mrow = m / W.mcu_w; mcol = m - mrow * W.mcu_w; }
    bool stop = kWrite && W.n >= W.n1;
    while (!stop && br.pos() < pos_end) {
        br.refill();
        const uint32_t win = br.top32();
        const int ci = inter ? (j < ny ? 0 : j - ny + 1) : 0;
        const int c = inter ? ci : c0;
        const HuffTab& tab = tabs2[(slots >> (2 * ci)) & 1u];
        const uint32_t e = huff_lookup(tab, win);
        const int len = (int)(e >> 8), sz = (int)(e & 255u);
        if (e == 0 || sz > 15) {
            if (kWrite) { bad = true; break; }
            br.skip(1);
            continue;
        }
        const int d = extend_bits(top_bits(win << len, sz), sz);
        br.skip(len + sz);
        if (c == 0) s0 += d; else if (c == 1) s1 += d; else s2 += d;
        if (kWrite) {
            const int pv = (c == 0 ? W.pred[0] : (c == 1 ? W.pred[1] : W.pred[2])) + d;
            if (c == 0) W.pred[0] = pv; else if (c == 1) W.pred[1] = pv; else W.pred[2] = pv;
            uint64_t blk;
            if (inter && c == 0) blk = W.coff[0] + (uint64_t)(W.vs * mrow + ((uint32_t)j >> (W.hs - 1u))) * W.bw[0] + W.hs * mcol + ((uint32_t)j & (W.hs - 1u));
            else blk = W.coff[c] + (uint64_t)mrow * W.bw[c] + mcol;
            W.head[blk * 8] = (int16_t)(pv << W.Al);
            if (++W.n >= W.n1) stop = true;
        }
        ++nb;
        if (++j == bpm) {
            j = 0;
            if (kWrite) { if (++mcol == W.mcu_w) { mcol = 0; ++mrow; } }
        }
    }
    pos_out = br.pos();
    j_out = j;
    nblk = nb;
    sum0 = s0; sum1 = s1; sum2 = s2;
}

// Exclusive prefix sum over the CTA's threads in thread order (warp scans, then the warps' totals
// through shared memory); total = the sum over all threads.  Every thread of the CTA calls it.
template <class T>
__device__ __forceinline__ T cta_exclusive_sum(T v, T* s_tmp, int wid, int lane, int warps, T& total) {
    const unsigned full = 0xffffffffu;
    T inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const T o = __shfl_up_sync(full, inc, d);
        if (lane >= d) inc += o;
    }
    __syncthreads();                                           // s_tmp may still be read from the previous call
    if (lane == 31) s_tmp[wid] = inc;
    __syncthreads();
    T before = 0, all = 0;
    for (int w = 0; w < warps; ++w) { const T t = s_tmp[w]; if (w < wid) before += t; all += t; }
    total = all;
    return before + inc - v;
}

// One CTA of kLongWarps warps per listed (scan, image) whose scan is one restart interval; first
// passes only.  The interval is cut into 32 * kLongWarps subsequences, one per thread.
__global__ void __launch_bounds__(32 * kLongWarps) first_pass_long_kernel(Params P, const uint32_t* __restrict__ list, uint32_t count) {
    __shared__ HuffTab tabs[2];
    __shared__ uint32_t s_pos[kLongWarps];                     // end state of every warp's last lane, for the next warp's first
    __shared__ int s_state[kLongWarps];
    __shared__ uint32_t s_u[kLongWarps];
    __shared__ int s_i[kLongWarps];
    __shared__ __align__(4) uint16_t s_lut[1 << kLutBits];    // the search pass's table (AC), or two byte tables (DC)
    const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
    const uint32_t it = blockIdx.x;
    if (it >= count) return;                                   // whole CTA
    const uint32_t si = list[it];
    const int s = (int)(si / (uint32_t)P.N), img = (int)(si % (uint32_t)P.N);
    const ScanDesc sd = P.scans[si];
    const ScanScript sc = P.script[s];
    const ImgDesc im = P.imgs[img];
    const Geometry g = make_geometry(im, P);
    const bool dc = sc.Ss == 0, inter = sc.ncomp > 1;
    const int c0 = sc.comp[0];
    const uint32_t mcu_w = inter ? g.mx : g.ubw[c0];
    const uint32_t mcu_h = inter ? g.my : g.ubh[c0];
    const uint32_t total = mcu_w * mcu_h;                      // MCUs of the scan (one interval)
    const unsigned full = 0xffffffffu;
    if (wid == 0) build_hufftab(tabs[0], P.rec + sd.tab_off[0], lane);
    if (wid == (kLongWarps > 1 ? 1 : 0) && sd.tab_off[1]) build_hufftab(tabs[1], P.rec + sd.tab_off[1], lane);
    __syncthreads();
    if (dc) {
        uint8_t* dl = reinterpret_cast<uint8_t*>(s_lut);
        for (int i = tid; i < (2 << kLutBits); i += 32 * kLongWarps) {
            const uint32_t t = ((i >> kLutBits) == 0 || sd.tab_off[1]) ? tabs[i >> kLutBits].lut[i & ((1 << kLutBits) - 1)] : 0u;
            dl[i] = (uint8_t)((t != 0 && (t & 255u) <= 15u) ? ((t >> 8) << 4) | (t & 15u) : 0u);
        }
    } else {
        for (int i = tid; i < (1 << kLutBits); i += 32 * kLongWarps) s_lut[i] = (uint16_t)ac_search_entry(tabs[0].lut[i]);
    }
    __syncthreads();
    const uint32_t* segtab = P.seg_start + sd.seg_base;
    const uint32_t bstart = segtab[0], bend = segtab[1] - 2u;
    if (bstart < sd.data_off || bend > sd.data_end || bend < bstart) {   // (the same for every thread)
        if (tid == 0) atomicMin(&P.status[img], kErrCorrupt);
        return;
    }
    const uint32_t* base = reinterpret_cast<const uint32_t*>(P.ubuf) + (bstart >> 2);
    const uint32_t lead = 8u * (bstart & 3u), endbit = lead + 8u * (bend - bstart);
    // subsequences of S bits (whole words, at least 8 of them)
    constexpr uint32_t kSubs = 32u * kLongWarps;
    const uint32_t nwords = (endbit + 31u) >> 5;
    const uint32_t S = 32u * max(8u, (nwords + kSubs - 1u) / kSubs);
    const uint32_t my_begin = min(max((uint32_t)tid * S, lead), endbit), my_end = min(((uint32_t)tid + 1u) * S, endbit);
    bool bad = false;
    // the state the previous thread ended in (its last lane's through shared memory for a warp's first lane)
    auto handed_on = [&](uint32_t pos_x, int st_x, uint32_t& ppos, int& pst) {
        if (lane == 31) { s_pos[wid] = pos_x; s_state[wid] = st_x; }
        __syncthreads();
        ppos = __shfl_up_sync(full, pos_x, 1);
        pst = __shfl_up_sync(full, st_x, 1);
        if (lane == 0 && wid > 0) { ppos = s_pos[wid - 1]; pst = s_state[wid - 1]; }
        ppos = min(ppos, endbit);
    };
    if (dc) {
        DcWrite W;
        W.head = P.head; W.mcu_w = mcu_w; W.Al = sc.Al; W.hs = (uint32_t)P.hs; W.vs = (uint32_t)P.vs;
        const uint32_t bpm = inter ? (uint32_t)(P.hs * P.vs + 2) : 1u;
#pragma unroll
        for (int c = 0; c < 3; ++c) { W.coff[c] = g.coff[c]; W.bw[c] = g.bw[c]; W.pred[c] = 0; }
        W.n = 0; W.n1 = total * bpm;
        // per block of the MCU: its table (one bit) and its component (two bits)
        uint32_t tbits = 0, cpack = 0;
        for (uint32_t jj = 0; jj < bpm; ++jj) {
            const uint32_t ny = (uint32_t)(P.hs * P.vs), ci = inter ? (jj < ny ? 0u : jj - ny + 1u) : 0u;
            tbits |= ((sd.slots >> (2u * ci)) & 1u) << jj;
            cpack |= (inter ? ci : (uint32_t)c0) << (2u * jj);
        }
        uint32_t pos = my_begin, pos_x = my_begin, nb = 0;
        int j = 0, j_x = 0, a0 = 0, a1 = 0, a2 = 0;
        bool again = true;
        for (int round = 0; round <= (int)kSubs; ++round) {
            if (again) dc_search_span(tabs, reinterpret_cast<const uint8_t*>(s_lut), tbits, cpack, (int)bpm, base, pos, j, my_end, pos_x, j_x, nb, a0, a1, a2);
            uint32_t ppos; int pj;
            handed_on(pos_x, j_x, ppos, pj);
            again = tid > 0 && (ppos != pos || pj != j);
            if (again) { pos = ppos; j = pj; }
            if (!__syncthreads_or(again)) break;
        }
        // first block and predictors of every thread: exclusive prefix sums
        uint32_t all;
        int t0, t1, t2;
        W.n = min(cta_exclusive_sum(nb, s_u, wid, lane, kLongWarps, all), W.n1);
        W.pred[0] = cta_exclusive_sum(a0, s_i, wid, lane, kLongWarps, t0);
        W.pred[1] = cta_exclusive_sum(a1, s_i, wid, lane, kLongWarps, t1);
        W.pred[2] = cta_exclusive_sum(a2, s_i, wid, lane, kLongWarps, t2);
        // the place inside the MCU follows from the block number (equal to the handed-on state unless
        // the stream is damaged; taking it from the block number keeps every store inside the image)
        if (nb && (uint32_t)j != W.n % bpm) bad = true;
        j = (int)(W.n % bpm);
        dc_first_span<true>(tabs, sd.slots, inter, c0, base, pos, j, my_end, pos_x, j_x, nb, a0, a1, a2, W, bad);
        if (all < total * bpm) bad = true;                     // the stream ends before the last block
    } else {
        const int c = c0, Ss = sc.Ss, Se = sc.Se;
        const ScanAux ax = P.saux[s];
        AcWrite W;
        W.plane = P.planes + g.coff[c] * 64; W.headp = P.head + g.coff[c] * 8;
        W.maskp = reinterpret_cast<unsigned long long*>(P.aux + ax.base + g.loff[c]);
        W.mcu_w = mcu_w; W.bw = g.bw[c]; W.m = 0; W.m1 = total; W.p1 = 1 << sc.Al;
        const HuffTab& tab = tabs[0];
        uint32_t pos = my_begin, pos_x = my_begin, nb = 0;
        int k = Ss, k_x = Ss;
        bool again = true;
        for (int round = 0; round <= (int)kSubs; ++round) {
            if (again) ac_search_span(tab, s_lut, base, pos, k, my_end, Ss, Se, pos_x, k_x, nb);
            uint32_t ppos; int pk;
            handed_on(pos_x, k_x, ppos, pk);
            again = tid > 0 && (ppos != pos || pk != k);
            if (again) { pos = ppos; k = pk; }
            if (!__syncthreads_or(again)) break;
        }
        uint32_t all;
        W.m = min(cta_exclusive_sum(nb, s_u, wid, lane, kLongWarps, all), total);
        ac_first_span<true>(tab, base, pos, k, my_end, Ss, Se, pos_x, k_x, nb, W, bad);
        if (all < total) bad = true;                                         // the stream ends before the last block
    }
    if (__syncthreads_or(bad) && tid == 0) atomicMin(&P.status[img], kErrCorrupt);
}

// ---------------------------------------------------------------------------------------
// A sequential (baseline) scan that is one restart interval: the same scheme as the first passes.
// The state a lane hands on is (bit position, block of the MCU, zigzag position inside the block;
// 0 = the block's DC symbol comes next); every lane counts the blocks it finishes and sums the DC
// differences it reads per component.
// ---------------------------------------------------------------------------------------
struct SeqWrite {
    int16_t* head;
    int16_t* planes;
    uint64_t coff[3];
    uint32_t bw[3];
    uint32_t mcu_w;
    uint32_t hs, vs;
    uint32_t n, n1;        // next block of the scan in scan order (the one being decoded), one past the last
    int pred[3];
};

template <bool kWrite>
__device__ __forceinline__ void seq_span(const HuffTab* tabs4, uint32_t slots, uint32_t slots_ac, int nc, const uint32_t* base,
                                         uint32_t pos, int j, int k, uint32_t pos_end, uint32_t& pos_out, int& j_out, int& k_out,
                                         uint32_t& nblk, int& sum0, int& sum1, int& sum2, SeqWrite& W, bool& bad) {
    WordReader br;
    br.init(base, pos);
    const int ny = (int)(W.hs * W.vs), bpm = nc == 3 ? ny + 2 : 1;
    uint32_t nb = 0;
    int s0 = 0, s1 = 0, s2 = 0;
    uint32_t mrow = 0, mcol = 0;
    if (kWrite) { const uint32_t m = W.n / (uint32_t)bpm; mrow = m / W.mcu_w; mcol = m - mrow * W.mcu_w; }
    bool stop = kWrite && W.n >= W.n1;
    while (!stop && br.pos() < pos_end) {
        br.refill();
        const uint32_t win = br.top32();
        const int c = nc == 3 ? (j < ny ? 0 : j - ny + 1) : 0;
        const bool is_dc = k == 0;
        const int ti = is_dc ? (int)((slots >> (2 * c)) & 1u) : 2 + (int)((slots_ac >> (2 * c)) & 1u);
        const uint32_t e = huff_lookup(tabs4[ti], win);
        const int len = (int)(e >> 8), r = is_dc ? 0 : (int)(e >> 4) & 15, sz = is_dc ? (int)(e & 255u) : (int)(e & 15u);
        const bool is_coef = sz != 0, is_zrl = !is_dc && sz == 0 && r == 15, is_eob = !is_dc && sz == 0 && r == 0;
        const int kk = k + r;
        if (e == 0 || sz > 15 || (!is_dc && !is_coef && !is_zrl && !is_eob) || (is_coef && kk > 63)) {
            if (kWrite) { bad = true; break; }
            br.skip(1);
            continue;
        }
        const int extra = is_coef ? sz : 0;
        const int v = extend_bits(top_bits(win << len, extra), extra);
        br.skip(len + extra);
        uint64_t blk = 0;
        if (kWrite) {
            if (nc == 3 && c == 0) blk = W.coff[0] + (uint64_t)(W.vs * mrow + ((uint32_t)j >> (W.hs - 1u))) * W.bw[0] + W.hs * mcol + ((uint32_t)j & (W.hs - 1u));
            else blk = W.coff[c] + (uint64_t)mrow * W.bw[c] + mcol;
        }
        if (is_dc) {
            if (c == 0) s0 += v; else if (c == 1) s1 += v; else s2 += v;
            if (kWrite) {
                const int pv = (c == 0 ? W.pred[0] : (c == 1 ? W.pred[1] : W.pred[2])) + v;
                if (c == 0) W.pred[0] = pv; else if (c == 1) W.pred[1] = pv; else W.pred[2] = pv;
                W.head[blk * 8] = (int16_t)pv;
            }
            k = 1;
        } else if (is_coef) {
            if (kWrite) {
                if (kk < 8) W.head[blk * 8 + kk] = (int16_t)v;
                else W.planes[blk * 64 + kk] = (int16_t)v;
            }
            k = kk + 1;
        } else if (is_zrl) {
            k += 16;
        }
        if (is_eob || k > 63) {                               // block finished
            k = 0;
            ++nb;
            if (kWrite && ++W.n >= W.n1) stop = true;
            if (++j == bpm) {
                j = 0;
                if (kWrite) { if (++mcol == W.mcu_w) { mcol = 0; ++mrow; } }
            }
        }
    }
    pos_out = br.pos();
    j_out = j;
    k_out = k;
    nblk = nb;
    sum0 = s0; sum1 = s1; sum2 = s2;
}

#ifndef PCR_SEQ_LONG_WARPS
#define PCR_SEQ_LONG_WARPS 4
#endif
constexpr int kSeqLongWarps = PCR_SEQ_LONG_WARPS;   // warps per image in sequential_long_kernel: 32 subsequences each

// One CTA of kSeqLongWarps warps per listed image whose (one) sequential scan is one restart interval.
__global__ void __launch_bounds__(32 * kSeqLongWarps) sequential_long_kernel(Params P, const uint32_t* __restrict__ list, uint32_t count) {
    __shared__ HuffTab tabs[4];                                // DC 0, DC 1, AC 0, AC 1
    __shared__ uint32_t s_pos[kSeqLongWarps];                  // end state of every warp's last lane, for the next warp's first
    __shared__ int s_state[kSeqLongWarps];
    __shared__ uint32_t s_u[kSeqLongWarps];
    __shared__ int s_i[kSeqLongWarps];
    const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
    const uint32_t it = blockIdx.x;
    if (it >= count) return;                                   // whole CTA
    const uint32_t si = list[it];
    const int img = (int)(si % (uint32_t)P.N);
    const ScanDesc sd = P.scans[si];
    const ImgDesc im = P.imgs[img];
    const Geometry g = make_geometry(im, P);
    const uint32_t mcu_w = g.mx, total = g.mx * g.my;
    const uint32_t bpm = P.nc == 3 ? (uint32_t)(P.hs * P.vs + 2) : 1u;
    const unsigned full = 0xffffffffu;
    // four tables, built by the warps in turn
    for (int t = wid; t < 4; t += kSeqLongWarps) {
        const uint32_t off = t == 0 ? sd.tab_off[0] : (t == 1 ? sd.tab_off[1] : (t == 2 ? sd.tab_ac[0] : sd.tab_ac[1]));
        if (off) build_hufftab(tabs[t], P.rec + off, lane);
    }
    __syncthreads();
    const uint32_t* segtab = P.seg_start + sd.seg_base;
    const uint32_t bstart = segtab[0], bend = segtab[1] - 2u;
    if (bstart < sd.data_off || bend > sd.data_end || bend < bstart) {   // (the same for every thread)
        if (tid == 0) atomicMin(&P.status[img], kErrCorrupt);
        return;
    }
    const uint32_t* base = reinterpret_cast<const uint32_t*>(P.ubuf) + (bstart >> 2);
    const uint32_t lead = 8u * (bstart & 3u), endbit = lead + 8u * (bend - bstart);
    constexpr uint32_t kSubs = 32u * kSeqLongWarps;
    const uint32_t nwords = (endbit + 31u) >> 5;
    const uint32_t S = 32u * max(8u, (nwords + kSubs - 1u) / kSubs);
    const uint32_t my_begin = min(max((uint32_t)tid * S, lead), endbit), my_end = min(((uint32_t)tid + 1u) * S, endbit);
    bool bad = false;
    SeqWrite W;
    W.head = P.head; W.planes = P.planes; W.mcu_w = mcu_w; W.hs = (uint32_t)P.hs; W.vs = (uint32_t)P.vs;
#pragma unroll
    for (int c = 0; c < 3; ++c) { W.coff[c] = g.coff[c]; W.bw[c] = g.bw[c]; W.pred[c] = 0; }
    W.n = 0; W.n1 = total * bpm;
    uint32_t pos = my_begin, pos_x = my_begin, nb = 0;
    int j = 0, k = 0, j_x = 0, k_x = 0, a0 = 0, a1 = 0, a2 = 0;
    bool again = true;
    for (int round = 0; round <= (int)kSubs; ++round) {
        if (again) seq_span<false>(tabs, sd.slots, sd.slots_ac, P.nc, base, pos, j, k, my_end, pos_x, j_x, k_x, nb, a0, a1, a2, W, bad);
        // the state the previous thread ended in (block of the MCU and zigzag position in one word)
        const int st_x = j_x * 64 + k_x;
        if (lane == 31) { s_pos[wid] = pos_x; s_state[wid] = st_x; }
        __syncthreads();
        uint32_t ppos = __shfl_up_sync(full, pos_x, 1);
        int pst = __shfl_up_sync(full, st_x, 1);
        if (lane == 0 && wid > 0) { ppos = s_pos[wid - 1]; pst = s_state[wid - 1]; }
        ppos = min(ppos, endbit);
        again = tid > 0 && (ppos != pos || pst != j * 64 + k);
        if (again) { pos = ppos; j = pst >> 6; k = pst & 63; }
        if (!__syncthreads_or(again)) break;
    }
    uint32_t all;
    int t0, t1, t2;
    W.n = min(cta_exclusive_sum(nb, s_u, wid, lane, kSeqLongWarps, all), W.n1);
    W.pred[0] = cta_exclusive_sum(a0, s_i, wid, lane, kSeqLongWarps, t0);
    W.pred[1] = cta_exclusive_sum(a1, s_i, wid, lane, kSeqLongWarps, t1);
    W.pred[2] = cta_exclusive_sum(a2, s_i, wid, lane, kSeqLongWarps, t2);
    // the place inside the MCU follows from the block number (equal to the handed-on state unless the
    // stream is damaged; taking it from the block number keeps every store inside the image)
    if ((nb || k) && (uint32_t)j != W.n % bpm) bad = true;
    j = (int)(W.n % bpm);
    seq_span<true>(tabs, sd.slots, sd.slots_ac, P.nc, base, pos, j, k, my_end, pos_x, j_x, k_x, nb, a0, a1, a2, W, bad);
    if (all < total * bpm) bad = true;                         // the stream ends before the last block
    if (__syncthreads_or(bad) && tid == 0) atomicMin(&P.status[img], kErrCorrupt);
}

// ---------------------------------------------------------------------------------------
// AC refinements of scans that are one restart interval.  The unit of work is a chain: one
// refinement scan of one (image, component) group; a group has at most four (its "levels", in
// scan order).  Side data written per block is that of entropy_kernel's refinement branch:
// {non-zero mask of the band after the scan, correction bits in reading order from bit 63 down,
// newly non-zero positions, the positive ones among them}.
//
// The time of a chain is the number of instructions one thread executes per symbol (every
// instruction waits for the one before), so the decoding thread only follows the chain: Huffman
// symbol -> run r -> position of the (r+1)-th still-zero coefficient -> number of correction bits
// passed -> next symbol.  For every symbol it leaves a record {bit position behind the sign, new
// position, number of correction bits}; the chain's helper warp lists the still-zero positions
// of the next 32 blocks meanwhile and afterwards turns the records of 32 blocks into the side
// data (one lane per block, reading sign and correction bits back from the ring).
//
// A later refinement of the same component needs the masks the earlier one leaves, block by
// block.  Both walk the same block grid in the same order, so the later chain runs behind the
// earlier one instead of after it: every chain publishes the number of blocks whose side data it
// has written (global memory, after a fence), and a helper that depends on it waits, with a
// bounded number of polls, until the blocks it is about to read are there.  A chain is only
// started after the chains it depends on (queue order), so its producer is running or done.
// ---------------------------------------------------------------------------------------
constexpr int kChainPairs = 16;          // chains per CTA of the persistent refinement launch (four per scheduler), two warps each
constexpr int kChainRing = 256;          // words of bitstream per chain in shared memory
constexpr int kChainRecs = 512;          // symbol records per batch of blocks (four bytes each)
constexpr int kChainLutBits = 9;         // refinement alphabets are small (runs 0..15 with size 0 or 1): short codes
constexpr uint32_t kChainBlockWords = 44;   // a block never needs more: 63 symbols of at most 17 bits, 3 sixteen-zero runs, one run length, 63 correction bits
constexpr uint32_t kSpinLimit = 1u << 22;   // polls (of at least 64 ns) before a wait gives up
constexpr int kErrTimeout = -4;

struct ChainBits {
    const uint32_t* ring;
    uint32_t w0, w1, w2;   // the word the next bit lies in and the two after it
    uint32_t bits;         // position of the next bit, counted from the first bit of ring word `org`
    uint32_t org;          // absolute index of that word (moved up at the start of every batch)
    __device__ __forceinline__ void init(const uint32_t* r, uint32_t first, uint32_t lead) {
        ring = r;
        w0 = r[first & (kChainRing - 1)]; w1 = r[(first + 1) & (kChainRing - 1)]; w2 = r[(first + 2) & (kChainRing - 1)];
        org = first;
        bits = lead;
    }
    __device__ __forceinline__ uint32_t win() const { return __funnelshift_l(w1, w0, bits); }   // the next 32 bits (shift taken mod 32)
    __device__ __forceinline__ uint32_t word() const { return org + (bits >> 5); }               // absolute index of the word of the next bit
    __device__ __forceinline__ void skip(uint32_t n) {
        const uint32_t nb = bits + n, adv = (nb >> 5) - (bits >> 5);
        bits = nb;
        if (adv) {
            const uint32_t wi = org + (nb >> 5);
            if (adv == 1u) { w0 = w1; w1 = w2; }
            else { w0 = ring[wi & (kChainRing - 1)]; w1 = ring[(wi + 1u) & (kChainRing - 1)]; }
            w2 = ring[(wi + 2u) & (kChainRing - 1)];
        }
    }
    __device__ __forceinline__ void rebase() { org += bits >> 5; bits &= 31u; }
};

// the n bits (1..32) at bit position p (counted from the first bit of word `base`) of the ring
__device__ __forceinline__ uint32_t ring_bits(const uint32_t* ring, uint32_t base, uint32_t p, uint32_t n) {
    const uint32_t a = ring[(base + (p >> 5)) & (kChainRing - 1)], b = ring[(base + (p >> 5) + 1u) & (kChainRing - 1)];
    return __funnelshift_l(b, a, p & 31u) >> (32u - n);
}

// Polls *flag until it reaches `need`, sleeping `ns` nanoseconds between polls; false after `limit` polls.
__device__ __forceinline__ bool wait_at_least(const volatile uint32_t* flag, uint32_t need, uint32_t limit, uint32_t ns = 64) {
#pragma unroll 1
    for (uint32_t i = 0; i < limit; ++i) {
        if (*flag >= need) return true;
        __nanosleep(ns);
    }
    return false;
}

// Entry of the chain's own lookup table on the next kChainLutBits bits, made from the Huffman table:
// bits 0..4 = bits to skip (code, plus the sign bit of a new coefficient), 5..11 = run r, 15 = a new
// coefficient follows the run; the end of band of a single block is entered as a run of 64 without a
// new coefficient (it passes over the rest of the band like a run that overshoots); 0 = everything
// else (longer end-of-band runs, codes longer than the index, undefined codes): the general path.
__device__ __noinline__ uint32_t chain_lookup(const HuffTabT<kChainLutBits>& tab, uint32_t win) { return huff_lookup(tab, win); }

struct ChainLists {
    uint64_t h[32];                    // positions of the band that are already non-zero, per block of the batch
    uint8_t zpos[64][32];              // [i][block]: position of the block's i-th still-zero coefficient of the band, minus i;
                                       // entry nz: Se + 1 - nz (as if position Se + 1 followed)
    uint8_t nz[32];                    // how many such positions there are (at most 63)
};
struct ChainRecs {
    uint32_t rec[kChainRecs];          // corrections | position << 8 | new << 15 | (bit position behind the sign bit - base) << 16
    uint32_t first[33];                // first record of each block of the batch
    uint32_t base;                     // bit position at which the batch starts
};
struct ChainMail {                     // what the two warps of a chain tell each other at a meeting point
    uint32_t nd, rd, err_c;            // decoder: blocks it decoded, oldest ring word it still needs, error
    uint32_t wr, err_h;                // helper: the ring is filled up to this word, error
};
struct ChainShared {
    HuffTabT<kChainLutBits> tab;
    uint32_t quick[1 << kChainLutBits];
    uint32_t ring[kChainRing];
    ChainLists lists[2];               // the batch being decoded and the one being prepared
    ChainRecs recs[2];                 // the batch being decoded and the one being turned into side data
    ChainMail mail[2];                 // by parity of the meeting point
    uint32_t job_gi, job_level;        // the pair's job (job_gi = 0xFFFFFFFF: none left)
    uint32_t Ss, Se, total, rd0, lead, limit;   // of the job, for the decoder
    volatile uint32_t phase_c, phase_h;         // meeting points each side has reached
};

// Polls *flag (another warp's progress word in global memory) until it reaches `need`; `seen` keeps
// the last value read, so that a consumer that is behind anyway polls once per many batches.
__device__ __forceinline__ bool wait_progress(const volatile uint32_t* flag, uint32_t need, uint32_t& seen, uint32_t limit) {
    if (seen >= need) return true;
#pragma unroll 1
    for (uint32_t i = 0; i < limit; ++i) {
        seen = *flag;
        if (seen >= need) return true;
        __nanosleep(64);
    }
    return false;
}

// Meeting point k of a chain's two warps: each side announces that it has arrived (everything it
// wrote to shared memory before is visible to the other behind the meeting) and waits, with a
// bounded number of polls, for the other.  false: the partner never came.
__device__ __forceinline__ bool meet_decoder(ChainShared& sh, uint32_t k) {          // one thread
    __threadfence_block();
    sh.phase_c = k;
    const bool ok = wait_at_least(&sh.phase_h, k, kSpinLimit);
    __threadfence_block();
    return ok;
}
__device__ __forceinline__ bool meet_helper(ChainShared& sh, uint32_t k, int lane) {  // a whole warp
    __syncwarp();
    if (lane == 0) { __threadfence_block(); sh.phase_h = k; }
    // (long sleeps: the helper is far ahead of the decoder, and its polls would take issue slots from the chains)
    bool ok = true;
    if (lane == 0) ok = wait_at_least(&sh.phase_c, k, kSpinLimit, 512);
    ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
    __threadfence_block();
    return ok;
}

// The decoding side of a chain: one thread.  It takes the pair's jobs (first the statically assigned
// one, then tickets of its scheduler's queue), and per job follows the bit stream batch by batch:
// the lists of still-zero positions of a batch come from the helper, the symbol records go back to it.
__device__ __forceinline__ void chain_decoder(const FinalizeList& fl, ChainShared& sh, const uint32_t* __restrict__ list, uint32_t n_groups,
                                              uint32_t* sync, uint32_t levels, uint32_t rounds, uint32_t q, uint32_t slot) {
    const uint32_t per_round = 4u * gridDim.x, statics = per_round * rounds;
    uint32_t mk = 0;                                           // meeting points so far
    bool first_job = true;
    for (;;) {
        uint32_t gi, level;
        for (;;) {
            if (first_job) {
                first_job = false;
                gi = (slot / levels) * per_round + 4u * blockIdx.x + q;
                level = slot % levels;
            } else {
                const uint32_t t = atomicAdd(&sync[q], 1u);
                gi = statics + 4u * (t / levels) + q;
                level = t % levels;
            }
            if (gi >= n_groups) { gi = 0xFFFFFFFFu; break; }  // the queue is empty (entries only grow)
            if ((int)level < fl.n[list[gi] >> 28]) break;      // (a component with fewer refinements has no such level)
        }
        sh.job_gi = gi; sh.job_level = level;
        if (!meet_decoder(sh, ++mk)) return;                   // the helper has the job
        if (gi == 0xFFFFFFFFu) return;
        if (!meet_decoder(sh, ++mk)) return;                   // tables, first lists and ring are ready
        if (sh.mail[mk & 1u].err_h) continue;                  // a scan whose bounds are off: the helper reports it
        uint32_t wr = sh.mail[mk & 1u].wr;
        const uint32_t Ss = sh.Ss, Se = sh.Se, total = sh.total, limit = sh.limit;
        ChainBits B;
        B.init(sh.ring, sh.rd0, sh.lead);
        uint32_t eobrun = 0, m = 0, p = 0;
        for (;;) {
            const uint32_t nblk = min(32u, total - m);
            const ChainLists& L = sh.lists[p];
            ChainRecs& R = sh.recs[p];
            // positions inside a batch count from the word the batch starts in (fewer than 2^16 bits: 32
            // blocks of kChainBlockWords words)
            B.rebase();
            const uint32_t base = (B.org - sh.rd0) * 32u;
            R.base = base;
            // a block is only begun while kChainBlockWords words lie ahead in the ring and the interval has
            // not ended: one comparison for both, told apart behind the loop
            const uint32_t avail = wr - B.org;
            const uint32_t pause_bits = avail > kChainBlockWords + 2u ? (avail - (kChainBlockWords + 2u)) << 5 : 0u;
            const uint32_t end_bits = limit >= base ? limit - base + 1u : 0u;      // first position that is past the end
            const uint32_t stop_bits = min(pause_bits, end_bits);
            uint32_t* recp = R.rec;
            uint32_t* const rec_stop = R.rec + (kChainRecs - 64);
            uint32_t nd = 0;
            int err = 0;
            for (; nd < nblk; ++nd) {
                if (B.bits >= stop_bits || recp > rec_stop) break;
                R.first[nd] = (uint32_t)(recp - R.rec);
                // zi: how many of the block's still-zero positions are passed; ep: the list entry of the last
                // one reached (entry t = position - t, so that the difference of two entries is the number of
                // non-zero positions between them: one correction bit each)
                const uint32_t nz = L.nz[nd];
                uint32_t zi = 0, ep = Ss;
                bool band_done = false;
                if (eobrun == 0) {
                    for (;;) {
                        const uint32_t win = B.win();
                        uint32_t qe = sh.quick[win >> (32 - kChainLutBits)];
                        if (qe == 0) {                         // not a plain (run, new coefficient) symbol
                            const uint32_t e = chain_lookup(sh.tab, win);
                            const uint32_t len = e >> 8, rs = e & 255u, newc = rs & 1u, r = rs >> 4;
                            if (e == 0 || (rs & 14u)) { err = kErrCorrupt; break; }   // a refinement symbol has size 0 or 1
                            if (!newc && r < 15u) {            // end of band for this block and eobrun - 1 more
                                eobrun = 1u << r;
                                if (r) eobrun += (win << len) >> (32u - r);
                                B.skip(len + r);
                                break;
                            }
                            qe = (len + newc) | (r << 5) | (newc << 15);   // a code longer than the table's index
                        }
                        // the target: the (r+1)-th still-zero position from here; a run past the last one ends
                        // at the list's closing entry (position Se + 1)
                        const uint32_t t = min(zi + ((qe >> 5) & 127u), nz);
                        const uint32_t e = L.zpos[t][nd];
                        const uint32_t cnt = e - ep, pos = e + t, n1 = qe & 31u;
                        *recp++ = ((B.bits + n1) << 16) | (pos << 8) | (qe & 0x8000u) | cnt;
                        B.skip(n1 + cnt);                      // code, sign and correction bits in one step
                        zi = t + 1u;
                        ep = e;
                        if (pos >= Se) { band_done = true; break; }
                    }
                }
                if (err) break;
                if (!band_done) {                              // inside an end-of-band run: corrections for the rest of the band
                    const uint32_t cnt = L.zpos[nz][nd] - ep;
                    *recp++ = (B.bits << 16) | cnt;
                    B.skip(cnt);
                    --eobrun;
                }
            }
            R.first[nd] = (uint32_t)(recp - R.rec);
            if (!err && B.bits >= end_bits) err = kErrCorrupt;     // read past the end of the interval
            ++mk;
            sh.mail[mk & 1u].nd = nd; sh.mail[mk & 1u].rd = B.word(); sh.mail[mk & 1u].err_c = (uint32_t)err;
            if (!meet_decoder(sh, mk)) return;
            wr = sh.mail[mk & 1u].wr;
            if (err || sh.mail[mk & 1u].err_h) break;
            m += nd;
            if (nd == nblk) {
                p ^= 1u;
                if (m >= total) break;
            } else {                                           // stopped early: the helper lists the blocks from m again
                if (!meet_decoder(sh, ++mk)) return;
                wr = sh.mail[mk & 1u].wr;
                if (sh.mail[mk & 1u].err_h) break;
                p ^= 1u;
            }
        }
    }
}

// The helper side of a chain: a whole warp.  Per job it builds the tables, then stays one batch ahead
// of the decoder with the masks and lists of still-zero positions (waiting, with bounded polls, for
// an earlier refinement of the same blocks when this launch decodes that too), keeps the ring of
// bitstream words filled, and one batch behind it turns the symbol records into side data.
__device__ __forceinline__ void chain_helper(const Params& P, const FinalizeList& fl, ChainShared& sh, const uint32_t* __restrict__ list,
                                             uint32_t* progress_all, int lane) {
    const unsigned full = 0xffffffffu;
    uint32_t mk = 0;
    for (;;) {
        if (!meet_helper(sh, ++mk, lane)) return;
        const uint32_t gi = sh.job_gi;
        const int level = (int)sh.job_level;
        if (gi == 0xFFFFFFFFu) return;
        const uint32_t entry = list[gi];
        const int c = (int)(entry >> 28), img = (int)(entry & 0x0FFFFFFFu);
        uint32_t* progress = progress_all + 4ull * gi;
        volatile uint32_t* my_progress = progress + level;
        const int s = fl.scan[c][level];
        const ScanDesc sd = P.scans[(uint32_t)s * (uint32_t)P.N + (uint32_t)img];
        const ScanScript sc = P.script[s];
        const Geometry g = make_geometry(P.imgs[img], P);
        const uint32_t Ss = (uint32_t)sc.Ss, Se = (uint32_t)sc.Se;
        const uint32_t mcu_w = g.ubw[c], total = g.ubw[c] * g.ubh[c], bw = g.bw[c];
        build_hufftab(sh.tab, P.rec + sd.tab_off[0], lane);
        for (int i = lane; i < (1 << kChainLutBits); i += 32) {
            const uint32_t e = sh.tab.lut[i], len = e >> 8, rs = e & 255u, newc = rs & 1u, r = rs >> 4;
            const bool plain = e != 0 && (rs & 14u) == 0 && (newc || r == 15u || r == 0u);   // run + new coefficient, sixteen zeros, end of band
            sh.quick[i] = plain ? ((len + newc) | ((rs == 0u ? 64u : r) << 5) | (newc << 15)) : 0u;
        }
        const uint32_t* segtab = P.seg_start + sd.seg_base;
        const uint32_t bstart = segtab[0], bend = segtab[1] - 2u;
        const bool bad = bstart < sd.data_off || bend > sd.data_end || bend < bstart;
        const uint32_t* words = reinterpret_cast<const uint32_t*>(P.ubuf);
        const uint32_t rd0 = bstart >> 2, lead = 8u * (bstart & 3u);
        const uint32_t wlim = ((bend + 3u) >> 2) + 2u;         // words beyond are not read (zeros instead)
        if (lane == 0) {
            sh.Ss = Ss; sh.Se = Se; sh.total = total; sh.rd0 = rd0; sh.lead = lead;
            sh.limit = lead + 8u * (bend - bstart);            // first bit behind the interval, counted from word rd0
        }
        // masks of the positions that are already non-zero: the union of up to four earlier scans; a
        // source that this launch decodes itself (an earlier level of the group) is waited for
        // (prod* = its progress word)
        const ScanAux ax = P.saux[s];
        const uint64_t band = low_mask((int)Se + 1) & ~low_mask((int)Ss);
        const uint64_t* src0 = nullptr; const uint64_t* src1 = nullptr; const uint64_t* src2 = nullptr; const uint64_t* src3 = nullptr;
        uint32_t st0 = 0, st1 = 0, st2 = 0, st3 = 0;
        const volatile uint32_t* prod0 = nullptr; const volatile uint32_t* prod1 = nullptr; const volatile uint32_t* prod2 = nullptr;
        {
            auto producer = [&](int scan) -> const volatile uint32_t* {
                for (int w = 0; w < level; ++w) if (fl.scan[c][w] == scan) return progress + w;
                return nullptr;
            };
            auto note = [&](const volatile uint32_t* q) { if (q) { if (!prod0) prod0 = q; else if (!prod1) prod1 = q; else prod2 = q; } };
            const ScanAux x0 = P.saux[ax.src[0]];
            src0 = P.aux + x0.base + g.loff[c] * x0.stride; st0 = x0.stride; note(producer(ax.src[0]));
            if (ax.nsrc > 1) { const ScanAux x = P.saux[ax.src[1]]; src1 = P.aux + x.base + g.loff[c] * x.stride; st1 = x.stride; note(producer(ax.src[1])); }
            if (ax.nsrc > 2) { const ScanAux x = P.saux[ax.src[2]]; src2 = P.aux + x.base + g.loff[c] * x.stride; st2 = x.stride; note(producer(ax.src[2])); }
            if (ax.nsrc > 3) { const ScanAux x = P.saux[ax.src[3]]; src3 = P.aux + x.base + g.loff[c] * x.stride; st3 = x.stride; note(producer(ax.src[3])); }
        }
        uint64_t* outp = P.aux + ax.base + g.loff[c] * 4ull;
        uint32_t* ring = sh.ring;
        uint32_t wr = rd0, seen0 = 0, seen1 = 0, seen2 = 0;
        int err = bad ? kErrCorrupt : 0;
        auto block_index = [&](uint32_t x) { const uint32_t row = x / mcu_w; return row * bw + (x - row * mcu_w); };
        // the masks of blocks m0 .. m0 + 31 and their lists of still-zero positions
        auto gather = [&](uint32_t m0, ChainLists& L) -> int {
            const uint32_t nblk = min(32u, total - m0);
            if (prod0 && !wait_progress(prod0, m0 + nblk, seen0, kSpinLimit)) return kErrTimeout;
            if (prod1 && !wait_progress(prod1, m0 + nblk, seen1, kSpinLimit)) return kErrTimeout;
            if (prod2 && !wait_progress(prod2, m0 + nblk, seen2, kSpinLimit)) return kErrTimeout;
            __threadfence();
            if ((uint32_t)lane < nblk) {
                const uint32_t bi = block_index(m0 + lane);
                uint64_t v = __ldcg(src0 + (uint64_t)bi * st0);    // not through L1: a line may hold blocks written later
                if (src1) v |= __ldcg(src1 + (uint64_t)bi * st1);
                if (src2) v |= __ldcg(src2 + (uint64_t)bi * st2);
                if (src3) v |= __ldcg(src3 + (uint64_t)bi * st3);
                v &= band;
                L.h[lane] = v;
                // the positions of the band that are still zero, in order: the target of a run r is then one
                // table look-up for the decoder (the (r+1)-th of those not yet passed).  (Listing the few non-zero
                // positions instead and stepping over them measured 18 % slower: the steps sit on the chain.)
                const uint64_t z = ~v & band;
                uint32_t n = 0;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t w = half ? (uint32_t)(z >> 32) : (uint32_t)z;
                    while (w) {
                        L.zpos[n][lane] = (uint8_t)(32 * half + __ffs((int)w) - 1 - (int)n);
                        ++n;
                        w &= w - 1u;
                    }
                }
                L.zpos[n][lane] = (uint8_t)(Se + 1u - n);      // closing entry: behind the band
                L.nz[lane] = (uint8_t)n;
            }
            return 0;
        };
        // the ring filled as far as it goes while word `oldest` is still needed
        auto top_up = [&](uint32_t oldest) {
            while (wr - oldest + 32u <= (uint32_t)kChainRing) {
                ring[(wr + lane) & (kChainRing - 1)] = wr + lane < wlim ? __ldg(words + wr + lane) : 0u;
                wr += 32u;
            }
        };
        // the records of blocks m0 .. m0 + nd - 1 -> side data, one block per lane; then the count
        auto side_data = [&](uint32_t m0, uint32_t nd, const ChainRecs& R, const ChainLists& L) {
            bool over = false;
            if ((uint32_t)lane < nd) {
                uint64_t cstr = 0, Nw = 0, NS = 0;
                uint32_t cn = 0;
                for (uint32_t i = R.first[lane]; i < R.first[lane + 1]; ++i) {
                    const uint32_t rc = R.rec[i], at = R.base + (rc >> 16);
                    uint32_t n = rc & 127u;
                    if (rc & 0x8000u) {
                        if (((rc >> 8) & 127u) > Se) { over = true; break; }   // a new coefficient behind the band
                        const uint64_t bit = 1ull << ((rc >> 8) & 63u);
                        Nw |= bit;
                        if (ring_bits(ring, rd0, at - 1u, 1u)) NS |= bit;
                    }
                    if (cn + n > 64u) { over = true; break; }
                    cn += n;
                    uint32_t bp = at;
                    while (n) {
                        const uint32_t nn = min(n, 32u);
                        cstr = (cstr << nn) | (uint64_t)ring_bits(ring, rd0, bp, nn);
                        bp += nn; n -= nn;
                    }
                }
                if (cn) cstr <<= 64u - cn;                     // first correction bit at bit 63
                ulonglong2* o = reinterpret_cast<ulonglong2*>(outp + (uint64_t)block_index(m0 + lane) * 4);
                o[0] = make_ulonglong2((L.h[lane] | Nw), cstr);
                o[1] = make_ulonglong2(Nw, NS);
            }
            if (__any_sync(full, over)) err = kErrCorrupt;
            __threadfence();                                   // the side data before the count
            __syncwarp(full);
            if (lane == 0) *my_progress = m0 + nd;
        };
        if (!bad) {
            err = gather(0, sh.lists[0]);
            top_up(rd0);
        }
        ++mk;
        if (lane == 0) { sh.mail[mk & 1u].wr = wr; sh.mail[mk & 1u].err_h = (uint32_t)err; }
        if (!meet_helper(sh, mk, lane)) return;
        uint32_t m = 0, p = 0, rd_c = rd0, pend_m = 0, pend_n = 0, pend_p = 0;
        while (!err) {
            const uint32_t nblk = min(32u, total - m);
            if (pend_n) { side_data(pend_m, pend_n, sh.recs[pend_p], sh.lists[pend_p]); pend_n = 0; }
            top_up(rd_c);
            if (m + nblk < total) { const int e = gather(m + nblk, sh.lists[p ^ 1u]); if (!err) err = e; }
            ++mk;
            if (lane == 0) { sh.mail[mk & 1u].wr = wr; sh.mail[mk & 1u].err_h = (uint32_t)err; }
            if (!meet_helper(sh, mk, lane)) return;
            const uint32_t nd = sh.mail[mk & 1u].nd;
            const int err_c = (int)sh.mail[mk & 1u].err_c;
            rd_c = sh.mail[mk & 1u].rd;
            if (err || err_c) { if (!err) err = err_c; break; }
            if (nd == nblk) {
                pend_m = m; pend_n = nd; pend_p = p;
                p ^= 1u;
                m += nd;
                if (m >= total) { side_data(pend_m, pend_n, sh.recs[pend_p], sh.lists[pend_p]); break; }
            } else {                                           // the decoder stopped early: its records now, the lists from m again
                if (nd) side_data(m, nd, sh.recs[p], sh.lists[p]);
                m += nd;
                top_up(rd_c);
                { const int e = gather(m, sh.lists[p ^ 1u]); if (!err) err = e; }
                ++mk;
                if (lane == 0) { sh.mail[mk & 1u].wr = wr; sh.mail[mk & 1u].err_h = (uint32_t)err; }
                if (!meet_helper(sh, mk, lane)) return;
                p ^= 1u;
            }
        }
        __syncwarp(full);
        if (lane == 0) {
            __threadfence();
            *my_progress = 0xFFFFFFFFu;                        // a scan that failed must not keep a later one waiting
            if (err) atomicMin(&P.status[img], err);
        }
    }
}

// Persistent launch: one CTA per SM with `pairs` chains, each a decoding warp (one thread of it
// works) and a helper warp; warp w and its helper w + pairs sit on scheduler w % 4.  The groups
// ((image, component) pairs, luminance first, most bytes first) are dealt to four queues, one per
// scheduler (group gi is in queue gi % 4); within a queue every group is followed through its levels
// (the refinement scans of the component that this call decodes, in script order), so a producer is
// always taken before its consumer.  The first `rounds` groups of each CTA's schedulers are assigned
// statically (group r * 4 * CTAs + 4 * CTA + q in round r: every scheduler of the device gets one
// long luminance chain before any gets a second, and a group's levels start together in one CTA);
// after that a decoder that has finished takes the next entry of its queue from a counter in global
// memory.  sync: four queue counters, then four progress words per group, all zero before the launch.
__global__ void __launch_bounds__(64 * kChainPairs, 1) ac_refine_group_kernel(Params P, FinalizeList fl, const uint32_t* __restrict__ list,
                                                                              uint32_t n_groups, uint32_t* __restrict__ sync, int levels, int rounds) {
    extern __shared__ __align__(16) unsigned char s_dyn[];     // one ChainShared per chain
    ChainShared* s_sh = reinterpret_cast<ChainShared*>(s_dyn);
    const int pairs = (int)(blockDim.x >> 6);
    const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if ((int)threadIdx.x < pairs) { s_sh[threadIdx.x].phase_c = 0; s_sh[threadIdx.x].phase_h = 0; }
    __syncthreads();
    if (wid < pairs) {
        if (lane == 0) chain_decoder(fl, s_sh[wid], list, n_groups, sync, (uint32_t)levels, (uint32_t)rounds, (uint32_t)wid & 3u, (uint32_t)wid >> 2);
    } else {
        chain_helper(P, fl, s_sh[wid - pairs], list, sync + 4, lane);
    }
}

// Test hook: the bounded wait on a flag that nothing sets; *result = 1 if it gave up as it should.
__global__ void bounded_wait_probe_kernel(uint32_t limit, int* result) {
    __shared__ uint32_t s_flag;
    if (threadIdx.x == 0) s_flag = 0;
    __syncthreads();
    const bool ok = wait_at_least(&s_flag, 1u, limit);
    if (threadIdx.x == 0) *result = ok ? 0 : 1;
}

}  // namespace pcr
