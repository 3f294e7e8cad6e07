/*
 * pcr_oracle — plain, slow, single-threaded CPU reference for decoding a Progressive
 * Compressed Record truncated at scan group k to int16 coefficients and RGB pixels.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may call this; it exists so that
 * the CUDA library can be compared with something obviously correct, and so that a CPU
 * baseline can be timed.  It shares no code with the CUDA library.
 *
 * What it follows:
 *  - Record semantics: the paper's Section 3 (metadata, then scan groups; reading from the
 *    start of the record to the end of scan group k gives fidelity k) and Section 5,
 *    "Decoding" (locate the offsets, take the image's scans 1..k, terminate with an EOI
 *    token, hand the byte string to a JPEG decoder).  oracle_reassemble() does exactly that
 *    and oracle_decode_image() decodes its result.
 *  - The JPEG decoder the paper treats as a black box ("progressive compression", Section 2)
 *    is ITU-T T.81, progressive DCT, Huffman coded, 8-bit: marker syntax (Annex B), Huffman
 *    decoding with MINCODE/MAXCODE/VALPTR one bit at a time (Annex F.2.2.3), progressive
 *    scan decoding (Annex G.2), restart handling (F.2.2.4 / E.2.4).
 *  - What a truncated stream shows: coefficients not yet received are zero and received
 *    values are scaled by 2^Al with no rounding bias and no smoothing across blocks.
 *  - Pixels: dequantisation, the 8x8 inverse DCT by its definition with 13-bit integer
 *    cosines and two rounding shifts, 2x2 chroma replication, full-range BT.601 (JFIF) colour
 *    conversion in 16-bit fixed point, crop to W x H, packed RGB.
 *
 * Pins (tests that tie this file to something other than itself): round trip against the
 * encoder's ground-truth coefficients, the closed-form band/bit-plane mask for k < G, a
 * third-party JPEG implementation in both directions, a double-precision inverse DCT within
 * +-1, constant-image closed forms, the colour cube against double precision.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_OK 0
#define ORC_E_ARG -1
#define ORC_E_FORMAT -2
#define ORC_E_CORRUPT -3
#define ORC_E_UNSUPPORTED -4

/* ------------------------------------------------------------------------- */
/* Record layout (little-endian "raw struct" metadata, paper Section 5)       */
/* ------------------------------------------------------------------------- */
static uint32_t rd32(const uint8_t* p) { return (uint32_t)p[0] | ((uint32_t)p[1] << 8) | ((uint32_t)p[2] << 16) | ((uint32_t)p[3] << 24); }
static uint64_t rd64(const uint8_t* p) { return (uint64_t)rd32(p) | ((uint64_t)rd32(p + 4) << 32); }

typedef struct { uint32_t N, G; uint64_t meta_off, index_off, data_off, total; } rec_hdr;

static int parse_hdr(const uint8_t* rec, size_t len, rec_hdr* h) {
    if (!rec || len < 64) return ORC_E_FORMAT;
    if (memcmp(rec, "PCR1", 4) != 0 || rd32(rec + 4) != 1) return ORC_E_FORMAT;
    h->N = rd32(rec + 8); h->G = rd32(rec + 12);
    h->meta_off = rd64(rec + 24); h->index_off = rd64(rec + 32); h->data_off = rd64(rec + 40); h->total = rd64(rec + 48);
    if (h->N == 0 || h->G == 0 || h->G > 64) return ORC_E_FORMAT;
    if (h->meta_off + 16ull * h->N > len) return ORC_E_FORMAT;
    if (h->index_off + 8ull * (h->G + 1) + 16ull * h->G * h->N > len) return ORC_E_FORMAT;
    return ORC_OK;
}

int oracle_record_info(const uint8_t* rec, size_t len, int* N, int* G) {
    rec_hdr h; int rc = parse_hdr(rec, len, &h);
    if (rc) return rc;
    *N = (int)h.N; *G = (int)h.G;
    return ORC_OK;
}

int oracle_image_info(const uint8_t* rec, size_t len, int i, uint32_t* W, uint32_t* H, int32_t* label) {
    rec_hdr h; int rc = parse_hdr(rec, len, &h);
    if (rc) return rc;
    if (i < 0 || (uint32_t)i >= h.N) return ORC_E_ARG;
    const uint8_t* m = rec + h.meta_off + 16ull * (uint32_t)i;
    *label = (int32_t)rd32(m); *W = rd32(m + 4); *H = rd32(m + 8);
    return ORC_OK;
}

/* bytes [0, end of scan group k): what a reader fetches for fidelity k (Section 3) */
long long oracle_prefix_bytes(const uint8_t* rec, size_t len, int k) {
    rec_hdr h; int rc = parse_hdr(rec, len, &h);
    if (rc) return rc;
    if (k < 1 || (uint32_t)k > h.G) return ORC_E_ARG;
    return (long long)rd64(rec + h.index_off + 8ull * (uint32_t)k);
}

/* Section 5, "Decoding": scans 1..k of image i, in order, then an EOI token.
 * `len` is how much of the record the caller has read; nothing at or beyond it is touched.
 * Returns the JPEG length, or a negative error; with out == NULL only the length. */
long long oracle_reassemble(const uint8_t* rec, size_t len, int i, int k, uint8_t* out, size_t cap) {
    rec_hdr h; int rc = parse_hdr(rec, len, &h);
    if (rc) return rc;
    if (i < 0 || (uint32_t)i >= h.N || k < 1 || (uint32_t)k > h.G) return ORC_E_ARG;
    const uint8_t* chunk = rec + h.index_off + 8ull * (h.G + 1);
    size_t n = 0;
    for (int g = 0; g < k; ++g) {
        const uint8_t* c = chunk + 16ull * ((uint64_t)g * h.N + (uint32_t)i);
        uint64_t off = rd64(c); uint32_t clen = rd32(c + 8);
        if (off + clen > len) return ORC_E_FORMAT;
        if (out) {
            if (n + clen + 2 > cap) return ORC_E_ARG;
            memcpy(out + n, rec + off, clen);
        }
        n += clen;
    }
    if (out) { out[n] = 0xFF; out[n + 1] = 0xD9; }
    return (long long)n + 2;
}

/* ------------------------------------------------------------------------- */
/* JPEG decoder state                                                         */
/* ------------------------------------------------------------------------- */
typedef struct {
    int defined;
    int mincode[17], maxcode[17], valptr[17];
    uint8_t huffval[256];
} htab;

typedef struct {
    int W, H, mx, my;
    int ncomp;
    int cid[3], hs[3], vs[3], tq[3];
    int bw[3], bh[3], ubw[3], ubh[3];
    size_t coff[3], nblocks;
    uint16_t q[4][64];      /* zigzag order, as stored in DQT */
    int qdef[4];
    htab dc[4], ac[4];
    int ri;
    int have_frame;
    int sequential;          /* frame header was SOF0: one interleaved scan carries whole blocks */
    int16_t* coef;          /* canonical layout: comp, block row, block col, zigzag */
} jdec;

/* zigzag position -> natural index: walk the anti-diagonals of the 8x8 grid,
 * alternating direction (T.81 Figure 5) */
static void zigzag_table(int zz[64]) {
    int r = 0, c = 0;
    for (int k = 0; k < 64; ++k) {
        zz[k] = r * 8 + c;
        if ((r + c) % 2 == 0) {            /* moving up-right */
            if (c == 7) ++r; else if (r == 0) ++c; else { --r; ++c; }
        } else {                           /* moving down-left */
            if (r == 7) ++c; else if (c == 0) ++r; else { ++r; --c; }
        }
    }
}

/* T.81 Annex C: code lengths -> canonical codes; F.2.2.3 decoder tables */
static int build_htab(htab* t, const uint8_t bits[17], const uint8_t* vals, int nvals) {
    int code = 0, p = 0;
    for (int l = 1; l <= 16; ++l) {
        if (bits[l] == 0) { t->maxcode[l] = -1; t->mincode[l] = 0; t->valptr[l] = p; }
        else {
            t->valptr[l] = p; t->mincode[l] = code;
            code += bits[l]; p += bits[l];
            t->maxcode[l] = code - 1;
            if (code > (1 << l)) return ORC_E_CORRUPT;
        }
        code <<= 1;
    }
    if (p != nvals) return ORC_E_CORRUPT;
    memcpy(t->huffval, vals, (size_t)nvals);
    t->defined = 1;
    return ORC_OK;
}

/* entropy-coded segment reader: one bit at a time, MSB first, FF00 -> FF */
typedef struct { const uint8_t* d; size_t pos, end; int cur, left; int starved; } bitr;

static int next_bit(bitr* b) {
    if (b->left == 0) {
        if (b->pos >= b->end) { b->starved = 1; return 0; }
        int v = b->d[b->pos];
        if (v == 0xFF) {
            if (b->pos + 1 < b->end && b->d[b->pos + 1] == 0x00) b->pos += 2;
            else { b->starved = 1; return 0; }      /* a marker: no more data in this interval */
        } else b->pos += 1;
        b->cur = v; b->left = 8;
    }
    --b->left;
    return (b->cur >> b->left) & 1;
}
static int receive(bitr* b, int n) { int v = 0; for (int i = 0; i < n; ++i) v = (v << 1) | next_bit(b); return v; }
static int extend(int v, int n) { return n == 0 ? 0 : (v < (1 << (n - 1)) ? v - (1 << n) + 1 : v); }
static int decode_sym(bitr* b, const htab* t, int* err) {
    int code = 0;
    for (int l = 1; l <= 16; ++l) {
        code = (code << 1) | next_bit(b);
        if (t->maxcode[l] >= 0 && code <= t->maxcode[l] && code >= t->mincode[l])
            return t->huffval[t->valptr[l] + code - t->mincode[l]];
    }
    *err = 1;
    return 0;
}

/* one successive-approximation correction of an already non-zero coefficient (G.1.2.3) */
static void correct(bitr* b, int16_t* c, int p1) {
    if (next_bit(b)) {
        if ((*c & p1) == 0) *c = (int16_t)(*c >= 0 ? *c + p1 : *c - p1);
    }
}

typedef struct { int ns; int ci[3]; int td[3], ta[3]; int Ss, Se, Ah, Al; } scan_hdr;

static int decode_scan(jdec* J, const scan_hdr* S, const uint8_t* data, size_t n, size_t* used) {
    int inter = S->ns > 1;
    int c0 = S->ci[0];
    int mcu_w = inter ? J->mx : J->ubw[c0];
    int mcu_h = inter ? J->my : J->ubh[c0];
    long total = (long)mcu_w * mcu_h;
    int pred[3] = {0, 0, 0};
    int eobrun = 0, err = 0;
    int p1 = 1 << S->Al;
    int rst_expect = 0;
    bitr b = {data, 0, n, 0, 0, 0};
    for (long m = 0; m < total; ++m) {
        if (J->ri && m > 0 && m % J->ri == 0) {
            /* restart: drop the padding bits, require RSTm, reset predictors and the EOB run */
            if (b.starved) return ORC_E_CORRUPT;
            b.left = 0;
            if (b.pos + 2 > b.end || b.d[b.pos] != 0xFF || b.d[b.pos + 1] != 0xD0 + rst_expect) return ORC_E_CORRUPT;
            b.pos += 2; rst_expect = (rst_expect + 1) & 7; b.starved = 0;
            pred[0] = pred[1] = pred[2] = 0; eobrun = 0;
        }
        int mrow = (int)(m / mcu_w), mcol = (int)(m % mcu_w);
        for (int si = 0; si < S->ns; ++si) {
            int c = S->ci[si];
            int nh = inter ? J->hs[c] : 1, nv = inter ? J->vs[c] : 1;
            for (int by = 0; by < nv; ++by)
                for (int bx = 0; bx < nh; ++bx) {
                    size_t brow = (size_t)mrow * nv + by, bcol = (size_t)mcol * nh + bx;
                    int16_t* blk = J->coef + (J->coff[c] + brow * J->bw[c] + bcol) * 64;
                    if (S->Ss == 0 && S->Se == 63) {
                        /* sequential DCT scan (F.2.2): the block's DC difference, then its AC
                         * coefficients as (run, size) symbols up to an end-of-block symbol */
                        int s0 = decode_sym(&b, &J->dc[S->td[si]], &err);
                        if (s0 > 15) err = 1;
                        pred[c] += extend(receive(&b, s0), s0);
                        blk[0] = (int16_t)pred[c];
                        int k = 1;
                        while (k <= 63 && !err) {
                            int rs = decode_sym(&b, &J->ac[S->ta[si]], &err);
                            int r = rs >> 4, s = rs & 15;
                            if (s != 0) {
                                k += r;
                                if (k > 63) { err = 1; break; }
                                blk[k] = (int16_t)extend(receive(&b, s), s);
                                ++k;
                            } else if (r == 15) k += 16;
                            else if (r == 0) break;                    /* end of block */
                            else { err = 1; break; }                   /* end-of-band runs exist in progressive scans only */
                        }
                    } else if (S->Ss == 0) {
                        if (S->Ah == 0) {                              /* DC first (G.2.1) */
                            int s = decode_sym(&b, &J->dc[S->td[si]], &err);
                            if (s > 15) err = 1;
                            int d = extend(receive(&b, s), s);
                            pred[c] += d;
                            blk[0] = (int16_t)(pred[c] * p1);
                        } else if (next_bit(&b)) blk[0] |= (int16_t)p1;  /* DC refine (G.2.1) */
                    } else if (S->Ah == 0) {                           /* AC first (G.2.2) */
                        if (eobrun > 0) { --eobrun; continue; }
                        int k = S->Ss;
                        while (k <= S->Se) {
                            int rs = decode_sym(&b, &J->ac[S->ta[si]], &err);
                            int r = rs >> 4, s = rs & 15;
                            if (s != 0) {
                                k += r;
                                if (k > S->Se) { err = 1; break; }
                                blk[k] = (int16_t)(extend(receive(&b, s), s) * p1);
                                ++k;
                            } else if (r == 15) k += 16;
                            else { eobrun = (1 << r) + (r ? receive(&b, r) : 0) - 1; break; }
                        }
                    } else {                                           /* AC refine (G.2.3) */
                        int k = S->Ss;
                        if (eobrun == 0) {
                            while (k <= S->Se) {
                                int rs = decode_sym(&b, &J->ac[S->ta[si]], &err);
                                int r = rs >> 4, s = rs & 15, newval = 0;
                                if (s != 0) {
                                    if (s != 1) err = 1;
                                    newval = next_bit(&b) ? p1 : -p1;
                                } else if (r < 15) {
                                    eobrun = (1 << r) + (r ? receive(&b, r) : 0);
                                    break;
                                }
                                while (k <= S->Se) {
                                    if (blk[k] != 0) correct(&b, &blk[k], p1);
                                    else if (r == 0) break;
                                    else --r;
                                    ++k;
                                }
                                if (s != 0 && k <= S->Se) blk[k] = (int16_t)newval;
                                ++k;
                            }
                        }
                        if (eobrun > 0) {
                            for (; k <= S->Se; ++k) if (blk[k] != 0) correct(&b, &blk[k], p1);
                            --eobrun;
                        }
                    }
                    if (err) return ORC_E_CORRUPT;
                }
        }
    }
    if (b.starved) return ORC_E_CORRUPT;
    *used = b.pos;
    return ORC_OK;
}

/* T.81 A.1.1 / A.2: component c has ceil(W * Hc / Hmax) x ceil(H * Vc / Vmax) samples; an
 * interleaved MCU holds Hc x Vc blocks of it, so the MCU-padded grid is (mx * Hc) x (my * Vc) blocks
 * with mx = ceil(W / (8 Hmax)).  A frame with one component is never interleaved: its grid is the
 * unpadded one and its sampling factors play no role (taken as 1 x 1). */
static void set_geometry(jdec* J) {
    int hmax = 1, vmax = 1;
    if (J->ncomp == 1) { J->hs[0] = 1; J->vs[0] = 1; }
    for (int c = 0; c < J->ncomp; ++c) { if (J->hs[c] > hmax) hmax = J->hs[c]; if (J->vs[c] > vmax) vmax = J->vs[c]; }
    J->mx = (J->W + 8 * hmax - 1) / (8 * hmax); J->my = (J->H + 8 * vmax - 1) / (8 * vmax);
    size_t off = 0;
    for (int c = 0; c < 3; ++c) {
        if (c >= J->ncomp) { J->bw[c] = J->bh[c] = J->ubw[c] = J->ubh[c] = 0; J->coff[c] = off; continue; }
        J->bw[c] = J->mx * J->hs[c]; J->bh[c] = J->my * J->vs[c];
        int wc = (J->W * J->hs[c] + hmax - 1) / hmax, hc = (J->H * J->vs[c] + vmax - 1) / vmax;
        J->ubw[c] = (wc + 7) / 8; J->ubh[c] = (hc + 7) / 8;
        J->coff[c] = off; off += (size_t)J->bw[c] * J->bh[c];
    }
    J->nblocks = off;
}

/* Walk the marker segments of a (possibly truncated-and-EOI-terminated) progressive file. */
static int jpeg_decode_coeffs(jdec* J, const uint8_t* d, size_t n, int16_t* coef, size_t ncoef) {
    memset(J, 0, sizeof *J);
    size_t p = 0;
    if (n < 4 || d[0] != 0xFF || d[1] != 0xD8) return ORC_E_FORMAT;
    p = 2;
    for (;;) {
        if (p + 2 > n) return ORC_E_CORRUPT;       /* ran out without an EOI */
        if (d[p] != 0xFF) return ORC_E_CORRUPT;
        while (p < n && d[p] == 0xFF) ++p;          /* fill bytes */
        if (p >= n) return ORC_E_CORRUPT;
        int mk = d[p++];
        if (mk == 0xD9) break;                      /* EOI */
        if (p + 2 > n) return ORC_E_CORRUPT;
        size_t L = ((size_t)d[p] << 8) | d[p + 1];
        if (L < 2 || p + L > n) return ORC_E_CORRUPT;
        const uint8_t* s = d + p + 2; size_t sl = L - 2;
        if (mk == 0xDB) {                           /* DQT */
            size_t q = 0;
            while (q < sl) {
                int pq = s[q] >> 4, tq = s[q] & 15; ++q;
                if (tq > 3 || pq > 1 || q + (pq ? 128 : 64) > sl) return ORC_E_CORRUPT;
                for (int k = 0; k < 64; ++k) {
                    J->q[tq][k] = pq ? (uint16_t)((s[q] << 8) | s[q + 1]) : s[q];
                    q += pq ? 2 : 1;
                }
                J->qdef[tq] = 1;
            }
        } else if (mk == 0xC2 || mk == 0xC0) {      /* SOF2: progressive, Huffman; SOF0: baseline sequential */
            J->sequential = mk == 0xC0;
            if (sl < 6 || s[0] != 8) return ORC_E_UNSUPPORTED;
            J->H = (s[1] << 8) | s[2]; J->W = (s[3] << 8) | s[4]; J->ncomp = s[5];
            if ((J->ncomp != 3 && J->ncomp != 1) || sl < (size_t)(6 + 3 * J->ncomp) || J->W == 0 || J->H == 0) return ORC_E_UNSUPPORTED;
            for (int c = 0; c < J->ncomp; ++c) {
                J->cid[c] = s[6 + 3 * c]; J->hs[c] = s[7 + 3 * c] >> 4; J->vs[c] = s[7 + 3 * c] & 15; J->tq[c] = s[8 + 3 * c];
                if (J->tq[c] > 3) return ORC_E_CORRUPT;
                if (J->hs[c] < 1 || J->hs[c] > 2 || J->vs[c] < 1 || J->vs[c] > 2) return ORC_E_UNSUPPORTED;
            }
            /* luminance 1 or 2 blocks per MCU in each direction, chroma one block: 4:4:4, 4:2:2, 4:4:0, 4:2:0, grey */
            if (J->ncomp == 3 && (J->hs[1] != 1 || J->vs[1] != 1 || J->hs[2] != 1 || J->vs[2] != 1)) return ORC_E_UNSUPPORTED;
            set_geometry(J);
            if (J->nblocks * 64 != ncoef) return ORC_E_ARG;
            J->coef = coef;
            memset(coef, 0, ncoef * sizeof(int16_t));
            J->have_frame = 1;
        } else if (mk == 0xC1 || (mk >= 0xC3 && mk <= 0xCF && mk != 0xC4 && mk != 0xC8 && mk != 0xCC)) {
            return ORC_E_UNSUPPORTED;               /* other frame types */
        } else if (mk == 0xC4) {                    /* DHT */
            size_t q = 0;
            while (q < sl) {
                if (q + 17 > sl) return ORC_E_CORRUPT;
                int tc = s[q] >> 4, th = s[q] & 15;
                if (tc > 1 || th > 3) return ORC_E_CORRUPT;
                uint8_t bits[17]; int nv = 0; bits[0] = 0;
                for (int l = 1; l <= 16; ++l) { bits[l] = s[q + l]; nv += bits[l]; }
                if (nv > 256 || q + 17 + (size_t)nv > sl) return ORC_E_CORRUPT;
                int rc = build_htab(tc ? &J->ac[th] : &J->dc[th], bits, s + q + 17, nv);
                if (rc) return rc;
                q += 17 + (size_t)nv;
            }
        } else if (mk == 0xDD) {                    /* DRI */
            if (sl != 2) return ORC_E_CORRUPT;
            J->ri = (s[0] << 8) | s[1];
        } else if (mk == 0xDA) {                    /* SOS */
            if (!J->have_frame) return ORC_E_CORRUPT;
            scan_hdr S; memset(&S, 0, sizeof S);
            if (sl < 1) return ORC_E_CORRUPT;
            S.ns = s[0];
            if (S.ns < 1 || S.ns > 3 || sl != (size_t)(4 + 2 * S.ns)) return ORC_E_CORRUPT;
            for (int i = 0; i < S.ns; ++i) {
                int id = s[1 + 2 * i], found = -1;
                for (int c = 0; c < J->ncomp; ++c) if (J->cid[c] == id) found = c;
                if (found < 0) return ORC_E_CORRUPT;
                S.ci[i] = found; S.td[i] = s[2 + 2 * i] >> 4; S.ta[i] = s[2 + 2 * i] & 15;
                if (S.td[i] > 3 || S.ta[i] > 3) return ORC_E_CORRUPT;
            }
            S.Ss = s[1 + 2 * S.ns]; S.Se = s[2 + 2 * S.ns]; S.Ah = s[3 + 2 * S.ns] >> 4; S.Al = s[3 + 2 * S.ns] & 15;
            if (S.Ss > S.Se || S.Se > 63 || S.Al > 13) return ORC_E_CORRUPT;
            if (J->sequential) {                                   /* one kind of scan: everything of its components */
                if (S.Ss != 0 || S.Se != 63 || S.Ah != 0 || S.Al != 0 || S.ns != J->ncomp) return ORC_E_UNSUPPORTED;
                for (int i = 0; i < S.ns; ++i)
                    if (!J->dc[S.td[i]].defined || !J->ac[S.ta[i]].defined) return ORC_E_CORRUPT;
            } else if (S.Ss == 0 && S.Se != 0) return ORC_E_CORRUPT;  /* DC and AC never share a progressive scan */
            if (S.Ss > 0 && S.ns != 1) return ORC_E_CORRUPT;       /* AC scans hold one component */
            if (S.Ah != 0 && S.Ah != S.Al + 1) return ORC_E_CORRUPT;
            for (int i = 0; i < S.ns; ++i) {
                if (S.Ss == 0 && S.Ah == 0 && !J->dc[S.td[i]].defined) return ORC_E_CORRUPT;
                if (S.Ss > 0 && !J->ac[S.ta[i]].defined) return ORC_E_CORRUPT;
            }
            size_t used = 0;
            int rc = decode_scan(J, &S, d + p + L, n - (p + L), &used);
            if (rc) return rc;
            p += L + used;
            continue;
        } else if (mk >= 0xD0 && mk <= 0xD7) {
            return ORC_E_CORRUPT;                   /* a restart marker outside a scan */
        }
        /* APPn, COM and anything else with a length: skipped */
        p += L;
    }
    if (!J->have_frame) return ORC_E_CORRUPT;
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Pixels from coefficients                                                   */
/* ------------------------------------------------------------------------- */
/* 8-point inverse DCT basis in 13-bit fixed point, straight from the definition
 * x(n) = 1/2 * sum_k c_k X(k) cos((2n+1) k pi / 16),  c_0 = 1/sqrt 2:
 * M[n][k] = round(8192 * c_k * cos((2n+1) k pi / 16)); the factor 1/2 of each pass is
 * folded into the rounding shifts below. */
static int32_t IDCT_M[8][8];
static int ZZT[64];
static int consts_ready = 0;
static void init_consts(void) {
    if (consts_ready) return;
    const double pi = 3.14159265358979323846;
    for (int n = 0; n < 8; ++n)
        for (int k = 0; k < 8; ++k)
            IDCT_M[n][k] = (int32_t)lround(8192.0 * (k == 0 ? sqrt(0.5) : 1.0) * cos((2 * n + 1) * k * pi / 16.0));
    zigzag_table(ZZT);
    consts_ready = 1;
}

static int32_t wrap32(int64_t v) { return (int32_t)(uint32_t)(uint64_t)v; }

/* one block: zigzag int16 coefficients x zigzag quantiser -> 64 samples, natural order */
static void block_to_samples(const int16_t* coef, const uint16_t* q, uint8_t out[64]) {
    int32_t F[64], T[64];
    for (int k = 0; k < 64; ++k) F[ZZT[k]] = wrap32((int64_t)coef[k] * q[k]);
    /* pass 1: along the vertical frequency index v of every column u; 2 extra fraction bits kept */
    for (int u = 0; u < 8; ++u)
        for (int y = 0; y < 8; ++y) {
            int64_t acc = 0;
            for (int v = 0; v < 8; ++v) acc += (int64_t)IDCT_M[y][v] * F[v * 8 + u];
            T[y * 8 + u] = wrap32((int64_t)wrap32(acc) + 2048) >> 12;
        }
    /* pass 2: along the horizontal frequency index u of every row y */
    for (int y = 0; y < 8; ++y)
        for (int x = 0; x < 8; ++x) {
            int64_t acc = 0;
            for (int u = 0; u < 8; ++u) acc += (int64_t)IDCT_M[x][u] * T[y * 8 + u];
            int32_t s = (wrap32((int64_t)wrap32(acc) + 32768) >> 16) + 128;
            out[y * 8 + x] = (uint8_t)(s < 0 ? 0 : (s > 255 ? 255 : s));
        }
}

static uint8_t clamp8(int v) { return (uint8_t)(v < 0 ? 0 : (v > 255 ? 255 : v)); }

/* full-range BT.601 (JFIF) in 16-bit fixed point, round half up */
static void ycc_to_rgb(int Y, int cb, int cr, uint8_t* rgb) {
    cb -= 128; cr -= 128;
    rgb[0] = clamp8(Y + ((91881 * cr + 32768) >> 16));
    rgb[1] = clamp8(Y + ((-22553 * cb - 46802 * cr + 32768) >> 16));
    rgb[2] = clamp8(Y + ((116130 * cb + 32768) >> 16));
}
void oracle_ycc_to_rgb(int Y, int cb, int cr, uint8_t* rgb) { ycc_to_rgb(Y, cb, cr, rgb); }
void oracle_ycc_to_rgb_array(const uint8_t* ycc, size_t n, uint8_t* rgb) {
    for (size_t i = 0; i < n; ++i) ycc_to_rgb(ycc[3 * i], ycc[3 * i + 1], ycc[3 * i + 2], rgb + 3 * i);
}

/* coefficients (canonical layout) + per-component zigzag quantisers -> packed RGB (H*W*3).
 * hs x vs: luminance blocks per MCU (chroma has one), ncomp 3 or 1.  Pixel (x, y) takes the
 * chroma sample (x / hs, y / vs) (replication); a greyscale image has no chroma: every pixel is
 * (Y, Y, Y), which is what the colour formula gives for Cb = Cr = 128.
 * planes, if not NULL, receives the sample planes over the padded grids
 * (Y: 8 hs mx x 8 vs my, then Cb and Cr: 8mx x 8my each). */
int oracle_pixels_from_coeffs_s(const int16_t* coef, uint32_t W, uint32_t H, int hs, int vs, int ncomp, const uint16_t* qy,
                                const uint16_t* qcb, const uint16_t* qcr, uint8_t* rgb, uint8_t* planes) {
    init_consts();
    if (!coef || W == 0 || H == 0 || (ncomp != 1 && ncomp != 3) || hs < 1 || hs > 2 || vs < 1 || vs > 2) return ORC_E_ARG;
    if (ncomp == 1) { hs = 1; vs = 1; }
    int mx = (int)((W + 8 * hs - 1) / (8 * hs)), my = (int)((H + 8 * vs - 1) / (8 * vs));
    int bw[3] = {hs * mx, mx, mx}, bh[3] = {vs * my, my, my};
    size_t psz[3] = {(size_t)64 * bw[0] * bh[0], (size_t)64 * mx * my, (size_t)64 * mx * my};
    if (ncomp == 1) psz[1] = psz[2] = 0;
    uint8_t* own = planes ? NULL : (uint8_t*)malloc(psz[0] + psz[1] + psz[2]);
    uint8_t* pl[3]; pl[0] = planes ? planes : own; pl[1] = pl[0] + psz[0]; pl[2] = pl[1] + psz[1];
    const uint16_t* q[3] = {qy, qcb, qcr};
    size_t boff = 0;
    for (int c = 0; c < ncomp; ++c) {
        int pw = bw[c] * 8;
        for (int by = 0; by < bh[c]; ++by)
            for (int bx = 0; bx < bw[c]; ++bx) {
                uint8_t s[64];
                block_to_samples(coef + (boff + (size_t)by * bw[c] + bx) * 64, q[c], s);
                for (int y = 0; y < 8; ++y)
                    memcpy(pl[c] + (size_t)(by * 8 + y) * pw + bx * 8, s + y * 8, 8);
            }
        boff += (size_t)bw[c] * bh[c];
    }
    if (rgb) {
        int yw = 8 * bw[0], cw = 8 * mx;
        for (uint32_t y = 0; y < H; ++y)
            for (uint32_t x = 0; x < W; ++x) {
                int Yv = pl[0][(size_t)y * yw + x];
                int cb = 128, cr = 128;
                if (ncomp == 3) {
                    cb = pl[1][(size_t)(y / (uint32_t)vs) * cw + (x / (uint32_t)hs)];   /* replication */
                    cr = pl[2][(size_t)(y / (uint32_t)vs) * cw + (x / (uint32_t)hs)];
                }
                ycc_to_rgb(Yv, cb, cr, rgb + ((size_t)y * W + x) * 3);
            }
    }
    free(own);
    return ORC_OK;
}

int oracle_pixels_from_coeffs(const int16_t* coef, uint32_t W, uint32_t H, const uint16_t* qy, const uint16_t* qcb,
                              const uint16_t* qcr, uint8_t* rgb, uint8_t* planes) {
    return oracle_pixels_from_coeffs_s(coef, W, H, 2, 2, 3, qy, qcb, qcr, rgb, planes);
}

/* A progressive JPEG byte string -> coefficients (+ optional RGB and planes).
 * ncoef must equal 64 * blocks of the padded grids.  W/H are returned. */
int oracle_jpeg_decode(const uint8_t* jpg, size_t n, int16_t* coef, size_t ncoef, uint8_t* rgb, uint8_t* planes,
                       uint32_t* W, uint32_t* H) {
    init_consts();
    jdec* J = (jdec*)malloc(sizeof *J);
    int rc = jpeg_decode_coeffs(J, jpg, n, coef, ncoef);
    if (rc == ORC_OK) {
        if (W) *W = (uint32_t)J->W;
        if (H) *H = (uint32_t)J->H;
        for (int c = 0; c < J->ncomp; ++c) if (!J->qdef[J->tq[c]]) rc = ORC_E_CORRUPT;
        if (rc == ORC_OK && (rgb || planes))
            rc = oracle_pixels_from_coeffs_s(coef, (uint32_t)J->W, (uint32_t)J->H, J->hs[0], J->vs[0], J->ncomp, J->q[J->tq[0]],
                                             J->q[J->tq[J->ncomp == 3 ? 1 : 0]], J->q[J->tq[J->ncomp == 3 ? 2 : 0]], rgb, planes);
    }
    free(J);
    return rc;
}

/* frame size, luminance sampling and component count of a JPEG byte string (reads up to the frame header) */
int oracle_jpeg_info(const uint8_t* d, size_t n, uint32_t* W, uint32_t* H, int* hs, int* vs, int* ncomp) {
    size_t p = 2;
    if (n < 4 || d[0] != 0xFF || d[1] != 0xD8) return ORC_E_FORMAT;
    while (p + 4 <= n) {
        if (d[p] != 0xFF) return ORC_E_CORRUPT;
        int mk = d[p + 1];
        if (mk == 0xFF) { ++p; continue; }
        size_t L = ((size_t)d[p + 2] << 8) | d[p + 3];
        if (mk == 0xC2 || mk == 0xC0) {
            if (p + 12 > n) return ORC_E_CORRUPT;
            *H = ((uint32_t)d[p + 5] << 8) | d[p + 6]; *W = ((uint32_t)d[p + 7] << 8) | d[p + 8];
            *ncomp = d[p + 9];
            *hs = *ncomp == 1 ? 1 : d[p + 11] >> 4; *vs = *ncomp == 1 ? 1 : d[p + 11] & 15;
            return ORC_OK;
        }
        if (mk == 0xDA || mk == 0xD9) break;
        p += 2 + L;
    }
    return ORC_E_FORMAT;
}

size_t oracle_num_blocks_s(uint32_t W, uint32_t H, int hs, int vs, int ncomp) {
    if (ncomp == 1) { hs = 1; vs = 1; }
    size_t mx = (W + 8 * (uint32_t)hs - 1) / (8 * (uint32_t)hs), my = (H + 8 * (uint32_t)vs - 1) / (8 * (uint32_t)vs);
    return ((size_t)hs * vs + (ncomp == 3 ? 2 : 0)) * mx * my;
}

/* frame size of a JPEG byte string without decoding it (reads up to the SOF2 segment) */
int oracle_jpeg_dims(const uint8_t* d, size_t n, uint32_t* W, uint32_t* H) {
    size_t p = 2;
    if (n < 4 || d[0] != 0xFF || d[1] != 0xD8) return ORC_E_FORMAT;
    while (p + 4 <= n) {
        if (d[p] != 0xFF) return ORC_E_CORRUPT;
        int mk = d[p + 1];
        if (mk == 0xFF) { ++p; continue; }
        size_t L = ((size_t)d[p + 2] << 8) | d[p + 3];
        if (mk == 0xC2 || mk == 0xC0) {
            if (p + 9 > n) return ORC_E_CORRUPT;
            *H = ((uint32_t)d[p + 5] << 8) | d[p + 6]; *W = ((uint32_t)d[p + 7] << 8) | d[p + 8];
            return ORC_OK;
        }
        if (mk == 0xDA || mk == 0xD9) break;
        p += 2 + L;
    }
    return ORC_E_FORMAT;
}

/* Image i of a record at fidelity k: reassemble as the paper's decoder does, then decode.
 * Only bytes below the end of scan group k are read. */
int oracle_decode_image(const uint8_t* rec, size_t len, int i, int k, int16_t* coef, size_t ncoef, uint8_t* rgb) {
    long long pre = oracle_prefix_bytes(rec, len, k);
    if (pre < 0) return (int)pre;
    if ((size_t)pre > len) return ORC_E_FORMAT;
    long long need = oracle_reassemble(rec, (size_t)pre, i, k, NULL, 0);
    if (need < 0) return (int)need;
    uint8_t* tmp = (uint8_t*)malloc((size_t)need);
    long long n = oracle_reassemble(rec, (size_t)pre, i, k, tmp, (size_t)need);
    int rc;
    if (n < 0) rc = (int)n;
    else rc = oracle_jpeg_decode(tmp, (size_t)n, coef, ncoef, rgb, NULL, NULL, NULL);
    free(tmp);
    return rc;
}

size_t oracle_num_blocks(uint32_t W, uint32_t H) {
    size_t mx = (W + 15) / 16, my = (H + 15) / 16;
    return 6 * mx * my;
}

/* the inverse DCT of one block alone (for the double-precision pin) */
void oracle_block_idct(const int16_t coef[64], const uint16_t q[64], uint8_t out[64]) {
    init_consts();
    block_to_samples(coef, q, out);
}
