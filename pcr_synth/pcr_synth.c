/*
 * pcr_synth — seeded synthetic inputs for the PCR decode path.
 *
 * This file makes the INPUTS only: synthetic images, their quantised DCT
 * coefficients (the ground truth of every test), a progressive-JPEG encoder
 * that serialises those coefficients with a scan script, and a writer that lays
 * the per-image scans out as a Progressive Compressed Record (metadata first,
 * then scan group 1 of every image, scan group 2 of every image, ... as in the
 * paper's Section 3 and its record-layout figure).
 *
 * It holds nothing of the decode path: no Huffman decoding, no inverse DCT, no
 * colour conversion.  Both the CPU oracle and the CUDA library consume the
 * bytes produced here; neither shares code with this file.
 *
 * The bit-level stream syntax is ITU-T T.81 (progressive, Huffman, 8-bit),
 * which the paper relies on through its JPEG citations.
 */
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define PI 3.14159265358979323846

/* ------------------------------------------------------------------------- */
/* Random numbers: splitmix64 stream, Box-Muller normals                      */
/* ------------------------------------------------------------------------- */
typedef struct { uint64_t s; int have; double spare; } rng_t;

static uint64_t rng_u64(rng_t* r) {
    uint64_t z = (r->s += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
static double rng_unit(rng_t* r) { return (double)(rng_u64(r) >> 11) * (1.0 / 9007199254740992.0); }
static double rng_range(rng_t* r, double a, double b) { return a + (b - a) * rng_unit(r); }
static double rng_normal(rng_t* r) {
    if (r->have) { r->have = 0; return r->spare; }
    double u1 = 1.0 - rng_unit(r), u2 = rng_unit(r);
    double m = sqrt(-2.0 * log(u1));
    r->spare = m * sin(2.0 * PI * u2);
    r->have = 1;
    return m * cos(2.0 * PI * u2);
}

/* ------------------------------------------------------------------------- */
/* Public structs                                                             */
/* ------------------------------------------------------------------------- */
typedef struct {
    uint32_t width, height;
    int32_t label;
    int32_t quality;   /* 1..100, scales the Annex K base tables              */
    double beta;       /* sinusoid amplitude ~ f^-beta                          */
    double gamma;      /* weight of the per-channel colour fields               */
    double sigma;      /* i.i.d. Gaussian pixel noise                           */
    int32_t blobs;     /* 1: add smooth elliptical luminance blobs              */
    int32_t rsvd;
    uint64_t seed;
} synth_image_spec;

/* Chroma sampling of the images made from here on (process-wide, like the scan script): the
 * luminance component has hs x vs blocks per MCU, the chroma components one each; ncomp = 1 makes
 * greyscale images (one component, no MCU padding: a lone component is never interleaved). */
static int g_hs = 2, g_vs = 2, g_nc = 3;
int synth_set_sampling(int hs, int vs, int ncomp) {
    if ((hs != 1 && hs != 2) || (vs != 1 && vs != 2) || (ncomp != 1 && ncomp != 3)) return -1;
    g_hs = ncomp == 1 ? 1 : hs; g_vs = ncomp == 1 ? 1 : vs; g_nc = ncomp;
    return 0;
}

typedef struct {
    int W, H, mx, my;
    int hs, vs, nc;       /* luminance blocks per MCU (horizontal, vertical), components */
    int bw[3], bh[3];     /* padded block grid per component                    */
    int ubw[3], ubh[3];   /* unpadded block grid per component                  */
    size_t coff[3];       /* first block of each component in the image array   */
    size_t nblocks;
} geom_t;

static void geom_init(geom_t* g, int W, int H) {
    g->W = W; g->H = H;
    g->hs = g_hs; g->vs = g_vs; g->nc = g_nc;
    g->mx = (W + 8 * g->hs - 1) / (8 * g->hs); g->my = (H + 8 * g->vs - 1) / (8 * g->vs);
    g->bw[0] = g->hs * g->mx; g->bh[0] = g->vs * g->my;
    g->bw[1] = g->bw[2] = g->nc == 3 ? g->mx : 0; g->bh[1] = g->bh[2] = g->nc == 3 ? g->my : 0;
    g->ubw[0] = (W + 7) / 8; g->ubh[0] = (H + 7) / 8;
    int cw = (W + g->hs - 1) / g->hs, ch = (H + g->vs - 1) / g->vs;
    g->ubw[1] = g->ubw[2] = g->nc == 3 ? (cw + 7) / 8 : 0; g->ubh[1] = g->ubh[2] = g->nc == 3 ? (ch + 7) / 8 : 0;
    g->coff[0] = 0;
    g->coff[1] = (size_t)g->bw[0] * g->bh[0];
    g->coff[2] = g->coff[1] + (size_t)g->bw[1] * g->bh[1];
    g->nblocks = g->coff[2] + (size_t)g->bw[2] * g->bh[2];
}

/* zigzag position -> natural (row-major) index, built by walking anti-diagonals */
static int ZZ[64];
static double COSM[8][8];   /* COSM[u][x] = c_u/2 * cos((2x+1)u*pi/16) */
static int tables_ready = 0;
static void init_tables(void) {
    if (tables_ready) return;
    int n = 0;
    for (int d = 0; d < 15; ++d) {
        if (d & 1) { for (int r = (d < 8 ? 0 : d - 7); r <= (d < 8 ? d : 7); ++r) ZZ[n++] = r * 8 + (d - r); }
        else       { for (int r = (d < 8 ? d : 7); r >= (d < 8 ? 0 : d - 7); --r) ZZ[n++] = r * 8 + (d - r); }
    }
    for (int u = 0; u < 8; ++u)
        for (int x = 0; x < 8; ++x)
            COSM[u][x] = (u == 0 ? sqrt(0.5) : 1.0) * 0.5 * cos((2 * x + 1) * u * PI / 16.0);
    tables_ready = 1;
}

/* T.81 Annex K example quantisation tables (natural order) */
static const uint8_t BASE_LUMA[64] = {
    16, 11, 10, 16, 24, 40, 51, 61,   12, 12, 14, 19, 26, 58, 60, 55,
    14, 13, 16, 24, 40, 57, 69, 56,   14, 17, 22, 29, 51, 87, 80, 62,
    18, 22, 37, 56, 68, 109, 103, 77, 24, 35, 55, 64, 81, 104, 113, 92,
    49, 64, 78, 87, 103, 121, 120, 101, 72, 92, 95, 98, 112, 100, 103, 99};
static const uint8_t BASE_CHROMA[64] = {
    17, 18, 24, 47, 99, 99, 99, 99,   18, 21, 26, 66, 99, 99, 99, 99,
    24, 26, 56, 99, 99, 99, 99, 99,   47, 66, 99, 99, 99, 99, 99, 99,
    99, 99, 99, 99, 99, 99, 99, 99,   99, 99, 99, 99, 99, 99, 99, 99,
    99, 99, 99, 99, 99, 99, 99, 99,   99, 99, 99, 99, 99, 99, 99, 99};

/* quality -> scaled table (natural order), the usual 200-2q / 5000/q rule */
void synth_quant_table(int quality, int chroma, uint8_t out[64]) {
    if (quality < 1) quality = 1;
    if (quality > 100) quality = 100;
    int s = quality < 50 ? 5000 / quality : 200 - 2 * quality;
    const uint8_t* base = chroma ? BASE_CHROMA : BASE_LUMA;
    for (int i = 0; i < 64; ++i) {
        int q = (base[i] * s + 50) / 100;
        if (q < 1) q = 1;
        if (q > 255) q = 255;
        out[i] = (uint8_t)q;
    }
}

/* ------------------------------------------------------------------------- */
/* Synthetic image: sum of sinusoids with 1/f^beta amplitudes, optional       */
/* elliptical blobs, per-channel colour fields, Gaussian noise                */
/* ------------------------------------------------------------------------- */
#define NSIN 8
typedef struct { double amp, fx, fy, phase; } wave_t;

static void make_field(rng_t* r, int W, int H, double beta, wave_t w[NSIN]) {
    double M = W > H ? W : H, m = W < H ? W : H;
    double fmax = m / 4.0; if (fmax < 1.0) fmax = 1.0;
    double power = 0.0;
    for (int j = 0; j < NSIN; ++j) {
        double f = exp(rng_range(r, 0.0, log(fmax)));
        double th = rng_range(r, 0.0, PI);
        w[j].phase = rng_range(r, 0.0, 2.0 * PI);
        w[j].amp = pow(f, -beta);
        w[j].fx = 2.0 * PI * f * cos(th) / M;
        w[j].fy = 2.0 * PI * f * sin(th) / M;
        power += 0.5 * w[j].amp * w[j].amp;
    }
    double scale = 40.0 / sqrt(power);
    for (int j = 0; j < NSIN; ++j) w[j].amp *= scale;
}

typedef struct { double cx, cy, ax, ay, ct, st, amp; } blob_t;

/* rgb: H*W*3 uint8, row-major */
void synth_image_rgb(const synth_image_spec* sp, uint8_t* rgb) {
    init_tables();
    int W = (int)sp->width, H = (int)sp->height;
    rng_t r = { sp->seed * 0x2545F4914F6CDD1Dull + 0x1234567ull, 0, 0.0 };
    wave_t fld[4][NSIN];
    for (int c = 0; c < 4; ++c) make_field(&r, W, H, sp->beta, fld[c]);
    blob_t blob[6]; int nblob = 0;
    if (sp->blobs) {
        nblob = 3 + (int)(rng_unit(&r) * 4.0); if (nblob > 6) nblob = 6;
        for (int b = 0; b < nblob; ++b) {
            blob[b].cx = rng_range(&r, 0.25, 0.75) * W;
            blob[b].cy = rng_range(&r, 0.25, 0.75) * H;
            blob[b].ax = rng_range(&r, 0.15, 0.45) * W;
            blob[b].ay = rng_range(&r, 0.15, 0.45) * H;
            double th = rng_range(&r, 0.0, PI);
            blob[b].ct = cos(th); blob[b].st = sin(th);
            blob[b].amp = (rng_unit(&r) < 0.5 ? -60.0 : 60.0);
        }
    }
    double* row = (double*)malloc(sizeof(double) * 4 * (size_t)W);
    for (int y = 0; y < H; ++y) {
        for (int i = 0; i < 4 * W; ++i) row[i] = 0.0;
        for (int c = 0; c < 4; ++c) {
            double* dst = row + (size_t)c * W;
            for (int j = 0; j < NSIN; ++j) {
                const wave_t* w = &fld[c][j];
                double p0 = w->fy * y + w->phase;
                double s = sin(p0), co = cos(p0), sd = sin(w->fx), cd = cos(w->fx);
                for (int x = 0; x < W; ++x) {
                    dst[x] += w->amp * s;
                    double ns = s * cd + co * sd;
                    co = co * cd - s * sd;
                    s = ns;
                }
            }
        }
        for (int x = 0; x < W; ++x) {
            double L = 128.0 + row[x];
            for (int b = 0; b < nblob; ++b) {
                double dx = x - blob[b].cx, dy = y - blob[b].cy;
                double u = (dx * blob[b].ct + dy * blob[b].st) / blob[b].ax;
                double v = (-dx * blob[b].st + dy * blob[b].ct) / blob[b].ay;
                L += blob[b].amp * exp(-0.5 * (u * u + v * v));
            }
            for (int c = 0; c < 3; ++c) {
                double v = L + sp->gamma * row[(size_t)(c + 1) * W + x] + sp->sigma * rng_normal(&r);
                double q = floor(v + 0.5);
                if (q < 0.0) q = 0.0;
                if (q > 255.0) q = 255.0;
                rgb[((size_t)y * W + x) * 3 + c] = (uint8_t)q;
            }
        }
    }
    free(row);
}

/* ------------------------------------------------------------------------- */
/* RGB -> quantised coefficients (canonical layout: comp, block row, block    */
/* col, zigzag position), all in double precision before the final rounding   */
/* ------------------------------------------------------------------------- */
static void fdct_quant_plane(const double* plane, int pw, int bw, int bh, const uint8_t q[64], int16_t* out) {
    for (int by = 0; by < bh; ++by)
        for (int bx = 0; bx < bw; ++bx) {
            double s[8][8], t[8][8];
            for (int y = 0; y < 8; ++y)
                for (int x = 0; x < 8; ++x) s[y][x] = plane[(size_t)(by * 8 + y) * pw + bx * 8 + x] - 128.0;
            for (int y = 0; y < 8; ++y)          /* rows: x -> u */
                for (int u = 0; u < 8; ++u) {
                    double a = 0.0;
                    for (int x = 0; x < 8; ++x) a += s[y][x] * COSM[u][x];
                    t[y][u] = a;
                }
            int16_t nat[64];
            for (int v = 0; v < 8; ++v)          /* columns: y -> v */
                for (int u = 0; u < 8; ++u) {
                    double a = 0.0;
                    for (int y = 0; y < 8; ++y) a += t[y][u] * COSM[v][y];
                    double c = a / q[v * 8 + u];
                    double rr = c < 0 ? -floor(-c + 0.5) : floor(c + 0.5);
                    int lim = (v == 0 && u == 0) ? 1023 : 1023;
                    if (rr > lim) rr = lim;
                    if (rr < -lim) rr = -lim;
                    nat[v * 8 + u] = (int16_t)rr;
                }
            int16_t* dst = out + ((size_t)by * bw + bx) * 64;
            for (int k = 0; k < 64; ++k) dst[k] = nat[ZZ[k]];
        }
}

void synth_rgb_to_coeffs(const uint8_t* rgb, int W, int H, const uint8_t qy[64], const uint8_t qc[64], int16_t* coef) {
    init_tables();
    geom_t g; geom_init(&g, W, H);
    int PW = 8 * g.hs * g.mx, PH = 8 * g.vs * g.my;
    double* Y = (double*)malloc(sizeof(double) * (size_t)PW * PH);
    double* Cb = (double*)malloc(sizeof(double) * (size_t)PW * PH);
    double* Cr = (double*)malloc(sizeof(double) * (size_t)PW * PH);
    for (int y = 0; y < PH; ++y) {
        int sy = y < H ? y : H - 1;
        for (int x = 0; x < PW; ++x) {
            int sx = x < W ? x : W - 1;
            const uint8_t* p = rgb + ((size_t)sy * W + sx) * 3;
            double R = p[0], G = p[1], B = p[2];
            Y[(size_t)y * PW + x] = 0.299 * R + 0.587 * G + 0.114 * B;
            Cb[(size_t)y * PW + x] = 128.0 - 0.168736 * R - 0.331264 * G + 0.5 * B;
            Cr[(size_t)y * PW + x] = 128.0 + 0.5 * R - 0.418688 * G - 0.081312 * B;
        }
    }
    int CW = PW / g.hs, CH = PH / g.vs;
    double* cb2 = (double*)malloc(sizeof(double) * (size_t)CW * CH);
    double* cr2 = (double*)malloc(sizeof(double) * (size_t)CW * CH);
    const double inv = 1.0 / (g.hs * g.vs);                    /* box average over the hs x vs pixels of a chroma sample */
    for (int y = 0; y < CH; ++y)
        for (int x = 0; x < CW; ++x) {
            double sb = 0.0, sr = 0.0;
            for (int dy = 0; dy < g.vs; ++dy)
                for (int dx = 0; dx < g.hs; ++dx) {
                    size_t a = (size_t)(g.vs * y + dy) * PW + g.hs * x + dx;
                    sb += Cb[a]; sr += Cr[a];
                }
            cb2[(size_t)y * CW + x] = inv * sb;
            cr2[(size_t)y * CW + x] = inv * sr;
        }
    fdct_quant_plane(Y, PW, g.bw[0], g.bh[0], qy, coef + g.coff[0] * 64);
    if (g.nc == 3) {
        fdct_quant_plane(cb2, CW, g.bw[1], g.bh[1], qc, coef + g.coff[1] * 64);
        fdct_quant_plane(cr2, CW, g.bw[2], g.bh[2], qc, coef + g.coff[2] * 64);
    }
    free(Y); free(Cb); free(Cr); free(cb2); free(cr2);
}

/* ------------------------------------------------------------------------- */
/* Growable byte buffer and the entropy-coded bit writer                      */
/* ------------------------------------------------------------------------- */
typedef struct { uint8_t* p; size_t n, cap; } bytebuf;
static void bb_reserve(bytebuf* b, size_t extra) {
    if (b->n + extra <= b->cap) return;
    size_t c = b->cap ? b->cap : 4096;
    while (c < b->n + extra) c *= 2;
    b->p = (uint8_t*)realloc(b->p, c); b->cap = c;
}
static void bb_put(bytebuf* b, int v) { bb_reserve(b, 1); b->p[b->n++] = (uint8_t)v; }
static void bb_put16(bytebuf* b, int v) { bb_put(b, v >> 8); bb_put(b, v & 255); }
static void bb_write(bytebuf* b, const void* src, size_t n) { bb_reserve(b, n); memcpy(b->p + b->n, src, n); b->n += n; }

typedef struct { bytebuf* out; uint32_t acc; int nacc; } bitw;
static void bw_put(bitw* w, uint32_t v, int n) {   /* n <= 24 */
    if (n == 0) return;
    w->acc = (w->acc << n) | (v & ((1u << n) - 1u));
    w->nacc += n;
    while (w->nacc >= 8) {
        int byte = (w->acc >> (w->nacc - 8)) & 255;
        bb_put(w->out, byte);
        if (byte == 255) bb_put(w->out, 0);
        w->nacc -= 8;
    }
}
static void bw_flush(bitw* w) {   /* pad the last byte with 1-bits */
    if (w->nacc > 0) bw_put(w, (1u << (8 - w->nacc)) - 1u, 8 - w->nacc);
    w->acc = 0; w->nacc = 0;
}

/* ------------------------------------------------------------------------- */
/* Scan script and the token stream of one scan                               */
/* ------------------------------------------------------------------------- */
typedef struct { int ncomp; int comp[3]; int Ss, Se, Ah, Al; } scan_spec;

/* the ten-scan script a stock encoder uses for three-component 4:2:0 images */
static const scan_spec SCRIPT10[10] = {
    {3, {0, 1, 2}, 0, 0, 0, 1}, {1, {0, 0, 0}, 1, 5, 0, 2},  {1, {2, 0, 0}, 1, 63, 0, 1},
    {1, {1, 0, 0}, 1, 63, 0, 1}, {1, {0, 0, 0}, 6, 63, 0, 2}, {1, {0, 0, 0}, 1, 63, 2, 1},
    {3, {0, 1, 2}, 0, 0, 1, 0}, {1, {2, 0, 0}, 1, 63, 1, 0},  {1, {1, 0, 0}, 1, 63, 1, 0},
    {1, {0, 0, 0}, 1, 63, 1, 0}};

/* The script in force (default: the ten-scan one).  synth_set_script replaces it for the records
 * made afterwards; n = 0 restores the default.  flat: 8 ints per scan (ncomp, comp[3], Ss, Se, Ah, Al). */
#define MAX_SCANS 16
static scan_spec g_script[MAX_SCANS];
static int g_nscans = 0;
static const scan_spec* cur_script(int* n) {
    if (g_nscans > 0) { *n = g_nscans; return g_script; }
    *n = 10; return SCRIPT10;
}
/* What a record really holds: for greyscale images the scans of the chroma components fall away
 * and an interleaved scan becomes a luminance scan. */
static int eff_script(scan_spec* out) {
    int n;
    const scan_spec* sc = cur_script(&n);
    int m = 0;
    for (int s = 0; s < n; ++s) {
        scan_spec t = sc[s];
        if (g_nc == 1) {
            int has_y = 0;
            for (int c = 0; c < t.ncomp; ++c) if (t.comp[c] == 0) has_y = 1;
            if (!has_y) continue;
            t.ncomp = 1; t.comp[0] = 0;
        }
        out[m++] = t;
    }
    return m;
}
int synth_set_script(const int* flat, int n) {
    if (n < 0 || n > MAX_SCANS) return -1;
    for (int s = 0; s < n; ++s) {
        scan_spec* sc = &g_script[s];
        sc->ncomp = flat[8 * s];
        for (int c = 0; c < 3; ++c) sc->comp[c] = flat[8 * s + 1 + c];
        sc->Ss = flat[8 * s + 4]; sc->Se = flat[8 * s + 5]; sc->Ah = flat[8 * s + 6]; sc->Al = flat[8 * s + 7];
    }
    g_nscans = n;
    return 0;
}

#define TOK_SYM 0u   /* [9:8] table slot, [7:0] symbol */
#define TOK_BITS 1u  /* [28:24] count, [23:0] value     */
#define TOK_RST 2u   /* [2:0] marker index              */
typedef struct { uint32_t* t; size_t n, cap; } tokbuf;
static void tk_push(tokbuf* b, uint32_t v) {
    if (b->n == b->cap) { b->cap = b->cap ? b->cap * 2 : 65536; b->t = (uint32_t*)realloc(b->t, b->cap * sizeof(uint32_t)); }
    b->t[b->n++] = v;
}
static void tk_sym(tokbuf* b, int slot, int sym) { tk_push(b, (TOK_SYM << 30) | ((uint32_t)slot << 8) | (uint32_t)sym); }
static void tk_bits(tokbuf* b, uint32_t v, int n) { if (n) tk_push(b, (TOK_BITS << 30) | ((uint32_t)n << 24) | (v & ((1u << n) - 1u))); }
static void tk_rst(tokbuf* b, int m) { tk_push(b, (TOK_RST << 30) | (uint32_t)(m & 7)); }

static int bitlen(int a) { int n = 0; while (a) { ++n; a >>= 1; } return n; }

typedef struct {
    tokbuf tok;
    uint8_t* corr; size_t ncorr, capcorr;   /* correction bits held back during an end-of-band run */
    int eobrun, eobslot;
} scan_enc;

static void corr_push(scan_enc* e, int bit) {
    if (e->ncorr == e->capcorr) { e->capcorr = e->capcorr ? e->capcorr * 2 : 4096; e->corr = (uint8_t*)realloc(e->corr, e->capcorr); }
    e->corr[e->ncorr++] = (uint8_t)bit;
}
static void flush_eobrun(scan_enc* e) {
    if (e->eobrun > 0) {
        int nb = bitlen(e->eobrun) - 1;
        tk_sym(&e->tok, e->eobslot, nb << 4);
        tk_bits(&e->tok, (uint32_t)(e->eobrun - (1 << nb)), nb);
        e->eobrun = 0;
    }
    for (size_t i = 0; i < e->ncorr; ++i) tk_bits(&e->tok, e->corr[i], 1);
    e->ncorr = 0;
}

static void enc_ac_first(scan_enc* e, const int16_t* blk, int Ss, int Se, int Al, int slot) {
    int run = 0;
    for (int k = Ss; k <= Se; ++k) {
        int v = blk[k], a = (v < 0 ? -v : v) >> Al;
        if (a == 0) { ++run; continue; }
        flush_eobrun(e);
        while (run > 15) { tk_sym(&e->tok, slot, 0xF0); run -= 16; }
        int s = bitlen(a);
        tk_sym(&e->tok, slot, (run << 4) | s);
        tk_bits(&e->tok, (uint32_t)(v < 0 ? ~a : a), s);
        run = 0;
    }
    if (run > 0) {
        e->eobslot = slot;
        if (++e->eobrun == 0x7FFF) flush_eobrun(e);
    }
}

/* a whole block of a sequential (baseline) scan: the AC part ends with a plain end-of-block
 * symbol unless position 63 is non-zero; there are no end-of-band runs */
static void enc_ac_sequential(scan_enc* e, const int16_t* blk, int slot) {
    int run = 0;
    for (int k = 1; k <= 63; ++k) {
        int v = blk[k], a = v < 0 ? -v : v;
        if (a == 0) { ++run; continue; }
        while (run > 15) { tk_sym(&e->tok, slot, 0xF0); run -= 16; }
        int s = bitlen(a);
        tk_sym(&e->tok, slot, (run << 4) | s);
        tk_bits(&e->tok, (uint32_t)(v < 0 ? ~a : a), s);
        run = 0;
    }
    if (run > 0) tk_sym(&e->tok, slot, 0x00);
}

static void enc_ac_refine(scan_enc* e, const int16_t* blk, int Ss, int Se, int Al, int slot) {
    int mag[64], last_new = -1;
    for (int k = Ss; k <= Se; ++k) {
        int v = blk[k];
        mag[k] = (v < 0 ? -v : v) >> Al;
        if (mag[k] == 1) last_new = k;
    }
    uint8_t pend[64]; int npend = 0;   /* correction bits waiting for the next symbol of this block */
    int run = 0;
    for (int k = Ss; k <= Se; ++k) {
        if (mag[k] == 0) { ++run; continue; }
        while (run > 15 && k <= last_new) {
            flush_eobrun(e);
            tk_sym(&e->tok, slot, 0xF0);
            run -= 16;
            for (int i = 0; i < npend; ++i) tk_bits(&e->tok, pend[i], 1);
            npend = 0;
        }
        if (mag[k] > 1) { pend[npend++] = (uint8_t)(mag[k] & 1); continue; }
        flush_eobrun(e);
        tk_sym(&e->tok, slot, (run << 4) | 1);
        tk_bits(&e->tok, blk[k] < 0 ? 0u : 1u, 1);
        for (int i = 0; i < npend; ++i) tk_bits(&e->tok, pend[i], 1);
        npend = 0;
        run = 0;
    }
    if (run > 0 || npend > 0) {
        e->eobslot = slot;
        ++e->eobrun;
        for (int i = 0; i < npend; ++i) corr_push(e, pend[i]);
        if (e->eobrun == 0x7FFF) flush_eobrun(e);
    }
}

/* ------------------------------------------------------------------------- */
/* Optimal Huffman code lengths (T.81 K.2): lengths <= 16, all-ones reserved  */
/* ------------------------------------------------------------------------- */
typedef struct { uint8_t bits[17]; uint8_t vals[256]; int nvals; uint16_t code[256]; uint8_t len[256]; } hufftab;

static void huff_build(const long freq_in[256], hufftab* h) {
    long freq[257]; int size[257], next[257];
    for (int i = 0; i < 256; ++i) freq[i] = freq_in[i];
    freq[256] = 1;                       /* placeholder that ends up with the all-ones code */
    for (int i = 0; i < 257; ++i) { size[i] = 0; next[i] = -1; }
    for (;;) {
        int a = -1, b = -1;
        for (int i = 0; i < 257; ++i) if (freq[i] > 0 && (a < 0 || freq[i] <= freq[a])) a = i;
        for (int i = 0; i < 257; ++i) if (freq[i] > 0 && i != a && (b < 0 || freq[i] <= freq[b])) b = i;
        if (b < 0) break;
        freq[a] += freq[b]; freq[b] = 0;
        int t = a;
        for (;;) { ++size[t]; if (next[t] < 0) break; t = next[t]; }
        next[t] = b;
        for (t = b; t >= 0; t = next[t]) ++size[t];
    }
    int count[40]; memset(count, 0, sizeof count);
    for (int i = 0; i < 257; ++i) if (size[i]) ++count[size[i] > 39 ? 39 : size[i]];
    for (int L = 39; L > 16; --L)
        while (count[L] > 0) {           /* shorten a pair of over-long codes */
            int j = L - 2;
            while (count[j] == 0) --j;
            count[L] -= 2; count[L - 1] += 1; count[j + 1] += 2; count[j] -= 1;
        }
    int L = 16; while (count[L] == 0) --L;
    --count[L];                          /* drop the placeholder */
    memset(h, 0, sizeof *h);
    for (int i = 1; i <= 16; ++i) h->bits[i] = (uint8_t)count[i];
    int n = 0;
    for (int s = 1; s <= 39; ++s)
        for (int i = 0; i < 256; ++i) if (size[i] == s) h->vals[n++] = (uint8_t)i;
    h->nvals = n;
    int code = 0, k = 0;
    for (int l = 1; l <= 16; ++l) {
        for (int i = 0; i < h->bits[l]; ++i) { int sym = h->vals[k++]; h->code[sym] = (uint16_t)code++; h->len[sym] = (uint8_t)l; }
        code <<= 1;
    }
}

static void write_dht(bytebuf* out, int tc, int th, const hufftab* h) {
    bb_put16(out, 0xFFC4);
    bb_put16(out, 2 + 1 + 16 + h->nvals);
    bb_put(out, (tc << 4) | th);
    for (int i = 1; i <= 16; ++i) bb_put(out, h->bits[i]);
    bb_write(out, h->vals, (size_t)h->nvals);
}

/* ------------------------------------------------------------------------- */
/* One scan: tokenise, build tables, write DHT / DRI / SOS / entropy bytes    */
/* ------------------------------------------------------------------------- */
typedef struct { scan_enc se; int cur_ri; } enc_state;

static void encode_scan(enc_state* st, const geom_t* g, const int16_t* coef, const scan_spec* sc,
                        int restart_rows, int restart_fixed, bytebuf* out) {
    scan_enc* e = &st->se;
    e->tok.n = 0; e->ncorr = 0; e->eobrun = 0; e->eobslot = 0;
    int inter = sc->ncomp > 1;
    int sequential = sc->Ss == 0 && sc->Se == 63;      /* DC and AC of every block in one scan: baseline */
    int c0 = sc->comp[0];
    int mcu_w = inter ? g->mx : g->ubw[c0];
    int mcu_h = inter ? g->my : g->ubh[c0];
    long total = (long)mcu_w * mcu_h;
    int ri = restart_fixed > 0 ? restart_fixed : (restart_rows ? mcu_w : 0);
    if (ri > 65535) ri = 0;
    int pred[3] = {0, 0, 0};
    int rst = 0;
    long m = 0;
    for (int my = 0; my < mcu_h; ++my)
        for (int mxi = 0; mxi < mcu_w; ++mxi, ++m) {
            if (ri && m > 0 && m % ri == 0) {
                flush_eobrun(e);
                tk_rst(&e->tok, rst); rst = (rst + 1) & 7;
                pred[0] = pred[1] = pred[2] = 0;
            }
            for (int ci = 0; ci < sc->ncomp; ++ci) {
                int c = sc->comp[ci];
                int hh = inter && c == 0 ? g->hs : 1, hv = inter && c == 0 ? g->vs : 1;
                for (int by = 0; by < hv; ++by)
                    for (int bx = 0; bx < hh; ++bx) {
                        size_t brow = (size_t)my * hv + by, bcol = (size_t)mxi * hh + bx;
                        const int16_t* blk = coef + (g->coff[c] + brow * g->bw[c] + bcol) * 64;
                        int slot = c == 0 ? 0 : 1;
                        if (sequential) {
                            int v = blk[0], d = v - pred[c]; pred[c] = v;
                            int a = d < 0 ? -d : d, s = bitlen(a);
                            tk_sym(&e->tok, slot, s);
                            tk_bits(&e->tok, (uint32_t)(d < 0 ? d - 1 : d), s);
                            enc_ac_sequential(e, blk, 2 + slot);
                        } else if (sc->Ss == 0) {
                            if (sc->Ah == 0) {
                                int v = blk[0] >> sc->Al;      /* arithmetic shift: floor */
                                int d = v - pred[c]; pred[c] = v;
                                int a = d < 0 ? -d : d, s = bitlen(a);
                                tk_sym(&e->tok, slot, s);
                                tk_bits(&e->tok, (uint32_t)(d < 0 ? d - 1 : d), s);
                            } else {
                                tk_bits(&e->tok, (uint32_t)((blk[0] >> sc->Al) & 1), 1);
                            }
                        } else if (sc->Ah == 0) enc_ac_first(e, blk, sc->Ss, sc->Se, sc->Al, slot);
                        else enc_ac_refine(e, blk, sc->Ss, sc->Se, sc->Al, slot);
                    }
            }
        }
    flush_eobrun(e);
    (void)total;

    /* statistics -> tables */
    long freq[4][256]; memset(freq, 0, sizeof freq);
    int used[4] = {0, 0, 0, 0};
    for (size_t i = 0; i < e->tok.n; ++i) {
        uint32_t t = e->tok.t[i];
        if ((t >> 30) == TOK_SYM) { int slot = (t >> 8) & 3; ++freq[slot][t & 255]; used[slot] = 1; }
    }
    hufftab tab[4];
    int is_dc = sc->Ss == 0;
    /* progressive scans use slots 0, 1 of one table class; a sequential scan uses DC tables 0, 1
     * (slots 0, 1) and AC tables 0, 1 (slots 2, 3) */
    for (int s = 0; s < 4; ++s)
        if (used[s]) {
            huff_build(freq[s], &tab[s]);
            if (sequential) write_dht(out, s >= 2 ? 1 : 0, s & 1, &tab[s]);
            else write_dht(out, is_dc ? 0 : 1, s, &tab[s]);
        }
    if (ri != st->cur_ri) {
        bb_put16(out, 0xFFDD); bb_put16(out, 4); bb_put16(out, ri);
        st->cur_ri = ri;
    }
    bb_put16(out, 0xFFDA);
    bb_put16(out, 6 + 2 * sc->ncomp);
    bb_put(out, sc->ncomp);
    for (int ci = 0; ci < sc->ncomp; ++ci) {
        int c = sc->comp[ci], slot = c == 0 ? 0 : 1;
        bb_put(out, c + 1);
        bb_put(out, sequential ? ((slot << 4) | slot) : (is_dc ? (slot << 4) : slot));
    }
    bb_put(out, sc->Ss); bb_put(out, sc->Se); bb_put(out, (sc->Ah << 4) | sc->Al);
    bitw w = {out, 0, 0};
    for (size_t i = 0; i < e->tok.n; ++i) {
        uint32_t t = e->tok.t[i];
        switch (t >> 30) {
        case TOK_SYM: { int slot = (t >> 8) & 3, sym = t & 255; bw_put(&w, tab[slot].code[sym], tab[slot].len[sym]); break; }
        case TOK_BITS: bw_put(&w, t & 0xFFFFFFu, (t >> 24) & 31); break;
        default: bw_flush(&w); bb_put16(out, 0xFFD0 + (t & 7)); break;
        }
    }
    bw_flush(&w);
}

/* ------------------------------------------------------------------------- */
/* One image -> progressive JPEG file, with the byte offset of every scan     */
/* ------------------------------------------------------------------------- */
/* restart_rows: 1 = restart interval of one MCU row in every scan;
 * restart_fixed > 0 overrides with a fixed interval in MCUs.
 * scan_end[s] = offset just past scan s's entropy data (EOI follows the last). */
static void encode_image(enc_state* st, const geom_t* g, const int16_t* coef, const uint8_t qy[64],
                         const uint8_t qc[64], int restart_rows, int restart_fixed, bytebuf* out, size_t scan_end[MAX_SCANS]) {
    st->cur_ri = 0;
    bb_put16(out, 0xFFD8);
    static const uint8_t jfif[] = {0xFF, 0xE0, 0, 16, 'J', 'F', 'I', 'F', 0, 1, 1, 0, 0, 1, 0, 1, 0, 0};
    bb_write(out, jfif, sizeof jfif);
    for (int t = 0; t < 2; ++t) {
        bb_put16(out, 0xFFDB); bb_put16(out, 67); bb_put(out, t);
        const uint8_t* q = t ? qc : qy;
        for (int k = 0; k < 64; ++k) bb_put(out, q[ZZ[k]]);
    }
    scan_spec script[MAX_SCANS];
    int ns = eff_script(script);
    int baseline = ns == 1 && script[0].Ss == 0 && script[0].Se == 63;
    bb_put16(out, baseline ? 0xFFC0 : 0xFFC2); bb_put16(out, 8 + 3 * g->nc); bb_put(out, 8);
    bb_put16(out, g->H); bb_put16(out, g->W); bb_put(out, g->nc);
    bb_put(out, 1); bb_put(out, (g->hs << 4) | g->vs); bb_put(out, 0);
    if (g->nc == 3) {
        bb_put(out, 2); bb_put(out, 0x11); bb_put(out, 1);
        bb_put(out, 3); bb_put(out, 0x11); bb_put(out, 1);
    }
    for (int s = 0; s < ns; ++s) {
        encode_scan(st, g, coef, &script[s], restart_rows, restart_fixed, out);
        scan_end[s] = out->n;
    }
    bb_put16(out, 0xFFD9);
}

/* ------------------------------------------------------------------------- */
/* Record: header, sample metadata, index, scan groups                        */
/* ------------------------------------------------------------------------- */
typedef struct synth_record {
    int n;
    uint8_t* bytes; size_t len;
    int16_t** truth; size_t* truth_n;     /* ground-truth coefficients per image */
    uint8_t** jpeg; size_t* jpeg_n;       /* the stand-alone progressive file of each image */
    uint32_t* W; uint32_t* H;
} synth_record;

static void put32(uint8_t* p, uint32_t v) { p[0] = v; p[1] = v >> 8; p[2] = v >> 16; p[3] = v >> 24; }
static void put64(uint8_t* p, uint64_t v) { put32(p, (uint32_t)v); put32(p + 4, (uint32_t)(v >> 32)); }

static void assemble_record(synth_record* r, const int32_t* labels, size_t (*scan_end)[MAX_SCANS]) {
    scan_spec eff[MAX_SCANS];
    int N = r->n, G = eff_script(eff);    /* one scan per group */
    size_t meta_off = 64;
    size_t index_off = meta_off + 16 * (size_t)N;
    size_t data_off = index_off + 8 * (size_t)(G + 1) + 16 * (size_t)G * N;
    data_off = (data_off + 255) & ~(size_t)255;
    size_t total = data_off;
    for (int g = 0; g < G; ++g) {
        for (int i = 0; i < N; ++i) {
            size_t a = g ? scan_end[i][g - 1] : 0, b = scan_end[i][g];
            total += (b - a + 15) & ~(size_t)15;
        }
        total = (total + 255) & ~(size_t)255;
    }
    r->bytes = (uint8_t*)calloc(total, 1); r->len = total;
    uint8_t* p = r->bytes;
    memcpy(p, "PCR1", 4); put32(p + 4, 1); put32(p + 8, (uint32_t)N); put32(p + 12, (uint32_t)G);
    put32(p + 16, 0); put32(p + 20, 0);
    put64(p + 24, meta_off); put64(p + 32, index_off); put64(p + 40, data_off); put64(p + 48, total);
    for (int i = 0; i < N; ++i) {
        uint8_t* m = p + meta_off + 16 * (size_t)i;
        put32(m, (uint32_t)labels[i]); put32(m + 4, r->W[i]); put32(m + 8, r->H[i]); put32(m + 12, 0);
    }
    uint8_t* gend = p + index_off;
    uint8_t* chunk = gend + 8 * (size_t)(G + 1);
    put64(gend, data_off);
    size_t pos = data_off;
    for (int g = 0; g < G; ++g) {
        for (int i = 0; i < N; ++i) {
            size_t a = g ? scan_end[i][g - 1] : 0, b = scan_end[i][g];
            memcpy(p + pos, r->jpeg[i] + a, b - a);
            uint8_t* c = chunk + 16 * ((size_t)g * N + i);
            put64(c, pos); put32(c + 8, (uint32_t)(b - a)); put32(c + 12, 0);
            pos += (b - a + 15) & ~(size_t)15;
        }
        pos = (pos + 255) & ~(size_t)255;
        put64(gend + 8 * (size_t)(g + 1), pos);
    }
}

static void free_scan_enc(enc_state* st) { free(st->se.tok.t); free(st->se.corr); }

/* Build a record from ready-made coefficient arrays (canonical layout).
 * coefs[i] has geom(W[i],H[i]).nblocks*64 entries; qy/qc are natural-order tables per image (64 each). */
synth_record* synth_record_from_coeffs(int n, const uint32_t* W, const uint32_t* H, const int32_t* labels,
                                       const int16_t* const* coefs, const uint8_t* qy, const uint8_t* qc,
                                       int restart_rows, int restart_fixed, int nthreads) {
    init_tables();
    synth_record* r = (synth_record*)calloc(1, sizeof *r);
    r->n = n;
    r->truth = (int16_t**)calloc((size_t)n, sizeof(void*)); r->truth_n = (size_t*)calloc((size_t)n, sizeof(size_t));
    r->jpeg = (uint8_t**)calloc((size_t)n, sizeof(void*)); r->jpeg_n = (size_t*)calloc((size_t)n, sizeof(size_t));
    r->W = (uint32_t*)calloc((size_t)n, 4); r->H = (uint32_t*)calloc((size_t)n, 4);
    size_t (*scan_end)[MAX_SCANS] = (size_t(*)[MAX_SCANS])calloc((size_t)n, sizeof(size_t[MAX_SCANS]));
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#endif
#pragma omp parallel
    {
        enc_state st; memset(&st, 0, sizeof st);
#pragma omp for schedule(dynamic, 1)
        for (int i = 0; i < n; ++i) {
            geom_t g; geom_init(&g, (int)W[i], (int)H[i]);
            r->W[i] = W[i]; r->H[i] = H[i];
            r->truth_n[i] = g.nblocks * 64;
            r->truth[i] = (int16_t*)malloc(r->truth_n[i] * sizeof(int16_t));
            memcpy(r->truth[i], coefs[i], r->truth_n[i] * sizeof(int16_t));
            /* blocks that exist only as MCU padding are outside every single-component scan,
             * so a progressive stream cannot carry their AC coefficients: the truth has none */
            for (int c = 0; c < 3; ++c)
                for (int by = 0; by < g.bh[c]; ++by)
                    for (int bx = 0; bx < g.bw[c]; ++bx)
                        if (bx >= g.ubw[c] || by >= g.ubh[c])
                            memset(r->truth[i] + (g.coff[c] + (size_t)by * g.bw[c] + bx) * 64 + 1, 0, 63 * sizeof(int16_t));
            bytebuf out = {0, 0, 0};
            encode_image(&st, &g, r->truth[i], qy + 64 * (size_t)i, qc + 64 * (size_t)i, restart_rows, restart_fixed, &out, scan_end[i]);
            r->jpeg[i] = out.p; r->jpeg_n[i] = out.n;
        }
        free_scan_enc(&st);
    }
    assemble_record(r, labels, scan_end);
    free(scan_end);
    return r;
}

/* Build a record from image recipes. */
synth_record* synth_record_create(const synth_image_spec* specs, int n, int restart_rows, int restart_fixed, int nthreads) {
    init_tables();
    int16_t** coefs = (int16_t**)calloc((size_t)n, sizeof(void*));
    uint32_t* W = (uint32_t*)malloc(4 * (size_t)n); uint32_t* H = (uint32_t*)malloc(4 * (size_t)n);
    int32_t* labels = (int32_t*)malloc(4 * (size_t)n);
    uint8_t* qy = (uint8_t*)malloc(64 * (size_t)n); uint8_t* qc = (uint8_t*)malloc(64 * (size_t)n);
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#endif
#pragma omp parallel for schedule(dynamic, 1)
    for (int i = 0; i < n; ++i) {
        const synth_image_spec* sp = &specs[i];
        W[i] = sp->width; H[i] = sp->height; labels[i] = sp->label;
        synth_quant_table(sp->quality, 0, qy + 64 * (size_t)i);
        synth_quant_table(sp->quality, 1, qc + 64 * (size_t)i);
        geom_t g; geom_init(&g, (int)sp->width, (int)sp->height);
        uint8_t* rgb = (uint8_t*)malloc((size_t)sp->width * sp->height * 3);
        synth_image_rgb(sp, rgb);
        coefs[i] = (int16_t*)malloc(g.nblocks * 64 * sizeof(int16_t));
        synth_rgb_to_coeffs(rgb, (int)sp->width, (int)sp->height, qy + 64 * (size_t)i, qc + 64 * (size_t)i, coefs[i]);
        free(rgb);
    }
    synth_record* r = synth_record_from_coeffs(n, W, H, labels, (const int16_t* const*)coefs, qy, qc, restart_rows, restart_fixed, nthreads);
    for (int i = 0; i < n; ++i) free(coefs[i]);
    free(coefs); free(W); free(H); free(labels); free(qy); free(qc);
    return r;
}

const uint8_t* synth_record_bytes(const synth_record* r, size_t* len) { *len = r->len; return r->bytes; }
int synth_record_num_images(const synth_record* r) { return r->n; }
size_t synth_record_truth_count(const synth_record* r, int i) { return r->truth_n[i]; }
const int16_t* synth_record_truth(const synth_record* r, int i) { return r->truth[i]; }
const uint8_t* synth_record_jpeg(const synth_record* r, int i, size_t* len) { *len = r->jpeg_n[i]; return r->jpeg[i]; }
void synth_record_dims(const synth_record* r, int i, uint32_t* W, uint32_t* H) { *W = r->W[i]; *H = r->H[i]; }
size_t synth_num_blocks(uint32_t W, uint32_t H) { geom_t g; geom_init(&g, (int)W, (int)H); return g.nblocks; }
void synth_zigzag(int32_t out[64]) { init_tables(); for (int k = 0; k < 64; ++k) out[k] = ZZ[k]; }

void synth_record_free(synth_record* r) {
    if (!r) return;
    for (int i = 0; i < r->n; ++i) { free(r->truth[i]); free(r->jpeg[i]); }
    free(r->truth); free(r->truth_n); free(r->jpeg); free(r->jpeg_n); free(r->W); free(r->H); free(r->bytes);
    free(r);
}
