// Structures shared by the host side and the kernels of the PCR decoder.
#pragma once
#include <stdint.h>

namespace pcr {

// One scan of the (record-wide) scan script: which components, which band, which bit.
struct ScanScript {
    int32_t ncomp;
    int32_t comp[3];
    int32_t Ss, Se, Ah, Al;
};

// Where an AC scan keeps its per-block side data in the auxiliary array (units of uint64,
// indexed by the block's number inside its component across the whole record):
//  - a first-pass AC scan writes one word per block: the mask of zigzag positions it made non-zero;
//  - an AC refinement scan writes four words per block: {mask of non-zero positions of its band
//    after the scan, correction bits in reading order (first bit at bit 63), mask of newly
//    non-zero positions, mask of those that are positive}.  The coefficient planes are updated
//    from these by the pixel kernel.
// A refinement scan finds the positions that were non-zero before it by OR-ing the masks of up
// to four earlier scans (src), each read with its own stride.
struct ScanAux {
    uint64_t base;        // first word of this scan's side data
    uint32_t stride;      // words per block: 1 or 4
    int32_t nsrc;
    int32_t src[4];       // scan indices
};

// Refinement scans to apply per component, in scan order (built per decode for the chosen k).
struct FinalizeList {
    int32_t n[3];
    int32_t scan[3][4];
    int32_t p1[3][4];      // 1 << Al of the scan
    uint64_t base[3][4];   // first word of the scan's side data
};

// One (scan, image) pair: where its entropy-coded bytes and Huffman tables live.
struct ScanDesc {
    uint32_t data_off;    // first entropy-coded byte (offset in the record)
    uint32_t data_end;    // one past the last byte of the chunk
    uint32_t seg_base;    // first entry of this pair in the segment table
    uint32_t nseg;        // restart intervals in the scan
    uint32_t ri;          // restart interval in MCUs (0 = none)
    uint32_t tab_off[2];  // offsets of up to two DHT table bodies (16 counts, then values)
    uint32_t slots;       // 2 bits per scan component: which of tab_off it uses
    uint32_t tab_ac[2];   // sequential scans only: up to two AC table bodies (tab_off then holds the DC tables)
    uint32_t slots_ac;    // 2 bits per scan component: which of tab_ac it uses
};

struct ImgDesc {
    uint32_t W, H, mx, my;
    uint64_t blk_base;    // first block of the image in the coefficient planes
    uint64_t out_off;     // first byte of the image in the output buffer
};

// Restart intervals one warp takes (one lane each).  Fewer than 32 leaves lanes idle but
// gives more warps to hide the latency of the serial decode chains.
#ifndef PCR_SEGS_PER_ITEM
#define PCR_SEGS_PER_ITEM 32
#endif
constexpr int kSegsPerItem = PCR_SEGS_PER_ITEM;

// Entropy work item: up to kSegsPerItem consecutive restart intervals of one (scan, image).
struct Item {
    uint32_t si;          // scan * N + image
    uint32_t seg0;        // first restart interval of the item
    uint32_t count;       // restart intervals in the item (<= kSegsPerItem)
    uint32_t next;        // 0, or 1 + (scan * N + image) of the image whose first intervals the item runs on into
};
constexpr uint32_t kItemOpen = 0xFFFFFFFFu;   // host only, while the list is built: the item may still be extended

// Crop rectangle of one image (pixels) and whether its columns are mirrored; the pixel kernel
// skips work units that lie outside it when one is given.
struct CropRect {
    uint32_t x0, y0, w, h, flip;
};

// Pixel work unit: a run of MCUs in one MCU row of one image.
struct Unit {
    uint32_t img;
    uint16_t mrow, mcol0;
};

struct Params {
    const uint8_t* rec;         // record bytes on the device
    uint8_t* ubuf;              // entropy-coded bytes without stuffing, big-endian words
    int16_t* planes;            // coefficient planes, 64 int16 per block, zigzag order
    int16_t* head;              // zigzag positions 0..7 of every block, dense (8 int16 = 16 bytes per
                                // block, same block numbering).  First passes store these positions
                                // here and only positions 8..63 in the 128-byte line: the dense
                                // plane stays in L2 while it is written, instead of one cold
                                // 128-byte line being read and written back per coefficient
    const ScanScript* script;   // [G]
    const ScanAux* saux;        // [G]
    uint64_t* aux;              // side data of the AC scans
    const ScanDesc* scans;      // [G][N]
    const ImgDesc* imgs;        // [N]
    uint32_t* seg_start;        // segment table: first byte of every restart interval
    const Item* items;
    const Unit* units;
    const uint16_t* qtab;       // [N][3][64] quantisers, zigzag order
    uint8_t* chroma;            // chroma sample planes (triangle upsampling only): per image, at 128 bytes
                                // per MCU in front of it, a Cb plane then a Cr plane of 8*my rows x 8*mx bytes
    const uint32_t* order;      // [N] processing order of the images
    const CropRect* roi;        // [N] or null: only work units that touch the image's rectangle are transformed
    int* status;                // [N]
    int32_t N;
    // chroma sampling of the record's images: the luminance component has hs x vs blocks per MCU
    // (1 or 2 each), every chroma component one; nc = 3, or 1 for greyscale (then hs = vs = 1 and
    // the block grid has no MCU padding)
    int32_t hs, vs, nc;
};

}  // namespace pcr
