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

// One (scan, image) pair: where its entropy-coded bytes and Huffman tables live.
struct ScanDesc {
    uint32_t data_off;    // first entropy-coded byte (offset in the record)
    uint32_t data_end;    // one past the last byte of the chunk
    uint32_t seg_base;    // first entry of this pair in the segment table
    uint32_t nseg;        // restart intervals in the scan
    uint32_t ri;          // restart interval in MCUs (0 = none)
    uint32_t tab_off[2];  // offsets of up to two DHT table bodies (16 counts, then values)
    uint32_t slots;       // 2 bits per scan component: which of tab_off it uses
};

struct ImgDesc {
    uint32_t W, H, mx, my;
    uint64_t blk_base;    // first block of the image in the coefficient planes
    uint64_t out_off;     // first byte of the image in the output buffer
};

// Entropy work item: up to 32 consecutive restart intervals of one (scan, image).
struct Item {
    uint32_t si;          // scan * N + image
    uint32_t seg0;        // first restart interval of the item
};

// Pixel work unit: a run of MCUs in one MCU row of one image.
struct Unit {
    uint32_t img;
    uint16_t mrow, mcol0;
};

struct Params {
    const uint8_t* rec;         // record bytes on the device
    int16_t* planes;            // coefficient planes, 64 int16 per block, zigzag order
    const ScanScript* script;   // [G]
    const ScanDesc* scans;      // [G][N]
    const ImgDesc* imgs;        // [N]
    uint32_t* seg_start;        // segment table: first byte of every restart interval
    const Item* items;
    const Unit* units;
    const uint16_t* qtab;       // [N][3][64] quantisers, zigzag order
    int* status;                // [N]
    int32_t N;
};

}  // namespace pcr
