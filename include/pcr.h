/*
 * pcr.h — C ABI of the B200 (sm_100a) decoder for Progressive Compressed Records.
 *
 * A record is the paper's storage unit (Section 3, and its record-layout figure): sample
 * metadata (labels) and record metadata (where every image's every scan lives) followed by
 * scan group 1 of all images, scan group 2 of all images, ...  Reading the record from its
 * start to the end of scan group k gives every image at fidelity k.  This library takes
 * those bytes and produces training pixels on the GPU: for every image, the progressive
 * JPEG decode of its scans 1..k (Section 2, "Progressive Image Compression"; Section 5,
 * "Decoding": scans 1..k of an image followed by an end-of-image token are a decodable
 * JPEG) -> int16 coefficient planes in device memory -> dequantise, 8x8 inverse DCT,
 * 2x2 chroma replication, YCbCr->RGB -> packed uint8 RGB.
 *
 * Record layout (little-endian, 16-byte aligned chunks; the "raw struct" form of Section 5):
 *   header  64 B : "PCR1", u32 version(1), u32 n_images N, u32 n_groups G, u32 flags, u32 rsvd,
 *                  u64 meta_off, u64 index_off, u64 data_off, u64 total_bytes, u64 rsvd
 *   meta         : N x { i32 label; u32 width; u32 height; u32 rsvd }            (scan group 0)
 *   index        : u64 group_end[G+1]  (group_end[0] = data_off; fidelity k needs bytes
 *                  [0, group_end[k]))  then  { u64 off; u32 len; u32 rsvd } chunk[G][N]
 *   data         : group 1 chunks of images 0..N-1, group 2 chunks, ...
 *   chunk (g, i) = the bytes of image i's progressive JPEG file that belong to scan g: for
 *   g = 1 from SOI (tables, frame header), for every g the scan's DHT/DRI/SOS segments and
 *   entropy-coded bytes.  The file's EOI is not stored.  One scan per group.
 *
 * Supported streams: 8-bit, Huffman coded; three components with the luminance at 1 or 2 blocks per
 * MCU in each direction and one block per chroma component (4:2:0, 4:2:2, 4:4:0, 4:4:4: the paper's
 * per-scan example for HAM10000 is a 4:4:4 file), or one component (greyscale: every output pixel
 * is (Y, Y, Y)); one sampling per record; progressive
 * (SOF2) with any scan script that is the same for all images of a record, or baseline
 * sequential (SOF0, one interleaved scan = one scan group: the conventional JPEG that the paper's
 * Table 2 compares against); any restart interval.
 *
 * All functions return an int status: PCR_OK (0) or a negative PCR_E_* code.  Nothing here
 * throws, aborts or prints.  Unless said otherwise pointers are HOST pointers.
 * A pcr_record may be used by one thread at a time.
 */
#ifndef PCR_H_
#define PCR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PCR_OK 0
#define PCR_E_ARG (-1)      /* NULL pointer, k outside 1..G, index out of range, misaligned output */
#define PCR_E_FORMAT (-2)   /* not a record: magic/version, offsets not monotone or past the end,
                               images disagree on the scan script, unsupported JPEG features     */
#define PCR_E_CORRUPT (-3)  /* found while decoding on the device: undefined Huffman code,
                               segment overrun, wrong number of restart markers                   */
#define PCR_E_TIMEOUT (-4)  /* a bounded device-side wait gave up: in records without restart
                               markers a refinement scan follows, block by block, the earlier
                               refinement of the same component that other warps of the same
                               launch decode, and a scan's decoding thread and helper warp meet
                               once per batch of blocks; the polls of these waits are counted   */
#define PCR_E_CUDA (-5)     /* a CUDA runtime call failed                                        */
#define PCR_E_NOMEM (-6)    /* host or device allocation failed                                  */

typedef struct pcr_record pcr_record; /* opaque; owned by the library */

typedef struct {
    uint32_t width, height;
    int32_t label;
    uint32_t rsvd;
    uint64_t out_offset; /* byte offset of the image's pixels inside the output buffer */
    uint64_t out_bytes;  /* 3 * width * height                                          */
} pcr_image_info;

/* Section 3 (metadata + scan groups) and Section 5 "Decoding" (locate the offsets).
 * Parses and validates the header, the group table, every chunk's position and every
 * image's JPEG frame, table and scan headers; allocates the per-record device state
 * (record bytes, coefficient planes, tables) on the current CUDA device.
 *   bytes : the whole record, HOST memory (pinned memory makes the copies asynchronous).
 *           BORROWED: it must stay valid and unchanged until pcr_close.
 *   len   : its length in bytes (< 4 GiB).
 *   rec   : receives the handle; NULL on failure.
 * The device tables are filled on an internal stream and the call does not wait for them: every
 * decode of the record waits (on the device) for that set-up first.  Different records may be
 * opened and used from different host threads at the same time (a loader parses the next record
 * while the current one decodes); one record belongs to one thread at a time.  Device buffers of
 * closed records are kept for later opens (pcr_release_cached_memory returns them).
 * Errors: PCR_E_ARG, PCR_E_FORMAT, PCR_E_NOMEM, PCR_E_CUDA. */
int pcr_open(const void* bytes, size_t len, pcr_record** rec);

/* Number of images N / scan groups G of the record (negative error for a NULL handle). */
int pcr_num_images(const pcr_record* rec);
int pcr_num_groups(const pcr_record* rec);

/* Sample metadata and output placement of image i (Section 3: labels are metadata). */
int pcr_get_image(const pcr_record* rec, int i, pcr_image_info* info);

/* Size the output buffer of pcr_decode must have.  Images are packed RGB, row-major,
 * 3*width bytes per row, image i at out_offset (a multiple of 128).  The size includes 16 spare
 * bytes behind the last image (never written; pcr_decode_tensor reads pixels as aligned words). */
size_t pcr_out_bytes(const pcr_record* rec);

/* Bytes [0, pcr_prefix_bytes(rec, k)) are what fidelity k reads (Section 3: "from the
 * start of the PCR to the end of the corresponding scan group").  0 for a bad k. */
size_t pcr_prefix_bytes(const pcr_record* rec, int k);

/* Decode all images at fidelity k (Sections 2, 3, 5): Huffman-decode scans 1..k into the
 * record's int16 coefficient planes (first passes, then successive-approximation
 * refinements in place), then dequantise, inverse-DCT, upsample, colour-convert and store.
 *   k      : 1..G.
 *   out    : DEVICE memory, caller-owned, at least pcr_out_bytes(rec) bytes, 16-byte aligned.
 *            Only the bytes of each image's 3*W*H pixels are written.
 *   stream : a cudaStream_t (NULL = the default stream).
 * Any part of the prefix [0, end_k) that is not yet resident on the device is first copied
 * from the borrowed host buffer on `stream`; resident bytes are kept for later calls.
 * The call enqueues the copy and the kernels and returns; the caller synchronises `stream`.
 * Every call decodes scans 1..k from scratch.  One decode in flight per record.
 * Bytes at or beyond end_k are never read.
 * Errors: PCR_E_ARG, PCR_E_CUDA (launch failures).  Stream errors found by the device are
 * reported by pcr_status. */
int pcr_decode(pcr_record* rec, int k, void* out, void* stream);

/* Raise the fidelity of the last decode (Section 3: "a task then merely needs to read subsequent
 * scan groups until the desired fidelity level is reached"; Section 4.3 switches fidelity while
 * training).  The coefficient planes and the side data of scans 1..k_prev stay on the device
 * after pcr_decode; this call copies the scan groups k_prev+1..k that are not yet resident,
 * decodes only those scans on top of the resident state and produces the pixels of fidelity k.
 * The result is identical to pcr_decode(rec, k, ...).
 *   k : k_prev < k <= G, where k_prev is the fidelity of the last pcr_decode / pcr_decode_more
 *       on this record (PCR_E_ARG otherwise, also when nothing has been decoded yet).
 *   out, stream : as for pcr_decode.  The previous call's work must be complete or ordered
 *       before this one (same stream, or synchronised).
 * Status words accumulate: an error flagged by the earlier decode stays set. */
int pcr_decode_more(pcr_record* rec, int k, void* out, void* stream);

/* Decode at fidelity k straight to a training batch (Section 6, experimental setup: the
 * experiments use resizing, crop and horizontal-flip augmentations, after which all inputs have
 * the same size: 224x224, or 160x160 crops in the appendix's second pipeline).  The decode is
 * pcr_decode's; the pixel stage transforms only the 16x16 MCUs that touch an image's crop
 * rectangle, and an epilogue kernel resamples the crop to size x size and writes the tensor:
 *   for output pixel (ox, oy): u = flip ? size-1-ox : ox;
 *   fx = clamp((u + 0.5) * w / size - 0.5, 0, w - 1), fy likewise with h (half-pixel centres,
 *   the crop's edge pixels repeated, no low-pass filter); v = bilinear interpolation of the four
 *   pixels around (x0 + fx, y0 + fy); tensor[i][c][oy][ox] = (v_c / 255 - mean[c]) / std[c],
 *   evaluated in single precision, stored as dtype (half, bfloat16: round to nearest even).
 *   crops  : HOST array of pcr_num_images entries (read before the call returns); every
 *            rectangle must lie inside its image, w, h >= 1, flip 0 or 1 (else PCR_E_ARG; also
 *            when an image has 2 GiB of pixels or more).
 *            The random draws of an augmentation policy are the caller's.
 *   size   : 1..4096.   mean, std : HOST, three floats each, std > 0.   dtype : PCR_F16 / PCR_F32 / PCR_BF16.
 *   rgb    : DEVICE scratch as pcr_decode's `out` (same size and alignment); afterwards it holds
 *            the decoded pixels of the transformed MCUs, other bytes are left as they were.
 *   tensor : DEVICE, pcr_num_images * 3 * size * size elements of dtype, image i at index i.
 * Restart intervals whose MCU rows lie outside the MCU rows an image's rectangle touches are not
 * entropy-decoded either, so afterwards the coefficient planes are incomplete: pcr_decode_more
 * refuses to continue from this call (PCR_E_ARG) and pcr_coeffs is meaningful only for the
 * decoded rows.
 * Enqueues on `stream` and returns; errors as pcr_decode.  The first call on a record allocates
 * a small device array for the rectangles. */
#define PCR_F16 0
#define PCR_F32 1
#define PCR_BF16 2
typedef struct {
    uint32_t x0, y0, w, h; /* crop rectangle in pixels of the decoded image */
    uint32_t flip;         /* 1: mirror the columns                         */
} pcr_crop;
int pcr_decode_tensor(pcr_record* rec, int k, const pcr_crop* crops, int size, const float* mean, const float* std,
                      int dtype, void* rgb, void* tensor, void* stream);

/* Multi-scale structural similarity between two decodes of the record, image by image (Section
 * 4.3 and the appendix figure on reconstruction quality: the MSSIM of the image decoded from scan
 * groups 1..k against the full-fidelity image is the paper's diagnostic for choosing k; scan
 * groups of 5 and more reach 95 % there).  The measure is Wang, Simoncelli and Bovik's (2003) in
 * its common form: luminance 0.299 R + 0.587 G + 0.114 B of the 8-bit pixels; per scale an 11x11
 * Gaussian window (sigma 1.5) at the positions where it fits; cs = (2 s_xy + C2) / (s_x^2 + s_y^2
 * + C2) and l = (2 m_x m_y + C1) / (m_x^2 + m_y^2 + C1) with C1 = 2.55^2, C2 = 7.65^2, averaged
 * over the scale; the next scale is the 2x2 block average (an odd last row or column dropped);
 * score = prod_j max(mean cs_j, 0)^w_j * max(mean l_M, 0)^w_M with the weights 0.0448, 0.2856,
 * 0.3001, 0.2363, 0.1333; an image with a side below 176 has fewer scales (M = the number of j
 * with min(W, H) >> j >= 11) and uses the first M weights rescaled to sum to one; M = 0: NaN.
 *   rgb_a, rgb_b : DEVICE, two outputs of pcr_decode / pcr_decode_more of THIS record.
 *   scratch      : DEVICE, pcr_msssim_scratch_bytes(rec) bytes, 16-byte aligned, caller-owned
 *                  (two luminance pyramids per image and the per-scale sums).
 *   dev_scores   : DEVICE, pcr_num_images floats, score of image i at index i.
 * Enqueues on `stream` and returns.  The first call on a record uploads a small per-image table
 * (one allocation).  Records of more than 65535 images are refused (PCR_E_ARG).
 * Errors: PCR_E_ARG, PCR_E_NOMEM, PCR_E_CUDA. */
size_t pcr_msssim_scratch_bytes(pcr_record* rec);
int pcr_msssim(pcr_record* rec, const void* rgb_a, const void* rgb_b, void* scratch, float* dev_scores, void* stream);

/* Chroma upsampling of the decodes that follow (pcr_decode, pcr_decode_more).  The paper hands
 * its reassembled files to stock decoders (Section 5) and does not name the filter.
 *   PCR_UPSAMPLE_REPLICATE (default): pixel (x, y) takes chroma sample (x >> 1, y >> 1).
 *   PCR_UPSAMPLE_TRIANGLE: the filter stock decoders apply by default: every pixel mixes its own
 *     sample with the horizontally nearer, the vertically nearer and the diagonal neighbour,
 *     (9 a + 3 b + 3 c + d + 8) >> 4; neighbours come from the decoded MCU-padded chroma planes,
 *     beyond their border the edge sample repeats.  Costs a second pass over the chroma blocks
 *     (their samples go through device memory: the first call allocates 128 bytes per MCU).
 * pcr_decode_tensor works with replication only (PCR_E_ARG otherwise).  The triangle filter is
 * built for 4:2:0 records (PCR_E_ARG for other samplings).
 * Errors: PCR_E_ARG, PCR_E_NOMEM. */
#define PCR_UPSAMPLE_REPLICATE 0
#define PCR_UPSAMPLE_TRIANGLE 1
int pcr_set_upsampling(pcr_record* rec, int mode);

/* Forget which record bytes are resident on the device: the next pcr_decode copies its whole
 * prefix again (what a loader that streams each record once from host memory pays). */
int pcr_evict(pcr_record* rec);

/* After the stream of the last pcr_decode has been synchronised: reads the per-image
 * status words back.  *code = PCR_OK, or the first failing image's error with its index in
 * *first_bad_image (-1 if none).  A corrupt image's pixels come from the coefficients
 * decoded before the error (never uninitialised memory). */
int pcr_status(pcr_record* rec, int* first_bad_image, int* code);

/* Test hook: the coefficient planes of the last decode, DEVICE memory owned by the record.
 * Call it after the decode's stream has been synchronised: it completes the canonical layout
 * (the decode keeps DC coefficients in a dense plane of their own; they are copied into the
 * blocks here, with a small kernel on the default stream that this call waits for).
 * Layout: image after image (image i's first block = its blocks_offset), within an image
 * component Y, Cb, Cr, block rows then block columns of the MCU-padded grid, 64 int16 per
 * block in zigzag order (128 bytes per block).  *bytes = total size. */
int pcr_coeffs(pcr_record* rec, const int16_t** dev_planes, size_t* bytes);

/* First block of image i inside the planes returned by pcr_coeffs, and its block count. */
int pcr_image_blocks(const pcr_record* rec, int i, uint64_t* first_block, uint64_t* n_blocks);

/* One scan of the record's scan script (Section 2: scans are ordered groups of deltas; the
 * spectral band Ss..Se and the bit positions Ah/Al are the two progressive dimensions) and
 * the dependency wave the decoder runs it in (scans of one wave touch disjoint data). */
typedef struct {
    int32_t ncomp;      /* components in the scan (1, or 3 interleaved)             */
    int32_t comp[3];    /* 0 = Y, 1 = Cb, 2 = Cr                                     */
    int32_t Ss, Se;     /* zigzag band                                               */
    int32_t Ah, Al;     /* successive approximation: previous / current bit position */
    int32_t wave;       /* 0-based dependency wave                                   */
    int32_t rsvd;
    uint64_t bytes;     /* bytes of this scan group in the record                    */
} pcr_scan_info;
int pcr_get_scan(const pcr_record* rec, int s, pcr_scan_info* info);   /* s in 0..G-1 */

/* Chroma sampling of the record's images (Section 2: chroma subsampling is part of the JPEG data):
 * *hs x *vs luminance blocks per MCU (2 x 2 = 4:2:0, 2 x 1 = 4:2:2, 1 x 2 = 4:4:0, 1 x 1 = 4:4:4),
 * *ncomp = 3, or 1 for greyscale (then 1 x 1).  The block grid of pcr_coeffs follows from it: the
 * luminance plane has hs*ceil(W/(8 hs)) x vs*ceil(H/(8 vs)) blocks, each chroma plane
 * ceil(W/(8 hs)) x ceil(H/(8 vs)). */
int pcr_get_sampling(const pcr_record* rec, int* hs, int* vs, int* ncomp);

/* Stage timing for benchmarks.  With profiling enabled every pcr_decode records CUDA events
 * on its stream around each stage; after the stream has been synchronised pcr_get_profile
 * returns, for the last decode, up to `cap` entries {name, milliseconds, kernel launches}.
 * Stages: "h2d" (prefix copy), "clear" (status and plane clearing), "index" (restart-interval
 * index and unstuffed copy), "entropy0".."entropyW" (one per wave that ran), "pixels" (in-place
 * update of the planes from the refinement scans, then the pixel stage).  *n = entries written. */
typedef struct {
    char name[24];
    float ms;
    int32_t launches;
} pcr_stage_time;
int pcr_set_profiling(pcr_record* rec, int enable);
int pcr_get_profile(pcr_record* rec, pcr_stage_time* out, int cap, int* n);

/* The pixel stage alone, for one image, without any allocation.  (The paper has no
 * counterpart; this is a convenience of this library.)
 *
 * Who needs it: code that is handed a fixed set of device buffers and must not grow the
 * device heap or call into an allocator while it runs: a data-loader plug-in running inside
 * another framework's memory pool, a worker that runs after the training job has claimed all
 * device memory, or code on a path where cudaMalloc's implicit device synchronisation is not
 * acceptable.  pcr_open/pcr_decode allocate their tables with cudaMalloc; this call does not
 * call cudaMalloc, cudaFree or any allocating library routine.
 *
 * It turns the int16 coefficient planes of ONE image into packed RGB exactly as pcr_decode's
 * last stage does (dequantise, inverse DCT, 2x2 chroma replication, colour conversion, crop).
 *   dev_coeffs : DEVICE, caller-owned: 6*ceil(W/16)*ceil(H/16) blocks of 64 int16 in the
 *                layout of pcr_coeffs (Y, Cb, Cr; block rows, block columns; zigzag), 16-byte
 *                aligned (the kernel reads whole 16-byte vectors; any other alignment is
 *                refused with PCR_E_ARG before anything is launched).  Not modified.
 *   width, height : at most 4096 each; larger images are refused with PCR_E_ARG.
 *   host_qtab  : HOST, 3 x 64 uint16 quantisers (Y, Cb, Cr) in zigzag order; copied by value.
 *   dev_rgb    : DEVICE, caller-owned, 3*W*H bytes, 4-byte aligned start recommended.
 *   stream     : a cudaStream_t (NULL = default stream).  The call only enqueues work.
 * The kernel's small tables (image descriptor, work-unit list, quantisers: about 65 KB) live
 * in one fixed array inside the library's device image, which every GPU that loads the
 * library holds until the process exits.  All calls on a device share that array and each
 * call rewrites the part it uses, so two calls whose work overlaps on the GPU (different
 * streams, no ordering between them) race; order them on one stream or with events.
 * The first call on each device looks the array's device address up (cudaGetSymbolAddress,
 * with that device current); make that first call before starting any stream capture.
 * Errors: PCR_E_ARG (NULL, zero or too-large size, misaligned coefficients, device index
 * beyond 63), PCR_E_CUDA. */
int pcr_pixels_noalloc(const int16_t* dev_coeffs, uint32_t width, uint32_t height, const uint16_t* host_qtab,
                       uint8_t* dev_rgb, void* stream);

/* Test hook for the bounded device-side wait behind PCR_E_TIMEOUT (the paper has no counterpart):
 * launches one warp that waits, with the decoder's own wait routine and a limit of 2000 polls,
 * for a flag that nothing sets.  *gave_up = 1 if the wait ended by its limit (the kernel returns
 * normally and the context stays usable), 0 if it claims to have seen the flag.
 * Errors: PCR_E_ARG, PCR_E_NOMEM, PCR_E_CUDA. */
int pcr_selftest_bounded_wait(int* gave_up);

/* Counts kernel launches issued by this library since it was loaded (all records). */
uint64_t pcr_launch_count(void);

/* Text for a status code. */
const char* pcr_strerror(int code);

/* Frees the record's host state and gives its device buffers up.  Waits for the last decode
 * enqueued on this record (not for the whole device).  NULL is allowed.  The borrowed bytes are
 * not touched.  The device buffers are kept in a per-process cache (up to 24 GiB) and handed to
 * later pcr_open calls, so that a loader that opens and closes record after record does not pay
 * cudaMalloc/cudaFree each time. */
void pcr_close(pcr_record* rec);

/* Cache of closed records (Section 5: a loader reads the same records epoch after epoch).  With a
 * limit above zero pcr_close parks the whole record (parse results, device tables and buffers:
 * about 1.5 GB for a 1024-image ImageNet-shaped record) instead of freeing it, and a later pcr_open
 * of the same record takes it back, which saves the host-side walk over every image's marker
 * segments and the table uploads (about 0.7 ms per 1024 images).  The handle it returns is fresh:
 * nothing resident, nothing decoded, default settings.  A record is recognised by the address and
 * length of its bytes, the PCR_SLICES / PCR_LONG_MIN_BYTES settings, the current device, and a
 * hash of its header, sample metadata, index (position and length of every chunk) and the first
 * 256 bytes of every image's first chunk (frame header, quantisation and Huffman tables).  Bytes
 * that changed elsewhere under the same address are the caller's responsibility, exactly as for
 * an open handle.
 *   max_device_bytes : device memory the parked records may hold together; the least recently
 *                      closed ones are freed beyond it; 0 (the default) switches the cache off
 *                      and frees what it holds.
 * Errors: none (always PCR_OK). */
int pcr_set_record_cache(size_t max_device_bytes);

/* Returns the cached device buffers of closed records (and parked records) to the driver. */
void pcr_release_cached_memory(void);

#ifdef __cplusplus
}
#endif
#endif /* PCR_H_ */
