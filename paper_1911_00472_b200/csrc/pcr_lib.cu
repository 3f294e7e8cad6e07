// Host side of the PCR decoder and its C ABI (see include/pcr.h).
//
// pcr_open walks the record's metadata and every image's JPEG marker segments once, on the
// host, and turns them into flat device tables (per (scan, image) byte ranges and Huffman
// table positions, per image geometry, work lists).  pcr_decode only enqueues work: the
// prefix copy, the restart-interval index, one entropy kernel per dependency wave of the
// scan script, and the fused pixel kernel.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <atomic>
#include <map>
#include <mutex>
#include <new>
#include <thread>
#include <utility>
#include <vector>

#include "../../include/pcr.h"
#include "pcr_entropy.cuh"
#include "pcr_long.cuh"
#include "pcr_msssim.cuh"
#include "pcr_pixels.cuh"
#include "pcr_types.h"

using namespace pcr;

static std::atomic<uint64_t> g_launches{0};

// Device buffers of closed records are kept for the next pcr_open instead of going back to the
// driver: cudaMalloc and cudaFree cost milliseconds and cudaFree waits for the whole device, which
// a loader that opens and closes one record after the other cannot afford.  Sizes are rounded up
// to classes with three mantissa bits (at most 12.5 % slack) so that records of similar size
// reuse each other's buffers.
namespace {
struct DeviceCache {
    std::mutex mu;
    std::multimap<std::pair<int, size_t>, void*> free_;
    size_t cached = 0;
    static constexpr size_t kLimit = 24ull << 30;
} g_cache;

size_t size_class(size_t n) {
    if (n < 4096) return 4096;
    int top = 63 - __builtin_clzll((unsigned long long)n);
    const size_t step = (size_t)1 << (top - 3);
    return (n + step - 1) & ~(step - 1);
}

void* dev_alloc(size_t n, int device) {
    const size_t cls = size_class(n);
    {
        std::lock_guard<std::mutex> lk(g_cache.mu);
        auto it = g_cache.free_.find({device, cls});
        if (it != g_cache.free_.end()) {
            void* p = it->second;
            g_cache.free_.erase(it);
            g_cache.cached -= cls;
            return p;
        }
    }
    void* p = nullptr;
    if (cudaMalloc(&p, cls) != cudaSuccess) {
        cudaGetLastError();
        // give cached buffers back and try once more
        std::lock_guard<std::mutex> lk(g_cache.mu);
        for (auto& kv : g_cache.free_) cudaFree(kv.second);
        g_cache.free_.clear();
        g_cache.cached = 0;
        if (cudaMalloc(&p, cls) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    }
    return p;
}

// internal streams and (non-timing) events are pooled the same way
struct HandlePool {
    std::mutex mu;
    std::multimap<int, cudaStream_t> streams;
    std::multimap<int, cudaEvent_t> events;
} g_handles;

cudaStream_t pool_stream_get(int device) {
    {
        std::lock_guard<std::mutex> lk(g_handles.mu);
        auto it = g_handles.streams.find(device);
        if (it != g_handles.streams.end()) { cudaStream_t q = it->second; g_handles.streams.erase(it); return q; }
    }
    cudaStream_t q = nullptr;
    if (cudaStreamCreateWithFlags(&q, cudaStreamNonBlocking) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return q;
}
void pool_stream_put(cudaStream_t q, int device) {
    if (!q) return;
    std::lock_guard<std::mutex> lk(g_handles.mu);
    g_handles.streams.insert({device, q});
}
cudaEvent_t pool_event_get(int device) {
    {
        std::lock_guard<std::mutex> lk(g_handles.mu);
        auto it = g_handles.events.find(device);
        if (it != g_handles.events.end()) { cudaEvent_t e = it->second; g_handles.events.erase(it); return e; }
    }
    cudaEvent_t e = nullptr;
    if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return e;
}
void pool_event_put(cudaEvent_t e, int device) {
    if (!e) return;
    std::lock_guard<std::mutex> lk(g_handles.mu);
    g_handles.events.insert({device, e});
}

void dev_release(void* p, size_t n, int device) {
    if (!p) return;
    const size_t cls = size_class(n);
    std::lock_guard<std::mutex> lk(g_cache.mu);
    if (g_cache.cached + cls <= DeviceCache::kLimit) {
        g_cache.free_.insert({{device, cls}, p});
        g_cache.cached += cls;
    } else {
        cudaFree(p);
    }
}
}  // namespace

struct pcr_record {
    const uint8_t* host = nullptr;
    size_t len = 0;
    int N = 0, G = 0;
    std::vector<uint64_t> group_end;
    std::vector<pcr_image_info> info;
    std::vector<uint64_t> blk_base, nblk;
    uint64_t total_blocks = 0, total_segs = 0;
    int hs = 2, vs = 2, nc = 3;     // chroma sampling, the same for every image of the record
    uint32_t unit_mcus = kPixMcus;  // MCUs of a pixel work unit
    unsigned dc_refine_chunks = 1;  // 256-MCU chunks of the largest image, at most 8 (dc_refine_kernel's grid)
    bool widths_mult16 = true;    // every image is a multiple of 16 pixels wide (the DC-only pixel kernel's condition)
    size_t out_bytes = 0;
    // scan script analysis
    std::vector<ScanScript> script;
    std::vector<int> wave_of_scan;
    int n_waves = 0;
    // images are cut into slices that run as independent pipelines on their own streams;
    // items are sorted by (slice, wave, scan), units by image
    int n_slices = 1;
    std::vector<uint32_t> slice_img;                            // [n_slices + 1] first image of each slice
    std::vector<uint32_t> slice_unit;                           // [n_slices + 1] first pixel unit of each slice
    std::vector<uint32_t> item_begin, item_count;               // [n_slices][G]
    // Scans that are one long restart interval take kernels of their own (pcr_long.cuh): first passes
    // as (scan, image) pairs sorted by (slice, wave, scan); AC refinements as (component, image)
    // groups sorted by slice (all refinement scans of the component that a call decodes, in one CTA)
    std::vector<uint32_t> long_begin, long_count;               // [n_slices][G]
    uint32_t* d_long = nullptr;
    uint32_t n_groups = 0;                                      // (image, component) pairs whose AC refinements are chains
    uint32_t* d_group = nullptr;                                // luminance first, most bytes first
    uint32_t* d_chain_sync = nullptr;                           // queue counters and progress words of the chain launch
    int n_sms = 1;
    cudaEvent_t ev_chain = nullptr;
    std::vector<cudaStream_t> streams;                          // one per slice
    std::vector<cudaEvent_t> ev_index;                          // [n_waves] index of wave w done (side stream)
    cudaEvent_t ev_start = nullptr;                             // index of the first wave done
    cudaEvent_t ev_fork = nullptr;
    cudaStream_t copy_stream = nullptr;                         // host-to-device copies of later scan groups
    cudaStream_t clear_stream = nullptr;                        // zeroing of the planes, beside the index kernels
    cudaEvent_t ev_clear = nullptr;
    std::vector<cudaEvent_t> ev_copy;                           // [n_waves] bytes of wave w have arrived
    std::vector<cudaEvent_t> ev_join;
    std::vector<std::vector<int>> wave_scans;
    uint32_t n_units = 0;
    // device state
    int device = 0;
    uint8_t* d_rec = nullptr;
    uint8_t* d_ubuf = nullptr;
    size_t resident = 0;
    int16_t* d_planes = nullptr;
    int16_t* d_head = nullptr;
    int decoded_k = 0;            // fidelity of the state the planes and side data hold (0: none)
    bool dc_merged = true;        // the planes hold the DC coefficients of the last decode
    bool planes_cleared = true;   // ... and zeros wherever the last decode left no coefficient
    ScanScript* d_script = nullptr;
    ScanAux* d_saux = nullptr;
    uint64_t* d_aux = nullptr;
    std::vector<ScanAux> saux;
    ScanDesc* d_scans = nullptr;
    ImgDesc* d_imgs = nullptr;
    uint32_t* d_seg = nullptr;
    Item* d_items = nullptr;
    Unit* d_units = nullptr;
    uint32_t* d_unit_prefix = nullptr;
    uint16_t* d_qtab = nullptr;
    uint32_t* d_order = nullptr;  // processing order of the images (slices are runs of it)
    MsDesc* d_ms = nullptr;       // per-image table of pcr_msssim (built on first use)
    size_t ms_scratch = 0;        // bytes of scratch pcr_msssim needs
    uint64_t ms_floats = 0;       // floats of all pyramids (the sums follow them)
    int upsampling = PCR_UPSAMPLE_REPLICATE;
    uint8_t* d_chroma = nullptr;  // chroma sample planes between the two passes of triangle upsampling
    CropRect* d_crops = nullptr;  // crop rectangles of the last pcr_decode_tensor (allocated on first use)
    int* d_status = nullptr;
    std::vector<int> h_status;
    std::vector<std::pair<void*, size_t>> bufs;   // every device buffer of the record with its size
    cudaStream_t up_stream = nullptr;             // pcr_open's uploads and memsets (never the default stream:
                                                  // that one would wait for every other record's decode)
    cudaEvent_t ev_ready = nullptr;               // the record's device state is set up
    cudaEvent_t ev_done = nullptr;                // end of the last decode enqueued
    bool decode_enqueued = false;
    // identity of the record for the cache of closed records (pcr_set_record_cache): valid when key_len != 0
    uint64_t key_hash = 0;
    size_t key_len = 0;
    uint32_t key_env = 0;                         // the tuning variables read when it was opened
    size_t device_bytes = 0;                      // what its device buffers add up to
    // optional stage timing
    bool profiling = false;
    std::vector<cudaEvent_t> events;
    std::vector<pcr_stage_time> stages;   // names and launch counts of the last decode
};

static const int kMaxStages = 16;

static inline uint32_t rd32(const uint8_t* p) { return (uint32_t)p[0] | ((uint32_t)p[1] << 8) | ((uint32_t)p[2] << 16) | ((uint32_t)p[3] << 24); }
static inline uint64_t rd64(const uint8_t* p) { return (uint64_t)rd32(p) | ((uint64_t)rd32(p + 4) << 32); }

// Writes the list of pixel work units at set-up: block = position of the processing order.
__global__ void __launch_bounds__(128) units_kernel(const ImgDesc* __restrict__ imgs, const uint32_t* __restrict__ order,
                                                    const uint32_t* __restrict__ prefix, Unit* __restrict__ units, uint32_t unit_mcus) {
    const uint32_t img = order[blockIdx.x];
    const uint32_t per_row = (imgs[img].mx + unit_mcus - 1) / unit_mcus, n = per_row * imgs[img].my;
    Unit* dst = units + prefix[blockIdx.x];
    for (uint32_t j = threadIdx.x; j < n; j += 128) {
        Unit un;
        un.img = img; un.mrow = (uint16_t)(j / per_row); un.mcol0 = (uint16_t)((j % per_row) * unit_mcus);
        dst[j] = un;
    }
}

namespace {

struct TableRef { uint32_t off = 0; };   // offset of the 16 length counts of a DHT table body; 0 = undefined

struct ImageParse {
    uint32_t W = 0, H = 0;
    int cid[3] = {0, 0, 0}, tq[3] = {0, 0, 0};
    uint16_t q[4][64];
    bool qdef[4] = {false, false, false, false};
    TableRef dc[4], ac[4];
    uint32_t ri = 0;
    bool have_frame = false;
    bool sequential = false;      // SOF0: one interleaved scan carries whole blocks
    int hs = 2, vs = 2, nc = 3;   // luminance blocks per MCU, components
};

struct ScanParse {
    ScanScript sc;
    uint32_t tab[3];       // table body offset per scan component (0 when the scan uses none)
    uint32_t tab_ac[3];    // sequential scans: the AC table per component (tab then holds the DC tables)
    uint32_t data_off, data_end, ri;
};

// Validate one DHT table body at p (inside [p, end)): returns its length or 0.
size_t check_dht_body(const uint8_t* p, size_t avail) {
    if (avail < 16) return 0;
    uint32_t code = 0, n = 0;
    for (int l = 1; l <= 16; ++l) {
        code += p[l - 1];
        n += p[l - 1];
        if (code > (1u << l)) return 0;
        code <<= 1;
    }
    if (n > 256 || 16 + (size_t)n > avail) return 0;
    return 16 + n;
}

// Walk the marker segments of chunk [off, off+len) of one image up to and including its SOS.
int parse_chunk(const uint8_t* rec, uint64_t off, uint32_t len, bool first, ImageParse& im, ScanParse& out) {
    uint64_t p = off, end = off + len;
    if (first) {
        if (len < 4 || rec[p] != 0xFF || rec[p + 1] != 0xD8) return PCR_E_FORMAT;
        p += 2;
    }
    for (;;) {
        if (p + 4 > end || rec[p] != 0xFF) return PCR_E_FORMAT;
        while (p < end && rec[p] == 0xFF) ++p;
        if (p >= end) return PCR_E_FORMAT;
        int mk = rec[p++];
        if (p + 2 > end) return PCR_E_FORMAT;
        uint32_t L = ((uint32_t)rec[p] << 8) | rec[p + 1];
        if (L < 2 || p + L > end) return PCR_E_FORMAT;
        const uint8_t* s = rec + p + 2;
        uint32_t sl = L - 2;
        if (mk == 0xDB) {
            uint32_t q = 0;
            while (q < sl) {
                int pq = s[q] >> 4, tq = s[q] & 15;
                ++q;
                if (tq > 3 || pq > 1 || q + (pq ? 128u : 64u) > sl) return PCR_E_FORMAT;
                for (int k = 0; k < 64; ++k) {
                    im.q[tq][k] = pq ? (uint16_t)((s[q] << 8) | s[q + 1]) : s[q];
                    q += pq ? 2 : 1;
                }
                im.qdef[tq] = true;
            }
        } else if (mk == 0xC2 || mk == 0xC0) {            // progressive / baseline sequential, Huffman
            if (im.have_frame || sl < 9 || s[0] != 8 || (s[5] != 3 && s[5] != 1) || sl < 6u + 3u * s[5]) return PCR_E_FORMAT;
            im.sequential = mk == 0xC0;
            im.H = ((uint32_t)s[1] << 8) | s[2];
            im.W = ((uint32_t)s[3] << 8) | s[4];
            im.nc = s[5];
            for (int c = 0; c < im.nc; ++c) {
                im.cid[c] = s[6 + 3 * c];
                int hv = s[7 + 3 * c];
                im.tq[c] = s[8 + 3 * c];
                if (im.tq[c] > 3) return PCR_E_FORMAT;
                // luminance 1 or 2 blocks per MCU in each direction, chroma one: 4:4:4, 4:2:2, 4:4:0, 4:2:0
                if (c == 0) { im.hs = hv >> 4; im.vs = hv & 15; if (im.hs < 1 || im.hs > 2 || im.vs < 1 || im.vs > 2) return PCR_E_FORMAT; }
                else if (hv != 0x11) return PCR_E_FORMAT;
            }
            if (im.nc == 1) im.hs = im.vs = 1;                // a lone component is never interleaved: no MCU padding
            if (im.W == 0 || im.H == 0) return PCR_E_FORMAT;
            im.have_frame = true;
        } else if (mk == 0xC4) {
            uint32_t q = 0;
            while (q < sl) {
                int tc = s[q] >> 4, th = s[q] & 15;
                if (tc > 1 || th > 3) return PCR_E_FORMAT;
                size_t n = check_dht_body(s + q + 1, sl - q - 1);
                if (!n) return PCR_E_FORMAT;
                (tc ? im.ac[th] : im.dc[th]).off = (uint32_t)(p + 2 + q + 1);
                q += 1 + (uint32_t)n;
            }
        } else if (mk == 0xDD) {
            if (sl != 2) return PCR_E_FORMAT;
            im.ri = ((uint32_t)s[0] << 8) | s[1];
        } else if (mk == 0xDA) {
            if (!im.have_frame || sl < 1) return PCR_E_FORMAT;
            int ns = s[0];
            if (ns < 1 || ns > 3 || sl != (uint32_t)(4 + 2 * ns)) return PCR_E_FORMAT;
            ScanScript& sc = out.sc;
            memset(&sc, 0, sizeof sc);
            sc.ncomp = ns;
            int td[3] = {0, 0, 0}, ta[3] = {0, 0, 0};
            for (int i = 0; i < ns; ++i) {
                int id = s[1 + 2 * i], found = -1;
                for (int c = 0; c < im.nc; ++c) if (im.cid[c] == id) found = c;
                if (found < 0) return PCR_E_FORMAT;
                for (int j = 0; j < i; ++j) if (sc.comp[j] >= found) return PCR_E_FORMAT;   // frame order
                sc.comp[i] = found;
                td[i] = s[2 + 2 * i] >> 4;
                ta[i] = s[2 + 2 * i] & 15;
                if (td[i] > 3 || ta[i] > 3) return PCR_E_FORMAT;
            }
            sc.Ss = s[1 + 2 * ns]; sc.Se = s[2 + 2 * ns];
            sc.Ah = s[3 + 2 * ns] >> 4; sc.Al = s[3 + 2 * ns] & 15;
            if (sc.Ss > sc.Se || sc.Se > 63 || sc.Al > 13) return PCR_E_FORMAT;
            if (im.sequential) {
                if (sc.Ss != 0 || sc.Se != 63 || sc.Ah != 0 || sc.Al != 0 || ns != im.nc) return PCR_E_FORMAT;
            } else if (sc.Ss == 0 && sc.Se != 0) return PCR_E_FORMAT;
            if (sc.Ss > 0 && ns != 1) return PCR_E_FORMAT;
            if (ns > 1 && ns != im.nc) return PCR_E_FORMAT; // interleaved scans hold all three components
            if (sc.Ah != 0 && sc.Ah != sc.Al + 1) return PCR_E_FORMAT;
            for (int i = 0; i < 3; ++i) out.tab[i] = out.tab_ac[i] = 0;
            for (int i = 0; i < ns && im.sequential; ++i) {
                out.tab_ac[i] = im.ac[ta[i]].off;
                if (!out.tab_ac[i]) return PCR_E_FORMAT;
            }
            for (int i = 0; i < ns; ++i) {
                if (sc.Ss == 0 && sc.Ah == 0) { out.tab[i] = im.dc[td[i]].off; if (!out.tab[i]) return PCR_E_FORMAT; }
                if (sc.Ss > 0) { out.tab[i] = im.ac[ta[i]].off; if (!out.tab[i]) return PCR_E_FORMAT; }
            }
            out.data_off = (uint32_t)(p + L);
            out.data_end = (uint32_t)end;
            out.ri = im.ri;
            return PCR_OK;
        } else if ((mk >= 0xC0 && mk <= 0xCF) || (mk >= 0xD0 && mk <= 0xD9)) {
            return PCR_E_FORMAT;     // other frame types, stray restart / SOI / EOI markers
        }
        p += L;
    }
}

void free_device(pcr_record* r) {
    // nothing is handed on before the record's set-up and its last decode have finished
    if (r->up_stream) cudaStreamSynchronize(r->up_stream);
    if (r->ev_done && r->decode_enqueued) cudaEventSynchronize(r->ev_done);
    if (r->ev_ready) pool_event_put(r->ev_ready, r->device);
    r->ev_ready = nullptr;
    if (r->up_stream) pool_stream_put(r->up_stream, r->device);
    r->up_stream = nullptr;
    r->decode_enqueued = false;
    for (cudaStream_t q : r->streams) pool_stream_put(q, r->device);
    r->streams.clear();
    if (r->ev_start) pool_event_put(r->ev_start, r->device);
    r->ev_start = nullptr;
    if (r->ev_chain) pool_event_put(r->ev_chain, r->device);
    r->ev_chain = nullptr;
    for (cudaEvent_t e : r->ev_index) pool_event_put(e, r->device);
    r->ev_index.clear();
    if (r->ev_fork) pool_event_put(r->ev_fork, r->device);
    r->ev_fork = nullptr;
    if (r->copy_stream) pool_stream_put(r->copy_stream, r->device);
    r->copy_stream = nullptr;
    if (r->clear_stream) pool_stream_put(r->clear_stream, r->device);
    r->clear_stream = nullptr;
    if (r->ev_clear) pool_event_put(r->ev_clear, r->device);
    r->ev_clear = nullptr;
    for (cudaEvent_t e : r->ev_copy) pool_event_put(e, r->device);
    r->ev_copy.clear();
    for (cudaEvent_t e : r->ev_join) pool_event_put(e, r->device);
    r->ev_join.clear();
    for (cudaEvent_t e : r->events) cudaEventDestroy(e);
    r->events.clear();
    // buffers go back to the cache once the record's last decode has finished
    if (r->ev_done) {
        if (r->decode_enqueued) cudaEventSynchronize(r->ev_done);
        pool_event_put(r->ev_done, r->device);
        r->ev_done = nullptr;
    }
    for (auto& b : r->bufs) dev_release(b.first, b.second, r->device);
    r->bufs.clear();
}

template <class T>
int take(pcr_record* r, T** dst, size_t bytes) {
    *dst = static_cast<T*>(dev_alloc(bytes, r->device));
    if (!*dst) return PCR_E_NOMEM;
    r->bufs.push_back({*dst, bytes});
    return PCR_OK;
}

template <class T>
int upload(pcr_record* r, T** dst, const std::vector<T>& v) {
    size_t n = std::max<size_t>(v.size(), 1) * sizeof(T);
    if (int rc = take(r, dst, n)) return rc;
    // pageable source: the call returns once the bytes sit in the driver's staging memory
    if (!v.empty() && cudaMemcpyAsync(*dst, v.data(), v.size() * sizeof(T), cudaMemcpyHostToDevice, r->up_stream) != cudaSuccess) return PCR_E_CUDA;
    return PCR_OK;
}

int open_impl(const uint8_t* rec, size_t len, pcr_record* r) {
    if (len < 64 || len >= (1ull << 32)) return PCR_E_FORMAT;
    if (memcmp(rec, "PCR1", 4) != 0 || rd32(rec + 4) != 1) return PCR_E_FORMAT;
    uint32_t N = rd32(rec + 8), G = rd32(rec + 12);
    uint64_t meta_off = rd64(rec + 24), index_off = rd64(rec + 32), data_off = rd64(rec + 40), total = rd64(rec + 48);
    if (N == 0 || G == 0 || G > 64 || N > (1u << 24)) return PCR_E_FORMAT;
    if (total != len) return PCR_E_FORMAT;
    if (meta_off < 64 || meta_off + 16ull * N > len) return PCR_E_FORMAT;
    if (index_off < 64 || index_off + 8ull * (G + 1) + 16ull * G * N > len) return PCR_E_FORMAT;
    if (data_off > len || data_off < index_off + 8ull * (G + 1) + 16ull * G * N) return PCR_E_FORMAT;
    r->host = rec; r->len = len; r->N = (int)N; r->G = (int)G;
    r->group_end.resize(G + 1);
    for (uint32_t g = 0; g <= G; ++g) r->group_end[g] = rd64(rec + index_off + 8ull * g);
    if (r->group_end[0] != data_off) return PCR_E_FORMAT;
    for (uint32_t g = 1; g <= G; ++g)
        if (r->group_end[g] < r->group_end[g - 1] || r->group_end[g] > len) return PCR_E_FORMAT;
    const uint8_t* chunk = rec + index_off + 8ull * (G + 1);

    std::vector<ScanDesc> scans((size_t)G * N);
    std::vector<ImgDesc> imgs(N);
    std::vector<uint16_t> qtab((size_t)N * 192);
    r->info.resize(N); r->blk_base.resize(N); r->nblk.resize(N);
    r->script.resize(G);
    // every image's chunks are walked independently (a few host threads for large records); the
    // running sums over images follow in one serial pass
    std::vector<ScanScript> scripts((size_t)N * G);
    std::vector<uint8_t> samplings(N, 0);
    auto parse_image = [&](uint32_t i) -> int {
        ImageParse im;
        const uint8_t* m = rec + meta_off + 16ull * i;
        for (uint32_t g = 0; g < G; ++g) {
            const uint8_t* c = chunk + 16ull * ((uint64_t)g * N + i);
            uint64_t off = rd64(c);
            uint32_t clen = rd32(c + 8);
            uint64_t padded = ((uint64_t)clen + 15) & ~15ull;
            if ((off & 15) || off < r->group_end[g] || off + padded > r->group_end[g + 1]) return PCR_E_FORMAT;
            if (clen >= (1u << 28)) return PCR_E_FORMAT;        // bit positions inside a scan are 32-bit
            ScanParse sp;
            int rc = parse_chunk(rec, off, clen, g == 0, im, sp);
            if (rc) return rc;
            scripts[(size_t)i * G + g] = sp.sc;
            ScanDesc& sd = scans[(size_t)g * N + i];
            sd.data_off = sp.data_off; sd.data_end = sp.data_end; sd.ri = sp.ri;
            // up to two distinct tables per scan
            sd.tab_ac[0] = sp.tab_ac[0]; sd.tab_ac[1] = 0; sd.slots_ac = 0;
            for (int ci = 1; ci < sp.sc.ncomp && sp.tab_ac[0]; ++ci) {
                if (sp.tab_ac[ci] == sd.tab_ac[0]) continue;
                if (sd.tab_ac[1] == 0) sd.tab_ac[1] = sp.tab_ac[ci];
                if (sp.tab_ac[ci] != sd.tab_ac[1]) return PCR_E_FORMAT;
                sd.slots_ac |= 1u << (2 * ci);
            }
            sd.tab_off[0] = sp.tab[0]; sd.tab_off[1] = 0; sd.slots = 0;
            for (int ci = 1; ci < sp.sc.ncomp; ++ci) {
                if (sp.tab[ci] == sd.tab_off[0]) continue;
                if (sd.tab_off[1] == 0) sd.tab_off[1] = sp.tab[ci];
                if (sp.tab[ci] != sd.tab_off[1]) return PCR_E_FORMAT;
                sd.slots |= 1u << (2 * ci);
            }
            uint32_t mx = (im.W + 8 * im.hs - 1) / (8 * im.hs), my = (im.H + 8 * im.vs - 1) / (8 * im.vs);
            uint64_t total_mcu;
            if (sp.sc.ncomp > 1) total_mcu = (uint64_t)mx * my;
            else {
                uint32_t wc = sp.sc.comp[0] == 0 ? im.W : (im.W + im.hs - 1) / im.hs, hc = sp.sc.comp[0] == 0 ? im.H : (im.H + im.vs - 1) / im.vs;
                total_mcu = (uint64_t)((wc + 7) / 8) * ((hc + 7) / 8);
            }
            sd.nseg = sd.ri ? (uint32_t)((total_mcu + sd.ri - 1) / sd.ri) : 1u;
        }
        if (!im.have_frame) return PCR_E_FORMAT;
        if (rd32(m + 4) != im.W || rd32(m + 8) != im.H) return PCR_E_FORMAT;   // metadata and frame header agree
        for (int c = 0; c < im.nc; ++c) {
            if (!im.qdef[im.tq[c]]) return PCR_E_FORMAT;
            memcpy(&qtab[(size_t)i * 192 + 64 * c], im.q[im.tq[c]], 128);
        }
        samplings[i] = (uint8_t)(im.hs | (im.vs << 2) | (im.nc << 4));
        pcr_image_info& inf = r->info[i];
        inf.width = im.W; inf.height = im.H; inf.label = (int32_t)rd32(m); inf.rsvd = 0;
        inf.out_bytes = 3ull * im.W * im.H;
        imgs[i].W = im.W; imgs[i].H = im.H;
        imgs[i].mx = (im.W + 8 * im.hs - 1) / (8 * im.hs); imgs[i].my = (im.H + 8 * im.vs - 1) / (8 * im.vs);
        return PCR_OK;
    };
    {
        const unsigned hw = std::max(1u, std::thread::hardware_concurrency());
        const unsigned nthreads = N >= 256 ? std::min(4u, hw) : 1u;
        std::vector<int> rcs(nthreads, PCR_OK);
        auto work = [&](unsigned t) {
            for (uint32_t i = t; i < N; i += nthreads) {
                const int rc = parse_image(i);
                if (rc != PCR_OK) { rcs[t] = rc; return; }
            }
        };
        std::vector<std::thread> pool;
        for (unsigned t = 1; t < nthreads; ++t) pool.emplace_back(work, t);
        work(0);
        for (auto& th : pool) th.join();
        for (int rc : rcs) if (rc != PCR_OK) return rc;
    }
    uint64_t blocks = 0, out_off = 0, segs = 0;
    r->hs = samplings[0] & 3; r->vs = (samplings[0] >> 2) & 3; r->nc = samplings[0] >> 4;
    const uint32_t bpm = (uint32_t)(r->hs * r->vs + (r->nc == 3 ? 2 : 0));      // blocks per MCU
    r->unit_mcus = r->nc == 3 && r->hs == 2 ? 8u : 16u;                         // a work unit is 128 pixels wide
    for (uint32_t g = 0; g < G; ++g) r->script[g] = scripts[g];
    for (uint32_t i = 0; i < N; ++i) {
        if (i && memcmp(&scripts[(size_t)i * G], &scripts[0], sizeof(ScanScript) * G) != 0) return PCR_E_FORMAT;   // one script per record
        for (uint32_t g = 0; g < G; ++g) {
            ScanDesc& sd = scans[(size_t)g * N + i];
            sd.seg_base = (uint32_t)segs;
            segs += sd.nseg + 1;                      // one closing entry per (scan, image)
            if (segs >= (1ull << 32)) return PCR_E_FORMAT;
        }
        pcr_image_info& inf = r->info[i];
        inf.out_offset = out_off;
        out_off += (inf.out_bytes + 127) & ~127ull;
        if (imgs[i].W & 15u) r->widths_mult16 = false;
        r->dc_refine_chunks = std::max(r->dc_refine_chunks, std::min(8u, (imgs[i].mx * imgs[i].my + 255u) / 256u));
        if (samplings[i] != samplings[0]) return PCR_E_FORMAT;                                  // one sampling per record
        r->blk_base[i] = blocks; r->nblk[i] = (uint64_t)bpm * imgs[i].mx * imgs[i].my;
        imgs[i].blk_base = blocks; imgs[i].out_off = inf.out_offset;
        blocks += r->nblk[i];
    }
    // 16 spare bytes behind the last image: the tensor epilogue reads pixels as aligned words and may
    // touch up to 8 bytes past a pixel pair
    r->total_blocks = blocks; r->out_bytes = out_off + 16; r->total_segs = segs;

    // dependency waves of the script: a scan waits for every earlier scan that touches an
    // overlapping coefficient band of one of its components
    r->wave_of_scan.assign(G, 0);
    for (uint32_t s = 0; s < G; ++s) {
        int w = 0;
        for (uint32_t t = 0; t < s; ++t) {
            bool share = false;
            for (int a = 0; a < r->script[s].ncomp; ++a)
                for (int b = 0; b < r->script[t].ncomp; ++b)
                    if (r->script[s].comp[a] == r->script[t].comp[b]) share = true;
            if (share && r->script[s].Ss <= r->script[t].Se && r->script[t].Ss <= r->script[s].Se)
                w = std::max(w, r->wave_of_scan[t] + 1);
        }
        r->wave_of_scan[s] = w;
        r->n_waves = std::max(r->n_waves, w + 1);
    }
    r->wave_scans.assign(r->n_waves, {});
    for (uint32_t s = 0; s < G; ++s) r->wave_scans[r->wave_of_scan[s]].push_back((int)s);
    // slices: enough images each to fill the machine, few enough to keep launches cheap
    {
        // four at most: one record decodes as fast with four slices as with eight, and two records
        // in flight then stay close to the eight hardware queues that streams are mapped onto
        int want = (int)std::min<uint32_t>(4, std::max<uint32_t>(1, N / 128));
        if (const char* e = getenv("PCR_SLICES")) want = std::max(1, std::min(64, atoi(e)));
        r->n_slices = (int)std::min<uint32_t>((uint32_t)want, N);
        r->slice_img.resize(r->n_slices + 1);
        for (int g = 0; g <= r->n_slices; ++g) r->slice_img[g] = (uint32_t)((uint64_t)N * g / r->n_slices);
    }
    // Processing order of the images: a slice is a run of this order.  The time a slice needs for
    // its entropy waves is set by its longest restart intervals, so the images are sorted by their
    // entropy-coded bytes per MCU row, most first: the slice of the heaviest rows starts first, slices
    // of light images finish their waves early and their pixel stage overlaps the waves of the heavy
    // ones.  (By width alone, the first version of this order: 2 % slower on the ImageNet-shaped record.)
    std::vector<uint32_t> order(N);
    for (uint32_t i = 0; i < N; ++i) order[i] = i;
    if (r->n_slices > 1) {
        std::vector<double> key(N);
        for (uint32_t i = 0; i < N; ++i) {
            uint64_t b = 0;
            for (uint32_t s2 = 0; s2 < G; ++s2) b += scans[(size_t)s2 * N + i].data_end - scans[(size_t)s2 * N + i].data_off;
            key[i] = (double)b / (double)std::max<uint32_t>(1, imgs[i].my);
        }
        std::stable_sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) { return key[a] > key[b]; });
    }
    std::vector<Item> items;
    items.reserve((size_t)(segs / 24 + (uint64_t)N * G));
    r->item_begin.assign((size_t)r->n_slices * G, 0); r->item_count.assign((size_t)r->n_slices * G, 0);
    // A scan that is one restart interval of at least this many bytes goes to the kernels for long
    // intervals; DC refinement scans have a kernel of their own and no items at all.
    uint32_t long_min = 64;
    if (const char* e = getenv("PCR_LONG_MIN_BYTES")) long_min = (uint32_t)std::max(0, atoi(e));
    auto is_long = [&](int s, uint32_t i) {
        const ScanScript& sc = r->script[s];
        const ScanDesc& sd = scans[(size_t)s * N + i];
        (void)sc;
        return sd.nseg == 1 && sd.data_end - sd.data_off >= long_min;
    };
    // the AC refinements of one component of one image go together: all of them one interval each,
    // at least one of them long
    std::vector<uint8_t> grouped((size_t)N * 3, 0);
    for (uint32_t i = 0; i < N; ++i)
        for (int c = 0; c < 3; ++c) {
            bool any = false, one_interval = true, big = false;
            for (uint32_t s = 0; s < G; ++s) {
                const ScanScript& sc = r->script[s];
                if (sc.Ss == 0 || sc.Ah == 0 || sc.comp[0] != c) continue;
                any = true;
                one_interval = one_interval && scans[(size_t)s * N + i].nseg == 1;
                big = big || is_long((int)s, i);
            }
            grouped[(size_t)i * 3 + c] = any && one_interval && big;
        }
    auto takes_long_kernel = [&](int s, uint32_t i) {
        const ScanScript& sc = r->script[s];
        if (sc.Ss > 0 && sc.Ah != 0) return grouped[(size_t)i * 3 + sc.comp[0]] != 0;
        return is_long(s, i);
    };
    std::vector<uint32_t> longs, groups;
    r->long_begin.assign((size_t)r->n_slices * G, 0); r->long_count.assign((size_t)r->n_slices * G, 0);
    for (int g = 0; g < r->n_slices; ++g) {
        for (int w = 0; w < r->n_waves; ++w)
            for (int s : r->wave_scans[w]) {
                const ScanScript& sc = r->script[s];
                if (sc.Ah != 0) continue;                      // first passes only
                r->long_begin[(size_t)g * G + s] = (uint32_t)longs.size();
                for (uint32_t pos = r->slice_img[g]; pos < r->slice_img[g + 1]; ++pos)
                    if (is_long(s, order[pos])) longs.push_back((uint32_t)(s * N + order[pos]));
                r->long_count[(size_t)g * G + s] = (uint32_t)longs.size() - r->long_begin[(size_t)g * G + s];
            }
    }
    // one list for the whole record: luminance first (its chains are the longest), within a
    // component the images with the most refinement bytes first
    for (int c = 0; c < 3; ++c) {
        std::vector<std::pair<uint64_t, uint32_t>> byw;
        for (uint32_t i = 0; i < N; ++i) {
            if (!grouped[(size_t)i * 3 + c]) continue;
            uint64_t bytes = 0;
            for (uint32_t s = 0; s < G; ++s) {
                const ScanScript& sc = r->script[s];
                if (sc.Ss > 0 && sc.Ah != 0 && sc.comp[0] == c) bytes += scans[(size_t)s * N + i].data_end - scans[(size_t)s * N + i].data_off;
            }
            byw.push_back({bytes, i});
        }
        std::stable_sort(byw.begin(), byw.end(), [](const std::pair<uint64_t, uint32_t>& a, const std::pair<uint64_t, uint32_t>& b) { return a.first > b.first; });
        for (auto& e : byw) groups.push_back(((uint32_t)c << 28) | e.second);
    }
    r->n_groups = (uint32_t)groups.size();
    for (int g = 0; g < r->n_slices; ++g)
        for (int w = 0; w < r->n_waves; ++w)
            for (int s : r->wave_scans[w]) {
                r->item_begin[(size_t)g * G + s] = (uint32_t)items.size();
                const bool ac = r->script[s].Ss > 0;
                const bool dc_refine = r->script[s].Ss == 0 && r->script[s].Ah != 0;
                for (uint32_t pos = r->slice_img[g]; pos < r->slice_img[g + 1] && !dc_refine; ++pos) {
                    const uint32_t i = order[pos];
                    if (takes_long_kernel((int)s, i)) continue;
                    const ScanDesc& sd = scans[(size_t)s * N + i];
                    // full warps of 32 restart intervals; in AC scans the last warp of an image
                    // runs on into the first intervals of the next image (two tables per warp)
                    uint32_t j = 0;
                    if (ac && !items.empty() && items.back().next == kItemOpen) {     // continued from the previous image
                        Item& prev = items.back();
                        const uint32_t take = std::min<uint32_t>(kSegsPerItem - prev.count, sd.nseg);
                        prev.count += take; prev.next = (uint32_t)(s * N + i) + 1u;
                        j = take;
                    }
                    for (; j < sd.nseg; j += kSegsPerItem) {
                        const uint32_t cnt = std::min<uint32_t>(kSegsPerItem, sd.nseg - j);
                        // kItemOpen marks an unfilled last item that the next image may extend
                        items.push_back(Item{(uint32_t)(s * N + i), j, cnt, (ac && cnt < (uint32_t)kSegsPerItem) ? kItemOpen : 0u});
                    }
                }
                if (!items.empty() && items.back().next == kItemOpen) items.back().next = 0;
                r->item_count[(size_t)g * G + s] = (uint32_t)items.size() - r->item_begin[(size_t)g * G + s];
            }
    // pixel work units (8 MCUs of one MCU row), image by image in processing order, inside an image
    // MCU row by MCU row.  The host only counts them; a small kernel writes the list at set-up.
    std::vector<uint32_t> unit_prefix(N + 1, 0);
    for (uint32_t pos = 0; pos < N; ++pos) {
        const ImgDesc& im = imgs[order[pos]];
        if (im.my > 65535 || im.mx > 65535) return PCR_E_FORMAT;
        const uint64_t nu = (uint64_t)((im.mx + r->unit_mcus - 1) / r->unit_mcus) * im.my;
        if (unit_prefix[pos] + nu >= (1ull << 32)) return PCR_E_FORMAT;
        unit_prefix[pos + 1] = unit_prefix[pos] + (uint32_t)nu;
    }
    r->slice_unit.assign(r->n_slices + 1, 0);
    for (int g = 0; g <= r->n_slices; ++g) r->slice_unit[g] = unit_prefix[r->slice_img[g]];
    r->n_units = unit_prefix[N];

    // side data of the AC scans: one word per block for a first pass, four for a refinement
    const uint64_t total_mcus = blocks / bpm;
    uint64_t aux_words = 0;
    r->saux.assign(G, ScanAux{});
    int n_refine[3] = {0, 0, 0};
    for (uint32_t s = 0; s < G; ++s)
        if (r->script[s].Ss > 0 && r->script[s].Ah > 0 && ++n_refine[r->script[s].comp[0]] > 4) return PCR_E_FORMAT;
    for (uint32_t s = 0; s < G; ++s) {
        const ScanScript& sc = r->script[s];
        ScanAux& ax = r->saux[s];
        if (sc.Ss == 0) continue;
        ax.stride = sc.Ah ? 4u : 1u;
        ax.base = aux_words;
        aux_words += (sc.comp[0] == 0 ? (uint64_t)(r->hs * r->vs) : 1ull) * total_mcus * ax.stride;
        aux_words = (aux_words + 1) & ~1ull;      // 16-byte alignment of every scan's area
        if (sc.Ah) {
            // positions already non-zero = union of the masks of earlier scans on this band; an
            // earlier scan is covered by a later refinement whose band contains its own
            std::vector<int> src;
            for (uint32_t t = 0; t < s; ++t) {
                const ScanScript& st = r->script[t];
                if (st.Ss == 0 || st.comp[0] != sc.comp[0] || st.Ss > sc.Se || sc.Ss > st.Se) continue;
                src.push_back((int)t);
            }
            std::vector<int> keep;
            for (int t : src) {
                bool covered = false;
                for (int u : src)
                    if (u > t && r->script[u].Ah && r->script[u].Ss <= r->script[t].Ss && r->script[u].Se >= r->script[t].Se) covered = true;
                if (!covered) keep.push_back(t);
            }
            if (keep.empty() || keep.size() > 4) return PCR_E_FORMAT;
            ax.nsrc = (int)keep.size();
            for (size_t i = 0; i < keep.size(); ++i) ax.src[i] = keep[i];
        }
    }

    // device state
    if (cudaGetDevice(&r->device) != cudaSuccess) return PCR_E_CUDA;
    if (!(r->up_stream = pool_stream_get(r->device))) return PCR_E_CUDA;
    if (int rc = take(r, &r->d_aux, (size_t)(std::max<uint64_t>(aux_words, 2) * 8))) return rc;
    // zeroing is enqueued after the table uploads: a copy from pageable memory first waits for
    // everything already in its stream
    std::vector<std::pair<void*, size_t>> zero;
    zero.push_back({r->d_aux, (size_t)(std::max<uint64_t>(aux_words, 2) * 8)});
    if (int rc = take(r, &r->d_rec, (size_t)(len + 64))) return rc;
    if (int rc = take(r, &r->d_ubuf, (size_t)(len + 256))) return rc;
    zero.push_back({r->d_ubuf, len + 256});
    if (int rc = take(r, &r->d_planes, (size_t)(std::max<uint64_t>(blocks, 1) * 128))) return rc;
    if (int rc = take(r, &r->d_head, (size_t)(std::max<uint64_t>(blocks, 1) * 16))) return rc;
    zero.push_back({r->d_head, (size_t)(std::max<uint64_t>(blocks, 1) * 16)});
    if (int rc = take(r, &r->d_seg, (size_t)((segs + 1) * 4))) return rc;
    if (int rc = take(r, &r->d_status, (size_t)((size_t)N * 4))) return rc;
    zero.push_back({r->d_seg, (size_t)((segs + 1) * 4)});
    zero.push_back({r->d_status, (size_t)N * 4});
    int rc;
    if ((rc = upload(r, &r->d_script, r->script))) return rc;
    if ((rc = upload(r, &r->d_saux, r->saux))) return rc;
    if ((rc = upload(r, &r->d_scans, scans))) return rc;
    if ((rc = upload(r, &r->d_imgs, imgs))) return rc;
    if ((rc = upload(r, &r->d_items, items))) return rc;
    if ((rc = upload(r, &r->d_long, longs))) return rc;
    if ((rc = upload(r, &r->d_group, groups))) return rc;
    if (r->n_groups) {
        if ((rc = take(r, &r->d_chain_sync, (size_t)(4 + 4 * (size_t)r->n_groups) * 4))) return rc;
        if (cudaDeviceGetAttribute(&r->n_sms, cudaDevAttrMultiProcessorCount, r->device) != cudaSuccess) return PCR_E_CUDA;
        if (cudaFuncSetAttribute(ac_refine_group_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kChainPairs * sizeof(ChainShared))) != cudaSuccess) return PCR_E_CUDA;
    }
    if ((rc = upload(r, &r->d_qtab, qtab))) return rc;
    if ((rc = upload(r, &r->d_unit_prefix, unit_prefix))) return rc;
    if ((rc = take(r, &r->d_units, (size_t)std::max<uint32_t>(r->n_units, 1) * sizeof(Unit)))) return rc;
    if ((rc = upload(r, &r->d_order, order))) return rc;
    units_kernel<<<N, 128, 0, r->up_stream>>>(r->d_imgs, r->d_order, r->d_unit_prefix, r->d_units, r->unit_mcus);
    ++g_launches;
    for (auto& z : zero)
        if (cudaMemsetAsync(z.first, 0, z.second, r->up_stream) != cudaSuccess) return PCR_E_CUDA;
    r->h_status.assign(N, 0);
    r->resident = 0;
    if (!(r->ev_done = pool_event_get(r->device))) return PCR_E_CUDA;
    // the set-up above runs on the record's own stream; every decode waits for this event first
    if (!(r->ev_ready = pool_event_get(r->device))) return PCR_E_CUDA;
    if (cudaEventRecord(r->ev_ready, r->up_stream) != cudaSuccess) return PCR_E_CUDA;
    if (r->n_slices > 1) {
        if (!(r->ev_fork = pool_event_get(r->device))) return PCR_E_CUDA;
        if (!(r->copy_stream = pool_stream_get(r->device))) return PCR_E_CUDA;
        if (!(r->clear_stream = pool_stream_get(r->device))) return PCR_E_CUDA;
        if (!(r->ev_clear = pool_event_get(r->device))) return PCR_E_CUDA;
        if (!(r->ev_start = pool_event_get(r->device))) return PCR_E_CUDA;
        if (!(r->ev_chain = pool_event_get(r->device))) return PCR_E_CUDA;
        for (int w = 0; w < r->n_waves; ++w) {
            cudaEvent_t e;
            if (!(e = pool_event_get(r->device))) return PCR_E_CUDA;
            r->ev_copy.push_back(e);
            if (!(e = pool_event_get(r->device))) return PCR_E_CUDA;
            r->ev_index.push_back(e);
        }
        for (int g = 0; g < r->n_slices; ++g) {
            cudaStream_t q; cudaEvent_t e;
            if (!(q = pool_stream_get(r->device))) return PCR_E_CUDA;
            r->streams.push_back(q);
            if (!(e = pool_event_get(r->device))) return PCR_E_CUDA;
            r->ev_join.push_back(e);

        }
    }
    return PCR_OK;
}

}  // namespace

// ---------------------------------------------------------------------------------------
// Cache of closed records.  A loader reads the same records epoch after epoch; with the cache
// on, pcr_close parks the whole record (parse results, device tables and buffers) and a later
// pcr_open of the same bytes takes it back instead of walking every image's marker segments and
// uploading the tables again.  A record is recognised by its address, its length, the tuning
// variables in force and a hash of its header, sample metadata, index (position and length of every
// chunk) and the head of every image's first chunk (frame header and tables).
// ---------------------------------------------------------------------------------------
namespace {
struct RecordCache {
    std::mutex mu;
    std::vector<pcr_record*> lru;     // most recently closed last
    size_t bytes = 0, limit = 0;
} g_rcache;

inline uint64_t mix64(uint64_t h, uint64_t v) {
    h ^= v + 0x9E3779B97F4A7C15ull + (h << 6) + (h >> 2);
    h *= 0xFF51AFD7ED558CCDull;
    return h ^ (h >> 29);
}
uint64_t hash_bytes(uint64_t h, const uint8_t* p, size_t n) {
    size_t i = 0;
    for (; i + 8 <= n; i += 8) { uint64_t v; memcpy(&v, p + i, 8); h = mix64(h, v); }
    uint64_t tail = 0;
    if (i < n) { memcpy(&tail, p + i, n - i); h = mix64(h, tail ^ ((uint64_t)(n - i) << 56)); }
    return h;
}
uint32_t env_key() {
    const char* a = getenv("PCR_SLICES"); const char* b = getenv("PCR_LONG_MIN_BYTES");
    return (uint32_t)((a ? atoi(a) + 1 : 0) * 1000003 + (b ? atoi(b) + 1 : 0));
}
// 0 when the bytes do not even look like a record (pcr_open then reports the error)
uint64_t record_identity(const uint8_t* rec, size_t len) {
    if (len < 64 || len >= (1ull << 32) || memcmp(rec, "PCR1", 4) != 0) return 0;
    const uint32_t N = rd32(rec + 8), G = rd32(rec + 12);
    const uint64_t index_off = rd64(rec + 32), data_off = rd64(rec + 40);
    if (N == 0 || G == 0 || G > 64 || N > (1u << 24) || data_off > len) return 0;
    if (index_off < 64 || index_off + 8ull * (G + 1) + 16ull * G * N > data_off) return 0;
    uint64_t h = hash_bytes(len, rec, (size_t)data_off);        // header, sample metadata, index
    const uint8_t* chunk = rec + index_off + 8ull * (G + 1);
    for (uint64_t j = 0; j < (uint64_t)N; ++j) {              // the chunks of scan group 1: frame header and tables of every image
        const uint64_t off = rd64(chunk + 16 * j);
        const uint32_t clen = rd32(chunk + 16 * j + 8);
        if (off > len || clen > len - off) return 0;
        h = hash_bytes(h, rec + off, std::min<size_t>(clen, 256));
    }
    return h ? h : 1;
}
void evict_records_locked(std::vector<pcr_record*>* out) {
    while (g_rcache.bytes > g_rcache.limit && !g_rcache.lru.empty()) {
        pcr_record* r = g_rcache.lru.front();
        g_rcache.lru.erase(g_rcache.lru.begin());
        g_rcache.bytes -= r->device_bytes;
        out->push_back(r);
    }
}
}  // namespace

extern "C" {

int pcr_set_record_cache(size_t max_device_bytes) {
    std::vector<pcr_record*> gone;
    {
        std::lock_guard<std::mutex> lk(g_rcache.mu);
        g_rcache.limit = max_device_bytes;
        evict_records_locked(&gone);
    }
    for (pcr_record* r : gone) { free_device(r); delete r; }
    return PCR_OK;
}

int pcr_open(const void* bytes, size_t len, pcr_record** rec) {
    if (rec) *rec = nullptr;
    if (!bytes || !rec) return PCR_E_ARG;
    uint64_t key = 0;
    const uint32_t ekey = env_key();
    if (g_rcache.limit) {
        key = record_identity(static_cast<const uint8_t*>(bytes), len);
        int dev = -1;
        cudaGetDevice(&dev);
        std::lock_guard<std::mutex> lk(g_rcache.mu);
        for (size_t i = g_rcache.lru.size(); key && i-- > 0;) {
            pcr_record* c = g_rcache.lru[i];
            if (c->host != bytes || c->key_len != len || c->key_hash != key || c->key_env != ekey || c->device != dev) continue;
            g_rcache.lru.erase(g_rcache.lru.begin() + (long)i);
            g_rcache.bytes -= c->device_bytes;
            // a fresh handle: nothing resident, nothing decoded, default settings
            c->resident = 0; c->decoded_k = 0; c->upsampling = PCR_UPSAMPLE_REPLICATE; c->profiling = false;
            c->decode_enqueued = false;
            *rec = c;
            return PCR_OK;
        }
    }
    pcr_record* r = new (std::nothrow) pcr_record();
    if (!r) return PCR_E_NOMEM;
    int rc;
    try {
        rc = open_impl(static_cast<const uint8_t*>(bytes), len, r);
    } catch (const std::bad_alloc&) {
        rc = PCR_E_NOMEM;
    }
    if (rc != PCR_OK) {
        free_device(r);
        delete r;
        return rc;
    }
    r->key_hash = key; r->key_len = key ? len : 0; r->key_env = ekey;
    for (auto& b : r->bufs) r->device_bytes += size_class(b.second);
    *rec = r;
    return PCR_OK;
}

int pcr_num_images(const pcr_record* rec) { return rec ? rec->N : PCR_E_ARG; }
int pcr_num_groups(const pcr_record* rec) { return rec ? rec->G : PCR_E_ARG; }

int pcr_get_image(const pcr_record* rec, int i, pcr_image_info* info) {
    if (!rec || !info || i < 0 || i >= rec->N) return PCR_E_ARG;
    *info = rec->info[i];
    return PCR_OK;
}

size_t pcr_out_bytes(const pcr_record* rec) { return rec ? rec->out_bytes : 0; }

size_t pcr_prefix_bytes(const pcr_record* rec, int k) {
    if (!rec || k < 1 || k > rec->G) return 0;
    return (size_t)rec->group_end[k];
}

int pcr_evict(pcr_record* rec) {
    if (!rec) return PCR_E_ARG;
    rec->resident = 0;
    return PCR_OK;
}

}  // extern "C"

template <int kSamp>
static void launch_pixels_sampled(bool refine, unsigned grid, cudaStream_t q, const Params& Q, const FinalizeList& fl, uint8_t* o8) {
    if (refine) pixel_kernel<true, 1, false, 0, kSamp><<<grid, kPixThreads, 0, q>>>(Q, fl, o8);
    else pixel_kernel<false, 1, false, 0, kSamp><<<grid, kPixThreads, 0, q>>>(Q, fl, o8);
}

// Decode scans k0 .. k-1 on top of the state scans 0 .. k0-1 left behind (k0 = 0: from scratch),
// then produce the pixels of fidelity k.
static int decode_range(pcr_record* rec, int k0, int k, void* out, void* stream, const TensorArgs* targs = nullptr) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t need = (size_t)rec->group_end[k];
    const bool prof = rec->profiling;
    rec->stages.clear();
    auto mark = [&](const char* name, int launches) {
        if (!prof || rec->stages.size() + 1 >= rec->events.size()) return;
        pcr_stage_time t;
        memset(&t, 0, sizeof t);
        strncpy(t.name, name, sizeof t.name - 1);
        t.launches = launches;
        rec->stages.push_back(t);
        cudaEventRecord(rec->events[rec->stages.size()], st);
    };
    if (cudaStreamWaitEvent(st, rec->ev_ready, 0) != cudaSuccess) return PCR_E_CUDA;      // pcr_open's uploads
    if (prof) cudaEventRecord(rec->events[0], st);
    const bool pipelined = rec->n_slices > 1 && !prof;
    if (!pipelined && rec->resident < need) {
        size_t from = rec->resident & ~(size_t)15;
        if (cudaMemcpyAsync(rec->d_rec + from, rec->host + from, need - from, cudaMemcpyHostToDevice, st) != cudaSuccess) return PCR_E_CUDA;
        rec->resident = need;
    }
    mark("h2d", 0);
    if (k0 == 0 && cudaMemsetAsync(rec->d_status, 0, (size_t)rec->N * 4, st) != cudaSuccess) return PCR_E_CUDA;
    Params P;
    P.rec = rec->d_rec; P.ubuf = rec->d_ubuf; P.planes = rec->d_planes; P.head = rec->d_head; P.script = rec->d_script; P.scans = rec->d_scans;
    P.saux = rec->d_saux; P.aux = rec->d_aux;
    P.imgs = rec->d_imgs; P.seg_start = rec->d_seg; P.items = rec->d_items; P.units = rec->d_units;
    P.qtab = rec->d_qtab; P.order = rec->d_order; P.status = rec->d_status; P.N = rec->N;
    P.hs = rec->hs; P.vs = rec->vs; P.nc = rec->nc;
    P.roi = targs ? targs->crops : nullptr;          // (only read by the crop-restricted kernels)
    P.chroma = rec->d_chroma;
    FinalizeList fl;
    memset(&fl, 0, sizeof fl);
    bool any_refine = false;
    for (int s = k0; s < k; ++s) {
        const ScanScript& sc = rec->script[s];
        if (sc.Ss == 0 || sc.Ah == 0) continue;
        const int c = sc.comp[0];
        if (fl.n[c] < 4) {
            fl.scan[c][fl.n[c]] = s;
            fl.p1[c][fl.n[c]] = 1 << sc.Al;
            fl.base[c][fl.n[c]] = rec->saux[s].base;
            ++fl.n[c];
            any_refine = true;
        }
    }
    int first_refine_wave = -1;                 // wave of the first AC refinement this call decodes
    for (int s = k0; s < k; ++s)
        if (rec->script[s].Ss > 0 && rec->script[s].Ah > 0 && (first_refine_wave < 0 || rec->wave_of_scan[s] < first_refine_wave))
            first_refine_wave = rec->wave_of_scan[s];
    const bool chains = first_refine_wave >= 0 && rec->n_groups > 0;
    const int chain_depth = kChainPairs / 4;    // chains per scheduler of the chain launch
    bool dc_only = true, head_only = true;      // no AC scan at all / no scan beyond zigzag position 7
    for (int s = 0; s < k; ++s) {
        if (rec->script[s].Ss > 0 || rec->script[s].Se > 0) dc_only = false;
        if (rec->script[s].Se > 7) head_only = false;
    }
    // the specialised pixel kernels (DC only, head plane only, crop-restricted) exist for 4:2:0
    const bool s420 = rec->hs == 2 && rec->vs == 2 && rec->nc == 3;
    if (!s420) { dc_only = false; head_only = false; }
    const bool roi = targs && s420;                 // decode only the MCU rows the crops touch
    rec->dc_merged = false;
    // the planes must be zero before the first AC scan writes into them
    const bool clear_planes = !head_only && (k0 == 0 || !rec->planes_cleared);
    const bool clear_dc = k0 == 0;
    if (k0 == 0) rec->planes_cleared = false;
    if (clear_planes) rec->planes_cleared = true;
    rec->decoded_k = k;
    const int G = rec->G;
    std::vector<char> copied(rec->n_waves, 0);      // wave w has to wait for its copy event
    // the stages of one slice; stage numbers: 0 clear, 1 index, 2+w entropy wave w, 2+W unused, 3+W pixels
    // (the pixel kernel also folds the refinement side data into the planes)
    const int W = rec->n_waves;
    std::vector<char> indexed(rec->n_waves, 0);     // wave w of the current slice has an index launch to wait for
    // restart-interval index of wave w of slice g on stream q: 1 launched, 0 nothing to do, -1 error
    auto launch_index = [&](int w, cudaStream_t q) -> int {
        ScanList sl;
        sl.n = 0;
        for (int s : rec->wave_scans[w]) if (s >= k0 && s < k) sl.s[sl.n++] = s;
        if (!sl.n) return 0;
        const uint32_t i0 = 0, i1 = (uint32_t)rec->N;      // one launch covers every slice
        if (copied[w] && cudaStreamWaitEvent(q, rec->ev_copy[w], 0) != cudaSuccess) return -1;
        const uint32_t warps = (uint32_t)sl.n * (i1 - i0);
        unstuff_index_kernel<<<(warps + 7) / 8, 256, 0, q>>>(P, sl, (int)i0, (int)(i1 - i0));
        ++g_launches;
        return 1;
    };
    auto run_stage = [&](int stage, int g, cudaStream_t q) -> bool {
        const uint32_t i0 = rec->slice_img[g], i1 = rec->slice_img[g + 1];
        const uint32_t u0 = rec->slice_unit[g], nu = rec->slice_unit[g + 1] - u0;
        if (stage == 0) {
            if (pipelined) return true;           // zeroed once for all slices on the clear stream
            if (g != 0) return true;              // the first slice zeroes for all (a slice's blocks are not contiguous)
            if (clear_dc && cudaMemsetAsync(rec->d_head, 0, rec->total_blocks * 16, q) != cudaSuccess) return false;
            if (!clear_planes) return true;       // no AC scan yet, or already zeroed by the decode this one continues
            return cudaMemsetAsync(rec->d_planes, 0, rec->total_blocks * 128, q) == cudaSuccess;
        }
        if (stage == 1) {
            if (pipelined) return true;          // done wave by wave, as the bytes arrive
            ScanList sl;
            sl.n = 0;
            for (int s = k0; s < k; ++s) sl.s[sl.n++] = s;
            const uint32_t warps = (uint32_t)sl.n * (i1 - i0);
            unstuff_index_kernel<<<(warps + 7) / 8, 256, 0, q>>>(P, sl, (int)i0, (int)(i1 - i0));
            ++g_launches;
            return true;
        }
        if (stage < 2 + W) {
            const int w = stage - 2;
            if (pipelined) {
                if (w == 0) {
                    if (cudaStreamWaitEvent(q, rec->ev_clear, 0) != cudaSuccess) return false;
                } else if (indexed[w]) {
                    // the later waves were indexed on the side stream, beside the first wave
                    if (cudaStreamWaitEvent(q, rec->ev_index[w], 0) != cudaSuccess) return false;
                }
            }
            const ScanScript& first = rec->script[rec->wave_scans[w][0]];
            const bool sequential = first.Ss == 0 && first.Se == 63;   // a baseline record: its one scan is sequential
            // the items of the wave's scans lie one after the other
            uint32_t begin = 0, count = 0;
            for (int s : rec->wave_scans[w]) {
                if (s >= k) break;   // scans of a wave are stored in ascending order
                if (s < k0) continue;
                if (!count) begin = rec->item_begin[(size_t)g * G + s];
                count += rec->item_count[(size_t)g * G + s];
            }
            if (sequential) {
                if (count) {
                    if (roi) sequential_kernel<true><<<(count + kSeqWarps - 1) / kSeqWarps, 32 * kSeqWarps, 0, q>>>(P, begin, count);
                    else sequential_kernel<false><<<(count + kSeqWarps - 1) / kSeqWarps, 32 * kSeqWarps, 0, q>>>(P, begin, count);
                    ++g_launches;
                }
                const int s0 = rec->wave_scans[w][0];      // the record's one scan
                const uint32_t lc = (s0 >= k0 && s0 < k) ? rec->long_count[(size_t)g * G + s0] : 0u;
                if (lc) {                                  // images whose scan is one long restart interval
                    sequential_long_kernel<<<lc, 32 * kSeqLongWarps, 0, q>>>(P, rec->d_long + rec->long_begin[(size_t)g * G + s0], lc);
                    ++g_launches;
                }
                return true;
            }
            if (count) {
                const unsigned nb = (count + kEntropyWarps - 1) / kEntropyWarps;
                if (roi) entropy_kernel<true><<<nb, 32 * kEntropyWarps, 0, q>>>(P, begin, count);
                else entropy_kernel<false><<<nb, 32 * kEntropyWarps, 0, q>>>(P, begin, count);
                ++g_launches;
            }
            // scans that are one long restart interval: the first passes of the wave (a contiguous run
            // of the list) ...
            {
                uint32_t lb = 0, lc = 0;
                bool lany = false;
                for (int s : rec->wave_scans[w]) {
                    if (s >= k) break;
                    if (s < k0 || rec->script[s].Ah != 0) continue;
                    if (!lany) { lb = rec->long_begin[(size_t)g * G + s]; lany = true; }
                    lc += rec->long_count[(size_t)g * G + s];
                }
                if (lc) {
                    first_pass_long_kernel<<<lc, 32 * kLongWarps, 0, q>>>(P, rec->d_long + lb, lc);
                    ++g_launches;
                }
            }
            // ... (their AC refinements follow in one launch for the whole record, once every slice
            // has finished its waves) and the DC refinement scans of every record
            for (int s : rec->wave_scans[w]) {
                if (s >= k) break;
                const ScanScript& sc = rec->script[s];
                if (s < k0 || sc.Ss != 0 || sc.Ah == 0) continue;
                for (uint32_t p0 = i0; p0 < i1; p0 += 65535u) {
                    dc_refine_kernel<<<dim3(rec->dc_refine_chunks, std::min(i1 - p0, 65535u)), 256, 0, q>>>(P, s, p0);
                    ++g_launches;
                }
            }
            return true;
        }
        Params Q = P;
        Q.units = P.units + u0;
        if (stage == 2 + W) {
            // the AC refinements of scans that are one long restart interval: one persistent launch
            // for all slices (the first slice's stream carries it; the caller has joined the others)
            if (g != 0 || !chains) return true;
            const int levels = std::max(fl.n[0], std::max(fl.n[1], fl.n[2]));
            const int rounds = std::max(1, chain_depth / levels);
            const int pairs = 4 * rounds * levels;          // chains per CTA: a decoding and a helper warp each
            if (cudaMemsetAsync(rec->d_chain_sync, 0, (size_t)(4 + 4 * (size_t)rec->n_groups) * 4, q) != cudaSuccess) return false;
            const unsigned grid = std::min<unsigned>((unsigned)rec->n_sms, (rec->n_groups + 3u) / 4u);
            ac_refine_group_kernel<<<grid, 64 * pairs, (size_t)pairs * sizeof(ChainShared), q>>>(P, fl, rec->d_group, rec->n_groups, rec->d_chain_sync, levels, rounds);
            ++g_launches;
            return true;
        }
        if (nu) {
            const unsigned grid = nu;
            uint8_t* o8 = static_cast<uint8_t*>(out);
            if (!s420) {
                // other samplings: one general kernel per sampling (positions 0..7 from the head plane, the
                // rest from the lines, which are always cleared for these records)
                const int code = rec->nc == 1 ? kSampGrey : (rec->hs == 2 ? kSamp422 : (rec->vs == 2 ? kSamp440 : kSamp444));
                if (code == kSamp422) launch_pixels_sampled<kSamp422>(any_refine, grid, q, Q, fl, o8);
                else if (code == kSamp440) launch_pixels_sampled<kSamp440>(any_refine, grid, q, Q, fl, o8);
                else if (code == kSamp444) launch_pixels_sampled<kSamp444>(any_refine, grid, q, Q, fl, o8);
                else launch_pixels_sampled<kSampGrey>(any_refine, grid, q, Q, fl, o8);
            } else if (!targs && rec->upsampling == PCR_UPSAMPLE_TRIANGLE) {
                // chroma pass (samples of every chroma block into the sample planes), then the pixel pass
                if (head_only && any_refine) {
                    pixel_kernel<true, 3, false, 1><<<grid, kPixThreads, 0, q>>>(Q, fl, o8);
                    pixel_kernel<true, 3, false, 2><<<grid, kPixThreads, 0, q>>>(Q, fl, o8);
                } else if (head_only) {
                    pixel_kernel<false, 3, false, 1><<<grid, kPixThreads, 0, q>>>(Q, fl, o8);
                    pixel_kernel<false, 3, false, 2><<<grid, kPixThreads, 0, q>>>(Q, fl, o8);
                } else if (any_refine) {
                    pixel_kernel<true, 1, false, 1><<<grid, kPixThreads, 0, q>>>(Q, fl, o8);
                    pixel_kernel<true, 1, false, 2><<<grid, kPixThreads, 0, q>>>(Q, fl, o8);
                } else {
                    pixel_kernel<false, 1, false, 1><<<grid, kPixThreads, 0, q>>>(Q, fl, o8);
                    pixel_kernel<false, 1, false, 2><<<grid, kPixThreads, 0, q>>>(Q, fl, o8);
                }
                ++g_launches;
            } else if (!targs) {
                if (dc_only && rec->widths_mult16) dc_pixel_kernel<false><<<grid, 128, 0, q>>>(Q, o8);
                else if (dc_only) dc_pixel_kernel<false, false><<<grid, 128, 0, q>>>(Q, o8);
                else if (head_only && any_refine) pixel_kernel<true, 3><<<grid, kPixThreads, 0, q>>>(Q, fl, o8);
                else if (head_only) pixel_kernel<false, 3><<<grid, kPixThreads, 0, q>>>(Q, fl, o8);
                else if (any_refine) pixel_kernel<true, 1><<<grid, kPixThreads, 0, q>>>(Q, fl, o8);
                else pixel_kernel<false, 1><<<grid, kPixThreads, 0, q>>>(Q, fl, o8);
            } else {
                if (dc_only && rec->widths_mult16) dc_pixel_kernel<true><<<grid, 128, 0, q>>>(Q, o8);
                else if (dc_only) dc_pixel_kernel<true, false><<<grid, 128, 0, q>>>(Q, o8);
                else if (head_only && any_refine) pixel_kernel<true, 3, true><<<grid, kPixThreads, 0, q>>>(Q, fl, o8);
                else if (head_only) pixel_kernel<false, 3, true><<<grid, kPixThreads, 0, q>>>(Q, fl, o8);
                else if (any_refine) pixel_kernel<true, 1, true><<<grid, kPixThreads, 0, q>>>(Q, fl, o8);
                else pixel_kernel<false, 1, true><<<grid, kPixThreads, 0, q>>>(Q, fl, o8);
            }
            ++g_launches;
            // the grid's second dimension (one image each) holds at most 65535 entries
            for (uint32_t p0 = i0; targs && p0 < i1; p0 += 65535u) {
                const dim3 tg((unsigned)((targs->size + kTensorRows - 1) / kTensorRows), std::min(i1 - p0, 65535u));
                if (targs->f32 == 2) tensor_kernel<__nv_bfloat16><<<tg, 256, 0, q>>>(P, *targs, static_cast<const uint8_t*>(out), p0);
                else if (targs->f32) tensor_kernel<float><<<tg, 256, 0, q>>>(P, *targs, static_cast<const uint8_t*>(out), p0);
                else tensor_kernel<__half><<<tg, 256, 0, q>>>(P, *targs, static_cast<const uint8_t*>(out), p0);
                ++g_launches;
            }
        }
        return true;
    };
    auto launched_in = [&](int stage) -> int {      // kernel launches of a stage over all slices (for the profile)
        if (stage == 0) return 0;
        if (stage == 2 + W) return chains ? 1 : 0;
        if (stage >= 2 && stage < 2 + W) {
            bool any = false;
            for (int s : rec->wave_scans[stage - 2]) if (s >= k0 && s < k) any = true;
            if (!any) return 0;
        }
        return rec->n_slices;
    };
    const int n_stages = 4 + W;
    if (rec->n_slices == 1 || prof) {
        // one stage after the other (also the timed layout of the stage profile); with several
        // slices the slices of a stage run side by side on their streams, between two joins
        for (int stage = 0; stage < n_stages; ++stage) {
            if (rec->n_slices == 1) {
                if (!run_stage(stage, 0, st)) return PCR_E_CUDA;
            } else {
                if (cudaEventRecord(rec->ev_fork, st) != cudaSuccess) return PCR_E_CUDA;
                for (int g = 0; g < rec->n_slices; ++g) {
                    cudaStream_t q = rec->streams[g];
                    if (cudaStreamWaitEvent(q, rec->ev_fork, 0) != cudaSuccess) return PCR_E_CUDA;
                    if (!run_stage(stage, g, q)) return PCR_E_CUDA;
                    if (cudaEventRecord(rec->ev_join[g], q) != cudaSuccess) return PCR_E_CUDA;
                    if (cudaStreamWaitEvent(st, rec->ev_join[g], 0) != cudaSuccess) return PCR_E_CUDA;
                }
            }
            char name[24];
            if (stage == 0) snprintf(name, sizeof name, "clear");
            else if (stage == 1) snprintf(name, sizeof name, "index");
            else if (stage < 2 + W) snprintf(name, sizeof name, "entropy%d", stage - 2);
            else if (stage == 2 + W) snprintf(name, sizeof name, "chains");
            else snprintf(name, sizeof name, "pixels");
            const int nl = launched_in(stage);
            if (stage <= 1 || stage == n_stages - 1 || nl) mark(name, nl);
        }
    } else {
        // every slice is its own pipeline on its own stream, forked from and joined to the caller's;
        // missing record bytes arrive on a copy stream, the scan groups of each wave behind an event
        if (cudaEventRecord(rec->ev_fork, st) != cudaSuccess) return PCR_E_CUDA;
        if (cudaStreamWaitEvent(rec->clear_stream, rec->ev_fork, 0) != cudaSuccess) return PCR_E_CUDA;
        if (clear_dc && cudaMemsetAsync(rec->d_head, 0, rec->total_blocks * 16, rec->clear_stream) != cudaSuccess) return PCR_E_CUDA;
        if (clear_planes && cudaMemsetAsync(rec->d_planes, 0, rec->total_blocks * 128, rec->clear_stream) != cudaSuccess) return PCR_E_CUDA;
        if (cudaEventRecord(rec->ev_clear, rec->clear_stream) != cudaSuccess) return PCR_E_CUDA;
        if (rec->resident < need) {
            if (cudaStreamWaitEvent(rec->copy_stream, rec->ev_fork, 0) != cudaSuccess) return PCR_E_CUDA;
            bool any = false;
            for (int w = 0; w < W; ++w) {
                size_t upto = 0;
                for (int s : rec->wave_scans[w]) if (s < k) upto = std::max(upto, (size_t)rec->group_end[s + 1]);
                if (upto > rec->resident) {
                    const size_t from = rec->resident & ~(size_t)15;
                    if (cudaMemcpyAsync(rec->d_rec + from, rec->host + from, upto - from, cudaMemcpyHostToDevice, rec->copy_stream) != cudaSuccess) return PCR_E_CUDA;
                    rec->resident = upto;
                    any = true;
                }
                if (any) {
                    if (cudaEventRecord(rec->ev_copy[w], rec->copy_stream) != cudaSuccess) return PCR_E_CUDA;
                    copied[w] = true;
                }
            }
        }
        // restart-interval index, one launch per wave for all slices: the first wave's on the caller's
        // stream, the later waves' on the side stream behind the memsets, beside the first entropy wave
        if (launch_index(0, st) < 0) return PCR_E_CUDA;
        if (cudaEventRecord(rec->ev_start, st) != cudaSuccess) return PCR_E_CUDA;
        for (int w = 1; w < W; ++w) {
            const int li = launch_index(w, rec->clear_stream);
            if (li < 0) return PCR_E_CUDA;
            indexed[w] = li > 0;
            if (li > 0 && cudaEventRecord(rec->ev_index[w], rec->clear_stream) != cudaSuccess) return PCR_E_CUDA;
        }
        // with a chain launch the slices meet once: it follows the entropy waves of all of them
        const int meet = chains ? 2 + W : n_stages;
        for (int g = 0; g < rec->n_slices; ++g) {
            cudaStream_t q = rec->streams[g];
            if (cudaStreamWaitEvent(q, rec->ev_start, 0) != cudaSuccess) return PCR_E_CUDA;
            for (int stage = 0; stage < meet; ++stage)
                if (!run_stage(stage, g, q)) return PCR_E_CUDA;
            if (cudaEventRecord(rec->ev_join[g], q) != cudaSuccess) return PCR_E_CUDA;
            if (!chains && cudaStreamWaitEvent(st, rec->ev_join[g], 0) != cudaSuccess) return PCR_E_CUDA;
        }
        if (chains) {
            cudaStream_t q0 = rec->streams[0];
            for (int g = 1; g < rec->n_slices; ++g)
                if (cudaStreamWaitEvent(q0, rec->ev_join[g], 0) != cudaSuccess) return PCR_E_CUDA;
            if (!run_stage(2 + W, 0, q0)) return PCR_E_CUDA;
            if (cudaEventRecord(rec->ev_chain, q0) != cudaSuccess) return PCR_E_CUDA;
            for (int g = 0; g < rec->n_slices; ++g) {
                cudaStream_t q = rec->streams[g];
                if (g && cudaStreamWaitEvent(q, rec->ev_chain, 0) != cudaSuccess) return PCR_E_CUDA;
                for (int stage = 3 + W; stage < n_stages; ++stage)
                    if (!run_stage(stage, g, q)) return PCR_E_CUDA;
                if (cudaEventRecord(rec->ev_join[g], q) != cudaSuccess) return PCR_E_CUDA;
                if (cudaStreamWaitEvent(st, rec->ev_join[g], 0) != cudaSuccess) return PCR_E_CUDA;
            }
        }
        // the side and copy streams rejoin the caller's stream too (implied by the slices' waits
        // whenever they carried work; stated so that every fork is joined)
        if (cudaEventRecord(rec->ev_clear, rec->clear_stream) != cudaSuccess) return PCR_E_CUDA;
        if (cudaStreamWaitEvent(st, rec->ev_clear, 0) != cudaSuccess) return PCR_E_CUDA;
        if (copied[W - 1] && cudaStreamWaitEvent(st, rec->ev_copy[W - 1], 0) != cudaSuccess) return PCR_E_CUDA;
    }
    if (cudaEventRecord(rec->ev_done, st) != cudaSuccess) return PCR_E_CUDA;
    rec->decode_enqueued = true;
    if (cudaGetLastError() != cudaSuccess) return PCR_E_CUDA;
    return PCR_OK;
}

extern "C" {

void pcr_release_cached_memory(void) {
    {
        std::vector<pcr_record*> gone;
        {
            std::lock_guard<std::mutex> lk(g_rcache.mu);
            gone.swap(g_rcache.lru);
            g_rcache.bytes = 0;
        }
        for (pcr_record* r : gone) { free_device(r); delete r; }
    }
    std::lock_guard<std::mutex> lk(g_cache.mu);
    for (auto& kv : g_cache.free_) cudaFree(kv.second);
    g_cache.free_.clear();
    g_cache.cached = 0;
}

int pcr_decode(pcr_record* rec, int k, void* out, void* stream) {
    if (!rec || !out || k < 1 || k > rec->G) return PCR_E_ARG;
    if (reinterpret_cast<uintptr_t>(out) & 15u) return PCR_E_ARG;
    return decode_range(rec, 0, k, out, stream);
}

int pcr_decode_more(pcr_record* rec, int k, void* out, void* stream) {
    if (!rec || !out || k < 1 || k > rec->G) return PCR_E_ARG;
    if (reinterpret_cast<uintptr_t>(out) & 15u) return PCR_E_ARG;
    if (rec->decoded_k < 1 || k <= rec->decoded_k) return PCR_E_ARG;
    return decode_range(rec, rec->decoded_k, k, out, stream);
}

int pcr_decode_tensor(pcr_record* rec, int k, const pcr_crop* crops, int size, const float* mean, const float* std_,
                      int dtype, void* rgb, void* tensor, void* stream) {
    if (!rec || !crops || !mean || !std_ || !rgb || !tensor || k < 1 || k > rec->G) return PCR_E_ARG;
    if (rec->upsampling != PCR_UPSAMPLE_REPLICATE) return PCR_E_ARG;      // the tensor path resamples replicated chroma only
    if (size < 1 || size > 4096 || (dtype != PCR_F16 && dtype != PCR_F32 && dtype != PCR_BF16)) return PCR_E_ARG;
    if (reinterpret_cast<uintptr_t>(rgb) & 15u) return PCR_E_ARG;
    if (reinterpret_cast<uintptr_t>(tensor) & (dtype == PCR_F32 ? 3u : 1u)) return PCR_E_ARG;
    static_assert(sizeof(pcr_crop) == sizeof(CropRect), "pcr_crop and CropRect have the same layout");
    for (int i = 0; i < rec->N; ++i) {
        const pcr_crop& c = crops[i];
        const pcr_image_info& inf = rec->info[i];
        if (inf.out_bytes >= (1ull << 31)) return PCR_E_ARG;      // the epilogue indexes an image's bytes with 32 bits
        if (c.w < 1 || c.h < 1 || c.flip > 1 || c.x0 > inf.width || c.y0 > inf.height || c.w > inf.width - c.x0 ||
            c.h > inf.height - c.y0) return PCR_E_ARG;
        if (!(std_[0] > 0.f) || !(std_[1] > 0.f) || !(std_[2] > 0.f)) return PCR_E_ARG;
    }
    if (!rec->d_crops) {
        if (int rc = take(rec, &rec->d_crops, (size_t)rec->N * sizeof(CropRect))) return rc;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(rec->d_crops, crops, (size_t)rec->N * sizeof(CropRect), cudaMemcpyHostToDevice, st) != cudaSuccess) return PCR_E_CUDA;
    TensorArgs T;
    T.crops = rec->d_crops; T.out = tensor; T.size = size; T.f32 = dtype == PCR_F32 ? 1 : (dtype == PCR_BF16 ? 2 : 0);
    for (int c = 0; c < 3; ++c) { T.mean[c] = mean[c]; T.inv_std[c] = 1.0f / std_[c]; }
    const int rc = decode_range(rec, 0, k, rgb, stream, &T);
    rec->decoded_k = 0;          // rows outside the crops were not decoded: nothing to raise the fidelity of
    return rc;
}

static void msssim_layout(pcr_record* rec, std::vector<MsDesc>* table) {
    uint64_t floats = 0;
    if (table) table->resize(rec->N);
    for (int i = 0; i < rec->N; ++i) {
        const uint32_t W = rec->info[i].width, H = rec->info[i].height;
        uint32_t M = 0;
        while (M < (uint32_t)kMsMaxScales && (std::min(W, H) >> M) >= (uint32_t)kMsWin) ++M;
        uint64_t len = 0;
        for (uint32_t j = 0; j < M; ++j) len += (uint64_t)(W >> j) * (H >> j);
        if (table) {
            MsDesc& d = (*table)[i];
            d.W = W; d.H = H; d.M = M; d.rsvd = 0;
            d.rgb_off = rec->info[i].out_offset; d.plane_off = floats; d.plane_len = len;
        }
        floats += 2 * len;
    }
    floats = (floats + 1) & ~1ull;                      // the double-precision sums start 8-byte aligned
    rec->ms_floats = floats;
    rec->ms_scratch = (size_t)(floats * 4 + (uint64_t)rec->N * kMsMaxScales * 2 * 8);
}

size_t pcr_msssim_scratch_bytes(pcr_record* rec) {
    if (!rec) return 0;
    if (!rec->ms_scratch) msssim_layout(rec, nullptr);
    return rec->ms_scratch;
}

int pcr_msssim(pcr_record* rec, const void* rgb_a, const void* rgb_b, void* scratch, float* dev_scores, void* stream) {
    if (!rec || !rgb_a || !rgb_b || !scratch || !dev_scores) return PCR_E_ARG;
    if ((reinterpret_cast<uintptr_t>(scratch) & 15u) || (reinterpret_cast<uintptr_t>(dev_scores) & 3u)) return PCR_E_ARG;
    if (rec->N > 65535) return PCR_E_ARG;       // one grid row per image
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!rec->d_ms) {
        std::vector<MsDesc> table;
        msssim_layout(rec, &table);
        if (int rc = upload(rec, &rec->d_ms, table)) return rc;
        if (cudaEventRecord(rec->ev_ready, rec->up_stream) != cudaSuccess) return PCR_E_CUDA;
    }
    if (cudaStreamWaitEvent(st, rec->ev_ready, 0) != cudaSuccess) return PCR_E_CUDA;
    float* planes = static_cast<float*>(scratch);
    double* sums = reinterpret_cast<double*>(planes + rec->ms_floats);
    if (cudaMemsetAsync(sums, 0, (size_t)rec->N * kMsMaxScales * 2 * 8, st) != cudaSuccess) return PCR_E_CUDA;
    MsWindow win;
    {
        double g[kMsWin], tot = 0.0;
        for (int k = 0; k < kMsWin; ++k) { const double x = k - (kMsWin - 1) / 2.0; g[k] = exp(-(x * x) / (2.0 * 1.5 * 1.5)); tot += g[k]; }
        for (int k = 0; k < kMsWin; ++k) win.g[k] = (float)(g[k] / tot);
    }
    const unsigned N = (unsigned)rec->N;
    ms_luma_kernel<<<dim3(64, N), 256, 0, st>>>(rec->d_ms, static_cast<const uint8_t*>(rgb_a), static_cast<const uint8_t*>(rgb_b), planes);
    ++g_launches;
    for (int j = 0; j < kMsMaxScales; ++j) {
        ms_scale_kernel<<<dim3(j == 0 ? 32 : (j == 1 ? 8 : 2), N), kMsTile * kMsTile, 0, st>>>(rec->d_ms, planes, sums, j, win);
        ++g_launches;
        if (j + 1 < kMsMaxScales) {
            ms_pool_kernel<<<dim3(j == 0 ? 32 : 8, N), 256, 0, st>>>(rec->d_ms, planes, j);
            ++g_launches;
        }
    }
    ms_final_kernel<<<(N + 255) / 256, 256, 0, st>>>(rec->d_ms, sums, dev_scores, (int)N);
    ++g_launches;
    // pcr_close waits for this event before it hands the record's buffers (the table above among them) on
    if (cudaEventRecord(rec->ev_done, st) != cudaSuccess) return PCR_E_CUDA;
    rec->decode_enqueued = true;
    if (cudaGetLastError() != cudaSuccess) return PCR_E_CUDA;
    return PCR_OK;
}

int pcr_set_upsampling(pcr_record* rec, int mode) {
    if (!rec || (mode != PCR_UPSAMPLE_REPLICATE && mode != PCR_UPSAMPLE_TRIANGLE)) return PCR_E_ARG;
    if (mode == PCR_UPSAMPLE_TRIANGLE && !(rec->hs == 2 && rec->vs == 2 && rec->nc == 3)) return PCR_E_ARG;   // built for 4:2:0
    if (mode == PCR_UPSAMPLE_TRIANGLE && !rec->d_chroma) {
        if (int rc = take(rec, &rec->d_chroma, (size_t)(std::max<uint64_t>(rec->total_blocks / 6, 1) * 128)   /* 4:2:0: six blocks per MCU */)) return rc;
    }
    rec->upsampling = mode;
    return PCR_OK;
}

int pcr_status(pcr_record* rec, int* first_bad_image, int* code) {
    if (!rec || !first_bad_image || !code) return PCR_E_ARG;
    if (cudaMemcpy(rec->h_status.data(), rec->d_status, (size_t)rec->N * 4, cudaMemcpyDeviceToHost) != cudaSuccess) return PCR_E_CUDA;
    *first_bad_image = -1; *code = PCR_OK;
    for (int i = 0; i < rec->N; ++i)
        if (rec->h_status[i] != 0) { *first_bad_image = i; *code = rec->h_status[i]; break; }
    return PCR_OK;
}

int pcr_coeffs(pcr_record* rec, const int16_t** dev_planes, size_t* bytes) {
    if (!rec || !dev_planes || !bytes) return PCR_E_ARG;
    // the decode keeps the DC coefficients in a dense plane of their own (and leaves the planes
    // alone when no AC scan was decoded): complete the canonical layout now
    if (!rec->planes_cleared) {
        if (cudaMemset(rec->d_planes, 0, rec->total_blocks * 128) != cudaSuccess) return PCR_E_CUDA;
        rec->planes_cleared = true;
    }
    if (!rec->dc_merged && rec->total_blocks) {
        Params P;
        memset(&P, 0, sizeof P);
        P.planes = rec->d_planes; P.head = rec->d_head;
        merge_head_kernel<<<(unsigned)((rec->total_blocks + 255) / 256), 256>>>(P, rec->total_blocks);
        ++g_launches;
        if (cudaDeviceSynchronize() != cudaSuccess) return PCR_E_CUDA;
        rec->dc_merged = true;
    }
    *dev_planes = rec->d_planes;
    *bytes = (size_t)rec->total_blocks * 128;
    return PCR_OK;
}

int pcr_image_blocks(const pcr_record* rec, int i, uint64_t* first_block, uint64_t* n_blocks) {
    if (!rec || !first_block || !n_blocks || i < 0 || i >= rec->N) return PCR_E_ARG;
    *first_block = rec->blk_base[i];
    *n_blocks = rec->nblk[i];
    return PCR_OK;
}

int pcr_get_scan(const pcr_record* rec, int s, pcr_scan_info* info) {
    if (!rec || !info || s < 0 || s >= rec->G) return PCR_E_ARG;
    const ScanScript& sc = rec->script[s];
    info->ncomp = sc.ncomp;
    for (int i = 0; i < 3; ++i) info->comp[i] = sc.comp[i];
    info->Ss = sc.Ss; info->Se = sc.Se; info->Ah = sc.Ah; info->Al = sc.Al;
    info->wave = rec->wave_of_scan[s];
    info->rsvd = 0;
    info->bytes = rec->group_end[s + 1] - rec->group_end[s];
    return PCR_OK;
}

int pcr_get_sampling(const pcr_record* rec, int* hs, int* vs, int* ncomp) {
    if (!rec || !hs || !vs || !ncomp) return PCR_E_ARG;
    *hs = rec->hs; *vs = rec->vs; *ncomp = rec->nc;
    return PCR_OK;
}

int pcr_set_profiling(pcr_record* rec, int enable) {
    if (!rec) return PCR_E_ARG;
    if (enable && rec->events.empty()) {
        for (int i = 0; i <= kMaxStages; ++i) {
            cudaEvent_t e;
            if (cudaEventCreate(&e) != cudaSuccess) return PCR_E_CUDA;
            rec->events.push_back(e);
        }
    }
    rec->profiling = enable != 0;
    return PCR_OK;
}

int pcr_get_profile(pcr_record* rec, pcr_stage_time* out, int cap, int* n) {
    if (!rec || !out || !n || cap < 0) return PCR_E_ARG;
    *n = 0;
    for (size_t i = 0; i < rec->stages.size() && (int)i < cap; ++i) {
        out[i] = rec->stages[i];
        if (cudaEventElapsedTime(&out[i].ms, rec->events[i], rec->events[i + 1]) != cudaSuccess) return PCR_E_CUDA;
        ++*n;
    }
    return PCR_OK;
}

uint64_t pcr_launch_count(void) { return g_launches.load(); }

int pcr_selftest_bounded_wait(int* gave_up) {
    if (!gave_up) return PCR_E_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return PCR_E_CUDA;
    int* d = static_cast<int*>(dev_alloc(sizeof(int), dev));
    if (!d) return PCR_E_NOMEM;
    int rc = PCR_OK;
    if (cudaMemset(d, 0xFF, sizeof(int)) != cudaSuccess) rc = PCR_E_CUDA;
    if (rc == PCR_OK) {
        bounded_wait_probe_kernel<<<1, 32>>>(2000u, d);      // 2000 polls of about 64 ns: the wait ends by itself
        ++g_launches;
        if (cudaMemcpy(gave_up, d, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) rc = PCR_E_CUDA;
    }
    dev_release(d, sizeof(int), dev);
    return rc;
}

const char* pcr_strerror(int code) {
    switch (code) {
    case PCR_OK: return "ok";
    case PCR_E_ARG: return "invalid argument";
    case PCR_E_FORMAT: return "not a valid or supported record";
    case PCR_E_CORRUPT: return "corrupt entropy-coded data";
    case PCR_E_TIMEOUT: return "device-side wait timed out";
    case PCR_E_CUDA: return "CUDA runtime error";
    case PCR_E_NOMEM: return "out of memory";
    default: return "unknown error";
    }
}

// ---------------------------------------------------------------------------------------
// pcr_pixels_noalloc: the pixel stage for one image, for callers that may not allocate.
// The pixel kernel reads an image descriptor, a work-unit list and the quantisers from
// global memory; pcr_open puts those in cudaMalloc'd tables.  Here they live in one
// file-scope device array that a small kernel fills on every call.
// ---------------------------------------------------------------------------------------
namespace {

constexpr uint32_t kNoAllocMaxDim = 4096;                                         // pixels per side
constexpr uint32_t kNoAllocMaxUnits = (kNoAllocMaxDim / 16) * (kNoAllocMaxDim / 16 / kPixMcus);
struct NoAllocScratch {
    ImgDesc img;
    uint16_t qtab[192];
    Unit units[kNoAllocMaxUnits];
};
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoAllocScratch)];

struct QuantArg { uint16_t q[192]; };

__global__ void noalloc_fill_kernel(uint32_t W, uint32_t H, QuantArg qa) {
    NoAllocScratch* s = reinterpret_cast<NoAllocScratch*>(g_noalloc_scratch);   // device code may name the array
    const uint32_t mx = (W + 15) / 16, my = (H + 15) / 16;
    const uint32_t per_row = (mx + kPixMcus - 1) / kPixMcus;
    const uint32_t tid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
    if (tid == 0) {
        s->img.W = W; s->img.H = H; s->img.mx = mx; s->img.my = my;
        s->img.blk_base = 0; s->img.out_off = 0;
    }
    if (tid < 192) s->qtab[tid] = qa.q[tid];
    for (uint32_t u = tid; u < per_row * my; u += nth) {
        Unit un;
        un.img = 0; un.mrow = (uint16_t)(u / per_row); un.mcol0 = (uint16_t)((u % per_row) * kPixMcus);
        s->units[u] = un;
    }
}

constexpr int kMaxDevices = 64;
void* g_noalloc_ptr[kMaxDevices];          // device address of the array, per device
std::atomic<int> g_noalloc_ready[kMaxDevices];

}  // namespace

int pcr_pixels_noalloc(const int16_t* dev_coeffs, uint32_t width, uint32_t height, const uint16_t* host_qtab,
                       uint8_t* dev_rgb, void* stream) {
    if (!dev_coeffs || !host_qtab || !dev_rgb || width == 0 || height == 0) return PCR_E_ARG;
    if (width > kNoAllocMaxDim || height > kNoAllocMaxDim) return PCR_E_ARG;   // beyond the fixed scratch
    // the pixel kernel reads every block as eight 16-byte vectors
    if (reinterpret_cast<uintptr_t>(dev_coeffs) & 15u) return PCR_E_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return PCR_E_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return PCR_E_ARG;
    if (!g_noalloc_ready[dev].load(std::memory_order_acquire)) {
        // In host code the array's name is only a handle; its device address has to be asked for,
        // once per device, with that device current.
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) { cudaGetLastError(); return PCR_E_CUDA; }
        g_noalloc_ptr[dev] = p;
        g_noalloc_ready[dev].store(1, std::memory_order_release);
    }
    NoAllocScratch* s = static_cast<NoAllocScratch*>(g_noalloc_ptr[dev]);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint32_t mx = (width + 15) / 16, my = (height + 15) / 16;
    const uint32_t n_units = ((mx + kPixMcus - 1) / kPixMcus) * my;
    QuantArg qa;
    memcpy(qa.q, host_qtab, sizeof qa.q);
    noalloc_fill_kernel<<<(n_units + 255) / 256, 256, 0, st>>>(width, height, qa);
    ++g_launches;
    Params P;
    memset(&P, 0, sizeof P);
    P.planes = const_cast<int16_t*>(dev_coeffs);     // read only by the pixel kernel
    P.imgs = &s->img; P.units = s->units; P.qtab = s->qtab; P.N = 1;
    FinalizeList none;
    memset(&none, 0, sizeof none);
    pixel_kernel<false, 0><<<n_units, kPixThreads, 0, st>>>(P, none, dev_rgb);
    ++g_launches;
    if (cudaGetLastError() != cudaSuccess) return PCR_E_CUDA;
    return PCR_OK;
}

void pcr_close(pcr_record* rec) {
    if (!rec) return;
    if (g_rcache.limit && rec->key_len) {
        // park it: its set-up and its last decode have to be complete before another handle may use it
        if (rec->up_stream) cudaStreamSynchronize(rec->up_stream);
        if (rec->ev_done && rec->decode_enqueued) cudaEventSynchronize(rec->ev_done);
        rec->device_bytes = 0;
        for (auto& b : rec->bufs) rec->device_bytes += size_class(b.second);
        std::vector<pcr_record*> gone;
        {
            std::lock_guard<std::mutex> lk(g_rcache.mu);
            if (rec->device_bytes <= g_rcache.limit) {
                g_rcache.lru.push_back(rec);
                g_rcache.bytes += rec->device_bytes;
                rec = nullptr;
                evict_records_locked(&gone);
            }
        }
        for (pcr_record* r : gone) { free_device(r); delete r; }
        if (!rec) return;
    }
    free_device(rec);
    delete rec;
}

}  // extern "C"
