// Shared definitions for the densify kernels: workspace layout, small device helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <utility>

#include "dst.h"

namespace dst {

// ---- fixed shape parameters -------------------------------------------------
constexpr int kRadixThreads = 512;          // threads of a radix-pass CTA (a multiple of 256, the number of digits; 256 threads: 1 % slower on the 64-slice case)
constexpr int kTile = kRadixThreads * 8;     // keys per CTA of a radix pass, at least (sizes the look-back descriptors)
constexpr int kClusterCtas = 8;             // the one-kernel index path for small inputs: CTAs per cluster,
constexpr int kFrontThreads = 1024;         // threads per CTA,
constexpr int kFrontMaxRows = 65535;        // largest input (positions are packed into 16 bits)
constexpr int kPrepItems = 8;               // indices per thread of the validation kernel
constexpr int kPrepThreads = 1024;
constexpr int kPrepTile = kPrepThreads * kPrepItems;
constexpr int kCountInPrepMaxVocab = 65536; // up to here a CTA of the validation kernel can hold a 16-bit counter per row in shared memory
constexpr int kMaxPasses = 4;               // 8-bit digits, keys below 2^31
constexpr int kFanIn = 8;                   // children per node of the heavy-row combine tree
constexpr int kMaxBatchUnits = 31;          // a light work item holds rows worth at most this many units (+ one row)
constexpr int kMaxChunkRows = 128;           // entries per chunk of a heavy row, at most (fewer chunks mean fewer drains of a warp's ring; more make the last items too long)
constexpr int kPipeWarpsTotal = 148 * 8;    // warps the row-reduction kernel runs with on a B200 (sizes the work items)
constexpr int kPipeWarps = 4;               // row-reduction kernel: warps per CTA, each with its own slot ring
constexpr int kPipeThreads = kPipeWarps * 32;
constexpr int kPipeSlots = 6;               // ring slots per warp, at most
constexpr int kPipeHeaderReserve = 1024;    // mbarriers in front of the slots
constexpr int kMaxBlockCols = 1024;         // columns per column block (32 fp32 accumulators per lane)
constexpr long long kWaitCycles = 1LL << 31; // SM clock cycles (about a second) before an mbarrier wait gives up
constexpr int kScanThreads = kRadixThreads;  // the scan tiles can ride in the launch of the first radix pass
constexpr int kScanItems = 4;               // rows per thread of a scan tile (8: the scan tiles outlast the first radix pass they ride in)
constexpr int kScanTile = kScanThreads * kScanItems;
constexpr int kSmCount = 148;               // B200; only used to pick the chunk length
constexpr unsigned kInvalidKey = 0xFFFFFFFFu;
constexpr unsigned kFlagMask = 0xC0000000u, kFlagAggregate = 0x40000000u, kFlagPrefix = 0x80000000u;
constexpr unsigned kValueMask = 0x3FFFFFFFu;
constexpr int64_t kMaxRows = (int64_t(1) << 30) - 1;  // look-back words keep 30 bits of count
constexpr int64_t kMaxVocab = int64_t(1) << 30;
constexpr int kSpinLimit = 1 << 20;
constexpr int kMaxDensePartners = 64;       // dense tensors one densify pass adds (their pointers travel as kernel parameters)

// ---- workspace --------------------------------------------------------------
struct WsHeader {          // zeroed at the start of every call
    int status;            // device-detected dst_status_t (max wins)
    int n_valid;           // rows with an index inside [0, vocab)
    int n_unique;
    int n_heavy;           // rows with more than `chunk` occurrences
    int n_chunks;          // work items those rows are split into
    int n_upper;           // combine-tree nodes above the chunk level
    int max_segment;
    unsigned int done;     // CTAs of the row-reduction kernel that have finished
    unsigned long long n_bad;
    unsigned int ticket[kMaxPasses];
    unsigned int work_counter;
    int n_batches;         // light work items (row batches)
    unsigned int scan_ticket;
    unsigned int scan_done;
    unsigned int copy_counter;   // small-input path: copy work items handed out
    int tables_ready;            // ... set by the index cluster once every table and this header are written
    int reserved[2];
    int bitmap_ready[kClusterCtas];   // ... CTA r of the index cluster has written its copy of the named-row bitmap
};
static_assert(sizeof(WsHeader) == 120, "header layout");
constexpr int kHeaderWordsBeforeFlags = (120 - 4 * kClusterCtas) / 4;   // words the index cluster's first CTA clears

struct SliceEntry {        // one IndexedSlices object of the (virtual) concatenation
    const void* indices;
    const void* values;
    long long start;       // global position of its first row
    long long n_rows;
};

constexpr int kHistSlices = 64;   // slices described per histogram launch (kernel-parameter space)
struct HistParams {
    SliceEntry s[kHistSlices];
    int n;                 // slices used in this launch
    int first;             // index of s[0] in the full slice table
};

struct HeavyInfo {         // a row whose segment is split into chunks
    int row;
    int chunk_base;        // id of its first chunk
    int upper_base;        // id of its first upper tree node
    int n_chunks;
    int begin;             // first entry of its segment in perm[]
    int count;             // entries in its segment
    int pad[2];
};
static_assert(sizeof(HeavyInfo) == 32, "heavy-row record layout");

struct ChunkDesc {         // one chunk work item (derived from HeavyInfo on the fly)
    int row;
    int begin;             // first entry in perm[]
    int len;
    int heavy;             // index into HeavyInfo
};

struct Layout {
    int64_t n_rows, vocab, d;
    int R, chunk, passes, batch_units;
    int64_t n_tiles, vocab_pad, heavy_max, chunk_max, upper_max, batch_max;
    size_t off_header, off_count, off_digit, off_desc, off_nodecnt, off_batches, off_scandesc, zero_bytes;
    size_t off_offsets, off_keys[2], off_pos[2], off_tab, off_heavy, off_partials, off_urow, off_uoff, off_bitmap;
    int bitmap_words;        // 32-bit words of the named-row bitmap (small-input path), 0 when that path cannot apply
    size_t total;
};

// arguments of the row-reduction kernels
struct MainArgs {
    WsHeader* hdr;
    const int* offsets;
    const unsigned* perm;
    const SliceEntry* tab;
    const HeavyInfo* heavy;
    const int2* batches;   // per row batch: first row + 1, last row + 1 (0: empty batch).  `compact`: an int per batch
                           // instead, the rank of its first named row, and one more int, the number of named rows
    const unsigned* urec;  // compact: the named rows by rank: row << 16 | first entry in perm[]; then the number of entries
                           // (and perm[] holds 16-bit positions)
    unsigned* node_cnt;
    float* partials;
    const void* dense_in;   // the first dense partner (nullptr: none)
    void* out;
    dst_result_t* result;
    long long d;
    int n_dense;            // dense partners in all: dense_in, then dense_more[0 .. n_dense - 2]
    const void* dense_more[kMaxDensePartners - 1];
    int vocab;
    int n_total;     // rows in all slices (capacity of perm)
    int R;
    int chunk;
    int chunk_max;   // partial rows of the chunk level; upper nodes follow
    int upper_max;   // combine-tree arrival counters per column block
    int W;           // columns per column block
    int ncb;         // column blocks per row
    int slot_bytes;
    int n_slots;
    int apply;       // 0: `out` receives the gradient; 1 SGD, 2 momentum, 3 Adam: `out` is an fp32 weight that takes the step
    float lr;        // learning rate of that step
    float grad_scale;           // the summed gradient is multiplied by this (reciprocal of the loss scale)
    float opt_a, opt_b;         // momentum: mu, -; Adam: beta1, beta2
    float opt_eps;              // Adam
    float opt_bc1, opt_bc2;     // Adam: 1 / (1 - beta1^t), 1 / (1 - beta2^t)
    void* state1;               // [vocab, d] fp32: momentum buffer / Adam's first moment
    void* state2;               // [vocab, d] fp32: Adam's second moment
    int compact;     // the row batches list only the named rows (urow / uoff); the others are not this item list's business
    // Overlapped small-input path: the kernel starts beside the index cluster.  Until tables_ready it gives the rows
    // nobody names their dense_in row (copy items of copy_rows consecutive rows, named ones skipped by the bitmap),
    // then it takes the named rows, then whatever copy items are left.
    int overlap;
    int copy_rows;              // rows per copy item: 8, 16 or 32 (a divisor of 32)
    int copy_slots;             // ring slots in use while copying (n_slots while reducing)
    const unsigned* bitmap;     // kClusterCtas interleaved copies, see Layout::off_bitmap
    int bitmap_words;
};

// How the row-reduction kernel cuts rows into column blocks and shared memory into slots.
struct PipeShape { int K, W, ncb, slot_bytes, n_slots; };
inline PipeShape pipe_shape(int value_size, int out_size, int64_t d) {
    PipeShape p{};
    const int vc = 16 / value_size;                        // columns per 16-byte group of a value row
    const int64_t w = d < kMaxBlockCols ? d : kMaxBlockCols;
    p.W = int(w > 0 ? w : 1);
    p.ncb = int(d > 0 ? (d + p.W - 1) / p.W : 1);
    p.K = 1;
    while (p.K * 32 * vc < p.W) p.K *= 2;                  // 16-byte groups per lane
    const int widest = value_size > out_size ? value_size : out_size;
    p.slot_bytes = (p.W * widest + 127) / 128 * 128;
    p.n_slots = kPipeSlots;                                // at most; the launcher may use fewer
    return p;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Everything about the workspace follows from the shapes alone, so the same
// shapes always give the same chunking and therefore the same summation order.
inline Layout make_layout(int64_t n_rows, int32_t R, int64_t d, int64_t vocab, int value_size, int out_size) {
    Layout L{};
    L.n_rows = n_rows; L.vocab = vocab; L.d = d; L.R = R;
    // Work-item sizes: about a third of a warp's fair share of units (one unit = one source row),
    // so that the tail of the row-reduction kernel stays short.
    const int64_t share = (vocab + n_rows) / (int64_t(kPipeWarpsTotal) * 3);
    int c = 16;
    const int64_t max_chunk = kMaxChunkRows;
    while (c < max_chunk && c * 2 <= share) c *= 2;
    L.batch_units = int(share < 8 ? 8 : (share > kMaxBatchUnits ? kMaxBatchUnits : share));
    {
        int pow2 = 8;                                     // the small-input path cuts items of the power of two below batch_units
        while (pow2 * 2 <= L.batch_units) pow2 *= 2;
        L.batch_max = (vocab + n_rows) / pow2 + 2;
    }
    // A large input that names one row only is nothing but chunk items of equal length: cut them so that a whole
    // number of rounds gives every warp the same number (with 128 entries, 3.46 items per warp meant four rounds
    // for some warps and three for others).  Small inputs keep the power of two their index path needs.
    if (c == max_chunk && n_rows > kFrontMaxRows) {
        const int64_t warps = int64_t(kSmCount) * (value_size == 2 ? 16 : 8);
        const int64_t rounds = (n_rows + warps * max_chunk - 1) / (warps * max_chunk);
        const int64_t even = (n_rows + warps * rounds - 1) / (warps * rounds);
        if (even >= max_chunk / 2 && even <= max_chunk) c = int(even);
    }
    L.chunk = c;
    int bits = 0;
    while (bits < 31 && (int64_t(1) << bits) < vocab) ++bits;   // keys are < vocab <= 2^bits
    L.passes = bits <= 8 ? 1 : (bits + 7) / 8;
    L.n_tiles = (n_rows + kTile - 1) / kTile;
    L.vocab_pad = (vocab + kScanItems - 1) / kScanItems * kScanItems;
    L.heavy_max = n_rows / (c + 1);
    L.chunk_max = n_rows / c + L.heavy_max;
    L.upper_max = L.chunk_max / 2 + L.heavy_max + 1;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    L.off_header = take(sizeof(WsHeader));
    L.off_count = take(size_t(L.vocab_pad) * 4);
    L.off_digit = take(size_t(kMaxPasses) * 256 * 4);
    L.off_desc = take(size_t(L.passes) * size_t(L.n_tiles) * 256 * 4);
    L.off_nodecnt = take(size_t(L.upper_max) * size_t(pipe_shape(value_size, out_size, d).ncb) * 4);
    L.off_batches = take(size_t(L.batch_max) * 8);
    L.off_scandesc = take(size_t((L.vocab_pad + kScanTile - 1) / kScanTile + 1) * 64);
    L.zero_bytes = o;
    L.off_offsets = take(size_t(L.vocab_pad + kScanItems) * 4);
    L.off_keys[0] = take(size_t(n_rows) * 4);
    L.off_keys[1] = take(size_t(n_rows) * 4);
    L.off_pos[0] = take(size_t(n_rows) * 4);
    L.off_pos[1] = take(size_t(n_rows) * 4);
    L.off_tab = take(size_t(R > 0 ? R : 1) * sizeof(SliceEntry));
    L.off_heavy = take(size_t(L.heavy_max + 1) * sizeof(HeavyInfo));
    {
        const int64_t cap = (n_rows < vocab ? n_rows : vocab) + 2;
        L.off_urow = take(size_t(cap) * 4);
        L.off_uoff = take(size_t(cap) * 4);
    }
    // named-row bitmap of the small-input path: one copy per CTA of the index cluster, word w of copy r at [w * 8 + r]
    L.bitmap_words = (n_rows <= kFrontMaxRows && vocab <= 65536) ? int((vocab + 31) / 32) : 0;
    L.off_bitmap = take(size_t(L.bitmap_words) * kClusterCtas * 4);
    L.off_partials = take(size_t(L.chunk_max + L.upper_max) * size_t(d) * 4);
    L.total = o;
    return L;
}

// ---- kernel launchers (defined next to their kernels) ----------------------------
struct ScanParams {
    WsHeader* hdr;
    const unsigned* count;
    int* offsets;
    HeavyInfo* heavy;
    void* unique_rows;
    int* counts_out;
    dst_result_t* result;
    int2* batches;
    int* scan_desc;
    int vocab, vocab_pad, chunk, batch_units;
    int wide;              // unique_rows holds 64-bit integers
};
// count != nullptr: the kernel also counts the entries of every row (vocab <= kCountInPrepMaxVocab)
cudaError_t launch_prep(const HistParams& P, int grid_x, int index_type, WsHeader* hdr, unsigned* digit_hist,
                        unsigned* keys, SliceEntry* tab, long long vocab, int passes, unsigned* count, cudaStream_t stream);
// out_keys == nullptr: the last pass, whose keys nobody reads; scan != nullptr: the scan tiles ride in this launch
// items: keys per thread, from radix_items(); a pass over n keys then has ceil(n / (kRadixThreads * items)) tiles
int radix_items(long long n, int extra_ctas, int sms);
int scan_tile_count(int vocab_pad);
cudaError_t launch_radix_pass(int items, int sms, WsHeader* hdr, const unsigned* in_keys, const unsigned* in_pos,
                              unsigned* out_keys, unsigned* out_pos, const unsigned* digit_hist, unsigned* desc,
                              int pass, int capacity, const ScanParams* scan, cudaStream_t stream);
struct FrontParams {
    HistParams P;
    WsHeader* hdr;
    SliceEntry* tab;
    unsigned* perm;
    HeavyInfo* heavy;
    void* unique_rows;
    int* counts_out;
    dst_result_t* result;
    unsigned* node_cnt;
    int* bfirst;               // light work items: rank of the first named row of each, then the number of named rows
    long long vocab;
    int n_total, chunk, batch_units, nodecnt_words;
    unsigned* urec;            // the named rows, ascending: row << 16 | first entry in perm[]; then the number of entries
    unsigned* bitmap;          // named-row bitmap, written early for the row-reduction kernel running beside this one
    int bitmap_words;
};
cudaError_t launch_front_cluster(int index_type, const FrontParams& p, cudaStream_t stream);
cudaError_t launch_bounds(const WsHeader* hdr, const unsigned* keys, unsigned* count, int capacity, int vocab,
                          cudaStream_t stream);
cudaError_t launch_scan(const ScanParams& p, cudaStream_t stream);
// ---- accumulation dispatcher (Algorithms 1 and 2) ----
constexpr int kSumFanIn = 8;                // dense tensors summed per launch
struct SumParams {
    const void* src[kSumFanIn];
    void* out;
    long long n_elems;
    int k;
    int vector_ok;                          // every pointer 16-byte aligned
};
cudaError_t launch_sum_dense(const SumParams& p, int out_type, int sm_count, cudaStream_t stream);
cudaError_t launch_iota(void* indices, long long n, int index_type, int sm_count, cudaStream_t stream);
cudaError_t launch_reduce_rows(const MainArgs& a, int value_type, int out_type, bool vector_ok, int sm_count,
                               cudaStream_t stream);
cudaError_t launch_selftest_wait(WsHeader* hdr, dst_result_t* result, long long limit, cudaStream_t stream);

// Launch with programmatic stream serialisation: the kernel may be scheduled while its predecessor
// in the stream is still running (once all of the predecessor's CTAs have called pdl_trigger), so the
// launch latency and the kernel's prologue overlap with the predecessor's tail.  Every kernel calls
// pdl_wait before it touches memory that an earlier kernel may still be writing.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// The opt-in to a kernel's dynamic shared memory size is made once per device and kernel (and again when a
// larger size is asked for), not on every call.  One cache object per kernel instantiation.
struct SmemOptIn { std::atomic<int> bytes[64]; };
template <typename Kernel>
inline cudaError_t ensure_dynamic_smem(Kernel kernel, size_t bytes, SmemOptIn& cache) {
    int dev = -1;
    const bool cached = cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64;
    if (cached && cache.bytes[dev].load() >= (int)bytes) return cudaSuccess;
    const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess && cached) cache.bytes[dev].store((int)bytes);
    return e;
}

// ---- device helpers ---------------------------------------------------------
#ifdef __CUDACC__
// the kernels after this one in the stream may be scheduled now / wait for the kernels before this one
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ int lane_id() { return threadIdx.x & 31; }
__device__ __forceinline__ int warp_id() { return threadIdx.x >> 5; }

__device__ __forceinline__ void raise_status(WsHeader* hdr, int code) { atomicMax(&hdr->status, code); }

// Lanes of the warp whose 8-bit digit equals this lane's, among the lanes with `valid` set
// (eight ballots; the result is meaningless for lanes without `valid`).
__device__ __forceinline__ unsigned match_digit(unsigned dg, bool valid) {
    unsigned m = __ballot_sync(0xFFFFFFFFu, valid);
#pragma unroll
    for (int b = 0; b < 8; ++b) {
        const bool bit = (dg >> b) & 1u;
        const unsigned bal = __ballot_sync(0xFFFFFFFFu, bit);
        m &= bit ? bal : ~bal;
    }
    return m;
}

// Units a row contributes to the light work items: its entries and the unit that closes it; a heavy
// row only keeps its place.
__host__ __device__ __forceinline__ int row_units(int cc, int chunk) { return cc > chunk ? 1 : cc + 1; }

// Number of combine-tree nodes above the chunk level for a row split into n chunks.
__host__ __device__ __forceinline__ int upper_nodes(int n) {
    int u = 0;
    while (n > 1) { n = (n + kFanIn - 1) / kFanIn; u += n; }
    return u;
}
#endif

}  // namespace dst
