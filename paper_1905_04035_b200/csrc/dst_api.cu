// C ABI of the densify library: argument checks, workspace carving, kernel sequencing.
#include <math.h>
#include <string.h>

#include <atomic>
#include <memory>
#include <new>
#include <mutex>

#include <nvtx3/nvToolsExt.h>

#include "dst_common.cuh"

namespace dst {

static thread_local cudaEvent_t t_ev_before = nullptr, t_ev_after = nullptr;
static std::atomic<long long> g_launches{0};
static std::atomic<int> g_ranges{0};    // NVTX ranges around the phases of a call: off unless dst_profile_ranges(1)

// An NVTX range on the calling host thread for as long as the object lives (nothing when ranges are off).
struct PhaseRange {
    bool on;
    explicit PhaseRange(const char* name) : on(g_ranges.load(std::memory_order_relaxed) != 0) { if (on) nvtxRangePushA(name); }
    ~PhaseRange() { if (on) nvtxRangePop(); }
};

static size_t index_size(int t) { return t == DST_I64 ? 8 : 4; }
static size_t dtype_size(int t) { return t == DST_F32 ? 4 : 2; }

static bool opts_ok(const dst_opts_t* o) {
    return o && (o->index_type == DST_I32 || o->index_type == DST_I64) &&
           (o->value_type == DST_F32 || o->value_type == DST_BF16) &&
           (o->out_type == DST_F32 || o->out_type == DST_BF16) && o->flags == 0;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int sm_count() {
    // asked of the runtime once per device ordinal
    constexpr int kDevices = 64;
    static std::atomic<int> cached[kDevices];
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return kSmCount;
    if (dev >= 0 && dev < kDevices && (n = cached[dev].load()) > 0) return n;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return kSmCount;
    if (dev >= 0 && dev < kDevices) cached[dev].store(n);
    return n;
}

// `dense`: the n_dense dense partners (n_dense <= kMaxDensePartners, no null among them), added after the value
// rows in the order given.
static int densify_impl(const dst_slice_t* slices, int32_t R, int64_t d, int64_t vocab, const void* const* dense,
                        int n_dense, void* out, cudaStream_t stream, const dst_opts_t* opts, void* workspace,
                        size_t workspace_bytes, void* unique_rows, int32_t* counts, dst_result_t* result,
                        const dst_optimizer_t* optimizer = nullptr) {
    if (!opts_ok(opts)) return opts ? DST_ERR_UNSUPPORTED : DST_ERR_INVALID_ARG;
    if (n_dense < 0 || n_dense > kMaxDensePartners || (n_dense > 0 && !dense)) return DST_ERR_INVALID_ARG;
    for (int p = 0; p < n_dense; ++p) if (!dense[p]) return DST_ERR_INVALID_ARG;
    const void* dense_in = n_dense > 0 ? dense[0] : nullptr;
    const bool apply = optimizer != nullptr;
    // with an optimizer `out` is the fp32 weight; value rows and dense_in share one type
    if (apply && opts->value_type != opts->out_type) return DST_ERR_UNSUPPORTED;
    if (apply && out && (out == optimizer->state1 || out == optimizer->state2))
        return DST_ERR_INVALID_ARG;                                    // the weight is not its own state
    for (int p = 0; apply && p < n_dense; ++p) if (dense[p] == out) return DST_ERR_INVALID_ARG;   // nor its own gradient
    if (apply) {
        const int k = optimizer->kind;
        if (k != DST_OPT_SGD && k != DST_OPT_MOMENTUM && k != DST_OPT_ADAM) return DST_ERR_INVALID_ARG;
        if (k != DST_OPT_SGD && vocab > 0 && d > 0 && !optimizer->state1) return DST_ERR_INVALID_ARG;
        if (k == DST_OPT_ADAM && vocab > 0 && d > 0 && (!optimizer->state2 || optimizer->state2 == optimizer->state1))
            return DST_ERR_INVALID_ARG;
        if (k == DST_OPT_ADAM && (optimizer->step < 1 || !(optimizer->beta1 >= 0.f && optimizer->beta1 < 1.f) ||
                                  !(optimizer->beta2 >= 0.f && optimizer->beta2 < 1.f)))
            return DST_ERR_INVALID_ARG;
    }
    if (R < 0 || d < 0 || vocab < 0 || (R > 0 && !slices)) return DST_ERR_INVALID_ARG;
    if (vocab > kMaxVocab) return DST_ERR_UNSUPPORTED;
    int64_t n_total = 0;
    for (int r = 0; r < R; ++r) {
        if (slices[r].n_rows < 0) return DST_ERR_INVALID_ARG;
        if (slices[r].n_rows > 0 && (!slices[r].indices || (!slices[r].values && d > 0))) return DST_ERR_INVALID_ARG;
        n_total += slices[r].n_rows;
        if (n_total > kMaxRows) return DST_ERR_UNSUPPORTED;
    }
    if (vocab == 0 || d == 0) return DST_OK;
    if (!out || !workspace) return DST_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return DST_ERR_INVALID_ARG;
    const Layout L = make_layout(n_total, R, d, vocab, int(dtype_size(opts->value_type)), int(dtype_size(opts->out_type)));
    if (workspace_bytes < L.total) return DST_ERR_WORKSPACE_TOO_SMALL;

    char* ws = static_cast<char*>(workspace);
    WsHeader* hdr = reinterpret_cast<WsHeader*>(ws + L.off_header);
    unsigned* count = reinterpret_cast<unsigned*>(ws + L.off_count);
    unsigned* digit = reinterpret_cast<unsigned*>(ws + L.off_digit);
    unsigned* desc = reinterpret_cast<unsigned*>(ws + L.off_desc);
    unsigned* nodecnt = reinterpret_cast<unsigned*>(ws + L.off_nodecnt);
    int2* batches = reinterpret_cast<int2*>(ws + L.off_batches);
    int* offsets = reinterpret_cast<int*>(ws + L.off_offsets);
    unsigned* keys[2] = {reinterpret_cast<unsigned*>(ws + L.off_keys[0]), reinterpret_cast<unsigned*>(ws + L.off_keys[1])};
    unsigned* pos[2] = {reinterpret_cast<unsigned*>(ws + L.off_pos[0]), reinterpret_cast<unsigned*>(ws + L.off_pos[1])};
    SliceEntry* tab = reinterpret_cast<SliceEntry*>(ws + L.off_tab);
    HeavyInfo* heavy = reinterpret_cast<HeavyInfo*>(ws + L.off_heavy);
    float* partials = reinterpret_cast<float*>(ws + L.off_partials);

    // the fast kernels need 16-byte aligned rows everywhere
    const size_t smallest = dtype_size(opts->value_type) < dtype_size(opts->out_type) ? dtype_size(opts->value_type)
                                                                                      : dtype_size(opts->out_type);
    bool vector_ok = d % int64_t(16 / smallest) == 0 && aligned16(out);
    for (int p = 0; p < n_dense; ++p) vector_ok = vector_ok && aligned16(dense[p]);
    if (apply) vector_ok = vector_ok && aligned16(optimizer->state1) && aligned16(optimizer->state2);
    for (int r = 0; r < R && vector_ok; ++r)
        if (slices[r].n_rows > 0 && !aligned16(slices[r].values)) vector_ok = false;

    const unsigned* perm = pos[L.passes & 1];
    bool compact = false, overlap = false;
    // Small input with no more input rows than vocabulary rows (and rows the vector kernels can take): one cluster
    // kernel does the whole index side.  Most output rows are then named by nobody: the tables list the named
    // rows only, and the row-reduction kernel, running beside the index cluster, gives the other rows their
    // dense_in row (or zeros, or the dense part of the SGD step) while the index work is under way.  In place
    // there is nothing to do for those rows.
    PhaseRange call_range(apply ? "dst: densify + optimizer step" : "dst: densify");
    const bool small = n_total <= kFrontMaxRows && vocab <= 65536 && R <= kHistSlices && vector_ok && n_total <= vocab;
    if (small) {
        PhaseRange index_range("dst: index cluster (validate, sort, tables)");
        FrontParams fp;
        memset(&fp.P, 0, sizeof fp.P);
        fp.P.n = R;
        int64_t start = 0;
        for (int i = 0; i < R; ++i) {
            fp.P.s[i] = SliceEntry{slices[i].indices, slices[i].values, (long long)start, (long long)slices[i].n_rows};
            start += slices[i].n_rows;
        }
        fp.hdr = hdr; fp.tab = tab; fp.perm = pos[0]; fp.heavy = heavy;
        fp.unique_rows = unique_rows; fp.counts_out = counts; fp.result = result;
        fp.node_cnt = nodecnt; fp.vocab = vocab; fp.n_total = int(n_total);
        fp.chunk = L.chunk; fp.batch_units = L.batch_units; fp.bfirst = reinterpret_cast<int*>(batches);
        fp.nodecnt_words = int((L.off_batches - L.off_nodecnt) / 4);
        compact = true;
        // (plain SGD without a dense partner leaves the rows nobody names alone; momentum and Adam move every row)
        // (several dense partners: every row is at least their sum)
        overlap = apply ? (n_dense > 0 || optimizer->kind != DST_OPT_SGD) : (n_dense > 1 || out != dense_in);
        fp.urec = reinterpret_cast<unsigned*>(ws + L.off_urow);
        fp.bitmap = reinterpret_cast<unsigned*>(ws + L.off_bitmap);
        fp.bitmap_words = L.bitmap_words;
        if (launch_front_cluster(opts->index_type, fp, stream) != cudaSuccess) return DST_ERR_CUDA;
        ++g_launches;
        perm = pos[0];
    } else {
        PhaseRange index_range("dst: index kernels (validate, radix passes, bounds, scan)");
        if (cudaMemsetAsync(ws, 0, L.zero_bytes, stream) != cudaSuccess) return DST_ERR_CUDA;
        // With a vocabulary small enough, the validation kernel counts the entries of every row itself; the
        // scan then rides in the launch of the first radix pass and no pass over the sorted keys is needed.
        const bool early_count = n_total > 0 && vocab <= kCountInPrepMaxVocab;
        ScanParams sp{hdr, count, offsets, heavy, unique_rows, counts, result, batches,
                      reinterpret_cast<int*>(ws + L.off_scandesc), int(vocab), int(L.vocab_pad), L.chunk, L.batch_units,
                      opts->index_type == DST_I64 ? 1 : 0};
        // a1: validate and narrow, at most kHistSlices slices per launch
        int64_t start = 0;
        for (int first = 0; first < R; first += kHistSlices) {
            HistParams P;
            memset(&P, 0, sizeof P);
            P.n = R - first < kHistSlices ? R - first : kHistSlices;
            P.first = first;
            int64_t longest = 0;
            for (int i = 0; i < P.n; ++i) {
                const dst_slice_t& s = slices[first + i];
                P.s[i] = SliceEntry{s.indices, s.values, (long long)start, (long long)s.n_rows};
                start += s.n_rows;
                if (s.n_rows > longest) longest = s.n_rows;
            }
            int grid_x = int((longest + kPrepTile - 1) / kPrepTile);
            if (grid_x < 1) grid_x = 1;   // still writes the slice table
            if (launch_prep(P, grid_x, opts->index_type, hdr, digit, keys[0], tab, vocab, L.passes,
                            early_count ? count : nullptr, stream) != cudaSuccess)
                return DST_ERR_CUDA;
            ++g_launches;
        }
        if (n_total > 0) {
            // a4: least significant digit first; keys/positions ping-pong between two buffers
            const int items = radix_items(n_total, early_count ? scan_tile_count(int(L.vocab_pad)) : 0, sm_count());
            for (int p = 0; p < L.passes; ++p) {
                // (the sorted keys of the last pass are read by the run-length kernel only)
                unsigned* keys_out = early_count && p == L.passes - 1 ? nullptr : keys[(p + 1) & 1];
                if (launch_radix_pass(items, sm_count(), hdr, keys[p & 1], p == 0 ? nullptr : pos[p & 1], keys_out,
                                      pos[(p + 1) & 1], digit + p * 256, desc + size_t(p) * size_t(L.n_tiles) * 256, p,
                                      int(n_total), early_count && p == 0 ? &sp : nullptr, stream) != cudaSuccess)
                    return DST_ERR_CUDA;
                ++g_launches;
            }
            // a2: run lengths of the sorted keys
            if (!early_count) {
                if (launch_bounds(hdr, keys[L.passes & 1], count, int(n_total), int(vocab), stream) != cudaSuccess)
                    return DST_ERR_CUDA;
                ++g_launches;
            }
        }
        // a3/a5/a6
        if (!early_count) {
            if (launch_scan(sp, stream) != cudaSuccess) return DST_ERR_CUDA;
            ++g_launches;
        }
    }
    // a7/a8
    MainArgs a;
    a.hdr = hdr; a.offsets = offsets; a.perm = perm; a.tab = tab; a.heavy = heavy;
    a.batches = batches; a.node_cnt = nodecnt; a.partials = partials; a.dense_in = dense_in; a.out = out;
    a.n_dense = n_dense;
    for (int p = 1; p < kMaxDensePartners; ++p) a.dense_more[p - 1] = p < n_dense ? dense[p] : nullptr;
    a.result = result; a.d = d; a.vocab = int(vocab); a.n_total = int(n_total); a.R = R; a.chunk = L.chunk;
    a.chunk_max = int(L.chunk_max); a.upper_max = int(L.upper_max);
    a.W = a.ncb = a.slot_bytes = a.n_slots = 0;   // set by the launcher
    a.compact = compact ? 1 : 0;
    a.overlap = overlap ? 1 : 0;
    a.bitmap = reinterpret_cast<const unsigned*>(ws + L.off_bitmap);
    a.bitmap_words = L.bitmap_words;
    a.copy_rows = 8; a.copy_slots = 0;     // set by the launcher
    a.apply = 0; a.lr = 0.f; a.grad_scale = 1.f; a.opt_a = a.opt_b = a.opt_eps = 0.f; a.opt_bc1 = a.opt_bc2 = 1.f;
    a.state1 = a.state2 = nullptr;
    if (apply) {
        a.apply = optimizer->kind + 1;               // the kernels' numbering: 1 SGD, 2 momentum, 3 Adam
        a.lr = optimizer->lr; a.grad_scale = optimizer->grad_scale;
        a.state1 = optimizer->state1; a.state2 = optimizer->state2;
        if (optimizer->kind == DST_OPT_MOMENTUM) a.opt_a = optimizer->momentum;
        if (optimizer->kind == DST_OPT_ADAM) {
            a.opt_a = optimizer->beta1; a.opt_b = optimizer->beta2; a.opt_eps = optimizer->eps;
            a.opt_bc1 = float(1.0 / (1.0 - pow(double(optimizer->beta1), double(optimizer->step))));
            a.opt_bc2 = float(1.0 / (1.0 - pow(double(optimizer->beta2), double(optimizer->step))));
        }
    }
    a.urec = reinterpret_cast<const unsigned*>(ws + L.off_urow);
    PhaseRange reduce_range("dst: row reduction");
    if (t_ev_before && cudaEventRecord(t_ev_before, stream) != cudaSuccess) return DST_ERR_CUDA;
    if (launch_reduce_rows(a, opts->value_type, opts->out_type, vector_ok, sm_count(), stream) != cudaSuccess)
        return DST_ERR_CUDA;
    ++g_launches;
    if (t_ev_after && cudaEventRecord(t_ev_after, stream) != cudaSuccess) return DST_ERR_CUDA;
    return DST_OK;
}

// ---- scratch for dst_densify_static ------------------------------------------------
// Device global memory that belongs to the library itself: every GPU that loads the
// library holds one copy until the process exits.  In host code this name is only a
// handle for the runtime's symbol look-up, never a device address; kernels get the
// address that cudaGetSymbolAddress returns for the current device.
static __device__ __align__(256) unsigned char g_static_workspace[DST_STATIC_WORKSPACE_BYTES];

constexpr int kMaxDevices = 64;
static std::mutex g_static_mutex;
static void* g_static_ptr[kMaxDevices];   // device address of the array, per device ordinal

// Address of the array on the current device; looked up once per device.
static cudaError_t static_workspace(void** ptr) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_workspace);
        if (e != cudaSuccess) return e;
        if (!p) return cudaErrorInvalidSymbol;
        g_static_ptr[dev] = p;
    }
    *ptr = g_static_ptr[dev];
    return cudaSuccess;
}

}  // namespace dst

using namespace dst;

extern "C" {

int dst_version(void) { return 100; }

void dst_profile_events(void* before, void* after) {
    t_ev_before = static_cast<cudaEvent_t>(before);
    t_ev_after = static_cast<cudaEvent_t>(after);
}

int64_t dst_kernel_launches(void) { return g_launches.load(); }

void dst_profile_ranges(int on) { g_ranges.store(on ? 1 : 0); }

const char* dst_status_string(int status) {
    switch (status) {
        case DST_OK: return "ok";
        case DST_ERR_INVALID_ARG: return "invalid argument";
        case DST_ERR_UNSUPPORTED: return "unsupported type or size";
        case DST_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case DST_ERR_INDEX_OUT_OF_RANGE: return "some indices were outside [0, vocab) and were skipped";
        case DST_ERR_TIMEOUT: return "a bounded device-side wait gave up; output invalid";
        case DST_ERR_CUDA: return "CUDA runtime error";
        default: return "unknown status";
    }
}

size_t dst_workspace_bytes(int64_t n_rows_total, int32_t R, int64_t d, int64_t vocab, const dst_opts_t* opts) {
    if (!opts_ok(opts) || n_rows_total < 0 || n_rows_total > kMaxRows || R < 0 || d < 0 || vocab < 0 || vocab > kMaxVocab)
        return 0;
    return make_layout(n_rows_total, R, d, vocab, int(dtype_size(opts->value_type)), int(dtype_size(opts->out_type))).total;
}

int dst_densify(const void* indices, const void* values, int64_t n_rows, int64_t d, int64_t vocab,
                const void* dense_in, void* out, dst_stream_t stream, const dst_opts_t* opts, void* workspace,
                size_t workspace_bytes, void* unique_rows, int32_t* counts, dst_result_t* result) {
    dst_slice_t s{indices, values, n_rows};
    return densify_impl(&s, 1, d, vocab, &dense_in, dense_in ? 1 : 0, out, stream, opts, workspace, workspace_bytes,
                        unique_rows, counts, result);
}

int dst_densify_concat(const dst_slice_t* slices, int32_t R, int64_t d, int64_t vocab, const void* dense_in,
                       void* out, dst_stream_t stream, const dst_opts_t* opts, void* workspace,
                       size_t workspace_bytes, void* unique_rows, int32_t* counts, dst_result_t* result) {
    return densify_impl(slices, R, d, vocab, &dense_in, dense_in ? 1 : 0, out, stream, opts, workspace, workspace_bytes,
                        unique_rows, counts, result);
}

int dst_densify_apply_sgd(const dst_slice_t* slices, int32_t R, int64_t d, int64_t vocab, const void* dense_in,
                          void* weight, float lr, dst_stream_t stream, const dst_opts_t* opts, void* workspace,
                          size_t workspace_bytes, void* unique_rows, int32_t* counts, dst_result_t* result) {
    if (opts_ok(opts) && (opts->value_type != DST_F32 || opts->out_type != DST_F32)) return DST_ERR_UNSUPPORTED;
    dst_optimizer_t sgd{};
    sgd.kind = DST_OPT_SGD; sgd.lr = lr; sgd.grad_scale = 1.f;
    return densify_impl(slices, R, d, vocab, &dense_in, dense_in ? 1 : 0, weight, stream, opts, workspace, workspace_bytes,
                        unique_rows, counts, result, &sgd);
}

int dst_densify_apply(const dst_slice_t* slices, int32_t R, int64_t d, int64_t vocab, const void* dense_in,
                      void* weight, const dst_optimizer_t* optimizer, dst_stream_t stream, const dst_opts_t* opts,
                      void* workspace, size_t workspace_bytes, void* unique_rows, int32_t* counts, dst_result_t* result) {
    if (!optimizer) return DST_ERR_INVALID_ARG;
    return densify_impl(slices, R, d, vocab, &dense_in, dense_in ? 1 : 0, weight, stream, opts, workspace, workspace_bytes,
                        unique_rows, counts, result, optimizer);
}

int dst_densify_static(const void* indices, const void* values, int64_t n_rows, int64_t d, int64_t vocab,
                       const void* dense_in, void* out, dst_stream_t stream, const dst_opts_t* opts,
                       void* unique_rows, int32_t* counts, dst_result_t* result) {
    if (!opts_ok(opts)) return opts ? DST_ERR_UNSUPPORTED : DST_ERR_INVALID_ARG;
    if (n_rows < 0 || d < 0 || vocab < 0) return DST_ERR_INVALID_ARG;
    if (n_rows > kMaxRows || vocab > kMaxVocab) return DST_ERR_UNSUPPORTED;
    if (vocab == 0 || d == 0) return DST_OK;
    // the shape decides the need; refuse before touching the device
    if (make_layout(n_rows, 1, d, vocab, int(dtype_size(opts->value_type)), int(dtype_size(opts->out_type))).total >
        size_t(DST_STATIC_WORKSPACE_BYTES)) return DST_ERR_WORKSPACE_TOO_SMALL;
    void* ws = nullptr;
    if (static_workspace(&ws) != cudaSuccess) return DST_ERR_CUDA;
    dst_slice_t s{indices, values, n_rows};
    return densify_impl(&s, 1, d, vocab, &dense_in, dense_in ? 1 : 0, out, stream, opts, ws, size_t(DST_STATIC_WORKSPACE_BYTES),
                        unique_rows, counts, result);
}

size_t dst_host_staging_bytes(int64_t n_rows_total, int64_t d, int64_t vocab, const dst_opts_t* opts) {
    if (!opts_ok(opts) || n_rows_total < 0 || d < 0 || vocab < 0) return 0;
    size_t o = 0;
    o = align_up(o + size_t(n_rows_total) * index_size(opts->index_type), 256);
    o = align_up(o + size_t(n_rows_total) * size_t(d) * dtype_size(opts->value_type), 256);
    o = align_up(o + size_t(vocab) * size_t(d) * dtype_size(opts->out_type), 256);
    o = align_up(o + sizeof(dst_result_t), 256);
    return o;
}

int dst_densify_concat_host(const dst_slice_t* slices, int32_t R, int64_t d, int64_t vocab,
                            const void* host_dense_in, void* host_out, dst_stream_t stream, const dst_opts_t* opts,
                            void* staging, size_t staging_bytes, void* workspace, size_t workspace_bytes,
                            dst_result_t* host_result) {
    if (!opts_ok(opts)) return opts ? DST_ERR_UNSUPPORTED : DST_ERR_INVALID_ARG;
    if (R < 0 || d < 0 || vocab < 0 || (R > 0 && !slices)) return DST_ERR_INVALID_ARG;
    int64_t n_total = 0;
    for (int r = 0; r < R; ++r) {
        if (slices[r].n_rows < 0) return DST_ERR_INVALID_ARG;
        if (slices[r].n_rows > 0 && (!slices[r].indices || (!slices[r].values && d > 0))) return DST_ERR_INVALID_ARG;
        n_total += slices[r].n_rows;
        if (n_total > kMaxRows) return DST_ERR_UNSUPPORTED;
    }
    if (vocab == 0 || d == 0) return DST_OK;
    if (!host_out || !staging || (reinterpret_cast<uintptr_t>(staging) & 255u)) return DST_ERR_INVALID_ARG;
    if (staging_bytes < dst_host_staging_bytes(n_total, d, vocab, opts)) return DST_ERR_WORKSPACE_TOO_SMALL;
    if (!workspace || workspace_bytes < dst_workspace_bytes(n_total, 1, d, vocab, opts)) return DST_ERR_WORKSPACE_TOO_SMALL;
    const size_t si = index_size(opts->index_type), sv = dtype_size(opts->value_type), so = dtype_size(opts->out_type);
    char* st = static_cast<char*>(staging);
    size_t o = 0;
    char* d_idx = st + o; o = align_up(o + size_t(n_total) * si, 256);
    char* d_val = st + o; o = align_up(o + size_t(n_total) * size_t(d) * sv, 256);
    char* d_out = st + o; o = align_up(o + size_t(vocab) * size_t(d) * so, 256);
    dst_result_t* d_res = reinterpret_cast<dst_result_t*>(st + o);
    // host -> device: the slices land back to back, i.e. as their concatenation
    size_t row = 0;
    for (int r = 0; r < R; ++r) {
        const size_t n = size_t(slices[r].n_rows);
        if (n == 0) continue;
        if (cudaMemcpyAsync(d_idx + row * si, slices[r].indices, n * si, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
            cudaMemcpyAsync(d_val + row * size_t(d) * sv, slices[r].values, n * size_t(d) * sv, cudaMemcpyHostToDevice,
                            stream) != cudaSuccess)
            return DST_ERR_CUDA;
        row += n;
    }
    const size_t out_bytes = size_t(vocab) * size_t(d) * so;
    if (host_dense_in &&
        cudaMemcpyAsync(d_out, host_dense_in, out_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return DST_ERR_CUDA;
    dst_slice_t s{d_idx, d_val, n_total};
    const void* partner = d_out;
    int rc = densify_impl(&s, 1, d, vocab, &partner, host_dense_in ? 1 : 0, d_out, stream, opts, workspace,
                          workspace_bytes, nullptr, nullptr, d_res);
    if (rc != DST_OK) return rc;
    if (cudaMemcpyAsync(host_out, d_out, out_bytes, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return DST_ERR_CUDA;
    if (host_result &&
        cudaMemcpyAsync(host_result, d_res, sizeof(dst_result_t), cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return DST_ERR_CUDA;
    return DST_OK;
}

// ---- Algorithms 1 and 2, Listing 1: which branch a list of gradients takes ----
int dst_accumulate_plan(const dst_grad_t* grads, int32_t n, int64_t d, int64_t vocab, int32_t strategy,
                        const dst_opts_t* opts, dst_accum_plan_t* plan) {
    if (!plan || n < 0 || d < 0 || vocab < 0 || (n > 0 && !grads)) return DST_ERR_INVALID_ARG;
    if (!opts_ok(opts)) return opts ? DST_ERR_UNSUPPORTED : DST_ERR_INVALID_ARG;
    if (strategy != DST_ACC_STOCK && strategy != DST_ACC_PROPOSED && strategy != DST_ACC_SPARSE_AS_DENSE)
        return DST_ERR_INVALID_ARG;
    dst_accum_plan_t p{};
    for (int i = 0; i < n; ++i) {
        if (grads[i].kind == DST_GRAD_DENSE) {
            ++p.n_dense;
        } else if (grads[i].kind == DST_GRAD_SLICES) {
            if (grads[i].n_rows < 0) return DST_ERR_INVALID_ARG;
            ++p.n_slices;
            p.n_slice_rows += grads[i].n_rows;
            if (p.n_slice_rows > kMaxRows) return DST_ERR_UNSUPPORTED;
        } else {
            return DST_ERR_INVALID_ARG;
        }
    }
    const int64_t sv = (int64_t)dtype_size(opts->value_type), so = (int64_t)dtype_size(opts->out_type);
    const int64_t si = (int64_t)index_size(opts->index_type);
    // Listing 1 converts each IndexedSlices gradient before Algorithm 1 looks at the list
    const bool all_dense = p.n_slices == 0 || strategy == DST_ACC_SPARSE_AS_DENSE;
    bool dense_out;
    if (n == 0) {
        p.branch = DST_BRANCH_EMPTY;
        p.out_kind = -1;
        *plan = p;
        return DST_OK;
    } else if (n < 2) {
        p.branch = DST_BRANCH_PASS_THROUGH;
        dense_out = all_dense;
    } else if (all_dense) {
        p.branch = DST_BRANCH_REDUCE;
        dense_out = true;
    } else if (strategy == DST_ACC_PROPOSED && p.n_dense > 0) {
        p.branch = DST_BRANCH_CONVERT_AND_REDUCE;
        dense_out = true;
    } else {
        p.branch = DST_BRANCH_GATHER;
        dense_out = false;
    }
    if (dense_out) {
        p.out_kind = DST_GRAD_DENSE;
        p.out_rows = vocab;
        p.out_bytes = vocab * d * so;
        p.converts = p.n_slices > 0;
    } else {
        p.out_kind = DST_GRAD_SLICES;
        p.out_rows = p.n_slice_rows + (int64_t)p.n_dense * vocab;
        p.out_bytes = p.out_rows * (d * sv + si);
    }
    *plan = p;
    return DST_OK;
}

int dst_accumulate(const dst_grad_t* grads, int32_t n, int64_t d, int64_t vocab, int32_t strategy,
                   void* out_dense, void* out_indices, void* out_values, int64_t out_capacity_rows,
                   dst_stream_t stream, const dst_opts_t* opts, void* workspace, size_t workspace_bytes,
                   dst_result_t* result, dst_accum_plan_t* plan_out) {
    dst_accum_plan_t p{};
    const int rc = dst_accumulate_plan(grads, n, d, vocab, strategy, opts, &p);
    if (rc != DST_OK) return rc;
    if (plan_out) *plan_out = p;
    if (p.branch == DST_BRANCH_EMPTY || vocab == 0 || d == 0) return DST_OK;
    for (int i = 0; i < n; ++i) {
        if (!grads[i].values) { if (grads[i].kind == DST_GRAD_DENSE || grads[i].n_rows > 0) return DST_ERR_INVALID_ARG; }
        if (grads[i].kind == DST_GRAD_SLICES && grads[i].n_rows > 0 && !grads[i].indices) return DST_ERR_INVALID_ARG;
    }
    const size_t sv = dtype_size(opts->value_type), so = dtype_size(opts->out_type), si = index_size(opts->index_type);

    if (p.out_kind == DST_GRAD_SLICES) {
        // gather (or the pass-through of one IndexedSlices gradient): concatenate in the order given
        if (p.out_rows > out_capacity_rows || p.out_rows > kMaxRows) return DST_ERR_INVALID_ARG;
        if (p.out_rows > 0 && (!out_indices || !out_values)) return DST_ERR_INVALID_ARG;
        if (p.n_dense > 0 && opts->value_type != opts->out_type) return DST_ERR_UNSUPPORTED;
        int64_t row = 0;
        for (int i = 0; i < n; ++i) {
            const bool dense = grads[i].kind == DST_GRAD_DENSE;
            const int64_t rows = dense ? vocab : grads[i].n_rows;
            if (rows == 0) continue;
            char* oi = static_cast<char*>(out_indices) + size_t(row) * si;
            char* ov = static_cast<char*>(out_values) + size_t(row) * size_t(d) * sv;
            if (dense) {
                // the rows of a dense tensor are its own indices (Section 3)
                if (launch_iota(oi, rows, opts->index_type, sm_count(), stream) != cudaSuccess) return DST_ERR_CUDA;
                ++g_launches;
            } else if (cudaMemcpyAsync(oi, grads[i].indices, size_t(rows) * si, cudaMemcpyDeviceToDevice, stream) != cudaSuccess) {
                return DST_ERR_CUDA;
            }
            if (cudaMemcpyAsync(ov, grads[i].values, size_t(rows) * size_t(d) * sv, cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
                return DST_ERR_CUDA;
            row += rows;
        }
        return DST_OK;
    }

    // dense output.  The dense gradients in the order given, except that one that is out_dense itself goes first
    // (it must be read before anything lands in out_dense).
    if (!out_dense) return DST_ERR_INVALID_ARG;
    const long long n_elems = (long long)vocab * d;
    std::unique_ptr<const void*[]> list(new (std::nothrow) const void*[p.n_dense + 1]);
    if (!list) return DST_ERR_INVALID_ARG;
    int n_list = 0, n_aliased = 0;
    for (int round = 0; round < 2; ++round)
        for (int i = 0; i < n; ++i)
            if (grads[i].kind == DST_GRAD_DENSE && (grads[i].values == out_dense) == (round == 0)) {
                list[n_list++] = grads[i].values;
                n_aliased += round == 0;
            }
    if (n_aliased > kSumFanIn) return DST_ERR_INVALID_ARG;

    // out_dense = list[0] + ... + list[count - 1], kSumFanIn tensors per pass, the running sum carried in out_dense
    auto sum_passes = [&](int count) -> int {
        SumParams sp{};
        sp.out = out_dense; sp.n_elems = n_elems; sp.vector_ok = aligned16(out_dense);
        bool first = true;
        for (int q = 0; q < count; ++q) {
            sp.src[sp.k++] = list[q];
            sp.vector_ok = sp.vector_ok && aligned16(list[q]);
            if (sp.k == kSumFanIn || q == count - 1) {
                const bool nothing = first && sp.k == 1 && sp.src[0] == out_dense;   // one tensor that already is the output
                if (!nothing && !(!first && sp.k == 1)) {
                    if (launch_sum_dense(sp, opts->out_type, sm_count(), stream) != cudaSuccess) return DST_ERR_CUDA;
                    ++g_launches;
                }
                first = false;
                sp.k = 0; sp.src[sp.k++] = out_dense; sp.vector_ok = aligned16(out_dense);
            }
        }
        return DST_OK;
    };

    const size_t ws_need = make_layout(p.n_slice_rows, p.n_slices, d, vocab, int(dtype_size(opts->value_type)),
                                       int(dtype_size(opts->out_type))).total;
    const bool have_ws = workspace && workspace_bytes >= ws_need && !(reinterpret_cast<uintptr_t>(workspace) & 255u);
    if (p.n_slices == 0 && (n_list <= kSumFanIn || !have_ws)) return sum_passes(n_list);   // a plain sum of dense tensors

    // One pass over everything (Fig. 3b of the paper, all ranks at once): every dense tensor and every value row
    // is read once on the way to its output row.  More dense tensors than one pass takes: the first ones are
    // summed into out_dense beforehand, which then stands for them.
    int first_in_pass = 0;
    if (n_list > kMaxDensePartners) {
        first_in_pass = n_list - (kMaxDensePartners - 1);
        const int rc2 = sum_passes(first_in_pass);
        if (rc2 != DST_OK) return rc2;
        list[--first_in_pass] = out_dense;
    }
    dst_slice_t stack_slices[64];
    dst_slice_t* sl = stack_slices;
    std::unique_ptr<dst_slice_t[]> heap;
    if (p.n_slices > 64) {
        heap.reset(new (std::nothrow) dst_slice_t[p.n_slices]);
        if (!heap) return DST_ERR_INVALID_ARG;
        sl = heap.get();
    }
    int r = 0;
    for (int i = 0; i < n; ++i)
        if (grads[i].kind == DST_GRAD_SLICES) sl[r++] = dst_slice_t{grads[i].indices, grads[i].values, grads[i].n_rows};
    return densify_impl(sl, p.n_slices, d, vocab, list.get() + first_in_pass, n_list - first_in_pass, out_dense, stream, opts,
                        workspace, workspace_bytes, nullptr, nullptr, result);
}

int dst_densify_batch(const dst_rank_grads_t* ranks, int32_t R, int64_t d, int64_t vocab, void* out, dst_stream_t stream,
                      const dst_opts_t* opts, void* workspace, size_t workspace_bytes, void* unique_rows,
                      int32_t* counts, dst_result_t* result) {
    if (R < 0 || (R > 0 && !ranks)) return DST_ERR_INVALID_ARG;
    const void* dense[kMaxDensePartners];
    int n_dense = 0;
    int64_t n_sl = 0;
    for (int r = 0; r < R; ++r) {
        if (ranks[r].n_slices < 0 || (ranks[r].n_slices > 0 && !ranks[r].slices)) return DST_ERR_INVALID_ARG;
        if (ranks[r].dense) {
            if (n_dense == kMaxDensePartners) return DST_ERR_UNSUPPORTED;
            dense[n_dense++] = ranks[r].dense;
        }
        n_sl += ranks[r].n_slices;
    }
    if (n_sl > (1 << 20)) return DST_ERR_UNSUPPORTED;
    std::unique_ptr<dst_slice_t[]> sl(new (std::nothrow) dst_slice_t[n_sl > 0 ? n_sl : 1]);
    if (!sl) return DST_ERR_INVALID_ARG;
    int64_t k = 0;
    for (int r = 0; r < R; ++r)
        for (int q = 0; q < ranks[r].n_slices; ++q) sl[k++] = ranks[r].slices[q];
    return densify_impl(sl.get(), int32_t(n_sl), d, vocab, dense, n_dense, out, stream, opts, workspace, workspace_bytes,
                        unique_rows, counts, result);
}

int dst_selftest_wait_limit(int64_t limit_cycles, void* workspace, size_t workspace_bytes, dst_stream_t stream,
                            dst_result_t* result) {
    if (limit_cycles <= 0 || limit_cycles > kWaitCycles || !workspace || workspace_bytes < 256) return DST_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return DST_ERR_INVALID_ARG;
    if (cudaMemsetAsync(workspace, 0, 256, stream) != cudaSuccess) return DST_ERR_CUDA;
    if (launch_selftest_wait(static_cast<WsHeader*>(workspace), result, (long long)limit_cycles, stream) != cudaSuccess)
        return DST_ERR_CUDA;
    ++g_launches;
    return DST_OK;
}

int dst_bytes_report(const int64_t* n_rows_per_slice, int32_t R, int64_t d, int64_t vocab, const dst_opts_t* opts,
                     dst_bytes_report_t* report) {
    if (!opts_ok(opts)) return opts ? DST_ERR_UNSUPPORTED : DST_ERR_INVALID_ARG;
    if (!report || R < 0 || d < 0 || vocab < 0 || (R > 0 && !n_rows_per_slice)) return DST_ERR_INVALID_ARG;
    const int64_t si = int64_t(index_size(opts->index_type)), sv = int64_t(dtype_size(opts->value_type)),
                  so = int64_t(dtype_size(opts->out_type));
    int64_t n_total = 0, gather_all = 0;
    for (int r = 0; r < R; ++r) {
        if (n_rows_per_slice[r] < 0) return DST_ERR_INVALID_ARG;
        n_total += n_rows_per_slice[r];
        gather_all += (vocab + n_rows_per_slice[r]) * d * sv;
    }
    report->n_rows_total = n_total;
    report->sparse_value_bytes = n_total * d * sv;
    report->sparse_index_bytes = n_total * si;
    report->sparse_bytes = report->sparse_value_bytes + report->sparse_index_bytes;
    report->dense_bytes = vocab * d * so;
    report->gather_all_value_bytes = gather_all;
    report->sparse_over_dense = report->dense_bytes ? double(report->sparse_bytes) / double(report->dense_bytes) : 0.0;
    report->gather_all_over_dense = report->dense_bytes ? double(gather_all) / double(report->dense_bytes) : 0.0;
    return DST_OK;
}

}  // extern "C"
