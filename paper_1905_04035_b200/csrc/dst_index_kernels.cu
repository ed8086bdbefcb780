// Index side of densify: validate, stable radix placement, segment bounds, scan to CSR offsets.
//
// Together these turn the row indices of the (virtually concatenated) IndexedSlices
// of the paper's Section 3 into
//   offsets[v] .. offsets[v+1]   the positions in perm[] that belong to output row v
//   perm[j]                      input row positions, ascending inside each segment
// plus the work-item tables the row-reduction kernel consumes.  Integer work only.
//
// Order of the kernels (large inputs):
//   k_prep        validate, narrow to 32-bit keys, digit histograms of all radix passes
//   k_radix_pass  one per 8-bit digit, least significant first, stable
//   k_bounds      run lengths of the sorted keys -> count[v]
//   k_scan        count[] -> offsets, unique rows, heavy-row chunks, row batches
// Small inputs take k_front_cluster (dst_front_cluster.cu), which does all of it in one kernel.
#include "dst_common.cuh"

namespace dst {

// ---------------------------------------------------------------------------
// a1: validate, narrow to 32-bit keys, per-pass digit histograms
// ---------------------------------------------------------------------------
template <typename IT>
__global__ void __launch_bounds__(kSortThreads)
k_prep(const __grid_constant__ HistParams P, WsHeader* __restrict__ hdr, unsigned* __restrict__ digit_hist,
       unsigned* __restrict__ keys, SliceEntry* __restrict__ tab, long long vocab, int passes) {
    __shared__ unsigned dh[kMaxPasses * 256];
    pdl_trigger();
    pdl_wait();

    const SliceEntry& se = P.s[blockIdx.y];
    if (blockIdx.x == 0 && threadIdx.x == 0) tab[P.first + blockIdx.y] = se;
    const long long n = se.n_rows;
    const long long t0 = (long long)blockIdx.x * kPrepTile;
    if (t0 >= n) return;

    for (int s = threadIdx.x; s < kMaxPasses * 256; s += kSortThreads) dh[s] = 0;
    __syncthreads();

    const IT* __restrict__ idx = static_cast<const IT*>(se.indices);
    const int lane = lane_id();
    unsigned bad = 0;
    long long vals[kPrepItems];          // every index of this thread first: one trip to memory, not kPrepItems
#pragma unroll
    for (int k = 0; k < kPrepItems; ++k) {
        const long long i = t0 + k * kSortThreads + threadIdx.x;
        vals[k] = -1;
        if (i < n) vals[k] = (long long)idx[i];
    }
#pragma unroll
    for (int k = 0; k < kPrepItems; ++k) {
        const long long i = t0 + k * kSortThreads + threadIdx.x;
        const bool in = i < n;
        const long long v = vals[k];
        const bool ok = in && v >= 0 && v < vocab;
        const unsigned key = ok ? (unsigned)v : kInvalidKey;
        if (in) keys[se.start + i] = key;
        bad += in && !ok;
        if (ok)
            for (int p = 0; p < passes; ++p) atomicAdd(&dh[p * 256 + ((key >> (8 * p)) & 255u)], 1u);
    }
    __syncthreads();
    for (int s = threadIdx.x; s < passes * 256; s += kSortThreads) {
        unsigned c = dh[s];
        if (c) atomicAdd(&digit_hist[s], c);
    }
    for (int o = 16; o > 0; o >>= 1) bad += __shfl_down_sync(0xFFFFFFFFu, bad, o);
    if (lane == 0 && bad) atomicAdd(&hdr->n_bad, (unsigned long long)bad);
}

// ---------------------------------------------------------------------------
// a4: one stable 8-bit radix pass (least significant digit first), single sweep
// over the keys with a decoupled look-back for the cross-tile prefix
// ---------------------------------------------------------------------------
// Exclusive prefix of digit d's count over the tiles before `tile`.  Every tile publishes its own
// count first ("aggregate"), then walks back over its predecessors, four at a time, until it meets
// one that has published its inclusive prefix.  Tiles start in ticket order, so every predecessor
// is running or done; the wait on a missing descriptor is bounded all the same.
__device__ __forceinline__ unsigned lookback_exclusive(volatile unsigned* desc, int tile, int d, unsigned cnt,
                                                       WsHeader* hdr) {
    if (tile == 0) { desc[d] = kFlagPrefix | cnt; return 0; }
    desc[(size_t)tile * 256 + d] = kFlagAggregate | cnt;
    unsigned excl = 0;
    bool ok = true, done = false;
    for (int t = tile - 1; t >= 0 && ok && !done; t -= 4) {
        unsigned v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) v[q] = t - q >= 0 ? desc[(size_t)(t - q) * 256 + d] : 0x80000000u;   // past tile 0: an empty prefix
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            if (done || !ok) break;
            unsigned w = v[q];
            int spins = 0;
            while ((w & kFlagMask) == 0) {
                if (++spins > kSpinLimit) { ok = false; break; }
                __nanosleep(20);
                w = desc[(size_t)(t - q) * 256 + d];
            }
            if (!ok) break;
            excl += w & kValueMask;
            if ((w & kFlagMask) == kFlagPrefix) done = true;
        }
    }
    if (!ok) { raise_status(hdr, DST_ERR_TIMEOUT); excl = 0; }
    desc[(size_t)tile * 256 + d] = kFlagPrefix | ((excl + cnt) & kValueMask);
    return excl;
}

__global__ void __launch_bounds__(kSortThreads)
k_radix_pass(WsHeader* __restrict__ hdr, const unsigned* __restrict__ in_keys, const unsigned* __restrict__ in_pos,
             unsigned* __restrict__ out_keys, unsigned* __restrict__ out_pos,
             const unsigned* __restrict__ digit_hist, unsigned* desc, int pass, int capacity) {
    constexpr int kWarps = kSortThreads / 32;
    __shared__ unsigned wh[kWarps][256];
    __shared__ unsigned bin_base[256];
    __shared__ unsigned wsum[kWarps];
    __shared__ unsigned s_tile;
    pdl_trigger();
    pdl_wait();
    if (threadIdx.x == 0) s_tile = atomicAdd(&hdr->ticket[pass], 1u);   // tiles start in id order
    // asked for now, needed later: these two trips to memory overlap the ticket's
    const unsigned n_bad = pass == 0 ? 0u : (unsigned)hdr->n_bad;
    const unsigned g = digit_hist[threadIdx.x];   // kSortThreads == 256 digits
    for (int s = threadIdx.x; s < kWarps * 256; s += kSortThreads) (&wh[0][0])[s] = 0;
    __syncthreads();
    const int tile = (int)s_tile;
    // pass 0 reads every input position (invalid rows carry kInvalidKey and drop out);
    // later passes read the survivors
    const int n_in = capacity - (int)n_bad;
    const long long t0 = (long long)tile * kTile;
    if (t0 >= n_in) return;

    const int lane = lane_id(), warp = warp_id();
    const int shift = 8 * pass;
    const unsigned lt_mask = (1u << lane) - 1u;
    unsigned key[kSortItems], pos[kSortItems], rank[kSortItems];
#pragma unroll
    for (int k = 0; k < kSortItems; ++k) {
        long long e = t0 + warp * (32 * kSortItems) + k * 32 + lane;
        key[k] = kInvalidKey; pos[k] = 0;
        if (e < n_in) {
            key[k] = in_keys[e];
            pos[k] = in_pos ? in_pos[e] : (unsigned)e;
        }
    }
    // stable rank inside the warp's consecutive keys
#pragma unroll
    for (int k = 0; k < kSortItems; ++k) {
        const bool valid = key[k] != kInvalidKey;
        unsigned dg = (key[k] >> shift) & 255u;
        unsigned m = match_digit(dg, valid);
        int leader = valid ? __ffs(m) - 1 : lane;
        unsigned pre = 0;
        if (valid && lane == leader) { pre = wh[warp][dg]; wh[warp][dg] = pre + __popc(m); }
        pre = __shfl_sync(0xFFFFFFFFu, pre, leader);
        rank[k] = pre + __popc(m & lt_mask);
        __syncwarp();
    }
    __syncthreads();
    // per digit: exclusive prefix over the warps of this tile, tile total
    const int d = threadIdx.x;   // kSortThreads == 256 digits
    unsigned cnt = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) { unsigned t = wh[w][d]; wh[w][d] = cnt; cnt += t; }
    // where digit d starts globally: exclusive scan of this pass's digit histogram
    unsigned ginc = g;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { unsigned t = __shfl_up_sync(0xFFFFFFFFu, ginc, o); if (lane >= o) ginc += t; }
    if (lane == 31) wsum[warp] = ginc;
    __syncthreads();
    unsigned gbase = ginc - g;
    for (int w = 0; w < warp; ++w) gbase += wsum[w];
    unsigned excl = lookback_exclusive(desc, tile, d, cnt, hdr);
    bin_base[d] = gbase + excl;
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kSortItems; ++k) {
        if (key[k] != kInvalidKey) {
            unsigned dg = (key[k] >> shift) & 255u;
            unsigned q = bin_base[dg] + wh[warp][dg] + rank[k];
            if (q < (unsigned)capacity) {
                out_keys[q] = key[k];
                out_pos[q] = pos[k];
            } else {
                raise_status(hdr, DST_ERR_TIMEOUT);   // only reachable after a failed look-back
            }
        }
    }
}

// ---------------------------------------------------------------------------
// a2: run lengths of the sorted keys.  The first entry of a run subtracts its position from
// count[key], the last one adds its position + 1: two atomics per distinct row, never contended.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
k_bounds(const WsHeader* __restrict__ hdr, const unsigned* __restrict__ keys, unsigned* __restrict__ count,
         int capacity, int vocab) {
    pdl_trigger();
    pdl_wait();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= capacity) return;
    // the three keys and the number of valid entries are asked for together: one trip to memory.
    // (Entries past the valid ones hold whatever the buffer held; they are read, never used.)
    const unsigned k = keys[i];
    const unsigned before = i > 0 ? keys[i - 1] : 0u;
    const unsigned after = i + 1 < capacity ? keys[i + 1] : 0u;
    const int n = capacity - (int)hdr->n_bad;
    if (i >= n) return;
    if (k >= (unsigned)vocab) return;                    // only after a failed look-back
    const unsigned prev = i > 0 ? before : ~k;
    const unsigned next = i + 1 < n ? after : ~k;
    if (prev != k) atomicSub(&count[k], (unsigned)i);
    if (next != k) atomicAdd(&count[k], (unsigned)i + 1u);
}

// ---------------------------------------------------------------------------
// a3 + a5 + a6: exclusive scan of count[], unique compaction, heavy-row chunking, row batches.
// One CTA per tile of kScanTile rows.  A tile publishes the sums over its own rows, then adds up
// what the tiles before it have published (a window of kScanThreads predecessors at a time, cut
// short at the nearest one that already knows its inclusive prefix).
// ---------------------------------------------------------------------------
struct Scan6 { int v[6]; };   // 0 offset, 1 unique, 2 heavy rows, 3 chunks, 4 upper nodes, 5 units of the light work items

struct ScanArgs {
    WsHeader* hdr;
    const unsigned* count;
    int* offsets;
    HeavyInfo* heavy;
    void* unique_rows;
    int* counts_out;
    dst_result_t* result;
    int2* batches;
    int* scan_desc;        // per tile: [0] flag (1 own sums, 2 inclusive prefix too), [2..7] own sums, [8..13] inclusive prefix
    int vocab, vocab_pad, chunk, batch_units, n_tiles;
};



// exclusive scan over the CTA (kScanThreads threads) of six counters at once
__device__ __forceinline__ Scan6 block_exclusive_scan(Scan6 x, Scan6& total, int (*sm)[6]) {
    constexpr int kWarps = kScanThreads / 32;
    const int lane = lane_id(), warp = warp_id();
    Scan6 inc = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
        for (int q = 0; q < 6; ++q) {
            int t = __shfl_up_sync(0xFFFFFFFFu, inc.v[q], o);
            if (lane >= o) inc.v[q] += t;
        }
    }
    if (lane == 31) {
#pragma unroll
        for (int q = 0; q < 6; ++q) sm[warp][q] = inc.v[q];
    }
    __syncthreads();
    Scan6 ex;
#pragma unroll
    for (int q = 0; q < 6; ++q) {
        int before = 0, all = 0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) { int t = sm[w][q]; if (w < warp) before += t; all += t; }
        ex.v[q] = inc.v[q] - x.v[q] + before;
        total.v[q] = all;
    }
    __syncthreads();
    return ex;
}

template <typename IT>
__global__ void __launch_bounds__(kScanThreads)
k_scan(const ScanArgs s) {
    __shared__ int sm[kScanThreads / 32][6];
    __shared__ int s_prefix[6];
    __shared__ int s_nearest;
    __shared__ int s_tile;
    __shared__ int s_fail;
    WsHeader* hdr = s.hdr;
    pdl_trigger();
    pdl_wait();
    const int chunk = s.chunk, B = s.batch_units, vocab = s.vocab;
    IT* unique_rows = static_cast<IT*>(s.unique_rows);
    if (threadIdx.x == 0) {
        s_tile = (int)atomicAdd(&hdr->scan_ticket, 1u);   // tiles start in id order
        // after a failed look-back count[] is not to be trusted: leave every table empty
        if (*reinterpret_cast<volatile int*>(&hdr->status) == DST_ERR_TIMEOUT) s_tile = -1;
        s_fail = 0; s_nearest = 0x7FFFFFFF;
    }
    if (threadIdx.x < 6) s_prefix[threadIdx.x] = 0;
    __syncthreads();
    const int tile = s_tile;
    if (tile < 0) return;
    volatile int* desc = s.scan_desc;
    const int e0 = tile * kScanTile + threadIdx.x * kScanItems;

    int c[kScanItems];
    if (e0 < s.vocab_pad) {
        const uint4* src = reinterpret_cast<const uint4*>(s.count + e0);
#pragma unroll
        for (int q = 0; q < kScanItems / 4; ++q) {
            uint4 t = __ldcg(src + q);
            c[4 * q] = (int)t.x; c[4 * q + 1] = (int)t.y; c[4 * q + 2] = (int)t.z; c[4 * q + 3] = (int)t.w;
        }
    } else {
#pragma unroll
        for (int q = 0; q < kScanItems; ++q) c[q] = 0;
    }
    int prev_cost = 0;                   // units of the row before this thread's first one
    if (e0 > 0 && e0 < s.vocab_pad) prev_cost = row_units((int)__ldcg(s.count + e0 - 1), chunk);
    Scan6 mine{};
    int maxseg = 0;
#pragma unroll
    for (int q = 0; q < kScanItems; ++q) {
        const int cc = c[q];
        mine.v[0] += cc;
        mine.v[1] += cc > 0;
        if (e0 + q < vocab) mine.v[5] += row_units(cc, chunk);
        if (cc > chunk) {
            const int n = (cc + chunk - 1) / chunk;
            mine.v[2] += 1; mine.v[3] += n; mine.v[4] += upper_nodes(n);
        }
        maxseg = max(maxseg, cc);
    }
    Scan6 total;
    Scan6 run = block_exclusive_scan(mine, total, sm);
    // publish this tile's own sums
    if (threadIdx.x == 0) {
#pragma unroll
        for (int q = 0; q < 6; ++q) desc[tile * 16 + 2 + q] = total.v[q];
        __threadfence();
        desc[tile * 16] = 1;
    }
    // add up the tiles before this one
    for (int w0 = 0; w0 < tile; w0 += kScanThreads) {
        const int dist = w0 + threadIdx.x;        // 0 = the tile right before this one
        const int p = tile - 1 - dist;
        int flag = 0;
        if (p >= 0) {
            int spins = 0;
            while ((flag = desc[p * 16]) == 0) {
                if (++spins > kSpinLimit) { s_fail = 1; break; }
                __nanosleep(20);
            }
            if (flag == 2) atomicMin(&s_nearest, dist);
        }
        __syncthreads();
        const int nearest = s_nearest;            // nearest predecessor that knows its inclusive prefix
        if (p >= 0 && flag != 0 && dist <= nearest) {
            __threadfence();
            const int off = p * 16 + (dist == nearest ? 8 : 2);
#pragma unroll
            for (int q = 0; q < 6; ++q) {
                const int t = desc[off + q];
                if (t) atomicAdd(&s_prefix[q], t);
            }
        }
        __syncthreads();
        if (nearest != 0x7FFFFFFF || s_fail) break;
    }
    __syncthreads();
    if (s_fail) {
        if (threadIdx.x == 0) raise_status(hdr, DST_ERR_TIMEOUT);
        return;
    }
    Scan6 prefix;
#pragma unroll
    for (int q = 0; q < 6; ++q) { prefix.v[q] = s_prefix[q]; run.v[q] += prefix.v[q]; }
    if (threadIdx.x == 0) {
#pragma unroll
        for (int q = 0; q < 6; ++q) desc[tile * 16 + 8 + q] = prefix.v[q] + total.v[q];
        __threadfence();
        desc[tile * 16] = 2;
    }

    if (e0 < s.vocab_pad) {
        int o[kScanItems];
        int rem = run.v[5] % B;          // units before row e0, modulo the batch size
        int b = run.v[5] / B;
#pragma unroll
        for (int q = 0; q < kScanItems; ++q) {
            const int cc = c[q];
            const int v = e0 + q;
            o[q] = run.v[0];
            if (cc > 0) {
                if (unique_rows) unique_rows[run.v[1]] = (IT)v;
                if (s.counts_out) s.counts_out[run.v[1]] = cc;
                run.v[1] += 1;
            }
            if (cc > chunk) {
                // a6: a heavy row becomes n chunk items and a combine tree
                const int n = (cc + chunk - 1) / chunk;
                s.heavy[run.v[2]] = HeavyInfo{v, run.v[3], run.v[4], n, run.v[0], cc, {0, 0}};
                run.v[2] += 1; run.v[3] += n; run.v[4] += upper_nodes(n);
            }
            run.v[0] += cc;
            if (v < vocab) {
                // light work items: row v belongs to batch floor(units before v / batch size)
                const int cost = row_units(cc, chunk);
                if (v == 0 || prev_cost > rem) s.batches[b].x = v + 1;      // the row before started in an earlier batch
                rem += cost;
                if (v == vocab - 1 || rem >= B) s.batches[b].y = v + 1;     // the next row starts in a later batch
                if (rem >= B) { b += rem / B; rem %= B; }
                prev_cost = cost;
            }
        }
        int4* dst = reinterpret_cast<int4*>(s.offsets + e0);
#pragma unroll
        for (int q = 0; q < kScanItems / 4; ++q) dst[q] = make_int4(o[4 * q], o[4 * q + 1], o[4 * q + 2], o[4 * q + 3]);
    }
    for (int o = 16; o > 0; o >>= 1) maxseg = max(maxseg, __shfl_down_sync(0xFFFFFFFFu, maxseg, o));
    if (lane_id() == 0 && maxseg > 0) atomicMax(&hdr->max_segment, maxseg);
    __syncthreads();
    if (threadIdx.x == 0) {
        if (tile == s.n_tiles - 1) {     // prefix + own sums = totals
            s.offsets[s.vocab_pad] = prefix.v[0] + total.v[0];
            hdr->n_valid = prefix.v[0] + total.v[0];
            hdr->n_unique = prefix.v[1] + total.v[1];
            hdr->n_heavy = prefix.v[2] + total.v[2];
            hdr->n_chunks = prefix.v[3] + total.v[3];
            hdr->n_upper = prefix.v[4] + total.v[4];
            const int units = prefix.v[5] + total.v[5];
            hdr->n_batches = units > 0 ? (units - 1) / B + 1 : 0;
        }
        __threadfence();
        if (atomicAdd(&hdr->scan_done, 1u) == (unsigned)s.n_tiles - 1u) {
            // every tile has finished: the header is complete
            __threadfence();
            const unsigned long long bad = *reinterpret_cast<volatile unsigned long long*>(&hdr->n_bad);
            if (bad) raise_status(hdr, DST_ERR_INDEX_OUT_OF_RANGE);
            if (s.result) {
                s.result->n_unique = *reinterpret_cast<volatile int*>(&hdr->n_unique);
                s.result->n_out_of_range = (long long)bad;
                s.result->max_segment = *reinterpret_cast<volatile int*>(&hdr->max_segment);
            }
        }
    }
}

// ---- host-side launchers ------------------------------------------------------
cudaError_t launch_prep(const HistParams& P, int grid_x, int index_type, WsHeader* hdr, unsigned* digit_hist,
                        unsigned* keys, SliceEntry* tab, long long vocab, int passes, cudaStream_t stream) {
    dim3 grid(grid_x, P.n);
    if (index_type == DST_I64)
        return launch_pdl(k_prep<long long>, grid, dim3(kSortThreads), 0, stream, P, hdr, digit_hist, keys, tab, vocab, passes);
    else
        return launch_pdl(k_prep<int>, grid, dim3(kSortThreads), 0, stream, P, hdr, digit_hist, keys, tab, vocab, passes);
}

cudaError_t launch_radix_pass(int n_tiles, WsHeader* hdr, const unsigned* in_keys, const unsigned* in_pos,
                              unsigned* out_keys, unsigned* out_pos, const unsigned* digit_hist, unsigned* desc,
                              int pass, int capacity, cudaStream_t stream) {
    return launch_pdl(k_radix_pass, dim3(n_tiles), dim3(kSortThreads), 0, stream, hdr, in_keys, in_pos, out_keys, out_pos,
                      digit_hist, desc, pass, capacity);
}

cudaError_t launch_bounds(const WsHeader* hdr, const unsigned* keys, unsigned* count, int capacity, int vocab,
                          cudaStream_t stream) {
    return launch_pdl(k_bounds, dim3((capacity + 255) / 256), dim3(256), 0, stream, hdr, keys, count, capacity, vocab);
}

cudaError_t launch_scan(int index_type, const ScanParams& p, cudaStream_t stream) {
    const int n_tiles = (p.vocab_pad + kScanTile - 1) / kScanTile;
    ScanArgs s{p.hdr, p.count, p.offsets, p.heavy, p.unique_rows, p.counts_out, p.result, p.batches,
               p.scan_desc, p.vocab, p.vocab_pad, p.chunk, p.batch_units, n_tiles};
    if (index_type == DST_I64) return launch_pdl(k_scan<long long>, dim3(n_tiles), dim3(kScanThreads), 0, stream, s);
    return launch_pdl(k_scan<int>, dim3(n_tiles), dim3(kScanThreads), 0, stream, s);
}

}  // namespace dst
