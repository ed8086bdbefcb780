// Index side of densify: validate, stable radix placement, segment bounds, scan to CSR offsets.
//
// Together these turn the row indices of the (virtually concatenated) IndexedSlices
// of the paper's Section 3 into
//   offsets[v] .. offsets[v+1]   the positions in perm[] that belong to output row v
//   perm[j]                      input row positions, ascending inside each segment
// plus the work-item tables the row-reduction kernel consumes.  Integer work only.
//
// Order of the kernels (large inputs):
//   k_prep        validate, narrow to 32-bit keys, digit histograms of all radix passes; for vocabularies of
//                 at most 65536 rows also count[v], in shared memory
//   k_radix_pass  one per 8-bit digit, least significant first, stable; when count[] is known already, the scan
//                 tiles ride in the launch of the first pass and nothing else follows the last one
//   k_bounds      (larger vocabularies) run lengths of the sorted keys -> count[v]
//   k_scan        (larger vocabularies) count[] -> offsets, unique rows, heavy-row chunks, row batches
// Small inputs take k_front_cluster (dst_front_cluster.cu), which does all of it in one kernel.
#include "dst_common.cuh"

namespace dst {

// ---------------------------------------------------------------------------
// a1: validate, narrow to 32-bit keys, per-pass digit histograms; a2 when the vocabulary is small
// enough for one 16-bit counter per row in a CTA's shared memory: the CTA counts its own entries
// there (a CTA sees at most kPrepTile < 65536 of them) and adds the rows it has met to count[].
// The counts are then known before the sort, not after it, and the scan that turns them into the
// row tables can run beside the radix passes.
// ---------------------------------------------------------------------------
template <typename IT, bool COUNT>
__global__ void __launch_bounds__(kPrepThreads)
k_prep(const __grid_constant__ HistParams P, WsHeader* __restrict__ hdr, unsigned* __restrict__ digit_hist,
       unsigned* __restrict__ keys, SliceEntry* __restrict__ tab, long long vocab, int passes,
       unsigned* __restrict__ count, int count_words) {
    __shared__ unsigned dh[kMaxPasses * 256];
    extern __shared__ __align__(16) unsigned rows16[];   // COUNT: two 16-bit counters per word, count_words words (a multiple of 4)
    const SliceEntry& se = P.s[blockIdx.y];
    const long long n = se.n_rows;
    const long long t0 = (long long)blockIdx.x * kPrepTile;
    // shared memory is this CTA's own: cleared before the wait on the kernels before this one
    if (t0 < n) {
        for (int s = threadIdx.x; s < kMaxPasses * 256; s += kPrepThreads) dh[s] = 0;
        if (COUNT)
            for (int s = threadIdx.x * 4; s < count_words; s += kPrepThreads * 4)
                *reinterpret_cast<uint4*>(rows16 + s) = make_uint4(0u, 0u, 0u, 0u);
    }
    pdl_trigger();
    pdl_wait();
    if (blockIdx.x == 0 && threadIdx.x == 0) tab[P.first + blockIdx.y] = se;
    if (t0 >= n) return;
    __syncthreads();

    const IT* __restrict__ idx = static_cast<const IT*>(se.indices);
    const int lane = lane_id();
    unsigned bad = 0;
    long long vals[kPrepItems];          // every index of this thread first: one trip to memory, not kPrepItems
#pragma unroll
    for (int k = 0; k < kPrepItems; ++k) {
        const long long i = t0 + k * kPrepThreads + threadIdx.x;
        vals[k] = -1;
        if (i < n) vals[k] = (long long)idx[i];
    }
#pragma unroll
    for (int k = 0; k < kPrepItems; ++k) {
        const long long i = t0 + k * kPrepThreads + threadIdx.x;
        const bool in = i < n;
        const long long v = vals[k];
        const bool ok = in && v >= 0 && v < vocab;
        const unsigned key = ok ? (unsigned)v : kInvalidKey;
        if (in) keys[se.start + i] = key;
        bad += in && !ok;
        // a warp whose 32 indices are all the same row (one very frequent row) adds once
        const unsigned k0 = __shfl_sync(0xFFFFFFFFu, key, 0);
        const bool same = __all_sync(0xFFFFFFFFu, ok && key == k0);
        if (same) {
            if (lane == 0) {
                for (int p = 0; p < passes; ++p) atomicAdd(&dh[p * 256 + ((key >> (8 * p)) & 255u)], 32u);
                if (COUNT) atomicAdd(&rows16[key >> 1], 32u << (16 * (key & 1u)));
            }
        } else if (ok) {
            for (int p = 0; p < passes; ++p) atomicAdd(&dh[p * 256 + ((key >> (8 * p)) & 255u)], 1u);
            if (COUNT) atomicAdd(&rows16[key >> 1], 1u << (16 * (key & 1u)));
        }
    }
    __syncthreads();
    for (int s = threadIdx.x; s < passes * 256; s += kPrepThreads) {
        unsigned c = dh[s];
        if (c) atomicAdd(&digit_hist[s], c);
    }
    if (COUNT) {
        // Two neighbouring rows per 64-bit add (a row's count stays below 2^32, so nothing carries over), and
        // neighbouring lanes on neighbouring words: the adds of one instruction fall into few 32-byte sectors.
        unsigned long long* count2 = reinterpret_cast<unsigned long long*>(count);
        for (int s = threadIdx.x; s < count_words; s += kPrepThreads) {
            const unsigned w = rows16[s];
            if (w) atomicAdd(&count2[s], (unsigned long long)(w & 0xFFFFu) | ((unsigned long long)(w >> 16) << 32));
        }
    }
    for (int o = 16; o > 0; o >>= 1) bad += __shfl_down_sync(0xFFFFFFFFu, bad, o);
    if (lane == 0 && bad) atomicAdd(&hdr->n_bad, (unsigned long long)bad);
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
    int wide;              // unique_rows holds 64-bit integers
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

// One scan tile.  Called by every thread of a CTA of kScanThreads threads, after the wait on the kernels before.
__device__ __forceinline__ void scan_tile(const ScanArgs& s) {
    __shared__ int sm[kScanThreads / 32][6];
    __shared__ int s_prefix[6];
    __shared__ int s_nearest;
    __shared__ int s_tile;
    __shared__ int s_fail;
    WsHeader* hdr = s.hdr;
    const int chunk = s.chunk, B = s.batch_units, vocab = s.vocab;
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
                if (s.unique_rows) {
                    if (s.wide) static_cast<long long*>(s.unique_rows)[run.v[1]] = v;
                    else static_cast<int*>(s.unique_rows)[run.v[1]] = v;
                }
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

__global__ void __launch_bounds__(kScanThreads)
k_scan(const ScanArgs s) {
    pdl_trigger();
    pdl_wait();
    scan_tile(s);
}

// ---------------------------------------------------------------------------
// a4: one stable 8-bit radix pass (least significant digit first), single sweep
// over the keys with a decoupled look-back for the cross-tile prefix
// ---------------------------------------------------------------------------
// Exclusive prefix of digit d's count over the tiles before `tile`.  Every tile publishes its own
// count first ("aggregate"), then walks back over its predecessors, four at a time, until it meets
// one that has published its inclusive prefix.  Tiles start in ticket order, so every predecessor
// is running or done; the wait on a missing descriptor is bounded all the same.
__device__ __forceinline__ void lookback_publish(volatile unsigned* desc, int tile, int d, unsigned cnt) {
    desc[(size_t)tile * 256 + d] = (tile == 0 ? kFlagPrefix : kFlagAggregate) | cnt;
}

constexpr int kLookback = 4;                // predecessors asked for per trip to memory (16 and 32: 0.5 % and 1 % slower on the 64-slice case)

__device__ __forceinline__ unsigned lookback_walk(volatile unsigned* desc, int tile, int d, unsigned cnt, WsHeader* hdr) {
    if (tile == 0) return 0;
    unsigned excl = 0;
    bool ok = true, done = false;
    for (int t = tile - 1; t >= 0 && ok && !done; t -= kLookback) {
        unsigned v[kLookback];
#pragma unroll
        for (int q = 0; q < kLookback; ++q) v[q] = t - q >= 0 ? desc[(size_t)(t - q) * 256 + d] : 0x80000000u;   // past tile 0: an empty prefix
#pragma unroll
        for (int q = 0; q < kLookback; ++q) {
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

// One pass: rank the tile's keys by digit (stable), publish the tile's digit counts, lay the tile out in
// shared memory in its sorted order while the predecessors publish theirs, fetch the cross-tile prefix,
// then write the tile out.  Entries of one digit are consecutive in shared memory and go to consecutive
// places in global memory, so the stores of a warp fall into a few runs instead of 32 separate sectors
// (written straight from the registers, the scatter alone took a quarter of the pass).
//
// ITEMS keys per thread, kRadixThreads * ITEMS per tile: the host picks the smallest tile with which every CTA of
// the launch has an SM of its own (two CTAs on one SM rank their keys at half the speed, and every tile after
// them in the order waits for their counts).  With all CTAs resident from the start the tile number is the CTA
// number; otherwise tiles take a ticket, so that a tile's predecessors are running or done when it starts.
template <int ITEMS>
__global__ void __launch_bounds__(kRadixThreads, ITEMS <= 8 ? 2 : 1)
k_radix_pass(WsHeader* __restrict__ hdr, const unsigned* __restrict__ in_keys, const unsigned* __restrict__ in_pos,
             unsigned* __restrict__ out_keys, unsigned* __restrict__ out_pos,
             const unsigned* __restrict__ digit_hist, unsigned* desc, int pass, int capacity,
             const __grid_constant__ ScanArgs scan, int scan_tiles, int ticketed) {
    constexpr int kWarps = kRadixThreads / 32;
    constexpr int kTileKeys = kRadixThreads * ITEMS;
    __shared__ unsigned short wh[kWarps][256];   // counts of one tile: at most 8192, which fits 16 bits
    extern __shared__ __align__(16) unsigned staged[];
    unsigned* skey = staged;
    unsigned* spos = staged + kTileKeys;
    __shared__ unsigned tile_off[256];      // where digit d starts inside the sorted tile
    __shared__ unsigned delta[256];         // global place of entry j of digit d = delta[d] + j
    __shared__ unsigned wsum[8], wsum2[8];
    __shared__ unsigned s_tile;
    pdl_trigger();
    pdl_wait();
    // The first CTAs of the launch are scan tiles when the row counts are known already: they need nothing
    // from the sort, and the row-reduction kernel needs their tables only after the last pass.
    if ((int)blockIdx.x < scan_tiles) { scan_tile(scan); return; }
    if (threadIdx.x == 0) s_tile = ticketed ? atomicAdd(&hdr->ticket[pass], 1u) : blockIdx.x - (unsigned)scan_tiles;
    // asked for now, needed later: these two trips to memory overlap the ticket's
    const unsigned n_bad = pass == 0 ? 0u : (unsigned)hdr->n_bad;
    const bool digit_thread = threadIdx.x < 256;   // thread d < 256 looks after digit d
    const unsigned g = digit_thread ? digit_hist[threadIdx.x] : 0u;
    for (int s = threadIdx.x; s < kWarps * 128; s += kRadixThreads) reinterpret_cast<unsigned*>(&wh[0][0])[s] = 0;
    __syncthreads();
    const int tile = (int)s_tile;
    // pass 0 reads every input position (invalid rows carry kInvalidKey and drop out);
    // later passes read the survivors
    const int n_in = capacity - (int)n_bad;
    const long long t0 = (long long)tile * kTileKeys;
    if (t0 >= n_in) return;

    const int lane = lane_id(), warp = warp_id();
    const int shift = 8 * pass;
    const unsigned lt_mask = (1u << lane) - 1u;
    unsigned key[ITEMS], pos[ITEMS], rank[ITEMS];
#pragma unroll
    for (int k = 0; k < ITEMS; ++k) {
        long long e = t0 + warp * (32 * ITEMS) + k * 32 + lane;
        key[k] = kInvalidKey; pos[k] = 0;
        if (e < n_in) {
            key[k] = in_keys[e];
            pos[k] = in_pos ? in_pos[e] : (unsigned)e;
        }
    }
    // stable rank inside the warp's consecutive keys
#pragma unroll
    for (int k = 0; k < ITEMS; ++k) {
        const bool valid = key[k] != kInvalidKey;
        unsigned dg = (key[k] >> shift) & 255u;
        unsigned m = match_digit(dg, valid);
        int leader = valid ? __ffs(m) - 1 : lane;
        unsigned pre = 0;
        if (valid && lane == leader) { pre = wh[warp][dg]; wh[warp][dg] = (unsigned short)(pre + __popc(m)); }
        pre = __shfl_sync(0xFFFFFFFFu, pre, leader);
        rank[k] = pre + __popc(m & lt_mask);
        __syncwarp();
    }
    __syncthreads();
    // per digit: exclusive prefix over the warps of this tile, tile total
    const int d = threadIdx.x & 255;
    unsigned cnt = 0;
    if (digit_thread) {
#pragma unroll
        for (int w = 0; w < kWarps; ++w) { unsigned t = wh[w][d]; wh[w][d] = (unsigned short)cnt; cnt += t; }
        lookback_publish(desc, tile, d, cnt);
    }
    // where digit d starts globally (exclusive scan of this pass's digit histogram) and inside the tile
    unsigned ginc = g, tinc = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        unsigned t = __shfl_up_sync(0xFFFFFFFFu, ginc, o), u = __shfl_up_sync(0xFFFFFFFFu, tinc, o);
        if (lane >= o) { ginc += t; tinc += u; }
    }
    if (lane == 31 && digit_thread) { wsum[warp] = ginc; wsum2[warp] = tinc; }
    __syncthreads();
    unsigned gbase = ginc - g, tbase = tinc - cnt, n_tile = 0;
    for (int w = 0; w < 8; ++w) {
        if (w < warp) { gbase += wsum[w]; tbase += wsum2[w]; }
        n_tile += wsum2[w];
    }
    if (digit_thread) tile_off[d] = tbase;
    __syncthreads();
#pragma unroll
    for (int k = 0; k < ITEMS; ++k) {
        if (key[k] != kInvalidKey) {
            const unsigned dg = (key[k] >> shift) & 255u;
            const unsigned li = tile_off[dg] + wh[warp][dg] + rank[k];
            skey[li] = key[k];
            spos[li] = pos[k];
        }
    }
    if (digit_thread) {
        const unsigned excl = lookback_walk(desc, tile, d, cnt, hdr);
        delta[d] = gbase + excl - tbase;
    }
    __syncthreads();
    for (unsigned j = threadIdx.x; j < n_tile; j += kRadixThreads) {
        const unsigned kk = skey[j];
        const unsigned q = delta[(kk >> shift) & 255u] + j;
        if (q < (unsigned)capacity) {
            if (out_keys) out_keys[q] = kk;
            out_pos[q] = spos[j];
        } else {
            raise_status(hdr, DST_ERR_TIMEOUT);   // only reachable after a failed look-back
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

// ---- host-side launchers ------------------------------------------------------
cudaError_t launch_prep(const HistParams& P, int grid_x, int index_type, WsHeader* hdr, unsigned* digit_hist,
                        unsigned* keys, SliceEntry* tab, long long vocab, int passes, unsigned* count, cudaStream_t stream) {
    dim3 grid(grid_x, P.n);
    const bool wide = index_type == DST_I64;
    if (!count) {
        if (wide)
            return launch_pdl(k_prep<long long, false>, grid, dim3(kPrepThreads), 0, stream, P, hdr, digit_hist, keys, tab,
                              vocab, passes, count, 0);
        return launch_pdl(k_prep<int, false>, grid, dim3(kPrepThreads), 0, stream, P, hdr, digit_hist, keys, tab, vocab,
                          passes, count, 0);
    }
    const int words = int(((vocab + 1) / 2 + 3) / 4 * 4);
    const size_t smem = size_t(words) * 4;
    static SmemOptIn optin_wide, optin_narrow;
    cudaError_t e = wide ? ensure_dynamic_smem(k_prep<long long, true>, smem, optin_wide)
                         : ensure_dynamic_smem(k_prep<int, true>, smem, optin_narrow);
    if (e != cudaSuccess) return e;
    if (wide)
        return launch_pdl(k_prep<long long, true>, grid, dim3(kPrepThreads), smem, stream, P, hdr, digit_hist, keys, tab,
                          vocab, passes, count, words);
    return launch_pdl(k_prep<int, true>, grid, dim3(kPrepThreads), smem, stream, P, hdr, digit_hist, keys, tab, vocab,
                      passes, count, words);
}

int scan_tile_count(int vocab_pad) { return (vocab_pad + kScanTile - 1) / kScanTile; }

static ScanArgs scan_args(const ScanParams& p) {
    const int n_tiles = scan_tile_count(p.vocab_pad);
    return ScanArgs{p.hdr, p.count, p.offsets, p.heavy, p.unique_rows, p.counts_out, p.result, p.batches,
                    p.scan_desc, p.vocab, p.vocab_pad, p.chunk, p.batch_units, n_tiles, p.wide};
}

// Items per thread of a radix pass over n keys, given the CTAs that ride along and the SMs of the device.
int radix_items(long long n, int extra_ctas, int sms) {
    const int choices[4] = {8, 10, 12, 16};
    for (int c = 0; c < 4; ++c) {
        const long long tile = (long long)kRadixThreads * choices[c];
        if ((n + tile - 1) / tile + extra_ctas <= sms) return choices[c];
    }
    return n > 4LL * sms * kRadixThreads * 8 ? 16 : 8;
}

template <int ITEMS>
static cudaError_t launch_radix_as(int n_tiles, cudaStream_t stream, int sms, WsHeader* hdr, const unsigned* in_keys,
                                   const unsigned* in_pos, unsigned* out_keys, unsigned* out_pos,
                                   const unsigned* digit_hist, unsigned* desc, int pass, int capacity,
                                   const ScanArgs& sa, int scan_tiles) {
    static SmemOptIn optin;
    const size_t smem = size_t(kRadixThreads) * ITEMS * 8;
    cudaError_t e = ensure_dynamic_smem(k_radix_pass<ITEMS>, smem, optin);
    if (e != cudaSuccess) return e;
    const int ticketed = n_tiles + scan_tiles > sms ? 1 : 0;
    return launch_pdl(k_radix_pass<ITEMS>, dim3(n_tiles + scan_tiles), dim3(kRadixThreads), smem, stream, hdr, in_keys,
                      in_pos, out_keys, out_pos, digit_hist, desc, pass, capacity, sa, scan_tiles, ticketed);
}

cudaError_t launch_radix_pass(int items, int sms, WsHeader* hdr, const unsigned* in_keys, const unsigned* in_pos,
                              unsigned* out_keys, unsigned* out_pos, const unsigned* digit_hist, unsigned* desc,
                              int pass, int capacity, const ScanParams* scan, cudaStream_t stream) {
    ScanArgs sa{};
    int scan_tiles = 0;
    if (scan) { sa = scan_args(*scan); scan_tiles = sa.n_tiles; }
    const int tile = kRadixThreads * items;
    const int n_tiles = (capacity + tile - 1) / tile;
#define DST_RADIX_CASE(I) case I: return launch_radix_as<I>(n_tiles, stream, sms, hdr, in_keys, in_pos, out_keys, out_pos, \
                                                            digit_hist, desc, pass, capacity, sa, scan_tiles)
    switch (items) {
        DST_RADIX_CASE(8);
        DST_RADIX_CASE(10);
        DST_RADIX_CASE(12);
        DST_RADIX_CASE(16);
    }
#undef DST_RADIX_CASE
    return cudaErrorInvalidValue;
}

cudaError_t launch_bounds(const WsHeader* hdr, const unsigned* keys, unsigned* count, int capacity, int vocab,
                          cudaStream_t stream) {
    return launch_pdl(k_bounds, dim3((capacity + 255) / 256), dim3(256), 0, stream, hdr, keys, count, capacity, vocab);
}

cudaError_t launch_scan(const ScanParams& p, cudaStream_t stream) {
    const ScanArgs s = scan_args(p);
    return launch_pdl(k_scan, dim3(s.n_tiles), dim3(kScanThreads), 0, stream, s);
}

}  // namespace dst
