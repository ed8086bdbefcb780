// Index side of densify: validate + histogram, scan to CSR offsets, stable radix placement.
//
// Together these turn the row indices of the (virtually concatenated) IndexedSlices
// of the paper's Section 3 into
//   offsets[v] .. offsets[v+1]   the positions in perm[] that belong to output row v
//   perm[j]                      input row positions, ascending inside each segment
// which is what the row-reduction kernel consumes.  Integer work only.
#include "dst_common.cuh"

namespace dst {

// ---------------------------------------------------------------------------
// a1 + a2: validate, narrow to 32-bit keys, per-row histogram, per-pass digit histograms
// ---------------------------------------------------------------------------
template <typename IT>
__global__ void __launch_bounds__(kSortThreads)
k_hist(const __grid_constant__ HistParams P, WsHeader* __restrict__ hdr, unsigned* __restrict__ count,
       unsigned* __restrict__ digit_hist, unsigned* __restrict__ keys, SliceEntry* __restrict__ tab,
       long long vocab, int passes) {
    __shared__ unsigned hkey[kHashSlots];
    __shared__ unsigned hcnt[kHashSlots];
    __shared__ unsigned dh[kMaxPasses * 256];

    const SliceEntry& se = P.s[blockIdx.y];
    if (blockIdx.x == 0 && threadIdx.x == 0) tab[P.first + blockIdx.y] = se;
    const long long n = se.n_rows;
    const long long t0 = (long long)blockIdx.x * kTile;
    if (t0 >= n) return;

    for (int s = threadIdx.x; s < kHashSlots; s += kSortThreads) { hkey[s] = kInvalidKey; hcnt[s] = 0; }
    for (int s = threadIdx.x; s < kMaxPasses * 256; s += kSortThreads) dh[s] = 0;
    __syncthreads();

    const IT* __restrict__ idx = static_cast<const IT*>(se.indices);
    unsigned bad = 0;
#pragma unroll
    for (int k = 0; k < kSortItems; ++k) {
        long long i = t0 + k * kSortThreads + threadIdx.x;
        if (i < n) {
            long long v = (long long)idx[i];
            bool ok = v >= 0 && v < vocab;
            unsigned key = ok ? (unsigned)v : kInvalidKey;
            keys[se.start + i] = key;
            if (ok) {
                // aggregate equal keys inside the CTA before touching global counters
                unsigned slot = (key * 2654435761u) >> 20;   // 12 bits
                for (int probe = 0; probe < kHashSlots; ++probe) {
                    unsigned old = atomicCAS(&hkey[slot], kInvalidKey, key);
                    if (old == kInvalidKey || old == key) { atomicAdd(&hcnt[slot], 1u); break; }
                    slot = (slot + 1) & (kHashSlots - 1);
                }
                for (int p = 0; p < passes; ++p) atomicAdd(&dh[p * 256 + ((key >> (8 * p)) & 255u)], 1u);
            } else {
                ++bad;
            }
        }
    }
    __syncthreads();
    for (int s = threadIdx.x; s < kHashSlots; s += kSortThreads) {
        unsigned k = hkey[s];
        if (k != kInvalidKey) atomicAdd(&count[k], hcnt[s]);
    }
    for (int s = threadIdx.x; s < passes * 256; s += kSortThreads) {
        unsigned c = dh[s];
        if (c) atomicAdd(&digit_hist[s], c);
    }
    for (int o = 16; o > 0; o >>= 1) bad += __shfl_down_sync(0xFFFFFFFFu, bad, o);
    if (lane_id() == 0 && bad) atomicAdd(&hdr->n_bad, (unsigned long long)bad);
}

// ---------------------------------------------------------------------------
// a3 + a5 + a6: exclusive scan of the histogram, unique compaction, heavy-row chunking
// ---------------------------------------------------------------------------
struct Scan5 { int v[6]; };   // 0 offset, 1 unique, 2 heavy rows, 3 chunks, 4 upper nodes, 5 units of the light work items

__device__ __forceinline__ Scan5 block_exclusive_scan(Scan5 x, Scan5& total, int (*sm)[6]) {
    const int lane = lane_id(), warp = warp_id();
    Scan5 inc = x;
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
    if (warp == 0) {
        Scan5 w;
#pragma unroll
        for (int q = 0; q < 6; ++q) w.v[q] = sm[lane][q];
        Scan5 winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
            for (int q = 0; q < 6; ++q) {
                int t = __shfl_up_sync(0xFFFFFFFFu, winc.v[q], o);
                if (lane >= o) winc.v[q] += t;
            }
        }
#pragma unroll
        for (int q = 0; q < 6; ++q) {
            sm[lane][q] = winc.v[q] - w.v[q];          // exclusive prefix of this warp
            if (lane == 31) sm[32][q] = winc.v[q];     // block total
        }
    }
    __syncthreads();
    Scan5 ex;
#pragma unroll
    for (int q = 0; q < 6; ++q) {
        ex.v[q] = inc.v[q] - x.v[q] + sm[warp][q];
        total.v[q] = sm[32][q];
    }
    __syncthreads();
    return ex;
}

template <typename IT>
__global__ void __launch_bounds__(kScanThreads)
k_scan(WsHeader* __restrict__ hdr, const unsigned* __restrict__ count, int* __restrict__ offsets,
       HeavyInfo* __restrict__ heavy, ChunkDesc* __restrict__ chunkdesc, IT* __restrict__ unique_rows,
       int* __restrict__ counts_out, dst_result_t* __restrict__ result, int2* __restrict__ batches, int vocab,
       int vocab_pad, int chunk, int batch_units) {
    __shared__ int sm[33][6];
    __shared__ int smax[32];
    Scan5 carry{};
    int maxseg = 0;
    constexpr int kRound = kScanThreads * kScanItems;
    for (int base = 0; base < vocab_pad; base += kRound) {
        const int e0 = base + threadIdx.x * kScanItems;
        unsigned c[kScanItems];
        if (e0 < vocab_pad) {
            const uint4* src = reinterpret_cast<const uint4*>(count + e0);
#pragma unroll
            for (int q = 0; q < kScanItems / 4; ++q) {
                uint4 t = src[q];
                c[4 * q] = t.x; c[4 * q + 1] = t.y; c[4 * q + 2] = t.z; c[4 * q + 3] = t.w;
            }
        } else {
#pragma unroll
            for (int q = 0; q < kScanItems; ++q) c[q] = 0;
        }
        Scan5 mine{};
#pragma unroll
        for (int q = 0; q < kScanItems; ++q) {
            int cc = (int)c[q];
            mine.v[0] += cc;
            mine.v[1] += cc > 0;
            if (e0 + q < vocab) mine.v[5] += cc > chunk ? 1 : cc + 1;
            if (cc > chunk) {
                int n = (cc + chunk - 1) / chunk;
                mine.v[2] += 1; mine.v[3] += n; mine.v[4] += upper_nodes(n);
            }
            maxseg = max(maxseg, cc);
        }
        Scan5 total;
        Scan5 run = block_exclusive_scan(mine, total, sm);
#pragma unroll
        for (int q = 0; q < 6; ++q) run.v[q] += carry.v[q];
        if (e0 < vocab_pad) {
            // units of the row before this thread's first one (decides whether that row opens a batch)
            int prev_cost = 0;
            if (e0 > 0) { int pc = (int)count[e0 - 1]; prev_cost = pc > chunk ? 1 : pc + 1; }
            int o[kScanItems];
#pragma unroll
            for (int q = 0; q < kScanItems; ++q) {
                int cc = (int)c[q];
                o[q] = run.v[0];
                if (cc > 0) {
                    if (unique_rows) unique_rows[run.v[1]] = (IT)(e0 + q);
                    if (counts_out) counts_out[run.v[1]] = cc;
                    run.v[1] += 1;
                }
                if (cc > chunk) {
                    int n = (cc + chunk - 1) / chunk;
                    heavy[run.v[2]] = HeavyInfo{e0 + q, run.v[3], run.v[4], n};
                    run.v[2] += 1; run.v[3] += n; run.v[4] += upper_nodes(n);
                }
                run.v[0] += cc;
                if (e0 + q < vocab) {
                    // light work items: row v belongs to batch floor(units before v / batch_units)
                    const int cost = cc > chunk ? 1 : cc + 1;
                    const int b = run.v[5] / batch_units;
                    const int v = e0 + q;
                    if (v == 0 || (run.v[5] - prev_cost) / batch_units != b) batches[b].x = v + 1;
                    if (v == vocab - 1 || (run.v[5] + cost) / batch_units != b) batches[b].y = v + 1;
                    run.v[5] += cost;
                    prev_cost = cost;
                }
            }
            int4* dst = reinterpret_cast<int4*>(offsets + e0);
#pragma unroll
            for (int q = 0; q < kScanItems / 4; ++q) dst[q] = make_int4(o[4 * q], o[4 * q + 1], o[4 * q + 2], o[4 * q + 3]);
        }
#pragma unroll
        for (int q = 0; q < 6; ++q) carry.v[q] += total.v[q];
    }
    for (int o = 16; o > 0; o >>= 1) maxseg = max(maxseg, __shfl_down_sync(0xFFFFFFFFu, maxseg, o));
    if (lane_id() == 0) smax[warp_id()] = maxseg;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < kScanThreads / 32; ++w) maxseg = max(maxseg, smax[w]);
        offsets[vocab_pad] = carry.v[0];
        hdr->n_valid = carry.v[0];
        hdr->n_unique = carry.v[1];
        hdr->n_heavy = carry.v[2];
        hdr->n_chunks = carry.v[3];
        hdr->n_upper = carry.v[4];
        hdr->max_segment = maxseg;
        hdr->n_batches = carry.v[5] > 0 ? (carry.v[5] - 1) / batch_units + 1 : 0;
        unsigned long long bad = hdr->n_bad;
        if (bad) raise_status(hdr, DST_ERR_INDEX_OUT_OF_RANGE);
        if (result) {
            result->n_unique = carry.v[1];
            result->n_out_of_range = (long long)bad;
            result->max_segment = maxseg;
        }
    }
    __syncthreads();   // this block's global writes (offsets, heavy) are visible to the whole block
    // a6: one descriptor per chunk of every heavy row
    const int n_heavy = carry.v[2];
    for (int h = warp_id(); h < n_heavy; h += kScanThreads / 32) {
        HeavyInfo hi = heavy[h];
        int seg_begin = offsets[hi.row], seg_end = offsets[hi.row + 1];
        for (int k = lane_id(); k < hi.n_chunks; k += 32) {
            int b = seg_begin + k * chunk;
            chunkdesc[hi.chunk_base + k] = ChunkDesc{hi.row, b, min(chunk, seg_end - b), h};
        }
    }
}

// ---------------------------------------------------------------------------
// a4: one stable 8-bit radix pass (least significant digit first), single sweep
// over the keys with a decoupled look-back for the cross-tile prefix
// ---------------------------------------------------------------------------
__device__ __forceinline__ unsigned lookback_exclusive(volatile unsigned* desc, int tile, int d, unsigned cnt,
                                                       WsHeader* hdr) {
    if (tile == 0) { desc[d] = kFlagPrefix | cnt; return 0; }
    desc[(size_t)tile * 256 + d] = kFlagAggregate | cnt;
    unsigned excl = 0;
    bool ok = true;
    for (int t = tile - 1; t >= 0; --t) {
        unsigned v;
        int spins = 0;
        while (((v = desc[(size_t)t * 256 + d]) & kFlagMask) == 0) {
            if (++spins > kSpinLimit) { ok = false; break; }
            __nanosleep(40);
        }
        if (!ok) break;
        excl += v & kValueMask;
        if ((v & kFlagMask) == kFlagPrefix) break;
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
    if (threadIdx.x == 0) s_tile = atomicAdd(&hdr->ticket[pass], 1u);   // tiles start in id order
    for (int s = threadIdx.x; s < kWarps * 256; s += kSortThreads) (&wh[0][0])[s] = 0;
    __syncthreads();
    const int tile = (int)s_tile;
    // pass 0 reads every input position (invalid rows carry kInvalidKey and drop out);
    // later passes read the n_valid survivors
    const int n_in = pass == 0 ? capacity : hdr->n_valid;
    const long long t0 = (long long)tile * kTile;
    if (t0 >= n_in) return;

    const int lane = lane_id(), warp = warp_id();
    const int shift = 8 * pass;
    const unsigned lt_mask = (1u << lane) - 1u;
    unsigned key[kSortItems], pos[kSortItems], rank[kSortItems];
    bool valid[kSortItems];
#pragma unroll
    for (int k = 0; k < kSortItems; ++k) {
        long long e = t0 + warp * (32 * kSortItems) + k * 32 + lane;
        valid[k] = false; key[k] = kInvalidKey; pos[k] = 0;
        if (e < n_in) {
            key[k] = in_keys[e];
            pos[k] = in_pos ? in_pos[e] : (unsigned)e;
            valid[k] = key[k] != kInvalidKey;
        }
    }
    // stable rank inside the warp's 256 consecutive keys
#pragma unroll
    for (int k = 0; k < kSortItems; ++k) {
        unsigned dg = valid[k] ? ((key[k] >> shift) & 255u) : (0x10000u | lane);
        unsigned m = __match_any_sync(0xFFFFFFFFu, dg);
        int leader = __ffs(m) - 1;
        unsigned pre = 0;
        if (valid[k] && lane == leader) { pre = wh[warp][dg]; wh[warp][dg] = pre + __popc(m); }
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
    unsigned g = digit_hist[d];
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
        if (valid[k]) {
            unsigned dg = (key[k] >> shift) & 255u;
            unsigned q = bin_base[dg] + wh[warp][dg] + rank[k];
            if (q < (unsigned)capacity) {
                if (out_keys) out_keys[q] = key[k];
                out_pos[q] = pos[k];
            } else {
                raise_status(hdr, DST_ERR_TIMEOUT);   // only reachable after a failed look-back
            }
        }
    }
}

// ---- host-side launchers ------------------------------------------------------
cudaError_t launch_hist(const HistParams& P, int grid_x, int index_type, WsHeader* hdr, unsigned* count,
                        unsigned* digit_hist, unsigned* keys, SliceEntry* tab, long long vocab, int passes,
                        cudaStream_t stream) {
    dim3 grid(grid_x, P.n);
    if (index_type == DST_I64)
        k_hist<long long><<<grid, kSortThreads, 0, stream>>>(P, hdr, count, digit_hist, keys, tab, vocab, passes);
    else
        k_hist<int><<<grid, kSortThreads, 0, stream>>>(P, hdr, count, digit_hist, keys, tab, vocab, passes);
    return cudaGetLastError();
}

cudaError_t launch_scan(int index_type, WsHeader* hdr, const unsigned* count, int* offsets, HeavyInfo* heavy,
                        ChunkDesc* chunkdesc, void* unique_rows, int* counts_out, dst_result_t* result,
                        int2* batches, int vocab, int vocab_pad, int chunk, int batch_units, cudaStream_t stream) {
    if (index_type == DST_I64)
        k_scan<long long><<<1, kScanThreads, 0, stream>>>(hdr, count, offsets, heavy, chunkdesc,
                                                          static_cast<long long*>(unique_rows), counts_out, result,
                                                          batches, vocab, vocab_pad, chunk, batch_units);
    else
        k_scan<int><<<1, kScanThreads, 0, stream>>>(hdr, count, offsets, heavy, chunkdesc,
                                                    static_cast<int*>(unique_rows), counts_out, result, batches,
                                                    vocab, vocab_pad, chunk, batch_units);
    return cudaGetLastError();
}

cudaError_t launch_radix_pass(int n_tiles, WsHeader* hdr, const unsigned* in_keys, const unsigned* in_pos,
                              unsigned* out_keys, unsigned* out_pos, const unsigned* digit_hist, unsigned* desc,
                              int pass, int capacity, cudaStream_t stream) {
    k_radix_pass<<<n_tiles, kSortThreads, 0, stream>>>(hdr, in_keys, in_pos, out_keys, out_pos, digit_hist, desc,
                                                       pass, capacity);
    return cudaGetLastError();
}

}  // namespace dst
