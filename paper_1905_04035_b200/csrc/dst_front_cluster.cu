// Index side of densify for small inputs, in one kernel: a thread-block cluster of kClusterCtas
// CTAs validates the indices, sorts them (two stable 8-bit radix passes), takes the run lengths and
// scans them into every table the row-reduction kernel needs.
//
// Why a cluster: for a Transformer batch of a few thousand tokens (the paper's Section 3 setting)
// the index work is pure latency.  Spread over separate kernels it costs more launches than work;
// in one CTA it is bound by one SM's instruction rate.  Eight CTAs on eight SMs share the work and
// exchange what they must through distributed shared memory and cluster barriers:
//   - the per-digit counts of each CTA (to place a CTA's entries behind those of the CTAs before it),
//   - the entries themselves: pass 0 scatters each packed entry (key << 16 | position) into the
//     shared memory of the CTA that owns that part of the sorted order,
//   - count[v], kept in shared memory, a slice of the vocabulary per CTA,
//   - the per-CTA sums of the final scan.
// Nothing spins: the only waits are cluster barriers that every thread of every CTA reaches the same
// number of times.  The kernel also clears the few global tables that must start at zero, so this
// path needs no memset.
//
// Limits: n_total <= kFrontMaxRows (positions fit 16 bits), vocab <= 65536 (keys fit 16 bits),
// R <= kHistSlices (the slice table travels as a kernel parameter).
#include <cooperative_groups.h>

#include <atomic>

#include "dst_common.cuh"

namespace cg = cooperative_groups;

namespace dst {

struct FrontArgs {
    HistParams P;              // the slices
    WsHeader* hdr;
    SliceEntry* tab;
    unsigned* perm;
    int* offsets;
    HeavyInfo* heavy;
    void* unique_rows;
    int* counts_out;
    dst_result_t* result;
    int2* batches;
    int* urow;
    int* uoff;
    int compact;
    unsigned* node_cnt;
    long long vocab;
    int n_total, vocab_pad, chunk, batch_units, batch_max, nodecnt_words;
    int lw;                    // entries per warp (multiple of 32); a CTA's slice of the sorted order holds 32 * lw
    int rpt;                   // vocabulary rows per thread in the scan; a CTA's slice of count[] holds 1024 * rpt
    const uint4* copy_src;     // clusters after the first: out = dense_in (or zeros), 16 bytes per thread and step
    uint4* copy_dst;
    long long copy_vecs;
    int copy_apply;            // out -= copy_lr * dense_in instead of out = dense_in (fp32 tensors)
    float copy_lr;
};

constexpr int kFrontWarps = kFrontThreads / 32;
constexpr int kFrontGroups = 8;       // groups of 32 entries per warp, at most (kFrontMaxRows / 256 / 32)
constexpr int kFrontRpt = 8;          // rows per thread, at most (65536 / 8192)

// one group of 32 entries: add it to the warp's running digit counters and return this lane's
// rank among the warp's entries so far with the same digit (wh: this warp's 256 counters)
__device__ __forceinline__ unsigned rank_step(unsigned short* wh, bool valid, unsigned dg, int lane) {
    const unsigned m = match_digit(dg & 255u, valid);
    const int leader = valid ? __ffs(m) - 1 : lane;
    unsigned pre = 0;
    if (valid && lane == leader) { pre = wh[dg]; wh[dg] = (unsigned short)(pre + __popc(m)); }
    pre = __shfl_sync(0xFFFFFFFFu, pre, leader);
    __syncwarp();
    return pre + __popc(m & ((1u << lane) - 1u));
}

// After every warp has counted its digits into wh[w][d]: turn the counts into the sorted position
// of the first entry of (digit d, this CTA, warp w).  One cluster barrier inside.  Returns the
// number of entries over the whole cluster.
__device__ __forceinline__ unsigned cluster_bases(cg::cluster_group& cluster, unsigned short (*wh)[256],
                                                  unsigned* cta_tot, unsigned* s_warp_tot, unsigned* s_total) {
    const int lane = lane_id(), warp = warp_id();
    const unsigned rank = cluster.block_rank();
    unsigned tot = 0;
    if (threadIdx.x < 256) {
#pragma unroll 8
        for (int w = 0; w < kFrontWarps; ++w) { unsigned t = wh[w][threadIdx.x]; wh[w][threadIdx.x] = (unsigned short)tot; tot += t; }
        cta_tot[threadIdx.x] = tot;
    }
    cluster.sync();                                   // every CTA's per-digit totals are in place
    unsigned before = 0, all = 0;
    if (threadIdx.x < 256) {
#pragma unroll
        for (unsigned c = 0; c < (unsigned)kClusterCtas; ++c) {
            const unsigned t = cluster.map_shared_rank(cta_tot, c)[threadIdx.x];
            if (c < rank) before += t;
            all += t;
        }
    }
    unsigned inc = all;                               // exclusive scan of the digit totals over the 256 digits
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { unsigned t = __shfl_up_sync(0xFFFFFFFFu, inc, o); if (lane >= o) inc += t; }
    if (lane == 31 && warp < 8) s_warp_tot[warp] = inc;
    __syncthreads();
    if (threadIdx.x < 256) {
        unsigned base = inc - all + before;
        for (int w = 0; w < warp; ++w) base += s_warp_tot[w];
#pragma unroll 8
        for (int w = 0; w < kFrontWarps; ++w) wh[w][threadIdx.x] = (unsigned short)(wh[w][threadIdx.x] + base);
        if (threadIdx.x == 255) *s_total = base - before + all;
    }
    __syncthreads();
    return *s_total;
}

struct Sum6 { int v[6]; };   // 0 offset, 1 unique, 2 heavy rows, 3 chunks, 4 upper nodes, 5 units of the light work items

template <typename IT>
__global__ void __cluster_dims__(kClusterCtas, 1, 1) __launch_bounds__(kFrontThreads, 1)
k_front_cluster(const __grid_constant__ FrontArgs f) {
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ unsigned short wh[kFrontWarps][256];
    __shared__ unsigned cta_tot[256];
    __shared__ unsigned s_warp_tot[8];
    __shared__ unsigned s_total;
    __shared__ int s_scan[kFrontWarps][6];
    __shared__ int cta_sum[6];
    __shared__ int s_before[6], s_grand[6];
    __shared__ int s_maxseg[kFrontWarps];
    pdl_trigger();
    pdl_wait();

    if (blockIdx.x >= (unsigned)kClusterCtas) {
        // Not the index cluster: meanwhile give every output row its dense_in row (or zeros).  The rows
        // that do get contributions are rewritten by the row-reduction kernel; for a batch of a few
        // thousand tokens against a vocabulary of tens of thousands that is a small part of the rows,
        // and this copy, most of the bytes of the whole operation, hides the index work entirely.
        const long long stride = (long long)(gridDim.x - kClusterCtas) * kFrontThreads;
        long long i = (long long)(blockIdx.x - kClusterCtas) * kFrontThreads + threadIdx.x;
        if (f.copy_src && f.copy_apply) {
            // the dense part of the SGD step for every row: weight -= lr * dense gradient
            const float4* src = reinterpret_cast<const float4*>(f.copy_src);
            float4* dst = reinterpret_cast<float4*>(f.copy_dst);
            const float nlr = -f.copy_lr;
            for (; i + 3 * stride < f.copy_vecs; i += 4 * stride) {
                float4 g[4], w[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) { g[q] = __ldcs(src + i + q * stride); w[q] = __ldcs(dst + i + q * stride); }
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    __stcs(dst + i + q * stride, make_float4(fmaf(nlr, g[q].x, w[q].x), fmaf(nlr, g[q].y, w[q].y),
                                                            fmaf(nlr, g[q].z, w[q].z), fmaf(nlr, g[q].w, w[q].w)));
            }
            for (; i < f.copy_vecs; i += stride) {
                const float4 g = __ldcs(src + i), w = __ldcs(dst + i);
                __stcs(dst + i, make_float4(fmaf(nlr, g.x, w.x), fmaf(nlr, g.y, w.y), fmaf(nlr, g.z, w.z), fmaf(nlr, g.w, w.w)));
            }
        } else if (f.copy_src) {
            for (; i + 7 * stride < f.copy_vecs; i += 8 * stride) {
                uint4 v[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) v[q] = __ldcs(f.copy_src + i + q * stride);
#pragma unroll
                for (int q = 0; q < 8; ++q) __stcs(f.copy_dst + i + q * stride, v[q]);
            }
            for (; i < f.copy_vecs; i += stride) __stcs(f.copy_dst + i, __ldcs(f.copy_src + i));
        } else {
            for (; i < f.copy_vecs; i += stride) __stcs(f.copy_dst + i, make_uint4(0u, 0u, 0u, 0u));
        }
        return;
    }
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int lane = lane_id(), warp = warp_id();
    const int S = 32 * f.lw;                         // entries of the sorted order this CTA owns
    const int Vs = kFrontThreads * f.rpt;            // rows of count[] this CTA owns
    unsigned* packed = reinterpret_cast<unsigned*>(dyn);                          // [S] key << 16 | position
    unsigned* cnt = packed + S;                                                   // [Vs]
    unsigned short* skey = reinterpret_cast<unsigned short*>(cnt + Vs);           // [S] sorted keys
    WsHeader* hdr = f.hdr;
    const int gt = rank * kFrontThreads + threadIdx.x;   // thread id in the cluster
    constexpr int kAllThreads = kClusterCtas * kFrontThreads;

    // ---- clear what must start at zero
    for (int i = threadIdx.x; i < Vs; i += kFrontThreads) cnt[i] = 0;
    for (int i = gt; i < f.batch_max; i += kAllThreads) f.batches[i] = make_int2(f.compact ? 0x7FFFFFFF : 0, 0);
    for (int i = gt; i < f.nodecnt_words; i += kAllThreads) f.node_cnt[i] = 0;
    if (rank == 0) {
        if (threadIdx.x < (int)(sizeof(WsHeader) / 4)) reinterpret_cast<unsigned*>(hdr)[threadIdx.x] = 0;
        if (threadIdx.x < f.P.n) f.tab[threadIdx.x] = f.P.s[threadIdx.x];
    }
    for (int s = lane; s < 128; s += 32) reinterpret_cast<unsigned*>(wh[warp])[s] = 0;

    // ---- a1: load and validate.  Warp gw of the cluster owns entries [gw * lw, gw * lw + lw).
    const int gw = rank * kFrontWarps + warp;
    const int ng = f.lw / 32;
    unsigned key[kFrontGroups];
    {
        int r = 0;
#pragma unroll
        for (int g = 0; g < kFrontGroups; ++g) {
            key[g] = kInvalidKey;
            const int e = gw * f.lw + g * 32 + lane;
            if (g < ng && e < f.n_total) {
                while (r + 1 < f.P.n && (long long)e >= f.P.s[r + 1].start) ++r;
                const long long v = (long long)static_cast<const IT*>(f.P.s[r].indices)[(long long)e - f.P.s[r].start];
                if (v >= 0 && v < f.vocab) key[g] = (unsigned)v;
            }
        }
    }
    __syncwarp();
    // ---- a4, pass 0: low digit; registers -> the shared memory of the CTA that owns the target position.
    // rk[g] is the entry's rank among the warp's entries with the same digit; once the counters have
    // become positions (cluster_bases) the target is wh[warp][digit] + rk[g].
    unsigned short rk[kFrontGroups];
#pragma unroll
    for (int g = 0; g < kFrontGroups; ++g) {
        rk[g] = 0;
        if (g < ng) rk[g] = (unsigned short)rank_step(wh[warp], key[g] != kInvalidKey, key[g] & 255u, lane);
    }
    __syncthreads();
    const int n_valid = (int)cluster_bases(cluster, wh, cta_tot, s_warp_tot, &s_total);
#pragma unroll
    for (int g = 0; g < kFrontGroups; ++g) {
        if (g < ng && key[g] != kInvalidKey) {
            const unsigned q = (unsigned)wh[warp][key[g] & 255u] + rk[g];
            const unsigned owner = q / (unsigned)S;
            cluster.map_shared_rank(packed, owner)[q - owner * (unsigned)S] =
                (key[g] << 16) | (unsigned)(gw * f.lw + g * 32 + lane);
        }
    }
    __syncthreads();                                  // every warp has read its positions
    for (int s = lane; s < 128; s += 32) reinterpret_cast<unsigned*>(wh[warp])[s] = 0;
    cluster.sync();                                   // all of pass 0 has landed
    // ---- pass 1: high digit; this CTA's slice [rank * S, rank * S + S) -> perm (global) and skey (owner's shared memory)
#pragma unroll
    for (int g = 0; g < kFrontGroups; ++g) {
        key[g] = kInvalidKey; rk[g] = 0;
        const int e = warp * f.lw + g * 32 + lane;
        if (g < ng) {
            const bool valid = rank * S + e < n_valid;
            const unsigned x = valid ? packed[e] : 0u;   // a packed entry (never 0xFFFFFFFF: positions stay below 65535)
            rk[g] = (unsigned short)rank_step(wh[warp], valid, x >> 24, lane);
            if (valid) key[g] = x;
        }
    }
    __syncthreads();
    cluster_bases(cluster, wh, cta_tot, s_warp_tot, &s_total);
#pragma unroll
    for (int g = 0; g < kFrontGroups; ++g) {
        if (g < ng && key[g] != kInvalidKey) {
            const unsigned x = key[g];
            const unsigned q = (unsigned)wh[warp][x >> 24] + rk[g];
            f.perm[q] = x & 0xFFFFu;
            const unsigned owner = q / (unsigned)S;
            cluster.map_shared_rank(skey, owner)[q - owner * (unsigned)S] = (unsigned short)(x >> 16);
        }
    }
    cluster.sync();                                   // the sorted keys are in place
    // ---- a2: run lengths.  The first entry of a run subtracts its position from count[key], the last
    // adds its position + 1; count[] lives in shared memory, rows [c * Vs, c * Vs + Vs) in CTA c.
    for (int e = threadIdx.x; e < S; e += kFrontThreads) {
        const int i = rank * S + e;
        if (i < n_valid) {
            const unsigned k = skey[e];
            unsigned prev = ~k, next = ~k;
            if (i > 0) prev = e > 0 ? skey[e - 1] : cluster.map_shared_rank(skey, rank - 1)[S - 1];
            if (i + 1 < n_valid) next = e + 1 < S ? skey[e + 1] : cluster.map_shared_rank(skey, rank + 1)[0];
            const unsigned owner = k / (unsigned)Vs;
            unsigned* c = cluster.map_shared_rank(cnt, owner) + (k - owner * (unsigned)Vs);
            if (prev != k) atomicSub(c, (unsigned)i);
            if (next != k) atomicAdd(c, (unsigned)i + 1u);
        }
    }
    cluster.sync();                                   // count[] is complete
    // ---- a3 + a5 + a6: scan of count[].  Thread t of CTA c owns rows c * Vs + t * rpt + [0, rpt).
    IT* unique_rows = static_cast<IT*>(f.unique_rows);
    const int chunk = f.chunk, B = f.batch_units, vocab = (int)f.vocab;
    const int l0 = threadIdx.x * f.rpt;              // first owned row, local
    const int e0 = rank * Vs + l0;                   // ... and global
    int c[kFrontRpt];
    Sum6 mine{};
    int maxseg = 0;
#pragma unroll
    for (int q = 0; q < kFrontRpt; ++q) {
        c[q] = q < f.rpt ? (int)cnt[l0 + q] : 0;
        const int cc = c[q];
        mine.v[0] += cc;
        mine.v[1] += cc > 0;
        if (q < f.rpt && e0 + q < vocab && !(f.compact && cc == 0)) mine.v[5] += row_units(cc, chunk);
        if (cc > chunk) {
            const int n = (cc + chunk - 1) / chunk;
            mine.v[2] += 1; mine.v[3] += n; mine.v[4] += upper_nodes(n);
        }
        maxseg = max(maxseg, cc);
    }
    int prev_cost = 0;                               // units of the row before this thread's first one
    if (e0 > 0 && e0 < f.vocab_pad) {
        const unsigned pc = l0 > 0 ? cnt[l0 - 1] : cluster.map_shared_rank(cnt, rank - 1)[Vs - 1];
        prev_cost = row_units((int)pc, chunk);
    }
    Sum6 inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
        for (int q = 0; q < 6; ++q) {
            int t = __shfl_up_sync(0xFFFFFFFFu, inc.v[q], o);
            if (lane >= o) inc.v[q] += t;
        }
    }
    for (int o = 16; o > 0; o >>= 1) maxseg = max(maxseg, __shfl_down_sync(0xFFFFFFFFu, maxseg, o));
    if (lane == 31) {
#pragma unroll
        for (int q = 0; q < 6; ++q) s_scan[warp][q] = inc.v[q];
    }
    if (lane == 0) s_maxseg[warp] = maxseg;
    __syncthreads();
    if (warp == 0) {
        // lane w holds warp w's sums: scan them, leave each warp's exclusive prefix and the CTA's sums
        Sum6 ws, wi;
#pragma unroll
        for (int q = 0; q < 6; ++q) { ws.v[q] = s_scan[lane][q]; wi.v[q] = ws.v[q]; }
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
            for (int q = 0; q < 6; ++q) {
                int t = __shfl_up_sync(0xFFFFFFFFu, wi.v[q], o);
                if (lane >= o) wi.v[q] += t;
            }
        }
#pragma unroll
        for (int q = 0; q < 6; ++q) {
            s_scan[lane][q] = wi.v[q] - ws.v[q];
            if (lane == 31) cta_sum[q] = wi.v[q];
        }
        int m = s_maxseg[lane];
        for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_down_sync(0xFFFFFFFFu, m, o));
        if (lane == 0 && m > 0) atomicMax(&hdr->max_segment, m);
    }
    __syncthreads();
    Sum6 run;
#pragma unroll
    for (int q = 0; q < 6; ++q) run.v[q] = inc.v[q] - mine.v[q] + s_scan[warp][q];
    cluster.sync();                                   // every CTA's sums are in place
    if (threadIdx.x < 6) {
        int before = 0, all = 0;
        for (int cc = 0; cc < kClusterCtas; ++cc) {
            const int t = cluster.map_shared_rank(cta_sum, cc)[threadIdx.x];
            if (cc < rank) before += t;
            all += t;
        }
        s_before[threadIdx.x] = before;
        s_grand[threadIdx.x] = all;
    }
    __syncthreads();
#pragma unroll
    for (int q = 0; q < 6; ++q) run.v[q] += s_before[q];
    if (e0 < f.vocab_pad) {
        int rem = run.v[5] % B;                      // units before row e0, modulo the batch size
        int b = run.v[5] / B;
#pragma unroll
        for (int q = 0; q < kFrontRpt; ++q) {
            const int v = e0 + q;
            if (q < f.rpt && v < f.vocab_pad) {
                const int cc = c[q];
                f.offsets[v] = run.v[0];
                if (cc > 0) {
                    if (unique_rows) unique_rows[run.v[1]] = (IT)v;
                    if (f.counts_out) f.counts_out[run.v[1]] = cc;
                    if (f.compact) {
                        // the row batches list named rows only: row number and first entry by rank among them
                        const int u = run.v[1];
                        f.urow[u] = v;
                        f.uoff[u] = run.v[0];
                        const int cost = row_units(cc, chunk);
                        atomicMin(&f.batches[b].x, u + 1);
                        atomicMax(&f.batches[b].y, u + 1);
                        rem += cost;
                        if (rem >= B) { b += rem / B; rem %= B; }
                    }
                    run.v[1] += 1;
                }
                if (cc > chunk) {
                    // a6: a heavy row becomes n chunk items and a combine tree
                    const int n = (cc + chunk - 1) / chunk;
                    f.heavy[run.v[2]] = HeavyInfo{v, run.v[3], run.v[4], n, run.v[0], cc, {0, 0}};
                    run.v[2] += 1; run.v[3] += n; run.v[4] += upper_nodes(n);
                }
                run.v[0] += cc;
                if (v < vocab && !f.compact) {
                    // light work items: row v belongs to batch floor(units before v / batch size)
                    const int cost = row_units(cc, chunk);
                    if (v == 0 || prev_cost > rem) f.batches[b].x = v + 1;
                    rem += cost;
                    if (v == vocab - 1 || rem >= B) f.batches[b].y = v + 1;
                    if (rem >= B) { b += rem / B; rem %= B; }
                    prev_cost = cost;
                }
            }
        }
    }
    cluster.sync();       // all tables and the header's max_segment are written; nobody reads a peer's shared memory after this
    if (rank == 0 && threadIdx.x == 0) {
        f.offsets[f.vocab_pad] = s_grand[0];
        if (f.compact) f.uoff[s_grand[1]] = s_grand[0];
        hdr->n_valid = s_grand[0];
        hdr->n_unique = s_grand[1];
        hdr->n_heavy = s_grand[2];
        hdr->n_chunks = s_grand[3];
        hdr->n_upper = s_grand[4];
        hdr->n_batches = s_grand[5] > 0 ? (s_grand[5] - 1) / B + 1 : 0;
        const long long bad = (long long)f.n_total - n_valid;
        hdr->n_bad = (unsigned long long)bad;
        if (bad) raise_status(hdr, DST_ERR_INDEX_OUT_OF_RANGE);
        if (f.result) {
            f.result->n_unique = s_grand[1];
            f.result->n_out_of_range = bad;
            f.result->max_segment = *reinterpret_cast<volatile int*>(&hdr->max_segment);
        }
    }
}

cudaError_t launch_front_cluster(int index_type, const FrontParams& p, cudaStream_t stream) {
    FrontArgs f;
    f.P = p.P; f.hdr = p.hdr; f.tab = p.tab; f.perm = p.perm; f.offsets = p.offsets; f.heavy = p.heavy;
    f.unique_rows = p.unique_rows; f.counts_out = p.counts_out; f.result = p.result; f.batches = p.batches;
    f.urow = p.urow; f.uoff = p.uoff; f.compact = p.compact;
    f.node_cnt = p.node_cnt; f.vocab = p.vocab; f.n_total = p.n_total; f.vocab_pad = p.vocab_pad; f.chunk = p.chunk;
    f.batch_units = p.batch_units; f.batch_max = p.batch_max; f.nodecnt_words = p.nodecnt_words;
    f.copy_src = static_cast<const uint4*>(p.copy_src); f.copy_dst = static_cast<uint4*>(p.copy_dst);
    f.copy_vecs = p.copy_bytes / 16;
    f.copy_apply = p.copy_apply; f.copy_lr = p.copy_lr;
    const int per_warp = (p.n_total + kClusterCtas * kFrontWarps - 1) / (kClusterCtas * kFrontWarps);
    f.lw = (per_warp + 31) / 32 * 32;
    if (f.lw < 32) f.lw = 32;
    f.rpt = (p.vocab_pad + kClusterCtas * kFrontThreads - 1) / (kClusterCtas * kFrontThreads);
    if (f.rpt < 1) f.rpt = 1;
    if (f.lw > 32 * kFrontGroups || f.rpt > kFrontRpt) return cudaErrorInvalidValue;
    const size_t S = size_t(32) * f.lw, Vs = size_t(kFrontThreads) * f.rpt;
    const size_t smem = S * 4 + Vs * 4 + S * 2;
    cudaError_t e;
    if (index_type == DST_I64)
        e = cudaFuncSetAttribute(k_front_cluster<long long>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    else
        e = cudaFuncSetAttribute(k_front_cluster<int>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    // Copy clusters: no more than can be resident beside the index cluster (a cluster needs eight free SMs of
    // one GPC; clusters that start late would finish late, their share of the rows being fixed).
    int copy_clusters = p.copy_clusters > 0 ? p.copy_clusters : 0;
    if (copy_clusters > 0) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(kClusterCtas * (1 + copy_clusters)); cfg.blockDim = dim3(kFrontThreads); cfg.dynamicSmemBytes = smem;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = kClusterCtas; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        // the answer depends on the device and on the shared memory asked for: remembered per index type
        static std::atomic<long long> cache[2];
        const int which = index_type == DST_I64 ? 1 : 0;
        int dev = 0;
        (void)cudaGetDevice(&dev);
        const long long key = ((long long)smem << 16) | ((long long)(dev & 0xFF) << 8);
        const long long seen = cache[which].load();
        int resident = 0;
        if ((seen & ~0xFFLL) == key && (seen & 0xFF) != 0) {
            resident = int(seen & 0xFF);
        } else {
            if (which) e = cudaOccupancyMaxActiveClusters(&resident, k_front_cluster<long long>, &cfg);
            else e = cudaOccupancyMaxActiveClusters(&resident, k_front_cluster<int>, &cfg);
            if (e != cudaSuccess) { (void)cudaGetLastError(); resident = 0; }
            if (resident > 0) cache[which].store(key | (resident > 255 ? 255 : resident));
        }
        if (resident >= 2 && copy_clusters > resident - 1) copy_clusters = resident - 1;
    }
    const int grid = kClusterCtas * (1 + copy_clusters);
    if (index_type == DST_I64)
        return launch_pdl(k_front_cluster<long long>, dim3(grid), dim3(kFrontThreads), smem, stream, f);
    return launch_pdl(k_front_cluster<int>, dim3(grid), dim3(kFrontThreads), smem, stream, f);
}

}  // namespace dst
