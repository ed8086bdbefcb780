// Index side of densify for small inputs, in one kernel: a thread-block cluster of kClusterCtas
// CTAs validates the indices, sorts them (two stable 8-bit radix passes) and walks the sorted
// order once to produce every table the row-reduction kernel needs.
//
// Why a cluster: for a Transformer batch of a few thousand tokens (the paper's Section 3 setting)
// the index work is pure latency.  Spread over separate kernels it costs more launches than work;
// in one CTA it is bound by one SM's instruction rate.  Eight CTAs on eight SMs share the work and
// exchange what they must through distributed shared memory and cluster barriers:
//   - the per-digit counts of each CTA (to place a CTA's entries behind those of the CTAs before it),
//   - the entries themselves: each pass scatters every packed entry (key << 16 | position) into the
//     shared memory of the CTA that owns that part of the sorted order,
//   - one summary per CTA of the segmented scan over the sorted entries.
// Nothing spins: the only waits are cluster barriers that every thread of every CTA reaches the same
// number of times.
//
// The row-reduction kernel is launched as a programmatic dependent of this one and runs beside it on
// the other SMs, moving most of the bytes of the call meanwhile, so every access this kernel makes to
// global memory queues behind that traffic.  Hence the shape of the kernel: global memory is read once
// (the indices) and written at two points only -- a bitmap of the named rows as soon as the indices are
// validated (the rows outside it only need their dense_in row, which the other kernel copies while the
// sort is still running), and all tables in one burst at the end, followed by one flag.  Everything in
// between lives in shared memory.  The header with the flags is cleared before the dependent launch is
// released.
//
// The tables list the named rows only (by rank u among them: urec[u] packs the row number and its first entry),
// which is why this path is taken only when there are no more input rows than vocabulary rows.
// Limits: n_total <= kFrontMaxRows (positions fit 16 bits), vocab <= 65536 (keys fit 16 bits),
// R <= kHistSlices (the slice table travels as a kernel parameter).
#include <cooperative_groups.h>

#include "dst_common.cuh"

namespace cg = cooperative_groups;

namespace dst {

struct FrontArgs {
    HistParams P;              // the slices
    WsHeader* hdr;
    SliceEntry* tab;
    unsigned short* perm;      // input positions in sorted order, 16 bits each
    HeavyInfo* heavy;
    void* unique_rows;
    int* counts_out;
    dst_result_t* result;
    unsigned* urec;            // per named row, by rank: row << 16 | first entry in perm; one more word holds the number of entries
    unsigned* node_cnt;
    int* bfirst;               // light work items: rank of the first named row of each; one more entry holds the number of named rows
    unsigned* bitmap;          // [bitmap_words][kClusterCtas]: this CTA's copy of the named-row bitmap at [w * 8 + rank]
    long long vocab;
    int n_total, chunk_log, batch_log, nodecnt_words, bitmap_words;
    int lw;                    // entries per warp (multiple of 32); a CTA's slice of the sorted order holds 32 * lw
};

constexpr int kFrontWarps = kFrontThreads / 32;
constexpr int kFrontGroups = 8;       // groups of 32 entries per warp, at most (kFrontMaxRows / 256 / 32)
constexpr int kFrontParts = 4;        // the warps of a CTA in four parts of eight for the digit prefix

// A note on the style of this file.  The code of this kernel is fetched cold on every launch, through a
// memory system that the row-reduction kernel keeps saturated meanwhile, and is executed once: its
// running time follows the bytes of straight-line code more than the instructions executed.  So loops
// stay rolled (#pragma unroll 1), per-entry state lives in shared memory instead of register arrays,
// and what is needed at several places exists once.

// Lanes of the warp whose 8-bit digit equals this lane's, among the lanes with `valid` set.
__device__ __forceinline__ unsigned match_digit_rolled(unsigned dg, bool valid) {
    unsigned m = __ballot_sync(0xFFFFFFFFu, valid);
#pragma unroll           // the one loop of this file that is unrolled: the ranking is bound by the instructions issued
    for (int b = 0; b < 8; ++b) {
        const bool bit = (dg >> b) & 1u;
        const unsigned bal = __ballot_sync(0xFFFFFFFFu, bit);
        m &= bit ? bal : ~bal;
    }
    return m;
}

struct DigitScratch {
    unsigned short wh[kFrontWarps][256];      // per warp and digit: count, then exclusive prefix inside the warp's part
    unsigned short part_tot[kFrontParts][256];
    unsigned cta_tot[256];                    // this CTA's entries per digit (read by the other CTAs)
    unsigned base[kFrontParts][256];          // sorted position of the first entry of (digit, this CTA, part)
    unsigned warp_tot[8];
    unsigned total;
};

// ---- the segmented scan over the sorted entries --------------------------------------------------
// What a stretch of consecutive sorted entries knows about the rows (runs of equal keys) it touches.
// A row is accounted for where its last entry (its tail) lies; its length needs the position of its
// first entry (its head), which may lie in an earlier stretch: such a tail stays open (`bt`) until
// the stretches are combined.  At most one tail of a stretch can be open: the first, when no head
// comes before it.
struct Seg {
    int nt;     // tails: rows that end in the stretch
    int nh;     // of those with a known length: heavy rows,
    int nc;     //   their chunks,
    int nu;     //   their upper combine-tree nodes,
    int un;     // of the rows with a known length: units of light work (entries + 1; a heavy row counts 1)
    int mx;     // longest known row
    int lh;     // position of the last head in the stretch, -1: none
    int bt;     // position of the open tail, -1: none
};
__device__ __forceinline__ Seg seg_identity() { return Seg{0, 0, 0, 0, 0, 0, -1, -1}; }
// Chunks and upper tree nodes of a heavy row, packed (nodes << 16 | chunks; a row has at most 4096 chunks).
// Out of line on purpose: heavy rows are few, and the code of this kernel is fetched cold on every
// launch, through a memory system that the row-reduction kernel keeps busy, so every kilobyte of
// straight-line code on the common path is paid for in time.
__device__ __noinline__ unsigned heavy_shape(int count, int chunk_log) {
    const int n = (count + (1 << chunk_log) - 1) >> chunk_log;
    return ((unsigned)upper_nodes(n) << 16) | (unsigned)n;
}
__device__ __forceinline__ void seg_add_row(Seg& s, int count, int chunk_log) {
    s.mx = max(s.mx, count);
    s.un += row_units(count, 1 << chunk_log);
    if (count > (1 << chunk_log)) {
        const unsigned hs = heavy_shape(count, chunk_log);
        s.nh += 1; s.nc += (int)(hs & 0xFFFFu); s.nu += (int)(hs >> 16);
    }
}
// stretch A followed by stretch B
__device__ __forceinline__ Seg seg_combine(const Seg& A, const Seg& B, int chunk_log) {
    Seg r;
    r.nt = A.nt + B.nt; r.nh = A.nh + B.nh; r.nc = A.nc + B.nc; r.nu = A.nu + B.nu; r.un = A.un + B.un;
    r.mx = max(A.mx, B.mx);
    if (B.bt >= 0 && A.lh >= 0) seg_add_row(r, B.bt - A.lh + 1, chunk_log);
    r.bt = A.bt >= 0 ? A.bt : (A.lh < 0 ? B.bt : -1);
    r.lh = B.lh >= 0 ? B.lh : A.lh;
    return r;
}
__device__ __forceinline__ Seg seg_shfl_up(const Seg& s, int o) {
    Seg t;
    t.nt = __shfl_up_sync(0xFFFFFFFFu, s.nt, o); t.nh = __shfl_up_sync(0xFFFFFFFFu, s.nh, o);
    t.nc = __shfl_up_sync(0xFFFFFFFFu, s.nc, o); t.nu = __shfl_up_sync(0xFFFFFFFFu, s.nu, o);
    t.un = __shfl_up_sync(0xFFFFFFFFu, s.un, o); t.mx = __shfl_up_sync(0xFFFFFFFFu, s.mx, o);
    t.lh = __shfl_up_sync(0xFFFFFFFFu, s.lh, o); t.bt = __shfl_up_sync(0xFFFFFFFFu, s.bt, o);
    return t;
}
__device__ __forceinline__ Seg seg_shfl(const Seg& s, int src) {
    Seg t;
    t.nt = __shfl_sync(0xFFFFFFFFu, s.nt, src); t.nh = __shfl_sync(0xFFFFFFFFu, s.nh, src);
    t.nc = __shfl_sync(0xFFFFFFFFu, s.nc, src); t.nu = __shfl_sync(0xFFFFFFFFu, s.nu, src);
    t.un = __shfl_sync(0xFFFFFFFFu, s.un, src); t.mx = __shfl_sync(0xFFFFFFFFu, s.mx, src);
    t.lh = __shfl_sync(0xFFFFFFFFu, s.lh, src); t.bt = __shfl_sync(0xFFFFFFFFu, s.bt, src);
    return t;
}
// inclusive scan over the lanes of a warp; `excl` receives the exclusive one
__device__ __forceinline__ Seg seg_warp_scan(Seg v, Seg& excl, int chunk_log) {
    const int lane = lane_id();
#pragma unroll 1
    for (int o = 1; o < 32; o <<= 1) {
        const Seg t = seg_shfl_up(v, o);
        if (lane >= o) v = seg_combine(t, v, chunk_log);
    }
    excl = seg_shfl_up(v, 1);
    if (lane == 0) excl = seg_identity();
    return v;
}

template <typename IT>
__global__ void __cluster_dims__(kClusterCtas, 1, 1) __launch_bounds__(kFrontThreads, 1)
k_front_cluster(const __grid_constant__ FrontArgs f) {
    extern __shared__ __align__(16) unsigned char dyn[];
    __shared__ DigitScratch dg;
    __shared__ Seg s_warp_seg[kFrontWarps];     // per warp: its stretch
    __shared__ Seg s_warp_pre[kFrontWarps];     // per warp: the stretch of the warps before it
    __shared__ Seg s_cta_seg;                   // this CTA's stretch (read by the other CTAs)
    __shared__ Seg s_before, s_grand;           // the stretch of the CTAs before this one / of all CTAs
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int lane = lane_id(), warp = warp_id();
    const int S = 32 * f.lw;                         // entries of the sorted order this CTA owns
    const int ng = f.lw / 32;                        // groups of 32 entries per warp = entries per thread
    // two buffers of packed entries (key << 16 | position; 0xFFFFFFFF: no entry): the passes go from one to the other
    unsigned* buf0 = reinterpret_cast<unsigned*>(dyn);                            // [S]
    unsigned* buf1 = buf0 + S;                                                    // [S]
    unsigned short* rks = reinterpret_cast<unsigned short*>(buf1 + S);            // [S] rank of an entry among its warp's entries with the same digit
    unsigned char* named = reinterpret_cast<unsigned char*>(rks + S);             // [32 * bitmap_words] 1: some valid entry names the row
    WsHeader* hdr = f.hdr;
    const int gt = rank * kFrontThreads + threadIdx.x;   // thread id in the cluster
    constexpr int kAllThreads = kClusterCtas * kFrontThreads;

    pdl_wait();
    const int gw = rank * kFrontWarps + warp;
    {
        // ask for the indices now (into L2): the trip to memory overlaps the set-up below
        int r = 0;
#pragma unroll 1
        for (int g = 0; g < ng; ++g) {
            const int e = gw * f.lw + g * 32 + lane;
            if (e < f.n_total) {
                while (r + 1 < f.P.n && (long long)e >= f.P.s[r + 1].start) ++r;
                asm volatile("prefetch.global.L2 [%0];" ::"l"(static_cast<const IT*>(f.P.s[r].indices) + ((long long)e - f.P.s[r].start)));
            }
        }
    }
    // The header (counters, flags) starts at zero; every CTA clears its own bitmap flag.  Only then may the
    // row-reduction kernel start beside this one: it polls those flags.
    if (rank == 0 && threadIdx.x < kHeaderWordsBeforeFlags) reinterpret_cast<unsigned*>(hdr)[threadIdx.x] = 0;
    if (threadIdx.x == 0) hdr->bitmap_ready[rank] = 0;
    for (int i = threadIdx.x; i < 2 * f.bitmap_words; i += kFrontThreads) reinterpret_cast<uint4*>(named)[i] = make_uint4(0u, 0u, 0u, 0u);
    __threadfence();
    __syncthreads();
    pdl_trigger();
    // ---- a1: load and validate.  Warp gw of the cluster owns entries [gw * lw, gw * lw + lw) of the input.
    {
        int r = 0;
#pragma unroll 1
        for (int g = 0; g < ng; ++g) {
            const int e = gw * f.lw + g * 32 + lane;
            unsigned x = 0xFFFFFFFFu;
            if (e < f.n_total) {
                while (r + 1 < f.P.n && (long long)e >= f.P.s[r + 1].start) ++r;
                const long long v = (long long)static_cast<const IT*>(f.P.s[r].indices)[(long long)e - f.P.s[r].start];
                if (v >= 0 && v < f.vocab) { x = ((unsigned)v << 16) | (unsigned)e; named[v] = 1; }   // everybody writes the same value
            }
            buf0[warp * f.lw + g * 32 + lane] = x;
        }
    }
    __syncthreads();
    // ---- the named rows, 32 per word, as this CTA sees them: the other kernel ORs the eight copies
    for (int w = threadIdx.x; w < f.bitmap_words; w += kFrontThreads) {
        const uint4 lo = reinterpret_cast<const uint4*>(named)[2 * w], hi = reinterpret_cast<const uint4*>(named)[2 * w + 1];
        const unsigned x[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
        unsigned word = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) word |= (((x[i] & 0x01010101u) * 0x01020408u) >> 24) << (4 * i);   // four 0/1 bytes -> four bits
        f.bitmap[w * kClusterCtas + rank] = word;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();                              // the words of every thread of this CTA, ordered by the barrier
        *reinterpret_cast<volatile int*>(&hdr->bitmap_ready[rank]) = 1;
    }
    // what else must start at zero or be in place before the tables are used
    for (int i = gt; i < f.nodecnt_words; i += kAllThreads) f.node_cnt[i] = 0;
    if (rank == 0 && threadIdx.x < f.P.n) f.tab[threadIdx.x] = f.P.s[threadIdx.x];
    // ---- a4: two stable passes, low digit of the key first.  A pass takes this CTA's slice of `src` (warp w:
    // entries [w * lw, w * lw + lw)) and sends every entry to the shared memory of the CTA that owns its
    // position in the order by digit: base[part][digit] + wh[warp][digit] + its rank among its warp's
    // entries with that digit.
    int n_valid = 0;
#pragma unroll 1
    for (int pass = 0; pass < 2; ++pass) {
        const unsigned* src = pass ? buf1 : buf0;
        unsigned* dst = pass ? buf0 : buf1;
        const int shift = 16 + 8 * pass;
        const int bound = pass ? n_valid - rank * S : S;          // entries of the slice that exist
        for (int s = lane; s < 128; s += 32) reinterpret_cast<unsigned*>(dg.wh[warp])[s] = 0;
        __syncwarp();
#pragma unroll 1
        for (int g = 0; g < ng; ++g) {
            const int e = warp * f.lw + g * 32 + lane;
            const unsigned x = e < bound ? src[e] : 0xFFFFFFFFu;
            const bool valid = x != 0xFFFFFFFFu;
            const unsigned d = (x >> shift) & 255u;
            const unsigned m = match_digit_rolled(d, valid);
            const int leader = valid ? __ffs(m) - 1 : lane;
            unsigned pre = 0;
            if (valid && lane == leader) { pre = dg.wh[warp][d]; dg.wh[warp][d] = (unsigned short)(pre + __popc(m)); }
            pre = __shfl_sync(0xFFFFFFFFu, pre, leader);
            __syncwarp();
            rks[e] = (unsigned short)(pre + __popc(m & ((1u << lane) - 1u)));
        }
        __syncthreads();
        {
            // per digit: prefix over the warps of this CTA (in four parts), then over the CTAs of the cluster
            const int d = threadIdx.x & 255, part = threadIdx.x >> 8;
            unsigned run = 0;
#pragma unroll 1
            for (int w = part * 8; w < part * 8 + 8; ++w) { const unsigned t = dg.wh[w][d]; dg.wh[w][d] = (unsigned short)run; run += t; }
            dg.part_tot[part][d] = (unsigned short)run;
            __syncthreads();
            unsigned pt[kFrontParts];
#pragma unroll
            for (int p = 0; p < kFrontParts; ++p) pt[p] = dg.part_tot[p][d];
            if (part == 0) dg.cta_tot[d] = pt[0] + pt[1] + pt[2] + pt[3];
            cluster.sync();                           // every CTA's per-digit totals are in place
            if (threadIdx.x < 256) {
                unsigned before = 0, all = 0;
#pragma unroll
                for (int c = 0; c < kClusterCtas; ++c) {
                    const unsigned t = cluster.map_shared_rank(dg.cta_tot, c)[d];
                    if (c < rank) before += t;
                    all += t;
                }
                unsigned inc = all;                   // exclusive scan of the digit totals over the 256 digits
#pragma unroll 1
                for (int o = 1; o < 32; o <<= 1) { unsigned t = __shfl_up_sync(0xFFFFFFFFu, inc, o); if (lane >= o) inc += t; }
                if (lane == 31) dg.warp_tot[warp] = inc;
                asm volatile("bar.sync 1, 256;" ::: "memory");   // the eight warps that hold the digits
                unsigned b = inc - all + before;
                for (int w = 0; w < warp; ++w) b += dg.warp_tot[w];
                if (threadIdx.x == 255) dg.total = b - before + all;
#pragma unroll
                for (int p = 0; p < kFrontParts; ++p) { dg.base[p][d] = b; b += pt[p]; }
            }
            __syncthreads();
        }
        if (pass == 0) n_valid = (int)dg.total;
#pragma unroll 1
        for (int g = 0; g < ng; ++g) {
            const int e = warp * f.lw + g * 32 + lane;
            const unsigned x = e < bound ? src[e] : 0xFFFFFFFFu;
            if (x != 0xFFFFFFFFu) {
                const unsigned d = (x >> shift) & 255u;
                const unsigned q = dg.base[warp >> 3][d] + (unsigned)dg.wh[warp][d] + (unsigned)rks[e];
                const unsigned owner = q / (unsigned)S;
                cluster.map_shared_rank(dst, owner)[q - owner * (unsigned)S] = x;
            }
        }
        cluster.sync();                               // the pass has landed everywhere
    }
    // ---- a2 + a3 + a5 + a6 in one walk over the sorted order (now in buf0).  Thread t of CTA c owns the ng
    // consecutive entries from position c * S + t * ng.  First walk: what this thread's stretch knows (Seg);
    // a scan over lanes, warps and CTAs gives every thread the stretch of everything before it; second
    // walk: the tables.
    const unsigned* sorted = buf0;
    const int e0 = threadIdx.x * ng;
    const int i0 = rank * S + e0;
    const int n_mine = max(0, min(ng, n_valid - i0));
    const int chunk_log = f.chunk_log;
    unsigned k_first_prev = 0xFFFFFFFFu, k_last_next = 0xFFFFFFFFu;      // keys beside the stretch; no key looks like this
    if (n_mine > 0) {
        if (i0 > 0) k_first_prev = (e0 > 0 ? sorted[e0 - 1] : cluster.map_shared_rank(buf0, rank - 1)[S - 1]) >> 16;
        if (i0 + ng < n_valid) k_last_next = (e0 + ng < S ? sorted[e0 + ng] : cluster.map_shared_rank(buf0, rank + 1)[0]) >> 16;
    }
    Seg mine = seg_identity();
    {
        unsigned kb = k_first_prev;
#pragma unroll 1
        for (int j = 0; j < n_mine; ++j) {
            const unsigned k = sorted[e0 + j] >> 16;
            const unsigned ka = j + 1 < n_mine ? sorted[e0 + j + 1] >> 16 : (j + 1 < ng ? 0xFFFFFFFFu : k_last_next);
            if (kb != k) mine.lh = i0 + j;
            if (ka != k) {
                mine.nt += 1;
                if (mine.lh >= 0) seg_add_row(mine, i0 + j - mine.lh + 1, chunk_log); else mine.bt = i0 + j;
            }
            kb = k;
        }
    }
    // three levels of one scan: lanes of a warp (every warp), then warps of the CTA and CTAs of the cluster
    // (warp 0; the barriers between the levels are for all)
    Seg lane_excl = seg_identity();
    {
        Seg v = mine;
#pragma unroll 1
        for (int level = 0; level < 3; ++level) {
            Seg excl = seg_identity(), incl = seg_identity();
            if (level == 0 || warp == 0) incl = seg_warp_scan(v, excl, chunk_log);
            if (level == 0) {
                lane_excl = excl;
                if (lane == 31) s_warp_seg[warp] = incl;
                __syncthreads();
                if (warp == 0) v = s_warp_seg[lane];
            } else if (level == 1) {
                if (warp == 0) { s_warp_pre[lane] = excl; if (lane == 31) s_cta_seg = incl; }
                cluster.sync();                       // every CTA's stretch is in place
                v = seg_identity();
                if (warp == 0 && lane < kClusterCtas) v = *cluster.map_shared_rank(&s_cta_seg, lane);
            } else {
                if (warp == 0) {
                    const Seg before = seg_shfl(excl, rank), grand = seg_shfl(incl, kClusterCtas - 1);
                    if (lane == 0) { s_before = before; s_grand = grand; }
                }
                __syncthreads();
            }
        }
    }
    {
        IT* unique_rows = static_cast<IT*>(f.unique_rows);
        Seg run = seg_combine(s_before, seg_combine(s_warp_pre[warp], lane_excl, chunk_log), chunk_log);
        const int B = 1 << f.batch_log;
        unsigned kb = k_first_prev;
        unsigned long long pw = 0;                       // up to four 16-bit positions on their way to perm
#pragma unroll 1
        for (int j = 0; j < n_mine; ++j) {
            const int i = i0 + j;
            const unsigned x = sorted[e0 + j];
            const unsigned k = x >> 16;
            const unsigned ka = j + 1 < n_mine ? sorted[e0 + j + 1] >> 16 : (j + 1 < ng ? 0xFFFFFFFFu : k_last_next);
            pw |= (unsigned long long)(x & 0xFFFFu) << (16 * (j & 3));
            if ((j & 3) == 3 || j == n_mine - 1) {
                // i0 is a multiple of ng: with ng a multiple of four this is one aligned 8-byte store
                if ((ng & 3) == 0) {
                    *reinterpret_cast<unsigned long long*>(f.perm + (i & ~3)) = pw;
                } else {
                    for (int q = 0; q <= (j & 3); ++q) f.perm[(i0 + (j & ~3)) + q] = (unsigned short)(pw >> (16 * q));
                }
                pw = 0;
            }
            if (kb != k) run.lh = i;
            if (ka != k) {
                // the row k ends here: rank u among the named rows, entries [run.lh, i]
                const int u = run.nt, cc = i - run.lh + 1;
                f.urec[u] = (k << 16) | (unsigned)run.lh;
                if (unique_rows) unique_rows[u] = (IT)k;
                if (f.counts_out) f.counts_out[u] = cc;
                if (cc > (1 << chunk_log))           // a6: a heavy row becomes chunk items and a combine tree
                    f.heavy[run.nh] = HeavyInfo{(int)k, run.nc, run.nu, (int)(heavy_shape(cc, chunk_log) & 0xFFFFu), run.lh, cc, {0, 0}};
                // Light work items: a row belongs to the item its first unit falls into, item b = units
                // [b * B, b * B + B).  The row whose units reach or cross the start of an item names the
                // next row as that item's first (an item no row starts in gets the same first row as the
                // item after it, and is empty).
                const int p0 = run.un, p1 = run.un + row_units(cc, 1 << chunk_log);
                if (u == 0) f.bfirst[0] = 0;
                for (int b = (p0 >> f.batch_log) + 1; b * B <= p1; ++b) f.bfirst[b] = u + 1;
                run.nt += 1;
                seg_add_row(run, cc, chunk_log);
            }
            kb = k;
        }
    }
    if (rank == 0 && threadIdx.x == 0) {
        const Seg g = s_grand;
        f.urec[g.nt] = (unsigned)n_valid;
        f.bfirst[g.un > 0 ? ((g.un - 1) >> f.batch_log) + 1 : 0] = g.nt;
        hdr->n_valid = n_valid;
        hdr->n_unique = g.nt;
        hdr->n_heavy = g.nh;
        hdr->n_chunks = g.nc;
        hdr->n_upper = g.nu;
        hdr->max_segment = g.mx;
        hdr->n_batches = g.un > 0 ? ((g.un - 1) >> f.batch_log) + 1 : 0;
        const long long bad = (long long)f.n_total - n_valid;
        hdr->n_bad = (unsigned long long)bad;
        if (bad) raise_status(hdr, DST_ERR_INDEX_OUT_OF_RANGE);
        if (f.result) {
            f.result->n_unique = g.nt;
            f.result->n_out_of_range = bad;
            f.result->max_segment = g.mx;
        }
    }
    cluster.sync();       // every table and the header have landed; nobody reads a peer's shared memory after this
    if (rank == 0 && threadIdx.x == 0) {
        __threadfence();
        *reinterpret_cast<volatile int*>(&hdr->tables_ready) = 1;
    }
}

cudaError_t launch_front_cluster(int index_type, const FrontParams& p, cudaStream_t stream) {
    FrontArgs f;
    f.P = p.P; f.hdr = p.hdr; f.tab = p.tab; f.perm = reinterpret_cast<unsigned short*>(p.perm); f.heavy = p.heavy;
    f.unique_rows = p.unique_rows; f.counts_out = p.counts_out; f.result = p.result;
    f.urec = p.urec; f.bfirst = p.bfirst;
    f.node_cnt = p.node_cnt; f.vocab = p.vocab; f.n_total = p.n_total;
    f.nodecnt_words = p.nodecnt_words;
    f.batch_log = 0;
    while ((2 << f.batch_log) <= p.batch_units) ++f.batch_log;            // items of 2^batch_log units: the power of two below batch_units
    f.bitmap = p.bitmap; f.bitmap_words = p.bitmap_words;
    f.chunk_log = 0;
    while ((1 << f.chunk_log) < p.chunk) ++f.chunk_log;
    if ((1 << f.chunk_log) != p.chunk) return cudaErrorInvalidValue;      // chunk lengths are powers of two
    const int per_warp = (p.n_total + kClusterCtas * kFrontWarps - 1) / (kClusterCtas * kFrontWarps);
    f.lw = (per_warp + 31) / 32 * 32;
    if (f.lw < 32) f.lw = 32;
    if (f.lw > 32 * kFrontGroups || (long long)p.bitmap_words * 32 < p.vocab) return cudaErrorInvalidValue;
    const size_t S = size_t(32) * f.lw;
    const size_t smem = S * 10 + size_t(32) * p.bitmap_words;   // S is a multiple of 1024: the byte map stays 16-byte aligned
    static SmemOptIn opt_in[2];
    const cudaError_t e = index_type == DST_I64 ? ensure_dynamic_smem(k_front_cluster<long long>, smem, opt_in[1])
                                                : ensure_dynamic_smem(k_front_cluster<int>, smem, opt_in[0]);
    if (e != cudaSuccess) return e;
    if (index_type == DST_I64)
        return launch_pdl(k_front_cluster<long long>, dim3(kClusterCtas), dim3(kFrontThreads), smem, stream, f);
    return launch_pdl(k_front_cluster<int>, dim3(kClusterCtas), dim3(kFrontThreads), smem, stream, f);
}

}  // namespace dst
