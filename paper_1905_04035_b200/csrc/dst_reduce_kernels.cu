// Row side of densify: segmented row reduction, fused dense add, one streaming write.
//
//   out[v, :] = sum_{j in segment(v)} values[perm[j], :]  +  dense_in[v, :]
//
// (Section 4 / Listing 1 of the paper: IndexedSlices -> dense; Algorithm 1 line 4:
// the dense tensors are then summed.)  This kernel moves practically all bytes of
// the operation.  It is HBM-bound: every value row, every dense_in row and every
// out row crosses the memory bus exactly once; no tensor cores are involved.
//
// Structure: persistent CTAs of kPipeWarps independent warps.  Each warp owns a small ring
// of shared-memory slots and streams "units" (one source row of one column block each)
// through it: lane 0 issues one bulk asynchronous copy (cp.async.bulk, completion on an
// mbarrier) per unit, up to n_slots ahead of the unit the warp is adding into its fp32
// registers, so the bytes in flight are set by shared memory, not by registers.  The
// units of a work item are laid out flat across the lanes (value rows of a segment, then
// the unit that closes the output row with its dense_in row), so the copies of one
// output row overlap with those of its neighbours.  The warp that read a slot is the
// one that refills it, so only "full" barriers are needed.
// Work items:
//   chunk items   `chunk` consecutive entries of a heavy row's segment -> fp32 partial row;
//                 partials are combined by a fixed fan-in tree whose nodes are
//                 evaluated by whichever CTA arrives last (children always summed
//                 in index order, so the result does not depend on timing)
//   row batches   consecutive output rows that are not heavy, about batch_units units' worth
// Rows wider than one slot are processed as independent column blocks.
//
// Small inputs (the paper's per-worker batches against a vocabulary of tens of thousands of rows):
// most output rows are named by nobody and only need their dense_in row, and the index work is a
// latency chain.  There the kernel is launched beside the index cluster and starts with
//   copy items    a few consecutive output rows, those a bitmap marks as named left out;
// when the index cluster flags its tables complete the warps turn to the chunk items and row
// batches (which then list named rows only), and finish whatever copy items are left.  The two
// kinds of item write disjoint rows, so no order between them is needed.
#include <type_traits>

#include "dst_common.cuh"

namespace dst {

// ---- typed column-group access ------------------------------------------------
template <int VC> struct Acc { float x[VC]; };

template <int VC> __device__ __forceinline__ void zero(Acc<VC>& a) {
#pragma unroll
    for (int i = 0; i < VC; ++i) a.x[i] = 0.f;
}
template <int VC> __device__ __forceinline__ void add(Acc<VC>& a, const Acc<VC>& b) {
#pragma unroll
    for (int i = 0; i < VC; ++i) a.x[i] += b.x[i];
}

__device__ __forceinline__ void unpack_bf16x2(unsigned w, float& lo, float& hi) {
    lo = __uint_as_float(w << 16);
    hi = __uint_as_float(w & 0xFFFF0000u);
}
__device__ __forceinline__ unsigned pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<unsigned*>(&t);
}

// The square root and the quotient of Adam's step, 32 of each per lane and output row: the IEEE-rounded ones
// cost about twenty instructions apiece and made the step instruction-bound; these are good to two units in
// the last place, a hundredth of what the step's own rounding allows for.
__device__ __forceinline__ float fast_sqrt(float x) {
    float r;
    asm("sqrt.approx.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

// VC consecutive elements at p (shared or global memory, generic address) -> fp32
__device__ __forceinline__ void load_elems(const float* p, Acc<4>& a) {
    float4 t = *reinterpret_cast<const float4*>(p);
    a.x[0] = t.x; a.x[1] = t.y; a.x[2] = t.z; a.x[3] = t.w;
}
__device__ __forceinline__ void load_elems(const float* p, Acc<8>& a) {
    float4 t = *reinterpret_cast<const float4*>(p);
    float4 u = *(reinterpret_cast<const float4*>(p) + 1);
    a.x[0] = t.x; a.x[1] = t.y; a.x[2] = t.z; a.x[3] = t.w;
    a.x[4] = u.x; a.x[5] = u.y; a.x[6] = u.z; a.x[7] = u.w;
}
__device__ __forceinline__ void load_elems(const __nv_bfloat16* p, Acc<8>& a) {
    uint4 t = *reinterpret_cast<const uint4*>(p);
    unpack_bf16x2(t.x, a.x[0], a.x[1]); unpack_bf16x2(t.y, a.x[2], a.x[3]);
    unpack_bf16x2(t.z, a.x[4], a.x[5]); unpack_bf16x2(t.w, a.x[6], a.x[7]);
}
__device__ __forceinline__ void load_elems(const __nv_bfloat16* p, Acc<4>& a) {
    uint2 t = *reinterpret_cast<const uint2*>(p);
    unpack_bf16x2(t.x, a.x[0], a.x[1]); unpack_bf16x2(t.y, a.x[2], a.x[3]);
}
// the dense result is written once and not read again: streaming stores
__device__ __forceinline__ void store_out(float* p, const Acc<4>& a) {
    __stcs(reinterpret_cast<float4*>(p), make_float4(a.x[0], a.x[1], a.x[2], a.x[3]));
}
__device__ __forceinline__ void store_out(float* p, const Acc<8>& a) {
    __stcs(reinterpret_cast<float4*>(p), make_float4(a.x[0], a.x[1], a.x[2], a.x[3]));
    __stcs(reinterpret_cast<float4*>(p) + 1, make_float4(a.x[4], a.x[5], a.x[6], a.x[7]));
}
__device__ __forceinline__ void store_out(__nv_bfloat16* p, const Acc<8>& a) {
    __stcs(reinterpret_cast<uint4*>(p), make_uint4(pack_bf16x2(a.x[0], a.x[1]), pack_bf16x2(a.x[2], a.x[3]),
                                                   pack_bf16x2(a.x[4], a.x[5]), pack_bf16x2(a.x[6], a.x[7])));
}
__device__ __forceinline__ void store_out(__nv_bfloat16* p, const Acc<4>& a) {
    __stcs(reinterpret_cast<uint2*>(p), make_uint2(pack_bf16x2(a.x[0], a.x[1]), pack_bf16x2(a.x[2], a.x[3])));
}
// partial rows: written by one CTA, read by another through L2
template <int VC> __device__ __forceinline__ void store_partial(float* p, const Acc<VC>& a) {
#pragma unroll
    for (int i = 0; i < VC; i += 4)
        __stcg(reinterpret_cast<float4*>(p + i), make_float4(a.x[i], a.x[i + 1], a.x[i + 2], a.x[i + 3]));
}
template <int VC> __device__ __forceinline__ void load_partial(const float* p, Acc<VC>& a) {
#pragma unroll
    for (int i = 0; i < VC; i += 4) {
        float4 t = __ldcg(reinterpret_cast<const float4*>(p + i));
        a.x[i] = t.x; a.x[i + 1] = t.y; a.x[i + 2] = t.z; a.x[i + 3] = t.w;
    }
}

// position in the virtual concatenation -> address of that value row
template <typename VT>
__device__ __forceinline__ const VT* resolve_row(const MainArgs& a, unsigned p) {
    int lo = 0;
    if (a.R > 1) {
        int hi = a.R - 1;                       // largest r with tab[r].start <= p
        while (lo < hi) {
            int mid = (lo + hi + 1) >> 1;
            if (__ldg(&a.tab[mid].start) <= (long long)p) lo = mid; else hi = mid - 1;
        }
    }
    const VT* base = reinterpret_cast<const VT*>(
        __ldg(reinterpret_cast<const unsigned long long*>(&a.tab[lo].values)));
    long long local = (long long)p - __ldg(&a.tab[lo].start);
    return base + local * a.d;
}

// ---- mbarrier / bulk-copy primitives (shared::cta addresses) -----------------------
__device__ __forceinline__ unsigned smem_addr(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned bar) {
    asm volatile("{ .reg .b64 st; mbarrier.arrive.shared::cta.b64 st, [%0]; }" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned bar, unsigned bytes) {
    asm volatile("{ .reg .b64 st; mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1; }" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up when the limit is reached or another thread has given up.
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity, volatile int* abort_flag,
                                          long long limit = kWaitCycles) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long start = clock64();
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag || clock64() - start > limit) return false;
    }
}
// global -> this CTA's shared memory, 16-byte aligned on both sides, bytes % 16 == 0
__device__ __forceinline__ void bulk_load(unsigned dst_smem, const void* src, unsigned bytes, unsigned bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// ---- per-warp slot ring --------------------------------------------------------------
enum : int {
    kUnitAdd = 1,        // slot holds a value row: add it
    kUnitFinal = 2,      // finish output row y (slot holds its dense_in row unless there is no dense_in)
    kUnitCopy = 4,       // with kUnitFinal: nobody names the row, out = dense_in bit for bit
    kUnitChunkEnd = 8,   // last entry of chunk y: store the partial row, climb the tree
    kUnitPoll = 16,      // (copy items) ask now whether the index cluster has finished; the answer is looked at after the item
    kUnitState1 = 32,    // optimizer step: the slot holds the row of state1 (momentum buffer / Adam's m) of output row y
    kUnitState2 = 64,    // optimizer step: ... of state2 (Adam's v)
    kUnitAddDense = 128  // slot holds a row of a dense partner (dense_in's type): add it
};

constexpr int kTabCache = 64;       // slices whose table is copied into shared memory
constexpr int kHeavyCache = 1024;   // heavy rows whose first chunk id is copied into shared memory
constexpr int kNamedWords = 65536 / 32;   // the overlapped path is for vocabularies of at most 65536 rows
template <bool OVERLAP>
struct CtaTables {
    long long start[kTabCache];
    unsigned long long values[kTabCache];
    int chunk_base[kHeavyCache];
    int n_heavy;
    int state;                     // overlapped path: 0 tables not loaded, 1 a warp is loading them, 2 loaded
    unsigned named[OVERLAP ? kNamedWords : 1];   // overlapped path: bit v set when some valid entry names row v
    // (only there: the other variants size their CTAs per SM by shared memory, and 8 KB more would cost the
    // bf16 kernel its fourth CTA)
};

// A block of at most 32 units, one per lane.
struct UnitBlock {
    const void* src;     // first byte to copy (nullptr: nothing to copy)
    unsigned bytes;
    int kind;
    int y;               // output row (kUnitFinal) or chunk id (kUnitChunkEnd)
};

// OPT: 0 writes the accumulated gradient; otherwise `out` holds an fp32 weight that takes an optimizer step
// with the gradient g = grad_scale * (dense_in + sum of value rows), which is never written:
//   kOptSgd       out <- out - lr * g
//   kOptMomentum  b <- mu * b + g;  out <- out - lr * b                                  (b: state1)
//   kOptAdam      m <- beta1 * m + (1 - beta1) * g;  v <- beta2 * v + (1 - beta2) * g * g  (m: state1, v: state2)
//                 out <- out - lr * (m / (1 - beta1^t)) / (sqrt(v / (1 - beta2^t)) + eps)
// The rows of the state ride the ring as further closing units of an output row (v, then m, then the
// weight), each read once and written once.  value rows and dense_in have one type (fp32 or bf16);
// weight and state are fp32.
// OVERLAP: the kernel runs beside the index cluster and starts with copy items (small inputs, see above).
enum : int { kOptNone = 0, kOptSgd = 1, kOptMomentum = 2, kOptAdam = 3 };

template <typename VT, typename OT, int K, int OPT = kOptNone, bool OVERLAP = false>
struct WarpPipe {
    static constexpr bool APPLY = OPT != kOptNone;
    using WT = std::conditional_t<APPLY, float, OT>;     // what `out` holds
    static constexpr int VC = 16 / sizeof(VT);     // columns per 16-byte group of a value row
    const MainArgs& a;
    const int lane;
    const unsigned ring;      // shared address of this warp's first slot
    const unsigned bars;      // shared address of this warp's first mbarrier (one per slot)
    char* const ring_ptr;     // generic address of the first slot
    volatile int* const abort_flag;
    CtaTables<OVERLAP>& tabs; // this CTA's shared copies of the slice table and of the heavy rows' first chunk ids
    HeavyInfo cur_heavy;      // the heavy row of the chunk item being processed
    int islot;                // slot the next issued unit goes to
    int cslot;                // slot of the next unit to consume
    unsigned cphase;          // bit s: parity to wait for on slot s
    unsigned issued_mask;     // slots with a copy that may still be in flight
    int polled;               // lane 0: tables_ready as last asked for (kUnitPoll)
    int ns;                   // slots of the ring in use (<= a.n_slots, the slots there are); changed only when the ring is empty
    Acc<VC> aux[K];           // kOptAdam: sqrt(vhat) + eps of the row being closed, between its v unit and its m unit

    __device__ WarpPipe(const MainArgs& args, unsigned ring_addr, unsigned bar_addr, char* ring_generic, volatile int* ab,
                        CtaTables<OVERLAP>& t)
        : a(args), lane(lane_id()), ring(ring_addr), bars(bar_addr), ring_ptr(ring_generic), abort_flag(ab), tabs(t), islot(0),
          cslot(0), cphase(0u), issued_mask(0u), polled(0), ns(args.n_slots) {}

    __device__ __forceinline__ int col(int k) const { return (k * 32 + lane) * VC; }

    // The optimizer's arithmetic on one column group.  `g` comes in as the raw sum (dense_in + value rows).
    // state unit of kOptMomentum: s holds b; leaves the new b in s and in g (what the weight unit subtracts)
    __device__ __forceinline__ void step_momentum(Acc<VC>& g, Acc<VC>& s) const {
#pragma unroll
        for (int i = 0; i < VC; ++i) { s.x[i] = fmaf(a.opt_a, s.x[i], a.grad_scale * g.x[i]); g.x[i] = s.x[i]; }
    }
    // first state unit of kOptAdam: s holds v; leaves the new v in s, the scaled gradient in g, the denominator in den
    __device__ __forceinline__ void step_adam_v(Acc<VC>& g, Acc<VC>& s, Acc<VC>& den) const {
#pragma unroll
        for (int i = 0; i < VC; ++i) {
            g.x[i] = a.grad_scale * g.x[i];
            s.x[i] = fmaf(a.opt_b, s.x[i], (1.f - a.opt_b) * (g.x[i] * g.x[i]));
            den.x[i] = fast_sqrt(s.x[i] * a.opt_bc2) + a.opt_eps;
        }
    }
    // second state unit of kOptAdam: s holds m; leaves the new m in s and the bias-corrected step direction in g
    __device__ __forceinline__ void step_adam_m(Acc<VC>& g, Acc<VC>& s, const Acc<VC>& den) const {
#pragma unroll
        for (int i = 0; i < VC; ++i) {
            s.x[i] = fmaf(a.opt_a, s.x[i], (1.f - a.opt_a) * g.x[i]);
            g.x[i] = __fdividef(s.x[i] * a.opt_bc1, den.x[i]);
        }
    }
    // the weight unit: w holds the weight row; g what the state units left (kOptSgd: the raw sum)
    __device__ __forceinline__ void step_weight(const Acc<VC>& g, Acc<VC>& w) const {
#pragma unroll
        for (int i = 0; i < VC; ++i) w.x[i] = fmaf(-a.lr, OPT == kOptSgd ? a.grad_scale * g.x[i] : g.x[i], w.x[i]);
    }
    // The units that close an output row, in ring order: its dense_in row (OPT: one more row to add), then,
    // with an optimizer, Adam's v row, the m / momentum row and last the weight row.
    // There may be several dense partners (one per rank of the paper's Fig. 3b: every rank's projection gradient);
    // each one's row of an output row is read once, on the way to that output row.
    __device__ __forceinline__ int n_closing() const {
        if constexpr (!APPLY) return a.n_dense > 1 ? a.n_dense : 1;
        return a.n_dense + (OPT == kOptAdam ? 2 : (OPT == kOptMomentum ? 1 : 0)) + 1;
    }
    __device__ __forceinline__ const OT* dense_row_of(int which, long long at) const {
        return static_cast<const OT*>(which == 0 ? a.dense_in : a.dense_more[which - 1]) + at;
    }
    __device__ __forceinline__ void closing_unit(UnitBlock& b, int c, long long at, long long wcols, bool named) const {
        const unsigned dbytes = (unsigned)(wcols * (long long)sizeof(OT));
        if constexpr (APPLY) {
            const unsigned fbytes = (unsigned)(wcols * 4);
            if (c < a.n_dense) { b.src = dense_row_of(c, at); b.bytes = dbytes; b.kind = kUnitAddDense; return; }
            c -= a.n_dense;
            if constexpr (OPT == kOptAdam) {
                if (c == 0) { b.src = static_cast<const float*>(a.state2) + at; b.bytes = fbytes; b.kind = kUnitState2; return; }
                --c;
            }
            if constexpr (OPT == kOptAdam || OPT == kOptMomentum) {
                if (c == 0) { b.src = static_cast<const float*>(a.state1) + at; b.bytes = fbytes; b.kind = kUnitState1; return; }
                --c;
            }
            b.src = static_cast<const float*>(a.out) + at; b.bytes = fbytes; b.kind = kUnitFinal;
        } else if (c + 1 < a.n_dense) {
            b.src = dense_row_of(c, at); b.bytes = dbytes; b.kind = kUnitAddDense;
        } else {
            // the last (or only) partner closes the row; a row nobody names with one partner is its copy, bit for bit
            b.kind = kUnitFinal | ((named || a.n_dense > 1) ? 0 : kUnitCopy);
            if (a.n_dense > 0) { b.src = dense_row_of(a.n_dense - 1, at); b.bytes = dbytes; }
        }
    }
    __device__ __forceinline__ float* state_row(int which, int y, long long cb) const {
        return static_cast<float*>(which == 1 ? a.state1 : a.state2) + (long long)y * a.d + cb;
    }

    // unit j of the block goes into the next slot
    __device__ __forceinline__ void issue(const UnitBlock& b, int j) {
        if (lane == j) {                                  // the lane that holds the unit talks to the copy engine
            const unsigned bar = bars + 8u * (unsigned)islot;
            if (b.bytes) {
                mbar_arrive_expect_tx(bar, b.bytes);
                bulk_load(ring + (unsigned)islot * (unsigned)a.slot_bytes, b.src, b.bytes, bar);
            } else {
                mbar_arrive(bar);
            }
        }
        issued_mask |= 1u << islot;
        islot = islot + 1 == ns ? 0 : islot + 1;
    }

    // position in the virtual concatenation -> address of that value row (slice table in shared memory)
    __device__ __forceinline__ const VT* row_address(unsigned p) const {
        if (a.R > kTabCache) return resolve_row<VT>(a, p);
        int lo = 0, hi = a.R - 1;                  // largest r with start[r] <= p
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (tabs.start[mid] <= (long long)p) lo = mid; else hi = mid - 1;
        }
        return reinterpret_cast<const VT*>(tabs.values[lo]) + ((long long)p - tabs.start[lo]) * a.d;
    }

    __device__ __forceinline__ float* partial_row(int slot) const { return a.partials + (long long)slot * a.d; }

    // a plain copy of `bytes` bytes into the next slot (lane 0 talks to the copy engine)
    __device__ __forceinline__ void issue_plain(const void* src, unsigned bytes) {
        if (lane == 0) {
            const unsigned bar = bars + 8u * (unsigned)islot;
            mbar_arrive_expect_tx(bar, bytes);
            bulk_load(ring + (unsigned)islot * (unsigned)a.slot_bytes, src, bytes, bar);
        }
        issued_mask |= 1u << islot;
        islot = islot + 1 == ns ? 0 : islot + 1;
    }

    // acc = child[0] + child[1] + ... in index order.  fp32 value rows: a slot of the ring holds one
    // partial row, so the children stream through the ring like any other unit, n_slots copies in
    // flight, and the sum costs about one trip to memory however busy the memory system is.
    // bf16 value rows (slots half as wide as a partial row): direct loads, half of the column
    // groups at a time to save registers.
    // `n_extra` more fp32 rows are added after the children: the rows at element offset `extra_at` of the dense
    // partners (at the root of a heavy row).
    __device__ __forceinline__ bool sum_children(Acc<VC> (&acc)[K], int first_slot, int n_children, long long cb, int wcols,
                                                 int n_extra, long long extra_at) {
        if constexpr (sizeof(VT) == 4) {
            const int n = n_children + n_extra;
            auto source = [&](int c) {
                return c < n_children ? static_cast<const float*>(partial_row(first_slot + c) + cb)
                                      : reinterpret_cast<const float*>(dense_row_of(c - n_children, extra_at));
            };
            // the partial rows were written with ordinary stores; the copy engine reads them
            asm volatile("fence.proxy.async;" ::: "memory");
#pragma unroll
            for (int k = 0; k < K; ++k) zero(acc[k]);
            const unsigned bytes = (unsigned)wcols * 4u;
            int issued = 0;
            for (; issued < n && issued < ns; ++issued) issue_plain(source(issued), bytes);
            for (int c = 0; c < n; ++c) {
                if (!mbar_wait(bars + 8u * (unsigned)cslot, (cphase >> cslot) & 1u, abort_flag)) { give_up(); return false; }
                cphase ^= 1u << cslot;
                issued_mask &= ~(1u << cslot);
                const VT* sp = reinterpret_cast<const VT*>(ring_ptr + (size_t)cslot * a.slot_bytes);
                Acc<VC> v[K];
#pragma unroll
                for (int k = 0; k < K; ++k) {
                    const int cc = col(k);
                    zero(v[k]);
                    if (cc < wcols) load_elems(sp + cc, v[k]);
                }
#pragma unroll
                for (int k = 0; k < K; ++k) add(acc[k], v[k]);
                __syncwarp();
                cslot = cslot + 1 == ns ? 0 : cslot + 1;
                if (issued < n) { issue_plain(source(issued), bytes); ++issued; }
            }
            return true;
        }
        constexpr int KH = (sizeof(VT) == 2 && K >= 4) ? K / 2 : K;   // the bf16 variants run at 128 registers
        const int n = n_children;
#pragma unroll
        for (int h0 = 0; h0 < K; h0 += KH) {
#pragma unroll
            for (int k = 0; k < KH; ++k) zero(acc[h0 + k]);
            for (int c = 0; c < n; c += 2) {
                const float* pa = partial_row(first_slot + c) + cb;
                const float* pb = (c + 1 < n) ? partial_row(first_slot + c + 1) + cb : nullptr;
                Acc<VC> va[KH], vb[KH];
#pragma unroll
                for (int k = 0; k < KH; ++k) {
                    const int cc = col(h0 + k);
                    zero(va[k]); zero(vb[k]);
                    if (cc < wcols) {
                        load_partial(pa + cc, va[k]);
                        if (pb) load_partial(pb + cc, vb[k]);
                    }
                }
#pragma unroll
                for (int k = 0; k < KH; ++k) { add(acc[h0 + k], va[k]); add(acc[h0 + k], vb[k]); }
            }
        }
        return true;
    }

    // Heavy row that owns chunk cid: the last h with heavy[h].chunk_base <= cid.
    __device__ __forceinline__ int find_heavy(int cid) const {
        int lo = 0, hi = tabs.n_heavy;
        if (hi <= kHeavyCache) {                     // the first chunk ids are in shared memory
            --hi;
            while (lo < hi) {
                const int mid = (lo + hi + 1) >> 1;
                if (tabs.chunk_base[mid] <= cid) lo = mid; else hi = mid - 1;
            }
            return lo;
        }
        while (hi - lo > 1) {                        // all lanes probe at once
            const int step = (hi - lo + 31) / 32;
            const int idx = lo + lane * step;
            const bool le = idx < hi && __ldg(&a.heavy[idx].chunk_base) <= cid;
            const int t = __popc(__ballot_sync(0xFFFFFFFFu, le));      // lane 0 always qualifies
            lo += (t - 1) * step;
            hi = min(hi, lo + step);
        }
        return lo;
    }
    __device__ __forceinline__ ChunkDesc chunk_of(int cid) {
        const int h = find_heavy(cid);
        const HeavyInfo hi = a.heavy[h];
        cur_heavy = hi;
        const int k = cid - hi.chunk_base;
        return ChunkDesc{hi.row, hi.begin + k * a.chunk, min(a.chunk, hi.count - k * a.chunk), h};
    }

    // The chunk's sum is in acc: store it as a partial row and climb the combine tree while this
    // warp is the last child to arrive.
    __device__ bool finish_chunk(Acc<VC> (&acc)[K], int cid, int cblk) {
        const HeavyInfo hi = cur_heavy;
        const long long cb = (long long)cblk * a.W;
        const int wcols = (int)min((long long)a.W, a.d - cb);
        {
            float* pr = partial_row(cid) + cb;
#pragma unroll
            for (int k = 0; k < K; ++k) {
                const int c = col(k);
                if (c < wcols) store_partial(pr + c, acc[k]);
            }
        }
        unsigned* node_cnt = a.node_cnt + (size_t)cblk * (size_t)a.upper_max;
        int j = cid - hi.chunk_base;     // index inside the current level
        int n_level = hi.n_chunks;       // nodes on the current level
        int child_first = hi.chunk_base; // partial slot of node 0 of the current level
        int upper_off = 0;               // offset of the parent level inside this row's upper nodes
        while (true) {
            const int parent = j / kFanIn;
            const int n_parent = (n_level + kFanIn - 1) / kFanIn;
            const int n_children = min(kFanIn, n_level - parent * kFanIn);
            const int node = hi.upper_base + upper_off + parent;
            __threadfence();
            __syncwarp();
            int last = 0;
            if (lane == 0) last = atomicAdd(&node_cnt[node], 1u) == (unsigned)(n_children - 1);
            last = __shfl_sync(0xFFFFFFFFu, last, 0);
            if (!last) return true;
            __threadfence();
            const bool root = n_parent == 1;
            // fp32 rows in, fp32 dense rows: the root's dense row rides the ring behind the children
            constexpr bool kDenseInRing = sizeof(VT) == 4 && sizeof(OT) == 4;
            const long long row_at = (long long)hi.row * a.d + cb;
            const int in_ring = (kDenseInRing && root) ? a.n_dense : 0;
            if (!sum_children(acc, child_first + parent * kFanIn, n_children, cb, wcols, in_ring, row_at)) return false;
            if (root) {
                // The output may be the dense input itself, so the compiler keeps loads and stores in
                // program order: read the whole dense row first, then store, or every column group
                // pays its own trip to memory.
                if constexpr (APPLY) {
                    // weight and state rows straight from memory (heavy rows are few): all loads of a step first
                    float* wrow = static_cast<float*>(a.out) + (long long)hi.row * a.d + cb;
                    if constexpr (!kDenseInRing) {
                        for (int p = 0; p < a.n_dense; ++p) {
                            const OT* drow = dense_row_of(p, row_at);
                            Acc<VC> dn[K];
#pragma unroll
                            for (int k = 0; k < K; ++k) { zero(dn[k]); if (col(k) < wcols) load_elems(drow + col(k), dn[k]); }
#pragma unroll
                            for (int k = 0; k < K; ++k) add(acc[k], dn[k]);
                        }
                    }
                    if constexpr (OPT == kOptMomentum || OPT == kOptAdam) {
                        float* srow = state_row(OPT == kOptAdam ? 2 : 1, hi.row, cb);
                        Acc<VC> st[K];
#pragma unroll
                        for (int k = 0; k < K; ++k) { zero(st[k]); if (col(k) < wcols) load_elems(srow + col(k), st[k]); }
#pragma unroll
                        for (int k = 0; k < K; ++k) {
                            if constexpr (OPT == kOptAdam) step_adam_v(acc[k], st[k], aux[k]); else step_momentum(acc[k], st[k]);
                            if (col(k) < wcols) store_out(srow + col(k), st[k]);
                        }
                    }
                    if constexpr (OPT == kOptAdam) {
                        float* srow = state_row(1, hi.row, cb);
                        Acc<VC> st[K];
#pragma unroll
                        for (int k = 0; k < K; ++k) { zero(st[k]); if (col(k) < wcols) load_elems(srow + col(k), st[k]); }
#pragma unroll
                        for (int k = 0; k < K; ++k) {
                            step_adam_m(acc[k], st[k], aux[k]);
                            if (col(k) < wcols) store_out(srow + col(k), st[k]);
                        }
                    }
                    Acc<VC> wt[K];
#pragma unroll
                    for (int k = 0; k < K; ++k) { zero(wt[k]); if (col(k) < wcols) load_elems(wrow + col(k), wt[k]); }
#pragma unroll
                    for (int k = 0; k < K; ++k) {
                        step_weight(acc[k], wt[k]);
                        if (col(k) < wcols) store_out(wrow + col(k), wt[k]);
                    }
                    return true;
                }
                // The output may be a dense partner itself, so the compiler keeps loads and stores in program
                // order: read a whole dense row first, then store, or every column group pays its own trip.
                OT* out = static_cast<OT*>(a.out) + row_at;
                constexpr int KH = (sizeof(VT) == 2 && K >= 4) ? K / 2 : K;
                const int direct = kDenseInRing ? 0 : a.n_dense;       // partners not yet added
#pragma unroll
                for (int h0 = 0; h0 < K; h0 += KH) {
                    for (int p = 0; p < direct; ++p) {
                        const OT* drow = dense_row_of(p, row_at);
                        Acc<VC> dn[KH];
#pragma unroll
                        for (int k = 0; k < KH; ++k) {
                            const int c = col(h0 + k);
                            zero(dn[k]);
                            if (c < wcols) load_elems(drow + c, dn[k]);
                        }
#pragma unroll
                        for (int k = 0; k < KH; ++k) add(acc[h0 + k], dn[k]);
                    }
#pragma unroll
                    for (int k = 0; k < KH; ++k) {
                        const int c = col(h0 + k);
                        if (c < wcols) store_out(out + c, acc[h0 + k]);
                    }
                }
                return true;
            }
            float* pr = partial_row(a.chunk_max + node) + cb;
#pragma unroll
            for (int k = 0; k < K; ++k) {
                const int c = col(k);
                if (c < wcols) store_partial(pr + c, acc[k]);
            }
            child_first = a.chunk_max + hi.upper_base + upper_off;
            upper_off += n_parent;
            j = parent;
            n_level = n_parent;
        }
    }

    __device__ __forceinline__ void give_up() const {
        raise_status(a.hdr, DST_ERR_TIMEOUT);
        *abort_flag = 1;
    }

    // Stream the n units of a block (lane j holds unit j) through the ring: up to n_slots copies in
    // flight, consumed in order.  Returns false when a wait gave up.
    __device__ bool run_block(Acc<VC> (&acc)[K], const UnitBlock& b, int n, int cblk) {
        const long long cb = (long long)cblk * a.W;
        const int wcols = (int)min((long long)a.W, a.d - cb);
        WT* const out = static_cast<WT*>(a.out);
        const int ahead = min(n, ns);
        for (int j = 0; j < ahead; ++j) issue(b, j);
        for (int j = 0; j < n; ++j) {
            const int kind = __shfl_sync(0xFFFFFFFFu, b.kind, j);
            const int y = __shfl_sync(0xFFFFFFFFu, b.y, j);
            if constexpr (OVERLAP)
                if ((kind & kUnitPoll) && lane == 0) polled = *reinterpret_cast<volatile int*>(&a.hdr->tables_ready);
            if (!mbar_wait(bars + 8u * (unsigned)cslot, (cphase >> cslot) & 1u, abort_flag)) { give_up(); return false; }
            cphase ^= 1u << cslot;
            issued_mask &= ~(1u << cslot);
            const char* sp = ring_ptr + (size_t)cslot * a.slot_bytes;
            if (kind & kUnitAdd) {
                // A block of full width (the usual case) takes plain loads: one predicate and eight cleared registers
                // per column group, in every unit, were a tenth of the bf16 kernel's instructions.  Only here, where
                // most units pass, and not in the optimizer kernels: the same split at the closing units, or in the
                // Adam kernel (200 registers as it is), made those slower.
                if (OPT == kOptNone && wcols == K * 32 * VC) {
                    Acc<VC> v[K];
#pragma unroll
                    for (int k = 0; k < K; ++k) load_elems(reinterpret_cast<const VT*>(sp) + col(k), v[k]);
#pragma unroll
                    for (int k = 0; k < K; ++k) add(acc[k], v[k]);
                } else {
#pragma unroll
                    for (int k = 0; k < K; ++k) {
                        const int c = col(k);
                        if (c < wcols) { Acc<VC> v; load_elems(reinterpret_cast<const VT*>(sp) + c, v); add(acc[k], v); }
                    }
                }
            }
            if (kind & kUnitAddDense) {
                Acc<VC> v[K];
#pragma unroll
                for (int k = 0; k < K; ++k) {
                    const int c = col(k);
                    zero(v[k]);
                    if (c < wcols) load_elems(reinterpret_cast<const OT*>(sp) + c, v[k]);
                }
#pragma unroll
                for (int k = 0; k < K; ++k) add(acc[k], v[k]);
            }
            if constexpr (OPT == kOptMomentum || OPT == kOptAdam) {
                if (kind & (kUnitState1 | kUnitState2)) {
                    // the slot holds a row of optimizer state: update it, keep what the next closing unit needs
                    float* srow = state_row((kind & kUnitState1) ? 1 : 2, y, cb);
                    Acc<VC> st[K];
#pragma unroll
                    for (int k = 0; k < K; ++k) {
                        const int c = col(k);
                        zero(st[k]);
                        if (c < wcols) load_elems(reinterpret_cast<const float*>(sp) + c, st[k]);
                    }
#pragma unroll
                    for (int k = 0; k < K; ++k) {
                        const int c = col(k);
                        if constexpr (OPT == kOptMomentum) {
                            step_momentum(acc[k], st[k]);
                        } else {
                            if (kind & kUnitState2) step_adam_v(acc[k], st[k], aux[k]); else step_adam_m(acc[k], st[k], aux[k]);
                        }
                        if (c < wcols) store_out(srow + c, st[k]);
                    }
                }
            }
            if (kind & kUnitFinal) {
                WT* orow = out + (long long)y * a.d + cb;
                Acc<VC> dn[K];                            // the dense row first, all of it, then the stores
#pragma unroll
                for (int k = 0; k < K; ++k) {
                    const int c = col(k);
                    zero(dn[k]);
                    if ((APPLY || a.n_dense > 0) && c < wcols) load_elems(reinterpret_cast<const WT*>(sp) + c, dn[k]);
                }
#pragma unroll
                for (int k = 0; k < K; ++k) {
                    const int c = col(k);
                    if constexpr (APPLY) {
                        step_weight(acc[k], dn[k]);       // the slot holds the weight row
                    } else {
                        if (!(kind & kUnitCopy)) add(dn[k], acc[k]);
                    }
                    if (c < wcols) store_out(orow + c, dn[k]);
                    zero(acc[k]);
                }
            }
            __syncwarp();                                 // every lane has read the slot
            cslot = cslot + 1 == ns ? 0 : cslot + 1;
            if (j + ns < n) issue(b, j + ns);   // refill it
            if (kind & kUnitChunkEnd) {
                if (!finish_chunk(acc, y, cblk)) return false;
#pragma unroll
                for (int k = 0; k < K; ++k) zero(acc[k]);
            }
        }
        return true;
    }

    __device__ bool do_chunk(int cid, int cblk) {
        const ChunkDesc cd = chunk_of(cid);
        const long long cb = (long long)cblk * a.W;
        const unsigned bytes = (unsigned)(min((long long)a.W, a.d - cb) * (long long)sizeof(VT));
        Acc<VC> acc[K];
#pragma unroll
        for (int k = 0; k < K; ++k) zero(acc[k]);
        for (int base = 0; base < cd.len; base += 32) {
            const int q = base + lane;
            UnitBlock b{nullptr, 0u, 0, cid};
            if (q < cd.len) {
                const unsigned p = a.compact ? reinterpret_cast<const unsigned short*>(a.perm)[cd.begin + q] : a.perm[cd.begin + q];
                if (p < (unsigned)a.n_total) { b.src = row_address(p) + cb; b.bytes = bytes; b.kind = kUnitAdd; }
                if (q == cd.len - 1) b.kind |= kUnitChunkEnd;
            }
            if (!run_block(acc, b, min(32, cd.len - base), cblk)) return false;
        }
        return true;
    }

    // A batch of consecutive output rows: their entries and their closing units, flattened
    __device__ bool do_rows(int batch, int cblk) {
        int v0, nrows;                                    // first row (compact: its rank among the named rows), rows
        if (a.compact) {
            const int* first = reinterpret_cast<const int*>(a.batches);
            v0 = first[batch];
            nrows = min(first[batch + 1] - v0, 31);
            if (nrows <= 0) return true;                  // no row starts in this batch
        } else {
            const int2 bt = a.batches[batch];
            if (bt.y == 0) return true;
            v0 = bt.x - 1;
            nrows = min(bt.y - bt.x + 1, 31);
        }
        const long long cb = (long long)cblk * a.W;
        const long long wcols = min((long long)a.W, a.d - cb);
        int o = 0, row = v0 + lane;
        if (a.compact) {
            if (lane <= nrows) {
                const unsigned rec = a.urec[v0 + lane];
                o = (int)(rec & 0xFFFFu); row = (int)(rec >> 16);     // (the word after the last row: the number of entries)
            }
        } else {
            if (lane <= nrows) o = a.offsets[v0 + lane];
        }
        const int o_next = __shfl_down_sync(0xFFFFFFFFu, o, 1);
        const int cnt = lane < nrows ? o_next - o : 0;
        const int nunits = (lane < nrows && cnt <= a.chunk) ? cnt + n_closing() : 0;   // heavy rows belong to the chunk items
        int incl = nunits;
#pragma unroll
        for (int s = 1; s < 32; s <<= 1) {
            int t = __shfl_up_sync(0xFFFFFFFFu, incl, s);
            if (lane >= s) incl += t;
        }
        const int total = __shfl_sync(0xFFFFFFFFu, incl, 31);
        Acc<VC> acc[K];
#pragma unroll
        for (int k = 0; k < K; ++k) zero(acc[k]);
        for (int base = 0; base < total; base += 32) {
            const int q = base + lane;
            int i = 0;                                   // row of unit q: rows whose units all come before q
#pragma unroll
            for (int step = 16; step > 0; step >>= 1)
                if (__shfl_sync(0xFFFFFFFFu, incl, i + step - 1) <= q) i += step;
            i = min(i, 31);
            const int e = q - (__shfl_sync(0xFFFFFFFFu, incl, i) - __shfl_sync(0xFFFFFFFFu, nunits, i));
            const int ci = __shfl_sync(0xFFFFFFFFu, cnt, i);
            const int oi = __shfl_sync(0xFFFFFFFFu, o, i);
            const int vi = __shfl_sync(0xFFFFFFFFu, row, i);
            UnitBlock b{nullptr, 0u, 0, vi};
            if (q < total) {
                if (e < ci) {
                    const unsigned p = a.compact ? reinterpret_cast<const unsigned short*>(a.perm)[oi + e] : a.perm[oi + e];
                    if (p < (unsigned)a.n_total) {
                        b.src = row_address(p) + cb;
                        b.bytes = (unsigned)(wcols * (long long)sizeof(VT));
                        b.kind = kUnitAdd;
                    }
                } else {
                    closing_unit(b, e - ci, (long long)b.y * a.d + cb, wcols, ci != 0);
                }
            }
            if (!run_block(acc, b, min(32, total - base), cblk)) return false;
        }
        return true;
    }

    // A few consecutive output rows that only need their dense_in row (or zeros; APPLY: the dense part of
    // the step): the rows of the item that the bitmap does not mark as named.
    __device__ bool do_copy(unsigned item) {
        const int groups = (a.vocab + a.copy_rows - 1) / a.copy_rows;
        const int cblk = (int)(item / (unsigned)groups);
        const int r0 = ((int)item - cblk * groups) * a.copy_rows;      // copy_rows divides 32: the rows share one bitmap word
        const int n_valid = min(a.copy_rows, a.vocab - r0);
        const unsigned span = n_valid >= 32 ? 0xFFFFFFFFu : ((1u << n_valid) - 1u);
        const unsigned want = ~(tabs.named[r0 >> 5] >> (r0 & 31)) & span;
        const int n = __popc(want);
        if (n == 0) {                                     // every row of the item is named: nothing to copy
            if (lane == 0) polled = *reinterpret_cast<volatile int*>(&a.hdr->tables_ready);
            return true;
        }
        const long long cb = (long long)cblk * a.W;
        const long long wcols = min((long long)a.W, a.d - cb);
        Acc<VC> acc[K];
#pragma unroll
        for (int k = 0; k < K; ++k) zero(acc[k]);
        const int per_row = n_closing();
        const int total = n * per_row;
        for (int base = 0; base < total; base += 32) {
            const int q = base + lane;
            UnitBlock b{nullptr, 0u, 0, 0};
            if (q < total) {
                b.y = r0 + (int)__fns(want, 0u, q / per_row + 1);          // the (q / per_row + 1)-th row that is wanted
                closing_unit(b, q % per_row, (long long)b.y * a.d + cb, wcols, false);
            }
            // the unit during which the last copies of the item are issued asks for the flag
            if (base + 32 >= total && q == max(base, total - 1 - ns)) b.kind |= kUnitPoll;
            if (!run_block(acc, b, min(32, total - base), cblk)) return false;
        }
        return true;
    }

    // Work items handed out through one counter.  While plenty of items are left the next one is
    // claimed one item ahead, so its number is back from the counter before it is needed.  Near the
    // end that would leave some warps with an extra item in hand while others have run dry: then a
    // warp claims only when it is out of work.
    struct Claim {
        unsigned* counter;
        unsigned n_items, base, item, pending;
        bool lazy;
    };
    // static_first: the first item of a warp is its own number (no traffic on the counter while the
    // whole grid starts up) and the counter hands out the numbers after those
    __device__ __forceinline__ void claim_begin(Claim& c, unsigned* counter, unsigned n_items, bool static_first) {
        const unsigned n_warps = gridDim.x * (unsigned)kPipeWarps;
        c.counter = counter; c.n_items = n_items; c.pending = 0xFFFFFFFFu;
        c.lazy = n_items < 2u * n_warps;
        if (static_first) {
            c.base = n_warps;
            c.item = blockIdx.x * (unsigned)kPipeWarps + (unsigned)warp_id();
        } else {
            c.base = 0;
            unsigned it = 0;
            if (lane == 0) it = atomicAdd(counter, 1u);
            c.item = __shfl_sync(0xFFFFFFFFu, it, 0);
        }
        if (lane == 0 && c.item < n_items && !c.lazy) c.pending = c.base + atomicAdd(counter, 1u);
    }
    __device__ __forceinline__ void claim_next(Claim& c) {
        const unsigned n_warps = gridDim.x * (unsigned)kPipeWarps;
        if (c.lazy) {
            unsigned it = 0;
            if (lane == 0) it = c.base + atomicAdd(c.counter, 1u);
            c.item = __shfl_sync(0xFFFFFFFFu, it, 0);
        } else {
            c.item = __shfl_sync(0xFFFFFFFFu, c.pending, 0);
            if (c.item < c.n_items && c.n_items - c.item < 2u * n_warps) c.lazy = true;
            if (lane == 0 && c.item < c.n_items && !c.lazy) c.pending = c.base + atomicAdd(c.counter, 1u);
        }
    }

    // Overlapped path: the slice table and the heavy rows' first chunk ids come into shared memory once
    // the index cluster has written them; the first warp of the CTA to get here loads them.
    __device__ bool load_tables_once() {
        int st = 0;
        if (lane == 0) st = atomicCAS(&tabs.state, 0, 1);
        st = __shfl_sync(0xFFFFFFFFu, st, 0);
        if (st == 0) {
            for (int r = lane; r < a.R; r += 32) {
                tabs.start[r] = a.tab[r].start;
                tabs.values[r] = reinterpret_cast<unsigned long long>(a.tab[r].values);
            }
            const int nh = a.hdr->n_heavy;
            if (lane == 0) tabs.n_heavy = nh;
            if (nh <= kHeavyCache)
                for (int h = lane; h < nh; h += 32) tabs.chunk_base[h] = a.heavy[h].chunk_base;
            __threadfence_block();
            __syncwarp();
            if (lane == 0) atomicExch(&tabs.state, 2);
        } else if (st == 1) {
            const long long start = clock64();
            volatile int* state = &tabs.state;
            while (*state != 2) {
                if (*abort_flag || clock64() - start > kWaitCycles) { give_up(); return false; }
            }
            __threadfence_block();
        }
        __syncwarp();
        return true;
    }

    __device__ void run() {
        bool ok = true;
        Claim copies{};
        unsigned n_copy = 0;
        if constexpr (OVERLAP) {
            // Until the index cluster says its tables are complete: copy items.  The flag is asked for
            // while the last copies of an item are under way and looked at after the item, so the trip
            // to memory costs nothing.
            n_copy = (unsigned)((a.vocab + a.copy_rows - 1) / a.copy_rows) * (unsigned)a.ncb;
            ns = a.copy_slots;
            claim_begin(copies, &a.hdr->copy_counter, n_copy, true);
            volatile int* ready_flag = &a.hdr->tables_ready;
            bool ready = false;
            while (ok && !ready) {
                int f = 0;
                bool waited = false;
                if (copies.item < n_copy) {
                    ok = do_copy(copies.item);
                    f = polled;
                    claim_next(copies);
                } else {
                    // nothing left to copy: wait for the tables, within the limit
                    waited = true;
                    if (lane == 0) {
                        const long long start = clock64();
                        f = *ready_flag;
                        while (!f) {
                            if (*abort_flag || clock64() - start > kWaitCycles) break;
                            __nanosleep(200);
                            f = *ready_flag;
                        }
                    }
                }
                ready = __shfl_sync(0xFFFFFFFFu, f, 0) != 0;
                if (waited && !ready) { give_up(); ok = false; }   // the wait ran out
            }
            if (ok) {
                __threadfence();        // the tables were written before the flag
                ok = load_tables_once();
            }
        }
        if constexpr (OVERLAP) { ns = a.n_slots; islot = cslot = 0; }      // the ring is empty between items
        if (ok) {
            const unsigned n_chunks = (unsigned)a.hdr->n_chunks;
            const unsigned n_base = n_chunks + (unsigned)a.hdr->n_batches;
            const unsigned n_items = n_base * (unsigned)a.ncb;
            Claim c{};
            claim_begin(c, &a.hdr->work_counter, n_items, !OVERLAP);
            while (ok && c.item < n_items) {
                const int cblk = (int)(c.item / n_base);
                const unsigned base = c.item - (unsigned)cblk * n_base;
                ok = base < n_chunks ? do_chunk((int)base, cblk) : do_rows((int)(base - n_chunks), cblk);
                claim_next(c);
            }
        }
        if constexpr (OVERLAP) {
            ns = a.copy_slots; islot = cslot = 0;
            while (ok && copies.item < n_copy) {      // the copy items that are left
                ok = do_copy(copies.item);
                claim_next(copies);
            }
        }
        if (!ok) {
            // a wait gave up: let every copy this warp has issued land before the CTA's shared memory goes away
            for (int s = 0; s < a.n_slots; ++s) {
                if (issued_mask & (1u << s)) {
                    const long long start = clock64();
                    while (!mbar_try_wait(bars + 8u * (unsigned)s, (cphase >> s) & 1u) && clock64() - start < kWaitCycles) {}
                }
            }
        }
    }
};

template <typename VT, typename OT, int K, int OPT = kOptNone, bool OVERLAP = false>
__global__ void __launch_bounds__(kPipeThreads, (sizeof(VT) == 2 && OPT == kOptNone) ? 4 : 2)
k_reduce_rows(const __grid_constant__ MainArgs a) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ int s_abort;
    __shared__ CtaTables<OVERLAP> tabs;
    unsigned long long* bar_base = reinterpret_cast<unsigned long long*>(smem_raw);
    char* slot_base = reinterpret_cast<char*>(smem_raw) + kPipeHeaderReserve;
    const int warp = warp_id();
    if (threadIdx.x == 0) {
        for (int s = 0; s < kPipeWarps * a.n_slots; ++s) mbar_init(smem_addr(&bar_base[s]), 1u);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    pdl_trigger();
    if constexpr (!OVERLAP) {
        pdl_wait();       // everything above overlaps with the tail of the kernel before
        if (a.R <= kTabCache) {
            for (int r = threadIdx.x; r < a.R; r += kPipeThreads) {
                tabs.start[r] = a.tab[r].start;
                tabs.values[r] = reinterpret_cast<unsigned long long>(a.tab[r].values);
            }
        }
        const int nh = a.hdr->n_heavy;
        if (threadIdx.x == 0) tabs.n_heavy = nh;
        if (nh <= kHeavyCache)
            for (int h = threadIdx.x; h < nh; h += kPipeThreads) tabs.chunk_base[h] = a.heavy[h].chunk_base;
    } else {
        // Running beside the index cluster (which cleared the header before it let this kernel start, and
        // which waited for everything earlier in the stream): first the bitmap of named rows, one copy per
        // CTA of that cluster, each flagged when written.
        if (threadIdx.x == 0) tabs.state = 0;
        if (warp == 0) {
            volatile const int* flags = a.hdr->bitmap_ready;
            const long long start = clock64();
            while (true) {
                const int v = lane_id() < kClusterCtas ? flags[lane_id()] : 1;
                if (__all_sync(0xFFFFFFFFu, v != 0)) break;
                if (clock64() - start > kWaitCycles) {
                    if (lane_id() == 0) { raise_status(a.hdr, DST_ERR_TIMEOUT); s_abort = 1; }
                    break;
                }
                __nanosleep(100);
            }
        }
        __syncthreads();
        if (!s_abort) {
            __threadfence();
            for (int w = threadIdx.x; w < a.bitmap_words; w += kPipeThreads) {
                const uint4 lo = __ldcg(reinterpret_cast<const uint4*>(a.bitmap) + 2 * w);
                const uint4 hi = __ldcg(reinterpret_cast<const uint4*>(a.bitmap) + 2 * w + 1);
                tabs.named[w] = lo.x | lo.y | lo.z | lo.w | hi.x | hi.y | hi.z | hi.w;
            }
        }
    }
    __syncthreads();
    {
        char* my_ring = slot_base + (size_t)warp * (size_t)a.n_slots * (size_t)a.slot_bytes;
        WarpPipe<VT, OT, K, OPT, OVERLAP> pipe(a, smem_addr(my_ring), smem_addr(&bar_base[warp * a.n_slots]), my_ring, &s_abort, tabs);
        // after a failed wait in an earlier kernel the tables are not to be trusted: touch nothing
        if (OVERLAP ? !s_abort : *reinterpret_cast<volatile int*>(&a.hdr->status) != DST_ERR_TIMEOUT) pipe.run();
    }
    if constexpr (OVERLAP) pdl_wait();   // nothing later in the stream may start before the index cluster has retired too
    __syncthreads();
    // the last CTA to finish reports the status word (it may have been raised by this kernel)
    if (threadIdx.x == 0 && a.result) {
        __threadfence();
        if (atomicAdd(&a.hdr->done, 1u) == gridDim.x - 1u) {
            __threadfence();
            a.result->status = *reinterpret_cast<volatile int*>(&a.hdr->status);
        }
    }
}

// Any d, any alignment: one thread per output element, segment summed in order.  With an optimizer
// (a.apply != 0) `out` is the fp32 weight and the state tensors take their step too.
template <typename VT, typename OT>
__global__ void __launch_bounds__(256)
k_reduce_rows_scalar(const MainArgs a) {
    const long long total = (long long)a.vocab * a.d;
    const int status = *reinterpret_cast<volatile int*>(&a.hdr->status);
    if (blockIdx.x == 0 && threadIdx.x == 0 && a.result) a.result->status = status;
    if (status == DST_ERR_TIMEOUT) return;     // a wait gave up in an earlier kernel: the tables are not to be trusted
    const OT* din = static_cast<const OT*>(a.dense_in);
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
        const int v = (int)(e / a.d);
        const long long c = e - (long long)v * a.d;
        const int beg = max(a.offsets[v], 0), end = min(a.offsets[v + 1], a.n_total);
        if (beg >= end && !a.apply && a.n_dense <= 1) { static_cast<OT*>(a.out)[e] = din ? din[e] : OT(0.f); continue; }
        float acc = 0.f;
        for (int j = beg; j < end; ++j) {
            unsigned p = a.perm[j];
            if (p < (unsigned)a.n_total) acc += (float)resolve_row<VT>(a, p)[c];
        }
        if (din) acc += (float)din[e];
        for (int q = 1; q < a.n_dense; ++q) acc += (float)static_cast<const OT*>(a.dense_more[q - 1])[e];
        if (!a.apply) { static_cast<OT*>(a.out)[e] = OT(acc); continue; }
        float* w = static_cast<float*>(a.out) + e;
        float g = a.grad_scale * acc;
        if (a.apply == kOptMomentum) {
            float* b = static_cast<float*>(a.state1) + e;
            g = fmaf(a.opt_a, *b, g);
            *b = g;
        } else if (a.apply == kOptAdam) {
            float* m = static_cast<float*>(a.state1) + e;
            float* vv = static_cast<float*>(a.state2) + e;
            const float v2 = fmaf(a.opt_b, *vv, (1.f - a.opt_b) * (g * g));
            const float m2 = fmaf(a.opt_a, *m, (1.f - a.opt_a) * g);
            *vv = v2; *m = m2;
            g = (m2 * a.opt_bc1) / (sqrtf(v2 * a.opt_bc2) + a.opt_eps);
        }
        *w = fmaf(-a.lr, g, *w);
    }
}

// Copies kept in flight by the whole grid.  Enough to cover the memory system's latency at full
// bandwidth with some slack; more only lengthens the queue every dependent access waits in (an
// index lookup, a node of a combine tree), which is what a short call is made of.
constexpr long long kInFlightBytes = 14ll << 20;

template <typename VT, typename OT, int K, int OPT, bool OVERLAP>
static cudaError_t launch_pipe_as(MainArgs a, int sm_count, cudaStream_t stream) {
    auto smem_for = [&](int slots) { return size_t(kPipeHeaderReserve) + size_t(kPipeWarps) * size_t(slots) * size_t(a.slot_bytes); };
    // the shared-memory opt-in and the occupancy answer are asked of the runtime once per device and variant
    static SmemOptIn opt_in;
    static std::atomic<int> resident_on[64];
    cudaError_t e = ensure_dynamic_smem(k_reduce_rows<VT, OT, K, OPT, OVERLAP>, smem_for(kPipeSlots), opt_in);
    if (e != cudaSuccess) return e;
    int dev = -1, resident = 0;                          // CTAs of this variant an SM holds with full rings
    const bool cached = cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64;
    if (cached) resident = resident_on[dev].load();
    if (resident < 1) {
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, k_reduce_rows<VT, OT, K, OPT, OVERLAP>, kPipeThreads, smem_for(kPipeSlots));
        if (e != cudaSuccess) return e;
        if (resident < 1) return cudaErrorLaunchOutOfResources;
        if (cached) resident_on[dev].store(resident);
    }
    const int grid = sm_count * resident;
    const long long per_slot = (long long)grid * kPipeWarps * a.slot_bytes;
    long long slots = kInFlightBytes / per_slot;
    a.n_slots = (int)(slots < 2 ? 2 : (slots > kPipeSlots ? kPipeSlots : slots));
    if (OVERLAP) {
        // the same ring depth for copy items and for the items that follow (six slots for the latter measured
        // no better: those run in waves that are bound by bandwidth and by their dependent look-ups, not by
        // the depth of one warp's ring)
        a.copy_slots = a.n_slots;
    }
    return launch_pdl(k_reduce_rows<VT, OT, K, OPT, OVERLAP>, dim3(grid), dim3(kPipeThreads), smem_for(a.n_slots), stream, a);
}

template <typename VT, typename OT, int K, int OPT>
static cudaError_t launch_pipe(const MainArgs& a, int sm_count, cudaStream_t stream) {
    return a.overlap ? launch_pipe_as<VT, OT, K, OPT, true>(a, sm_count, stream)
                     : launch_pipe_as<VT, OT, K, OPT, false>(a, sm_count, stream);
}

template <typename VT, typename OT, int OPT = kOptNone>
static cudaError_t launch_typed(MainArgs a, bool vector_ok, int sm_count, cudaStream_t stream) {
    if (!vector_ok) {
        long long total = (long long)a.vocab * a.d;
        long long blocks = (total + 255) / 256;
        if (blocks > 148LL * 32) blocks = 148LL * 32;
        if (blocks < 1) blocks = 1;
        k_reduce_rows_scalar<VT, OT><<<(int)blocks, 256, 0, stream>>>(a);
        return cudaGetLastError();
    }
    // slots hold value rows, dense_in rows and, with an optimizer, fp32 weight and state rows
    const PipeShape ps = pipe_shape((int)sizeof(VT), OPT != kOptNone ? 4 : (int)sizeof(OT), a.d);
    a.W = ps.W; a.ncb = ps.ncb; a.slot_bytes = ps.slot_bytes; a.n_slots = ps.n_slots;
    {
        // a copy item: about 32 KB worth of consecutive rows, 8 to 32 of them
        const long long row_bytes = (long long)ps.W * (OPT != kOptNone ? 4ll : (long long)sizeof(OT));
        a.copy_rows = row_bytes * 32 <= 32768 ? 32 : (row_bytes * 16 <= 32768 ? 16 : 8);
    }
    constexpr int kMaxK = sizeof(VT) == 4 ? 8 : 4;
    if (ps.K == 1) return launch_pipe<VT, OT, 1, OPT>(a, sm_count, stream);
    if (ps.K == 2) return launch_pipe<VT, OT, 2, OPT>(a, sm_count, stream);
    if (ps.K == 4 || kMaxK == 4) return launch_pipe<VT, OT, 4, OPT>(a, sm_count, stream);
    return launch_pipe<VT, OT, kMaxK, OPT>(a, sm_count, stream);
}

// The give-up path of the bounded waits, on its own: one CTA waits on a barrier nobody arrives on, with
// the limit the caller gives, and must come back with DST_ERR_TIMEOUT in the header and in `result`.
__global__ void __launch_bounds__(kPipeThreads) k_selftest_wait(WsHeader* hdr, dst_result_t* result, long long limit) {
    __shared__ unsigned long long bar;
    __shared__ int s_abort;
    if (threadIdx.x == 0) {
        mbar_init(smem_addr(&bar), 1u);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (!mbar_wait(smem_addr(&bar), 0u, &s_abort, limit)) {      // what WarpPipe::give_up does
        raise_status(hdr, DST_ERR_TIMEOUT);
        s_abort = 1;
    }
    __syncthreads();
    if (threadIdx.x == 0 && result) {
        __threadfence();
        result->status = *reinterpret_cast<volatile int*>(&hdr->status);
    }
}

cudaError_t launch_selftest_wait(WsHeader* hdr, dst_result_t* result, long long limit, cudaStream_t stream) {
    k_selftest_wait<<<1, kPipeThreads, 0, stream>>>(hdr, result, limit);
    return cudaGetLastError();
}

cudaError_t launch_reduce_rows(const MainArgs& a, int value_type, int out_type, bool vector_ok, int sm_count,
                               cudaStream_t stream) {
    if (a.apply) {
        // value rows and dense_in of one type; weight and state fp32
        if (value_type != out_type) return cudaErrorInvalidValue;
        if (value_type == DST_F32) {
            if (a.apply == kOptSgd) return launch_typed<float, float, kOptSgd>(a, vector_ok, sm_count, stream);
            if (a.apply == kOptMomentum) return launch_typed<float, float, kOptMomentum>(a, vector_ok, sm_count, stream);
            if (a.apply == kOptAdam) return launch_typed<float, float, kOptAdam>(a, vector_ok, sm_count, stream);
        } else {
            if (a.apply == kOptSgd) return launch_typed<__nv_bfloat16, __nv_bfloat16, kOptSgd>(a, vector_ok, sm_count, stream);
            if (a.apply == kOptMomentum) return launch_typed<__nv_bfloat16, __nv_bfloat16, kOptMomentum>(a, vector_ok, sm_count, stream);
            if (a.apply == kOptAdam) return launch_typed<__nv_bfloat16, __nv_bfloat16, kOptAdam>(a, vector_ok, sm_count, stream);
        }
        return cudaErrorInvalidValue;
    }
    if (value_type == DST_F32 && out_type == DST_F32) return launch_typed<float, float>(a, vector_ok, sm_count, stream);
    if (value_type == DST_F32 && out_type == DST_BF16) return launch_typed<float, __nv_bfloat16>(a, vector_ok, sm_count, stream);
    if (value_type == DST_BF16 && out_type == DST_F32) return launch_typed<__nv_bfloat16, float>(a, vector_ok, sm_count, stream);
    return launch_typed<__nv_bfloat16, __nv_bfloat16>(a, vector_ok, sm_count, stream);
}

}  // namespace dst
