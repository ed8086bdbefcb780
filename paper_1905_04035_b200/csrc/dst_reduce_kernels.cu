// Row side of densify: segmented row reduction, fused dense add, one streaming write.
//
//   out[v, :] = sum_{j in segment(v)} values[perm[j], :]  +  dense_in[v, :]
//
// (Section 4 / Listing 1 of the paper: IndexedSlices -> dense; Algorithm 1 line 4:
// the dense tensors are then summed.)  This kernel moves practically all bytes of
// the operation.  It is HBM-bound: every value row, every dense_in row and every
// out row crosses the memory bus exactly once; no tensor cores are involved.
//
// Work decomposition (one warp per work item, items handed out by a counter):
//   chunk items   `chunk` consecutive entries of a heavy row's segment -> fp32 partial row;
//                 partials are combined by a fixed fan-in tree whose nodes are
//                 evaluated by whichever warp arrives last (children always summed
//                 in index order, so the result does not depend on timing)
//   row batches   kRowsPerBatch consecutive output rows that are not heavy
// A lane owns VC consecutive columns per 16-byte value load and K such groups.
#include "dst_common.cuh"

namespace dst {

// ---- typed column-group access ------------------------------------------------
template <int VC> struct Acc { float x[VC]; };

template <int VC> __device__ __forceinline__ void zero(Acc<VC>& a) {
#pragma unroll
    for (int i = 0; i < VC; ++i) a.x[i] = 0.f;
}

__device__ __forceinline__ void unpack_bf16x2(unsigned w, float& lo, float& hi) {
    lo = __uint_as_float(w << 16);
    hi = __uint_as_float(w & 0xFFFF0000u);
}
__device__ __forceinline__ unsigned pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<unsigned*>(&t);
}

// read-only input rows (never written during the kernel)
__device__ __forceinline__ void load_in(const float* p, Acc<4>& a) {
    float4 t = __ldg(reinterpret_cast<const float4*>(p));
    a.x[0] = t.x; a.x[1] = t.y; a.x[2] = t.z; a.x[3] = t.w;
}
__device__ __forceinline__ void load_in(const float* p, Acc<8>& a) {
    float4 t = __ldg(reinterpret_cast<const float4*>(p));
    float4 u = __ldg(reinterpret_cast<const float4*>(p) + 1);
    a.x[0] = t.x; a.x[1] = t.y; a.x[2] = t.z; a.x[3] = t.w;
    a.x[4] = u.x; a.x[5] = u.y; a.x[6] = u.z; a.x[7] = u.w;
}
__device__ __forceinline__ void load_in(const __nv_bfloat16* p, Acc<8>& a) {
    uint4 t = __ldg(reinterpret_cast<const uint4*>(p));
    unpack_bf16x2(t.x, a.x[0], a.x[1]); unpack_bf16x2(t.y, a.x[2], a.x[3]);
    unpack_bf16x2(t.z, a.x[4], a.x[5]); unpack_bf16x2(t.w, a.x[6], a.x[7]);
}
__device__ __forceinline__ void load_in(const __nv_bfloat16* p, Acc<4>& a) {
    uint2 t = __ldg(reinterpret_cast<const uint2*>(p));
    unpack_bf16x2(t.x, a.x[0], a.x[1]); unpack_bf16x2(t.y, a.x[2], a.x[3]);
}
// dense_in may alias out: plain (coherent) loads
__device__ __forceinline__ void load_dense(const float* p, Acc<4>& a) {
    float4 t = *reinterpret_cast<const float4*>(p);
    a.x[0] = t.x; a.x[1] = t.y; a.x[2] = t.z; a.x[3] = t.w;
}
__device__ __forceinline__ void load_dense(const float* p, Acc<8>& a) {
    float4 t = *reinterpret_cast<const float4*>(p);
    float4 u = *(reinterpret_cast<const float4*>(p) + 1);
    a.x[0] = t.x; a.x[1] = t.y; a.x[2] = t.z; a.x[3] = t.w;
    a.x[4] = u.x; a.x[5] = u.y; a.x[6] = u.z; a.x[7] = u.w;
}
__device__ __forceinline__ void load_dense(const __nv_bfloat16* p, Acc<8>& a) {
    uint4 t = *reinterpret_cast<const uint4*>(p);
    unpack_bf16x2(t.x, a.x[0], a.x[1]); unpack_bf16x2(t.y, a.x[2], a.x[3]);
    unpack_bf16x2(t.z, a.x[4], a.x[5]); unpack_bf16x2(t.w, a.x[6], a.x[7]);
}
__device__ __forceinline__ void load_dense(const __nv_bfloat16* p, Acc<4>& a) {
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
// partial rows: written by one warp, read by another through L2
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
template <int VC> __device__ __forceinline__ void add(Acc<VC>& a, const Acc<VC>& b) {
#pragma unroll
    for (int i = 0; i < VC; ++i) a.x[i] += b.x[i];
}

template <typename T> __device__ __forceinline__ const T* shfl_ptr(const T* p, int src) {
    unsigned long long u = reinterpret_cast<unsigned long long>(p);
    u = __shfl_sync(0xFFFFFFFFu, u, src);
    return reinterpret_cast<const T*>(u);
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

template <typename VT, typename OT, int K>
struct RowReducer {
    static constexpr int VC = 16 / sizeof(VT);          // columns per 16-byte value load
    static constexpr int kColsPerPass = K * 32 * VC;
    const MainArgs& a;
    const int lane;
    __device__ RowReducer(const MainArgs& args) : a(args), lane(lane_id()) {}

    __device__ __forceinline__ long long col(int cb, int k) const { return (long long)cb + (long long)(k * 32 + lane) * VC; }

    // acc += sum of value rows perm[begin .. begin+len), ascending
    __device__ __forceinline__ void accumulate_segment(Acc<VC> (&acc)[K], int begin, int len, long long cb) const {
        for (int base = 0; base < len; base += 32) {
            const int m = min(32, len - base);
            const VT* ptr = nullptr;
            if (lane < m) {
                unsigned p = a.perm[begin + base + lane];
                if (p < (unsigned)a.n_total) ptr = resolve_row<VT>(a, p);
            }
            for (int j = 0; j < m; j += 2) {
                const VT* pa = shfl_ptr(ptr, j);
                const VT* pb = shfl_ptr(ptr, (j + 1) & 31);
                if (j + 1 >= m) pb = nullptr;
                Acc<VC> va[K], vb[K];
#pragma unroll
                for (int k = 0; k < K; ++k) {
                    long long c = col(cb, k);
                    zero(va[k]); zero(vb[k]);
                    if (c < a.d) {
                        if (pa) load_in(pa + c, va[k]);
                        if (pb) load_in(pb + c, vb[k]);
                    }
                }
#pragma unroll
                for (int k = 0; k < K; ++k) { add(acc[k], va[k]); add(acc[k], vb[k]); }
            }
        }
    }

    __device__ __forceinline__ void finish_row(Acc<VC> (&acc)[K], int row, long long cb) const {
        const OT* din = static_cast<const OT*>(a.dense_in);
        OT* out = static_cast<OT*>(a.out);
#pragma unroll
        for (int k = 0; k < K; ++k) {
            long long c = col(cb, k);
            if (c < a.d) {
                if (din) { Acc<VC> dn; load_dense(din + (long long)row * a.d + c, dn); add(acc[k], dn); }
                store_out(out + (long long)row * a.d + c, acc[k]);
            }
        }
    }

    // rows nobody names: a straight copy of dense_in (bit-exact), or zeros
    __device__ __forceinline__ void copy_row(int row) const {
        const OT* din = static_cast<const OT*>(a.dense_in);
        OT* out = static_cast<OT*>(a.out);
        for (long long cb = 0; cb < a.d; cb += kColsPerPass) {
            Acc<VC> t[K];
#pragma unroll
            for (int k = 0; k < K; ++k) {
                long long c = col(cb, k);
                zero(t[k]);
                if (din && c < a.d) load_dense(din + (long long)row * a.d + c, t[k]);
            }
#pragma unroll
            for (int k = 0; k < K; ++k) {
                long long c = col(cb, k);
                if (c < a.d) store_out(out + (long long)row * a.d + c, t[k]);
            }
        }
    }

    __device__ void do_row_batch(int batch) const {
        const int v0 = batch * kRowsPerBatch;
        const int nrows = min(kRowsPerBatch, a.vocab - v0);
        int o = 0;
        if (lane <= nrows) o = a.offsets[v0 + lane];
        for (int i = 0; i < nrows; ++i) {
            const int beg = __shfl_sync(0xFFFFFFFFu, o, i);
            const int cnt = __shfl_sync(0xFFFFFFFFu, o, i + 1) - beg;
            if (cnt > a.chunk) continue;                 // heavy: produced by the chunk items
            if (cnt == 0) { copy_row(v0 + i); continue; }
            for (long long cb = 0; cb < a.d; cb += kColsPerPass) {
                Acc<VC> acc[K];
#pragma unroll
                for (int k = 0; k < K; ++k) zero(acc[k]);
                accumulate_segment(acc, beg, cnt, cb);
                finish_row(acc, v0 + i, cb);
            }
        }
    }

    __device__ __forceinline__ float* partial_row(int slot) const { return a.partials + (long long)slot * a.d; }

    // acc = child[0] + child[1] + ... in index order
    __device__ __forceinline__ void sum_children(Acc<VC> (&acc)[K], int first_slot, int n, long long cb) const {
#pragma unroll
        for (int k = 0; k < K; ++k) zero(acc[k]);
        for (int c = 0; c < n; c += 2) {
            const float* pa = partial_row(first_slot + c);
            const float* pb = (c + 1 < n) ? partial_row(first_slot + c + 1) : nullptr;
            Acc<VC> va[K], vb[K];
#pragma unroll
            for (int k = 0; k < K; ++k) {
                long long cc = col(cb, k);
                zero(va[k]); zero(vb[k]);
                if (cc < a.d) {
                    load_partial(pa + cc, va[k]);
                    if (pb) load_partial(pb + cc, vb[k]);
                }
            }
#pragma unroll
            for (int k = 0; k < K; ++k) { add(acc[k], va[k]); add(acc[k], vb[k]); }
        }
    }

    __device__ void do_chunk(int cid) const {
        const ChunkDesc cd = a.chunkdesc[cid];
        for (long long cb = 0; cb < a.d; cb += kColsPerPass) {
            Acc<VC> acc[K];
#pragma unroll
            for (int k = 0; k < K; ++k) zero(acc[k]);
            accumulate_segment(acc, cd.begin, cd.len, cb);
            float* pr = partial_row(cid);
#pragma unroll
            for (int k = 0; k < K; ++k) {
                long long c = col(cb, k);
                if (c < a.d) store_partial(pr + c, acc[k]);
            }
        }
        // climb the combine tree while this warp is the last child to arrive
        const HeavyInfo hi = a.heavy[cd.heavy];
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
            if (lane == 0) last = atomicAdd(&a.node_cnt[node], 1u) == (unsigned)(n_children - 1);
            last = __shfl_sync(0xFFFFFFFFu, last, 0);
            if (!last) return;
            __threadfence();
            const int first_child_slot = child_first + parent * kFanIn;
            const bool root = n_parent == 1;
            for (long long cb = 0; cb < a.d; cb += kColsPerPass) {
                Acc<VC> acc[K];
                sum_children(acc, first_child_slot, n_children, cb);
                if (root) {
                    finish_row(acc, hi.row, cb);
                } else {
                    float* pr = partial_row(a.chunk_max + node);
#pragma unroll
                    for (int k = 0; k < K; ++k) {
                        long long c = col(cb, k);
                        if (c < a.d) store_partial(pr + c, acc[k]);
                    }
                }
            }
            if (root) return;
            child_first = a.chunk_max + hi.upper_base + upper_off;
            upper_off += n_parent;
            j = parent;
            n_level = n_parent;
        }
    }
};

template <typename VT, typename OT, int K>
__global__ void __launch_bounds__(kMainThreads)
k_reduce_rows(const MainArgs a) {
    RowReducer<VT, OT, K> rr(a);
    const int n_chunks = a.hdr->n_chunks;
    const unsigned n_items = (unsigned)n_chunks + (unsigned)((a.vocab + kRowsPerBatch - 1) / kRowsPerBatch);
    if (blockIdx.x == 0 && threadIdx.x == 0 && a.result) a.result->status = a.hdr->status;
    while (true) {
        unsigned item = 0;
        if (rr.lane == 0) item = atomicAdd(&a.hdr->work_counter, 1u);
        item = __shfl_sync(0xFFFFFFFFu, item, 0);
        if (item >= n_items) break;
        if (item < (unsigned)n_chunks) rr.do_chunk((int)item);
        else rr.do_row_batch((int)(item - (unsigned)n_chunks));
    }
}

// Any d, any alignment: one thread per output element, segment summed in order.
template <typename VT, typename OT>
__global__ void __launch_bounds__(256)
k_reduce_rows_scalar(const MainArgs a) {
    const long long total = (long long)a.vocab * a.d;
    if (blockIdx.x == 0 && threadIdx.x == 0 && a.result) a.result->status = a.hdr->status;
    const OT* din = static_cast<const OT*>(a.dense_in);
    OT* out = static_cast<OT*>(a.out);
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
        const int v = (int)(e / a.d);
        const long long c = e - (long long)v * a.d;
        const int beg = a.offsets[v], end = a.offsets[v + 1];
        if (beg == end) { out[e] = din ? din[e] : OT(0.f); continue; }
        float acc = 0.f;
        for (int j = beg; j < end; ++j) {
            unsigned p = a.perm[j];
            if (p < (unsigned)a.n_total) acc += (float)resolve_row<VT>(a, p)[c];
        }
        if (din) acc += (float)din[e];
        out[e] = OT(acc);
    }
}

template <typename VT, typename OT>
static cudaError_t launch_typed(const MainArgs& a, bool vector_ok, int grid, cudaStream_t stream) {
    if (!vector_ok) {
        long long total = (long long)a.vocab * a.d;
        long long blocks = (total + 255) / 256;
        if (blocks > 148LL * 32) blocks = 148LL * 32;
        if (blocks < 1) blocks = 1;
        k_reduce_rows_scalar<VT, OT><<<(int)blocks, 256, 0, stream>>>(a);
        return cudaGetLastError();
    }
    constexpr int VC = 16 / sizeof(VT);
    const long long groups = (a.d + 32LL * VC - 1) / (32LL * VC);   // 16-byte groups per lane needed for one pass
    constexpr int kMaxK = sizeof(VT) == 4 ? 8 : 4;
    if (groups <= 1) k_reduce_rows<VT, OT, 1><<<grid, kMainThreads, 0, stream>>>(a);
    else if (groups <= 2) k_reduce_rows<VT, OT, 2><<<grid, kMainThreads, 0, stream>>>(a);
    else if (groups <= 4 || kMaxK == 4) k_reduce_rows<VT, OT, 4><<<grid, kMainThreads, 0, stream>>>(a);
    else k_reduce_rows<VT, OT, kMaxK><<<grid, kMainThreads, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_reduce_rows(const MainArgs& a, int value_type, int out_type, bool vector_ok, int grid,
                               cudaStream_t stream) {
    if (value_type == DST_F32 && out_type == DST_F32) return launch_typed<float, float>(a, vector_ok, grid, stream);
    if (value_type == DST_F32 && out_type == DST_BF16) return launch_typed<float, __nv_bfloat16>(a, vector_ok, grid, stream);
    if (value_type == DST_BF16 && out_type == DST_F32) return launch_typed<__nv_bfloat16, float>(a, vector_ok, grid, stream);
    return launch_typed<__nv_bfloat16, __nv_bfloat16>(a, vector_ok, grid, stream);
}

}  // namespace dst
