// Kernels of the accumulation dispatcher (Algorithms 1 and 2): the sum of dense gradients
// ("reduce" branch) and the row numbers a dense gradient gets when the "gather" branch turns
// it into IndexedSlices.  Both are plain streaming kernels bound by HBM bandwidth.
#include "dst_common.cuh"

namespace dst {

__device__ __forceinline__ void unpack8(const uint4& t, float (&f)[8]) {
    f[0] = __uint_as_float(t.x << 16); f[1] = __uint_as_float(t.x & 0xFFFF0000u);
    f[2] = __uint_as_float(t.y << 16); f[3] = __uint_as_float(t.y & 0xFFFF0000u);
    f[4] = __uint_as_float(t.z << 16); f[5] = __uint_as_float(t.z & 0xFFFF0000u);
    f[6] = __uint_as_float(t.w << 16); f[7] = __uint_as_float(t.w & 0xFFFF0000u);
}
__device__ __forceinline__ unsigned pack2(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const unsigned*>(&v);
}

// out = src[0] + src[1] + ... + src[k-1], left to right in fp32; out may be one of the sources.
// 16 bytes per thread and step; the tail that does not fill 16 bytes, and unaligned tensors, go
// element by element.
template <typename T>
__global__ void __launch_bounds__(256) k_sum_dense(const __grid_constant__ SumParams p) {
    pdl_trigger();
    pdl_wait();
    const long long stride = (long long)gridDim.x * blockDim.x;
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long n_vec = p.vector_ok ? p.n_elems * (long long)sizeof(T) / 16 : 0;
    for (long long i = tid; i < n_vec; i += stride) {
        uint4 v[kSumFanIn];
#pragma unroll
        for (int s = 0; s < kSumFanIn; ++s)
            if (s < p.k) v[s] = __ldcs(reinterpret_cast<const uint4*>(p.src[s]) + i);
        uint4 o;
        if (sizeof(T) == 4) {
            float4 acc = *reinterpret_cast<const float4*>(&v[0]);
#pragma unroll
            for (int s = 1; s < kSumFanIn; ++s)
                if (s < p.k) {
                    const float4 t = *reinterpret_cast<const float4*>(&v[s]);
                    acc.x += t.x; acc.y += t.y; acc.z += t.z; acc.w += t.w;
                }
            o = *reinterpret_cast<const uint4*>(&acc);
        } else {
            float acc[8];
            unpack8(v[0], acc);
#pragma unroll
            for (int s = 1; s < kSumFanIn; ++s)
                if (s < p.k) {
                    float t[8];
                    unpack8(v[s], t);
#pragma unroll
                    for (int q = 0; q < 8; ++q) acc[q] += t[q];
                }
            o = make_uint4(pack2(acc[0], acc[1]), pack2(acc[2], acc[3]), pack2(acc[4], acc[5]), pack2(acc[6], acc[7]));
        }
        __stcs(reinterpret_cast<uint4*>(p.out) + i, o);
    }
    const long long first = n_vec * 16 / (long long)sizeof(T);
    for (long long e = first + tid; e < p.n_elems; e += stride) {
        float acc = (float)static_cast<const T*>(p.src[0])[e];
        for (int s = 1; s < p.k; ++s) acc += (float)static_cast<const T*>(p.src[s])[e];
        static_cast<T*>(p.out)[e] = T(acc);
    }
}

// indices[i] = i for the `n` rows of a dense tensor seen as IndexedSlices
template <typename IT>
__global__ void __launch_bounds__(256) k_iota(IT* __restrict__ indices, long long n) {
    pdl_trigger();
    pdl_wait();
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) indices[i] = (IT)i;
}

cudaError_t launch_sum_dense(const SumParams& p, int out_type, int sm_count, cudaStream_t stream) {
    long long work = p.n_elems / 8 + 1;
    long long blocks = (work + 255) / 256;
    const long long cap = (long long)sm_count * 8;
    if (blocks > cap) blocks = cap;
    if (out_type == DST_F32) return launch_pdl(k_sum_dense<float>, dim3((unsigned)blocks), dim3(256), 0, stream, p);
    return launch_pdl(k_sum_dense<__nv_bfloat16>, dim3((unsigned)blocks), dim3(256), 0, stream, p);
}

cudaError_t launch_iota(void* indices, long long n, int index_type, int sm_count, cudaStream_t stream) {
    long long blocks = (n + 255) / 256;
    const long long cap = (long long)sm_count * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    if (index_type == DST_I64)
        return launch_pdl(k_iota<long long>, dim3((unsigned)blocks), dim3(256), 0, stream, static_cast<long long*>(indices), n);
    return launch_pdl(k_iota<int>, dim3((unsigned)blocks), dim3(256), 0, stream, static_cast<int*>(indices), n);
}

}  // namespace dst
