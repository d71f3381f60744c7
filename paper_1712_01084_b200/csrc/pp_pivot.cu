// Listing 1's group fetch as a pre-pass of its own: out[b][j] = x[b][gather_idx[j]] (0 where the
// index is -1) for every pivoted column j < n_pad.  Used when the layer kernel cannot permute x in
// shared memory itself (several batch columns, or an input too long to hold twice): the kernel
// then copies the pivoted rows straight into place.  One CTA per batch row; the row goes through
// shared memory so that the read of x and the write of out are both coalesced.
#include <cuda_fp16.h>

#include "pp_gemv.cuh"

namespace pp {
namespace {

template <typename T>
__global__ void pivot_x_kernel(const T* __restrict__ x, int ldx, int n, const int32_t* __restrict__ gather_idx, int n_pad,
                               T* __restrict__ out, int use_smem) {
    extern __shared__ __align__(16) unsigned char smem_row[];
    T* row = reinterpret_cast<T*>(smem_row);
    const int b = blockIdx.x;
    const T* src = x + (size_t)b * ldx;
    if (use_smem) {
        for (int j = threadIdx.x; j < n; j += blockDim.x) row[j] = src[j];
        __syncthreads();
    }
    T* dst = out + (size_t)b * n_pad;
    // 8 independent index loads per thread before the first use, so that their latencies overlap
    for (int j0 = threadIdx.x; j0 < n_pad; j0 += 8 * blockDim.x) {
        int idx[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int j = j0 + q * blockDim.x;
            idx[q] = j < n_pad ? __ldg(gather_idx + j) : -1;
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int j = j0 + q * blockDim.x;
            if (j < n_pad) dst[j] = idx[q] >= 0 ? (use_smem ? row[idx[q]] : src[idx[q]]) : T(0.0f);
        }
    }
}

}  // namespace

cudaError_t launch_pivot_x(pp_dtype_t dt, const void* x, int ldx, int n, const int32_t* gather_idx, int n_pad, void* out,
                           int batch, cudaStream_t stream) {
    const size_t esz = dt == PP_F16 ? 2 : 4;
    const size_t row_bytes = ((size_t)n * esz + 15) / 16 * 16;
    const int use_smem = row_bytes <= 48 * 1024;
    const size_t smem = use_smem ? row_bytes : 0;
    if (dt == PP_F16)
        pivot_x_kernel<__half><<<batch, 1024, smem, stream>>>(static_cast<const __half*>(x), ldx, n, gather_idx, n_pad,
                                                           static_cast<__half*>(out), use_smem);
    else
        pivot_x_kernel<float><<<batch, 1024, smem, stream>>>(static_cast<const float*>(x), ldx, n, gather_idx, n_pad,
                                                         static_cast<float*>(out), use_smem);
    return cudaGetLastError();
}

}  // namespace pp
