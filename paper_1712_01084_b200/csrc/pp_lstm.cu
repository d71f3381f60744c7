// Recurrent use of one pivoted gate layer as an LSTM cell: z_t = [x_t ; h_{t-1}], g = W z_t,
// original rows [0,H) input gate, [H,2H) forget gate, [2H,3H) candidate, [3H,4H) output gate;
// c_t = sig(f) c_{t-1} + sig(i) tanh(g), h_t = sig(o) tanh(c_t); no bias.  (The paper only names
// recurrent networks as users of FC layers; the cell is the workload's definition.)
//
// Cross-layer permutation fusion (Section 4.2.1) applied to the recurrence: the layer input lives
// in the layer's pivoted column order for all steps, so the matrix-vector kernel copies it without
// any gather; the gate kernel reads the four pre-activations of a unit through the inverse row
// permutation and writes h_t straight to the pivoted positions the next step reads.
#include <cuda_fp16.h>

#include "pp_lstm.cuh"

namespace pp {
namespace {

template <typename T> __device__ __forceinline__ float to_float(T v);
template <> __device__ __forceinline__ float to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_float<__half>(__half v) { return __half2float(v); }
template <typename T> __device__ __forceinline__ T from_float(float v);
template <> __device__ __forceinline__ float from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ __half from_float<__half>(float v) { return __float2half_rn(v); }

template <typename T>
__global__ void lstm_prepare_kernel(const LstmArgs a) {
    const long long total = (long long)(a.steps + 1) * a.n_pad;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
         e += (long long)gridDim.x * blockDim.x) {
        const int t = (int)(e / a.n_pad), j = (int)(e - (long long)t * a.n_pad);
        const int src = __ldg(a.gather_idx + j);
        T v = from_float<T>(0.0f);
        if (src >= 0 && src < a.I) {
            if (t < a.steps) v = static_cast<const T*>(a.x_seq)[(size_t)t * a.I + src];
        } else if (src >= a.I && t == 0) {
            v = static_cast<const T*>(a.h)[src - a.I];
        } else if (src >= a.I) {
            continue;                      // written by the gate kernel of step t - 1
        }
        static_cast<T*>(a.z)[e] = v;
    }
}

__device__ __forceinline__ float sigmoidf_(float v) { return 1.0f / (1.0f + expf(-v)); }

template <typename T>
__global__ void lstm_gates_kernel(const LstmArgs a, int t) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next step may prefetch its weights
    asm volatile("griddepcontrol.wait;" ::: "memory");                // g_piv comes from the kernel just before
    const int u = blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= a.H) return;
    const float gi = a.g_piv[__ldg(a.inv_row + u)];
    const float gf = a.g_piv[__ldg(a.inv_row + a.H + u)];
    const float gg = a.g_piv[__ldg(a.inv_row + 2 * a.H + u)];
    const float go = a.g_piv[__ldg(a.inv_row + 3 * a.H + u)];
    const float c = sigmoidf_(gf) * a.c[u] + sigmoidf_(gi) * tanhf(gg);
    const float h = sigmoidf_(go) * tanhf(c);
    a.c[u] = c;
    const T hv = from_float<T>(h);
    static_cast<T*>(a.z)[(size_t)(t + 1) * a.n_pad + __ldg(a.inv_col + a.I + u)] = hv;
    if (t == a.steps - 1) static_cast<T*>(a.h)[u] = hv;
}

}  // namespace

cudaError_t launch_lstm_prepare(const LstmArgs& a, cudaStream_t stream) {
    const long long total = (long long)(a.steps + 1) * a.n_pad;
    const int blocks = (int)((total + 255) / 256 < 1184 ? (total + 255) / 256 : 1184);
    if (a.f16) lstm_prepare_kernel<__half><<<blocks, 256, 0, stream>>>(a);
    else lstm_prepare_kernel<float><<<blocks, 256, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_lstm_gates(const LstmArgs& a, int t, cudaStream_t stream) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)((a.H + 127) / 128));
    cfg.blockDim = dim3(128);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return a.f16 ? cudaLaunchKernelEx(&cfg, lstm_gates_kernel<__half>, a, t)
                 : cudaLaunchKernelEx(&cfg, lstm_gates_kernel<float>, a, t);
}

}  // namespace pp
