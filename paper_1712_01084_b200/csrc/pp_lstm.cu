// Recurrent use of one pivoted gate layer as an LSTM cell: z_t = [x_t ; h_{t-1}], g = W z_t,
// original rows [0,H) input gate, [H,2H) forget gate, [2H,3H) candidate, [3H,4H) output gate;
// c_t = sig(f) c_{t-1} + sig(i) tanh(g), h_t = sig(o) tanh(c_t); a bias given to the layer is part of g.
// (The paper only names recurrent networks as users of FC layers; the cell is the workload's definition.)
//
// Cross-layer permutation fusion (Section 4.2.1) applied to the recurrence: the layer input lives
// in the layer's pivoted column order for all steps, so the matrix-vector kernel copies it without
// any gather; the gate kernel reads the four pre-activations of a unit through the inverse row
// permutation and writes h_t straight to the pivoted positions the next step reads.
#include <cuda_fp16.h>

#include "pp_lstm.cuh"
#include "pp_stream.cuh"

namespace pp {
namespace {

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

// =====================================================================================================
// Persistent cell.  The gate matrix of the recurrent workload (12.75 MiB) is smaller than the shared
// memory of the whole GPU, so a cooperative grid keeps it there for all steps: CTA c copies the
// fragments of its strips (16-row groups) into shared memory once; per step it multiplies them with
// z_t (8 KiB, also in shared memory) and publishes its pre-activations as tagged packets; EVERY CTA
// collects all of them and evaluates all H units (each thread keeps the cell state of its units in
// registers), writing h_t straight into its own shared-memory copy of z_{t+1} -- one exchange per step,
// no weight traffic at all.  Every wait for a packet is bounded; a time-out raises the status word and
// ends the kernel.
namespace pp {
namespace {

constexpr int kPersistThreads = 512;
constexpr int kPersistWarps = kPersistThreads / 32;
constexpr int kPersistUnits = 4;               // units per thread: H <= 4 * 512
constexpr unsigned kSpinLimit = 1u << 20;      // re-reads of one packet before a wait gives up (about a second)

__device__ __forceinline__ void cp16(void* smem_dst, const void* gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;"
                 :: "r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ uint4 ld_volatile_v4(const uint4* p) {
    uint4 v;
    asm volatile("ld.volatile.global.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
// Every CTA evaluates every unit, so the gate functions use the hardware exponential and reciprocal:
// absolute error of a few 1e-7, far inside what the fp16 weights and the fp16 h already cost.
__device__ __forceinline__ float fast_sigmoid(float v) { return __fdividef(1.0f, 1.0f + __expf(-v)); }
__device__ __forceinline__ float fast_tanh(float v) { return 1.0f - __fdividef(2.0f, 1.0f + __expf(2.0f * v)); }
__device__ __forceinline__ void mma16816(float (&d)[4], const uint4& a, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}

__global__ void __launch_bounds__(kPersistThreads, 1) lstm_persist_kernel(const LstmPersistArgs a) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t4 = lane & 3;
    const int ns = a.strips_per_cta;
    const int s0 = min((int)blockIdx.x * ns, a.n_strips), s1 = min(s0 + ns, a.n_strips);
    const int f0 = __ldg(a.strip_start + s0), f1 = __ldg(a.strip_start + s1);
    const int nf = f1 - f0;

    // shared memory: weights | xoff | red | z (two buffers) | all pre-activations of the step
    uint4* wsm = reinterpret_cast<uint4*>(smem);
    int* xo_sm = reinterpret_cast<int*>(smem + (size_t)nf * 512);
    float* red = reinterpret_cast<float*>(xo_sm + ((nf + 3) & ~3));            // [kPersistWarps][16]
    __half* zbuf = reinterpret_cast<__half*>(red + kPersistWarps * 16);        // [2][n_pad]
    float* gsm = reinterpret_cast<float*>(zbuf + 2 * (size_t)a.n_pad);         // [m_pad]
    __shared__ int s_abort;
    if (tid == 0) s_abort = 0;

    // once: this CTA's weights and column offsets, and z_0
    const uint4* wsrc = reinterpret_cast<const uint4*>(a.values) + (size_t)f0 * 32;
    for (int i = tid; i < nf * 32; i += kPersistThreads) cp16(wsm + i, wsrc + i);
    for (int i = tid; i < nf; i += kPersistThreads) xo_sm[i] = __ldg(a.xoff + f0 + i);
    const __half* zglob = static_cast<const __half*>(a.z);
    for (int i = tid; i < a.n_pad / 8; i += kPersistThreads) cp16(zbuf + 8 * i, zglob + 8 * i);
    asm volatile("cp.async.commit_group;" ::: "memory");

    // the units whose cell state this thread keeps (the same units in every CTA)
    // together with where their four pre-activations sit in pivoted row order and where h goes in z
    float cst[kPersistUnits];
    int ri[kPersistUnits], rf[kPersistUnits], rg[kPersistUnits], ro[kPersistUnits], hz[kPersistUnits];
#pragma unroll
    for (int q = 0; q < kPersistUnits; ++q) {
        const int u = tid + q * kPersistThreads;
        const bool live = u < a.H;
        cst[q] = live ? a.c[u] : 0.0f;
        ri[q] = live ? __ldg(a.inv_row + u) : 0;
        rf[q] = live ? __ldg(a.inv_row + a.H + u) : 0;
        rg[q] = live ? __ldg(a.inv_row + 2 * a.H + u) : 0;
        ro[q] = live ? __ldg(a.inv_row + 3 * a.H + u) : 0;
        hz[q] = live ? __ldg(a.inv_col + a.I + u) : 0;
    }

    // warp -> (strip of this CTA, part of its fragments)
    const int wps = kPersistWarps / ns;               // warps per strip
    const int si = warp / wps, part = warp % wps;
    int wf0 = 0, wf1 = 0;
    if (s0 + si < s1) {
        const int sb = __ldg(a.strip_start + s0 + si) - f0, se = __ldg(a.strip_start + s0 + si + 1) - f0;
        wf0 = sb + (int)(((long long)(se - sb) * part) / wps);
        wf1 = sb + (int)(((long long)(se - sb) * (part + 1)) / wps);
    }
    // the row this thread publishes (threads [0, 16 * strips of this CTA)) and its bias
    const int my_row = (s0 + (tid >> 4)) * 16 + (tid & 15);
    const float my_bias = tid < 16 * (s1 - s0) ? __ldg(a.bias_piv + my_row) : 0.0f;
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();

    for (int t = 0; t < a.steps; ++t) {
        __half* zcur = zbuf + (size_t)(t & 1) * a.n_pad;
        __half* znext = zbuf + (size_t)((t + 1) & 1) * a.n_pad;
        // prefetch x_{t+1} (pivoted, zeros at the h positions) into the other buffer
        const __half* znext_g = zglob + (size_t)(t + 1) * a.n_pad;
        for (int i = tid; i < a.n_pad / 8; i += kPersistThreads) cp16(znext + 8 * i, znext_g + 8 * i);
        asm volatile("cp.async.commit_group;" ::: "memory");

        // pre-activations of this CTA's rows
        // four independent accumulator chains, so that the loads and tensor-core instructions of
        // neighbouring fragments overlap
        float acc[4][4];
#pragma unroll
        for (int j = 0; j < 4; ++j) { acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.0f; }
        const __half* zlane = zcur + 2 * t4;
        for (int f = wf0; f < wf1; f += 4) {
            int xo[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) xo[j] = xo_sm[min(f + j, wf1 - 1)];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (f + j < wf1) {                       // warp-uniform
                    const uint4 wa = wsm[(size_t)(f + j) * 32 + lane];
                    uint32_t b0 = 0u, b1 = 0u;
                    if (g == 0) {
                        b0 = *reinterpret_cast<const uint32_t*>(zlane + xo[j]);
                        b1 = *reinterpret_cast<const uint32_t*>(zlane + xo[j] + 8);
                    }
                    mma16816(acc[j], wa, b0, b1);
                }
            }
        }
        if (t4 == 0) {                                   // column 0 = the only batch column
            red[warp * 16 + g] = (acc[0][0] + acc[1][0]) + (acc[2][0] + acc[3][0]);
            red[warp * 16 + g + 8] = (acc[0][2] + acc[1][2]) + (acc[2][2] + acc[3][2]);
        }
        __syncthreads();
        // Exchange.  Every pre-activation travels as an 8-byte packet {value, tag = t + 1} written by one
        // store, so a reader that sees the tag has the value: no fence, no separate barrier.  Two packet
        // buffers alternate by step parity: buffer t & 1 is rewritten at step t + 2, which a CTA starts
        // only after it has read all of step t + 1, i.e. after every CTA has finished reading step t.
        uint2* gpk = a.g_pk + (size_t)(t & 1) * a.m_pad;
        const uint32_t tag = (uint32_t)(t + 1);
        if (tid < 16 * (s1 - s0)) {
            const int ls = tid >> 4, r = tid & 15;
            float v = 0.0f;
            for (int pw = 0; pw < wps; ++pw) v += red[(ls * wps + pw) * 16 + r];
            v += my_bias;
            asm volatile("st.volatile.global.v2.u32 [%0], {%1, %2};" :: "l"(gpk + my_row), "r"(__float_as_uint(v)), "r"(tag) : "memory");
        }
        // every CTA collects all packets (two per 16-byte load), bounded retries on the ones not there yet
        bool gave_up = false;
        const unsigned spin_limit = a.spin_limit ? a.spin_limit : kSpinLimit;
        const int n_pairs = a.m_pad / 2;
        for (int base = 0; base < n_pairs; base += 8 * kPersistThreads) {
            uint4 v[8];
            unsigned pending = 0u;                      // bit k: packet pair k has not shown this step's tag yet
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int i = base + k * kPersistThreads + tid;
                v[k] = make_uint4(0u, tag, 0u, tag);
                if (i < n_pairs) v[k] = ld_volatile_v4(reinterpret_cast<const uint4*>(gpk) + i);
            }
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if (v[k].y != tag || v[k].w != tag) pending |= 1u << k;
            // Re-read ALL missing pairs per round, so that a round costs one trip to L2 however many are missing
            // (one pair after the other cost a trip each: 2.7 us per step for the collection, now about 1.4).
            unsigned spins = 0;
            while (pending) {
                if (++spins > spin_limit || ((spins & 1023u) == 0 && *reinterpret_cast<volatile int*>(a.status))) {
                    gave_up = true;
                    break;
                }
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    if (pending & (1u << k))
                        v[k] = ld_volatile_v4(reinterpret_cast<const uint4*>(gpk) + (base + k * kPersistThreads + tid));
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    if ((pending & (1u << k)) && v[k].y == tag && v[k].w == tag) pending &= ~(1u << k);
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int i = base + k * kPersistThreads + tid;
                if (i < n_pairs)
                    *reinterpret_cast<float2*>(gsm + 2 * i) = make_float2(__uint_as_float(v[k].x), __uint_as_float(v[k].z));
            }
        }
        if (gave_up) { *a.status = 1; s_abort = 1; }
        asm volatile("cp.async.wait_group 0;" ::: "memory");      // x_{t+1} has landed in the other z buffer
        __syncthreads();
        if (s_abort) break;

        // every CTA evaluates all units; h_t goes into this CTA's own copy of z_{t+1}
#pragma unroll
        for (int q = 0; q < kPersistUnits; ++q) {
            const int u = tid + q * kPersistThreads;
            if (u < a.H) {
                const float c = fast_sigmoid(gsm[rf[q]]) * cst[q] + fast_sigmoid(gsm[ri[q]]) * fast_tanh(gsm[rg[q]]);
                const float h = fast_sigmoid(gsm[ro[q]]) * fast_tanh(c);
                cst[q] = c;
                const __half hv = __float2half_rn(h);
                znext[hz[q]] = hv;
                if (t == a.steps - 1 && blockIdx.x == 0) { static_cast<__half*>(a.h)[u] = hv; a.c[u] = c; }
            }
        }
        __syncthreads();
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

}  // namespace

size_t lstm_persist_smem(int max_frags, int n_pad, int m_pad) {
    const size_t bytes = (size_t)max_frags * 512 + (size_t)((max_frags + 3) & ~3) * 4 + kPersistWarps * 16 * 4 +
                         2 * (size_t)n_pad * 2 + (size_t)m_pad * 4;
    return bytes <= 220 * 1024 ? bytes : 0;
}

cudaError_t launch_lstm_persist(const LstmPersistArgs& a_in, int grid, size_t smem, cudaStream_t stream) {
    static PerDeviceOnce configured;
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (!configured.is_done(dev)) {
        e = cudaFuncSetAttribute(lstm_persist_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
        if (e != cudaSuccess) return e;
        configured.mark(dev);
    }
    LstmPersistArgs a = a_in;
    a.spin_limit = (unsigned)g_stream_wait_polls;
    void* args[] = {&a};
    return cudaLaunchCooperativeKernel(reinterpret_cast<void*>(lstm_persist_kernel), dim3((unsigned)grid),
                                       dim3(kPersistThreads), args, smem, stream);
}

}  // namespace pp
