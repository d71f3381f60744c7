// Persistent streaming block-sparse matrix-vector kernels for sm_100a (batch 1 .. 8).
//
// The packed tile values of a layer form one linear sequence of 512-byte fragments (strip =
// row-group of a block-row; a strip's fragments are contiguous and strips follow each other).
// The host cuts that sequence into one contiguous range per CTA (2 CTAs per SM), and every warp
// of a CTA streams an equal, contiguous share of its CTA's range:
//   * Listing 1's group fetch is done ONCE per CTA for the whole pivoted input:
//     xs[j] = x[gather_idx[j]] goes to shared memory while the first weight fragments are already
//     in flight; after one barrier no warp waits for another until its range is finished;
//   * each warp keeps kUnroll 128-bit loads (4 KiB) in flight and refills a slot as soon as it is
//     consumed, so the load queue never drains at work-unit boundaries;
//   * where a warp's range crosses a strip boundary it parks the finished 16(32)-row partial sum
//     in shared memory; after the final barrier the CTA adds the parks of every strip in warp
//     order.  A strip shared by several CTAs (Section 4.1.5's "additional reduction step") goes
//     through one global partial sum per CTA, added in CTA order by the last CTA to arrive.
// Results are therefore independent of scheduling.  fp16 tiles: warp-level 16x8x16 tensor-core
// instruction, batch on the 8-wide side, fp32 accumulate.  fp32 tiles: plain FMAs.
#include <cuda_fp16.h>

#include "pp_gemv.cuh"
#include "pp_stream.cuh"

namespace pp {
namespace {

constexpr int kThreads = kStreamWarps * 32;
constexpr int kUnroll = 8;

__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ float ld_cg(const float* p) {
    float v;
    asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}

__device__ __forceinline__ void mma_16x8x16(float (&d)[4], const uint4& a, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}

__device__ __forceinline__ int x_index(const StreamArgs& a, int pj) {
    if (a.gather_idx) return __ldg(a.gather_idx + pj);
    return pj < a.x_limit ? pj : -1;
}

// Shared-memory header shared by both kernels (all sizes in 4-byte words).
struct SmemLayout {
    int* sstart;    // [kStreamMaxStrips + 1] strip starts of this CTA's strips
    int* wlohi;     // [kStreamMaxStrips] first | last << 8 warp that parked a partial for the strip
    int* flags;     // [2]
    float* segp;    // [kStreamSegSlots][RG][batch]
    void* xs;       // staged x
};
constexpr int kHeaderWords = 128;   // sstart (49) + wlohi (48) + flags (2), padded

__device__ __forceinline__ SmemLayout carve(unsigned char* raw, int rg, int batch) {
    SmemLayout L;
    int* w = reinterpret_cast<int*>(raw);
    L.sstart = w;
    L.wlohi = w + 56;
    L.flags = w + 112;
    L.segp = reinterpret_cast<float*>(w + kHeaderWords);
    L.xs = L.segp + kStreamSegSlots * rg * batch;
    return L;
}

__device__ __forceinline__ int warp_begin(const CtaDesc& d, int w) {
    return d.p_begin + (int)(((long long)(d.p_end - d.p_begin) * w) / kStreamWarps);
}

// Everything after the last barrier of the streaming phase: per-strip sums, cross-CTA reduction,
// bias + activation + (scatter | pivoted store).  RG = rows per strip.
template <int RG>
__device__ __forceinline__ void finalize(const StreamArgs& a, const CtaDesc& d, const SmemLayout& L) {
    const int tid = threadIdx.x;
    const int batch = a.batch;
    const int per_strip = RG * batch;

    auto emit = [&](int i, int b, float v) {
        v += __ldg(a.bias_piv + i);
        if (a.act == PP_ACT_RELU) v = fmaxf(v, 0.0f);
        if (a.out_mode == OUT_SCATTER_F32) {
            const int dst = __ldg(a.scatter_idx + i);
            if (dst >= 0) static_cast<float*>(a.y)[(size_t)b * a.ldy + dst] = v;
        } else if (a.out_mode == OUT_PIVOTED_F32) {
            static_cast<float*>(a.y)[(size_t)b * a.ldy + i] = v;
        } else {
            static_cast<__half*>(a.y)[(size_t)b * a.ldy + i] = __float2half_rn(v);
        }
    };

    // which warps parked a partial for each strip (their ranges intersect the strip inside this CTA)
    for (int ls = tid; ls < d.s_count; ls += kThreads) {
        const int lo = max(L.sstart[ls], d.p_begin), hi = min(L.sstart[ls + 1], d.p_end);
        int w_lo = 1, w_hi = 0;
        if (lo < hi) {
            w_lo = w_hi = 0;
            for (int w = 1; w < kStreamWarps; ++w) {
                const int wb = warp_begin(d, w);
                if (wb <= lo) w_lo = w;
                if (wb <= hi - 1) w_hi = w;
            }
        }
        L.wlohi[ls] = w_lo | (w_hi << 8);
    }
    __syncthreads();

    bool shared_any = false;
    const int n_out = d.s_count * per_strip;
    for (int e = tid; e < n_out; e += kThreads) {
        const int ls = e / per_strip, rem = e - ls * per_strip;
        const int r = rem / batch, b = rem - r * batch;
        const int wl = L.wlohi[ls] & 0xff, wh = L.wlohi[ls] >> 8;
        float v = 0.0f;
        for (int w = wl; w <= wh; ++w)      // warps with an empty range parked nothing
            if (warp_begin(d, w) < warp_begin(d, w + 1)) v += L.segp[((ls + w) * RG + r) * batch + b];
        const int s = d.s_first + ls;
        const int4 info = __ldg(reinterpret_cast<const int4*>(a.strip_info) + s);
        if (info.y == 1) {
            emit(s * RG + r, b, v);
        } else {
            a.partials[(size_t)(info.z + (int)blockIdx.x - info.x) * (RG * kStreamMaxBatch) + rem] = v;
            shared_any = true;
        }
    }
    // only the first and the last strip of a CTA can be shared with a neighbour
    const int ls_edge[2] = {0, d.s_count - 1};
    int4 edge[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        edge[k] = make_int4(0, 1, 0, 0);
        if (d.s_count > 0 && (k == 0 || d.s_count > 1))
            edge[k] = __ldg(reinterpret_cast<const int4*>(a.strip_info) + d.s_first + ls_edge[k]);
    }
    if (edge[0].y == 1 && edge[1].y == 1) return;      // uniform for the CTA
    (void)shared_any;
    __threadfence();
    __syncthreads();
    if (tid < 2) {
        int last = 0;
        if (edge[tid].y > 1) {
            const int old = atomicAdd(a.counters + d.s_first + ls_edge[tid], 1);
            last = (old == edge[tid].y - 1);
        }
        L.flags[tid] = last;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        if (!L.flags[k]) continue;
        __threadfence();
        const int s = d.s_first + ls_edge[k];
        const float* base = a.partials + (size_t)edge[k].z * (RG * kStreamMaxBatch);
        for (int e = tid; e < per_strip; e += kThreads) {
            float v = 0.0f;
            for (int p = 0; p < edge[k].y; ++p) v += ld_cg(base + (size_t)p * (RG * kStreamMaxBatch) + e);
            const int r = e / batch, b = e - r * batch;
            emit(s * RG + r, b, v);
        }
        if (tid == 0) a.counters[s] = 0;
    }
}

// ------------------------------------------------------------------ fp16 tiles
__global__ void __launch_bounds__(kThreads, 2) stream_f16_kernel(const StreamArgs a) {
    constexpr int RG = 16;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const SmemLayout L = carve(smem_raw, RG, a.batch);
    __half* xs = static_cast<__half*>(L.xs);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int4 dd = __ldg(reinterpret_cast<const int4*>(a.cta_desc) + blockIdx.x);
    const CtaDesc d{dd.x, dd.y, dd.z, dd.w};
    const int wbeg = warp_begin(d, warp), wend = warp_begin(d, warp + 1);

    // 1. first weight fragments (and their x offsets) in flight
    const uint4* vals = reinterpret_cast<const uint4*>(a.values) + lane;
    uint4 w[kUnroll];
    int xo[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
        const int p = wbeg + u;
        if (p < wend) {
            w[u] = ldg_stream(vals + (size_t)p * 32);
            xo[u] = __ldg(a.xoff + p);
        }
    }

    // 2. group fetch of the whole pivoted x, once per CTA
    for (int i = tid; i <= d.s_count; i += kThreads) L.sstart[i] = __ldg(a.strip_start + d.s_first + i);
    const __half* x = static_cast<const __half*>(a.x);
    for (int j = tid; j < a.n_pad; j += kThreads) {
        const int idx = x_index(a, j);
        for (int b = 0; b < a.batch; ++b)
            xs[b * a.xs_stride + j] = idx >= 0 ? x[(size_t)b * a.ldx + idx] : __float2half(0.0f);
    }
    __syncthreads();

    // 3. stream this warp's share
    float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    auto park = [&](int slot) {
        float* r0 = L.segp + (slot * RG + g) * a.batch;
        float* r1 = r0 + 8 * a.batch;
        if (2 * t < a.batch) { r0[2 * t] = acc[0]; r1[2 * t] = acc[2]; }
        if (2 * t + 1 < a.batch) { r0[2 * t + 1] = acc[1]; r1[2 * t + 1] = acc[3]; }
    };
    if (wbeg < wend) {
        int ls = 0;
        while (ls + 1 < d.s_count && L.sstart[ls + 1] <= wbeg) ++ls;
        int seg_end = min(wend, L.sstart[ls + 1]);
        const bool has_x = g < a.batch;
        const __half* xrow = xs + g * a.xs_stride + 2 * t;
        for (int base = wbeg; base < wend; base += kUnroll) {
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const int p = base + u;
                if (p < wend) {
                    if (p == seg_end) {
                        park(ls + warp);
                        acc[0] = acc[1] = acc[2] = acc[3] = 0.0f;
                        do { ++ls; } while (L.sstart[ls + 1] <= p);
                        seg_end = min(wend, L.sstart[ls + 1]);
                    }
                    const uint4 wa = w[u];
                    const int xoff = xo[u];
                    if (p + kUnroll < wend) {
                        w[u] = ldg_stream(vals + (size_t)(p + kUnroll) * 32);
                        xo[u] = __ldg(a.xoff + p + kUnroll);
                    }
                    uint32_t b0 = 0u, b1 = 0u;
                    if (has_x) {
                        b0 = *reinterpret_cast<const uint32_t*>(xrow + xoff);
                        b1 = *reinterpret_cast<const uint32_t*>(xrow + xoff + 8);
                    }
                    mma_16x8x16(acc, wa, b0, b1);
                }
            }
        }
        park(ls + warp);
    }
    __syncthreads();
    finalize<RG>(a, d, L);
}

// ------------------------------------------------------------------ fp32 tiles
template <int RG, int NB>
__global__ void __launch_bounds__(kThreads, 2) stream_f32_kernel(const StreamArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const SmemLayout L = carve(smem_raw, RG, a.batch);
    float* xs = static_cast<float*>(L.xs);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int4 dd = __ldg(reinterpret_cast<const int4*>(a.cta_desc) + blockIdx.x);
    const CtaDesc d{dd.x, dd.y, dd.z, dd.w};
    const int wbeg = warp_begin(d, warp), wend = warp_begin(d, warp + 1);

    const uint4* vals = reinterpret_cast<const uint4*>(a.values) + lane;
    uint4 w[kUnroll];
    int xo[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
        const int p = wbeg + u;
        if (p < wend) {
            w[u] = ldg_stream(vals + (size_t)p * 32);
            xo[u] = __ldg(a.xoff + p);
        }
    }

    for (int i = tid; i <= d.s_count; i += kThreads) L.sstart[i] = __ldg(a.strip_start + d.s_first + i);
    const float* x = static_cast<const float*>(a.x);
    for (int j = tid; j < a.n_pad; j += kThreads) {
        const int idx = x_index(a, j);
        for (int b = 0; b < a.batch; ++b)
            xs[b * a.xs_stride + j] = idx >= 0 ? __ldg(x + (size_t)b * a.ldx + idx) : 0.0f;
    }
    __syncthreads();

    float acc[NB][2];
#pragma unroll
    for (int b = 0; b < NB; ++b) acc[b][0] = acc[b][1] = 0.0f;
    auto park = [&](int slot) {
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            float v = acc[b][0] + acc[b][1];
            if (RG == 16) v += __shfl_xor_sync(0xffffffffu, v, 16);
            if (lane < RG && b < a.batch) L.segp[(slot * RG + lane) * a.batch + b] = v;
            acc[b][0] = acc[b][1] = 0.0f;
        }
    };
    if (wbeg < wend) {
        int ls = 0;
        while (ls + 1 < d.s_count && L.sstart[ls + 1] <= wbeg) ++ls;
        int seg_end = min(wend, L.sstart[ls + 1]);
        const float* xlane = xs + (lane / RG) * 4;
        for (int base = wbeg; base < wend; base += kUnroll) {
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const int p = base + u;
                if (p < wend) {
                    if (p == seg_end) {
                        park(ls + warp);
                        do { ++ls; } while (L.sstart[ls + 1] <= p);
                        seg_end = min(wend, L.sstart[ls + 1]);
                    }
                    const uint4 wa = w[u];
                    const int xoff = xo[u];
                    if (p + kUnroll < wend) {
                        w[u] = ldg_stream(vals + (size_t)(p + kUnroll) * 32);
                        xo[u] = __ldg(a.xoff + p + kUnroll);
                    }
                    const float w0 = __uint_as_float(wa.x), w1 = __uint_as_float(wa.y);
                    const float w2 = __uint_as_float(wa.z), w3 = __uint_as_float(wa.w);
#pragma unroll
                    for (int b = 0; b < NB; ++b) {
                        if (b < a.batch) {
                            const float4 xv = *reinterpret_cast<const float4*>(xlane + b * a.xs_stride + xoff);
                            acc[b][0] = fmaf(w0, xv.x, acc[b][0]);
                            acc[b][1] = fmaf(w1, xv.y, acc[b][1]);
                            acc[b][0] = fmaf(w2, xv.z, acc[b][0]);
                            acc[b][1] = fmaf(w3, xv.w, acc[b][1]);
                        }
                    }
                }
            }
        }
        park(ls + warp);
    }
    __syncthreads();
    finalize<RG>(a, d, L);
}

template <auto Kernel>
cudaError_t launch_one(const StreamArgs& a, int grid, size_t smem, cudaStream_t stream) {
    static bool configured = false;   // one flag per kernel instantiation
    if (smem > kStreamSmemLimit) return cudaErrorInvalidValue;
    if (!configured && smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(Kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)kStreamSmemLimit);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    Kernel<<<grid, kThreads, smem, stream>>>(a);
    return cudaGetLastError();
}

template <int RG>
cudaError_t launch_f32(const StreamArgs& a, int grid, size_t smem, cudaStream_t stream) {
    if (a.batch == 1) return launch_one<stream_f32_kernel<RG, 1>>(a, grid, smem, stream);
    if (a.batch == 2) return launch_one<stream_f32_kernel<RG, 2>>(a, grid, smem, stream);
    if (a.batch <= 4) return launch_one<stream_f32_kernel<RG, 4>>(a, grid, smem, stream);
    return launch_one<stream_f32_kernel<RG, 8>>(a, grid, smem, stream);
}

int xs_stride_for(pp_dtype_t dt, int n_pad) { return dt == PP_F16 ? n_pad + 8 : n_pad + 4; }

}  // namespace

size_t stream_smem_bytes(pp_dtype_t dt, int B, int n_pad, int batch) {
    const int rg = frag_geom(dt, B).rg_rows;
    const size_t esz = dt == PP_F16 ? 2 : 4;
    return (size_t)kHeaderWords * 4 + (size_t)kStreamSegSlots * rg * batch * 4 +
           (size_t)batch * xs_stride_for(dt, n_pad) * esz + 16;
}

cudaError_t launch_stream(pp_dtype_t dt, int B, const StreamArgs& a_in, int grid, cudaStream_t stream) {
    if (grid <= 0) return cudaSuccess;
    StreamArgs a = a_in;
    if (a.batch < 1 || a.batch > kStreamMaxBatch) return cudaErrorInvalidValue;
    a.xs_stride = xs_stride_for(dt, a.n_pad);
    const size_t smem = stream_smem_bytes(dt, B, a.n_pad, a.batch);
    if (dt == PP_F16) return launch_one<stream_f16_kernel>(a, grid, smem, stream);
    return B < 32 ? launch_f32<16>(a, grid, smem, stream) : launch_f32<32>(a, grid, smem, stream);
}

}  // namespace pp
