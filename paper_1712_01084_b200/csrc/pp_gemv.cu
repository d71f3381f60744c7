// Streaming block-sparse matrix-vector kernels for sm_100a (batch 1 .. 32).
//
// One CTA (8 warps) per work item = a run of consecutive kept tiles of one
// block-row.  The CTA follows Listing 1: group-fetch the x segment of its tiles
// through the column index array into shared memory, multiply, and store through
// the row index array -- with two changes for this GPU:
//   * the tile values are pre-ordered on the host into 512-byte fragments so that
//     every 128-bit load of a warp is contiguous, and each warp keeps kUnroll such
//     loads in flight (the weight loads are issued BEFORE the x gather so the two
//     latencies overlap);
//   * tiles that share a block-row (Section 4.1.5) are reduced in a fixed order:
//     across the warps of a CTA through shared memory, and across the CTAs of a
//     split block-row through per-part partial sums that the last-arriving CTA
//     adds in part order -- results do not depend on scheduling.
// fp16 tiles use the warp-level 16x8x16 tensor-core instruction with the batch as
// the 8-wide dimension (fp16 x fp16 products are exact in the fp32 accumulator);
// fp32 tiles use plain fp32 FMAs (no TF32 anywhere).
#include <cuda_fp16.h>

#include "pp_gemv.cuh"

namespace pp {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
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

__device__ __forceinline__ void cp_async_4(void* smem_dst, const void* gsrc, bool valid) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    const int n = valid ? 4 : 0;   // src-size 0 -> the 4 destination bytes are zero-filled
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" :: "r"(d), "l"(gsrc), "r"(n));
}

__device__ __forceinline__ WorkItem load_item(const WorkItem* items, int idx) {
    const int4* p = reinterpret_cast<const int4*>(items + idx);
    const int4 a = __ldg(p), b = __ldg(p + 1);
    WorkItem it;
    it.frag_base = a.x; it.rg_stride = a.y; it.nf = a.z; it.col_off = a.w;
    it.ntiles = b.x; it.br = b.y; it.part_nparts = b.z; it.slot_base = b.w;
    return it;
}

// Pivoted column pj -> index into x (or -1).
__device__ __forceinline__ int x_index(const GemvArgs& a, int pj) {
    if (a.gather_idx) return __ldg(a.gather_idx + pj);
    return pj < a.x_limit ? pj : -1;
}

// Tail shared by both kernels.  red holds per-warp partial sums as
// red[(warp * RG + row_in_group) * NC + b]; warps [rg*WPR, (rg+1)*WPR) cover row-group rg.
template <int B, int RG, int WPR, int NC>
__device__ __forceinline__ void reduce_and_store(const GemvArgs& a, const WorkItem& it, const float* red,
                                                 int* s_flag) {
    const int tid = threadIdx.x;
    const int batch = a.batch;
    const int part = it.part_nparts & 0xffff, nparts = it.part_nparts >> 16;
    const int n_out = B * batch;

    auto emit = [&](int r, int b, float v) {
        const int i = it.br * B + r;
        v += __ldg(a.bias_piv + i);
        if (a.act == PP_ACT_RELU) v = fmaxf(v, 0.0f);
        if (a.out_mode == OUT_SCATTER_F32 || a.out_mode == OUT_SCATTER_F16) {
            const int dst = __ldg(a.scatter_idx + i);
            if (dst >= 0) {
                if (a.out_mode == OUT_SCATTER_F32) static_cast<float*>(a.y)[(size_t)b * a.ldy + dst] = v;
                else static_cast<__half*>(a.y)[(size_t)b * a.ldy + dst] = __float2half_rn(v);
            }
        } else if (a.out_mode == OUT_PIVOTED_F32) {
            static_cast<float*>(a.y)[(size_t)b * a.ldy + i] = v;
        } else {
            static_cast<__half*>(a.y)[(size_t)b * a.ldy + i] = __float2half_rn(v);
        }
    };
    auto cta_sum = [&](int r, int b) {
        const int rg = r / RG, rr = r % RG;
        float v = 0.0f;
#pragma unroll
        for (int ws = 0; ws < WPR; ++ws) v += red[((rg * WPR + ws) * RG + rr) * NC + b];
        return v;
    };

    if (nparts == 1) {
        for (int e = tid; e < n_out; e += kThreads) {
            const int r = e / batch, b = e - r * batch;
            emit(r, b, cta_sum(r, b));
        }
        return;
    }
    // split block-row: publish this part, the last part to arrive adds all parts in order
    float* slot = a.partials + (size_t)(it.slot_base + part) * (B * kMaxGroupBatch);
    for (int e = tid; e < n_out; e += kThreads) {
        const int r = e / batch, b = e - r * batch;
        slot[e] = cta_sum(r, b);
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int old = atomicAdd(a.counters + it.br, 1);
        *s_flag = (old == nparts - 1);
    }
    __syncthreads();
    if (!*s_flag) return;
    __threadfence();
    const float* base = a.partials + (size_t)it.slot_base * (B * kMaxGroupBatch);
    for (int e = tid; e < n_out; e += kThreads) {
        float v = 0.0f;
        for (int p = 0; p < nparts; ++p) v += ld_cg(base + (size_t)p * (B * kMaxGroupBatch) + e);
        const int r = e / batch, b = e - r * batch;
        emit(r, b, v);
    }
    if (tid == 0) a.counters[it.br] = 0;   // ready for the next launch on this stream
}

// ------------------------------------------------------------------ fp16 tiles
template <int B, int NT>
__global__ void __launch_bounds__(kThreads) gemv_f16_kernel(const GemvArgs a) {
    constexpr int NRG = B / 16, WPR = kWarps / NRG, NC = NT * 8;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ int s_flag;
    float* red = reinterpret_cast<float*>(smem_raw);                       // [kWarps][16][NC]
    __half* xs = reinterpret_cast<__half*>(smem_raw + kWarps * 16 * NC * 4);  // [batch][xs_stride]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rg = warp / WPR, ws = warp % WPR;
    const int g = lane >> 2, t = lane & 3;
    const WorkItem it = load_item(a.items, blockIdx.x);
    const int nf = it.nf;

    // 1. first weight fragments in flight
    const uint4* wbase = reinterpret_cast<const uint4*>(a.values) +
                         ((size_t)it.frag_base + (size_t)rg * it.rg_stride) * 32 + lane;
    uint4 w[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
        const int i = ws + u * WPR;
        if (i < nf) w[u] = ldg_stream(wbase + (size_t)i * 32);
    }

    // 2. group fetch: x segment of this run's tiles through the column index array
    const int nk = it.ntiles * B;
    const __half* x = static_cast<const __half*>(a.x);
    for (int c = tid; c < nk; c += kThreads) {
        const int col = __ldg(a.tile_col + it.col_off + c / B);
        const int idx = x_index(a, col * B + (c % B));
        for (int b = 0; b < a.batch; ++b)
            xs[b * a.xs_stride + c] = idx >= 0 ? x[(size_t)b * a.ldx + idx] : __float2half(0.0f);
    }
    __syncthreads();

    // 3. stream the fragments
    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[nt][q] = 0.0f;

    for (int i0 = ws; i0 < nf; i0 += kUnroll * WPR) {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int i = i0 + u * WPR;
            if (i < nf) {
                const uint4 wa = w[u];
                const int nxt = i + kUnroll * WPR;
                if (nxt < nf) w[u] = ldg_stream(wbase + (size_t)nxt * 32);
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const int n = nt * 8 + g;
                    uint32_t b0 = 0u, b1 = 0u;
                    if (n < a.batch) {
                        const __half* xp = xs + n * a.xs_stride + i * 16 + 2 * t;
                        b0 = *reinterpret_cast<const uint32_t*>(xp);
                        b1 = *reinterpret_cast<const uint32_t*>(xp + 8);
                    }
                    mma_16x8x16(acc[nt], wa, b0, b1);
                }
            }
        }
    }

    // 4. per-warp partial sums -> shared memory
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        float* r0 = red + (warp * 16 + g) * NC + nt * 8 + 2 * t;
        r0[0] = acc[nt][0]; r0[1] = acc[nt][1];
        r0[8 * NC] = acc[nt][2]; r0[8 * NC + 1] = acc[nt][3];
    }
    __syncthreads();
    reduce_and_store<B, 16, WPR, NC>(a, it, red, &s_flag);
}

// ------------------------------------------------------------------ fp32 tiles
template <int B, int NB>
__global__ void __launch_bounds__(kThreads) gemv_f32_kernel(const GemvArgs a) {
    constexpr int RG = B < 32 ? B : 32, KF = 128 / RG, NRG = B / RG, WPR = kWarps / NRG;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ int s_flag;
    float* red = reinterpret_cast<float*>(smem_raw);                 // [kWarps][RG][NB]
    float* xs = red + kWarps * RG * NB;                              // [batch][xs_stride]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int rg = warp / WPR, ws = warp % WPR;
    const WorkItem it = load_item(a.items, blockIdx.x);
    const int nf = it.nf;

    const uint4* wbase = reinterpret_cast<const uint4*>(a.values) +
                         ((size_t)it.frag_base + (size_t)rg * it.rg_stride) * 32 + lane;
    uint4 w[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
        const int i = ws + u * WPR;
        if (i < nf) w[u] = ldg_stream(wbase + (size_t)i * 32);
    }

    // group fetch with 4-byte asynchronous copies (padding columns are zero-filled)
    const int nk = it.ntiles * B;
    const float* x = static_cast<const float*>(a.x);
    for (int c = tid; c < nk; c += kThreads) {
        const int col = __ldg(a.tile_col + it.col_off + c / B);
        const int idx = x_index(a, col * B + (c % B));
        for (int b = 0; b < a.batch; ++b)
            cp_async_4(xs + b * a.xs_stride + c, x + (size_t)b * a.ldx + (idx >= 0 ? idx : 0), idx >= 0);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();

    float acc[NB][2];
#pragma unroll
    for (int b = 0; b < NB; ++b) acc[b][0] = acc[b][1] = 0.0f;
    const int xoff = (lane / RG) * 4;    // 16-row tiles: upper half-warp takes columns 4..7 of the fragment

    for (int i0 = ws; i0 < nf; i0 += kUnroll * WPR) {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int i = i0 + u * WPR;
            if (i < nf) {
                const uint4 wa = w[u];
                const int nxt = i + kUnroll * WPR;
                if (nxt < nf) w[u] = ldg_stream(wbase + (size_t)nxt * 32);
                const float w0 = __uint_as_float(wa.x), w1 = __uint_as_float(wa.y);
                const float w2 = __uint_as_float(wa.z), w3 = __uint_as_float(wa.w);
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    if (b < a.batch) {
                        const float4 xv = *reinterpret_cast<const float4*>(xs + b * a.xs_stride + i * KF + xoff);
                        acc[b][0] = fmaf(w0, xv.x, acc[b][0]);
                        acc[b][1] = fmaf(w1, xv.y, acc[b][1]);
                        acc[b][0] = fmaf(w2, xv.z, acc[b][0]);
                        acc[b][1] = fmaf(w3, xv.w, acc[b][1]);
                    }
                }
            }
        }
    }

#pragma unroll
    for (int b = 0; b < NB; ++b) {
        float v = acc[b][0] + acc[b][1];
        if (RG == 16) v += __shfl_xor_sync(0xffffffffu, v, 16);
        if (lane < RG) red[(warp * RG + lane) * NB + b] = v;
    }
    __syncthreads();
    reduce_and_store<B, RG, WPR, NB>(a, it, red, &s_flag);
}

template <auto Kernel>
cudaError_t launch_one(const GemvArgs& a, int n_items, size_t smem, cudaStream_t stream) {
    static PerDeviceOnce configured;   // one table per kernel instantiation (Kernel is a template argument)
    if (smem > 200 * 1024) return cudaErrorInvalidValue;
    if (smem > 48 * 1024) {
        int dev = -1;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (!configured.is_done(dev)) {
            e = cudaFuncSetAttribute(Kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
            if (e != cudaSuccess) return e;
            configured.mark(dev);
        }
    }
    Kernel<<<n_items, kThreads, smem, stream>>>(a);
    return cudaGetLastError();
}

template <int B>
cudaError_t launch_f16(const GemvArgs& a, int n_items, cudaStream_t stream) {
    const int nt = (a.batch + 7) / 8;
    const size_t xs_bytes = (size_t)a.batch * a.xs_stride * 2;
    if (nt == 1) return launch_one<gemv_f16_kernel<B, 1>>(a, n_items, kWarps * 16 * 8 * 4 + xs_bytes, stream);
    if (nt == 2) return launch_one<gemv_f16_kernel<B, 2>>(a, n_items, kWarps * 16 * 16 * 4 + xs_bytes, stream);
    return launch_one<gemv_f16_kernel<B, 4>>(a, n_items, kWarps * 16 * 32 * 4 + xs_bytes, stream);
}

template <int B>
cudaError_t launch_f32(const GemvArgs& a, int n_items, cudaStream_t stream) {
    constexpr int RG = B < 32 ? B : 32;
    const size_t xs_bytes = (size_t)a.batch * a.xs_stride * 4;
    if (a.batch == 1) return launch_one<gemv_f32_kernel<B, 1>>(a, n_items, kWarps * RG * 1 * 4 + xs_bytes, stream);
    if (a.batch == 2) return launch_one<gemv_f32_kernel<B, 2>>(a, n_items, kWarps * RG * 2 * 4 + xs_bytes, stream);
    if (a.batch <= 4) return launch_one<gemv_f32_kernel<B, 4>>(a, n_items, kWarps * RG * 4 * 4 + xs_bytes, stream);
    return launch_one<gemv_f32_kernel<B, 8>>(a, n_items, kWarps * RG * 8 * 4 + xs_bytes, stream);
}

}  // namespace

cudaError_t launch_gemv(pp_dtype_t dt, int B, const GemvArgs& a_in, int n_items, int max_item_tiles,
                        cudaStream_t stream) {
    if (n_items <= 0) return cudaSuccess;
    GemvArgs a = a_in;
    if (a.batch < 1 || a.batch > gemv_group_batch(dt)) return cudaErrorInvalidValue;
    if (dt == PP_F16) {
        a.xs_stride = max_item_tiles * B + 8;   // +4 words: rows of the staged x land on distinct banks
        switch (B) {
            case 16: return launch_f16<16>(a, n_items, stream);
            case 32: return launch_f16<32>(a, n_items, stream);
            case 64: return launch_f16<64>(a, n_items, stream);
        }
    } else {
        a.xs_stride = max_item_tiles * B + 4;
        switch (B) {
            case 16: return launch_f32<16>(a, n_items, stream);
            case 32: return launch_f32<32>(a, n_items, stream);
            case 64: return launch_f32<64>(a, n_items, stream);
        }
    }
    return cudaErrorInvalidValue;
}

}  // namespace pp
