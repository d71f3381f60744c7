// Batched tile path for sm_100a (fp16 layers with B = 64, batch >= 64): every kept tile is a real
// dense contraction, so it runs on the 5th-generation tensor cores.
//
// Per block-row the kernel accumulates  D[128 x 64] += X_piv_seg[128 x 64] * W_tile^T  over the
// block-row's kept tiles: the batch chunk (128 rows of the permuted input) is the M side, the
// tile's 64 output rows the N side, the tile's 64 columns the K side (4 instructions of K = 16).
//   * Listing 1's group fetch is a pre-pass (gather_x_kernel): x_piv[b][j] = x[b][gather_idx[j]],
//     one CTA per batch row through shared memory, written as one 16 KiB block per tile-column that
//     already has the 128-byte-swizzled shared-memory image the tensor core wants; the packer stores
//     every weight tile as such an image (8 KiB) too;
//   * warp 0 streams (X block, W tile) pairs into a ring of shared-memory stages with two bulk
//     asynchronous copies per tile (cp.async.bulk, one request each, no multicast), signalling
//     mbarriers (2-D tensor-map loads of 128-byte rows were request-rate bound: 60 us vs the
//     same data as two contiguous copies);
//   * warp 1 issues tcgen05.mma (kind::f16, accumulator in tensor memory) from shared-memory matrix
//     descriptors and frees each stage with tcgen05.commit;
//   * warps 2..5 read the accumulator with tcgen05.ld and run the fused epilogue: bias, activation,
//     store through the row index array (Listing 1's last step).
// Every wait on an mbarrier is bounded; on a time-out the kernel raises the layer's status word,
// stops issuing work, lets its outstanding copies land, frees its tensor memory and returns.
#include <cuda_fp16.h>

#include "pp_gemv.cuh"
#include "pp_tile.cuh"

namespace pp {
namespace {

constexpr int kStages = 8;
constexpr int kProducers = 4;      // lanes of warp 0 that issue bulk copies (kStages is a multiple of it)
constexpr int kXBytes = kTileBatch * 64 * 2;     // 128 x 64 fp16 = 16 KiB
constexpr int kWBytes = 64 * 64 * 2;             // 64 x 64 fp16 = 8 KiB
constexpr int kStageBytes = kXBytes + kWBytes;
constexpr int kTmemCols = 64;
constexpr int kThreads = 192;
constexpr int kPollLimit = 1 << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* b, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(b)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* b, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* b) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* b, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false after kPollLimit polls, or at once when another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity, volatile int* abort_flag) {
    for (int i = 0; i < kPollLimit; ++i) {
        if (mbar_try_wait(b, parity)) return true;
        if ((i & 1023) == 1023 && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}

__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes, 8-row groups
// 1024 bytes apart (stride byte offset), descriptor version 1.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3fff);
    d |= (uint64_t)1 << 16;                       // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;             // stride byte offset
    d |= (uint64_t)1 << 46;                       // version
    d |= (uint64_t)2 << 61;                       // SWIZZLE_128B
    return d;
}

// Instruction descriptor: D = f32, A = B = f16, both K-major, N = 64, M = 128.
constexpr uint32_t kInstrDesc = (1u << 4) | ((64u >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, bool accumulate) {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.u32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
        :: "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(kInstrDesc), "r"((uint32_t)accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 :: "r"(smem_u32(bar)) : "memory");
}

struct TileSmem {
    uint64_t full[kStages];
    uint64_t empty[kStages];
    uint64_t acc_full;
    uint32_t tmem_base;
    int abort_flag;
};

__global__ void __launch_bounds__(kThreads, 1)
tile_f16_kernel(const TileArgs a) {
    extern __shared__ unsigned char smem_raw[];
    // stage buffers need 1024-byte alignment for the 128-byte swizzle
    unsigned char* stages = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    TileSmem* sm = reinterpret_cast<TileSmem*>(stages + kStages * kStageBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int br = blockIdx.x;
    const int t0 = __ldg(a.row_ptr + br), k = __ldg(a.row_ptr + br + 1) - t0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&sm->full[s], 1); mbar_init(&sm->empty[s], 1); }
        mbar_init(&sm->acc_full, 1);
        sm->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(smem_u32(&sm->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = sm->tmem_base;
    volatile int* abort_flag = &sm->abort_flag;

    if (warp == 0) {
        // ---------------- producers: kProducers lanes, lane p feeds tiles p, p + kProducers, ...
        // (one thread issues a bulk copy every ~0.15 us at best, which alone would cap the CTA)
        if (lane < kProducers) {
            int last = -1;
            const int cbase = __ldg(a.col_ptr + br);
            const int rot = k > 0 ? (int)(((long long)br * k) / gridDim.x) : 0;
            for (int t = lane; t < k; t += kProducers) {
                const int s = t % kStages;
                if (t >= kStages && !mbar_wait(&sm->empty[s], ((t / kStages) & 1) ^ 1, abort_flag)) break;
                // block-rows start at different tiles of their lists, so that CTAs running side by side
                // do not all ask the L2 for the same X segment at the same moment
                const int tt = (t + rot) % k;
                const int col = __ldg(a.tile_col + cbase + tt);
                mbar_expect_tx(&sm->full[s], kStageBytes);
                bulk_load(stages + s * kStageBytes, a.x_sw + (size_t)col * kXBytes, kXBytes, &sm->full[s]);
                bulk_load(stages + s * kStageBytes + kXBytes, a.tiles_sw + (size_t)(t0 + tt) * kWBytes, kWBytes, &sm->full[s]);
                last = t;
            }
            if (*abort_flag) {
                // let this lane's copies still in flight land before shared memory goes away
                for (int t = last; t >= 0 && t > last - kStages; t -= kProducers)
                    for (int i = 0; i < kPollLimit && !mbar_try_wait(&sm->full[t % kStages], (t / kStages) & 1); ++i) {}
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (one lane)
        if (lane == 0) {
            bool ok = true;
            for (int t = 0; t < k && ok; ++t) {
                const int s = t % kStages;
                ok = mbar_wait(&sm->full[s], (t / kStages) & 1, abort_flag);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t xa = smem_u32(stages + s * kStageBytes), wa = xa + kXBytes;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    umma_f16(tmem, smem_desc_sw128(xa + kk * 32), smem_desc_sw128(wa + kk * 32), t > 0 || kk > 0);
                umma_commit(&sm->empty[s]);          // frees the stage once these MMAs have read it
            }
            if (k > 0 && ok) umma_commit(&sm->acc_full);   // accumulator complete
            else mbar_arrive(&sm->acc_full);               // nothing to wait for (no tile, or giving up)
        }
    } else {
        // ---------------- epilogue: 4 warps, warp (w % 4) owns tensor-memory lanes 32 (w % 4) ..
        const int q = warp & 3;
        // the tensor-memory loads below are warp-wide instructions: the whole warp takes one decision
        const bool ok = __all_sync(0xffffffffu, mbar_wait(&sm->acc_full, 0, abort_flag) && !*abort_flag);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int b = q * 32 + lane;                 // batch row inside the chunk
        if (ok) {
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t r[32];
                if (k > 0) {
                    asm volatile(
                        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                        : "r"(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)c0));
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = 0u;
                }
                if (b < a.batch) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const int i = br * 64 + c0 + j;
                        float v = __uint_as_float(r[j]) + __ldg(a.bias_piv + i);
                        if (a.act == PP_ACT_RELU) v = fmaxf(v, 0.0f);
                        const int dst = __ldg(a.scatter_idx + i);
                        if (dst >= 0) a.y[(size_t)b * a.ldy + dst] = v;
                    }
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0 && sm->abort_flag) *a.status = 1;
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// Byte offset of element (row r, column c) inside a 128-byte-swizzled block of 128-byte rows:
// the 16-byte chunk index is XOR-ed with the row index modulo 8.
__host__ __device__ __forceinline__ uint32_t sw128_offset(int r, int c) {
    return (uint32_t)r * 128u + (uint32_t)(((c >> 3) ^ (r & 7)) << 4) + (uint32_t)(c & 7) * 2u;
}

// x_piv[b][j] = x[b][gather_idx[j]] for the rows of one batch chunk; rows past the batch and padding
// columns are zero.  One CTA per row: the row goes to shared memory coalesced and leaves permuted, into
// the swizzled 16 KiB block of its tile-column (row b of the block).
__global__ void gather_x_kernel(const __half* __restrict__ x, int ldx, int n, const int32_t* __restrict__ gather_idx,
                                int n_pad, unsigned char* __restrict__ x_sw, int batch) {
    extern __shared__ __half row[];
    const int b = blockIdx.x;
    if (b < batch) {
        // 16-byte copies where the row allows it (base and pitch 16-byte aligned), element copies otherwise
        const __half* src = x + (size_t)b * ldx;
        const bool vec = ((reinterpret_cast<uintptr_t>(src) & 15u) == 0);
        const int n8 = vec ? n / 8 : 0;
        for (int i = threadIdx.x; i < n8; i += blockDim.x)
            reinterpret_cast<uint4*>(row)[i] = __ldg(reinterpret_cast<const uint4*>(src) + i);
        for (int j = n8 * 8 + threadIdx.x; j < n; j += blockDim.x) row[j] = src[j];
    }
    __syncthreads();
    // 8 independent index loads per thread before the first use, so their latencies overlap
    for (int j0 = threadIdx.x; j0 < n_pad; j0 += 8 * blockDim.x) {
        int idx[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int j = j0 + q * blockDim.x;
            idx[q] = (b < batch && j < n_pad) ? __ldg(gather_idx + j) : -1;
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int j = j0 + q * blockDim.x;
            if (j < n_pad) {
                const __half v = idx[q] >= 0 ? row[idx[q]] : __float2half(0.0f);
                *reinterpret_cast<__half*>(x_sw + (size_t)(j >> 6) * kXBytes + sw128_offset(b, j & 63)) = v;
            }
        }
    }
}

}  // namespace

void swizzle_tile_64x64(const void* row_major, void* out) {
    const unsigned char* src = static_cast<const unsigned char*>(row_major);
    unsigned char* dst = static_cast<unsigned char*>(out);
    for (int r = 0; r < 64; ++r)
        for (int ch = 0; ch < 8; ++ch)
            for (int k = 0; k < 16; ++k) dst[r * 128 + ((ch ^ (r & 7)) << 4) + k] = src[r * 128 + ch * 16 + k];
}

cudaError_t launch_tile(const TileArgs& a, const void* x, int ldx, int n, const int32_t* gather_idx, int n_pad, int Mb,
                        cudaStream_t stream) {
    if (a.batch < 1 || a.batch > kTileBatch) return cudaErrorInvalidValue;
    static bool configured = false;
    const size_t smem = (size_t)kStages * kStageBytes + sizeof(TileSmem) + 1024;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(tile_f16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    if ((size_t)n * 2 > 48 * 1024) return cudaErrorInvalidValue;
    gather_x_kernel<<<kTileBatch, 1024, ((size_t)n * 2 + 15) / 16 * 16, stream>>>(static_cast<const __half*>(x), ldx, n, gather_idx, n_pad,
                                                              const_cast<unsigned char*>(a.x_sw), a.batch);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    tile_f16_kernel<<<Mb, kThreads, smem, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace pp
