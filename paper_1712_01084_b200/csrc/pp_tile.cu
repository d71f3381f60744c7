// Batched tile path for sm_100a (fp16 layers with B = 64, batch >= 64): every kept tile is a real
// dense contraction, so it runs on the 5th-generation tensor cores.
//
// Per block-row the kernel accumulates  D[128 x 64] += X_piv_seg[128 x 64] * W_tile^T  over the
// block-row's kept tiles: the batch chunk (128 rows of the permuted input) is the M side, the
// tile's 64 output rows the N side, the tile's 64 columns the K side (4 instructions of K = 16).
//   * Listing 1's group fetch is a pre-pass (gather_x_kernel): x_piv[b][j] = x[b][gather_idx[j]],
//     one CTA per batch row, through shared memory so that both sides are coalesced;
//   * warp 0 streams (X segment, W tile) pairs into a ring of shared-memory stages with TMA
//     (cp.async.bulk.tensor, 128-byte swizzle, no multicast), signalling mbarriers;
//   * warp 1 issues tcgen05.mma (kind::f16, accumulator in tensor memory) from shared-memory matrix
//     descriptors and frees each stage with tcgen05.commit;
//   * warps 2..5 read the accumulator with tcgen05.ld and run the fused epilogue: bias, activation,
//     store through the row index array (Listing 1's last step).
// Every wait on an mbarrier is bounded; on a time-out the kernel raises the layer's status word,
// stops issuing work, lets its outstanding copies land, frees its tensor memory and returns.
#include <cuda.h>
#include <cuda_fp16.h>

#include <new>

#include "pp_gemv.cuh"
#include "pp_tile.cuh"

namespace pp {
namespace {

constexpr int kStages = 6;
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

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int c0, int c1, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 :: "r"(smem_u32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(smem_u32(bar)) : "memory");
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
tile_f16_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, const TileArgs a) {
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
        // ---------------- TMA producer (one lane)
        if (lane == 0) {
            int issued = 0;
            for (int t = 0; t < k; ++t) {
                const int s = t % kStages;
                if (t >= kStages && !mbar_wait(&sm->empty[s], ((t / kStages) & 1) ^ 1, abort_flag)) break;
                const int col = __ldg(a.tile_col + __ldg(a.col_ptr + br) + t);
                mbar_expect_tx(&sm->full[s], kStageBytes);
                tma_load_2d(stages + s * kStageBytes, &map_x, col * 64, 0, &sm->full[s]);
                tma_load_2d(stages + s * kStageBytes + kXBytes, &map_w, 0, (t0 + t) * 64, &sm->full[s]);
                issued = t + 1;
            }
            if (*abort_flag) {
                // let the copies still in flight land before shared memory goes away
                for (int t = issued > kStages ? issued - kStages : 0; t < issued; ++t)
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

// x_piv[b][j] = x[b][gather_idx[j]] for the rows of one batch chunk; rows past the batch and padding
// columns are zero.  One CTA per row: the row goes to shared memory coalesced and leaves permuted.
__global__ void gather_x_kernel(const __half* __restrict__ x, int ldx, int n, const int32_t* __restrict__ gather_idx,
                                int n_pad, __half* __restrict__ x_piv, int batch) {
    extern __shared__ __half row[];
    const int b = blockIdx.x;
    __half* out = x_piv + (size_t)b * n_pad;
    if (b >= batch) {
        for (int j = threadIdx.x; j < n_pad; j += blockDim.x) out[j] = __float2half(0.0f);
        return;
    }
    for (int j = threadIdx.x; j < n; j += blockDim.x) row[j] = x[(size_t)b * ldx + j];
    __syncthreads();
    for (int j = threadIdx.x; j < n_pad; j += blockDim.x) {
        const int idx = __ldg(gather_idx + j);
        out[j] = idx >= 0 ? row[idx] : __float2half(0.0f);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

bool encode_2d(CUtensorMap* map, void* base, uint64_t cols, uint64_t rows, uint32_t box_cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) ==
           CUDA_SUCCESS;
}

}  // namespace

struct TilePlan {
    CUtensorMap map_x, map_w;
    bool has_w;
};

TilePlan* tile_plan_create(void* d_tiles_rm, int64_t T, void* d_x_piv, int n_pad) {
    TilePlan* p = new (std::nothrow) TilePlan();
    if (!p) return nullptr;
    p->has_w = T > 0;
    bool ok = encode_2d(&p->map_x, d_x_piv, (uint64_t)n_pad, kTileBatch, 64, kTileBatch);
    if (ok && T > 0) ok = encode_2d(&p->map_w, d_tiles_rm, 64, (uint64_t)T * 64, 64, 64);
    if (ok && T == 0) p->map_w = p->map_x;      // never dereferenced: no block-row has a tile
    if (!ok) { delete p; return nullptr; }
    return p;
}

void tile_plan_destroy(TilePlan* p) { delete p; }

cudaError_t launch_tile(const TilePlan* plan, const TileArgs& a, const void* x, int ldx, int n, const int32_t* gather_idx,
                        int n_pad, void* d_x_piv, int Mb, cudaStream_t stream) {
    if (a.batch < 1 || a.batch > kTileBatch) return cudaErrorInvalidValue;
    static bool configured = false;
    const size_t smem = (size_t)kStages * kStageBytes + sizeof(TileSmem) + 1024;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(tile_f16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    if ((size_t)n * 2 > 200 * 1024) return cudaErrorInvalidValue;
    gather_x_kernel<<<kTileBatch, 256, (size_t)n * 2, stream>>>(static_cast<const __half*>(x), ldx, n, gather_idx, n_pad,
                                                              static_cast<__half*>(d_x_piv), a.batch);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    tile_f16_kernel<<<Mb, kThreads, smem, stream>>>(plan->map_x, plan->map_w, a);
    return cudaGetLastError();
}

}  // namespace pp
