// Batched tile path for sm_100a (fp16 layers with B = 64, batch > 8): every kept tile is a real
// dense contraction, so it runs on the 5th-generation tensor cores.
//
// Per block-row the kernel accumulates  D[128 x 64] += X_piv_seg[128 x 64] * W_tile^T  over the
// block-row's kept tiles: the batch chunk (128 rows of the permuted input) is the M side, the
// tile's 64 output rows the N side, the tile's 64 columns the K side (4 instructions of K = 16).
//   * Listing 1's group fetch is a pre-pass (gather_x_kernel): x_piv[b][j] = x[b][gather_idx[j]],
//     one CTA per batch row through shared memory, written as one 16 KiB block per tile-column that
//     already has the 128-byte-swizzled shared-memory image the tensor core wants; the packer stores
//     every weight tile as such an image (8 KiB) too;
//   * warps 0..3 (one lane each) stream (X block, W tile) pairs into a ring of shared-memory stages
//     with two bulk asynchronous copies per tile (cp.async.bulk, one request each, every CTA fetching for itself),
//     signalling mbarriers (2-D tensor-map loads of 128-byte rows were request-rate bound: 60 us vs
//     the same data as two contiguous copies);
//   * warps 4..7 (one lane each) issue tcgen05.mma (kind::f16, accumulators in tensor memory) from
//     shared-memory matrix descriptors and free each stage with tcgen05.commit; the tiles go round robin to
//     the four warps, each with an accumulator of its own, because one thread cannot issue faster than
//     a tile per 0.28 us;
//   * warps 8..11 read the accumulators with tcgen05.ld, add them and run the fused epilogue: bias,
//     activation, store through the row index array (Listing 1's last step).
// A second kernel (further down) lets a cluster of four CTAs share the X blocks of four block-rows, a third
// gives every SM an equal share of the work; both are slower (measured) and run only on request.
// Every wait on an mbarrier is bounded; on a time-out the kernel raises the layer's status word,
// stops issuing work, lets its outstanding copies land, frees its tensor memory and returns.
#include <cuda_fp16.h>

#include "pp_gemv.cuh"
#include "pp_stream.cuh"
#include "pp_tile.cuh"

namespace pp {
namespace {

constexpr int kProducers = 4;      // producer warps (one lane each issues bulk copies; the stage count is a multiple of it)
constexpr int kXBytes = kTileBatch * 64 * 2;     // 128 x 64 fp16 = 16 KiB
constexpr int kWBytes = 64 * 64 * 2;             // 64 x 64 fp16 = 8 KiB
// One-block-row kernel: the thread that issues the tensor-core instructions spends about 0.16 us per tile on the
// hand-shake alone (wait for the stage, fence, commit) plus 0.03 us per instruction, whatever the instruction's
// shape and whether any data moves at all (measured with the copies and the instructions taken out in turn), while
// the copies of a tile take 0.17 us.  So kIssuers warps share the tiles of the block-row round robin, each with an
// accumulator of its own in tensor memory; the epilogue adds the accumulators in a fixed order.
constexpr int kIssuers = 4;
constexpr int kTmemCols = 64 * kIssuers;
constexpr int kThreads = 32 * (kProducers + kIssuers + 4);    // producers, MMA issuers, 4 epilogue warps
constexpr int kPollLimit = 1 << 22;
constexpr int kIdxCap = 512;       // tiles of a block-row whose indices are staged in shared memory

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
__device__ __forceinline__ bool mbar_test_wait(uint64_t* b, uint32_t parity) {     // never suspends the thread
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false after the poll limit, or at once when another role already gave up.  polls == 0 is the
// normal case (kPollLimit polls that may each suspend the thread for a while: seconds in all).  A caller-set
// limit counts polls that return at once, so that a test can make a wait run out on purpose.
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity, volatile int* abort_flag, int polls) {
    if (polls > 0) {
        for (int i = 0; i < polls; ++i) {
            if (mbar_test_wait(b, parity)) return true;
            if (*abort_flag) return false;
        }
        *abort_flag = 1;
        return false;
    }
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

// The descriptor of the same operand layout `bytes` further on (bytes a multiple of 16; shared-memory
// addresses stay below 256 KiB, so the 14-bit address field cannot carry into its neighbours).
__device__ __forceinline__ uint64_t desc_advance(uint64_t d, uint32_t bytes) { return d + (uint64_t)(bytes >> 4); }

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

#ifdef PP_TRACE
__device__ __forceinline__ void tile_stamp(const TileArgs& a, int slot) {
    if (a.trace) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t) :: "memory");
        a.trace[(size_t)blockIdx.x * 8 + slot] = t;
    }
}
#else
__device__ __forceinline__ void tile_stamp(const TileArgs&, int) {}
#endif

// STAGES stages of (XB bytes of the X block + one tile).  A stage is re-used once per STAGES tiles and a
// copy takes 1.5-2 us to land, so small batches (which need only the first 8-row groups of the X block)
// trade the unused part of the X region for more stages in flight.
template <int STAGES>
struct TileSmem {
    uint64_t full[STAGES];
    uint64_t empty[STAGES];
    uint64_t acc_full;
    uint32_t tmem_base;
    int abort_flag;
    float bias[64];           // bias and destination rows of the block-row
    int dst[64];
    int col[kIdxCap];         // tile-column and image position of the block-row's first kIdxCap tiles
    int pos[kIdxCap];
};

template <int STAGES, int XB>
__global__ void __launch_bounds__(kThreads, 1)
tile_f16_kernel(const TileArgs a) {
    constexpr int kStages = STAGES;
    constexpr int kStageBytes = XB + kWBytes;
    static_assert(STAGES % kProducers == 0 && XB % 1024 == 0 && XB <= kXBytes, "stage geometry");
    extern __shared__ unsigned char smem_raw[];
    // stage buffers need 1024-byte alignment for the 128-byte swizzle
    unsigned char* stages = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    // The A operand of every MMA spans 128 rows (16 KiB) from the start of its stage's X region, whatever XB is:
    // the rows past XB are dead batch rows read from the bytes that follow (the stage's tile, the next stage).
    // kXBytes - XB spare bytes behind the last stage keep that read inside the allocation.
    TileSmem<STAGES>* sm = reinterpret_cast<TileSmem<STAGES>*>(stages + kStages * kStageBytes + (kXBytes - XB));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int br = blockIdx.x;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next call's gather kernel may fetch its index entries meanwhile
    if (threadIdx.x == 0 && blockIdx.x < 148) tile_stamp(a, 0);
    const int t0 = __ldg(a.row_ptr + br), k = __ldg(a.row_ptr + br + 1) - t0;

    // The block-row's tile list goes to shared memory once, by the whole CTA, while tensor memory is set
    // up: a producer that fetched each tile's indices from global memory just before its copies spent one
    // L2 round trip per tile on that and capped the kernel at four tiles per round trip.
    {
        const int cbase0 = __ldg(a.col_ptr + br);
        for (int i = threadIdx.x; i < k && i < kIdxCap; i += kThreads) {
            sm->col[i] = __ldg(a.tile_col + cbase0 + i);
            sm->pos[i] = __ldg(a.tile_pos + t0 + i);
        }
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&sm->full[s], 1); mbar_init(&sm->empty[s], 1); }
        mbar_init(&sm->acc_full, kIssuers);
        sm->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kProducers) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(smem_u32(&sm->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = sm->tmem_base;
    volatile int* abort_flag = &sm->abort_flag;

    if (warp < kProducers) {
        // ---------------- producers: one lane of each of kProducers warps, warp p feeds tiles p, p + kProducers, ...
        // (a thread is held for a few hundred ns per bulk copy it issues, and the lanes of one warp would
        // take turns, so the requests come from different warps)
        if (lane == 0) {
            int last = -1;
            // Only the 8-row groups (1 KiB each) that hold live batch rows are fetched.  The rows of the
            // stage beyond them keep whatever they held: a row of the A operand only reaches its own row
            // of the accumulator, and rows past the batch are never stored.
            const uint32_t xbytes = (uint32_t)((a.batch + 7) / 8) * 1024u;
            const int cbase = __ldg(a.col_ptr + br);
            const int rot = k > 0 ? (int)(((long long)br * k) / gridDim.x) : 0;
            for (int t = warp; t < k; t += kProducers) {
                const int s = t % kStages;
                if (t >= kStages && !mbar_wait(&sm->empty[s], ((t / kStages) & 1) ^ 1, abort_flag, a.polls)) break;
                // block-rows start at different tiles of their lists, so that CTAs running side by side
                // do not all ask the L2 for the same X segment at the same moment
                const int tt = (t + rot) % k;
                const int col = tt < kIdxCap ? sm->col[tt] : __ldg(a.tile_col + cbase + tt);
                const int pos = tt < kIdxCap ? sm->pos[tt] : __ldg(a.tile_pos + t0 + tt);
                mbar_expect_tx(&sm->full[s], xbytes + kWBytes);
                bulk_load(stages + s * kStageBytes + XB, a.tiles_sw + (size_t)pos * kWBytes, kWBytes, &sm->full[s]);
                // the permuted input comes from the gather kernel launched just before: everything up to here
                // (set-up, the first weight copies) may overlap its tail
                if (t == warp) asm volatile("griddepcontrol.wait;" ::: "memory");
                bulk_load(stages + s * kStageBytes, a.x_sw + (size_t)col * kXBytes, xbytes, &sm->full[s]);
                last = t;
            }
            if (*abort_flag) {
                // let this lane's copies still in flight land before shared memory goes away
                for (int t = last; t >= 0 && t > last - kStages; t -= kProducers)
                    for (int i = 0; i < kPollLimit && !mbar_try_wait(&sm->full[t % kStages], (t / kStages) & 1); ++i) {}
            }
        }
    } else if (warp < kProducers + kIssuers) {
        // ---------------- MMA issuers (one lane each): issuer i takes tiles i, i + kIssuers, ... into accumulator i
        if (lane == 0) {
            const int me = warp - kProducers;
            const uint32_t acc = tmem + (uint32_t)(me * 64);
            bool ok = true, issued = false;
            const uint64_t desc0 = smem_desc_sw128(smem_u32(stages));
            for (int t = me; t < k && ok; t += kIssuers) {
                const int s = t % kStages;
                ok = mbar_wait(&sm->full[s], (t / kStages) & 1, abort_flag, a.polls);
                if (!ok) break;
                if (t == 0 && blockIdx.x < 148) tile_stamp(a, 1);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint64_t xd = desc_advance(desc0, (uint32_t)(s * kStageBytes)), wd = desc_advance(xd, XB);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    umma_f16(acc, desc_advance(xd, kk * 32), desc_advance(wd, kk * 32), issued || kk > 0);
                issued = true;
                umma_commit(&sm->empty[s]);          // frees the stage once these MMAs have read it
            }
            // this issuer's accumulator is complete; when giving up after some tiles, the epilogue (and the release
            // of tensor memory behind it) still waits for the instructions already issued
            if (issued) umma_commit(&sm->acc_full);
            else mbar_arrive(&sm->acc_full);               // nothing was issued: nothing to wait for
            if (me == 0 && blockIdx.x < 148) tile_stamp(a, 2);
        }
    } else {
        // ---------------- epilogue: 4 warps, warp (w % 4) owns tensor-memory lanes 32 (w % 4) ..
        const int q = warp & 3;
        const int b = q * 32 + lane;                 // batch row inside the chunk
        // while the main loop runs: bias and destination rows into shared memory (read by all four warps
        // after the named barrier below)
        if (b < 64) {
            sm->bias[b] = __ldg(a.bias_piv + br * 64 + b);
            sm->dst[b] = a.pivoted ? br * 64 + b : __ldg(a.scatter_idx + br * 64 + b);
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        // the tensor-memory loads below are warp-wide instructions: the whole warp takes one decision
        const bool ok = __all_sync(0xffffffffu, mbar_wait(&sm->acc_full, 0, abort_flag, 0) && !*abort_flag);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (threadIdx.x == 32 * (kProducers + kIssuers) && blockIdx.x < 148) tile_stamp(a, 3);
        if (ok && q * 32 < a.batch) {
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                // the sum of the accumulators that received tiles (issuer i did iff k > i), in issuer order
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = 0.0f;
#pragma unroll
                for (int i = 0; i < kIssuers; ++i) {
                    if (i < k) {                 // the same decision in every lane: the load is a warp-wide instruction
                        uint32_t r[32];
                        asm volatile(
                            "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                            "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                            "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                            : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                              "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                              "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                              "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                            : "r"(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(i * 64 + c0)));
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] += __uint_as_float(r[j]);
                    }
                }
                // Transpose the 32 x 32 block through shared memory (the stages are idle by now), so that the
                // lanes of a store run over output rows: 32 scattered words of ONE row of y.  With lanes over
                // batch rows the words of a store lie a whole row pitch apart and crowd a few L2 slices.
                float* xpose = reinterpret_cast<float*>(stages) + q * (32 * 33);
#pragma unroll
                for (int j = 0; j < 32; ++j) xpose[lane * 33 + j] = v[j];
                __syncwarp();
                const float bias = sm->bias[c0 + lane];
                const int dst = sm->dst[c0 + lane];
#pragma unroll 8
                for (int rr = 0; rr < 32; ++rr) {
                    const int bb = q * 32 + rr;
                    float o = xpose[rr * 33 + lane] + bias;
                    if (a.act == PP_ACT_RELU) o = fmaxf(o, 0.0f);
                    if (dst >= 0 && bb < a.batch) a.y[(size_t)bb * a.ldy + dst] = o;
                }
                __syncwarp();
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0 && blockIdx.x < 148) tile_stamp(a, 4);
    if (threadIdx.x == 0 && sm->abort_flag) *a.status = 1;
    if (warp == kProducers) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------
// Clustered variant.  With one block-row per CTA every CTA pulls the whole permuted input through
// its L2 port (2 MiB of X for 1 MiB of weights at 8192 columns), every tile costs two copy requests
// and every MMA re-reads its 128 x 16 slice of X from shared memory for just 64 output columns.
// Here kTileRows consecutive block-rows form a group computed by a cluster of kTileRows CTAs:
//   * CTA r owns a contiguous quarter of the group's tile-columns ("steps").  Per step it fetches
//     the X block ONCE and, with one more request, the tiles all block-rows of the group have in that
//     column (the packer stores them next to each other); four producer warps issue the requests;
//   * the block-rows' accumulators sit side by side in tensor memory (4 x 64 columns), so the tiles
//     of consecutive block-rows are the B operand of ONE instruction with N up to 256;
//   * at the end the cluster meets at its hardware barrier (everybody's stage buffers are free),
//     every CTA sends its partial accumulator of block-row j to CTA j with remote shared-memory
//     stores, the cluster meets again, and CTA j adds the four partials in rank order and runs the
//     epilogue for block-row j -- no global scratch, no atomics, the same bits on every run.
constexpr int kCStages = 4;
constexpr int kCProducers = 4;                                 // producer warps; warp w feeds stage w
constexpr int kCStageBytes = kXBytes + kTileRows * kWBytes;    // 48 KiB: one X block + up to 4 tiles
constexpr int kCTmemCols = 64 * kTileRows;
static_assert(kTileRows * 64 * kTileBatch * 4 + 4 * 32 * 33 * 4 <= kCStages * kCStageBytes, "exchange buffers reuse the stages");
__device__ __forceinline__ int q_of_warp(int warp) { return warp & 3; }
constexpr int kCThreads = 32 * (kCProducers + 1 + 4);          // producers, MMA issuer, 4 epilogue warps
constexpr int kStepCap = 96;                                   // step records of a CTA staged in shared memory
static_assert(kCStages == kCProducers, "one stage per producer warp");

struct ClusterSmem {
    uint64_t full[kCStages];
    uint64_t empty[kCStages];
    uint64_t acc_full;
    uint32_t tmem_base;
    int abort_flag;
    uint32_t acc_mask;        // accumulators that received at least one tile
    float bias[64];           // bias and destination rows of the block-row this CTA finishes
    int dst[64];
    int4 steps[kStepCap][2];  // this CTA's first kStepCap step records
};
static_assert(sizeof(TileStep) == 2 * sizeof(int4), "a step record is staged as two 16-byte words");

__device__ __forceinline__ TileStep load_step(const TileStep* p) {
    const int4 lo = __ldg(reinterpret_cast<const int4*>(p)), hi = __ldg(reinterpret_cast<const int4*>(p) + 1);
    TileStep s;
    s.col = lo.x; s.tile[0] = lo.y; s.tile[1] = lo.z; s.tile[2] = lo.w; s.tile[3] = hi.x; s.ntiles = hi.y; s.pos = hi.z;
    s.pad = 0;
    return s;
}
__device__ __forceinline__ TileStep unpack_step(const int4 lo, const int4 hi) {
    TileStep s;
    s.col = lo.x; s.tile[0] = lo.y; s.tile[1] = lo.z; s.tile[2] = lo.w; s.tile[3] = hi.x; s.ntiles = hi.y; s.pos = hi.z;
    s.pad = 0;
    return s;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t peer_addr(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    return remote;
}
__device__ __forceinline__ void st_peer_v4(uint32_t remote_addr, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" :: "r"(remote_addr), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
// tcgen05.mma with M = 128 and N = 64 * n_tiles (instruction descriptor built on the fly)
__device__ __forceinline__ void umma_f16_n(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, int n_tiles, bool accumulate) {
    const uint32_t idesc = (1u << 4) | (((uint32_t)(64 * n_tiles) >> 3) << 17) | ((128u >> 4) << 24);
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.u32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
        :: "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"((uint32_t)accumulate) : "memory");
}

__global__ void __cluster_dims__(kTileRows, 1, 1) __launch_bounds__(kCThreads, 1)
tile_cluster_f16_kernel(const TileArgs a) {
    static_assert(kTileRows == 4, "step records carry four tile slots");
    extern __shared__ unsigned char smem_raw[];
    unsigned char* stages = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    ClusterSmem* sm = reinterpret_cast<ClusterSmem*>(stages + kCStages * kCStageBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint32_t rank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next call's gather kernel may fetch its index entries meanwhile
    const int grp = blockIdx.x / kTileRows, n_groups = gridDim.x / kTileRows;
    const int p0 = __ldg(a.parts + grp * (kTileRows + 1) + rank);
    const int n_steps = __ldg(a.parts + grp * (kTileRows + 1) + rank + 1) - p0;
    // clusters start at different steps of their ranges, so that the CTAs of equal rank (which walk the
    // same tile-columns) do not all ask the L2 for the same X block at the same moment
    const int rot = n_steps > 0 ? (int)(((long long)grp * n_steps) / n_groups) : 0;

    // This CTA's step records go to shared memory once, by all threads, while tensor memory is set up: read
    // from global memory inside the loops they cost the producers and the MMA issuer one L2 round trip per step.
    for (int i = threadIdx.x; i < 2 * n_steps && i < 2 * kStepCap; i += kCThreads)
        sm->steps[i >> 1][i & 1] = __ldg(reinterpret_cast<const int4*>(a.steps + p0) + i);
    auto step_at = [&](int i) {
        return i < kStepCap ? unpack_step(sm->steps[i][0], sm->steps[i][1]) : load_step(a.steps + p0 + i);
    };
    if (threadIdx.x == 0) {
        for (int s = 0; s < kCStages; ++s) { mbar_init(&sm->full[s], 1); mbar_init(&sm->empty[s], 1); }
        mbar_init(&sm->acc_full, 2);          // the tensor core's commit + the issuing thread's own arrival
        sm->abort_flag = 0;
        sm->acc_mask = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kCProducers) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(smem_u32(&sm->tmem_base)), "r"(kCTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = sm->tmem_base;
    volatile int* abort_flag = &sm->abort_flag;
    // after the main loop the stage buffers hold what the peers send: [sender][16 row quads][128 batch][4]
    // floats (a warp's remote store is one contiguous 512-byte run), and behind them a 32 x 33
    // transposition tile per epilogue warp
    float* recv = reinterpret_cast<float*>(stages);
    float* xpose = recv + kTileRows * 64 * kTileBatch + q_of_warp(threadIdx.x >> 5) * (32 * 33);

    if (warp < kCProducers) {
        // ---------------- producers: warp w (one lane) feeds steps w, w + kCProducers, ... into stage w
        if (lane == 0) {
            const int s = warp;
            int last = -1;
            const uint32_t xbytes = (uint32_t)((a.batch + 7) / 8) * 1024u;   // live 8-row groups of the X block only
            for (int t = warp; t < n_steps; t += kCProducers) {
                if (t >= kCStages && !mbar_wait(&sm->empty[s], ((t / kCStages) & 1) ^ 1, abort_flag, a.polls)) break;
                const TileStep st = step_at((t + rot) % n_steps);
                unsigned char* dst = stages + s * kCStageBytes;
                mbar_expect_tx(&sm->full[s], xbytes + (uint32_t)(st.ntiles * kWBytes));
                bulk_load(dst + kXBytes, a.tiles_sw + (size_t)st.pos * kWBytes, (uint32_t)(st.ntiles * kWBytes), &sm->full[s]);
                // the permuted input comes from the gather kernel launched just before: everything up to here
                // (set-up, the first weight copies) may overlap its tail
                if (t == warp) asm volatile("griddepcontrol.wait;" ::: "memory");
                bulk_load(dst, a.x_sw + (size_t)st.col * kXBytes, xbytes, &sm->full[s]);
                last = t;
            }
            if (*abort_flag && last >= 0) {
                // let the copies still in flight land before shared memory is reused or goes away
                for (int i = 0; i < kPollLimit && !mbar_try_wait(&sm->full[s], (last / kCStages) & 1); ++i) {}
            }
        }
    } else if (warp == kCProducers) {
        // ---------------- MMA issuer (one lane)
        if (lane == 0) {
            bool ok = true;
            uint32_t mask = 0u;
            for (int t = 0; t < n_steps && ok; ++t) {
                const int s = t % kCStages;
                const TileStep st = step_at((t + rot) % n_steps);
                ok = mbar_wait(&sm->full[s], (t / kCStages) & 1, abort_flag, a.polls);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t xa = smem_u32(stages + s * kCStageBytes);
                // runs of consecutive block-rows that have a tile here and are in the same state (first tile
                // or not) share one instruction: the tiles are consecutive in the stage, the accumulators in
                // tensor memory
                int slot = 0;
                for (int j = 0; j < kTileRows;) {
                    if (st.tile[j] < 0) { ++j; continue; }
                    const bool started = ((mask >> j) & 1u) != 0u;
                    int n = 1;
                    while (j + n < kTileRows && st.tile[j + n] >= 0 && (((mask >> (j + n)) & 1u) != 0u) == started) ++n;
                    const uint32_t wa = xa + kXBytes + slot * kWBytes;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        umma_f16_n(tmem + (uint32_t)(j * 64), smem_desc_sw128(xa + kk * 32), smem_desc_sw128(wa + kk * 32), n,
                                   started || kk > 0);
                    mask |= ((1u << n) - 1u) << j;
                    slot += n;
                    j += n;
                }
                umma_commit(&sm->empty[s]);          // frees the stage once these MMAs have read it
            }
            sm->acc_mask = ok ? mask : 0u;
            if (mask != 0u) umma_commit(&sm->acc_full);         // accumulators complete (also when giving up: whatever was issued must finish)
            else mbar_arrive(&sm->acc_full);                    // nothing was issued: nothing to wait for
            mbar_arrive(&sm->acc_full);                         // releases acc_mask to the epilogue warps
        }
    }
    // ---------------- epilogue warps: warp (w % 4) owns tensor-memory lanes 32 (w % 4) ..
    const bool epi = warp > kCProducers;
    const int q = warp & 3, b = q * 32 + lane;
    const int br = grp * kTileRows + (int)rank;
    bool ok = true;
    if (epi) {
        // while the main loop runs: bias and destination rows of this CTA's block-row into shared memory
        if (b < 64) {
            const bool live = br < a.Mb;
            sm->bias[b] = live ? __ldg(a.bias_piv + br * 64 + b) : 0.0f;
            sm->dst[b] = live ? (a.pivoted ? br * 64 + b : __ldg(a.scatter_idx + br * 64 + b)) : -1;
        }
        ok = __all_sync(0xffffffffu, mbar_wait(&sm->acc_full, 0, abort_flag, 0) && !*abort_flag);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    // Every CTA of the cluster gets here, also one that gave up (the barrier is the hardware's).  Past it
    // no CTA of the cluster reads or fills its stage buffers any more.
    cluster_sync_all();
    if (epi && ok && q * 32 < a.batch) {          // a warp whose 32 batch rows all lie past the batch has nothing to send
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t mask = sm->acc_mask;
        const uint32_t mine = smem_u32(recv) + (uint32_t)(((int)rank * 16) * kTileBatch + b) * 16u;   // [sender = rank][0][b][0]
#pragma unroll 1
        for (int j = 0; j < kTileRows; ++j) {
            const uint32_t dst = peer_addr(mine, (uint32_t)j);
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t r[32];
                if ((mask >> j) & 1u) {           // warp-uniform
                    asm volatile(
                        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                        : "r"(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(j * 64 + c0)));
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = 0u;
                }
#pragma unroll
                for (int i = 0; i < 32; i += 4)
                    st_peer_v4(dst + (uint32_t)(((c0 + i) >> 2) * kTileBatch) * 16u, r[i], r[i + 1], r[i + 2], r[i + 3]);
            }
        }
    }
    cluster_sync_all();          // all partials have arrived (release / acquire at cluster scope)
    if (epi && br < a.Mb && !sm->abort_flag && q * 32 < a.batch) {
        // ---------------- block-row `rank` of the group: add the four partials in sender order, epilogue.
        // Lanes run over the output rows here: one store instruction then writes 32 scattered words of ONE
        // row of y (lanes over batch rows would write words a whole row pitch apart, which all land in the
        // same few L2 slices).
#pragma unroll 1
        for (int c0 = 0; c0 < 64; c0 += 32) {
#pragma unroll
            for (int i = 0; i < 32; i += 4) {            // lanes over batch rows: contiguous, conflict-free reads
                const float4* src = reinterpret_cast<const float4*>(recv) + ((c0 + i) >> 2) * kTileBatch + b;
                float4 v = src[0];
#pragma unroll
                for (int p = 1; p < kTileRows; ++p) {
                    const float4 w = src[p * 16 * kTileBatch];
                    v.x += w.x; v.y += w.y; v.z += w.z; v.w += w.w;
                }
                xpose[lane * 33 + i] = v.x; xpose[lane * 33 + i + 1] = v.y;
                xpose[lane * 33 + i + 2] = v.z; xpose[lane * 33 + i + 3] = v.w;
            }
            __syncwarp();
            const float bias = sm->bias[c0 + lane];
            const int dst = sm->dst[c0 + lane];
#pragma unroll 8
            for (int r = 0; r < 32; ++r) {               // lanes over output rows
                const int bb = q * 32 + r;
                float v = xpose[r * 33 + lane] + bias;
                if (a.act == PP_ACT_RELU) v = fmaxf(v, 0.0f);
                if (dst >= 0 && bb < a.batch) a.y[(size_t)bb * a.ldy + dst] = v;
            }
            __syncwarp();
        }
    }
    __syncthreads();
    if (threadIdx.x == 0 && sm->abort_flag) *a.status = 1;
    if (warp == kCProducers) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"(kCTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------
// Persistent variant: every SM streams an equal share of the layer.
// The steps of all groups (a step = one tile-column of a group of kTileRows block-rows: one X block and the
// up to kTileRows tiles the group has there) form one sequence, which the host cuts into one contiguous range
// per CTA, balanced by bytes; one CTA per SM.  The part of a group that falls into one CTA's range is a unit:
//   * the producers and the MMA issuer walk the CTA's steps without a break; consecutive units alternate between
//     two sets of kTileRows accumulators in tensor memory (512 columns in all), so that the epilogue warps work
//     on one unit while the next one is being multiplied;
//   * a unit that covers its whole group stores the group's rows itself (bias, activation, row index array);
//   * otherwise every unit of the group writes its partial sums to its own slots in global memory ([chunk]
//     [quad of output rows][batch row][4 floats]: a warp's 16-byte stores and loads are contiguous) and counts
//     itself in at the group's arrival counter; the group's 8 chunks of 32 output rows are dealt out to the
//     units, and each unit, once all have arrived (bounded wait), adds the partial sums of its chunks in unit
//     order and stores those rows.  No atomics on data, the same bits on every run; the last unit to finish
//     reading puts the group's two counters back to zero.
constexpr int kPStages = 4;
constexpr int kPStageBytes = kXBytes + kTileRows * kWBytes;    // 48 KiB: one X block + up to 4 tiles
constexpr int kPTmemCols = 2 * 64 * kTileRows;                 // two accumulator sets
constexpr int kPThreads = 32 * (kProducers + 1 + 4);
constexpr int kPChunks = 2 * kTileRows;                        // chunks of 32 output rows per group
constexpr int kGroupPolls = 1 << 22;

struct PersistSmem {
    uint64_t full[kPStages];
    uint64_t empty[kPStages];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint32_t tmem_base;
    int abort_flag;
    int group_ready;          // written by one epilogue thread after its bounded wait for the group's units
    uint32_t acc_mask[2];     // per accumulator set: block-rows that received at least one tile
    float xpose[4][32 * 33];  // one transposition tile per epilogue warp
    int4 steps[kStepCap][2];  // this CTA's first kStepCap step records
};

__device__ __forceinline__ void tmem_ld32(uint32_t addr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(addr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ TileUnit load_unit(const TileUnit* p) {
    const int4 lo = __ldg(reinterpret_cast<const int4*>(p)), hi = __ldg(reinterpret_cast<const int4*>(p) + 1);
    TileUnit u;
    u.step_begin = lo.x; u.step_end = lo.y; u.group = lo.z; u.part = lo.w; u.n_parts = hi.x; u.first_unit = hi.y;
    u.pad[0] = u.pad[1] = 0;
    return u;
}


// Which unit of a group finishes chunk q of the group's rows.
__device__ __forceinline__ int chunk_owner(int q, int n_parts) { return n_parts <= kPChunks ? q % n_parts : q; }

__global__ void __launch_bounds__(kPThreads, 1)
tile_persist_f16_kernel(const TileArgs a) {
    static_assert(kTileRows == 4, "step records carry four tile slots");
    extern __shared__ unsigned char smem_raw[];
    unsigned char* stages = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    PersistSmem* sm = reinterpret_cast<PersistSmem*>(stages + kPStages * kPStageBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next call's gather kernel may fetch its index entries meanwhile
    const int u0 = __ldg(a.cta_unit + blockIdx.x), u1 = __ldg(a.cta_unit + blockIdx.x + 1);
    int cs = 0, ce = 0;                       // this CTA's steps: from its first unit's first step to its last unit's last
    if (u0 < u1) {
        cs = __ldg(&a.units[u0].step_begin);
        ce = __ldg(&a.units[u1 - 1].step_end);
    }
    // This CTA's step records go to shared memory once: read from global memory inside the loops they cost the
    // producers and the MMA issuer one L2 round trip per step.
    for (int i = threadIdx.x; i < 2 * (ce - cs) && i < 2 * kStepCap; i += kPThreads)
        sm->steps[i >> 1][i & 1] = __ldg(reinterpret_cast<const int4*>(a.steps + cs) + i);
    auto step_at = [&](int i) {
        return i < kStepCap ? unpack_step(sm->steps[i][0], sm->steps[i][1]) : load_step(a.steps + cs + i);
    };
    if (threadIdx.x == 0) {
        for (int s = 0; s < kPStages; ++s) { mbar_init(&sm->full[s], 1); mbar_init(&sm->empty[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&sm->acc_full[s], 2); mbar_init(&sm->acc_empty[s], 4); }
        sm->abort_flag = 0;
        sm->acc_mask[0] = sm->acc_mask[1] = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kProducers) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(smem_u32(&sm->tmem_base)), "r"(kPTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = sm->tmem_base;
    volatile int* abort_flag = &sm->abort_flag;
    if (threadIdx.x == 0) tile_stamp(a, 0);

    if (warp < kProducers) {
        // ---------------- producers: warp w (one lane) feeds steps cs + w, cs + w + kProducers, ... into stage w
        if (lane == 0) {
            const int s = warp;
            int last = -1;
            const uint32_t xbytes = (uint32_t)((a.batch + 7) / 8) * 1024u;   // live 8-row groups of the X block only
            for (int t = warp; t < ce - cs; t += kProducers) {
                if (t >= kPStages && !mbar_wait(&sm->empty[s], ((t / kPStages) & 1) ^ 1, abort_flag, a.polls)) break;
                const TileStep st = step_at(t);
                unsigned char* dst = stages + s * kPStageBytes;
                mbar_expect_tx(&sm->full[s], xbytes + (uint32_t)(st.ntiles * kWBytes));
                bulk_load(dst + kXBytes, a.tiles_sw + (size_t)st.pos * kWBytes, (uint32_t)(st.ntiles * kWBytes), &sm->full[s]);
                // the permuted input comes from the gather kernel launched just before: everything up to here
                // (set-up, the first weight copies) may overlap its tail
                if (t == warp) asm volatile("griddepcontrol.wait;" ::: "memory");
                bulk_load(dst, a.x_sw + (size_t)st.col * kXBytes, xbytes, &sm->full[s]);
                last = t;
            }
            if (*abort_flag && last >= 0) {
                // let the copy still in flight land before shared memory goes away
                for (int i = 0; i < kPollLimit && !mbar_try_wait(&sm->full[s], (last / kPStages) & 1); ++i) {}
            }
        }
    } else if (warp == kProducers) {
        // ---------------- MMA issuer (one lane): unit after unit, alternating between the two accumulator sets
        if (lane == 0) {
            bool ok = true;
            int t = 0;                                   // steps issued so far, over all units
            for (int u = u0; u < u1; ++u) {
                const int set = (u - u0) & 1, use = (u - u0) >> 1;
                const int n = __ldg(&a.units[u].step_end) - __ldg(&a.units[u].step_begin);
                uint32_t mask = 0u;
                // the epilogue must have drained this set's previous unit
                if (ok && use > 0) ok = mbar_wait(&sm->acc_empty[set], (use - 1) & 1, abort_flag, 0);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                for (int i = 0; i < n && ok; ++i, ++t) {
                    const int s = t % kPStages;
                    const TileStep st = step_at(t);
                    ok = mbar_wait(&sm->full[s], (t / kPStages) & 1, abort_flag, a.polls);
                    if (!ok) break;
                    if (t == 0) tile_stamp(a, 1);
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t xa = smem_u32(stages + s * kPStageBytes);
                    int slot = 0;
                    for (int j = 0; j < kTileRows;) {
                        if (st.tile[j] < 0) { ++j; continue; }
                        const bool started = ((mask >> j) & 1u) != 0u;
                        int nn = 1;
                        while (j + nn < kTileRows && st.tile[j + nn] >= 0 && (((mask >> (j + nn)) & 1u) != 0u) == started) ++nn;
                        const uint32_t wa = xa + kXBytes + slot * kWBytes;
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            umma_f16_n(tmem + (uint32_t)(set * 64 * kTileRows + j * 64), smem_desc_sw128(xa + kk * 32),
                                       smem_desc_sw128(wa + kk * 32), nn, started || kk > 0);
                        mask |= ((1u << nn) - 1u) << j;
                        slot += nn;
                        j += nn;
                    }
                    umma_commit(&sm->empty[s]);          // frees the stage once these MMAs have read it
                }
                sm->acc_mask[set] = ok ? mask : 0u;
                if (mask != 0u) umma_commit(&sm->acc_full[set]);   // whatever was issued must finish, also when giving up
                else mbar_arrive(&sm->acc_full[set]);
                mbar_arrive(&sm->acc_full[set]);                   // releases acc_mask to the epilogue warps
            }
            tile_stamp(a, 2);
        }
    } else {
        // ---------------- epilogue warps: warp (w % 4) owns tensor-memory lanes 32 (w % 4) .., thread = batch row
        const int q = warp & 3, b = q * 32 + lane;
        const bool live_warp = q * 32 < a.batch;          // a warp whose 32 batch rows all lie past the batch only keeps the barriers
        float* xpose = sm->xpose[q];
        bool ok = true;
        // rows [c0, c0 + 32) of a block-row: bias, activation, store.  The 32 x 32 block is transposed through
        // shared memory so that the lanes of a store run over output rows (32 scattered words of ONE row of y).
        auto store_chunk = [&](const uint32_t (&r)[32], float bias, int dst) {
#pragma unroll
            for (int j = 0; j < 32; ++j) xpose[lane * 33 + j] = __uint_as_float(r[j]);
            __syncwarp();
#pragma unroll 8
            for (int rr = 0; rr < 32; ++rr) {
                const int bb = q * 32 + rr;
                float v = xpose[rr * 33 + lane] + bias;
                if (a.act == PP_ACT_RELU) v = fmaxf(v, 0.0f);
                if (dst >= 0 && bb < a.batch) a.y[(size_t)bb * a.ldy + dst] = v;
            }
            __syncwarp();
        };
        // bias and destination row of the chunks of unit `un` that this unit stores (lane = row of the chunk)
        auto chunk_rows = [&](const TileUnit& un, float (&cbias)[kPChunks], int (&cdst)[kPChunks]) {
#pragma unroll
            for (int c = 0; c < kPChunks; ++c) {
                const int br = un.group * kTileRows + (c >> 1), row = br * 64 + (c & 1) * 32 + lane;
                const bool mine = (un.n_parts == 1 || chunk_owner(c, un.n_parts) == un.part) && br < a.Mb;
                cbias[c] = mine ? __ldg(a.bias_piv + row) : 0.0f;
                cdst[c] = !mine ? -1 : (a.pivoted ? row : __ldg(a.scatter_idx + row));
            }
        };
        // First pass, unit after unit as the accumulators complete: a unit that owns its whole group stores the
        // rows; any other writes its partial sums to its slots and counts itself in at the group's counter.
        // Nothing here waits for another CTA, so no CTA's publication can be held up by a neighbour's.
        for (int u = u0; u < u1; ++u) {
            const int set = (u - u0) & 1, use = (u - u0) >> 1;
            const TileUnit un = load_unit(a.units + u);
            float cbias[kPChunks];
            int cdst[kPChunks];
            if (un.n_parts == 1) chunk_rows(un, cbias, cdst);        // requested while the unit is still being multiplied
            ok = __all_sync(0xffffffffu, ok && mbar_wait(&sm->acc_full[set], use & 1, abort_flag, 0) && !*abort_flag);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t mask = sm->acc_mask[set];
            const uint32_t tbase = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(set * 64 * kTileRows);
            if (ok && live_warp) {
                float* mine = a.unit_partials + (size_t)u * (kPChunks * kTileBatch * 32);
#pragma unroll
                for (int c = 0; c < kPChunks; ++c) {
                    uint32_t r[32];
                    if ((mask >> (c >> 1)) & 1u) {              // warp-uniform: the tensor-memory load is a warp-wide instruction
                        tmem_ld32(tbase + (uint32_t)(c * 32), r);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) r[j] = 0u;
                    }
                    if (un.n_parts == 1) {
                        store_chunk(r, cbias[c], cdst[c]);
                    } else if (b < a.batch) {
                        // [chunk][row quad j][batch row][4]: the 32 lanes of a store write one contiguous 512-byte run
                        uint4* dst = reinterpret_cast<uint4*>(mine) + (size_t)c * (8 * kTileBatch) + b;
#pragma unroll
                        for (int j = 0; j < 8; ++j) dst[(size_t)j * kTileBatch] = make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            if (lane == 0) mbar_arrive(&sm->acc_empty[set]);         // the accumulator set may be reused
            if (un.n_parts > 1) {
                __threadfence();
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (ok && warp == kProducers + 1 && lane == 0) atomicAdd(a.group_sync + 2 * un.group, 1);
            }
        }
        if (warp == kProducers + 1 && lane == 0) tile_stamp(a, 3);
        // Second pass: for every split group this CTA has a unit of, wait (bounded) until all units of the group
        // have arrived, add the partial sums of this unit's chunks in unit order and store those rows; the last
        // unit to finish reading puts the group's counters back to zero.
        for (int u = u0; u < u1; ++u) {
            const TileUnit un = load_unit(a.units + u);
            if (un.n_parts == 1) continue;
            float cbias[kPChunks];
            int cdst[kPChunks];
            chunk_rows(un, cbias, cdst);
            int* gsync = a.group_sync + 2 * un.group;
            if (warp == kProducers + 1 && lane == 0) {
                int ready = 0;
                if (ok) {
                    const int limit = a.polls > 0 ? a.polls : kGroupPolls;
                    for (int i = 0; i < limit && !ready; ++i) {
                        int seen;
                        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(gsync) : "memory");
                        ready = seen >= un.n_parts;
                        if (!ready && (i & 63) == 63 && *reinterpret_cast<volatile int*>(a.status)) break;
                    }
                    if (!ready) { *abort_flag = 1; *a.status = 1; }
                }
                sm->group_ready = ready;
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
            ok = ok && sm->group_ready != 0;
            if (ok && live_warp) {
#pragma unroll
                for (int c = 0; c < kPChunks; ++c) {
                    if (chunk_owner(c, un.n_parts) != un.part) continue;
                    uint32_t r[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = 0u;
                    if (b < a.batch) {
                        // the partial sums were written by other SMs: read them past the L1 (ld.global.cg); the loads of
                        // two units are in flight together, the additions stay in unit order
                        const uint4* base = reinterpret_cast<const uint4*>(a.unit_partials) +
                                            ((size_t)un.first_unit * kPChunks + c) * (8 * kTileBatch) + b;
                        const size_t unit_stride = (size_t)kPChunks * 8 * kTileBatch;
                        for (int p = 0; p < un.n_parts; p += 2) {
                            const bool two = p + 1 < un.n_parts;
                            uint4 v0[8], v1[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) v0[j] = __ldcg(base + (size_t)p * unit_stride + (size_t)j * kTileBatch);
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                v1[j] = two ? __ldcg(base + (size_t)(p + 1) * unit_stride + (size_t)j * kTileBatch) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                r[4 * j] = __float_as_uint(__uint_as_float(r[4 * j]) + __uint_as_float(v0[j].x));
                                r[4 * j + 1] = __float_as_uint(__uint_as_float(r[4 * j + 1]) + __uint_as_float(v0[j].y));
                                r[4 * j + 2] = __float_as_uint(__uint_as_float(r[4 * j + 2]) + __uint_as_float(v0[j].z));
                                r[4 * j + 3] = __float_as_uint(__uint_as_float(r[4 * j + 3]) + __uint_as_float(v0[j].w));
                            }
                            if (two) {
#pragma unroll
                                for (int j = 0; j < 8; ++j) {
                                    r[4 * j] = __float_as_uint(__uint_as_float(r[4 * j]) + __uint_as_float(v1[j].x));
                                    r[4 * j + 1] = __float_as_uint(__uint_as_float(r[4 * j + 1]) + __uint_as_float(v1[j].y));
                                    r[4 * j + 2] = __float_as_uint(__uint_as_float(r[4 * j + 2]) + __uint_as_float(v1[j].z));
                                    r[4 * j + 3] = __float_as_uint(__uint_as_float(r[4 * j + 3]) + __uint_as_float(v1[j].w));
                                }
                            }
                        }
                    }
                    store_chunk(r, cbias[c], cdst[c]);
                }
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");           // every warp has read; group_ready may be rewritten
            if (ok && warp == kProducers + 1 && lane == 0) {
                if (atomicAdd(gsync + 1, 1) == un.n_parts - 1) { gsync[0] = 0; gsync[1] = 0; }
            }
        }
        if (warp == kProducers + 1 && lane == 0) tile_stamp(a, 4);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0 && sm->abort_flag) *a.status = 1;
    if (warp == kProducers) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"(kPTmemCols) : "memory");
    }
}

// Byte offset of element (row r, column c) inside a 128-byte-swizzled block of 128-byte rows:
// the 16-byte chunk index is XOR-ed with the row index modulo 8.
__host__ __device__ __forceinline__ uint32_t sw128_offset(int r, int c) {
    return (uint32_t)r * 128u + (uint32_t)(((c >> 3) ^ (r & 7)) << 4) + (uint32_t)(c & 7) * 2u;
}

// x_piv[b][j] = x[b][gather_idx[j]] for the rows of one batch chunk; padding columns are zero.  One CTA per row: the row goes to shared memory coalesced and leaves permuted, into
// the swizzled 16 KiB block of its tile-column (row b of the block).
__global__ void gather_x_kernel(const __half* __restrict__ x, int ldx, int n, const int32_t* __restrict__ gather_idx,
                                int n_pad, unsigned char* __restrict__ x_sw, int batch) {
    extern __shared__ __half row[];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the tile kernel may set up meanwhile
    const int b = blockIdx.x;
    if (b >= batch) return;
    // A thread produces whole 16-byte chunks of the destination (8 consecutive pivoted columns).  The index
    // entries of its first chunk are requested before the row itself, so that the two round trips overlap.
    const int n_chunks = n_pad / 8;
    const int4* idx4 = reinterpret_cast<const int4*>(gather_idx);
    int i = threadIdx.x;
    int4 ia = make_int4(-1, -1, -1, -1), ib = ia;
    if (i < n_chunks) { ia = __ldg(idx4 + 2 * i); ib = __ldg(idx4 + 2 * i + 1); }
    // Launched with programmatic stream serialization behind whatever precedes it in the stream (typically the
    // previous call's tile kernel, which may still read the permuted-input blocks this kernel is about to
    // overwrite, or the producer of x): the index entries above are the layer's own, everything below waits.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    {
        // 16-byte copies where the row allows it (base and pitch 16-byte aligned), element copies otherwise
        const __half* src = x + (size_t)b * ldx;
        const bool vec = ((reinterpret_cast<uintptr_t>(src) & 15u) == 0);
        const int n8 = vec ? n / 8 : 0;
        for (int c = threadIdx.x; c < n8; c += blockDim.x)
            reinterpret_cast<uint4*>(row)[c] = __ldg(reinterpret_cast<const uint4*>(src) + c);
        for (int j = n8 * 8 + threadIdx.x; j < n; j += blockDim.x) row[j] = src[j];
    }
    __syncthreads();
    const unsigned short* rowu = reinterpret_cast<const unsigned short*>(row);
    auto pick = [&](int idx) { return idx >= 0 ? (uint32_t)rowu[idx] : 0u; };
    for (bool first = true; i < n_chunks; i += blockDim.x, first = false) {
        if (!first) { ia = __ldg(idx4 + 2 * i); ib = __ldg(idx4 + 2 * i + 1); }
        uint4 v;
        v.x = pick(ia.x) | (pick(ia.y) << 16);
        v.y = pick(ia.z) | (pick(ia.w) << 16);
        v.z = pick(ib.x) | (pick(ib.y) << 16);
        v.w = pick(ib.z) | (pick(ib.w) << 16);
        const int j = 8 * i;
        *reinterpret_cast<uint4*>(x_sw + (size_t)(j >> 6) * kXBytes + sw128_offset(b, j & 63)) = v;
    }
}

}  // namespace

#ifdef PP_TRACE
unsigned long long* g_tile_trace = nullptr;
#endif

void swizzle_tile_64x64(const void* row_major, void* out) {
    const unsigned char* src = static_cast<const unsigned char*>(row_major);
    unsigned char* dst = static_cast<unsigned char*>(out);
    for (int r = 0; r < 64; ++r)
        for (int ch = 0; ch < 8; ++ch)
            for (int k = 0; k < 16; ++k) dst[r * 128 + ((ch ^ (r & 7)) << 4) + k] = src[r * 128 + ch * 16 + k];
}

// Launch with programmatic stream serialization: the kernel may start while the gather kernel before it
// still runs; its producers wait for that kernel (griddepcontrol.wait) before they touch the permuted input.
// cooperative: the CTAs wait on one another (units of a group), so all of them must be resident at once.
static cudaError_t launch_after_gather(void (*kernel)(const TileArgs), int grid, int threads, size_t smem, const TileArgs& a,
                                       cudaStream_t stream, bool cooperative = false) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeCooperative;
    attr[1].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = cooperative ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, kernel, a);
}

template <int STAGES, int XB>
cudaError_t launch_one_row(const TileArgs& a, int Mb, cudaStream_t stream) {
    static PerDeviceOnce configured;
    const size_t smem = (size_t)STAGES * (XB + kWBytes) + (kXBytes - XB) + sizeof(TileSmem<STAGES>) + 1024;
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (!configured.is_done(dev)) {
        e = cudaFuncSetAttribute(tile_f16_kernel<STAGES, XB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured.mark(dev);
    }
    return launch_after_gather(tile_f16_kernel<STAGES, XB>, Mb, kThreads, smem, a, stream);
}

cudaError_t launch_tile(const TileArgs& a_in, const void* x, int ldx, int n, const int32_t* gather_idx, int n_pad, int Mb,
                        int kernel, cudaStream_t stream) {
    const bool use_cluster = kernel == 2;
    TileArgs a = a_in;
    a.polls = g_stream_wait_polls;
    a.trace = nullptr;
#ifdef PP_TRACE
    a.trace = g_tile_trace;
#endif
    if (a.batch < 1 || a.batch > kTileBatch) return cudaErrorInvalidValue;
    if ((size_t)n * 2 > 48 * 1024) return cudaErrorInvalidValue;
    // rows past the batch keep whatever an earlier call left there: every row of the product is independent
    // and the epilogue drops those rows
    cudaError_t e;
    {
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)a.batch);
        cfg.blockDim = dim3(1024);
        cfg.dynamicSmemBytes = ((size_t)n * 2 + 15) / 16 * 16;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = g_stream_pdl ? 1 : 0;
        e = cudaLaunchKernelEx(&cfg, gather_x_kernel, static_cast<const __half*>(x), ldx, n, gather_idx, n_pad,
                               const_cast<unsigned char*>(a.x_sw), a.batch);
    }
    if (e != cudaSuccess) return e;
    if (kernel == 3 && a.units && a.cta_unit && a.persist_ctas > 0 && a.unit_partials && a.group_sync) {
        static PerDeviceOnce configured_p;
        const size_t smem_p = (size_t)kPStages * kPStageBytes + sizeof(PersistSmem) + 1024;
        int dev = -1;
        e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (!configured_p.is_done(dev)) {
            e = cudaFuncSetAttribute(tile_persist_f16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_p);
            if (e != cudaSuccess) return e;
            configured_p.mark(dev);
        }
        return launch_after_gather(tile_persist_f16_kernel, a.persist_ctas, kPThreads, smem_p, a, stream, true);
    }
    if (use_cluster && a.steps && a.parts) {
        static PerDeviceOnce configured_c;
        const size_t smem_c = (size_t)kCStages * kCStageBytes + sizeof(ClusterSmem) + 1024;
        int dev = -1;
        e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (!configured_c.is_done(dev)) {
            e = cudaFuncSetAttribute(tile_cluster_f16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_c);
            if (e != cudaSuccess) return e;
            configured_c.mark(dev);
        }
        const int groups = (Mb + kTileRows - 1) / kTileRows;
        return launch_after_gather(tile_cluster_f16_kernel, groups * kTileRows, kCThreads, smem_c, a, stream);
    }
    if (a.batch <= 32) return launch_one_row<16, 4 * 1024>(a, Mb, stream);
    if (a.batch <= 64) return launch_one_row<12, 8 * 1024>(a, Mb, stream);
    return launch_one_row<8, kXBytes>(a, Mb, stream);
}

}  // namespace pp

#ifdef PP_TRACE
// Diagnostic builds only: launches of the persistent tile kernel write their phase stamps to `device_buffer`
// (148 x 8 unsigned 64-bit words, overwritten by every launch).
extern "C" void pp_trace_set_tile_buffer(void* device_buffer) { pp::g_tile_trace = static_cast<unsigned long long*>(device_buffer); }
#endif
