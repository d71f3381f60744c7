// Persistent streaming block-sparse matrix-vector kernels for sm_100a (batch 1 .. 8).
//
// The packed tile values of a layer form one linear sequence of 512-byte fragments (strip =
// row-group of a block-row; a strip's fragments are contiguous and strips follow each other).
// The host cuts that sequence into one contiguous range per CTA, and every warp of a CTA
// streams an equal, contiguous share of its CTA's range:
//   * Listing 1's group fetch is done ONCE per CTA for the whole layer input: x and the column
//     index array are copied to shared memory with 16-byte asynchronous copies (issued first,
//     so they are not queued behind the weight loads) and permuted there into pivoted order
//     while the first weight fragments are in flight; after that barrier no warp waits for
//     another until its range is finished;
//   * the weights never pass through registers on their way in: each warp owns a ring of U
//     512-byte slots in shared memory and keeps U 16-byte-per-lane asynchronous copies
//     (cp.async groups) in flight, refilling a slot right after reading it (a register ring of
//     plain loads serialises on the load scoreboard and measured 30 % slower; it also blocked the
//     shared-memory permutation of x behind the outstanding weight loads);
//   * where a warp's range crosses a strip boundary it parks the finished 16(32)-row partial sum
//     in shared memory; after the final barrier the CTA adds the parks of every strip in warp
//     order.  A strip shared by several CTAs (the extra sum Section 4.1.5 asks for where blocks share rows) goes
//     through one global partial sum per CTA, added in CTA order by the last CTA to arrive.
//   * everything the epilogue needs (row index array, pivoted bias, strip table) is fetched
//     asynchronously at kernel start, so the tail is shared-memory work plus the stores;
//   * the kernel is launched with programmatic stream serialization: it releases its successor
//     at once (griddepcontrol.launch_dependents) and fetches tables and first weights before
//     griddepcontrol.wait, so back-to-back layers overlap launch latency and prologue with the
//     previous kernel's tail.  x is read, and y and scratch are written, only after the wait.
// Results are independent of scheduling.  fp16 tiles: warp-level 16x8x16 tensor-core
// instruction, batch on the 8-wide side, fp32 accumulate.  fp32 tiles: plain FMAs.
#include <cuda_fp16.h>

#include "pp_gemv.cuh"
#include "pp_stream.cuh"

namespace pp {
namespace {

constexpr int kThreads = kStreamWarps * 32;
constexpr int kParamCtas = 320;       // CTA ranges that travel in the kernel parameters

struct StreamLaunch {
    StreamArgs a;
    CtaDesc table[kParamCtas];
};

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

__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;"
                 :: "r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc));
}
__device__ __forceinline__ void cp_async_4(void* smem_dst, const void* gsrc) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;"
                 :: "r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc));
}

#ifdef PP_TRACE
// Diagnostic builds only: thread 0 of every CTA stamps the global nanosecond timer at the kernel's phases.
__device__ __forceinline__ void trace_stamp(const StreamArgs& a, int slot) {
    if (a.trace && threadIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        a.trace[(size_t)blockIdx.x * 8 + slot] = t;
        if (slot == 0) {
            unsigned smid;
            asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
            a.trace[(size_t)blockIdx.x * 8 + 7] = smid;
        }
    }
}
#else
__device__ __forceinline__ void trace_stamp(const StreamArgs&, int) {}
#endif

__device__ __forceinline__ int x_index(const StreamArgs& a, int pj) {
    if (a.gather_idx) return __ldg(a.gather_idx + pj);
    return pj < a.x_limit ? pj : -1;
}

// Shared memory: fixed header, then the regions whose size depends on the launch.
struct SmemLayout {
    int* sstart;     // [kStreamMaxStrips + 1] strip starts of this CTA's strips
    int* wlohi;      // [kStreamMaxStrips] bit w set: warp w parked a partial sum for the strip
    int* flags;      // [2]
    int* wb;         // [kStreamWarps + 1] fragment position where each warp's range starts
    uint64_t* xbar;  // mbarrier the bulk copies of x complete on
    int4* sinfo;     // [kStreamMaxStrips] strip table entries of this CTA's strips
    int* rowdst;     // [max_rows] scatter_idx of this CTA's pivoted rows
    float* rowbias;  // [max_rows] bias_piv of this CTA's pivoted rows
    float* segp;     // [strips a CTA may list + kStreamWarps][RG][batch] parked partial sums (slot = local strip + warp)
    uint4* ring;     // [kStreamWarps][U][32] weight fragments in flight
    void* xs;        // staged pivoted x   [batch][xs_stride] (absent in staging mode 3)
    int* idxs;       // staging modes 1, 3: gather_idx [n_pad]
    void* raw;       // staging modes 1, 3: x as given [batch][raw_stride]
};
constexpr int kHeaderBytes = 512 + kStreamMaxStrips * 16;   // 512 B: sstart, wlohi, xbar, flags, wb; then sinfo (the regions
                                                            // behind the header keep their 128-byte alignment)
static_assert(kStreamMaxStrips <= 48, "header words 56..103 hold wlohi, 104..105 the x barrier");

__host__ __device__ __forceinline__ size_t xs_bytes(int batch, int xs_stride, int esz) {
    return ((size_t)batch * xs_stride * esz + 15) / 16 * 16;
}

// Bytes of the park slots: a CTA lists at most max_rows / rg strips and a warp parks in slot (local strip + warp);
// rounded to 128 bytes so that the weight ring behind it keeps its alignment.
__host__ __device__ __forceinline__ size_t segp_bytes(int max_rows, int rg, int batch) {
    return ((size_t)(max_rows / rg + kStreamWarps) * rg * batch * 4 + 127) / 128 * 128;
}

__device__ __forceinline__ SmemLayout carve(unsigned char* base, int rg, int U, const StreamArgs& a, int esz) {
    SmemLayout L;
    int* w = reinterpret_cast<int*>(base);
    L.sstart = w;
    L.wlohi = w + 56;
    L.flags = w + 108;
    L.wb = w + 110;
    L.xbar = reinterpret_cast<uint64_t*>(w + 104);
    L.sinfo = reinterpret_cast<int4*>(base + 512);
    L.rowdst = reinterpret_cast<int*>(base + kHeaderBytes);
    L.rowbias = reinterpret_cast<float*>(L.rowdst + a.max_rows);
    L.segp = L.rowbias + a.max_rows;
    L.ring = reinterpret_cast<uint4*>(reinterpret_cast<unsigned char*>(L.segp) + segp_bytes(a.max_rows, rg, a.batch));
    unsigned char* p = reinterpret_cast<unsigned char*>(L.ring + kStreamWarps * U * 32);
    L.xs = p;
    if (a.stage_mode < 3) p += xs_bytes(a.batch, a.xs_stride, esz);
    L.idxs = reinterpret_cast<int*>(p);
    L.raw = p + (size_t)a.n_pad * (a.stage_mode == 4 ? 2 : 4) + 16;     // 16 spare bytes in front: raw[-1] is the zero that index -1 reads
    return L;
}

__device__ __forceinline__ int warp_begin(const CtaDesc& d, int w) {
    return d.p_begin + (int)(((long long)(d.p_end - d.p_begin) * w) / kStreamWarps);
}

__device__ __forceinline__ CtaDesc cta_range(const StreamLaunch& P) {
    if (gridDim.x <= kParamCtas) return P.table[blockIdx.x];
    const int4 dd = __ldg(reinterpret_cast<const int4*>(P.a.cta_desc) + blockIdx.x);
    return CtaDesc{dd.x, dd.y, dd.z, dd.w};
}

// Phase 1a: asynchronous copies of the layer's own (immutable) tables: strip starts, strip table,
// row index array and pivoted bias of this CTA's rows, and the column index array.  Nothing
// here depends on the previous kernel in the stream, so it runs before griddepcontrol.wait.
template <int RG>
__device__ __forceinline__ void issue_static(const StreamArgs& a, const CtaDesc& d, const SmemLayout& L) {
    const int tid = threadIdx.x;
    for (int i = tid; i <= d.s_count; i += kThreads) cp_async_4(L.sstart + i, a.strip_start + d.s_first + i);
    for (int i = tid; i < d.s_count; i += kThreads) cp_async_16(L.sinfo + i, a.strip_info + d.s_first + i);
    const int n_rows = d.s_count * RG, row0 = d.s_first * RG;
    for (int i = tid; i < n_rows; i += kThreads) {
        cp_async_4(L.rowdst + i, a.scatter_idx + row0 + i);
        cp_async_4(L.rowbias + i, a.bias_piv + row0 + i);
    }
    if (a.stage_mode == 1 || a.stage_mode == 3)
        for (int i = tid; i < a.n_pad / 4; i += kThreads) cp_async_16(L.idxs + 4 * i, a.gather_idx + 4 * i);
    if (a.stage_mode == 4)      // 16-bit table: entry = index + 1, 0 = the zero in front of the copied x
        for (int i = tid; i < a.n_pad / 8; i += kThreads)
            cp_async_16(reinterpret_cast<uint16_t*>(L.idxs) + 8 * i, a.gather16 + 8 * i);
    asm volatile("cp.async.commit_group;" ::: "memory");
}

// Before griddepcontrol.wait: touch the pages of x and y with L2 prefetches so that their address
// translations are already cached when the copy of x and the stores to y are issued.  (A prefetch
// reads no value into the SM; the data itself is read and written only after the wait.)
__device__ __forceinline__ void warm_translations(const StreamArgs& a) {
    if (threadIdx.x == 0) {
        asm volatile("prefetch.global.L2 [%0];" :: "l"(a.x));
        asm volatile("prefetch.global.L2 [%0];" :: "l"(a.y));
    }
}

// Phase 1b (after griddepcontrol.wait): Listing 1's group fetch, for the whole layer input.
// Mode 1 copies x to shared memory (permuted in phase 3 through the index array copied in
// phase 1a), mode 3 (batch 1) copies x and lets the multiply loop read it through the index
// array, mode 2 (input already in pivoted order) copies straight into place; mode 0 leaves the
// gather to phase 3.
template <typename T>
__device__ __forceinline__ void issue_x(const StreamArgs& a, const SmemLayout& L) {
    constexpr int EPC = 16 / (int)sizeof(T);
    if (a.stage_mode != 0 && threadIdx.x == 0) {
        const bool via_raw = a.stage_mode != 2;
        const T* x = static_cast<const T*>(a.x);
        T* dst = via_raw ? static_cast<T*>(L.raw) : static_cast<T*>(L.xs);
        const int dst_stride = via_raw ? a.raw_stride : a.xs_stride;
        // modes 1, 3, 4 copy every element a gather index may name (x_len); mode 2 copies the N real
        // columns (the padding columns up to n_pad are zero-filled in phase 3).  One bulk copy per input
        // row, issued by one thread and completing on an mbarrier: the same bytes as 16-byte copies from
        // every thread took 0.8-1.6 us longer per call (one request per row instead of a thousand).
        const uint32_t bytes = (uint32_t)((via_raw ? a.x_len : a.x_limit) / EPC) * 16u;
        if (bytes) {
            const uint32_t bar = (uint32_t)__cvta_generic_to_shared(L.xbar);
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes * (uint32_t)a.batch) : "memory");
            for (int b = 0; b < a.batch; ++b)
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             :: "r"((uint32_t)__cvta_generic_to_shared(dst + b * dst_stride)), "l"(x + (size_t)b * a.ldx),
                                "r"(bytes), "r"(bar) : "memory");
        }
    }
}

// Kernel start: the mbarrier of the x copies (one arrival: the issuing thread's expect_tx).
__device__ __forceinline__ void init_xbar(const SmemLayout& L) {
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"((uint32_t)__cvta_generic_to_shared(L.xbar)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
}

// Which warps will park a partial sum for each of this CTA's strips (their ranges intersect the strip
// inside the CTA).  Runs right after the staging barrier; the barrier that ends the streaming phase
// publishes the result.  Sixteen lanes share a strip: lane w tests where warp w's range starts against the
// strip's first and last fragment inside the CTA, and since those starts ascend the highest lane that passes
// names the warp (one thread per strip walking all warps held warp 0 back by 0.6 us, which is the whole
// multiply phase of a small layer).
static_assert(kStreamWarps == 16, "plan_parks gives half a warp to every strip");
__device__ __forceinline__ void plan_parks(const CtaDesc& d, const SmemLayout& L) {
    const int w = threadIdx.x & 15, half = (threadIdx.x >> 4) & 1;
    const int total = d.s_count * kStreamWarps;
    for (int base = 0; base < total; base += kThreads) {
        const int e = base + (int)threadIdx.x, ls = e >> 4;
        const bool in = e < total;
        int lo = 0, hi = 0;
        bool at_lo = false, at_hi = false, live = false;
        if (in) {
            lo = max(L.sstart[ls], d.p_begin);
            hi = min(L.sstart[ls + 1], d.p_end);
            const int wbeg = L.wb[w];
            at_lo = wbeg <= lo;
            at_hi = wbeg <= hi - 1;
            live = wbeg < L.wb[w + 1];                    // a warp with an empty range parks nothing
        }
        const unsigned m_lo = (__ballot_sync(0xffffffffu, at_lo) >> (16 * half)) & 0xffffu;
        const unsigned m_hi = (__ballot_sync(0xffffffffu, at_hi) >> (16 * half)) & 0xffffu;
        const unsigned m_live = (__ballot_sync(0xffffffffu, live) >> (16 * half)) & 0xffffu;
        if (in && w == 0) {
            unsigned mask = 0u;                           // an empty intersection: no warp parks
            if (lo < hi) {                                // warp 0 starts at the CTA's first fragment, so bit 0 is set in both
                const int w_lo = 31 - __clz((int)m_lo), w_hi = 31 - __clz((int)m_hi);
                mask = m_live & ((2u << w_hi) - 1u) & ~((1u << w_lo) - 1u);
            }
            L.wlohi[ls] = (int)mask;
        }
    }
}

constexpr int kXWaitPolls = 1 << 22;   // default polls of the x barrier before the kernel gives up (seconds; a copy that lands never gets near it)

// Phase 3: wait for the copies of phases 1 and 2, finish the staged pivoted x.  x_parity: phase of the x barrier
// this use completes (0 for the first use in a kernel, alternating after that).  The park plan, which needs the
// CTA's tables but not x, is made while the copy of x is still on its way.
template <typename T, int U>
__device__ __forceinline__ void finish_stage(const StreamArgs& a, const CtaDesc& d, const SmemLayout& L, uint32_t x_parity = 0u) {
    constexpr int EPC = 16 / (int)sizeof(T);
    const int tid = threadIdx.x;
    const T* x = static_cast<const T*>(a.x);
    T* xs = static_cast<T*>(L.xs);
    if (a.stage_mode != 0) {
        // ragged tail of each row (fewer than 16 bytes) and, in mode 2, the zero padding
        const bool via_raw = a.stage_mode != 2;
        T* dst = via_raw ? static_cast<T*>(L.raw) : xs;
        const int dst_stride = via_raw ? a.raw_stride : a.xs_stride;
        const int n_src = via_raw ? a.x_len : a.x_limit;
        const int n_dst = via_raw ? a.x_len : a.n_pad;
        if (a.stage_mode >= 3 && tid < a.batch) dst[tid * dst_stride - 1] = T(0.0f);   // what index -1 reads, in front of every row
        const int done = n_src / EPC * EPC;
        for (int b = 0; b < a.batch; ++b)
            for (int j = done + tid; j < n_dst; j += kThreads)
                dst[b * dst_stride + j] = j < n_src ? x[(size_t)b * a.ldx + j] : T(0.0f);
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");   // tables and first weight fragments have landed
    __syncthreads();                                        // ... for every thread, and the stores above are visible
    plan_parks(d, L);
    if (a.stage_mode != 0 && (a.stage_mode != 2 ? a.x_len : a.x_limit) >= EPC) {   // and so must x
        const uint32_t bar = (uint32_t)__cvta_generic_to_shared(L.xbar);
        uint32_t ok = 0u;
        // Normally up to kXWaitPolls polls that may each suspend the thread for a while (seconds in all).  A
        // caller-set limit counts polls that return at once, so that a test can make the wait run out on purpose.
        if (a.wait_polls > 0) {
            for (int i = 0; i < a.wait_polls && !ok; ++i)
                asm volatile("{\n.reg .pred p;\nmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                             : "=r"(ok) : "r"(bar), "r"(x_parity) : "memory");
        } else {
            for (int i = 0; i < kXWaitPolls && !ok; ++i)
                asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                             : "=r"(ok) : "r"(bar), "r"(x_parity) : "memory");
        }
        if (!ok) {
            // bounded wait gave up: the output of this call is invalid.  The copy is still in flight; it must have
            // landed before this CTA's shared memory is given back, so wait once more with the kernel's own limit.
            if (a.status) *a.status = 1;
            for (int i = 0; i < kXWaitPolls && !ok; ++i)
                asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                             : "=r"(ok) : "r"(bar), "r"(x_parity) : "memory");
        }
    }
    if (a.stage_mode == 1) {
        __syncthreads();
        const T* raw = static_cast<const T*>(L.raw);
#pragma unroll 8
        for (int j = tid; j < a.n_pad; j += kThreads) {
            const int idx = L.idxs[j];
            for (int b = 0; b < a.batch; ++b)
                xs[b * a.xs_stride + j] = idx >= 0 ? raw[b * a.raw_stride + idx] : T(0.0f);
        }
    } else if (a.stage_mode == 0) {
        for (int j0 = tid; j0 < a.n_pad; j0 += 8 * kThreads) {
            int idx[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const int j = j0 + q * kThreads;
                idx[q] = j < a.n_pad ? x_index(a, j) : -1;
            }
            for (int b = 0; b < a.batch; ++b) {
                T v[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) v[q] = idx[q] >= 0 ? x[(size_t)b * a.ldx + idx[q]] : T(0.0f);
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    if (j0 + q * kThreads < a.n_pad) xs[b * a.xs_stride + j0 + q * kThreads] = v[q];
            }
        }
    }
    // modes 2..4 wrote nothing to shared memory since the barrier above (every thread has seen the x barrier
    // complete itself); the permutation passes of modes 0 and 1 did
    if (a.stage_mode < 2) __syncthreads();
}

constexpr unsigned kEmptySlot = 0xffffffffu;   // exchange slots rest at this NaN pattern

// Sum of the partial sums the warps parked for element `rem` (row * batch + column) of local strip `ls`, in warp
// order.  All sixteen candidate loads are issued before the first addition (a loop that tested and loaded warp after
// warp was a chain of sixteen shared-memory round trips on every call's tail).
template <int RG>
__device__ __forceinline__ float sum_parks_of(const SmemLayout& L, int ls, int rem, int per_strip) {
    const unsigned m = (unsigned)L.wlohi[ls];
    const float* base = L.segp + (size_t)ls * per_strip + rem;
    float s[kStreamWarps];
#pragma unroll
    for (int w = 0; w < kStreamWarps; ++w) s[w] = (m >> w) & 1u ? base[w * per_strip] : 0.0f;
    float v = 0.0f;
#pragma unroll
    for (int w = 0; w < kStreamWarps; ++w)
        if ((m >> w) & 1u) v += s[w];
    return v;
}

// Everything after the last barrier of the streaming phase: per-strip sums, cross-CTA reduction,
// bias + activation + (scatter | pivoted store).  RG = rows per strip.
//
// A strip shared by exactly two CTAs needs no counter and no fence: each CTA swaps its partial sum
// into the strip's exchange slot; whoever gets the resting pattern back was first and is done,
// the other gets the first one's partial sum back, adds its own (a + b == b + a bit for bit, so the
// order of arrival cannot change the result), stores the row and puts the resting pattern back.
// Strips shared by three or more CTAs publish one partial sum per CTA and the last CTA to bump the
// strip's counter adds them in CTA order.
template <int RG>
__device__ __forceinline__ void finalize(const StreamArgs& a, const CtaDesc& d, const SmemLayout& L) {
    const int tid = threadIdx.x;
    const int batch = a.batch;
    const int per_strip = RG * batch;

    auto emit = [&](int ls, int r, int b, float v) {
        const int lr = ls * RG + r;
        v += L.rowbias[lr];
        if (a.act == PP_ACT_RELU) v = fmaxf(v, 0.0f);
        if (a.out_mode == OUT_SCATTER_F32 || a.out_mode == OUT_SCATTER_F16) {
            const int dst = L.rowdst[lr];
            if (dst >= 0) {
                if (a.out_mode == OUT_SCATTER_F32) static_cast<float*>(a.y)[(size_t)b * a.ldy + dst] = v;
                else static_cast<__half*>(a.y)[(size_t)b * a.ldy + dst] = __float2half_rn(v);
            }
        } else {
            const int i = d.s_first * RG + lr;
            if (a.out_mode == OUT_PIVOTED_F32) static_cast<float*>(a.y)[(size_t)b * a.ldy + i] = v;
            else static_cast<__half*>(a.y)[(size_t)b * a.ldy + i] = __float2half_rn(v);
        }
    };

    // One input vector (the common case) needs no index arithmetic beyond a shift: element e is row e of
    // the CTA's strips.  Kept apart from the general loop so that this path is a short run of code.
    const bool single = batch == 1;
    if (single) {
        for (int e = tid; e < d.s_count * RG; e += kThreads) {
            const int ls = e / RG, r = e % RG;
            float v = sum_parks_of<RG>(L, ls, r, per_strip);
            const int4 info = L.sinfo[ls];
            if (info.y == 2) {
                unsigned* slot = reinterpret_cast<unsigned*>(a.partials + (size_t)info.z * (RG * kStreamMaxBatch) + r);
                unsigned mine = __float_as_uint(v);
                if (mine == kEmptySlot) mine = 0x7fc00000u;
                const unsigned other = atomicExch(slot, mine);
                if (other == kEmptySlot) continue;
                v += __uint_as_float(other);
                *slot = kEmptySlot;
            } else if (info.y != 1) {
                a.partials[(size_t)(info.z + (int)blockIdx.x - info.x) * (RG * kStreamMaxBatch) + r] = v;
                continue;
            }
            emit(ls, r, 0, v);
        }
    }
    const int n_out = single ? 0 : d.s_count * per_strip;
    for (int e = tid; e < n_out; e += kThreads) {
        const int ls = e / per_strip, rem = e - ls * per_strip;
        const int r = rem / batch, b = rem - r * batch;
        const float v = sum_parks_of<RG>(L, ls, rem, per_strip);
        const int4 info = L.sinfo[ls];
        if (info.y == 1) {
            emit(ls, r, b, v);
        } else if (info.y == 2) {
            unsigned* slot = reinterpret_cast<unsigned*>(a.partials + (size_t)info.z * (RG * kStreamMaxBatch) + rem);
            unsigned mine = __float_as_uint(v);
            if (mine == kEmptySlot) mine = 0x7fc00000u;          // a NaN stays a NaN, but not the resting pattern
            const unsigned other = atomicExch(slot, mine);
            if (other != kEmptySlot) {
                emit(ls, r, b, v + __uint_as_float(other));
                *slot = kEmptySlot;
            }
        } else {
            a.partials[(size_t)(info.z + (int)blockIdx.x - info.x) * (RG * kStreamMaxBatch) + rem] = v;
        }
    }
    // only the first and the last strip of a CTA can be shared with a neighbour
    const int ls_edge[2] = {0, d.s_count - 1};
    int4 edge[2];
    edge[0] = L.sinfo[0];
    edge[1] = d.s_count > 1 ? L.sinfo[d.s_count - 1] : make_int4(0, 1, 0, 0);
    if (edge[0].y <= 2 && edge[1].y <= 2) return;      // uniform for the CTA
    __threadfence();
    __syncthreads();
    if (tid < 2) {
        int last = 0;
        if (edge[tid].y > 2) {
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
        const float* base = a.partials + (size_t)edge[k].z * (RG * kStreamMaxBatch);
        for (int e = tid; e < per_strip; e += kThreads) {
            float v = 0.0f;
            for (int p = 0; p < edge[k].y; ++p) v += ld_cg(base + (size_t)p * (RG * kStreamMaxBatch) + e);
            const int r = e / batch, b = e - r * batch;
            emit(ls_edge[k], r, b, v);
        }
        if (tid == 0) a.counters[d.s_first + ls_edge[k]] = 0;
    }
}

// Per-warp weight ring.  prologue(): fill the U slots (one cp.async group per slot, committed even
// when empty so that group counting stays uniform).  Inside the main loop, slot u is read after
// cp.async.wait_group U-1 and refilled with fragment p + U.
template <int U>
struct WeightRing {
    uint4* slot;           // this lane's 16 bytes of slot 0; slot u is slot + 32 * u
    const uint4* vals;     // this lane's 16 bytes of fragment 0
    __device__ __forceinline__ void fill(int u, int p, int wend) const {
        if (p < wend) cp_async_16(slot + 32 * u, vals + (size_t)p * 32);
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    __device__ __forceinline__ void refill(int u, int p) const {       // p is known to be inside the warp's range
        cp_async_16(slot + 32 * u, vals + (size_t)p * 32);
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    __device__ __forceinline__ void prologue(int wbeg, int wend) const {
#pragma unroll
        for (int u = 0; u < U; ++u) fill(u, wbeg + u, wend);
    }
    __device__ __forceinline__ uint4 take(int u) const {
        asm volatile("cp.async.wait_group %0;" :: "n"(U - 1) : "memory");
        return slot[32 * u];
    }
};

// A read-only global load that is issued where it stands: the compiler may move an ordinary load down to the first
// use of its value, which for a table fetched ahead of the dependency wait puts a trip to L2 or DRAM (0.7 us) back on
// the critical path behind the wait.
__device__ __forceinline__ int ld_nc_here(const int32_t* p) {
    int v;
    asm volatile("ld.global.nc.s32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}

// Column offsets of 32 consecutive fragments, one per lane, fetched one block ahead.
struct XoffWindow {
    const int32_t* xoff;
    int cur, nxt, base;    // cur covers fragments [base, base + 32)
    __device__ __forceinline__ void init(const int32_t* table, int wbeg, int wend, int lane) {
        xoff = table; base = wbeg;
        cur = wbeg + lane < wend ? ld_nc_here(xoff + wbeg + lane) : 0;
        nxt = wbeg + 32 + lane < wend ? ld_nc_here(xoff + wbeg + 32 + lane) : 0;
    }
    __device__ __forceinline__ int get(int p, int wend, int lane) {
        if (p - base == 32) {
            base += 32; cur = nxt;
            nxt = base + 32 + lane < wend ? ld_nc_here(xoff + base + 32 + lane) : 0;
        }
        return __shfl_sync(0xffffffffu, cur, p - base);
    }
};

// ------------------------------------------------------------------ fp16 tiles
// How a layer body meets the producer of its input.  release(): the consumer of this layer's output may start
// its own prologue.  wait(): called by all threads after a CTA barrier; on return everything the producer wrote
// is visible; false when a bounded wait gave up (the CTA then leaves the kernel).
struct LaunchDependency {      // the producer is the previous kernel in the stream (programmatic dependent launch)
    bool x_ready;              // x does not come from a kernel still in flight: only the writes have to wait
    __device__ __forceinline__ void release() const { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
    __device__ __forceinline__ bool wait() const {
        if (!x_ready) asm volatile("griddepcontrol.wait;" ::: "memory");
        return true;
    }
    // called right before the layer's first write to global memory (y, exchange slots, counters)
    __device__ __forceinline__ void wait_before_writes() const {
        if (x_ready) asm volatile("griddepcontrol.wait;" ::: "memory");
    }
};

// What a layer requests before it meets its producer: its tables and the first U weight fragments of every warp
// (nothing here depends on the producer).  The cp.async groups it commits are the caller's to wait for.
template <int U>
__device__ __forceinline__ void stream_f16_prologue(const StreamArgs& a, const CtaDesc d, unsigned char* smem_raw) {
    const SmemLayout L = carve(smem_raw, 16, U, a, 2);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int wbeg = warp_begin(d, warp), wend = warp_begin(d, warp + 1);
    if (tid <= kStreamWarps) L.wb[tid] = warp_begin(d, tid);
    issue_static<16>(a, d, L);
    const WeightRing<U> ring{L.ring + (warp * U) * 32 + lane, reinterpret_cast<const uint4*>(a.values) + lane};
    ring.prologue(wbeg, wend);
}

struct NothingEarly {
    __device__ __forceinline__ void operator()() const {}
};

// One fp16 layer on this CTA's range `d`: prologue (tables, first weights; skipped when the caller has already
// requested them into this layer's shared memory), dependency wait, x, multiply, epilogue.  `early` runs between
// the prologue and the dependency wait (a chain requests the next layer's prologue there).
// The x barrier must have been initialised (init_xbar) and published by a CTA barrier or be past an earlier use.
// Returns false when the dependency wait gave up; nothing of x or y has been touched then.
template <int U, class Dep, class Early = NothingEarly>
__device__ __forceinline__ bool stream_f16_layer(const StreamArgs& a, const CtaDesc d, unsigned char* smem_raw,
                                                 uint32_t x_parity, const Dep& dep, bool prologue_done = false,
                                                 const Early& early = Early{}) {
    constexpr int RG = 16;
    const SmemLayout L = carve(smem_raw, RG, U, a, 2);
    __half* xs = static_cast<__half*>(L.xs);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int wbeg = warp_begin(d, warp), wend = warp_begin(d, warp + 1);

    // 1. the consumer of this layer may start its own prologue; this one prefetches what does
    //    not depend on its producer: tables, first U weight fragments, column offsets
    trace_stamp(a, 0);
    dep.release();
    if (!prologue_done) stream_f16_prologue<U>(a, d, smem_raw);
    const WeightRing<U> ring{L.ring + (warp * U) * 32 + lane, reinterpret_cast<const uint4*>(a.values) + lane};
    early();
    XoffWindow xw;
    xw.init(a.xoff, wbeg, wend, lane);
    warm_translations(a);

    // 2. everything the producer wrote is complete from here on: fetch x
    //    (the barrier publishes the mbarrier's initialisation to the threads that will wait on it)
    __syncthreads();
    trace_stamp(a, 1);
    if (!dep.wait()) {
        asm volatile("cp.async.wait_group 0;" ::: "memory");     // the prologue's copies land before shared memory is given back
        return false;
    }
    trace_stamp(a, 2);
    issue_x<__half>(a, L);

    // 3. pivoted x in shared memory
    finish_stage<__half, U>(a, d, L, x_parity);
    trace_stamp(a, 3);

    // 4. stream this warp's share
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
        const bool direct = a.stage_mode >= 3, idx16 = a.stage_mode == 4;
        const unsigned short* rawu = static_cast<const unsigned short*>(L.raw);
        const __half* xrow = xs + g * a.xs_stride + 2 * t;
        uint32_t mb0 = 0u, mb1 = 0u;
        // batch 1: x is read through the index array (index -1 reads raw[-1] = 0).  Every 8 fragments the
        // warp builds their 8 B-operands at once, 4 lanes per fragment (lane 4f + t holds columns 2t, 2t+1,
        // 2t+8, 2t+9 of fragment f), and hands them to the lanes that feed the tensor core with two
        // shuffles per fragment.
        auto gather8 = [&](int p) {
            (void)xw.get(p, wend, lane);                       // moves the window when needed
            const int xo = __shfl_sync(0xffffffffu, xw.cur, (p - xw.base) + g);
            int2 i0, i1;
            if (idx16) {
                const uint16_t* t16 = reinterpret_cast<const uint16_t*>(L.idxs) + xo + 2 * t;
                const uint32_t p0 = *reinterpret_cast<const uint32_t*>(t16);
                const uint32_t p1 = *reinterpret_cast<const uint32_t*>(t16 + 8);
                i0 = make_int2((int)(p0 & 0xffffu) - 1, (int)(p0 >> 16) - 1);
                i1 = make_int2((int)(p1 & 0xffffu) - 1, (int)(p1 >> 16) - 1);
            } else {
                i0 = *reinterpret_cast<const int2*>(L.idxs + xo + 2 * t);
                i1 = *reinterpret_cast<const int2*>(L.idxs + xo + 2 * t + 8);
            }
            mb0 = (uint32_t)rawu[i0.x] | ((uint32_t)rawu[i0.y] << 16);
            mb1 = (uint32_t)rawu[i1.x] | ((uint32_t)rawu[i1.y] << 16);
        };
        // Several input vectors read through the index array: lane (g, t) fetches its own four entries of
        // input row g for every fragment (no pivoted copy of x in shared memory, no permutation pass).
        const bool direct1 = direct && a.batch == 1;
        const unsigned short* rawg = rawu + g * a.raw_stride;
        auto gather_row = [&](int xo, uint32_t& b0, uint32_t& b1) {
            if (!has_x) return;
            int2 i0, i1;
            if (idx16) {
                const uint16_t* t16 = reinterpret_cast<const uint16_t*>(L.idxs) + xo + 2 * t;
                const uint32_t p0 = *reinterpret_cast<const uint32_t*>(t16);
                const uint32_t p1 = *reinterpret_cast<const uint32_t*>(t16 + 8);
                i0 = make_int2((int)(p0 & 0xffffu) - 1, (int)(p0 >> 16) - 1);
                i1 = make_int2((int)(p1 & 0xffffu) - 1, (int)(p1 >> 16) - 1);
            } else {
                i0 = *reinterpret_cast<const int2*>(L.idxs + xo + 2 * t);
                i1 = *reinterpret_cast<const int2*>(L.idxs + xo + 2 * t + 8);
            }
            b0 = (uint32_t)rawg[i0.x] | ((uint32_t)rawg[i0.y] << 16);
            b1 = (uint32_t)rawg[i1.x] | ((uint32_t)rawg[i1.y] << 16);
        };
        // Fragments are taken in groups of GRP; fragment wbeg + i sits in ring slot i % U.  A group of 8
        // that lies inside one strip, with all its refills inside the warp's range, runs without any
        // per-fragment test (the common case: a strip is hundreds of fragments long).
        constexpr int GRP = (8 % U == 0) ? 8 : U;
        for (int base = wbeg; base < wend; base += GRP) {
            if (GRP == 8 && base + 8 + U <= wend && base + 8 <= seg_end) {
                if (direct1) gather8(base);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    uint32_t b0 = 0u, b1 = 0u;
                    if (direct1) {
                        b0 = __shfl_sync(0xffffffffu, mb0, j * 4 + t);
                        b1 = __shfl_sync(0xffffffffu, mb1, j * 4 + t);
                    } else if (direct) {
                        gather_row(xw.get(base + j, wend, lane), b0, b1);
                    } else {
                        const int xoff = xw.get(base + j, wend, lane);
                        if (has_x) {
                            b0 = *reinterpret_cast<const uint32_t*>(xrow + xoff);
                            b1 = *reinterpret_cast<const uint32_t*>(xrow + xoff + 8);
                        }
                    }
                    const uint4 wa = ring.take(j % U);
                    ring.refill(j % U, base + j + U);
                    mma_16x8x16(acc, wa, b0, b1);
                }
                continue;
            }
            if (GRP == 8 && direct) {
                // A group that ends the warp's range or crosses a strip boundary.  One input vector: the B operands
                // of the (up to) eight fragments are built at once (several vectors: every lane fetches its own entries
                // per fragment, as in the full groups above), then one pass per strip the group touches
                // (nearly always one).  A fragment costs two tests, two shuffles, the ring slot and the tensor-core
                // instruction: while the weights are in shared memory the SM is bound by instruction issue (eight
                // warps per scheduler), and the per-fragment bookkeeping of the general loop below took three times
                // as many instructions, which is most of the multiply phase of a sparse layer.
                if (direct1) gather8(base);
                else (void)xw.get(base, wend, lane);              // moves the window when needed
                const int gend = min(base + 8, wend);
                int p = base;
                while (true) {
                    if (p == seg_end) {
                        park(ls + warp);
                        acc[0] = acc[1] = acc[2] = acc[3] = 0.0f;
                        do { ++ls; } while (L.sstart[ls + 1] <= p);
                        seg_end = min(wend, L.sstart[ls + 1]);
                    }
                    const int end = min(gend, seg_end);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int q = base + j;
                        if (q >= p && q < end) {
                            uint32_t b0 = 0u, b1 = 0u;
                            if (direct1) {
                                b0 = __shfl_sync(0xffffffffu, mb0, j * 4 + t);
                                b1 = __shfl_sync(0xffffffffu, mb1, j * 4 + t);
                            } else {
                                gather_row(__shfl_sync(0xffffffffu, xw.cur, q - xw.base), b0, b1);
                            }
                            const uint4 wa = ring.take(j % U);
                            ring.fill(j % U, q + U, wend);
                            mma_16x8x16(acc, wa, b0, b1);
                        }
                    }
                    p = end;
                    if (p >= gend) break;
                }
                continue;
            }
            if (GRP == 8) {
                // The same pass per strip for an input staged in pivoted order (a chain's inner layers): a lane reads its
                // operand words straight from the staged row.
                (void)xw.get(base, wend, lane);              // moves the window when needed
                const int gend = min(base + 8, wend);
                int p = base;
                while (true) {
                    if (p == seg_end) {
                        park(ls + warp);
                        acc[0] = acc[1] = acc[2] = acc[3] = 0.0f;
                        do { ++ls; } while (L.sstart[ls + 1] <= p);
                        seg_end = min(wend, L.sstart[ls + 1]);
                    }
                    const int end = min(gend, seg_end);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int q = base + j;
                        if (q >= p && q < end) {
                            const int xoff = __shfl_sync(0xffffffffu, xw.cur, q - xw.base);
                            uint32_t b0 = 0u, b1 = 0u;
                            if (has_x) {
                                b0 = *reinterpret_cast<const uint32_t*>(xrow + xoff);
                                b1 = *reinterpret_cast<const uint32_t*>(xrow + xoff + 8);
                            }
                            const uint4 wa = ring.take(j % U);
                            ring.fill(j % U, q + U, wend);
                            mma_16x8x16(acc, wa, b0, b1);
                        }
                    }
                    p = end;
                    if (p >= gend) break;
                }
                continue;
            }
            if constexpr (GRP != 8) {            // rings of 6: fragment by fragment
#pragma unroll
            for (int j = 0; j < GRP; ++j) {
                const int p = base + j;
                if (p < wend) {
                    if (p == seg_end) {
                        park(ls + warp);
                        acc[0] = acc[1] = acc[2] = acc[3] = 0.0f;
                        do { ++ls; } while (L.sstart[ls + 1] <= p);
                        seg_end = min(wend, L.sstart[ls + 1]);
                    }
                    uint32_t b0 = 0u, b1 = 0u;
                    if (direct1) {
                        const int in_group = (p - wbeg) & 7;
                        if (in_group == 0) gather8(p);
                        b0 = __shfl_sync(0xffffffffu, mb0, in_group * 4 + t);
                        b1 = __shfl_sync(0xffffffffu, mb1, in_group * 4 + t);
                    } else if (direct) {
                        gather_row(xw.get(p, wend, lane), b0, b1);
                    } else {
                        const int xoff = xw.get(p, wend, lane);        // warp-wide shuffle: outside the lane test
                        if (has_x) {
                            b0 = *reinterpret_cast<const uint32_t*>(xrow + xoff);
                            b1 = *reinterpret_cast<const uint32_t*>(xrow + xoff + 8);
                        }
                    }
                    const uint4 wa = ring.take(j % U);
                    ring.fill(j % U, p + U, wend);
                    mma_16x8x16(acc, wa, b0, b1);
                }
            }
            }
        }
        park(ls + warp);
    }
    trace_stamp(a, 6);
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    trace_stamp(a, 4);
    dep.wait_before_writes();
    finalize<RG>(a, d, L);
    trace_stamp(a, 5);
    return true;
}

template <int U>
__global__ void __launch_bounds__(kThreads, 2) stream_f16_kernel(const __grid_constant__ StreamLaunch P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    init_xbar(carve(smem_raw, 16, U, P.a, 2));
    stream_f16_layer<U>(P.a, cta_range(P), smem_raw, 0u, LaunchDependency{P.a.x_ready != 0});
}

// ------------------------------------------------------------------ a whole chain of fp16 layers in one kernel
// Cooperative launch (every CTA resident).  CTA c runs its range of layer 0, then of layer 1, ...; between two
// layers the grid meets at a counter in global memory: a CTA that has stored its part of layer l adds one, and
// before it reads layer l's output it waits until all CTAs have done so.  The tables and the first weights of
// layer l + 1 are requested BEFORE that wait, so they arrive while the slowest CTA of layer l finishes; for layers
// of a few MiB that is the whole layer.  The wait is bounded: when it gives up the CTA raises the status word and
// leaves; every other CTA sees the word inside its own wait and leaves too.
struct GridCounterDependency {
    unsigned* counter;
    unsigned target;         // arrivals that complete the producer layer (0: nothing to wait for)
    int* status;
    int polls;
    __device__ __forceinline__ void release() const {}
    __device__ __forceinline__ void wait_before_writes() const {}
    __device__ __forceinline__ bool wait() const {
        __shared__ int ok_flag;
        if (threadIdx.x == 0) {
            int ok = target == 0u;
            for (int i = 0; i < polls && !ok; ++i) {
                unsigned seen;
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
                ok = seen >= target;
                if (!ok && (i & 63) == 63 && *reinterpret_cast<volatile int*>(status)) break;
            }
            if (!ok) *status = 1;
            // the producer's stores came through the generic proxy; x is fetched by bulk copies (asynchronous proxy)
            asm volatile("fence.proxy.async.global;" ::: "memory");
            ok_flag = ok;
        }
        __syncthreads();
        return ok_flag != 0;
    }
};

constexpr int kChainPolls = 1 << 22;

template <int U>
__global__ void __launch_bounds__(kThreads, 1) chain_f16_kernel(const ChainLaunch P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ StreamArgs args[kChainMaxLayers];
    __shared__ CtaDesc desc[kChainMaxLayers];
    const unsigned n_ctas = gridDim.x;
    // Two shared-memory regions alternate between the layers: while layer l works in one, the tables and first
    // weights of layer l + 1 arrive in the other.
    auto region = [&](int l) { return smem_raw + (size_t)(l & 1) * P.region_bytes; };
    // programmatic dependent launch: the next kernel in the stream may be scheduled as CTAs of this one retire
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x < 2) {          // the x barrier sits at the same place in every layer's carving of a region
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"((uint32_t)__cvta_generic_to_shared(region(threadIdx.x) + 104 * 4)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // all layers' arguments and this CTA's range of every layer, in two rounds of loads
    {
        const int n_words = P.n_layers * (int)(sizeof(StreamArgs) / 4);
        for (int i = threadIdx.x; i < n_words; i += kThreads)
            reinterpret_cast<uint32_t*>(args)[i] = __ldg(reinterpret_cast<const uint32_t*>(P.layers) + i);
        __syncthreads();
        if (threadIdx.x < P.n_layers) {
            const int l = threadIdx.x;
            CtaDesc dd{0, 0, 0, -1};                         // s_count < 0: this CTA is not part of the layer's plan
            if ((int)blockIdx.x < __ldg(P.grids + l)) {
                const int4 v = __ldg(reinterpret_cast<const int4*>(args[l].cta_desc) + blockIdx.x);
                dd = CtaDesc{v.x, v.y, v.z, v.w};
            }
            desc[l] = dd;
            if (l == 0) args[l].x = P.x;                      // the call's input and output; everything between is the chain's
            if (l == P.n_layers - 1) args[l].y = P.y;
            args[l].wait_polls = P.polls;
#ifdef PP_TRACE
            args[l].trace = P.trace ? P.trace + (size_t)l * 320 * 8 : nullptr;
#endif
        }
        __syncthreads();
    }
    if (desc[0].s_count >= 0) stream_f16_prologue<U>(args[0], desc[0], region(0));
    // everything before this kernel in the stream (the previous call on these buffers) is complete from here on
    asm volatile("griddepcontrol.wait;" ::: "memory");
    uint32_t x_uses[2] = {0u, 0u};
    bool alive = true;
    for (int l = 0; l < P.n_layers && alive; ++l) {
        const StreamArgs& a = args[l];
        const GridCounterDependency dep{P.counter, l == 0 ? 0u : n_ctas * (unsigned)l, P.status,
                                        P.polls > 0 ? P.polls : kChainPolls};
        auto next_prologue = [&]() {
            if (l + 1 < P.n_layers && desc[l + 1].s_count >= 0)
                stream_f16_prologue<U>(args[l + 1], desc[l + 1], region(l + 1));
        };
        if (desc[l].s_count >= 0) {
            const bool has_x = a.stage_mode != 0 && (a.stage_mode != 2 ? a.x_len : a.x_limit) >= 8;
            alive = stream_f16_layer<U>(a, desc[l], region(l), x_uses[l & 1] & 1u, dep, true, next_prologue);
            if (alive && has_x) ++x_uses[l & 1];
        } else {
            next_prologue();
            __syncthreads();
            alive = dep.wait();
        }
        if (alive && l + 1 < P.n_layers) {
            // this CTA's part of layer l is stored: make it visible, then count this CTA in
            __threadfence();
            __syncthreads();
            if (threadIdx.x == 0) atomicAdd(P.counter, 1u);
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    // Last use of the counter by this CTA.  Whoever is last of all puts it back to zero for the next launch; a
    // launch that gave up leaves it for the host to clear (pp_chain_status).
    if (alive && threadIdx.x == 0) {
        const unsigned total = n_ctas * (unsigned)P.n_layers;
        if (atomicAdd(P.counter, 1u) == total - 1u) *P.counter = 0u;
    }
}

// ------------------------------------------------------------------ fp32 tiles
template <int RG, int NB, int U>
__global__ void __launch_bounds__(kThreads, 2) stream_f32_kernel(const __grid_constant__ StreamLaunch P) {
    const StreamArgs& a = P.a;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const SmemLayout L = carve(smem_raw, RG, U, a, 4);
    float* xs = static_cast<float*>(L.xs);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const CtaDesc d = cta_range(P);
    const int wbeg = warp_begin(d, warp), wend = warp_begin(d, warp + 1);
    if (tid <= kStreamWarps) L.wb[tid] = warp_begin(d, tid);

    trace_stamp(a, 0);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    init_xbar(L);
    issue_static<RG>(a, d, L);
    const WeightRing<U> ring{L.ring + (warp * U) * 32 + lane, reinterpret_cast<const uint4*>(a.values) + lane};
    ring.prologue(wbeg, wend);
    XoffWindow xw;
    xw.init(a.xoff, wbeg, wend, lane);
    warm_translations(a);
    __syncthreads();
    trace_stamp(a, 1);
    if (!a.x_ready) asm volatile("griddepcontrol.wait;" ::: "memory");
    trace_stamp(a, 2);
    issue_x<float>(a, L);
    finish_stage<float, U>(a, d, L);
    trace_stamp(a, 3);

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
        const bool direct = a.stage_mode >= 3, idx16 = a.stage_mode == 4;
        const float* rawf = static_cast<const float*>(L.raw);
        // one fragment: 4 columns of RG rows (lane = row; with 16-row strips the upper half-warp takes the next 4 columns)
        auto multiply = [&](const uint4 wa, int xoff) {
            const float w0 = __uint_as_float(wa.x), w1 = __uint_as_float(wa.y);
            const float w2 = __uint_as_float(wa.z), w3 = __uint_as_float(wa.w);
            if (direct) {            // batch 1: read x through the index array (index -1 reads raw[-1] = 0)
                int4 ii;
                if (idx16) {
                    const uint2 pp2 = *reinterpret_cast<const uint2*>(reinterpret_cast<const uint16_t*>(L.idxs) + xoff + (lane / RG) * 4);
                    ii = make_int4((int)(pp2.x & 0xffffu) - 1, (int)(pp2.x >> 16) - 1, (int)(pp2.y & 0xffffu) - 1, (int)(pp2.y >> 16) - 1);
                } else {
                    ii = *reinterpret_cast<const int4*>(L.idxs + xoff + (lane / RG) * 4);
                }
                acc[0][0] = fmaf(w0, rawf[ii.x], acc[0][0]);
                acc[0][1] = fmaf(w1, rawf[ii.y], acc[0][1]);
                acc[0][0] = fmaf(w2, rawf[ii.z], acc[0][0]);
                acc[0][1] = fmaf(w3, rawf[ii.w], acc[0][1]);
                return;
            }
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
        };
        auto next_strip = [&](int p) {
            park(ls + warp);
            do { ++ls; } while (L.sstart[ls + 1] <= p);
            seg_end = min(wend, L.sstart[ls + 1]);
        };
        if (wend - wbeg <= U) {
            // A short range was requested whole by the prologue and finish_stage has waited for it: plain
            // shared-memory loads, nothing to wait for and nothing to refill.
            // One input vector: four fragments of one strip at a time, every load of the four issued before the first
            // use (offset -> index entries -> x values is a chain of three shared-memory round trips, about 0.2 us
            // when every fragment walks it alone).  The sums are added in the same order as one by one.
#pragma unroll 1
            for (int p = wbeg; p < wend;) {
                if (p == seg_end) next_strip(p);
                if (direct && p + 4 <= seg_end) {
                    int xo[4];
                    uint4 wa[4];
                    int4 ii[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) xo[j] = xw.get(p + j, wend, lane);
#pragma unroll
                    for (int j = 0; j < 4; ++j) wa[j] = ring.slot[32 * (p + j - wbeg)];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (idx16) {
                            const uint2 pp2 = *reinterpret_cast<const uint2*>(reinterpret_cast<const uint16_t*>(L.idxs) + xo[j] + (lane / RG) * 4);
                            ii[j] = make_int4((int)(pp2.x & 0xffffu) - 1, (int)(pp2.x >> 16) - 1, (int)(pp2.y & 0xffffu) - 1, (int)(pp2.y >> 16) - 1);
                        } else {
                            ii[j] = *reinterpret_cast<const int4*>(L.idxs + xo[j] + (lane / RG) * 4);
                        }
                    }
                    float xv[4][4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        xv[j][0] = rawf[ii[j].x]; xv[j][1] = rawf[ii[j].y]; xv[j][2] = rawf[ii[j].z]; xv[j][3] = rawf[ii[j].w];
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        acc[0][0] = fmaf(__uint_as_float(wa[j].x), xv[j][0], acc[0][0]);
                        acc[0][1] = fmaf(__uint_as_float(wa[j].y), xv[j][1], acc[0][1]);
                        acc[0][0] = fmaf(__uint_as_float(wa[j].z), xv[j][2], acc[0][0]);
                        acc[0][1] = fmaf(__uint_as_float(wa[j].w), xv[j][3], acc[0][1]);
                    }
                    p += 4;
                    continue;
                }
                multiply(ring.slot[32 * (p - wbeg)], xw.get(p, wend, lane));
                ++p;
            }
        } else {
            for (int base = wbeg; base < wend; base += U) {
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int p = base + u;
                    if (p < wend) {
                        if (p == seg_end) next_strip(p);
                        const int xoff = xw.get(p, wend, lane);
                        const uint4 wa = ring.take(u);
                        ring.fill(u, p + U, wend);
                        multiply(wa, xoff);
                    }
                }
            }
        }
        park(ls + warp);
    }
    trace_stamp(a, 6);
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    trace_stamp(a, 4);
    if (a.x_ready) asm volatile("griddepcontrol.wait;" ::: "memory");    // y and scratch may still be in use by the previous kernel
    finalize<RG>(a, d, L);
    trace_stamp(a, 5);
}

template <auto Kernel>
cudaError_t launch_one(const StreamLaunch& P, int grid, size_t smem, cudaStream_t stream) {
    static PerDeviceOnce configured;   // one table per kernel instantiation; the attribute belongs to the device
    if (smem > kStreamSmemLimit) return cudaErrorInvalidValue;
    if (smem > 48 * 1024) {
        int dev = -1;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (!configured.is_done(dev)) {
            e = cudaFuncSetAttribute(Kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStreamSmemLimit);
            if (e != cudaSuccess) return e;
            configured.mark(dev);
        }
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = g_stream_pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, Kernel, P);
}

template <int RG, int U>
cudaError_t launch_f32(const StreamLaunch& P, int grid, size_t smem, cudaStream_t stream) {
    if (P.a.batch == 1) return launch_one<stream_f32_kernel<RG, 1, U>>(P, grid, smem, stream);
    if (P.a.batch == 2) return launch_one<stream_f32_kernel<RG, 2, U>>(P, grid, smem, stream);
    if (P.a.batch <= 4) return launch_one<stream_f32_kernel<RG, 4, U>>(P, grid, smem, stream);
    return launch_one<stream_f32_kernel<RG, 8, U>>(P, grid, smem, stream);
}

// Row stride (elements) of the shared-memory copy of x as given.  With several rows, 8 elements more than the
// 16-element multiple: the rows then start 4 (fp16) or 8 (fp32) banks apart instead of in the same bank, which
// matters when lanes of different rows read the same column.
int raw_stride_for(int x_len, int batch) { return (x_len + 15) / 16 * 16 + (batch > 1 ? 8 : 0); }
int xs_stride_for(pp_dtype_t dt, int n_pad) { return dt == PP_F16 ? n_pad + 8 : n_pad + 4; }

}  // namespace

#ifdef PP_TRACE
unsigned long long* g_stream_trace = nullptr;   // diagnostic builds: [calls][kTraceCtas][8] stamps, filled call after call
int g_stream_trace_calls = 0, g_stream_trace_next = 0;
constexpr int kTraceCtas = 320;
#endif
int g_stream_wait_polls = 0;   // polls before a bounded device-side wait gives up; 0 = the kernels' defaults
int g_stream_depth = 0;   // ring slots per warp: 4, 6 or 8; 0 = chosen per launch
int g_stream_pdl = 1;     // launch with programmatic stream serialization (prologue overlaps the previous kernel)
int g_stream_x_ready = 0; // launches fetch x before the dependency wait (the caller's promise, tuning key 17)

namespace {
size_t smem_bytes_at(pp_dtype_t dt, int B, int n_pad, int x_len, int max_rows, int batch, int stage_mode, int depth);
}

// Fragments a warp of the plan streams on average (the ring depth is chosen by it).
int stream_frags_per_warp(const CtaDesc* host_table, int grid) {
    if (!host_table || grid <= 0) return 0;
    long long frags = 0;
    for (int c = 0; c < grid; ++c) frags += host_table[c].p_end - host_table[c].p_begin;
    return (int)(frags / ((long long)grid * kStreamWarps));
}

constexpr int kDeepRingFrags = 17;   // between 13.8 (density 0.25, 4 copies faster) and 20.8 (0.375, 8 copies faster) on 8192 x 8192

// Weight copies each warp keeps in flight.  Two CTAs share an SM when the grid is larger than the SM
// count and a CTA needs at most half of the SM's shared memory: then 4 per warp (64 KiB in flight per
// SM).  A CTA that has the SM to itself takes the deepest ring that still fits.
int stream_pick_depth(pp_dtype_t dt, int B, int n_pad, int x_len, int max_rows, int batch, int stage_mode, int grid,
                      int frags_per_warp) {
    if (g_stream_depth) return g_stream_depth;
    if (grid > 148 && smem_bytes_at(dt, B, n_pad, x_len, max_rows, batch, stage_mode, 4) <= 113 * 1024) {
        // Two CTAs per SM.  Long ranges of fp16 fragments stream faster with 8 copies per warp in flight when two
        // such CTAs still fit an SM (8192 x 8192 at density 1 / 0.5 / 0.375: 23.2 / 12.8 / 10.3 us with 4 copies,
        // 22.7 / 12.3 / 9.8 us with 8); short ranges are slower that way (density 0.25 and below: a call is one burst
        // of requests, and the deeper prologue only queues the copy of x behind more weight traffic).
        if (dt == PP_F16 && frags_per_warp >= kDeepRingFrags &&
            smem_bytes_at(dt, B, n_pad, x_len, max_rows, batch, stage_mode, 8) <= 113 * 1024)
            return 8;
        return 4;
    }
    for (int d : {8, 6})
        if (smem_bytes_at(dt, B, n_pad, x_len, max_rows, batch, stage_mode, d) <= kStreamSmemLimit) return d;
    return 4;
}

size_t stream_smem_bytes(pp_dtype_t dt, int B, int n_pad, int x_len, int max_rows, int batch, int stage_mode) {
    // sized for the shallowest ring a launch may pick (a launch with the SM to itself takes a deeper one if it fits)
    return smem_bytes_at(dt, B, n_pad, x_len, max_rows, batch, stage_mode, g_stream_depth ? g_stream_depth : 4);
}

namespace {
size_t smem_bytes_at(pp_dtype_t dt, int B, int n_pad, int x_len, int max_rows, int batch, int stage_mode, int depth) {
    const int rg = frag_geom(dt, B).rg_rows;
    const int esz = dt == PP_F16 ? 2 : 4;
    max_rows = (max_rows + 31) / 32 * 32;          // as the launcher rounds it
    size_t bytes = (size_t)kHeaderBytes + (size_t)max_rows * 8 + segp_bytes(max_rows, rg, batch) +
                   (size_t)kStreamWarps * depth * 512;
    if (stage_mode < 3) bytes += xs_bytes(batch, xs_stride_for(dt, n_pad), esz);
    if (stage_mode == 1 || stage_mode >= 3)
        bytes += (size_t)n_pad * (stage_mode == 4 ? 2 : 4) + 16 + (size_t)batch * raw_stride_for(x_len, batch) * esz;
    return bytes;
}
}  // namespace

void stream_finish_args(pp_dtype_t dt, StreamArgs& a) {
    a.xs_stride = xs_stride_for(dt, a.n_pad);
    a.raw_stride = raw_stride_for(a.x_len, a.batch);
    a.max_rows = (a.max_rows + 31) / 32 * 32;      // whole strips of either height; keeps the regions behind 128-byte aligned
    a.wait_polls = g_stream_wait_polls;
    a.trace = nullptr;
}

namespace {
template <int U>
int chain_resident_ctas_u(size_t smem) {
    int dev = 0, sms = 0, per_sm = 0, coop = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop ||
        cudaFuncSetAttribute(chain_f16_kernel<U>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStreamSmemLimit) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, chain_f16_kernel<U>, kThreads, smem) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return per_sm * sms;
}

template <int U>
cudaError_t launch_chain_u(const ChainLaunch& P, int grid, size_t smem, cudaStream_t stream) {
    static PerDeviceOnce configured;
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (!configured.is_done(dev)) {
        e = cudaFuncSetAttribute(chain_f16_kernel<U>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStreamSmemLimit);
        if (e != cudaSuccess) return e;
        configured.mark(dev);
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = g_stream_pdl ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, chain_f16_kernel<U>, P);
}
}  // namespace

int chain_resident_ctas(size_t smem, int depth) {
    return depth == 8 ? chain_resident_ctas_u<8>(smem) : chain_resident_ctas_u<4>(smem);
}

cudaError_t launch_chain_f16(const ChainLaunch& P_in, int grid, size_t smem, int depth, cudaStream_t stream) {
    if (smem > kStreamSmemLimit || grid < 1 || (depth != 4 && depth != 8)) return cudaErrorInvalidValue;
    ChainLaunch P = P_in;
    if (P.polls <= 0) P.polls = g_stream_wait_polls;
    if (P.n_layers < 1 || P.n_layers > kChainMaxLayers || smem < 2 * (size_t)P.region_bytes) return cudaErrorInvalidValue;
    P.trace = nullptr;
#ifdef PP_TRACE
    if (g_stream_trace && g_stream_trace_next + P.n_layers <= g_stream_trace_calls && grid <= kTraceCtas) {
        P.trace = g_stream_trace + (size_t)g_stream_trace_next * kTraceCtas * 8;
        g_stream_trace_next += P.n_layers;
    }
#endif
    return depth == 8 ? launch_chain_u<8>(P, grid, smem, stream) : launch_chain_u<4>(P, grid, smem, stream);
}

size_t stream_launch_smem(pp_dtype_t dt, int B, int n_pad, int x_len, int max_rows, int batch, int stage_mode, int depth) {
    return smem_bytes_at(dt, B, n_pad, x_len, max_rows, batch, stage_mode, depth);
}

cudaError_t launch_stream(pp_dtype_t dt, int B, const StreamArgs& a_in, const CtaDesc* host_table, int grid,
                          cudaStream_t stream) {
    if (grid <= 0) return cudaSuccess;
    StreamLaunch P;
    P.a = a_in;
    StreamArgs& a = P.a;
    if (a.batch < 1 || a.batch > kStreamMaxBatch || (a.stage_mode >= 3 && a.batch != 1 && dt != PP_F16) ||
        (a.stage_mode == 4 && !a.gather16))
        return cudaErrorInvalidValue;
    stream_finish_args(dt, a);
#ifdef PP_TRACE
    if (g_stream_trace && g_stream_trace_next < g_stream_trace_calls && grid <= kTraceCtas)
        a.trace = g_stream_trace + (size_t)(g_stream_trace_next++) * kTraceCtas * 8;
#endif
    if (grid <= kParamCtas)
        for (int c = 0; c < grid; ++c) P.table[c] = host_table[c];
    const int depth = stream_pick_depth(dt, B, a.n_pad, a.x_len, a.max_rows, a.batch, a.stage_mode, grid,
                                        stream_frags_per_warp(host_table, grid));
    const size_t smem = smem_bytes_at(dt, B, a.n_pad, a.x_len, a.max_rows, a.batch, a.stage_mode, depth);
    if (dt == PP_F16) {
        if (depth == 8) return launch_one<stream_f16_kernel<8>>(P, grid, smem, stream);
        if (depth == 6) return launch_one<stream_f16_kernel<6>>(P, grid, smem, stream);
        return launch_one<stream_f16_kernel<4>>(P, grid, smem, stream);
    }
    if (B < 32) {
        if (depth == 8) return launch_f32<16, 8>(P, grid, smem, stream);
        if (depth == 6) return launch_f32<16, 6>(P, grid, smem, stream);
        return launch_f32<16, 4>(P, grid, smem, stream);
    }
    if (depth == 8) return launch_f32<32, 8>(P, grid, smem, stream);
    if (depth == 6) return launch_f32<32, 6>(P, grid, smem, stream);
    return launch_f32<32, 4>(P, grid, smem, stream);
}

}  // namespace pp

#ifdef PP_TRACE
// Diagnostic builds only: the next `calls` launches of the persistent kernel write their phase stamps to
// `device_buffer` (calls x 320 x 8 unsigned 64-bit words).
extern "C" void pp_trace_set_buffer(void* device_buffer, int calls) {
    pp::g_stream_trace = static_cast<unsigned long long*>(device_buffer);
    pp::g_stream_trace_calls = calls;
    pp::g_stream_trace_next = 0;
}
#endif
