// Forward entry point for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc on the inference path: real-time loops that
// were handed one fixed device arena at start-up, processes whose memory pool is owned by another
// runtime, or code running where an allocation (an implicit device synchronisation) is not
// allowed.  pp_forward_noalloc serves them: the caller uploads the packed layer image into memory
// it owns, and the cross-CTA reduction scratch of the persistent kernel lives in the fixed-size
// device array below, which every GPU that loads this library holds until the process exits.
#include <cuda_runtime.h>

#include <cstring>

#include "pp_gemv.cuh"
#include "pp_internal.h"
#include "pp_stream.cuh"

namespace {

constexpr size_t kStaticScratchBytes = 1u << 20;   // 1 MiB per GPU, shared by every call
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Raised by the kernel when its bounded wait for the copy of x gives up (the output of that call is invalid).
static __device__ __align__(16) int g_static_status;

constexpr int kMaxDevices = 64;
unsigned char* g_scratch_addr[kMaxDevices] = {};   // device address of g_static_scratch, per device
int* g_status_addr[kMaxDevices] = {};              // device address of g_static_status, per device

// The array's name is only a host-side handle; its device address must be asked for, once per
// device, with that device current.
cudaError_t scratch_address(unsigned char** out, int** status_out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!g_scratch_addr[dev] || !g_status_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        void* q = nullptr;
        e = cudaGetSymbolAddress(&q, g_static_status);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = static_cast<unsigned char*>(p);
        g_status_addr[dev] = static_cast<int*>(q);
    }
    *out = g_scratch_addr[dev];
    *status_out = g_status_addr[dev];
    return cudaSuccess;
}

size_t round256(size_t n) { return (n + 255) / 256 * 256; }

// Sections of the device image, in order: strip_start, strip_info, scatter_idx, bias_piv,
// gather_idx, xoff, values.  (The CTA ranges travel with each launch and are not part of it.)
struct ImageLayout {
    size_t off[7];
    size_t size[7];
    size_t bytes;
};

ImageLayout image_layout(const pp_packed* pk) {
    const size_t S = pk->strip_info.size();
    ImageLayout im;
    const size_t sz[7] = {(S + 1) * 4, S * sizeof(pp::StripInfo), (size_t)pk->Mpad * 4, (size_t)pk->Mpad * 4,
                          (size_t)pk->Npad * 4, pk->xoff.size() * 4, pk->values.size()};
    size_t pos = 0;
    for (int i = 0; i < 7; ++i) { im.off[i] = pos; im.size[i] = sz[i]; pos += round256(sz[i]); }
    im.bytes = pos ? pos : 256;
    return im;
}

constexpr int kParamTableCtas = 320;   // CTA ranges the persistent kernel carries in its parameters

}  // namespace

extern "C" {

pp_status_t pp_pack_device_image_bytes(const pp_packed_t* p, int64_t* bytes) {
    if (!p || !bytes) return PP_ERR_INVALID_ARG;
    *bytes = (int64_t)image_layout(p).bytes;
    return PP_OK;
}

pp_status_t pp_pack_device_image(const pp_packed_t* p, void* host_dst, int64_t bytes) {
    if (!p || !host_dst) return PP_ERR_INVALID_ARG;
    const ImageLayout im = image_layout(p);
    if (bytes < (int64_t)im.bytes) return PP_ERR_INVALID_ARG;
    unsigned char* d = static_cast<unsigned char*>(host_dst);
    std::memset(d, 0, im.bytes);
    const void* src[7] = {p->strip_start.data(), p->strip_info.data(), p->scatter_idx.data(), p->bias_piv.data(),
                          p->gather_idx.data(), p->xoff.data(), p->values.data()};
    for (int i = 0; i < 7; ++i)
        if (im.size[i]) std::memcpy(d + im.off[i], src[i], im.size[i]);
    return PP_OK;
}

pp_status_t pp_forward_noalloc(const pp_packed_t* p, const void* device_image, const void* x, void* y, int batch,
                               pp_act_t act, void* cuda_stream) {
    if (!p || !device_image || !x || !y || x == y) return PP_ERR_INVALID_ARG;
    if (act != PP_ACT_IDENTITY && act != PP_ACT_RELU) return PP_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(device_image) & 255u) || (reinterpret_cast<uintptr_t>(x) & 15u) ||
        (reinterpret_cast<uintptr_t>(y) & 15u))
        return PP_ERR_INVALID_ARG;
    if (batch < 1 || batch > pp::kStreamMaxBatch) return PP_ERR_UNSUPPORTED;   // the persistent kernel only
    const pp::FragGeom g = pp::frag_geom(p->wdtype, p->B);
    const size_t S = p->strip_info.size();
    const size_t slot_bytes = round256((size_t)p->stream_slots * g.rg_rows * pp::kStreamMaxBatch * 4);
    const size_t counter_bytes = round256((S ? S : 1) * 4);
    if (slot_bytes + counter_bytes > kStaticScratchBytes) return PP_ERR_UNSUPPORTED;   // more scratch than the fixed array holds
    if (p->cta_desc.size() > (size_t)kParamTableCtas) return PP_ERR_UNSUPPORTED;        // CTA ranges must fit the kernel parameters

    const int x_elt = p->wdtype == PP_F16 ? 2 : 4;
    int max_rows = 0;
    for (const pp::CtaDesc& c : p->cta_desc)
        max_rows = c.s_count * g.rg_rows > max_rows ? c.s_count * g.rg_rows : max_rows;
    const bool rows_aligned = batch == 1 || ((size_t)p->N * x_elt) % 16 == 0;
    const int fast = batch == 1 ? 3 : 1;
    int stage_mode = -1;
    if (rows_aligned && pp::stream_smem_bytes(p->wdtype, p->B, p->Npad, p->N, max_rows, batch, fast) <= pp::kStreamSmemLimit)
        stage_mode = fast;
    else if (pp::stream_smem_bytes(p->wdtype, p->B, p->Npad, p->N, max_rows, batch, 0) <= pp::kStreamSmemLimit)
        stage_mode = 0;
    if (stage_mode < 0) return PP_ERR_UNSUPPORTED;

    unsigned char* scratch = nullptr;
    int* status_word = nullptr;
    if (scratch_address(&scratch, &status_word) != cudaSuccess) { cudaGetLastError(); return PP_ERR_CUDA; }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // the array keeps whatever the last call left: exchange slots must rest at all ones, counters at zero
    if (slot_bytes && cudaMemsetAsync(scratch, 0xff, slot_bytes, stream) != cudaSuccess) return PP_ERR_CUDA;
    if (cudaMemsetAsync(scratch + slot_bytes, 0, counter_bytes, stream) != cudaSuccess) return PP_ERR_CUDA;

    const ImageLayout im = image_layout(p);
    const unsigned char* img = static_cast<const unsigned char*>(device_image);
    pp::StreamArgs s{};
    s.stage_mode = stage_mode;
    s.strip_start = reinterpret_cast<const int32_t*>(img + im.off[0]);
    s.strip_info = reinterpret_cast<const pp::StripInfo*>(img + im.off[1]);
    s.scatter_idx = reinterpret_cast<const int32_t*>(img + im.off[2]);
    s.bias_piv = reinterpret_cast<const float*>(img + im.off[3]);
    s.gather_idx = reinterpret_cast<const int32_t*>(img + im.off[4]);
    s.xoff = reinterpret_cast<const int32_t*>(img + im.off[5]);
    s.values = img + im.off[6];
    s.cta_desc = nullptr;                      // plans larger than the parameter table were refused above
    s.x = x; s.y = y;
    s.partials = reinterpret_cast<float*>(scratch);
    s.counters = reinterpret_cast<int*>(scratch + slot_bytes);
    s.status = status_word;
    s.ldx = p->N; s.ldy = p->M; s.x_limit = p->N; s.n_pad = p->Npad; s.x_len = p->N; s.max_rows = max_rows;
    s.batch = batch; s.act = (int)act; s.out_mode = pp::OUT_SCATTER_F32;
    return pp::launch_stream(p->wdtype, p->B, s, p->cta_desc.data(), (int)p->cta_desc.size(), stream) == cudaSuccess
               ? PP_OK : PP_ERR_CUDA;
}

// PP_ERR_TIMEOUT when a pp_forward_noalloc kernel on the current device gave up its bounded wait since the
// last query; the word is cleared by the read.  Synchronises with the device; allocates nothing.
pp_status_t pp_noalloc_status(pp_status_t* status) {
    if (!status) return PP_ERR_INVALID_ARG;
    *status = PP_OK;
    unsigned char* scratch = nullptr;
    int* status_word = nullptr;
    if (scratch_address(&scratch, &status_word) != cudaSuccess) { cudaGetLastError(); return PP_ERR_CUDA; }
    int flag = 0;
    if (cudaMemcpy(&flag, status_word, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return PP_ERR_CUDA;
    if (flag) {
        *status = PP_ERR_TIMEOUT;
        if (cudaMemset(status_word, 0, sizeof(int)) != cudaSuccess) return PP_ERR_CUDA;
    }
    return PP_OK;
}

}  // extern "C"
