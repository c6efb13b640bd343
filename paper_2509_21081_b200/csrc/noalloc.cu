// typhoon_mla_naive_shared_noalloc: shared-prefix attention for callers that
// must not allocate device memory.
//
// The regular entry point takes a caller-allocated workspace for the KV-split
// partials of the naive shared-prefix attention.  Some callers have no way to
// provide one: a serving process that handed every free byte of HBM to its
// KV-cache pool at start-up (a later cudaMalloc would simply fail), or a
// latency-critical loop in which cudaMalloc/cudaFree are banned because they
// synchronise the device and take the driver's allocator lock.  For them this
// file keeps the scratch in a fixed device array that is part of the library
// image.  CUDA loads the module that holds the array lazily, at the first
// lookup of its address on a device, and loading it is what takes the 32 MiB
// of device memory.  typhoon_mla_prepare_shared therefore does that lookup for
// its device (preparing a prefix allocates anyway and happens before serving
// starts); from then on the array stays until the process exits, and this
// entry point only reads a cached pointer.
#include <mutex>

#include "handle.h"
#include "kernels.h"

using namespace tmla;

namespace {

// Split partials: per (split, request, head) 128 fp32 outputs + 1 fp32 LSE.
constexpr size_t kScratchBytes = TYPHOON_MLA_NOALLOC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

// In host code `g_noalloc_scratch` is only a handle for the runtime, not an
// address a kernel can use; the device address is looked up once per device.
constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {};

// Cached address for device `dev`, or null if it has not been resolved yet.
void* cached_scratch(int dev) {
    if (dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_mu);
    return g_scratch_ptr[dev];
}

}  // namespace

int tmla::noalloc_resolve_scratch_for_current_device() {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return api_cuda_fail(e);
    if (dev < 0 || dev >= kMaxDevices) return TYPHOON_MLA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess || p == nullptr) {
            cudaGetLastError();
            return api_cuda_fail(e != cudaSuccess ? e : cudaErrorInvalidSymbol);
        }
        g_scratch_ptr[dev] = p;
    }
    return TYPHOON_MLA_OK;
}

extern "C" int typhoon_mla_naive_shared_noalloc(const typhoon_mla_shared_t* sh, const void* q_nope, const void* q_pe,
                                                 int32_t B, float softmax_scale, void* out, float* lse_out,
                                                 void* stream) {
    api_set_last_launches(0);
    if (!sh || !q_nope || !q_pe || !out || B < 1) return TYPHOON_MLA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(q_nope) | reinterpret_cast<uintptr_t>(q_pe) | reinterpret_cast<uintptr_t>(out)) & 15u)
        return TYPHOON_MLA_ERR_INVALID_ARG;
    if (!(softmax_scale > 0.f) || softmax_scale > 3.0e38f) return TYPHOON_MLA_ERR_INVALID_ARG;   // positive, finite
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return api_cuda_fail(e);
    if (dev != sh->device) return TYPHOON_MLA_ERR_INVALID_ARG;   // the handle's caches live on another device
    const int H = sh->dims.num_heads;
    const size_t rows = (size_t)B * H;
    const size_t per_split = rows * 128 * sizeof(float) + ((rows * sizeof(float) + 255) / 256) * 256;
    if (per_split > kScratchBytes) return TYPHOON_MLA_ERR_STATIC_SCRATCH_EXCEEDED;

    // resolved when the handle was prepared on this device
    void* scratch = cached_scratch(sh->device);
    if (!scratch) return TYPHOON_MLA_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);

    // Work decomposition of the shared-prefix kernel (the same tcgen05 kernel the regular entry point runs): the
    // library's choice if its partial slots fit the array, else one tile range per head, which needs one slot.
    const int n_sm = sh->num_sms > 0 ? sh->num_sms : 148;
    int n_ranges = 0, n_slots = 0;
    if (sh->Ls > 0) {
        naive_sm100_plan(B, H, sh->Ls, n_sm, 0, &n_ranges, &n_slots, sh->fp8 != 0);
        if ((size_t)n_slots * per_split > kScratchBytes) {
            n_ranges = H;
            n_slots = 1;
        }
    }
    float* o_part = reinterpret_cast<float*>(scratch);
    float* lse_part = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(scratch) +
                                               (size_t)(n_slots > 0 ? n_slots : 1) * rows * 128 * sizeof(float));
    // Every (slot, request, head) entry that the combine reads is written by the attention kernel of the same
    // call (slots a head does not use get lse = -inf), so nothing has to start at zero and the previous call's
    // contents never leak into this one.
    tl_pdl = false;   // ordinary stream-ordered launches
    int launches = 0;
    if (n_slots > 0) {
        NaiveAttnSm100 na{q_nope, q_pe, &sh->tm_kn, &sh->tm_kp, &sh->tm_vt, B, H, (int)sh->Ls, n_ranges, n_slots,
                          softmax_scale, o_part, lse_part, sh->status, B};
        if (sh->fp8) na.fp8_mult = sh->fp8_f;
        e = launch_naive_attn_sm100(na, s);
        if (e != cudaSuccess) return api_cuda_fail(e);
        ++launches;
    }
    e = launch_combine(o_part, lse_part, n_slots, nullptr, nullptr, B, H, out, lse_out, s);
    if (e != cudaSuccess) return api_cuda_fail(e);
    api_set_last_launches(launches + 1);
    return TYPHOON_MLA_OK;
}
