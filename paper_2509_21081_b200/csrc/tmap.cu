// Host helper: tiled bf16 tensor maps (TMA descriptors) with 128-byte swizzle.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstring>
#include <mutex>

#include "sm100.cuh"

namespace tmla {
namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
std::once_flag g_once;
}  // namespace

cudaError_t make_tmap_bf16(CUtensorMap* out, const void* base, int rank, const uint64_t* dims,
                           const uint64_t* strides_bytes, const uint32_t* box) {
    std::call_once(g_once, [] {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            g_encode = reinterpret_cast<EncodeTiledFn>(fn);
        else
            cudaGetLastError();
    });
    if (!g_encode) return cudaErrorNotSupported;
    if (rank < 2 || rank > 5) return cudaErrorInvalidValue;
    // A decode step re-creates the same handful of descriptors (queries, workspace buffers, page arrays)
    // every call.  The encoding is a pure function of its arguments, so each host thread remembers results in a
    // direct-mapped table (a serving loop with several steps in flight has a few dozen live descriptors) and a
    // repeated request costs one hash and one comparison instead of a driver call.
    struct Key {
        const void* base; int rank; uint64_t dims[5]; uint64_t strides[4]; uint32_t box[5];
    };
    struct Entry { Key key; CUtensorMap map; bool valid; };
    constexpr int kCacheEntries = 256;
    thread_local Entry cache[kCacheEntries] = {};
    Key key;
    std::memset(&key, 0, sizeof(key));
    key.base = base; key.rank = rank;
    for (int i = 0; i < rank; ++i) {
        key.dims[i] = dims[i];
        key.box[i] = box[i];
        if (i > 0) key.strides[i - 1] = strides_bytes[i - 1];
    }
    uint64_t hsh = 1469598103934665603ull;   // FNV-1a over the key's bytes
    {
        const unsigned char* kb = reinterpret_cast<const unsigned char*>(&key);
        for (size_t i = 0; i < sizeof(Key); ++i) hsh = (hsh ^ kb[i]) * 1099511628211ull;
    }
    Entry& slot = cache[(hsh ^ (hsh >> 17)) % kCacheEntries];
    if (slot.valid && std::memcmp(&slot.key, &key, sizeof(Key)) == 0) {
        *out = slot.map;
        return cudaSuccess;
    }
    cuuint64_t gdim[5];
    cuuint64_t gstr[5];
    cuuint32_t bx[5], es[5];
    for (int i = 0; i < rank; ++i) {
        gdim[i] = dims[i];
        bx[i] = box[i];
        es[i] = 1;
        if (i > 0) gstr[i - 1] = strides_bytes[i - 1];
    }
    CUresult r = g_encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gdim, gstr,
                          bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    slot.key = key;
    slot.map = *out;
    slot.valid = true;
    return cudaSuccess;
}

}  // namespace tmla
