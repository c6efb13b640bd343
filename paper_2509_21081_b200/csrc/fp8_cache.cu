// 8-bit (E4M3) storage of the expanded shared-prefix cache: per-head power-of-two scales and the encoding
// pass that runs once when a prefix is prepared.  The paper only assumes 8-bit caches in its memory-footprint
// analysis (Section 4, "HBM Footprint"); format, rounding and scaling are this library's reading of it: OCP
// E4M3 (no infinities, largest value 448), round to nearest even, saturating, one scale 2^e per head and tensor
// with e the smallest integer such that amax / 2^e <= 448.  What is encoded is the 16-bit expanded cache, so the
// 16-bit path's rounding comes first.
#include <cuda_fp8.h>

#include <algorithm>

#include "common.cuh"
#include "kernels.h"

namespace tmla {
namespace {

// amax per head over a head-major bf16 array (padding tokens are zero and do not matter)
__global__ void amax_kernel(const uint4* __restrict__ src, size_t vec_per_head, uint32_t* __restrict__ amax_bits) {
    const int h = blockIdx.y;
    const uint4* p = src + (size_t)h * vec_per_head;
    uint32_t m = 0;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < vec_per_head; i += (size_t)gridDim.x * blockDim.x) {
        const uint4 v = p[i];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            m = max(m, w[k] & 0x7fffu);            // |low element| as an ordered integer
            m = max(m, (w[k] >> 16) & 0x7fffu);    // |high element|
        }
    }
    m = __reduce_max_sync(0xffffffffu, m);
    if ((threadIdx.x & 31) == 0 && m) atomicMax(&amax_bits[h], m);
}

// scale[h] = 2^e, e the smallest integer with amax <= 448 * 2^e (e = 0 for an all-zero head)
__global__ void scale_kernel(const uint32_t* __restrict__ amax_bits, int H, float* __restrict__ scale) {
    const int h = blockIdx.x * blockDim.x + threadIdx.x;
    if (h >= H) return;
    const float amax = __uint_as_float(amax_bits[h] << 16);
    int e = 0;
    if (amax > 0.f && amax < INFINITY) {
        const int E = ilogbf(amax);                       // amax = m * 2^E, 1 <= m < 2
        const float m = ldexpf(amax, -E);
        e = (m <= 1.75f) ? E - 8 : E - 7;                 // 448 = 1.75 * 2^8
    }
    scale[h] = ldexpf(1.f, e);
}

__device__ __forceinline__ uint32_t encode4(uint2 v, float inv_scale) {
    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v.x));
    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v.y));
    const uint32_t c0 = __nv_cvt_float_to_fp8(a.x * inv_scale, __NV_SATFINITE, __NV_E4M3);
    const uint32_t c1 = __nv_cvt_float_to_fp8(a.y * inv_scale, __NV_SATFINITE, __NV_E4M3);
    const uint32_t c2 = __nv_cvt_float_to_fp8(b.x * inv_scale, __NV_SATFINITE, __NV_E4M3);
    const uint32_t c3 = __nv_cvt_float_to_fp8(b.y * inv_scale, __NV_SATFINITE, __NV_E4M3);
    return c0 | (c1 << 8) | (c2 << 16) | (c3 << 24);
}

// K_nope: bf16 [H, Lp/64, 2 slabs, 64 tokens, 64 dims] -> codes [H, Lp tokens, 128 dims]; one thread per 4 codes
__global__ void quantize_k_kernel(const uint2* __restrict__ src, const float* __restrict__ scale, int64_t Lp,
                                  uint32_t* __restrict__ dst) {
    const int h = blockIdx.y;
    const float inv = __fdiv_rn(1.f, scale[h]);   // a power of two: exact
    const int64_t n = Lp * 32;                            // 4-code groups of this head
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t t = i >> 5;
        const int dg = (int)(i & 31), slab = dg >> 4;
        const int64_t s = (((int64_t)h * (Lp / 64) + t / 64) * 2 + slab) * 4096 + (t % 64) * 64 + (dg & 15) * 4;
        dst[(int64_t)h * n + i] = encode4(src[s >> 2], inv);
    }
}

// V^T: bf16 [H, Lp/64, 128 dims, 64 tokens] -> codes in the same order
__global__ void quantize_v_kernel(const uint2* __restrict__ src, const float* __restrict__ scale, int64_t Lp,
                                  uint32_t* __restrict__ dst) {
    const int h = blockIdx.y;
    const float inv = __fdiv_rn(1.f, scale[h]);   // a power of two: exact
    const int64_t n = Lp * 32;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        dst[(int64_t)h * n + i] = encode4(src[(int64_t)h * n + i], inv);
}

}  // namespace

cudaError_t launch_quantize_e4m3(const void* src_bf16, bool is_v, int H, int64_t Ls_pad, void* dst_codes, uint32_t* amax_bits,
                                 float* scale_out, cudaStream_t s) {
    if (H <= 0 || Ls_pad <= 0) return cudaSuccess;
    cudaError_t e = cudaMemsetAsync(amax_bits, 0, (size_t)H * sizeof(uint32_t), s);
    if (e != cudaSuccess) return e;
    const size_t vec_per_head = (size_t)Ls_pad * 128 * 2 / 16;
    const int bx = (int)std::min<size_t>((vec_per_head + 255) / 256, 64);
    amax_kernel<<<dim3(bx, H), 256, 0, s>>>(reinterpret_cast<const uint4*>(src_bf16), vec_per_head, amax_bits);
    scale_kernel<<<(H + 127) / 128, 128, 0, s>>>(amax_bits, H, scale_out);
    const int qx = (int)std::min<int64_t>((Ls_pad * 32 + 255) / 256, 256);
    if (is_v)
        quantize_v_kernel<<<dim3(qx, H), 256, 0, s>>>(reinterpret_cast<const uint2*>(src_bf16), scale_out, Ls_pad,
                                                      reinterpret_cast<uint32_t*>(dst_codes));
    else
        quantize_k_kernel<<<dim3(qx, H), 256, 0, s>>>(reinterpret_cast<const uint2*>(src_bf16), scale_out, Ls_pad,
                                                      reinterpret_cast<uint32_t*>(dst_codes));
    return cudaGetLastError();
}

}  // namespace tmla
