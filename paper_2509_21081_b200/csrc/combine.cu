// Vector kernels of the path: merge of absorb chunk partials, the final LSE
// combine (Algorithm 1 line 8; Section 3.2 "CombineLSE") and layout helpers
// used once per prefix by the expansion step.
#include "common.cuh"
#include "kernels.h"

namespace tmla {
namespace {

// One block of 128 threads per (b, h); each thread owns 4 of the 512 latent columns.
__global__ void __launch_bounds__(128) merge_latent_kernel(const float* __restrict__ o_part,
                                                           const float* __restrict__ lse_part, int n_chunks,
                                                           int BH, __nv_bfloat16* __restrict__ o_lat,
                                                           float* __restrict__ lse) {
    const int bh = blockIdx.x;
    float m = -INFINITY;
    for (int c = 0; c < n_chunks; ++c) m = fmaxf(m, lse_part[(int64_t)c * BH + bh]);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float z = 0.f;
    if (m != -INFINITY) {
        for (int c = 0; c < n_chunks; ++c) {
            float l = lse_part[(int64_t)c * BH + bh];
            if (l == -INFINITY) continue;  // empty chunk: its O slot was never written
            float w = __expf(l - m);
            float4 v = *reinterpret_cast<const float4*>(o_part + ((int64_t)c * BH + bh) * 512 + threadIdx.x * 4);
            acc.x += w * v.x; acc.y += w * v.y; acc.z += w * v.z; acc.w += w * v.w;
            z += w;
        }
        float inv = 1.f / z;
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    }
    uint2 pk = make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
    *reinterpret_cast<uint2*>(o_lat + (int64_t)bh * 512 + threadIdx.x * 4) = pk;
    if (threadIdx.x == 0) lse[bh] = (m == -INFINITY) ? -INFINITY : m + __logf(z);
}

// One warp per (b, h); each lane owns 4 of the 128 output columns.
__global__ void __launch_bounds__(256) combine_kernel(const float* __restrict__ o_naive,
                                                      const float* __restrict__ lse_naive, int n_naive,
                                                      const float* __restrict__ o_abs,
                                                      const float* __restrict__ lse_abs, int BH,
                                                      __nv_bfloat16* __restrict__ out, float* __restrict__ lse_out) {
    const int bh = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (bh >= BH) return;
    float m = -INFINITY;
    for (int i = 0; i < n_naive; ++i) m = fmaxf(m, lse_naive[(int64_t)i * BH + bh]);
    float la = -INFINITY;
    if (o_abs != nullptr) {
        la = lse_abs[bh];
        m = fmaxf(m, la);
    }
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float z = 0.f;
    if (m != -INFINITY) {
        for (int i = 0; i < n_naive; ++i) {
            float l = lse_naive[(int64_t)i * BH + bh];
            if (l == -INFINITY) continue;
            float w = __expf(l - m);
            float4 v = *reinterpret_cast<const float4*>(o_naive + ((int64_t)i * BH + bh) * 128 + lane * 4);
            acc.x += w * v.x; acc.y += w * v.y; acc.z += w * v.z; acc.w += w * v.w;
            z += w;
        }
        if (la != -INFINITY) {
            float w = __expf(la - m);
            float4 v = *reinterpret_cast<const float4*>(o_abs + (int64_t)bh * 128 + lane * 4);
            acc.x += w * v.x; acc.y += w * v.y; acc.z += w * v.z; acc.w += w * v.w;
            z += w;
        }
        float inv = 1.f / z;
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    }
    uint2 pk = make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
    *reinterpret_cast<uint2*>(out + (int64_t)bh * 128 + lane * 4) = pk;
    if (lse_out != nullptr && lane == 0) lse_out[bh] = (m == -INFINITY) ? -INFINITY : m + __logf(z);
}

__global__ void __launch_bounds__(256) transpose_bf16_kernel(const __nv_bfloat16* __restrict__ in,
                                                             __nv_bfloat16* __restrict__ out, int R, int C) {
    __shared__ __nv_bfloat16 tile[32][34];
    const int64_t off = (int64_t)blockIdx.z * R * C;
    const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int i = ty; i < 32; i += 8) {
        int r = r0 + i, c = c0 + tx;
        tile[i][tx] = (r < R && c < C) ? in[off + (int64_t)r * C + c] : __float2bfloat16(0.f);
    }
    __syncthreads();
    for (int i = ty; i < 32; i += 8) {
        int c = c0 + i, r = r0 + tx;
        if (r < R && c < C) out[off + (int64_t)c * R + r] = tile[tx][i];
    }
}

__global__ void __launch_bounds__(256) copy_pad_rows_kernel(const __nv_bfloat16* __restrict__ in, int64_t ld_in,
                                                            __nv_bfloat16* __restrict__ out, int L, int Lp, int W8) {
    int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
    int64_t total = (int64_t)Lp * W8;
    if (idx >= total) return;
    int row = (int)(idx / W8), ch = (int)(idx % W8);
    uint4 v = make_uint4(0, 0, 0, 0);
    if (row < L) v = *reinterpret_cast<const uint4*>(in + (int64_t)row * ld_in + ch * 8);
    *reinterpret_cast<uint4*>(out + ((int64_t)row * W8 + ch) * 8) = v;
}

// Longest-first launch order for ragged suffixes: perm[] = request indices sorted by descending
// suffix length (ties by index, so the order is deterministic).  One block, bitonic sort in
// shared memory of up to 4096 keys.
__global__ void __launch_bounds__(1024) order_by_length_kernel(const int32_t* __restrict__ seq_lens, int B,
                                                               int32_t* __restrict__ perm) {
    __shared__ unsigned long long keys[4096];
    block_order_by_length(seq_lens, B, perm, keys);
}

}  // namespace

cudaError_t launch_order_by_length(const int32_t* seq_lens, int B, int32_t* perm, cudaStream_t s) {
    if (B <= 0 || B > 4096) return cudaErrorInvalidValue;
    order_by_length_kernel<<<1, 1024, 0, s>>>(seq_lens, B, perm);
    return cudaGetLastError();
}

cudaError_t launch_merge_latent(const float* o_part, const float* lse_part, int n_chunks, int B, int H,
                                void* o_lat_bf16, float* lse, cudaStream_t s) {
    if (B * H <= 0) return cudaSuccess;
    merge_latent_kernel<<<B * H, 128, 0, s>>>(o_part, lse_part, n_chunks, B * H,
                                              reinterpret_cast<__nv_bfloat16*>(o_lat_bf16), lse);
    return cudaGetLastError();
}

cudaError_t launch_combine(const float* o_naive, const float* lse_naive, int n_naive, const float* o_abs,
                           const float* lse_abs, int B, int H, void* out_bf16, float* lse_out, cudaStream_t s) {
    int BH = B * H;
    if (BH <= 0) return cudaSuccess;
    combine_kernel<<<(BH + 7) / 8, 256, 0, s>>>(o_naive, lse_naive, n_naive, o_abs, lse_abs, BH,
                                                reinterpret_cast<__nv_bfloat16*>(out_bf16), lse_out);
    return cudaGetLastError();
}

cudaError_t launch_transpose_bf16(const void* in, void* out, int R, int C, int batch, cudaStream_t s) {
    if (R <= 0 || C <= 0 || batch <= 0) return cudaSuccess;
    dim3 grid((C + 31) / 32, (R + 31) / 32, batch);
    transpose_bf16_kernel<<<grid, 256, 0, s>>>(reinterpret_cast<const __nv_bfloat16*>(in),
                                               reinterpret_cast<__nv_bfloat16*>(out), R, C);
    return cudaGetLastError();
}

cudaError_t launch_copy_pad_rows(const void* in, int64_t ld_in, void* out, int L, int Lp, int W, cudaStream_t s) {
    if (Lp <= 0) return cudaSuccess;
    int W8 = W / 8;
    int64_t total = (int64_t)Lp * W8;
    copy_pad_rows_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(
        reinterpret_cast<const __nv_bfloat16*>(in), ld_in, reinterpret_cast<__nv_bfloat16*>(out), L, Lp, W8);
    return cudaGetLastError();
}

}  // namespace tmla
