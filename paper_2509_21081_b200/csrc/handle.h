// The prepared-prefix handle behind typhoon_mla_shared_t (host object; see typhoon_mla_prepare_shared).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/typhoon_mla.h"

struct typhoon_mla_shared {
    typhoon_mla_dims_t dims;
    int64_t Ls, Ls_pad;
    void* k_nope;   // bf16 [H, Ls_pad/64, 2, 64, 64]: 64-token x 64-dim tiles, each contiguous
    void* v_t;      // bf16 [H, Ls_pad/64, 128, 64]: V^T in contiguous 64-token blocks
    void* ckv;      // bf16 [Ls_pad, 512]
    void* kpe;      // bf16 [Ls_pad, 64]
    void* w_uk_t;   // bf16 [H, 512, 128]
    const void* w_uv;  // borrowed, bf16 [H, 128, 512]
    CUtensorMap tm_kn, tm_kp, tm_vt;   // TMA descriptors of k_nope, kpe, v_t (valid if Ls > 0)
    CUtensorMap tm_wuk_t;              // TMA descriptor of w_uk_t
    CUtensorMap tm_ckv, tm_kpe_tok;    // TMA descriptors of ckv, kpe as 64-token pages (valid if Ls > 0)
    cudaStream_t side_stream;          // absorb branch of a hybrid step runs here, beside the naive kernel
    cudaEvent_t ev_fork, ev_join;
    int* status;    // device word: non-zero after a bounded in-kernel wait expired
    size_t owned_bytes;
    int device;     // device the handle was prepared on; every call checks that it is the current one
    int num_sms;    // multiprocessors of that device (the work decompositions fill them)
    // 8-bit expanded cache (typhoon_mla_prepare_shared_fp8): k_nope and v_t are null, the codes live here and
    // tm_kn / tm_vt describe the code arrays
    int fp8;
    void* k8;       // E4M3 codes [H, Ls_pad, 128]: token rows of 128 dims
    void* v8;       // E4M3 codes [H, Ls_pad/64, 128, 64]: V^T in 64-token blocks
    float* fp8_f;   // device [2][H] floats: scale of K_nope, scale of V; then [H] words of scratch for the amax reduction
};
