// Internal launch interfaces between the C ABI (api.cu) and the kernels.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace tmla {

// Launch with the programmatic-stream-serialization attribute when enabled (see sm100::pdl_wait): the
// kernel must call pdl_wait() before its first access to global memory.  The switch is per thread: an API
// call copies its snapshot of the process-wide setting here before it launches anything.
extern thread_local bool tl_pdl;

// Opt-in shared-memory sizes of the kernels, set once per device (by typhoon_mla_prepare_shared, with that
// device current) instead of before every launch.
cudaError_t set_attrs_naive_sm100();
cudaError_t set_attrs_absorb_sm100();
cudaError_t set_attrs_stacked_sm100();
cudaError_t set_attrs_gemm_sm100();
cudaError_t set_attrs_q_absorb_sm100();
cudaError_t set_attrs_attn_mma();
cudaError_t set_attrs_gemm_tn();
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = tl_pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}


// C[z][m][n] = sum_k A[z][m][k] * B[z][n][k]   (both operands K-major, bf16, fp32 accumulate)
struct GemmTN {
    const void* A; int64_t lda; int64_t a_batch;   // elements
    const void* B; int64_t ldb; int64_t b_batch;
    void* C; int64_t ldc; int64_t c_batch;
    int M, N, K, batch;
    bool out_fp32;
    // 0: C[m][n] at m*ldc + n.  64: N is stored in blocks of 64 columns, each block a contiguous
    // [M][64] matrix: C[m][n] at (n/64)*M*64 + m*64 + n%64 (ldc ignored).
    int c_block_n = 0;
    // true: C is stored as 64 x 64 tiles, tile (m/64, n/64) contiguous and row-major inside,
    // tiles ordered by m/64 then n/64: C[m][n] at ((m/64)*(N/64) + n/64)*4096 + (m%64)*64 + n%64.
    bool c_tile64 = false;
};
cudaError_t launch_gemm_tn(const GemmTN& g, cudaStream_t s);
// tcgen05/TMEM/TMA version (bf16 output only; N % 128 == 0, K % 64 == 0).  `status` (device int,
// may be null) is set non-zero if a bounded wait inside the kernel expired.
// Optional fused epilogue (N must be 128): the accumulator row of (request m, head z) is taken as the
// normalised absorb-side output and merged with n_naive naive-side partials by their LSEs.
struct CombineEpilogue {
    const float* o_naive = nullptr;    // [n_naive][B][H][128]
    const float* lse_naive = nullptr;  // [n_naive][B][H]
    int n_naive = 0;
    const float* lse_abs = nullptr;    // [B][H]
    void* out = nullptr;               // bf16 [B][H][128]
    float* lse_out = nullptr;          // optional [B][H]
    int H = 0;
    int out_fp32 = 0;                  // `out` is fp32 [B][H][128] (a partial result for a later merge)
};
cudaError_t launch_gemm_tn_sm100(const GemmTN& g, int* status, cudaStream_t s, const CombineEpilogue* ce = nullptr);

// Query absorption on tcgen05 (one CTA per head and 128 requests); tm_w from make_q_absorb_tmap.
cudaError_t make_q_absorb_tmap(const void* w_uk_t, int H, CUtensorMap* tm_w);
// With seq_lens and order given (B <= 4096) one extra block also writes the longest-first request order and,
// with desc given, one int4 per launch position {request, clamped suffix length, first page, second page}
// (-1 where the block table has no such column) that saves the absorb kernel three dependent loads.
// walk_ctas > 0 (and B <= 128): that many CTAs walk through the heads instead of one CTA per head (for launches that share the
// GPU with a kernel that leaves only a few SMs free).
cudaError_t launch_q_absorb_sm100(const void* q_nope, const CUtensorMap* tm_w, void* q_abs, int B, int H, int n_sm, int walk_ctas, int* status,
                                  const int32_t* seq_lens, int32_t* order, const int32_t* block_table, int max_pages,
                                  int page_size, int32_t* desc, cudaStream_t s);

// Naive shared-prefix attention partials (Algorithm 1 line 4).
struct NaiveAttn {
    const void* q_nope; const void* q_pe;          // [B,H,128], [B,H,64]
    const void* k_nope; const void* v_t; const void* kpe;  // [H,Lp/64,2,64,64], [H,Lp/64,128,64], [Lp,64]
    int B, H; int Ls, Ls_pad; int n_split;
    float scale;
    float* o_part;   // [n_split][B][H][128], each normalised
    float* lse_part; // [n_split][B][H], natural log
};
cudaError_t launch_naive_attn_mma(const NaiveAttn& p, cudaStream_t s);

// tcgen05/TMEM/TMA version.  The tensor maps of the expanded cache are built once per prefix
// (make_naive_sm100_tmaps); number of tile ranges and partial slots come from naive_sm100_plan.
struct NaiveAttnSm100 {
    const void* q_nope; const void* q_pe;
    const CUtensorMap* tm_kn; const CUtensorMap* tm_kp; const CUtensorMap* tm_vt;   // host pointers
    int B, H; int Ls; int n_ranges, n_slots;
    float scale;
    float* o_part;   // [slots][part_rows][H][128], pointing at this launch's first row
    float* lse_part; // [slots][part_rows][H]
    int* status;     // device word, set non-zero if a bounded wait expired
    int part_rows = 0;   // rows of the partial arrays; 0 = B (a launch may fill a row range of a larger batch)
    // 8-bit cache: device [2][H] power-of-two scales of K_nope and V (tm_kn / tm_vt then describe the code arrays,
    // see make_naive_fp8_tmaps); null for the 16-bit cache
    const float* fp8_mult = nullptr;
};
int naive_sm100_tile_tokens(int B, bool fp8 = false);   // KV tile width the kernel uses for this batch size (64 or 128)
// CTAs (at most n_sm, each with an equal contiguous share of all (head, row group, tile) work) and
// partial slots for a problem size; a pure function of its arguments.
// schedule: 0 = chosen by the plan, 1 = column split, 2 = stream-K
void naive_sm100_plan(int B, int H, int64_t Ls, int n_sm, int schedule, int* n_ranges, int* n_slots, bool fp8 = false);
cudaError_t launch_naive_attn_sm100(const NaiveAttnSm100& a, cudaStream_t s);
cudaError_t make_naive_sm100_tmaps(const void* k_nope, const void* kpe, const void* v_t, int H, int64_t Ls_pad,
                                   CUtensorMap* tm_kn, CUtensorMap* tm_kp, CUtensorMap* tm_vt);
// Tensor maps of the E4M3 code arrays k8 [H, Ls_pad/64, 64 tokens, 128 dims] and v8 [H, Ls_pad/64, 128 dims,
// 64 tokens] (one byte per code; every 64-token block is 8 KB, copied as 64 rows of 128 bytes) and of the rope keys.
cudaError_t make_naive_fp8_tmaps(const void* k8, const void* kpe, const void* v8, int H, int64_t Ls_pad,
                                 CUtensorMap* tm_k8, CUtensorMap* tm_kp, CUtensorMap* tm_v8);
// Expanded 16-bit cache of one tensor (k_nope or v_t layout) -> per-head power-of-two scale (smallest 2^e with
// amax / 2^e <= 448) and E4M3 codes (round to nearest even) in the layouts above.  scale_out[h] = 2^e; amax_bits is
// a scratch of H words.
cudaError_t launch_quantize_e4m3(const void* src_bf16, bool is_v, int H, int64_t Ls_pad, void* dst_codes, uint32_t* amax_bits,
                                 float* scale_out, cudaStream_t s);

// Absorb attention partials over latent tokens (Algorithm 1 line 6).
struct AbsorbAttn {
    const void* q_abs; const void* q_pe;           // [B,H,512], [B,H,64]
    const void* ckv_shared; const void* kpe_shared; int Ls_absorb;  // shared prefix handled here (ABSORB mode) or 0
    const void* ckv_pages; const void* kpe_pages;
    int64_t ckv_stride, kpe_stride; int page_size;
    int num_pages;                                 // physical pages in ckv_pages / kpe_pages; ids outside are not read
    const int32_t* block_table; int max_pages; const int32_t* seq_lens;
    const int32_t* order;                          // optional [B]: request handled by block z (longest first)
    const int32_t* desc;                           // optional [B][4]: per launch position, see launch_q_absorb_sm100
    int B, H; int chunk;                           // tokens per chunk
    int n_shared_chunks, n_suffix_chunks;
    float scale;
    float* o_part;   // [n_chunks][B][H][512], each normalised
    float* lse_part; // [n_chunks][B][H]
    int* status = nullptr;   // device word: bit 0x100 is set when a page id was out of range
    bool stacked = false;    // tcgen05 kernel: shared-prefix chunks take 64-row groups of the stacked [B*H] queries
};
cudaError_t launch_absorb_attn_mma(const AbsorbAttn& p, cudaStream_t s);

// tcgen05/TMEM/TMA version (chunk must be a multiple of 64).  The tensor maps of the handle's copy of the
// shared latent cache come from make_absorb_shared_tmaps (used when n_shared_chunks > 0).
// With a single chunk in total the kernel writes the merged bf16 latent output [B,H,512] and its LSE [B,H]
// directly to o_lat_direct / lse_direct (no merge step needed); otherwise it writes the partials.
cudaError_t launch_absorb_attn_sm100(const AbsorbAttn& a, const CUtensorMap* tm_ckv_sh, const CUtensorMap* tm_kpe_sh,
                                     void* o_lat_direct, float* lse_direct, int* status, cudaStream_t s);
cudaError_t make_absorb_shared_tmaps(const void* ckv, const void* kpe, int64_t Ls_pad, CUtensorMap* tm_ckv,
                                     CUtensorMap* tm_kpe);

// perm[0..B) = request indices by descending suffix length (B <= 4096).
// -inf into n_slots segments of `count` floats, `stride` floats apart.
cudaError_t launch_fill_neg_inf(float* dst, int n_slots, int64_t stride, int64_t count, cudaStream_t s);
// Page table and lengths of the (request, query token) rows of a step with S_q query tokens per request.
cudaError_t launch_expand_query_rows(const int32_t* block_table, const int32_t* seq_lens, int B, int max_pages, int S_q,
                                     int32_t* bt_rows, int32_t* len_rows, cudaStream_t s);
cudaError_t launch_order_by_length(const int32_t* seq_lens, int B, int32_t* perm, cudaStream_t s);

// Merge absorb chunk partials -> bf16 latent output [B,H,512] + lse [B,H].
cudaError_t launch_merge_latent(const float* o_part, const float* lse_part, int n_chunks, int B, int H,
                                void* o_lat_bf16, float* lse, cudaStream_t s);

// Absorb-only step with one or two requests: merge of the chunk partials + W_UV projection (Algorithm 1 line 7)
// + final rounding in one launch; w_uv is [H, 128, 512] bf16; out bf16 (or fp32) [B, H, 128], lse_out optional.
cudaError_t launch_merge_project(const float* o_part, const float* lse_part, int n_chunks, int B, int H, const void* w_uv,
                                 void* out, float* lse_out, bool out_fp32, cudaStream_t s);

// Final LSE combine (Algorithm 1 line 8) of n_naive naive partials and an optional absorb partial;
// `out` is bf16 [B,H,128], or fp32 with out_fp32.
cudaError_t launch_combine(const float* o_naive, const float* lse_naive, int n_naive,
                           const float* o_abs, const float* lse_abs,
                           int B, int H, void* out, float* lse_out, cudaStream_t s, bool out_fp32 = false);

// One block that waits, with the given deadline in SM clocks, on a barrier nothing arrives on, then ORs `code`
// into *status (test of the bounded-wait mechanism; no copies, no tensor memory).
cudaError_t launch_wait_expiry_selftest(int* status, long long deadline_cycles, int code, cudaStream_t s);

// typhoon_mla_naive_shared_noalloc: looks up (once per device) the device address of the built-in scratch array
// for the current device.  Returns a TYPHOON_MLA_* status.
int noalloc_resolve_scratch_for_current_device();
// Bookkeeping shared by the entry points that live outside api.cu: records the CUDA error behind a
// TYPHOON_MLA_ERR_CUDA (returns that status) and the number of kernels the call launched, both per thread.
int api_cuda_fail(cudaError_t e);
void api_set_last_launches(int n);

// out[c][r] = in[r][c] for each of `batch` matrices [R][C] bf16.
cudaError_t launch_transpose_bf16(const void* in, void* out, int R, int C, int batch, cudaStream_t s);

// rows [L, W] with stride ld_in -> contiguous padded [Lp, W] (padding zero), bf16
cudaError_t launch_copy_pad_rows(const void* in, int64_t ld_in, void* out, int L, int Lp, int W, cudaStream_t s);

}  // namespace tmla
