/*
 * typhoon_mla.h -- C ABI of the B200 (sm_100a) MLA decode-attention library.
 *
 * The operation is the decode attention of Multi-Head Latent Attention when
 * many requests share a long prefix of the KV cache (Algorithm 1, "TyphoonMLA
 * Decode Attention Kernel"):
 *
 *   - the shared prefix is attended in the naive formulation over per-head
 *     keys/values that were expanded once from the shared latent cache
 *     (Section 3.1 "Prefill"; Algorithm 1 line 4);
 *   - each request's own suffix is attended in the absorb formulation: q_nope
 *     is moved through W_UK (= W_KVb1) into the latent space, attention runs
 *     over the paged latent cache plus the rope keys, and the latent output is
 *     projected through W_UV (= W_KVb2) (Algorithm 1 lines 5-7);
 *   - the two normalised partial results are merged by their log-sum-exps
 *     (Algorithm 1 line 8; Section 3.2 "CombineLSE");
 *   - below a batch threshold the whole context runs in absorb form
 *     (Section 3.1 "Fall-back to Absorb"; Eq. 1).
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless its comment says "host".
 *   - Tensors are bf16 (raw uint16 storage) unless stated; accumulation,
 *     softmax statistics, split partials and the combine are fp32.
 *   - q_pe and all cached rope keys arrive already rotated: no RoPE is applied.
 *   - softmax_scale multiplies the sum of the nope and the rope logits; it must be
 *     positive and finite.
 *   - Log-sum-exps are natural logarithms of sum(exp(scaled logit)).
 *   - A single decode query attends to every cached token (no mask).
 *   - Every call returns a status (0 = OK); nothing throws, aborts or traps.
 *     Work is enqueued on the given cudaStream_t (passed as void*) and the call
 *     returns without synchronising unless stated.
 *   - Inputs are never modified.  `out` rows 0..B-1 are fully overwritten.
 *   - There is no CPU fallback: without a CUDA device every compute entry
 *     point returns TYPHOON_MLA_ERR_CUDA.
 *
 * Supported dimensions: d_nope = 128, d_rope = 64, d_v = 128,
 * kv_lora_rank = 512, num_heads a multiple of 16 up to 128 (DeepSeek-v3: 128,
 * Kimi-K2: 64), page_size 64 or 128, base pointers 16-byte aligned.
 */
#ifndef TYPHOON_MLA_H_
#define TYPHOON_MLA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct typhoon_mla_shared typhoon_mla_shared_t; /* opaque host object */

typedef struct {
    int32_t num_heads;     /* H   */
    int32_t d_nope;        /* D_n */
    int32_t d_rope;        /* D_r */
    int32_t d_v;           /* D_v */
    int32_t kv_lora_rank;  /* D_l */
} typhoon_mla_dims_t;

enum {
    TYPHOON_MLA_OK = 0,
    TYPHOON_MLA_ERR_INVALID_ARG = 1,
    TYPHOON_MLA_ERR_UNSUPPORTED_DIMS = 2,
    TYPHOON_MLA_ERR_WORKSPACE_TOO_SMALL = 3,
    TYPHOON_MLA_ERR_ALLOC = 4,
    TYPHOON_MLA_ERR_CUDA = 5,
    TYPHOON_MLA_ERR_DEVICE_CHECK = 6,
    TYPHOON_MLA_ERR_STATIC_SCRATCH_EXCEEDED = 7 /* problem too large for the built-in scratch array */
};

enum {
    TYPHOON_MLA_MODE_AUTO = 0,   /* crossover rule decides (ABSORB or HYBRID; NAIVE if max_pages == 0) */
    TYPHOON_MLA_MODE_ABSORB = 1, /* whole context in absorb form (the fall-back) */
    TYPHOON_MLA_MODE_HYBRID = 2, /* Algorithm 1: naive over the prefix, absorb over the suffix */
    TYPHOON_MLA_MODE_NAIVE = 3   /* shared prefix only (Algorithm 1 line 4 + combine); suffixes ignored */
};

/* Kinds for typhoon_mla_cost_model (rows of Table 1). */
enum { TYPHOON_MLA_COST_NAIVE = 0, TYPHOON_MLA_COST_ABSORB = 1, TYPHOON_MLA_COST_TYPHOON = 2 };

/*
 * Expand the shared prefix (Section 3.1 "Prefill": the shared part of the
 * latent cache is passed through the up-projection to form per-head K and V).
 *
 *   ckv_shared  bf16 [Ls, 512], row stride ld_ckv elements (>= 512)
 *   kpe_shared  bf16 [Ls, 64],  row stride ld_kpe elements (>= 64)
 *   w_uk        bf16 [H, 128, 512] contiguous   (W_KVb1)
 *   w_uv        bf16 [H, 128, 512] contiguous   (W_KVb2)
 *
 * The handle OWNS (cudaMalloc) the expanded per-head keys K_nope, stored as
 * contiguous 64-token x 64-dim tiles [H, Ls'/64, 2, 64, 64],
 * the expanded values stored transposed in 64-token blocks V^T [H, Ls'/64, 128, 64]
 * (each block contiguous, so one KV tile is one contiguous 16 KB read), a copy of the shared
 * latent cache and rope keys, and a transposed copy of W_UK; Ls' is Ls rounded
 * up to a multiple of 128, the padding is zero.  It BORROWS w_uv: the caller
 * keeps w_uv alive and unchanged until typhoon_mla_free.  Ls may be 0.
 * The work is enqueued on `stream`; the handle may be used on that stream at
 * once, on other streams after the caller has ordered them behind it.
 * Errors: NULL arguments or bad strides -> INVALID_ARG; other dimensions ->
 * UNSUPPORTED_DIMS; cudaMalloc failure -> ALLOC (nothing is leaked).
 */
int typhoon_mla_prepare_shared(const typhoon_mla_dims_t* dims /* host */,
                               const void* ckv_shared, const void* kpe_shared,
                               int64_t Ls, int64_t ld_ckv, int64_t ld_kpe,
                               const void* w_uk, const void* w_uv,
                               void* stream, typhoon_mla_shared_t** out_handle /* host */);

/*
 * The same with the expanded K_nope and V stored in 8 bits (half the footprint and half the
 * bytes a step streams; the paper assumes 8-bit caches only in its memory-footprint
 * analysis, Section 4 "HBM Footprint", and does not fix an encoding; this is the library's):
 * OCP E4M3 codes (1-4-3 bits, bias 7, no infinities, largest value 448), round to
 * nearest even, saturating, of the 16-bit expanded cache divided by one power of two per
 * head and tensor (the smallest 2^e with amax / 2^e <= 448).  Rope keys, the copy of the
 * latent cache, the per-request caches and the queries stay 16-bit; the attention kernel
 * widens the codes exactly and computes as in the 16-bit path (half-precision operands,
 * fp32 accumulation), so the only error added is that of the encoding.  Queries must be
 * within half precision's range (|q| < 65504).  The handle is used like any other
 * (decode, decode_tree, decode_partial, the no-alloc call; AUTO / ABSORB / HYBRID /
 * NAIVE).  The option trades speed for memory: widening the codes inside the kernel
 * costs more than the halved traffic saves, and the shared-prefix kernel then works on
 * row groups of at most 128 requests (measured on B200: steps 1.15 to 1.6 times as long
 * as with the 16-bit cache).  A 16-bit scratch of the size of one expanded tensor is taken
 * from and returned to the stream's memory pool inside the call.
 * Arguments and errors as typhoon_mla_prepare_shared.
 */
int typhoon_mla_prepare_shared_fp8(const typhoon_mla_dims_t* dims /* host */,
                                   const void* ckv_shared, const void* kpe_shared,
                                   int64_t Ls, int64_t ld_ckv, int64_t ld_kpe,
                                   const void* w_uk, const void* w_uv,
                                   void* stream, typhoon_mla_shared_t** out_handle /* host */);

/* Release the handle and the device memory it owns (synchronises the device).
 * NULL is accepted. */
int typhoon_mla_free(typhoon_mla_shared_t* shared);

/* Bytes of scratch typhoon_mla_decode needs for this problem size in `mode`
 * (TYPHOON_MLA_MODE_AUTO: the worst case over the modes AUTO may resolve to, so the
 * same workspace serves every step whatever the crossover rule picks).  Host, pure:
 * it reads the handle and touches no process-wide state, so it may be called from
 * any thread at any time.  Returns 0 on invalid arguments. */
size_t typhoon_mla_workspace_bytes(const typhoon_mla_shared_t* shared, int32_t B,
                                   int32_t max_pages, int32_t page_size, int32_t mode);

/*
 * One decode-attention step for B requests (Algorithm 1).
 *
 *   q_nope       bf16 [B, H, 128] contiguous
 *   q_pe         bf16 [B, H, 64]  contiguous, RoPE already applied
 *   ckv_pages    bf16 latent cache, token (page p, slot s) at
 *                ckv_pages + (p * page_size + s) * ckv_token_stride, 512 wide
 *   kpe_pages    bf16 rope keys, same addressing with kpe_token_stride, 64 wide
 *                (strides in elements, multiples of 8; a fused 576-wide page
 *                layout can be passed by pointing both into it)
 *   num_pages    number of physical pages in ckv_pages / kpe_pages (>= 1 when
 *                max_pages > 0).  It bounds every read of the paged cache: a
 *                block-table entry inside a request's length that is negative
 *                or >= num_pages is never dereferenced -- its tokens read as
 *                zeros -- and sets bit TYPHOON_MLA_STATUS_BAD_PAGE of the
 *                handle's status word (typhoon_mla_check_status); the output
 *                rows of that request are then meaningless, the call does not
 *                fault.
 *   block_table  int32 [B, max_pages]: physical page of each logical page;
 *                entries at or beyond ceil(seq_lens[b] / page_size) are ignored
 *   seq_lens     int32 [B]: suffix length of each request, may be 0; values
 *                above max_pages * page_size are clamped to it
 *   out          bf16 [B, H, 128]
 *   lse_out      optional fp32 [B, H] (NULL to skip): ln sum exp over the whole
 *                context of each (request, head)
 *   workspace    at least typhoon_mla_workspace_bytes() bytes, 256-byte
 *                aligned; contents are scratch.  Calls that overlap in time
 *                need distinct workspaces.
 *
 * Token slots past a request's length and unused block-table entries are never
 * read into the result.  A request with no context at all (Ls = 0 and
 * seq_lens[b] = 0) gets a zero output row and lse = -inf.
 * The call never allocates and never synchronises.  It only enqueues kernels on
 * `stream` and, in HYBRID mode, on the handle's side stream (forked from and
 * joined back to `stream` with events inside the call), so it may be captured
 * into a CUDA graph; a replay reads the buffers' contents at replay time and
 * uses the pointers, sizes and mode given at capture time (AUTO is resolved at
 * capture).  Calls on the same handle from several host threads at once are not
 * supported (the side stream and its events belong to the handle).
 * Errors: INVALID_ARG (NULL/misaligned pointers, B < 1, bad mode or page size),
 * WORKSPACE_TOO_SMALL, CUDA (launch failure; see typhoon_mla_last_cuda_error).
 */
int typhoon_mla_decode(const typhoon_mla_shared_t* shared,
                       const void* q_nope, const void* q_pe, int32_t B,
                       const void* ckv_pages, const void* kpe_pages,
                       int64_t ckv_token_stride, int64_t kpe_token_stride,
                       int32_t page_size, int32_t num_pages,
                       const int32_t* block_table, int32_t max_pages,
                       const int32_t* seq_lens,
                       float softmax_scale, int32_t mode,
                       void* out, float* lse_out,
                       void* workspace, size_t workspace_bytes, void* stream);

/*
 * A context sharded over several devices (Section 3.1: the shared part "can be
 * parallelized across attention heads", the latent part across the sequence).
 *
 * Sequence sharding: every device holds a slice of the tokens (a slice of the
 * shared prefix prepared as its own handle, and the suffix pages of the
 * requests it owns; requests it does not own get seq_len 0) and calls
 * typhoon_mla_decode_partial, which is typhoon_mla_decode except that the
 * result over this device's tokens is returned un-rounded: out_partial fp32
 * [B, H, 128] (normalised over this device's tokens) and lse_partial fp32
 * [B, H] (natural log; -inf with a zero row where the device holds no token of
 * a request; required).  The partials of all devices are gathered (one
 * all-gather of B*H*129 floats per device) and merged by
 * typhoon_mla_combine_partials: the log-sum-exp combine of Algorithm 1 line 8
 * over n_parts partials, o_parts fp32 [n_parts, B, H, 128] and lse_parts fp32
 * [n_parts, B, H] (device, 16-byte aligned) -> out bf16 [B, H, 128] and the
 * optional lse_out fp32 [B, H].  Rows whose partials are all empty give zeros
 * and -inf.  Head sharding needs no call of its own: a device prepares and
 * decodes H / G heads (weights and queries sliced by head) and the bf16
 * outputs are gathered along the head axis.
 * Errors: as typhoon_mla_decode; INVALID_ARG for a null lse_partial or
 * n_parts < 1.  Both calls only enqueue work on `stream`.
 */
int typhoon_mla_decode_partial(const typhoon_mla_shared_t* shared,
                               const void* q_nope, const void* q_pe, int32_t B,
                               const void* ckv_pages, const void* kpe_pages,
                               int64_t ckv_token_stride, int64_t kpe_token_stride,
                               int32_t page_size, int32_t num_pages,
                               const int32_t* block_table, int32_t max_pages,
                               const int32_t* seq_lens,
                               float softmax_scale, int32_t mode,
                               float* out_partial, float* lse_partial,
                               void* workspace, size_t workspace_bytes, void* stream);
int typhoon_mla_combine_partials(const float* o_parts, const float* lse_parts, int32_t n_parts,
                                 int32_t B, int32_t H, void* out, float* lse_out, void* stream);

/* Bytes of device staging typhoon_mla_decode_host needs (host, pure). */
size_t typhoon_mla_host_staging_bytes(const typhoon_mla_shared_t* shared, int32_t B, int32_t max_pages);

/*
 * The same step with the per-step tensors in HOST memory (pinned memory makes
 * the copies asynchronous): q_nope, q_pe, block_table, seq_lens are copied to
 * `staging` (device), the step runs, and `out` (host, bf16 [B, H, 128]) is
 * copied back, all on `stream`.  The caches (ckv_pages, kpe_pages) stay device
 * pointers.  The call returns after enqueueing; synchronise the stream before
 * reading `out`.
 */
int typhoon_mla_decode_host(const typhoon_mla_shared_t* shared,
                            const void* q_nope_host, const void* q_pe_host, int32_t B,
                            const void* ckv_pages, const void* kpe_pages,
                            int64_t ckv_token_stride, int64_t kpe_token_stride,
                            int32_t page_size, int32_t num_pages,
                            const int32_t* block_table_host, int32_t max_pages,
                            const int32_t* seq_lens_host,
                            float softmax_scale, int32_t mode,
                            void* out_host,
                            void* staging, size_t staging_bytes,
                            void* workspace, size_t workspace_bytes, void* stream);

/*
 * Crossover rule (Section 3.1 "Fall-back to Absorb"; Eq. 1), host, pure.
 * Returns TYPHOON_MLA_MODE_ABSORB or _HYBRID (or _NAIVE when
 * total_suffix_tokens == 0 and Ls > 0) for a batch of B requests against this
 * prefix; total_suffix_tokens < 0 means unknown.  The rule compares modelled
 * times t_hybrid and t_absorb built from the Table 1 work terms, the hardware
 * model set by typhoon_mla_set_hw_model and a fixed per-launch cost; ties go
 * to ABSORB.
 */
int typhoon_mla_choose_mode(const typhoon_mla_shared_t* shared, int32_t B, int64_t total_suffix_tokens);

/* The same rule from the dimensions and the prefix length alone (no handle, no device). */
int typhoon_mla_choose_mode_for(const typhoon_mla_dims_t* dims /* host */, int64_t Ls, int32_t B,
                                int64_t total_suffix_tokens);

/* Hardware model of the crossover rule: sustained tensor throughput in FLOP/s,
 * HBM bandwidth in bytes/s, fixed cost of the extra hybrid launches in
 * seconds.  Non-positive values restore the defaults (B200 measured values).
 * Process-wide; not thread-safe against concurrent decode calls. */
int typhoon_mla_set_hw_model(double tensor_flops, double hbm_bytes_per_s, double hybrid_fixed_s);

/* Fraction of `tensor_flops` the absorb formulation reaches over the shared prefix in this
 * implementation (default 0.5, calibrated on B200; 1.0 gives the paper's zero-overhead rule of Eq. 1).
 * Values outside (0, 1] restore the default. */
int typhoon_mla_set_absorb_efficiency(double fraction);

/* Eq. 1: B_theta = (D_qk + D_v) / (S_q (2 D_l + D_r)) * T / M.  Host, pure. */
double typhoon_mla_batch_threshold(const typhoon_mla_dims_t* dims /* host */, int32_t S_q, double T, double M);

/* Table 1: MACs and HBM words of the attention part for one of the three
 * formulations (kind = TYPHOON_MLA_COST_*).  Host, pure.  L_n is the suffix
 * length of every request. */
int typhoon_mla_cost_model(const typhoon_mla_dims_t* dims /* host */, int32_t kind,
                           int64_t B, int64_t S_q, int64_t L_s, int64_t L_n,
                           int64_t* macs /* host */, int64_t* hbm_words /* host */);

/*
 * Several shared prefixes in one step (Section 3.1: tree-structured prompts, e.g. a system prompt
 * shared by all requests and one further prompt per group of requests).  A level partitions the
 * requests 0..B-1 into consecutive groups; group g = requests [group_begin[g], group_begin[g+1]) shares
 * prefixes[g] (NULL: that group has no prefix at this level).  A request attends to the prefix of its
 * group at every level and to its own suffix; all parts are merged by the LSE combine (Algorithm 1
 * line 8 with more partials).  Line 4 runs once per (level, group) over that group's query rows; lines
 * 5-7 run once for the whole batch.  All handles must have the same head count and were prepared with
 * the same weights (the first non-NULL handle's are used for the projections).  Both arrays are host
 * arrays; at most 8 levels and 256 non-empty (level, group) pairs.  tcgen05 kernel path only
 * (UNSUPPORTED_DIMS otherwise).  Other arguments, errors and the stream behaviour are those of
 * typhoon_mla_decode in HYBRID mode.  The paper describes this extension and does not evaluate it.
 */
typedef struct {
    const typhoon_mla_shared_t* const* prefixes; /* host array [n_groups] */
    const int32_t* group_begin;                  /* host array [n_groups + 1]: 0 = [0] <= ... <= [n_groups] = B */
    int32_t n_groups;
} typhoon_mla_prefix_level_t;

size_t typhoon_mla_tree_workspace_bytes(const typhoon_mla_prefix_level_t* levels /* host */, int32_t n_levels,
                                        int32_t B, int32_t max_pages, int32_t page_size);

int typhoon_mla_decode_tree(const typhoon_mla_prefix_level_t* levels /* host */, int32_t n_levels,
                            const void* q_nope, const void* q_pe, int32_t B,
                            const void* ckv_pages, const void* kpe_pages,
                            int64_t ckv_token_stride, int64_t kpe_token_stride,
                            int32_t page_size, int32_t num_pages,
                            const int32_t* block_table, int32_t max_pages,
                            const int32_t* seq_lens, float softmax_scale,
                            void* out, float* lse_out,
                            void* workspace, size_t workspace_bytes, void* stream);

/* Several query tokens per request (S_q of Table 1, e.g. the verification step of speculative
 * decoding): the cache already holds the S_q new tokens of every request and query token j
 * (0 <= j < S_q) attends to the shared prefix and to the first seq_lens[b] - (S_q - 1 - j) suffix
 * tokens (causal among the new tokens).  The path treats every (request, query token) pair as a row:
 * this call writes the page table block_table_rows int32 [B * S_q, max_pages] and the lengths
 * seq_lens_rows int32 [B * S_q] of the rows (row = b * S_q + j; negative lengths become 0), which
 * typhoon_mla_decode then takes with B * S_q in place of B and q arrays of B * S_q rows.  All pointers
 * are device pointers; asynchronous on `stream`; no allocation.  The paper states the cost model for
 * S_q (Table 1, Eq. 1) and evaluates S_q = 1 only. */
int typhoon_mla_expand_query_rows(const int32_t* block_table, const int32_t* seq_lens, int32_t B,
                                  int32_t max_pages, int32_t S_q, int32_t* block_table_rows,
                                  int32_t* seq_lens_rows, void* stream);

/*
 * Device-side checks.  The handle owns one status word in device memory, zero after
 * typhoon_mla_prepare_shared.  Kernels never trap or assert; instead they OR a bit into the word:
 *   TYPHOON_MLA_STATUS_WAIT_EXPIRED  a bounded in-kernel wait ran out (every wait on a copy or a tensor-core
 *                                    completion has a deadline of about one second); the kernel abandoned its
 *                                    work and the results of that launch are invalid
 *   TYPHOON_MLA_STATUS_BAD_PAGE      a block-table entry inside a request's length was negative or >= num_pages;
 *                                    it was not dereferenced (its tokens read as zeros)
 * typhoon_mla_check_status synchronises `stream`, copies the word to *word (host, may be NULL), clears it on the
 * device when `clear` is non-zero, and returns TYPHOON_MLA_ERR_DEVICE_CHECK if it was non-zero, else OK.  This is
 * the library's stand-in for a memory checker on systems where none can be run; it is off the hot path (a decode
 * call never reads the word back).  Bits 0-7 of the word name the kernel whose wait expired (diagnostic only).
 */
enum { TYPHOON_MLA_STATUS_WAIT_EXPIRED = 0xff, TYPHOON_MLA_STATUS_BAD_PAGE = 0x100 };
int typhoon_mla_check_status(const typhoon_mla_shared_t* shared, void* stream, int32_t* word /* host */, int32_t clear);

/*
 * Shared-prefix attention without any allocation (the paper has no counterpart:
 * this is a packaging variant of Algorithm 1 line 4 followed by the combine,
 * i.e. what TYPHOON_MLA_MODE_NAIVE computes, for requests with no suffix).
 *
 * For callers that cannot obtain device memory at call time -- a server whose
 * cache pool already owns all free HBM, so that cudaMalloc fails; a real-time
 * loop where cudaMalloc/cudaFree are forbidden because they synchronise the
 * device -- and therefore cannot pass a workspace.  The KV-split partials live
 * in a fixed array of TYPHOON_MLA_NOALLOC_SCRATCH_BYTES inside the library
 * image.  CUDA loads the part of the image that holds the array when its
 * address is first looked up on a device, and it is that load which takes the
 * 32 MiB of device memory: typhoon_mla_prepare_shared does the lookup (with
 * its device current, checking the result), so the memory is taken while the
 * caller is still setting up and allocation is still possible, and this entry
 * point only reads a cached device pointer.  From then on every GPU on which
 * a prefix was prepared holds the array until the process exits.
 *
 *   q_nope bf16 [B, H, 128], q_pe bf16 [B, H, 64], out bf16 [B, H, 128],
 *   lse_out optional fp32 [B, H]; all device pointers, 16-byte aligned.
 *
 * Limit: B * H * 516 bytes (rounded up to 256) must fit in the array, i.e.
 * B * H <= 65024 (B <= 508 at H = 128); larger problems are rejected with
 * TYPHOON_MLA_ERR_STATIC_SCRATCH_EXCEEDED, a bad scale or a handle of another
 * device with INVALID_ARG; a rejected call launches nothing and writes nothing.
 * The call uses no cudaMalloc/cudaFree and no allocating library routine, and
 * runs the same shared-prefix kernel as typhoon_mla_decode (with fewer partial
 * slots when the library's own choice would not fit the array).  Because the
 * address lookup happens in typhoon_mla_prepare_shared, prepare the prefix
 * before any stream capture begins.  All calls on a device share the one
 * array, which keeps the previous call's contents; every slot a call reads it
 * has written itself, so no clearing is needed, but two calls whose kernels
 * overlap on the GPU (different streams) race on it: serialise them.
 */
#define TYPHOON_MLA_NOALLOC_SCRATCH_BYTES (32u << 20)
int typhoon_mla_naive_shared_noalloc(const typhoon_mla_shared_t* shared,
                                     const void* q_nope, const void* q_pe, int32_t B,
                                     float softmax_scale, void* out, float* lse_out, void* stream);

/* The cudaError_t (as int) behind the last TYPHOON_MLA_ERR_CUDA of this thread. */
int typhoon_mla_last_cuda_error(void);

const char* typhoon_mla_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* TYPHOON_MLA_H_ */
