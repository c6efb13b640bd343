// C ABI of the library: argument validation, the prepared-prefix handle, the
// workspace plan, the crossover rule (Eq. 1 / Table 1) and the launch sequence
// of one decode step (Algorithm 1).
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <new>

#include "../../include/typhoon_mla.h"
#include "../../include/typhoon_mla_internal.h"
#include "kernels.h"

using namespace tmla;

#include "handle.h"

thread_local bool tmla::tl_pdl = true;

namespace {

thread_local int g_last_launches = 0;
thread_local int g_last_cuda_error = 0;

// Optional CUDA-event timing of one kernel kind inside decode calls.
struct Profile {
    int kernel_id = -1;
    int capacity = 0, used = 0;
    cudaEvent_t* ev = nullptr;  // 2 per recorded launch
};
Profile g_prof;

inline void prof_before(int id, cudaStream_t s) {
    if (id == g_prof.kernel_id && g_prof.used < g_prof.capacity) cudaEventRecord(g_prof.ev[2 * g_prof.used], s);
}
inline void prof_after(int id, cudaStream_t s) {
    if (id == g_prof.kernel_id && g_prof.used < g_prof.capacity) {
        cudaEventRecord(g_prof.ev[2 * g_prof.used + 1], s);
        ++g_prof.used;
    }
}

// Process-wide switches (test and measurement hooks) and the hardware model of the crossover rule.  They
// are atomics; an API call takes one snapshot at its start and plans and launches from that snapshot only.
std::atomic<int> g_kernel_path{TYPHOON_MLA_PATH_TCGEN05};
std::atomic<bool> g_overlap{true};          // absorb branch of a hybrid step on the handle's side stream
std::atomic<bool> g_pdl{true};              // programmatic dependent launch of the step's kernels
std::atomic<int> g_naive_schedule{0};
std::atomic<bool> g_stacked_absorb{true};   // absorb-only steps: batch-stacked kernel over the shared prefix
constexpr double kDefTensor = 1.0e15, kDefHbm = 6.0e12, kDefFixed = 6.0e-6, kDefAbsorbEff = 0.5;
std::atomic<double> g_tensor_flops{kDefTensor};        // sustained rate the attention kernels reach, FLOP/s
std::atomic<double> g_hbm_bytes{kDefHbm};              // bytes/s
std::atomic<double> g_hybrid_fixed_s{kDefFixed};       // extra launches + combine of the hybrid path
std::atomic<double> g_absorb_efficiency{kDefAbsorbEff};   // absorb kernel's share of g_tensor_flops (calibrated on B200)

struct Settings {
    int kernel_path, naive_schedule;
    bool overlap, pdl, stacked_absorb;
    bool tc() const { return kernel_path == TYPHOON_MLA_PATH_TCGEN05; }
};
Settings snapshot() {
    return Settings{g_kernel_path.load(), g_naive_schedule.load(), g_overlap.load(), g_pdl.load(), g_stacked_absorb.load()};
}

inline int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool dims_supported(const typhoon_mla_dims_t& d) {
    return d.d_nope == 128 && d.d_rope == 64 && d.d_v == 128 && d.kv_lora_rank == 512 && d.num_heads >= 16 &&
           d.num_heads <= 128 && d.num_heads % 16 == 0;
}

int cuda_fail(cudaError_t e) {
    g_last_cuda_error = (int)e;
    return TYPHOON_MLA_ERR_CUDA;
}
}  // namespace
int tmla::api_cuda_fail(cudaError_t e) { return cuda_fail(e); }
void tmla::api_set_last_launches(int n) { g_last_launches = n; }
namespace {

// ---- workspace plan --------------------------------------------------------
struct Plan {
    int mode;
    int n_split_naive;       // KV splits of the warp-MMA naive kernel / tile ranges of the tcgen05 one
    int n_slots_naive;       // partial slots the naive kernel writes (>= n_split_naive)
    int chunk;               // tokens per absorb chunk
    int n_shared_chunks;     // absorb chunks over the shared prefix (ABSORB mode)
    int n_suffix_chunks;
    // byte offsets into the workspace
    size_t off_order, off_desc, off_qabs, off_opart_a, off_lsepart_a, off_olat, off_lse_a, off_oabs, off_opart_n, off_lsepart_n, total;
};

constexpr int kDefaultNumSM = 148;        // a B200; used where no device is at hand (pure planning queries)
constexpr int kMaxAbsorbChunks = 1024;   // chunks per request the merge kernel accepts

int naive_splits(int B, int H, int64_t Ls, int n_sm) {
    if (Ls <= 0) return 0;
    int n_tiles = (int)((Ls + 63) / 64);
    int base = ((B + 63) / 64) * H;
    int want = (4 * n_sm + base - 1) / base;
    return std::max(1, std::min({want, n_tiles, 64}));
}

void absorb_chunks(bool tc, bool stacked, int n_sm, int B, int H, int64_t Ls_absorb, int64_t cap_suffix, int* chunk, int* n_sh,
                   int* n_sf) {
    const int units = B * ((H + 63) / 64);
    // CTAs per shared-prefix chunk: 64-row groups of the stacked [B * H] query matrix, or of each request
    const int units_sh = (tc && stacked) ? (int)(((int64_t)B * H + 63) / 64) : units;
    const int64_t longest = std::max<int64_t>(std::max(Ls_absorb, cap_suffix), 1);
    int64_t c;
    if (tc) {
        // One CTA per SM: minimise waves x (tiles per chunk + fixed cost in tile units) over the number of
        // chunks the longest segment is cut into.
        const double fixed = 3.0;
        double best_cost = 1e30;
        c = round_up(longest, 64);
        for (int parts = 1; parts <= 512; ++parts) {
            const int64_t ch = round_up((longest + parts - 1) / parts, 64);
            const int64_t per_req = (Ls_absorb + ch - 1) / ch + (cap_suffix + ch - 1) / ch;
            const int64_t ctas = (int64_t)units_sh * ((Ls_absorb + ch - 1) / ch) + (int64_t)units * ((cap_suffix + ch - 1) / ch);
            if (per_req > kMaxAbsorbChunks) continue;   // limit of the merge kernel
            const int64_t waves = (ctas + n_sm - 1) / n_sm;
            // a split segment writes and re-reads fp32 partials (64 heads x 2 KB, both ways): about 3.5 tiles
            // worth of traffic per chunk
            const double split_cost = (per_req > 1) ? 3.5 : 0.0;
            const double cost = (double)waves * ((double)ch / 64.0 + fixed + split_cost);
            if (cost < best_cost - 1e-9) {
                best_cost = cost;
                c = ch;
            }
            if (ch <= 64) break;
        }
    } else {
        const int target = std::max(1, (2 * n_sm + units - 1) / units);
        c = std::max<int64_t>(round_up((longest + target - 1) / target, 64), 256);
        while ((Ls_absorb + c - 1) / c + (cap_suffix + c - 1) / c > kMaxAbsorbChunks) c *= 2;
    }
    *chunk = (int)c;
    *n_sh = (int)((Ls_absorb + c - 1) / c);
    *n_sf = (int)((cap_suffix + c - 1) / c);
}

// `mode` is resolved (ABSORB, HYBRID or NAIVE); `tc` and `schedule` come from the caller's settings snapshot.
Plan make_plan(const typhoon_mla_shared* sh, bool tc, int schedule, int B, int max_pages, int page_size, int mode,
               int naive_slots_override = -1, bool stacked = true) {
    Plan p{};
    const int H = sh->dims.num_heads;
    const int n_sm = sh->num_sms > 0 ? sh->num_sms : kDefaultNumSM;
    p.mode = mode;
    const int64_t cap = (int64_t)max_pages * page_size;
    const bool use_naive = (mode != TYPHOON_MLA_MODE_ABSORB) && sh->Ls > 0;
    const bool use_absorb = (mode != TYPHOON_MLA_MODE_NAIVE);
    if (naive_slots_override >= 0) {   // several shared-prefix launches planned by the caller
        p.n_split_naive = naive_slots_override > 0 ? 1 : 0;
        p.n_slots_naive = naive_slots_override;
    } else if (use_naive && tc) {
        naive_sm100_plan(B, H, sh->Ls, n_sm, schedule, &p.n_split_naive, &p.n_slots_naive, sh->fp8 != 0);   // n_split_naive = tile ranges
    } else {
        p.n_split_naive = use_naive ? naive_splits(B, H, sh->Ls, n_sm) : 0;
        p.n_slots_naive = p.n_split_naive;
    }
    if (use_absorb) {
        absorb_chunks(tc, stacked, n_sm, B, H, mode == TYPHOON_MLA_MODE_ABSORB ? sh->Ls : 0, cap, &p.chunk, &p.n_shared_chunks,
                      &p.n_suffix_chunks);
    }
    const int n_chunks = p.n_shared_chunks + p.n_suffix_chunks;
    const size_t BH = (size_t)B * H;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t o = off;
        off += round_up((int64_t)bytes, 256);
        return o;
    };
    p.off_order = take((size_t)B * 4);
    p.off_desc = take((size_t)B * 16);
    p.off_qabs = take(BH * 512 * 2);
    p.off_opart_a = take((size_t)n_chunks * BH * 512 * 4);
    p.off_lsepart_a = take((size_t)n_chunks * BH * 4);
    p.off_olat = take(BH * 512 * 2);
    p.off_lse_a = take(BH * 4);
    p.off_oabs = take(BH * 128 * 4);
    p.off_opart_n = take((size_t)p.n_slots_naive * BH * 128 * 4);
    p.off_lsepart_n = take((size_t)p.n_slots_naive * BH * 4);
    p.total = off;
    return p;
}

// The handle's buffers, stream and events live on the device it was prepared on.
bool on_handle_device(const typhoon_mla_shared* sh) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == sh->device;
}

int resolve_mode(const typhoon_mla_shared* sh, int B, int max_pages, int mode) {
    if (mode == TYPHOON_MLA_MODE_AUTO) {
        if (max_pages == 0 && sh->Ls > 0) return TYPHOON_MLA_MODE_NAIVE;
        return typhoon_mla_choose_mode(sh, B, -1);
    }
    if (mode == TYPHOON_MLA_MODE_HYBRID && sh->Ls == 0) return TYPHOON_MLA_MODE_ABSORB;
    return mode;
}

}  // namespace

extern "C" {

const char* typhoon_mla_status_string(int status) {
    switch (status) {
        case TYPHOON_MLA_OK: return "ok";
        case TYPHOON_MLA_ERR_INVALID_ARG: return "invalid argument";
        case TYPHOON_MLA_ERR_UNSUPPORTED_DIMS: return "unsupported dimensions";
        case TYPHOON_MLA_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case TYPHOON_MLA_ERR_ALLOC: return "device allocation failed";
        case TYPHOON_MLA_ERR_CUDA: return "CUDA error";
        case TYPHOON_MLA_ERR_DEVICE_CHECK: return "device-side check failed";
        case TYPHOON_MLA_ERR_STATIC_SCRATCH_EXCEEDED: return "problem exceeds the built-in scratch array";
        default: return "unknown status";
    }
}

int typhoon_mla_last_launch_count(void) { return g_last_launches; }
int typhoon_mla_last_cuda_error(void) { return g_last_cuda_error; }

double typhoon_mla_batch_threshold(const typhoon_mla_dims_t* d, int32_t S_q, double T, double M) {
    if (!d || S_q < 1 || !(M > 0.0)) return -1.0;
    const double d_qk = (double)d->d_nope + d->d_rope;
    return (d_qk + d->d_v) / ((double)S_q * (2.0 * d->kv_lora_rank + d->d_rope)) * (T / M);
}

int typhoon_mla_naive_plan(int32_t num_heads, int32_t B, int64_t L_s, int32_t schedule, int32_t num_sms,
                           int32_t* tile_tokens, int32_t* n_ranges, int32_t* row_groups, int32_t* n_slots) {
    if (B < 1 || L_s < 1 || L_s > (int64_t)1 << 30 || schedule < 0 || schedule > 2 || num_sms < 0) return TYPHOON_MLA_ERR_INVALID_ARG;
    if (num_heads < 16 || num_heads > 128 || num_heads % 16) return TYPHOON_MLA_ERR_INVALID_ARG;
    if (!tile_tokens || !n_ranges || !row_groups || !n_slots) return TYPHOON_MLA_ERR_INVALID_ARG;
    int r = 0, sl = 0;
    naive_sm100_plan(B, num_heads, L_s, num_sms > 0 ? num_sms : kDefaultNumSM, schedule, &r, &sl);
    *tile_tokens = naive_sm100_tile_tokens(B);
    *n_ranges = r;
    *row_groups = B <= 128 ? 1 : (B + 255) / 256;
    *n_slots = sl;
    return TYPHOON_MLA_OK;
}

int typhoon_mla_cost_model(const typhoon_mla_dims_t* d, int32_t kind, int64_t B, int64_t S_q, int64_t L_s,
                           int64_t L_n, int64_t* macs, int64_t* hbm_words) {
    if (!d || B < 0 || S_q < 1 || L_s < 0 || L_n < 0) return TYPHOON_MLA_ERR_INVALID_ARG;
    const int64_t H = d->num_heads;
    const int64_t w_naive = H * ((int64_t)d->d_nope + d->d_rope + d->d_v);      // per (query, token) / per token
    const int64_t w_abs_mac = H * (2 * (int64_t)d->kv_lora_rank + d->d_rope);
    const int64_t w_abs_mem = (int64_t)d->kv_lora_rank + d->d_rope;
    int64_t m, w;
    switch (kind) {
        case TYPHOON_MLA_COST_NAIVE:
            m = B * S_q * (L_s + L_n) * w_naive;
            w = (L_s + B * L_n) * w_naive;
            break;
        case TYPHOON_MLA_COST_ABSORB:
            m = B * S_q * (L_s + L_n) * w_abs_mac;
            w = (L_s + B * L_n) * w_abs_mem;
            break;
        case TYPHOON_MLA_COST_TYPHOON:
            m = B * S_q * (L_s * w_naive + L_n * w_abs_mac);
            w = L_s * w_naive + B * L_n * w_abs_mem;
            break;
        default: return TYPHOON_MLA_ERR_INVALID_ARG;
    }
    if (macs) *macs = m;
    if (hbm_words) *hbm_words = w;
    return TYPHOON_MLA_OK;
}

int typhoon_mla_set_hw_model(double tensor_flops, double hbm_bytes_per_s, double hybrid_fixed_s) {
    g_tensor_flops.store(tensor_flops > 0 ? tensor_flops : kDefTensor);
    g_hbm_bytes.store(hbm_bytes_per_s > 0 ? hbm_bytes_per_s : kDefHbm);
    g_hybrid_fixed_s.store(hybrid_fixed_s >= 0 ? hybrid_fixed_s : kDefFixed);
    return TYPHOON_MLA_OK;
}

int typhoon_mla_set_absorb_efficiency(double fraction) {
    g_absorb_efficiency.store((fraction > 0.0 && fraction <= 1.0) ? fraction : kDefAbsorbEff);
    return TYPHOON_MLA_OK;
}

// `naive_time_factor`: how much longer the shared-prefix kernel takes than the model says (1 for the 16-bit cache; the
// 8-bit cache's kernel is bound by its widening step: measured 1.4-1.7 times the 16-bit kernel's time)
static int choose_mode_impl(const typhoon_mla_dims_t* dims, int64_t Ls, int32_t B, int64_t total_suffix_tokens,
                            double naive_time_factor) {
    if (!dims || B < 1 || Ls <= 0) return TYPHOON_MLA_MODE_ABSORB;
    if (total_suffix_tokens == 0) return TYPHOON_MLA_MODE_NAIVE;
    // Shared-prefix part only: the suffix part is identical in both modes.
    // Work terms are Table 1's, with the rope keys of the expanded cache read
    // once per token instead of once per head.
    const typhoon_mla_dims_t& d = *dims;
    const double H = d.num_heads, L = (double)Ls;
    const double f_naive = 2.0 * B * H * L * (d.d_nope + d.d_rope + d.d_v);
    // (the absorb kernel works on groups of 64 rows of the stacked [B * H] query matrix: a partial group costs as
    // much as a full one)
    const double rows_abs = std::ceil(B * H / 64.0) * 64.0;
    const double f_absorb = 2.0 * rows_abs * L * (2.0 * d.kv_lora_rank + d.d_rope);
    const double by_naive = 2.0 * L * (H * (d.d_nope + d.d_v) + d.d_rope);
    const double by_absorb = 2.0 * L * (d.kv_lora_rank + d.d_rope);
    // The absorb kernel re-reads the prefix per request and runs M = 64 tiles: measured on B200 it
    // reaches about half of the tensor throughput the naive kernel does, hence the factor.
    const double T = g_tensor_flops.load(), M = g_hbm_bytes.load();
    const double t_hybrid = naive_time_factor * std::max(f_naive / T, by_naive / M) + g_hybrid_fixed_s.load();
    const double t_absorb = std::max(f_absorb / (g_absorb_efficiency.load() * T), by_absorb / M);
    return t_hybrid < t_absorb ? TYPHOON_MLA_MODE_HYBRID : TYPHOON_MLA_MODE_ABSORB;
}

int typhoon_mla_choose_mode_for(const typhoon_mla_dims_t* dims, int64_t Ls, int32_t B, int64_t total_suffix_tokens) {
    return choose_mode_impl(dims, Ls, B, total_suffix_tokens, 1.0);
}

int typhoon_mla_choose_mode(const typhoon_mla_shared_t* sh, int32_t B, int64_t total_suffix_tokens) {
    if (!sh) return TYPHOON_MLA_MODE_ABSORB;
    return choose_mode_impl(&sh->dims, sh->Ls, B, total_suffix_tokens, sh->fp8 ? 1.5 : 1.0);
}

int typhoon_mla_free(typhoon_mla_shared_t* sh) {
    if (!sh) return TYPHOON_MLA_OK;
    // the handle's buffers, stream and events belong to the device it was prepared on, whatever device is current now
    int cur = -1;
    const bool switched = cudaGetDevice(&cur) == cudaSuccess && cur != sh->device && cudaSetDevice(sh->device) == cudaSuccess;
    cudaDeviceSynchronize();
    cudaFree(sh->k_nope);
    cudaFree(sh->v_t);
    cudaFree(sh->ckv);
    cudaFree(sh->kpe);
    cudaFree(sh->w_uk_t);
    cudaFree(sh->status);
    cudaFree(sh->k8);
    cudaFree(sh->v8);
    cudaFree(sh->fp8_f);
    if (sh->side_stream) cudaStreamDestroy(sh->side_stream);
    if (sh->ev_fork) cudaEventDestroy(sh->ev_fork);
    if (sh->ev_join) cudaEventDestroy(sh->ev_join);
    if (switched) cudaSetDevice(cur);
    cudaGetLastError();   // a failure while releasing must not surface in the caller's next launch
    delete sh;
    return TYPHOON_MLA_OK;
}

static int prepare_impl(const typhoon_mla_dims_t* dims, const void* ckv_shared, const void* kpe_shared,
                        int64_t Ls, int64_t ld_ckv, int64_t ld_kpe, const void* w_uk, const void* w_uv,
                        void* stream, typhoon_mla_shared_t** out_handle, bool fp8) {
    if (!dims || !out_handle || !w_uk || !w_uv || Ls < 0) return TYPHOON_MLA_ERR_INVALID_ARG;
    *out_handle = nullptr;
    if (!dims_supported(*dims)) return TYPHOON_MLA_ERR_UNSUPPORTED_DIMS;
    if (Ls > 0 && (!ckv_shared || !kpe_shared || ld_ckv < 512 || ld_kpe < 64 || ld_ckv % 8 || ld_kpe % 8 ||
                   !aligned16(ckv_shared) || !aligned16(kpe_shared)))
        return TYPHOON_MLA_ERR_INVALID_ARG;
    if (!aligned16(w_uk) || !aligned16(w_uv) || Ls > (int64_t)1 << 24) return TYPHOON_MLA_ERR_INVALID_ARG;
    int dev = 0, n_sm = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    // opt-in shared-memory sizes of every kernel, once per device and off the decode path
    if (e == cudaSuccess) e = set_attrs_naive_sm100();
    if (e == cudaSuccess) e = set_attrs_absorb_sm100();
    if (e == cudaSuccess) e = set_attrs_gemm_sm100();
    if (e == cudaSuccess) e = set_attrs_q_absorb_sm100();
    if (e == cudaSuccess) e = set_attrs_attn_mma();
    if (e == cudaSuccess) e = set_attrs_gemm_tn();
    if (e != cudaSuccess) return cuda_fail(e);
    // The allocation-free entry point keeps its scratch in a device array of the library image.  The module
    // that holds it is loaded lazily, and loading it takes device memory: do it here, where allocating is
    // allowed, so that the entry point itself never has to.
    {
        const int st = noalloc_resolve_scratch_for_current_device();
        if (st != TYPHOON_MLA_OK) return st;
    }
    const Settings cfg = snapshot();
    tmla::tl_pdl = cfg.pdl;

    typhoon_mla_shared* sh = new (std::nothrow) typhoon_mla_shared();
    if (!sh) return TYPHOON_MLA_ERR_ALLOC;
    std::memset(sh, 0, sizeof(*sh));
    sh->dims = *dims;
    sh->Ls = Ls;
    sh->Ls_pad = round_up(Ls, 128);
    sh->w_uv = w_uv;
    sh->device = dev;
    sh->num_sms = n_sm;
    const int H = dims->num_heads;
    const size_t Lp = (size_t)sh->Ls_pad;
    const size_t b_k = (size_t)H * Lp * 128 * 2, b_ckv = Lp * 512 * 2, b_kpe = Lp * 64 * 2,
                 b_w = (size_t)H * 512 * 128 * 2;
    auto alloc = [&](void** p, size_t bytes) {
        if (bytes == 0) { *p = nullptr; return true; }
        if (cudaMalloc(p, bytes) != cudaSuccess) { cudaGetLastError(); *p = nullptr; return false; }
        sh->owned_bytes += bytes;
        return true;
    };
    sh->fp8 = (fp8 && Ls > 0) ? 1 : 0;
    bool ok_alloc = alloc(&sh->ckv, b_ckv) && alloc(&sh->kpe, b_kpe) && alloc(&sh->w_uk_t, b_w) &&
                    alloc(reinterpret_cast<void**>(&sh->status), 256);
    if (ok_alloc && !sh->fp8) ok_alloc = alloc(&sh->k_nope, b_k) && alloc(&sh->v_t, b_k);
    if (ok_alloc && sh->fp8)
        ok_alloc = alloc(&sh->k8, b_k / 2) && alloc(&sh->v8, b_k / 2) &&
                   alloc(reinterpret_cast<void**>(&sh->fp8_f), (size_t)H * 3 * sizeof(float));
    if (!ok_alloc) {
        typhoon_mla_free(sh);
        return TYPHOON_MLA_ERR_ALLOC;
    }
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    // 8-bit cache: each tensor is expanded into a 16-bit scratch of the stream's memory pool, encoded from there,
    // and the scratch is handed back in stream order (no synchronisation)
    void* scratch16 = nullptr;
    if (sh->fp8 && cudaMallocAsync(&scratch16, b_k, s) != cudaSuccess) {
        cudaGetLastError();
        typhoon_mla_free(sh);
        return TYPHOON_MLA_ERR_ALLOC;
    }
    void* const k_dst = sh->fp8 ? scratch16 : sh->k_nope;
    void* const v_dst = sh->fp8 ? scratch16 : sh->v_t;
    const bool tc = cfg.tc();
    {
        int lo = 0, hi = 0;
        cudaDeviceGetStreamPriorityRange(&lo, &hi);   // hi is the numerically lowest = highest priority
        e = cudaStreamCreateWithPriority(&sh->side_stream, cudaStreamNonBlocking, hi);
    }
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&sh->ev_fork, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&sh->ev_join, cudaEventDisableTiming);
    if (e != cudaSuccess) {
        if (scratch16) cudaFreeAsync(scratch16, s);
        typhoon_mla_free(sh);
        return cuda_fail(e);
    }
    e = cudaMemsetAsync(sh->status, 0, 256, s);
    if (e == cudaSuccess) e = launch_transpose_bf16(w_uk, sh->w_uk_t, 128, 512, H, s);
    if (e == cudaSuccess && Ls > 0) {
        e = launch_copy_pad_rows(ckv_shared, ld_ckv, sh->ckv, (int)Ls, (int)Lp, 512, s);
        if (e == cudaSuccess) e = launch_copy_pad_rows(kpe_shared, ld_kpe, sh->kpe, (int)Ls, (int)Lp, 64, s);
        if (e == cudaSuccess) {  // K_nope[h] = ckv * W_UK[h]^T
            GemmTN g{sh->ckv, 512, 0, w_uk, 512, 128 * 512, k_dst, 128, (int64_t)Lp * 128,
                     (int)Lp, 128, 512, H, false, 0, true};
            e = tc ? launch_gemm_tn_sm100(g, sh->status, s) : launch_gemm_tn(g, s);
            if (e == cudaSuccess && sh->fp8)
                e = launch_quantize_e4m3(k_dst, false, H, (int64_t)Lp, sh->k8, reinterpret_cast<uint32_t*>(sh->fp8_f + 2 * H),
                                         sh->fp8_f, s);
        }
        if (e == cudaSuccess) {  // V^T[h] = W_UV[h] * ckv^T
            GemmTN g{w_uv, 512, 128 * 512, sh->ckv, 512, 0, v_dst, (int64_t)Lp, (int64_t)(128 * Lp),
                     128, (int)Lp, 512, H, false, 64};
            e = tc ? launch_gemm_tn_sm100(g, sh->status, s) : launch_gemm_tn(g, s);
            if (e == cudaSuccess && sh->fp8)
                e = launch_quantize_e4m3(v_dst, true, H, (int64_t)Lp, sh->v8, reinterpret_cast<uint32_t*>(sh->fp8_f + 2 * H),
                                         sh->fp8_f + H, s);
        }
    }
    if (scratch16) {
        const cudaError_t ef = cudaFreeAsync(scratch16, s);
        if (e == cudaSuccess) e = ef;
    }
    if (e == cudaSuccess && Ls > 0)
        e = sh->fp8 ? make_naive_fp8_tmaps(sh->k8, sh->kpe, sh->v8, H, sh->Ls_pad, &sh->tm_kn, &sh->tm_kp, &sh->tm_vt)
                    : make_naive_sm100_tmaps(sh->k_nope, sh->kpe, sh->v_t, H, sh->Ls_pad, &sh->tm_kn, &sh->tm_kp, &sh->tm_vt);
    if (e == cudaSuccess) e = make_q_absorb_tmap(sh->w_uk_t, H, &sh->tm_wuk_t);
    if (e == cudaSuccess && Ls > 0) e = make_absorb_shared_tmaps(sh->ckv, sh->kpe, sh->Ls_pad, &sh->tm_ckv, &sh->tm_kpe_tok);
    if (e != cudaSuccess) {
        typhoon_mla_free(sh);
        return cuda_fail(e);
    }
    *out_handle = sh;
    return TYPHOON_MLA_OK;
}

int typhoon_mla_prepare_shared(const typhoon_mla_dims_t* dims, const void* ckv_shared, const void* kpe_shared,
                               int64_t Ls, int64_t ld_ckv, int64_t ld_kpe, const void* w_uk, const void* w_uv,
                               void* stream, typhoon_mla_shared_t** out_handle) {
    return prepare_impl(dims, ckv_shared, kpe_shared, Ls, ld_ckv, ld_kpe, w_uk, w_uv, stream, out_handle, false);
}

int typhoon_mla_prepare_shared_fp8(const typhoon_mla_dims_t* dims, const void* ckv_shared, const void* kpe_shared,
                                   int64_t Ls, int64_t ld_ckv, int64_t ld_kpe, const void* w_uk, const void* w_uv,
                                   void* stream, typhoon_mla_shared_t** out_handle) {
    return prepare_impl(dims, ckv_shared, kpe_shared, Ls, ld_ckv, ld_kpe, w_uk, w_uv, stream, out_handle, true);
}

int typhoon_mla_shared_view(const typhoon_mla_shared_t* sh, const void** k_nope, const void** v_t, int64_t* Ls,
                            int64_t* Ls_padded, int64_t* owned_bytes) {
    if (!sh) return TYPHOON_MLA_ERR_INVALID_ARG;
    if (k_nope) *k_nope = sh->k_nope;
    if (v_t) *v_t = sh->v_t;
    if (Ls) *Ls = sh->Ls;
    if (Ls_padded) *Ls_padded = sh->Ls_pad;
    if (owned_bytes) *owned_bytes = (int64_t)sh->owned_bytes;
    return TYPHOON_MLA_OK;
}

int typhoon_mla_expand_query_rows(const int32_t* block_table, const int32_t* seq_lens, int32_t B, int32_t max_pages,
                                  int32_t S_q, int32_t* block_table_rows, int32_t* seq_lens_rows, void* stream) {
    if (!seq_lens || !seq_lens_rows || B < 1 || S_q < 1 || max_pages < 0) return TYPHOON_MLA_ERR_INVALID_ARG;
    if (max_pages > 0 && (!block_table || !block_table_rows)) return TYPHOON_MLA_ERR_INVALID_ARG;
    if ((int64_t)B * S_q > INT32_MAX) return TYPHOON_MLA_ERR_INVALID_ARG;
    cudaError_t e = launch_expand_query_rows(block_table, seq_lens, B, max_pages, S_q, block_table_rows, seq_lens_rows,
                                             reinterpret_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? TYPHOON_MLA_OK : cuda_fail(e);
}

int typhoon_mla_order_by_length(const int32_t* seq_lens, int32_t B, int32_t* perm, void* stream) {
    if (!seq_lens || !perm || B < 1 || B > 4096) return TYPHOON_MLA_ERR_INVALID_ARG;
    cudaError_t e = launch_order_by_length(seq_lens, B, perm, reinterpret_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? TYPHOON_MLA_OK : cuda_fail(e);
}

int typhoon_mla_set_overlap(int32_t enable) {
    g_overlap.store(enable != 0);
    return TYPHOON_MLA_OK;
}

int typhoon_mla_set_programmatic_launch(int32_t enable) {
    g_pdl.store(enable != 0);
    return TYPHOON_MLA_OK;
}

int typhoon_mla_set_naive_schedule(int32_t schedule) {
    if (schedule < 0 || schedule > 2) return TYPHOON_MLA_ERR_INVALID_ARG;
    g_naive_schedule.store(schedule);
    return TYPHOON_MLA_OK;
}

int typhoon_mla_set_kernel_path(int32_t path) {
    if (path != TYPHOON_MLA_PATH_TCGEN05 && path != TYPHOON_MLA_PATH_WARP_MMA) return TYPHOON_MLA_ERR_INVALID_ARG;
    g_kernel_path.store(path);
    return TYPHOON_MLA_OK;
}

int typhoon_mla_set_stacked_absorb(int32_t enable) {
    g_stacked_absorb.store(enable != 0);
    return TYPHOON_MLA_OK;
}

int typhoon_mla_check_status(const typhoon_mla_shared_t* sh, void* stream, int32_t* word, int32_t clear) {
    if (!sh) return TYPHOON_MLA_ERR_INVALID_ARG;
    int v = 0;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(&v, sh->status, sizeof(int), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess && clear) e = cudaMemsetAsync(sh->status, 0, sizeof(int), s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(e);
    if (word) *word = v;
    return v == 0 ? TYPHOON_MLA_OK : TYPHOON_MLA_ERR_DEVICE_CHECK;
}

int typhoon_mla_test_wait_expiry(const typhoon_mla_shared_t* sh, int64_t deadline_cycles, int32_t code, void* stream) {
    if (!sh || code < 1 || code > 255) return TYPHOON_MLA_ERR_INVALID_ARG;
    const long long d = std::min<long long>(std::max<long long>(deadline_cycles, 1000), 100000000LL);
    const cudaError_t e = launch_wait_expiry_selftest(sh->status, d, code, reinterpret_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? TYPHOON_MLA_OK : cuda_fail(e);
}

int typhoon_mla_shared_export(const typhoon_mla_shared_t* sh, void* k_nope_dst, void* v_t_dst, void* stream) {
    if (!sh || !k_nope_dst || !v_t_dst || sh->fp8) return TYPHOON_MLA_ERR_INVALID_ARG;
    const size_t bytes = (size_t)sh->dims.num_heads * (size_t)sh->Ls_pad * 128 * 2;
    if (bytes == 0) return TYPHOON_MLA_OK;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(k_nope_dst, sh->k_nope, bytes, cudaMemcpyDeviceToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(v_t_dst, sh->v_t, bytes, cudaMemcpyDeviceToDevice, s);
    return e == cudaSuccess ? TYPHOON_MLA_OK : cuda_fail(e);
}

int typhoon_mla_shared_export_fp8(const typhoon_mla_shared_t* sh, void* k_codes_dst, void* v_codes_dst, float* scales_dst,
                                  void* stream) {
    if (!sh || !k_codes_dst || !v_codes_dst || !scales_dst || !sh->fp8) return TYPHOON_MLA_ERR_INVALID_ARG;
    const int H = sh->dims.num_heads;
    const size_t n = (size_t)H * (size_t)sh->Ls_pad * 128;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(k_codes_dst, sh->k8, n, cudaMemcpyDeviceToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(v_codes_dst, sh->v8, n, cudaMemcpyDeviceToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(scales_dst, sh->fp8_f, (size_t)2 * H * sizeof(float), cudaMemcpyDeviceToDevice, s);
    return e == cudaSuccess ? TYPHOON_MLA_OK : cuda_fail(e);
}

size_t typhoon_mla_workspace_bytes(const typhoon_mla_shared_t* sh, int32_t B, int32_t max_pages, int32_t page_size,
                                   int32_t mode) {
    if (!sh || B < 1 || max_pages < 0 || (page_size != 64 && page_size != 128)) return 0;
    if (mode < TYPHOON_MLA_MODE_AUTO || mode > TYPHOON_MLA_MODE_NAIVE) return 0;
    // Worst case over the modes `mode` can resolve to, over both kernel implementations and over the work
    // decompositions a test hook may select: a workspace sized here serves whatever the switches are set to when
    // the step runs.  Only local values are used; no process-wide state is read or written.
    size_t worst = 0;
    for (int m : {TYPHOON_MLA_MODE_ABSORB, TYPHOON_MLA_MODE_HYBRID, TYPHOON_MLA_MODE_NAIVE}) {
        if (mode != TYPHOON_MLA_MODE_AUTO && mode != m && !(mode == TYPHOON_MLA_MODE_HYBRID && sh->Ls == 0)) continue;
        const int pages = m == TYPHOON_MLA_MODE_NAIVE ? 0 : max_pages;
        for (bool tc : {true, false})
            for (int schedule : {0, 1, 2})
                for (bool stacked : {true, false})
                    worst = std::max(worst, make_plan(sh, tc, schedule, B, pages, page_size, m, -1, stacked).total);
    }
    return worst + 256;
}

// One launch of the shared-prefix kernel: `rows` requests starting at `row0` against the prefix of
// `sh`, partial slots [slot0, slot0 + n_slots_level) of the step's partial arrays.
struct NaiveJob {
    const typhoon_mla_shared* sh;
    int row0, rows;
    int n_ranges;         // tile ranges (tcgen05 path) or KV splits (warp-MMA path)
    int n_slots_level;    // slots of this job's level (the kernel marks the ones it does not fill as empty)
    int slot0;
};
// Rows of a level that have no prefix: their slots get weight zero in the combine.
struct EmptySlots {
    int slot0, n_slots, row0, rows;
};

// Launch sequence of one step.  `sh` provides the weights, the absorb-side tensor maps, the side stream
// and the status word; `mode` is resolved (ABSORB, HYBRID or NAIVE); `pl.n_slots_naive` is the total
// number of naive partial slots.
constexpr int kMergeProjectMaxB = 2;   // measured: from 3 requests on the GEMM form (weights read once) is faster

static int decode_core(const Settings& cfg, const typhoon_mla_shared* sh, const NaiveJob* jobs, int n_jobs,
                const EmptySlots* empties, int n_empties,
                const Plan& pl, const void* q_nope, const void* q_pe, int32_t B, const void* ckv_pages,
                const void* kpe_pages, int64_t ckv_token_stride, int64_t kpe_token_stride, int32_t page_size, int32_t num_pages,
                const int32_t* block_table, int32_t max_pages, const int32_t* seq_lens, float softmax_scale, int32_t mode,
                void* out, float* lse_out, void* workspace, void* stream, bool out_fp32 = false) {
    const bool use_absorb = mode != TYPHOON_MLA_MODE_NAIVE;
    tmla::tl_pdl = cfg.pdl;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    char* ws = reinterpret_cast<char*>(workspace);
    const int H = sh->dims.num_heads;
    cudaError_t e = cudaSuccess;
    int launches = 0;

    float* o_part_n = reinterpret_cast<float*>(ws + pl.off_opart_n);
    float* lse_part_n = reinterpret_cast<float*>(ws + pl.off_lsepart_n);
    float* o_abs = reinterpret_cast<float*>(ws + pl.off_oabs);
    float* lse_a = reinterpret_cast<float*>(ws + pl.off_lse_a);

    const int n_chunks = pl.n_shared_chunks + pl.n_suffix_chunks;
    const bool have_absorb = use_absorb && n_chunks > 0;
    const bool tc = cfg.tc();
    // In a hybrid step the absorb branch (lines 5-6) does not depend on the naive kernel (line 4): it runs
    // on the handle's (high-priority) side stream, forked behind the caller's stream here and joined
    // before the projection.
    if (!tc)   // row ranges and the 8-bit cache need the tcgen05 kernel
        for (int j = 0; j < n_jobs; ++j)
            if (jobs[j].rows != B || jobs[j].sh->fp8) return TYPHOON_MLA_ERR_UNSUPPORTED_DIMS;
    cudaStream_t s_main = s;
    const bool forked = cfg.overlap && have_absorb && n_jobs > 0 && sh->side_stream != nullptr;
    if (forked) {
        e = cudaEventRecord(sh->ev_fork, s_main);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(sh->side_stream, sh->ev_fork, 0);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    // A failure after the fork still joins the side stream back into the caller's stream, so that the caller's stream
    // stays the only one with work of this call pending (and a stream capture is not left with an open branch).
    bool open_fork = forked;
    auto fail = [&](cudaError_t err) {
        if (open_fork && cudaEventRecord(sh->ev_join, sh->side_stream) == cudaSuccess) cudaStreamWaitEvent(s_main, sh->ev_join, 0);
        return cuda_fail(err);
    };

    // --- naive shared-prefix attention (Algorithm 1 line 4), one launch per (prefix, row range)
    for (int j = 0; j < n_jobs; ++j) {
        const NaiveJob& jb = jobs[j];
        const char* qn = reinterpret_cast<const char*>(q_nope) + (size_t)jb.row0 * H * 128 * 2;
        const char* qp = reinterpret_cast<const char*>(q_pe) + (size_t)jb.row0 * H * 64 * 2;
        float* op = o_part_n + ((size_t)jb.slot0 * B + jb.row0) * H * 128;
        float* lp = lse_part_n + ((size_t)jb.slot0 * B + jb.row0) * H;
        prof_before(TYPHOON_MLA_KERNEL_NAIVE_ATTN, s);
        if (tc) {
            NaiveAttnSm100 na{qn, qp, &jb.sh->tm_kn, &jb.sh->tm_kp, &jb.sh->tm_vt, jb.rows, H, (int)jb.sh->Ls,
                              jb.n_ranges, jb.n_slots_level, softmax_scale, op, lp, sh->status, B};
            if (jb.sh->fp8) na.fp8_mult = jb.sh->fp8_f;
            e = launch_naive_attn_sm100(na, s);
        } else {
            NaiveAttn na{qn, qp, jb.sh->k_nope, jb.sh->v_t, jb.sh->kpe, B, H, (int)jb.sh->Ls, (int)jb.sh->Ls_pad,
                         jb.n_ranges, softmax_scale, op, lp};
            e = launch_naive_attn_mma(na, s);
        }
        prof_after(TYPHOON_MLA_KERNEL_NAIVE_ATTN, s);
        if (e != cudaSuccess) return fail(e);
        ++launches;
    }
    for (int j = 0; j < n_empties; ++j) {
        const EmptySlots& es = empties[j];
        e = launch_fill_neg_inf(lse_part_n + ((size_t)es.slot0 * B + es.row0) * H, es.n_slots, (int64_t)B * H,
                                (int64_t)es.rows * H, s);
        if (e != cudaSuccess) return fail(e);
        ++launches;
    }
    bool combined = false;
    if (forked) s = sh->side_stream;
    if (have_absorb) {
        // ragged suffixes: the longest requests are launched first (order computed on the device, no host
        // sync): by an extra block of the query-absorption kernel on the tcgen05 path, by its own kernel otherwise
        int32_t* order = nullptr;
        int32_t* desc = nullptr;   // per-position descriptors, written next to the order on the tcgen05 path
        if (pl.n_suffix_chunks > 0 && B > 1 && B <= 4096) order = reinterpret_cast<int32_t*>(ws + pl.off_order);
        // --- query absorption Q_A = Q_N W_UK (Algorithm 1 line 5)
        void* q_abs = ws + pl.off_qabs;
        prof_before(TYPHOON_MLA_KERNEL_Q_ABSORB, s);
        if (tc) {
            if (order) desc = reinterpret_cast<int32_t*>(ws + pl.off_desc);
            // Beside the shared-prefix kernel the absorb branch has the SMs that kernel's CTAs leave free: if those are few,
            // that many CTAs walk through the heads (each resident for the whole launch) instead of one CTA per head
            // queueing for them.
            int walk_ctas = 0;
            if (forked) {
                int naive_ctas = 0;
                for (int j = 0; j < n_jobs; ++j) {
                    const int rows = jobs[j].rows;
                    const int groups = jobs[j].sh->fp8 ? (rows + 127) / 128 : (rows <= 128 ? 1 : (rows + 255) / 256);
                    naive_ctas = std::max(naive_ctas, jobs[j].n_ranges * groups);
                }
                const int free_sms = sh->num_sms - naive_ctas;
                if (n_jobs == 1 && free_sms >= 8 && free_sms < H) {
                    // ... but only if the shared-prefix kernel lasts about as long as the walk (measured: about 5 us per head
                    // for a walking CTA, 0.7 us per 64-token tile for a shared-prefix CTA; B = 64, H = 128: the walk wins
                    // from 3072 prefix tokens on and loses at 2048); under a short shared-prefix kernel one CTA per head,
                    // which spreads over the whole GPU as soon as that kernel ends, is faster.
                    const int64_t tok = jobs[0].rows <= 128 || jobs[0].sh->fp8 ? 64 : 128;
                    const int64_t tiles_per_cta = ((jobs[0].sh->Ls + tok - 1) / tok * H + jobs[0].n_ranges - 1) / jobs[0].n_ranges;
                    const int heads_per_cta = (H + free_sms - 1) / free_sms;
                    if ((double)tiles_per_cta * (tok == 64 ? 0.7 : 3.0) >= 4.0 * heads_per_cta) walk_ctas = free_sms;
                }
            }
            e = launch_q_absorb_sm100(q_nope, &sh->tm_wuk_t, q_abs, B, H, sh->num_sms, walk_ctas, sh->status, order ? seq_lens : nullptr, order,
                                      block_table, max_pages, page_size, desc, s);
        } else {
            GemmTN g1{q_nope, (int64_t)H * 128, 128, sh->w_uk_t, 128, 512 * 128, q_abs, (int64_t)H * 512, 512,
                      B, 512, 128, H, false};
            e = launch_gemm_tn(g1, s);
            if (e == cudaSuccess && order) {
                e = launch_order_by_length(seq_lens, B, order, s);
                ++launches;
            }
        }
        prof_after(TYPHOON_MLA_KERNEL_Q_ABSORB, s);
        if (e != cudaSuccess) return fail(e);
        ++launches;
        // --- absorb attention over latent tokens (Algorithm 1 line 6)
        float* o_part_a = reinterpret_cast<float*>(ws + pl.off_opart_a);
        float* lse_part_a = reinterpret_cast<float*>(ws + pl.off_lsepart_a);
        void* o_lat = ws + pl.off_olat;
        AbsorbAttn ab{q_abs, q_pe, sh->ckv, sh->kpe, mode == TYPHOON_MLA_MODE_ABSORB ? (int)sh->Ls : 0,
                      ckv_pages, kpe_pages, ckv_token_stride, kpe_token_stride, page_size, num_pages, block_table, max_pages,
                      seq_lens, order, desc, B, H, pl.chunk, pl.n_shared_chunks, pl.n_suffix_chunks, softmax_scale,
                      o_part_a, lse_part_a, sh->status, cfg.stacked_absorb};
        prof_before(TYPHOON_MLA_KERNEL_ABSORB_ATTN, s);
        e = tc ? launch_absorb_attn_sm100(ab, &sh->tm_ckv, &sh->tm_kpe_tok, o_lat, lse_a, sh->status, s)
               : launch_absorb_attn_mma(ab, s);
        prof_after(TYPHOON_MLA_KERNEL_ABSORB_ATTN, s);
        if (e != cudaSuccess) return fail(e);
        ++launches;
        if (n_jobs == 0 && n_empties == 0 && n_chunks > 1 && B <= kMergeProjectMaxB) {
            // absorb-only, a handful of requests: merge + projection + rounding in one launch
            prof_before(TYPHOON_MLA_KERNEL_MERGE, s);
            e = launch_merge_project(o_part_a, lse_part_a, n_chunks, B, H, sh->w_uv, out, lse_out, out_fp32, s);
            prof_after(TYPHOON_MLA_KERNEL_MERGE, s);
            if (e != cudaSuccess) return fail(e);
            g_last_launches = launches + 1;
            return TYPHOON_MLA_OK;
        }
        if (!(tc && n_chunks == 1)) {   // a single-chunk tcgen05 launch has already written the merged result
            prof_before(TYPHOON_MLA_KERNEL_MERGE, s);
            e = launch_merge_latent(o_part_a, lse_part_a, n_chunks, B, H, o_lat, lse_a, s);
            prof_after(TYPHOON_MLA_KERNEL_MERGE, s);
            if (e != cudaSuccess) return fail(e);
            ++launches;
        }
        if (forked) {
            e = cudaEventRecord(sh->ev_join, sh->side_stream);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(s_main, sh->ev_join, 0);
            open_fork = false;
            if (e != cudaSuccess) return cuda_fail(e);
            s = s_main;
        }
        // --- output projection O_A W_UV^T (Algorithm 1 line 7); on the tcgen05 path its epilogue also does the
        //     LSE combine (line 8)
        prof_before(TYPHOON_MLA_KERNEL_W_UV, s);
        if (tc) {
            GemmTN g2{o_lat, (int64_t)H * 512, 512, sh->w_uv, 512, 128 * 512, nullptr, 0, 0, B, 128, 512, H, false};
            CombineEpilogue ce;
            ce.o_naive = o_part_n; ce.lse_naive = lse_part_n; ce.n_naive = pl.n_slots_naive;
            ce.lse_abs = lse_a; ce.out = out; ce.lse_out = lse_out; ce.H = H;
            ce.out_fp32 = out_fp32 ? 1 : 0;
            e = launch_gemm_tn_sm100(g2, sh->status, s, &ce);
            combined = true;
        } else {
            GemmTN g2{o_lat, (int64_t)H * 512, 512, sh->w_uv, 512, 128 * 512, o_abs, (int64_t)H * 128, 128,
                      B, 128, 512, H, true};
            e = launch_gemm_tn(g2, s);
        }
        prof_after(TYPHOON_MLA_KERNEL_W_UV, s);
        if (e != cudaSuccess) return fail(e);
        ++launches;
    }
    // --- LSE combine (Algorithm 1 line 8)
    if (!combined) {
        prof_before(TYPHOON_MLA_KERNEL_COMBINE, s);
        e = launch_combine(o_part_n, lse_part_n, pl.n_slots_naive, have_absorb ? o_abs : nullptr, lse_a, B, H, out,
                           lse_out, s, out_fp32);
        prof_after(TYPHOON_MLA_KERNEL_COMBINE, s);
        if (e != cudaSuccess) return fail(e);
        ++launches;
    }
    g_last_launches = launches;
    return TYPHOON_MLA_OK;
}

static int decode_impl(const typhoon_mla_shared_t* sh, const void* q_nope, const void* q_pe, int32_t B,
                       const void* ckv_pages, const void* kpe_pages, int64_t ckv_token_stride,
                       int64_t kpe_token_stride, int32_t page_size, int32_t num_pages, const int32_t* block_table,
                       int32_t max_pages, const int32_t* seq_lens, float softmax_scale, int32_t mode, void* out,
                       float* lse_out, void* workspace, size_t workspace_bytes, void* stream, bool out_fp32) {
    g_last_launches = 0;
    if (!sh || !q_nope || !q_pe || !out || B < 1 || max_pages < 0) return TYPHOON_MLA_ERR_INVALID_ARG;
    if (!on_handle_device(sh)) return TYPHOON_MLA_ERR_INVALID_ARG;
    const Settings cfg = snapshot();
    if (page_size != 64 && page_size != 128) return TYPHOON_MLA_ERR_INVALID_ARG;
    if (mode < TYPHOON_MLA_MODE_AUTO || mode > TYPHOON_MLA_MODE_NAIVE) return TYPHOON_MLA_ERR_INVALID_ARG;
    if (!aligned16(q_nope) || !aligned16(q_pe) || !aligned16(out)) return TYPHOON_MLA_ERR_INVALID_ARG;
    if (!(softmax_scale > 0.f) || softmax_scale > 3.0e38f) return TYPHOON_MLA_ERR_INVALID_ARG;   // positive, finite
    mode = resolve_mode(sh, B, max_pages, mode);
    const bool use_absorb = mode != TYPHOON_MLA_MODE_NAIVE;
    if (use_absorb && max_pages > 0) {
        if (!ckv_pages || !kpe_pages || !block_table || !seq_lens || num_pages < 1) return TYPHOON_MLA_ERR_INVALID_ARG;
        if (!aligned16(ckv_pages) || !aligned16(kpe_pages) || ckv_token_stride < 512 || kpe_token_stride < 64 ||
            ckv_token_stride % 8 || kpe_token_stride % 8)
            return TYPHOON_MLA_ERR_INVALID_ARG;
    }
    if (mode == TYPHOON_MLA_MODE_NAIVE && sh->Ls == 0) max_pages = 0;
    const Plan pl = make_plan(sh, cfg.tc(), cfg.naive_schedule, B, use_absorb ? max_pages : 0, page_size, mode, -1, cfg.stacked_absorb);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return TYPHOON_MLA_ERR_INVALID_ARG;
    if (workspace_bytes < pl.total) return TYPHOON_MLA_ERR_WORKSPACE_TOO_SMALL;

    NaiveJob job{sh, 0, B, pl.n_split_naive, pl.n_slots_naive, 0};
    return decode_core(cfg, sh, &job, pl.n_split_naive > 0 ? 1 : 0, nullptr, 0, pl, q_nope, q_pe, B, ckv_pages, kpe_pages,
                       ckv_token_stride, kpe_token_stride, page_size, num_pages, block_table, use_absorb ? max_pages : 0,
                       seq_lens, softmax_scale, mode, out, lse_out, workspace, stream, out_fp32);
}

int typhoon_mla_decode(const typhoon_mla_shared_t* sh, const void* q_nope, const void* q_pe, int32_t B,
                       const void* ckv_pages, const void* kpe_pages, int64_t ckv_token_stride,
                       int64_t kpe_token_stride, int32_t page_size, int32_t num_pages, const int32_t* block_table,
                       int32_t max_pages, const int32_t* seq_lens, float softmax_scale, int32_t mode, void* out,
                       float* lse_out, void* workspace, size_t workspace_bytes, void* stream) {
    return decode_impl(sh, q_nope, q_pe, B, ckv_pages, kpe_pages, ckv_token_stride, kpe_token_stride, page_size, num_pages,
                       block_table, max_pages, seq_lens, softmax_scale, mode, out, lse_out, workspace, workspace_bytes, stream,
                       false);
}

// ---- context sharded over several devices: per-device partial + merge -----------------------------
int typhoon_mla_decode_partial(const typhoon_mla_shared_t* sh, const void* q_nope, const void* q_pe, int32_t B,
                               const void* ckv_pages, const void* kpe_pages, int64_t ckv_token_stride,
                               int64_t kpe_token_stride, int32_t page_size, int32_t num_pages,
                               const int32_t* block_table, int32_t max_pages, const int32_t* seq_lens,
                               float softmax_scale, int32_t mode, float* out_partial, float* lse_partial,
                               void* workspace, size_t workspace_bytes, void* stream) {
    if (!lse_partial) return TYPHOON_MLA_ERR_INVALID_ARG;
    return decode_impl(sh, q_nope, q_pe, B, ckv_pages, kpe_pages, ckv_token_stride, kpe_token_stride, page_size, num_pages,
                       block_table, max_pages, seq_lens, softmax_scale, mode, out_partial, lse_partial, workspace,
                       workspace_bytes, stream, true);
}

int typhoon_mla_combine_partials(const float* o_parts, const float* lse_parts, int32_t n_parts, int32_t B, int32_t H,
                                 void* out, float* lse_out, void* stream) {
    if (!o_parts || !lse_parts || !out || n_parts < 1 || B < 1 || H < 1) return TYPHOON_MLA_ERR_INVALID_ARG;
    if (!aligned16(o_parts) || !aligned16(out)) return TYPHOON_MLA_ERR_INVALID_ARG;
    tmla::tl_pdl = g_pdl.load();
    const cudaError_t e = launch_combine(o_parts, lse_parts, n_parts, nullptr, nullptr, B, H, out, lse_out,
                                         reinterpret_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e);
    g_last_launches = 1;
    return TYPHOON_MLA_OK;
}
// ---- several shared prefixes per step (tree-structured prompts) ------------------------------------
namespace {
constexpr int kMaxLevels = 8, kMaxTreeJobs = 256;
struct TreePlan {
    const typhoon_mla_shared* sh0 = nullptr;   // first prefix: weights, absorb-side tensor maps, side stream, status
    NaiveJob jobs[kMaxTreeJobs];
    EmptySlots empties[kMaxTreeJobs];
    int n_jobs = 0, n_empties = 0, total_slots = 0;
};
int plan_tree(const typhoon_mla_prefix_level_t* levels, int n_levels, int B, int schedule, TreePlan* tp) {
    if (!levels || n_levels < 1 || n_levels > kMaxLevels || B < 1) return TYPHOON_MLA_ERR_INVALID_ARG;
    for (int l = 0; l < n_levels && !tp->sh0; ++l) {
        if (!levels[l].prefixes || !levels[l].group_begin || levels[l].n_groups < 1) return TYPHOON_MLA_ERR_INVALID_ARG;
        for (int g = 0; g < levels[l].n_groups && !tp->sh0; ++g) tp->sh0 = levels[l].prefixes[g];
    }
    if (!tp->sh0) return TYPHOON_MLA_ERR_INVALID_ARG;
    const int H = tp->sh0->dims.num_heads;
    int slot0 = 0;
    for (int l = 0; l < n_levels; ++l) {
        const typhoon_mla_prefix_level_t& lv = levels[l];
        if (!lv.prefixes || !lv.group_begin || lv.n_groups < 1) return TYPHOON_MLA_ERR_INVALID_ARG;
        if (lv.group_begin[0] != 0 || lv.group_begin[lv.n_groups] != B) return TYPHOON_MLA_ERR_INVALID_ARG;
        const int first_job = tp->n_jobs;
        int level_slots = 0;
        for (int g = 0; g < lv.n_groups; ++g) {
            const int r0 = lv.group_begin[g], r1 = lv.group_begin[g + 1];
            if (r1 < r0) return TYPHOON_MLA_ERR_INVALID_ARG;
            const typhoon_mla_shared* sh = lv.prefixes[g];
            if (sh && (sh->dims.num_heads != H || sh->device != tp->sh0->device)) return TYPHOON_MLA_ERR_INVALID_ARG;
            if (!sh || sh->Ls == 0 || r1 == r0) continue;
            if (tp->n_jobs == kMaxTreeJobs) return TYPHOON_MLA_ERR_INVALID_ARG;
            int ranges = 0, slots = 0;
            naive_sm100_plan(r1 - r0, H, sh->Ls, sh->num_sms > 0 ? sh->num_sms : kDefaultNumSM, schedule, &ranges, &slots,
                             sh->fp8 != 0);
            tp->jobs[tp->n_jobs++] = NaiveJob{sh, r0, r1 - r0, ranges, 0, slot0};
            level_slots = std::max(level_slots, slots);
        }
        if (level_slots == 0) continue;   // no prefix at this level at all: no slots
        for (int j = first_job; j < tp->n_jobs; ++j) tp->jobs[j].n_slots_level = level_slots;
        for (int g = 0; g < lv.n_groups; ++g) {
            const int r0 = lv.group_begin[g], r1 = lv.group_begin[g + 1];
            const typhoon_mla_shared* sh = lv.prefixes[g];
            if ((sh && sh->Ls > 0) || r1 == r0) continue;
            if (tp->n_empties == kMaxTreeJobs) return TYPHOON_MLA_ERR_INVALID_ARG;
            tp->empties[tp->n_empties++] = EmptySlots{slot0, level_slots, r0, r1 - r0};
        }
        slot0 += level_slots;
    }
    tp->total_slots = slot0;
    return TYPHOON_MLA_OK;
}
}  // namespace

size_t typhoon_mla_tree_workspace_bytes(const typhoon_mla_prefix_level_t* levels, int32_t n_levels, int32_t B,
                                        int32_t max_pages, int32_t page_size) {
    if (max_pages < 0 || (page_size != 64 && page_size != 128)) return 0;
    // worst case over the work decompositions a test hook may select (the tree step needs the tcgen05 kernels)
    size_t worst = 0;
    for (int schedule : {0, 1, 2}) {
        TreePlan tp;
        if (plan_tree(levels, n_levels, B, schedule, &tp) != TYPHOON_MLA_OK) return 0;
        worst = std::max(worst, make_plan(tp.sh0, true, schedule, B, max_pages, page_size, TYPHOON_MLA_MODE_HYBRID, tp.total_slots).total);
    }
    return worst + 256;
}

int typhoon_mla_decode_tree(const typhoon_mla_prefix_level_t* levels, int32_t n_levels, const void* q_nope,
                            const void* q_pe, int32_t B, const void* ckv_pages, const void* kpe_pages,
                            int64_t ckv_token_stride, int64_t kpe_token_stride, int32_t page_size, int32_t num_pages,
                            const int32_t* block_table, int32_t max_pages, const int32_t* seq_lens, float softmax_scale,
                            void* out, float* lse_out, void* workspace, size_t workspace_bytes, void* stream) {
    g_last_launches = 0;
    if (!q_nope || !q_pe || !out || B < 1 || max_pages < 0) return TYPHOON_MLA_ERR_INVALID_ARG;
    if (page_size != 64 && page_size != 128) return TYPHOON_MLA_ERR_INVALID_ARG;
    if (!aligned16(q_nope) || !aligned16(q_pe) || !aligned16(out)) return TYPHOON_MLA_ERR_INVALID_ARG;
    if (!(softmax_scale > 0.f) || softmax_scale > 3.0e38f) return TYPHOON_MLA_ERR_INVALID_ARG;
    const Settings cfg = snapshot();
    if (!cfg.tc()) return TYPHOON_MLA_ERR_UNSUPPORTED_DIMS;
    if (max_pages > 0) {
        if (!ckv_pages || !kpe_pages || !block_table || !seq_lens || num_pages < 1) return TYPHOON_MLA_ERR_INVALID_ARG;
        if (!aligned16(ckv_pages) || !aligned16(kpe_pages) || ckv_token_stride < 512 || kpe_token_stride < 64 ||
            ckv_token_stride % 8 || kpe_token_stride % 8)
            return TYPHOON_MLA_ERR_INVALID_ARG;
    }
    TreePlan tp;
    const int rc = plan_tree(levels, n_levels, B, cfg.naive_schedule, &tp);
    if (rc != TYPHOON_MLA_OK) return rc;
    if (!on_handle_device(tp.sh0)) return TYPHOON_MLA_ERR_INVALID_ARG;
    // NAIVE when there is no page table (nothing for the absorb branch), else Algorithm 1 with several line-4 launches
    const int mode = max_pages == 0 ? TYPHOON_MLA_MODE_NAIVE : TYPHOON_MLA_MODE_HYBRID;
    const Plan pl = make_plan(tp.sh0, true, cfg.naive_schedule, B, max_pages, page_size, mode, tp.total_slots);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return TYPHOON_MLA_ERR_INVALID_ARG;
    if (workspace_bytes < pl.total) return TYPHOON_MLA_ERR_WORKSPACE_TOO_SMALL;
    return decode_core(cfg, tp.sh0, tp.jobs, tp.n_jobs, tp.empties, tp.n_empties, pl, q_nope, q_pe, B, ckv_pages, kpe_pages,
                       ckv_token_stride, kpe_token_stride, page_size, num_pages, block_table, max_pages, seq_lens,
                       softmax_scale, mode, out, lse_out, workspace, stream);
}

int typhoon_mla_profile_begin(int32_t kernel_id, int32_t max_launches) {
    if (kernel_id < 0 || kernel_id >= TYPHOON_MLA_NUM_KERNELS || max_launches < 1) return TYPHOON_MLA_ERR_INVALID_ARG;
    if (g_prof.ev) return TYPHOON_MLA_ERR_INVALID_ARG;
    g_prof.ev = new (std::nothrow) cudaEvent_t[2 * (size_t)max_launches];
    if (!g_prof.ev) return TYPHOON_MLA_ERR_ALLOC;
    for (int i = 0; i < 2 * max_launches; ++i) {
        cudaError_t e = cudaEventCreate(&g_prof.ev[i]);
        if (e != cudaSuccess) {
            for (int j = 0; j < i; ++j) cudaEventDestroy(g_prof.ev[j]);
            delete[] g_prof.ev;
            g_prof.ev = nullptr;
            return cuda_fail(e);
        }
    }
    g_prof.capacity = max_launches;
    g_prof.used = 0;
    g_prof.kernel_id = kernel_id;
    return TYPHOON_MLA_OK;
}

int typhoon_mla_profile_end(double* total_ms, int32_t* launches) {
    if (!g_prof.ev) return TYPHOON_MLA_ERR_INVALID_ARG;
    double tot = 0.0;
    int st = TYPHOON_MLA_OK;
    for (int i = 0; i < g_prof.used; ++i) {
        float ms = 0.f;
        cudaError_t e = cudaEventSynchronize(g_prof.ev[2 * i + 1]);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, g_prof.ev[2 * i], g_prof.ev[2 * i + 1]);
        if (e != cudaSuccess) { st = cuda_fail(e); break; }
        tot += ms;
    }
    if (total_ms) *total_ms = tot;
    if (launches) *launches = g_prof.used;
    for (int i = 0; i < 2 * g_prof.capacity; ++i) cudaEventDestroy(g_prof.ev[i]);
    delete[] g_prof.ev;
    g_prof = Profile();
    return st;
}

size_t typhoon_mla_host_staging_bytes(const typhoon_mla_shared_t* sh, int32_t B, int32_t max_pages) {
    if (!sh || B < 1 || max_pages < 0) return 0;
    const size_t BH = (size_t)B * sh->dims.num_heads;
    return round_up(BH * 128 * 2, 256) + round_up(BH * 64 * 2, 256) + round_up((size_t)B * std::max(max_pages, 1) * 4, 256) +
           round_up((size_t)B * 4, 256) + round_up(BH * 128 * 2, 256);
}

int typhoon_mla_decode_host(const typhoon_mla_shared_t* sh, const void* q_nope_host, const void* q_pe_host, int32_t B,
                            const void* ckv_pages, const void* kpe_pages, int64_t ckv_token_stride,
                            int64_t kpe_token_stride, int32_t page_size, int32_t num_pages,
                            const int32_t* block_table_host, int32_t max_pages, const int32_t* seq_lens_host,
                            float softmax_scale, int32_t mode,
                            void* out_host, void* staging, size_t staging_bytes, void* workspace,
                            size_t workspace_bytes, void* stream) {
    if (!sh || !q_nope_host || !q_pe_host || !out_host || !staging || B < 1 || max_pages < 0)
        return TYPHOON_MLA_ERR_INVALID_ARG;
    if (max_pages > 0 && (!block_table_host || !seq_lens_host)) return TYPHOON_MLA_ERR_INVALID_ARG;
    if (staging_bytes < typhoon_mla_host_staging_bytes(sh, B, max_pages)) return TYPHOON_MLA_ERR_WORKSPACE_TOO_SMALL;
    if (reinterpret_cast<uintptr_t>(staging) & 255u) return TYPHOON_MLA_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const size_t BH = (size_t)B * sh->dims.num_heads;
    char* st = reinterpret_cast<char*>(staging);
    char* d_qn = st;
    char* d_qp = d_qn + round_up(BH * 128 * 2, 256);
    char* d_bt = d_qp + round_up(BH * 64 * 2, 256);
    char* d_sl = d_bt + round_up((size_t)B * std::max(max_pages, 1) * 4, 256);
    char* d_out = d_sl + round_up((size_t)B * 4, 256);
    cudaError_t e = cudaMemcpyAsync(d_qn, q_nope_host, BH * 128 * 2, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d_qp, q_pe_host, BH * 64 * 2, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess && max_pages > 0) {
        e = cudaMemcpyAsync(d_bt, block_table_host, (size_t)B * max_pages * 4, cudaMemcpyHostToDevice, s);
        if (e == cudaSuccess) e = cudaMemcpyAsync(d_sl, seq_lens_host, (size_t)B * 4, cudaMemcpyHostToDevice, s);
    }
    if (e != cudaSuccess) return cuda_fail(e);
    int st_code = typhoon_mla_decode(sh, d_qn, d_qp, B, ckv_pages, kpe_pages, ckv_token_stride, kpe_token_stride,
                                     page_size, num_pages, reinterpret_cast<const int32_t*>(d_bt), max_pages,
                                     reinterpret_cast<const int32_t*>(d_sl), softmax_scale, mode, d_out, nullptr,
                                     workspace, workspace_bytes, stream);
    if (st_code != TYPHOON_MLA_OK) return st_code;
    e = cudaMemcpyAsync(out_host, d_out, BH * 128 * 2, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return cuda_fail(e);
    return TYPHOON_MLA_OK;
}

}  // extern "C"
