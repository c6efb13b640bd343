// Naive shared-prefix attention (Algorithm 1 line 4) on tcgen05 / TMEM / TMA.
//
// Per head h the step is a dense contraction over all B query rows:
//     S = Q_h [B,192] * [K_nope_h | k_pe]^T [192, L_s],  O = softmax(S) * V_h [L_s,128].
//
// Work decomposition.  The KV tiles of all heads form one sequence of T = H * n_tiles tiles, which
// is cut into R equal contiguous ranges.  A CTA owns one range and one group of query rows (128
// rows for B <= 128, else 256; CTAs of the same range are adjacent in the grid, so the row groups
// of a head walk the same KV tiles at about the same time and share them through L2).  A CTA works
// through its range as a few "segments" (head, tile range), each a complete flash-attention pass
// with its own Q tile that ends in a normalised fp32 partial plus LSE; the combine step merges the
// partials of a (request, head).  The host picks R: a multiple of H (every range inside one head,
// "column split") or the number of SMs over the number of row groups ("stream-K": one resident CTA
// per SM, every SM gets the same number of tiles whatever H and L_s are).
//
// Inside a segment two independent attention "streams" share the TMA/MMA machinery:
//   * B > 128  (mode X, 128-token KV tiles): stream i = query rows [256g + 128i, +128); both
//     streams consume every KV tile (tiles are loaded once).  Compute-bound regime: N = 128 per
//     S MMA halves the re-reads of Q from shared memory, the streams ping-pong between tensor
//     core and softmax.
//   * B <= 128 (mode Y, 64-token KV tiles): both streams use the same 128 query rows; stream i
//     takes every second KV tile with its own softmax state, and at the end of the segment
//     stream 0 merges the two accumulators (same tensor-memory lanes) into one partial.
//     HBM-bound regime: small tiles give deep K and V rings.
//     With B <= 64 the MMAs are issued with M = 64 (template flag M64): accumulator row r then
//     sits in lane 32 (r / 16) + r % 16 and half of the softmax lanes hold no row.
//
// Warp roles (384 threads): warp 0 = TMA producer for Q and the K ring, warp 2 = TMA producer
// for the V ring, warp 1 = issuer of the S = Q K^T MMAs and TMEM owner, warp 3 = issuer of the
// O += P V MMAs, warps 4-7 / 8-11 = softmax warpgroup of stream 0 / 1 (thread = one query row).
// Role warps run their loops with all lanes and predicate the issuing instruction on one
// elected lane.  Ring positions, S-buffer uses and accumulator completions are counted across
// segments, so the pipeline never drains inside a CTA except for the Q tile of a new segment.
//
// Tensor memory (512 columns).  64-token tiles: S[i][buf] (64 fp32 columns, double buffered; P
// in bf16 overwrites the first 32) at (2i+buf)*64, O[i] at 256 + 128 i.  128-token tiles: S[i]
// (128 columns, P overwrites the first 64) at 128 i, O[i] at 256 + 128 i.
//
// The expanded cache is stored in 64-token blocks: K_nope [H, L/64, 2 slabs, 64, 64],
// V^T [H, L/64, 128, 64], rope keys [L, 64]; every TMA box is a contiguous 8 or 16 KB.
//
// With the expanded cache stored as E4M3 codes (template flag FP8; 64-token tiles, row groups of at most 128
// requests) four more warps (12-15, 512 threads) widen the copied code blocks into half-precision operand
// tiles; see the conversion warps below.
//
// Every mbarrier wait has a deadline; on expiry all roles fall through to the common teardown
// and the status word is set.
#include <cstddef>

#include "kernels.h"
#include "sm100.cuh"



namespace tmla {
namespace {

using namespace sm100;

constexpr int Q_TILE_BYTES = 128 * 192 * 2;   // 3 slabs [128][64] bf16

constexpr int MAX_STAGES = 4;
constexpr int MAX_Q_STAGES = 8;
constexpr int kNaiveSmemMax = 227 * 1024;   // opt-in limit set once per device; every launch stays below it

struct NaiveSm100Params {
    int B, H, Ls, Ls_pad;
    int part_rows;         // rows of the partial arrays (>= B: a launch may fill a row range of a larger batch)
    int m_groups;          // query-row groups per head
    int n_tiles;           // KV tiles per head
    int n_ranges;          // R (grid = R * m_groups CTAs)
    int per, rem;          // T = R * per + rem: ranges [0, rem) hold per + 1 tiles, the others per
    int n_seg_max;         // partial slots per head (one per segment of the head)
    int k_stages, v_stages;
    int kq_stages, vq_stages;   // 8-bit cache: depth of the staging rings the copies land in
    const float* mult;          // 8-bit cache: [2][H] power-of-two scales of K_nope and of V, per head
    float scale_log2;
    float* o_part;     // [n_slots][part_rows][H][128]
    float* lse_part;   // [n_slots][part_rows][H]
    int* status;
};

struct Barriers {
    uint64_t q_full, q_free;
    uint64_t k_full[MAX_STAGES], k_empty[MAX_STAGES];
    uint64_t v_full[MAX_STAGES], v_empty[MAX_STAGES];
    // p_half (128-token tiles): the first 64 tokens' probabilities of a tile are in place, so the PV product can start
    // on them while the softmax warpgroup is still working on the second 64
    uint64_t s_ready[2][2], p_ready[2][2], p_half[2], sbuf_free[2][2], o_free[2];
    // 64-token tiles: stream 1 has published its softmax state (merge_m / merge_l) and its accumulator is
    // complete; stream 0 then merges the two streams' results into one partial (128 arrivals per segment)
    uint64_t merge_ready;
    // completion of PV product u of stream i goes to o_done[i][u & 1]: a waiter that knows product
    // u-2 has landed (every wait below does) then sees a barrier at most one completion from the
    // awaited one, which is what a parity wait can tell apart
    uint64_t o_done[2][2];
    // 8-bit cache: staging rings filled by bulk copies (K codes + rope keys; V codes) and emptied by the conversion
    // warpgroup, which fills the 16-bit rings k_full / v_full guard; q_conv: the query tile is in half precision
    uint64_t kq_full[MAX_Q_STAGES], kq_empty[MAX_Q_STAGES], vq_full[MAX_Q_STAGES], vq_empty[MAX_Q_STAGES], q_conv;
    uint32_t tmem_base;
    int abort_flag;
    float merge_m[128], merge_l[128];   // stream 1's reference exponent and row sum, per query row
};

// One segment of a CTA's tile range.
struct Segment {
    int t0, cnt;           // first tile, number of tiles
    int h, row0;           // head, first query row
    int slot_seg;          // index of this segment among the head's segments
    bool last_of_col;      // this segment ends the head
    int n_str0, n_str1;    // tiles per stream
};

// TOK = tokens per KV tile: 64 (mode Y, B <= 128) or 128 (mode X, B > 128).
// FP8: the expanded cache is stored as E4M3 codes (see the conversion warpgroup below); 64 query rows per CTA.
template <int TOK, bool M64, bool FP8>
__global__ void __launch_bounds__(FP8 ? 512 : 384, 1)
naive_attn_sm100_kernel(const __grid_constant__ CUtensorMap tm_qn, const __grid_constant__ CUtensorMap tm_qp,
                        const __grid_constant__ CUtensorMap tm_kn, const __grid_constant__ CUtensorMap tm_kp,
                        const __grid_constant__ CUtensorMap tm_vt, NaiveSm100Params p) {
    constexpr bool MODE_Y = TOK == 64;
    // 128-token tiles (compute-bound regime): pairs of exponentials computed on the FMA pipe instead of the
    // special-function unit, by position of the pair within a group of eight (bit set = polynomial).  Measured at
    // B = 512: one pair in four is the best mix (-4 % kernel time); one in eight and three in eight gain 1-2 %, every
    // second pair changes the compiler's register allocation for the worse (+5 %).
    constexpr unsigned kPolyExpMask = TOK == 128 ? 0x88u : 0u;
    constexpr int NB = MODE_Y ? 2 : 1;                  // S buffers per stream
    constexpr int BLK = TOK / 64;                       // 64-token blocks per tile
    constexpr int K_SLAB = TOK * 128;                   // bytes of one [TOK][64] K slab
    constexpr int K_TILE_BYTES = (FP8 ? 2 : 3) * K_SLAB;   // (8-bit cache: the rope slab stays in the staging ring)
    constexpr int V_TILE_BYTES = BLK * 16384;           // BLK slabs [128 dims][64 tokens]
    constexpr int ROWS = FP8 ? (M64 ? 64 : 128) : (MODE_Y ? 128 : 256);   // query rows per column
    static_assert(!FP8 || TOK == 64, "the 8-bit cache path is built for 64-token tiles");
    constexpr int Q_SLAB = ((FP8 && M64) ? 64 : 128) * 128;   // bytes of one [rows][64] slab of the query tile
    constexpr int Q_BYTES = 3 * Q_SLAB;
    constexpr int KQ_BYTES = 16384, VQ_BYTES = 8192;    // staging slots: K codes 8 KB + rope keys 8 KB; V codes 8 KB

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    constexpr int n_q_tiles = MODE_Y ? 1 : 2;
    uint8_t* sQ = smem;
    uint8_t* sK = sQ + n_q_tiles * Q_BYTES;
    uint8_t* sV = sK + p.k_stages * K_TILE_BYTES;
    uint8_t* sKq = sV + p.v_stages * V_TILE_BYTES;      // staging rings (8-bit cache only)
    uint8_t* sVq = sKq + (FP8 ? p.kq_stages : 0) * KQ_BYTES;
    Barriers* bar = reinterpret_cast<Barriers*>(sVq + (FP8 ? p.vq_stages : 0) * VQ_BYTES);
    const int k_depth = FP8 ? p.kq_stages : p.k_stages, v_depth = FP8 ? p.vq_stages : p.v_stages;   // rings the copies land in
    volatile int* abort_flag = &bar->abort_flag;

    const int warp = warp_index_uniform(), lane = threadIdx.x & 31;
    const int rng = blockIdx.x / p.m_groups, grp = blockIdx.x % p.m_groups;
    pdl_trigger();   // the next kernel of the stream may be scheduled as soon as every CTA of this one has started
    pdl_wait();      // nothing below touches global memory before the stream's earlier kernels are done

    // this CTA's contiguous range of the global tile sequence (T < 2^31: 32-bit arithmetic)
    const int g_begin = rng * p.per + min(rng, p.rem);
    const int g_end = g_begin + p.per + (rng < p.rem ? 1 : 0);

    // Segment starting at global tile g (g_begin <= g < g_end).
    auto segment_at = [&](int g) {
        Segment s;
        s.h = g / p.n_tiles;
        s.t0 = g - s.h * p.n_tiles;
        s.cnt = min(p.n_tiles - s.t0, g_end - g);
        s.row0 = grp * ROWS;
        // first range that reaches into this head: the one containing the head's first tile
        const int first_tile = s.h * p.n_tiles, big = p.rem * (p.per + 1);
        const int r_first = first_tile < big ? first_tile / (p.per + 1) : p.rem + (first_tile - big) / p.per;
        s.slot_seg = rng - r_first;
        s.last_of_col = (s.t0 + s.cnt == p.n_tiles);
        if (MODE_Y) {
            s.n_str0 = (s.cnt + 1) >> 1;
            s.n_str1 = s.cnt >> 1;
        } else {
            s.n_str0 = s.cnt;
            s.n_str1 = (s.row0 + 128 < p.B) ? s.cnt : 0;   // second row tile entirely past B: skip it
        }
        return s;
    };
    // Softmax attention does not depend on the order in which KV tiles are visited.  Segments of
    // different heads start at different tiles and wrap around, so that the CTAs resident at any
    // moment do not all read the same offset of their (power-of-two strided) per-head arrays
    // (the row groups of one range use the same order).
    auto tile_of = [&](const Segment& s, int e) {
        const int rot = (int)(((unsigned)s.h * 37u + (unsigned)s.slot_seg * 11u) % (unsigned)s.cnt);
        const int t = e + rot;
        return s.t0 + (t >= s.cnt ? t - s.cnt : t);
    };
    // ring position (within the segment) of the KV tile used by stream i at step j; S columns of use u
    auto entry_of = [&](int j, int i) { return MODE_Y ? 2 * j + i : j; };
    auto s_col = [&](int i, int u) { return (uint32_t)(MODE_Y ? (2 * i + (u & 1)) * 64 : i * 128); };

    const uint32_t ld0 = (warp == 0 && elect_one()) ? 1u : 0u;
    auto issue_q = [&](const Segment& s) {
        const int nq = (s.n_str1 > 0 && !MODE_Y) ? 2 : 1;
        mbar_arrive_expect_tx_if(ld0, &bar->q_full, nq * Q_BYTES);
        for (int t = 0; t < nq; ++t) {
            uint8_t* dst = sQ + t * Q_BYTES;
            tma_load_3d_if(ld0, dst, &tm_qn, &bar->q_full, 0, s.h, s.row0 + t * 128);
            tma_load_3d_if(ld0, dst + Q_SLAB, &tm_qn, &bar->q_full, 64, s.h, s.row0 + t * 128);
            tma_load_3d_if(ld0, dst + 2 * Q_SLAB, &tm_qp, &bar->q_full, 0, s.h, s.row0 + t * 128);
        }
    };
    auto issue_k = [&](const Segment& s, int e, int ring_pos) {
        if (FP8) {   // one 64-token block of codes (as 64 rows of 128 bytes) and its rope keys into a staging slot
            const int sq = ring_pos % p.kq_stages;
            uint8_t* dst = sKq + sq * KQ_BYTES;
            const int blk = tile_of(s, e);
            mbar_arrive_expect_tx_if(ld0, &bar->kq_full[sq], KQ_BYTES);
            tma_load_3d_if(ld0, dst, &tm_kn, &bar->kq_full[sq], 0, blk * 64, s.h);
            tma_load_2d_if(ld0, dst + 8192, &tm_kp, &bar->kq_full[sq], 0, blk * 64);
            return;
        }
        const int st = ring_pos % p.k_stages;
        uint8_t* dst = sK + st * K_TILE_BYTES;
        const int blk0 = tile_of(s, e) * BLK;
        mbar_arrive_expect_tx_if(ld0, &bar->k_full[st], K_TILE_BYTES);
#pragma unroll
        for (int bi = 0; bi < BLK; ++bi) {
            const int gb = s.h * (p.Ls_pad / 64) + blk0 + bi;
            tma_load_3d_if(ld0, dst + bi * 8192, &tm_kn, &bar->k_full[st], 0, 0, gb);
            tma_load_3d_if(ld0, dst + K_SLAB + bi * 8192, &tm_kn, &bar->k_full[st], 0, 64, gb);
            tma_load_2d_if(ld0, dst + 2 * K_SLAB + bi * 8192, &tm_kp, &bar->k_full[st], 0, (blk0 + bi) * 64);
        }
    };
    auto issue_v = [&](const Segment& s, int e, int ring_pos, uint32_t ld) {
        if (FP8) {
            const int sq = ring_pos % p.vq_stages;
            mbar_arrive_expect_tx_if(ld, &bar->vq_full[sq], VQ_BYTES);
            tma_load_3d_if(ld, sVq + sq * VQ_BYTES, &tm_vt, &bar->vq_full[sq], 0, tile_of(s, e) * 64, s.h);
            return;
        }
        const int st = ring_pos % p.v_stages;
        const int blk0 = tile_of(s, e) * BLK;
        mbar_arrive_expect_tx_if(ld, &bar->v_full[st], V_TILE_BYTES);
#pragma unroll
        for (int bi = 0; bi < BLK; ++bi)
            tma_load_4d_if(ld, sV + st * V_TILE_BYTES + bi * 16384, &tm_vt, &bar->v_full[st], 0, 0, blk0 + bi, s.h);
    };

    // Warp 0 initialises the barriers (one per lane) and at once issues the first segment's Q and
    // first K tiles; warp 2 fetches the tensor maps while the barriers are set up and then issues the
    // first V tiles.  The first copies are thus in flight while the rest of the CTA sets up.
    const uint32_t ld2 = (warp == 2 && elect_one()) ? 1u : 0u;
    int n_pre_k = 0, n_pre_v = 0;
    if (g_begin < g_end) {
        const Segment s0 = segment_at(g_begin);
        n_pre_k = min(k_depth, s0.cnt);
        n_pre_v = min(v_depth, s0.cnt);
        if (warp == 2) {
            if (lane == 0) prefetch_tmap(&tm_qn);
            if (lane == 1) prefetch_tmap(&tm_qp);
            if (lane == 2) prefetch_tmap(&tm_kn);
            if (lane == 3) prefetch_tmap(&tm_kp);
            if (lane == 4) prefetch_tmap(&tm_vt);
            asm volatile("bar.sync 1, 64;\n" ::: "memory");   // warp 0 has initialised the barriers
            asm volatile("bar.sync 2, 64;\n" ::: "memory");   // ... and issued Q and the first K tile (needed first)
            for (int e = 0; e < n_pre_v; ++e) issue_v(s0, e, e, ld2);
        }
        if (warp == 0) {
            // the mbarriers are the leading uint64_t members of the struct; p_ready and o_free count the
            // 128 threads of a softmax warpgroup, all others one arrival
            uint64_t* all = &bar->q_full;
            constexpr int n_bars = (int)(offsetof(Barriers, tmem_base) / sizeof(uint64_t));
            for (int i = lane; i < n_bars; i += 32) {
                uint64_t* m = all + i;
                const bool wg = (m >= &bar->p_ready[0][0] && m < &bar->sbuf_free[0][0]) || (m >= &bar->o_free[0] && m < &bar->o_done[0][0]);   // o_free, merge_ready
                mbar_init(m, wg ? 128 : 1);
            }
            if (lane == 0) bar->abort_flag = 0;
            fence_mbar_init();
            __syncwarp();
            asm volatile("bar.sync 1, 64;\n" ::: "memory");
            issue_q(s0);
            issue_k(s0, 0, 0);
            asm volatile("bar.sync 2, 64;\n" ::: "memory");
            for (int e = 1; e < n_pre_k; ++e) issue_k(s0, e, e);
        }
    } else if (threadIdx.x == 0) {
        bar->abort_flag = 0;
    }
    if (warp == 1) tmem_alloc(&bar->tmem_base, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // broadcast through a shuffle so that the compiler knows the value is warp-uniform
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, bar->tmem_base, 0);

    int k_issued = 0, v_issued = 0, q_issued = 0;   // producer warps: copies issued (upper bounds), for the abort path
    if (warp == 0) {
        // ---------------- Q + K producer
        int ring = 0, seg = 0;
        bool ok = true;
        for (int g = g_begin; g < g_end && ok; ++seg) {
            const Segment s = segment_at(g);
            // K tiles first (they only need free ring slots), so that they are in flight while the
            // previous segment's last S products still hold the Q tile
            const int head_k = min(s.cnt, k_depth);
            uint64_t* const k_slot_free = FP8 ? bar->kq_empty : bar->k_empty;   // ring the K copies land in
            int e = 0;
            for (; e < head_k && ok; ++e, ++ring) {
                if (ring < n_pre_k) continue;                 // issued before the setup barrier
                ok = mbar_wait_warp(&k_slot_free[ring % k_depth], ((ring / k_depth) & 1) ^ 1, abort_flag);
                if (ok) issue_k(s, e, ring);
            }
            if (seg > 0 && ok) {
                ok = mbar_wait_warp(&bar->q_free, (seg - 1) & 1, abort_flag);   // previous segment's S products done
                if (ok) issue_q(s);
            }
            for (; e < s.cnt && ok; ++e, ++ring) {
                ok = mbar_wait_warp(&k_slot_free[ring % k_depth], ((ring / k_depth) & 1) ^ 1, abort_flag);
                if (ok) issue_k(s, e, ring);
            }
            g += s.cnt;
        }
        k_issued = ring;
        q_issued = max(seg, 1);
    } else if (warp == 2) {
        // ---------------- V producer
        const uint32_t ld = ld2;
        int ring = 0;
        bool ok = true;
        for (int g = g_begin; g < g_end && ok;) {
            const Segment s = segment_at(g);
            for (int e = 0; e < s.cnt && ok; ++e, ++ring) {
                if (ring < n_pre_v) continue;                 // issued before the setup barrier
                uint64_t* const v_slot_free = FP8 ? bar->vq_empty : bar->v_empty;
                ok = mbar_wait_warp(&v_slot_free[ring % v_depth], ((ring / v_depth) & 1) ^ 1, abort_flag);
                if (ok) issue_v(s, e, ring, ld);
            }
            g += s.cnt;
        }
        v_issued = ring;
    } else if (warp == 1) {
        // ---------------- S = Q K^T issuer.  With two S buffers per stream it runs ahead of the softmax by
        // up to two steps; with one it follows the PV product of the previous step.
        const uint32_t ld = elect_one() ? 1u : 0u;
        constexpr uint32_t idesc_s = idesc_bf16(M64 ? 64 : 128, TOK, false, false);
        constexpr uint32_t idesc_s_nope = FP8 ? idesc_f16(M64 ? 64 : 128, TOK, false, false) : idesc_s;
        int ring_base = 0, seg = 0;
        int used0 = 0, used1 = 0;                              // S-buffer uses so far, per stream
        bool ok = true;
        for (int g = g_begin; g < g_end && ok; ++seg) {
            const Segment s = segment_at(g);
            ok = mbar_wait_warp(&bar->q_full, seg & 1, abort_flag);
            if (FP8 && ok) ok = mbar_wait_warp(&bar->q_conv, seg & 1, abort_flag);   // nope part converted to half precision
            for (int j = 0; j < s.n_str0 && ok; ++j) {
                for (int i = 0; i < 2 && ok; ++i) {
                    if (j >= (i == 0 ? s.n_str0 : s.n_str1)) continue;
                    const int ring = ring_base + entry_of(j, i);
                    const int st = ring % p.k_stages;
                    // Awaited: the K tile (mode X: stream 1 reuses stream 0's), with the 8-bit cache also the staging slot
                    // whose rope keys the product reads, and, from the NB-th use on, the PV product that read P from this
                    // S buffer NB uses ago.  The barriers are tested together: each test of a barrier costs about 200
                    // clocks even when its phase is complete, and this warp's loop is the pace of the 64-token kernels.
                    const int u = (i == 0 ? used0 : used1) + j;
                    const bool need_k = MODE_Y || i == 0, need_s = u >= NB;
                    uint64_t* const kf = &bar->k_full[st];
                    uint64_t* const kq = &bar->kq_full[FP8 ? ring % p.kq_stages : 0];
                    uint64_t* const sf = &bar->sbuf_free[i][u % NB];
                    const uint32_t kf_par = (ring / p.k_stages) & 1, kq_par = FP8 ? (ring / p.kq_stages) & 1 : 0;
                    const uint32_t sf_par = ((u / NB) - 1) & 1;
                    if (need_k && need_s)
                        ok = FP8 ? mbar_wait3_warp(kf, kf_par, kq, kq_par, sf, sf_par, abort_flag)
                                 : mbar_wait2_warp(kf, kf_par, sf, sf_par, abort_flag);
                    else if (need_k)
                        ok = FP8 ? mbar_wait2_warp(kf, kf_par, kq, kq_par, abort_flag) : mbar_wait_warp(kf, kf_par, abort_flag);
                    else if (need_s)
                        ok = mbar_wait_warp(sf, sf_par, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t qa = smem_u32(sQ + (MODE_Y ? 0 : i) * Q_BYTES);
                    const uint32_t ka = smem_u32(sK + st * K_TILE_BYTES);
                    const uint32_t rope = FP8 ? smem_u32(sKq + (ring % p.kq_stages) * KQ_BYTES + 8192) : ka + 2 * K_SLAB;
                    const uint32_t d = tmem_base + s_col(i, u);
                    const bool last_user = MODE_Y || i == 1 || s.n_str1 == 0;
#pragma unroll
                    for (int slab = 0; slab < 3; ++slab) {
                        const uint64_t da = smem_desc_k_sw128(qa + slab * Q_SLAB);
                        const uint64_t db = smem_desc_k_sw128(slab == 2 ? rope : ka + slab * K_SLAB);
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            umma_ss_if(ld, d, da + 2 * k, db + 2 * k, slab == 2 ? idesc_s : idesc_s_nope, (slab | k) != 0);
                    }
                    umma_commit_if(ld, &bar->s_ready[i][u % NB]);
                    if (last_user) umma_commit_if(ld, &bar->k_empty[st]);   // last user releases the ring slot
                    if (FP8) umma_commit_if(ld, &bar->kq_empty[ring % p.kq_stages]);   // ... and the staging slot (rope keys read, codes widened before)
                }
            }
            umma_commit_if(ld, &bar->q_free);                     // the Q tile may be replaced
            used0 += s.n_str0;
            used1 += s.n_str1;
            ring_base += s.cnt;
            g += s.cnt;
        }
    } else if (warp == 3) {
        // ---------------- O += P V issuer
        const uint32_t ld = elect_one() ? 1u : 0u;
        constexpr uint32_t idesc_o = FP8 ? idesc_f16(M64 ? 64 : 128, 128, false, false) : idesc_bf16(M64 ? 64 : 128, 128, false, false);
        int ring_base = 0, seg = 0;
        int used0 = 0, used1 = 0;
        bool ok = true;
        for (int g = g_begin; g < g_end && ok; ++seg) {
            const Segment s = segment_at(g);
            for (int j = 0; j < s.n_str0 && ok; ++j) {
                for (int i = 0; i < 2 && ok; ++i) {
                    if (j >= (i == 0 ? s.n_str0 : s.n_str1)) continue;
                    const int ring = ring_base + entry_of(j, i);
                    const int st = ring % p.v_stages;
                    // the V tile and the probabilities, tested together (see the S issuer)
                    const int u = (i == 0 ? used0 : used1) + j;
                    uint64_t* const pf = MODE_Y ? &bar->p_ready[i][u % NB] : &bar->p_half[i];
                    const uint32_t pf_par = MODE_Y ? (u / NB) & 1 : u & 1;
                    if (MODE_Y || i == 0) ok = mbar_wait2_warp(&bar->v_full[st], (ring / p.v_stages) & 1, pf, pf_par, abort_flag);
                    else ok = mbar_wait_warp(pf, pf_par, abort_flag);
                    if (!ok) break;
                    if (j == 0 && seg > 0) {   // the previous segment's epilogue has read this accumulator
                        ok = mbar_wait_warp(&bar->o_free[i], (seg - 1) & 1, abort_flag);
                        if (!ok) break;
                    }
                    tc_fence_after();
                    const uint32_t va = smem_u32(sV + st * V_TILE_BYTES);
                    const uint32_t pa = tmem_base + s_col(i, u);
                    const uint32_t d = tmem_base + 256u + (uint32_t)i * 128u;
                    const bool last_user = MODE_Y || i == 1 || s.n_str1 == 0;
#pragma unroll
                    for (int bi = 0; bi < BLK; ++bi) {
                        if (bi == 1) {   // second 64 tokens of a 128-token tile: the rest of the probabilities
                            ok = mbar_wait_warp(&bar->p_ready[i][u % NB], (u / NB) & 1, abort_flag);
                            if (!ok) break;
                            tc_fence_after();
                        }
                        const uint64_t db = smem_desc_k_sw128(va + bi * 16384);
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            umma_ts_if(ld, d, pa + 8 * (bi * 4 + k), db + 2 * k, idesc_o, (j | bi | k) != 0);
                    }
                    if (!ok) break;
                    umma_commit_if(ld, &bar->o_done[i][u & 1]);
                    umma_commit_if(ld, &bar->sbuf_free[i][u % NB]);
                    if (last_user) umma_commit_if(ld, &bar->v_empty[st]);
                }
            }
            used0 += s.n_str0;
            used1 += s.n_str1;
            ring_base += s.cnt;
            g += s.cnt;
        }
    } else if (warp >= 4 && warp < 12) {
        // ---------------- softmax warpgroups
        const int i = (warp - 4) >> 2;            // stream
        const int lg = (warp & 3) * 32;           // TMEM lane group of this warp
        const int r = lg + lane;                  // this thread's tensor-memory lane
        // query row of this thread within the tile: the lane itself, or, with M = 64 accumulators, 16 rows in
        // the first 16 lanes of every 32-lane group (the other lanes hold no row; they only keep in step)
        const bool lane_has_row = !M64 || lane < 16;
        const int row = M64 ? (warp & 3) * 16 + lane : r;
        int used = 0;                             // S-buffer uses (= PV products) of this stream so far
        int segi = 0;                             // segments finished by this CTA
        bool ok = true;
        for (int g = g_begin; g < g_end && ok;) {
            const Segment s = segment_at(g);
            const int tile_row0 = s.row0 + (MODE_Y ? 0 : i * 128);
            const int b = lane_has_row ? tile_row0 + row : 0x3fffffff;
            const int nt = i == 0 ? s.n_str0 : s.n_str1;
            const bool warp_has_rows = tile_row0 + (M64 ? (warp & 3) * 16 : lg) < p.B;   // warp-uniform: the warp's first row is a real request
            float m_ref = -INFINITY, m_ref_b = -INFINITY;   // (M = 64: reference exponents of this thread's rows A and B)
            uint64_t l_sum2 = pack_f32x2(0.f, 0.f), l_sum2b = pack_f32x2(0.f, 0.f);   // row sum of the probabilities, as four partial sums
            // (8-bit cache: the accumulated logits are the true ones divided by the scale of this head's K, see below)
            const float scale_l2 = FP8 ? p.scale_log2 * p.mult[s.h] : p.scale_log2;
            const uint64_t scale2 = pack_f32x2(scale_l2, scale_l2);
            for (int j = 0; j < nt && ok; ++j) {
                const int u = used + j;
                const int buf = u % NB;
                ok = __all_sync(0xffffffffu, mbar_wait(&bar->s_ready[i][buf], (u / NB) & 1, abort_flag));
                if (!ok) break;
                tc_fence_after();
                if (!warp_has_rows) {
                    // all 32 rows of this warp are padding past B: their P rows may hold anything (rows of
                    // the MMA are independent and these output rows are never stored); just keep in step
                    tc_fence_before();
                    if (!MODE_Y) mbar_arrive(&bar->p_half[i]);
                    mbar_arrive(&bar->p_ready[i][buf]);
                    continue;
                }
                const uint32_t s_addr = tmem_base + ((uint32_t)lg << 16) + s_col(i, u);
                const int tile = tile_of(s, entry_of(j, i));
                const int valid = min(TOK, p.Ls - tile * TOK);
                if (M64) {
                    // M = 64 accumulators: the warp's 16 rows sit in the first 16 lanes of its lane group.  They are
                    // read as fragments, so that all 32 threads work: thread t holds 16 of the 64 logits of row
                    // t/4 ("A") and of row t/4 + 8 ("B"), in column pairs 8g + 2(t%4) + {0, 1}, which are exactly the
                    // token pairs that share a packed P column (4g + t%4).  Row maxima need two shuffles within the
                    // four threads of a row; row sums stay per thread until the end of the segment.
                    uint32_t sr[32];
                    tmem_ld_16x256b_x8(s_addr, sr);
                    tmem_ld_wait();
                    const int q4 = lane & 3;
                    if (valid < TOK) {
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (8 * (c >> 2) + 2 * q4 + (c & 1) >= valid) sr[c] = 0xff800000u;   // -inf
                    }
                    float mxa = -INFINITY, mxb = -INFINITY, mxa2 = -INFINITY, mxb2 = -INFINITY;
#pragma unroll
                    for (int gq = 0; gq < 8; gq += 2) {
                        mxa = max3(mxa, __uint_as_float(sr[4 * gq]), __uint_as_float(sr[4 * gq + 1]));
                        mxb = max3(mxb, __uint_as_float(sr[4 * gq + 2]), __uint_as_float(sr[4 * gq + 3]));
                        mxa2 = max3(mxa2, __uint_as_float(sr[4 * gq + 4]), __uint_as_float(sr[4 * gq + 5]));
                        mxb2 = max3(mxb2, __uint_as_float(sr[4 * gq + 6]), __uint_as_float(sr[4 * gq + 7]));
                    }
                    mxa = fmaxf(mxa, mxa2);
                    mxb = fmaxf(mxb, mxb2);
                    mxa = fmaxf(mxa, __shfl_xor_sync(0xffffffffu, mxa, 1));
                    mxb = fmaxf(mxb, __shfl_xor_sync(0xffffffffu, mxb, 1));
                    mxa = fmaxf(mxa, __shfl_xor_sync(0xffffffffu, mxa, 2)) * scale_l2;
                    mxb = fmaxf(mxb, __shfl_xor_sync(0xffffffffu, mxb, 2)) * scale_l2;
                    // lazy rescale: only when some row's maximum grew by more than 2^8
                    const bool grow_a = mxa > m_ref + 8.f, grow_b = mxb > m_ref_b + 8.f;
                    if (j == 0) {
                        m_ref = mxa;
                        m_ref_b = mxb;
                    } else if (__any_sync(0xffffffffu, grow_a || grow_b)) {
                        // the previous PV of this stream must have landed before O is touched
                        ok = __all_sync(0xffffffffu, mbar_wait(&bar->o_done[i][(u - 1) & 1], ((u - 1) >> 1) & 1, abort_flag));
                        if (!ok) break;
                        tc_fence_after();
                        const float fa = grow_a ? fast_exp2(m_ref - mxa) : 1.f, fb = grow_b ? fast_exp2(m_ref_b - mxb) : 1.f;
                        if (grow_a) m_ref = mxa;
                        if (grow_b) m_ref_b = mxb;
                        l_sum2 = mul_f32x2(l_sum2, pack_f32x2(fa, fa));
                        l_sum2b = mul_f32x2(l_sum2b, pack_f32x2(fb, fb));
                        // the accumulator is rescaled row by row through the one-lane-per-thread shape: lane l < 16 of
                        // the group holds row l, whose factor lives in the threads 4 (l % 8) .. + 3 (A for l < 8, else B)
                        const float va = __shfl_sync(0xffffffffu, fa, 4 * (lane & 7)), vb = __shfl_sync(0xffffffffu, fb, 4 * (lane & 7));
                        const float f = (lane & 8) ? vb : va;
                        const uint32_t o_addr = tmem_base + ((uint32_t)lg << 16) + 256u + (uint32_t)i * 128u;
#pragma unroll 1
                        for (int c = 0; c < 4; ++c) {
                            uint32_t orr[32];
                            tmem_ld32(o_addr + c * 32, orr);
                            tmem_ld_wait();
#pragma unroll
                            for (int qq = 0; qq < 32; ++qq) orr[qq] = __float_as_uint(__uint_as_float(orr[qq]) * f);
                            tmem_st32(o_addr + c * 32, orr);
                        }
                        tmem_st_wait();
                    }
                    const uint64_t nma = pack_f32x2(-m_ref, -m_ref), nmb = pack_f32x2(-m_ref_b, -m_ref_b);
                    uint32_t pk[16];
#pragma unroll
                    for (int gq = 0; gq < 8; ++gq) {
                        float x0, x1, y0, y1;
                        unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(sr[4 * gq]), __uint_as_float(sr[4 * gq + 1])), scale2, nma), x0, x1);
                        unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(sr[4 * gq + 2]), __uint_as_float(sr[4 * gq + 3])), scale2, nmb), y0, y1);
                        const float pa0 = fast_exp2(x0), pa1 = fast_exp2(x1), pb0 = fast_exp2(y0), pb1 = fast_exp2(y1);
                        // (8-bit cache: V is converted to half precision, so the probabilities are too)
                        pk[2 * gq] = FP8 ? pack_f16(pa0, pa1) : pack_bf16(pa0, pa1);          // row A, P column 4 gq + t%4
                        pk[2 * gq + 1] = FP8 ? pack_f16(pb0, pb1) : pack_bf16(pb0, pb1);      // row B, same column
                        l_sum2 = add_f32x2(l_sum2, pack_f32x2(pa0, pa1));
                        l_sum2b = add_f32x2(l_sum2b, pack_f32x2(pb0, pb1));
                    }
                    tmem_st_16x128b_x8(s_addr, pk);
                    tmem_st_wait();
                    tc_fence_before();
                    mbar_arrive(&bar->p_ready[i][buf]);
                    continue;
                }
                // pass 1: row maximum of the raw logits (the scale is positive, so it commutes with the
                // maximum); the ragged tail is masked with -inf in place
                // (four independent running maxima and, below, two pairs of running sums: the tile's softmax is one
                // link of the chain S product -> softmax -> PV product -> next S product of its stream, so the length
                // of its dependent instruction chains counts, not only the number of instructions)
                float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
                uint32_t sr[2][32];
#pragma unroll
                for (int half = 0; half < BLK; ++half) {
                    tmem_ld32(s_addr + half * 64, sr[0]);
                    tmem_ld32(s_addr + half * 64 + 32, sr[1]);
                    tmem_ld_wait();
                    if (valid < TOK) {
#pragma unroll
                        for (int c = 0; c < 64; ++c)
                            if (half * 64 + c >= valid) sr[c >> 5][c & 31] = 0xff800000u;   // -inf
                    }
#pragma unroll
                    for (int c = 0; c < 64; c += 2)
                        mx4[(c >> 1) & 3] = max3(mx4[(c >> 1) & 3], __uint_as_float(sr[c >> 5][c & 31]),
                                                 __uint_as_float(sr[(c + 1) >> 5][(c + 1) & 31]));
                }
                const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * scale_l2;
                // lazy rescale: only when some row's maximum grew by more than 2^8
                const bool grow = lane_has_row && mx > m_ref + 8.f;
                if (j == 0) {
                    m_ref = mx;
                } else if (__any_sync(0xffffffffu, grow)) {
                    // the previous PV of this stream must have landed before O is touched
                    ok = __all_sync(0xffffffffu, mbar_wait(&bar->o_done[i][(u - 1) & 1], ((u - 1) >> 1) & 1, abort_flag));
                    if (!ok) break;
                    tc_fence_after();
                    const float m_new = grow ? mx : m_ref;
                    const float f = fast_exp2(m_ref - m_new);
                    m_ref = m_new;
                    l_sum2 = mul_f32x2(add_f32x2(l_sum2, l_sum2b), pack_f32x2(f, f));
                    l_sum2b = pack_f32x2(0.f, 0.f);
                    const uint32_t o_addr = tmem_base + ((uint32_t)lg << 16) + 256u + (uint32_t)i * 128u;
#pragma unroll 1
                    for (int c = 0; c < 4; ++c) {
                        uint32_t orr[32];
                        tmem_ld32(o_addr + c * 32, orr);
                        tmem_ld_wait();
#pragma unroll
                        for (int q = 0; q < 32; ++q) orr[q] = __float_as_uint(__uint_as_float(orr[q]) * f);
                        tmem_st32(o_addr + c * 32, orr);
                    }
                    tmem_st_wait();
                }
                // pass 2: p = 2^(s * scale - m_ref) (one FMA and one ex2 per element), packed to bf16 over
                // the S columns (P column c holds tokens 2c, 2c+1); with 128-token tiles the logits are read
                // again, 64 at a time, to stay within the register budget
                const uint64_t neg_m2 = pack_f32x2(-m_ref, -m_ref);
                // probabilities of 32 logits held in `src`: 16 packed bf16 pairs, sums into the four partial sums
                auto probs32 = [&](const uint32_t (&src)[32], uint32_t (&dst)[16]) {
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        // two logits per instruction: distance to the reference exponent, probabilities, running sums
                        float x0, x1;
                        unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(src[2 * c]), __uint_as_float(src[2 * c + 1])), scale2, neg_m2), x0, x1);
                        float p0, p1;
                        if ((kPolyExpMask >> (c & 7)) & 1) {
                            exp2_poly_x2(x0, x1, p0, p1);
                        } else {
                            p0 = fast_exp2(x0);
                            p1 = fast_exp2(x1);
                        }
                        dst[c] = FP8 ? pack_f16(p0, p1) : pack_bf16(p0, p1);
                        if (c & 1) l_sum2b = add_f32x2(l_sum2b, pack_f32x2(p0, p1));
                        else l_sum2 = add_f32x2(l_sum2, pack_f32x2(p0, p1));
                    }
                };
                if (BLK == 1) {
                    // the 64 logits of pass 1 are still in registers
                    uint32_t pk[2][16];
                    probs32(sr[0], pk[0]);
                    tmem_st16(s_addr, pk[0]);
                    probs32(sr[1], pk[1]);
                    tmem_st16(s_addr + 16, pk[1]);
                } else {
                    // 128-token tiles: the logits are read again, 32 at a time with the next 32 already requested, to stay
                    // within the register budget.  Quarter q covers S columns [32 q, 32 q + 32) and writes P columns
                    // [16 q, 16 q + 16): those overlap only S columns that are already in registers or consumed.
                    tmem_ld32(s_addr, sr[0]);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        tmem_ld_wait();
                        if (q < 3) tmem_ld32(s_addr + (q + 1) * 32, sr[(q + 1) & 1]);
                        if (valid < TOK) {
#pragma unroll
                            for (int c = 0; c < 32; ++c)
                                if (q * 32 + c >= valid) sr[q & 1][c] = 0xff800000u;
                        }
                        uint32_t pk[16];
                        probs32(sr[q & 1], pk);
                        tmem_st16(s_addr + q * 16, pk);
                        if (q == 1) {   // first half of the tile's probabilities in place
                            tmem_st_wait();
                            tc_fence_before();
                            mbar_arrive(&bar->p_half[i]);
                        }
                    }
                }
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(&bar->p_ready[i][buf]);
            }
            if (!ok) break;
            float l_sum;
            if (M64) {
                // this thread's partial sums of rows A and B -> whole-row sums (four threads per row), then the values
                // of the row that the one-lane-per-thread epilogue below handles in this lane: lane l < 16 holds row l
                float a0, a1, b0, b1;
                unpack_f32x2(l_sum2, a0, a1);
                unpack_f32x2(l_sum2b, b0, b1);
                float la = a0 + a1, lb = b0 + b1;
                la += __shfl_xor_sync(0xffffffffu, la, 1);
                lb += __shfl_xor_sync(0xffffffffu, lb, 1);
                la += __shfl_xor_sync(0xffffffffu, la, 2);
                lb += __shfl_xor_sync(0xffffffffu, lb, 2);
                const int src = 4 * (lane & 7);
                const float la_r = __shfl_sync(0xffffffffu, la, src), lb_r = __shfl_sync(0xffffffffu, lb, src);
                const float ma_r = __shfl_sync(0xffffffffu, m_ref, src), mb_r = __shfl_sync(0xffffffffu, m_ref_b, src);
                l_sum = (lane & 8) ? lb_r : la_r;
                m_ref = (lane & 8) ? mb_r : ma_r;
            } else {
                float a, c;
                unpack_f32x2(add_f32x2(l_sum2, l_sum2b), a, c);
                l_sum = a + c;
            }
            // ---- segment epilogue: normalised partial + LSE into this segment's slot.  With 64-token tiles the two
            // streams worked on the same query rows: stream 1 publishes its softmax state, stream 0 merges both
            // accumulators (same tensor-memory lanes) and writes one partial.
            const int slot = s.slot_seg;
            const bool owns_rows = MODE_Y ? i == 0 : (i == 0 || s.row0 + 128 < p.B);
            if (nt > 0) {
                const int u_last = used + nt - 1;
                ok = __all_sync(0xffffffffu, mbar_wait(&bar->o_done[i][u_last & 1], (u_last >> 1) & 1, abort_flag));
                if (!ok) break;
                tc_fence_after();
            }
            if (MODE_Y && i == 1) {
                if (segi > 0) {   // stream 0 has read what the previous segment published (it frees O1 after that)
                    ok = __all_sync(0xffffffffu, mbar_wait(&bar->o_free[1], (segi - 1) & 1, abort_flag));
                    if (!ok) break;
                }
                bar->merge_m[r] = nt > 0 ? m_ref : -INFINITY;
                bar->merge_l[r] = nt > 0 ? l_sum : 0.f;
                tc_fence_before();
                mbar_arrive(&bar->merge_ready);
            } else {
                float a0 = 0.f, a1 = 0.f, lse2 = -INFINITY;   // weights of the two accumulators, LSE in base 2
                if (MODE_Y) {
                    ok = __all_sync(0xffffffffu, mbar_wait(&bar->merge_ready, segi & 1, abort_flag));
                    if (!ok) break;
                    tc_fence_after();
                    const float m1 = bar->merge_m[r], l1 = bar->merge_l[r];
                    const float m = fmaxf(m_ref, m1);           // stream 0 always has a tile: m_ref is finite
                    const float e0 = fast_exp2(m_ref - m), e1 = l1 > 0.f ? fast_exp2(m1 - m) : 0.f;
                    const float l = l_sum * e0 + l1 * e1;
                    a0 = e0 / l;
                    a1 = e1 / l;
                    lse2 = m + log2f(l);
                } else if (nt > 0) {
                    a0 = 1.f / l_sum;
                    lse2 = m_ref + log2f(l_sum);
                }
                if (FP8) {   // the accumulators hold P times the V codes' values: the true values divided by the scale
                    const float vm = p.mult[p.H + s.h];
                    a0 *= vm;
                    a1 *= vm;
                }
                if (nt > 0 && warp_has_rows) {
                    const uint32_t o_addr = tmem_base + ((uint32_t)lg << 16) + 256u + (uint32_t)(MODE_Y ? 0 : i) * 128u;
                    float* dst = p.o_part + (((int64_t)slot * p.part_rows + b) * p.H + s.h) * 128;
#pragma unroll 1
                    for (int c = 0; c < 4; ++c) {
                        uint32_t orr[32];
                        tmem_ld32(o_addr + c * 32, orr);
                        tmem_ld_wait();
                        float v[32];
#pragma unroll
                        for (int q = 0; q < 32; ++q) v[q] = __uint_as_float(orr[q]) * a0;
                        if (MODE_Y && s.n_str1 > 0) {   // uniform over the CTA (the tensor-memory load is warp-collective)
                            tmem_ld32(o_addr + 128u + c * 32, orr);
                            tmem_ld_wait();
#pragma unroll
                            for (int q = 0; q < 32; ++q) v[q] = fmaf(__uint_as_float(orr[q]), a1, v[q]);
                        }
                        if (b < p.B) {
#pragma unroll
                            for (int q = 0; q < 8; ++q)
                                *reinterpret_cast<float4*>(dst + c * 32 + 4 * q) = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                        }
                    }
                    if (b < p.B) p.lse_part[((int64_t)slot * p.part_rows + b) * p.H + s.h] = lse2 * kLn2;
                } else if (nt == 0 && owns_rows && b < p.B) {
                    p.lse_part[((int64_t)slot * p.part_rows + b) * p.H + s.h] = -INFINITY;   // this stream had no tile
                }
                // the segment that ends a head marks the head's unused slots as empty
                if (s.last_of_col && owns_rows && b < p.B) {
                    for (int ss = s.slot_seg + 1; ss < p.n_seg_max; ++ss)
                        p.lse_part[((int64_t)ss * p.part_rows + b) * p.H + s.h] = -INFINITY;
                }
                // the accumulator(s) just read may be overwritten by the next segment
                tc_fence_before();
                mbar_arrive(&bar->o_free[i]);
                if (MODE_Y) mbar_arrive(&bar->o_free[1]);
            }
            ++segi;
            used += nt;
            g += s.cnt;
        }
    } else if (FP8) {
        // ---------------- conversion warps (8-bit cache only): warps 12-13 for K and the query tile, warps 14-15 for V.
        // The expanded K_nope and V of the prefix are stored as E4M3 codes with one power-of-two scale per head.
        // Bulk copies bring 8 KB blocks of codes into staging slots; these warps rewrite each block as the
        // half-precision operand tile the MMAs read (same 128-byte-swizzled layouts as the 16-bit path).  Every E4M3
        // value is a half-precision value, so widening is exact (one conversion instruction per pair of codes).  The
        // scales go where they cost nothing.  K: the query's nope part is only converted to half precision (once
        // per segment, here), its rope part is divided by the scale (a power of two: exact), so the accumulated
        // logits are the true ones divided by it, and the softmax scale is multiplied by it.  V: into the final
        // normalisation.
        const bool is_v = warp >= 14;
        const int ct = threadIdx.x - (is_v ? 448 : 384);          // 0..63 within the pair of warps
        auto pair_sync = [&] {
            if (is_v) asm volatile("bar.sync 4, 64;\n" ::: "memory");
            else asm volatile("bar.sync 3, 64;\n" ::: "memory");
        };
        // The two warps of a pair must take the same decision before either of them goes to the pair's barrier: one
        // may have seen the abort flag in a wait that the other left through its fast path.
        auto pair_vote_or = [&](bool pred) {
            uint32_t r;
            if (is_v)
                asm volatile("{\n.reg .pred p, q;\nsetp.ne.b32 q, %1, 0;\nbar.red.or.pred p, 4, 64, q;\nselp.u32 %0, 1, 0, p;\n}\n"
                             : "=r"(r) : "r"(pred ? 1u : 0u) : "memory");
            else
                asm volatile("{\n.reg .pred p, q;\nsetp.ne.b32 q, %1, 0;\nbar.red.or.pred p, 3, 64, q;\nselp.u32 %0, 1, 0, p;\n}\n"
                             : "=r"(r) : "r"(pred ? 1u : 0u) : "memory");
            return r != 0;
        };
        auto widen = [](uint32_t w, uint32_t& lo, uint32_t& hi) {
            asm("{\n.reg .b16 a, b;\nmov.b32 {a, b}, %2;\ncvt.rn.f16x2.e4m3x2 %0, a;\ncvt.rn.f16x2.e4m3x2 %1, b;\n}\n"
                : "=r"(lo), "=r"(hi)
                : "r"(w));
        };
        // one 8 KB staging block (64 rows of 128 bytes, 16-byte chunks swizzled by the row) -> 16 KB operand tile.
        // K: row = token, chunk = 16 dims, tile = two [64 tokens][64 dims] slabs.  V: row = two dims (64 tokens
        // each), chunk = 16 tokens of one dim, tile = [128 dims][64 tokens].
        auto convert = [&](const uint8_t* src, uint8_t* dst) {
#pragma unroll
            for (int it = 0; it < 8; ++it) {
                // Eight consecutive lanes take chunks 0-3 of one row and chunks 4-7 of the next (or the other way round):
                // their eight 16-byte reads fall on eight different bank groups, and so do their writes (the two
                // rows' swizzles differ in the lowest bit, the two halves of a K row go to different slabs).
                const int u = it * 64 + ct, j = u & 7, grp = u >> 3;
                const int r = 2 * (grp >> 1) + (j >> 2), c = (j & 3) + 4 * ((j >> 2) ^ (grp & 1));
                const uint4 w = *reinterpret_cast<const uint4*>(src + r * 128 + ((c ^ (r & 7)) << 4));
                uint4 o0, o1;
                widen(w.x, o0.x, o0.y);
                widen(w.y, o0.z, o0.w);
                widen(w.z, o1.x, o1.y);
                widen(w.w, o1.z, o1.w);
                const int row = is_v ? 2 * r + (c >> 2) : r;          // row of the operand tile
                const int slab = is_v ? 0 : (c >> 2);
                const int c0 = 2 * (c & 3);
                uint8_t* d = dst + slab * 8192 + row * 128;
                *reinterpret_cast<uint4*>(d + ((c0 ^ (row & 7)) << 4)) = o0;
                *reinterpret_cast<uint4*>(d + (((c0 + 1) ^ (row & 7)) << 4)) = o1;
            }
        };
        // ring position `ring`: staging slot -> 16-bit slot, then hand both on
        auto convert_tile = [&](int ring) {
            const int q_depth = is_v ? p.vq_stages : p.kq_stages, depth = is_v ? p.v_stages : p.k_stages;
            const int sq = ring % q_depth, st = ring % depth;
            uint64_t* const staged = is_v ? &bar->vq_full[sq] : &bar->kq_full[sq];
            uint64_t* const slot_free = is_v ? &bar->v_empty[st] : &bar->k_empty[st];
            // (both barriers tested together first: in the steady state both phases are complete)
            bool ok = __all_sync(0xffffffffu, mbar_try_wait2(staged, (ring / q_depth) & 1, slot_free, ((ring / depth) & 1) ^ 1));
            if (!ok) {
                ok = __all_sync(0xffffffffu, mbar_wait(staged, (ring / q_depth) & 1, abort_flag));
                ok = ok && __all_sync(0xffffffffu, mbar_wait(slot_free, ((ring / depth) & 1) ^ 1, abort_flag));
            }
            if (pair_vote_or(!ok)) return false;
            if (is_v) convert(sVq + sq * VQ_BYTES, sV + st * V_TILE_BYTES);
            else convert(sKq + sq * KQ_BYTES, sK + st * K_TILE_BYTES);
            fence_proxy_async();   // the MMAs read the tile through the async proxy
            pair_sync();
            if (ct == 0) {
                mbar_arrive(is_v ? &bar->v_full[st] : &bar->k_full[st]);
                // A K staging slot is released by the logits product that reads its rope keys: that product waits for
                // this tile's k_full, so it cannot complete before the codes have been read.
                if (is_v) mbar_arrive(&bar->vq_empty[sq]);
            }
            return true;
        };
        int ring_base = 0, seg = 0;
        bool ok = true;
        for (int g = g_begin; g < g_end && ok; ++seg) {
            const Segment s = segment_at(g);
            if (!is_v) {
                // query tile (three slabs): nope part to half precision, rope part divided by the K scale
                ok = !pair_vote_or(!__all_sync(0xffffffffu, mbar_wait(&bar->q_full, seg & 1, abort_flag)));
                if (!ok) break;
                const float inv_ks = __fdiv_rn(1.f, p.mult[s.h]);   // a power of two: exact
#pragma unroll
                constexpr int N_IT = Q_BYTES / 16 / 64;   // 16-byte pieces per thread; the first two thirds are the nope slabs
#pragma unroll 8
                for (int it = 0; it < N_IT; ++it) {
                    uint4* qv = reinterpret_cast<uint4*>(sQ) + it * 64 + ct;
                    uint4 w = *qv;
                    uint32_t* e = reinterpret_cast<uint32_t*>(&w);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const float2 f = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&e[k]));
                        e[k] = it < 2 * N_IT / 3 ? pack_f16(f.x, f.y) : pack_bf16(f.x * inv_ks, f.y * inv_ks);
                    }
                    *qv = w;
                }
                fence_proxy_async();
                pair_sync();
                if (ct == 0) mbar_arrive(&bar->q_conv);
            }
            for (int e = 0; e < s.cnt && ok; ++e) ok = convert_tile(ring_base + e);
            ring_base += s.cnt;
            g += s.cnt;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // A wait gave up.  Before the CTA's shared memory is released, each producer warp waits (with a limit) on the
        // barriers of the ring positions it issued last: the copies against them are the only ones that can still be
        // in flight.
        if (warp == 0 && g_begin < g_end) {
            uint64_t* const k_landed = FP8 ? bar->kq_full : bar->k_full;
            for (int pos = max(0, k_issued - k_depth); pos < k_issued; ++pos)
                mbar_drain(&k_landed[pos % k_depth], (pos / k_depth) & 1);
            mbar_drain(&bar->q_full, (q_issued - 1) & 1);
        }
        if (warp == 2 && g_begin < g_end) {
            uint64_t* const v_landed = FP8 ? bar->vq_full : bar->v_full;
            for (int pos = max(0, v_issued - v_depth); pos < v_issued; ++pos)
                mbar_drain(&v_landed[pos % v_depth], (pos / v_depth) & 1);
        }
        if (threadIdx.x == 0 && p.status) atomicOr(p.status, 2);
        __syncthreads();
    }
    if (warp == 1) tmem_dealloc(tmem_base, 512);
}

}  // namespace


int naive_sm100_tile_tokens(int B, bool fp8) { return (fp8 || B <= 128) ? 64 : 128; }

// Host-side plan (pure function of the sizes): number of tile ranges R and of partial slots.
//
// Two schedules are weighed.  "Column split" cuts every head into ns equal parts (R = H * ns, CTAs
// may run in several waves); ns minimises waves x (tiles per CTA + a fixed cost of about six tile
// times for the Q load and the pipeline fill).  "Stream-K" uses R = SMs / row groups resident
// CTAs and gives every SM the same number of tiles at the price of a few more segments (each
// pays the fixed cost and a partial slot; with 64-token tiles a further slot per head is also charged
// the extra read it causes in the combine).  Stream-K is taken when its modelled cost is lower (by at
// least 5% in the HBM-bound regime of 64-token tiles).
void naive_sm100_plan(int B, int H, int64_t Ls, int n_sm, int schedule, int* n_ranges, int* n_slots, bool fp8) {
    // (8-bit cache: always 64-token tiles, row groups of 128 requests)
    const bool mode_y = fp8 || B <= 128;
    const int tok = mode_y ? 64 : 128;
    const int m_groups = fp8 ? (B + 127) / 128 : (mode_y ? 1 : (B + 255) / 256);
    const int n_tiles = (int)((Ls + tok - 1) / tok);
    const long long T = (long long)H * n_tiles;
    if (T <= 0) {
        *n_ranges = 0;
        *n_slots = 0;
        return;
    }
    // partial slots a head needs when the T tiles are cut into R ranges (ranges [0, rem) hold per + 1 tiles)
    auto slots_for = [&](long long R) {
        const long long per = T / R, rem = T % R, big = rem * (per + 1);
        auto range_of = [&](long long t) { return t < big ? t / (per + 1) : rem + (t - big) / per; };
        int seg_max = 1;
        for (long long h = 0; h < H; ++h) {
            const long long first = h * n_tiles, last = first + n_tiles - 1;
            seg_max = std::max(seg_max, (int)(range_of(last) - range_of(first)) + 1);
        }
        return seg_max;
    };
    // column split
    const long long base = (long long)H * m_groups;
    const double fixed = 6.0;
    // every further partial slot is one more dependent read of B x H x 128 floats in the combine that follows
    // (about 5 us, i.e. 8 tile times, measured with 64-token tiles; not significant next to 128-token tiles)
    const double slot_cost = mode_y ? 8.0 : 0.0;
    int ns_best = 1;
    double cost_best = 1e30, eff_best = 0.0;
    for (int ns = 1; ns <= std::min(n_tiles, 32); ++ns) {
        const int per = (n_tiles + ns - 1) / ns;
        if (n_tiles % ns != 0) continue;   // equal parts only: every range stays inside one head
        const long long waves = (ns * base + n_sm - 1) / n_sm;
        const double cost = (double)waves * (per + fixed) + slot_cost * (ns - 1);
        if (cost < cost_best - 1e-9) {
            cost_best = cost;
            ns_best = ns;
            eff_best = (double)(T * m_groups) / ((double)waves * per * n_sm);
        }
    }
    // stream-K: equal ranges; a CTA meets at most (tiles per range / tiles per head) + 2 segments
    const int r_stream = (int)std::min<long long>(std::max(1, n_sm / m_groups), T);
    const long long per_stream = (T + r_stream - 1) / r_stream;
    const long long waves_stream = ((long long)r_stream * m_groups + n_sm - 1) / n_sm;
    const double segs_stream = (per_stream >= n_tiles) ? (double)per_stream / n_tiles + 1.0 : 2.0;
    const double cost_stream = (double)waves_stream * (per_stream + segs_stream * fixed) + slot_cost * (slots_for(r_stream) - 1);
    bool stream_k;
    if (schedule == 1) stream_k = false;
    else if (schedule == 2) stream_k = true;
    else {
        // With at most 64 query rows a CTA keeps up with its share of HBM: more resident CTAs do not
        // help as long as most SMs are busy, and spare SMs go to the concurrent absorb branch.
        const bool hbm_bound_small = mode_y && B <= 64 && eff_best >= 0.8;
        // 64-token tiles (HBM-bound regime): column split must lose by 5%, since it often leaves SMs to
        // the concurrent absorb branch and writes fewer partials
        stream_k = !hbm_bound_small && cost_stream < (mode_y ? 0.95 : 1.0) * cost_best;
    }
    const int R = stream_k ? r_stream : H * ns_best;
    *n_ranges = R;
    *n_slots = slots_for(R);   // the kernel uses the same partition
}

cudaError_t launch_naive_attn_sm100(const NaiveAttnSm100& a, cudaStream_t s) {
    if (a.B <= 0 || a.Ls <= 0 || a.n_ranges <= 0) return cudaSuccess;
    const bool fp8 = a.fp8_mult != nullptr;
    CUtensorMap tm_qn, tm_qp;
    {
        uint64_t dims[3] = {128, (uint64_t)a.H, (uint64_t)a.B};
        uint64_t str[2] = {128 * 2, (uint64_t)a.H * 128 * 2};
        uint32_t box[3] = {64, 1, (fp8 && a.B <= 64) ? 64u : 128u};
        cudaError_t e = make_tmap_bf16(&tm_qn, a.q_nope, 3, dims, str, box);
        if (e != cudaSuccess) return e;
    }
    {
        uint64_t dims[3] = {64, (uint64_t)a.H, (uint64_t)a.B};
        uint64_t str[2] = {64 * 2, (uint64_t)a.H * 64 * 2};
        uint32_t box[3] = {64, 1, (fp8 && a.B <= 64) ? 64u : 128u};
        cudaError_t e = make_tmap_bf16(&tm_qp, a.q_pe, 3, dims, str, box);
        if (e != cudaSuccess) return e;
    }
    const bool mode_y = fp8 || a.B <= 128;
    const int tok = mode_y ? 64 : 128;
    NaiveSm100Params p{};
    p.B = a.B; p.H = a.H; p.Ls = a.Ls; p.Ls_pad = (a.Ls + 127) / 128 * 128;
    p.part_rows = a.part_rows > 0 ? a.part_rows : a.B;
    p.m_groups = fp8 ? (a.B + 127) / 128 : (mode_y ? 1 : (a.B + 255) / 256);
    p.n_tiles = (a.Ls + tok - 1) / tok;
    p.n_ranges = a.n_ranges;
    {
        const long long T = (long long)a.H * p.n_tiles;
        if (T >= (1LL << 31) || a.n_ranges > T) return cudaErrorInvalidValue;
        p.per = (int)(T / a.n_ranges);
        p.rem = (int)(T % a.n_ranges);
    }
    p.n_seg_max = a.n_slots;
    p.k_stages = fp8 ? (a.B <= 64 ? 3 : 2) : (mode_y ? 4 : 2);   // (8-bit cache: the 128-row query tile takes 24 KB more)
    p.v_stages = fp8 ? (a.B <= 64 ? 3 : 2) : (mode_y ? 4 : 1);
    p.kq_stages = fp8 ? 4 : 0;
    p.vq_stages = fp8 ? 4 : 0;
    p.mult = a.fp8_mult;
    p.scale_log2 = a.scale * kLog2e;
    p.o_part = a.o_part; p.lse_part = a.lse_part; p.status = a.status;
    const int k_tile = fp8 ? 16384 : tok * 384, v_tile = mode_y ? 16384 : 32768;
    const int smem = ((fp8 && a.B <= 64) ? Q_TILE_BYTES / 2 : (mode_y ? 1 : 2) * Q_TILE_BYTES) + p.k_stages * k_tile + p.v_stages * v_tile +
                     p.kq_stages * 16384 + p.vq_stages * 8192 + 1024 + (int)sizeof(Barriers) + 64;
    dim3 grid(p.n_ranges * p.m_groups, 1, 1);
    if (smem > kNaiveSmemMax) return cudaErrorInvalidValue;
    if (fp8) {
        if (a.B <= 64)
            return launch_pdl(naive_attn_sm100_kernel<64, true, true>, grid, dim3(512), smem, s, tm_qn, tm_qp, *a.tm_kn, *a.tm_kp, *a.tm_vt, p);
        return launch_pdl(naive_attn_sm100_kernel<64, false, true>, grid, dim3(512), smem, s, tm_qn, tm_qp, *a.tm_kn, *a.tm_kp, *a.tm_vt, p);
    }
    if (mode_y) {
        if (a.B <= 64)   // half-height MMAs: the padding rows 64..127 of the query tile cost tensor-pipe time and power
            return launch_pdl(naive_attn_sm100_kernel<64, true, false>, grid, dim3(384), smem, s, tm_qn, tm_qp, *a.tm_kn, *a.tm_kp, *a.tm_vt, p);
        return launch_pdl(naive_attn_sm100_kernel<64, false, false>, grid, dim3(384), smem, s, tm_qn, tm_qp, *a.tm_kn, *a.tm_kp, *a.tm_vt, p);
    }
    return launch_pdl(naive_attn_sm100_kernel<128, false, false>, grid, dim3(384), smem, s, tm_qn, tm_qp, *a.tm_kn, *a.tm_kp, *a.tm_vt, p);
}

cudaError_t set_attrs_naive_sm100() {
    cudaError_t e = cudaFuncSetAttribute(naive_attn_sm100_kernel<64, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kNaiveSmemMax);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(naive_attn_sm100_kernel<64, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kNaiveSmemMax);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(naive_attn_sm100_kernel<128, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kNaiveSmemMax);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(naive_attn_sm100_kernel<64, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kNaiveSmemMax);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(naive_attn_sm100_kernel<64, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kNaiveSmemMax);
    return e;
}

cudaError_t make_naive_sm100_tmaps(const void* k_nope, const void* kpe, const void* v_t, int H, int64_t Ls_pad,
                                   CUtensorMap* tm_kn, CUtensorMap* tm_kp, CUtensorMap* tm_vt) {
    {
        // K_nope is stored as contiguous 64-token blocks of two [64 tokens][64 dims] slabs;
        // one box = one slab of one block (8 KB)
        uint64_t dims[3] = {64, 128, (uint64_t)H * (uint64_t)(Ls_pad / 64)};
        uint64_t str[2] = {64 * 2, 128 * 64 * 2};
        uint32_t box[3] = {64, 64, 1};
        cudaError_t e = make_tmap_bf16(tm_kn, k_nope, 3, dims, str, box);
        if (e != cudaSuccess) return e;
    }
    {
        uint64_t dims[2] = {64, (uint64_t)Ls_pad};
        uint64_t str[1] = {64 * 2};
        uint32_t box[2] = {64, 64};
        cudaError_t e = make_tmap_bf16(tm_kp, kpe, 2, dims, str, box);
        if (e != cudaSuccess) return e;
    }
    {
        // V^T is stored in 64-token blocks, each a contiguous [128 dims][64 tokens] matrix
        uint64_t dims[4] = {64, 128, (uint64_t)(Ls_pad / 64), (uint64_t)H};
        uint64_t str[3] = {64 * 2, 128 * 64 * 2, (uint64_t)Ls_pad * 128 * 2};
        uint32_t box[4] = {64, 128, 1, 1};
        cudaError_t e = make_tmap_bf16(tm_vt, v_t, 4, dims, str, box);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t make_naive_fp8_tmaps(const void* k8, const void* kpe, const void* v8, int H, int64_t Ls_pad,
                                 CUtensorMap* tm_k8, CUtensorMap* tm_kp, CUtensorMap* tm_v8) {
    // Both code arrays are [H][Ls_pad rows of 128 bytes]: a 64-token block of K is 64 token rows of 128 dims, a
    // 64-token block of V^T is 128 dim rows of 64 tokens = 64 rows of 128 bytes.  The copies treat a row as 64
    // 16-bit elements (the conversion warpgroup undoes the 128-byte swizzle when it reads the block).
    for (int t = 0; t < 2; ++t) {
        uint64_t dims[3] = {64, (uint64_t)Ls_pad, (uint64_t)H};
        uint64_t str[2] = {128, (uint64_t)Ls_pad * 128};
        uint32_t box[3] = {64, 64, 1};
        cudaError_t e = make_tmap_bf16(t == 0 ? tm_k8 : tm_v8, t == 0 ? k8 : v8, 3, dims, str, box);
        if (e != cudaSuccess) return e;
    }
    uint64_t dims[2] = {64, (uint64_t)Ls_pad};
    uint64_t str[1] = {64 * 2};
    uint32_t box[2] = {64, 64};
    return make_tmap_bf16(tm_kp, kpe, 2, dims, str, box);
}

}  // namespace tmla
