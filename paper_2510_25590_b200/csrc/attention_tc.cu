// Region attention with the Region-Instruction KV cache on the 5th-generation
// tensor cores (Sec. 4 "Region-Aware Generation", the attention equation):
// queries of the recomputed tokens against [fresh keys | cached keys] without
// materialising the concatenation.
//
// One CTA = one (request, head, pair of 128-row query tiles).  Warp roles:
//   warps 0-3  softmax / correction / epilogue of query tile 0 (thread = row)
//   warps 4-7  the same for query tile 1
//   warp  8    TMA producer: Q once, then K_j, V_j tiles (128 keys) through a ring
//              of shared-memory stages; the cached segment and the fresh segment
//              are two tensor maps walked one after the other.  In the full step that
//              refreshes the Region-Instruction KV cache the whole warp also copies the
//              retained rows of the staged K / V tiles from shared memory to the cache
//   warps 9,10 issuers of the O_t += P_t V_j products, one per query tile (the whole
//              warp walks the loop, one elected lane issues); warp 9 owns the
//              tensor-memory allocation
//   warp  11   issuer of the S = Q_t K_j^T products of both query tiles
//   (warps 8-11 form the third warpgroup; it gives registers up to the softmax
//   warpgroups with setmaxnreg)
//
// Tensor memory (512 columns): S | P0 | P1 | O0 | O1 = 128 + 64 + 64 + 128 + 128.
// There is ONE S buffer (fp32, 128 logits per row), a staging place that the two
// query tiles share: a product lands there, the softmax warps of its tile read their
// row into registers and give the buffer back at once, and the next product (the other
// tile's, or the same tile's next key tile) may follow while the exponentials are
// still being computed.  The probabilities go to the tile's own P region as packed
// bf16, in two chunks of 64 keys, and O_t += P_t V_j runs straight from tensor memory:
// the product of the first chunk is issued while the exponentials of the second are
// computed.  Because P does not live in the S buffer, S_t(j+1) never waits for the
// products P_t(j) V_j: the dependency chain of a tile is  S ready -> row maximum ->
// exponentials -> (S of the next key tile is already there),  with both kinds of
// product off it.  What a tile must wait for before it overwrites P_t or rescales O_t
// is the completion of its previous key tile's products (a barrier of their own), and
// that has long happened by then.  The two tiles run their exponentials whenever they
// are ready; nothing sequences them.  A pair with a single live query tile does not
// leave the second tile's warps idle: they run the same query tile against the odd key
// tiles of the segment (own accumulator, maximum and sum), the first tile's warps take
// the even ones, and the epilogue merges the halves.
//
// Online softmax in the exp2 domain; O is rescaled in tensor memory only when
// a row maximum grows by more than 2^8.  Keys past a segment's live count are
// masked in the softmax and their V rows zeroed in shared memory, so garbage
// (even NaN) behind the live prefix cannot leak.
//
// Scheduling: the kernel is persistent, one CTA per SM.  A "step" is one key tile of one
// (request, head, query pair) item; all steps of the launch form one sequence, item after item,
// laid out on a cost axis (a step of a pair with one live query tile costs half a step of a full
// pair, and every item starts with a fixed cost for draining and refilling the pipeline), which is cut into equal contiguous shares, one per CTA (a stream-K decomposition:
// the grid is always one balanced wave, whatever the number of items).  A CTA's share is a few
// segments, each a run of key tiles of one item.  A segment that covers its item completely writes
// the output rows directly; otherwise it writes its unnormalised output and (max, sum) pair to a
// slot of the caller's workspace and a small second kernel merges the slots of such items (the
// attention kernel leaves it a table of the items that its share boundaries cut).  The share
// length is bounded below so that no item is spread over more slots than the workspace holds.
// Counts live in device memory, so every CTA derives the same plan from them.  Output rows go to
// out[b, i] or, with a row list, to out[b, out_rows[b, i]] (the scatter of the attention rows back
// into the joint sequence, done by whichever kernel writes the row).
//
// Every wait is bounded: if a barrier does not complete within ~2 s the CTA
// records REGIONE_DEV_TIMEOUT, all roles leave their loops, tensor memory is
// released and the kernel ends normally.
#include <cuda.h>
#include <cstddef>
#include <type_traits>

#include <algorithm>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace regione {

constexpr int kAttnThreads = 384;        // 2 softmax warpgroups + 1 of producer / issuers
constexpr int kBM = 128;                 // query rows per tile
constexpr int kBN = 128;                 // key rows per shared-memory tile
constexpr int kBH = 64;                  // key rows per P chunk (half a tile)
constexpr int kPolyEvery = 4;             // one pair in kPolyEvery computes one of its two exponentials on the FMA pipe
constexpr int kHalfBytes = 128 * 64 * 2; // one 128-row x 64-column bf16 box (128-byte rows)
constexpr long long kTimeoutCycles = 4000000000LL;   // default bound of every wait (about 2 s)

template <int D>
struct AttnCfg {
    static constexpr int kHalves = D / 64;
    static constexpr int kTileBytes = kHalves * kHalfBytes;
    static constexpr int kStages = (D == 128) ? 4 : 6;
    // 2 query tiles + the ring + one more stage that only a lone query tile uses (its ring is that
    // stage, the ordinary ring and the idle second query tile: kStages + 2 stages)
    static constexpr int kSmemTiles = (2 + kStages + 1) * kTileBytes;
    static constexpr int kCtrlBytes = 256;
    static constexpr int kSmemBytes = kSmemTiles + 1024 /*alignment slack*/ + kCtrlBytes +
                                      kBM * 8 /*(max, sum) of a lone tile's second half*/;
};

struct AttnCtrl {
    uint64_t q_full;
    uint64_t kv_full[8];        // up to AttnCfg::kStages + 2 stages
    uint64_t kv_empty[8];
    uint64_t s_full[2];         // [query tile]
    uint64_t p_full[2][2];      // [query tile][chunk of 64 keys]
    uint64_t o_final[2];        // completes once, after the tile's last P*V product
    uint64_t pv_done[2];        // [query tile] completes after every key tile's last product: P may be
                                // overwritten and O rescaled
    uint64_t s_free;            // the shared S buffer has been read by the softmax warps it was computed for
    uint64_t half_done;         // lone query tile: the odd key tiles' (max, sum) are in shared memory
    uint32_t tmem_base;
    int abort_flag;
};

// The barriers of AttnCtrl as one array starting at q_full.
constexpr int kBarKvEmpty = 9, kBarSFull = 17, kBarPFull = 19, kBarOFinal = 23, kBarPvDone = 25, kBarSFree = 27,
              kBarHalfDone = 28, kNumBarriers = 29;
static_assert(offsetof(AttnCtrl, kv_empty) == kBarKvEmpty * 8 && offsetof(AttnCtrl, s_full) == kBarSFull * 8 &&
              offsetof(AttnCtrl, p_full) == kBarPFull * 8 && offsetof(AttnCtrl, o_final) == kBarOFinal * 8 &&
              offsetof(AttnCtrl, pv_done) == kBarPvDone * 8 && offsetof(AttnCtrl, s_free) == kBarSFree * 8 &&
              offsetof(AttnCtrl, half_done) == kBarHalfDone * 8 && offsetof(AttnCtrl, tmem_base) == kNumBarriers * 8,
              "barrier layout");

// What share c tells the merge kernel: the item that the boundary between shares c - 1 and c
// cuts, if c is the second share of that item (so every cut item is named exactly once).
struct alignas(16) CutItem {
    int valid, b, h, qp, n_slots, nq, pad0, pad1;
};

struct AttnParams {
    const int32_t* n_q;
    const int32_t* n_fresh;
    const int32_t* n_cache;
    int B, Nq_cap, Nf_cap, Nc_cap, H;
    int P_cap;           // query pairs per (request, head) at capacity
    int max_slots;       // workspace slots per item (>= 2)
    float scale_log2e;
    uint16_t* out;       // [B, out_cap, H, D]
    const int32_t* out_rows;   // nullptr: query row i goes to out row i; else to row out_rows[b, i]
    int out_cap;         // rows per request of `out` (Nq_cap without out_rows)
    int32_t* dev_status;
    float* part_o;       // [B, H, P_cap, max_slots, 256, D] unnormalised outputs
    float2* part_ml;     // [B, H, P_cap, max_slots, 256]    (running max in the exp2 domain, sum)
    CutItem* cut;        // [grid] the item that the start of each share cuts, for the merge kernel
    long long timeout_cycles;   // bound of every barrier wait, in SM clock cycles
};

// Cache refresh fused into a full step: the rows keep_rows[b, 0..n_keep[b]) (ascending) of the fresh
// K and V are also written to k_store / v_store [B, store_cap, H, D].  A parameter of its own, of
// the kernel that refreshes the cache only: the plain attention kernel's parameters do not grow.
struct StoreParams {
    const int32_t* keep_rows;
    const int32_t* n_keep;
    int store_cap;
    uint16_t* k_store;
    uint16_t* v_store;
};


// ---- the plan every CTA (and the merge kernel) derives from the device-side counts ------------
// Shares are cut on a cost axis measured in ticks, not in steps, so that they take about the same
// time: a key tile of a full query pair costs kTickPair, a key tile of a pair with one live query
// tile kTickSingle (its even and odd key tiles run side by side on the two tile roles; measured per
// thread block against its share's composition: 0.55 to 0.56 of a pair's step, not half), and every
// item starts with kTickStart ticks that stand for the drain of the previous segment and the fill of
// the new one (measured the same way: 3.5 to 6 pair steps depending on the workload, 5 on the
// layers of configurations 2 and 4).
constexpr int kTickPair = 16, kTickSingle = 9, kTickStart = 80;

struct ReqShape {
    int nq, nf, nc;      // clamped counts
    int np;              // live query pairs
    int nt_c, nt;        // cached key tiles, all key tiles
    long long items;     // H * np
    int steps;           // steps of an item: max(nt, 1) (an item without keys writes zeros in one step)
    int w_last;          // ticks per step of the last query pair
    long long ticks_full, ticks_last, head_ticks, ticks;   // per full-pair item, last item, head, request
};

// NO_CACHE: the launch has no cached segment at all (p.n_cache is not read).
template <bool NO_CACHE>
__device__ __forceinline__ ReqShape req_shape(const AttnParams& p, int b, bool* bad = nullptr) {
    ReqShape r;
    int nq = p.n_q[b], nf = p.n_fresh[b], nc = NO_CACHE ? 0 : p.n_cache[b];
    if (nq < 0 || nq > p.Nq_cap || nf < 0 || nf > p.Nf_cap || nc < 0 || nc > p.Nc_cap) {
        if (bad) *bad = true;
        nq = max(0, min(nq, p.Nq_cap));
        nf = max(0, min(nf, p.Nf_cap));
        nc = max(0, min(nc, p.Nc_cap));
    }
    r.nq = nq; r.nf = nf; r.nc = nc;
    r.np = (nq + 2 * kBM - 1) / (2 * kBM);
    r.nt_c = (nc + kBN - 1) / kBN;
    r.nt = r.nt_c + (nf + kBN - 1) / kBN;
    r.items = (long long)p.H * r.np;
    r.steps = max(r.nt, 1);
    r.w_last = (nq - (r.np - 1) * 2 * kBM > kBM) ? kTickPair : kTickSingle;
    r.ticks_full = kTickStart + (long long)kTickPair * r.steps;
    r.ticks_last = kTickStart + (long long)r.w_last * r.steps;
    r.head_ticks = r.np > 0 ? (r.np - 1) * r.ticks_full + r.ticks_last : 0;
    r.ticks = p.H * r.head_ticks;
    return r;
}

// How the launch's work is cut into shares, one per CTA.
//  - whole items: when handing out whole items wastes at most 6 % of the grid's last round, items
//    are dealt round-robin and never split (no workspace traffic, no merge): positions count items.
//  - otherwise positions count ticks and CTA c owns the steps whose first tick lies in
//    [c * chunk, (c + 1) * chunk); shares may cut items.  The share length is bounded below so
//    that an item never meets more than max_slots shares.
struct Plan {
    bool whole_items;
    long long total, chunk;
};

template <bool NO_CACHE>
__device__ __forceinline__ Plan plan_shares(const AttnParams& p, int grid, bool* bad = nullptr) {
    Plan pl;
    long long items = 0, ticks = 0, span = 0;      // span: first tick of an item's last step, at most
    for (int b = 0; b < p.B; ++b) {
        const ReqShape r = req_shape<NO_CACHE>(p, b, bad);
        items += r.items;
        ticks += r.ticks;
        if (r.np > 0) span = max(span, (long long)(r.np > 1 ? kTickPair : r.w_last) * (r.steps - 1));
    }
    const long long per = (items + grid - 1) / grid;
    pl.whole_items = per * grid * 100 <= items * 106;
    if (pl.whole_items) {
        pl.total = items;
        pl.chunk = max(per, 1LL);
    } else {
        pl.total = ticks;
        pl.chunk = (ticks + grid - 1) / grid;
        // an item meets at most span / chunk + 2 shares: keep that within max_slots; and a share is
        // at least one step long, so that every share between an item's first and last holds a
        // step of it (and writes its slot)
        const long long floor_len = max(span / (p.max_slots - 1) + 1, (long long)kTickPair);
        if (pl.chunk < floor_len) pl.chunk = floor_len;
    }
    return pl;
}

// The part of one item that a CTA works on.
struct Segment {
    int b, h, qp;
    ReqShape r;
    int j_first, n_steps;   // steps [j_first, j_first + n_steps) of the item; n_steps may be 0
    int slot, n_slots;      // this share's slot among the shares that hold steps of the item
    long long next;         // position behind the item
};

// a / b for non-negative a and positive b; positions fit 32 bits in every realistic launch, and a
// 32-bit division is several times shorter than a 64-bit one (the lookups below sit between two
// segments, on every thread's path).
__device__ __forceinline__ long long div_pos(long long a, long long b) {
    if (((a | b) >> 32) == 0) return (long long)((unsigned)a / (unsigned)b);
    return a / b;
}

// Shares that hold steps of the item whose step 0 starts at tick `first_tick`.
__device__ __forceinline__ void item_slots(const Plan& pl, long long first_tick, int w, int steps,
                                           int& c_first, int& n_slots) {
    c_first = (int)div_pos(first_tick, pl.chunk);
    n_slots = (int)div_pos(first_tick + (long long)w * (steps - 1), pl.chunk) - c_first + 1;
}

// Whole-item plan: the item with index `idx`.
template <bool NO_CACHE>
__device__ __forceinline__ Segment segment_whole(const AttnParams& p, long long idx) {
    Segment sg;
    long long base = 0;
    int b = 0;
    ReqShape r = req_shape<NO_CACHE>(p, 0);
    while (idx >= base + r.items && b + 1 < p.B) {
        base += r.items;
        ++b;
        r = req_shape<NO_CACHE>(p, b);
    }
    const long long item = idx - base;
    sg.b = b; sg.r = r;
    sg.h = r.np > 0 ? (int)(item / r.np) : 0;
    sg.qp = (int)(item - (long long)sg.h * r.np);
    sg.j_first = 0;
    sg.n_steps = r.np > 0 ? r.steps : 0;
    sg.slot = 0; sg.n_slots = 1;
    sg.next = idx + 1;
    return sg;
}

// Tick plan: the item that contains tick `pos`, and the steps of it that share `c` owns.
template <bool NO_CACHE>
__device__ __forceinline__ Segment segment_ticks(const AttnParams& p, const Plan& pl, long long pos,
                                                 int c) {
    Segment sg;
    long long base = 0;
    int b = 0;
    ReqShape r = req_shape<NO_CACHE>(p, 0);
    while (pos >= base + r.ticks && b + 1 < p.B) {
        base += r.ticks;
        ++b;
        r = req_shape<NO_CACHE>(p, b);
    }
    sg.b = b; sg.r = r;
    if (r.np == 0) {                                  // nothing left behind the last live request
        sg.h = sg.qp = sg.j_first = sg.n_steps = sg.slot = 0;
        sg.n_slots = 1;
        sg.next = pl.total;
        return sg;
    }
    const long long rel = pos - base;
    sg.h = (int)div_pos(rel, r.head_ticks);
    const long long rem = rel - (long long)sg.h * r.head_ticks;
    sg.qp = (int)min(div_pos(rem, r.ticks_full), (long long)(r.np - 1));
    const long long t0 = base + (long long)sg.h * r.head_ticks + (long long)sg.qp * r.ticks_full;
    const bool last = sg.qp == r.np - 1;
    const int w = last ? r.w_last : kTickPair;
    const long long first_tick = t0 + kTickStart;
    const long long lo = (long long)c * pl.chunk, hi = lo + pl.chunk;
    long long s_lo = lo <= first_tick ? 0 : div_pos(lo - first_tick + w - 1, w);
    long long s_hi = hi <= first_tick ? 0 : div_pos(hi - first_tick + w - 1, w);
    s_lo = min(s_lo, (long long)r.steps);
    s_hi = min(s_hi, (long long)r.steps);
    sg.j_first = (int)s_lo;
    sg.n_steps = (int)(s_hi - s_lo);
    int c_first;
    item_slots(pl, first_tick, w, r.steps, c_first, sg.n_slots);
    sg.slot = c - c_first;
    sg.next = t0 + (last ? r.ticks_last : r.ticks_full);
    return sg;
}

// Bounded wait on phase `parity` of an mbarrier: true when the phase completed, false when another
// role has already given up or `limit` cycles have passed (then the abort flag is raised and
// REGIONE_DEV_TIMEOUT recorded; the caller leaves its loop, nothing traps).
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                         int32_t* dev_status, long long limit) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > limit) {
            *abort_flag = 1;
            record_status(dev_status, REGIONE_DEV_TIMEOUT);
            return false;
        }
    }
}

// Keys >= valid of a 64-logit chunk are dead (behind a segment's live prefix): their logits become
// -inf, after which the chunk goes through the same code as a full one (maximum unaffected,
// probability 0 or, on the polynomial path, 2^-126).  A short separate pass instead of masked
// variants of the long unrolled loops: those would run once per item, from a cold instruction cache.
__device__ __forceinline__ void mask_dead_keys(uint32_t* s, int valid) {
#pragma unroll
    for (int i = 0; i < kBH; ++i)
        if (i >= valid) s[i] = 0xff800000u;
}

// Maximum of 64 logits held in registers.
__device__ __forceinline__ float chunk_max(const uint32_t* s) {
    float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
    for (int i = 0; i < kBH; ++i) mx[i & 3] = fmaxf(mx[i & 3], __uint_as_float(s[i]));
    return fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
}

// 2^x for x <= 0 on the FMA pipe: x = n + f with n = round(x) (the magic-number addition leaves n in
// the low mantissa bits of t), 2^f by a cubic on [-0.5, 0.5] (relative error 7.5e-5, far below the
// bf16 rounding of the probabilities), n added to the exponent field.  Used for part of the
// exponentials so that they do not all queue on the special-function unit.
__device__ __forceinline__ float poly_exp2(float x) {
    x = fmaxf(x, -126.f);
    const float t = x + 12582912.f;
    const float f = x - (t - 12582912.f);
    float p = fmaf(f, 0.0551716f, 0.2426111f);
    p = fmaf(p, f, 0.6932610f);
    p = fmaf(p, f, 0.9999281f);
    return __int_as_float(__float_as_int(p) + (__float_as_int(t) << 23));
}

// p = 2^(s*c - m) for 64 logits, written to tensor memory at `tP` (32 columns) as packed bf16;
// returns their fp32 sum.
__device__ __forceinline__ float chunk_probabilities(uint32_t tP, const uint32_t* s, float c, float m) {
    float sum[4] = {0.f, 0.f, 0.f, 0.f};
    uint32_t pk[kBH / 2];
#pragma unroll
    for (int i = 0; i < kBH / 2; ++i) {
        const float p0 = fast_exp2(fmaf(__uint_as_float(s[2 * i]), c, -m));
        const float p1 = (i % kPolyEvery == 1) ? poly_exp2(fmaf(__uint_as_float(s[2 * i + 1]), c, -m))
                                               : fast_exp2(fmaf(__uint_as_float(s[2 * i + 1]), c, -m));
        sum[i & 3] += p0 + p1;
        pk[i] = pack_bf16x2(p0, p1);
    }
    ptx::tmem_st32(tP, pk);
    return (sum[0] + sum[1]) + (sum[2] + sum[3]);
}

// The segments of one CTA's share, for one of the two kinds of warpgroup: the softmax warpgroups
// (SOFTMAX_WG, many registers) or the producer / issuer warpgroup (few).  The two instantiations
// are called from the two sides of the setmaxnreg split so that each is compiled for its own
// register budget; both execute the same sequence of CTA-wide barriers.
// STORE: the instantiation for the full step that also refreshes the cache (warp 11 writes the
// retained K / V rows); the plain instantiation contains none of that code.
template <int D, bool SOFTMAX_WG, bool STORE>
__device__ __forceinline__ void run_share(const CUtensorMap* tm_q_, const CUtensorMap* tm_kf_,
                                          const CUtensorMap* tm_vf_, const CUtensorMap* tm_kc_,
                                          const CUtensorMap* tm_vc_, const AttnParams& p,
                                          const StoreParams& sp,
                                          long long pos, const long long hi, const Plan pl,
                                          AttnCtrl* ctrl, uint8_t* smem_gen, const uint32_t sQ,
                                          const uint32_t sKV, const int warp, const int lane) {
    using Cfg = AttnCfg<D>;
    constexpr int kStages = Cfg::kStages;
    constexpr int kTileBytes = Cfg::kTileBytes;
    volatile int* abort_flag = &ctrl->abort_flag;
    const CUtensorMap& tm_q = *tm_q_;
    const CUtensorMap& tm_kf = *tm_kf_;
    const CUtensorMap& tm_vf = *tm_vf_;
    const CUtensorMap& tm_kc = *tm_kc_;
    const CUtensorMap& tm_vc = *tm_vc_;
    bool first_segment = true;
    while (pos < hi) {
    // ---- the segment: key tiles [j_first, j_first + n_tiles) of item (b, h, query pair) ----
    const Segment it = pl.whole_items ? segment_whole<STORE>(p, pos)
                                      : segment_ticks<STORE>(p, pl, pos, (int)blockIdx.x);
    if (first_segment && SOFTMAX_WG && threadIdx.x == 0) {
        // tell the merge kernel which item the start of this share cuts
        CutItem ci;
        ci.valid = (!pl.whole_items && it.r.np > 0 && it.n_slots >= 2 && it.slot == 1) ? 1 : 0;
        ci.b = it.b; ci.h = it.h; ci.qp = it.qp; ci.n_slots = it.n_slots; ci.nq = it.r.nq;
        ci.pad0 = ci.pad1 = 0;
        p.cut[blockIdx.x] = ci;
    }
    first_segment = false;
    if (it.n_steps == 0) {                              // (uniform for the CTA)
        pos = pl.whole_items ? pos + gridDim.x : it.next;
        continue;
    }
    const int b = it.b, h = it.h;
    const int q0 = it.qp * (2 * kBM);
    const int nq = it.r.nq, nf = it.r.nf, nc = it.r.nc, nt_c = it.r.nt_c;
    const int ntq = (nq - q0 > kBM) ? 2 : 1;            // live query tiles of this segment
    const int j_first = it.j_first;
    const int n_tiles = it.r.nt == 0 ? 0 : it.n_steps;
    // slot of this segment among the shares that touch the item; a lone segment writes the output
    const int slot = it.slot;
    const bool direct = it.n_slots == 1;
    // A lone query tile would leave half of the CTA idle and run at the speed of its dependency
    // chain.  Instead the roles of "tile 1" work on the same query tile against the odd key tiles
    // of the segment while "tile 0" takes the even ones; the two halves (own accumulator, maximum
    // and sum) are merged in the epilogue.  `lanes` = query-tile roles at work.
    const bool split = ntq == 1 && n_tiles >= 2;
    const int lanes = split ? 2 : ntq;
    // a lone tile's ring starts at the idle second query tile and runs over the extra stage: two
    // stages more, because its two halves consume K/V tiles at twice the rate per chain
    const int n_stages = split ? kStages + 2 : kStages;
    // cache refresh: every item walks all key tiles of its (request, head); key tile j is written to
    // the cache by the item of query pair j mod np, so every (request, head, key tile) is written
    // exactly once and the copies are spread evenly over the thread blocks
    const bool store_item = STORE && n_tiles > 0;
    const uint32_t ring = split ? sQ + kTileBytes : sKV;
    uint8_t* const ring_gen = smem_gen + (split ? 1 : 2) * kTileBytes;

    // thread i sets barrier i of the control block up (and takes it down after the segment)
    if (threadIdx.x < kNumBarriers) {
        const int i = threadIdx.x;
        int count = 1;                                               // q_full, kv_full, s_full, o_final
        if (i >= kBarKvEmpty && i < kBarSFull) count = (split ? 1 : ntq) + (store_item ? 1 : 0);   // commits per stage (+ the cache writer)
        else if ((i >= kBarPFull && i < kBarOFinal) || i >= kBarSFree) count = kBM / 32;   // one arrival per warp
        ptx::mbar_init(ptx::smem_addr(&ctrl->q_full + i), count);
        ptx::fence_barrier_init();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = ctrl->tmem_base;

    // key tile jl of this segment -> (segment of the KV sequence, first row, live rows); a tile
    // yields one P chunk when at most 64 of its keys are live, else two
    auto tile_seg = [&](int jl, bool& cached, int& row0, int& valid) {
        const int j = j_first + jl;
        cached = j < nt_c;
        const int jj = cached ? j : j - nt_c;
        row0 = jj * kBN;
        valid = min(kBN, (cached ? nc : nf) - row0);
    };
    auto tile_chunks = [&](int jl) {
        bool cached; int row0, valid;
        tile_seg(jl, cached, row0, valid);
        return valid > kBH ? 2 : 1;
    };
    // key tiles of query-tile role t: all of them, or every second one of a lone query tile
    auto role_tiles = [&](int t) { return split ? (n_tiles + 1 - t) >> 1 : n_tiles; };
    auto role_tile = [&](int t, int j) { return split ? 2 * j + t : j; };

    if constexpr (!SOFTMAX_WG) {
    if (warp == 8) {
        // ================= TMA producer (and, in the cache-refreshing kernel, the cache writer) =================
        if (n_tiles > 0) {
            if (lane == 0) {
                ptx::prefetch_tensormap(&tm_q);
                ptx::prefetch_tensormap(j_first < nt_c ? &tm_kc : &tm_kf);
                ptx::prefetch_tensormap(j_first < nt_c ? &tm_vc : &tm_vf);
                const uint32_t qbar = ptx::smem_addr(&ctrl->q_full);
                ptx::mbar_arrive_expect_tx(qbar, ntq * kTileBytes);
                for (int t = 0; t < ntq; ++t)
                    for (int hf = 0; hf < Cfg::kHalves; ++hf)
                        ptx::tma_load_4d(sQ + t * kTileBytes + hf * kHalfBytes, &tm_q, qbar, hf * 64, h,
                                         q0 + t * kBM, b);
            }
            // ---- cache writer state (whole warp; used by the cache-refreshing kernel only) ----
            // The retained rows of every K / V tile this segment stages are copied from shared memory
            // to their slots in the cache, two ring items behind the loads (an item has landed by
            // then), before its stage is given back.
            constexpr int kCpr = D / 8;                 // 16-byte chunks per row of one head
            constexpr int kRowsPer = 32 / kCpr;         // rows a warp instruction moves
            constexpr int kLag = 2;
            const int32_t* keep = nullptr;
            int nk = 0, lo = 0, cnt = 0;
            bool mine = false;                          // the key tile being written belongs to this item
            int r[kBN / 32];
            if (STORE && store_item) {
                keep = sp.keep_rows + (size_t)b * sp.store_cap;
                nk = sp.n_keep[b];
                if (nk < 0 || nk > sp.store_cap) {
                    record_status(p.dev_status, REGIONE_DEV_BOUNDS);
                    nk = max(0, min(nk, sp.store_cap));
                }
            }
            // number of retained rows below `row_first` (the list is ascending): 32-ary search, one
            // coalesced probe per level
            auto rows_below = [&](int row_first) {
                int at0 = 0, len = nk;
                while (len > 0) {
                    const int step = (len + 31) / 32;
                    const int at = at0 + min(lane * step, len - 1);
                    const bool below = (lane * step < len) && keep[at] < row_first;
                    const int nb = __popc(__ballot_sync(0xffffffffu, below));   // probes below the target
                    // the answer lies behind probe nb - 1 and at or before probe nb
                    const int new_lo = nb == 0 ? at0 : at0 + (nb - 1) * step + 1;
                    const int new_hi = nb == 0 ? at0 : min(at0 + nb * step, at0 + len);
                    len = (step == 1) ? 0 : new_hi - new_lo;
                    at0 = (step == 1) ? at0 + nb : new_lo;
                }
                return at0;
            };
            // copies ring item x (K of key tile x / 2, or V) to the cache if that tile is this item's to
            // write, and releases its stage
            auto write_item = [&](int x) -> bool {
                const int jl = x >> 1, is_v = x & 1, stage = x % n_stages;
                bool cached; int row0, valid;
                tile_seg(jl, cached, row0, valid);
                if (!is_v) {
                    mine = (j_first + jl) % it.r.np == it.qp;
                    if (mine) {
                        // retained rows of this tile: at most kBN consecutive entries of the ascending list
                        lo = rows_below(row0);
                        cnt = 0;                        // length of the run of entries inside this tile
                        bool run_open = true;
#pragma unroll
                        for (int k = 0; k < kBN / 32; ++k) {
                            const int i = lo + k * 32 + lane;
                            r[k] = i < nk ? keep[i] - row0 : kBN;
                            if (r[k] < 0) {             // the list is not ascending
                                record_status(p.dev_status, REGIONE_DEV_BOUNDS);
                                r[k] = kBN;
                            }
                            const uint32_t inside = __ballot_sync(0xffffffffu, r[k] < valid);
                            if (run_open) cnt += inside == 0xffffffffu ? 32 : __ffs(~inside) - 1;
                            run_open = run_open && inside == 0xffffffffu;
                        }
                        // entries left over behind the last key tile name rows that do not exist
                        if (j_first + jl == it.r.nt - 1 && lo + cnt < nk)
                            record_status(p.dev_status, REGIONE_DEV_BOUNDS);
                    }
                }
                if (mine) {
                    if (!wait_bar(ptx::smem_addr(&ctrl->kv_full[stage]), (x / n_stages) & 1, abort_flag,
                                  p.dev_status, p.timeout_cycles))
                        return false;
                    const uint8_t* tile = ring_gen + stage * kTileBytes;
                    uint16_t* dst_base = (is_v ? sp.v_store : sp.k_store) +
                                         (((size_t)b * sp.store_cap + lo) * p.H + h) * D;
                    const int q = lane % kCpr;          // this lane's 16-byte chunk of the row
#pragma unroll
                    for (int k = 0; k < kBN / 32; ++k) {
                        if (k * 32 >= cnt) break;                       // (uniform)
#pragma unroll 1
                        for (int e0 = 0; e0 < 32; e0 += 4 * kRowsPer) {
                            // four warp-wide moves at a time: all loads are issued before the first store
                            uint4 x4[4];
                            int el[4];
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                el[u] = e0 + u * kRowsPer + lane / kCpr;    // entry of the tile's run: k * 32 + el
                                const int rr = __shfl_sync(0xffffffffu, r[k], el[u]);
                                if (k * 32 + el[u] < cnt)
                                    x4[u] = *reinterpret_cast<const uint4*>(
                                        tile + (q >> 3) * kHalfBytes + rr * 128 + (((q & 7) ^ (rr & 7)) << 4));
                            }
#pragma unroll
                            for (int u = 0; u < 4; ++u)
                                if (k * 32 + el[u] < cnt)
                                    *reinterpret_cast<uint4*>(dst_base + (size_t)(k * 32 + el[u]) * p.H * D + q * 8) = x4[u];
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctrl->kv_empty[stage]));
                return true;
            };
            bool ok = true;
            const int n_items = 2 * n_tiles;
            for (int i = 0; i < n_items + (STORE && store_item ? kLag : 0) && ok; ++i) {
                if (STORE && store_item && i >= kLag) ok = write_item(i - kLag);
                if (i < n_items && ok) {
                    if (lane == 0) {
                        const int j = i >> 1, is_v = i & 1;
                        const int stage = i % n_stages, use = i / n_stages;
                        if (use > 0)
                            ok = wait_bar(ptx::smem_addr(&ctrl->kv_empty[stage]), (use - 1) & 1, abort_flag,
                                          p.dev_status, p.timeout_cycles);
                        if (ok) {
                            bool cached; int row0, valid;
                            tile_seg(j, cached, row0, valid);
                            const CUtensorMap* map = cached ? (is_v ? &tm_vc : &tm_kc) : (is_v ? &tm_vf : &tm_kf);
                            const uint32_t bar = ptx::smem_addr(&ctrl->kv_full[stage]);
                            ptx::mbar_arrive_expect_tx(bar, kTileBytes);
                            for (int hf = 0; hf < Cfg::kHalves; ++hf)
                                ptx::tma_load_4d(ring + stage * kTileBytes + hf * kHalfBytes, map, bar, hf * 64, h,
                                                 row0, b);
                        }
                    }
                    if (STORE) ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;     // (the writer's lanes follow lane 0)
                }
            }
        }
    } else if (warp == 11) {
        // ================= issuer of the S products of both query tiles =================
        // S = Q_t K_j^T goes to ONE staging buffer in tensor memory that the two query tiles share:
        // a product is issued as soon as its K tile has landed and the buffer's previous contents
        // have been read into registers by the softmax warps they were computed for.  It does not
        // have to wait for the P*V products of its own tile, which read P from a place of their own.
        if (n_tiles > 0) {
            constexpr uint32_t idesc_s = ptx::idesc_bf16_f32(kBM, kBN, false);
            constexpr uint32_t hi_k = ptx::smem_desc_hi_sw128(1024);   // 8-row groups 1024 B apart
            const uint32_t k_lo = ptx::smem_desc_lo(ring, 16);
            bool ok = wait_bar(ptx::smem_addr(&ctrl->q_full), 0, abort_flag, p.dev_status, p.timeout_cycles);
            int n_issued = 0;                                   // products so far = uses of the staging buffer
            for (int jl = 0; jl < n_tiles && ok; ++jl) {
                const int ik = 2 * jl, sk = ik % n_stages;
                ok = wait_bar(ptx::smem_addr(&ctrl->kv_full[sk]), (ik / n_stages) & 1, abort_flag,
                              p.dev_status, p.timeout_cycles);
                // the roles this key tile feeds: both query tiles, or one half of a lone query tile
                const int t_first = split ? (jl & 1) : 0, t_last = split ? (jl & 1) : ntq - 1;
                for (int t = t_first; t <= t_last && ok; ++t) {
                    if (n_issued > 0)
                        ok = wait_bar(ptx::smem_addr(&ctrl->s_free), (n_issued - 1) & 1, abort_flag,
                                      p.dev_status, p.timeout_cycles);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    if (ptx::elect_one()) {
                        const uint32_t q_lo = ptx::smem_desc_lo(sQ + (split ? 0 : t) * kTileBytes, 16);
                        const uint32_t b0 = k_lo + ((sk * kTileBytes) >> 4);
#pragma unroll
                        for (int kk = 0; kk < D / 16; ++kk) {
                            const uint32_t off = ((kk >> 2) * kHalfBytes + (kk & 3) * 32) >> 4;
                            ptx::mma_ss(tmem, ptx::smem_desc_join(q_lo + off, hi_k),
                                        ptx::smem_desc_join(b0 + off, hi_k), idesc_s, kk > 0);
                        }
                        ptx::mma_commit(ptx::smem_addr(&ctrl->s_full[t]));
                        ptx::mma_commit(ptx::smem_addr(&ctrl->kv_empty[sk]));
                    }
                    __syncwarp();
                    ++n_issued;
                }
            }
        }
    } else if (warp == 9 || warp == 10) {
        // ================= issuers of the P*V products: warp 9 for query tile 0, warp 10 for query tile 1 ========
        // Each whole warp walks its loop and waits on the barriers; one elected lane issues.
        const int t = warp - 9;
        if (t < lanes && n_tiles > 0) {
            const int n_my = role_tiles(t);
            constexpr uint32_t idesc_pv = ptx::idesc_bf16_f32(kBM, D, true);
            constexpr uint32_t hi_k = ptx::smem_desc_hi_sw128(1024);   // 8-key groups 1024 B apart
            // V is MN-major: 64-column boxes kHalfBytes apart (LBO), 8-key groups 1024 B apart (SBO)
            const uint32_t v_lo = ptx::smem_desc_lo(ring, kHalfBytes);
            const uint32_t tPt = tmem + kBN + t * (kBN / 2), tOt = tmem + 256 + t * D;
            // O_t (+)= P_t[chunk] V[64 chunk .. 64 chunk + 64) : A from tensor memory (bf16 pairs,
            // 8 columns per 16 keys)
            auto issue_pv = [&](int stage, int chunk, bool accumulate) {
                const uint32_t b0 = v_lo + ((stage * kTileBytes + chunk * (kBH / 16) * 2048) >> 4);
#pragma unroll
                for (int kk = 0; kk < kBH / 16; ++kk)
                    ptx::mma_ts(tOt, tPt + chunk * (kBH / 2) + kk * 8,
                                ptx::smem_desc_join(b0 + ((kk * 2048) >> 4), hi_k), idesc_pv,
                                (accumulate || kk > 0) ? 1u : 0u);
            };
            bool ok = true;
            int nb = 0;                                     // second chunks seen so far
            for (int j = 0; j < n_my && ok; ++j) {
                const int jl = role_tile(t, j);
                const int iv = 2 * jl + 1, sv = iv % n_stages;
                const bool more = (j + 1 < n_my);
                const int chunks = tile_chunks(jl);
                ok = wait_bar(ptx::smem_addr(&ctrl->kv_full[sv]), (iv / n_stages) & 1, abort_flag,
                              p.dev_status, p.timeout_cycles);
                if (ok)
                    ok = wait_bar(ptx::smem_addr(&ctrl->p_full[t][0]), j & 1, abort_flag,
                                  p.dev_status, p.timeout_cycles);
                if (!ok) break;
                if (chunks == 2) {
                    ptx::tc_fence_after_sync();
                    if (ptx::elect_one()) issue_pv(sv, 0, j > 0);
                    __syncwarp();
                    ok = wait_bar(ptx::smem_addr(&ctrl->p_full[t][1]), nb & 1, abort_flag,
                                  p.dev_status, p.timeout_cycles);
                    ++nb;
                    if (!ok) break;
                }
                ptx::tc_fence_after_sync();
                if (ptx::elect_one()) {
                    issue_pv(sv, chunks - 1, j > 0 || chunks == 2);
                    ptx::mma_commit(ptx::smem_addr(&ctrl->pv_done[t]));
                    if (!more) ptx::mma_commit(ptx::smem_addr(&ctrl->o_final[t]));
                    ptx::mma_commit(ptx::smem_addr(&ctrl->kv_empty[sv]));
                }
                __syncwarp();
            }
        }
    }
    } else if (warp < 4 * lanes) {
        // ================= softmax / correction / epilogue =================
        const int t = warp >> 2;
        const int row = ((warp & 3) << 5) + lane;                  // row of the query tile
        const uint32_t lane_sel = (uint32_t)((warp & 3) << 5) << 16;
        const uint32_t tS = tmem + lane_sel;                       // the S staging buffer both tiles share
        const uint32_t tP = tmem + lane_sel + kBN + t * (kBN / 2); // this tile's probabilities (bf16 pairs)
        const uint32_t tO = tmem + lane_sel + 256 + t * D;
        const float c = p.scale_log2e;
        float m = -INFINITY, l = 0.f;
        bool ok = true;

        const int n_my = n_tiles > 0 ? role_tiles(t) : 0;
        for (int j = 0; j < n_my; ++j) {
            bool cached; int row0, valid;
            tile_seg(role_tile(t, j), cached, row0, valid);
            const int chunks = valid > kBH ? 2 : 1;
            ok = wait_bar(ptx::smem_addr(&ctrl->s_full[t]), j & 1, abort_flag, p.dev_status, p.timeout_cycles);
            if (!ok) break;
            ptx::tc_fence_after_sync();
            uint32_t s[kBN];
            ptx::tmem_ld32(tS, s);
            ptx::tmem_ld32(tS + 32, s + 32);
            if (chunks == 2) {
                ptx::tmem_ld32(tS + 64, s + 64);
                ptx::tmem_ld32(tS + 96, s + 96);
            }
            ptx::tmem_wait_ld();
            // the logits are in registers: the staging buffer may take the next product (of the other
            // query tile, or of this tile's next key tile)
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctrl->s_free));
            float mt;
            if (chunks == 2) {
                if (valid < kBN) mask_dead_keys(s + kBH, valid - kBH);
                mt = fmaxf(chunk_max(s), chunk_max(s + kBH));
            } else {
                if (valid < kBH) mask_dead_keys(s, valid);
                mt = chunk_max(s);
            }
            mt *= c;
            // P_t and O_t belong to the products of the key tile before this one until they have
            // completed (they run in the shadow of this tile's wait for S and of its row maximum)
            if (j > 0) {
                ok = wait_bar(ptx::smem_addr(&ctrl->pv_done[t]), (j - 1) & 1, abort_flag, p.dev_status,
                              p.timeout_cycles);
                if (!ok) break;
                ptx::tc_fence_after_sync();
            }
            if (j == 0) {
                m = mt;
            } else if (__any_sync(0xffffffffu, mt > m + 8.f)) {
                const float m_new = fmaxf(m, mt);
                const float alpha = fast_exp2(m - m_new);
                uint32_t r[32];
#pragma unroll 1
                for (int ch = 0; ch < D / 32; ++ch) {
                    ptx::tmem_ld32(tO + ch * 32, r);
                    ptx::tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                    ptx::tmem_st32(tO + ch * 32, r);
                }
                l *= alpha;
                m = m_new;
            }
            // first chunk of probabilities (keys 0..63 of the tile)
            l += chunk_probabilities(tP, s, c, m);
            ptx::tmem_wait_st();
            if (valid < kBN) {
                // last tile of a segment: zero the V rows behind the live prefix (0 * NaN = NaN)
                const int iv = 2 * role_tile(t, j) + 1, sv = iv % n_stages;
                ok = wait_bar(ptx::smem_addr(&ctrl->kv_full[sv]), (iv / n_stages) & 1, abort_flag,
                              p.dev_status, p.timeout_cycles);
                if (!ok) break;
                if (row >= valid) {
                    uint8_t* vrow = ring_gen + sv * kTileBytes + row * 128;
#pragma unroll
                    for (int hf = 0; hf < Cfg::kHalves; ++hf)
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            reinterpret_cast<uint4*>(vrow + hf * kHalfBytes)[q] = make_uint4(0, 0, 0, 0);
                }
                ptx::fence_proxy_async_smem();
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctrl->p_full[t][0]));
            if (chunks == 2) {
                // second chunk (keys 64..127) while the first chunk's product runs
                l += chunk_probabilities(tP + kBH / 2, s + kBH, c, m);
                ptx::tmem_wait_st();
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctrl->p_full[t][1]));
            }
        }
        // epilogue (rows past n_q are not written).  A thread holds one row, so storing straight
        // from registers would touch 32 different rows per warp instruction; instead each warp
        // passes 128-byte row pieces through its own 4 KB corner of the (now idle) query tile in
        // shared memory and stores four whole pieces per instruction.
        const int wrow0 = q0 + (split ? 0 : t) * kBM + ((warp & 3) << 5);   // first query row of this warp
        const int live_rows = min(max(nq - wrow0, 0), 32);
        const bool live = lane < live_rows;
        // where this thread's query row goes in `out` (-1: the row is dead); the lookup is issued
        // ahead of the wait for the last product and used after it
        int dst_row = -1;
        if (live && direct)
            dst_row = p.out_rows != nullptr ? p.out_rows[(size_t)b * p.Nq_cap + wrow0 + lane] : wrow0 + lane;
        if (n_tiles > 0 && ok) {
            ok = wait_bar(ptx::smem_addr(&ctrl->o_final[t]), 0, abort_flag, p.dev_status, p.timeout_cycles);
            if (ok) ptx::tc_fence_after_sync();
        }
        // lone query tile: role 1 leaves its (max, sum) in shared memory (its accumulator stays in
        // tensor memory) and is done; role 0 merges the halves
        float2* const half_ml = reinterpret_cast<float2*>(smem_gen + Cfg::kSmemTiles + Cfg::kCtrlBytes);
        float w_own = 1.f, w_other = 0.f;                   // weights of the two accumulators
        if (split && t == 1) {
            half_ml[row] = make_float2(m, l);
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctrl->half_done));
        } else if (split && ok) {
            ok = wait_bar(ptx::smem_addr(&ctrl->half_done), 0, abort_flag, p.dev_status, p.timeout_cycles);
            if (ok) ok = wait_bar(ptx::smem_addr(&ctrl->o_final[1]), 0, abort_flag, p.dev_status, p.timeout_cycles);
            if (ok) {
                ptx::tc_fence_after_sync();
                const float2 other = half_ml[row];
                const float m_all = fmaxf(m, other.x);
                w_own = fast_exp2(m - m_all);
                w_other = other.y > 0.f ? fast_exp2(other.x - m_all) : 0.f;
                l = w_own * l + w_other * other.y;
                m = m_all;
            }
        }
        // lone tile: 32 columns of this row's two accumulators, weighted and added
        auto load_merged = [&](int col, uint32_t* r) {
            uint32_t r1[32];
            ptx::tmem_ld32(tO + col, r);
            ptx::tmem_ld32(tO + D + col, r1);
            ptx::tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i)
                r[i] = __float_as_uint(fmaf(w_own, __uint_as_float(r[i]), w_other * __uint_as_float(r1[i])));
        };
        if (!(split && t == 1)) {
        uint8_t* const stage = smem_gen + t * kTileBytes + (warp & 3) * (kTileBytes / 4);
        // `to` = this lane's destination row (counted from g_row0), -1 to drop the row
        auto store_pieces = [&](const uint4 (&v)[8], uint8_t* g_row0, size_t row_stride, int to) {
            // piece q of row r sits at 16-byte column q ^ (r & 7): both the row-wise writes and
            // the piece-wise reads are free of bank conflicts without padding
            uint4* dst = reinterpret_cast<uint4*>(stage + lane * 128);
#pragma unroll
            for (int q = 0; q < 8; ++q) dst[q ^ (lane & 7)] = v[q];
            __syncwarp();
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int rr = i * 4 + (lane >> 3);
                const uint4 x = *reinterpret_cast<const uint4*>(stage + rr * 128 +
                                                                 (((lane & 7) ^ (rr & 7)) << 4));
                const int to_rr = __shfl_sync(0xffffffffu, to, rr);
                if (to_rr >= 0)
                    *reinterpret_cast<uint4*>(g_row0 + to_rr * row_stride + (lane & 7) * 16) = x;
            }
            __syncwarp();
        };
        if (direct) {
            // O / l -> bf16 -> out
            if (dst_row >= p.out_cap || (dst_row < 0 && live)) {     // destination out of range: dropped
                record_status(p.dev_status, REGIONE_DEV_BOUNDS);
                dst_row = -1;
            }
            const size_t row_stride = (size_t)p.H * D * 2;
            uint8_t* g_row0 = reinterpret_cast<uint8_t*>(p.out) +
                              (((size_t)b * p.out_cap) * p.H + h) * D * 2;      // row 0 of the request
            if (n_tiles == 0) {
                if (dst_row >= 0)
                    for (int q = 0; q < D / 8; ++q)
                        reinterpret_cast<uint4*>(g_row0 + dst_row * row_stride)[q] = make_uint4(0, 0, 0, 0);
            } else if (ok) {
                const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll 1
                for (int c64 = 0; c64 < D / 64; ++c64) {
                    uint32_t r[64];
                    if (!split) {
                        ptx::tmem_ld32(tO + c64 * 64, r);
                        ptx::tmem_ld32(tO + c64 * 64 + 32, r + 32);
                        ptx::tmem_wait_ld();
                    } else {
                        load_merged(c64 * 64, r);
                        load_merged(c64 * 64 + 32, r + 32);
                    }
                    uint4 v[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        v[q].x = pack_bf16x2(__uint_as_float(r[8 * q + 0]) * inv, __uint_as_float(r[8 * q + 1]) * inv);
                        v[q].y = pack_bf16x2(__uint_as_float(r[8 * q + 2]) * inv, __uint_as_float(r[8 * q + 3]) * inv);
                        v[q].z = pack_bf16x2(__uint_as_float(r[8 * q + 4]) * inv, __uint_as_float(r[8 * q + 5]) * inv);
                        v[q].w = pack_bf16x2(__uint_as_float(r[8 * q + 6]) * inv, __uint_as_float(r[8 * q + 7]) * inv);
                    }
                    store_pieces(v, g_row0 + c64 * 128, row_stride, dst_row);
                }
            }
        } else {
            // unnormalised O and (m, l) of this segment -> its workspace slot
            const size_t item_idx = ((size_t)b * p.H + h) * p.P_cap + it.qp;
            const size_t prow_w = (item_idx * p.max_slots + slot) * (2 * kBM) + (split ? 0 : t) * kBM +
                                  ((warp & 3) << 5);
            if (n_tiles == 0) {
                if (live) p.part_ml[prow_w + lane] = make_float2(-INFINITY, 0.f);
            } else if (ok) {
                uint8_t* g_row0 = reinterpret_cast<uint8_t*>(p.part_o + prow_w * D);
#pragma unroll 1
                for (int ch = 0; ch < D / 32; ++ch) {
                    uint32_t r[32];
                    if (!split) {
                        ptx::tmem_ld32(tO + ch * 32, r);
                        ptx::tmem_wait_ld();
                    } else {
                        load_merged(ch * 32, r);
                    }
                    uint4 v[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) v[q] = make_uint4(r[4 * q], r[4 * q + 1], r[4 * q + 2], r[4 * q + 3]);
                    store_pieces(v, g_row0 + ch * 128, (size_t)D * 4, live ? lane : -1);
                }
                if (live) p.part_ml[prow_w + lane] = make_float2(m, l);
            }
        }
        }   // all roles but the second half of a lone tile
        ptx::fence_proxy_async_smem();      // the next segment's query tile arrives by TMA
    }

    // ---- end of the segment: every role is done with shared and tensor memory ----
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    if (threadIdx.x < kNumBarriers) ptx::mbar_inval(ptx::smem_addr(&ctrl->q_full + threadIdx.x));
    pos = pl.whole_items ? pos + gridDim.x : it.next;
    if (*abort_flag) break;
    }   // segments
}

template <int D, bool STORE>
__device__ __forceinline__ void attention_kernel_body(const CUtensorMap& tm_q, const CUtensorMap& tm_kf,
                                                      const CUtensorMap& tm_vf, const CUtensorMap& tm_kc,
                                                      const CUtensorMap& tm_vc, const AttnParams& p,
                                                      const StoreParams& sp) {
    using Cfg = AttnCfg<D>;
    constexpr int kTileBytes = Cfg::kTileBytes;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_addr(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_addr(smem_raw));
    const uint32_t sQ = smem_base;                      // 2 query tiles
    const uint32_t sKV = smem_base + 2 * kTileBytes;    // ring of K/V stages
    AttnCtrl* ctrl = reinterpret_cast<AttnCtrl*>(smem_gen + Cfg::kSmemTiles);
    volatile int* abort_flag = &ctrl->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    grid_dependency_wait();                             // (everything below reads the launch's inputs)
    // this CTA's share [pos, hi) of the item sequence or of the cost axis
    bool bad = false;
    const Plan pl = plan_shares<STORE>(p, gridDim.x, &bad);
    if (bad && blockIdx.x == 0 && threadIdx.x == 0) record_status(p.dev_status, REGIONE_DEV_BOUNDS);
    // (whole items are dealt round-robin, so that the CTAs running at any one time work on
    // neighbouring items, which share K/V tiles in L2; a share of steps is one contiguous range)
    long long pos = pl.whole_items ? (long long)blockIdx.x : (long long)blockIdx.x * pl.chunk;
    const long long hi = pl.whole_items ? pl.total : min(pos + pl.chunk, pl.total);
    if (pos >= hi) {                                    // uniform for the CTA
        if (threadIdx.x == 0) p.cut[blockIdx.x].valid = 0;
        return;
    }

    grid_launch_dependents();                      // the merge kernel may queue up behind this CTA
    if (threadIdx.x == 0) ctrl->abort_flag = 0;
    if (warp == 9) {
        ptx::tmem_alloc(ptx::smem_addr(&ctrl->tmem_base), 512);
        ptx::tmem_relinquish();
    }
    if (warp >= 8) {
        ptx::reg_dealloc<56>();                         // producer / issuer warpgroup gives registers up
        run_share<D, false, STORE>(&tm_q, &tm_kf, &tm_vf, &tm_kc, &tm_vc, p, sp, pos, hi, pl, ctrl, smem_gen,
                                   sQ, sKV, warp, lane);
    } else {
        ptx::reg_alloc<224>();                          // a row of 128 logits stays in registers
        run_share<D, true, STORE>(&tm_q, &tm_kf, &tm_vf, &tm_kc, &tm_vc, p, sp, pos, hi, pl, ctrl, smem_gen,
                                  sQ, sKV, warp, lane);
    }

    // ================= teardown =================
    if (*abort_flag) {
        // give copies and MMAs that are still in flight time to land before tensor memory and
        // shared memory are given back
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 9) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(ctrl->tmem_base, 512);
    }
}

// The attention kernel, and the one that also refreshes the cache (one parameter more).
template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1)
region_attention_tc_kernel(const __grid_constant__ CUtensorMap tm_q,
                           const __grid_constant__ CUtensorMap tm_kf,
                           const __grid_constant__ CUtensorMap tm_vf,
                           const __grid_constant__ CUtensorMap tm_kc,
                           const __grid_constant__ CUtensorMap tm_vc, const AttnParams p) {
    const StoreParams none = {};
    attention_kernel_body<D, false>(tm_q, tm_kf, tm_vf, tm_kc, tm_vc, p, none);
}
template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1)
region_attention_store_kernel(const __grid_constant__ CUtensorMap tm_q,
                              const __grid_constant__ CUtensorMap tm_kf,
                              const __grid_constant__ CUtensorMap tm_vf,
                              const __grid_constant__ CUtensorMap tm_kc,
                              const __grid_constant__ CUtensorMap tm_vc, const AttnParams p,
                              const StoreParams sp) {
    attention_kernel_body<D, true>(tm_q, tm_kf, tm_vf, tm_kc, tm_vc, p, sp);
}

// Merges the workspace slots of the items that were spread over several shares:
// out = sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s.  blockIdx.x + 1 names a share boundary; the
// attention kernel has left the item cut there (if any) in `cut`.  One warp per query row of the
// item's pair of tiles (blockIdx.y * 8 + warp); a lane owns D / 32 consecutive columns.  The kernel
// is launched behind the attention kernel with programmatic serialization and reads nothing before
// the dependency wait; all slots' loads are issued before the first use, so a warp pays one
// memory round trip, not one per slot.
// MAXS >= AttnParams::max_slots bounds the slots held in registers (the host knows max_slots, and
// the smaller instantiations let more warps be resident).
template <int D, int MAXS>
__global__ void __launch_bounds__(256)
region_attention_combine_kernel(const AttnParams p) {
    constexpr int kCombineMaxSlots = MAXS;
    constexpr int E = D / 32;
    using Vec = typename std::conditional<E == 4, float4, float2>::type;
    grid_dependency_wait();
    const int4* cp = reinterpret_cast<const int4*>(p.cut + blockIdx.x + 1);
    const int4 c0 = cp[0], c1 = cp[1];
    const int b = c0.y, h = c0.z, qp = c0.w, n_slots = c1.x, nq = c1.y;
    // (the fields are checked so that a table left incomplete by an aborted launch cannot send
    // this kernel out of bounds)
    if (c0.x != 1 || b < 0 || b >= p.B || h < 0 || h >= p.H || qp < 0 || qp >= p.P_cap ||
        n_slots < 2 || n_slots > p.max_slots || n_slots > kCombineMaxSlots || nq > p.Nq_cap)
        return;
    const int lane = threadIdx.x & 31;
    const int r_local = blockIdx.y * 8 + (threadIdx.x >> 5);
    const int qrow = qp * (2 * kBM) + r_local;
    if (qrow >= nq) return;
    const size_t item_idx = ((size_t)b * p.H + h) * p.P_cap + qp;
    const size_t prow0 = item_idx * p.max_slots * (2 * kBM) + r_local;
    // (issued together with the slots' loads, used after them)
    const int dst_row = p.out_rows != nullptr ? p.out_rows[(size_t)b * p.Nq_cap + qrow] : qrow;

    float2 ml[kCombineMaxSlots];
    Vec o[kCombineMaxSlots];
#pragma unroll
    for (int s = 0; s < kCombineMaxSlots; ++s) {
        if (s < n_slots) {
            const size_t prow = prow0 + (size_t)s * (2 * kBM);
            ml[s] = p.part_ml[prow];
            o[s] = *reinterpret_cast<const Vec*>(p.part_o + prow * D + lane * E);
        }
    }
    float M = -INFINITY;
#pragma unroll
    for (int s = 0; s < kCombineMaxSlots; ++s)
        if (s < n_slots && ml[s].y > 0.f) M = fmaxf(M, ml[s].x);
    float acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;
    float L = 0.f;
#pragma unroll
    for (int s = 0; s < kCombineMaxSlots; ++s) {
        if (s < n_slots && ml[s].y > 0.f) {           // a slot without keys carries no weight
            const float wgt = fast_exp2(ml[s].x - M);
            L = fmaf(wgt, ml[s].y, L);
            const float* po = reinterpret_cast<const float*>(&o[s]);
#pragma unroll
            for (int e = 0; e < E; ++e) acc[e] = fmaf(wgt, po[e], acc[e]);
        }
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
    if (dst_row < 0 || dst_row >= p.out_cap) {             // destination out of range: dropped
        if (lane == 0) record_status(p.dev_status, REGIONE_DEV_BOUNDS);
        return;
    }
    uint16_t* orow = p.out + (((size_t)b * p.out_cap + dst_row) * p.H + h) * D + lane * E;
    uint32_t packed[E / 2];
#pragma unroll
    for (int e = 0; e < E; e += 2) packed[e / 2] = pack_bf16x2(acc[e] * inv, acc[e + 1] * inv);
    if constexpr (E == 4)
        *reinterpret_cast<uint2*>(orow) = make_uint2(packed[0], packed[1]);
    else
        *reinterpret_cast<uint32_t*>(orow) = packed[0];
}

// Self-test of the bounded wait: one thread waits, through the same wait_bar the attention
// kernel's roles use, on an mbarrier that nobody ever arrives on.  No copy and no tensor-core
// operation is in flight, so giving up is all that happens: the wait must return false after
// `limit` cycles with REGIONE_DEV_TIMEOUT recorded, and the kernel ends normally.
// out[0] = 1 if the wait reported a completed phase (it must not), out[1] = cycles spent waiting.
__global__ void bounded_wait_selftest_kernel(long long limit, int32_t* dev_status, long long* out) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        ptx::mbar_init(ptx::smem_addr(&bar), 1);
        ptx::fence_barrier_init();
        const long long t0 = clock64();
        const bool done = wait_bar(ptx::smem_addr(&bar), 0, &abort_flag, dev_status, limit);
        const long long spent = clock64() - t0;
        if (out != nullptr) {
            out[0] = done ? 1 : 0;
            out[1] = spent;
            out[2] = abort_flag;
        }
        ptx::mbar_inval(ptx::smem_addr(&bar));
    }
}

// ---- host side ---------------------------------------------------------------------------------

constexpr int kMaxDevices = 64;

// Ordinal of the current device, or -1 (no device / an ordinal beyond the per-device caches).
static int current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
    return dev;
}

// SM count of the current device (cached per device; 148 when it cannot be read).
static int sm_count() {
    static int cached[kMaxDevices] = {};
    const int dev = current_device();
    if (dev < 0) return 148;
    int n = __atomic_load_n(&cached[dev], __ATOMIC_ACQUIRE);
    if (n == 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0)
            return 148;
        n = v;
        __atomic_store_n(&cached[dev], n, __ATOMIC_RELEASE);
    }
    return n;
}

// Launch shape from the capacities alone (so the workspace query and the launch agree): a
// persistent grid of one CTA per SM (fewer if there are fewer steps), and enough workspace slots
// per item that the longest item can be spread over the shares it meets at that grid size.
struct LaunchPlan {
    int grid, P_cap, max_slots;
};

static LaunchPlan plan_launch(int B, int Nq_cap, int Nf_cap, int Nc_cap, int H) {
    LaunchPlan lp;
    lp.P_cap = (Nq_cap + 2 * kBM - 1) / (2 * kBM);
    const long long nt_cap = std::max(1, (Nf_cap + kBN - 1) / kBN + (Nc_cap + kBN - 1) / kBN);
    const long long total_cap = (long long)B * H * lp.P_cap * nt_cap;
    lp.grid = (int)std::min<long long>(sm_count(), std::max<long long>(total_cap, 1));
    const long long share = (total_cap + lp.grid - 1) / lp.grid;
    lp.max_slots = (int)std::min<long long>(8, std::max<long long>(2, (nt_cap + share - 1) / share + 1));
    return lp;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* f = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &qres) ==
                cudaSuccess && qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(f);
    }
    return fn;
}

// [B, rows, H, D] bf16 as a 4-D tensor (D, H, rows, B); box = 64 columns x 1 head x 128 rows.
static bool make_map(CUtensorMap* map, const void* base, int B, int rows, int H, int D) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    if (rows <= 0) rows = 1;     // never loaded from; keeps the encoder happy
    cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)H, (cuuint64_t)rows, (cuuint64_t)B};
    cuuint64_t strides[3] = {(cuuint64_t)D * 2, (cuuint64_t)H * D * 2, (cuuint64_t)rows * H * D * 2};
    cuuint32_t box[4] = {64, 1, (cuuint32_t)kBN, 1};
    cuuint32_t elem[4] = {1, 1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box,
              elem, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static inline size_t slot_rows(const LaunchPlan& lp, int B, int H) {
    return (size_t)B * H * lp.P_cap * lp.max_slots * (2 * kBM);
}

size_t region_attention_tc_workspace(int B, int Nq_cap, int Nf_cap, int Nc_cap, int H, int D) {
    const LaunchPlan lp = plan_launch(B, Nq_cap, Nf_cap, Nc_cap, H);
    const size_t rows = slot_rows(lp, B, H);
    return ((rows * D * sizeof(float) + 255) & ~(size_t)255) +
           ((rows * sizeof(float2) + 255) & ~(size_t)255) + (size_t)lp.grid * sizeof(CutItem);
}

template <int D, bool STORE>
static int launch_main(const CUtensorMap* maps, const AttnParams& prm, const StoreParams& sp, int grid,
                       cudaStream_t st) {
    using Cfg = AttnCfg<D>;
    // the opt-in to large dynamic shared memory is a per-device attribute of the kernel
    static int configured[kMaxDevices] = {};
    const int dev = current_device();
    if (dev < 0) return REGIONE_CUDA_ERROR;
    if (!__atomic_load_n(&configured[dev], __ATOMIC_ACQUIRE)) {
        const cudaError_t e =
            STORE ? cudaFuncSetAttribute(region_attention_store_kernel<D>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes)
                  : cudaFuncSetAttribute(region_attention_tc_kernel<D>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes);
        if (e != cudaSuccess) return REGIONE_CUDA_ERROR;
        __atomic_store_n(&configured[dev], 1, __ATOMIC_RELEASE);
    }
    cudaError_t e;
    if constexpr (STORE)
        e = launch_overlapped(region_attention_store_kernel<D>, dim3(grid), dim3(kAttnThreads),
                              Cfg::kSmemBytes, st, maps[0], maps[1], maps[2], maps[3], maps[4], prm, sp);
    else
        e = launch_overlapped(region_attention_tc_kernel<D>, dim3(grid), dim3(kAttnThreads),
                              Cfg::kSmemBytes, st, maps[0], maps[1], maps[2], maps[3], maps[4], prm);
    return e == cudaSuccess ? REGIONE_OK : REGIONE_CUDA_ERROR;
}

template <int D>
static int launch_tc(const CUtensorMap* maps, const AttnParams& prm, const StoreParams* sp, int grid,
                     cudaStream_t st) {
    const StoreParams none = {};
    const int rc = sp != nullptr ? launch_main<D, true>(maps, prm, *sp, grid, st)
                                 : launch_main<D, false>(maps, prm, none, grid, st);
    if (rc != REGIONE_OK) return rc;
    // the merge kernel may become resident while the attention kernel drains (it waits for that
    // kernel's completion before it reads a slot)
    if (grid < 2) return launch_status(cudaGetLastError());     // a single share cuts nothing
    const dim3 cgrid((unsigned)(grid - 1), (2 * kBM) / 8, 1);
    cudaError_t e;
    if (prm.max_slots <= 2)
        e = launch_overlapped(region_attention_combine_kernel<D, 2>, cgrid, dim3(256), 0, st, prm);
    else if (prm.max_slots <= 3)
        e = launch_overlapped(region_attention_combine_kernel<D, 3>, cgrid, dim3(256), 0, st, prm);
    else if (prm.max_slots <= 4)
        e = launch_overlapped(region_attention_combine_kernel<D, 4>, cgrid, dim3(256), 0, st, prm);
    else
        e = launch_overlapped(region_attention_combine_kernel<D, 8>, cgrid, dim3(256), 0, st, prm);
    if (e != cudaSuccess) return REGIONE_CUDA_ERROR;
    return launch_status(cudaGetLastError());
}

int launch_region_attention_tc(const uint16_t* q, const uint16_t* k_fresh, const uint16_t* v_fresh,
                               const uint16_t* k_cache, const uint16_t* v_cache, const int32_t* n_q,
                               const int32_t* n_fresh, const int32_t* n_cache, int B, int Nq_cap,
                               int Nf_cap, int Nc_cap, int H, int D, float scale, uint16_t* out,
                               const int32_t* out_rows, int out_cap, void* workspace,
                               size_t workspace_bytes, int32_t* dev_status, cudaStream_t st,
                               const CacheStore* store) {
    (void)workspace_bytes;
    CUtensorMap maps[5];
    // an absent segment still needs a valid (never dereferenced) base address
    const void* kf = Nf_cap > 0 ? (const void*)k_fresh : (const void*)q;
    const void* vf = Nf_cap > 0 ? (const void*)v_fresh : (const void*)q;
    const void* kc = Nc_cap > 0 ? (const void*)k_cache : (const void*)q;
    const void* vc = Nc_cap > 0 ? (const void*)v_cache : (const void*)q;
    if (!make_map(&maps[0], q, B, Nq_cap, H, D) || !make_map(&maps[1], kf, B, Nf_cap, H, D) ||
        !make_map(&maps[2], vf, B, Nf_cap, H, D) || !make_map(&maps[3], kc, B, Nc_cap, H, D) ||
        !make_map(&maps[4], vc, B, Nc_cap, H, D))
        return REGIONE_CUDA_ERROR;
    const LaunchPlan lp = plan_launch(B, Nq_cap, Nf_cap, Nc_cap, H);
    AttnParams prm;
    prm.n_q = n_q; prm.n_fresh = n_fresh; prm.n_cache = n_cache;
    prm.B = B; prm.Nq_cap = Nq_cap; prm.Nf_cap = Nf_cap; prm.Nc_cap = Nc_cap; prm.H = H;
    prm.P_cap = lp.P_cap; prm.max_slots = lp.max_slots;
    prm.scale_log2e = scale * 1.4426950408889634f;
    prm.out = out; prm.dev_status = dev_status;
    prm.out_rows = out_rows;
    prm.out_cap = out_rows != nullptr ? out_cap : Nq_cap;
    prm.timeout_cycles = kTimeoutCycles;
    StoreParams sp = {};
    if (store != nullptr) {
        sp.keep_rows = store->keep_rows; sp.n_keep = store->n_keep; sp.store_cap = store->cap;
        sp.k_store = store->k_cache; sp.v_store = store->v_cache;
    }
    const size_t rows = slot_rows(lp, B, H);
    prm.part_o = reinterpret_cast<float*>(workspace);
    uint8_t* const ws = reinterpret_cast<uint8_t*>(workspace);
    const size_t off_ml = (rows * D * sizeof(float) + 255) & ~(size_t)255;
    prm.part_ml = reinterpret_cast<float2*>(ws + off_ml);
    prm.cut = reinterpret_cast<CutItem*>(ws + off_ml + ((rows * sizeof(float2) + 255) & ~(size_t)255));
    const StoreParams* spp = store != nullptr ? &sp : nullptr;
    return D == 64 ? launch_tc<64>(maps, prm, spp, lp.grid, st) : launch_tc<128>(maps, prm, spp, lp.grid, st);
}

// ---- variant with library-owned scratch -----------------------------------------------------
// The split-KV partials of regione_region_attention_static live here instead of in a caller
// workspace.  The array is part of the library image: every GPU that loads the library keeps
// these bytes resident until the process exits.
constexpr size_t kStaticScratchBytes = (size_t)64 << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {
void* g_static_scratch_addr[kMaxDevices] = {};      // device address of the array, per device
}  // namespace

// Device address of g_static_scratch on the current device (in host code the symbol itself is
// only a stand-in and must never be handed to a kernel).  Resolved on the first call per device.
static int static_scratch_address(void** out) {
    const int dev = current_device();
    if (dev < 0) return REGIONE_CUDA_ERROR;
    void* addr = __atomic_load_n(&g_static_scratch_addr[dev], __ATOMIC_ACQUIRE);
    if (addr == nullptr) {
        if (cudaGetSymbolAddress(&addr, g_static_scratch) != cudaSuccess || addr == nullptr) {
            (void)cudaGetLastError();
            return REGIONE_CUDA_ERROR;
        }
        __atomic_store_n(&g_static_scratch_addr[dev], addr, __ATOMIC_RELEASE);
    }
    *out = addr;
    return REGIONE_OK;
}

}  // namespace regione

extern "C" int regione_selftest_bounded_wait(long long limit_cycles, int32_t* dev_status,
                                             long long* out, void* stream) {
    using namespace regione;
    // the limit is capped well below the attention kernel's own so that the self-test stays short
    if (limit_cycles < 1 || limit_cycles > 100000000LL) return REGIONE_INVALID_ARG;
    bounded_wait_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(limit_cycles, dev_status, out);
    return launch_status(cudaGetLastError());
}

extern "C" int regione_region_attention_static(
    const regione_bf16* q, const regione_bf16* k_fresh, const regione_bf16* v_fresh,
    const regione_bf16* k_cache, const regione_bf16* v_cache, const int32_t* n_q,
    const int32_t* n_fresh, const int32_t* n_cache, int B, int Nq_cap, int Nf_cap, int Nc_cap, int H,
    int D, float softmax_scale, regione_bf16* out, int32_t* dev_status, void* stream) {
    using namespace regione;
    bool nothing = false;
    const int args_rc = check_attention_args(q, k_fresh, v_fresh, k_cache, v_cache, n_q, n_fresh,
                                             n_cache, B, Nq_cap, Nf_cap, Nc_cap, H, D, out, &nothing);
    if (args_rc != REGIONE_OK || nothing) return args_rc;
    // the partials of this shape must fit the fixed array: refuse, never truncate
    const size_t need = region_attention_tc_workspace(B, Nq_cap, Nf_cap, Nc_cap, H, D);
    if (need > kStaticScratchBytes) return REGIONE_WORKSPACE_TOO_SMALL;
    void* scratch = nullptr;
    const int rc = static_scratch_address(&scratch);
    if (rc != REGIONE_OK) return rc;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)D);
    // Nothing in the scratch has to start at zero: every word the merge kernel reads is written
    // by the attention kernel of the same call, so the previous call's contents are harmless.
    return launch_region_attention_tc(q, k_fresh, v_fresh, k_cache, v_cache, n_q, n_fresh, n_cache,
                                      B, Nq_cap, Nf_cap, Nc_cap, H, D, scale, out, nullptr, 0, scratch,
                                      kStaticScratchBytes, dev_status, (cudaStream_t)stream, nullptr);
}
