// One persistent kernel per forward for head dim 64 at sizes where three launches cost more than
// they compute (the SD-v2.1 and SD-XL 2048 levels): split-N state, fixed-order reduction and apply
// (Prop. 2, Eq. 5) in a single launch, on the same TMA + tcgen05 machinery as stream_kernels.cuh.
//
// Units are (slab, 128-token tile) pairs, numbered slab-major.  The slabs are cut into one or two
// WAVES (wave 0 = slabs [0, split), wave 1 = the rest); inside a wave CTA g of G owns the
// contiguous run [g*U/G, (g+1)*U/G) of the wave's U units.  A CTA walks through
//
//      K/V of its wave-0 run, K/V of its wave-1 run, Q of its wave-0 run, Q of its wave-1 run
//
// as one uninterrupted TMA stream.  The only cross-CTA dependency is "every partial state of slab
// s is summed before anyone applies slab s".  With two waves it costs nothing: the states of the
// wave-0 slabs are exchanged while the CTAs are busy with the K/V of wave 1, those of wave 1 while
// they apply wave 0.  The exchange, per slab, among the P CTAs whose runs meet it (Prop. 2's sum
// over tokens, split over CTAs):
//
//   1. three warps of the state group drain the tensor-memory accumulator into fp32 registers,
//      write the CTA's partial S_p | z_p and add to the slab's first counter (release);
//   2. the state group (four warps) of contributor r waits for all P partials, sums slice r of the
//      state over them in CTA order (fixed order), writes the slice into the slab's fp32 state and
//      adds to the slab's second counter;
//   3. it waits for all P slices, reads the whole state, converts it to the 16-bit B operand
//      S^T | z of the apply MMA in one of two shared-memory buffers and tells the MMA thread.
//
// A slab that lies entirely inside one CTA's run (P = 1) needs none of this: its operand is built
// straight from the registers the accumulator was drained into.
// Every contributor reads the same fp32 state, so all CTAs of a slab apply the same bits.  The
// counters are never reset: each grows by a fixed amount per forward, and an epoch word (advanced
// by the CTA that finishes last) tells a kernel where they stood when it started.  All CTAs must
// be resident together (grid <= SM count, one CTA per SM); a CTA that cannot be placed for a
// while only delays the others, and every wait is bounded.
#pragma once

#include "stream_kernels.cuh"

namespace lf {

struct FusedCfg {
    static constexpr int TILE = 128;
    static constexpr int GROUPS = 3;  // consumer warpgroups
    static constexpr int CONSUMER_WARPS = 4 * GROUPS;
    static constexpr int STATE_WARP0 = CONSUMER_WARPS;  // warps 12..15; 12, 13, 14 = TMEM lane quarters 0, 1, 2
    static constexpr int STATE_WARPS = 4;
    static constexpr int STATE_THREADS = 32 * STATE_WARPS;
    static constexpr int PRODUCER_WARP = CONSUMER_WARPS + 4;
    static constexpr int MMA_WARP = CONSUMER_WARPS + 5;
    static constexpr int STORE_WARP = CONSUMER_WARPS + 6;
    static constexpr int THREADS = 32 * (CONSUMER_WARPS + 7);
    static constexpr int SLOT_BYTES = TILE * kStreamRowBytes;  // 16 KB: one tile of one tensor
    static constexpr int SLOTS = 12;                           // phase 2: one Q / Y tile per slot
    static constexpr int KV_STAGES = SLOTS / 2;                // phase 1: K in slot 2s, V in slot 2s+1
    static constexpr int KV_STAGE_BYTES = 2 * SLOT_BYTES;
    static constexpr int ONES_BYTES = 16 * kStreamRowBytes;
    static constexpr int B_ROWS = StreamApplyCfg::B_ROWS;
    static constexpr int B_BYTES = B_ROWS * kStreamRowBytes;   // 10 KB, two of them
    static constexpr int SEGMENT_TILES = 32;
    static constexpr int TMEM_COLS = 512;        // [0,128): two state accumulators; 128 + 128 g: group g's A | D
    static constexpr int TMEM_APPLY0 = 128;
    static constexpr int TMEM_COLS_PER_GROUP = 128;
    static constexpr int FLUSH_ARRIVALS = 3;     // arrivals on a slab's first counter per contributing CTA
    static constexpr int SLICE_ARRIVALS = 4;     // arrivals on its second counter per contributing CTA
    static constexpr int STATE_VEC4 = kStreamStateFloats / 4;  // 1040 float4: S rows, then z
    static constexpr int SMEM_BYTES = SLOTS * SLOT_BYTES + ONES_BYTES + 2 * B_BYTES + 1024 /*align*/ + 1024 /*barriers*/;
};
static_assert(FusedCfg::STATE_WARP0 % 4 == 0, "flush warps must cover TMEM lane quarters 0, 1, 2");
static_assert((FusedCfg::SLOTS * FusedCfg::SLOT_BYTES + FusedCfg::ONES_BYTES) % 1024 == 0 && FusedCfg::B_BYTES % 1024 == 0,
              "B operands on 1024-byte boundaries");
static_assert(FusedCfg::TMEM_APPLY0 + FusedCfg::GROUPS * FusedCfg::TMEM_COLS_PER_GROUP <= FusedCfg::TMEM_COLS, "TMEM budget");
static_assert(FusedCfg::SMEM_BYTES > 116 * 1024 && FusedCfg::SMEM_BYTES <= 227 * 1024, "one CTA per SM");

// Control words of the fused path in the workspace: ctrl[0] = epoch (forwards completed),
// ctrl[1] = CTAs of the running forward that have finished.
constexpr int kFusedCtrlWords = 2;

// How the units are dealt: `split` = first slab of wave 1 (= slabs when there is one wave).
struct FusedPlan {
    int tiles_per_slab;
    int slabs;
    int split;
    int whole;  // nonzero: runs are made of whole slabs (small slabs: no slab is shared between CTAs)
};

__host__ __device__ __forceinline__ int fused_waves(const FusedPlan& p) { return p.split < p.slabs ? 2 : 1; }
__host__ __device__ __forceinline__ long long fused_wave_units(const FusedPlan& p, int w)
{
    return static_cast<long long>(w == 0 ? p.split : p.slabs - p.split) * p.tiles_per_slab;
}
// Run of CTA g in wave w, in global unit numbers (slab * tiles_per_slab + tile).
__host__ __device__ __forceinline__ void fused_run(const FusedPlan& p, long long g, long long G, int w, long long* b,
                                                   long long* e)
{
    const long long U = fused_wave_units(p, w);
    const long long base = w == 0 ? 0 : static_cast<long long>(p.split) * p.tiles_per_slab;
    if (p.whole != 0) {
        const long long S = U / p.tiles_per_slab;  // the wave's slabs, dealt whole
        *b = base + unit_begin(g, S, G) * p.tiles_per_slab;
        *e = base + unit_begin(g + 1, S, G) * p.tiles_per_slab;
        return;
    }
    *b = base + unit_begin(g, U, G);
    *e = base + unit_begin(g + 1, U, G);
}
// Slabs a run touches.
__host__ __device__ __forceinline__ int fused_run_slabs(long long b, long long e, int tiles_per_slab)
{
    return e > b ? static_cast<int>((e - 1) / tiles_per_slab - b / tiles_per_slab) + 1 : 0;
}

// The walk of one CTA: position `it` of its concatenated runs -> global unit.
struct FusedWalk {
    long long b0, b1;
    int n0, n;  // units in wave 0; in both waves
    __device__ __forceinline__ long long unit(int it) const { return it < n0 ? b0 + it : b1 + (it - n0); }
    // Positions from `it` to the end of its slab within its wave's run.
    __device__ __forceinline__ int left_in_slab(int it, int tiles_per_slab) const
    {
        const long long u = unit(it);
        const int to_slab_end = tiles_per_slab - static_cast<int>(u % tiles_per_slab);
        const int to_run_end = (it < n0 ? n0 : n) - it;
        return to_slab_end < to_run_end ? to_slab_end : to_run_end;
    }
};

__device__ __forceinline__ FusedWalk fused_walk(const FusedPlan& p, long long g, long long G)
{
    FusedWalk w;
    long long e0, e1 = 0;
    fused_run(p, g, G, 0, &w.b0, &e0);
    w.n0 = static_cast<int>(e0 - w.b0);
    w.b1 = 0;
    w.n = w.n0;
    if (fused_waves(p) == 2) {
        fused_run(p, g, G, 1, &w.b1, &e1);
        w.n += static_cast<int>(e1 - w.b1);
    }
    return w;
}

// One warp waits for a counter nobody advances: the bounded wait must give up and leave the error
// word behind.  Run by the library's self-test only.
__global__ void __launch_bounds__(32)
counter_wait_selftest_kernel(uint32_t* __restrict__ status, const uint32_t* __restrict__ ctr)
{
    bool ok = true;
    if (threadIdx.x == 0) ok = counter_wait(ctr, ld_acquire_gpu(ctr), 1u);
    if (!ok) report_wait_expired(status);
}

// CTAs [g0, g1) are those whose wave-w run meets slab `slab` (a slab of wave w).
__device__ __forceinline__ void fused_contributors(const FusedPlan& p, int slab, int w, long long G, int* g0_out, int* g1_out)
{
    long long U = fused_wave_units(p, w);
    long long lo = static_cast<long long>(slab - (w == 0 ? 0 : p.split)) * p.tiles_per_slab, hi = lo + p.tiles_per_slab;
    if (p.whole != 0) {  // the same search over whole slabs
        U /= p.tiles_per_slab;
        lo /= p.tiles_per_slab;
        hi = lo + 1;
    }
    long long g0 = (lo * G) / U;
    while (g0 + 1 < G && unit_begin(g0 + 1, U, G) <= lo) ++g0;
    while (g0 > 0 && unit_begin(g0, U, G) > lo) --g0;
    long long g1 = (hi * G) / U;
    while (g1 < G && unit_begin(g1, U, G) < hi) ++g1;
    while (g1 > 0 && unit_begin(g1 - 1, U, G) >= hi) --g1;
    *g0_out = static_cast<int>(g0);
    *g1_out = static_cast<int>(g1);
}
// Partials CTA g writes before it enters wave w (one per slab its earlier runs touch).
__host__ __device__ __forceinline__ int fused_slots_before_wave(const FusedPlan& p, long long g, long long G, int w)
{
    if (w == 0) return 0;
    long long b, e;
    fused_run(p, g, G, 0, &b, &e);
    return fused_run_slabs(b, e, p.tiles_per_slab);
}
// Index, among the partials CTA g writes (in the order of its walk), of its partial for `slab` of wave w.
__device__ __forceinline__ int fused_partial_slot(const FusedPlan& p, long long g, long long G, int slab, int w)
{
    long long b, e;
    fused_run(p, g, G, w, &b, &e);
    return fused_slots_before_wave(p, g, G, w) + slab - static_cast<int>(b / p.tiles_per_slab);
}

template <int KIND>
__global__ void __launch_bounds__(FusedCfg::THREADS, 1)
stream_fused_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                    const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_y,
                    float* __restrict__ partials, float* __restrict__ state, uint32_t* __restrict__ arrive,
                    uint32_t* __restrict__ ctrl, uint32_t* __restrict__ status, int N, FusedPlan plan, int spans,
                    int H, ApplyScales sc)
{
    using C = FusedCfg;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    unsigned char* ones = smem + C::SLOTS * C::SLOT_BYTES;
    unsigned char* bsm = ones + C::ONES_BYTES;                        // two B operands
    uint64_t* full1 = reinterpret_cast<uint64_t*>(bsm + 2 * C::B_BYTES);  // phase 1, per K/V stage
    uint64_t* empty1 = full1 + C::KV_STAGES;
    uint64_t* k_ready = empty1 + C::KV_STAGES;
    uint64_t* acc_done = k_ready + C::KV_STAGES;  // [2]
    uint64_t* acc_free = acc_done + 2;            // [2]
    uint64_t* full2 = acc_free + 2;               // phase 2, per slot
    uint64_t* empty2 = full2 + C::SLOTS;
    uint64_t* y_ready = empty2 + C::SLOTS;
    uint64_t* a_ready = y_ready + C::SLOTS;       // per group
    uint64_t* mma_done = a_ready + C::GROUPS;     // per group
    uint64_t* b_ready = mma_done + C::GROUPS;     // [2] operand buffer holds the slab's S^T | z
    uint64_t* b_free = b_ready + 2;               // [2] the MMAs that read the buffer are complete
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(b_free + 2);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long G = gridDim.x, g = blockIdx.x;
    const int tiles_per_slab = plan.tiles_per_slab;
    const FusedWalk walk = fused_walk(plan, g, G);
    const int n_units = walk.n;
    uint32_t* arrive2 = arrive + plan.slabs;  // second counter of every slab

    if (tid == 0) {
        for (int s = 0; s < C::KV_STAGES; ++s) {
            mbar_init(&full1[s], 1);
            mbar_init(&empty1[s], 1);
            mbar_init(&k_ready[s], 4);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&acc_done[b], 1);
            mbar_init(&acc_free[b], 3);
            mbar_init(&b_ready[b], C::STATE_WARPS);
            mbar_init(&b_free[b], 1);
        }
        for (int s = 0; s < C::SLOTS; ++s) {
            mbar_init(&full2[s], 1);
            mbar_init(&empty2[s], 1);
            mbar_init(&y_ready[s], 4);
        }
        for (int q = 0; q < C::GROUPS; ++q) {
            mbar_init(&a_ready[q], 4);
            mbar_init(&mma_done[q], 1);
        }
        mbar_fence_init();
    }
    // Constant block of the state MMA's A operand (a one at (token t, row 64); see stream_state_kernel),
    // and the zero rows 65..79 of both B operands, which are never written again.
    for (int i = tid; i < C::ONES_BYTES / 4; i += C::THREADS) reinterpret_cast<uint32_t*>(ones)[i] = 0u;
    for (int i = tid; i < 2 * 15 * 128 / 16; i += C::THREADS)
        reinterpret_cast<uint4*>(bsm + (i / 120) * C::B_BYTES + 65 * 128)[i % 120] = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();
    if (tid < 16)
        *reinterpret_cast<uint16_t*>(ones + tid * 128 + ((tid & 7) << 4)) = static_cast<uint16_t>(ones_pair<KIND>() & 0xffffu);
    fence_proxy_async_smem();
    if (warp == 0) tmem_alloc(tmem_slot, C::TMEM_COLS);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    if (warp == C::PRODUCER_WARP && lane == 0) {
        prefetch_tmap(&tmap_k);
        prefetch_tmap(&tmap_v);
        prefetch_tmap(&tmap_q);
    }
    if (warp == C::STORE_WARP && lane == 0) prefetch_tmap(&tmap_y);
    pdl_launch_dependents();
    pdl_wait();

    if (warp == C::PRODUCER_WARP) {
        // ---------------- producer: K/V tiles of the walk, then its Q tiles ----------------
        if (lane == 0) {
            const uint64_t policy = policy_evict_first();
            bool ok = true;
            int issued1 = 0, issued2 = 0;
            for (int it = 0; it < n_units && ok; ++it) {
                const int s = it % C::KV_STAGES;
                ok = mbar_wait(&empty1[s], ((it / C::KV_STAGES) & 1) ^ 1);
                if (!ok) break;
                const long long u = walk.unit(it);
                const int slab = static_cast<int>(u / tiles_per_slab), tile = static_cast<int>(u % tiles_per_slab);
                unsigned char* dst = smem + s * C::KV_STAGE_BYTES;
                mbar_expect_tx(&full1[s], C::KV_STAGE_BYTES);
                tma_load_4d(dst, &tmap_k, 0, tile * C::TILE, slab % H, slab / H, &full1[s], policy);
                tma_load_4d(dst + C::SLOT_BYTES, &tmap_v, 0, tile * C::TILE, slab % H, slab / H, &full1[s], policy);
                ++issued1;
            }
            for (int it = 0; it < n_units && ok; ++it) {
                const int s2 = it % C::SLOTS;
                if (it < C::SLOTS) {
                    // First use of the slot in this phase: the state MMAs that read K/V stage s2/2 for
                    // the last time must be complete.  (That barrier sees no further arrivals, so its
                    // phase stays put and the parity of that last use can still be waited on.)
                    const int st = s2 / 2;
                    if (st < n_units) {
                        const int last = st + C::KV_STAGES * ((n_units - 1 - st) / C::KV_STAGES);
                        ok = mbar_wait(&empty1[st], (last / C::KV_STAGES) & 1);
                    }
                } else {
                    ok = mbar_wait(&empty2[s2], ((it / C::SLOTS) & 1) ^ 1);
                }
                if (!ok) break;
                const long long u = walk.unit(it);
                const int slab = static_cast<int>(u / tiles_per_slab), tile = static_cast<int>(u % tiles_per_slab);
                mbar_expect_tx(&full2[s2], C::SLOT_BYTES);
                tma_load_4d(smem + s2 * C::SLOT_BYTES, &tmap_q, 0, tile * C::TILE, slab % H, slab / H, &full2[s2], policy);
                ++issued2;
            }
            if (!ok) report_wait_expired(status);
            drain_loads<C::KV_STAGES>(full1, 0, issued1, status);
            drain_loads<C::SLOTS>(full2, 0, issued2, status);
        }
    } else if (warp == C::MMA_WARP) {
        // ---------------- MMA warp: every tcgen05.mma of the CTA is issued by this one thread ----------------
        if (lane == 0) {
            bool ok = true;
            {
                const uint32_t idesc = umma_idesc_f32acc(kind_dtype(KIND), 128, 64, kUmmaAMnMajor | kUmmaBMnMajor);
                const uint32_t ones_addr = smem_u32(ones);
                int cur_slab = -1, in_segment = 0, segments = 0, buf = 1;
                for (int it = 0; it < n_units; ++it) {
                    const int s = it % C::KV_STAGES;
                    const int slab = static_cast<int>(walk.unit(it) / tiles_per_slab);
                    if (slab != cur_slab || in_segment == C::SEGMENT_TILES) {
                        if (cur_slab >= 0) umma_commit(&acc_done[buf]);
                        buf ^= 1;
                        if (segments >= 2 && !mbar_wait(&acc_free[buf], ((segments - 2) >> 1) & 1)) {
                            ok = false;
                            break;
                        }
                        ++segments;
                        cur_slab = slab;
                        in_segment = 0;
                    }
                    if (!mbar_wait(&k_ready[s], (it / C::KV_STAGES) & 1)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint32_t k_addr = smem_u32(smem + s * C::KV_STAGE_BYTES), v_addr = k_addr + C::SLOT_BYTES;
                    const uint32_t d_tmem = tmem_base + buf * 64;
#pragma unroll
                    for (int k = 0; k < C::TILE / 16; ++k) {
                        const uint32_t va = v_addr + k * 2048;
                        const uint64_t a_desc = umma_desc_mnmajor_sw128(va, ones_addr - va, 1024);
                        const uint64_t b_desc = umma_desc_mnmajor_sw128(k_addr + k * 2048, 0, 1024);
                        umma_ss(d_tmem, a_desc, b_desc, idesc, (in_segment == 0 && k == 0) ? 0u : 1u);
                    }
                    ++in_segment;
                    umma_commit(&empty1[s]);
                }
                if (cur_slab >= 0) umma_commit(&acc_done[buf]);
            }
            if (ok) {
                const uint32_t idesc = umma_idesc_f32acc(kind_dtype(KIND), C::TILE, C::B_ROWS);
                int cur_slab = -1, seg = -1;
                uint64_t b_desc = 0;
                for (int it = 0; it < n_units; ++it) {
                    const int q = it % C::GROUPS;
                    const int slab = static_cast<int>(walk.unit(it) / tiles_per_slab);
                    if (slab != cur_slab) {
                        // the MMAs of the slab before are all issued: its buffer is free once they are complete
                        if (seg >= 0) umma_commit(&b_free[seg & 1]);
                        ++seg;
                        if (!mbar_wait(&b_ready[seg & 1], (seg >> 1) & 1)) {
                            ok = false;
                            break;
                        }
                        b_desc = umma_desc_kmajor_sw128(smem_u32(bsm + (seg & 1) * C::B_BYTES));
                        cur_slab = slab;
                    }
                    if (!mbar_wait(&a_ready[q], (it / C::GROUPS) & 1)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint32_t a_tmem = tmem_base + C::TMEM_APPLY0 + q * C::TMEM_COLS_PER_GROUP, d_tmem = a_tmem + 32;
#pragma unroll
                    for (int k = 0; k < 4; ++k) umma_ts(d_tmem, a_tmem + 8 * k, b_desc + 2 * k, idesc, k > 0 ? 1u : 0u);
                    umma_commit(&mma_done[q]);
                }
            }
            if (!ok) report_wait_expired(status);
        }
    } else if (warp == C::STORE_WARP) {
        // ---------------- store warp ----------------
        if (lane == 0) {
            const uint64_t policy = policy_evict_first();
            for (int it = 0; it < n_units; ++it) {
                const int s2 = it % C::SLOTS;
                if (!mbar_wait(&y_ready[s2], (it / C::SLOTS) & 1)) {
                    report_wait_expired(status);
                    break;
                }
                const long long u = walk.unit(it);
                const int slab = static_cast<int>(u / tiles_per_slab), tile = static_cast<int>(u % tiles_per_slab);
                tma_store_4d(&tmap_y, smem + s2 * C::SLOT_BYTES, 0, tile * C::TILE, slab % H, slab / H, policy);
                tma_store_wait_read();
                mbar_arrive(&empty2[s2]);
            }
            tma_store_wait_all();
        }
    } else if (warp >= C::STATE_WARP0 && warp < C::STATE_WARP0 + C::STATE_WARPS) {
        // ---------------- state group: drain accumulators, exchange the slabs' states, build the operands ----------------
        // The walk is a sequence of slab VISITS (maximal runs of units of one slab inside one wave's
        // run), visit k's operand goes to buffer k & 1.  Warps 12..14 drain (TMEM lane quarters
        // 0..2 = rows of S^T, row 64 = z); warp 15 joins for the exchange only.
        const int wq = warp & 3;
        const bool drains = wq < 3;
        const int stid = tid - 32 * C::STATE_WARP0;
        const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(wq * 32) << 16);
        const uint32_t epoch = ld_acquire_gpu(&ctrl[0]);
        const float4* part4 = reinterpret_cast<const float4*>(partials);
        const float scale = sc.operand;
        bool ok = true;

        // The exchange of visit kx through global memory, in two halves so that a CTA whose run
        // meets several slabs delivers its slice of every one of them (first half) before it waits
        // for anybody else's (second half): a CTA that waited for slab s to be complete before it
        // contributed its slice of slab s+1 would chain the slabs' exchanges one behind the other
        // across the grid.  (For a slab that is local to this CTA but could not take the register
        // shortcut, both halves together are a plain copy.)
        struct Visit {
            int slab, P, r, g0, w;
        };
        auto visit_of = [&](int kx) {
            int it = 0;
            for (int i = 0; i < kx; ++i) it += walk.left_in_slab(it, tiles_per_slab);
            Visit v;
            v.slab = static_cast<int>(walk.unit(it) / tiles_per_slab);
            v.w = it < walk.n0 ? 0 : 1;
            int g1;
            fused_contributors(plan, v.slab, v.w, G, &v.g0, &g1);
            v.P = g1 - v.g0;
            v.r = static_cast<int>(g) - v.g0;
            return v;
        };
        // First half (step 2 above): wait for the slab's partials, sum this CTA's slice, deliver it.
        auto exchange_slice = [&](int kx) {
            const Visit vis = visit_of(kx);
            const int slab = vis.slab, w = vis.w, g0 = vis.g0, P = vis.P, r = vis.r;
            // 1. every contributor's partial is written (P = 1: this CTA's own three draining warps)
            int seen = 1;
            if (lane == 0) seen = counter_wait(&arrive[slab], epoch * static_cast<uint32_t>(P * C::FLUSH_ARRIVALS),
                                               static_cast<uint32_t>(P * C::FLUSH_ARRIVALS)) ? 1 : 0;
            seen = __shfl_sync(0xffffffffu, seen, 0);
            __syncwarp();
            if (seen == 0) return false;
            // 2. slice r of the state, summed over the contributors in CTA order
            float4* st4 = reinterpret_cast<float4*>(state + static_cast<size_t>(slab) * kStreamStateFloats);
            {
                // Lane l of every warp keeps the offset of contributor l's partial (at most 32
                // contributors per slab: the host's plan).  Contributor g0 may have entered the
                // slab earlier in its run; the later ones' wave-w runs start inside it.
                size_t my_base = 0;
                if (lane < P) {
                    const int slot = lane == 0 ? fused_partial_slot(plan, g0, G, slab, w)
                                               : fused_slots_before_wave(plan, g0 + lane, G, w);
                    my_base = (static_cast<size_t>(g0 + lane) * spans + slot) * C::STATE_VEC4;
                }
                const int lo = (r * C::STATE_VEC4) / P, hi = ((r + 1) * C::STATE_VEC4) / P;
                const int n_idx = (hi - lo + C::STATE_THREADS - 1) / C::STATE_THREADS;
                const int total = n_idx * P;  // (index, contributor) pairs, index-major
                int i_ld = 0, c_ld = 0, i_ad = 0, c_ad = 0;
                float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int t0 = 0; t0 < total; t0 += 8) {
                    float4 v[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        // uniform across the warp: every lane walks the same (index, contributor) sequence
                        const unsigned long long base = __shfl_sync(0xffffffffu, static_cast<unsigned long long>(my_base), c_ld & 31);
                        const int idx = lo + stid + C::STATE_THREADS * i_ld;
                        v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (t0 + j < total && idx < hi) v[j] = __ldcg(part4 + base + idx);
                        if (++c_ld == P) {
                            c_ld = 0;
                            ++i_ld;
                        }
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        if (t0 + j < total) {
                            if (c_ad == 0) {
                                sum = v[j];
                            } else {
                                sum.x += v[j].x;
                                sum.y += v[j].y;
                                sum.z += v[j].z;
                                sum.w += v[j].w;
                            }
                            if (++c_ad == P) {
                                const int idx = lo + stid + C::STATE_THREADS * i_ad;
                                if (idx < hi) st4[idx] = sum;
                                c_ad = 0;
                                ++i_ad;
                            }
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) red_release_gpu_add(&arrive2[slab], 1u);  // each of the four warps counts once
            return true;
        };
        // Second half (step 3 above): every slice of every contributor is in; build the operand.
        auto exchange_operand = [&](int kx) {
            const Visit vis = visit_of(kx);
            const int slab = vis.slab, P = vis.P;
            float4* st4 = reinterpret_cast<float4*>(state + static_cast<size_t>(slab) * kStreamStateFloats);
            int seen = 1;
            if (lane == 0)
                seen = counter_wait(&arrive2[slab], epoch * static_cast<uint32_t>(P * C::SLICE_ARRIVALS),
                                    static_cast<uint32_t>(P * C::SLICE_ARRIVALS)) ? 1 : 0;
            seen = __shfl_sync(0xffffffffu, seen, 0);
            __syncwarp();
            if (seen == 0) return false;
            // the buffer's previous user (two visits back) must be through
            if (kx >= 2 && !mbar_wait(&b_free[kx & 1], ((kx - 2) >> 1) & 1)) return false;
            // The whole state -> the 16-bit operand.  Thread t takes feature c = t & 63 and output
            // channels 32 (t >> 6) .. + 31: for a fixed channel the lanes' values are neighbours in
            // a row of B (no bank conflicts).
            unsigned char* B = bsm + (kx & 1) * C::B_BYTES;
            {
                const int c = stid & 63, e4_0 = 8 * (stid >> 6);
                float4 v[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] = __ldcg(st4 + c * 16 + e4_0 + j);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float f[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int row = 4 * (e4_0 + j) + i;  // S[c][row] -> B row `row`, column c
                        *reinterpret_cast<uint16_t*>(B + row * 128 + (((c >> 3) ^ (row & 7)) << 4) + (c & 7) * 2) =
                            static_cast<uint16_t>(pack_pair<KIND>(f[i] * scale, 0.0f) & 0xffffu);
                    }
                }
            }
            if (stid < 16) {
                // z[4 t .. 4 t + 3] -> row 64 (64 & 7 = 0: chunks in place)
                const float4 zv = __ldcg(st4 + 1024 + stid);
                uint2 wv;
                wv.x = pack_pair<KIND>(zv.x * scale, zv.y * scale);
                wv.y = pack_pair<KIND>(zv.z * scale, zv.w * scale);
                *reinterpret_cast<uint2*>(B + 64 * 128 + stid * 8) = wv;
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(&b_ready[kx & 1]);
            return true;
        };

        float acc[64];
#pragma unroll
        for (int c = 0; c < 64; ++c) acc[c] = 0.0f;
        int aseg = 0, k = 0, k_s = 0, k_x = 0;  // visits drained; with their slice delivered; with their operand built
        bool visit_from_tile0 = walk.unit(0) % tiles_per_slab == 0;
        for (int it = 0; it < n_units && ok;) {
            const long long u = walk.unit(it);
            const int slab = static_cast<int>(u / tiles_per_slab);
            const int left = walk.left_in_slab(it, tiles_per_slab);
            const int len = left > C::SEGMENT_TILES ? C::SEGMENT_TILES : left;
            const bool visit_ends_slab = static_cast<int>(u % tiles_per_slab) + left == tiles_per_slab;
            it += len;
            const int buf = aseg & 1;
            ok = mbar_wait(&acc_done[buf], (aseg >> 1) & 1);
            ++aseg;
            __syncwarp();
            if (!ok) break;
            if (drains) {
                tc_fence_after_sync();
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    uint32_t d[16];
                    tmem_load_16cols(t_lane + buf * 64 + 16 * q4, d);
#pragma unroll
                    for (int c = 0; c < 16; ++c) acc[16 * q4 + c] += __uint_as_float(d[c]);
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&acc_free[buf]);
            }
            if (len != left) continue;
            // Visit k is complete.  If the whole slab lay inside it, the sum is final.
            const bool local = visit_from_tile0 && visit_ends_slab;
            if (local && k == k_x && k < 2) {
                // operand buffer k is still untouched: build it from the registers, no exchange
                unsigned char* B = bsm + (k & 1) * C::B_BYTES;
                float* dst = state + static_cast<size_t>(slab) * kStreamStateFloats;
                if (wq < 2) {
                    const int e = wq * 32 + lane;  // row e of S^T = column e of S along c = row e of B
#pragma unroll
                    for (int c = 0; c < 64; ++c) dst[c * 64 + e] = acc[c];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        uint4 wv;
                        wv.x = pack_pair<KIND>(acc[8 * j + 0] * scale, acc[8 * j + 1] * scale);
                        wv.y = pack_pair<KIND>(acc[8 * j + 2] * scale, acc[8 * j + 3] * scale);
                        wv.z = pack_pair<KIND>(acc[8 * j + 4] * scale, acc[8 * j + 5] * scale);
                        wv.w = pack_pair<KIND>(acc[8 * j + 6] * scale, acc[8 * j + 7] * scale);
                        *reinterpret_cast<uint4*>(B + e * 128 + ((j ^ (e & 7)) << 4)) = wv;
                    }
                } else if (wq == 2 && lane == 0) {
#pragma unroll
                    for (int c = 0; c < 64; ++c) dst[64 * 64 + c] = acc[c];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        uint4 wv;
                        wv.x = pack_pair<KIND>(acc[8 * j + 0] * scale, acc[8 * j + 1] * scale);
                        wv.y = pack_pair<KIND>(acc[8 * j + 2] * scale, acc[8 * j + 3] * scale);
                        wv.z = pack_pair<KIND>(acc[8 * j + 4] * scale, acc[8 * j + 5] * scale);
                        wv.w = pack_pair<KIND>(acc[8 * j + 6] * scale, acc[8 * j + 7] * scale);
                        *reinterpret_cast<uint4*>(B + 64 * 128 + (j << 4)) = wv;
                    }
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&b_ready[k & 1]);
                k_s = k_x = k + 1;
            } else if (drains) {
                // partial k of this CTA: row e of S^T (lanes 0..63), z (lane 64)
                float* dst = partials + (static_cast<size_t>(g) * spans + k) * kStreamStateFloats;
                if (wq < 2) {
                    const int e = wq * 32 + lane;
#pragma unroll
                    for (int c = 0; c < 64; ++c) dst[c * 64 + e] = acc[c];
                } else if (lane == 0) {
#pragma unroll
                    for (int c = 0; c < 64; ++c) dst[64 * 64 + c] = acc[c];
                }
                // All lanes' stores are ordered before lane 0's release by the warp barrier.
                __syncwarp();
                if (lane == 0) red_release_gpu_add(&arrive[slab], 1u);
            }
            ++k;
            visit_from_tile0 = true;  // the next visit starts a new slab (tile 0) unless it opens a wave's run mid-slab
            if (it < n_units) visit_from_tile0 = walk.unit(it) % tiles_per_slab == 0;
            // Wave 0 is drained and wave 1 is streaming: exchange what fits in the two free buffers now.
            if (it == walk.n0 && walk.n0 < n_units) {
                while (ok && k_s < k) ok = exchange_slice(k_s++);
                while (ok && k_x < k && k_x < 2) ok = exchange_operand(k_x++);
            }
            // (cleared after the exchange, so that the sums are not kept alive across it)
#pragma unroll
            for (int c = 0; c < 64; ++c) acc[c] = 0.0f;
        }
        while (ok && k_s < k) ok = exchange_slice(k_s++);
        while (ok && k_x < k) ok = exchange_operand(k_x++);
        if (!ok && lane == 0) report_wait_expired(status);
    } else {
        // ---------------- consumer warpgroups ----------------
        const int group = warp >> 2, wq = warp & 3;
        const int row = wq * 32 + lane;
        const uint32_t sw = row & 7;
        const uint32_t row_base = smem_u32(smem) + row * 128;
        bool ok = true;
        // phase 1: thread r of group q rewrites token r's K row of every third tile as phi(K)
        for (int it = group; it < n_units; it += C::GROUPS) {
            const int s = it % C::KV_STAGES;
            if (!mbar_wait(&full1[s], (it / C::KV_STAGES) & 1)) {
                ok = false;
                break;
            }
            const int tile = static_cast<int>(walk.unit(it) % tiles_per_slab);
            const uint32_t base = row_base + s * C::KV_STAGE_BYTES;
            if (tile * C::TILE + row < N) {
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    uint32_t x0, x1, x2, x3;
                    const uint32_t addr = base + ((c ^ sw) << 4);
                    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(x0), "=r"(x1), "=r"(x2), "=r"(x3) : "r"(addr));
                    x0 = phi_packed_pair<KIND>(x0);
                    x1 = phi_packed_pair<KIND>(x1);
                    x2 = phi_packed_pair<KIND>(x2);
                    x3 = phi_packed_pair<KIND>(x3);
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(x0), "r"(x1), "r"(x2), "r"(x3)
                                 : "memory");
                }
            }
            // rows past N were zero-filled by TMA and stay zero (phi(0) = 1 must not count)
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(&k_ready[s]);
        }
        // phase 2: group q takes every third Q tile of the walk
        if (ok) {
            const uint32_t a_tmem = tmem_base + (static_cast<uint32_t>(wq * 32) << 16) + C::TMEM_APPLY0 +
                                    group * C::TMEM_COLS_PER_GROUP;
            const uint32_t d_tmem = a_tmem + 32;
            uint32_t tiles_done = 0;
            for (int it = group; it < n_units; it += C::GROUPS) {
                const int s2 = it % C::SLOTS;
                if (!mbar_wait(&full2[s2], (it / C::SLOTS) & 1)) {
                    ok = false;
                    break;
                }
                const uint32_t base = row_base + s2 * C::SLOT_BYTES;
                {
                    uint32_t a[32];
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        uint32_t x0, x1, x2, x3;
                        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                                     : "=r"(x0), "=r"(x1), "=r"(x2), "=r"(x3)
                                     : "r"(base + ((c ^ sw) << 4)));
                        a[4 * c + 0] = phi_packed_pair<KIND>(x0);
                        a[4 * c + 1] = phi_packed_pair<KIND>(x1);
                        a[4 * c + 2] = phi_packed_pair<KIND>(x2);
                        a[4 * c + 3] = phi_packed_pair<KIND>(x3);
                    }
                    tmem_store_32cols(a_tmem, a);
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&a_ready[group]);
                ok = mbar_wait(&mma_done[group], tiles_done & 1);
                ++tiles_done;
                __syncwarp();
                if (!ok) break;
                tc_fence_after_sync();
                const float den = __uint_as_float(tmem_load_1col(d_tmem + 64));  // phi(Q_i) . z
                const float inv = row_scale(den, sc);
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t d[32];
                    tmem_load_32cols(d_tmem + 32 * half, d);
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const uint32_t v0 = pack_pair<KIND>(__uint_as_float(d[8 * c + 0]) * inv, __uint_as_float(d[8 * c + 1]) * inv);
                        const uint32_t v1 = pack_pair<KIND>(__uint_as_float(d[8 * c + 2]) * inv, __uint_as_float(d[8 * c + 3]) * inv);
                        const uint32_t v2 = pack_pair<KIND>(__uint_as_float(d[8 * c + 4]) * inv, __uint_as_float(d[8 * c + 5]) * inv);
                        const uint32_t v3 = pack_pair<KIND>(__uint_as_float(d[8 * c + 6]) * inv, __uint_as_float(d[8 * c + 7]) * inv);
                        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(base + (((4 * half + c) ^ sw) << 4)),
                                     "r"(v0), "r"(v1), "r"(v2), "r"(v3)
                                     : "memory");
                    }
                }
                tc_fence_before_sync();
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&y_ready[s2]);
            }
        }
        if (!ok && lane == 0) report_wait_expired(status);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
    // The CTA that finishes last closes the forward: the counters now stand at (epoch + 1) times
    // their per-forward increments.
    if (tid == 0) {
        __threadfence();
        const uint32_t done = atomicAdd(&ctrl[1], 1u);
        if (done == gridDim.x - 1) {
            ctrl[1] = 0u;
            atomicAdd(&ctrl[0], 1u);
        }
    }
}

}  // namespace lf
