// The attention fed from the layer input X instead of from Q, K, V (head dim 64): the projections
// that produce K and V (and, in producer_apply_kernel, Q) run on tcgen05 inside the kernel that
// consumes them, so that K, V and Q never exist in global memory.
//
//   V = X W_V                                                     (Eq. 2)
//   K = g'(X) = X W_K + T_K,   Q = f'(X) = X W_Q + T_Q            (Sec. 3.1, implementation details)
//
// where T = LeakyReLU(LayerNorm(X W_1 + b_1)) is the output of the non-linear branch, computed
// beforehand by producer_hidden_kernel + producer_norm_kernel (LayerNorm runs over a token's whole
// feature vector, all heads, so it cannot be taken tile by tile per head) and added tile by tile
// here; without that branch (its output is zero at the paper's initialization) T is absent.
//
// producer_state2_kernel — per (batch, head pair) and 128-token tile:
//     D1[128 x 256] = X_tile[128 x C] [W_K,h0 | W_K,h1 | W_V,h0 | W_V,h1]   K loop over C in chunks of 64,
//                                                           operands by TMA (X: K-major; W: [c_in][c_out]
//                                                           rows = MN-major), accumulator in tensor memory
//     epilogue (one warpgroup per head): K = D1 columns (+ T row), phi(K) and V rounded to 16 bits into
//               padded shared-memory tiles; S^T rows += phi(K)^T V and z on warp-level MMAs (Prop. 2, Eq. 5)
//   producer_reduce_kernel sums the CTAs' partial states in CTA order (fixed order).
// producer_apply_kernel — per (batch, head pair) and 128-token tile:
//     D1[128 x 128] = X_tile [W_Q,h0 | W_Q,h1] ; epilogue per head: Q (+ T tile), phi(Q) -> tensor memory as
//     the A operand; D2[128 x 80] = phi(Q) [S | z] ; Y = D2[:, 0:64] / (D2[:, 64] + eps) -> shared -> TMA store
//
// Roles per CTA (one per SM): two producer warps (TMA: X chunks; W chunks), MMA warp (one thread issues
// every tcgen05.mma), two epilogue warpgroups (one per head of the pair), a store warp where Y or U is
// written.  Every wait is bounded.
#pragma once

#include <cuda_fp16.h>

#include "stream_kernels.cuh"

namespace lf {

// 3-D tiled TMA load (x = channel, y = token, z = batch) and 2-D (x = output column, y = input row).
__device__ __forceinline__ void tma_load_3d(void* smem_dst, const void* tmap, int x, int y, int z, uint64_t* bar,
                                            uint64_t cache_policy)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%2, %3, %4}], [%5], %6;" ::"r"(smem_u32(smem_dst)),
        "l"(tmap), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar)), "l"(cache_policy)
        : "memory");
}
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const void* tmap, int x, int y, uint64_t* bar,
                                            uint64_t cache_policy)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%2, %3}], [%4], %5;" ::"r"(smem_u32(smem_dst)),
        "l"(tmap), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(cache_policy)
        : "memory");
}
// Position in a ring of STAGES stages: stage index and the parity of its current use.  The K loops
// below run on one thread each (the TMA issuer, the MMA issuer); at four MMAs per chunk the thread's
// own instruction stream sets the pace, so the loops carry running positions and descriptors instead
// of recomputing them (no divisions, no descriptor assembly per chunk).
template <int STAGES>
struct RingPos {
    int s = 0;
    uint32_t phase = 0;
    __device__ __forceinline__ void next()
    {
        if (++s == STAGES) {
            s = 0;
            phase ^= 1u;
        }
    }
};
// mbar_wait on a shared-memory address that is already 32-bit.
__device__ __forceinline__ bool mbar_wait_addr(uint32_t addr, uint32_t parity)
{
    if (mbar_try_wait(addr, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    do {
        if (mbar_try_wait(addr, parity)) return true;
    } while (global_timer_ns() - t0 < kMaxBarrierWaitNs);
    return false;
}
__device__ __forceinline__ void mbar_expect_tx_addr(uint32_t addr, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(addr), "r"(bytes) : "memory");
}
__device__ __forceinline__ void umma_commit_addr(uint32_t addr)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(addr) : "memory");
}
// TMA loads with shared-memory addresses already 32-bit.
__device__ __forceinline__ void tma_load_3d_addr(uint32_t dst, const void* tmap, int x, int y, int z, uint32_t bar, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%2, %3, %4}], [%5], %6;" ::"r"(dst), "l"(tmap), "r"(x), "r"(y), "r"(z), "r"(bar), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void tma_load_2d_addr(uint32_t dst, const void* tmap, int x, int y, uint32_t bar, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%2, %3}], [%4], %5;" ::"r"(dst), "l"(tmap), "r"(x), "r"(y), "r"(bar), "l"(policy)
        : "memory");
}

// Heads are taken in pairs (2p, 2p + 1); with an odd head count the last pair's second head does
// not exist: its weight boxes and T tile lie past the tensors' extents (TMA fills zeros), and nothing
// of it is stored.
__host__ __device__ __forceinline__ int head_pairs(int H) { return (H + 1) / 2; }

__device__ __forceinline__ uint64_t policy_evict_last()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}

// What the epilogues need besides the accumulator: whether a tile of the non-linear branch's
// output is added, and the token count (rows past it must count for nothing).
struct ProducerArgs {
    int N;        // tokens per batch element
    int H;        // heads
    int chunks;   // C / 64: K-loop length
    int has_t;    // nonzero: T tiles are loaded and added
};

// ---------------------------------------------------------------------------------------------
// State from X, two heads per unit.  One tcgen05.mma costs its issuing thread about 125 cycles
// whatever its N, so the projection runs at N = 256: D1[128 x 256] = X_tile [W_K,h0 | W_K,h1 | W_V,h0 | W_V,h1].
// A double-buffered accumulator of that width is all of tensor memory, so the state contraction
// itself moves to the epilogue warps: group e (four warps) writes phi(K_e) | V_e of the tile into
// padded shared memory and accumulates S_e^T-by-rows with warp-level MMAs, fp32 in registers, exactly
// as the split path does (warp w of the group owns features 16 w .. 16 w + 15 of S and z).
// Units are (batch, head pair, 128-token tile), pair-major; CTA g of G owns a contiguous run; a run is
// a sequence of visits to (batch, head pair)s; partials[((g * spans + visit) * 2 + e)][S 64x64 | z 64].
// ---------------------------------------------------------------------------------------------
struct ProdState2Cfg {
    static constexpr int TILE = 128;
    static constexpr int KC = 64;
    static constexpr int STAGES = 3;
    static constexpr int X_BYTES = TILE * 128;       // 16 KB
    static constexpr int W_BYTES = 4 * KC * 128;     // 32 KB: 64 input rows x four 64-column blocks
    static constexpr int STAGE_BYTES = X_BYTES + W_BYTES;
    static constexpr int PITCH = 144;                // bytes per token row of a staged tile: odd in 16-byte units
    static constexpr int KV_BYTES = 2 * TILE * PITCH;  // phi(K) tile then V tile of one head
    static constexpr int EPI_GROUPS = 2;
    static constexpr int EPI_WARPS = 4 * EPI_GROUPS;
    static constexpr int PRODUCER_WARP = EPI_WARPS;
    static constexpr int MMA_WARP = EPI_WARPS + 1;
    static constexpr int WPRODUCER_WARP = EPI_WARPS + 2;
    static constexpr int THREADS = 32 * (EPI_WARPS + 3);
    static constexpr int TMEM_COLS = 512;            // two projection accumulators of 256 columns
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_GROUPS * KV_BYTES + 1024 + 1024;
};
static_assert(ProdState2Cfg::SMEM_BYTES > 116 * 1024 && ProdState2Cfg::SMEM_BYTES <= 227 * 1024, "one CTA per SM");
static_assert(ProdState2Cfg::STAGE_BYTES % 1024 == 0, "operands on 1024-byte boundaries");

// Barrier over `threads` threads that also tells everybody whether `ok` held for all of them, so
// that a group leaves a loop that contains barriers together or not at all.
__device__ __forceinline__ bool named_barrier_all(int id, int threads, bool ok)
{
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.and.pred p, %2, %3, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"(ok ? 1u : 0u), "r"(id), "r"(threads)
        : "memory");
    return r != 0u;
}

template <int KIND>
__global__ void __launch_bounds__(ProdState2Cfg::THREADS, 1)
producer_state2_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_wk,
                       const __grid_constant__ CUtensorMap tmap_wv, const __nv_bfloat16* __restrict__ t_k,
                       float* __restrict__ partials, uint32_t* __restrict__ status, ProducerArgs pa,
                       int tiles_per_slab, long long W, int spans)
{
    using C = ProdState2Cfg;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    unsigned char* kv = smem + C::STAGES * C::STAGE_BYTES;  // per head of the pair: phi(K) tile | V tile, padded rows
    uint64_t* full = reinterpret_cast<uint64_t*>(kv + C::EPI_GROUPS * C::KV_BYTES);
    uint64_t* empty = full + C::STAGES;
    uint64_t* d1_done = empty + C::STAGES;  // [2]
    uint64_t* d1_free = d1_done + 2;        // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(d1_free + 2);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long G = gridDim.x, g = blockIdx.x;
    const long long u0 = unit_begin(g, W, G), u1 = unit_begin(g + 1, W, G);
    const int n_units = static_cast<int>(u1 - u0);
    const int KCH = pa.chunks;
    const int HP = head_pairs(pa.H);

    if (tid == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            mbar_init(&full[s], 2);
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&d1_done[b], 1);
            mbar_init(&d1_free[b], 8);
        }
        mbar_fence_init();
    }
    if (warp == 0) tmem_alloc(tmem_slot, C::TMEM_COLS);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    if (warp == C::PRODUCER_WARP && lane == 0) prefetch_tmap(&tmap_x);
    if (warp == C::WPRODUCER_WARP && lane == 0) {
        prefetch_tmap(&tmap_wk);
        prefetch_tmap(&tmap_wv);
    }
    pdl_launch_dependents();
    pdl_wait();

    if (warp == C::WPRODUCER_WARP) {
        // ---------------- W producer: [W_K | W_V] chunks of both heads (a head past the last: zero fill) ----------------
        if (lane == 0) {
            const uint64_t pol_w = policy_evict_last();
            const uint32_t full0 = smem_u32(full), empty0 = smem_u32(empty), w0 = smem_u32(smem) + C::X_BYTES;
            RingPos<C::STAGES> r;
            bool ok = true;
            for (int it = 0; it < n_units && ok; ++it) {
                const int h0 = static_cast<int>(((u0 + it) / tiles_per_slab) % HP) * 2;
                for (int kc = 0; kc < KCH; ++kc, r.next()) {
                    ok = mbar_wait_addr(empty0 + 8 * r.s, r.phase ^ 1u);
                    if (!ok) break;
                    const uint32_t dst = w0 + r.s * C::STAGE_BYTES, bar = full0 + 8 * r.s;
                    mbar_expect_tx_addr(bar, C::W_BYTES);
                    // one box per weight matrix: 64 input rows x the 64-column blocks of both heads
                    tma_load_3d_addr(dst, &tmap_wk, 0, kc * C::KC, h0, bar, pol_w);
                    tma_load_3d_addr(dst + 16384, &tmap_wv, 0, kc * C::KC, h0, bar, pol_w);
                }
            }
            if (!ok) report_wait_expired(status);
        }
    } else if (warp == C::PRODUCER_WARP) {
        // ---------------- X producer (its drain covers the W loads too) ----------------
        if (lane == 0) {
            const uint64_t pol_x = policy_evict_first();
            const uint32_t full0 = smem_u32(full), empty0 = smem_u32(empty), x0 = smem_u32(smem);
            RingPos<C::STAGES> r;
            bool ok = true;
            int issued = 0;
            for (int it = 0; it < n_units && ok; ++it) {
                const long long u = u0 + it;
                const int ps = static_cast<int>(u / tiles_per_slab), tile = static_cast<int>(u % tiles_per_slab);
                const int b = ps / HP;
                for (int kc = 0; kc < KCH; ++kc, r.next()) {
                    ok = mbar_wait_addr(empty0 + 8 * r.s, r.phase ^ 1u);
                    if (!ok) break;
                    const uint32_t bar = full0 + 8 * r.s;
                    mbar_expect_tx_addr(bar, C::X_BYTES);
                    tma_load_3d_addr(x0 + r.s * C::STAGE_BYTES, &tmap_x, kc * C::KC, tile * C::TILE, b, bar, pol_x);
                    ++issued;
                }
            }
            if (!ok) report_wait_expired(status);
            drain_loads<C::STAGES>(full, 0, issued, status);
        }
    } else if (warp == C::MMA_WARP) {
        // ---------------- MMA warp: the projections only ----------------
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_f32acc(kind_dtype(KIND), 128, 256, kUmmaBMnMajor);
            const uint64_t a_desc0 = umma_desc_kmajor_sw128(smem_u32(smem));
            const uint64_t b_desc0 = umma_desc_mnmajor_sw128(smem_u32(smem) + C::X_BYTES, C::KC * 128, 1024);
            const uint32_t full0 = smem_u32(full), empty0 = smem_u32(empty);
            RingPos<C::STAGES> r;
            bool ok = true;
            for (int it = 0; it < n_units && ok; ++it) {
                const int buf = it & 1;
                if (it >= 2) ok = mbar_wait(&d1_free[buf], ((it >> 1) - 1) & 1);
                if (!ok) break;
                const uint32_t d1 = tmem_base + buf * 256;
                for (int kc = 0; kc < KCH; ++kc, r.next()) {
                    ok = mbar_wait_addr(full0 + 8 * r.s, r.phase);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint64_t step = static_cast<uint64_t>(r.s * (C::STAGE_BYTES >> 4));
                    const uint64_t a_desc = a_desc0 + step, b_desc = b_desc0 + step;
                    umma_ss(d1, a_desc, b_desc, idesc, kc > 0 ? 1u : 0u);
#pragma unroll
                    for (int k = 1; k < C::KC / 16; ++k) umma_ss(d1, a_desc + 2 * k, b_desc + 128 * k, idesc, 1u);
                    umma_commit_addr(empty0 + 8 * r.s);
                }
                if (!ok) break;
                umma_commit(&d1_done[buf]);
            }
            if (!ok) report_wait_expired(status);
        }
    } else {
        // ---------------- epilogue warpgroups: group e owns head e of every pair ----------------
        const int e = warp >> 2, wg = warp & 3;
        const int row = wg * 32 + lane;
        const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(wg * 32) << 16) + e * 64;  // K_e at +0, V_e at +128
        unsigned char* Ksm = kv + e * C::KV_BYTES;
        unsigned char* Vsm = Ksm + C::TILE * C::PITCH;
        const uint32_t k_row = smem_u32(Ksm) + row * C::PITCH, v_row = smem_u32(Vsm) + row * C::PITCH;
        // ldmatrix.trans lane addressing of the state MMA (A = phi(K)^T from the tile stored [token][feature],
        // B = V from the tile stored [token][channel]); warp wg owns features 16 wg .. 16 wg + 15
        const uint32_t a_off = smem_u32(Ksm) + ((lane & 7) + ((lane >> 4) << 3)) * C::PITCH + (wg * 16 + ((lane >> 3) & 1) * 8) * 2;
        const uint32_t b_off = smem_u32(Vsm) + ((lane & 7) + (((lane >> 3) & 1) << 3)) * C::PITCH + ((lane >> 4) * 8) * 2;
        const uint32_t ones = ones_pair<KIND>();
        const int gq = lane >> 2, tq = lane & 3;
        const int Cdim = pa.H * 64;
        float acc[9][4];
#pragma unroll
        for (int nb = 0; nb < 9; ++nb)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[nb][i] = 0.0f;
        bool ok = true;
        int visit = -1, cur_ps = -1;
        for (int it = 0; it < n_units; ++it) {
            const long long u = u0 + it;
            const int ps = static_cast<int>(u / tiles_per_slab), tile = static_cast<int>(u % tiles_per_slab);
            const int b = ps / HP, h = 2 * (ps % HP) + e;
            const bool head = h < pa.H;
            const int tok = tile * C::TILE + row;
            const bool live = tok < pa.N && head;  // rows past N (and a head that does not exist) count for nothing
            if (ps != cur_ps) {
                cur_ps = ps;
                ++visit;
            }
            // the T row of this token and head, if any, on its way while the projection completes
            uint4 tr[8];
            if (pa.has_t != 0 && live) {
                const uint4* src = reinterpret_cast<const uint4*>(t_k + (static_cast<size_t>(b) * pa.N + tok) * Cdim + h * 64);
#pragma unroll
                for (int c = 0; c < 8; ++c) tr[c] = ld_stream_16B(src + c);
            }
            const int buf = it & 1;
            ok = named_barrier_all(3 + e, 128, mbar_wait(&d1_done[buf], (it >> 1) & 1));
            if (!ok) break;
            tc_fence_after_sync();
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t d[32];
                tmem_load_32cols(t_lane + buf * 256 + 32 * half, d);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    float f[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(d[8 * c + i]);
                    if (pa.has_t != 0 && live) {
                        const uint4 t4 = tr[4 * half + c];
                        f[0] += pair_lo<KIND>(t4.x); f[1] += pair_hi<KIND>(t4.x);
                        f[2] += pair_lo<KIND>(t4.y); f[3] += pair_hi<KIND>(t4.y);
                        f[4] += pair_lo<KIND>(t4.z); f[5] += pair_hi<KIND>(t4.z);
                        f[6] += pair_lo<KIND>(t4.w); f[7] += pair_hi<KIND>(t4.w);
                    }
                    uint32_t p0 = 0u, p1 = 0u, p2 = 0u, p3 = 0u;
                    if (live) {
                        p0 = pack_pair<KIND>(phi<KIND>(f[0]), phi<KIND>(f[1]));
                        p1 = pack_pair<KIND>(phi<KIND>(f[2]), phi<KIND>(f[3]));
                        p2 = pack_pair<KIND>(phi<KIND>(f[4]), phi<KIND>(f[5]));
                        p3 = pack_pair<KIND>(phi<KIND>(f[6]), phi<KIND>(f[7]));
                    }
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(k_row + (4 * half + c) * 16), "r"(p0), "r"(p1),
                                 "r"(p2), "r"(p3)
                                 : "memory");
                }
            }
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t d[32];
                tmem_load_32cols(t_lane + buf * 256 + 128 + 32 * half, d);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint32_t p0 = pack_pair<KIND>(__uint_as_float(d[8 * c + 0]), __uint_as_float(d[8 * c + 1]));
                    const uint32_t p1 = pack_pair<KIND>(__uint_as_float(d[8 * c + 2]), __uint_as_float(d[8 * c + 3]));
                    const uint32_t p2 = pack_pair<KIND>(__uint_as_float(d[8 * c + 4]), __uint_as_float(d[8 * c + 5]));
                    const uint32_t p3 = pack_pair<KIND>(__uint_as_float(d[8 * c + 6]), __uint_as_float(d[8 * c + 7]));
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(v_row + (4 * half + c) * 16), "r"(p0), "r"(p1),
                                 "r"(p2), "r"(p3)
                                 : "memory");
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&d1_free[buf]);
            named_barrier_sync(1 + e, 128);  // the group's tiles are complete
            // S^T rows 16 wg .. += phi(K)^T V over the tile's 128 tokens, z from a block of ones
#pragma unroll
            for (int ks = 0; ks < C::TILE / 16; ++ks) {
                uint32_t a0, a1, a2, a3;
                ldmatrix_x4_trans(a_off + ks * 16 * C::PITCH, a0, a1, a2, a3);
#pragma unroll
                for (int nbp = 0; nbp < 4; ++nbp) {
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4_trans(b_off + ks * 16 * C::PITCH + nbp * 32, b0, b1, b2, b3);
                    mma_16816<KIND>(acc[2 * nbp], a0, a1, a2, a3, b0, b1);
                    mma_16816<KIND>(acc[2 * nbp + 1], a0, a1, a2, a3, b2, b3);
                }
                mma_16816<KIND>(acc[8], a0, a1, a2, a3, ones, ones);
            }
            named_barrier_sync(1 + e, 128);  // everybody has read the tiles: the next unit may overwrite them
            const bool visit_ends = it + 1 == n_units || static_cast<int>((u + 1) / tiles_per_slab) != ps;
            if (visit_ends) {
                // this CTA's share of slab (b, h): S [64][64] (row = feature c) then z [64]
                if (head) {
                    float* dst = partials + ((static_cast<size_t>(g) * spans + visit) * 2 + e) * kStreamStateFloats;
                    const int c0 = wg * 16 + gq, c1 = c0 + 8;
#pragma unroll
                    for (int nb = 0; nb < 8; ++nb) {
                        const int ee = nb * 8 + 2 * tq;
                        *reinterpret_cast<float2*>(dst + c0 * 64 + ee) = make_float2(acc[nb][0], acc[nb][1]);
                        *reinterpret_cast<float2*>(dst + c1 * 64 + ee) = make_float2(acc[nb][2], acc[nb][3]);
                    }
                    if (tq == 0) {
                        dst[64 * 64 + c0] = acc[8][0];
                        dst[64 * 64 + c1] = acc[8][2];
                    }
                }
#pragma unroll
                for (int nb = 0; nb < 9; ++nb)
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[nb][i] = 0.0f;
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
}

// The second stage for producer_state2_kernel's partials: grid (17, slabs), 256 threads; slab (b, h) is
// head h % 2 of pair-slab (b, h / 2); its partials come from the CTAs whose run meets that pair-slab,
// summed in CTA order.  Output as stream_reduce_kernel's: fp32 S | z, the 16-bit operand image, the tile counter.
__global__ void __launch_bounds__(256)
producer_reduce_kernel(const float* __restrict__ partials, float* __restrict__ state,
                       unsigned char* __restrict__ operand, int* __restrict__ tile_counters, int tiles_per_slab,
                       long long W, int G, int spans, int H, int dtype, float operand_scale)
{
    __shared__ float sums[256];
    const int tid = threadIdx.x;
    const int idx = blockIdx.x * 256 + tid;
    const int slab = blockIdx.y;
    pdl_launch_dependents();
    pdl_wait();
    if (blockIdx.x == 0 && tid == 0) tile_counters[slab] = 0;
    float sum = 0.0f;
    if (idx < kStreamStateFloats) {
        const int HP = head_pairs(H);
        const int ps = (slab / H) * HP + (slab % H) / 2, e = (slab % H) & 1;
        const long long lo = static_cast<long long>(ps) * tiles_per_slab, hi = lo + tiles_per_slab;
        long long g0 = (lo * G) / W;
        while (g0 + 1 < G && unit_begin(g0 + 1, W, G) <= lo) ++g0;
        while (g0 > 0 && unit_begin(g0, W, G) > lo) --g0;
        long long g1 = (hi * G) / W;
        while (g1 < G && unit_begin(g1, W, G) < hi) ++g1;
        while (g1 > 0 && unit_begin(g1 - 1, W, G) >= hi) --g1;
        // visit index of pair-slab ps in CTA g0's run; every later CTA starts inside it (its visit 0)
        const int slot0 = ps - static_cast<int>(unit_begin(g0, W, G) / tiles_per_slab);
        const size_t F = kStreamStateFloats;
        const float* src = partials + idx;
        sum += src[((static_cast<size_t>(g0) * spans + slot0) * 2 + e) * F];
#pragma unroll 4
        for (long long g = g0 + 1; g < g1; ++g) sum += src[((static_cast<size_t>(g) * spans) * 2 + e) * F];
        state[static_cast<size_t>(slab) * F + idx] = sum;
    }
    sums[tid] = sum;
    __syncthreads();
    emit_state_operand(sums, operand + static_cast<size_t>(slab) * kStreamOperandBytes, dtype, operand_scale);
}

struct ProdApplyCfg {
    static constexpr int TILE = 128;
    static constexpr int KC = 64;
    // One tcgen05.mma of this thread costs about 125 cycles to issue whatever its N (measured: the
    // K loop took the same time per chunk with N = 64 as with N = 128), so a unit takes TWO heads:
    // D1[128 x 128] = X_tile [W_Q,h0 | W_Q,h1], twice the work per instruction.
    static constexpr int STAGES = 4;
    static constexpr int X_BYTES = TILE * 128;     // 16 KB
    static constexpr int W_BYTES = 2 * KC * 128;   // 16 KB: 64 input rows x (64 | 64) Q columns of the two heads
    static constexpr int STAGE_BYTES = X_BYTES + W_BYTES;
    static constexpr int Y_BYTES = TILE * 128;     // per head of the pair: T tile in, Y tile out
    static constexpr int B_ROWS = StreamApplyCfg::B_ROWS;
    static constexpr int B_BYTES = StreamApplyCfg::B_BYTES;  // S^T | z operand image of one head
    static constexpr int EPI_GROUPS = 2;           // group e works on head e of every pair
    static constexpr int EPI_WARPS = 4 * EPI_GROUPS;
    static constexpr int PRODUCER_WARP = EPI_WARPS;
    static constexpr int MMA_WARP = EPI_WARPS + 1;
    static constexpr int STORE_WARP = EPI_WARPS + 2;
    static constexpr int WPRODUCER_WARP = EPI_WARPS + 3;  // W chunks (the producer warp issues the X chunks)
    static constexpr int THREADS = 32 * (EPI_WARPS + 4);
    static constexpr int TMEM_COLS = 512;
    // [0,256): two projection accumulators of 128 columns; per head e: phi(Q) operand (32) and output accumulator (80)
    static constexpr int TMEM_A0 = 256, TMEM_A_STEP = 32, TMEM_D2_0 = 320, TMEM_D2_STEP = 80;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_GROUPS * Y_BYTES + 4 * B_BYTES + 1024 + 1024;
};
static_assert((ProdApplyCfg::STAGES * ProdApplyCfg::STAGE_BYTES + ProdApplyCfg::EPI_GROUPS * ProdApplyCfg::Y_BYTES) % 1024 == 0 &&
                  ProdApplyCfg::B_BYTES % 1024 == 0 && ProdApplyCfg::STAGE_BYTES % 1024 == 0,
              "operands on 1024-byte boundaries");
static_assert(ProdApplyCfg::TMEM_D2_0 + 2 * ProdApplyCfg::TMEM_D2_STEP <= ProdApplyCfg::TMEM_COLS, "TMEM budget");
static_assert(ProdApplyCfg::SMEM_BYTES > 116 * 1024 && ProdApplyCfg::SMEM_BYTES <= 227 * 1024, "one CTA per SM");

// Y from X and the reduced state.  Units are (batch, head pair, 128-token tile), numbered
// pair-major; CTA g of G owns the contiguous run [g*W/G, (g+1)*W/G).  A run is a sequence of VISITS
// to (batch, head pair)s; visit k's two operand images S^T | z go to shared-memory buffers 2 (k & 1) + e.
template <int KIND>
__global__ void __launch_bounds__(ProdApplyCfg::THREADS, 1)
producer_apply_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_wq,
                      const __grid_constant__ CUtensorMap tmap_t, const __grid_constant__ CUtensorMap tmap_y,
                      const unsigned char* __restrict__ operand, uint32_t* __restrict__ status, ProducerArgs pa,
                      int tiles_per_slab, long long W, ApplyScales sc)
{
    using C = ProdApplyCfg;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    unsigned char* ybuf = smem + C::STAGES * C::STAGE_BYTES;
    unsigned char* bsm = ybuf + C::EPI_GROUPS * C::Y_BYTES;
    uint64_t* full = reinterpret_cast<uint64_t*>(bsm + 4 * C::B_BYTES);
    uint64_t* empty = full + C::STAGES;
    uint64_t* d1_done = empty + C::STAGES;  // [2] projection accumulator (unit parity) complete
    uint64_t* d1_free = d1_done + 2;        // [2] read by both heads' epilogues
    uint64_t* t_full = d1_free + 2;         // [2] per head: T tile landed in the head's tile buffer
    uint64_t* a_ready = t_full + 2;         // [2] per head: phi(Q) rows in tensor memory
    uint64_t* d2_done = a_ready + 2;        // [2] per head: output accumulator complete
    uint64_t* y_ready = d2_done + 2;        // [2] per head: Y tile in the tile buffer
    uint64_t* y_free = y_ready + 2;         // [2] per head: the store has read it
    uint64_t* b_ready = y_free + 2;         // [2] per visit parity: operand images in shared memory
    uint64_t* b_free = b_ready + 2;         // [2] the MMAs that read them are complete
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(b_free + 2);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long G = gridDim.x, g = blockIdx.x;
    const long long u0 = unit_begin(g, W, G), u1 = unit_begin(g + 1, W, G);
    const int n_units = static_cast<int>(u1 - u0);
    const int KCH = pa.chunks;
    const int HP = head_pairs(pa.H);

    if (tid == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            mbar_init(&full[s], 2);  // the X and the W issuer each announce their bytes
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&d1_done[b], 1);
            mbar_init(&d1_free[b], 8);
            mbar_init(&t_full[b], 1);
            mbar_init(&a_ready[b], 4);
            mbar_init(&d2_done[b], 1);
            mbar_init(&y_ready[b], 4);
            mbar_init(&y_free[b], 1);
            mbar_init(&b_ready[b], 1);
            mbar_init(&b_free[b], 1);
        }
        mbar_fence_init();
    }
    if (warp == 0) tmem_alloc(tmem_slot, C::TMEM_COLS);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    if (warp == C::PRODUCER_WARP && lane == 0) {
        prefetch_tmap(&tmap_x);
        if (pa.has_t != 0) prefetch_tmap(&tmap_t);
    }
    if (warp == C::WPRODUCER_WARP && lane == 0) prefetch_tmap(&tmap_wq);
    if (warp == C::STORE_WARP && lane == 0) prefetch_tmap(&tmap_y);
    pdl_launch_dependents();
    pdl_wait();

    if (warp == C::WPRODUCER_WARP) {
        // ---------------- W producer: the weight chunks of every unit ----------------
        if (lane == 0) {
            const uint64_t pol_w = policy_evict_last();
            const uint32_t full0 = smem_u32(full), empty0 = smem_u32(empty), w0 = smem_u32(smem) + C::X_BYTES;
            RingPos<C::STAGES> r;
            bool ok = true;
            for (int it = 0; it < n_units && ok; ++it) {
                const int h0 = static_cast<int>(((u0 + it) / tiles_per_slab) % HP) * 2;
                for (int kc = 0; kc < KCH; ++kc, r.next()) {
                    ok = mbar_wait_addr(empty0 + 8 * r.s, r.phase ^ 1u);
                    if (!ok) break;
                    const uint32_t bar = full0 + 8 * r.s;
                    mbar_expect_tx_addr(bar, C::W_BYTES);
                    // one box: 64 input rows x the 64-column blocks of both heads
                    tma_load_3d_addr(w0 + r.s * C::STAGE_BYTES, &tmap_wq, 0, kc * C::KC, h0, bar, pol_w);
                }
            }
            if (!ok) report_wait_expired(status);
        }
    } else if (warp == C::PRODUCER_WARP) {
        // ---------------- producer warp (lane 0 issues the X chunks and T tiles; all lanes copy the
        // operand images; its drain at the end covers the W loads too) ----------------
        uint64_t pol_x = 0;
        if (lane == 0) pol_x = policy_evict_first();
        const uint32_t full0 = smem_u32(full), empty0 = smem_u32(empty), x0 = smem_u32(smem);
        RingPos<C::STAGES> r;
        bool ok = true;
        int issued = 0, visit = -1, cur_ps = -1;
        for (int it = 0; it < n_units && ok; ++it) {
            const long long u = u0 + it;
            const int ps = static_cast<int>(u / tiles_per_slab), tile = static_cast<int>(u % tiles_per_slab);
            const int b = ps / HP, h0 = 2 * (ps % HP);
            if (lane == 0) {
                for (int kc = 0; kc < KCH; ++kc, r.next()) {
                    ok = mbar_wait_addr(empty0 + 8 * r.s, r.phase ^ 1u);
                    if (!ok) break;
                    const uint32_t bar = full0 + 8 * r.s;
                    mbar_expect_tx_addr(bar, C::X_BYTES);
                    tma_load_3d_addr(x0 + r.s * C::STAGE_BYTES, &tmap_x, kc * C::KC, tile * C::TILE, b, bar, pol_x);
                    ++issued;
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            if (ps != cur_ps) {
                // A new visit: its operand images, after the unit's own loads are on their way (the MMA
                // thread frees the buffers of two visits back only once it reaches the visit before this one).
                cur_ps = ps;
                ++visit;
                if (visit >= 2) {
                    if (lane == 0) ok = mbar_wait(&b_free[visit & 1], ((visit >> 1) - 1) & 1);
                    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                    if (!ok) break;
                }
                for (int e = 0; e < 2; ++e) {
                    if (h0 + e >= pa.H) break;
                    const int slab = b * pa.H + h0 + e;
                    const uint4* src = reinterpret_cast<const uint4*>(operand + static_cast<size_t>(slab) * C::B_BYTES);
                    uint4* dst = reinterpret_cast<uint4*>(bsm + (2 * (visit & 1) + e) * C::B_BYTES);
                    for (int i = lane; i < C::B_BYTES / 16; i += 32) dst[i] = __ldg(src + i);
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&b_ready[visit & 1]);
            }
            if (pa.has_t != 0 && lane == 0) {
                // T tiles of the two heads into their tile buffers, once the stores of the unit before
                // have read them (a head past the last one: the box lies outside the tensor, zeros)
                for (int e = 0; e < 2 && ok; ++e) {
                    if (it >= 1) ok = mbar_wait(&y_free[e], (it - 1) & 1);
                    if (ok) {
                        mbar_expect_tx(&t_full[e], C::Y_BYTES);
                        tma_load_4d(ybuf + e * C::Y_BYTES, &tmap_t, 0, tile * C::TILE, h0 + e, b, &t_full[e], pol_x);
                    }
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        }
        if (lane == 0) {
            if (!ok) report_wait_expired(status);
            drain_loads<C::STAGES>(full, 0, issued, status);
        }
    } else if (warp == C::MMA_WARP) {
        // ---------------- MMA warp ----------------
        if (lane == 0) {
            const uint32_t idesc1 = umma_idesc_f32acc(kind_dtype(KIND), 128, 128, kUmmaBMnMajor);
            const uint32_t idesc2 = umma_idesc_f32acc(kind_dtype(KIND), C::TILE, C::B_ROWS);
            bool ok = true;
            int visit = -1, cur_ps = -1;
            uint64_t b_desc[2] = {0, 0};
            // Output MMAs of unit j, head by head: D2_e = phi(Q_e) [S_e | z_e].
            auto apply_mma = [&](int j) {
                const int ps = static_cast<int>((u0 + j) / tiles_per_slab);
                if (ps != cur_ps) {
                    if (visit >= 0) umma_commit(&b_free[visit & 1]);  // the visit before: all its MMAs are issued
                    ++visit;
                    cur_ps = ps;
                    if (!mbar_wait(&b_ready[visit & 1], (visit >> 1) & 1)) return false;
                    b_desc[0] = umma_desc_kmajor_sw128(smem_u32(bsm + (2 * (visit & 1)) * C::B_BYTES));
                    b_desc[1] = umma_desc_kmajor_sw128(smem_u32(bsm + (2 * (visit & 1) + 1) * C::B_BYTES));
                }
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    if (!mbar_wait(&a_ready[e], j & 1)) return false;
                    tc_fence_after_sync();
                    const uint32_t a_tmem = tmem_base + C::TMEM_A0 + e * C::TMEM_A_STEP;
                    const uint32_t d_tmem = tmem_base + C::TMEM_D2_0 + e * C::TMEM_D2_STEP;
#pragma unroll
                    for (int k = 0; k < 4; ++k) umma_ts(d_tmem, a_tmem + 8 * k, b_desc[e] + 2 * k, idesc2, k > 0 ? 1u : 0u);
                    umma_commit(&d2_done[e]);
                }
                return true;
            };
            // Descriptors of stage 0 (a stage further on adds STAGE_BYTES / 16 to the address field); the W
            // chunk's two 64-column blocks (the two heads) are 8 KB apart.
            const uint64_t a_desc0 = umma_desc_kmajor_sw128(smem_u32(smem));
            const uint64_t w_desc0 = umma_desc_mnmajor_sw128(smem_u32(smem) + C::X_BYTES, C::KC * 128, 1024);
            const uint32_t full0 = smem_u32(full), empty0 = smem_u32(empty);
            RingPos<C::STAGES> r;
            for (int it = 0; it < n_units && ok; ++it) {
                const int buf = it & 1;
                if (it >= 2) ok = mbar_wait(&d1_free[buf], ((it >> 1) - 1) & 1);
                if (!ok) break;
                const uint32_t d1 = tmem_base + buf * 128;
                for (int kc = 0; kc < KCH; ++kc, r.next()) {
                    ok = mbar_wait_addr(full0 + 8 * r.s, r.phase);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint64_t step = static_cast<uint64_t>(r.s * (C::STAGE_BYTES >> 4));
                    const uint64_t a_desc = a_desc0 + step, w_desc = w_desc0 + step;
                    umma_ss(d1, a_desc, w_desc, idesc1, kc > 0 ? 1u : 0u);
#pragma unroll
                    for (int k = 1; k < C::KC / 16; ++k) umma_ss(d1, a_desc + 2 * k, w_desc + 128 * k, idesc1, 1u);
                    umma_commit_addr(empty0 + 8 * r.s);
                }
                if (!ok) break;
                umma_commit(&d1_done[buf]);
                if (it >= 1) ok = apply_mma(it - 1);
            }
            if (ok && n_units > 0) ok = apply_mma(n_units - 1);
            if (!ok) report_wait_expired(status);
        }
    } else if (warp == C::STORE_WARP) {
        // ---------------- store warp ----------------
        if (lane == 0) {
            const uint64_t policy = policy_evict_first();
            bool ok = true;
            for (int it = 0; it < n_units && ok; ++it) {
                const long long u = u0 + it;
                const int ps = static_cast<int>(u / tiles_per_slab), tile = static_cast<int>(u % tiles_per_slab);
                const int b = ps / HP, h0 = 2 * (ps % HP);
                for (int e = 0; e < 2; ++e) {
                    if (!mbar_wait(&y_ready[e], it & 1)) {
                        report_wait_expired(status);
                        ok = false;
                        break;
                    }
                    if (h0 + e < pa.H) {
                        tma_store_4d(&tmap_y, ybuf + e * C::Y_BYTES, 0, tile * C::TILE, h0 + e, b, policy);
                        tma_store_wait_read();
                    }
                    mbar_arrive(&y_free[e]);
                }
            }
            tma_store_wait_all();
        }
    } else {
        // ---------------- epilogue warpgroups: group e works on head e of every unit's pair ----------------
        const int e = warp >> 2, wq = warp & 3;
        const int row = wq * 32 + lane;
        const uint32_t sw = row & 7;
        const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(wq * 32) << 16);
        const uint32_t a_tmem = t_lane + C::TMEM_A0 + e * C::TMEM_A_STEP;
        const uint32_t d2_tmem = t_lane + C::TMEM_D2_0 + e * C::TMEM_D2_STEP;
        const uint32_t y_row = smem_u32(ybuf + e * C::Y_BYTES) + row * 128;
        bool ok = true;
        for (int it = 0; it < n_units; ++it) {
            const int buf = it & 1;
            ok = mbar_wait(&d1_done[buf], (it >> 1) & 1);
            if (ok && pa.has_t != 0) ok = mbar_wait(&t_full[e], it & 1);
            __syncwarp();
            if (!ok) break;
            tc_fence_after_sync();
            {
                // Q row of this head (+ T row), phi in fp32, rounded: the row of the output MMA's A operand
                uint32_t a[32];
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t d[32];
                    tmem_load_32cols(t_lane + buf * 128 + e * 64 + 32 * half, d);
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        float f[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(d[8 * c + i]);
                        if (pa.has_t != 0) {
                            uint32_t t0, t1, t2, t3;
                            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                                         : "=r"(t0), "=r"(t1), "=r"(t2), "=r"(t3)
                                         : "r"(y_row + (((4 * half + c) ^ sw) << 4)));
                            f[0] += pair_lo<KIND>(t0); f[1] += pair_hi<KIND>(t0);
                            f[2] += pair_lo<KIND>(t1); f[3] += pair_hi<KIND>(t1);
                            f[4] += pair_lo<KIND>(t2); f[5] += pair_hi<KIND>(t2);
                            f[6] += pair_lo<KIND>(t3); f[7] += pair_hi<KIND>(t3);
                        }
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            a[16 * half + 4 * c + i] = pack_pair<KIND>(phi<KIND>(f[2 * i]), phi<KIND>(f[2 * i + 1]));
                    }
                }
                tmem_store_32cols(a_tmem, a);
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&d1_free[buf]);
                mbar_arrive(&a_ready[e]);
            }
            ok = mbar_wait(&d2_done[e], it & 1);
            // without a T tile nobody has waited yet for the store of the unit before to let go of the buffer
            if (ok && pa.has_t == 0 && it >= 1) ok = mbar_wait(&y_free[e], (it - 1) & 1);
            __syncwarp();
            if (!ok) break;
            tc_fence_after_sync();
            const float den = __uint_as_float(tmem_load_1col(d2_tmem + 64));  // phi(Q_i) . z
            const float inv = row_scale(den, sc);
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t d[32];
                tmem_load_32cols(d2_tmem + 32 * half, d);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint32_t v0 = pack_pair<KIND>(__uint_as_float(d[8 * c + 0]) * inv, __uint_as_float(d[8 * c + 1]) * inv);
                    const uint32_t v1 = pack_pair<KIND>(__uint_as_float(d[8 * c + 2]) * inv, __uint_as_float(d[8 * c + 3]) * inv);
                    const uint32_t v2 = pack_pair<KIND>(__uint_as_float(d[8 * c + 4]) * inv, __uint_as_float(d[8 * c + 5]) * inv);
                    const uint32_t v3 = pack_pair<KIND>(__uint_as_float(d[8 * c + 6]) * inv, __uint_as_float(d[8 * c + 7]) * inv);
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(y_row + (((4 * half + c) ^ sw) << 4)),
                                 "r"(v0), "r"(v1), "r"(v2), "r"(v3)
                                 : "memory");
                }
            }
            tc_fence_before_sync();
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(&y_ready[e]);
        }
        if (!ok && lane == 0) report_wait_expired(status);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

// 3-D tiled TMA store (x = channel, y = token, z = batch), clipped at the tensor's extents.
__device__ __forceinline__ void tma_store_3d(const void* tmap, const void* smem_src, int x, int y, int z,
                                             uint64_t cache_policy)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group.L2::cache_hint [%0, {%1, %2, %3}], [%4], %5;"
        ::"l"(tmap), "r"(x), "r"(y), "r"(z), "r"(smem_u32(smem_src)), "l"(cache_policy)
        : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

// ---------------------------------------------------------------------------------------------
// The non-linear branch of f' / g' (Sec. 3.1, implementation details): T = LeakyReLU(LayerNorm(X W_1 + b_1)).
// LayerNorm runs over a token's whole feature vector, so it is taken in two steps:
//   producer_hidden_kernel — U = X W_1 + b_1 on tcgen05, 128 tokens x 256 output columns at a time,
//                            rounded to 16 bits and stored by TMA; the thread that owns a token row
//                            sums u and u^2 (fp32, before rounding) over all its column blocks and
//                            leaves the row's mean and 1 / sqrt(variance + ln_eps);
//   producer_norm_kernel   — T = LeakyReLU((U - mean) * rstd * gamma + beta), elementwise, in place.
// ---------------------------------------------------------------------------------------------
struct ProdHiddenCfg {
    static constexpr int TILE = 128;
    static constexpr int KC = 64;
    static constexpr int NB_COLS = 256;              // output columns per block: the widest MMA one CTA can issue
    static constexpr int STAGES = 3;
    static constexpr int X_BYTES = TILE * 128;
    static constexpr int W_BYTES = 4 * KC * 128;     // 64 input rows x four 64-column blocks (one TMA box)
    static constexpr int STAGE_BYTES = X_BYTES + W_BYTES;
    static constexpr int OUT_BYTES = 4 * TILE * 128;  // 128 rows x four 64-column blocks
    static constexpr int MAX_C = 2048;
    static constexpr int EPI_WARPS = 4;
    static constexpr int PRODUCER_WARP = EPI_WARPS;
    static constexpr int MMA_WARP = EPI_WARPS + 1;
    static constexpr int STORE_WARP = EPI_WARPS + 2;
    static constexpr int WPRODUCER_WARP = EPI_WARPS + 3;  // W chunks (the producer warp issues the X chunks)
    static constexpr int THREADS = 32 * (EPI_WARPS + 4);
    static constexpr int TMEM_COLS = 512;            // two accumulators of 256 columns
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + OUT_BYTES + MAX_C * 4 + 1024 + 1024;
};
static_assert(ProdHiddenCfg::SMEM_BYTES <= 227 * 1024, "shared memory budget");

// grid: CTA g of G owns token tiles [g*W/G, (g+1)*W/G) of the W = B * tiles tiles.  stats: [B*N][2] fp32.
template <int KIND>
__global__ void __launch_bounds__(ProdHiddenCfg::THREADS, 1)
producer_hidden_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w1,
                       const __grid_constant__ CUtensorMap tmap_u, const __nv_bfloat16* __restrict__ bias,
                       float* __restrict__ stats, uint32_t* __restrict__ status, int N, int Cdim, int tiles_per_batch,
                       long long W, float ln_eps)
{
    using C = ProdHiddenCfg;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    unsigned char* outb = smem + C::STAGES * C::STAGE_BYTES;
    float* bias_s = reinterpret_cast<float*>(outb + C::OUT_BYTES);
    uint64_t* full = reinterpret_cast<uint64_t*>(reinterpret_cast<unsigned char*>(bias_s) + C::MAX_C * 4);
    uint64_t* empty = full + C::STAGES;
    uint64_t* d1_done = empty + C::STAGES;  // [2]
    uint64_t* d1_free = d1_done + 2;        // [2]
    uint64_t* out_ready = d1_free + 2;      // the staged block is complete
    uint64_t* out_free = out_ready + 1;     // the stores have read it
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(out_free + 1);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long G = gridDim.x, g = blockIdx.x;
    const long long u0 = unit_begin(g, W, G), u1 = unit_begin(g + 1, W, G);
    const int n_units = static_cast<int>(u1 - u0);
    const int KCH = Cdim / C::KC;
    const int NB = (Cdim + C::NB_COLS - 1) / C::NB_COLS;
    const int n_blocks = n_units * NB;  // (tile, column block) pairs of this CTA, in order

    if (tid == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            mbar_init(&full[s], 2);  // the X and the W issuer each announce their bytes
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&d1_done[b], 1);
            mbar_init(&d1_free[b], 4);
        }
        mbar_init(out_ready, 4);
        mbar_init(out_free, 1);
        mbar_fence_init();
    }
    if (warp == 0) tmem_alloc(tmem_slot, C::TMEM_COLS);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    if (warp == C::PRODUCER_WARP && lane == 0) prefetch_tmap(&tmap_x);
    if (warp == C::WPRODUCER_WARP && lane == 0) prefetch_tmap(&tmap_w1);
    if (warp == C::STORE_WARP && lane == 0) prefetch_tmap(&tmap_u);
    pdl_launch_dependents();
    pdl_wait();
    // the bias as fp32, for every role that wants it (zero when there is none)
    for (int i = tid; i < Cdim; i += C::THREADS)
        bias_s[i] = bias != nullptr ? (kind_dtype(KIND) == kDtypeFp16 ? __half2float(reinterpret_cast<const __half*>(bias)[i])
                                                                    : __bfloat162float(bias[i]))
                                    : 0.0f;
    __syncthreads();

    if (warp == C::WPRODUCER_WARP) {
        if (lane == 0) {
            const uint64_t pol_w = policy_evict_last();
            const uint32_t full0 = smem_u32(full), empty0 = smem_u32(empty), w0 = smem_u32(smem) + C::X_BYTES;
            RingPos<C::STAGES> r;
            bool ok = true;
            for (int j = 0; j < n_blocks && ok; ++j) {
                const int blk64 = (j % NB) * (C::NB_COLS / 64);  // first 64-column block of this column block
                for (int kc = 0; kc < KCH; ++kc, r.next()) {
                    ok = mbar_wait_addr(empty0 + 8 * r.s, r.phase ^ 1u);
                    if (!ok) break;
                    const uint32_t bar = full0 + 8 * r.s;
                    mbar_expect_tx_addr(bar, C::W_BYTES);
                    // one box of four 64-column blocks (those past the last column: zero fill)
                    tma_load_3d_addr(w0 + r.s * C::STAGE_BYTES, &tmap_w1, 0, kc * C::KC, blk64, bar, pol_w);
                }
            }
            if (!ok) report_wait_expired(status);
        }
    } else if (warp == C::PRODUCER_WARP) {
        if (lane == 0) {
            const uint64_t pol_x = policy_evict_first();
            const uint32_t full0 = smem_u32(full), empty0 = smem_u32(empty), x0 = smem_u32(smem);
            RingPos<C::STAGES> r;
            bool ok = true;
            int issued = 0;
            for (int j = 0; j < n_blocks && ok; ++j) {
                const long long u = u0 + j / NB;
                const int b = static_cast<int>(u / tiles_per_batch), tile = static_cast<int>(u % tiles_per_batch);
                for (int kc = 0; kc < KCH; ++kc, r.next()) {
                    ok = mbar_wait_addr(empty0 + 8 * r.s, r.phase ^ 1u);
                    if (!ok) break;
                    const uint32_t bar = full0 + 8 * r.s;
                    mbar_expect_tx_addr(bar, C::X_BYTES);
                    tma_load_3d_addr(x0 + r.s * C::STAGE_BYTES, &tmap_x, kc * C::KC, tile * C::TILE, b, bar, pol_x);
                    ++issued;
                }
            }
            if (!ok) report_wait_expired(status);
            drain_loads<C::STAGES>(full, 0, issued, status);  // covers the W loads too (same barriers)
        }
    } else if (warp == C::MMA_WARP) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_f32acc(kind_dtype(KIND), 128, 256, kUmmaBMnMajor);
            bool ok = true;
            const uint64_t a_desc0 = umma_desc_kmajor_sw128(smem_u32(smem));
            const uint64_t b_desc0 = umma_desc_mnmajor_sw128(smem_u32(smem) + C::X_BYTES, C::KC * 128, 1024);
            const uint32_t full0 = smem_u32(full), empty0 = smem_u32(empty);
            RingPos<C::STAGES> r;
            for (int j = 0; j < n_blocks && ok; ++j) {
                const int e = j & 1;
                if (j >= 2) ok = mbar_wait(&d1_free[e], ((j >> 1) - 1) & 1);
                if (!ok) break;
                const uint32_t d1 = tmem_base + e * 256;
                for (int kc = 0; kc < KCH; ++kc, r.next()) {
                    ok = mbar_wait_addr(full0 + 8 * r.s, r.phase);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint64_t step = static_cast<uint64_t>(r.s * (C::STAGE_BYTES >> 4));
                    const uint64_t a_desc = a_desc0 + step, b_desc = b_desc0 + step;
                    umma_ss(d1, a_desc, b_desc, idesc, kc > 0 ? 1u : 0u);
#pragma unroll
                    for (int k = 1; k < C::KC / 16; ++k) umma_ss(d1, a_desc + 2 * k, b_desc + 128 * k, idesc, 1u);
                    umma_commit_addr(empty0 + 8 * r.s);
                }
                if (!ok) break;
                umma_commit(&d1_done[e]);
            }
            if (!ok) report_wait_expired(status);
        }
    } else if (warp == C::STORE_WARP) {
        if (lane == 0) {
            const uint64_t policy = policy_evict_last();  // read again soon by the normalization
            for (int j = 0; j < n_blocks; ++j) {
                if (!mbar_wait(out_ready, j & 1)) {
                    report_wait_expired(status);
                    break;
                }
                const long long u = u0 + j / NB;
                const int nb = j % NB;
                const int b = static_cast<int>(u / tiles_per_batch), tile = static_cast<int>(u % tiles_per_batch);
                for (int q = 0; q < C::NB_COLS / 64; ++q)
                    if (nb * C::NB_COLS + 64 * q < Cdim)
                        tma_store_3d(&tmap_u, outb + q * (C::TILE * 128), nb * C::NB_COLS + 64 * q, tile * C::TILE, b, policy);
                tma_store_wait_read();
                mbar_arrive(out_free);
            }
            tma_store_wait_all();
        }
    } else {
        // ---------------- epilogue warpgroup: thread r owns token row r of every tile ----------------
        const int wq = warp & 3;
        const int row = wq * 32 + lane;
        const uint32_t sw = row & 7;
        float sum = 0.0f, sq = 0.0f;
        bool ok = true;
        for (int j = 0; j < n_blocks; ++j) {
            const int e = j & 1, nb = j % NB;
            ok = mbar_wait(&d1_done[e], (j >> 1) & 1);
            if (ok && j >= 1) ok = mbar_wait(out_free, (j - 1) & 1);
            __syncwarp();
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(wq * 32) << 16) + e * 256;
            const uint32_t o_row = smem_u32(outb) + row * 128;
#pragma unroll
            for (int q = 0; q < C::NB_COLS / 32; ++q) {
                // columns 32 q .. + 31 of the block: half q / 2 of the staging tile, chunks 4 (q % 2) ..
                uint32_t d[32];
                tmem_load_32cols(t_row + 32 * q, d);
                const int col0 = nb * C::NB_COLS + 32 * q;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    float f[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int col = col0 + 8 * c + i;
                        f[i] = 0.0f;
                        if (col < Cdim) {
                            f[i] = __uint_as_float(d[8 * c + i]) + bias_s[col];
                            sum += f[i];
                            sq += f[i] * f[i];
                        }
                    }
                    const uint32_t addr = o_row + (q >> 1) * (C::TILE * 128) + (((4 * (q & 1) + c) ^ sw) << 4);
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(pack_pair<KIND>(f[0], f[1])),
                                 "r"(pack_pair<KIND>(f[2], f[3])), "r"(pack_pair<KIND>(f[4], f[5])),
                                 "r"(pack_pair<KIND>(f[6], f[7]))
                                 : "memory");
                }
            }
            tc_fence_before_sync();
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&d1_free[e]);
                mbar_arrive(out_ready);
            }
            if (nb == NB - 1) {
                // the row is complete: mean and 1 / sqrt(biased variance + ln_eps) over its Cdim features
                const long long u = u0 + j / NB;
                const int b = static_cast<int>(u / tiles_per_batch), tile = static_cast<int>(u % tiles_per_batch);
                const int tok = tile * C::TILE + row;
                if (tok < N) {
                    const float mean = sum / static_cast<float>(Cdim);
                    const float var = fmaxf(sq / static_cast<float>(Cdim) - mean * mean, 0.0f);
                    float2* dst = reinterpret_cast<float2*>(stats) + static_cast<size_t>(b) * N + tok;
                    *dst = make_float2(mean, rsqrtf(var + ln_eps));
                }
                sum = 0.0f;
                sq = 0.0f;
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
}

// T = LeakyReLU((U - mean) * rstd * gamma + beta), in place over t [rows][Cdim] (16-bit), eight
// channels per thread; stats [rows][2] = (mean, rstd) per row.
template <int KIND>
__global__ void __launch_bounds__(256)
producer_norm_kernel(__nv_bfloat16* __restrict__ t, const float* __restrict__ stats,
                     const __nv_bfloat16* __restrict__ gamma, const __nv_bfloat16* __restrict__ beta, long long rows,
                     int Cdim, float slope)
{
    pdl_launch_dependents();
    pdl_wait();
    const int vecs = Cdim / 8;
    const long long total = rows * vecs;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const long long row = i / vecs;
        const int c8 = static_cast<int>(i - row * vecs);
        const float2 st = __ldg(reinterpret_cast<const float2*>(stats) + row);
        uint4* p = reinterpret_cast<uint4*>(t + row * Cdim) + c8;
        const uint4 u = *p;
        const uint4 gm = __ldg(reinterpret_cast<const uint4*>(gamma) + c8);
        const uint4 bt = __ldg(reinterpret_cast<const uint4*>(beta) + c8);
        const uint32_t uu[4] = {u.x, u.y, u.z, u.w}, gg[4] = {gm.x, gm.y, gm.z, gm.w}, bb[4] = {bt.x, bt.y, bt.z, bt.w};
        uint32_t out[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            float lo = (pair_lo<KIND>(uu[k]) - st.x) * st.y * pair_lo<KIND>(gg[k]) + pair_lo<KIND>(bb[k]);
            float hi = (pair_hi<KIND>(uu[k]) - st.x) * st.y * pair_hi<KIND>(gg[k]) + pair_hi<KIND>(bb[k]);
            lo = lo >= 0.0f ? lo : slope * lo;
            hi = hi >= 0.0f ? hi : slope * hi;
            out[k] = pack_pair<KIND>(lo, hi);
        }
        *p = make_uint4(out[0], out[1], out[2], out[3]);
    }
}


}  // namespace lf
