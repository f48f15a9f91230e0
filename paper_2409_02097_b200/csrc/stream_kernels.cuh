// Persistent, TMA-pipelined kernels for head dim 64 (the SD-v2.1 / SD-XL shapes), where the
// operator is bound by HBM bandwidth: every byte of Q, K, V is read once through
// cp.async.bulk.tensor into 128-byte-swizzled shared-memory stages, Y is written once with TMA
// stores, and both contractions run on tcgen05 with their accumulators in tensor memory.
//
// The state kernel's work is cut into units of one token tile of one slab, numbered slab-major;
// CTA g of G owns the contiguous run of units [g*W/G, (g+1)*W/G).  That split is a pure function of
// the shape and the grid size, so the summation order — and with it every output bit — is fixed.
//
//   stream_state_kernel   — per CTA and per slab it touches: partial S_p = sum phi(K_j)^T V_j and
//                           z_p (Prop. 2, Eq. 5) on tcgen05.  A K/V tile of 128 tokens is eight
//                           MMA steps of 16 tokens: D[128 x 64] += A * B with A = [V^T ; 1 ; 0]
//                           (the raw V tile plus a constant block whose single row of ones
//                           yields z) and B = phi(K)^T, both read from shared memory in the
//                           token-major form TMA delivers (MN-major operands).  Each of 128
//                           threads of a warpgroup applies phi to its token's K row in place;
//                           one thread issues the MMAs; the accumulator lives in tensor memory
//                           and is drained into fp32 registers of three flush warps every 32
//                           tiles (keeps the tensor core's accumulation chains short).  Each
//                           (CTA, slab) writes its own fp32 partial; nothing is combined with
//                           atomics.
//   stream_reduce_kernel  — sums the partials of a slab in CTA order; also lays S^T | z out
//                           as the 16-bit, K-major, 128-byte-swizzled B operand the apply kernel
//                           copies into shared memory.
//   stream_apply_kernel   — Y_i = phi(Q_i) S / (phi(Q_i) . z + eps) on tcgen05: a 128-row Q tile
//                           is one MMA tile (M = 128).  Each of the 128 threads of a warpgroup
//                           reads its row from the stage, applies phi in packed 16-bit
//                           arithmetic and writes the row to tensor memory as the A operand; one
//                           thread of the CTA
//                           issues D[128 x 80] = A[128 x 64] * B[64 x 80] (B = S^T rows, then z,
//                           then zero padding, from shared memory); the threads read their row
//                           of D back, divide by the z column, write the 16-bit row over the Q
//                           row in the stage, and a TMA store sends the tile to Y.  Q tiles are
//                           handed out per slab through an atomic counter (the result of a tile
//                           does not depend on which CTA computes it).
//
// One extra warp per CTA is the TMA producer (the apply kernel has a store warp and an MMA warp
// too).  All mbarrier waits are bounded; a wait that expires records kStatusWaitExpired in the
// status word and the CTA drains and exits.
#pragma once

#include "common.cuh"

namespace lf {

constexpr int kStreamD = 64;
constexpr int kStreamStateFloats = kStreamD * (kStreamD + 1);  // S [64][64] then z [64]
constexpr int kStreamRowBytes = kStreamD * 2;                  // 128: one swizzle span

struct StreamStateCfg {
    static constexpr int TILE = 128;   // tokens per stage = 8 MMA steps of 16
    static constexpr int GROUPS = 3;   // warpgroups applying phi, each to its own tile
    static constexpr int PHI_WARPS = 4 * GROUPS;
    static constexpr int PRODUCER_WARP = PHI_WARPS;
    static constexpr int MMA_WARP = PHI_WARPS + 1;
    static constexpr int CLEAR_WARP = PHI_WARPS + 2;   // zeroes the apply kernel's per-slab words
    static constexpr int FLUSH_WARP0 = PHI_WARPS + 4;  // three warps whose index is 0, 1, 2 mod 4
    static constexpr int THREADS = 32 * (PHI_WARPS + 7);
    static constexpr int STAGES = 6;
    static constexpr int CTAS_PER_SM = 1;
    static constexpr int TILE_BYTES = TILE * kStreamRowBytes;  // 16 KB per tensor
    static constexpr int STAGE_BYTES = 2 * TILE_BYTES;         // K then V
    static constexpr int ONES_BYTES = 16 * kStreamRowBytes;    // constant block of A for one MMA step
    static constexpr int SEGMENT_TILES = 32;                   // tiles accumulated in TMEM before a drain
    static constexpr int TMEM_COLS = 128;                      // two accumulators of 64 fp32 columns
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + ONES_BYTES + 1024 /*align*/ + 1024 /*barriers*/;
};
static_assert(StreamStateCfg::FLUSH_WARP0 % 4 == 0, "flush warps must cover TMEM lane quarters 0, 1, 2");
static_assert(StreamStateCfg::SMEM_BYTES > 116 * 1024, "one state CTA per SM");

struct StreamApplyCfg {
    static constexpr int TILE = 128;   // tokens per stage = rows of one MMA tile = TMEM lanes
    static constexpr int GROUPS = 4;   // warpgroups, each working on its own tile
    static constexpr int CONSUMER_WARPS = 4 * GROUPS;
    static constexpr int PRODUCER_WARP = CONSUMER_WARPS;
    static constexpr int STORE_WARP = CONSUMER_WARPS + 1;
    static constexpr int MMA_WARP = CONSUMER_WARPS + 2;
    static constexpr int THREADS = 32 * (CONSUMER_WARPS + 3);
    static constexpr int STAGE_BYTES = TILE * kStreamRowBytes;  // 16 KB: a Q tile, later its Y tile
    static constexpr int STAGES = 12;
    static constexpr int B_ROWS = 80;  // N of the MMA: 64 channels of S^T, z, padding to a multiple of 16
    static constexpr int B_BYTES = B_ROWS * kStreamRowBytes;    // 10 KB
    static constexpr int B_BUFFERS = 2;                         // the next slab's operand is copied while the last one is in use
    static constexpr int TMEM_COLS_PER_GROUP = 128;             // A: 32 columns, D: 80
    static constexpr int TMEM_COLS = 512;                       // a power of two >= GROUPS * 128
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + B_BUFFERS * B_BYTES + 1024 /*align*/ + 1024 /*barriers, meta*/;
};
static_assert(StreamApplyCfg::GROUPS * StreamApplyCfg::TMEM_COLS_PER_GROUP <= StreamApplyCfg::TMEM_COLS, "TMEM budget");
static_assert(StreamApplyCfg::STAGES >= 2 * StreamApplyCfg::GROUPS + 2, "end markers need released stages");
// Shared memory beyond half an SM's keeps a second CTA (and its TMEM allocation) off the SM.
static_assert(StreamApplyCfg::SMEM_BYTES > 116 * 1024, "one apply CTA per SM");

// First unit of CTA g when W units are dealt to G CTAs.
__host__ __device__ __forceinline__ long long unit_begin(long long g, long long W, long long G)
{
    return (g * W) / G;
}

__device__ __forceinline__ void report_wait_expired(uint32_t* status)
{
    atomicExch(status, kStatusWaitExpired);
}

__device__ __forceinline__ uint32_t ld_acquire_gpu(const uint32_t* p)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_gpu_add(uint32_t* p, uint32_t v)
{
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Spin (bounded by the global timer, like the mbarrier waits) until the counter has advanced by at
// least `need` from `base`.  Counters only grow; the difference is taken modulo 2^32.
__device__ __forceinline__ bool counter_wait(const uint32_t* ctr, uint32_t base, uint32_t need)
{
    if (ld_acquire_gpu(ctr) - base >= need) return true;
    const unsigned long long t0 = global_timer_ns();
    do {
        __nanosleep(40);
        if (ld_acquire_gpu(ctr) - base >= need) return true;
    } while (global_timer_ns() - t0 < kMaxBarrierWaitNs);
    return false;
}

// Barrier among `threads` threads of the CTA (ids 1..15; 0 is __syncthreads).
__device__ __forceinline__ void named_barrier_sync(int id, int threads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// One warp waits on an mbarrier that nothing ever arrives on: the bounded wait must give up after
// kMaxBarrierWaitNs and leave the error word behind, and the kernel must end normally.  Run by the
// library's self-test of its failure reporting, never on the attention path.
__global__ void __launch_bounds__(32)
wait_selftest_kernel(uint32_t* __restrict__ status)
{
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mbar_fence_init();
    }
    __syncwarp();
    if (!mbar_wait(&bar, 0) && threadIdx.x == 0) report_wait_expired(status);
}

// Before the producer leaves: a bounded wait for every bulk copy it still has in flight, so
// that no copy lands in shared memory after the CTA has gone.
// Loads [first, issued) are waited for; a load whose stage has been armed again since (its phase
// is then two behind and can no longer be waited on) must not be in that range.
template <int STAGES>
__device__ __forceinline__ void drain_loads(uint64_t* full, int first, int issued, uint32_t* status)
{
    if (first < issued - STAGES) first = issued - STAGES;
    if (first < 0) first = 0;
    for (int it = first; it < issued; ++it)
        if (!mbar_wait(&full[it % STAGES], (it / STAGES) & 1)) {
            report_wait_expired(status);
            return;
        }
}

// ---------------------------------------------------------------------------------------------
// State: partials[g * spans + slot][kStreamStateFloats], slot = slab - first slab of CTA g's run.
//
// Roles in a CTA (one per SM): producer warp (TMA loads of K and V tiles); 3 warpgroups (thread r
// of a group rewrites token r's K row as phi(K), zero past N); MMA warp (one thread issues every
// tcgen05.mma; the stage is released by a commit once the MMAs that read it are complete); three
// flush warps (TMEM lanes 0..63 = rows of S^T, lane 64 = z).  The run of a CTA is cut into
// segments of at most SEGMENT_TILES tiles of one slab; segments alternate between two TMEM
// accumulators, and the flush warps add each finished segment into fp32 registers (round to
// nearest) and write the partial when the slab ends.
// Per stage s: full[s] -> k_ready[s] (4 warps) -> empty[s] (commit).  Per accumulator b:
// acc_done[b] (commit) -> acc_free[b] (3 flush warps).
// ---------------------------------------------------------------------------------------------
template <int KIND>
__global__ void __launch_bounds__(StreamStateCfg::THREADS, StreamStateCfg::CTAS_PER_SM)
stream_state_kernel(const __grid_constant__ CUtensorMap tmap_k,
                    const __grid_constant__ CUtensorMap tmap_v, float* __restrict__ partials,
                    uint32_t* __restrict__ status, int N, int tiles_per_slab, long long W, int spans, int H,
                    uint32_t* __restrict__ clear_words, int n_clear)
{
    using C = StreamStateCfg;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    unsigned char* ones = smem + C::STAGES * C::STAGE_BYTES;  // on a 1024-byte boundary
    uint64_t* full = reinterpret_cast<uint64_t*>(ones + C::ONES_BYTES);
    uint64_t* empty = full + C::STAGES;
    uint64_t* k_ready = empty + C::STAGES;
    uint64_t* acc_done = k_ready + C::STAGES;  // [2]
    uint64_t* acc_free = acc_done + 2;         // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_free + 2);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long G = gridDim.x, g = blockIdx.x;
    const long long u0 = unit_begin(g, W, G), u1 = unit_begin(g + 1, W, G);
    const int n_units = static_cast<int>(u1 - u0);
    const int slab_first = static_cast<int>(u0 / tiles_per_slab);

    if (tid == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
            mbar_init(&k_ready[s], 4);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&acc_done[b], 1);
            mbar_init(&acc_free[b], 3);
        }
        mbar_fence_init();
    }
    // Constant block of A (rows 64..127 of [V^T ; 1 ; 0] for 16 tokens): a one at (token t, row 64),
    // which is the first value of token t's 128-byte row, moved by the swizzle to chunk t & 7.
    for (int i = tid; i < C::ONES_BYTES / 4; i += C::THREADS) reinterpret_cast<uint32_t*>(ones)[i] = 0u;
    __syncthreads();
    if (tid < 16)
        *reinterpret_cast<uint16_t*>(ones + tid * 128 + ((tid & 7) << 4)) = static_cast<uint16_t>(ones_pair<KIND>() & 0xffffu);
    fence_proxy_async_smem();
    if (warp == 0) tmem_alloc(tmem_slot, C::TMEM_COLS);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // Set-up done (barriers, tensor memory): let the next kernel in the stream be scheduled behind
    // this one, and wait for the one before it to be complete before touching global memory.  (The
    // tensor maps are kernel parameters: fetching them does not depend on earlier work.)
    if (warp == C::PRODUCER_WARP && lane == 0) {
        prefetch_tmap(&tmap_k);
        prefetch_tmap(&tmap_v);
    }
    pdl_launch_dependents();
    pdl_wait();

    if (warp == C::PRODUCER_WARP) {
        // ---------------- producer ----------------
        if (lane == 0) {
            const uint64_t policy = policy_evict_first();
            int issued = 0;
            for (int it = 0; it < n_units; ++it) {
                const int s = it % C::STAGES;
                if (!mbar_wait(&empty[s], ((it / C::STAGES) & 1) ^ 1)) {
                    report_wait_expired(status);
                    break;
                }
                const long long u = u0 + it;
                const int slab = static_cast<int>(u / tiles_per_slab);
                const int tile = static_cast<int>(u % tiles_per_slab);
                unsigned char* dst = smem + s * C::STAGE_BYTES;
                mbar_expect_tx(&full[s], C::STAGE_BYTES);
                tma_load_4d(dst, &tmap_k, 0, tile * C::TILE, slab % H, slab / H, &full[s], policy);
                tma_load_4d(dst + C::TILE_BYTES, &tmap_v, 0, tile * C::TILE, slab % H, slab / H, &full[s], policy);
                ++issued;
            }
            drain_loads<C::STAGES>(full, 0, issued, status);
        }
    } else if (warp == C::MMA_WARP) {
        // ---------------- MMA warp ----------------
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_f32acc(kind_dtype(KIND), 128, 64, kUmmaAMnMajor | kUmmaBMnMajor);
            const uint32_t ones_addr = smem_u32(ones);
            int cur_slab = -1, in_segment = 0, segments = 0, buf = 1;
            for (int it = 0; it < n_units; ++it) {
                const int s = it % C::STAGES;
                const int slab = static_cast<int>((u0 + it) / tiles_per_slab);
                if (slab != cur_slab || in_segment == C::SEGMENT_TILES) {
                    if (cur_slab >= 0) umma_commit(&acc_done[buf]);  // the segment's accumulator is complete
                    buf ^= 1;
                    // this accumulator held the segment before last: its drain must be over
                    if (segments >= 2 && !mbar_wait(&acc_free[buf], ((segments - 2) >> 1) & 1)) {
                        report_wait_expired(status);
                        break;
                    }
                    ++segments;
                    cur_slab = slab;
                    in_segment = 0;
                }
                if (!mbar_wait(&k_ready[s], (it / C::STAGES) & 1)) {
                    report_wait_expired(status);
                    break;
                }
                tc_fence_after_sync();
                const uint32_t k_addr = smem_u32(smem + s * C::STAGE_BYTES), v_addr = k_addr + C::TILE_BYTES;
                const uint32_t d_tmem = tmem_base + buf * 64;
#pragma unroll
                for (int k = 0; k < C::TILE / 16; ++k) {
                    // A: 64 rows from the V tile, 64 from the constant block (lbo = their distance);
                    // 16 tokens = two 8-row groups 1024 bytes apart.
                    const uint32_t va = v_addr + k * 2048;
                    const uint64_t a_desc = umma_desc_mnmajor_sw128(va, ones_addr - va, 1024);
                    const uint64_t b_desc = umma_desc_mnmajor_sw128(k_addr + k * 2048, 0, 1024);
                    umma_ss(d_tmem, a_desc, b_desc, idesc, (in_segment == 0 && k == 0) ? 0u : 1u);
                }
                ++in_segment;
                umma_commit(&empty[s]);  // the stage is free once these MMAs have read it
            }
            if (cur_slab >= 0) umma_commit(&acc_done[buf]);
        }
    } else if (warp >= C::FLUSH_WARP0 && warp < C::FLUSH_WARP0 + 3) {
        // ---------------- flush warps ----------------
        // The same walk over the run as the MMA thread's, segment by segment.
        const int wq = warp & 3;
        const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(wq * 32) << 16);
        float acc[64];
#pragma unroll
        for (int c = 0; c < 64; ++c) acc[c] = 0.0f;
        int seg = 0;
        bool ok = true;
        for (int it = 0; it < n_units && ok;) {
            const int slab = static_cast<int>((u0 + it) / tiles_per_slab);
            const long long slab_end = static_cast<long long>(slab + 1) * tiles_per_slab - u0;  // first it of the next slab
            int len = static_cast<int>(slab_end < n_units ? slab_end : n_units) - it;
            if (len > C::SEGMENT_TILES) len = C::SEGMENT_TILES;
            it += len;
            const int buf = seg & 1;
            ok = mbar_wait(&acc_done[buf], (seg >> 1) & 1);
            ++seg;
            __syncwarp();
            if (!ok) {
                if (lane == 0) report_wait_expired(status);
                break;
            }
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
            if (it == n_units || it == slab_end) {
                // the slab's share of this CTA is complete: row e of S^T (lanes 0..63), z (lane 64)
                float* dst = partials + (static_cast<size_t>(g) * spans + (slab - slab_first)) * kStreamStateFloats;
                if (wq < 2) {
                    const int e = wq * 32 + lane;
#pragma unroll
                    for (int c = 0; c < 64; ++c) dst[c * 64 + e] = acc[c];
                } else if (lane == 0) {
#pragma unroll
                    for (int c = 0; c < 64; ++c) dst[64 * 64 + c] = acc[c];
                }
#pragma unroll
                for (int c = 0; c < 64; ++c) acc[c] = 0.0f;
            }
        }
    } else if (warp == C::CLEAR_WARP) {
        // ---------------- the apply kernel's per-slab words (tile counters, ready flags) start every forward
        // at zero; the forward before has completed (dependency wait above) ----------------
        for (int i = static_cast<int>(g) * 32 + lane; i < n_clear; i += static_cast<int>(G) * 32) clear_words[i] = 0u;
    } else if (warp < C::PHI_WARPS) {
        // ---------------- phi warpgroups ----------------
        const int group = warp >> 2;
        const int row = (warp & 3) * 32 + lane;
        const uint32_t row_base = smem_u32(smem) + row * 128;
        const uint32_t sw = row & 7;
        for (int it = group; it < n_units; it += C::GROUPS) {
            const int s = it % C::STAGES;
            if (!mbar_wait(&full[s], (it / C::STAGES) & 1)) {
                if (lane == 0) report_wait_expired(status);
                break;
            }
            const int tile = static_cast<int>((u0 + it) % tiles_per_slab);
            const uint32_t base = row_base + s * C::STAGE_BYTES;
            if (tile * C::TILE + row < N) {
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    // a quarter-warp touches eight different chunk positions: no bank conflicts
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
            // else: a row past N.  TMA filled it with zeros and it must count for nothing; phi(0) = 1,
            // so the zeros are left as they are.  (Only the last tile of a slab has such rows.)
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(&k_ready[s]);
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

// Operand image of S | z for the apply kernel, per slab: the MMA's B operand in its shared-memory
// form — 80 rows of 128 bytes, row n < 64 = column n of S (64 values of the storage type along c), row 64 = z, rows 65-79
// zero; 16-byte chunk j of row n sits at chunk position j ^ (n & 7) (the 128-byte swizzle).
constexpr int kStreamOperandBytes = StreamApplyCfg::B_BYTES;

// Block blockIdx.x of a (17, slabs) grid of 256 threads holds elements 256*blockIdx.x .. of one
// slab's fp32 state (S rows 4*blockIdx.x .., or z in block 16) in `sums`; write their share of the
// operand image `img` of that slab.
__device__ __forceinline__ void emit_state_operand(const float* sums, unsigned char* img, int dtype, float scale)
{
    const int tid = threadIdx.x;
    if (blockIdx.x < 16) {
        // S rows c0 .. c0+3 are in sums[r*64 + e]; thread e < 64 writes the four values of column e
        if (tid < 64) {
            const int c0 = 4 * blockIdx.x, e = tid;
            uint2 v;
            v.x = to_storage16(sums[e] * scale, dtype) | (static_cast<uint32_t>(to_storage16(sums[64 + e] * scale, dtype)) << 16);
            v.y = to_storage16(sums[128 + e] * scale, dtype) |
                  (static_cast<uint32_t>(to_storage16(sums[192 + e] * scale, dtype)) << 16);
            *reinterpret_cast<uint2*>(img + e * 128 + (((c0 >> 3) ^ (e & 7)) << 4) + (c0 & 7) * 2) = v;
        }
    } else {
        // z -> row 64 (64 & 7 = 0: chunks in place), zeros -> rows 65..79
        if (tid < 32) {
            *reinterpret_cast<uint32_t*>(img + 64 * 128 + tid * 4) =
                to_storage16(sums[2 * tid] * scale, dtype) |
                (static_cast<uint32_t>(to_storage16(sums[2 * tid + 1] * scale, dtype)) << 16);
        } else if (tid < 32 + 120) {
            reinterpret_cast<uint4*>(img + 65 * 128)[tid - 32] = make_uint4(0u, 0u, 0u, 0u);
        }
    }
}

// grid (17, slabs), 256 threads: state[slab] = sum over the CTAs whose run meets the slab, in
// increasing CTA index (fp32, fixed order).  Also writes the 16-bit operand
// image of S | z for the apply kernel and clears the slab's tile counter for it.
__global__ void __launch_bounds__(256)
stream_reduce_kernel(const float* __restrict__ partials, float* __restrict__ state,
                     unsigned char* __restrict__ operand, int* __restrict__ tile_counters,
                     int tiles_per_slab, long long W, int G, int spans, int dtype, float operand_scale)
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
        const long long lo = static_cast<long long>(slab) * tiles_per_slab, hi = lo + tiles_per_slab;
        // g0: the CTA whose run contains unit `lo`; g1: the first CTA whose run starts at or after `hi`.
        long long g0 = (lo * G) / W;
        while (g0 + 1 < G && unit_begin(g0 + 1, W, G) <= lo) ++g0;
        while (g0 > 0 && unit_begin(g0, W, G) > lo) --g0;
        long long g1 = (hi * G) / W;
        while (g1 < G && unit_begin(g1, W, G) < hi) ++g1;
        while (g1 > 0 && unit_begin(g1 - 1, W, G) >= hi) --g1;
        const int slot0 = slab - static_cast<int>(unit_begin(g0, W, G) / tiles_per_slab);
        const size_t F = kStreamStateFloats;
        const float* src = partials + idx;
        sum += src[(static_cast<size_t>(g0) * spans + slot0) * F];
        // Every later CTA starts inside this slab: its partial for it is in slot 0.
#pragma unroll 4
        for (long long g = g0 + 1; g < g1; ++g) sum += src[(static_cast<size_t>(g) * spans) * F];
        state[static_cast<size_t>(slab) * F + idx] = sum;
    }
    sums[tid] = sum;
    __syncthreads();
    emit_state_operand(sums, operand + static_cast<size_t>(slab) * kStreamOperandBytes, dtype, operand_scale);
}

// grid (17, slabs), 256 threads: rebuild the 16-bit operand image (and clear the tile counters) from
// fp32 states that were changed or live outside the reduction — the state after a sum over devices
// of a token-sharded forward (Sec. 4.3), or the devices' states themselves, which are then summed
// here in index order (loads from peers' memory when the list holds peers' buffers).
__global__ void __launch_bounds__(256)
stream_pack_kernel(PeerStates states, unsigned char* __restrict__ operand,
                   int* __restrict__ tile_counters, int dtype, float operand_scale)
{
    __shared__ float sums[256];
    const int tid = threadIdx.x;
    const int idx = blockIdx.x * 256 + tid;
    const int slab = blockIdx.y;
    pdl_launch_dependents();
    pdl_wait();
    if (blockIdx.x == 0 && tid == 0) tile_counters[slab] = 0;
    sums[tid] = idx < kStreamStateFloats ? peer_sum(states, static_cast<size_t>(slab) * kStreamStateFloats + idx) : 0.0f;
    __syncthreads();
    emit_state_operand(sums, operand + static_cast<size_t>(slab) * kStreamOperandBytes, dtype, operand_scale);
}

// ---------------------------------------------------------------------------------------------
// Apply.  Tiles are handed out per slab through an atomic counter: CTA g starts on its home slab
// g*slabs/G and moves to the next slab that still has tiles when one runs dry, so the CTAs of a
// slab share its tail and early finishers help elsewhere.  Each output tile depends only on its
// own Q rows and the slab's S | z, so the result does not depend on who computes it.  For short
// runs with the same number of CTAs on every slab the host asks for fixed runs instead (static_runs).
//
// Roles in a CTA (one CTA per SM; it owns all 512 TMEM columns):
//   producer warp — claims tiles, copies the slab's B operand into shared memory when the slab
//                   changes (after every posted tile has left), loads Q tiles with TMA;
//   4 warpgroups  — group g takes the tiles posted g-th, (g+4)-th, ...; thread r of a group owns
//                   row r of the tile = TMEM lane r (a warp may only touch the 32 lanes of its
//                   quarter, so warp w of the CTA works on rows 32*(w%4) ..);
//   MMA warp      — one thread issues every tcgen05.mma of the CTA, in posting order;
//   store warp    — one thread sends finished Y tiles out with TMA, in posting order, and
//                   releases the stage once the store has read it.
// Per stage s: full[s] (TMA bytes landed) -> a_ready[g] (4 warps: phi(Q) rows in TMEM) ->
// mma_done[g] (tcgen05.commit) -> y_ready[s] (4 warps: Y rows in the stage) -> empty[s].
// ---------------------------------------------------------------------------------------------
// The second stage of the state reduction done by the apply kernel itself (no kernel of its own between
// the state kernel and the apply kernel): every apply CTA sums, in CTA order, the partials of its HOME slab
// (the slab it starts on) straight into its shared-memory operand; the lowest-numbered CTA of a slab's
// home CTAs also leaves the fp32 state and the 16-bit operand image in global memory and then raises the
// slab's ready flag, which a CTA that later helps out on that slab waits for (bounded) before it copies
// the image.  Every slab needs a home CTA: the host enables this only when slabs <= grid size.
struct MergedReduce {
    const float* partials;   // of stream_state_kernel
    float* state;            // [slab][S 64x64 | z 64] fp32
    unsigned char* operand;  // [slab] 16-bit images
    uint32_t* ready;         // [slab] flags, zero at kernel start
    long long W;             // the state kernel's units, grid and partial slots per CTA
    int G, spans, tiles_per_slab;
    int dtype;
    float scale;
    int enabled;
};

template <int KIND>
__global__ void __launch_bounds__(StreamApplyCfg::THREADS, 1)
stream_apply_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_y,
                    const unsigned char* __restrict__ operand, int* __restrict__ tile_counters,
                    uint32_t* __restrict__ status, int tiles_per_slab, int slabs, ApplyScales sc, int H, MergedReduce mr,
                    int static_runs)
{
    using C = StreamApplyCfg;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    unsigned char* bsm = smem + C::STAGES * C::STAGE_BYTES;  // B operands (two buffers), on 1024-byte boundaries
    uint64_t* full = reinterpret_cast<uint64_t*>(bsm + C::B_BUFFERS * C::B_BYTES);
    uint64_t* empty = full + C::STAGES;
    uint64_t* y_ready = empty + C::STAGES;
    uint64_t* a_ready = y_ready + C::STAGES;  // per group
    uint64_t* mma_done = a_ready + C::GROUPS;  // per group
    uint64_t* b_ready = mma_done + C::GROUPS;  // [B_BUFFERS]: a slab's operand has been put into that buffer
    uint64_t* home_done = b_ready + C::B_BUFFERS;  // the home slab's operand has been summed into buffer 0
    int2* meta = reinterpret_cast<int2*>(home_done + 1);  // (slab, tile) of each stage; slab < 0 ends
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(meta + C::STAGES);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    if (tid == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
            mbar_init(&y_ready[s], 4);
        }
        for (int g = 0; g < C::GROUPS; ++g) {
            mbar_init(&a_ready[g], 4);
            mbar_init(&mma_done[g], 1);
        }
        for (int b = 0; b < C::B_BUFFERS; ++b) mbar_init(&b_ready[b], 1);
        mbar_init(home_done, 1);
        mbar_fence_init();
    }
    if (warp == 0) tmem_alloc(tmem_slot, C::TMEM_COLS);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // Set-up done (barriers, tensor memory): let the next kernel in the stream be scheduled behind
    // this one, and wait for the one before it to be complete before touching global memory.  (The
    // tensor maps are kernel parameters: fetching them does not depend on earlier work.)
    if (warp == C::PRODUCER_WARP && lane == 0) prefetch_tmap(&tmap_q);
    if (warp == C::STORE_WARP && lane == 0) prefetch_tmap(&tmap_y);
    const int home = static_cast<int>((static_cast<long long>(blockIdx.x) * slabs) / gridDim.x);
    constexpr int TEAM = C::THREADS - 32;  // every warp but the producer
    const int ttid = tid < 32 * C::PRODUCER_WARP ? tid : tid - 32;
    int* ctrb = reinterpret_cast<int*>(tmem_slot + 1);  // g0, g1, first contributor's slot
    if (mr.enabled != 0 && warp != C::PRODUCER_WARP) {
        // (pure index arithmetic and shared memory: done while the kernel ahead is still running)
        if (ttid == 0) {
            const long long lo = static_cast<long long>(home) * mr.tiles_per_slab, hi = lo + mr.tiles_per_slab;
            const long long Gs = mr.G, Ws = mr.W;
            long long g0 = (lo * Gs) / Ws;
            while (g0 + 1 < Gs && unit_begin(g0 + 1, Ws, Gs) <= lo) ++g0;
            while (g0 > 0 && unit_begin(g0, Ws, Gs) > lo) --g0;
            long long g1 = (hi * Gs) / Ws;
            while (g1 < Gs && unit_begin(g1, Ws, Gs) < hi) ++g1;
            while (g1 > 0 && unit_begin(g1 - 1, Ws, Gs) >= hi) --g1;
            ctrb[0] = static_cast<int>(g0);
            ctrb[1] = static_cast<int>(g1);
            ctrb[2] = home - static_cast<int>(unit_begin(g0, Ws, Gs) / mr.tiles_per_slab);
        }
        for (int i = ttid; i < 15 * 128 / 16; i += TEAM) reinterpret_cast<uint4*>(bsm + 65 * 128)[i] = make_uint4(0u, 0u, 0u, 0u);
    }
    pdl_launch_dependents();
    pdl_wait();

    if (mr.enabled != 0 && warp != C::PRODUCER_WARP) {
        // ---------------- every warp but the producer (which is already fetching Q tiles): the home
        // slab's state, summed over the state kernel's CTAs ----------------
        named_barrier_sync(1, TEAM);
        const int g0 = ctrb[0], g1 = ctrb[1], slot0 = ctrb[2];
        const bool writer = blockIdx.x == 0 ||
                            static_cast<int>((static_cast<long long>(blockIdx.x - 1) * slabs) / gridDim.x) != home;
        const float4* part4 = reinterpret_cast<const float4*>(mr.partials);
        constexpr int V4 = kStreamStateFloats / 4;  // 1040: S rows as 16 float4 each, then z as 16
        float4* st4 = reinterpret_cast<float4*>(mr.state + static_cast<size_t>(home) * kStreamStateFloats);
        // contributor g0's partial of this slab sits in its slot `slot0`; every later contributor's run starts
        // inside the slab (its slot 0).  A thread walks through the (element, contributor) pairs of its
        // elements with twelve 16-byte loads in flight and adds them in CTA order.
        auto emit = [&](int idx, const float4& sum) {
            if (writer) st4[idx] = sum;
            const float f[4] = {sum.x * mr.scale, sum.y * mr.scale, sum.z * mr.scale, sum.w * mr.scale};
            if (idx < 1024) {
                const int c = idx >> 4, e0 = (idx & 15) * 4;  // S[c][e0 .. e0+3] -> B rows e0 .., column c
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int row = e0 + i;
                    *reinterpret_cast<uint16_t*>(bsm + row * 128 + (((c >> 3) ^ (row & 7)) << 4) + (c & 7) * 2) =
                        to_storage16(f[i], mr.dtype);
                }
            } else {
                // z[4 t .. 4 t + 3] -> row 64 (64 & 7 = 0: chunks in place)
                const int t4 = idx - 1024;
                uint2 wv;
                wv.x = to_storage16(f[0], mr.dtype) | (static_cast<uint32_t>(to_storage16(f[1], mr.dtype)) << 16);
                wv.y = to_storage16(f[2], mr.dtype) | (static_cast<uint32_t>(to_storage16(f[3], mr.dtype)) << 16);
                *reinterpret_cast<uint2*>(bsm + 64 * 128 + t4 * 8) = wv;
            }
        };
        {
            constexpr int kInFlight = 12;
            int idx = ttid, gc = g0;
            float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
            while (idx < V4) {
                float4 v[kInFlight];
                int idx2 = idx, gc2 = gc;
#pragma unroll
                for (int u = 0; u < kInFlight; ++u) {
                    if (idx2 < V4) {
                        v[u] = __ldcg(part4 + (static_cast<size_t>(gc2) * mr.spans + (gc2 == g0 ? slot0 : 0)) * V4 + idx2);
                        if (++gc2 == g1) {
                            gc2 = g0;
                            idx2 += TEAM;
                        }
                    }
                }
#pragma unroll
                for (int u = 0; u < kInFlight; ++u) {
                    if (idx < V4) {
                        if (gc == g0) {
                            sum = v[u];  // the first term as it is: the same bits as a sum that starts from it
                        } else {
                            sum.x += v[u].x;
                            sum.y += v[u].y;
                            sum.z += v[u].z;
                            sum.w += v[u].w;
                        }
                        if (++gc == g1) {
                            emit(idx, sum);
                            gc = g0;
                            idx += TEAM;
                        }
                    }
                }
            }
        }
        fence_proxy_async_smem();
        named_barrier_sync(1, TEAM);
        if (ttid == 0) mbar_arrive(home_done);
        if (writer && static_runs == 0) {
            // (with fixed runs nobody works on another CTA's slab: no image, no flag)
            uint4* img = reinterpret_cast<uint4*>(mr.operand + static_cast<size_t>(home) * C::B_BYTES);
            for (int i = ttid; i < C::B_BYTES / 16; i += TEAM) img[i] = reinterpret_cast<const uint4*>(bsm)[i];
            named_barrier_sync(1, TEAM);
            if (ttid == 0) {
                __threadfence();
                red_release_gpu_add(&mr.ready[home], 1u);
            }
        }
    }

    if (warp == C::PRODUCER_WARP) {
        // ---------------- producer warp (lane 0 issues; all lanes help to find work and copy B) ----------------
        uint64_t policy = 0;
        if (lane == 0) policy = policy_evict_first();
        int slab = home;
        // Two operand buffers: the operand of the slab being posted sits in buffer cur_buf; when the slab
        // changes the new operand goes to the other buffer, which was last read by the tiles posted before
        // the previous change (long gone, as a rule), so the ring is not drained for it.  Buffer 0 starts
        // as the home slab's, summed in place by the other warps (complete once home_done).
        int cur_buf = 0;
        const bool home_in_place = mr.enabled != 0;
        bool home_pending = mr.enabled != 0;          // the other warps may still be writing buffer 0
        int it = 0, issued = 0, loaded_slab = -1, last_switch_it = 0;
        bool ok = true;
        // static_runs > 0 (the grid is static_runs CTAs per slab): this CTA takes a fixed run of its home
        // slab's tiles and nothing else.  A CTA's share is then shorter than the ring is deep, and tiles
        // claimed through the counters would go to whichever CTA asks first, leave the others short, and
        // send them to other slabs for a tile or two at the price of draining the ring for the new operand.
        const int run = static_runs > 0 ? static_cast<int>(blockIdx.x) % static_runs : 0;
        int s_next = static_runs > 0 ? static_cast<int>((static_cast<long long>(run) * tiles_per_slab) / static_runs) : 0;
        const int s_end = static_runs > 0 ? static_cast<int>((static_cast<long long>(run + 1) * tiles_per_slab) / static_runs) : 0;
        auto claim = [&]() {
            if (static_runs > 0) return s_next < s_end ? s_next++ : tiles_per_slab;
            return atomicAdd(&tile_counters[slab], 1);
        };
        int next = 0;
        if (lane == 0) next = claim();
        while (true) {
            const int tile = __shfl_sync(0xffffffffu, next, 0);
            if (tile >= tiles_per_slab) {
                if (static_runs > 0) break;
                // Next slab, in cyclic order, whose counter has not run past its tiles.
                int found = -1;
                for (int base = 0; base < slabs && found < 0; base += 32) {
                    const int off = base + lane;
                    const int cand = (slab + 1 + off) % slabs;
                    const bool has = off < slabs &&
                                     *reinterpret_cast<volatile int*>(&tile_counters[cand]) < tiles_per_slab;
                    const unsigned m = __ballot_sync(0xffffffffu, has);
                    if (m != 0u) found = (slab + 1 + base + __ffs(m) - 1) % slabs;
                }
                if (found < 0) break;
                slab = found;
                if (lane == 0) next = claim();
                continue;
            }
            // Claim the tile after this one now: the atomic's round trip (comparable to the time a
            // tile takes) overlaps the wait for a free stage and the copy below.
            if (lane == 0) next = claim();
            const bool new_slab = slab != loaded_slab;
            const bool first_slab = loaded_slab < 0;
            const bool copy_b = new_slab && !(first_slab && home_in_place);
            const int use_buf = new_slab ? (first_slab ? 0 : cur_buf ^ 1) : cur_buf;
            if (copy_b && !first_slab) {
                // The tiles that read buffer use_buf are those posted before the previous change of slab:
                // they must have left (their MMAs are then complete as well) before it is overwritten.
                if (lane == 0) {
                    for (int j = it > C::STAGES ? it - C::STAGES : 0; j < last_switch_it && ok; ++j)
                        ok = mbar_wait(&empty[j % C::STAGES], (j / C::STAGES) & 1);
                    if (!ok) report_wait_expired(status);
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
            }
            const int s = it % C::STAGES;
            if (lane == 0) {
                ok = mbar_wait(&empty[s], ((it / C::STAGES) & 1) ^ 1);
                if (ok) {
                    meta[s] = make_int2(slab, tile | (use_buf << 30));
                    mbar_expect_tx(&full[s], C::STAGE_BYTES);
                    tma_load_4d(smem + s * C::STAGE_BYTES, &tmap_q, 0, tile * C::TILE, slab % H, slab / H, &full[s], policy);
                    ++issued;
                } else {
                    report_wait_expired(status);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            ++it;
            if (new_slab) {
                // The slab's operand, copied while the tile above is on its way (unless the buffer holds
                // it already: the home slab's, summed above); the MMA thread waits for b_ready before
                // the first MMA of a slab.
                if (copy_b) {
                    if (mr.enabled != 0) {
                        // buffer 0 must not be overwritten while the home slab's sum is still being written
                        // into it; the image is written during this kernel by the slab's first home CTA
                        if (lane == 0 && home_pending && use_buf == 0) ok = mbar_wait(home_done, 0);
                        if (use_buf == 0) home_pending = false;
                        if (lane == 0 && ok) ok = counter_wait(&mr.ready[slab], 0u, 1u);
                        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                        if (!ok) {
                            if (lane == 0) report_wait_expired(status);
                            break;
                        }
                    }
                    const uint4* src = reinterpret_cast<const uint4*>(operand + static_cast<size_t>(slab) * C::B_BYTES);
                    uint4* dst = reinterpret_cast<uint4*>(bsm + use_buf * C::B_BYTES);
                    for (int i = lane; i < C::B_BYTES / 16; i += 32) dst[i] = __ldcg(src + i);
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&b_ready[use_buf]);
                loaded_slab = slab;
                cur_buf = use_buf;
                last_switch_it = it - 1;  // the tile just posted is the first of this slab
            }
        }
        if (lane == 0) {
            int first = 0;
            if (ok) {
                // One end marker per warpgroup, in consecutive stages (group g reads every third
                // posting).  Those stages held loads issued - STAGES .., released by now.
                for (int e = 0; e < C::GROUPS && ok; ++e) {
                    const int s = it % C::STAGES;
                    ok = mbar_wait(&empty[s], ((it / C::STAGES) & 1) ^ 1);
                    if (ok) {
                        meta[s] = make_int2(-1, 0);
                        mbar_arrive(&full[s]);
                        ++it;
                    } else {
                        report_wait_expired(status);
                    }
                }
                first = issued - C::STAGES + C::GROUPS;
            }
            drain_loads<C::STAGES>(full, first, issued, status);
        }
    } else if (warp == C::STORE_WARP) {
        // ---------------- store warp ----------------
        if (lane == 0) {
            const uint64_t policy = policy_evict_first();
            for (int it = 0;; ++it) {
                const int s = it % C::STAGES;
                if (!mbar_wait(&y_ready[s], (it / C::STAGES) & 1)) {
                    report_wait_expired(status);
                    break;
                }
                const int2 m = meta[s];
                if (m.x < 0) break;  // the first end marker: every tile posted before it has left
                tma_store_4d(&tmap_y, smem + s * C::STAGE_BYTES, 0, (m.y & 0x3fffffff) * C::TILE, m.x % H, m.x / H, policy);
                tma_store_wait_read();
                mbar_arrive(&empty[s]);
            }
            tma_store_wait_all();
        }
    } else if (warp == C::MMA_WARP) {
        // ---------------- MMA warp ----------------
        // (tcgen05.mma issued by the leaders of several warpgroups at once lost completions now and
        // then; with a single issuing thread it has not.)
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_f32acc(kind_dtype(KIND), C::TILE, C::B_ROWS);
            const uint64_t b_desc0 = umma_desc_kmajor_sw128(smem_u32(bsm));
            uint64_t b_desc = b_desc0;
            int cur_slab = -1;
            uint32_t operands_seen[C::B_BUFFERS] = {0u, 0u};
            if (mr.enabled != 0 && !mbar_wait(home_done, 0)) report_wait_expired(status);
            for (int it = 0;; ++it) {
                const int s = it % C::STAGES, g = it % C::GROUPS;
                if (!mbar_wait(&full[s], (it / C::STAGES) & 1)) {
                    report_wait_expired(status);
                    break;
                }
                const int2 m = meta[s];
                const int slab = m.x;
                if (slab < 0) break;
                if (slab != cur_slab) {
                    const int buf = (m.y >> 30) & 1;
                    if (!mbar_wait(&b_ready[buf], operands_seen[buf] & 1u)) {
                        report_wait_expired(status);
                        break;
                    }
                    ++operands_seen[buf];
                    cur_slab = slab;
                    b_desc = b_desc0 + static_cast<uint64_t>(buf * (C::B_BYTES >> 4));  // start address field, 16-byte units
                }
                if (!mbar_wait(&a_ready[g], (it / C::GROUPS) & 1)) {
                    report_wait_expired(status);
                    break;
                }
                tc_fence_after_sync();
                const uint32_t a_tmem = tmem_base + g * C::TMEM_COLS_PER_GROUP, d_tmem = a_tmem + 32;
                // K = 64 as four steps of 16: A advances 8 columns (two 16-bit values per column), B 32 bytes
#pragma unroll
                for (int k = 0; k < 4; ++k) umma_ts(d_tmem, a_tmem + 8 * k, b_desc + 2 * k, idesc, k > 0 ? 1u : 0u);
                umma_commit(&mma_done[g]);
            }
        }
    } else {
        // ---------------- consumer warpgroups ----------------
        const int group = warp >> 2, wq = warp & 3;
        const int row = wq * 32 + lane;
        const uint32_t a_tmem = tmem_base + (static_cast<uint32_t>(wq * 32) << 16) + group * C::TMEM_COLS_PER_GROUP;
        const uint32_t d_tmem = a_tmem + 32;
        const uint32_t row_base = smem_u32(smem) + row * 128;
        const uint32_t sw = row & 7;
        uint32_t tiles_done = 0;
        for (int it = group;; it += C::GROUPS) {
            const int s = it % C::STAGES;
            if (!mbar_wait(&full[s], (it / C::STAGES) & 1)) {
                if (lane == 0) report_wait_expired(status);
                break;
            }
            const int slab = meta[s].x;
            __syncwarp();
            if (slab < 0) {
                if (lane == 0) mbar_arrive(&y_ready[s]);  // hand the end marker on to the store warp
                break;
            }
            const uint32_t base = row_base + s * C::STAGE_BYTES;
            {
                // the row's eight 16-byte chunks; a quarter-warp reads eight different chunk
                // positions (the swizzle), so the loads are free of bank conflicts
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
            const bool ok = mbar_wait(&mma_done[group], tiles_done & 1);
            ++tiles_done;
            __syncwarp();
            if (!ok) {
                if (lane == 0) report_wait_expired(status);
                break;
            }
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
            tc_fence_before_sync();  // orders the loads of D before the next tile's MMA (through a_ready)
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(&y_ready[s]);
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

}  // namespace lf
