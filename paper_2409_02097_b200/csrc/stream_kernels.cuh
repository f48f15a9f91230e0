// Persistent, TMA-pipelined kernels for head dim 64 (the SD-v2.1 / SD-XL shapes), where the
// operator is bound by HBM bandwidth: every byte of Q, K, V is read once through
// cp.async.bulk.tensor into 128-byte-swizzled shared-memory stages, and Y is written once with
// 16-byte stores.
//
// Work is cut into units of one token tile of one slab, numbered slab-major; CTA g of G owns
// the contiguous run of units [g*W/G, (g+1)*W/G).  That split is a pure function of the shape
// and the grid size, so the summation order — and with it every output bit — is fixed.
//
//   stream_state_kernel   — per CTA and per slab it touches: partial S_p = sum phi(K_j)^T V_j and
//                           z_p (Prop. 2, Eq. 5).  Eight consumer warps: warp w owns rows
//                           16*(w&3).. of the state and the token half (w>>2) of each 128-token
//                           tile; A = phi(K)^T and B = V come out of the stage with
//                           ldmatrix.trans, phi is applied to the A fragments in registers, and a
//                           ninth column block of ones produces z.  Each (CTA, slab, half) writes
//                           its own fp32 partial; nothing is combined with atomics.
//   stream_reduce_kernel  — sums the partials of a slab in (CTA, half) order; also lays S | z out
//                           as the bf16 MMA B-fragments the apply kernel loads.
//   stream_apply_kernel   — Y_i = phi(Q_i) S / (phi(Q_i) . z + eps).  S | z sit in registers as
//                           bf16 MMA B-fragments (reloaded when the CTA moves to another slab);
//                           Q tiles are handed out per slab through an atomic counter (the
//                           result of a tile does not depend on which CTA computes it);
//                           A = phi(Q) comes from the stage with ldmatrix; the
//                           columns of S are permuted so that every lane ends up with 8
//                           contiguous output channels and stores them as one 16-byte vector.
//
// One extra warp per CTA is the TMA producer.  All mbarrier waits are bounded; a wait that
// expires records kStatusWaitExpired in the status word and the CTA drains and exits.
#pragma once

#include "common.cuh"

namespace lf {

constexpr int kStreamD = 64;
constexpr int kStreamStateFloats = kStreamD * (kStreamD + 1);  // S [64][64] then z [64]
constexpr int kStreamRowBytes = kStreamD * 2;                  // 128: one swizzle span

struct StreamStateCfg {
    static constexpr int TILE = 128;  // tokens per stage
    static constexpr int CONSUMER_WARPS = 8;
    static constexpr int THREADS = 32 * (CONSUMER_WARPS + 1);
    static constexpr int STAGES = 2;
    static constexpr int CTAS_PER_SM = 3;
    static constexpr int TILE_BYTES = TILE * kStreamRowBytes;  // 16 KB per tensor
    static constexpr int STAGE_BYTES = 2 * TILE_BYTES;         // K then V
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*align*/ + 256 /*barriers*/;
};

template <int CW>
struct StreamApplyCfg {
    static constexpr int CONSUMER_WARPS = CW;
    static constexpr int TILE = 16 * CW;  // tokens per stage: one m16 block per consumer warp
    static constexpr int THREADS = 32 * (CW + 1);
    static constexpr int STAGE_BYTES = TILE * kStreamRowBytes;
    static constexpr int STAGES = (198 * 1024) / STAGE_BYTES;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 + 512;  // + align, barriers, meta
};

// First unit of CTA g when W units are dealt to G CTAs.
__host__ __device__ __forceinline__ long long unit_begin(long long g, long long W, long long G)
{
    return (g * W) / G;
}

__device__ __forceinline__ void report_wait_expired(uint32_t* status)
{
    atomicExch(status, kStatusWaitExpired);
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
// State: partials[(g * spans + slot) * 2 + half][kStreamStateFloats]
// ---------------------------------------------------------------------------------------------
template <int PHI>
__global__ void __launch_bounds__(StreamStateCfg::THREADS, StreamStateCfg::CTAS_PER_SM)
stream_state_kernel(const __grid_constant__ CUtensorMap tmap_k,
                    const __grid_constant__ CUtensorMap tmap_v, float* __restrict__ partials,
                    uint32_t* __restrict__ status, int N, int tiles_per_slab, long long W, int spans, int H)
{
    using C = StreamStateCfg;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + C::STAGES * C::STAGE_BYTES);
    uint64_t* empty = full + C::STAGES;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long G = gridDim.x, g = blockIdx.x;
    const long long u0 = unit_begin(g, W, G), u1 = unit_begin(g + 1, W, G);
    const int n_units = static_cast<int>(u1 - u0);

    if (tid == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], C::CONSUMER_WARPS);
        }
        mbar_fence_init();
    }
    __syncthreads();

    if (warp == C::CONSUMER_WARPS) {
        // ---------------- producer ----------------
        if (lane == 0) {
            prefetch_tmap(&tmap_k);
            prefetch_tmap(&tmap_v);
            const uint64_t policy = policy_evict_first();
            int issued = 0;
            for (int it = 0; it < n_units; ++it) {
                const int s = it % C::STAGES;
                const uint32_t ph = (it / C::STAGES) & 1;
                if (!mbar_wait(&empty[s], ph ^ 1)) {
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
        return;
    }

    // ---------------- consumers ----------------
    const int mb = warp & 3, half = warp >> 2;
    const int g8 = lane >> 2, t4 = lane & 3;
    float acc[9][4];
#pragma unroll
    for (int nb = 0; nb < 9; ++nb)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[nb][i] = 0.0f;

    // Lane offsets inside a swizzled tile: byte = row*128 + ((chunk ^ (row & 7)) << 4), and
    // row & 7 == lane & 7 for every row a lane addresses.
    const int sw = lane & 7;
    const uint32_t a_lane = (half * 64 + (lane & 7) + ((lane >> 4) << 3)) * 128 +
                            (((mb * 2 + ((lane >> 3) & 1)) ^ sw) << 4);
    const uint32_t b_lane = (half * 64 + (lane & 7) + (((lane >> 3) & 1) << 3)) * 128 +
                            (((lane >> 4) ^ sw) << 4);
    const uint32_t ones = 0x3F803F80u;
    const uint32_t smem_base = smem_u32(smem);

    auto flush = [&](int slab_first, int slab) {
        const int slot = slab - slab_first;
        float* dst = partials + ((static_cast<size_t>(g) * spans + slot) * 2 + half) * kStreamStateFloats;
        const int c0 = mb * 16 + g8, c1 = c0 + 8;
#pragma unroll
        for (int nb = 0; nb < 8; ++nb) {
            const int e = nb * 8 + 2 * t4;
            *reinterpret_cast<float2*>(dst + c0 * 64 + e) = make_float2(acc[nb][0], acc[nb][1]);
            *reinterpret_cast<float2*>(dst + c1 * 64 + e) = make_float2(acc[nb][2], acc[nb][3]);
        }
        if (t4 == 0) {
            dst[64 * 64 + c0] = acc[8][0];
            dst[64 * 64 + c1] = acc[8][2];
        }
#pragma unroll
        for (int nb = 0; nb < 9; ++nb)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[nb][i] = 0.0f;
    };

    const int slab_first = static_cast<int>(u0 / tiles_per_slab);
    int cur_slab = slab_first;
    bool failed = false;
    for (int it = 0; it < n_units; ++it) {
        const int s = it % C::STAGES;
        const uint32_t ph = (it / C::STAGES) & 1;
        const long long u = u0 + it;
        const int slab = static_cast<int>(u / tiles_per_slab);
        const int tile = static_cast<int>(u % tiles_per_slab);
        if (slab != cur_slab) {
            flush(slab_first, cur_slab);
            cur_slab = slab;
        }
        if (!failed && !mbar_wait(&full[s], ph)) {
            if (lane == 0) report_wait_expired(status);
            failed = true;
        }
        if (!failed) {
            const uint32_t kbase = smem_base + s * C::STAGE_BYTES;
            const uint32_t vbase = kbase + C::TILE_BYTES;
            const int valid = N - tile * C::TILE - half * 64;  // tokens of this warp's half inside N
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                uint32_t a0, a1, a2, a3;
                ldmatrix_x4_trans(kbase + a_lane + ks * 2048, a0, a1, a2, a3);
                a0 = phi_packed_bf16x2<PHI>(a0);
                a1 = phi_packed_bf16x2<PHI>(a1);
                a2 = phi_packed_bf16x2<PHI>(a2);
                a3 = phi_packed_bf16x2<PHI>(a3);
                if (valid < 64) {
                    // Rows past N were zero-filled by TMA, but phi(0) = 1: clear them explicitly.
                    // a0/a1 hold tokens j, j+1; a2/a3 hold j+8, j+9 with j = 16*ks + 2*t4.
                    const int j = ks * 16 + 2 * t4;
                    const uint32_t m01 = (j < valid ? 0x0000ffffu : 0u) | (j + 1 < valid ? 0xffff0000u : 0u);
                    const uint32_t m23 = (j + 8 < valid ? 0x0000ffffu : 0u) | (j + 9 < valid ? 0xffff0000u : 0u);
                    a0 &= m01;
                    a1 &= m01;
                    a2 &= m23;
                    a3 &= m23;
                }
#pragma unroll
                for (int nbp = 0; nbp < 4; ++nbp) {
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4_trans(vbase + ((b_lane + ks * 2048) ^ (nbp << 5)), b0, b1, b2, b3);
                    mma_bf16_16816(acc[2 * nbp], a0, a1, a2, a3, b0, b1);
                    mma_bf16_16816(acc[2 * nbp + 1], a0, a1, a2, a3, b2, b3);
                }
                mma_bf16_16816(acc[8], a0, a1, a2, a3, ones, ones);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[s]);
    }
    if (n_units > 0) flush(slab_first, cur_slab);
}

// Operand image of S | z for the apply kernel: bf16 MMA B-fragments in the order the lanes load
// them, [k block 4][column-block pair 5][lane 32][4 words] per slab.  Word w of pair p holds
// register (w & 1) of column block 2p + (w >> 1); block 8 is z, block 9 does not exist.
constexpr int kStreamFragWords = 4 * 5 * 32 * 4;

// Output channel carried by column slot g8 of column block nb (nb < 8): with this permutation a
// lane ends up owning channels 8*t4 .. 8*t4+7 (blocks 0-3) and 32+8*t4 .. (blocks 4-7) of its rows.
__host__ __device__ __forceinline__ int apply_channel_of(int nb, int g8)
{
    return 32 * (nb >> 2) + 8 * (g8 >> 1) + 2 * (nb & 3) + (g8 & 1);
}

// Block blockIdx.x of a (17, slabs) grid of 256 threads holds elements 256*blockIdx.x .. of one
// slab's fp32 state (S rows 4*blockIdx.x .., or z in block 16) in `sums`; write their share of the
// fragment image `fr` of that slab.
__device__ __forceinline__ void emit_state_fragments(const float* sums, uint32_t* fr)
{
    const int tid = threadIdx.x;
    if (blockIdx.x < 16) {
        // rows c = 4*blockIdx.x + tid/64 of S; even rows pack (S[c][e], S[c+1][e])
        const int r = tid >> 6, e = tid & 63;
        if ((r & 1) == 0) {
            const int c = 4 * blockIdx.x + r;
            const uint32_t pair = pack_bf16x2(sums[tid], sums[tid + 64]);
            const int kb = c >> 4, reg = (c >> 3) & 1, t4 = (c & 7) >> 1;
            const int r32 = e & 31;
            const int nb = 4 * (e >> 5) + ((r32 & 7) >> 1);
            const int g8 = 2 * (r32 >> 3) + (r32 & 1);
            fr[((kb * 5 + (nb >> 1)) * 32 + g8 * 4 + t4) * 4 + (nb & 1) * 2 + reg] = pair;
        }
    } else if (tid < 64 && (tid & 1) == 0) {
        // z: pair (z[c], z[c+1]) goes to every column slot of block 8
        const int c = tid;
        const uint32_t pair = pack_bf16x2(sums[tid], sums[tid + 1]);
        const int kb = c >> 4, reg = (c >> 3) & 1, t4 = (c & 7) >> 1;
        for (int g8 = 0; g8 < 8; ++g8) fr[((kb * 5 + 4) * 32 + g8 * 4 + t4) * 4 + reg] = pair;
    }
}

// grid (17, slabs), 256 threads: state[slab] = sum over the CTAs whose run meets the slab, in
// increasing CTA index, half 0 then half 1 (fp32, fixed order).  Also writes the bf16 fragment
// image of S | z for the apply kernel and clears the slab's tile counter for it.
__global__ void __launch_bounds__(256)
stream_reduce_kernel(const float* __restrict__ partials, float* __restrict__ state,
                     uint32_t* __restrict__ frags, int* __restrict__ tile_counters,
                     int tiles_per_slab, long long W, int G, int spans)
{
    __shared__ float sums[256];
    const int tid = threadIdx.x;
    const int idx = blockIdx.x * 256 + tid;
    const int slab = blockIdx.y;
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
        sum += src[((static_cast<size_t>(g0) * spans + slot0) * 2) * F];
        sum += src[((static_cast<size_t>(g0) * spans + slot0) * 2 + 1) * F];
        // Every later CTA starts inside this slab: its partial for it is in slot 0.
#pragma unroll 4
        for (long long g = g0 + 1; g < g1; ++g) {
            sum += src[(static_cast<size_t>(g) * spans * 2) * F];
            sum += src[(static_cast<size_t>(g) * spans * 2 + 1) * F];
        }
        state[static_cast<size_t>(slab) * F + idx] = sum;
    }
    sums[tid] = sum;
    __syncthreads();
    emit_state_fragments(sums, frags + static_cast<size_t>(slab) * kStreamFragWords);
}

// grid (17, slabs), 256 threads: rebuild the bf16 fragment image (and clear the tile counters) from
// an fp32 state that was changed outside the library — the sum over devices of a token-sharded
// forward (Sec. 4.3).
__global__ void __launch_bounds__(256)
stream_pack_kernel(const float* __restrict__ state, uint32_t* __restrict__ frags,
                   int* __restrict__ tile_counters)
{
    __shared__ float sums[256];
    const int tid = threadIdx.x;
    const int idx = blockIdx.x * 256 + tid;
    const int slab = blockIdx.y;
    if (blockIdx.x == 0 && tid == 0) tile_counters[slab] = 0;
    sums[tid] = idx < kStreamStateFloats ? state[static_cast<size_t>(slab) * kStreamStateFloats + idx] : 0.0f;
    __syncthreads();
    emit_state_fragments(sums, frags + static_cast<size_t>(slab) * kStreamFragWords);
}

// ---------------------------------------------------------------------------------------------
// Apply.  Tiles are handed out per slab through an atomic counter: CTA g starts on its home slab
// g*slabs/G and moves to the next slab that still has tiles when one runs dry, so the CTAs of a
// slab share its tail and early finishers help elsewhere.  Each output tile depends only on its
// own Q rows and the slab's S | z, so the result does not depend on who computes it.
// ---------------------------------------------------------------------------------------------
template <int PHI, int CW>
__global__ void __launch_bounds__(StreamApplyCfg<CW>::THREADS, 1)
stream_apply_kernel(const __grid_constant__ CUtensorMap tmap_q, const uint32_t* __restrict__ frags,
                    __nv_bfloat16* __restrict__ Y, int* __restrict__ tile_counters,
                    uint32_t* __restrict__ status, int N, int tiles_per_slab, int slabs, float eps, SlabLayout L)
{
    using C = StreamApplyCfg<CW>;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + C::STAGES * C::STAGE_BYTES);
    uint64_t* empty = full + C::STAGES;
    int2* meta = reinterpret_cast<int2*>(empty + C::STAGES);  // (slab, tile) of each stage; slab < 0 ends

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    if (tid == 0) {
        for (int s = 0; s < C::STAGES; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], C::CONSUMER_WARPS);
        }
        mbar_fence_init();
    }
    __syncthreads();

    if (warp == C::CONSUMER_WARPS) {
        // ---------------- producer warp (lane 0 issues; all lanes help to find work) ----------------
        uint64_t policy = 0;
        if (lane == 0) {
            prefetch_tmap(&tmap_q);
            policy = policy_evict_first();
        }
        int slab = static_cast<int>((static_cast<long long>(blockIdx.x) * slabs) / gridDim.x);
        int it = 0, issued = 0;
        bool ok = true;
        while (true) {
            int tile = 0;
            if (lane == 0) tile = atomicAdd(&tile_counters[slab], 1);
            tile = __shfl_sync(0xffffffffu, tile, 0);
            if (tile >= tiles_per_slab) {
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
                continue;
            }
            const int s = it % C::STAGES;
            if (lane == 0) {
                ok = mbar_wait(&empty[s], ((it / C::STAGES) & 1) ^ 1);
                if (ok) {
                    meta[s] = make_int2(slab, tile);
                    mbar_expect_tx(&full[s], C::STAGE_BYTES);
                    tma_load_4d(smem + s * C::STAGE_BYTES, &tmap_q, 0, tile * C::TILE, slab % L.H, slab / L.H, &full[s], policy);
                    ++issued;
                } else {
                    report_wait_expired(status);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            ++it;
        }
        if (lane == 0) {
            int first = 0;
            if (ok) {
                // End marker in the next stage (consumers leave when they see it).  Its stage held
                // load number issued - STAGES, which the consumers have released by now.
                const int s = it % C::STAGES;
                if (mbar_wait(&empty[s], ((it / C::STAGES) & 1) ^ 1)) {
                    meta[s] = make_int2(-1, 0);
                    mbar_arrive(&full[s]);
                    first = issued - C::STAGES + 1;
                } else {
                    report_wait_expired(status);
                }
            }
            drain_loads<C::STAGES>(full, first, issued, status);
        }
        return;
    }

    // ---------------- consumers ----------------
    const int g8 = lane >> 2, t4 = lane & 3;
    // A-fragment lane offset in the swizzled Q stage (non-transposed ldmatrix).
    const int sw = lane & 7;
    const uint32_t q_row = (warp * 16 + (lane & 7) + (((lane >> 3) & 1) << 3)) * 128;
    const uint32_t q_hi = lane >> 4;  // 16-byte chunk parity inside a 16-channel k block
    const uint32_t smem_base = smem_u32(smem);

    uint32_t sfrag[4][9][2];  // [k block][column block][b0, b1], bf16x2
    auto load_state = [&](int slab) {
        const uint4* fr = reinterpret_cast<const uint4*>(frags + static_cast<size_t>(slab) * kStreamFragWords) + lane;
#pragma unroll
        for (int kb = 0; kb < 4; ++kb) {
#pragma unroll
            for (int nbp = 0; nbp < 5; ++nbp) {
                const uint4 v = __ldg(fr + (kb * 5 + nbp) * 32);
                sfrag[kb][2 * nbp][0] = v.x;
                sfrag[kb][2 * nbp][1] = v.y;
                if (nbp < 4) {
                    sfrag[kb][2 * nbp + 1][0] = v.z;
                    sfrag[kb][2 * nbp + 1][1] = v.w;
                }
            }
        }
    };

    int cur_slab = -1;
    for (int it = 0;; ++it) {
        const int s = it % C::STAGES;
        if (!mbar_wait(&full[s], (it / C::STAGES) & 1)) {
            if (lane == 0) report_wait_expired(status);
            break;
        }
        const int2 m = meta[s];
        const int slab = m.x, tile = m.y;
        if (slab < 0) break;
        if (slab != cur_slab) {
            load_state(slab);
            cur_slab = slab;
        }
        const uint32_t qbase = smem_base + s * C::STAGE_BYTES + q_row;
        float acc[9][4];
#pragma unroll
        for (int kb = 0; kb < 4; ++kb) {
            uint32_t a0, a1, a2, a3;
            ldmatrix_x4(qbase + ((((kb << 1) | q_hi) ^ sw) << 4), a0, a1, a2, a3);
            a0 = phi_packed_bf16x2<PHI>(a0);
            a1 = phi_packed_bf16x2<PHI>(a1);
            a2 = phi_packed_bf16x2<PHI>(a2);
            a3 = phi_packed_bf16x2<PHI>(a3);
#pragma unroll
            for (int nb = 0; nb < 9; ++nb) {
                if (kb == 0)
                    mma_bf16_16816_init(acc[nb], a0, a1, a2, a3, sfrag[kb][nb][0], sfrag[kb][nb][1]);
                else
                    mma_bf16_16816(acc[nb], a0, a1, a2, a3, sfrag[kb][nb][0], sfrag[kb][nb][1]);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[s]);  // stage is free as soon as the fragments are read

        const float inv0 = 1.0f / (acc[8][0] + eps);
        const float inv1 = 1.0f / (acc[8][2] + eps);
        const long long r0 = static_cast<long long>(tile) * C::TILE + warp * 16 + g8, r1 = r0 + 8;
        __nv_bfloat16* y0 = Y + slab_base(L, slab) + static_cast<size_t>(r0) * L.row_stride;
        __nv_bfloat16* y1 = y0 + 8 * static_cast<size_t>(L.row_stride);
#pragma unroll
        for (int hi = 0; hi < 2; ++hi) {
            uint4 v0, v1;
            v0.x = pack_bf16x2(acc[4 * hi + 0][0] * inv0, acc[4 * hi + 0][1] * inv0);
            v0.y = pack_bf16x2(acc[4 * hi + 1][0] * inv0, acc[4 * hi + 1][1] * inv0);
            v0.z = pack_bf16x2(acc[4 * hi + 2][0] * inv0, acc[4 * hi + 2][1] * inv0);
            v0.w = pack_bf16x2(acc[4 * hi + 3][0] * inv0, acc[4 * hi + 3][1] * inv0);
            v1.x = pack_bf16x2(acc[4 * hi + 0][2] * inv1, acc[4 * hi + 0][3] * inv1);
            v1.y = pack_bf16x2(acc[4 * hi + 1][2] * inv1, acc[4 * hi + 1][3] * inv1);
            v1.z = pack_bf16x2(acc[4 * hi + 2][2] * inv1, acc[4 * hi + 2][3] * inv1);
            v1.w = pack_bf16x2(acc[4 * hi + 3][2] * inv1, acc[4 * hi + 3][3] * inv1);
            if (r0 < N) st_stream_16B(y0 + 32 * hi + 8 * t4, v0);
            if (r1 < N) st_stream_16B(y1 + 32 * hi + 8 * t4, v1);
        }
    }
}

}  // namespace lf
