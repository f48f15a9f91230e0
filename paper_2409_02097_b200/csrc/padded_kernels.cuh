// One persistent TMA + tcgen05 kernel per forward for head widths that are not a multiple of 64
// (the SD-v1.5 widths 40, 80 and 160): split-N state, fixed-order reduction and apply (Prop. 2,
// Eq. 5) in a single launch.
//
// Layout in shared memory.  A tile is 128 tokens of one tensor of one (batch, head) slab.  TMA
// delivers it as ceil(D / 64) blocks of 64 channels ("atoms": 128 rows of 128 bytes in the 128-byte
// swizzle); the channels past D of the last atom lie outside the tensor and arrive as zeros.  The
// tcgen05 descriptors address the atoms directly, so the padding costs shared memory but no HBM
// traffic and no extra instruction.  The padding also carries the normalizer: thread r of a
// warpgroup writes a one into channel D of token r's V row, so that row D of the state MMA's result
// is z = sum phi(K_j) (Eq. 5) and no separate operand block of ones is needed.
//
// Work split.  Every slab is cut into `per_slab` runs of whole tiles, one CTA per run (grid =
// slabs * per_slab <= SM count; all CTAs resident together; per_slab = 1 and grid = SM count when
// there are more slabs than SMs).  A CTA
//   1. streams the K and V tiles of its run through a ring of tile slots, applies phi to the K
//      rows in place, and accumulates  D[e][c] += sum_j [V | 1]_je phi(K)_jc  in tensor memory
//      (A = [V | 1]^T and B = phi(K)^T, both MN-major as TMA delivers them);
//   2. writes the accumulator to its fp32 partial in global memory (stored [c][e] like S itself:
//      the lanes of a warp hold consecutive e) and adds to the slab's counter; meanwhile its
//      producer already fetches the Q tiles of the same run into the slots that have been released;
//   3. waits (bounded) until all `per_slab` partials of the slab are there and sums them in run
//      order (the same order in every CTA of the slab, so all of them hold the same bits) into the
//      16-bit B operand of the apply MMA in shared memory — S | z with the channels e along
//      128-byte rows, one row per feature c, in the 128-byte swizzle (MN-major, the orientation of
//      S itself, so nothing is transposed anywhere); the CTAs of a slab share the writing of the
//      fp32 state;
//   4. per Q tile: phi in place, D[i][e] = sum_c phi(Q)_ic B_ce on tcgen05 (both operands from
//      shared memory), each thread divides its row by the z column (Eq. 5), writes the 16-bit row
//      over the Q row, and a TMA store (clipped at D channels and N tokens) sends the tile to Y.
// Every CTA of a slab reads all of its partials, so the host keeps per_slab small enough for that
// to stay a few hundred KB — or, where that would leave long runs (large partials: d = 160), asks for the
// shared form of step 3 (`scatter`): CTA r sums only its share of the rows c, publishes that share of the
// operand and of the fp32 state, and after a second counter round every CTA copies the whole operand.  A CTA that has its slab to itself (per_slab = 1) skips 2-3: it builds
// the operand and the fp32 state straight from the accumulator; with more slabs than SMs such a CTA
// takes several whole slabs one after the other (the K/V tiles of the next slab are fetched while the
// current one is applied).  The counters are zeroed again by the CTA that finishes last, so every
// forward starts from zero.
#pragma once

#include "stream_kernels.cuh"

namespace lf {

template <int D>
struct PaddedCfg {
    static_assert(D % 8 == 0 && D % 64 != 0 && D > 0 && D < 192, "widths with padding in their last 64-channel atom");
    static constexpr int TILE = 128;                        // tokens per tile = rows of an MMA tile
    static constexpr int NA = (D + 63) / 64;                // 64-channel atoms per row
    static constexpr int ATOM_BYTES = TILE * 128;           // 16 KB
    static constexpr int SLOT_BYTES = NA * ATOM_BYTES;      // one tile of one tensor
    static constexpr int DKN = (D + 15) / 16 * 16;          // N of the state MMA = K extent of the apply MMA
    static constexpr int DVN = (D + 1 + 15) / 16 * 16;      // N of the apply MMA: D channels, z, padding
    static constexpr int PARTIAL_FLOATS = DKN * DVN;        // partial[c][e]: e < D = S[c][e], e = D = z[c], then zeros
    static constexpr int ECHUNKS = D / 8 + 1;               // 8-channel chunks of a partial row that are used
    static constexpr int B_ATOM_BYTES = DKN * 128;          // one 64-channel atom of the apply operand: DKN rows c
    static constexpr int B_ATOMS = (DVN + 63) / 64;
    static constexpr int B_BYTES = B_ATOMS * B_ATOM_BYTES;
    static constexpr int STATE_MMAS = NA == 3 ? 2 : 1;      // rows e 0..127, then 128..191
    static constexpr int STATE_COLS = STATE_MMAS * DKN;
    static constexpr int APPLY_GROUPS = 2;
    static constexpr int TMEM_NEED = STATE_COLS > APPLY_GROUPS * DVN ? STATE_COLS : APPLY_GROUPS * DVN;
    static constexpr int TMEM_COLS = TMEM_NEED <= 32 ? 32 : TMEM_NEED <= 64 ? 64 : TMEM_NEED <= 128 ? 128 : TMEM_NEED <= 256 ? 256 : 512;
    static constexpr int CONSUMER_WARPS = 4 * APPLY_GROUPS;
    static constexpr int CONSUMER_THREADS = 32 * CONSUMER_WARPS;
    static constexpr int PRODUCER_WARP = CONSUMER_WARPS;
    static constexpr int MMA_WARP = CONSUMER_WARPS + 1;
    static constexpr int STORE_WARP = CONSUMER_WARPS + 2;
    static constexpr int THREADS = 32 * (CONSUMER_WARPS + 3);
    static constexpr int TAIL_BYTES = 1024 /*align*/ + 1024 /*barriers*/;
    static constexpr int SLOTS_FIT = (227 * 1024 - B_BYTES - TAIL_BYTES) / SLOT_BYTES;
    static constexpr int SLOTS = SLOTS_FIT > 12 ? 12 : SLOTS_FIT;
    static constexpr int SMEM_BYTES = SLOTS * SLOT_BYTES + B_BYTES + TAIL_BYTES;
    // One accumulation chain in tensor memory per run: 512 tiles = 4096 MMA steps (a 70 000-step chain was
    // measured to drift 8e-5 relative, far below the 16-bit operands' 4e-3).
    static constexpr int MAX_TILES_PER_CTA = 512;
    static constexpr int ARRIVALS = CONSUMER_WARPS;         // arrivals on the slab's counter per CTA
};

// First tile of run `r` when a slab's `tiles` tiles are cut into `runs` nearly equal runs.
__host__ __device__ __forceinline__ int padded_run_begin(int r, int tiles, int runs)
{
    return static_cast<int>((static_cast<long long>(r) * tiles) / runs);
}

// Control words behind the per-slab counters: ctrl[0] = CTAs of the running forward that have finished.
constexpr int kPaddedCtrlWords = 1;

// 16 columns of the lane's TMEM row into registers, without waiting: r[] may be read only after a
// tmem_wait_loads() that follows.  Lets the next block's load run while the previous one is consumed.
__device__ __forceinline__ void tmem_load_16cols_async(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_wait_loads() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// phi on the D real channels of one 128-token row held as atoms of 128-byte rows (`row_addr` = the
// row inside atom 0, `sw` = row & 7: 16-byte chunk c of a row sits at chunk position c ^ sw).
template <int D, int KIND>
__device__ __forceinline__ void phi_row_in_place(uint32_t row_addr, uint32_t sw)
{
    using C = PaddedCfg<D>;
#pragma unroll
    for (int c = 0; c < D / 8; ++c) {
        const uint32_t addr = row_addr + (c >> 3) * C::ATOM_BYTES + (((c & 7) ^ sw) << 4);
        uint32_t x0, x1, x2, x3;
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(x0), "=r"(x1), "=r"(x2), "=r"(x3) : "r"(addr));
        x0 = phi_packed_pair<KIND>(x0);
        x1 = phi_packed_pair<KIND>(x1);
        x2 = phi_packed_pair<KIND>(x2);
        x3 = phi_packed_pair<KIND>(x3);
        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(x0), "r"(x1), "r"(x2), "r"(x3) : "memory");
    }
}

// grid = slabs * per_slab CTAs; CTA g works on slab g / per_slab, run g % per_slab of its tiles (per_slab = 1:
// grid <= slabs, CTA g on slabs g, g + grid, ...).
// partials: [slab][run][DKN][DVN] fp32; state: [slab][D*D + D] fp32 (S [c][e], then z [c]); images (scatter
// only): [slab][B_BYTES], zero wherever nothing is ever written; counters: two words per slab, zero between
// forwards; ctrl: kPaddedCtrlWords words, zero between forwards.  SCATTER != 0: instead of every CTA of a slab
// summing all of its partials, CTA r sums its share of the rows c, publishes that share of the 16-bit operand
// (and of the fp32 state), and every CTA copies the whole operand once all shares are there — two exchange
// rounds instead of one, but per_slab times less to read: for slabs whose partials are large (d = 160).
template <int D, int KIND, int SCATTER>
__global__ void __launch_bounds__(PaddedCfg<D>::THREADS, 1)
padded_fused_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                    const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_y,
                    float* __restrict__ partials, float* __restrict__ state, unsigned char* __restrict__ images,
                    uint32_t* __restrict__ counters, uint32_t* __restrict__ ctrl, uint32_t* __restrict__ status, int N,
                    int tiles_per_slab, int per_slab, int slabs, int H, ApplyScales sc)
{
    using C = PaddedCfg<D>;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    unsigned char* bsm = smem + C::SLOTS * C::SLOT_BYTES;  // on a 1024-byte boundary
    uint64_t* full = reinterpret_cast<uint64_t*>(bsm + C::B_BYTES);
    uint64_t* empty = full + C::SLOTS;
    uint64_t* k_ready = empty + C::SLOTS;
    uint64_t* y_ready = k_ready + C::SLOTS;
    uint64_t* q_ready = y_ready + C::SLOTS;   // [APPLY_GROUPS]
    uint64_t* mma_done = q_ready + C::APPLY_GROUPS;  // [APPLY_GROUPS]
    uint64_t* acc_done = mma_done + C::APPLY_GROUPS;
    uint64_t* b_ready = acc_done + 1;
    uint64_t* drained = b_ready + 1;  // every consumer warp is through with the apply tiles of a visit
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drained + 1);
    // Ring positions the producer has issued so far.  A consumer looks at a slot's `full` barrier only once
    // the position it wants has been issued: the parity of an mbarrier wait tells phase n from phase n + 1,
    // not from phase n - 1, and a warpgroup whose first tile already sits in a reused slot would otherwise
    // take the completion of the slot's earlier use for its own.
    uint32_t* issued_pos = tmem_slot + 1;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // A CTA visits one run of one slab (per_slab > 1) or, with its slabs to itself, the whole slabs
    // blockIdx.x, blockIdx.x + gridDim.x, ... one after the other (more slabs than SMs).
    const int run = per_slab > 1 ? static_cast<int>(blockIdx.x) % per_slab : 0;
    const int first_slab = per_slab > 1 ? static_cast<int>(blockIdx.x) / per_slab : static_cast<int>(blockIdx.x);
    const int slab_step = static_cast<int>(gridDim.x);
    const int visits = per_slab > 1 ? 1 : (slabs - first_slab + slab_step - 1) / slab_step;
    const int t0 = padded_run_begin(run, tiles_per_slab, per_slab);
    const int n = padded_run_begin(run + 1, tiles_per_slab, per_slab) - t0;  // tiles per visit (>= 1)

    if (tid == 0) {
        for (int s = 0; s < C::SLOTS; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
            mbar_init(&k_ready[s], 4);
            mbar_init(&y_ready[s], 4);
        }
        for (int g = 0; g < C::APPLY_GROUPS; ++g) {
            mbar_init(&q_ready[g], 4);
            mbar_init(&mma_done[g], 1);
        }
        mbar_init(acc_done, 1);
        mbar_init(b_ready, C::CONSUMER_WARPS);
        mbar_init(drained, C::CONSUMER_WARPS);
        *issued_pos = 0u;
        mbar_fence_init();
    }
    // The apply operand's padding (rows c >= D everywhere; channels e > D where a CTA builds the operand
    // itself) stays zero.
    for (int i = tid; i < C::B_BYTES / 16; i += C::THREADS) reinterpret_cast<uint4*>(bsm)[i] = make_uint4(0u, 0u, 0u, 0u);
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
    // Set-up done: the next kernel of the stream may be scheduled behind this one; nothing in global
    // memory is touched before the kernel ahead has completed.
    pdl_launch_dependents();
    pdl_wait();

    // Ring positions of visit v, from base = 3 n v: K of state tile i at base + 2i, V at base + 2i + 1; Q (later Y)
    // of apply tile j at base + 2n + j.
    auto slot_of = [](int pos) { return pos % C::SLOTS; };
    auto phase_of = [](int pos) { return static_cast<uint32_t>((pos / C::SLOTS) & 1); };

    if (warp == C::PRODUCER_WARP) {
        // ---------------- producer ----------------
        if (lane == 0) {
            const uint64_t policy = policy_evict_first();
            int issued = 0;
            bool ok = true;
            for (int visit = 0; visit < visits && ok; ++visit) {
                const int slab = first_slab + visit * slab_step, head = slab % H, batch = slab / H;
                for (int pos = 0; pos < 3 * n && ok; ++pos) {
                    const int gp = visit * 3 * n + pos, s = slot_of(gp);
                    if (!mbar_wait(&empty[s], phase_of(gp) ^ 1u)) {
                        report_wait_expired(status);
                        ok = false;
                        break;
                    }
                    const void* map = pos >= 2 * n ? &tmap_q : ((pos & 1) != 0 ? &tmap_v : &tmap_k);
                    const int tile = t0 + (pos >= 2 * n ? pos - 2 * n : pos >> 1);
                    unsigned char* dst = smem + s * C::SLOT_BYTES;
                    mbar_expect_tx(&full[s], C::SLOT_BYTES);
#pragma unroll
                    for (int a = 0; a < C::NA; ++a)
                        tma_load_4d(dst + a * C::ATOM_BYTES, map, 64 * a, tile * C::TILE, head, batch, &full[s], policy);
                    ++issued;
                    asm volatile("st.release.cta.shared.u32 [%0], %1;" ::"r"(smem_u32(issued_pos)), "r"(static_cast<uint32_t>(issued)) : "memory");
                }
            }
            drain_loads<C::SLOTS>(full, 0, issued, status);
        }
    } else if (warp == C::MMA_WARP) {
        // ---------------- MMA warp: one thread issues every tcgen05.mma ----------------
        if (lane == 0) {
            bool ok = true;
            const uint32_t idesc_state = umma_idesc_f32acc(kind_dtype(KIND), 128, C::DKN, kUmmaAMnMajor | kUmmaBMnMajor);
            const uint32_t idesc_apply = umma_idesc_f32acc(kind_dtype(KIND), C::TILE, C::DVN, kUmmaBMnMajor);
            const uint32_t b_addr = smem_u32(bsm);
            uint32_t k_phase = 0u;  // bit s = phase of k_ready[s] to wait for next
            int jj = 0;             // apply tiles so far, over all visits: tile jj belongs to warpgroup jj % APPLY_GROUPS
            for (int visit = 0; visit < visits && ok; ++visit) {
                const int base = visit * 3 * n;
                // The accumulator shares its columns with the apply tiles of the visit before: those must
                // have been read out.
                if (visit > 0 && !mbar_wait(drained, static_cast<uint32_t>((visit - 1) & 1))) {
                    report_wait_expired(status);
                    ok = false;
                    break;
                }
                // state: D[e][c] += [V | 1]^T phi(K), 16 tokens per step
                for (int i = 0; i < n && ok; ++i) {
                    const int sk = slot_of(base + 2 * i), sv = slot_of(base + 2 * i + 1);
                    if (!mbar_wait(&k_ready[sk], (k_phase >> sk) & 1u)) {
                        report_wait_expired(status);
                        ok = false;
                        break;
                    }
                    k_phase ^= 1u << sk;
                    tc_fence_after_sync();
                    const uint32_t k_addr = smem_u32(smem + sk * C::SLOT_BYTES), v_addr = smem_u32(smem + sv * C::SLOT_BYTES);
#pragma unroll
                    for (int ks = 0; ks < C::TILE / 16; ++ks) {
                        const uint32_t acc = (i == 0 && ks == 0) ? 0u : 1u;
                        const uint64_t b_desc = umma_desc_mnmajor_sw128(k_addr + ks * 2048, C::ATOM_BYTES, 1024);
                        // rows e 0..127: atoms 0 and 1 of V (one atom: both halves read atom 0, rows 64.. are not used)
                        const uint64_t a_desc = umma_desc_mnmajor_sw128(v_addr + ks * 2048, C::NA >= 2 ? C::ATOM_BYTES : 0, 1024);
                        umma_ss(tmem_base, a_desc, b_desc, idesc_state, acc);
                        if (C::STATE_MMAS == 2) {
                            // rows e 128..191: atom 2 (read twice; rows 192.. are not used)
                            const uint64_t a2 = umma_desc_mnmajor_sw128(v_addr + 2 * C::ATOM_BYTES + ks * 2048, 0, 1024);
                            umma_ss(tmem_base + C::DKN, a2, b_desc, idesc_state, acc);
                        }
                    }
                    umma_commit(&empty[sk]);  // the slots are free once these MMAs have read them
                    umma_commit(&empty[sv]);
                }
                if (!ok) break;
                umma_commit(acc_done);
                // apply: D[i][e] = phi(Q) (S | z), 16 features per step
                if (!mbar_wait(b_ready, static_cast<uint32_t>(visit & 1))) {
                    report_wait_expired(status);
                    ok = false;
                    break;
                }
                for (int j = 0; j < n; ++j, ++jj) {
                    const int g = jj % C::APPLY_GROUPS, s = slot_of(base + 2 * n + j);
                    if (!mbar_wait(&q_ready[g], static_cast<uint32_t>((jj / C::APPLY_GROUPS) & 1))) {
                        report_wait_expired(status);
                        ok = false;
                        break;
                    }
                    tc_fence_after_sync();
                    const uint32_t q_addr = smem_u32(smem + s * C::SLOT_BYTES);
                    const uint32_t d_tmem = tmem_base + g * C::DVN;
#pragma unroll
                    for (int ks = 0; ks < C::DKN / 16; ++ks) {
                        const uint64_t a_desc = umma_desc_kmajor_sw128(q_addr + (ks >> 2) * C::ATOM_BYTES + (ks & 3) * 32);
                        const uint64_t b_desc = umma_desc_mnmajor_sw128(b_addr + ks * 2048, C::B_ATOM_BYTES, 1024);
                        umma_ss(d_tmem, a_desc, b_desc, idesc_apply, ks > 0 ? 1u : 0u);
                    }
                    umma_commit(&mma_done[g]);
                }
            }
        }
    } else if (warp == C::STORE_WARP) {
        // ---------------- store warp: Y tiles out, slots back to the producer ----------------
        if (lane == 0) {
            const uint64_t policy = policy_evict_first();
            uint32_t y_phase = 0u;
            bool ok = true;
            for (int visit = 0; visit < visits && ok; ++visit) {
                const int slab = first_slab + visit * slab_step, head = slab % H, batch = slab / H;
                for (int j = 0; j < n; ++j) {
                    const int s = slot_of(visit * 3 * n + 2 * n + j);
                    if (!mbar_wait(&y_ready[s], (y_phase >> s) & 1u)) {
                        report_wait_expired(status);
                        ok = false;
                        break;
                    }
                    y_phase ^= 1u << s;
                    const unsigned char* src = smem + s * C::SLOT_BYTES;
#pragma unroll
                    for (int a = 0; a < C::NA; ++a)
                        tma_store_4d(&tmap_y, src + a * C::ATOM_BYTES, 64 * a, (t0 + j) * C::TILE, head, batch, policy);
                    tma_store_wait_read();
                    mbar_arrive(&empty[s]);
                }
            }
            tma_store_wait_all();
        }
    } else {
        // ---------------- consumer warpgroups ----------------
        const int group = warp >> 2, wq = warp & 3;
        const int row = wq * 32 + lane;
        const int ctid = tid;  // 0 .. CONSUMER_THREADS-1
        const uint32_t sw = row & 7;
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(wq * 32) << 16);
        bool ok = true;
        // Until the producer has issued ring position `pos` (bounded like every other wait).
        auto wait_issued = [&](int pos) {
            const uint32_t addr = smem_u32(issued_pos);
            uint32_t v;
            asm volatile("ld.acquire.cta.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
            if (v > static_cast<uint32_t>(pos)) return true;
            const unsigned long long t0 = global_timer_ns();
            do {
                __nanosleep(20);
                asm volatile("ld.acquire.cta.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
                if (v > static_cast<uint32_t>(pos)) return true;
            } while (global_timer_ns() - t0 < kMaxBarrierWaitNs);
            return false;
        };

        uint32_t tiles_done = 0;  // apply tiles of this warpgroup so far, over all visits
        const uint32_t d_tmem = lane_base + group * C::DVN;
        const int dtype = kind_dtype(KIND);
        for (int visit = 0; visit < visits && ok; ++visit) {
        const int slab = first_slab + visit * slab_step, base = visit * 3 * n;
        // 1. phi(K) in place, a one into channel D of V
        for (int i = group; i < n && ok; i += C::APPLY_GROUPS) {
            const int sk = slot_of(base + 2 * i), sv = slot_of(base + 2 * i + 1);
            ok = wait_issued(base + 2 * i + 1) && mbar_wait(&full[sk], phase_of(base + 2 * i)) &&
                 mbar_wait(&full[sv], phase_of(base + 2 * i + 1));
            __syncwarp();
            if (!ok) {
                if (lane == 0) report_wait_expired(status);
                break;
            }
            // rows past N arrive as zeros and must count for nothing: phi(0) = 1, so they are left alone
            if ((t0 + i) * C::TILE + row < N) {
                phi_row_in_place<D, KIND>(smem_u32(smem + sk * C::SLOT_BYTES) + row * 128, sw);
                const uint32_t one_addr = smem_u32(smem + sv * C::SLOT_BYTES) + (D / 64) * C::ATOM_BYTES + row * 128 +
                                          ((((D % 64) / 8) ^ sw) << 4);
                asm volatile("st.shared.u16 [%0], %1;" ::"r"(one_addr), "h"(static_cast<uint16_t>(ones_pair<KIND>() & 0xffffu)) : "memory");
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(&k_ready[sk]);
        }

        float* st = state + static_cast<size_t>(slab) * (D * D + D);

        // 2. the accumulator (row e = TMEM lane, DKN columns c)
        if (ok) {
            ok = mbar_wait(acc_done, static_cast<uint32_t>(visit & 1));
            __syncwarp();
            if (!ok && lane == 0) report_wait_expired(status);
        }
        if (ok) {
            tc_fence_after_sync();
            const int e = group * 128 + row;  // group 0 reads the first state MMA's rows, group 1 the second's
            // rows D < e < DVN of the accumulator are exact zeros (channels of V that TMA filled with zeros)
            const bool warp_has_rows = group < C::STATE_MMAS && group * 128 + wq * 32 < C::DVN;
            if (warp_has_rows) {
                float* dst = partials + (static_cast<size_t>(slab) * per_slab + run) * C::PARTIAL_FLOATS + e;
                const uint32_t b_row = smem_u32(bsm) + (e >> 6) * C::B_ATOM_BYTES + (e & 7) * 2;
                uint32_t dd[2][16];
                tmem_load_16cols_async(lane_base + group * C::DKN, dd[0]);
#pragma unroll
                for (int c0 = 0; c0 < C::DKN; c0 += 16) {
                    uint32_t (&d)[16] = dd[(c0 >> 4) & 1];
                    tmem_wait_loads();
                    if (c0 + 16 < C::DKN) tmem_load_16cols_async(lane_base + group * C::DKN + c0 + 16, dd[((c0 >> 4) + 1) & 1]);
                    if (e < C::DVN) {
                        if (per_slab == 1) {
                            // alone on the slab: S[c][e] | z[c] -> operand row c, channel e (eight lanes fill one
                            // 16-byte chunk), and the fp32 state
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                const int c = c0 + i;
                                const float v = __uint_as_float(d[i]);
                                asm volatile("st.shared.u16 [%0], %1;" ::"r"(b_row + c * 128 + ((((e & 63) >> 3) ^ (c & 7)) << 4)),
                                             "h"(to_storage16(v * sc.operand, dtype))
                                             : "memory");
                                if (c < D && e <= D) st[e < D ? c * D + e : D * D + c] = v;
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 16; ++i) __stcg(dst + (c0 + i) * C::DVN, __uint_as_float(d[i]));
                        }
                    }
                }
            }
            tc_fence_before_sync();
        }
        __syncwarp();

        if (per_slab > 1) {
            // 3. all partials of the slab, summed in run order -> the apply operand; this CTA's share of the
            //    rows c also goes to the fp32 state
            uint32_t* cnt = counters + 2 * slab;
            unsigned char* image = images + static_cast<size_t>(slab) * C::B_BYTES;
            if (lane == 0) red_release_gpu_add(cnt, 1u);  // also after a failure: the others must not wait for it
            if (ok) {
                uint32_t arrived = 0u;
                if (lane == 0) arrived = counter_wait(cnt, 0u, static_cast<uint32_t>(C::ARRIVALS * per_slab)) ? 1u : 0u;
                arrived = __shfl_sync(0xffffffffu, arrived, 0);
                if (arrived == 0u) {
                    ok = false;
                    if (lane == 0) report_wait_expired(status);
                }
            }
            if (ok) {
                // Work items are (row c, 8-channel chunk j) x (partial p), consecutive threads on consecutive
                // chunks of a row; a thread walks through the partials of its items with eight 32-byte loads
                // in flight and adds them in run order.
                const float* src0 = partials + static_cast<size_t>(slab) * per_slab * C::PARTIAL_FLOATS;
                const int c_begin = padded_run_begin(run, D, per_slab), c_end = padded_run_begin(run + 1, D, per_slab);
                const uint32_t b_addr = smem_u32(bsm);
                // rows c >= D of the operand stay zero; with scatter only this CTA's rows are summed here
                const int row0 = SCATTER != 0 ? c_begin : 0;
                const int kItems = (SCATTER != 0 ? c_end - c_begin : D) * C::ECHUNKS;  // a constant without SCATTER
                int item = ctid, p = 0;
                float acc[8];
                while (item < kItems) {
                    float4 a[8], b[8];
                    int it2 = item, p2 = p;
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        if (it2 < kItems) {
                            const int r2 = it2 / C::ECHUNKS, j2 = it2 - r2 * C::ECHUNKS, c2 = row0 + r2;
                            const float4* sp = reinterpret_cast<const float4*>(src0 + static_cast<size_t>(p2) * C::PARTIAL_FLOATS +
                                                                              c2 * C::DVN + j2 * 8);
                            a[u] = __ldcg(sp);
                            b[u] = __ldcg(sp + 1);
                            if (++p2 == per_slab) {
                                p2 = 0;
                                it2 += C::CONSUMER_THREADS;
                            }
                        }
                    }
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        if (item < kItems) {
                            if (p == 0) {
                                acc[0] = a[u].x; acc[1] = a[u].y; acc[2] = a[u].z; acc[3] = a[u].w;
                                acc[4] = b[u].x; acc[5] = b[u].y; acc[6] = b[u].z; acc[7] = b[u].w;
                            } else {
                                acc[0] += a[u].x; acc[1] += a[u].y; acc[2] += a[u].z; acc[3] += a[u].w;
                                acc[4] += b[u].x; acc[5] += b[u].y; acc[6] += b[u].z; acc[7] += b[u].w;
                            }
                            if (++p == per_slab) {
                                const int r = item / C::ECHUNKS, j = item - r * C::ECHUNKS, c = row0 + r;
                                const uint32_t v0 = to_storage16(acc[0] * sc.operand, dtype) | (static_cast<uint32_t>(to_storage16(acc[1] * sc.operand, dtype)) << 16);
                                const uint32_t v1 = to_storage16(acc[2] * sc.operand, dtype) | (static_cast<uint32_t>(to_storage16(acc[3] * sc.operand, dtype)) << 16);
                                const uint32_t v2 = to_storage16(acc[4] * sc.operand, dtype) | (static_cast<uint32_t>(to_storage16(acc[5] * sc.operand, dtype)) << 16);
                                const uint32_t v3 = to_storage16(acc[6] * sc.operand, dtype) | (static_cast<uint32_t>(to_storage16(acc[7] * sc.operand, dtype)) << 16);
                                // operand row c, channels 8 j .. 8 j + 7: atom j / 8, chunk position (j % 8) ^ (c % 8)
                                const uint32_t b_off = (j >> 3) * C::B_ATOM_BYTES + c * 128 + (((j & 7) ^ (c & 7)) << 4);
                                if (SCATTER != 0)
                                    __stcg(reinterpret_cast<uint4*>(image + b_off), make_uint4(v0, v1, v2, v3));
                                else
                                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(b_addr + b_off), "r"(v0), "r"(v1), "r"(v2), "r"(v3)
                                                 : "memory");
                                if (c >= c_begin && c < c_end) {
                                    if (j < D / 8) {
                                        float4* sp = reinterpret_cast<float4*>(st + c * D + j * 8);
                                        sp[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
                                        sp[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
                                    } else {
                                        st[D * D + c] = acc[0];  // channel D of the row: z[c]
                                    }
                                }
                                p = 0;
                                item += C::CONSUMER_THREADS;
                            }
                        }
                    }
                }
            }
            if (SCATTER != 0) {
                // second round: every share of the operand image is there -> copy it (eight loads in flight)
                __syncwarp();
                if (lane == 0) red_release_gpu_add(&cnt[1], 1u);
                if (ok) {
                    uint32_t arrived = 0u;
                    if (lane == 0) arrived = counter_wait(&cnt[1], 0u, static_cast<uint32_t>(C::ARRIVALS * per_slab)) ? 1u : 0u;
                    arrived = __shfl_sync(0xffffffffu, arrived, 0);
                    if (arrived == 0u) {
                        ok = false;
                        if (lane == 0) report_wait_expired(status);
                    }
                }
                if (ok) {
                    const uint4* src = reinterpret_cast<const uint4*>(image);
                    uint4* dst = reinterpret_cast<uint4*>(bsm);
                    constexpr int kVec = C::B_BYTES / 16;
                    for (int i0 = ctid; i0 < kVec; i0 += 8 * C::CONSUMER_THREADS) {
                        uint4 v[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u)
                            if (i0 + u * C::CONSUMER_THREADS < kVec) v[u] = __ldcg(src + i0 + u * C::CONSUMER_THREADS);
#pragma unroll
                        for (int u = 0; u < 8; ++u)
                            if (i0 + u * C::CONSUMER_THREADS < kVec) dst[i0 + u * C::CONSUMER_THREADS] = v[u];
                    }
                }
            }
        }
        if (ok) fence_proxy_async_smem();
        __syncwarp();
        if (ok && lane == 0) mbar_arrive(b_ready);

        // 4. apply: tile j of this visit is tile visit * n + j overall, and goes to warpgroup (visit * n + j) % APPLY_GROUPS
        const int j_first = ((group - visit * n) % C::APPLY_GROUPS + C::APPLY_GROUPS) % C::APPLY_GROUPS;
        for (int j = j_first; j < n && ok; j += C::APPLY_GROUPS) {
            const int pos = base + 2 * n + j, s = slot_of(pos);
            ok = wait_issued(pos) && mbar_wait(&full[s], phase_of(pos));
            __syncwarp();
            if (!ok) {
                if (lane == 0) report_wait_expired(status);
                break;
            }
            const uint32_t row_addr = smem_u32(smem + s * C::SLOT_BYTES) + row * 128;
            if ((t0 + j) * C::TILE + row < N) phi_row_in_place<D, KIND>(row_addr, sw);
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(&q_ready[group]);
            ok = mbar_wait(&mma_done[group], tiles_done & 1u);
            ++tiles_done;
            __syncwarp();
            if (!ok) {
                if (lane == 0) report_wait_expired(status);
                break;
            }
            tc_fence_after_sync();
            uint32_t dd[2][16];
            tmem_load_16cols_async(d_tmem, dd[0]);
            const float den = __uint_as_float(tmem_load_1col(d_tmem + D));  // phi(Q_i) . z (waits for both loads)
            const float inv = row_scale(den, sc);
#pragma unroll
            for (int cb = 0; cb < C::DKN / 16; ++cb) {
                uint32_t (&d)[16] = dd[cb & 1];
                if (cb > 0) tmem_wait_loads();
                if (cb + 1 < C::DKN / 16) tmem_load_16cols_async(d_tmem + 16 * (cb + 1), dd[(cb + 1) & 1]);
#pragma unroll
                for (int h2 = 0; h2 < 2; ++h2) {
                    const int cc = 2 * cb + h2;  // 16-byte chunk of the output row
                    const uint32_t v0 = pack_pair<KIND>(__uint_as_float(d[8 * h2 + 0]) * inv, __uint_as_float(d[8 * h2 + 1]) * inv);
                    const uint32_t v1 = pack_pair<KIND>(__uint_as_float(d[8 * h2 + 2]) * inv, __uint_as_float(d[8 * h2 + 3]) * inv);
                    const uint32_t v2 = pack_pair<KIND>(__uint_as_float(d[8 * h2 + 4]) * inv, __uint_as_float(d[8 * h2 + 5]) * inv);
                    const uint32_t v3 = pack_pair<KIND>(__uint_as_float(d[8 * h2 + 6]) * inv, __uint_as_float(d[8 * h2 + 7]) * inv);
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(row_addr + (cc >> 3) * C::ATOM_BYTES + (((cc & 7) ^ sw) << 4)),
                                 "r"(v0), "r"(v1), "r"(v2), "r"(v3)
                                 : "memory");
                }
            }
            tc_fence_before_sync();  // orders the loads of D before the group's next MMA (through q_ready)
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(&y_ready[s]);
        }
        // this warp has read its last tile of the visit out of tensor memory
        __syncwarp();
        if (ok && lane == 0) mbar_arrive(drained);
        }  // visits
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
    // The CTA that finishes last puts the counters back to zero for the next forward (every CTA is
    // past its wait by then).
    if (tid == 0) {
        __threadfence();
        if (atomicAdd(&ctrl[0], 1u) == gridDim.x - 1) {
            for (int s = 0; s < 2 * slabs; ++s) counters[s] = 0u;
            ctrl[0] = 0u;
            __threadfence();
        }
    }
}

}  // namespace lf
