// Kernels for any supported pair of widths (DK = d', the feature width of Q and K; DV = d, the
// channel width of V and Y; Prop. 3 — the released model has DK = DV), multiples of 8 up to 160,
// built on warp-level tensor-core MMAs with operands staged in shared memory by plain 16-byte loads:
//
//   state_partial_kernel  — split-N partial state  S_p = sum_{j in chunk} phi(K_j)^T V_j,
//                           z_p = sum phi(K_j)                        (Prop. 2, Eq. 5)
//   state_reduce_kernel   — fixed-order sum of the partials into S | z
//   apply_kernel          — Y_i = phi(Q_i) S / (phi(Q_i) . z + eps)
//   cluster_fused_kernel  — all three in one launch: one thread-block cluster per slab, the
//                           partial states summed in rank order through distributed shared memory
//
// MMA roles.  State: D[c][e] += A[c][j] B[j][e] with A = phi(K)^T and B = V, the contraction
// running over tokens j; one warp owns one 16-row block of c and every column block of e,
// plus one extra column block fed with ones, which yields z.  Apply: D[i][e] += A[i][c] B[c][e]
// with A = phi(Q) and B = S (held transposed, in the 16-bit storage type), one warp per 16 tokens, plus one
// extra column block holding z in every column, which yields the denominator.
#pragma once

#include <cooperative_groups.h>

#include "common.cuh"

namespace lf {

namespace cg = cooperative_groups;

template <int DK, int DV>
struct SplitCfg {
    static_assert(DK % 8 == 0 && DK >= 8 && DK <= 160, "feature width must be a multiple of 8 in [8, 160]");
    static_assert(DV % 8 == 0 && DV >= 8 && DV <= 160, "value width must be a multiple of 8 in [8, 160]");
    static constexpr int DKP = (DK + 15) / 16 * 16;  // features padded to the MMA's 16
    static constexpr int DVP = (DV + 15) / 16 * 16;  // value channels padded to the MMA's 16
    static constexpr int MB = DKP / 16;              // 16-row blocks of the state = warps per CTA
    static constexpr int NBV = DV / 8;               // 8-column blocks over V channels
    static constexpr int NBT = NBV + 1;              // + the ones / z block
    static constexpr int CHK = DKP / 8;              // 16-byte chunks per padded row of Q / K
    static constexpr int CHV = DVP / 8;              // ... of V
    static constexpr int PITCHK = (CHK | 1) * 16;    // smem row pitches, odd in 16-byte units
    static constexpr int PITCHV = (CHV | 1) * 16;
    static constexpr int NT = 32 * MB;               // threads per CTA
    static constexpr int TILE_KV = 64;               // tokens per K/V tile
    static constexpr int TILE_Q = 16 * MB;           // tokens per Q tile (one m16 block per warp)
    static constexpr int LD_K = TILE_KV * CHK / NT;  // 16-byte chunks per thread per tile
    static constexpr int LD_V = (TILE_KV * CHV + NT - 1) / NT;
    static constexpr int LD_Q = TILE_Q * CHK / NT;
    static_assert(TILE_KV * CHK % NT == 0 && TILE_Q * CHK % NT == 0, "tile must split evenly");
    static constexpr int ST_ROWS = (DV + 8 + 15) / 16 * 16;  // S^T rows: DV channels, 8 z rows, pad
    static constexpr int STATE_FLOATS = DK * (DV + 1);       // S [DK][DV] then z [DK]

    static constexpr int SMEM_KV = TILE_KV * (PITCHK + PITCHV);  // phi(K) tile + V tile
    static constexpr int SMEM_Q = TILE_Q * PITCHK;
    static constexpr int SMEM_ST = ST_ROWS * PITCHK;
    static constexpr int SMEM_APPLY = SMEM_ST + SMEM_Q;
    static constexpr int SMEM_STAGE = (SMEM_KV > SMEM_Q ? SMEM_KV : SMEM_Q);
    static constexpr int SMEM_CLUSTER = STATE_FLOATS * 4 + SMEM_ST + SMEM_STAGE;
};

constexpr int kMaxClusterSize = 16;  // beyond the portable 8: needs the non-portable launch attribute

// First tile of chunk `p` when `tiles` tiles are cut into `chunks` nearly equal runs.
__host__ __device__ __forceinline__ int chunk_begin(int p, int tiles, int chunks)
{
    return static_cast<int>((static_cast<long long>(p) * tiles) / chunks);
}

// ---------------------------------------------------------------------------------------------
// State accumulation over K/V tiles [tile0, tile1) of one slab.  acc[nb][.] holds this warp's
// 16 x 8 block (rows c = 16*warp + ..., columns 8*nb + ...), acc[NBV] the z block.  `rsk`, `rsv`:
// elements from one token row to the next in K and in V.
// ---------------------------------------------------------------------------------------------
template <int DK, int DV, int KIND>
__device__ __forceinline__ void accumulate_state(const __nv_bfloat16* __restrict__ Ks,
                                                 const __nv_bfloat16* __restrict__ Vs, int N, int rsk, int rsv,
                                                 int tile0, int tile1, unsigned char* smem_kv,
                                                 float (&acc)[SplitCfg<DK, DV>::NBT][4])
{
    using C = SplitCfg<DK, DV>;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned char* Ksm = smem_kv;
    unsigned char* Vsm = smem_kv + C::TILE_KV * C::PITCHK;

#pragma unroll
    for (int nb = 0; nb < C::NBT; ++nb)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[nb][i] = 0.0f;

    uint4 kreg[C::LD_K], vreg[C::LD_V];
    const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);

    auto load_tile = [&](int tile) {
#pragma unroll
        for (int i = 0; i < C::LD_K; ++i) {
            int idx = tid + i * C::NT;
            int row = idx / C::CHK, ch = idx % C::CHK;
            long long j = static_cast<long long>(tile) * C::TILE_KV + row;
            bool ok = (j < N) && (ch * 8 < DK);
            kreg[i] = ok ? ld_stream_16B(Ks + j * rsk + ch * 8) : zero4;
        }
#pragma unroll
        for (int i = 0; i < C::LD_V; ++i) {
            int idx = tid + i * C::NT;
            int row = idx / C::CHV, ch = idx % C::CHV;
            long long j = static_cast<long long>(tile) * C::TILE_KV + row;
            bool ok = (idx < C::TILE_KV * C::CHV) && (j < N) && (ch * 8 < DV);
            vreg[i] = ok ? ld_stream_16B(Vs + j * rsv + ch * 8) : zero4;
        }
    };
    auto store_tile = [&](int tile) {
#pragma unroll
        for (int i = 0; i < C::LD_K; ++i) {
            int idx = tid + i * C::NT;
            int row = idx / C::CHK, ch = idx % C::CHK;
            long long j = static_cast<long long>(tile) * C::TILE_KV + row;
            bool ok = (j < N) && (ch * 8 < DK);
            uint4 pk = zero4;  // rows past N and pad channels contribute nothing (not phi(0) = 1)
            if (ok) {
                pk.x = phi_pair<KIND>(kreg[i].x);
                pk.y = phi_pair<KIND>(kreg[i].y);
                pk.z = phi_pair<KIND>(kreg[i].z);
                pk.w = phi_pair<KIND>(kreg[i].w);
            }
            *reinterpret_cast<uint4*>(Ksm + row * C::PITCHK + ch * 16) = pk;
        }
#pragma unroll
        for (int i = 0; i < C::LD_V; ++i) {
            int idx = tid + i * C::NT;
            int row = idx / C::CHV, ch = idx % C::CHV;
            if (idx < C::TILE_KV * C::CHV) *reinterpret_cast<uint4*>(Vsm + row * C::PITCHV + ch * 16) = vreg[i];
        }
    };

    const uint32_t ksm_base = smem_u32(Ksm), vsm_base = smem_u32(Vsm);
    // ldmatrix.trans lane addressing.  A (16 c x 16 j) from the phi(K) tile stored [j][c]:
    // matrices (j0, c0), (j0, c0+8), (j0+8, c0), (j0+8, c0+8).  B (16 j x 16 e) from the V tile
    // stored [j][e]: matrices (j0, e0), (j0+8, e0), (j0, e0+8), (j0+8, e0+8).
    const uint32_t a_off = ((lane & 7) + ((lane >> 4) << 3)) * C::PITCHK +
                           (warp * 16 + ((lane >> 3) & 1) * 8) * 2;
    const uint32_t b_off = ((lane & 7) + (((lane >> 3) & 1) << 3)) * C::PITCHV + ((lane >> 4) * 8) * 2;
    const uint32_t ones = ones_pair<KIND>();

    if (tile0 < tile1) load_tile(tile0);
    for (int tile = tile0; tile < tile1; ++tile) {
        store_tile(tile);
        __syncthreads();
        if (tile + 1 < tile1) load_tile(tile + 1);
#pragma unroll
        for (int ks = 0; ks < C::TILE_KV / 16; ++ks) {
            uint32_t a0, a1, a2, a3;
            ldmatrix_x4_trans(ksm_base + ks * 16 * C::PITCHK + a_off, a0, a1, a2, a3);
#pragma unroll
            for (int nbp = 0; nbp < (C::NBV + 1) / 2; ++nbp) {
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4_trans(vsm_base + ks * 16 * C::PITCHV + b_off + nbp * 32, b0, b1, b2, b3);
                mma_16816<KIND>(acc[2 * nbp], a0, a1, a2, a3, b0, b1);
                if (2 * nbp + 1 < C::NBV) mma_16816<KIND>(acc[2 * nbp + 1], a0, a1, a2, a3, b2, b3);
            }
            mma_16816<KIND>(acc[C::NBV], a0, a1, a2, a3, ones, ones);
        }
        __syncthreads();
    }
}

// Write this warp's rows of the state as fp32: S [DK][DV] then z [DK] at `dst` (global or shared).
template <int DK, int DV>
__device__ __forceinline__ void store_state(float* dst, const float (&acc)[SplitCfg<DK, DV>::NBT][4])
{
    using C = SplitCfg<DK, DV>;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int c0 = warp * 16 + g, c1 = c0 + 8;
#pragma unroll
    for (int nb = 0; nb < C::NBV; ++nb) {
        int e = nb * 8 + 2 * t;
        if (c0 < DK) g_store(reinterpret_cast<float2*>(dst + c0 * DV + e), make_float2(acc[nb][0], acc[nb][1]));
        if (c1 < DK) g_store(reinterpret_cast<float2*>(dst + c1 * DV + e), make_float2(acc[nb][2], acc[nb][3]));
    }
    if (t == 0) {
        if (c0 < DK) g_store(dst + DK * DV + c0, acc[C::NBV][0]);
        if (c1 < DK) g_store(dst + DK * DV + c1, acc[C::NBV][2]);
    }
}

// ---------------------------------------------------------------------------------------------
// Apply over Q tiles [tile0, tile1) of one slab, with S^T | z resident in shared memory in the
// 16-bit storage type.  `rsq`, `rsy`: elements from one token row to the next in Q and in Y.
// ---------------------------------------------------------------------------------------------
template <int DK, int DV, int KIND>
__device__ __forceinline__ void apply_tiles(const __nv_bfloat16* __restrict__ Qs,
                                            __nv_bfloat16* __restrict__ Ys, int N, int rsq, int rsy, int tile0,
                                            int tile1, const unsigned char* St, unsigned char* Qsm,
                                            ApplyScales sc)
{
    using C = SplitCfg<DK, DV>;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
    uint4 qreg[C::LD_Q];

    auto load_tile = [&](int tile) {
#pragma unroll
        for (int i = 0; i < C::LD_Q; ++i) {
            int idx = tid + i * C::NT;
            int row = idx / C::CHK, ch = idx % C::CHK;
            long long r = static_cast<long long>(tile) * C::TILE_Q + row;
            bool ok = (r < N) && (ch * 8 < DK);
            qreg[i] = ok ? ld_stream_16B(Qs + r * rsq + ch * 8) : zero4;
        }
    };
    auto store_tile = [&](int tile) {
#pragma unroll
        for (int i = 0; i < C::LD_Q; ++i) {
            int idx = tid + i * C::NT;
            int row = idx / C::CHK, ch = idx % C::CHK;
            long long r = static_cast<long long>(tile) * C::TILE_Q + row;
            bool ok = (r < N) && (ch * 8 < DK);
            uint4 pq = zero4;
            if (ok) {
                pq.x = phi_pair<KIND>(qreg[i].x);
                pq.y = phi_pair<KIND>(qreg[i].y);
                pq.z = phi_pair<KIND>(qreg[i].z);
                pq.w = phi_pair<KIND>(qreg[i].w);
            }
            *reinterpret_cast<uint4*>(Qsm + row * C::PITCHK + ch * 16) = pq;
        }
    };

    // Non-transposed ldmatrix.  A (16 i x 16 c) from the phi(Q) tile stored [i][c]: matrices
    // (i0, c0), (i0+8, c0), (i0, c0+8), (i0+8, c0+8).  B (16 c x 16 e) from S^T stored [e][c]:
    // matrices (e0, c0), (e0, c0+8), (e0+8, c0), (e0+8, c0+8).
    const uint32_t q_base = smem_u32(Qsm) + (warp * 16 + (lane & 7) + (((lane >> 3) & 1) << 3)) * C::PITCHK +
                            ((lane >> 4) * 8) * 2;
    const uint32_t s_base = smem_u32(St) + ((lane & 7) + ((lane >> 4) << 3)) * C::PITCHK +
                            (((lane >> 3) & 1) * 8) * 2;

    if (tile0 < tile1) load_tile(tile0);
    for (int tile = tile0; tile < tile1; ++tile) {
        store_tile(tile);
        __syncthreads();
        if (tile + 1 < tile1) load_tile(tile + 1);

        float acc[C::NBT][4];
#pragma unroll
        for (int nb = 0; nb < C::NBT; ++nb)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[nb][i] = 0.0f;
#pragma unroll
        for (int kb = 0; kb < C::MB; ++kb) {
            uint32_t a0, a1, a2, a3;
            ldmatrix_x4(q_base + kb * 32, a0, a1, a2, a3);
#pragma unroll
            for (int nbp = 0; nbp < (C::NBT + 1) / 2; ++nbp) {
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4(s_base + nbp * 16 * C::PITCHK + kb * 32, b0, b1, b2, b3);
                mma_16816<KIND>(acc[2 * nbp], a0, a1, a2, a3, b0, b1);
                if (2 * nbp + 1 < C::NBT) mma_16816<KIND>(acc[2 * nbp + 1], a0, a1, a2, a3, b2, b3);
            }
        }
        // Every column of the z block holds phi(Q_i) . z for its row.
        const float inv0 = row_scale(acc[C::NBV][0], sc);
        const float inv1 = row_scale(acc[C::NBV][2], sc);
        const long long r0 = static_cast<long long>(tile) * C::TILE_Q + warp * 16 + g, r1 = r0 + 8;
#pragma unroll
        for (int nb = 0; nb < C::NBV; ++nb) {
            int e = nb * 8 + 2 * t;
            if (r0 < N) st_stream_4B(Ys + r0 * rsy + e, pack_pair<KIND>(acc[nb][0] * inv0, acc[nb][1] * inv0));
            if (r1 < N) st_stream_4B(Ys + r1 * rsy + e, pack_pair<KIND>(acc[nb][2] * inv1, acc[nb][3] * inv1));
        }
        __syncthreads();
    }
}

// Fill the shared S^T | z operand (16-bit storage type, scaled; rows = output channel e, then 8 rows of z, then zero
// rows; columns = feature c padded with zeros) from fp32 S [DK][DV], z [DK].  `read(idx)` returns
// element idx of that fp32 state.
template <int DK, int DV, typename ReadFn>
__device__ __forceinline__ void fill_state_operand(unsigned char* St, ReadFn read, int dtype, float scale)
{
    using C = SplitCfg<DK, DV>;
    constexpr int kBatch = 8;  // the reads of one batch are issued together, then stored
    const int total = C::DKP * C::ST_ROWS, stride = blockDim.x;
    for (int base = threadIdx.x; base < total; base += kBatch * stride) {
        float val[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int idx = base + u * stride;
            const int c = idx / C::ST_ROWS, e = idx % C::ST_ROWS;
            val[u] = 0.0f;
            if (idx < total && c < DK) {
                if (e < DV) val[u] = read(c * DV + e);
                else if (e < DV + 8) val[u] = read(DK * DV + c);
            }
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int idx = base + u * stride;
            const int c = idx / C::ST_ROWS, e = idx % C::ST_ROWS;
            if (idx < total)
                *reinterpret_cast<uint16_t*>(St + e * C::PITCHK + c * 2) = to_storage16(val[u] * scale, dtype);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Kernels
// ---------------------------------------------------------------------------------------------

// grid (chunks, slabs).  partials: [slab][chunk][DK*(DV+1)] fp32.  LK, LV: where a slab's rows sit
// in K and in V (they differ only when DK != DV).
template <int DK, int DV, int KIND>
__global__ void __launch_bounds__(SplitCfg<DK, DV>::NT)
state_partial_kernel(const __nv_bfloat16* __restrict__ K, const __nv_bfloat16* __restrict__ V,
                     float* __restrict__ partials, int N, int chunks, SlabLayout LK, SlabLayout LV)
{
    // Programmatic dependent launch: the next kernel of the stream may be scheduled behind this
    // one; nothing in global memory is touched before the kernel ahead has completed.
    pdl_launch_dependents();
    pdl_wait();
    using C = SplitCfg<DK, DV>;
    extern __shared__ __align__(128) unsigned char smem[];
    const int slab = blockIdx.y, p = blockIdx.x;
    const int tiles = (N + C::TILE_KV - 1) / C::TILE_KV;
    float acc[C::NBT][4];
    accumulate_state<DK, DV, KIND>(K + slab_base(LK, slab), V + slab_base(LV, slab), N, LK.row_stride, LV.row_stride,
                                  chunk_begin(p, tiles, chunks), chunk_begin(p + 1, tiles, chunks), smem, acc);
    store_state<DK, DV>(partials + (static_cast<size_t>(slab) * chunks + p) * C::STATE_FLOATS, acc);
}

// One element of the fp32 state S [dk][dv] | z [dk] -> its place(s) in the apply kernel's operand image:
// S[c][e] to row e, column c; z[c] to column c of rows dv .. dv+7.
__device__ __forceinline__ void put_state_operand(unsigned char* img, int idx, uint16_t b, int dk, int dv, int pitch)
{
    if (idx < dk * dv) {
        const int c = idx / dv, e = idx - c * dv;
        g_store(reinterpret_cast<uint16_t*>(img + e * pitch + c * 2), b);
    } else {
        const int c = idx - dk * dv;
        for (int j = 0; j < 8; ++j) g_store(reinterpret_cast<uint16_t*>(img + (dv + j) * pitch + c * 2), b);
    }
}

// grid (ceil(state_floats / 256), slabs).  Sums `chunks` partials per slab in index order.  If
// `st_image` is not null it also receives the S^T | z operand of the apply kernel (16-bit storage
// type `dtype`, values times `operand_scale`), laid out
// exactly as that kernel holds it in shared memory (`image_bytes` per slab, rows `pitch` bytes
// apart: row e < dv holds S[.][e], rows dv .. dv+7 hold z; pad bytes stay as the host zeroed them).
__global__ void __launch_bounds__(256)
state_reduce_kernel(const float* __restrict__ partials, float* __restrict__ state, int state_floats,
                    int chunks, unsigned char* __restrict__ st_image, int dk, int dv, int pitch, int image_bytes,
                    int dtype, float operand_scale)
{
    // Programmatic dependent launch: the next kernel of the stream may be scheduled behind this
    // one; nothing in global memory is touched before the kernel ahead has completed.
    pdl_launch_dependents();
    pdl_wait();
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= state_floats) return;
    const int slab = blockIdx.y;
    const float* src = partials + static_cast<size_t>(slab) * chunks * state_floats + idx;
    float sum = 0.0f;
    for (int p = 0; p < chunks; ++p) sum += g_load(src + static_cast<size_t>(p) * state_floats);
    g_store(state + static_cast<size_t>(slab) * state_floats + idx, sum);
    if (st_image != nullptr)
        put_state_operand(st_image + static_cast<size_t>(slab) * image_bytes, idx,
                          to_storage16(sum * operand_scale, dtype), dk, dv, pitch);
}

// grid (ceil(state_floats / 256), slabs): the apply kernel's operand image from the sum, in index
// order, of the fp32 states of the devices of a token-sharded forward (Sec. 4.3; loads from peers'
// memory when the list holds peers' buffers).  Same image layout as state_reduce_kernel writes.
__global__ void __launch_bounds__(256)
peer_sum_image_kernel(PeerStates states, int state_floats, unsigned char* __restrict__ st_image, int dk, int dv,
                      int pitch, int image_bytes, int dtype, float operand_scale)
{
    pdl_launch_dependents();
    pdl_wait();
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= state_floats) return;
    const int slab = blockIdx.y;
    const float sum = peer_sum(states, static_cast<size_t>(slab) * state_floats + idx);
    put_state_operand(st_image + static_cast<size_t>(slab) * image_bytes, idx,
                      to_storage16(sum * operand_scale, dtype), dk, dv, pitch);
}

// grid (chunks, slabs).  `st_image` (may be null) is the operand image written by
// state_reduce_kernel; without it every CTA converts the fp32 state itself.
template <int DK, int DV, int KIND>
__global__ void __launch_bounds__(SplitCfg<DK, DV>::NT)
apply_kernel(const __nv_bfloat16* __restrict__ Q, const float* __restrict__ state,
             __nv_bfloat16* __restrict__ Y, int N, int chunks, ApplyScales sc, SlabLayout LK, SlabLayout LV,
             const unsigned char* __restrict__ st_image)
{
    // Programmatic dependent launch: the next kernel of the stream may be scheduled behind this
    // one; nothing in global memory is touched before the kernel ahead has completed.
    pdl_launch_dependents();
    pdl_wait();
    using C = SplitCfg<DK, DV>;
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* St = smem;
    unsigned char* Qsm = smem + C::SMEM_ST;
    const int slab = blockIdx.y, p = blockIdx.x;
    const int tiles = (N + C::TILE_Q - 1) / C::TILE_Q;
    if (st_image != nullptr) {
        // The reduction kernel left the operand in its shared-memory layout: plain 16-byte copy.
        const uint4* img = reinterpret_cast<const uint4*>(st_image + static_cast<size_t>(slab) * C::SMEM_ST);
        for (int i = threadIdx.x; i < C::SMEM_ST / 16; i += blockDim.x)
            reinterpret_cast<uint4*>(St)[i] = g_load_ro(img + i);
    } else {
        const float* st = state + static_cast<size_t>(slab) * C::STATE_FLOATS;
        fill_state_operand<DK, DV>(St, [&](int i) { return g_load_ro(st + i); }, kind_dtype(KIND), sc.operand);
    }
    __syncthreads();
    apply_tiles<DK, DV, KIND>(Q + slab_base(LK, slab), Y + slab_base(LV, slab), N, LK.row_stride, LV.row_stride,
                             chunk_begin(p, tiles, chunks), chunk_begin(p + 1, tiles, chunks), St, Qsm, sc);
}

// The state fragments of accumulate_state() -> the 16-bit S^T | z operand in shared memory (which must
// have been cleared: pad rows and columns stay zero).  For a CTA that holds a slab's whole state.
template <int DK, int DV, int KIND>
__device__ __forceinline__ void state_fragments_to_operand(unsigned char* St, const float (&acc)[SplitCfg<DK, DV>::NBT][4],
                                                           float scale)
{
    using C = SplitCfg<DK, DV>;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int c0 = warp * 16 + g, c1 = c0 + 8;
    auto put = [&](int row, int c, float v) {
        *reinterpret_cast<uint16_t*>(St + row * C::PITCHK + c * 2) = to_storage16(v * scale, kind_dtype(KIND));
    };
#pragma unroll
    for (int nb = 0; nb < C::NBV; ++nb) {
        const int e = nb * 8 + 2 * t;  // S[c][e] goes to row e, column c
        if (c0 < DK) {
            put(e, c0, acc[nb][0]);
            put(e + 1, c0, acc[nb][1]);
        }
        if (c1 < DK) {
            put(e, c1, acc[nb][2]);
            put(e + 1, c1, acc[nb][3]);
        }
    }
    // z[c] to column c of rows DV .. DV+7: lane t of a quad writes rows DV + 2t, DV + 2t + 1 (every
    // column of the z block holds the same sum)
    if (c0 < DK) {
        put(DV + 2 * t, c0, acc[C::NBV][0]);
        put(DV + 2 * t + 1, c0, acc[C::NBV][0]);
    }
    if (c1 < DK) {
        put(DV + 2 * t, c1, acc[C::NBV][2]);
        put(DV + 2 * t + 1, c1, acc[C::NBV][2]);
    }
}

// One cluster of `cluster_size` CTAs per slab (grid.x = cluster_size, grid.y = slabs).  CTA r
// accumulates the partial state of its run of K/V tiles into its own shared memory; after a
// cluster barrier CTA r sums slice r of the partials over ranks 0, 1, ... in that order and pushes
// the result into every CTA's operand through distributed shared memory (so all CTAs hold the same
// bits); after a second barrier every CTA applies to its run of Q.  state_out (may be null)
// receives S | z in fp32.
template <int DK, int DV, int KIND>
__global__ void __launch_bounds__(SplitCfg<DK, DV>::NT)
cluster_fused_kernel(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K,
                     const __nv_bfloat16* __restrict__ V, __nv_bfloat16* __restrict__ Y,
                     float* __restrict__ state_out, int N, ApplyScales sc, SlabLayout LK, SlabLayout LV)
{
    using C = SplitCfg<DK, DV>;
    extern __shared__ __align__(128) unsigned char smem[];
    float* part = reinterpret_cast<float*>(smem);
    unsigned char* St = smem + C::STATE_FLOATS * 4;
    unsigned char* stage = St + C::SMEM_ST;

    cg::cluster_group cluster = cg::this_cluster();
    const int rank = static_cast<int>(cluster.block_rank());
    const int csize = static_cast<int>(cluster.num_blocks());
    const int slab = blockIdx.y;
    const size_t off_k = slab_base(LK, slab), off_v = slab_base(LV, slab);

    if (csize == 1) {
        // One CTA holds the slab's whole state: nothing to exchange.  The state goes from the MMA
        // fragments straight into the apply operand (and, in fp32, to state_out).
        pdl_launch_dependents();
        pdl_wait();
        for (int i = threadIdx.x; i < C::SMEM_ST / 16; i += blockDim.x)
            reinterpret_cast<uint4*>(St)[i] = make_uint4(0u, 0u, 0u, 0u);
        const int tiles = (N + C::TILE_KV - 1) / C::TILE_KV;
        float acc[C::NBT][4];
        accumulate_state<DK, DV, KIND>(K + off_k, V + off_v, N, LK.row_stride, LV.row_stride, 0, tiles, stage, acc);
        // (accumulate_state ends with a barrier: the clear above is complete)
        state_fragments_to_operand<DK, DV, KIND>(St, acc, sc.operand);
        if (state_out != nullptr) store_state<DK, DV>(state_out + static_cast<size_t>(slab) * C::STATE_FLOATS, acc);
        __syncthreads();
        const int qtiles = (N + C::TILE_Q - 1) / C::TILE_Q;
        apply_tiles<DK, DV, KIND>(Q + off_k, Y + off_v, N, LK.row_stride, LV.row_stride, 0, qtiles, St, stage, sc);
        return;
    }

    {
        const int tiles = (N + C::TILE_KV - 1) / C::TILE_KV;
        float acc[C::NBT][4];
        accumulate_state<DK, DV, KIND>(K + off_k, V + off_v, N, LK.row_stride, LV.row_stride,
                                      chunk_begin(rank, tiles, csize), chunk_begin(rank + 1, tiles, csize), stage, acc);
        store_state<DK, DV>(part, acc);
    }
    // Clear the own S^T | z operand (pad rows and columns must be zero) before any peer writes to it.
    for (int i = threadIdx.x; i < C::SMEM_ST / 16; i += blockDim.x)
        reinterpret_cast<uint4*>(St)[i] = make_uint4(0u, 0u, 0u, 0u);
    cluster.sync();

    // Reduce-scatter with push: CTA r sums slice r of the state over ranks 0, 1, ... in that order
    // (fixed order), and stores the 16-bit result into the S^T | z operand of every CTA of the
    // cluster through distributed shared memory (remote stores do not stall the writer), and the
    // fp32 result into state_out.
    {
        const int slice = (C::STATE_FLOATS + csize - 1) / csize;
        const int begin = rank * slice;
        const int end = begin + slice < C::STATE_FLOATS ? begin + slice : C::STATE_FLOATS;
        float* gout = state_out != nullptr ? state_out + static_cast<size_t>(slab) * C::STATE_FLOATS : nullptr;
        constexpr int kBatch = 8;  // elements in flight per thread; ranks are visited in order
        for (int base = begin + threadIdx.x; base < end; base += kBatch * blockDim.x) {
            float sum[kBatch];
#pragma unroll
            for (int u = 0; u < kBatch; ++u) sum[u] = 0.0f;
#pragma unroll 1
            for (int r = 0; r < csize; ++r) {
                const float* src = cluster.map_shared_rank(part, r);
                float v[kBatch];
#pragma unroll
                for (int u = 0; u < kBatch; ++u) {
                    const int i = base + u * blockDim.x;
                    v[u] = i < end ? src[i] : 0.0f;
                }
#pragma unroll
                for (int u = 0; u < kBatch; ++u) sum[u] += v[u];
            }
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const int i = base + u * blockDim.x;
                if (i >= end) continue;
                if (gout != nullptr) g_store(gout + i, sum[u]);
                const uint16_t b = to_storage16(sum[u] * sc.operand, kind_dtype(KIND));
                // S[c][e] goes to row e, column c of the operand; z[c] to column c of rows DV .. DV+7.
                const bool is_z = i >= DK * DV;
                const int c = is_z ? i - DK * DV : i / DV;
                const int row0 = is_z ? DV : i - c * DV;
                const int rows = is_z ? 8 : 1;
#pragma unroll 1
                for (int r = 0; r < csize; ++r) {
                    unsigned char* dst = cluster.map_shared_rank(St, r) + row0 * C::PITCHK + c * 2;
#pragma unroll 1
                    for (int j = 0; j < rows; ++j) *reinterpret_cast<uint16_t*>(dst + j * C::PITCHK) = b;
                }
            }
        }
    }
    cluster.sync();  // every operand is complete; no CTA leaves while a peer still reads `part`

    const int qtiles = (N + C::TILE_Q - 1) / C::TILE_Q;
    apply_tiles<DK, DV, KIND>(Q + off_k, Y + off_v, N, LK.row_stride, LV.row_stride, chunk_begin(rank, qtiles, csize),
                             chunk_begin(rank + 1, qtiles, csize), St, stage, sc);
}

}  // namespace lf
