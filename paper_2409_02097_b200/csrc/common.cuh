// Device helpers shared by the attention kernels: the activation phi, 16-bit packing,
// warp-level tensor-core fragments (ldmatrix / mma.sync), bounded mbarrier + TMA wrappers, and the
// tcgen05 (tensor memory, 5th-generation MMA) wrappers of the stream, fused and producer kernels.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace lf {

constexpr int kPhiEluPlusOne = 0;
constexpr int kPhiIdentity = 1;

// Storage type of Q, K, V, Y (and of the MMA operands).  Kernels are instantiated on one integer
// KIND = phi | (dtype << 1); pointers to 16-bit data are typed __nv_bfloat16 whatever the dtype.
constexpr int kDtypeBf16 = 0;
constexpr int kDtypeFp16 = 1;
__host__ __device__ constexpr int make_kind(int phi, int dtype) { return phi | (dtype << 1); }
__host__ __device__ constexpr int kind_phi(int kind) { return kind & 1; }
__host__ __device__ constexpr int kind_dtype(int kind) { return kind >> 1; }

// Status word values written by kernels (0 = fine).
constexpr uint32_t kStatusOk = 0u;
constexpr uint32_t kStatusWaitExpired = 1u;

// Upper bound on the time one mbarrier wait may take, in nanoseconds of the global timer: far beyond
// any legitimate wait here (microseconds, or the length of a kernel for the waits that span one),
// so that a lost transaction ends the kernel with an error word instead of a hang.
constexpr unsigned long long kMaxBarrierWaitNs = 250ull * 1000ull * 1000ull;
// How long one try_wait may keep the thread suspended (it wakes as soon as the phase completes):
// long, so that a waiting warp issues next to no instructions.
constexpr uint32_t kBarrierSuspendHintNs = 1000u * 1000u;

// Where the rows of one (batch, head) slab sit in a tensor, in elements.  Head-major [B,H,N,d]:
// batch_stride = H*N*d, head_stride = N*d, row_stride = d.  Token-major [B,N,H,d] (what a UNet
// holds before it splits heads): batch_stride = N*H*d, head_stride = d, row_stride = H*d.
struct SlabLayout {
    long long batch_stride;
    long long head_stride;
    int row_stride;
    int H;
};

__host__ __device__ __forceinline__ size_t slab_base(const SlabLayout& L, int slab)
{
    return static_cast<size_t>(slab / L.H) * L.batch_stride + static_cast<size_t>(slab % L.H) * L.head_stride;
}

// ---------------------------------------------------------------------------------------------
// phi (Sec. 2.2: non-negative activation on the K and Q features).  elu(x) + 1:
// x + 1 for x > 0, exp(x) otherwise; both branches give 1 at 0.  exp(min(x, 0)) is 1 on the
// positive side, so phi = max(x, 0) + exp(min(x, 0)) without a branch.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int KIND>
__device__ __forceinline__ float phi(float x)
{
    if (kind_phi(KIND) == kPhiIdentity) return x;
    return fmaxf(x, 0.0f) + ex2_approx(fminf(x, 0.0f) * 1.4426950408889634f);
}

// Row scale of the apply step: 1 / (phi(Q_i) . z + eps) (Eq. 5), or `unnormalized_scale` for the
// operator without its normalizer, which the host requests by passing a negative eps.  (With fp16
// operands S | z are held scaled by a power of two s so that z fits the format; the scale cancels
// in the quotient when eps is scaled too, and unnormalized_scale = 1/s undoes it otherwise.)
constexpr float kEpsUnnormalized = -1.0f;
struct ApplyScales {
    float eps;           // eps * operand, or kEpsUnnormalized
    float unnormalized;  // 1 / operand
    float operand;       // the power of two s that S | z are multiplied by when they become an MMA operand
};
__device__ __forceinline__ float row_scale(float den, const ApplyScales& sc)
{
    return sc.eps < 0.0f ? sc.unnormalized : 1.0f / (den + sc.eps);
}

// The fp32 states S | z of the devices of a token-sharded forward (Sec. 4.3), as device addresses
// this GPU can load from (its own buffer, and peers' buffers mapped over NVLink).  Kernels sum them
// in index order with plain loads, so every device that is given the same list gets the same bits.
constexpr int kMaxPeers = 16;
struct PeerStates {
    const float* p[kMaxPeers];
    int n;
};

__device__ __forceinline__ float bf16_lo(uint32_t p) { return __uint_as_float(p << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t p) { return __uint_as_float(p & 0xffff0000u); }

// Two floats -> packed bf16x2 (lo in the low half), round-to-nearest-even.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Packed pair of the kernel's storage type <-> two floats.
template <int KIND>
__device__ __forceinline__ uint32_t pack_pair(float lo, float hi)
{
    return kind_dtype(KIND) == kDtypeFp16 ? pack_f16x2(lo, hi) : pack_bf16x2(lo, hi);
}
template <int KIND>
__device__ __forceinline__ float pair_lo(uint32_t p)
{
    if (kind_dtype(KIND) == kDtypeFp16) {
        float f;
        asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %1;\n\tcvt.f32.f16 %0, l;\n\t}" : "=f"(f) : "r"(p));
        return f;
    }
    return bf16_lo(p);
}
template <int KIND>
__device__ __forceinline__ float pair_hi(uint32_t p)
{
    if (kind_dtype(KIND) == kDtypeFp16) {
        float f;
        asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %1;\n\tcvt.f32.f16 %0, h;\n\t}" : "=f"(f) : "r"(p));
        return f;
    }
    return bf16_hi(p);
}
// The pair (1, 1).
template <int KIND>
__device__ __forceinline__ constexpr uint32_t ones_pair()
{
    return kind_dtype(KIND) == kDtypeFp16 ? 0x3C003C00u : 0x3F803F80u;
}
// One float -> the 16-bit storage type, by a run-time dtype (kernels that are not instantiated per kind).
__device__ __forceinline__ uint16_t to_storage16(float x, int dtype)
{
    const uint32_t p = dtype == kDtypeFp16 ? pack_f16x2(x, 0.0f) : pack_bf16x2(x, 0.0f);
    return static_cast<uint16_t>(p & 0xffffu);
}

template <int KIND>
__device__ __forceinline__ uint32_t phi_pair(uint32_t p)
{
    return pack_pair<KIND>(phi<KIND>(pair_lo<KIND>(p)), phi<KIND>(pair_hi<KIND>(p)));
}

// The same activation on a packed pair, entirely in packed 16-bit arithmetic (6 PTX instructions per
// pair instead of 13 through fp32).  log2(e) is split into a head and a tail of the format so that
// t = min(x,0) * log2(e) is the correctly rounded product (one fused rounding).  bf16: rounding t
// adds a relative error of about |x| * 2^-9 to exp(x), and the bf16 exponential instruction rounds
// its result toward zero (measured mean -0.27 % on the negative side, where the fp32 route has
// none) — both of the order of the bf16 rounding the MMA operand gets anyway.  fp16 has three more
// mantissa bits and the same structure.
template <int KIND>
__device__ __forceinline__ uint32_t phi_packed_pair(uint32_t p)
{
    if (kind_phi(KIND) == kPhiIdentity) return p;
    const uint32_t zero = 0u;
    uint32_t m, u, t, e, r;
    if (kind_dtype(KIND) == kDtypeFp16) {
        const uint32_t log2e_hi = 0x3DC53DC5u;  // fp16 pair 1.4423828125
        const uint32_t log2e_lo = 0x0D1E0D1Eu;  // fp16 pair log2(e) - 1.4423828125 = 3.1233e-4
        asm("min.f16x2 %0, %1, %2;" : "=r"(m) : "r"(p), "r"(zero));
        asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(u) : "r"(m), "r"(log2e_lo));
        asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(t) : "r"(m), "r"(log2e_hi), "r"(u));
        asm("ex2.approx.f16x2 %0, %1;" : "=r"(e) : "r"(t));
        asm("max.f16x2 %0, %1, %2;" : "=r"(r) : "r"(p), "r"(zero));
        asm("add.rn.f16x2 %0, %1, %2;" : "=r"(r) : "r"(r), "r"(e));
        return r;
    }
    const uint32_t log2e_hi = 0x3FB93FB9u;  // bf16 pair 1.4453125
    const uint32_t log2e_lo = 0xBB2CBB2Cu;  // bf16 pair log2(e) - 1.4453125 = -0.0026245
    asm("min.bf16x2 %0, %1, %2;" : "=r"(m) : "r"(p), "r"(zero));
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(u) : "r"(m), "r"(log2e_lo));
    asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(t) : "r"(m), "r"(log2e_hi), "r"(u));
    asm("ex2.approx.ftz.bf16x2 %0, %1;" : "=r"(e) : "r"(t));
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(p), "r"(zero));
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(r), "r"(e));
    return r;
}

// ---------------------------------------------------------------------------------------------
// Shared-memory addressing and fragment loads
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                            uint32_t& r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1,
                                                  uint32_t& r2, uint32_t& r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}

// D(16x8, fp32) += A(16x16, row) * B(16x8, col), operands bf16 or fp16 by KIND
template <int KIND>
__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1)
{
    if (kind_dtype(KIND) == kDtypeFp16)
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
            "{%0,%1,%2,%3};"
            : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    else
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
            "{%0,%1,%2,%3};"
            : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// ---------------------------------------------------------------------------------------------
// Checked build (-DLF_CHECKED; a second library, for debugging, never the one that is benchmarked).
// The host registers the byte ranges a forward may touch (Q, K, V, Y, the workspace, peers' states);
// every global-memory access the split / cluster kernels compute an address for goes through
// lf_in_bounds(): an access that does not lie wholly inside one registered range is counted and
// SKIPPED (a load returns zeros) — no trap, no fault, the kernel runs to its end and the host reads
// the count.  Addresses in shared memory (the cluster kernel keeps partial states there) pass.
// In the normal build lf_in_bounds() is the constant true and costs nothing.
// ---------------------------------------------------------------------------------------------
#ifdef LF_CHECKED
constexpr int kCheckedMaxRanges = 24;
struct CheckedRanges {
    unsigned long long lo[kCheckedMaxRanges];
    unsigned long long hi[kCheckedMaxRanges];
    int n;
};
__device__ CheckedRanges g_checked_ranges;
__device__ unsigned int g_checked_violations;
__device__ __forceinline__ bool lf_in_bounds(const void* p, unsigned int bytes)
{
    if (!__isGlobal(p)) return true;
    const unsigned long long a = reinterpret_cast<unsigned long long>(p);
    for (int i = 0; i < g_checked_ranges.n; ++i)
        if (a >= g_checked_ranges.lo[i] && a + bytes <= g_checked_ranges.hi[i]) return true;
    atomicAdd(&g_checked_violations, 1u);
    return false;
}
#else
__device__ __forceinline__ constexpr bool lf_in_bounds(const void*, unsigned int) { return true; }
#endif

// Plain global loads and stores of the split / cluster kernels, through the check above.
template <typename T>
__device__ __forceinline__ T g_load(const T* p)
{
    if (!lf_in_bounds(p, sizeof(T))) return T{};
    return *p;
}
template <typename T>
__device__ __forceinline__ T g_load_ro(const T* p)  // read-only data path
{
    if (!lf_in_bounds(p, sizeof(T))) return T{};
    return __ldg(p);
}
template <typename T>
__device__ __forceinline__ void g_store(T* p, T v)
{
    if (lf_in_bounds(p, sizeof(T))) *p = v;
}

// Element i of the sum of the devices' states, in list order (see PeerStates).
__device__ __forceinline__ float peer_sum(const PeerStates& ps, size_t i)
{
    float sum = 0.0f;
    for (int r = 0; r < ps.n; ++r) sum += g_load(ps.p[r] + i);
    return sum;
}

// ---------------------------------------------------------------------------------------------
// Global memory access with streaming hints (each byte of Q, K, V, Y is touched once)
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 ld_stream_16B(const void* p)
{
    uint4 v;
    if (!lf_in_bounds(p, 16)) return make_uint4(0u, 0u, 0u, 0u);
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ void st_stream_16B(void* p, uint4 v)
{
    if (!lf_in_bounds(p, 16)) return;
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
                 "r"(v.w)
                 : "memory");
}

__device__ __forceinline__ void st_stream_4B(void* p, uint32_t v)
{
    if (!lf_in_bounds(p, 4)) return;
    asm volatile("st.global.cs.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// ---------------------------------------------------------------------------------------------
// mbarrier + TMA (cp.async.bulk.tensor) wrappers.  Every wait is bounded.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_fence_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
                 "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t addr, uint32_t parity)
{
    uint32_t done;
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t"
        "}"
        : "=r"(done)
        : "r"(addr), "r"(parity), "r"(kBarrierSuspendHintNs)
        : "memory");
    return done != 0u;
}

// Returns true once the phase with the given parity has completed, false if the time budget
// ran out (the caller records the failure and leaves).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity)
{
    const uint32_t addr = smem_u32(bar);
    if (mbar_try_wait(addr, parity)) return true;
    const unsigned long long t0 = global_timer_ns();
    do {
        if (mbar_try_wait(addr, parity)) return true;
    } while (global_timer_ns() - t0 < kMaxBarrierWaitNs);
    return false;
}

// 4-D tiled TMA load: box at (x, y, z, w) = (channel, token, head, batch) of the tensor map ->
// shared memory, completion counted in bytes on `bar`; head-major and token-major tensors differ
// only in the strides of the tensor map.  x * element size must be a multiple of 16 bytes (the
// kernels here always pass x = 0).
__device__ __forceinline__ void tma_load_4d(void* smem_dst, const void* tmap, int x, int y, int z, int w,
                                            uint64_t* bar, uint64_t cache_policy)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%2, %3, %4, %5}], [%6], %7;" ::"r"(smem_u32(smem_dst)),
        "l"(tmap), "r"(x), "r"(y), "r"(z), "r"(w), "r"(smem_u32(bar)), "l"(cache_policy)
        : "memory");
}

__device__ __forceinline__ uint64_t policy_evict_first()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}

__device__ __forceinline__ void prefetch_tmap(const void* tmap)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(tmap) : "memory");
}

// 4-D tiled TMA store: shared memory -> the box at (x, y, z, w) of the tensor map, clipped at the
// tensor's extents (rows past N are not written).  The copy joins the executing thread's current
// bulk group, which is committed at once.  The coordinate rules of tma_load_4d apply; no
// coordinate may be negative.
__device__ __forceinline__ void tma_store_4d(const void* tmap, const void* smem_src, int x, int y, int z, int w,
                                             uint64_t cache_policy)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group.L2::cache_hint [%0, {%1, %2, %3, %4}], [%5], %6;"
        ::"l"(tmap), "r"(x), "r"(y), "r"(z), "r"(w), "r"(smem_u32(smem_src)), "l"(cache_policy)
        : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// Until the executing thread's bulk stores have read their shared-memory source / have completed.
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// Generic-proxy writes to shared memory made visible to the async proxy (TMA stores, tcgen05.mma).
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ---------------------------------------------------------------------------------------------
// Programmatic dependent launch.  A kernel launched with the programmatic-stream-serialization
// attribute may be scheduled while the kernel before it in the stream is still running, once every
// CTA of that kernel has called pdl_launch_dependents() (or has exited).  Its CTAs land on SMs as the
// earlier kernel's CTAs leave, run their set-up, and block in pdl_wait() until the earlier kernel has
// completed and its writes are visible: nothing that depends on earlier work in the stream may be
// touched before pdl_wait().  Without the attribute both calls do nothing.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---------------------------------------------------------------------------------------------
// tcgen05: tensor memory (TMEM) and the 5th-generation MMA.  A TMEM address is (lane << 16) |
// column; warp w of a CTA may touch lanes 32*(w%4) .. 32*(w%4)+31 only.
// ---------------------------------------------------------------------------------------------
// One warp allocates ncols columns (a power of two >= 32) for the CTA; the base address lands in
// *dst_smem.  The same warp frees them before the CTA exits.
__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Lane i of the warp writes r[0..31] to columns taddr.col .. +31 of TMEM lane (taddr.lane + i),
// and waits until the write has landed.
__device__ __forceinline__ void tmem_store_32cols(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};\n\t"
        "tcgen05.wait::st.sync.aligned;" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
        "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
        "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
// The reverse: 32 columns of the lane's TMEM row into registers; the wait is part of the same
// statement so that no use of r[] can be scheduled before the data has arrived.
__device__ __forceinline__ void tmem_load_32cols(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,"
        "%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_load_16cols(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ uint32_t tmem_load_1col(uint32_t taddr)
{
    uint32_t r;
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];\n\ttcgen05.wait::ld.sync.aligned;"
                 : "=r"(r)
                 : "r"(taddr)
                 : "memory");
    return r;
}

// Shared-memory matrix descriptor of a K-major bf16 operand whose rows are 128 bytes (64 values
// along K) in the 128-byte swizzle, 8-row groups 1024 bytes apart; the tile starts on a 1024-byte
// boundary.  Adding 2 to the descriptor moves the start 32 bytes = one K step of 16 values.
__device__ __forceinline__ uint64_t umma_desc_kmajor_sw128(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);  // start address, 16-byte units
    d |= static_cast<uint64_t>(1024 >> 4) << 32;              // stride between 8-row groups
    d |= static_cast<uint64_t>(1) << 46;                      // descriptor version of sm_100
    d |= static_cast<uint64_t>(2) << 61;                      // 128-byte swizzle
    return d;
}
// The same for an operand stored the other way round (MN-major): 64 values along M (or N) are one
// 128-byte row, 8 rows along K are one 1024-byte swizzle group.  `sbo` = bytes from one 8-row group
// to the next along K, `lbo` = bytes from one 64-value block to the next along M/N.  Moving the
// start by 16 rows (2048 bytes) is one K step.
__device__ __forceinline__ uint64_t umma_desc_mnmajor_sw128(uint32_t smem_addr, uint32_t lbo, uint32_t sbo)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>((lbo >> 4) & 0x3FFFu) << 16;
    d |= static_cast<uint64_t>((sbo >> 4) & 0x3FFFu) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(2) << 61;
    return d;
}
// Instruction descriptor of kind::f16 with bf16 or fp16 A and B and fp32 accumulation, M x N; the operands
// are K-major unless the flags say MN-major.
constexpr uint32_t kUmmaAMnMajor = 1u << 15;
constexpr uint32_t kUmmaBMnMajor = 1u << 16;
__host__ __device__ constexpr uint32_t umma_idesc_f32acc(int dtype, int M, int N, uint32_t major_flags = 0u)
{
    // A and B formats: 0 = fp16, 1 = bf16 (both operands always have the same type)
    return (1u << 4) /*D fp32*/ | ((dtype == kDtypeFp16 ? 0u : 1u) << 7) | ((dtype == kDtypeFp16 ? 0u : 1u) << 10) | major_flags |
           (static_cast<uint32_t>(N >> 3) << 17) | (static_cast<uint32_t>(M >> 4) << 24);
}
// D[tmem] (+)= A[tmem] * B[smem]; one thread issues it for the CTA.  A and B have the same 16-bit type.
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The same with A from shared memory as well.
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// One arrival on `bar` once every tcgen05.mma this thread has issued so far is complete.
__device__ __forceinline__ void umma_commit(uint64_t* bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

}  // namespace lf
