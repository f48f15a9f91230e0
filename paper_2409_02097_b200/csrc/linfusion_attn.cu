// Host side of the C ABI declared in include/linfusion_attn.h: descriptor validation, the
// fixed split of N, workspace layout, tensor-map encoding and kernel launches.
#include "../../include/linfusion_attn.h"

#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>

#include "split_kernels.cuh"
#include "stream_kernels.cuh"
#include "fused_kernels.cuh"
#include "producer_kernels.cuh"
#include "padded_kernels.cuh"

using namespace lf;

namespace {

// In the stream and fused kernels a ring stage is always served by the same warpgroup (stage = it % STAGES,
// group = it % GROUPS), so a group has consumed a stage's previous use before it waits for the next one and
// the parity of its mbarrier wait is unambiguous.  That needs the ring depth to be a multiple of the group
// count.  (The padded-width kernel's ring can be odd; it guards its waits with the producer's issue count.)
static_assert(StreamStateCfg::STAGES % StreamStateCfg::GROUPS == 0 && StreamApplyCfg::STAGES % StreamApplyCfg::GROUPS == 0 &&
                  FusedCfg::SLOTS % FusedCfg::GROUPS == 0 && FusedCfg::KV_STAGES % FusedCfg::GROUPS == 0,
              "a ring stage must stay with one warpgroup");

constexpr int kDefaultSmCount = 148;
using ApplyCfg = StreamApplyCfg;

enum Variant { kSplit = 1, kStream = 2, kCluster = 3, kFused = 4 };

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool supported_d(int d)
{
    return d == 32 || d == 40 || d == 64 || d == 80 || d == 128 || d == 160;
}

// Feature width d' of Q and K (Prop. 3); the descriptor's 0 means "same as d".
int dk_of(const linfusion_attn_desc_t& d) { return d.d_qk > 0 ? d.d_qk : d.d; }

// (d', d) pairs the split and cluster kernels are instantiated for: every supported square case,
// and the widened / narrowed feature widths below.
bool supported_widths(int dk, int dv)
{
    if (dk == dv) return supported_d(dv);
    return (dk == 128 && dv == 64) || (dk == 80 && dv == 40) || (dk == 32 && dv == 64);
}

// Head widths of the single-launch tcgen05 kernel for widths that are not a multiple of 64
// (padded_kernels.cuh), d' = d.
bool padded_width(int dk, int dv) { return dk == dv && (dv == 40 || dv == 80 || dv == 160); }
int padded_partial_floats(int d) { return ((d + 15) / 16 * 16) * ((d + 1 + 15) / 16 * 16); }
// Bytes of its apply operand per slab (64-channel atoms of one 128-byte row per feature).
size_t padded_image_bytes(int d) { return static_cast<size_t>(((d + 1 + 15) / 16 * 16 + 63) / 64) * ((d + 15) / 16 * 16) * 128; }

// CTAs per slab of that kernel, or 0 where it does not apply: a CTA's run of tiles must fit one
// accumulation in tensor memory (with more slabs than SMs a CTA takes whole slabs, several in turn).
// Every CTA of a slab reads all of the slab's partials (9 KB each at d = 40, 30 KB at 80, 110 KB at 160),
// so their number is kept to what makes that at most 192 KB, or a quarter of what the CTA streams of Q, K
// and V anyway (long slabs), or what the longest run demands; then the smallest count that gives the CTAs
// the same longest run is taken.
int padded_per_slab(int N, int slabs, int sm_count, int d, int* scatter = nullptr)
{
    if (scatter != nullptr) *scatter = 0;
    const int tiles = (N + 127) / 128;
    constexpr int kMaxRun = PaddedCfg<40>::MAX_TILES_PER_CTA;  // tiles a CTA may accumulate in one chain
    if (slabs > sm_count) return tiles <= kMaxRun ? 1 : 0;
    const int k_max = sm_count / slabs < tiles ? sm_count / slabs : tiles;
    int k = k_max;
    const int need = (tiles + kMaxRun - 1) / kMaxRun;  // CTAs that the longest run allows
    if (k < need) return 0;
    const long long partial_bytes = 4ll * padded_partial_floats(d), tile_bytes = 3ll * 128 * d * 2;
    while (k > need && k > 1) {
        const long long streamed = (tiles + k - 1) / k * tile_bytes;
        const long long allowed = streamed / 4 > 192 * 1024 ? streamed / 4 : 192 * 1024;
        if (k * partial_bytes <= allowed) break;
        --k;
    }
    int longest = (tiles + k - 1) / k;
    if (longest > kMaxRun) return 0;
    // Where that rule leaves runs of four tiles or more and every SM's worth of CTAs would at least halve
    // them, the CTAs of a slab share the summing instead (two exchange rounds, see the kernel): each reads
    // one partial's worth and the 16-bit operand, however many they are.  Needs a row of S per CTA.
    const int k_all = k_max < d ? k_max : d;
    const int longest_all = (tiles + k_all - 1) / k_all;
    if (longest >= 4 && 2 * longest_all <= longest) {
        if (scatter != nullptr) *scatter = 1;
        longest = longest_all;
    }
    return (tiles + longest - 1) / longest;
}

// Everything that follows from (descriptor, SM count) alone.
struct Plan {
    int variant = 0;
    int slabs = 0;
    int state_floats = 0;
    // split
    int chunks_state = 0, chunks_apply = 0;
    // stream
    int tiles_state = 0, tiles_apply = 0;  // per slab
    long long W_state = 0, W_apply = 0;
    int G_state = 0, G_apply = 0, spans = 0;
    int merged_reduce = 0;  // stream: the apply kernel sums the partials itself (two launches)
    int apply_static_runs = 0;  // stream: CTAs per slab when the apply kernel's CTAs take fixed runs of tiles
    // cluster
    int cluster_size = 0;
    // stream, fed from X (token-major handles): units are (batch, head pair, tile)
    long long W_x = 0;
    int G_x = 0, spans_x = 0;
    // fused
    int fused_split = 0, fused_whole = 0;
    int padded_per_slab = 0;  // fused, widths 40 / 80 / 160: CTAs per slab
    int padded_scatter = 0;   // ... and whether they share the summing of the partial states (two rounds)
    // workspace (bytes, offsets)
    size_t partial_bytes = 0, state_off = 0, operand_off = 0, counters_off = 0, status_off = 0, total_bytes = 0;
    int launches = 0;
};

int tile_q_of(int d) { return 16 * ((d + 15) / 16); }

linfusion_status_t validate(const linfusion_attn_desc_t* d)
{
    if (d == nullptr) return LINFUSION_ERR_INVALID_ARG;
    if (d->B <= 0 || d->H <= 0 || d->N <= 0 || d->d <= 0) return LINFUSION_ERR_INVALID_ARG;
    if (!std::isfinite(d->eps) || d->eps < 0.0f) return LINFUSION_ERR_INVALID_ARG;
    if (d->device < 0) return LINFUSION_ERR_INVALID_ARG;
    if (static_cast<long long>(d->B) * d->H > 65535) return LINFUSION_ERR_UNSUPPORTED;
    if (d->d_qk < 0) return LINFUSION_ERR_INVALID_ARG;
    if (!supported_widths(dk_of(*d), d->d)) return LINFUSION_ERR_UNSUPPORTED;
    if (d->phi != LINFUSION_PHI_ELU_PLUS_ONE && d->phi != LINFUSION_PHI_IDENTITY)
        return LINFUSION_ERR_UNSUPPORTED;
    if ((d->flags & ~(LINFUSION_VARIANT_MASK | LINFUSION_LAYOUT_TOKEN_MAJOR | LINFUSION_FLAG_UNNORMALIZED |
                      LINFUSION_DTYPE_FP16)) != 0u)
        return LINFUSION_ERR_UNSUPPORTED;
    uint32_t v = d->flags & LINFUSION_VARIANT_MASK;
    if (v > LINFUSION_VARIANT_FUSED) return LINFUSION_ERR_UNSUPPORTED;
    const bool square64 = d->d == kStreamD && dk_of(*d) == kStreamD;
    if (v == LINFUSION_VARIANT_STREAM && !square64) return LINFUSION_ERR_UNSUPPORTED;
    if (v == LINFUSION_VARIANT_FUSED && !square64 && !padded_width(dk_of(*d), d->d)) return LINFUSION_ERR_UNSUPPORTED;
    return LINFUSION_OK;
}

// Up to this many 64-token K/V tiles one CTA takes a slab alone: one launch, no partial states, the
// state goes from the MMA fragments straight into the apply operand.  Measured: 15.8 vs 22.4 us (three
// chained launches) at N = 64, d = 160 x 16 slabs and 9.8 vs 12.3 us (the persistent tcgen05 launch) at
// N = 144, d = 64 x 40 slabs; at four tiles (N = 256, d = 160) one CTA per slab is already the slower
// (35 vs 24.5 us: 16 CTAs working through their tiles one after the other).
constexpr int kLocalMaxTilesKv = 3;

int largest_cluster(int tiles_kv)
{
    if (tiles_kv <= kLocalMaxTilesKv) return 1;
    int c = kMaxClusterSize;
    while (c > 1 && c > tiles_kv) c >>= 1;
    return c;
}

linfusion_status_t make_plan(const linfusion_attn_desc_t* d, int sm_count, Plan* p)
{
    linfusion_status_t st = validate(d);
    if (st != LINFUSION_OK) return st;
    if (sm_count <= 0) sm_count = kDefaultSmCount;
    *p = Plan();
    const int slabs = d->B * d->H;
    p->slabs = slabs;
    const int dk = dk_of(*d), dv = d->d;
    const bool square64 = dk == kStreamD && dv == kStreamD;
    p->state_floats = dk * (dv + 1);
    const int tiles_kv = (d->N + 63) / 64;
    const int tiles_q = (d->N + tile_q_of(dk) - 1) / tile_q_of(dk);

    uint32_t v = d->flags & LINFUSION_VARIANT_MASK;
    if (v == LINFUSION_VARIANT_AUTO) {
        // Measured on B200 over the SD-v1.5 / v2.1 / XL layer shapes, forwards back to back.  The
        // persistent TMA + tcgen05 kernels (d = 64; two launches, the apply kernel sums the partial states
        // itself) pay a few microseconds of set-up (tensor-memory allocation, one CTA per SM working through
        // its tiles in turn) and win from about two 128-token tiles per SM on (18.8 vs 22.8 us at
        // N = 2304 x 20 slabs, 24.8 vs 30.1 us at N = 9216 x 10, 36 vs 43 us at N = 4096 x 40, 46 vs 73 us at
        // N = 16384 x 20).  Below that the three chained launches of the split path, the single persistent
        // launch (many small slabs) or one CTA per slab (N <= 192) are faster.
        const long long stream_tiles = static_cast<long long>(slabs) * ((d->N + StreamStateCfg::TILE - 1) / StreamStateCfg::TILE);
        // The single persistent launch wins where no state has to cross CTAs: slabs of at most eight
        // 128-token tiles, enough of them to occupy a quarter of the SMs, each handled whole by one
        // CTA (10.9 vs 12.9 us at N = 144 x 40 slabs, 15.2 vs 18.6 us at N = 576 x 40).  Where slabs
        // are shared between CTAs its exchange through global memory costs more than two kernel
        // boundaries (32 vs 22 us at N = 2304 x 20, 106 vs 47 us at N = 16384 x 20), so it is not
        // chosen there.
        const int fused_tiles = (d->N + FusedCfg::TILE - 1) / FusedCfg::TILE;
        // Widths 40 / 80 / 160 (the SD-v1.5 levels): the single TMA + tcgen05 launch wherever its limits allow
        // (19.4 vs 20.8 us for three chained launches at N = 4096, d = 40 x 16 slabs; 16.6 vs 17.4 us at
        // N = 1024, d = 80; 19.4 vs 24.6 us at N = 256, d = 160; 13.5 vs 14.7 us for one CTA per slab of the
        // warp-level kernel at N = 64, d = 160).
        // Not where it would leave most of the machine idle on runs of more than three tiles (few CTAs per slab
        // because the partial states are large and sharing their summing does not pay: padded_per_slab()).
        const int pk = padded_width(dk, dv) ? padded_per_slab(d->N, slabs, sm_count, dv) : 0;
        const int padded_ctas = slabs > sm_count ? sm_count : slabs * pk;
        const int padded_run = pk > 0 ? (fused_tiles + pk - 1) / pk : 0;
        if (pk > 0 && (2 * padded_ctas >= sm_count || padded_run <= 3))
            v = LINFUSION_VARIANT_FUSED;
        else if (tiles_kv <= kLocalMaxTilesKv)
            v = LINFUSION_VARIANT_CLUSTER;  // resolves to one CTA per slab (largest_cluster())
        else if (square64 && stream_tiles >= 2ll * sm_count)
            v = LINFUSION_VARIANT_STREAM;
        else if (square64 && fused_tiles <= 8 && 4 * slabs >= sm_count && stream_tiles < 4ll * sm_count)
            v = LINFUSION_VARIANT_FUSED;
        else
            v = LINFUSION_VARIANT_SPLIT;
    }
    p->variant = static_cast<int>(v);

    size_t partial_floats = 0;
    if (v == LINFUSION_VARIANT_SPLIT) {
        int cs = (2 * sm_count + slabs - 1) / slabs;
        p->chunks_state = cs < 1 ? 1 : (cs > tiles_kv ? tiles_kv : cs);
        int ca = (4 * sm_count + slabs - 1) / slabs;
        p->chunks_apply = ca < 1 ? 1 : (ca > tiles_q ? tiles_q : ca);
        partial_floats = static_cast<size_t>(slabs) * p->chunks_state * p->state_floats;
        p->launches = 3;
    } else if (v == LINFUSION_VARIANT_STREAM) {
        p->tiles_state = (d->N + StreamStateCfg::TILE - 1) / StreamStateCfg::TILE;
        p->tiles_apply = (d->N + ApplyCfg::TILE - 1) / ApplyCfg::TILE;
        p->W_state = static_cast<long long>(slabs) * p->tiles_state;
        p->W_apply = static_cast<long long>(slabs) * p->tiles_apply;
        long long gs = static_cast<long long>(sm_count) * StreamStateCfg::CTAS_PER_SM;
        long long ga = sm_count;
        // The same number of CTAs on every slab, where that keeps at least four fifths of the SMs busy:
        // (1) token-major: the 128-byte rows of all heads of a token are adjacent in memory, and with equal
        // counts the CTAs of different heads walk through the same tokens at the same time, so DRAM pages
        // are used while they are open: 140 CTAs (7 per slab) beat 148 by 7-8 % at 20 slabs, and 120 (3 per
        // slab) equal 148 at 40; (2) either layout when a CTA's share is only a few dozen tiles: with 7 CTAs
        // on some slabs and 8 on others the kernels end with a tail that the tile hand-out cannot level
        // (41.8 vs 46.3 us at N = 16384 x 20 slabs, 31.0 vs 36.3 us at N = 4096 x 40).
        if ((d->flags & LINFUSION_LAYOUT_TOKEN_MAJOR) != 0u || p->W_state < 64ll * sm_count) {
            const long long aligned = (static_cast<long long>(sm_count) / slabs) * slabs;
            if (aligned * 5 >= static_cast<long long>(sm_count) * 4) gs = ga = aligned;
        }
        p->G_state = static_cast<int>(gs < p->W_state ? gs : p->W_state);
        p->G_apply = static_cast<int>(ga < p->W_apply ? ga : p->W_apply);
        int spans = 1;
        for (int g = 0; g < p->G_state; ++g) {
            long long b = unit_begin(g, p->W_state, p->G_state);
            long long e = unit_begin(g + 1, p->W_state, p->G_state);
            if (e > b) {
                int s = static_cast<int>((e - 1) / p->tiles_state - b / p->tiles_state) + 1;
                if (s > spans) spans = s;
            }
        }
        p->spans = spans;
        partial_floats = static_cast<size_t>(p->G_state) * spans * kStreamStateFloats;
        if ((d->flags & LINFUSION_LAYOUT_TOKEN_MAJOR) != 0u) {
            // The state from X (state_x): two heads per unit, the same number of CTAs on every (batch, head
            // pair) where that keeps at least four fifths of the SMs busy (the CTAs of a token's head pairs
            // then walk through X in step and share its tiles in L2); two partials per visit.
            const long long groups = static_cast<long long>(d->B) * head_pairs(d->H);
            p->W_x = groups * p->tiles_state;
            long long gx = sm_count;
            const long long aligned_x = (gx / groups) * groups;
            if (aligned_x * 5 >= gx * 4) gx = aligned_x;
            if (gx > p->W_x) gx = p->W_x;
            p->G_x = static_cast<int>(gx);
            int sx = 1;
            for (int g = 0; g < p->G_x; ++g) {
                long long b = unit_begin(g, p->W_x, p->G_x), e = unit_begin(g + 1, p->W_x, p->G_x);
                if (e > b) {
                    int n = static_cast<int>((e - 1) / p->tiles_state - b / p->tiles_state) + 1;
                    if (n > sx) sx = n;
                }
            }
            p->spans_x = sx;
            const size_t need = static_cast<size_t>(p->G_x) * sx * 2 * kStreamStateFloats;
            if (need > partial_floats) partial_floats = need;
        }
        // Every slab needs an apply CTA that starts on it for the apply kernel to take over the second
        // stage of the reduction (see MergedReduce); otherwise the reduction keeps its own kernel.
        p->merged_reduce = slabs <= p->G_apply ? 1 : 0;
        // Fixed runs of tiles in the apply kernel where every slab has the same number of CTAs and a CTA's
        // share is a few dozen tiles (measured: the hand-out through counters ends such kernels with a tail
        // of 7 us at N = 4096 x 40 slabs and N = 16384 x 20 slabs — CTAs that got fewer tiles than their
        // neighbours move to other slabs for a tile or two and drain their ring for each new operand).
        if (p->G_apply % slabs == 0 && p->G_apply / slabs <= p->tiles_apply &&
            p->tiles_apply <= 64ll * (p->G_apply / slabs))
            p->apply_static_runs = p->G_apply / slabs;
        p->launches = p->merged_reduce != 0 ? 2 : 3;
    } else if (v == LINFUSION_VARIANT_FUSED && !square64) {
        // One persistent launch, widths 40 / 80 / 160: per_slab CTAs on every slab, one partial each.
        p->padded_per_slab = padded_per_slab(d->N, slabs, sm_count, dv, &p->padded_scatter);
        if (p->padded_per_slab == 0) return LINFUSION_ERR_UNSUPPORTED;
        p->tiles_state = p->tiles_apply = (d->N + 127) / 128;
        p->G_state = p->G_apply = slabs > sm_count ? sm_count : slabs * p->padded_per_slab;
        partial_floats = p->padded_per_slab > 1 ? static_cast<size_t>(p->G_state) * padded_partial_floats(dv) : 0;
        p->launches = 1;
    } else if (v == LINFUSION_VARIANT_FUSED) {
        // One persistent launch.  Two waves of slabs once every CTA has a couple of tiles in each
        // (the exchange of one wave's states then hides behind the other wave's streaming); at
        // most 32 CTAs per slab (the reducer warp keeps one contributor per lane).
        const int tiles = (d->N + FusedCfg::TILE - 1) / FusedCfg::TILE;
        p->tiles_state = p->tiles_apply = tiles;
        p->W_state = p->W_apply = static_cast<long long>(slabs) * tiles;
        const bool two = slabs >= 2 && p->W_state >= 4ll * sm_count;
        p->fused_split = two ? (slabs + 1) / 2 : slabs;
        // Small slabs are dealt whole, one CTA per slab or more slabs per CTA: nothing is exchanged.
        p->fused_whole = (!two && tiles <= 8 && 4 * slabs >= sm_count) ? 1 : 0;
        const FusedPlan fp = {tiles, slabs, p->fused_split, p->fused_whole};
        long long G = sm_count;
        if (p->fused_whole != 0) {
            if (G > slabs) G = slabs;
        } else {
            if (G > fused_wave_units(fp, 0)) G = fused_wave_units(fp, 0);
            const long long min_wave_slabs = two ? slabs - p->fused_split : slabs;
            if (G > 30 * min_wave_slabs) G = 30 * min_wave_slabs;
        }
        p->G_state = p->G_apply = static_cast<int>(G);
        int spans = 1;
        for (int g = 0; g < p->G_state; ++g) {
            int touched = 0;
            for (int w = 0; w < fused_waves(fp); ++w) {
                long long b, e;
                fused_run(fp, g, G, w, &b, &e);
                touched += fused_run_slabs(b, e, tiles);
            }
            if (touched > spans) spans = touched;
        }
        p->spans = spans;
        partial_floats = static_cast<size_t>(p->G_state) * spans * kStreamStateFloats;
        p->launches = 1;
    } else {
        p->cluster_size = largest_cluster(tiles_kv);
        partial_floats = 0;
        p->launches = 1;
    }
    p->partial_bytes = align_up(partial_floats * sizeof(float), 256);
    p->state_off = p->partial_bytes;
    p->operand_off = p->state_off + align_up(static_cast<size_t>(slabs) * p->state_floats * sizeof(float), 256);
    // 16-bit operand image of S | z for the apply kernel (in its shared-memory layout), and for the
    // stream variant one tile counter per slab.
    const int dkp = (dk + 15) / 16 * 16;
    const size_t split_image = static_cast<size_t>((dv + 8 + 15) / 16 * 16) * (((dkp / 8) | 1) * 16);
    const size_t frag_bytes = v == LINFUSION_VARIANT_STREAM  ? static_cast<size_t>(slabs) * kStreamOperandBytes
                              : v == LINFUSION_VARIANT_SPLIT ? static_cast<size_t>(slabs) * split_image
                              : p->padded_scatter != 0       ? static_cast<size_t>(slabs) * padded_image_bytes(dv)
                                                             : 0;
    // Stream: one tile counter and one ready flag per slab.  Fused: two arrival counters per slab, then the control words.
    const size_t counter_bytes = v == LINFUSION_VARIANT_STREAM  ? align_up(static_cast<size_t>(slabs) * 8, 256)
                                 : v == LINFUSION_VARIANT_FUSED ? align_up(static_cast<size_t>(slabs) * 8, 256) + 256
                                                                : 0;
    p->counters_off = p->operand_off + align_up(frag_bytes, 256);
    p->status_off = p->counters_off + counter_bytes;
    p->total_bytes = p->status_off + 256;
    return LINFUSION_OK;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// KIND the kernels are instantiated on: phi and the 16-bit storage type.
int kind_of(const linfusion_attn_desc_t& d)
{
    return make_kind(d.phi == LINFUSION_PHI_IDENTITY ? kPhiIdentity : kPhiEluPlusOne,
                     (d.flags & LINFUSION_DTYPE_FP16) != 0u ? kDtypeFp16 : kDtypeBf16);
}
int dtype_of(const linfusion_attn_desc_t& d) { return kind_dtype(kind_of(d)); }

// Power of two that S | z are multiplied by when they become the apply kernel's MMA operand.  bf16
// has fp32's range: 1.  fp16 tops out at 65504 and z ~ N, so 2^-ceil(log2 N): z stays below ~8,
// S at its natural 1/sqrt(N) relative size.  The scale cancels in the quotient of Eq. 5.
float operand_scale(const linfusion_attn_desc_t& d)
{
    if (dtype_of(d) != kDtypeFp16) return 1.0f;
    int k = 0;
    while ((1ll << k) < d.N) ++k;
    return std::ldexp(1.0f, -k);
}

// What the apply kernels take besides the tensors: a negative eps selects the operator without
// its normalizer (whose result must have the operand scale taken out again).
ApplyScales apply_scales(const linfusion_attn_desc_t& d)
{
    ApplyScales sc;
    sc.operand = operand_scale(d);
    sc.unnormalized = 1.0f / sc.operand;
    sc.eps = (d.flags & LINFUSION_FLAG_UNNORMALIZED) != 0u ? kEpsUnnormalized : d.eps * sc.operand;
    return sc;
}

#define LF_DISPATCH_KIND(kval, CALL) \
    switch (kval) {                  \
        case 0: CALL(0); break;      \
        case 1: CALL(1); break;      \
        case 2: CALL(2); break;      \
        case 3: CALL(3); break;      \
        default: break;              \
    }

// Element strides of a slab's rows, `width` channels each, for the layout the descriptor asks for.
SlabLayout layout_of(const linfusion_attn_desc_t& d, int width)
{
    SlabLayout L;
    L.H = d.H;
    if ((d.flags & LINFUSION_LAYOUT_TOKEN_MAJOR) != 0u) {  // [B, N, H, width]
        L.batch_stride = static_cast<long long>(d.N) * d.H * width;
        L.head_stride = width;
        L.row_stride = d.H * width;
    } else {  // [B, H, N, width]
        L.batch_stride = static_cast<long long>(d.H) * d.N * width;
        L.head_stride = static_cast<long long>(d.N) * width;
        L.row_stride = width;
    }
    return L;
}
SlabLayout layout_qk(const linfusion_attn_desc_t& d) { return layout_of(d, dk_of(d)); }  // Q and K
SlabLayout layout_vy(const linfusion_attn_desc_t& d) { return layout_of(d, d.d); }       // V and Y
// Bytes of Q (or K), and of V (or Y).
size_t bytes_qk(const linfusion_attn_desc_t& d) { return static_cast<size_t>(d.B) * d.H * d.N * dk_of(d) * 2; }
size_t bytes_vy(const linfusion_attn_desc_t& d) { return static_cast<size_t>(d.B) * d.H * d.N * d.d * 2; }

// 16-bit (bf16 or fp16) tensor seen as (channel 64, token N, head H, batch B) -> boxes of tile_rows tokens of one
// (b, h) slab, 128-byte swizzle, zero fill past N.  The layout only changes the strides.
bool encode_slab_map(CUtensorMap* map, const void* base, const linfusion_attn_desc_t& d, int tile_rows)
{
    EncodeTiledFn fn = get_encode_fn();
    if (fn == nullptr) return false;
    const SlabLayout L = layout_vy(d);  // these kernels have d' = d = 64
    cuuint64_t dims[4] = {static_cast<cuuint64_t>(kStreamD), static_cast<cuuint64_t>(d.N),
                          static_cast<cuuint64_t>(d.H), static_cast<cuuint64_t>(d.B)};
    cuuint64_t strides[3] = {static_cast<cuuint64_t>(L.row_stride) * 2, static_cast<cuuint64_t>(L.head_stride) * 2,
                             static_cast<cuuint64_t>(L.batch_stride) * 2};
    cuuint32_t box[4] = {static_cast<cuuint32_t>(kStreamD), static_cast<cuuint32_t>(tile_rows), 1u, 1u};
    cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    // Head-major rows of a slab are contiguous: let L2 fetch 256 bytes per miss.  Token-major rows
    // are 128-byte segments between other heads' data: fetch only what this CTA will use.
    const CUtensorMapL2promotion promo = (d.flags & LINFUSION_LAYOUT_TOKEN_MAJOR) != 0u
                                             ? CU_TENSOR_MAP_L2_PROMOTION_L2_128B
                                             : CU_TENSOR_MAP_L2_PROMOTION_L2_256B;
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box,
                    estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    promo, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// The same view for the widths 40 / 80 / 160: the channel extent is d, the box is 64 channels wide, so
// the part of a box past channel d lies outside the tensor (zeros on loads, not written by stores).
bool encode_padded_map(CUtensorMap* map, const void* base, const linfusion_attn_desc_t& d)
{
    EncodeTiledFn fn = get_encode_fn();
    if (fn == nullptr) return false;
    const SlabLayout L = layout_vy(d);  // d' = d
    cuuint64_t dims[4] = {static_cast<cuuint64_t>(d.d), static_cast<cuuint64_t>(d.N), static_cast<cuuint64_t>(d.H),
                          static_cast<cuuint64_t>(d.B)};
    cuuint64_t strides[3] = {static_cast<cuuint64_t>(L.row_stride) * 2, static_cast<cuuint64_t>(L.head_stride) * 2,
                             static_cast<cuuint64_t>(L.batch_stride) * 2};
    cuuint32_t box[4] = {64u, 128u, 1u, 1u};
    cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

}  // namespace

struct linfusion_attn {
    linfusion_attn_desc_t desc;
    Plan plan;
    int sm_count;
    void* ws;  // device workspace in use
    size_t ws_bytes;
    bool owns_ws;
    float* partials;
    float* state;
    unsigned char* operand;  // 16-bit operand image of S | z for the apply kernels
    int* tile_counters;
    uint32_t* status;
    cudaStream_t last_stream;
    void* stage[4];  // staging for the host-buffer entry point (allocated on first use)
    // Optional per-kernel timing: `timing_slots` sets of 4 events, used round-robin by forward().
    cudaEvent_t* events;
    int timing_slots;
    long long timed_calls;
    int timing_stride;        // every timing_stride-th forward is bracketed with events
    long long forward_calls;  // forwards since timing was enabled
    bool sample_now;          // the forward being enqueued is one of them
    struct HostPipe* pipe;  // copy/compute pipeline of the host-buffer entry point (first use)
    // forward_x(): row statistics of the non-linear branches' LayerNorm and the branches' outputs
    // T_q, T_k (allocated on first use)
    float* x_stats;
    void* x_t[2];
};

// forward_host() cuts the slabs into groups and overlaps the upload of group i+1, the kernels of
// group i and the download of group i-1 on three streams.
constexpr int kMaxHostGroups = 20;
struct HostPipe {
    int groups = 1;
    linfusion_attn* sub = nullptr;  // handle for one group of slabs (null when groups == 1)
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    cudaEvent_t entry = nullptr, out = nullptr;
    cudaEvent_t in[kMaxHostGroups] = {}, done[kMaxHostGroups] = {};
};

namespace {

void bind_workspace(linfusion_attn* h, void* ws)
{
    h->ws = ws;
    h->ws_bytes = h->plan.total_bytes;
    unsigned char* base = static_cast<unsigned char*>(ws);
    h->partials = reinterpret_cast<float*>(base);
    h->state = reinterpret_cast<float*>(base + h->plan.state_off);
    h->operand = base + h->plan.operand_off;
    h->tile_counters = reinterpret_cast<int*>(base + h->plan.counters_off);
    h->status = reinterpret_cast<uint32_t*>(base + h->plan.status_off);
}

// Zero the operand image, the tile counters and the status word, and return only when that is done:
// a forward enqueued right afterwards on any stream (non-blocking side streams included, which the
// legacy default stream does not order against) must find them cleared and must not be overtaken
// by the clear.
bool clear_workspace_tail(linfusion_attn* h)
{
    if (cudaMemsetAsync(h->operand, 0, h->plan.total_bytes - h->plan.operand_off, nullptr) != cudaSuccess ||
        cudaStreamSynchronize(nullptr) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return true;
}

struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || (cudaSetDevice(dev) == cudaSuccess);
    }
    ~DeviceGuard()
    {
        if (ok && prev >= 0) cudaSetDevice(prev);
    }
};

// Record timing event `i` (0..3) of the current forward, when kernel timing is enabled.
inline void mark(const linfusion_attn* h, int i, cudaStream_t s)
{
    if (h->sample_now)
        cudaEventRecord(h->events[(h->timed_calls % h->timing_slots) * 4 + i], s);
}

template <int DK, int DV, int KIND>
cudaError_t set_split_attrs()
{
    using C = SplitCfg<DK, DV>;
    cudaError_t e;
    e = cudaFuncSetAttribute(state_partial_kernel<DK, DV, KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_KV);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(apply_kernel<DK, DV, KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_APPLY);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(cluster_fused_kernel<DK, DV, KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             C::SMEM_CLUSTER);
    if (e != cudaSuccess) return e;
    // Clusters of 16 CTAs are beyond the portable size of 8; create() shrinks the cluster when
    // the device cannot co-schedule it.
    e = cudaFuncSetAttribute(cluster_fused_kernel<DK, DV, KIND>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    return e;
}

template <int KIND>
cudaError_t set_stream_attrs()
{
    cudaError_t e;
    e = cudaFuncSetAttribute(stream_state_kernel<KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             StreamStateCfg::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(stream_apply_kernel<KIND>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, ApplyCfg::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(stream_fused_kernel<KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             FusedCfg::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(producer_apply_kernel<KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             ProdApplyCfg::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(producer_state2_kernel<KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             ProdState2Cfg::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(producer_hidden_kernel<KIND>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             ProdHiddenCfg::SMEM_BYTES);
    return e;
}

// Launch with the programmatic-stream-serialization attribute (see pdl_wait() in common.cuh): the
// kernel's CTAs may be placed, and run their set-up, while the kernel before it drains.
template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                           Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Checked build: tell the kernels, in stream order, which byte ranges this call may touch (Q and K,
// V and Y, the workspace, and for the peer-summed apply the devices' state buffers).  One table per
// device: checked calls on different streams must not overlap.  Nothing in the normal build.
#ifdef LF_CHECKED
// Self-test of the check: the registered Y range is cut short by this many bytes, so that the (valid)
// stores to the end of Y are reported and skipped.
std::atomic<size_t> g_checked_shrink_y{0};
#endif

void register_checked_ranges(const linfusion_attn* h, const void* q, const void* k, const void* v, const void* y,
                             cudaStream_t s, const PeerStates* peers = nullptr)
{
#ifdef LF_CHECKED
    CheckedRanges r;
    r.n = 0;
    auto add = [&](const void* p, size_t bytes) {
        if (p == nullptr || r.n >= kCheckedMaxRanges) return;
        r.lo[r.n] = reinterpret_cast<unsigned long long>(p);
        r.hi[r.n] = r.lo[r.n] + bytes;
        ++r.n;
    };
    add(q, bytes_qk(h->desc));
    add(k, bytes_qk(h->desc));
    add(v, bytes_vy(h->desc));
    const size_t shrink = g_checked_shrink_y.load();
    add(y, bytes_vy(h->desc) > shrink ? bytes_vy(h->desc) - shrink : 0);
    add(h->ws, h->ws_bytes);
    if (peers != nullptr)
        for (int i = 0; i < peers->n; ++i) add(peers->p[i], static_cast<size_t>(h->plan.slabs) * h->plan.state_floats * 4);
    cudaMemcpyToSymbolAsync(g_checked_ranges, &r, sizeof(r), 0, cudaMemcpyHostToDevice, s);
#else
    (void)h; (void)q; (void)k; (void)v; (void)y; (void)s; (void)peers;
#endif
}

template <int DK, int DV, int KIND>
cudaError_t launch_split(const linfusion_attn* h, const __nv_bfloat16* q, const __nv_bfloat16* k,
                         const __nv_bfloat16* v, __nv_bfloat16* y, cudaStream_t s)
{
    register_checked_ranges(h, q, k, v, y, s);
    using C = SplitCfg<DK, DV>;
    const Plan& p = h->plan;
    const int N = h->desc.N;
    cudaError_t e;
    mark(h, 0, s);
    e = launch_chained(state_partial_kernel<DK, DV, KIND>, dim3(p.chunks_state, p.slabs), dim3(C::NT), C::SMEM_KV, s, k, v,
                       h->partials, N, p.chunks_state, layout_qk(h->desc), layout_vy(h->desc));
    if (e != cudaSuccess) return e;
    mark(h, 1, s);
    // h->operand (when the workspace has it) receives the apply kernel's 16-bit operand image.
    unsigned char* image = h->operand;
    e = launch_chained(state_reduce_kernel, dim3((C::STATE_FLOATS + 255) / 256, p.slabs), dim3(256), 0, s,
                       h->partials, h->state, C::STATE_FLOATS, p.chunks_state, image, DK, DV, C::PITCHK, C::SMEM_ST,
                       dtype_of(h->desc), operand_scale(h->desc));
    if (e != cudaSuccess) return e;
    mark(h, 2, s);
    e = launch_chained(apply_kernel<DK, DV, KIND>, dim3(p.chunks_apply, p.slabs), dim3(C::NT), C::SMEM_APPLY, s, q,
                       h->state, y, N, p.chunks_apply, apply_scales(h->desc), layout_qk(h->desc), layout_vy(h->desc), image);
    if (e != cudaSuccess) return e;
    mark(h, 3, s);
    return cudaGetLastError();
}

template <int DK, int DV>
void cluster_config(cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr, int cluster_size, int slabs,
                    cudaStream_t s)
{
    using C = SplitCfg<DK, DV>;
    *cfg = cudaLaunchConfig_t{};
    cfg->gridDim = dim3(cluster_size, slabs, 1);
    cfg->blockDim = dim3(C::NT, 1, 1);
    cfg->dynamicSmemBytes = C::SMEM_CLUSTER;
    cfg->stream = s;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster_size;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg->attrs = attr;
    cfg->numAttrs = 1;
}

template <int DK, int DV, int KIND>
cudaError_t launch_cluster(const linfusion_attn* h, const __nv_bfloat16* q, const __nv_bfloat16* k,
                           const __nv_bfloat16* v, __nv_bfloat16* y, cudaStream_t s)
{
    register_checked_ranges(h, q, k, v, y, s);
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    cluster_config<DK, DV>(&cfg, attr, h->plan.cluster_size, h->plan.slabs, s);
    mark(h, 0, s);
    cudaError_t e;
    if (h->plan.cluster_size == 1)  // one CTA per slab: a plain launch, chained to its neighbours in the stream
        e = launch_chained(cluster_fused_kernel<DK, DV, KIND>, cfg.gridDim, cfg.blockDim, cfg.dynamicSmemBytes, s, q, k,
                           v, y, h->state, h->desc.N, apply_scales(h->desc), layout_qk(h->desc), layout_vy(h->desc));
    else
        e = cudaLaunchKernelEx(&cfg, cluster_fused_kernel<DK, DV, KIND>, q, k, v, y, h->state, h->desc.N,
                               apply_scales(h->desc), layout_qk(h->desc), layout_vy(h->desc));
    mark(h, 1, s);
    return e;
}

template <int KIND>
cudaError_t launch_stream(const linfusion_attn* h, const __nv_bfloat16* q, const __nv_bfloat16* k,
                          const __nv_bfloat16* v, __nv_bfloat16* y, cudaStream_t s)
{
    const Plan& p = h->plan;
    const int N = h->desc.N;
    CUtensorMap mq, mk, mv, my;
    if (!encode_slab_map(&mk, k, h->desc, StreamStateCfg::TILE) ||
        !encode_slab_map(&mv, v, h->desc, StreamStateCfg::TILE) ||
        !encode_slab_map(&mq, q, h->desc, ApplyCfg::TILE) || !encode_slab_map(&my, y, h->desc, ApplyCfg::TILE))
        return cudaErrorInvalidValue;
    cudaError_t e;
    MergedReduce mr = {};
    uint32_t* per_slab_words = reinterpret_cast<uint32_t*>(h->tile_counters);  // tile counters, then ready flags
    if (p.merged_reduce != 0) {
        mr.partials = h->partials;
        mr.state = h->state;
        mr.operand = h->operand;
        mr.ready = per_slab_words + p.slabs;
        mr.W = p.W_state;
        mr.G = p.G_state;
        mr.spans = p.spans;
        mr.tiles_per_slab = p.tiles_state;
        mr.dtype = dtype_of(h->desc);
        mr.scale = operand_scale(h->desc);
        mr.enabled = 1;
    }
    mark(h, 0, s);
    e = launch_chained(stream_state_kernel<KIND>, dim3(p.G_state), dim3(StreamStateCfg::THREADS),
                       StreamStateCfg::SMEM_BYTES, s, mk, mv, h->partials, h->status, N, p.tiles_state, p.W_state,
                       p.spans, h->desc.H, p.merged_reduce != 0 ? per_slab_words : nullptr,
                       p.merged_reduce != 0 ? 2 * p.slabs : 0);
    if (e != cudaSuccess) return e;
    mark(h, 1, s);
    if (p.merged_reduce == 0) {
        e = launch_chained(stream_reduce_kernel, dim3((kStreamStateFloats + 255) / 256, p.slabs), dim3(256), 0, s,
                           h->partials, h->state, h->operand, h->tile_counters, p.tiles_state, p.W_state, p.G_state,
                           p.spans, dtype_of(h->desc), operand_scale(h->desc));
        if (e != cudaSuccess) return e;
        mark(h, 2, s);
    }
    e = launch_chained(stream_apply_kernel<KIND>, dim3(p.G_apply), dim3(ApplyCfg::THREADS), ApplyCfg::SMEM_BYTES, s,
                       mq, my, h->operand, h->tile_counters, h->status, p.tiles_apply, p.slabs,
                       apply_scales(h->desc), h->desc.H, mr, p.apply_static_runs);
    if (e != cudaSuccess) return e;
    mark(h, p.merged_reduce != 0 ? 2 : 3, s);
    return cudaGetLastError();
}

template <int KIND>
cudaError_t launch_fused(const linfusion_attn* h, const __nv_bfloat16* q, const __nv_bfloat16* k,
                         const __nv_bfloat16* v, __nv_bfloat16* y, cudaStream_t s)
{
    const Plan& p = h->plan;
    CUtensorMap mq, mk, mv, my;
    if (!encode_slab_map(&mk, k, h->desc, FusedCfg::TILE) || !encode_slab_map(&mv, v, h->desc, FusedCfg::TILE) ||
        !encode_slab_map(&mq, q, h->desc, FusedCfg::TILE) || !encode_slab_map(&my, y, h->desc, FusedCfg::TILE))
        return cudaErrorInvalidValue;
    uint32_t* arrive = reinterpret_cast<uint32_t*>(h->tile_counters);
    uint32_t* ctrl = arrive + align_up(static_cast<size_t>(p.slabs) * 8, 256) / 4;
    const FusedPlan fp = {p.tiles_state, p.slabs, p.fused_split, p.fused_whole};
    mark(h, 0, s);
    cudaError_t e = launch_chained(stream_fused_kernel<KIND>, dim3(p.G_state), dim3(FusedCfg::THREADS),
                                   FusedCfg::SMEM_BYTES, s, mk, mv, mq, my, h->partials, h->state, arrive, ctrl,
                                   h->status, h->desc.N, fp, p.spans, h->desc.H, apply_scales(h->desc));
    if (e != cudaSuccess) return e;
    mark(h, 1, s);
    return cudaGetLastError();
}

template <int D, int KIND>
cudaError_t launch_padded(const linfusion_attn* h, const __nv_bfloat16* q, const __nv_bfloat16* k,
                          const __nv_bfloat16* v, __nv_bfloat16* y, cudaStream_t s)
{
    using C = PaddedCfg<D>;
    const Plan& p = h->plan;
    CUtensorMap mq, mk, mv, my;
    if (!encode_padded_map(&mk, k, h->desc) || !encode_padded_map(&mv, v, h->desc) ||
        !encode_padded_map(&mq, q, h->desc) || !encode_padded_map(&my, y, h->desc))
        return cudaErrorInvalidValue;
    uint32_t* counters = reinterpret_cast<uint32_t*>(h->tile_counters);
    uint32_t* ctrl = counters + align_up(static_cast<size_t>(p.slabs) * 8, 256) / 4;
    mark(h, 0, s);
    cudaError_t e =
        p.padded_scatter != 0
            ? launch_chained(padded_fused_kernel<D, KIND, 1>, dim3(p.G_state), dim3(C::THREADS), C::SMEM_BYTES, s, mk, mv, mq,
                             my, h->partials, h->state, h->operand, counters, ctrl, h->status, h->desc.N, p.tiles_state,
                             p.padded_per_slab, p.slabs, h->desc.H, apply_scales(h->desc))
            : launch_chained(padded_fused_kernel<D, KIND, 0>, dim3(p.G_state), dim3(C::THREADS), C::SMEM_BYTES, s, mk, mv, mq,
                             my, h->partials, h->state, h->operand, counters, ctrl, h->status, h->desc.N, p.tiles_state,
                             p.padded_per_slab, p.slabs, h->desc.H, apply_scales(h->desc));
    if (e != cudaSuccess) return e;
    mark(h, 1, s);
    return cudaGetLastError();
}

template <int D>
cudaError_t launch_padded_d(const linfusion_attn* h, const __nv_bfloat16* q, const __nv_bfloat16* k,
                            const __nv_bfloat16* v, __nv_bfloat16* y, cudaStream_t s)
{
    cudaError_t e = cudaErrorInvalidValue;
#define LF_K(KV) e = launch_padded<D, KV>(h, q, k, v, y, s)
    LF_DISPATCH_KIND(kind_of(h->desc), LF_K)
#undef LF_K
    return e;
}

template <int DK, int DV>
cudaError_t set_attrs_d(int kind)
{
    cudaError_t e = cudaErrorInvalidValue;
#define LF_K(KV) e = set_split_attrs<DK, DV, KV>()
    LF_DISPATCH_KIND(kind, LF_K)
#undef LF_K
    if constexpr (DK == DV && (DV == 40 || DV == 80 || DV == 160)) {
        if (e != cudaSuccess) return e;
#define LF_K(KV) \
    e = cudaFuncSetAttribute(padded_fused_kernel<DV, KV, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, PaddedCfg<DV>::SMEM_BYTES)
        LF_DISPATCH_KIND(kind, LF_K)
#undef LF_K
        if (e != cudaSuccess) return e;
#define LF_K(KV) \
    e = cudaFuncSetAttribute(padded_fused_kernel<DV, KV, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, PaddedCfg<DV>::SMEM_BYTES)
        LF_DISPATCH_KIND(kind, LF_K)
#undef LF_K
    }
    return e;
}

template <int DK, int DV>
cudaError_t launch_d(const linfusion_attn* h, const __nv_bfloat16* q, const __nv_bfloat16* k,
                     const __nv_bfloat16* v, __nv_bfloat16* y, cudaStream_t s)
{
    cudaError_t e = cudaErrorInvalidValue;
    if (h->plan.variant == kCluster) {
#define LF_K(KV) e = launch_cluster<DK, DV, KV>(h, q, k, v, y, s)
        LF_DISPATCH_KIND(kind_of(h->desc), LF_K)
#undef LF_K
    } else {
#define LF_K(KV) e = launch_split<DK, DV, KV>(h, q, k, v, y, s)
        LF_DISPATCH_KIND(kind_of(h->desc), LF_K)
#undef LF_K
    }
    return e;
}

// CALL(DK, DV) for the descriptor's pair of widths (supported_widths() lists the same pairs).
#define LF_DISPATCH_D(desc, CALL)               \
    switch (dk_of(desc) * 1000 + (desc).d) {    \
        case 32032: CALL(32, 32); break;        \
        case 40040: CALL(40, 40); break;        \
        case 64064: CALL(64, 64); break;        \
        case 80080: CALL(80, 80); break;        \
        case 128128: CALL(128, 128); break;     \
        case 160160: CALL(160, 160); break;     \
        case 128064: CALL(128, 64); break;      \
        case 80040: CALL(80, 40); break;        \
        case 32064: CALL(32, 64); break;        \
        default: break;                         \
    }

template <int DK, int DV>
bool cluster_fits(int kind, int cluster_size, int slabs)
{
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    cluster_config<DK, DV>(&cfg, attr, cluster_size, slabs, nullptr);
    int n = 0;
    cudaError_t e = cudaErrorInvalidValue;
#define LF_K(KV) e = cudaOccupancyMaxActiveClusters(&n, cluster_fused_kernel<DK, DV, KV>, &cfg)
    LF_DISPATCH_KIND(kind, LF_K)
#undef LF_K
    if (e != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return n > 0;
}

}  // namespace

extern "C" {

const char* linfusion_status_string(linfusion_status_t s)
{
    switch (s) {
        case LINFUSION_OK: return "ok";
        case LINFUSION_ERR_INVALID_ARG: return "invalid argument";
        case LINFUSION_ERR_UNSUPPORTED: return "unsupported head dim, activation, variant or device";
        case LINFUSION_ERR_ALLOC: return "workspace allocation failed or workspace too small";
        case LINFUSION_ERR_CUDA: return "CUDA call failed";
        case LINFUSION_ERR_TIMEOUT: return "a bounded device-side wait expired";
        default: return "unknown status";
    }
}

linfusion_status_t linfusion_attn_workspace_bytes(const linfusion_attn_desc_t* desc, int sm_count,
                                                  size_t* bytes)
{
    if (bytes == nullptr) return LINFUSION_ERR_INVALID_ARG;
    Plan p;
    linfusion_status_t st = make_plan(desc, sm_count, &p);
    if (st != LINFUSION_OK) return st;
    *bytes = p.total_bytes;
    return LINFUSION_OK;
}

linfusion_status_t linfusion_attn_plan(const linfusion_attn_desc_t* desc, int sm_count, int32_t* variant,
                                       int32_t* launches, int32_t* ctas)
{
    Plan p;
    linfusion_status_t st = make_plan(desc, sm_count, &p);
    if (st != LINFUSION_OK) return st;
    if (variant != nullptr) *variant = p.variant;
    if (launches != nullptr) *launches = p.launches;
    if (ctas != nullptr) *ctas = p.G_state > p.G_apply ? p.G_state : p.G_apply;
    return LINFUSION_OK;
}

linfusion_status_t linfusion_attn_create(const linfusion_attn_desc_t* desc, linfusion_attn_t** out)
{
    if (out == nullptr) return LINFUSION_ERR_INVALID_ARG;
    *out = nullptr;
    linfusion_status_t st = validate(desc);
    if (st != LINFUSION_OK) return st;

    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess) {
        cudaGetLastError();
        return LINFUSION_ERR_CUDA;
    }
    if (desc->device >= ndev) return LINFUSION_ERR_INVALID_ARG;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, desc->device) != cudaSuccess) return LINFUSION_ERR_CUDA;
    if (prop.major != 10) return LINFUSION_ERR_UNSUPPORTED;

    DeviceGuard guard(desc->device);
    if (!guard.ok) return LINFUSION_ERR_CUDA;

    linfusion_attn* h = new (std::nothrow) linfusion_attn();
    if (h == nullptr) return LINFUSION_ERR_ALLOC;
    h->desc = *desc;
    h->sm_count = prop.multiProcessorCount;
    h->ws = nullptr;
    h->owns_ws = false;
    h->last_stream = nullptr;
    for (int i = 0; i < 4; ++i) h->stage[i] = nullptr;
    h->events = nullptr;
    h->timing_slots = 0;
    h->timed_calls = 0;
    h->timing_stride = 1;
    h->forward_calls = 0;
    h->sample_now = false;
    h->pipe = nullptr;
    h->x_stats = nullptr;
    h->x_t[0] = h->x_t[1] = nullptr;
    st = make_plan(desc, h->sm_count, &h->plan);
    if (st != LINFUSION_OK) {
        delete h;
        return st;
    }

    cudaError_t e = cudaSuccess;
#define LF_SET(DKV, DVV) e = set_attrs_d<DKV, DVV>(kind_of(*desc))
    LF_DISPATCH_D(*desc, LF_SET)
#undef LF_SET
    if (e == cudaSuccess && desc->d == kStreamD && dk_of(*desc) == kStreamD) {
#define LF_K(KV) e = set_stream_attrs<KV>()
        LF_DISPATCH_KIND(kind_of(*desc), LF_K)
#undef LF_K
    }
    if (e != cudaSuccess) {
        cudaGetLastError();
        delete h;
        return LINFUSION_ERR_CUDA;
    }

    if (h->plan.variant == kCluster) {
        // Shrink the cluster until the device can co-schedule it; else fall back to three launches.
        bool fits = false;
        const bool forced = (desc->flags & LINFUSION_VARIANT_MASK) == LINFUSION_VARIANT_CLUSTER;
        while (true) {
#define LF_FIT(DKV, DVV) fits = cluster_fits<DKV, DVV>(kind_of(*desc), h->plan.cluster_size, h->plan.slabs)
            LF_DISPATCH_D(*desc, LF_FIT)
#undef LF_FIT
            if (fits || h->plan.cluster_size == 1) break;
            h->plan.cluster_size >>= 1;
        }
        if (!fits) {
            if (forced) {
                delete h;
                return LINFUSION_ERR_UNSUPPORTED;
            }
            linfusion_attn_desc_t d2 = *desc;
            d2.flags = (d2.flags & ~LINFUSION_VARIANT_MASK) | LINFUSION_VARIANT_SPLIT;
            make_plan(&d2, h->sm_count, &h->plan);
        }
    }

    void* ws = nullptr;
    if (cudaMalloc(&ws, h->plan.total_bytes) != cudaSuccess) {
        cudaGetLastError();
        delete h;
        return LINFUSION_ERR_ALLOC;
    }
    h->owns_ws = true;
    bind_workspace(h, ws);
    if (!clear_workspace_tail(h)) {
        cudaFree(ws);
        delete h;
        return LINFUSION_ERR_CUDA;
    }
    *out = h;
    return LINFUSION_OK;
}

linfusion_status_t linfusion_attn_set_workspace(linfusion_attn_t* h, void* dev_ptr, size_t bytes)
{
    if (h == nullptr || dev_ptr == nullptr) return LINFUSION_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(dev_ptr) & 255u) != 0) return LINFUSION_ERR_INVALID_ARG;
    if (bytes < h->plan.total_bytes) return LINFUSION_ERR_ALLOC;
    DeviceGuard guard(h->desc.device);
    if (!guard.ok) return LINFUSION_ERR_CUDA;
    cudaStreamSynchronize(h->last_stream);
    if (h->owns_ws && h->ws != nullptr) cudaFree(h->ws);
    h->owns_ws = false;
    bind_workspace(h, dev_ptr);
    if (!clear_workspace_tail(h)) return LINFUSION_ERR_CUDA;
    return LINFUSION_OK;
}

linfusion_status_t linfusion_attn_forward(linfusion_attn_t* h, const void* q, const void* k,
                                          const void* v, void* y, void* cuda_stream)
{
    if (h == nullptr || q == nullptr || k == nullptr || v == nullptr || y == nullptr)
        return LINFUSION_ERR_INVALID_ARG;
    const uintptr_t pq = reinterpret_cast<uintptr_t>(q), pk = reinterpret_cast<uintptr_t>(k),
                    pv = reinterpret_cast<uintptr_t>(v), py = reinterpret_cast<uintptr_t>(y);
    if (((pq | pk | pv | py) & 15u) != 0) return LINFUSION_ERR_INVALID_ARG;
    const size_t nqk = bytes_qk(h->desc), nvy = bytes_vy(h->desc);
    auto overlaps = [&](uintptr_t a, size_t n) { return a < py + nvy && py < a + n; };
    if (overlaps(pq, nqk) || overlaps(pk, nqk) || overlaps(pv, nvy)) return LINFUSION_ERR_INVALID_ARG;

    DeviceGuard guard(h->desc.device);
    if (!guard.ok) return LINFUSION_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const __nv_bfloat16* Q = static_cast<const __nv_bfloat16*>(q);
    const __nv_bfloat16* K = static_cast<const __nv_bfloat16*>(k);
    const __nv_bfloat16* V = static_cast<const __nv_bfloat16*>(v);
    __nv_bfloat16* Y = static_cast<__nv_bfloat16*>(y);

    h->sample_now = h->events != nullptr && h->forward_calls % h->timing_stride == 0;
    cudaError_t e = cudaErrorInvalidValue;
    if (h->plan.variant == kStream) {
#define LF_K(KV) e = launch_stream<KV>(h, Q, K, V, Y, s)
        LF_DISPATCH_KIND(kind_of(h->desc), LF_K)
#undef LF_K
    } else if (h->plan.variant == kFused && h->plan.padded_per_slab > 0) {
        switch (h->desc.d) {
            case 40: e = launch_padded_d<40>(h, Q, K, V, Y, s); break;
            case 80: e = launch_padded_d<80>(h, Q, K, V, Y, s); break;
            case 160: e = launch_padded_d<160>(h, Q, K, V, Y, s); break;
            default: break;
        }
    } else if (h->plan.variant == kFused) {
#define LF_K(KV) e = launch_fused<KV>(h, Q, K, V, Y, s)
        LF_DISPATCH_KIND(kind_of(h->desc), LF_K)
#undef LF_K
    } else {
#define LF_LAUNCH(DKV, DVV) e = launch_d<DKV, DVV>(h, Q, K, V, Y, s)
        LF_DISPATCH_D(h->desc, LF_LAUNCH)
#undef LF_LAUNCH
    }
    h->last_stream = s;
    if (h->events != nullptr) ++h->forward_calls;
    if (h->sample_now) ++h->timed_calls;
    h->sample_now = false;
    if (e != cudaSuccess) {
        cudaGetLastError();
        return LINFUSION_ERR_CUDA;
    }
    return LINFUSION_OK;
}

linfusion_status_t linfusion_attn_enable_kernel_timing(linfusion_attn_t* h, int32_t slots)
{
    if (h == nullptr || slots < 0 || slots > 4096) return LINFUSION_ERR_INVALID_ARG;
    DeviceGuard guard(h->desc.device);
    if (!guard.ok) return LINFUSION_ERR_CUDA;
    if (h->events != nullptr) {
        cudaStreamSynchronize(h->last_stream);
        for (int i = 0; i < h->timing_slots * 4; ++i) cudaEventDestroy(h->events[i]);
        delete[] h->events;
        h->events = nullptr;
    }
    h->timing_slots = 0;
    h->timed_calls = 0;
    h->forward_calls = 0;
    h->sample_now = false;
    if (slots == 0) return LINFUSION_OK;
    cudaEvent_t* ev = new (std::nothrow) cudaEvent_t[slots * 4];
    if (ev == nullptr) return LINFUSION_ERR_ALLOC;
    for (int i = 0; i < slots * 4; ++i) {
        if (cudaEventCreate(&ev[i]) != cudaSuccess) {
            for (int j = 0; j < i; ++j) cudaEventDestroy(ev[j]);
            delete[] ev;
            cudaGetLastError();
            return LINFUSION_ERR_CUDA;
        }
    }
    h->events = ev;
    h->timing_slots = slots;
    return LINFUSION_OK;
}

linfusion_status_t linfusion_attn_set_kernel_timing_stride(linfusion_attn_t* h, int32_t stride)
{
    if (h == nullptr || stride < 1) return LINFUSION_ERR_INVALID_ARG;
    h->timing_stride = stride;
    return LINFUSION_OK;
}

linfusion_status_t linfusion_attn_kernel_times(linfusion_attn_t* h, float* ms_sum, int32_t* calls)
{
    if (h == nullptr || ms_sum == nullptr || calls == nullptr) return LINFUSION_ERR_INVALID_ARG;
    ms_sum[0] = ms_sum[1] = ms_sum[2] = 0.0f;
    *calls = 0;
    if (h->events == nullptr) return LINFUSION_OK;
    DeviceGuard guard(h->desc.device);
    if (!guard.ok) return LINFUSION_ERR_CUDA;
    if (cudaStreamSynchronize(h->last_stream) != cudaSuccess) {
        cudaGetLastError();
        return LINFUSION_ERR_CUDA;
    }
    const int n = static_cast<int>(h->timed_calls < h->timing_slots ? h->timed_calls : h->timing_slots);
    const int kernels = h->plan.launches;
    for (int c = 0; c < n; ++c) {
        for (int k = 0; k < kernels; ++k) {
            float ms = 0.0f;
            if (cudaEventElapsedTime(&ms, h->events[c * 4 + k], h->events[c * 4 + k + 1]) != cudaSuccess) {
                cudaGetLastError();
                return LINFUSION_ERR_CUDA;
            }
            ms_sum[k] += ms;
        }
    }
    *calls = n;
    h->timed_calls = 0;
    return LINFUSION_OK;
}

linfusion_status_t linfusion_attn_forward_host(linfusion_attn_t* h, const void* q_host,
                                               const void* k_host, const void* v_host, void* y_host,
                                               void* cuda_stream)
{
    if (h == nullptr || q_host == nullptr || k_host == nullptr || v_host == nullptr || y_host == nullptr)
        return LINFUSION_ERR_INVALID_ARG;
    DeviceGuard guard(h->desc.device);
    if (!guard.ok) return LINFUSION_ERR_CUDA;
    // Staging buffers 0..3 hold Q, K, V, Y: Q and K are d' wide, V and Y d wide.
    const size_t nqk = bytes_qk(h->desc), nvy = bytes_vy(h->desc);
    const size_t stage_bytes[4] = {nqk, nqk, nvy, nvy};
    const size_t bytes = nvy;
    if (h->stage[0] == nullptr) {
        for (int i = 0; i < 4; ++i) {
            if (cudaMalloc(&h->stage[i], stage_bytes[i]) != cudaSuccess) {
                cudaGetLastError();
                for (int j = 0; j < i; ++j) cudaFree(h->stage[j]);
                for (int j = 0; j < 4; ++j) h->stage[j] = nullptr;
                return LINFUSION_ERR_ALLOC;
            }
        }
    }
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (h->pipe == nullptr) {
        // First use: decide the grouping, make the group handle, the copy streams and the events.
        HostPipe* p = new (std::nothrow) HostPipe();
        if (p == nullptr) return LINFUSION_ERR_ALLOC;
        const int slabs = h->plan.slabs;
        // Groups are runs of whole slabs, which are contiguous in memory only in the head-major layout.
        const bool head_major = (h->desc.flags & LINFUSION_LAYOUT_TOKEN_MAJOR) == 0u;
        for (int g = kMaxHostGroups; head_major && g >= 2; --g)
            if (slabs % g == 0 && bytes / g >= (size_t(32) << 20)) {
                p->groups = g;
                break;
            }
        bool ok = true;
        if (p->groups > 1) {
            linfusion_attn_desc_t d = h->desc;
            d.B = 1;
            d.H = slabs / p->groups;
            d.flags = static_cast<uint32_t>(h->plan.variant) |
                      (h->desc.flags & (LINFUSION_FLAG_UNNORMALIZED | LINFUSION_DTYPE_FP16));  // head-major only (see the grouping rule above)
            ok = linfusion_attn_create(&d, &p->sub) == LINFUSION_OK;
            ok = ok && cudaStreamCreateWithFlags(&p->copy_in, cudaStreamNonBlocking) == cudaSuccess;
            ok = ok && cudaStreamCreateWithFlags(&p->copy_out, cudaStreamNonBlocking) == cudaSuccess;
            ok = ok && cudaEventCreateWithFlags(&p->entry, cudaEventDisableTiming) == cudaSuccess;
            ok = ok && cudaEventCreateWithFlags(&p->out, cudaEventDisableTiming) == cudaSuccess;
            for (int i = 0; ok && i < p->groups; ++i)
                ok = cudaEventCreateWithFlags(&p->in[i], cudaEventDisableTiming) == cudaSuccess &&
                     cudaEventCreateWithFlags(&p->done[i], cudaEventDisableTiming) == cudaSuccess;
        }
        if (!ok) {
            cudaGetLastError();
            p->groups = 1;  // fall back to one group on the caller's stream
        }
        h->pipe = p;
    }
    HostPipe* p = h->pipe;
    if (p->groups == 1) {
        // K and V first: they feed the first kernel.
        if (cudaMemcpyAsync(h->stage[1], k_host, nqk, cudaMemcpyHostToDevice, s) != cudaSuccess ||
            cudaMemcpyAsync(h->stage[2], v_host, nvy, cudaMemcpyHostToDevice, s) != cudaSuccess ||
            cudaMemcpyAsync(h->stage[0], q_host, nqk, cudaMemcpyHostToDevice, s) != cudaSuccess) {
            cudaGetLastError();
            return LINFUSION_ERR_CUDA;
        }
        linfusion_status_t st = linfusion_attn_forward(h, h->stage[0], h->stage[1], h->stage[2], h->stage[3], s);
        if (st != LINFUSION_OK) return st;
        if (cudaMemcpyAsync(y_host, h->stage[3], nvy, cudaMemcpyDeviceToHost, s) != cudaSuccess) {
            cudaGetLastError();
            return LINFUSION_ERR_CUDA;
        }
        return LINFUSION_OK;
    }

    // Uploads run ahead on copy_in, kernels follow on the caller's stream, downloads trail on
    // copy_out; everything is ordered after the caller's earlier work and before its later work.
    const size_t gbytes = nvy / p->groups, gbytes_qk = nqk / p->groups;
    auto at = [&](const void* base, int i, size_t gb) { return static_cast<const unsigned char*>(base) + i * gb; };
    auto dev = [&](int which, int i) {
        return static_cast<unsigned char*>(h->stage[which]) + i * (which < 2 ? gbytes_qk : gbytes);
    };
    bool ok = cudaEventRecord(p->entry, s) == cudaSuccess &&
              cudaStreamWaitEvent(p->copy_in, p->entry, 0) == cudaSuccess &&
              cudaStreamWaitEvent(p->copy_out, p->entry, 0) == cudaSuccess;
    for (int i = 0; ok && i < p->groups; ++i) {
        ok = cudaMemcpyAsync(dev(1, i), at(k_host, i, gbytes_qk), gbytes_qk, cudaMemcpyHostToDevice, p->copy_in) == cudaSuccess &&
             cudaMemcpyAsync(dev(2, i), at(v_host, i, gbytes), gbytes, cudaMemcpyHostToDevice, p->copy_in) == cudaSuccess &&
             cudaMemcpyAsync(dev(0, i), at(q_host, i, gbytes_qk), gbytes_qk, cudaMemcpyHostToDevice, p->copy_in) == cudaSuccess &&
             cudaEventRecord(p->in[i], p->copy_in) == cudaSuccess &&
             cudaStreamWaitEvent(s, p->in[i], 0) == cudaSuccess;
        if (!ok) break;
        linfusion_status_t st = linfusion_attn_forward(p->sub, dev(0, i), dev(1, i), dev(2, i), dev(3, i), s);
        if (st != LINFUSION_OK) return st;
        ok = cudaEventRecord(p->done[i], s) == cudaSuccess &&
             cudaStreamWaitEvent(p->copy_out, p->done[i], 0) == cudaSuccess &&
             cudaMemcpyAsync(static_cast<unsigned char*>(y_host) + i * gbytes, dev(3, i), gbytes,
                             cudaMemcpyDeviceToHost, p->copy_out) == cudaSuccess;
    }
    ok = ok && cudaEventRecord(p->out, p->copy_out) == cudaSuccess &&
         cudaStreamWaitEvent(s, p->out, 0) == cudaSuccess;
    h->last_stream = s;
    if (!ok) {
        cudaGetLastError();
        return LINFUSION_ERR_CUDA;
    }
    return LINFUSION_OK;
}

linfusion_status_t linfusion_attn_status(linfusion_attn_t* h)
{
    if (h == nullptr) return LINFUSION_ERR_INVALID_ARG;
    DeviceGuard guard(h->desc.device);
    if (!guard.ok) return LINFUSION_ERR_CUDA;
    if (cudaStreamSynchronize(h->last_stream) != cudaSuccess) {
        cudaGetLastError();
        return LINFUSION_ERR_CUDA;
    }
    uint32_t word = 0;
    if (cudaMemcpy(&word, h->status, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess) {
        cudaGetLastError();
        return LINFUSION_ERR_CUDA;
    }
    if (word != kStatusOk) return LINFUSION_ERR_TIMEOUT;
    if (h->pipe != nullptr && h->pipe->sub != nullptr) return linfusion_attn_status(h->pipe->sub);
    return LINFUSION_OK;
}

static linfusion_status_t selftest_wait_impl(linfusion_attn_t* h, float* waited_ms, bool counter);

linfusion_status_t linfusion_attn_selftest_wait(linfusion_attn_t* h, float* waited_ms)
{
    return selftest_wait_impl(h, waited_ms, false);
}

linfusion_status_t linfusion_attn_selftest_counter_wait(linfusion_attn_t* h, float* waited_ms)
{
    return selftest_wait_impl(h, waited_ms, true);
}

static linfusion_status_t selftest_wait_impl(linfusion_attn_t* h, float* waited_ms, bool counter)
{
    if (h == nullptr || h->status == nullptr) return LINFUSION_ERR_INVALID_ARG;
    DeviceGuard guard(h->desc.device);
    if (!guard.ok) return LINFUSION_ERR_CUDA;
    cudaStream_t s = h->last_stream;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) {
        if (e0 != nullptr) cudaEventDestroy(e0);
        cudaGetLastError();
        return LINFUSION_ERR_CUDA;
    }
    cudaEventRecord(e0, s);
    if (counter)  // a word nothing advances: the second word behind the status word (always zero)
        counter_wait_selftest_kernel<<<1, 32, 0, s>>>(h->status, h->status + 1);
    else
        wait_selftest_kernel<<<1, 32, 0, s>>>(h->status);
    cudaEventRecord(e1, s);
    uint32_t word = 0;
    float ms = 0.0f;
    bool ok = cudaStreamSynchronize(s) == cudaSuccess && cudaEventElapsedTime(&ms, e0, e1) == cudaSuccess &&
              cudaMemcpy(&word, h->status, sizeof(word), cudaMemcpyDeviceToHost) == cudaSuccess &&
              cudaMemset(h->status, 0, sizeof(word)) == cudaSuccess;  // the handle stays usable
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (!ok) {
        cudaGetLastError();
        return LINFUSION_ERR_CUDA;
    }
    if (waited_ms != nullptr) *waited_ms = ms;
    return word != kStatusOk ? LINFUSION_ERR_TIMEOUT : LINFUSION_OK;
}

linfusion_status_t linfusion_attn_read_state(linfusion_attn_t* h, float* S_host, float* z_host)
{
    if (h == nullptr) return LINFUSION_ERR_INVALID_ARG;
    DeviceGuard guard(h->desc.device);
    if (!guard.ok) return LINFUSION_ERR_CUDA;
    if (cudaStreamSynchronize(h->last_stream) != cudaSuccess) {
        cudaGetLastError();
        return LINFUSION_ERR_CUDA;
    }
    const int dk = dk_of(h->desc), dv = h->desc.d, sf = h->plan.state_floats;
    for (int s = 0; s < h->plan.slabs; ++s) {
        const float* src = h->state + static_cast<size_t>(s) * sf;
        if (S_host != nullptr &&
            cudaMemcpy(S_host + static_cast<size_t>(s) * dk * dv, src, sizeof(float) * dk * dv,
                       cudaMemcpyDeviceToHost) != cudaSuccess)
            return LINFUSION_ERR_CUDA;
        if (z_host != nullptr &&
            cudaMemcpy(z_host + static_cast<size_t>(s) * dk, src + dk * dv, sizeof(float) * dk,
                       cudaMemcpyDeviceToHost) != cudaSuccess)
            return LINFUSION_ERR_CUDA;
    }
    return LINFUSION_OK;
}

const char* linfusion_attn_variant_name(const linfusion_attn_t* h)
{
    if (h == nullptr) return "";
    switch (h->plan.variant) {
        case kSplit: return "split";
        case kStream: return "stream";
        case kCluster: return "cluster";
        case kFused: return "fused";
        default: return "";
    }
}

int32_t linfusion_attn_launches_per_forward(const linfusion_attn_t* h)
{
    return h == nullptr ? 0 : h->plan.launches;
}

linfusion_status_t linfusion_attn_destroy(linfusion_attn_t* h)
{
    if (h == nullptr) return LINFUSION_OK;
    DeviceGuard guard(h->desc.device);
    linfusion_status_t st = LINFUSION_OK;
    if (guard.ok) {
        if (h->owns_ws && h->ws != nullptr && cudaFree(h->ws) != cudaSuccess) st = LINFUSION_ERR_CUDA;
        for (int i = 0; i < 4; ++i)
            if (h->stage[i] != nullptr && cudaFree(h->stage[i]) != cudaSuccess) st = LINFUSION_ERR_CUDA;
        if (h->x_stats != nullptr && cudaFree(h->x_stats) != cudaSuccess) st = LINFUSION_ERR_CUDA;
        for (int i = 0; i < 2; ++i)
            if (h->x_t[i] != nullptr && cudaFree(h->x_t[i]) != cudaSuccess) st = LINFUSION_ERR_CUDA;
        if (h->events != nullptr) {
            for (int i = 0; i < h->timing_slots * 4; ++i) cudaEventDestroy(h->events[i]);
            delete[] h->events;
        }
        if (h->pipe != nullptr) {
            HostPipe* p = h->pipe;
            if (p->sub != nullptr && linfusion_attn_destroy(p->sub) != LINFUSION_OK) st = LINFUSION_ERR_CUDA;
            if (p->copy_in != nullptr) cudaStreamDestroy(p->copy_in);
            if (p->copy_out != nullptr) cudaStreamDestroy(p->copy_out);
            if (p->entry != nullptr) cudaEventDestroy(p->entry);
            if (p->out != nullptr) cudaEventDestroy(p->out);
            for (int i = 0; i < kMaxHostGroups; ++i) {
                if (p->in[i] != nullptr) cudaEventDestroy(p->in[i]);
                if (p->done[i] != nullptr) cudaEventDestroy(p->done[i]);
            }
            delete p;
        }
    } else {
        st = LINFUSION_ERR_CUDA;
    }
    delete h;
    return st;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Allocation-free forward (see the header): the split-N partials and the reduced state live in a
// fixed array in device global memory that is part of this library's image, so nothing is ever
// requested from the CUDA allocator.  Every device that loads the library carries the array
// until the process exits.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr size_t kNoAllocScratchBytes = size_t(16) << 20;  // 16 MiB
constexpr int kNoAllocMaxDevices = 64;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

struct NoAllocDevice {
    std::atomic<bool> ready{false};
    unsigned char* scratch = nullptr;  // device address of g_noalloc_scratch on this device
    int sm_count = 0;
    std::atomic<uint64_t> configured{0};  // bit (width-pair index * 4 + kind): shared-memory limits raised
};
NoAllocDevice g_noalloc_dev[kNoAllocMaxDevices];
std::mutex g_noalloc_mutex;  // serializes the set-up below (first calls from several host threads)

// Index of a supported (d', d) pair.
int width_pair_index(int dk, int dv)
{
    switch (dk * 1000 + dv) {
        case 32032: return 0;
        case 40040: return 1;
        case 64064: return 2;
        case 80080: return 3;
        case 128128: return 4;
        case 160160: return 5;
        case 128064: return 6;
        case 80040: return 7;
        case 32064: return 8;
        default: return -1;
    }
}

// The two kernels this entry point launches per (head dim, kind); the cluster kernel is not among them.
template <int DK, int DV>
cudaError_t set_noalloc_attrs_d(int kind)
{
    using C = SplitCfg<DK, DV>;
    cudaError_t e = cudaErrorInvalidValue;
#define LF_K(KV)                                                                                                         \
    e = cudaFuncSetAttribute(state_partial_kernel<DK, DV, KV>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_KV); \
    if (e == cudaSuccess)                                                                                                \
    e = cudaFuncSetAttribute(apply_kernel<DK, DV, KV>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_APPLY)
    LF_DISPATCH_KIND(kind, LF_K)
#undef LF_K
    return e;
}

// With `device` current.  Once per device: resolve the array's device address (the symbol's name
// is only a host-side stand-in and must never be handed to a kernel) and read the SM count.  Once
// per (device, head dim, kind): raise the two kernels' dynamic shared-memory limits.  Later calls
// find both done and make no CUDA call here.  Safe for first calls made by several host threads
// at once: the set-up runs under a mutex and is published with release / acquire.
linfusion_status_t noalloc_setup(const linfusion_attn_desc_t& desc, int kind)
{
    const int device = desc.device;
    NoAllocDevice& dev = g_noalloc_dev[device];
    const uint64_t bit = uint64_t(1) << (width_pair_index(dk_of(desc), desc.d) * 4 + kind);
    if (dev.ready.load(std::memory_order_acquire) && (dev.configured.load(std::memory_order_acquire) & bit) != 0u)
        return LINFUSION_OK;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!dev.ready.load(std::memory_order_relaxed)) {
        int ndev = 0;
        if (cudaGetDeviceCount(&ndev) != cudaSuccess) {
            cudaGetLastError();
            return LINFUSION_ERR_CUDA;
        }
        if (device >= ndev) return LINFUSION_ERR_INVALID_ARG;
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) {
            cudaGetLastError();
            return LINFUSION_ERR_CUDA;
        }
        if (prop.major != 10) return LINFUSION_ERR_UNSUPPORTED;
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return LINFUSION_ERR_CUDA;
        }
        dev.scratch = static_cast<unsigned char*>(ptr);
        dev.sm_count = prop.multiProcessorCount;
        dev.ready.store(true, std::memory_order_release);
    }
    if ((dev.configured.load(std::memory_order_relaxed) & bit) == 0u) {
        cudaError_t e = cudaErrorInvalidValue;
#define LF_SET(DKV, DVV) e = set_noalloc_attrs_d<DKV, DVV>(kind)
        LF_DISPATCH_D(desc, LF_SET)
#undef LF_SET
        if (e != cudaSuccess) {
            cudaGetLastError();
            return LINFUSION_ERR_CUDA;
        }
        dev.configured.fetch_or(bit, std::memory_order_release);
    }
    return LINFUSION_OK;
}

// Where a problem's partial states and reduced state sit in the fixed array: `chunks` partials of
// per_chunk bytes from offset 0, the state at the next 256-byte boundary.  The split of N is the
// split path's plan for `sm_count` SMs, cut down to as many chunks as leave room for the state.
// ALLOC when not even one chunk and the state fit.  Pure host arithmetic.
linfusion_status_t noalloc_layout(const linfusion_attn_desc_t* desc, int sm_count, Plan* plan, size_t* state_off,
                                  size_t* bytes_used)
{
    linfusion_status_t st = validate(desc);
    if (st != LINFUSION_OK) return st;
    if ((desc->flags & LINFUSION_VARIANT_MASK) > LINFUSION_VARIANT_SPLIT) return LINFUSION_ERR_UNSUPPORTED;
    const size_t per_chunk = static_cast<size_t>(desc->B) * desc->H * dk_of(*desc) * (desc->d + 1) * 4;
    const size_t state_bytes = align_up(per_chunk, 256);
    if (state_bytes + per_chunk + 256 > kNoAllocScratchBytes) return LINFUSION_ERR_ALLOC;
    linfusion_attn_desc_t d = *desc;
    d.flags = (desc->flags & (LINFUSION_LAYOUT_TOKEN_MAJOR | LINFUSION_FLAG_UNNORMALIZED | LINFUSION_DTYPE_FP16)) |
              LINFUSION_VARIANT_SPLIT;
    st = make_plan(&d, sm_count, plan);
    if (st != LINFUSION_OK) return st;
    const size_t room = (kNoAllocScratchBytes - state_bytes - 256) / per_chunk;
    if (static_cast<size_t>(plan->chunks_state) > room) plan->chunks_state = static_cast<int>(room);
    *state_off = align_up(per_chunk * static_cast<size_t>(plan->chunks_state), 256);
    *bytes_used = *state_off + per_chunk;
    return LINFUSION_OK;
}

}  // namespace

extern "C" linfusion_status_t linfusion_attn_noalloc_layout(const linfusion_attn_desc_t* desc, int sm_count,
                                                            int32_t* chunks, size_t* state_offset,
                                                            size_t* bytes_used, size_t* capacity)
{
    Plan plan;
    size_t off = 0, used = 0;
    linfusion_status_t st = noalloc_layout(desc, sm_count, &plan, &off, &used);
    if (capacity != nullptr) *capacity = kNoAllocScratchBytes;
    if (st != LINFUSION_OK) return st;
    if (chunks != nullptr) *chunks = plan.chunks_state;
    if (state_offset != nullptr) *state_offset = off;
    if (bytes_used != nullptr) *bytes_used = used;
    return LINFUSION_OK;
}

extern "C" linfusion_status_t linfusion_attn_forward_noalloc(const linfusion_attn_desc_t* desc,
                                                             const void* q, const void* k,
                                                             const void* v, void* y,
                                                             void* cuda_stream)
{
    // Descriptor and capacity first: they depend on the descriptor alone (the chunk count is
    // settled below, once the device's SM count is known).
    linfusion_attn view;
    size_t state_off = 0, bytes_used = 0;
    linfusion_status_t st = noalloc_layout(desc, 0, &view.plan, &state_off, &bytes_used);
    if (st != LINFUSION_OK) return st;
    if (desc->device >= kNoAllocMaxDevices) return LINFUSION_ERR_INVALID_ARG;
    if (q == nullptr || k == nullptr || v == nullptr || y == nullptr) return LINFUSION_ERR_INVALID_ARG;
    const uintptr_t pq = reinterpret_cast<uintptr_t>(q), pk = reinterpret_cast<uintptr_t>(k),
                    pv = reinterpret_cast<uintptr_t>(v), py = reinterpret_cast<uintptr_t>(y);
    if (((pq | pk | pv | py) & 15u) != 0) return LINFUSION_ERR_INVALID_ARG;
    const size_t nqk = bytes_qk(*desc), nvy = bytes_vy(*desc);
    auto overlaps = [&](uintptr_t a, size_t n) { return a < py + nvy && py < a + n; };
    if (overlaps(pq, nqk) || overlaps(pk, nqk) || overlaps(pv, nvy)) return LINFUSION_ERR_INVALID_ARG;

    // (A device ordinal the process does not have fails in cudaSetDevice here, or in the first
    // call's set-up, which asks for the device count.)
    DeviceGuard guard(desc->device);
    if (!guard.ok) {
        cudaGetLastError();
        return g_noalloc_dev[desc->device].ready.load(std::memory_order_acquire) ? LINFUSION_ERR_CUDA
                                                                                 : LINFUSION_ERR_INVALID_ARG;
    }
    st = noalloc_setup(*desc, kind_of(*desc));
    if (st != LINFUSION_OK) return st;
    const NoAllocDevice& dev = g_noalloc_dev[desc->device];

    // A handle-shaped view on the stack: the three-launch split plan, with as many chunks of N
    // as the fixed array has room for.  Nothing in the array has to start at zero: every partial
    // and every state element that is read in this call is written earlier in the same call.
    view.desc = *desc;
    view.desc.flags = (desc->flags & (LINFUSION_LAYOUT_TOKEN_MAJOR | LINFUSION_FLAG_UNNORMALIZED | LINFUSION_DTYPE_FP16)) |
                      LINFUSION_VARIANT_SPLIT;
    st = noalloc_layout(desc, dev.sm_count, &view.plan, &state_off, &bytes_used);
    if (st != LINFUSION_OK) return st;
    if (bytes_used > kNoAllocScratchBytes) return LINFUSION_ERR_ALLOC;  // cannot happen; the array is never overrun
    view.sm_count = dev.sm_count;
    view.ws = dev.scratch;
    view.ws_bytes = bytes_used;
    view.owns_ws = false;
    view.partials = reinterpret_cast<float*>(dev.scratch);
    view.state = reinterpret_cast<float*>(dev.scratch + state_off);
    view.operand = nullptr;
    view.tile_counters = nullptr;
    view.status = nullptr;
    view.last_stream = nullptr;
    for (int i = 0; i < 4; ++i) view.stage[i] = nullptr;
    view.events = nullptr;
    view.timing_slots = 0;
    view.timed_calls = 0;
    view.timing_stride = 1;
    view.forward_calls = 0;
    view.sample_now = false;
    view.pipe = nullptr;
    view.x_stats = nullptr;
    view.x_t[0] = view.x_t[1] = nullptr;

    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const __nv_bfloat16* Q = static_cast<const __nv_bfloat16*>(q);
    const __nv_bfloat16* K = static_cast<const __nv_bfloat16*>(k);
    const __nv_bfloat16* V = static_cast<const __nv_bfloat16*>(v);
    __nv_bfloat16* Y = static_cast<__nv_bfloat16*>(y);
    cudaError_t e = cudaErrorInvalidValue;
#define LF_LAUNCH(DKV, DVV) e = launch_d<DKV, DVV>(&view, Q, K, V, Y, s)
    LF_DISPATCH_D(view.desc, LF_LAUNCH)
#undef LF_LAUNCH
    if (e != cudaSuccess) {
        cudaGetLastError();
        return LINFUSION_ERR_CUDA;
    }
    return LINFUSION_OK;
}

// ---------------------------------------------------------------------------------------------
// Token-sharded (sequence-parallel) use, Sec. 4.3: every device owns a run of the tokens of Q, K, V
// and Y, builds the state of its own K/V tokens, the devices sum their S | z (the only exchange,
// d x (d+1) floats per slab whatever N is), and each applies the summed state to its own Q tokens.
// The library runs the two halves; the sum over devices is the caller's collective on the buffer
// that linfusion_attn_state_buffer() exposes.
// ---------------------------------------------------------------------------------------------
namespace {

template <int DK, int DV, int KIND>
cudaError_t launch_split_half(const linfusion_attn* h, bool state_half, const __nv_bfloat16* a,
                              const __nv_bfloat16* b, __nv_bfloat16* y, cudaStream_t s, const PeerStates* peers)
{
    using C = SplitCfg<DK, DV>;
    const SlabLayout LK = layout_qk(h->desc), LV = layout_vy(h->desc);
    if (state_half)
        register_checked_ranges(h, nullptr, a, b, nullptr, s);
    else
        register_checked_ranges(h, a, nullptr, nullptr, y, s, peers);
    const Plan& p = h->plan;
    const int N = h->desc.N;
    if (state_half) {
        state_partial_kernel<DK, DV, KIND><<<dim3(p.chunks_state, p.slabs), C::NT, C::SMEM_KV, s>>>(
            a, b, h->partials, N, p.chunks_state, LK, LV);
        state_reduce_kernel<<<dim3((C::STATE_FLOATS + 255) / 256, p.slabs), 256, 0, s>>>(
            h->partials, h->state, C::STATE_FLOATS, p.chunks_state, nullptr, DK, DV, C::PITCHK, C::SMEM_ST,
            dtype_of(h->desc), operand_scale(h->desc));
    } else if (peers != nullptr) {
        // Sum the devices' states into the operand image, then apply from the image.
        peer_sum_image_kernel<<<dim3((C::STATE_FLOATS + 255) / 256, p.slabs), 256, 0, s>>>(
            *peers, C::STATE_FLOATS, h->operand, DK, DV, C::PITCHK, C::SMEM_ST, dtype_of(h->desc), operand_scale(h->desc));
        apply_kernel<DK, DV, KIND><<<dim3(p.chunks_apply, p.slabs), C::NT, C::SMEM_APPLY, s>>>(
            a, h->state, y, N, p.chunks_apply, apply_scales(h->desc), LK, LV, h->operand);
    } else {
        // The fp32 state may have been summed over devices: convert it here, not from an image.
        apply_kernel<DK, DV, KIND><<<dim3(p.chunks_apply, p.slabs), C::NT, C::SMEM_APPLY, s>>>(
            a, h->state, y, N, p.chunks_apply, apply_scales(h->desc), LK, LV, nullptr);
    }
    return cudaGetLastError();
}

template <int KIND>
cudaError_t launch_stream_half(const linfusion_attn* h, bool state_half, const __nv_bfloat16* a,
                               const __nv_bfloat16* b, __nv_bfloat16* y, cudaStream_t s, const PeerStates* peers)
{
    const Plan& p = h->plan;
    const int N = h->desc.N;
    const dim3 rgrid((kStreamStateFloats + 255) / 256, p.slabs);
    if (state_half) {
        CUtensorMap mk, mv;
        if (!encode_slab_map(&mk, a, h->desc, StreamStateCfg::TILE) ||
            !encode_slab_map(&mv, b, h->desc, StreamStateCfg::TILE))
            return cudaErrorInvalidValue;
        stream_state_kernel<KIND><<<p.G_state, StreamStateCfg::THREADS, StreamStateCfg::SMEM_BYTES, s>>>(
            mk, mv, h->partials, h->status, N, p.tiles_state, p.W_state, p.spans, h->desc.H, nullptr, 0);
        stream_reduce_kernel<<<rgrid, 256, 0, s>>>(h->partials, h->state, h->operand, h->tile_counters,
                                                  p.tiles_state, p.W_state, p.G_state, p.spans,
                                                  dtype_of(h->desc), operand_scale(h->desc));
    } else {
        CUtensorMap mq, my;
        if (!encode_slab_map(&mq, a, h->desc, ApplyCfg::TILE) || !encode_slab_map(&my, y, h->desc, ApplyCfg::TILE))
            return cudaErrorInvalidValue;
        // The state may have been summed over devices since the reduction, or is summed over the
        // devices' buffers here: rebuild its 16-bit image.
        PeerStates own;
        own.p[0] = h->state;
        own.n = 1;
        stream_pack_kernel<<<rgrid, 256, 0, s>>>(peers != nullptr ? *peers : own, h->operand, h->tile_counters,
                                                dtype_of(h->desc), operand_scale(h->desc));
        stream_apply_kernel<KIND><<<p.G_apply, ApplyCfg::THREADS, ApplyCfg::SMEM_BYTES, s>>>(
            mq, my, h->operand, h->tile_counters, h->status, p.tiles_apply, p.slabs, apply_scales(h->desc), h->desc.H,
            MergedReduce{}, p.apply_static_runs);
    }
    return cudaGetLastError();
}

template <int DK, int DV>
cudaError_t split_half_d(const linfusion_attn* h, bool state_half, const __nv_bfloat16* a, const __nv_bfloat16* b,
                         __nv_bfloat16* y, cudaStream_t s, const PeerStates* peers)
{
    cudaError_t e = cudaErrorInvalidValue;
#define LF_K(KV) e = launch_split_half<DK, DV, KV>(h, state_half, a, b, y, s, peers)
    LF_DISPATCH_KIND(kind_of(h->desc), LF_K)
#undef LF_K
    return e;
}

linfusion_status_t run_half(linfusion_attn* h, bool state_half, const void* a, const void* b, void* y,
                            void* cuda_stream, const PeerStates* peers = nullptr)
{
    if (h == nullptr || a == nullptr || (state_half ? b == nullptr : y == nullptr))
        return LINFUSION_ERR_INVALID_ARG;
    if (h->plan.variant == kCluster || h->plan.variant == kFused) return LINFUSION_ERR_UNSUPPORTED;
    const uintptr_t pa = reinterpret_cast<uintptr_t>(a), pb = reinterpret_cast<uintptr_t>(b),
                    py = reinterpret_cast<uintptr_t>(y);
    if (((pa | pb | py) & 15u) != 0) return LINFUSION_ERR_INVALID_ARG;
    if (!state_half && pa < py + bytes_vy(h->desc) && py < pa + bytes_qk(h->desc)) return LINFUSION_ERR_INVALID_ARG;
    DeviceGuard guard(h->desc.device);
    if (!guard.ok) return LINFUSION_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const __nv_bfloat16* A = static_cast<const __nv_bfloat16*>(a);
    const __nv_bfloat16* B = static_cast<const __nv_bfloat16*>(b);
    __nv_bfloat16* Y = static_cast<__nv_bfloat16*>(y);
    cudaError_t e = cudaErrorInvalidValue;
    if (h->plan.variant == kStream) {
#define LF_K(KV) e = launch_stream_half<KV>(h, state_half, A, B, Y, s, peers)
        LF_DISPATCH_KIND(kind_of(h->desc), LF_K)
#undef LF_K
    } else {
#define LF_HALF(DKV, DVV) e = split_half_d<DKV, DVV>(h, state_half, A, B, Y, s, peers)
        LF_DISPATCH_D(h->desc, LF_HALF)
#undef LF_HALF
    }
    h->last_stream = s;
    if (e != cudaSuccess) {
        cudaGetLastError();
        return LINFUSION_ERR_CUDA;
    }
    return LINFUSION_OK;
}

}  // namespace

extern "C" linfusion_status_t linfusion_attn_state(linfusion_attn_t* h, const void* k, const void* v,
                                                   void* cuda_stream)
{
    return run_half(h, true, k, v, nullptr, cuda_stream);
}

extern "C" linfusion_status_t linfusion_attn_apply(linfusion_attn_t* h, const void* q, void* y,
                                                   void* cuda_stream)
{
    return run_half(h, false, q, nullptr, y, cuda_stream);
}

extern "C" linfusion_status_t linfusion_attn_apply_peers(linfusion_attn_t* h, const void* q, void* y,
                                                         const float* const* peer_states, int32_t n_peers,
                                                         void* cuda_stream)
{
    if (h == nullptr || peer_states == nullptr || n_peers < 1 || n_peers > kMaxPeers) return LINFUSION_ERR_INVALID_ARG;
    PeerStates ps;
    ps.n = n_peers;
    for (int r = 0; r < kMaxPeers; ++r) ps.p[r] = nullptr;
    for (int r = 0; r < n_peers; ++r) {
        if (peer_states[r] == nullptr || (reinterpret_cast<uintptr_t>(peer_states[r]) & 3u) != 0)
            return LINFUSION_ERR_INVALID_ARG;
        ps.p[r] = peer_states[r];
    }
    return run_half(h, false, q, nullptr, y, cuda_stream, &ps);
}

extern "C" linfusion_status_t linfusion_attn_state_buffer(linfusion_attn_t* h, float** dev_ptr,
                                                          size_t* floats)
{
    if (h == nullptr || dev_ptr == nullptr || floats == nullptr) return LINFUSION_ERR_INVALID_ARG;
    *dev_ptr = h->state;
    *floats = static_cast<size_t>(h->plan.slabs) * h->plan.state_floats;
    return LINFUSION_OK;
}


// ---------------------------------------------------------------------------------------------
// The attention fed from the layer input X (Sec. 3.1, implementation details; Eq. 2): the
// projections run inside the kernels that consume their results (producer_kernels.cuh).
// ---------------------------------------------------------------------------------------------
namespace {

// X [B, N, C] (16-bit, C = H * 64) -> boxes of 128 tokens x 64 channels, 128-byte swizzle, zero fill past N.
bool encode_x_map(CUtensorMap* map, const void* x, const linfusion_attn_desc_t& d)
{
    EncodeTiledFn fn = get_encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t C = static_cast<cuuint64_t>(d.H) * kStreamD;
    cuuint64_t dims[3] = {C, static_cast<cuuint64_t>(d.N), static_cast<cuuint64_t>(d.B)};
    cuuint64_t strides[2] = {C * 2, static_cast<cuuint64_t>(d.N) * C * 2};
    cuuint32_t box[3] = {64u, static_cast<cuuint32_t>(ProdState2Cfg::TILE), 1u};
    cuuint32_t estr[3] = {1u, 1u, 1u};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(x), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// A weight matrix W [C_in][C_out] (16-bit, row = input channel) seen as (column within head 64, input row C, head H) -> boxes of 64 input rows x the
// 64-column blocks of `heads` consecutive heads, which land in shared memory as consecutive 8 KB blocks
// (head, row, column): one copy per weight matrix and K chunk.  A head index past the last head reads as zeros.
bool encode_w_pair_map(CUtensorMap* map, const void* w, int C, int H, int heads = 2)
{
    EncodeTiledFn fn = get_encode_fn();
    if (fn == nullptr) return false;
    cuuint64_t dims[3] = {64u, static_cast<cuuint64_t>(C), static_cast<cuuint64_t>(H)};
    cuuint64_t strides[2] = {static_cast<cuuint64_t>(C) * 2, 128u};
    cuuint32_t box[3] = {64u, 64u, static_cast<cuuint32_t>(heads)};
    cuuint32_t estr[3] = {1u, 1u, 1u};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(w), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Handles that can take X: head dim 64 on both sides, the three-launch TMA + tcgen05 plan, and the
// token-major layout (X and Y are [B, N, C]: the heads of a token side by side).
bool takes_x(const linfusion_attn* h)
{
    return h->plan.variant == kStream && (h->desc.flags & LINFUSION_LAYOUT_TOKEN_MAJOR) != 0u;
}

template <int KIND>
cudaError_t launch_state_x(const linfusion_attn* h, const void* x, const void* w_k, const void* w_v, const void* t_k,
                           cudaStream_t s)
{
    const Plan& p = h->plan;
    const int C = h->desc.H * kStreamD;
    CUtensorMap mx, mwk, mwv;
    if (!encode_x_map(&mx, x, h->desc) || !encode_w_pair_map(&mwk, w_k, C, h->desc.H) ||
        !encode_w_pair_map(&mwv, w_v, C, h->desc.H))
        return cudaErrorInvalidValue;
    ProducerArgs pa;
    pa.N = h->desc.N;
    pa.H = h->desc.H;
    pa.chunks = C / ProdState2Cfg::KC;
    pa.has_t = t_k != nullptr ? 1 : 0;
    cudaError_t e = launch_chained(producer_state2_kernel<KIND>, dim3(p.G_x), dim3(ProdState2Cfg::THREADS),
                                   ProdState2Cfg::SMEM_BYTES, s, mx, mwk, mwv, static_cast<const __nv_bfloat16*>(t_k),
                                   h->partials, h->status, pa, p.tiles_state, p.W_x, p.spans_x);
    if (e != cudaSuccess) return e;
    e = launch_chained(producer_reduce_kernel, dim3((kStreamStateFloats + 255) / 256, p.slabs), dim3(256), 0, s,
                       h->partials, h->state, h->operand, h->tile_counters, p.tiles_state, p.W_x, p.G_x, p.spans_x,
                       h->desc.H, dtype_of(h->desc), operand_scale(h->desc));
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

template <int KIND>
cudaError_t launch_apply_x(const linfusion_attn* h, const void* x, const void* w_q, const void* t_q, void* y,
                           cudaStream_t s)
{
    const Plan& p = h->plan;
    const int C = h->desc.H * kStreamD;
    CUtensorMap mx, mwq, mt, my;
    if (!encode_x_map(&mx, x, h->desc) || !encode_w_pair_map(&mwq, w_q, C, h->desc.H) ||
        !encode_slab_map(&mt, t_q != nullptr ? t_q : x, h->desc, ProdApplyCfg::TILE) ||
        !encode_slab_map(&my, y, h->desc, ProdApplyCfg::TILE))
        return cudaErrorInvalidValue;
    ProducerArgs pa;
    pa.N = h->desc.N;
    pa.H = h->desc.H;
    pa.chunks = C / ProdApplyCfg::KC;
    pa.has_t = t_q != nullptr ? 1 : 0;
    // The fp32 state may have been summed over devices since it was reduced: rebuild its 16-bit image.
    PeerStates own;
    own.p[0] = h->state;
    own.n = 1;
    cudaError_t e = launch_chained(stream_pack_kernel, dim3((kStreamStateFloats + 255) / 256, p.slabs), dim3(256), 0, s,
                                   own, h->operand, h->tile_counters, dtype_of(h->desc), operand_scale(h->desc));
    if (e != cudaSuccess) return e;
    // Units are (batch, head pair, tile); the same number of CTAs on every (batch, head pair) where that
    // keeps at least four fifths of the SMs busy, so that the CTAs of a token's head pairs walk through
    // X in step and share its tiles in L2.
    const long long groups = static_cast<long long>(h->desc.B) * head_pairs(h->desc.H);
    const long long W = groups * p.tiles_apply;
    long long G = h->sm_count;
    const long long aligned = (G / groups) * groups;
    if (aligned * 5 >= G * 4) G = aligned;
    if (G > W) G = W;
    e = launch_chained(producer_apply_kernel<KIND>, dim3(static_cast<unsigned>(G)), dim3(ProdApplyCfg::THREADS),
                       ProdApplyCfg::SMEM_BYTES, s, mx, mwq, mt, my, h->operand, h->status, pa, p.tiles_apply,
                       W, apply_scales(h->desc));
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

// T = LeakyReLU(LayerNorm(X W_1 + b_1; gamma, beta)) into `t` [B, N, C].
template <int KIND>
cudaError_t launch_branch_x(const linfusion_attn* h, const void* x, const void* w_1, const void* b_1, const void* gamma,
                            const void* beta, float ln_eps, float slope, void* t, cudaStream_t s)
{
    const int C = h->desc.H * kStreamD, N = h->desc.N, B = h->desc.B;
    CUtensorMap mx, mw, mu;
    if (!encode_x_map(&mx, x, h->desc) || !encode_w_pair_map(&mw, w_1, C, h->desc.H, ProdHiddenCfg::NB_COLS / 64) ||
        !encode_x_map(&mu, t, h->desc))
        return cudaErrorInvalidValue;
    const int tiles = (N + ProdHiddenCfg::TILE - 1) / ProdHiddenCfg::TILE;
    const long long W = static_cast<long long>(B) * tiles;
    const int G = static_cast<int>(W < h->sm_count ? W : h->sm_count);
    cudaError_t e = launch_chained(producer_hidden_kernel<KIND>, dim3(G), dim3(ProdHiddenCfg::THREADS),
                                   ProdHiddenCfg::SMEM_BYTES, s, mx, mw, mu, static_cast<const __nv_bfloat16*>(b_1),
                                   h->x_stats, h->status, N, C, tiles, W, ln_eps);
    if (e != cudaSuccess) return e;
    const long long rows = static_cast<long long>(B) * N, total = rows * (C / 8);
    long long blocks = (total + 255) / 256;
    if (blocks > 8ll * 148 * 8) blocks = 8ll * 148 * 8;
    e = launch_chained(producer_norm_kernel<KIND>, dim3(static_cast<unsigned>(blocks)), dim3(256), 0, s,
                       static_cast<__nv_bfloat16*>(t), static_cast<const float*>(h->x_stats),
                       static_cast<const __nv_bfloat16*>(gamma), static_cast<const __nv_bfloat16*>(beta), rows, C, slope);
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Row statistics buffer of the branches' LayerNorm, on first use.
linfusion_status_t ensure_x_stats(linfusion_attn* h)
{
    if (h->x_stats != nullptr) return LINFUSION_OK;
    void* p = nullptr;
    if (cudaMalloc(&p, static_cast<size_t>(h->desc.B) * h->desc.N * 2 * sizeof(float)) != cudaSuccess) {
        cudaGetLastError();
        return LINFUSION_ERR_ALLOC;
    }
    h->x_stats = static_cast<float*>(p);
    return LINFUSION_OK;
}

}  // namespace

extern "C" linfusion_status_t linfusion_attn_branch_x(linfusion_attn_t* h, const void* x, const void* w_1,
                                                      const void* b_1, const void* gamma, const void* beta,
                                                      float ln_eps, float leaky_slope, void* t_out,
                                                      void* cuda_stream)
{
    if (h == nullptr || x == nullptr || w_1 == nullptr || gamma == nullptr || beta == nullptr || t_out == nullptr)
        return LINFUSION_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(w_1) || !aligned16(gamma) || !aligned16(beta) || !aligned16(t_out) ||
        (reinterpret_cast<uintptr_t>(b_1) & 1u) != 0)
        return LINFUSION_ERR_INVALID_ARG;
    if (!std::isfinite(ln_eps) || ln_eps < 0.0f || !std::isfinite(leaky_slope)) return LINFUSION_ERR_INVALID_ARG;
    if (!takes_x(h)) return LINFUSION_ERR_UNSUPPORTED;
    if (h->desc.H * kStreamD > ProdHiddenCfg::MAX_C) return LINFUSION_ERR_UNSUPPORTED;
    const uintptr_t px = reinterpret_cast<uintptr_t>(x), pt = reinterpret_cast<uintptr_t>(t_out);
    const size_t bytes = bytes_vy(h->desc);
    if (px < pt + bytes && pt < px + bytes) return LINFUSION_ERR_INVALID_ARG;
    DeviceGuard guard(h->desc.device);
    if (!guard.ok) return LINFUSION_ERR_CUDA;
    linfusion_status_t st = ensure_x_stats(h);
    if (st != LINFUSION_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaErrorInvalidValue;
#define LF_K(KV) e = launch_branch_x<KV>(h, x, w_1, b_1, gamma, beta, ln_eps, leaky_slope, t_out, s)
    LF_DISPATCH_KIND(kind_of(h->desc), LF_K)
#undef LF_K
    h->last_stream = s;
    if (e != cudaSuccess) {
        cudaGetLastError();
        return LINFUSION_ERR_CUDA;
    }
    return LINFUSION_OK;
}

extern "C" linfusion_status_t linfusion_attn_forward_x(linfusion_attn_t* h, const void* x,
                                                       const linfusion_module_weights_t* w, void* y,
                                                       void* cuda_stream)
{
    if (h == nullptr || x == nullptr || w == nullptr || y == nullptr) return LINFUSION_ERR_INVALID_ARG;
    if (w->q.w_lin == nullptr || w->k.w_lin == nullptr || w->w_v == nullptr) return LINFUSION_ERR_INVALID_ARG;
    if (!takes_x(h)) return LINFUSION_ERR_UNSUPPORTED;
    const linfusion_mlp_weights_t* br[2] = {&w->q, &w->k};
    const void* t[2] = {nullptr, nullptr};
    for (int i = 0; i < 2; ++i) {
        if (br[i]->w_1 == nullptr) continue;  // the branch is absent: it contributes nothing
        if (h->x_t[i] == nullptr) {
            DeviceGuard guard(h->desc.device);
            if (!guard.ok) return LINFUSION_ERR_CUDA;
            if (cudaMalloc(&h->x_t[i], bytes_vy(h->desc)) != cudaSuccess) {
                cudaGetLastError();
                h->x_t[i] = nullptr;
                return LINFUSION_ERR_ALLOC;
            }
        }
        linfusion_status_t st = linfusion_attn_branch_x(h, x, br[i]->w_1, br[i]->b_1, br[i]->gamma, br[i]->beta,
                                                        w->ln_eps, w->leaky_slope, h->x_t[i], cuda_stream);
        if (st != LINFUSION_OK) return st;
        t[i] = h->x_t[i];
    }
    linfusion_status_t st = linfusion_attn_state_x(h, x, w->k.w_lin, w->w_v, t[1], cuda_stream);
    if (st != LINFUSION_OK) return st;
    return linfusion_attn_apply_x(h, x, w->q.w_lin, t[0], y, cuda_stream);
}

extern "C" linfusion_status_t linfusion_attn_apply_x(linfusion_attn_t* h, const void* x, const void* w_q,
                                                     const void* t_q, void* y, void* cuda_stream)
{
    if (h == nullptr || x == nullptr || w_q == nullptr || y == nullptr) return LINFUSION_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(w_q) || !aligned16(t_q) || !aligned16(y)) return LINFUSION_ERR_INVALID_ARG;
    if (!takes_x(h)) return LINFUSION_ERR_UNSUPPORTED;
    const uintptr_t px = reinterpret_cast<uintptr_t>(x), py = reinterpret_cast<uintptr_t>(y);
    const size_t bytes = bytes_vy(h->desc);
    if (px < py + bytes && py < px + bytes) return LINFUSION_ERR_INVALID_ARG;
    DeviceGuard guard(h->desc.device);
    if (!guard.ok) return LINFUSION_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaErrorInvalidValue;
#define LF_K(KV) e = launch_apply_x<KV>(h, x, w_q, t_q, y, s)
    LF_DISPATCH_KIND(kind_of(h->desc), LF_K)
#undef LF_K
    h->last_stream = s;
    if (e != cudaSuccess) {
        cudaGetLastError();
        return LINFUSION_ERR_CUDA;
    }
    return LINFUSION_OK;
}

extern "C" linfusion_status_t linfusion_attn_state_x(linfusion_attn_t* h, const void* x, const void* w_k,
                                                     const void* w_v, const void* t_k, void* cuda_stream)
{
    if (h == nullptr || x == nullptr || w_k == nullptr || w_v == nullptr) return LINFUSION_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(w_k) || !aligned16(w_v) || !aligned16(t_k)) return LINFUSION_ERR_INVALID_ARG;
    if (!takes_x(h)) return LINFUSION_ERR_UNSUPPORTED;
    DeviceGuard guard(h->desc.device);
    if (!guard.ok) return LINFUSION_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaErrorInvalidValue;
#define LF_K(KV) e = launch_state_x<KV>(h, x, w_k, w_v, t_k, s)
    LF_DISPATCH_KIND(kind_of(h->desc), LF_K)
#undef LF_K
    h->last_stream = s;
    if (e != cudaSuccess) {
        cudaGetLastError();
        return LINFUSION_ERR_CUDA;
    }
    return LINFUSION_OK;
}


// ---------------------------------------------------------------------------------------------
// The bounds-checked debugging build (see lf_in_bounds() in common.cuh).
// ---------------------------------------------------------------------------------------------
extern "C" int32_t linfusion_attn_checked_build(void)
{
#ifdef LF_CHECKED
    return 1;
#else
    return 0;
#endif
}

extern "C" linfusion_status_t linfusion_attn_checked_shrink_y(size_t bytes)
{
#ifdef LF_CHECKED
    g_checked_shrink_y.store(bytes);
    return LINFUSION_OK;
#else
    (void)bytes;
    return LINFUSION_ERR_UNSUPPORTED;
#endif
}

extern "C" linfusion_status_t linfusion_attn_checked_violations(int32_t device, uint32_t* count, int32_t reset)
{
    if (count == nullptr || device < 0) return LINFUSION_ERR_INVALID_ARG;
#ifdef LF_CHECKED
    DeviceGuard guard(device);
    if (!guard.ok) return LINFUSION_ERR_CUDA;
    unsigned int c = 0;
    if (cudaDeviceSynchronize() != cudaSuccess ||
        cudaMemcpyFromSymbol(&c, g_checked_violations, sizeof(c)) != cudaSuccess) {
        cudaGetLastError();
        return LINFUSION_ERR_CUDA;
    }
    *count = c;
    if (reset != 0) {
        c = 0;
        if (cudaMemcpyToSymbol(g_checked_violations, &c, sizeof(c)) != cudaSuccess) {
            cudaGetLastError();
            return LINFUSION_ERR_CUDA;
        }
    }
    return LINFUSION_OK;
#else
    (void)reset;
    *count = 0;
    return LINFUSION_ERR_UNSUPPORTED;
#endif
}
