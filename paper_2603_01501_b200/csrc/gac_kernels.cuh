// Device code of the GAC hot path for sm_100a: chunk descriptors, element
// access for the supported element-type pairs, the fused triple reduction with
// its fixed-order second stage and decision, the in-place projection with state
// refresh, and the projection fused with AdamW.  Included by gac.cu only; the
// host side of the C ABI lives there.
#pragma once

#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include <type_traits>

#include "gac.h"

namespace {

#ifndef GAC_CHUNK
#define GAC_CHUNK 16384
#endif
// load flavour: 0 plain ld.global, 1 streaming (ld.global.cs), 2 read-only path (ld.global.nc)
#ifndef GAC_LD_STATS
#define GAC_LD_STATS 0
#endif
#ifndef GAC_LD_PROJECT
#define GAC_LD_PROJECT 0
#endif
#ifndef GAC_ST      // 0 plain st.global, 1 streaming (st.global.cs), 2 write-through (st.global.wt)
#define GAC_ST 1
#endif
#ifndef GAC_PHASE_BARRIER   // 1: the fused AdamW pass keeps the warps of a CTA in step (see phase_barrier)
#define GAC_PHASE_BARRIER 1
#endif
constexpr int kDefaultChunk = GAC_CHUNK; // elements per chunk
constexpr int kMaxCtasPerSm = 16;

constexpr uint32_t kChunkAligned = 1u;  // both bases 16-byte aligned: vector path

struct __align__(16) Chunk {
    uint64_t g;      // device address of the chunk's first g element
    uint64_t d;      // device address of the chunk's first d element
    uint32_t n;      // elements in the chunk (<= chunk_elems)
    uint32_t flags;
    uint64_t pad;
};
static_assert(sizeof(Chunk) == 32, "chunk descriptors are read as two 16-byte words");

// Hyper-parameters as the kernels see them.
struct DevHP {
    double c_low, c_high, eps, beta, alpha_fixed;
    int mode, state_mode, zero_on_violation, first_step;
    unsigned long long step;
    unsigned staleness;
    int decide;      // 0: only publish the three sums (sharded form)
    double clip_max, clip_eps;
    int swapped;     // exchange mode: 1 when the table's d addresses hold this step's gradient
    // peer exchange of the three sums (sharded form without a collective library): 0 ranks = off
    unsigned xchg_world, xchg_rank;
    const unsigned long long *xchg_peers;   // device table: address of every rank's slot array, as seen from this GPU
};

// One rank's contribution to one step, as it lies in a slot array: 32 bytes, the flag last.
struct __align__(32) PeerSlot {
    double dot, gg, dd;
    unsigned long long step;   // Algorithm 1's t for which the three numbers hold; 0 = never written
};
// A slot array holds two sets of `world` slots, used by odd and even steps in turn: a rank can
// be at most one step ahead of a peer that has not yet read the previous step's slots.
__device__ __forceinline__ size_t peer_slot_index(unsigned long long step, unsigned world, unsigned rank) {
    return size_t(step & 1ull) * world + rank;
}

struct F4 {
    float x, y, z, w;
};

// ---------------------------------------------------------------- element I/O

template <int LD, typename V>
__device__ __forceinline__ V ld_vec(const V *p) {
    if (LD == 1) return __ldcs(p);
    if (LD == 2) return __ldg(p);
    return *p;
}
template <typename V>
__device__ __forceinline__ void st_vec(V *p, V v) {
#if GAC_ST == 1
    __stcs(p, v);
#elif GAC_ST == 2
    __stwt(p, v);
#else
    *p = v;
#endif
}

template <typename GT>
struct Elem;

// Raw = four elements as they lie in memory (what a thread keeps in registers
// while loads are in flight); unpack/pack convert to and from four binary32 values.
template <>
struct Elem<float> {
    using Raw = float4;
    static __device__ __forceinline__ Raw zero() { return make_float4(0.f, 0.f, 0.f, 0.f); }
    template <int LD>
    static __device__ __forceinline__ Raw load_raw(const void *base, uint32_t v) {
        return ld_vec<LD>(reinterpret_cast<const float4 *>(base) + v);
    }
    static __device__ __forceinline__ void store_raw(void *base, uint32_t v, Raw r) {
        st_vec(reinterpret_cast<float4 *>(base) + v, r);
    }
    static __device__ __forceinline__ F4 unpack(Raw t) { return F4{t.x, t.y, t.z, t.w}; }
    static __device__ __forceinline__ Raw pack(F4 a) { return make_float4(a.x, a.y, a.z, a.w); }
    template <int LD>
    static __device__ __forceinline__ F4 load4(const void *base, uint32_t v) {
        return unpack(load_raw<LD>(base, v));
    }
    static __device__ __forceinline__ void store4(void *base, uint32_t v, F4 a) { store_raw(base, v, pack(a)); }
    static __device__ __forceinline__ float load1(const void *base, uint32_t i) {
        return reinterpret_cast<const float *>(base)[i];
    }
    static __device__ __forceinline__ void store1(void *base, uint32_t i, float a) {
        reinterpret_cast<float *>(base)[i] = a;
    }
};

// bfloat16 = the upper 16 bits of a binary32 pattern.
struct bf16_t {
    uint16_t bits;
};

// Element-type pairs (gradient, stored direction).  A kernel's type parameter
// is one of these tags: float = (binary32, binary32), bf16_t = (bfloat16,
// binary32), bf16_pair_t = (bfloat16, bfloat16): a snapshot of half the size.
struct bf16_pair_t {};
template <typename P>
struct PairOf {
    using G = P;
    using D = float;
};
template <>
struct PairOf<bf16_pair_t> {
    using G = bf16_t;
    using D = bf16_t;
};
template <typename P>
using GOf = typename PairOf<P>::G;
template <typename P>
using DOf = typename PairOf<P>::D;

// Launch geometry.  All kernels here are bound by HBM, and on B200 their speed
// depends on how many bytes each SM keeps in flight: too few starve the memory
// system, too many make the reads and write-backs of many chunks collide in
// DRAM (the read+write passes are fastest with ONE CTA per SM and 48-64 KB of
// reads in flight).  The table holds the measured best per element-type pair:
//   T     threads per CTA
//   U     four-element vectors in flight per thread and operand
//   UK    the same for a step that leaves g alone (only g read, only d written)
//   C     resident CTAs per SM the grid is sized for (0 = all that fit)
//   MINB  occupancy asked of the compiler through __launch_bounds__
//   BAR   projection: __syncthreads() after a batch's loads (bit 0) and/or after its stores (bit 1)
//   PF    projection: 1 = the next chunk's descriptor is fetched while the current chunk is worked on
// A build that times variants substitutes its own table with
// -DGAC_GEOMETRY_HEADER='"file.h"'.
template <typename P>
struct StatsGeom;   // fused triple reduction
template <typename P>
struct ProjGeom;    // projection + state refresh
template <typename P>
struct ExchGeom;    // projection in exchange mode (two reads, one write per element)
template <typename P>
struct AdamGeom;    // projection fused with AdamW
#ifdef GAC_GEOMETRY_HEADER
#include GAC_GEOMETRY_HEADER
#else
template <> struct StatsGeom<float>       { static constexpr int T = 256, U = 8, C = 0, MINB = 4; };
template <> struct StatsGeom<bf16_t>      { static constexpr int T = 256, U = 8, C = 0, MINB = 4; };
template <> struct StatsGeom<bf16_pair_t> { static constexpr int T = 256, U = 8, C = 0, MINB = 4; };
template <> struct ProjGeom<float>        { static constexpr int T = 256, U = 8, UK = 16, C = 1, MINB = 1, BAR = 2, PF = 1; };
template <> struct ProjGeom<bf16_t>       { static constexpr int T = 512, U = 4, UK = 8, C = 1, MINB = 1, BAR = 1, PF = 1; };
template <> struct ProjGeom<bf16_pair_t>  { static constexpr int T = 512, U = 8, UK = 8, C = 1, MINB = 1, BAR = 1, PF = 0; };
template <> struct ExchGeom<float>        { static constexpr int T = 512, U = 4, UK = 8, C = 1, MINB = 1, BAR = 1, PF = 0; };
template <> struct ExchGeom<bf16_t>       { static constexpr int T = 512, U = 4, UK = 8, C = 1, MINB = 1, BAR = 1, PF = 0; };   // pair not served
template <> struct ExchGeom<bf16_pair_t>  { static constexpr int T = 512, U = 4, UK = 8, C = 2, MINB = 2, BAR = 1, PF = 0; };
// AdamGeom: T threads for the plain rule (beta = 1, no clipping), TG for the general one, C CTAs per SM.
// float32 gradients: one CTA of 1024 threads (a 64 KB chunk is exactly four batches); bfloat16
// gradients move fewer bytes per batch, and two CTAs of 512 threads, each in step with itself
// only, overlap one CTA's arithmetic with the other's memory phase (+5-7 % there, -3 % for float32).
template <> struct AdamGeom<float>        { static constexpr int T = 1024, TG = 1024, U = 1, C = 1; };
template <> struct AdamGeom<bf16_t>       { static constexpr int T = 512, TG = 512, U = 1, C = 2; };
template <> struct AdamGeom<bf16_pair_t>  { static constexpr int T = 512, TG = 512, U = 1, C = 2; };
#endif

__device__ __forceinline__ uint32_t pack_bf16x2_rn(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

template <>
struct Elem<bf16_t> {
    using Raw = uint2;   // four bfloat16 values stay packed (two registers) until they are used
    static __device__ __forceinline__ Raw zero() { return make_uint2(0u, 0u); }
    template <int LD>
    static __device__ __forceinline__ Raw load_raw(const void *base, uint32_t v) {
        return ld_vec<LD>(reinterpret_cast<const uint2 *>(base) + v);
    }
    static __device__ __forceinline__ void store_raw(void *base, uint32_t v, Raw r) {
        st_vec(reinterpret_cast<uint2 *>(base) + v, r);
    }
    static __device__ __forceinline__ F4 unpack(Raw t) {
        return F4{__uint_as_float(t.x << 16), __uint_as_float(t.x & 0xFFFF0000u),
                  __uint_as_float(t.y << 16), __uint_as_float(t.y & 0xFFFF0000u)};
    }
    static __device__ __forceinline__ Raw pack(F4 a) {
        return make_uint2(pack_bf16x2_rn(a.x, a.y), pack_bf16x2_rn(a.z, a.w));
    }
    template <int LD>
    static __device__ __forceinline__ F4 load4(const void *base, uint32_t v) {
        return unpack(load_raw<LD>(base, v));
    }
    static __device__ __forceinline__ void store4(void *base, uint32_t v, F4 a) { store_raw(base, v, pack(a)); }
    static __device__ __forceinline__ float load1(const void *base, uint32_t i) {
        return __uint_as_float(uint32_t(reinterpret_cast<const uint16_t *>(base)[i]) << 16);
    }
    static __device__ __forceinline__ void store1(void *base, uint32_t i, float a) {
        reinterpret_cast<uint16_t *>(base)[i] = uint16_t(pack_bf16x2_rn(a, 0.0f) & 0xFFFFu);
    }
};

// swapped (exchange mode): the two address columns of the table trade roles.
__device__ __forceinline__ Chunk load_chunk(const Chunk *table, uint32_t c, int swapped = 0) {
    const uint4 *p = reinterpret_cast<const uint4 *>(table + c);
    uint4 a = __ldg(p), b = __ldg(p + 1);
    Chunk ch;
    ch.g = (uint64_t(a.y) << 32) | a.x;
    ch.d = (uint64_t(a.w) << 32) | a.z;
    if (swapped) {
        const uint64_t t = ch.g;
        ch.g = ch.d;
        ch.d = t;
    }
    ch.n = b.x;
    ch.flags = b.y;
    ch.pad = 0;
    return ch;
}

// 16 bytes global -> shared without passing through registers; completion is awaited with
// cp_async_wait_all() by the thread that issued the copies.
__device__ __forceinline__ void cp_async16(void *smem, const void *gmem) {
    const unsigned sa = static_cast<unsigned>(__cvta_generic_to_shared(smem));
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(sa), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// Keeps the warps of a CTA in step in a pass that reads AND writes: every warp issues its
// batch of loads, then every warp stores its results, and only then does the next batch of
// loads start.  Without it the warps drift apart and each SM sends DRAM an even mix of reads
// and writes.  Measured on B200, fused AdamW pass on the 1.5 B float32 list (5 read + 4 write
// streams, 32 warps per SM): 5.96 TB/s without, 6.36 TB/s with this barrier, 6.60 TB/s once
// the chunk descriptors are also fetched ahead (adamw_walk), so that the CTA does not stall
// as one at every chunk boundary.
// Every thread of the CTA reaches it: the loops around it have CTA-uniform trip counts.
__device__ __forceinline__ void phase_barrier() {
#if GAC_PHASE_BARRIER
    __syncthreads();
#endif
}

// ------------------------------------------------------- decision (O(1) work)

// Global-norm clipping folded into the update (Table 2: "Gradient clipping
// True").  The squared norm of what a step sends on follows from the three
// sums alone: |beta g + k d|^2 = beta^2 <g,g> + 2 beta k <g,d> + k^2 <d,d> in the
// projection regime (k = the binary32 coefficient actually applied), <g,g> in
// the safe regime; a skipped step sends nothing on.  Factor as in the usual
// global-norm clip: min(1, max_norm / (norm + clip_eps)).
__device__ __forceinline__ double clip_factor(int regime, double dot, double gg, double dd, double beta,
                                              double k, double clip_max, double clip_eps, double *norm_out) {
    double n2 = gg;
    if (regime == GAC_REGIME_PROJECT)
        n2 = __dadd_rn(__dadd_rn(__dmul_rn(__dmul_rn(beta, beta), gg),
                                 __dmul_rn(__dmul_rn(2.0 * beta, k), dot)),
                       __dmul_rn(__dmul_rn(k, k), dd));
    const double norm = __dsqrt_rn(fmax(n2, 0.0));
    *norm_out = norm;
    if (!(clip_max > 0.0) || regime == GAC_REGIME_VIOLATION) return 1.0;
    const double f = __ddiv_rn(clip_max, __dadd_rn(norm, clip_eps));
    return f < 1.0 ? f : 1.0;
}

// Cosine with eps outside the root (App. A.1), the inclusive branches of
// Algorithm 1, alpha = c_low/|c| (Eq. 5) or the caller's gain (Eq. 3), and the
// multiplier of d in the rank-one form of App. A.2.
__device__ void take_regime(double dot, double gg, double dd, const DevHP &hp, gac_result *r) {
    if (gg == 0.0 || dd == 0.0) {   // zero reference: u = 0, projector = identity
        r->cos = 0.0;
        r->regime = GAC_REGIME_SAFE;
        r->clip_scale = clip_factor(r->regime, dot, gg, dd, hp.beta, 0.0, hp.clip_max, hp.clip_eps, &r->out_norm);
        return;
    }
    double c = __ddiv_rn(dot, __dadd_rn(__dsqrt_rn(__dmul_rn(gg, dd)), hp.eps));
    double ac = fabs(c);
    r->cos = c;
    if (hp.mode == GAC_MODE_FIXED) {
        r->regime = GAC_REGIME_PROJECT;
        r->alpha = hp.alpha_fixed;
    } else if (ac <= hp.c_low) {
        r->regime = GAC_REGIME_SAFE;
        r->clip_scale = clip_factor(r->regime, dot, gg, dd, hp.beta, 0.0, hp.clip_max, hp.clip_eps, &r->out_norm);
        return;
    } else if (ac >= hp.c_high) {
        r->regime = GAC_REGIME_VIOLATION;
        return;
    } else {
        r->regime = GAC_REGIME_PROJECT;
        r->alpha = __ddiv_rn(hp.c_low, ac);
    }
    double k = __ddiv_rn(__dmul_rn(__dadd_rn(r->alpha, -hp.beta), dot), dd);
    r->coef64 = k;
    r->coef = __double2float_rn(k);
    r->clip_scale = clip_factor(r->regime, dot, gg, dd, hp.beta, double(r->coef), hp.clip_max, hp.clip_eps,
                                &r->out_norm);
}

// The record of one step: the three sums, the zero reference of the first step
// (Algorithm 1: g_0 = 0), the non-finite reading, the regime and gains, and --
// for exchange mode -- which buffer set holds what the step sends on.
__device__ void take_decision(double dot, double gg, double dd, const DevHP &hp, bool zero_reference,
                              gac_result *r) {
    if (zero_reference) {   // Algorithm 1: g_0 = 0
        dot = 0.0;
        dd = 0.0;
    }
    r->dot = dot;
    r->gg = gg;
    r->dd = dd;
    r->alpha = 1.0;
    r->coef64 = 0.0;
    r->coef = 0.0f;
    r->out_norm = 0.0;
    r->clip_scale = 1.0;
    r->staleness = hp.staleness;
    r->step = hp.step;
    r->g_set = uint32_t(hp.swapped);
    r->out_set = r->g_set;
    r->timed_out = 0u;   // ref_lost is not touched here: the pass that closes the step owns it
    r->nonfinite = !(isfinite(dot) && isfinite(gg) && isfinite(dd));
    if (r->nonfinite) {
        r->cos = __longlong_as_double(0x7FF8000000000000LL);
        r->regime = GAC_REGIME_VIOLATION;
        return;
    }
    take_regime(dot, gg, dd, hp, r);
    if (hp.state_mode == GAC_STATE_EXCHANGE) {
        // exchange mode writes whatever differs from g into the buffers that held d
        const bool writes = r->regime == GAC_REGIME_PROJECT ||
                            (r->regime == GAC_REGIME_VIOLATION && hp.zero_on_violation) ||
                            (r->regime == GAC_REGIME_SAFE && r->clip_scale != 1.0);
        if (writes) r->out_set = r->g_set ^ 1u;
    }
}

// ------------------------------------------------------------- stats kernel

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// Sums (a, b, c) over the CTA in a fixed order; the result is valid in thread 0.
template <int T>
__device__ __forceinline__ void block_sum3(double &a, double &b, double &c, double (*sm)[3]) {
    a = warp_sum(a);
    b = warp_sum(b);
    c = warp_sum(c);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) {
        sm[warp][0] = a;
        sm[warp][1] = b;
        sm[warp][2] = c;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        a = sm[0][0];
        b = sm[0][1];
        c = sm[0][2];
        for (int w = 1; w < T / 32; ++w) {
            a += sm[w][0];
            b += sm[w][1];
            c += sm[w][2];
        }
    }
    __syncthreads();
}

template <typename GT, bool READ_D>
__device__ __forceinline__ void stats_chunk(const Chunk &ch, double &a_dot, double &a_gg,
                                            double &a_dd) {
    const void *g = reinterpret_cast<const void *>(ch.g);
    const void *d = reinterpret_cast<const void *>(ch.d);
    const uint32_t tid = threadIdx.x;
    constexpr int T = StatsGeom<GT>::T, U = StatsGeom<GT>::U;
    if (ch.flags & kChunkAligned) {
        const uint32_t nvec = ch.n >> 2;
        for (uint32_t base = 0; base < nvec; base += T * U) {
            typename Elem<GOf<GT>>::Raw gr[U];
            typename Elem<DOf<GT>>::Raw dr[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t v = base + u * T + tid;
                gr[u] = Elem<GOf<GT>>::zero();
                dr[u] = Elem<DOf<GT>>::zero();
                if (v < nvec) {
                    gr[u] = Elem<GOf<GT>>::template load_raw<GAC_LD_STATS>(g, v);
                    if (READ_D) dr[u] = Elem<DOf<GT>>::template load_raw<GAC_LD_STATS>(d, v);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const F4 gq = Elem<GOf<GT>>::unpack(gr[u]), dq = Elem<DOf<GT>>::unpack(dr[u]);
                const float ge[4] = {gq.x, gq.y, gq.z, gq.w};
                const float de[4] = {dq.x, dq.y, dq.z, dq.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const double x = double(ge[e]);
                    a_gg = fma(x, x, a_gg);
                    if (READ_D) {
                        const double y = double(de[e]);
                        a_dot = fma(x, y, a_dot);
                        a_dd = fma(y, y, a_dd);
                    }
                }
            }
        }
        const uint32_t done = nvec << 2;
        if (tid < ch.n - done) {   // ragged tail of a tensor: < 4 elements
            const double x = double(Elem<GOf<GT>>::load1(g, done + tid));
            a_gg = fma(x, x, a_gg);
            if (READ_D) {
                const double y = double(Elem<DOf<GT>>::load1(d, done + tid));
                a_dot = fma(x, y, a_dot);
                a_dd = fma(y, y, a_dd);
            }
        }
    } else {   // a base that is not 16-byte aligned: element-wise, still coalesced
        for (uint32_t i = tid; i < ch.n; i += T) {
            const double x = double(Elem<GOf<GT>>::load1(g, i));
            a_gg = fma(x, x, a_gg);
            if (READ_D) {
                const double y = double(Elem<DOf<GT>>::load1(d, i));
                a_dot = fma(x, y, a_dot);
                a_dd = fma(y, y, a_dd);
            }
        }
    }
}

// partials: gridDim.x x 3 doubles, each slot written once per launch.
// ticket: zero on entry; the last CTA to arrive reduces the slots in index
// order, publishes the result and puts the ticket back to zero.  No CTA waits.
template <typename GT>
__global__ void __launch_bounds__(StatsGeom<GT>::T, StatsGeom<GT>::MINB)
gac_stats_kernel(const Chunk *__restrict__ chunks, uint32_t n_chunks, double *partials,
                 unsigned *ticket, gac_result *rec, double *sums_out, DevHP hp) {
    constexpr int T = StatsGeom<GT>::T;
    __shared__ double sm[T / 32][3];
    __shared__ bool is_last;
    double a_dot = 0.0, a_gg = 0.0, a_dd = 0.0;
    // Exchange mode after a non-finite step: the stored direction is gone, the
    // step is taken against the zero reference like the first one.  Every CTA
    // reads the flag here, before the last CTA can rewrite the record.
    const bool zero_reference = hp.first_step || (hp.state_mode == GAC_STATE_EXCHANGE && rec->ref_lost);
    if (zero_reference) {
        for (uint32_t c = blockIdx.x; c < n_chunks; c += gridDim.x)
            stats_chunk<GT, false>(load_chunk(chunks, c, hp.swapped), a_dot, a_gg, a_dd);
    } else {
        for (uint32_t c = blockIdx.x; c < n_chunks; c += gridDim.x)
            stats_chunk<GT, true>(load_chunk(chunks, c, hp.swapped), a_dot, a_gg, a_dd);
    }
    block_sum3<T>(a_dot, a_gg, a_dd, sm);
    if (threadIdx.x == 0) {
        double *slot = partials + 3 * size_t(blockIdx.x);
        slot[0] = a_dot;
        slot[1] = a_gg;
        slot[2] = a_dd;
        __threadfence();
        const unsigned t = atomicAdd(ticket, 1u);
        is_last = (t == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // second stage: thread t adds slots t, t+T, t+2T, ... in that order, then the
    // same fixed tree as above
    double s0 = 0.0, s1 = 0.0, s2 = 0.0;
    for (uint32_t b = threadIdx.x; b < gridDim.x; b += T) {
        const double *slot = partials + 3 * size_t(b);
        s0 += __ldcg(slot + 0);
        s1 += __ldcg(slot + 1);
        s2 += __ldcg(slot + 2);
    }
    block_sum3<T>(s0, s1, s2, sm);
    if (threadIdx.x == 0) {
        *ticket = 0u;
        if (sums_out) {
            sums_out[0] = zero_reference ? 0.0 : s0;
            sums_out[1] = s1;
            sums_out[2] = zero_reference ? 0.0 : s2;
        }
        if (hp.xchg_world) {
            // App. A.1's one collective, done here: this rank's three numbers go into its slot of
            // EVERY rank's slot array (its own included) with plain stores, then -- after a
            // system-wide fence -- the step number that marks them valid.  Nothing is waited for.
            const size_t idx = peer_slot_index(hp.step, hp.xchg_world, hp.xchg_rank);
            for (unsigned r = 0; r < hp.xchg_world; ++r) {
                volatile PeerSlot *slot = reinterpret_cast<volatile PeerSlot *>(hp.xchg_peers[r]) + idx;
                slot->dot = zero_reference ? 0.0 : s0;
                slot->gg = s1;
                slot->dd = zero_reference ? 0.0 : s2;
            }
            __threadfence_system();
            for (unsigned r = 0; r < hp.xchg_world; ++r) {
                volatile PeerSlot *slot = reinterpret_cast<volatile PeerSlot *>(hp.xchg_peers[r]) + idx;
                slot->step = hp.step;
            }
        }
        if (hp.decide) take_decision(s0, s1, s2, hp, zero_reference, rec);
    }
}

__global__ void gac_decide_kernel(const double *sums_in, gac_result *rec, DevHP hp) {
    if (threadIdx.x == 0 && blockIdx.x == 0)
        take_decision(sums_in[0], sums_in[1], sums_in[2], hp, hp.first_step != 0, rec);
}

__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Second half of the peer exchange: thread r waits until rank r's slot of THIS rank's array
// carries the step number, then thread 0 adds the slots in rank order -- every rank performs
// the same additions in the same order, so all hold bit-identical sums -- and takes the
// decision.  The wait is bounded twice (wall time and iterations); when it runs out the record
// is marked timed_out, no decision is taken, and the pass that follows writes nothing.
constexpr int kExchangeThreads = 128;
__global__ void __launch_bounds__(kExchangeThreads, 1)
gac_decide_exchange_kernel(const PeerSlot *slots, gac_result *rec, DevHP hp, unsigned long long timeout_ns) {
    __shared__ int missing;
    if (threadIdx.x == 0) missing = 0;
    __syncthreads();
    const PeerSlot *mine = slots + size_t(hp.step & 1ull) * hp.xchg_world;
    for (unsigned r = threadIdx.x; r < hp.xchg_world; r += kExchangeThreads) {
        const volatile unsigned long long *flag = &mine[r].step;
        const unsigned long long t0 = global_ns();
        const unsigned long long max_polls = timeout_ns / 64ull + 1024ull;   // second bound, should the timer stand still
        bool there = false;
        for (unsigned long long poll = 0; poll < max_polls; ++poll) {
            if (*flag == hp.step) {
                there = true;
                break;
            }
            if (global_ns() - t0 > timeout_ns) break;
            __nanosleep(256);
        }
        if (!there) atomicAdd(&missing, 1);
    }
    __syncthreads();
    if (threadIdx.x != 0) return;
    if (missing) {
        rec->timed_out = 1u;
        rec->step = hp.step;
        return;
    }
    __threadfence_system();   // the flags were seen: now the numbers they guard
    double s0 = 0.0, s1 = 0.0, s2 = 0.0;
    for (unsigned r = 0; r < hp.xchg_world; ++r) {
        const volatile PeerSlot *slot = mine + r;
        s0 += slot->dot;
        s1 += slot->gg;
        s2 += slot->dd;
    }
    // the posted numbers already carry the zero reference where it applies
    take_decision(s0, s1, s2, hp, false, rec);
}

// ----------------------------------------------------------- project kernel

enum GOp { G_KEEP = 0, G_FMA = 1, G_ZERO = 2, G_SCALE = 3, G_FMA1 = 4 };   // G_FMA1: beta = 1 and no clip factor
enum DOp { D_KEEP = 0, D_RAW = 1, D_NEW = 2, D_OUT = 3 };   // D_OUT: the new g goes into d's buffer, g stays (exchange mode)

template <bool BETA1>
__device__ __forceinline__ float rank_one(float g, float d, float k, double beta, double s) {
    if (BETA1) return fmaf(k, d, g);   // beta = 1, no clipping: one rounding
    // general beta and/or an active clip factor s: binary64 (rounded product + exact product), times s
    return __double2float_rn(
        __dmul_rn(s, __dadd_rn(__dmul_rn(beta, double(g)), __dmul_rn(double(k), double(d)))));
}
__device__ __forceinline__ float scaled(float g, double s) { return __double2float_rn(__dmul_rn(s, double(g))); }

template <typename GT, int GOP, int DOP, bool BETA1, int T, int U, int BAR>
__device__ __forceinline__ void project_chunk(const Chunk &ch, float k, double beta, double s) {
    void *g = reinterpret_cast<void *>(ch.g);
    void *d = reinterpret_cast<void *>(ch.d);
    void *o = (DOP == D_OUT) ? d : g;   // where the outgoing gradient is stored
    const uint32_t tid = threadIdx.x;
    constexpr bool kReadG = (GOP == G_FMA) || (GOP == G_SCALE) || (DOP == D_RAW);
    constexpr bool kReadD = (GOP == G_FMA);
    if (ch.flags & kChunkAligned) {
        const uint32_t nvec = ch.n >> 2;
        for (uint32_t base = 0; base < nvec; base += T * U) {
            typename Elem<GOf<GT>>::Raw gr[U];
            typename Elem<DOf<GT>>::Raw dr[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t v = base + u * T + tid;
                gr[u] = Elem<GOf<GT>>::zero();
                dr[u] = Elem<DOf<GT>>::zero();
                if (v < nvec) {
                    if (kReadG) gr[u] = Elem<GOf<GT>>::template load_raw<GAC_LD_PROJECT>(g, v);
                    if (kReadD) dr[u] = Elem<DOf<GT>>::template load_raw<GAC_LD_PROJECT>(d, v);
                }
            }
            if (BAR & 1) __syncthreads();   // keeps the warps of the CTA in step (see phase_barrier)
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t v = base + u * T + tid;
                if (v >= nvec) continue;
                const F4 gq = Elem<GOf<GT>>::unpack(gr[u]);
                F4 out = gq;
                if (GOP == G_ZERO) out = F4{0.f, 0.f, 0.f, 0.f};
                if (GOP == G_FMA) {
                    const F4 dq = Elem<DOf<GT>>::unpack(dr[u]);
                    out.x = rank_one<BETA1>(gq.x, dq.x, k, beta, s);
                    out.y = rank_one<BETA1>(gq.y, dq.y, k, beta, s);
                    out.z = rank_one<BETA1>(gq.z, dq.z, k, beta, s);
                    out.w = rank_one<BETA1>(gq.w, dq.w, k, beta, s);
                }
                if (GOP == G_SCALE) out = F4{scaled(gq.x, s), scaled(gq.y, s), scaled(gq.z, s), scaled(gq.w, s)};
                if (GOP != G_KEEP) Elem<GOf<GT>>::store4(o, v, out);
                if (DOP == D_RAW) Elem<DOf<GT>>::store4(d, v, gq);
                if (DOP == D_NEW) {
                    if (GOP == G_FMA || GOP == G_SCALE) out = Elem<GOf<GT>>::template load4<GAC_LD_PROJECT>(g, v);   // the value as stored (rounded)
                    Elem<DOf<GT>>::store4(d, v, out);
                }
            }
            if (BAR & 2) __syncthreads();
        }
        const uint32_t done = nvec << 2;
        if (tid < ch.n - done) {
            const uint32_t i = done + tid;
            const float x = kReadG ? Elem<GOf<GT>>::load1(g, i) : 0.f;
            float out = (GOP == G_ZERO) ? 0.f : x;
            if (GOP == G_FMA) out = rank_one<BETA1>(x, Elem<DOf<GT>>::load1(d, i), k, beta, s);
            if (GOP == G_SCALE) out = scaled(x, s);
            if (GOP != G_KEEP) Elem<GOf<GT>>::store1(o, i, out);
            if (DOP == D_RAW) Elem<DOf<GT>>::store1(d, i, x);
            if (DOP == D_NEW) {
                if (GOP == G_FMA || GOP == G_SCALE) out = Elem<GOf<GT>>::load1(g, i);
                Elem<DOf<GT>>::store1(d, i, out);
            }
        }
    } else {
        for (uint32_t i = tid; i < ch.n; i += T) {
            const float x = kReadG ? Elem<GOf<GT>>::load1(g, i) : 0.f;
            float out = (GOP == G_ZERO) ? 0.f : x;
            if (GOP == G_FMA) out = rank_one<BETA1>(x, Elem<DOf<GT>>::load1(d, i), k, beta, s);
            if (GOP == G_SCALE) out = scaled(x, s);
            if (GOP != G_KEEP) Elem<GOf<GT>>::store1(o, i, out);
            if (DOP == D_RAW) Elem<DOf<GT>>::store1(d, i, x);
            if (DOP == D_NEW) {
                if (GOP == G_FMA || GOP == G_SCALE) out = Elem<GOf<GT>>::load1(g, i);
                Elem<DOf<GT>>::store1(d, i, out);
            }
        }
    }
}

// Geometry of the projection kernel for a state mode.
template <typename GT, int STATE>
using ProjGeomOf = typename std::conditional<STATE == GAC_STATE_EXCHANGE, ExchGeom<GT>, ProjGeom<GT>>::type;

// The descriptor of chunk c, read with loads the compiler may not move: a prefetch only helps if it
// is issued where it is written, ahead of the chunk's work.
__device__ __forceinline__ void load_chunk_words(const Chunk *table, uint32_t c, uint4 &a, uint4 &b) {
    const uint4 *p = reinterpret_cast<const uint4 *>(table + c);
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w) : "l"(p));
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w) : "l"(p + 1));
}
__device__ __forceinline__ Chunk chunk_from_words(uint4 a, uint4 b, int swapped) {
    Chunk ch;
    ch.g = (uint64_t(a.y) << 32) | a.x;
    ch.d = (uint64_t(a.w) << 32) | a.z;
    if (swapped) {
        const uint64_t t = ch.g;
        ch.g = ch.d;
        ch.d = t;
    }
    ch.n = b.x;
    ch.flags = b.y;
    ch.pad = 0;
    return ch;
}

// A CTA's walk over its chunks.  How the warps of the CTA line up decides how well DRAM is used
// (see phase_barrier), and two arrangements work on B200:
//   PF = 0  every thread reads the descriptor when it gets to the chunk; the short wait for it lets
//           the warps fall into step again at every chunk boundary (with BAR = 1 on top: +0.5-1 %);
//   PF = 1  the next descriptor is fetched while the current chunk is worked on, and barriers alone
//           keep the warps in step.  With BAR = 2 this is the fastest form for float32 pairs
//           (6.67 against 6.54 TB/s on the 1.5 B list) and the slowest for bfloat16 gradients; with
//           BAR = 1 it leaves the projection of bf16/f32 lists as it was and speeds up their steps
//           that only refresh the stored direction by 2 %.
template <typename GT, int GOP, int DOP, bool BETA1, int T, int U, int PF, int BAR>
__device__ __forceinline__ void project_walk_tu(const Chunk *chunks, uint32_t n_chunks, float k,
                                                double beta, double s, int swapped) {
    if (PF) {
        uint32_t c = blockIdx.x;
        if (c >= n_chunks) return;
        uint4 wa, wb;
        load_chunk_words(chunks, c, wa, wb);
        for (; c < n_chunks; c += gridDim.x) {
            const Chunk ch = chunk_from_words(wa, wb, swapped);
            if (c + gridDim.x < n_chunks) load_chunk_words(chunks, c + gridDim.x, wa, wb);
            project_chunk<GT, GOP, DOP, BETA1, T, U, BAR>(ch, k, beta, s);
        }
    } else {
        for (uint32_t c = blockIdx.x; c < n_chunks; c += gridDim.x)
            project_chunk<GT, GOP, DOP, BETA1, T, U, BAR>(load_chunk(chunks, c, swapped), k, beta, s);
    }
}
template <typename GT, int GOP, int DOP, bool BETA1>
__device__ __forceinline__ void project_walk(const Chunk *chunks, uint32_t n_chunks, float k,
                                             double beta, double s, int swapped) {
    using Geom = typename std::conditional<DOP == D_OUT, ExchGeom<GT>, ProjGeom<GT>>::type;
    project_walk_tu<GT, GOP, DOP, BETA1, Geom::T, Geom::U, Geom::PF, Geom::BAR>(chunks, n_chunks, k, beta, s, swapped);
}

// The regime is read from the device-resident record, so no host round trip
// separates the two passes; every CTA takes the same (uniform) branch.  What
// the host already knows (state mode, beta == 1, zero_on_violation) is fixed at
// compile time so that each instantiation holds only the loops it can reach.
template <typename GT, int STATE, bool BETA1, bool ZERO>
__global__ void __launch_bounds__((ProjGeomOf<GT, STATE>::T), (ProjGeomOf<GT, STATE>::MINB))
gac_project_kernel(const Chunk *__restrict__ chunks, uint32_t n_chunks, gac_result *rec,
                   float coef_override, int use_override, double beta, double clip_max, double clip_eps,
                   int swapped) {
    // Exchange mode: the roles swap whatever the step did, so a non-finite step loses the stored
    // direction.  The flag is written here, by the pass that closes the step (never by the
    // reduction, which may run more than once per step), and nobody reads it during this launch.
    const bool closed = rec->nonfinite || rec->timed_out;   // no decision to act on: touch nothing
    if (STATE == GAC_STATE_EXCHANGE && blockIdx.x == 0 && threadIdx.x == 0) rec->ref_lost = closed ? 1u : 0u;
    if (closed) return;
    const int regime = rec->regime;
    const float k = use_override ? coef_override : rec->coef;
    constexpr int dop = STATE == GAC_STATE_RAW ? D_RAW
                        : (STATE == GAC_STATE_PROJECTED ? D_NEW : (STATE == GAC_STATE_EXCHANGE ? D_OUT : D_KEEP));
    double s = 1.0;
    if (clip_max > 0.0) {
        // recomputed here so that it belongs to the coefficient actually applied
        double norm;
        s = clip_factor(regime, rec->dot, rec->gg, rec->dd, beta, double(k), clip_max, clip_eps, &norm);
        if (use_override && blockIdx.x == 0 && threadIdx.x == 0) {
            rec->out_norm = norm;       // nobody reads these two fields during this launch
            rec->clip_scale = s;
        }
    }
    if (regime == GAC_REGIME_PROJECT) {
        if (s != 1.0) project_walk<GT, G_FMA, dop, false>(chunks, n_chunks, k, beta, s, swapped);
        else project_walk<GT, G_FMA, dop, BETA1>(chunks, n_chunks, k, beta, 1.0, swapped);
    } else if (ZERO && regime == GAC_REGIME_VIOLATION) {
        project_walk<GT, G_ZERO, dop, true>(chunks, n_chunks, k, 1.0, 1.0, swapped);
    } else if (s != 1.0) {
        project_walk<GT, G_SCALE, dop, true>(chunks, n_chunks, k, 1.0, s, swapped);   // safe step, clipped: g'' = s g
    } else if (STATE != GAC_STATE_HOLD && STATE != GAC_STATE_EXCHANGE) {
        // d' = g, g untouched
        project_walk_tu<GT, G_KEEP, D_RAW, true, ProjGeom<GT>::T, ProjGeom<GT>::UK, ProjGeom<GT>::PF, ProjGeom<GT>::BAR>(
            chunks, n_chunks, k, 1.0, 1.0, 0);
    }
    // exchange mode, g unchanged: nothing to move -- the buffers that hold g become the stored direction
}

// ------------------------------------------------ projection fused with AdamW

struct __align__(16) OptChunk {
    uint64_t p, m, v, pad;   // device addresses of the chunk's first parameter / moment elements
};
static_assert(sizeof(OptChunk) == 32, "optimizer chunk descriptors are read as two 16-byte words");

// What the host knows of the optimizer, passed by value: kernel arguments live in the constant
// bank, where an instruction can use them as an operand without holding a register for them.
struct AdamDev {
    double lr, b1, b2, eps;
    double c1, c2, lr_wd;      // 1 - b1, 1 - b2, lr * weight_decay (computed on the host, same arithmetic)
};

// What depends on the count of applied updates, which lives on the device.
struct AdamStep {
    double step_size, inv_sqrt_bc2;   // lr / (1 - b1^t), 1 / sqrt(1 - b2^t)
    float coef;                       // the multiplier of d applied in this launch
};

// The outgoing gradient in binary64, unrounded: the moments are differences of
// nearly equal terms often enough that a binary32 g' would cost them digits.
template <int GOP>
__device__ __forceinline__ double outgoing64(float g, float d, float k, double beta, double s) {
    // beta = 1, s = 1: the product of two binary32 values is exact in binary64, so this single fused
    // operation gives the same number as the general form below
    if (GOP == G_FMA1) return fma(double(k), double(d), double(g));
    if (GOP == G_FMA)
        return __dmul_rn(s, __dadd_rn(__dmul_rn(beta, double(g)), __dmul_rn(double(k), double(d))));
    if (GOP == G_SCALE) return __dmul_rn(s, double(g));
    return double(g);
}

// One element of: g' -> AdamW, in binary64 so that p - delta stays accurate
// even where it cancels (tiny parameters).  The square root and the reciprocal
// start from the hardware's binary64 approximations (about 20 good bits, no
// conversion to binary32 and back) and take one Newton step each (relative
// error ~1e-12), far cheaper than the full binary64 routines.  m, v and p are
// each rounded once on the way out.
__device__ __forceinline__ double rsqrt_approx64(double x) {
    double y;
    asm("rsqrt.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(x));
    return y;
}
__device__ __forceinline__ double rcp_approx64(double x) {
    double y;
    asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(x));
    return y;
}
__device__ __forceinline__ void adamw_elem(double g64, float &p, float &m, float &v, const AdamDev &a,
                                           const AdamStep &st) {
    const double m64 = fma(a.b1, double(m), a.c1 * g64);
    const double v64 = fma(a.b2, double(v), (a.c2 * g64) * g64);
    double root = 0.0;
    if (v64 > 1e-300) {                                  // below that the root is far under any eps
        const double y = rsqrt_approx64(v64);
        const double r = v64 * y;
        root = fma(fma(-r, r, v64), 0.5 * y, r);         // r + (v - r^2) / (2 sqrt(v))
    }
    const double denom = fma(root, st.inv_sqrt_bc2, a.eps);
    const double q = rcp_approx64(denom);
    const double inv = q * fma(-denom, q, 2.0);          // q (2 - denom q)
    const double delta = fma(a.lr_wd, double(p), st.step_size * (m64 * inv));
    p = __double2float_rn(double(p) - delta);
    m = __double2float_rn(m64);
    v = __double2float_rn(v64);
}

// The two descriptors of the chunk a CTA is working on, in shared memory: everybody picks an
// address up where it is used.  At 1024 threads a thread has 64 registers; five 64-bit base
// addresses held across the loop would take ten of them.
struct __align__(16) AdamChunk {
    Chunk ch;
    OptChunk oc;
};

template <typename GT, int GOP, bool STORE_D, int T>
__device__ __forceinline__ void adamw_chunk(const volatile AdamChunk &ck, int swapped, double beta, double s,
                                            const AdamDev &a, const AdamStep &st) {
    const uint32_t tid = threadIdx.x;
    constexpr int U = AdamGeom<GT>::U;
    constexpr bool kReadD = (GOP == G_FMA || GOP == G_FMA1);
    const uint32_t n = ck.ch.n;
    const bool vec = (ck.ch.flags & kChunkAligned) && ((ck.oc.p | ck.oc.m | ck.oc.v) % 16 == 0);
    // exchange mode: the two address columns of the table trade roles
    #define CK_G (swapped ? ck.ch.d : ck.ch.g)
    #define CK_D (swapped ? ck.ch.g : ck.ch.d)
    if (vec) {
        const uint32_t nvec = n >> 2;
        for (uint32_t base = 0; base < nvec; base += T * U) {
            typename Elem<GOf<GT>>::Raw gr[U];
            typename Elem<DOf<GT>>::Raw dr[U];
            float4 p4[U], m4[U], v4[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t w = base + u * T + tid;
                gr[u] = Elem<GOf<GT>>::zero();
                dr[u] = Elem<DOf<GT>>::zero();
                p4[u] = m4[u] = v4[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (w < nvec) {
                    gr[u] = Elem<GOf<GT>>::template load_raw<GAC_LD_PROJECT>(reinterpret_cast<const void *>(CK_G), w);
                    if (kReadD) dr[u] = Elem<DOf<GT>>::template load_raw<GAC_LD_PROJECT>(reinterpret_cast<const void *>(CK_D), w);
                    p4[u] = Elem<float>::load_raw<GAC_LD_PROJECT>(reinterpret_cast<const void *>(ck.oc.p), w);
                    m4[u] = Elem<float>::load_raw<GAC_LD_PROJECT>(reinterpret_cast<const void *>(ck.oc.m), w);
                    v4[u] = Elem<float>::load_raw<GAC_LD_PROJECT>(reinterpret_cast<const void *>(ck.oc.v), w);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t w = base + u * T + tid;
                if (w >= nvec) continue;
                const F4 gq = Elem<GOf<GT>>::unpack(gr[u]), dq = Elem<DOf<GT>>::unpack(dr[u]);
                const float ge[4] = {gq.x, gq.y, gq.z, gq.w};
                float pe[4] = {p4[u].x, p4[u].y, p4[u].z, p4[u].w};
                float me[4] = {m4[u].x, m4[u].y, m4[u].z, m4[u].w};
                float ve[4] = {v4[u].x, v4[u].y, v4[u].z, v4[u].w};
                const float de[4] = {dq.x, dq.y, dq.z, dq.w};
                if (STORE_D) Elem<DOf<GT>>::store4(reinterpret_cast<void *>(CK_D), w, gq);   // d' = g, the raw gradient
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    adamw_elem(outgoing64<GOP>(ge[e], de[e], st.coef, beta, s), pe[e], me[e], ve[e], a, st);
                }
                Elem<float>::store4(reinterpret_cast<void *>(ck.oc.p), w, F4{pe[0], pe[1], pe[2], pe[3]});
                Elem<float>::store4(reinterpret_cast<void *>(ck.oc.m), w, F4{me[0], me[1], me[2], me[3]});
                Elem<float>::store4(reinterpret_cast<void *>(ck.oc.v), w, F4{ve[0], ve[1], ve[2], ve[3]});
            }
            phase_barrier();
        }
    }
    const uint32_t first = vec ? ((n >> 2) << 2) : 0u;
    for (uint32_t i = first + tid; i < n; i += T) {
        const float x = Elem<GOf<GT>>::load1(reinterpret_cast<const void *>(CK_G), i);
        const float dx = kReadD ? Elem<DOf<GT>>::load1(reinterpret_cast<const void *>(CK_D), i) : 0.f;
        float pe = Elem<float>::load1(reinterpret_cast<const void *>(ck.oc.p), i);
        float me = Elem<float>::load1(reinterpret_cast<const void *>(ck.oc.m), i);
        float ve = Elem<float>::load1(reinterpret_cast<const void *>(ck.oc.v), i);
        adamw_elem(outgoing64<GOP>(x, dx, st.coef, beta, s), pe, me, ve, a, st);
        if (STORE_D) Elem<DOf<GT>>::store1(reinterpret_cast<void *>(CK_D), i, x);
        Elem<float>::store1(reinterpret_cast<void *>(ck.oc.p), i, pe);
        Elem<float>::store1(reinterpret_cast<void *>(ck.oc.m), i, me);
        Elem<float>::store1(reinterpret_cast<void *>(ck.oc.v), i, ve);
    }
    #undef CK_G
    #undef CK_D
}

__device__ __forceinline__ OptChunk load_opt_chunk(const OptChunk *table, uint32_t c) {
    const uint4 *q = reinterpret_cast<const uint4 *>(table + c);
    uint4 a = __ldg(q), b = __ldg(q + 1);
    OptChunk oc;
    oc.p = (uint64_t(a.y) << 32) | a.x;
    oc.m = (uint64_t(a.w) << 32) | a.z;
    oc.v = (uint64_t(b.y) << 32) | b.x;
    oc.pad = 0;
    return oc;
}

template <typename GT, int GOP, bool STORE_D, int T>
__device__ __forceinline__ void adamw_walk(const Chunk *chunks, const OptChunk *opt_chunks, uint32_t n_chunks,
                                           int swapped, double beta, double s, const AdamDev &a,
                                           const AdamStep &st) {
    // Two slots: while the CTA works on the chunk in one, thread 0 has the descriptors of the next
    // chunk copied into the other (asynchronously, past the registers), so that nobody waits for
    // them at the chunk boundary.
    __shared__ AdamChunk slots[2];
    auto fetch = [&](uint32_t c, AdamChunk &out) {
        cp_async16(&out.ch, chunks + c);
        cp_async16(reinterpret_cast<char *>(&out.ch) + 16, reinterpret_cast<const char *>(chunks + c) + 16);
        cp_async16(&out.oc, opt_chunks + c);
        cp_async16(reinterpret_cast<char *>(&out.oc) + 16, reinterpret_cast<const char *>(opt_chunks + c) + 16);
    };
    uint32_t c = blockIdx.x;
    if (c >= n_chunks) return;
    if (threadIdx.x == 0) fetch(c, slots[0]);
    int cur = 0;
    for (; c < n_chunks; c += gridDim.x, cur ^= 1) {
        if (threadIdx.x == 0) cp_async_wait_all();   // the copies into slots[cur] have landed
        __syncthreads();                             // ... for everybody; and nobody reads slots[cur ^ 1] any more
        if (threadIdx.x == 0 && c + gridDim.x < n_chunks) fetch(c + gridDim.x, slots[cur ^ 1]);
        adamw_chunk<GT, GOP, STORE_D, T>(slots[cur], swapped, beta, s, a, st);
    }
}

// Same decision logic as gac_project_kernel; a safe or projection step feeds
// AdamW, a violation step only refreshes the stored direction.  The count of
// applied updates lives in the decision record: every CTA reads it on entry,
// and the last CTA to FINISH (arrival ticket, nobody waits) writes it back
// incremented, so no CTA can see the new value during this launch.
// EXCH (exchange mode): d' = g costs nothing -- the buffers swap roles -- so no
// state is stored and a skipped step moves no data at all.
// PLAIN (chosen by the host: beta = 1 and clipping off) holds only the loops of the paper's own
// rule; the general instantiation also serves Eq. 3's beta and an active clip factor.
template <typename GT, bool PLAIN>
struct AdamThreads {
    static constexpr int T = PLAIN ? AdamGeom<GT>::T : AdamGeom<GT>::TG;
};
template <typename GT, bool EXCH, bool PLAIN>
__global__ void __launch_bounds__((AdamThreads<GT, PLAIN>::T), (AdamGeom<GT>::C))
gac_adamw_kernel(const Chunk *__restrict__ chunks, const OptChunk *__restrict__ opt_chunks,
                 uint32_t n_chunks, gac_result *rec, unsigned *ticket, float coef_override,
                 int use_override, double beta, double clip_max, double clip_eps, AdamDev o, int swapped) {
    const bool closed = rec->nonfinite || rec->timed_out;
    if (EXCH && blockIdx.x == 0 && threadIdx.x == 0) rec->ref_lost = closed ? 1u : 0u;
    if (closed) return;
    const int regime = rec->regime;
    const float k = use_override ? coef_override : rec->coef;
    const unsigned long long t_prev = rec->applied_steps;
    double s = 1.0;
    if (clip_max > 0.0) {
        double norm;
        s = clip_factor(regime, rec->dot, rec->gg, rec->dd, beta, double(k), clip_max, clip_eps, &norm);
        if (use_override && blockIdx.x == 0 && threadIdx.x == 0) {
            rec->out_norm = norm;
            rec->clip_scale = s;
        }
    }
    const bool applies = (regime != GAC_REGIME_VIOLATION);
    if (applies) {
        const double t = double(t_prev + 1ull);
        const double bc1 = 1.0 - pow(o.b1, t), bc2 = 1.0 - pow(o.b2, t);
        // the two step-dependent factors live in shared memory: read where they are used, they do
        // not hold registers across the loop (at 1024 threads a thread has 64)
        __shared__ AdamStep st_shared;
        if (threadIdx.x == 0) {
            st_shared.step_size = o.lr / bc1;
            st_shared.inv_sqrt_bc2 = 1.0 / sqrt(bc2);
            st_shared.coef = k;
        }
        __syncthreads();
        const AdamStep &st = st_shared;
        // one uniform choice per launch; each branch holds only the loop it needs
        constexpr int T = AdamThreads<GT, PLAIN>::T;
        const int gop = regime == GAC_REGIME_PROJECT ? ((beta == 1.0 && s == 1.0) ? G_FMA1 : G_FMA)
                                                     : (s != 1.0 ? G_SCALE : G_KEEP);
        if (gop == G_FMA1) adamw_walk<GT, G_FMA1, !EXCH, T>(chunks, opt_chunks, n_chunks, swapped, 1.0, 1.0, o, st);
        else if (gop == G_KEEP) adamw_walk<GT, G_KEEP, !EXCH, T>(chunks, opt_chunks, n_chunks, swapped, 1.0, 1.0, o, st);
        else if (!PLAIN && gop == G_FMA) adamw_walk<GT, G_FMA, !EXCH, T>(chunks, opt_chunks, n_chunks, swapped, beta, s, o, st);
        else if (!PLAIN) adamw_walk<GT, G_SCALE, !EXCH, T>(chunks, opt_chunks, n_chunks, swapped, 1.0, s, o, st);
    } else if (!EXCH) {
        // skipped step: d' = g only
        project_walk_tu<GT, G_KEEP, D_RAW, true, AdamThreads<GT, PLAIN>::T, AdamGeom<GT>::U, 0, 1>(chunks, n_chunks, k, 1.0, 1.0, 0);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned done = atomicAdd(ticket, 1u);
        if (done == gridDim.x - 1) {
            // read again rather than held across the loop: nobody has written it during this launch
            rec->applied_steps = rec->applied_steps + (rec->regime != GAC_REGIME_VIOLATION ? 1ull : 0ull);
            __threadfence();
            *ticket = 0u;
        }
    }
}

using ProjectKernel = void (*)(const Chunk *, uint32_t, gac_result *, float, int, double, double, double, int);

template <typename GT, int STATE>
ProjectKernel pick_project(bool beta1, bool zero) {
    if (beta1) return zero ? gac_project_kernel<GT, STATE, true, true> : gac_project_kernel<GT, STATE, true, false>;
    return zero ? gac_project_kernel<GT, STATE, false, true> : gac_project_kernel<GT, STATE, false, false>;
}
// Exchange mode stores g' with g's element type into d's buffers: only pairs of one type have it.
template <typename GT>
using SameTypes = std::integral_constant<bool, std::is_same<GOf<GT>, DOf<GT>>::value>;
template <typename GT>
ProjectKernel pick_exchange(bool beta1, bool zero, std::true_type) {
    return pick_project<GT, GAC_STATE_EXCHANGE>(beta1, zero);
}
template <typename GT>
ProjectKernel pick_exchange(bool, bool, std::false_type) {
    return nullptr;
}
template <typename GT>
ProjectKernel pick_project(int state, bool beta1, bool zero) {
    if (state == GAC_STATE_RAW) return pick_project<GT, GAC_STATE_RAW>(beta1, zero);
    if (state == GAC_STATE_PROJECTED) return pick_project<GT, GAC_STATE_PROJECTED>(beta1, zero);
    if (state == GAC_STATE_EXCHANGE) return pick_exchange<GT>(beta1, zero, SameTypes<GT>{});
    return pick_project<GT, GAC_STATE_HOLD>(beta1, zero);
}

}  // namespace
