// CUDA implementation (sm_100a) of the GAC per-step hot path behind the C ABI in
// include/gac.h.
//
//   chunk table      the list of parameter tensors is cut into fixed-size
//                    chunks, none spanning two tensors; one launch walks them
//                    all (App. A.1: the gradient is the flattened
//                    concatenation of all parameter gradients -- presented
//                    here without the flatten copy)
//   gac_stats_kernel fused <g,d>, <g,g>, <d,d> (App. A.1) with binary64
//                    accumulation, per-CTA partials, and a fixed-order second
//                    stage run by the last CTA to finish, which also takes the
//                    decision of Algorithm 1 / Eq. 5
//   gac_project_kernel  g' = beta g + coef d in place and d' = g (App. A.2)
//
// The work is bound by HBM bandwidth: 3 FMAs per 8 bytes read in the first
// pass, 1 FMA per 16 bytes moved in the second.  There is no dense contraction
// here, hence no tensor-core path.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <mutex>
#include <new>
#include <vector>

#include "gac.h"

namespace {

// Launch geometry.  Both kernels are bound by HBM, and on B200 their speed
// depends on how many bytes each SM keeps in flight: too few starve the
// memory system, too many make reads and write-backs of many chunks collide in
// DRAM.  The macros exist so that variants can be built and timed side by side;
// the defaults are the measured best per element type (T threads per CTA,
// U four-element vectors in flight per thread and operand, C resident CTAs per
// SM the grid is sized for with 0 = all that fit, MINB = occupancy asked of the
// compiler with 0 = no request).
#ifndef GAC_STATS_T_F32
#define GAC_STATS_T_F32 256
#endif
#ifndef GAC_STATS_U_F32
#define GAC_STATS_U_F32 8
#endif
#ifndef GAC_STATS_C_F32
#define GAC_STATS_C_F32 0
#endif
#ifndef GAC_STATS_MINB_F32
#define GAC_STATS_MINB_F32 4
#endif
#ifndef GAC_STATS_T_BF16
#define GAC_STATS_T_BF16 256
#endif
#ifndef GAC_STATS_U_BF16
#define GAC_STATS_U_BF16 8
#endif
#ifndef GAC_STATS_C_BF16
#define GAC_STATS_C_BF16 0
#endif
#ifndef GAC_STATS_MINB_BF16
#define GAC_STATS_MINB_BF16 4
#endif
#ifndef GAC_PROJ_T_F32
#define GAC_PROJ_T_F32 256
#endif
#ifndef GAC_PROJ_U_F32
#define GAC_PROJ_U_F32 8
#endif
#ifndef GAC_PROJ_C_F32
#define GAC_PROJ_C_F32 1
#endif
#ifndef GAC_PROJ_MINB_F32
#define GAC_PROJ_MINB_F32 1
#endif
#ifndef GAC_PROJ_T_BF16
#define GAC_PROJ_T_BF16 512
#endif
#ifndef GAC_PROJ_U_BF16
#define GAC_PROJ_U_BF16 4
#endif
#ifndef GAC_PROJ_C_BF16
#define GAC_PROJ_C_BF16 1
#endif
#ifndef GAC_PROJ_MINB_BF16
#define GAC_PROJ_MINB_BF16 1
#endif
// (bfloat16 g, bfloat16 d): half the bytes per vector of the mixed pair
#ifndef GAC_STATS_T_BF16X
#define GAC_STATS_T_BF16X GAC_STATS_T_BF16
#endif
#ifndef GAC_STATS_U_BF16X
#define GAC_STATS_U_BF16X GAC_STATS_U_BF16
#endif
#ifndef GAC_STATS_C_BF16X
#define GAC_STATS_C_BF16X GAC_STATS_C_BF16
#endif
#ifndef GAC_STATS_MINB_BF16X
#define GAC_STATS_MINB_BF16X GAC_STATS_MINB_BF16
#endif
#ifndef GAC_PROJ_T_BF16X
#define GAC_PROJ_T_BF16X GAC_PROJ_T_BF16
#endif
#ifndef GAC_PROJ_U_BF16X
#define GAC_PROJ_U_BF16X 8
#endif
#ifndef GAC_PROJ_C_BF16X
#define GAC_PROJ_C_BF16X GAC_PROJ_C_BF16
#endif
#ifndef GAC_PROJ_MINB_BF16X
#define GAC_PROJ_MINB_BF16X GAC_PROJ_MINB_BF16
#endif
#ifndef GAC_ADAMW_T_F32
#define GAC_ADAMW_T_F32 1024
#endif
#ifndef GAC_ADAMW_U_F32
#define GAC_ADAMW_U_F32 1
#endif
#ifndef GAC_ADAMW_C_F32
#define GAC_ADAMW_C_F32 1
#endif
#ifndef GAC_ADAMW_T_BF16
#define GAC_ADAMW_T_BF16 1024
#endif
#ifndef GAC_ADAMW_U_BF16
#define GAC_ADAMW_U_BF16 1
#endif
#ifndef GAC_ADAMW_C_BF16
#define GAC_ADAMW_C_BF16 1
#endif
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
};

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

template <>
struct Elem<float> {
    template <int LD>
    static __device__ __forceinline__ F4 load4(const void *base, uint32_t v) {
        float4 t = ld_vec<LD>(reinterpret_cast<const float4 *>(base) + v);
        return F4{t.x, t.y, t.z, t.w};
    }
    static __device__ __forceinline__ void store4(void *base, uint32_t v, F4 a) {
        st_vec(reinterpret_cast<float4 *>(base) + v, make_float4(a.x, a.y, a.z, a.w));
    }
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

template <typename GT>
struct StatsGeom;
template <>
struct StatsGeom<float> {
    static constexpr int T = GAC_STATS_T_F32, U = GAC_STATS_U_F32, C = GAC_STATS_C_F32, MINB = GAC_STATS_MINB_F32;
};
template <>
struct StatsGeom<bf16_t> {
    static constexpr int T = GAC_STATS_T_BF16, U = GAC_STATS_U_BF16, C = GAC_STATS_C_BF16, MINB = GAC_STATS_MINB_BF16;
};
template <typename GT>
struct AdamGeom;
template <>
struct AdamGeom<float> {
    static constexpr int T = GAC_ADAMW_T_F32, U = GAC_ADAMW_U_F32, C = GAC_ADAMW_C_F32;
};
template <>
struct AdamGeom<bf16_t> {
    static constexpr int T = GAC_ADAMW_T_BF16, U = GAC_ADAMW_U_BF16, C = GAC_ADAMW_C_BF16;
};
template <>
struct StatsGeom<bf16_pair_t> {
    static constexpr int T = GAC_STATS_T_BF16X, U = GAC_STATS_U_BF16X, C = GAC_STATS_C_BF16X, MINB = GAC_STATS_MINB_BF16X;
};
template <>
struct AdamGeom<bf16_pair_t> : AdamGeom<bf16_t> {};
template <typename GT>
struct ProjGeom;
template <>
struct ProjGeom<float> {
    static constexpr int T = GAC_PROJ_T_F32, U = GAC_PROJ_U_F32, C = GAC_PROJ_C_F32, MINB = GAC_PROJ_MINB_F32;
};
template <>
struct ProjGeom<bf16_t> {
    static constexpr int T = GAC_PROJ_T_BF16, U = GAC_PROJ_U_BF16, C = GAC_PROJ_C_BF16, MINB = GAC_PROJ_MINB_BF16;
};
template <>
struct ProjGeom<bf16_pair_t> {
    static constexpr int T = GAC_PROJ_T_BF16X, U = GAC_PROJ_U_BF16X, C = GAC_PROJ_C_BF16X, MINB = GAC_PROJ_MINB_BF16X;
};

__device__ __forceinline__ uint32_t pack_bf16x2_rn(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

template <>
struct Elem<bf16_t> {
    template <int LD>
    static __device__ __forceinline__ F4 load4(const void *base, uint32_t v) {
        uint2 t = ld_vec<LD>(reinterpret_cast<const uint2 *>(base) + v);
        return F4{__uint_as_float(t.x << 16), __uint_as_float(t.x & 0xFFFF0000u),
                  __uint_as_float(t.y << 16), __uint_as_float(t.y & 0xFFFF0000u)};
    }
    static __device__ __forceinline__ void store4(void *base, uint32_t v, F4 a) {
        st_vec(reinterpret_cast<uint2 *>(base) + v,
               make_uint2(pack_bf16x2_rn(a.x, a.y), pack_bf16x2_rn(a.z, a.w)));
    }
    static __device__ __forceinline__ float load1(const void *base, uint32_t i) {
        return __uint_as_float(uint32_t(reinterpret_cast<const uint16_t *>(base)[i]) << 16);
    }
    static __device__ __forceinline__ void store1(void *base, uint32_t i, float a) {
        reinterpret_cast<uint16_t *>(base)[i] = uint16_t(pack_bf16x2_rn(a, 0.0f) & 0xFFFFu);
    }
};

__device__ __forceinline__ Chunk load_chunk(const Chunk *table, uint32_t c) {
    const uint4 *p = reinterpret_cast<const uint4 *>(table + c);
    uint4 a = __ldg(p), b = __ldg(p + 1);
    Chunk ch;
    ch.g = (uint64_t(a.y) << 32) | a.x;
    ch.d = (uint64_t(a.w) << 32) | a.z;
    ch.n = b.x;
    ch.flags = b.y;
    ch.pad = 0;
    return ch;
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
__device__ void take_decision(double dot, double gg, double dd, const DevHP &hp, gac_result *r) {
    if (hp.first_step) {   // Algorithm 1: g_0 = 0
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
    r->nonfinite = !(isfinite(dot) && isfinite(gg) && isfinite(dd));
    if (r->nonfinite) {
        r->cos = __longlong_as_double(0x7FF8000000000000LL);
        r->regime = GAC_REGIME_VIOLATION;
        return;
    }
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
            F4 gv[U], dv[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t v = base + u * T + tid;
                if (v < nvec) {
                    gv[u] = Elem<GOf<GT>>::template load4<GAC_LD_STATS>(g, v);
                    if (READ_D) dv[u] = Elem<DOf<GT>>::template load4<GAC_LD_STATS>(d, v);
                } else {
                    gv[u] = F4{0.f, 0.f, 0.f, 0.f};
                    if (READ_D) dv[u] = F4{0.f, 0.f, 0.f, 0.f};
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const float ge[4] = {gv[u].x, gv[u].y, gv[u].z, gv[u].w};
                const float de[4] = {dv[u].x, dv[u].y, dv[u].z, dv[u].w};
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
    if (hp.first_step) {
        for (uint32_t c = blockIdx.x; c < n_chunks; c += gridDim.x)
            stats_chunk<GT, false>(load_chunk(chunks, c), a_dot, a_gg, a_dd);
    } else {
        for (uint32_t c = blockIdx.x; c < n_chunks; c += gridDim.x)
            stats_chunk<GT, true>(load_chunk(chunks, c), a_dot, a_gg, a_dd);
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
            sums_out[0] = hp.first_step ? 0.0 : s0;
            sums_out[1] = s1;
            sums_out[2] = hp.first_step ? 0.0 : s2;
        }
        if (hp.decide) take_decision(s0, s1, s2, hp, rec);
    }
}

__global__ void gac_decide_kernel(const double *sums_in, gac_result *rec, DevHP hp) {
    if (threadIdx.x == 0 && blockIdx.x == 0)
        take_decision(sums_in[0], sums_in[1], sums_in[2], hp, rec);
}

// ----------------------------------------------------------- project kernel

enum GOp { G_KEEP = 0, G_FMA = 1, G_ZERO = 2, G_SCALE = 3 };
enum DOp { D_KEEP = 0, D_RAW = 1, D_NEW = 2 };

template <bool BETA1>
__device__ __forceinline__ float rank_one(float g, float d, float k, double beta, double s) {
    if (BETA1) return fmaf(k, d, g);   // beta = 1, no clipping: one rounding
    // general beta and/or an active clip factor s: binary64 (rounded product + exact product), times s
    return __double2float_rn(
        __dmul_rn(s, __dadd_rn(__dmul_rn(beta, double(g)), __dmul_rn(double(k), double(d)))));
}
__device__ __forceinline__ float scaled(float g, double s) { return __double2float_rn(__dmul_rn(s, double(g))); }

template <typename GT, int GOP, int DOP, bool BETA1, int T, int U>
__device__ __forceinline__ void project_chunk(const Chunk &ch, float k, double beta, double s) {
    void *g = reinterpret_cast<void *>(ch.g);
    void *d = reinterpret_cast<void *>(ch.d);
    const uint32_t tid = threadIdx.x;
    constexpr bool kReadG = (GOP == G_FMA) || (GOP == G_SCALE) || (DOP == D_RAW);
    constexpr bool kReadD = (GOP == G_FMA);
    if (ch.flags & kChunkAligned) {
        const uint32_t nvec = ch.n >> 2;
        for (uint32_t base = 0; base < nvec; base += T * U) {
            F4 gv[U], dv[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t v = base + u * T + tid;
                gv[u] = F4{0.f, 0.f, 0.f, 0.f};
                dv[u] = F4{0.f, 0.f, 0.f, 0.f};
                if (v < nvec) {
                    if (kReadG) gv[u] = Elem<GOf<GT>>::template load4<GAC_LD_PROJECT>(g, v);
                    if (kReadD) dv[u] = Elem<DOf<GT>>::template load4<GAC_LD_PROJECT>(d, v);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t v = base + u * T + tid;
                if (v >= nvec) continue;
                F4 out = gv[u];
                if (GOP == G_ZERO) out = F4{0.f, 0.f, 0.f, 0.f};
                if (GOP == G_FMA) {
                    out.x = rank_one<BETA1>(gv[u].x, dv[u].x, k, beta, s);
                    out.y = rank_one<BETA1>(gv[u].y, dv[u].y, k, beta, s);
                    out.z = rank_one<BETA1>(gv[u].z, dv[u].z, k, beta, s);
                    out.w = rank_one<BETA1>(gv[u].w, dv[u].w, k, beta, s);
                }
                if (GOP == G_SCALE) out = F4{scaled(gv[u].x, s), scaled(gv[u].y, s), scaled(gv[u].z, s), scaled(gv[u].w, s)};
                if (GOP != G_KEEP) Elem<GOf<GT>>::store4(g, v, out);
                if (DOP == D_RAW) Elem<DOf<GT>>::store4(d, v, gv[u]);
                if (DOP == D_NEW) {
                    if (GOP == G_FMA || GOP == G_SCALE) out = Elem<GOf<GT>>::template load4<GAC_LD_PROJECT>(g, v);   // the value as stored (rounded)
                    Elem<DOf<GT>>::store4(d, v, out);
                }
            }
        }
        const uint32_t done = nvec << 2;
        if (tid < ch.n - done) {
            const uint32_t i = done + tid;
            const float x = kReadG ? Elem<GOf<GT>>::load1(g, i) : 0.f;
            float out = (GOP == G_ZERO) ? 0.f : x;
            if (GOP == G_FMA) out = rank_one<BETA1>(x, Elem<DOf<GT>>::load1(d, i), k, beta, s);
            if (GOP == G_SCALE) out = scaled(x, s);
            if (GOP != G_KEEP) Elem<GOf<GT>>::store1(g, i, out);
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
            if (GOP != G_KEEP) Elem<GOf<GT>>::store1(g, i, out);
            if (DOP == D_RAW) Elem<DOf<GT>>::store1(d, i, x);
            if (DOP == D_NEW) {
                if (GOP == G_FMA || GOP == G_SCALE) out = Elem<GOf<GT>>::load1(g, i);
                Elem<DOf<GT>>::store1(d, i, out);
            }
        }
    }
}

template <typename GT, int GOP, int DOP, bool BETA1>
__device__ __forceinline__ void project_walk(const Chunk *chunks, uint32_t n_chunks, float k,
                                             double beta, double s) {
    for (uint32_t c = blockIdx.x; c < n_chunks; c += gridDim.x)
        project_chunk<GT, GOP, DOP, BETA1, ProjGeom<GT>::T, ProjGeom<GT>::U>(load_chunk(chunks, c), k, beta, s);
}

// The regime is read from the device-resident record, so no host round trip
// separates the two passes; every CTA takes the same (uniform) branch.  What
// the host already knows (state mode, beta == 1, zero_on_violation) is fixed at
// compile time so that each instantiation holds only the loops it can reach.
template <typename GT, int STATE, bool BETA1, bool ZERO>
__global__ void __launch_bounds__(ProjGeom<GT>::T, ProjGeom<GT>::MINB)
gac_project_kernel(const Chunk *__restrict__ chunks, uint32_t n_chunks, gac_result *rec,
                   float coef_override, int use_override, double beta, double clip_max, double clip_eps) {
    if (rec->nonfinite) return;   // reading taken for NaN/Inf: touch nothing
    const int regime = rec->regime;
    const float k = use_override ? coef_override : rec->coef;
    constexpr int dop = STATE == GAC_STATE_RAW ? D_RAW : (STATE == GAC_STATE_PROJECTED ? D_NEW : D_KEEP);
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
        if (s != 1.0) project_walk<GT, G_FMA, dop, false>(chunks, n_chunks, k, beta, s);
        else project_walk<GT, G_FMA, dop, BETA1>(chunks, n_chunks, k, beta, 1.0);
    } else if (ZERO && regime == GAC_REGIME_VIOLATION) {
        project_walk<GT, G_ZERO, dop, true>(chunks, n_chunks, k, 1.0, 1.0);
    } else if (s != 1.0) {
        project_walk<GT, G_SCALE, dop, true>(chunks, n_chunks, k, 1.0, s);   // safe step, clipped: g'' = s g
    } else if (STATE != GAC_STATE_HOLD) {
        project_walk<GT, G_KEEP, D_RAW, true>(chunks, n_chunks, k, 1.0, 1.0);   // d' = g, g untouched
    }
}

// ------------------------------------------------ projection fused with AdamW

struct __align__(16) OptChunk {
    uint64_t p, m, v, pad;   // device addresses of the chunk's first parameter / moment elements
};
static_assert(sizeof(OptChunk) == 32, "optimizer chunk descriptors are read as two 16-byte words");

struct AdamDev {
    double lr, beta1, beta2, eps, weight_decay;
};

struct AdamConst {
    double b1, c1, b2, c2;                       // moment recurrences
    double step_size, inv_sqrt_bc2, eps, lr_wd;  // lr/(1-b1^t), 1/sqrt(1-b2^t), eps, lr*wd
};

// The outgoing gradient in binary64, unrounded: the moments are differences of
// nearly equal terms often enough that a binary32 g' would cost them digits.
template <int GOP>
__device__ __forceinline__ double outgoing64(float g, float d, float k, double beta, double s) {
    if (GOP == G_FMA)
        return __dmul_rn(s, __dadd_rn(__dmul_rn(beta, double(g)), __dmul_rn(double(k), double(d))));
    if (GOP == G_SCALE) return __dmul_rn(s, double(g));
    return double(g);
}

// One element of: g' -> AdamW, in binary64 so that p - delta stays accurate
// even where it cancels (tiny parameters).  The square root and the reciprocal
// start from binary32 hardware results and take one Newton step each in
// binary64 (relative error ~1e-14), far cheaper than the binary64 library
// routines.  m, v and p are each rounded once on the way out.
__device__ __forceinline__ void adamw_elem(double g64, float &p, float &m, float &v, const AdamConst &a) {
    const double m64 = __dadd_rn(__dmul_rn(a.b1, double(m)), __dmul_rn(a.c1, g64));
    const double v64 = __dadd_rn(__dmul_rn(a.b2, double(v)), __dmul_rn(__dmul_rn(a.c2, g64), g64));
    double root = 0.0;
    const float r32 = __fsqrt_rn(__double2float_rn(v64));
    if (r32 > 0.0f) {
        const double r = double(r32);
        root = fma(fma(-r, r, v64), double(__fdividef(0.5f, r32)), r);   // r + (v - r^2)/(2r)
    }
    const double denom = fma(root, a.inv_sqrt_bc2, a.eps);
    const double q = double(__frcp_rn(__double2float_rn(denom)));
    const double inv = q * fma(-denom, q, 2.0);                           // q (2 - denom q)
    const double delta = fma(a.lr_wd, double(p), a.step_size * (m64 * inv));
    p = __double2float_rn(double(p) - delta);
    m = __double2float_rn(m64);
    v = __double2float_rn(v64);
}

template <typename GT, int GOP>
__device__ __forceinline__ void adamw_chunk(const Chunk &ch, const OptChunk &oc, float k, double beta,
                                            double s, const AdamConst &a) {
    const void *g = reinterpret_cast<const void *>(ch.g);
    void *d = reinterpret_cast<void *>(ch.d);
    void *pp = reinterpret_cast<void *>(oc.p);
    void *pm = reinterpret_cast<void *>(oc.m);
    void *pv = reinterpret_cast<void *>(oc.v);
    const uint32_t tid = threadIdx.x;
    constexpr int T = AdamGeom<GT>::T, U = AdamGeom<GT>::U;
    const bool vec = (ch.flags & kChunkAligned) && ((oc.p | oc.m | oc.v) % 16 == 0);
    if (vec) {
        const uint32_t nvec = ch.n >> 2;
        for (uint32_t base = 0; base < nvec; base += T * U) {
            F4 gv[U], dv[U], p4[U], m4[U], v4[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t w = base + u * T + tid;
                dv[u] = F4{0.f, 0.f, 0.f, 0.f};
                if (w < nvec) {
                    gv[u] = Elem<GOf<GT>>::template load4<GAC_LD_PROJECT>(g, w);
                    if (GOP == G_FMA) dv[u] = Elem<DOf<GT>>::template load4<GAC_LD_PROJECT>(d, w);
                    p4[u] = Elem<float>::load4<GAC_LD_PROJECT>(pp, w);
                    m4[u] = Elem<float>::load4<GAC_LD_PROJECT>(pm, w);
                    v4[u] = Elem<float>::load4<GAC_LD_PROJECT>(pv, w);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t w = base + u * T + tid;
                if (w >= nvec) continue;
                float ge[4] = {gv[u].x, gv[u].y, gv[u].z, gv[u].w};
                float pe[4] = {p4[u].x, p4[u].y, p4[u].z, p4[u].w};
                float me[4] = {m4[u].x, m4[u].y, m4[u].z, m4[u].w};
                float ve[4] = {v4[u].x, v4[u].y, v4[u].z, v4[u].w};
                const float de[4] = {dv[u].x, dv[u].y, dv[u].z, dv[u].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    adamw_elem(outgoing64<GOP>(ge[e], de[e], k, beta, s), pe[e], me[e], ve[e], a);
                }
                Elem<DOf<GT>>::store4(d, w, gv[u]);                       // d' = g, the raw gradient
                Elem<float>::store4(pp, w, F4{pe[0], pe[1], pe[2], pe[3]});
                Elem<float>::store4(pm, w, F4{me[0], me[1], me[2], me[3]});
                Elem<float>::store4(pv, w, F4{ve[0], ve[1], ve[2], ve[3]});
            }
        }
    }
    const uint32_t first = vec ? ((ch.n >> 2) << 2) : 0u;
    for (uint32_t i = first + tid; i < ch.n; i += T) {
        const float x = Elem<GOf<GT>>::load1(g, i);
        const float dx = (GOP == G_FMA) ? Elem<DOf<GT>>::load1(d, i) : 0.f;
        float pe = Elem<float>::load1(pp, i), me = Elem<float>::load1(pm, i), ve = Elem<float>::load1(pv, i);
        adamw_elem(outgoing64<GOP>(x, dx, k, beta, s), pe, me, ve, a);
        Elem<DOf<GT>>::store1(d, i, x);
        Elem<float>::store1(pp, i, pe);
        Elem<float>::store1(pm, i, me);
        Elem<float>::store1(pv, i, ve);
    }
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

// Same decision logic as gac_project_kernel; a safe or projection step feeds
// AdamW, a violation step only refreshes the stored direction.  The count of
// applied updates lives in the decision record: every CTA reads it on entry,
// and the last CTA to FINISH (arrival ticket, nobody waits) writes it back
// incremented, so no CTA can see the new value during this launch.
template <typename GT>
__global__ void __launch_bounds__(AdamGeom<GT>::T, AdamGeom<GT>::C)
gac_adamw_kernel(const Chunk *__restrict__ chunks, const OptChunk *__restrict__ opt_chunks,
                 uint32_t n_chunks, gac_result *rec, unsigned *ticket, float coef_override,
                 int use_override, double beta, double clip_max, double clip_eps, AdamDev o) {
    if (rec->nonfinite) return;
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
        const double bc1 = 1.0 - pow(o.beta1, t), bc2 = 1.0 - pow(o.beta2, t);
        AdamConst a;
        a.b1 = o.beta1;
        a.c1 = 1.0 - o.beta1;
        a.b2 = o.beta2;
        a.c2 = 1.0 - o.beta2;
        a.step_size = o.lr / bc1;
        a.inv_sqrt_bc2 = 1.0 / sqrt(bc2);
        a.eps = o.eps;
        a.lr_wd = o.lr * o.weight_decay;
        for (uint32_t c = blockIdx.x; c < n_chunks; c += gridDim.x) {
            const Chunk ch = load_chunk(chunks, c);
            const OptChunk oc = load_opt_chunk(opt_chunks, c);
            if (regime == GAC_REGIME_PROJECT) adamw_chunk<GT, G_FMA>(ch, oc, k, beta, s, a);
            else if (s != 1.0) adamw_chunk<GT, G_SCALE>(ch, oc, k, 1.0, s, a);
            else adamw_chunk<GT, G_KEEP>(ch, oc, k, 1.0, 1.0, a);
        }
    } else {
        for (uint32_t c = blockIdx.x; c < n_chunks; c += gridDim.x)   // skipped step: d' = g only
            project_chunk<GT, G_KEEP, D_RAW, true, AdamGeom<GT>::T, AdamGeom<GT>::U>(load_chunk(chunks, c), k, 1.0, 1.0);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned done = atomicAdd(ticket, 1u);
        if (done == gridDim.x - 1) {
            rec->applied_steps = t_prev + (applies ? 1ull : 0ull);
            __threadfence();
            *ticket = 0u;
        }
    }
}

using ProjectKernel = void (*)(const Chunk *, uint32_t, gac_result *, float, int, double, double, double);

template <typename GT, int STATE>
ProjectKernel pick_project(bool beta1, bool zero) {
    if (beta1) return zero ? gac_project_kernel<GT, STATE, true, true> : gac_project_kernel<GT, STATE, true, false>;
    return zero ? gac_project_kernel<GT, STATE, false, true> : gac_project_kernel<GT, STATE, false, false>;
}
template <typename GT>
ProjectKernel pick_project(int state, bool beta1, bool zero) {
    if (state == GAC_STATE_RAW) return pick_project<GT, GAC_STATE_RAW>(beta1, zero);
    if (state == GAC_STATE_PROJECTED) return pick_project<GT, GAC_STATE_PROJECTED>(beta1, zero);
    return pick_project<GT, GAC_STATE_HOLD>(beta1, zero);
}

}  // namespace

// ===================================================================== host

struct gac_ctx {
    int device = 0;
    int g_dt = GAC_F32, d_dt = GAC_F32;
    int pair = 0;   // PairId of (g_dt, d_dt)
    gac_hparams hp{};
    std::vector<gac_tensor> list;
    uint64_t total = 0;
    uint32_t misaligned = 0;

    Chunk *d_chunks = nullptr;
    uint64_t n_chunks = 0;
    double *d_partials = nullptr;
    unsigned *d_ticket = nullptr;
    gac_result *d_rec = nullptr;
    gac_result *h_rec = nullptr;   // pinned

    int sms = 0;
    int chunk_elems = kDefaultChunk;
    int ctas_per_sm = 0;           // 0 = what occupancy allows
    int grid_stats = 0, grid_project = 0;
    int threads_stats = 0, threads_project = 0;
    const void *project_fn = nullptr;   // instantiation chosen from the hyper-parameters
    OptChunk *d_opt_chunks = nullptr;   // optimizer state table of gac_attach_adamw
    std::vector<gac_opt_tensor> opt_list;
    int grid_adamw = 0, threads_adamw = 0;

    uint64_t last_projected_step = 0;
    uint64_t pending_step = 0;
    uint32_t pending_staleness = 0;
    bool stats_pending = false;    // a partial reduction waits for gac_decide
    bool decision_ready = false;   // a decision waits for gac_project
    bool started = false;
    uint64_t launches = 0;
    char err[512] = {0};
};

namespace {

thread_local char g_init_err[512] = "no error";

int fail(gac_ctx *ctx, int code, const char *fmt, const char *a = "", long long b = 0) {
    char *dst = ctx ? ctx->err : g_init_err;
    snprintf(dst, 512, fmt, a, b);
    return code;
}

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        ok = (cudaSetDevice(dev) == cudaSuccess);
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

#define GAC_CUDA(ctx, call)                                                          \
    do {                                                                             \
        cudaError_t e_ = (call);                                                     \
        if (e_ != cudaSuccess)                                                       \
            return fail((ctx), GAC_ERR_CUDA, "%s (CUDA error %lld): " #call,        \
                        cudaGetErrorString(e_), (long long)e_);                      \
    } while (0)

size_t elem_size(int dt) { return dt == GAC_BF16 ? 2 : 4; }

void release_device(gac_ctx *c) {
    if (c->d_chunks) cudaFree(c->d_chunks);
    if (c->d_opt_chunks) cudaFree(c->d_opt_chunks);
    c->d_opt_chunks = nullptr;
    if (c->d_partials) cudaFree(c->d_partials);
    if (c->d_ticket) cudaFree(c->d_ticket);
    if (c->d_rec) cudaFree(c->d_rec);
    if (c->h_rec) cudaFreeHost(c->h_rec);
    c->d_chunks = nullptr;
    c->d_partials = nullptr;
    c->d_ticket = nullptr;
    c->d_rec = nullptr;
    c->h_rec = nullptr;
}

template <typename K>
int resident_ctas(K kernel, int threads) {
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, threads, 0) != cudaSuccess || n < 1)
        n = 1;
    return std::min(n, kMaxCtasPerSm);
}

// Supported element-type pairs and the kernels instantiated for them.
enum PairId { kPairF32 = 0, kPairBf16F32 = 1, kPairBf16Bf16 = 2, kPairCount = 3 };

int pair_id(int g_dt, int d_dt) {
    if (g_dt == GAC_F32 && d_dt == GAC_F32) return kPairF32;
    if (g_dt == GAC_BF16 && d_dt == GAC_F32) return kPairBf16F32;
    if (g_dt == GAC_BF16 && d_dt == GAC_BF16) return kPairBf16Bf16;
    return -1;
}

template <typename F>
auto with_pair(int pair, F f) {
    switch (pair) {
        case kPairF32: return f(float{});
        case kPairBf16F32: return f(bf16_t{});
        default: return f(bf16_pair_t{});
    }
}

using StatsKernel = void (*)(const Chunk *, uint32_t, double *, unsigned *, gac_result *, double *, DevHP);
using AdamKernel = void (*)(const Chunk *, const OptChunk *, uint32_t, gac_result *, unsigned *, float, int,
                            double, double, double, AdamDev);

StatsKernel stats_kernel_of(int pair) {
    return with_pair(pair, [](auto tag) -> StatsKernel { return gac_stats_kernel<decltype(tag)>; });
}
int stats_threads_of(int pair) {
    return with_pair(pair, [](auto tag) { return StatsGeom<decltype(tag)>::T; });
}
int stats_cap_of(int pair) {
    return with_pair(pair, [](auto tag) { return StatsGeom<decltype(tag)>::C; });
}

// Optimizer-state table parallel to the chunk table (same cuts), if state is attached.
int build_opt_table(gac_ctx *c) {
    if (c->d_opt_chunks) {
        cudaFree(c->d_opt_chunks);
        c->d_opt_chunks = nullptr;
    }
    if (c->opt_list.empty()) return GAC_OK;
    const uint64_t ce = uint64_t(c->chunk_elems);
    std::vector<OptChunk> table;
    table.reserve(c->n_chunks);
    for (size_t i = 0; i < c->list.size(); ++i) {
        const gac_opt_tensor &o = c->opt_list[i];
        for (uint64_t off = 0; off < c->list[i].numel; off += ce) {
            OptChunk oc;
            oc.p = reinterpret_cast<uint64_t>(o.p) + off * 4;
            oc.m = reinterpret_cast<uint64_t>(o.m) + off * 4;
            oc.v = reinterpret_cast<uint64_t>(o.v) + off * 4;
            oc.pad = 0;
            table.push_back(oc);
        }
    }
    GAC_CUDA(c, cudaMalloc(&c->d_opt_chunks, table.size() * sizeof(OptChunk)));
    GAC_CUDA(c, cudaMemcpy(c->d_opt_chunks, table.data(), table.size() * sizeof(OptChunk),
                           cudaMemcpyHostToDevice));
    c->threads_adamw = with_pair(c->pair, [](auto tag) { return AdamGeom<decltype(tag)>::T; });
    const int ctas = with_pair(c->pair, [](auto tag) { return AdamGeom<decltype(tag)>::C; });
    c->grid_adamw = int(std::min<uint64_t>(uint64_t(c->sms) * ctas, c->n_chunks));
    return GAC_OK;
}

// Cuts the list into chunks and uploads the table; sizes both grids.
int build_table(gac_ctx *c) {
    const uint64_t ce = uint64_t(c->chunk_elems);
    uint64_t n_chunks = 0;
    for (const gac_tensor &t : c->list) n_chunks += (t.numel + ce - 1) / ce;
    if (n_chunks > 0xFFFFFFF0ull)
        return fail(c, GAC_ERR_INVALID_ARG, "too many chunks (%s%lld); raise chunk_elems", "",
                    (long long)n_chunks);
    std::vector<Chunk> table;
    table.reserve(n_chunks);
    const size_t gs = elem_size(c->g_dt), ds = elem_size(c->d_dt);
    c->misaligned = 0;
    for (const gac_tensor &t : c->list) {
        const uint64_t gb = reinterpret_cast<uint64_t>(t.g), db = reinterpret_cast<uint64_t>(t.d);
        const bool aligned = (gb % 16 == 0) && (db % 16 == 0);
        if (!aligned) ++c->misaligned;
        for (uint64_t off = 0; off < t.numel; off += ce) {
            Chunk ch;
            ch.g = gb + off * gs;
            ch.d = db + off * ds;
            ch.n = uint32_t(std::min<uint64_t>(ce, t.numel - off));
            ch.flags = aligned ? kChunkAligned : 0u;
            ch.pad = 0;
            table.push_back(ch);
        }
    }
    if (c->d_chunks) {
        cudaFree(c->d_chunks);
        c->d_chunks = nullptr;
    }
    GAC_CUDA(c, cudaMalloc(&c->d_chunks, table.size() * sizeof(Chunk)));
    GAC_CUDA(c, cudaMemcpy(c->d_chunks, table.data(), table.size() * sizeof(Chunk),
                           cudaMemcpyHostToDevice));
    c->n_chunks = table.size();

    c->threads_stats = stats_threads_of(c->pair);
    c->threads_project = with_pair(c->pair, [](auto tag) { return ProjGeom<decltype(tag)>::T; });
    int occ_s = resident_ctas(stats_kernel_of(c->pair), c->threads_stats);
    const bool beta1 = (c->hp.beta == 1.0), zero = (c->hp.zero_on_violation != 0);
    const int state_mode = c->hp.state_mode;
    ProjectKernel pk = with_pair(c->pair, [=](auto tag) -> ProjectKernel {
        return pick_project<decltype(tag)>(state_mode, beta1, zero);
    });
    c->project_fn = reinterpret_cast<const void *>(pk);
    int occ_p = resident_ctas(pk, c->threads_project);
    const int cap_s = stats_cap_of(c->pair);
    const int cap_p = with_pair(c->pair, [](auto tag) { return ProjGeom<decltype(tag)>::C; });
    if (cap_s > 0) occ_s = std::min(occ_s, cap_s);
    if (cap_p > 0) occ_p = std::min(occ_p, cap_p);
    if (c->ctas_per_sm > 0) {
        occ_s = std::min(occ_s, c->ctas_per_sm);
        occ_p = std::min(occ_p, c->ctas_per_sm);
    }
    c->grid_stats = int(std::min<uint64_t>(uint64_t(c->sms) * occ_s, c->n_chunks));
    c->grid_project = int(std::min<uint64_t>(uint64_t(c->sms) * occ_p, c->n_chunks));
    return build_opt_table(c);
}

int check_hparams(const gac_hparams *hp) {
    if (!(hp->eps >= 0.0) || !isfinite(hp->eps)) return fail(nullptr, GAC_ERR_INVALID_ARG, "eps must be finite and >= 0%s");
    if (!isfinite(hp->beta)) return fail(nullptr, GAC_ERR_INVALID_ARG, "beta must be finite%s");
    if (hp->mode == GAC_MODE_ADAPTIVE) {
        if (!(hp->c_low > 0.0) || !(hp->c_low < hp->c_high) || !isfinite(hp->c_high))
            return fail(nullptr, GAC_ERR_INVALID_ARG, "thresholds must satisfy 0 < c_low < c_high%s");
    } else if (hp->mode == GAC_MODE_FIXED) {
        if (!(hp->alpha_fixed >= 0.0) || !isfinite(hp->alpha_fixed))
            return fail(nullptr, GAC_ERR_INVALID_ARG, "alpha_fixed must be finite and >= 0%s");
    } else {
        return fail(nullptr, GAC_ERR_INVALID_ARG, "unknown mode%s");
    }
    if (hp->state_mode < GAC_STATE_RAW || hp->state_mode > GAC_STATE_HOLD)
        return fail(nullptr, GAC_ERR_INVALID_ARG, "unknown state_mode%s");
    if (hp->zero_on_violation != 0 && hp->zero_on_violation != 1)
        return fail(nullptr, GAC_ERR_INVALID_ARG, "zero_on_violation must be 0 or 1%s");
    if (hp->reserved != 0) return fail(nullptr, GAC_ERR_INVALID_ARG, "reserved field must be 0%s");
    if (!(hp->clip_max_norm >= 0.0) || !isfinite(hp->clip_max_norm) || !(hp->clip_eps >= 0.0) || !isfinite(hp->clip_eps))
        return fail(nullptr, GAC_ERR_INVALID_ARG, "clip_max_norm and clip_eps must be finite and >= 0%s");
    return GAC_OK;
}

DevHP dev_hp(const gac_ctx *c, uint64_t step, uint32_t staleness, int decide) {
    DevHP h;
    h.c_low = c->hp.c_low;
    h.c_high = c->hp.c_high;
    h.eps = c->hp.eps;
    h.beta = c->hp.beta;
    h.alpha_fixed = c->hp.alpha_fixed;
    h.mode = c->hp.mode;
    h.state_mode = c->hp.state_mode;
    h.zero_on_violation = c->hp.zero_on_violation;
    h.first_step = (step == 1);
    h.step = step;
    h.staleness = staleness;
    h.decide = decide;
    h.clip_max = c->hp.clip_max_norm;
    h.clip_eps = c->hp.clip_eps;
    return h;
}

int read_back(gac_ctx *c, cudaStream_t s, gac_result *host_out) {
    GAC_CUDA(c, cudaMemcpyAsync(c->h_rec, c->d_rec, sizeof(gac_result), cudaMemcpyDeviceToHost, s));
    GAC_CUDA(c, cudaStreamSynchronize(s));
    *host_out = *c->h_rec;
    if (host_out->nonfinite)
        return fail(c, GAC_ERR_NONFINITE, "NaN or Inf met in the gradient or the stored direction%s");
    return GAC_OK;
}

int launch_stats(gac_ctx *c, uint64_t step, uint32_t staleness, cudaStream_t s, double *sums_out,
                 int decide) {
    if (step == 0) return fail(c, GAC_ERR_INVALID_ARG, "step counts from 1 (Algorithm 1)%s");
    if (c->started && step <= c->last_projected_step)
        return fail(c, GAC_ERR_STATE, "step %s%lld was already projected", "", (long long)step);
    const DevHP h = dev_hp(c, step, staleness, decide);
    const uint32_t nc = uint32_t(c->n_chunks);
    stats_kernel_of(c->pair)<<<c->grid_stats, c->threads_stats, 0, s>>>(c->d_chunks, nc, c->d_partials, c->d_ticket,
                                                                        c->d_rec, sums_out, h);
    GAC_CUDA(c, cudaGetLastError());
    ++c->launches;
    c->pending_step = step;
    return GAC_OK;
}

}  // namespace

extern "C" {

void gac_default_hparams(gac_hparams *hp) {
    if (!hp) return;
    memset(hp, 0, sizeof(*hp));
    hp->c_low = 0.05;
    hp->c_high = 0.3;
    hp->eps = 1e-8;
    hp->beta = 1.0;
    hp->mode = GAC_MODE_ADAPTIVE;
    hp->state_mode = GAC_STATE_RAW;
    hp->clip_max_norm = 0.0;
    hp->clip_eps = 1e-6;
}

int gac_init(gac_ctx **out, const gac_tensor *list, uint32_t n, int g_dtype, int d_dtype,
             const gac_hparams *hp, int cuda_device) {
    if (!out) return fail(nullptr, GAC_ERR_INVALID_ARG, "out is NULL%s");
    *out = nullptr;
    if (!list || n == 0) return fail(nullptr, GAC_ERR_INVALID_ARG, "empty tensor list%s");
    if (!hp) return fail(nullptr, GAC_ERR_INVALID_ARG, "hp is NULL%s");
    if (pair_id(g_dtype, d_dtype) < 0)
        return fail(nullptr, GAC_ERR_DTYPE, "supported (g,d) element types: (f32,f32), (bf16,f32), (bf16,bf16)%s");
    if (int rc = check_hparams(hp)) return rc;
    const size_t gs = elem_size(g_dtype), ds = elem_size(d_dtype);
    for (uint32_t i = 0; i < n; ++i) {
        if (!list[i].g || !list[i].d)
            return fail(nullptr, GAC_ERR_INVALID_ARG, "tensor %s%lld has a NULL pointer", "", i);
        if (list[i].numel == 0)
            return fail(nullptr, GAC_ERR_INVALID_ARG, "tensor %s%lld has no elements", "", i);
        if (list[i].numel > (1ull << 40))
            return fail(nullptr, GAC_ERR_INVALID_ARG, "tensor %s%lld is larger than 2^40 elements", "", i);
        const uint64_t gb = reinterpret_cast<uint64_t>(list[i].g), db = reinterpret_cast<uint64_t>(list[i].d);
        if (gb % gs || db % ds)
            return fail(nullptr, GAC_ERR_INVALID_ARG, "tensor %s%lld is not element-aligned", "", i);
        // g is updated in place while d is read: the two ranges must not overlap
        if (gb < db + list[i].numel * ds && db < gb + list[i].numel * gs)
            return fail(nullptr, GAC_ERR_INVALID_ARG, "tensor %s%lld: g and d overlap", "", i);
    }
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev == 0)
        return fail(nullptr, GAC_ERR_CUDA, "no CUDA device is available%s");
    if (cuda_device < 0 || cuda_device >= n_dev)
        return fail(nullptr, GAC_ERR_INVALID_ARG, "cuda_device %s%lld out of range", "", cuda_device);

    gac_ctx *c = new (std::nothrow) gac_ctx;
    if (!c) return fail(nullptr, GAC_ERR_INVALID_ARG, "out of host memory%s");
    c->device = cuda_device;
    c->g_dt = g_dtype;
    c->d_dt = d_dtype;
    c->pair = pair_id(g_dtype, d_dtype);
    c->hp = *hp;
    c->list.assign(list, list + n);
    for (uint32_t i = 0; i < n; ++i) c->total += list[i].numel;

    DeviceGuard guard(cuda_device);
    int rc = GAC_OK;
    auto setup = [&]() -> int {
        if (!guard.ok) return fail(c, GAC_ERR_CUDA, "cudaSetDevice failed%s");
        GAC_CUDA(c, cudaDeviceGetAttribute(&c->sms, cudaDevAttrMultiProcessorCount, cuda_device));
        // small inputs: shorter chunks so that every SM still gets work
        while (c->chunk_elems > 4096 && c->total / uint64_t(c->chunk_elems) < uint64_t(4 * c->sms))
            c->chunk_elems /= 2;
        if (int r = build_table(c)) return r;
        GAC_CUDA(c, cudaMalloc(&c->d_partials, size_t(c->sms) * kMaxCtasPerSm * 3 * sizeof(double)));
        GAC_CUDA(c, cudaMalloc(&c->d_ticket, sizeof(unsigned)));
        GAC_CUDA(c, cudaMemset(c->d_ticket, 0, sizeof(unsigned)));
        GAC_CUDA(c, cudaMalloc(&c->d_rec, sizeof(gac_result)));
        GAC_CUDA(c, cudaMemset(c->d_rec, 0, sizeof(gac_result)));
        GAC_CUDA(c, cudaMallocHost(&c->h_rec, sizeof(gac_result)));
        return GAC_OK;
    };
    rc = setup();
    if (rc != GAC_OK) {
        memcpy(g_init_err, c->err, sizeof(g_init_err));
        release_device(c);
        delete c;
        return rc;
    }
    *out = c;
    return GAC_OK;
}

int gac_set_launch(gac_ctx *ctx, int chunk_elems, int ctas_per_sm) {
    if (!ctx) return fail(nullptr, GAC_ERR_INVALID_ARG, "ctx is NULL%s");
    if (ctx->started) return fail(ctx, GAC_ERR_STATE, "launch geometry is fixed once a step has run%s");
    if (chunk_elems > 0) {
        if (chunk_elems % 1024) return fail(ctx, GAC_ERR_INVALID_ARG, "chunk_elems must be a multiple of 1024%s");
        ctx->chunk_elems = chunk_elems;
    }
    if (ctas_per_sm > 0) ctx->ctas_per_sm = std::min(ctas_per_sm, kMaxCtasPerSm);
    DeviceGuard guard(ctx->device);
    return build_table(ctx);
}

int gac_stats(gac_ctx *ctx, uint64_t step, uint32_t staleness, void *cuda_stream, gac_result *host_out) {
    if (!ctx) return fail(nullptr, GAC_ERR_INVALID_ARG, "ctx is NULL%s");
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (int rc = launch_stats(ctx, step, staleness, s, nullptr, 1)) return rc;
    ctx->started = true;
    ctx->stats_pending = false;
    ctx->decision_ready = true;
    return host_out ? read_back(ctx, s, host_out) : GAC_OK;
}

int gac_stats_partial(gac_ctx *ctx, uint64_t step, uint32_t staleness, void *cuda_stream, double *sums_out) {
    if (!ctx) return fail(nullptr, GAC_ERR_INVALID_ARG, "ctx is NULL%s");
    if (!sums_out) return fail(ctx, GAC_ERR_INVALID_ARG, "sums_out is NULL%s");
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (int rc = launch_stats(ctx, step, staleness, s, sums_out, 0)) return rc;
    ctx->started = true;
    ctx->stats_pending = true;
    ctx->decision_ready = false;
    ctx->pending_staleness = staleness;
    return GAC_OK;
}

int gac_decide(gac_ctx *ctx, void *cuda_stream, const double *sums_in, gac_result *host_out) {
    if (!ctx) return fail(nullptr, GAC_ERR_INVALID_ARG, "ctx is NULL%s");
    if (!sums_in) return fail(ctx, GAC_ERR_INVALID_ARG, "sums_in is NULL%s");
    if (!ctx->stats_pending) return fail(ctx, GAC_ERR_STATE, "gac_decide needs a gac_stats_partial first%s");
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const DevHP h = dev_hp(ctx, ctx->pending_step, ctx->pending_staleness, 1);
    gac_decide_kernel<<<1, 32, 0, s>>>(sums_in, ctx->d_rec, h);
    GAC_CUDA(ctx, cudaGetLastError());
    ++ctx->launches;
    ctx->stats_pending = false;
    ctx->decision_ready = true;
    return host_out ? read_back(ctx, s, host_out) : GAC_OK;
}

int gac_project(gac_ctx *ctx, void *cuda_stream, const float *coef_override, gac_result *host_out) {
    if (!ctx) return fail(nullptr, GAC_ERR_INVALID_ARG, "ctx is NULL%s");
    if (!ctx->decision_ready)
        return fail(ctx, GAC_ERR_STATE, "gac_project needs the decision of gac_stats / gac_decide for this step%s");
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const float k = coef_override ? *coef_override : 0.0f;
    const int use = coef_override ? 1 : 0;
    const uint32_t nc = uint32_t(ctx->n_chunks);
    reinterpret_cast<ProjectKernel>(const_cast<void *>(ctx->project_fn))<<<ctx->grid_project, ctx->threads_project, 0, s>>>(
        ctx->d_chunks, nc, ctx->d_rec, k, use, ctx->hp.beta, ctx->hp.clip_max_norm, ctx->hp.clip_eps);
    GAC_CUDA(ctx, cudaGetLastError());
    ++ctx->launches;
    ctx->decision_ready = false;
    ctx->last_projected_step = ctx->pending_step;
    return host_out ? read_back(ctx, s, host_out) : GAC_OK;
}

void gac_default_adamw(gac_adamw *opt) {
    if (!opt) return;
    opt->lr = 1e-6;
    opt->beta1 = 0.9;
    opt->beta2 = 0.999;
    opt->eps = 1e-8;
    opt->weight_decay = 1e-2;
}

int gac_attach_adamw(gac_ctx *ctx, const gac_opt_tensor *list, uint32_t n, uint64_t applied_steps) {
    if (!ctx) return fail(nullptr, GAC_ERR_INVALID_ARG, "ctx is NULL%s");
    if (!list || n != ctx->list.size())
        return fail(ctx, GAC_ERR_INVALID_ARG, "optimizer state list must have one entry per tensor of the context%s");
    if (ctx->hp.state_mode != GAC_STATE_RAW)
        return fail(ctx, GAC_ERR_INVALID_ARG, "the fused optimizer step needs state_mode RAW%s");
    for (uint32_t i = 0; i < n; ++i) {
        const void *ptrs[3] = {list[i].p, list[i].m, list[i].v};
        for (const void *q : ptrs) {
            if (!q) return fail(ctx, GAC_ERR_INVALID_ARG, "optimizer tensor %s%lld has a NULL pointer", "", i);
            if (reinterpret_cast<uint64_t>(q) % 4)
                return fail(ctx, GAC_ERR_INVALID_ARG, "optimizer tensor %s%lld is not element-aligned", "", i);
        }
    }
    DeviceGuard guard(ctx->device);
    ctx->opt_list.assign(list, list + n);
    if (int rc = build_opt_table(ctx)) return rc;
    const unsigned long long t0 = applied_steps;
    GAC_CUDA(ctx, cudaMemcpy(&ctx->d_rec->applied_steps, &t0, sizeof(t0), cudaMemcpyHostToDevice));
    return GAC_OK;
}

int gac_project_adamw(gac_ctx *ctx, void *cuda_stream, const gac_adamw *opt, const float *coef_override,
                      gac_result *host_out) {
    if (!ctx) return fail(nullptr, GAC_ERR_INVALID_ARG, "ctx is NULL%s");
    if (!opt) return fail(ctx, GAC_ERR_INVALID_ARG, "opt is NULL%s");
    if (!ctx->d_opt_chunks) return fail(ctx, GAC_ERR_STATE, "gac_project_adamw needs gac_attach_adamw first%s");
    if (!ctx->decision_ready)
        return fail(ctx, GAC_ERR_STATE, "gac_project_adamw needs the decision of gac_stats / gac_decide for this step%s");
    if (!(opt->lr >= 0.0) || !(opt->beta1 >= 0.0 && opt->beta1 < 1.0) || !(opt->beta2 >= 0.0 && opt->beta2 < 1.0) ||
        !(opt->eps >= 0.0) || !(opt->weight_decay >= 0.0) || !isfinite(opt->lr) || !isfinite(opt->eps) ||
        !isfinite(opt->weight_decay))
        return fail(ctx, GAC_ERR_INVALID_ARG, "AdamW needs lr, eps, weight_decay >= 0 and betas in [0,1)%s");
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const float k = coef_override ? *coef_override : 0.0f;
    const int use = coef_override ? 1 : 0;
    const uint32_t nc = uint32_t(ctx->n_chunks);
    const AdamDev o{opt->lr, opt->beta1, opt->beta2, opt->eps, opt->weight_decay};
    const AdamKernel ak = with_pair(ctx->pair, [](auto tag) -> AdamKernel { return gac_adamw_kernel<decltype(tag)>; });
    ak<<<ctx->grid_adamw, ctx->threads_adamw, 0, s>>>(ctx->d_chunks, ctx->d_opt_chunks, nc, ctx->d_rec, ctx->d_ticket,
                                                      k, use, ctx->hp.beta, ctx->hp.clip_max_norm, ctx->hp.clip_eps, o);
    GAC_CUDA(ctx, cudaGetLastError());
    ++ctx->launches;
    ctx->decision_ready = false;
    ctx->last_projected_step = ctx->pending_step;
    return host_out ? read_back(ctx, s, host_out) : GAC_OK;
}

int gac_free(gac_ctx *ctx) {
    if (!ctx) return GAC_OK;
    {
        DeviceGuard guard(ctx->device);
        release_device(ctx);
    }
    delete ctx;
    return GAC_OK;
}

const char *gac_last_error(const gac_ctx *ctx) { return ctx ? ctx->err : g_init_err; }

int gac_get_info(const gac_ctx *ctx, gac_info *out) {
    if (!ctx || !out) return GAC_ERR_INVALID_ARG;
    out->total_elems = ctx->total;
    out->n_chunks = ctx->n_chunks;
    out->n_tensors = uint32_t(ctx->list.size());
    out->grid = uint32_t(ctx->grid_stats);
    out->threads = uint32_t(ctx->threads_stats);
    out->chunk_elems = uint32_t(ctx->chunk_elems);
    out->launches = ctx->launches;
    out->misaligned_tensors = ctx->misaligned;
    out->reserved = 0;
    return GAC_OK;
}

}  // extern "C"

// ------------------------------------------------ allocation-free statistics
//
// Everything gac_stats needs beyond its inputs and outputs -- the chunk table,
// the per-CTA partial sums and the arrival ticket -- laid out in one array that
// is part of the loaded library image, so that no call ever has to ask the
// driver for device memory.  Every device that loads the library carries its
// own copy (about 2.1 MiB) until the process exits.
namespace {

constexpr uint32_t kStaticMaxChunks = GAC_STATIC_MAX_CHUNKS;
constexpr uint32_t kStaticMaxCtas = 148 * 16 + 256;             // grid never exceeds SMs x resident CTAs
constexpr size_t kStaticTicketOff = 0;                           // one unsigned, rest of the 256 bytes unused
constexpr size_t kStaticPartialsOff = 256;
constexpr size_t kStaticChunksOff = kStaticPartialsOff + ((size_t(kStaticMaxCtas) * 3 * sizeof(double) + 255) / 256) * 256;
constexpr size_t kStaticBytes = kStaticChunksOff + size_t(kStaticMaxChunks) * sizeof(Chunk);
static_assert(kStaticBytes == GAC_STATIC_SCRATCH_BYTES, "the header states the size of the built-in scratch");

static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
struct StaticSetup {
    bool ready = false;
    unsigned char *base = nullptr;   // DEVICE address of g_static_scratch on that device
    int sms = 0;
    int occ[kPairCount] = {0, 0, 0};
};
StaticSetup g_static_setup[kMaxDevices];
std::mutex g_static_mutex;

// Runs once per device, with that device current.  The array's name is only a
// host-side handle here; the address a kernel can use comes from the runtime.
int static_setup(int dev, StaticSetup **out) {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticSetup &st = g_static_setup[dev];
    if (!st.ready) {
        void *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess || !ptr)
            return fail(nullptr, GAC_ERR_CUDA, "cudaGetSymbolAddress failed: %s (CUDA error %lld)",
                        cudaGetErrorString(e), (long long)e);
        e = cudaDeviceGetAttribute(&st.sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess)
            return fail(nullptr, GAC_ERR_CUDA, "cudaDeviceGetAttribute failed: %s (CUDA error %lld)",
                        cudaGetErrorString(e), (long long)e);
        for (int pr = 0; pr < kPairCount; ++pr) {
            st.occ[pr] = resident_ctas(stats_kernel_of(pr), stats_threads_of(pr));
            if (stats_cap_of(pr) > 0) st.occ[pr] = std::min(st.occ[pr], stats_cap_of(pr));
        }
        st.base = static_cast<unsigned char *>(ptr);
        st.ready = true;
    }
    *out = &st;
    return GAC_OK;
}

}  // namespace

extern "C" int gac_stats_static(const gac_tensor *list, uint32_t n, int g_dtype, int d_dtype,
                                const gac_hparams *hp, uint64_t step, uint32_t staleness,
                                int cuda_device, void *cuda_stream, gac_result *result_dev) {
    if (!list || n == 0) return fail(nullptr, GAC_ERR_INVALID_ARG, "empty tensor list%s");
    if (!hp) return fail(nullptr, GAC_ERR_INVALID_ARG, "hp is NULL%s");
    if (!result_dev) return fail(nullptr, GAC_ERR_INVALID_ARG, "result_dev is NULL%s");
    if (step == 0) return fail(nullptr, GAC_ERR_INVALID_ARG, "step counts from 1 (Algorithm 1)%s");
    if (pair_id(g_dtype, d_dtype) < 0)
        return fail(nullptr, GAC_ERR_DTYPE, "supported (g,d) element types: (f32,f32), (bf16,f32), (bf16,bf16)%s");
    if (int rc = check_hparams(hp)) return rc;
    if (cuda_device < 0 || cuda_device >= kMaxDevices)
        return fail(nullptr, GAC_ERR_INVALID_ARG, "cuda_device %s%lld out of range", "", cuda_device);

    // count the chunks first and refuse what does not fit the built-in scratch
    const uint64_t ce = kDefaultChunk;
    const size_t gs = elem_size(g_dtype), ds = elem_size(d_dtype);
    uint64_t n_chunks = 0;
    for (uint32_t i = 0; i < n; ++i) {
        if (!list[i].g || !list[i].d || list[i].numel == 0)
            return fail(nullptr, GAC_ERR_INVALID_ARG, "tensor %s%lld has a NULL pointer or no elements", "", i);
        if (reinterpret_cast<uint64_t>(list[i].g) % gs || reinterpret_cast<uint64_t>(list[i].d) % ds)
            return fail(nullptr, GAC_ERR_INVALID_ARG, "tensor %s%lld is not element-aligned", "", i);
        n_chunks += (list[i].numel + ce - 1) / ce;
        if (n_chunks > kStaticMaxChunks)
            return fail(nullptr, GAC_ERR_INVALID_ARG,
                        "list needs more than %s%lld chunks of 16384 elements: beyond the built-in scratch; "
                        "use gac_init/gac_stats", "", (long long)kStaticMaxChunks);
    }

    DeviceGuard guard(cuda_device);
    if (!guard.ok) return fail(nullptr, GAC_ERR_CUDA, "cudaSetDevice failed%s");
    StaticSetup *st = nullptr;
    if (int rc = static_setup(cuda_device, &st)) return rc;

    // host-side image of the table (host memory only), then one copy into the scratch
    static thread_local std::vector<Chunk> table;
    table.clear();
    table.reserve(n_chunks);
    for (uint32_t i = 0; i < n; ++i) {
        const uint64_t gb = reinterpret_cast<uint64_t>(list[i].g), db = reinterpret_cast<uint64_t>(list[i].d);
        const bool aligned = (gb % 16 == 0) && (db % 16 == 0);
        for (uint64_t off = 0; off < list[i].numel; off += ce) {
            Chunk ch;
            ch.g = gb + off * gs;
            ch.d = db + off * ds;
            ch.n = uint32_t(std::min<uint64_t>(ce, list[i].numel - off));
            ch.flags = aligned ? kChunkAligned : 0u;
            ch.pad = 0;
            table.push_back(ch);
        }
    }
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    Chunk *d_chunks = reinterpret_cast<Chunk *>(st->base + kStaticChunksOff);
    double *d_partials = reinterpret_cast<double *>(st->base + kStaticPartialsOff);
    unsigned *d_ticket = reinterpret_cast<unsigned *>(st->base + kStaticTicketOff);
    // the scratch keeps whatever the previous call left: the ticket must start at zero
    GAC_CUDA(nullptr, cudaMemsetAsync(d_ticket, 0, sizeof(unsigned), s));
    // source is pageable host memory: the call returns once it has been staged, so `table` may be reused
    GAC_CUDA(nullptr, cudaMemcpyAsync(d_chunks, table.data(), table.size() * sizeof(Chunk),
                                      cudaMemcpyHostToDevice, s));
    gac_ctx shell;            // only carries the hyper-parameters into dev_hp()
    shell.hp = *hp;
    const DevHP h = dev_hp(&shell, step, staleness, 1);
    const int pair = pair_id(g_dtype, d_dtype);
    const int occ = st->occ[pair];
    const uint32_t grid = uint32_t(std::min<uint64_t>(std::min<uint64_t>(uint64_t(st->sms) * occ, kStaticMaxCtas), n_chunks));
    stats_kernel_of(pair)<<<grid, stats_threads_of(pair), 0, s>>>(d_chunks, uint32_t(n_chunks), d_partials, d_ticket,
                                                                  result_dev, nullptr, h);
    GAC_CUDA(nullptr, cudaGetLastError());
    return GAC_OK;
}
