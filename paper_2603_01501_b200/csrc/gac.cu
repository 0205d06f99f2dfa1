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
#include <nvtx3/nvToolsExt.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <utility>
#include <mutex>
#include <new>
#include <vector>

#include "gac.h"

#include "gac_kernels.cuh"

// The ABI's structs as laid out for callers in other languages (the Python binding mirrors them).
static_assert(sizeof(gac_tensor) == 24, "gac_tensor layout");
static_assert(sizeof(gac_hparams) == 72, "gac_hparams layout");
static_assert(sizeof(gac_result) == 112, "gac_result layout");
static_assert(sizeof(gac_opt_tensor) == 24 && sizeof(gac_adamw) == 40, "optimizer structs layout");

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
    // peer exchange of the three sums (gac_exchange_attach)
    uint32_t xchg_world = 0, xchg_rank = 0;
    unsigned long long *d_peers = nullptr;   // device table of every rank's slot array, as addressable from this GPU
    PeerSlot *xchg_slots = nullptr;          // this rank's own slot array (caller-owned)
    unsigned long long xchg_timeout_ns = 0;
    bool posted = false;                     // the pending partial reduction was posted to the peers
    OptChunk *d_opt_chunks = nullptr;   // optimizer state table of gac_attach_adamw
    std::vector<gac_opt_tensor> opt_list;
    int grid_adamw = 0, threads_adamw = 0;

    uint64_t last_projected_step = 0;
    uint64_t pending_step = 0;
    uint32_t pending_staleness = 0;
    bool stats_pending = false;    // a partial reduction waits for gac_decide
    bool decision_ready = false;   // a decision waits for gac_project
    bool started = false;
    int swapped = 0;               // exchange mode: 1 while the list's `d` pointers hold the gradient
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

// Named range around the host side of a call, visible in a timeline profiler; costs one
// pointer test when no tool is attached.
struct Range {
    explicit Range(const char *name) { nvtxRangePushA(name); }
    ~Range() { nvtxRangePop(); }
};

void release_device(gac_ctx *c) {
    if (c->d_chunks) cudaFree(c->d_chunks);
    if (c->d_opt_chunks) cudaFree(c->d_opt_chunks);
    c->d_opt_chunks = nullptr;
    if (c->d_peers) cudaFree(c->d_peers);
    c->d_peers = nullptr;
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
                            double, double, double, AdamDev, int);

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
    const bool plain = (c->hp.beta == 1.0 && c->hp.clip_max_norm == 0.0);   // the paper's own rule: the leaner instantiation
    c->threads_adamw = with_pair(c->pair, [plain](auto tag) {
        return plain ? AdamGeom<decltype(tag)>::T : AdamGeom<decltype(tag)>::TG;
    });
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
    const bool exch = (c->hp.state_mode == GAC_STATE_EXCHANGE);
    c->threads_project = with_pair(c->pair, [exch](auto tag) {
        return exch ? ExchGeom<decltype(tag)>::T : ProjGeom<decltype(tag)>::T;
    });
    int occ_s = resident_ctas(stats_kernel_of(c->pair), c->threads_stats);
    const bool beta1 = (c->hp.beta == 1.0), zero = (c->hp.zero_on_violation != 0);
    const int state_mode = c->hp.state_mode;
    ProjectKernel pk = with_pair(c->pair, [=](auto tag) -> ProjectKernel {
        return pick_project<decltype(tag)>(state_mode, beta1, zero);
    });
    if (!pk) return fail(c, GAC_ERR_DTYPE, "no projection kernel for this state mode and element-type pair%s");
    c->project_fn = reinterpret_cast<const void *>(pk);
    int occ_p = resident_ctas(pk, c->threads_project);
    const int cap_s = stats_cap_of(c->pair);
    const int cap_p = with_pair(c->pair, [exch](auto tag) {
        return exch ? ExchGeom<decltype(tag)>::C : ProjGeom<decltype(tag)>::C;
    });
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
    if (hp->state_mode < GAC_STATE_RAW || hp->state_mode > GAC_STATE_EXCHANGE)
        return fail(nullptr, GAC_ERR_INVALID_ARG, "unknown state_mode%s");
    if (hp->zero_on_violation != 0 && hp->zero_on_violation != 1)
        return fail(nullptr, GAC_ERR_INVALID_ARG, "zero_on_violation must be 0 or 1%s");
    if (hp->reserved != 0) return fail(nullptr, GAC_ERR_INVALID_ARG, "reserved field must be 0%s");
    if (!(hp->clip_max_norm >= 0.0) || !isfinite(hp->clip_max_norm) || !(hp->clip_eps >= 0.0) || !isfinite(hp->clip_eps))
        return fail(nullptr, GAC_ERR_INVALID_ARG, "clip_max_norm and clip_eps must be finite and >= 0%s");
    return GAC_OK;
}

// Pointer, size and overlap checks of a tensor list (host only).
int check_list(gac_ctx *ctx, const gac_tensor *list, uint32_t n, size_t gs, size_t ds) {
    for (uint32_t i = 0; i < n; ++i) {
        if (!list[i].g || !list[i].d)
            return fail(ctx, GAC_ERR_INVALID_ARG, "tensor %s%lld has a NULL pointer", "", i);
        if (list[i].numel == 0)
            return fail(ctx, GAC_ERR_INVALID_ARG, "tensor %s%lld has no elements", "", i);
        if (list[i].numel > (1ull << 40))
            return fail(ctx, GAC_ERR_INVALID_ARG, "tensor %s%lld is larger than 2^40 elements", "", i);
        const uint64_t gb = reinterpret_cast<uint64_t>(list[i].g), db = reinterpret_cast<uint64_t>(list[i].d);
        if (gb % gs || db % ds)
            return fail(ctx, GAC_ERR_INVALID_ARG, "tensor %s%lld is not element-aligned", "", i);
        // g is updated in place while d is read: the two ranges must not overlap
        if (gb < db + list[i].numel * ds && db < gb + list[i].numel * gs)
            return fail(ctx, GAC_ERR_INVALID_ARG, "tensor %s%lld: g and d overlap", "", i);
    }
    {   // every g and every d is written in place: all 2n ranges must be pairwise disjoint
        std::vector<std::pair<uint64_t, uint64_t>> ranges;
        ranges.reserve(2 * size_t(n));
        for (uint32_t i = 0; i < n; ++i) {
            const uint64_t gb = reinterpret_cast<uint64_t>(list[i].g), db = reinterpret_cast<uint64_t>(list[i].d);
            ranges.emplace_back(gb, gb + list[i].numel * gs);
            ranges.emplace_back(db, db + list[i].numel * ds);
        }
        std::sort(ranges.begin(), ranges.end());
        for (size_t i = 1; i < ranges.size(); ++i)
            if (ranges[i].first < ranges[i - 1].second)
                return fail(ctx, GAC_ERR_INVALID_ARG, "buffers of different tensors overlap%s");
    }
    return GAC_OK;
}

DevHP dev_hp(const gac_ctx *c, uint64_t step, uint32_t staleness, int decide, bool exchange = false) {
    DevHP h;
    h.xchg_world = exchange ? c->xchg_world : 0u;
    h.xchg_rank = c->xchg_rank;
    h.xchg_peers = c->d_peers;
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
    h.swapped = c->swapped;
    return h;
}

int read_back(gac_ctx *c, cudaStream_t s, gac_result *host_out) {
    GAC_CUDA(c, cudaMemcpyAsync(c->h_rec, c->d_rec, sizeof(gac_result), cudaMemcpyDeviceToHost, s));
    GAC_CUDA(c, cudaStreamSynchronize(s));
    *host_out = *c->h_rec;
    if (host_out->timed_out)
        return fail(c, GAC_ERR_TIMEOUT, "the sums of step %s%lld did not arrive from every rank within the limit", "",
                    (long long)host_out->step);
    if (host_out->nonfinite)
        return fail(c, GAC_ERR_NONFINITE, "NaN or Inf met in the gradient or the stored direction%s");
    return GAC_OK;
}

int launch_stats(gac_ctx *c, uint64_t step, uint32_t staleness, cudaStream_t s, double *sums_out,
                 int decide, bool exchange = false) {
    if (step == 0) return fail(c, GAC_ERR_INVALID_ARG, "step counts from 1 (Algorithm 1)%s");
    if (c->started && step <= c->last_projected_step)
        return fail(c, GAC_ERR_STATE, "step %s%lld was already projected", "", (long long)step);
    const DevHP h = dev_hp(c, step, staleness, decide, exchange);
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
    if (hp->state_mode == GAC_STATE_EXCHANGE && g_dtype != d_dtype)
        return fail(nullptr, GAC_ERR_DTYPE, "exchange mode swaps the roles of the g and d buffers: both need one element type%s");
    const size_t gs = elem_size(g_dtype), ds = elem_size(d_dtype);
    if (int rc = check_list(nullptr, list, n, gs, ds)) return rc;
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

int gac_rebind(gac_ctx *ctx, const gac_tensor *list, uint32_t n) {
    if (!ctx) return fail(nullptr, GAC_ERR_INVALID_ARG, "ctx is NULL%s");
    if (!list || n != ctx->list.size())
        return fail(ctx, GAC_ERR_INVALID_ARG, "gac_rebind needs one entry per tensor of the context%s");
    for (uint32_t i = 0; i < n; ++i)
        if (list[i].numel != ctx->list[i].numel)
            return fail(ctx, GAC_ERR_INVALID_ARG, "tensor %s%lld changed its element count; create a new context", "", i);
    if (ctx->stats_pending || ctx->decision_ready)
        return fail(ctx, GAC_ERR_STATE, "gac_rebind between gac_stats and gac_project would split a step%s");
    if (int rc = check_list(ctx, list, n, elem_size(ctx->g_dt), elem_size(ctx->d_dt))) return rc;
    DeviceGuard guard(ctx->device);
    ctx->list.assign(list, list + n);
    ctx->swapped = 0;   // exchange mode starts over: the new `g` pointers hold the next gradient
    return build_table(ctx);
}

int gac_stats(gac_ctx *ctx, uint64_t step, uint32_t staleness, void *cuda_stream, gac_result *host_out) {
    if (!ctx) return fail(nullptr, GAC_ERR_INVALID_ARG, "ctx is NULL%s");
    Range range("gac_stats");
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (int rc = launch_stats(ctx, step, staleness, s, nullptr, 1)) return rc;
    ctx->started = true;
    ctx->stats_pending = false;
    ctx->posted = false;
    ctx->decision_ready = true;
    return host_out ? read_back(ctx, s, host_out) : GAC_OK;
}

int gac_stats_partial(gac_ctx *ctx, uint64_t step, uint32_t staleness, void *cuda_stream, double *sums_out) {
    if (!ctx) return fail(nullptr, GAC_ERR_INVALID_ARG, "ctx is NULL%s");
    Range range("gac_stats_partial");
    if (!sums_out) return fail(ctx, GAC_ERR_INVALID_ARG, "sums_out is NULL%s");
    if (reinterpret_cast<uint64_t>(sums_out) % 8)
        return fail(ctx, GAC_ERR_INVALID_ARG, "sums_out must be 8-byte aligned (three doubles)%s");
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (int rc = launch_stats(ctx, step, staleness, s, sums_out, 0)) return rc;
    ctx->started = true;
    ctx->stats_pending = true;
    ctx->posted = false;
    ctx->decision_ready = false;
    ctx->pending_staleness = staleness;
    return GAC_OK;
}

int gac_decide(gac_ctx *ctx, void *cuda_stream, const double *sums_in, gac_result *host_out) {
    if (!ctx) return fail(nullptr, GAC_ERR_INVALID_ARG, "ctx is NULL%s");
    Range range("gac_decide");
    if (!sums_in) return fail(ctx, GAC_ERR_INVALID_ARG, "sums_in is NULL%s");
    if (reinterpret_cast<uint64_t>(sums_in) % 8)
        return fail(ctx, GAC_ERR_INVALID_ARG, "sums_in must be 8-byte aligned (three doubles)%s");
    if (!ctx->stats_pending || ctx->posted)
        return fail(ctx, GAC_ERR_STATE, "gac_decide needs a gac_stats_partial first%s");
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

size_t gac_exchange_bytes(uint32_t world) { return size_t(world) * 2 * sizeof(PeerSlot); }

int gac_exchange_attach(gac_ctx *ctx, uint32_t rank, uint32_t world, void *const *slots, uint32_t timeout_ms) {
    if (!ctx) return fail(nullptr, GAC_ERR_INVALID_ARG, "ctx is NULL%s");
    if (world == 0 || world > GAC_EXCHANGE_MAX_RANKS || rank >= world)
        return fail(ctx, GAC_ERR_INVALID_ARG, "peer exchange needs 1 <= world <= %s%lld and rank < world", "",
                    (long long)GAC_EXCHANGE_MAX_RANKS);
    if (!slots) return fail(ctx, GAC_ERR_INVALID_ARG, "slots is NULL%s");
    if (ctx->stats_pending || ctx->decision_ready)
        return fail(ctx, GAC_ERR_STATE, "gac_exchange_attach between the calls of a step would split it%s");
    unsigned long long table[GAC_EXCHANGE_MAX_RANKS];   // on the stack: this call must not throw
    for (uint32_t r = 0; r < world; ++r) {
        const uint64_t a = reinterpret_cast<uint64_t>(slots[r]);
        if (!a || a % sizeof(PeerSlot))
            return fail(ctx, GAC_ERR_INVALID_ARG, "slot array of rank %s%lld is NULL or not 32-byte aligned", "", r);
        table[r] = a;
    }
    DeviceGuard guard(ctx->device);
    if (ctx->d_peers) {
        cudaFree(ctx->d_peers);
        ctx->d_peers = nullptr;
    }
    GAC_CUDA(ctx, cudaMalloc(&ctx->d_peers, world * sizeof(unsigned long long)));
    GAC_CUDA(ctx, cudaMemcpy(ctx->d_peers, table, world * sizeof(unsigned long long), cudaMemcpyHostToDevice));
    ctx->xchg_world = world;
    ctx->xchg_rank = rank;
    ctx->xchg_slots = static_cast<PeerSlot *>(slots[rank]);
    ctx->xchg_timeout_ns = uint64_t(timeout_ms ? timeout_ms : 1000u) * 1000000ull;
    return GAC_OK;
}

int gac_stats_exchange(gac_ctx *ctx, uint64_t step, uint32_t staleness, void *cuda_stream) {
    if (!ctx) return fail(nullptr, GAC_ERR_INVALID_ARG, "ctx is NULL%s");
    Range range("gac_stats_exchange");
    if (!ctx->xchg_world) return fail(ctx, GAC_ERR_STATE, "gac_stats_exchange needs gac_exchange_attach first%s");
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (int rc = launch_stats(ctx, step, staleness, s, nullptr, 0, true)) return rc;
    ctx->started = true;
    ctx->stats_pending = true;
    ctx->posted = true;
    ctx->decision_ready = false;
    ctx->pending_staleness = staleness;
    return GAC_OK;
}

int gac_decide_exchange(gac_ctx *ctx, void *cuda_stream, gac_result *host_out) {
    if (!ctx) return fail(nullptr, GAC_ERR_INVALID_ARG, "ctx is NULL%s");
    Range range("gac_decide_exchange");
    if (!ctx->stats_pending || !ctx->posted)
        return fail(ctx, GAC_ERR_STATE, "gac_decide_exchange needs a gac_stats_exchange first%s");
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const DevHP h = dev_hp(ctx, ctx->pending_step, ctx->pending_staleness, 1, true);
    gac_decide_exchange_kernel<<<1, kExchangeThreads, 0, s>>>(ctx->xchg_slots, ctx->d_rec, h, ctx->xchg_timeout_ns);
    GAC_CUDA(ctx, cudaGetLastError());
    ++ctx->launches;
    if (host_out) {
        const int rc = read_back(ctx, s, host_out);
        if (rc == GAC_ERR_TIMEOUT) return rc;   // still pending: the call may be repeated once the peers have posted
        ctx->stats_pending = false;
        ctx->posted = false;
        ctx->decision_ready = true;
        return rc;
    }
    ctx->stats_pending = false;
    ctx->posted = false;
    ctx->decision_ready = true;
    return GAC_OK;
}

int gac_project(gac_ctx *ctx, void *cuda_stream, const float *coef_override, gac_result *host_out) {
    if (!ctx) return fail(nullptr, GAC_ERR_INVALID_ARG, "ctx is NULL%s");
    Range range("gac_project");
    if (!ctx->decision_ready)
        return fail(ctx, GAC_ERR_STATE, "gac_project needs the decision of gac_stats / gac_decide for this step%s");
    DeviceGuard guard(ctx->device);
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const float k = coef_override ? *coef_override : 0.0f;
    const int use = coef_override ? 1 : 0;
    const uint32_t nc = uint32_t(ctx->n_chunks);
    reinterpret_cast<ProjectKernel>(const_cast<void *>(ctx->project_fn))<<<ctx->grid_project, ctx->threads_project, 0, s>>>(
        ctx->d_chunks, nc, ctx->d_rec, k, use, ctx->hp.beta, ctx->hp.clip_max_norm, ctx->hp.clip_eps, ctx->swapped);
    GAC_CUDA(ctx, cudaGetLastError());
    ++ctx->launches;
    ctx->decision_ready = false;
    ctx->last_projected_step = ctx->pending_step;
    if (ctx->hp.state_mode == GAC_STATE_EXCHANGE) ctx->swapped ^= 1;   // the buffers that held g are the stored direction now
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
    if (ctx->hp.state_mode != GAC_STATE_RAW && ctx->hp.state_mode != GAC_STATE_EXCHANGE)
        return fail(ctx, GAC_ERR_INVALID_ARG, "the fused optimizer step needs state_mode RAW or EXCHANGE%s");
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
    Range range("gac_project_adamw");
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
    const AdamDev o{opt->lr, opt->beta1, opt->beta2, opt->eps, 1.0 - opt->beta1, 1.0 - opt->beta2,
                    opt->lr * opt->weight_decay};
    const bool exch = (ctx->hp.state_mode == GAC_STATE_EXCHANGE);
    const bool plain = (ctx->hp.beta == 1.0 && ctx->hp.clip_max_norm == 0.0);
    const AdamKernel ak = with_pair(ctx->pair, [exch, plain](auto tag) -> AdamKernel {
        using P = decltype(tag);
        if (plain) return exch ? gac_adamw_kernel<P, true, true> : gac_adamw_kernel<P, false, true>;
        return exch ? gac_adamw_kernel<P, true, false> : gac_adamw_kernel<P, false, false>;
    });
    ak<<<ctx->grid_adamw, ctx->threads_adamw, 0, s>>>(ctx->d_chunks, ctx->d_opt_chunks, nc, ctx->d_rec, ctx->d_ticket,
                                                      k, use, ctx->hp.beta, ctx->hp.clip_max_norm, ctx->hp.clip_eps, o,
                                                      ctx->swapped);
    GAC_CUDA(ctx, cudaGetLastError());
    ++ctx->launches;
    ctx->decision_ready = false;
    ctx->last_projected_step = ctx->pending_step;
    if (exch) ctx->swapped ^= 1;
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

int gac_next_gradient_set(const gac_ctx *ctx, int *set_out) {
    if (!ctx || !set_out) return GAC_ERR_INVALID_ARG;
    *set_out = ctx->swapped ? GAC_SET_D : GAC_SET_G;
    return GAC_OK;
}

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
Chunk g_static_host_table[kStaticMaxChunks];   // host image of the chunk table, filled under the mutex

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
    if (reinterpret_cast<uint64_t>(result_dev) % 8)
        return fail(nullptr, GAC_ERR_INVALID_ARG, "result_dev must be 8-byte aligned (a gac_result holds doubles)%s");
    if (step == 0) return fail(nullptr, GAC_ERR_INVALID_ARG, "step counts from 1 (Algorithm 1)%s");
    if (pair_id(g_dtype, d_dtype) < 0)
        return fail(nullptr, GAC_ERR_DTYPE, "supported (g,d) element types: (f32,f32), (bf16,f32), (bf16,bf16)%s");
    if (int rc = check_hparams(hp)) return rc;
    if (hp->state_mode == GAC_STATE_EXCHANGE)
        return fail(nullptr, GAC_ERR_INVALID_ARG, "exchange mode needs a context (gac_init) to follow the buffer roles%s");
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
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    {
        // A captured copy node would read the library's shared host table when the graph is
        // replayed, after other calls have refilled it: refuse instead of replaying a stale table.
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        GAC_CUDA(nullptr, cudaStreamIsCapturing(s, &cap));
        if (cap != cudaStreamCaptureStatusNone)
            return fail(nullptr, GAC_ERR_STATE,
                        "gac_stats_static cannot be captured in a CUDA graph: its table copy reads a host buffer "
                        "that every call rewrites%s");
    }
    StaticSetup *st = nullptr;
    if (int rc = static_setup(cuda_device, &st)) return rc;

    // Host-side image of the table in a fixed buffer of the library (no heap use either), then one
    // copy into the device scratch.  The lock covers filling and staging: the copy call returns once
    // the pageable source has been staged, after which the buffer may be refilled by another caller.
    Chunk *d_chunks = reinterpret_cast<Chunk *>(st->base + kStaticChunksOff);
    double *d_partials = reinterpret_cast<double *>(st->base + kStaticPartialsOff);
    unsigned *d_ticket = reinterpret_cast<unsigned *>(st->base + kStaticTicketOff);
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        uint64_t filled = 0;
        for (uint32_t i = 0; i < n; ++i) {
            const uint64_t gb = reinterpret_cast<uint64_t>(list[i].g), db = reinterpret_cast<uint64_t>(list[i].d);
            const bool aligned = (gb % 16 == 0) && (db % 16 == 0);
            for (uint64_t off = 0; off < list[i].numel; off += ce) {
                Chunk &ch = g_static_host_table[filled++];
                ch.g = gb + off * gs;
                ch.d = db + off * ds;
                ch.n = uint32_t(std::min<uint64_t>(ce, list[i].numel - off));
                ch.flags = aligned ? kChunkAligned : 0u;
                ch.pad = 0;
            }
        }
        // the scratch keeps whatever the previous call left: the ticket must start at zero
        GAC_CUDA(nullptr, cudaMemsetAsync(d_ticket, 0, sizeof(unsigned), s));
        // the caller's record may hold anything: fields the reduction does not write (applied_steps,
        // ref_lost) read as zero afterwards
        GAC_CUDA(nullptr, cudaMemsetAsync(result_dev, 0, sizeof(gac_result), s));
        GAC_CUDA(nullptr, cudaMemcpyAsync(d_chunks, g_static_host_table, filled * sizeof(Chunk),
                                          cudaMemcpyHostToDevice, s));
    }
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
