// stream_probe -- what HBM delivers for the access patterns of this library's kernels, with the
// arithmetic taken out: R read streams and W write streams of float4, each its own allocation,
// cut into 64 KB chunks that the CTAs take round-robin (chunk c -> CTA c mod grid), T threads
// with U vectors of every read stream in flight per thread, streaming stores.  "in place" means
// that the W results overwrite the last W of the R streams read (as the kernels update g, d, p,
// m, v where they lie); otherwise the results go to W further allocations.  "barriers" keeps
// the warps of a CTA in step: 1 = __syncthreads() after a batch's loads, 2 = after its stores.
//
// The figures it prints are the ceilings the kernels are measured against besides the plain
// copy rate: a kernel that matches the probe of its own pattern is limited by how DRAM serves
// that mix of streams, not by its instructions.
//
//   stream_probe [elements per stream, default 2^30] [stagger bytes, default 0]
//
// With a stagger, stream i starts i x stagger bytes into its allocation (a multiple of 16), so
// that the streams no longer share their low address bits: allocations of one size that come
// from one allocator usually do.
//
// Patterns: 2+0 (fused triple reduction), 2+2 (projection + state refresh),
// 2+1 (projection in exchange mode), 5+4 and 5+3 (projection fused with AdamW, with and
// without the state copy).  One line per pattern and geometry:
//   streams stagger=.. R=.. W=.. place=in|out after=same|read barriers=0..3 T=.. U=.. ctas/sm=.. elems=.. ms=.. GB/s=..
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdio>
#include <cstdlib>

#define CK(x)                                                                          \
    do {                                                                               \
        cudaError_t e_ = (x);                                                          \
        if (e_ != cudaSuccess) {                                                       \
            fprintf(stderr, "CUDA error %s at line %d\n", cudaGetErrorString(e_), __LINE__); \
            return 1;                                                                  \
        }                                                                              \
    } while (0)

constexpr int kChunkVec = 4096;   // 16384 floats = 64 KB per stream and chunk
constexpr int kMaxStreams = 10;

struct Streams {
    float4 *p[kMaxStreams];
};

// BAR bit 0: __syncthreads() between a batch's loads and its stores; bit 1: after its stores.
// The barriers keep the warps of a CTA in step, so that an SM alternates between issuing reads
// and issuing writes instead of sending DRAM an even mix of both.
template <int R, int W, int T, int U, bool INPLACE, int BAR>
__global__ void __launch_bounds__(T, 1) walk(Streams s, size_t n_chunks, uint32_t chunk_vec) {
    constexpr int kFirstOut = INPLACE ? R - W : R;
    const uint32_t tid = threadIdx.x;
    for (size_t c = blockIdx.x; c < n_chunks; c += gridDim.x) {
        float4 *in[R], *out[W > 0 ? W : 1];   // the chunk's first vector in every stream
#pragma unroll
        for (int i = 0; i < R; ++i) in[i] = s.p[i] + c * size_t(chunk_vec);
#pragma unroll
        for (int i = 0; i < W; ++i) out[i] = s.p[kFirstOut + i] + c * size_t(chunk_vec);
        for (uint32_t base = 0; base < chunk_vec; base += T * U) {   // a run-time bound, as in the kernels
            float4 v[R][U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t i = base + u * T + tid;
#pragma unroll
                for (int r = 0; r < R; ++r) v[r][u] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (i < chunk_vec) {
#pragma unroll
                    for (int r = 0; r < R; ++r) v[r][u] = in[r][i];
                }
            }
            if (BAR & 1) __syncthreads();
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t i = base + u * T + tid;
                if (i >= chunk_vec) continue;
                float4 acc = v[0][u];
#pragma unroll
                for (int r = 1; r < R; ++r) {
                    acc.x += v[r][u].x;
                    acc.y += v[r][u].y;
                    acc.z += v[r][u].z;
                    acc.w += v[r][u].w;
                }
#pragma unroll
                for (int w = 0; w < W; ++w) __stcs(&out[w][i], acc);
                if (W == 0 && acc.x == 12345.678f) s.p[0][0] = acc;   // never true: keeps the loads alive
            }
            if (BAR & 2) __syncthreads();
        }
    }
}

template <int R, int W, int T, int U, bool INPLACE = false, int BAR = 0>
int run(size_t n_elems, int ctas_per_sm, size_t stagger, bool after_read = false) {
    static_assert(R + W <= kMaxStreams, "too many streams");
    static_assert(!INPLACE || W <= R, "in place: every result overwrites a stream that was read");
    static_assert(R >= 2, "the read-only pass walks the first two streams");
    constexpr int kAlloc = INPLACE ? R : R + W;
    const size_t n_chunks = n_elems / (size_t(kChunkVec) * 4);
    const size_t bytes = n_chunks * size_t(kChunkVec) * sizeof(float4);
    Streams s;
    void *base[kMaxStreams];
    for (int i = 0; i < kAlloc; ++i) {
        CK(cudaMalloc(&base[i], bytes + stagger * kMaxStreams));
        CK(cudaMemset(base[i], 0x3c + i, bytes + stagger * kMaxStreams));
        s.p[i] = reinterpret_cast<float4 *>(static_cast<char *>(base[i]) + stagger * i);
    }
    int sms = 0;
    CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0));
    cudaEvent_t a, b;
    CK(cudaEventCreate(&a));
    CK(cudaEventCreate(&b));
    // Every timed launch has its own pair of events.  With `after_read` a read-only pass over the
    // first two streams runs before it (untimed), as the reduction runs before the update in a
    // step: the timed pass then starts on an L2 full of clean lines instead of the dirty lines its
    // predecessor left behind.
    const int reps = 10;
    float total = 0.f;
    for (int i = 0; i < 3 + reps; ++i) {
        if (after_read) walk<2, 0, 256, 8, false, 0><<<sms * 4, 256>>>(s, n_chunks, kChunkVec);
        CK(cudaEventRecord(a));
        walk<R, W, T, U, INPLACE, BAR><<<sms * ctas_per_sm, T>>>(s, n_chunks, kChunkVec);
        CK(cudaEventRecord(b));
        CK(cudaEventSynchronize(b));
        float ms1 = 0.f;
        CK(cudaEventElapsedTime(&ms1, a, b));
        if (i >= 3) total += ms1;
    }
    const float ms = total / reps;
    printf("streams stagger=%zu R=%d W=%d place=%s after=%s barriers=%d T=%d U=%d ctas/sm=%d elems=%zu ms=%.3f GB/s=%.0f\n", stagger, R, W,
           INPLACE ? "in" : "out", after_read ? "read" : "same", BAR, T, U, ctas_per_sm, n_chunks * size_t(kChunkVec) * 4, ms,
           double(bytes) * (R + W) / (ms * 1e-3) / 1e9);
    for (int i = 0; i < kAlloc; ++i) cudaFree(base[i]);
    cudaEventDestroy(a);
    cudaEventDestroy(b);
    return 0;
}

int main(int argc, char **argv) {
    const size_t n = argc > 1 ? strtoull(argv[1], nullptr, 10) : (size_t(1) << 30);
    if (n < (size_t(1) << 24) || n > (size_t(1) << 31)) {
        fprintf(stderr, "elements per stream must lie in [2^24, 2^31]\n");
        return 2;
    }
    const size_t g = argc > 2 ? strtoull(argv[2], nullptr, 10) : 0;
    if (g % 16 || g > (size_t(1) << 24)) {
        fprintf(stderr, "stagger must be a multiple of 16 bytes, at most 2^24\n");
        return 2;
    }
    int rc = 0;
    rc |= run<2, 1, 256, 8>(n, 4, g);
    rc |= run<2, 0, 256, 8>(n, 4, g);
    rc |= run<2, 2, 256, 8>(n, 1, g);
    rc |= run<2, 2, 512, 4>(n, 1, g);
    rc |= run<2, 2, 256, 4>(n, 4, g);
    rc |= run<2, 1, 512, 4>(n, 1, g);
    rc |= run<5, 4, 1024, 1>(n, 1, g);
    rc |= run<5, 4, 896, 1>(n, 1, g);
    rc |= run<5, 4, 640, 1>(n, 1, g);
    rc |= run<5, 4, 512, 2>(n, 1, g);
    rc |= run<5, 4, 256, 2>(n, 2, g);
    rc |= run<5, 4, 256, 1>(n, 4, g);
    rc |= run<5, 3, 896, 1>(n, 1, g);
    // the same mixes with the results written over the streams that were read
    rc |= run<2, 2, 256, 8, true>(n, 1, g);
    rc |= run<2, 2, 512, 4, true>(n, 1, g);
    rc |= run<5, 4, 1024, 1, true>(n, 1, g);
    rc |= run<5, 4, 896, 1, true>(n, 1, g);
    rc |= run<5, 4, 640, 1, true>(n, 1, g);
    rc |= run<5, 4, 512, 2, true>(n, 1, g);
    rc |= run<5, 4, 256, 2, true>(n, 2, g);
    rc |= run<5, 4, 256, 4, true>(n, 1, g);
    rc |= run<5, 3, 896, 1, true>(n, 1, g);
    // ... with the warps of a CTA kept in step: barrier after the loads (1), after the stores (2), both (3)
    rc |= run<2, 2, 256, 8, true, 1>(n, 1, g);
    rc |= run<2, 2, 256, 8, true, 2>(n, 1, g);
    rc |= run<2, 2, 256, 8, true, 3>(n, 1, g);
    rc |= run<2, 2, 512, 4, true, 1>(n, 1, g);
    rc |= run<2, 2, 512, 4, true, 2>(n, 1, g);
    rc |= run<2, 1, 512, 4, false, 2>(n, 1, g);
    rc |= run<5, 4, 1024, 1, true, 1>(n, 1, g);
    rc |= run<5, 4, 1024, 1, true, 2>(n, 1, g);
    rc |= run<5, 4, 896, 1, true, 2>(n, 1, g);
    rc |= run<5, 4, 640, 1, true, 2>(n, 1, g);
    rc |= run<5, 4, 512, 2, true, 2>(n, 1, g);
    rc |= run<5, 3, 1024, 1, true, 2>(n, 1, g);
    // ... and each such pass after a read-only pass, as in a step
    rc |= run<2, 2, 256, 8, true>(n, 1, g, true);
    rc |= run<2, 2, 512, 4, true>(n, 1, g, true);
    rc |= run<2, 1, 512, 4>(n, 1, g, true);
    rc |= run<5, 4, 896, 1, true>(n, 1, g, true);
    rc |= run<5, 4, 640, 1, true>(n, 1, g, true);
    rc |= run<5, 4, 256, 2, true>(n, 2, g, true);
    return rc;
}
