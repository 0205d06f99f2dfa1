// stream_probe -- what HBM delivers for the access patterns of this library's kernels, with the
// arithmetic taken out: R read streams and W write streams of float4, each its own allocation,
// cut into 64 KB chunks that the CTAs take round-robin (chunk c -> CTA c mod grid), T threads
// with U vectors of every read stream in flight per thread, streaming stores.
//
// The figures it prints are the ceilings the kernels are measured against besides the plain
// copy rate: a kernel that matches the probe of its own pattern is limited by how DRAM serves
// that mix of streams, not by its instructions.
//
//   stream_probe [elements per stream, default 2^30]
//
// Patterns: 1+1 (copy), 2+0 (fused triple reduction), 2+2 (projection + state refresh),
// 2+1 (projection in exchange mode), 5+4 and 5+3 (projection fused with AdamW, with and
// without the state copy).  One line per pattern and geometry:
//   streams R=.. W=.. T=.. U=.. ctas/sm=.. elems=.. ms=.. GB/s=..
#include <cuda_runtime.h>

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

template <int R, int W, int T, int U>
__global__ void __launch_bounds__(T, 1) walk(Streams s, size_t n_chunks) {
    for (size_t c = blockIdx.x; c < n_chunks; c += gridDim.x) {
        const size_t off = c * size_t(kChunkVec);
        for (int base = 0; base < kChunkVec; base += T * U) {
            float4 v[R][U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int i = base + u * T + threadIdx.x;
#pragma unroll
                for (int r = 0; r < R; ++r) v[r][u] = i < kChunkVec ? s.p[r][off + i] : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int i = base + u * T + threadIdx.x;
                float4 acc = v[0][u];
#pragma unroll
                for (int r = 1; r < R; ++r) {
                    acc.x += v[r][u].x;
                    acc.y += v[r][u].y;
                    acc.z += v[r][u].z;
                    acc.w += v[r][u].w;
                }
                if (i < kChunkVec) {
#pragma unroll
                    for (int w = 0; w < W; ++w) __stcs(&s.p[R + w][off + i], acc);
                }
                if (W == 0 && acc.x == 12345.678f) s.p[0][0] = acc;   // never true: keeps the loads alive
            }
        }
    }
}

template <int R, int W, int T, int U>
int run(size_t n_elems, int ctas_per_sm) {
    static_assert(R + W <= kMaxStreams, "too many streams");
    const size_t n_chunks = n_elems / (size_t(kChunkVec) * 4);
    const size_t bytes = n_chunks * size_t(kChunkVec) * sizeof(float4);
    Streams s;
    for (int i = 0; i < R + W; ++i) {
        CK(cudaMalloc(&s.p[i], bytes));
        CK(cudaMemset(s.p[i], 0, bytes));
    }
    int sms = 0;
    CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0));
    cudaEvent_t a, b;
    CK(cudaEventCreate(&a));
    CK(cudaEventCreate(&b));
    for (int i = 0; i < 3; ++i) walk<R, W, T, U><<<sms * ctas_per_sm, T>>>(s, n_chunks);
    CK(cudaDeviceSynchronize());
    const int reps = 10;
    CK(cudaEventRecord(a));
    for (int i = 0; i < reps; ++i) walk<R, W, T, U><<<sms * ctas_per_sm, T>>>(s, n_chunks);
    CK(cudaEventRecord(b));
    CK(cudaEventSynchronize(b));
    float ms = 0.f;
    CK(cudaEventElapsedTime(&ms, a, b));
    ms /= reps;
    printf("streams R=%d W=%d T=%d U=%d ctas/sm=%d elems=%zu ms=%.3f GB/s=%.0f\n", R, W, T, U, ctas_per_sm,
           n_chunks * size_t(kChunkVec) * 4, ms, double(bytes) * (R + W) / (ms * 1e-3) / 1e9);
    for (int i = 0; i < R + W; ++i) cudaFree(s.p[i]);
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
    int rc = 0;
    rc |= run<1, 1, 256, 8>(n, 1);
    rc |= run<1, 1, 256, 8>(n, 4);
    rc |= run<2, 0, 256, 8>(n, 4);
    rc |= run<2, 2, 256, 8>(n, 1);
    rc |= run<2, 2, 512, 4>(n, 1);
    rc |= run<2, 2, 256, 4>(n, 4);
    rc |= run<2, 1, 512, 4>(n, 1);
    rc |= run<5, 4, 1024, 1>(n, 1);
    rc |= run<5, 4, 896, 1>(n, 1);
    rc |= run<5, 4, 640, 1>(n, 1);
    rc |= run<5, 4, 512, 2>(n, 1);
    rc |= run<5, 4, 256, 2>(n, 2);
    rc |= run<5, 4, 256, 1>(n, 4);
    rc |= run<5, 3, 896, 1>(n, 1);
    return rc;
}
