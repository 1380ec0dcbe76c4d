// Ceiling probe, independent of the library: how fast can this GPU gather (or scatter) rows of
// S bytes that lie at random places of a large array, when nothing else is in the way?  One plain
// kernel: a warp takes R rows at a time and copies them with eight 16-byte loads in flight per
// lane; the only indirection is one 4-byte index per row.  `bench.py --suite row_gather` builds it
// with nvcc and reports GB/s (bytes read + written) per row size.  The small-slab results of the
// library are read against these figures: they show that random S-byte access is not DRAM-limited
// on B200 down to 256-byte rows.
#include <cuda_runtime.h>
#include <stdint.h>

template <int U>
__global__ void __launch_bounds__(256)
rows_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, const int *__restrict__ idx, int n_rows,
            int vpr, int R, int scatter)
{
    const int lane = threadIdx.x & 31;
    const long warp = ((long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long nwarps = ((long)gridDim.x * blockDim.x) >> 5;
    for (long base = warp * R; base < n_rows; base += nwarps * R) {
        const int rows = (int)min((long)R, n_rows - base);
        const int total = rows * vpr;  // 16-byte vectors in this batch of rows
        for (int v0 = 0; v0 < total; v0 += 32 * U) {
            uint4 r[U];
            size_t to[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * 32 + lane;
                if (v < total) {
                    const int row = v / vpr, off = v - row * vpr;
                    const size_t rnd = (size_t)__ldg(idx + base + row) * vpr + off;
                    const size_t lin = (size_t)(base + row) * vpr + off;
                    const uint4 *from = src + (scatter ? lin : rnd);
                    to[u] = scatter ? rnd : lin;
                    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                                 : "=r"(r[u].x), "=r"(r[u].y), "=r"(r[u].z), "=r"(r[u].w)
                                 : "l"(from));
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int v = v0 + u * 32 + lane;
                if (v < total)
                    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(dst + to[u]), "r"(r[u].x),
                                 "r"(r[u].y), "r"(r[u].z), "r"(r[u].w)
                                 : "memory");
            }
        }
    }
}

// gather: dst[i] = src[idx[i]]; scatter: dst[idx[i]] = src[i]; rows of row_bytes (a multiple of 16).
extern "C" int probe_rows(const void *src, void *dst, const int *idx, int n_rows, int row_bytes, int rows_per_warp,
                          int scatter, int grid, void *stream)
{
    rows_kernel<8><<<grid, 256, 0, (cudaStream_t)stream>>>((const uint4 *)src, (uint4 *)dst, idx, n_rows,
                                                           row_bytes / 16, rows_per_warp, scatter);
    return (int)cudaGetLastError();
}

// Three linear streams over one large array, for context: how far is a copy from what the memory
// does when it only reads, or only writes?  Every thread keeps U 16-byte accesses in flight.
//   mode 0: read only (the values are folded into one word per thread, stored if it is ever zero
//           so that the loads cannot be dropped);  mode 1: write only;  mode 2: copy src -> dst.
template <int U>
__global__ void __launch_bounds__(256)
stream_kernel(const uint4 *__restrict__ src, uint4 *__restrict__ dst, size_t n_vec, int mode, uint32_t *sink)
{
    const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t nthreads = (size_t)gridDim.x * blockDim.x;
    uint32_t acc = 1;
    for (size_t v0 = tid; v0 < n_vec; v0 += nthreads * U) {
        uint4 r[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t v = v0 + (size_t)u * nthreads;
            r[u] = make_uint4(1u, 2u, 3u, (uint32_t)v);
            if (mode != 1 && v < n_vec)
                asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                             : "=r"(r[u].x), "=r"(r[u].y), "=r"(r[u].z), "=r"(r[u].w)
                             : "l"(src + v));
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const size_t v = v0 + (size_t)u * nthreads;
            if (v >= n_vec)
                continue;
            if (mode == 0)
                acc |= r[u].x ^ r[u].y ^ r[u].z ^ r[u].w;
            else
                asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(dst + v), "r"(r[u].x), "r"(r[u].y),
                             "r"(r[u].z), "r"(r[u].w)
                             : "memory");
        }
    }
    if (acc == 0)
        *sink = 0;
}

extern "C" int probe_stream(const void *src, void *dst, size_t bytes, int mode, int grid, void *sink, void *stream)
{
    stream_kernel<8><<<grid, 256, 0, (cudaStream_t)stream>>>((const uint4 *)src, (uint4 *)dst, bytes / 16, mode,
                                                             (uint32_t *)sink);
    return (int)cudaGetLastError();
}
