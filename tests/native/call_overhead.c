/* Host cost and device throughput of the per-chunk entry points, measured from C (no Python in
 * the loop): Sec. 5.1 of the paper contrasts 640 small transfers with 21 large ones; this is
 * the same question for kernel launches.
 *
 *   call_overhead <pool_blocks> <request_blocks> <reps>
 *
 * 8B KV shape (32 layers, K and V, 16-token blocks, 8 KV heads, head dim 128, 2-byte elements).
 * For chunk sizes of 16, 256 and 2048 tokens the request is packed with one kvc_pack call per
 * chunk, on one stream and rotated over four, then unpacked the same way; and once with one
 * batched call.  Also: host time of kvc_pack_batch and kvc_pack_batch_static for 2048 and 8192
 * blocks.  Prints one JSON object per line.  Exit code 0 on success. */
#define _POSIX_C_SOURCE 200809L
#include <cuda_runtime.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <time.h>

#include "kvc.h"

#define CK(x)                                                                                  \
    do {                                                                                       \
        kvc_status s_ = (x);                                                                   \
        if (s_ != KVC_OK) {                                                                    \
            fprintf(stderr, "line %d: %s\n", __LINE__, kvc_status_str(s_));                    \
            return 1;                                                                          \
        }                                                                                      \
    } while (0)
#define CU(x)                                                                                  \
    do {                                                                                       \
        cudaError_t e_ = (x);                                                                  \
        if (e_ != cudaSuccess) {                                                               \
            fprintf(stderr, "line %d: %s\n", __LINE__, cudaGetErrorString(e_));                \
            return 1;                                                                          \
        }                                                                                      \
    } while (0)

static double now_us(void)
{
    struct timespec t;
    clock_gettime(CLOCK_MONOTONIC, &t);
    return t.tv_sec * 1e6 + t.tv_nsec * 1e-3;
}

static int cmp_double(const void *a, const void *b)
{
    double x = *(const double *)a, y = *(const double *)b;
    return x < y ? -1 : x > y;
}

static double median(double *v, int n)
{
    qsort(v, (size_t)n, sizeof(double), cmp_double);
    return n % 2 ? v[n / 2] : 0.5 * (v[n / 2 - 1] + v[n / 2]);
}

#define NSTREAMS 4

int main(int argc, char **argv)
{
    const uint32_t NB = argc > 1 ? (uint32_t)atoi(argv[1]) : 6000;
    const uint32_t n = argc > 2 ? (uint32_t)atoi(argv[2]) : 5000;
    const int reps = argc > 3 ? atoi(argv[3]) : 7;
    const uint32_t L = 32, P = 2, B = 16, H = 8, D = 128, e = 2;
    if (n > NB || reps < 1 || reps > 64)
        return 2;
    const uint64_t per_block = (uint64_t)L * P * B * H * D * e;
    unsigned char *pool = NULL, *staging = NULL;
    CU(cudaMalloc((void **)&pool, per_block * NB));
    CU(cudaMalloc((void **)&staging, per_block * n));
    CU(cudaMemset(pool, 0x5a, per_block * NB));
    int32_t *ids = malloc(sizeof(int32_t) * n);
    uint32_t x = 12345;
    for (uint32_t i = 0; i < n; ++i) { /* distinct ids: a stride coprime with the pool size */
        x = (uint32_t)(((uint64_t)i * 7919u + 13u) % NB);
        ids[i] = (int32_t)x;
    }
    cudaStream_t st[NSTREAMS];
    cudaEvent_t ev0, ev1, fork, join[NSTREAMS];
    for (int i = 0; i < NSTREAMS; ++i) {
        CU(cudaStreamCreateWithFlags(&st[i], cudaStreamNonBlocking));
        CU(cudaEventCreateWithFlags(&join[i], cudaEventDisableTiming));
    }
    CU(cudaEventCreate(&ev0));
    CU(cudaEventCreate(&ev1));
    CU(cudaEventCreateWithFlags(&fork, cudaEventDisableTiming));

    /* the floor: the smallest stream operation the runtime can enqueue (a 16-byte memset), 5000 times */
    {
        double host_us[64], dev_ms[64];
        for (int r = -2; r < reps; ++r) {
            CU(cudaDeviceSynchronize());
            CU(cudaEventRecord(ev0, st[0]));
            const double t0 = now_us();
            for (int c = 0; c < 5000; ++c)
                CU(cudaMemsetAsync(staging + 256 * (c % 64), 0, 16, st[0]));
            const double t1 = now_us();
            CU(cudaEventRecord(ev1, st[0]));
            CU(cudaEventSynchronize(ev1));
            float ms = 0;
            CU(cudaEventElapsedTime(&ms, ev0, ev1));
            if (r >= 0) {
                host_us[r] = (t1 - t0) / 5000;
                dev_ms[r] = ms;
            }
        }
        const double hm = median(host_us, reps), dm = median(dev_ms, reps);
        printf("{\"case\": \"floor_16_byte_memset\", \"calls\": 5000, \"streams\": 1, "
               "\"host_us_per_call\": %.3f, \"device_ms\": %.4f, \"device_us_per_call\": %.3f}\n",
               hm, dm, dm * 1e3 / 5000);
    }

    const uint32_t chunk_tokens[3] = {16, 256, 2048};
    for (int ci = 0; ci < 3; ++ci) {
        kvc_layout_desc desc;
        CK(kvc_layout_desc_init_dense(&desc, pool, L, P, NB, B, H, D, e, chunk_tokens[ci], KVC_CHUNK_LAYER_MAJOR));
        kvc_layout *lay = NULL;
        CK(kvc_layout_create(&desc, &lay));
        const uint32_t bpc = kvc_layout_blocks_per_chunk(lay);
        const uint32_t n_chunks = kvc_layout_num_chunks(lay, n);
        for (int v = 0; v < 3; ++v) {
        /* v = 1: the caller vouches that slots are device memory; v = 2: and that consecutive
         * launches are independent of one another (pdl = 3) */
        const int hint = v >= 1, independent = v == 2;
        kvc_tuning tun;
        memset(&tun, 0, sizeof(tun));
        tun.slot_memory = (uint32_t)hint;
        tun.pdl = independent ? 3u : 0u;
        CK(kvc_layout_set_tuning(lay, &tun));
        if (v == 1 && ci != 0)
            continue;
        for (int dir = 0; dir < 2; ++dir) {
            for (int ns = 1; ns <= NSTREAMS; ns += NSTREAMS - 1) {
                double host_us[64], dev_ms[64];
                for (int r = -2; r < reps; ++r) { /* two warm-up rounds */
                    CU(cudaDeviceSynchronize());
                    CU(cudaEventRecord(ev0, st[0]));
                    CU(cudaEventRecord(fork, st[0]));
                    for (int s = 1; s < ns; ++s)
                        CU(cudaStreamWaitEvent(st[s], fork, 0));
                    const double t0 = now_us();
                    uint64_t off = 0;
                    for (uint32_t c = 0; c < n_chunks; ++c) {
                        const uint32_t first = c * bpc, nb = first + bpc <= n ? bpc : n - first;
                        const uint64_t bytes = kvc_layout_chunk_bytes(lay, nb);
                        if (dir == 0)
                            CK(kvc_pack(lay, ids + first, nb, 0, staging + off, bytes, st[c % ns]));
                        else
                            CK(kvc_unpack(lay, staging + off, bytes, ids + first, nb, 0, st[c % ns]));
                        off += bytes;
                    }
                    const double t1 = now_us();
                    for (int s = 1; s < ns; ++s) {
                        CU(cudaEventRecord(join[s], st[s]));
                        CU(cudaStreamWaitEvent(st[0], join[s], 0));
                    }
                    CU(cudaEventRecord(ev1, st[0]));
                    CU(cudaEventSynchronize(ev1));
                    float ms = 0;
                    CU(cudaEventElapsedTime(&ms, ev0, ev1));
                    if (r >= 0) {
                        host_us[r] = (t1 - t0) / n_chunks;
                        dev_ms[r] = ms;
                    }
                }
                const double hm = median(host_us, reps), dm = median(dev_ms, reps);
                printf("{\"case\": \"per_chunk\", \"direction\": \"%s\", \"chunk_tokens\": %u, \"calls\": %u, "
                       "\"streams\": %d, \"slot_memory_hint\": %d, \"independent_launches\": %d, \"host_us_per_call\": %.3f, "
                       "\"device_ms\": %.4f, \"device_us_per_call\": %.3f, \"gbs\": %.1f}\n",
                       dir ? "unpack" : "pack", chunk_tokens[ci], n_chunks, ns, hint, independent, hm, dm,
                       dm * 1e3 / n_chunks, 2.0 * per_block * n / dm / 1e6);
            }
        }
        }
        uint32_t skipped = 0, expired = 0;
        CK(kvc_poll_device_status(lay, st[0], &skipped, &expired));
        if (skipped || expired)
            return 3;
        CK(kvc_layout_destroy(lay));
    }

    /* batched entry points: host time of one call, allocating and static */
    {
        kvc_layout_desc desc;
        CK(kvc_layout_desc_init_dense(&desc, pool, L, P, NB, B, H, D, e, 256, KVC_CHUNK_LAYER_MAJOR));
        kvc_layout *lay = NULL;
        CK(kvc_layout_create(&desc, &lay));
        const uint32_t sizes[2] = {2048, 8192};
        for (int si = 0; si < 2; ++si) {
            const uint32_t nb_total = sizes[si] <= n ? sizes[si] : n;
            const uint32_t n_ops = kvc_layout_num_chunks(lay, nb_total);
            kvc_chunk_op *ops = calloc(n_ops, sizeof(kvc_chunk_op));
            uint64_t off = 0;
            for (uint32_t c = 0; c < n_ops; ++c) {
                const uint32_t first = c * 16, nb = first + 16 <= nb_total ? 16 : nb_total - first;
                ops[c].slot = staging + off;
                ops[c].ids = ids + first;
                ops[c].n_blocks = nb;
                off += kvc_layout_chunk_bytes(lay, nb);
            }
            for (int which = 0; which < 2; ++which) {
                double idle_us[64], busy_us[64];
                for (int r = -2; r < reps; ++r) {
                    /* idle stream: the call's own cost */
                    CU(cudaDeviceSynchronize());
                    double t0 = now_us();
                    CK(which ? kvc_pack_batch_static(lay, ops, n_ops, st[0]) : kvc_pack_batch(lay, ops, n_ops, 0, st[0]));
                    double t1 = now_us();
                    if (r >= 0)
                        idle_us[r] = t1 - t0;
                    /* busy stream: a second call while the first one's kernel still runs -- does
                     * the call wait for the stream? */
                    t0 = now_us();
                    CK(which ? kvc_pack_batch_static(lay, ops, n_ops, st[0]) : kvc_pack_batch(lay, ops, n_ops, 0, st[0]));
                    t1 = now_us();
                    if (r >= 0)
                        busy_us[r] = t1 - t0;
                }
                CU(cudaDeviceSynchronize());
                printf("{\"case\": \"batched_call_host_time\", \"entry\": \"%s\", \"blocks\": %u, \"ops\": %u, "
                       "\"host_us_idle_stream\": %.2f, \"host_us_busy_stream\": %.2f}\n",
                       which ? "kvc_pack_batch_static" : "kvc_pack_batch", nb_total, n_ops,
                       median(idle_us, reps), median(busy_us, reps));
            }
            free(ops);
        }
        uint32_t a = 0, b = 0;
        CK(kvc_poll_static_status(st[0], &a, &b));
        if (a || b)
            return 3;
        CK(kvc_layout_destroy(lay));
    }
    printf("{\"case\": \"done\"}\n");
    return 0;
}
