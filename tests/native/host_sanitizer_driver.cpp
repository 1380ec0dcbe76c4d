// Exercises the host-only parts of the library (slot policy, chunk files) under
// AddressSanitizer / UBSan.  Usage: driver <scratch directory>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <vector>

#include "kvc.h"

#define CHECK(x)                                                      \
    do {                                                              \
        if (!(x)) {                                                   \
            printf("FAILED line %d: %s\n", __LINE__, #x);             \
            return 1;                                                 \
        }                                                             \
    } while (0)

int main(int argc, char **argv)
{
    if (argc < 2)
        return 2;
    // slot policy: fill, join, reclaim, cancel, release everything
    kvc_slot_pool *pool = nullptr;
    CHECK(kvc_slot_pool_create(5, 2, 2, 1, &pool) == KVC_OK);
    uint32_t slot = 0;
    int joined = 0;
    std::vector<uint32_t> held;
    for (uint64_t k = 0; k < 8; ++k) {
        kvc_status s = kvc_slot_pool_acquire(pool, k % 2 ? KVC_CLASS_PRELOAD : KVC_CLASS_DEMAND_LOAD, k % 5,
                                             &slot, &joined);
        CHECK(s == KVC_OK || s == KVC_ERR_WOULD_BLOCK);
        if (s == KVC_OK)
            held.push_back(slot);
    }
    CHECK(kvc_slot_pool_mark_staged(pool, 99) == KVC_ERR_INVALID_ARG);
    for (uint32_t s : held) {
        kvc_slot_pool_mark_staged(pool, s);  // STATE for joined duplicates: ignored on purpose
        CHECK(kvc_slot_pool_release(pool, s) == KVC_OK);
    }
    kvc_slot_pool_counters c;
    CHECK(kvc_slot_pool_get_counters(pool, &c) == KVC_OK);
    CHECK(c.n_in_flight == 0 && c.n_free + c.n_staged + c.n_retained == 5);
    CHECK(kvc_slot_pool_destroy(pool) == KVC_OK);

    // chunk files: publish, duplicate, read back, wrong size, missing
    kvc_store *st = nullptr;
    CHECK(kvc_store_open(argv[1], "san", 1, &st) == KVC_OK);
    const uint64_t n = 3 * 4096;
    void *buf = nullptr, *back = nullptr;
    CHECK(posix_memalign(&buf, 4096, n) == 0 && posix_memalign(&back, 4096, n) == 0);
    memset(buf, 0x5a, n);
    CHECK(kvc_store_publish(st, 42, buf, n) == KVC_OK);
    CHECK(kvc_store_publish(st, 42, buf, n) == KVC_ERR_EXISTS);
    CHECK(kvc_store_read(st, 42, back, n) == KVC_OK && memcmp(buf, back, n) == 0);
    CHECK(kvc_store_read(st, 42, back, 4096) == KVC_ERR_INVALID_ARG);
    CHECK(kvc_store_read(st, 43, back, n) == KVC_ERR_NOT_FOUND);
    uint64_t sz = 1;
    CHECK(kvc_store_lookup(st, 43, &sz) == KVC_ERR_NOT_FOUND && sz == 0);
    char path[64];
    CHECK(kvc_store_path(st, 42, path, sizeof(path)) == KVC_ERR_INVALID_ARG || strlen(path) < 64);
    int32_t toks[4] = {1, 2, 3, 4};
    CHECK(kvc_chain_hash(0, toks, 4) != kvc_chain_hash(1, toks, 4));
    CHECK(kvc_fnv1a64("a", 1) == 0xaf63dc4c8601ec8cull);
    free(buf);
    free(back);
    CHECK(kvc_store_close(st) == KVC_OK);
    printf("ok\n");
    return 0;
}
