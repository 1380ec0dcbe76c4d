// Chunk files behind the staging ring (host only): the step immediately downstream of pack and
// upstream of unpack in the paper's design.
//   Sec. 6.3: an entry's path is derived from the model configuration and the prefix-block hash,
//             with intermediate directories spreading entries over the namespace; files are read
//             and written with direct I/O; a store writes a uniquely named temporary file in the
//             target directory, then creates the final name with a hard link (atomic, fails if
//             the name exists: first writer wins) and removes the temporary name; readers open
//             only final names, so an entry is either absent or complete.
//   Sec. 2.1: a block's hash covers its tokens and the hash of the preceding block, so equal
//             hashes mean equal prefixes.
#include <errno.h>
#include <fcntl.h>
#include <stdio.h>
#include <string.h>
#include <sys/stat.h>
#include <sys/types.h>
#include <unistd.h>

#include <atomic>
#include <new>
#include <string>

#include "kvc.h"

struct kvc_store {
    std::string root;       // root/model_tag
    bool want_direct;
    std::atomic<int> direct_refused;  // times O_DIRECT was refused and buffered I/O used instead
    std::atomic<uint64_t> seq;        // makes temporary names unique inside the process
    std::atomic<uint64_t> reads, read_bytes, publishes, publish_bytes;  // completed operations
};

namespace {

bool mkdir_p(const std::string &path)
{
    for (size_t i = 1; i <= path.size(); ++i) {
        if (i == path.size() || path[i] == '/') {
            std::string sub = path.substr(0, i);
            if (mkdir(sub.c_str(), 0777) != 0 && errno != EEXIST)
                return false;
        }
    }
    return true;
}

// root/ab/cd/<16 hex digits>.kv : two directory levels from the top two bytes of the hash
void entry_dir(const kvc_store *st, uint64_t hash, std::string *dir)
{
    char buf[16];
    snprintf(buf, sizeof(buf), "/%02x/%02x", (unsigned)(hash >> 56) & 0xff, (unsigned)(hash >> 48) & 0xff);
    *dir = st->root + buf;
}

void entry_path(const kvc_store *st, uint64_t hash, std::string *path)
{
    std::string dir;
    entry_dir(st, hash, &dir);
    char buf[32];
    snprintf(buf, sizeof(buf), "/%016llx.kv", (unsigned long long)hash);
    *path = dir + buf;
}

bool direct_ok(const void *buf, uint64_t bytes)
{
    return ((uintptr_t)buf % 4096) == 0 && (bytes % 4096) == 0 && bytes > 0;
}

int plain_open(const char *path, int flags, unsigned mode) { return open(path, flags, (mode_t)mode); }
std::atomic<kvc_open_fn> g_open{plain_open};

// Opens with O_DIRECT when asked for and possible; falls back to buffered I/O when the file
// system refuses the flag (tmpfs, some overlay file systems).  A refused O_DIRECT open with
// O_CREAT may already have created the (empty) file before failing: it is removed, or the
// buffered retry with O_EXCL would find it and fail.
int open_maybe_direct(kvc_store *st, const char *path, int flags, mode_t mode, bool direct)
{
    const kvc_open_fn do_open = g_open.load();
    if (direct) {
        int fd = do_open(path, flags | O_DIRECT, (unsigned)mode);
        if (fd >= 0 || errno != EINVAL)
            return fd;
        st->direct_refused.fetch_add(1);
        if ((flags & (O_CREAT | O_EXCL)) == (O_CREAT | O_EXCL))
            unlink(path);
    }
    return do_open(path, flags, (unsigned)mode);
}

kvc_status write_all(int fd, const unsigned char *p, uint64_t n)
{
    while (n) {
        ssize_t w = write(fd, p, n > (1u << 30) ? (1u << 30) : (size_t)n);
        if (w < 0) {
            if (errno == EINTR)
                continue;
            return KVC_ERR_IO;
        }
        p += w;
        n -= (uint64_t)w;
    }
    return KVC_OK;
}

kvc_status read_all(int fd, unsigned char *p, uint64_t n)
{
    while (n) {
        ssize_t r = read(fd, p, n > (1u << 30) ? (1u << 30) : (size_t)n);
        if (r < 0) {
            if (errno == EINTR)
                continue;
            return KVC_ERR_IO;
        }
        if (r == 0)
            return KVC_ERR_IO;  // shorter than the caller expects
        p += r;
        n -= (uint64_t)r;
    }
    return KVC_OK;
}

}  // namespace

extern "C" {

uint64_t kvc_chain_hash(uint64_t prev, const int32_t *tokens, uint32_t n_tokens)
{
    // FNV-1a (64 bit) over the previous hash (8 bytes, little endian) followed by the tokens'
    // bytes.  prev = 0 starts a chain.
    uint64_t h = 0xcbf29ce484222325ull;
    const uint64_t prime = 0x100000001b3ull;
    for (int i = 0; i < 8; ++i) {
        h ^= (prev >> (8 * i)) & 0xff;
        h *= prime;
    }
    const unsigned char *p = reinterpret_cast<const unsigned char *>(tokens);
    for (uint64_t i = 0; i < (uint64_t)n_tokens * 4; ++i) {
        h ^= p[i];
        h *= prime;
    }
    return h;
}

uint64_t kvc_fnv1a64(const void *data, uint64_t n)
{
    uint64_t h = 0xcbf29ce484222325ull;
    const unsigned char *p = static_cast<const unsigned char *>(data);
    for (uint64_t i = 0; i < n; ++i) {
        h ^= p[i];
        h *= 0x100000001b3ull;
    }
    return h;
}

kvc_status kvc_store_open(const char *root, const char *model_tag, int direct_io, kvc_store **out)
{
    try {
        if (!root || !model_tag || !out || !*root || !*model_tag || strchr(model_tag, '/'))
            return KVC_ERR_INVALID_ARG;
        *out = nullptr;
        kvc_store *st = new (std::nothrow) kvc_store();
        if (!st)
            return KVC_ERR_NOMEM;
        try {
            st->root = std::string(root) + "/" + model_tag;
        } catch (const std::bad_alloc &) {
            delete st;
            return KVC_ERR_NOMEM;
        }
        st->want_direct = direct_io != 0;
        st->direct_refused = 0;
        st->seq = 0;
        st->reads = st->read_bytes = st->publishes = st->publish_bytes = 0;
        if (!mkdir_p(st->root)) {
            delete st;
            return KVC_ERR_IO;
        }
        *out = st;
        return KVC_OK;
    } catch (const std::bad_alloc &) {
        return KVC_ERR_NOMEM;  // path strings are the only allocations in here
    }
}

kvc_status kvc_store_close(kvc_store *st)
{
    if (!st)
        return KVC_ERR_INVALID_ARG;
    delete st;
    return KVC_OK;
}

kvc_status kvc_store_path(const kvc_store *st, uint64_t hash, char *buf, uint32_t cap)
{
    try {
        if (!st || !buf)
            return KVC_ERR_INVALID_ARG;
        std::string p;
        entry_path(st, hash, &p);
        if (p.size() + 1 > cap)
            return KVC_ERR_INVALID_ARG;
        memcpy(buf, p.c_str(), p.size() + 1);
        return KVC_OK;
    } catch (const std::bad_alloc &) {
        return KVC_ERR_NOMEM;  // path strings are the only allocations in here
    }
}

kvc_status kvc_store_lookup(const kvc_store *st, uint64_t hash, uint64_t *bytes)
{
    try {
        if (!st || !bytes)
            return KVC_ERR_INVALID_ARG;
        std::string p;
        entry_path(st, hash, &p);
        struct stat sb;
        if (stat(p.c_str(), &sb) != 0) {
            *bytes = 0;
            return errno == ENOENT ? KVC_ERR_NOT_FOUND : KVC_ERR_IO;
        }
        *bytes = (uint64_t)sb.st_size;
        return KVC_OK;
    } catch (const std::bad_alloc &) {
        return KVC_ERR_NOMEM;  // path strings are the only allocations in here
    }
}

kvc_status kvc_store_publish(kvc_store *st, uint64_t hash, const void *host_buf, uint64_t bytes)
{
    try {
        if (!st || !host_buf || bytes == 0)
            return KVC_ERR_INVALID_ARG;
        std::string dir, final_path;
        entry_dir(st, hash, &dir);
        entry_path(st, hash, &final_path);
        struct stat sb;
        if (stat(final_path.c_str(), &sb) == 0)
            return KVC_ERR_EXISTS;  // already published: nothing to write
        if (!mkdir_p(dir))
            return KVC_ERR_IO;
        char tmp_name[96];
        snprintf(tmp_name, sizeof(tmp_name), "/.tmp.%016llx.%ld.%llu", (unsigned long long)hash,
                 (long)getpid(), (unsigned long long)st->seq.fetch_add(1));
        const std::string tmp = dir + tmp_name;
        const bool direct = st->want_direct && direct_ok(host_buf, bytes);
        int fd = open_maybe_direct(st, tmp.c_str(), O_WRONLY | O_CREAT | O_EXCL, 0666, direct);
        if (fd < 0) {
            unlink(tmp.c_str());  // a failed create may still have left the name behind
            return KVC_ERR_IO;
        }
        kvc_status rc = write_all(fd, static_cast<const unsigned char *>(host_buf), bytes);
        if (close(fd) != 0 && rc == KVC_OK)
            rc = KVC_ERR_IO;
        if (rc == KVC_OK) {
            // atomic publication: the link fails if another writer got there first
            if (link(tmp.c_str(), final_path.c_str()) != 0)
                rc = errno == EEXIST ? KVC_ERR_EXISTS : KVC_ERR_IO;
        }
        unlink(tmp.c_str());
        if (rc == KVC_OK) {
            st->publishes.fetch_add(1);
            st->publish_bytes.fetch_add(bytes);
        }
        return rc;
    } catch (const std::bad_alloc &) {
        return KVC_ERR_NOMEM;  // path strings are the only allocations in here
    }
}

kvc_status kvc_store_read(kvc_store *st, uint64_t hash, void *host_buf, uint64_t bytes)
{
    try {
        if (!st || !host_buf || bytes == 0)
            return KVC_ERR_INVALID_ARG;
        std::string p;
        entry_path(st, hash, &p);
        const bool direct = st->want_direct && direct_ok(host_buf, bytes);
        int fd = open_maybe_direct(st, p.c_str(), O_RDONLY, 0, direct);
        if (fd < 0)
            return errno == ENOENT ? KVC_ERR_NOT_FOUND : KVC_ERR_IO;
        struct stat sb;
        kvc_status rc = KVC_OK;
        if (fstat(fd, &sb) != 0)
            rc = KVC_ERR_IO;
        else if ((uint64_t)sb.st_size != bytes)
            rc = KVC_ERR_INVALID_ARG;  // the entry is not the size the caller's layout implies
        else
            rc = read_all(fd, static_cast<unsigned char *>(host_buf), bytes);
        close(fd);
        if (rc == KVC_OK) {
            st->reads.fetch_add(1);
            st->read_bytes.fetch_add(bytes);
        }
        return rc;
    } catch (const std::bad_alloc &) {
        return KVC_ERR_NOMEM;  // path strings are the only allocations in here
    }
}

int kvc_store_direct_io_refused(const kvc_store *st) { return st ? st->direct_refused.load() : 0; }

kvc_status kvc_store_get_counters(const kvc_store *st, kvc_store_counters *out)
{
    if (!st || !out)
        return KVC_ERR_INVALID_ARG;
    out->reads = st->reads.load();
    out->read_bytes = st->read_bytes.load();
    out->publishes = st->publishes.load();
    out->publish_bytes = st->publish_bytes.load();
    return KVC_OK;
}

kvc_status kvc_store_set_open_fn(kvc_open_fn fn)
{
    g_open.store(fn ? fn : plain_open);
    return KVC_OK;
}

}  // extern "C"
