// TapChannel, co-located form: per-source mailbox slots in the draft process's device
// memory (CUDA IPC), sequence stamps in host shared memory, bounded host-side waits.
// Paper Section 3.3; the handshake is described in tap_channel.h.
#include <cuda_runtime.h>
#include <fcntl.h>
#include <sys/mman.h>
#include <sys/stat.h>
#include <unistd.h>

#include <atomic>
#include <chrono>
#include <cstdlib>
#include <cstring>
#include <new>
#include <thread>

#include "tap_channel.h"

namespace {

thread_local int g_last_cuda_error = 0;

#define TAP_CUDA_CHECK(expr)                      \
    do {                                          \
        cudaError_t e__ = (expr);                 \
        if (e__ != cudaSuccess) {                 \
            g_last_cuda_error = (int)e__;         \
            return TAP_ECUDA;                     \
        }                                         \
    } while (0)

constexpr uint64_t kMagic = 0x54415043484e4c31ull;   // "TAPCHNL1"
constexpr int kMaxSources = 256;

struct alignas(64) SlotCtrl {
    std::atomic<uint64_t> stamp;   // 0 = empty, s > 0 = taps of sequence s complete
    std::atomic<uint64_t> bytes;   // payload size of the published taps
};
static_assert(sizeof(SlotCtrl) == 64, "one cache line per slot");
static_assert(std::atomic<uint64_t>::is_always_lock_free, "stamps must be plain 64-bit atomics");

struct CtrlBlock {
    uint64_t magic;
    int32_t n_sources;
    int32_t reserved;
    uint64_t slot_bytes;
    char pad[40];
    SlotCtrl slot[1];
};

size_t ctrl_bytes(int n) { return sizeof(CtrlBlock) + (size_t)(n - 1) * sizeof(SlotCtrl); }

}  // namespace

struct tap_ctrl {
    CtrlBlock *blk;
    size_t bytes;
    char name[128];
};

struct tap_mailbox {
    tap_ctrl *ctrl;
    char *slots;          // device
    uint64_t slot_bytes;  // rounded to 256
    int n_sources;
};

struct tap_source {
    tap_ctrl *ctrl;
    char *slots;          // device pointer of slot 0 in THIS process
    bool mapped_by_ipc;
    int source;
};

extern "C" const char *tap_status_string(int status) {
    switch (status) {
        case TAP_OK: return "ok";
        case TAP_EINVAL: return "invalid argument";
        case TAP_ESYS: return "shared memory could not be created or mapped";
        case TAP_ECUDA: return "CUDA runtime error";
        case TAP_ETIMEOUT: return "bounded wait ran out";
        case TAP_ESTATE: return "handshake violated (slot not empty or wrong stamp)";
        default: return "unknown status";
    }
}

extern "C" int tap_last_cuda_error(void) { return g_last_cuda_error; }

extern "C" uint64_t tap_payload_bytes(uint64_t n_rows, const uint32_t *feature_dims, int n_sources,
                                      uint32_t elem_bytes) {
    if (!feature_dims || n_sources < 0) return 0;
    uint64_t sum = 0;
    for (int s = 0; s < n_sources; ++s) sum += feature_dims[s];
    return (uint64_t)elem_bytes * n_rows * sum;
}

// ------------------------------------------------------------------ control block

static int map_block(const char *name, bool create, int n_sources, uint64_t slot_bytes, tap_ctrl **out) {
    if (!out) return TAP_EINVAL;
    *out = nullptr;
    if (!name || name[0] != '/' || strlen(name) >= sizeof(((tap_ctrl *)0)->name)) return TAP_EINVAL;
    int fd;
    size_t bytes;
    if (create) {
        if (n_sources < 1 || n_sources > kMaxSources || slot_bytes == 0) return TAP_EINVAL;
        bytes = ctrl_bytes(n_sources);
        shm_unlink(name);   // a stale block of an earlier run with the same name
        fd = shm_open(name, O_CREAT | O_EXCL | O_RDWR, 0600);
        if (fd < 0) return TAP_ESYS;
        if (ftruncate(fd, (off_t)bytes) != 0) { close(fd); shm_unlink(name); return TAP_ESYS; }
    } else {
        fd = shm_open(name, O_RDWR, 0600);
        if (fd < 0) return TAP_ESYS;
        struct stat st;
        if (fstat(fd, &st) != 0 || (size_t)st.st_size < sizeof(CtrlBlock)) { close(fd); return TAP_ESYS; }
        bytes = (size_t)st.st_size;
    }
    void *p = mmap(nullptr, bytes, PROT_READ | PROT_WRITE, MAP_SHARED, fd, 0);
    close(fd);
    if (p == MAP_FAILED) { if (create) shm_unlink(name); return TAP_ESYS; }
    CtrlBlock *blk = (CtrlBlock *)p;
    if (create) {
        memset(p, 0, bytes);
        blk->n_sources = n_sources;
        blk->slot_bytes = slot_bytes;
        for (int s = 0; s < n_sources; ++s) {
            new (&blk->slot[s].stamp) std::atomic<uint64_t>(0);
            new (&blk->slot[s].bytes) std::atomic<uint64_t>(0);
        }
        std::atomic_thread_fence(std::memory_order_release);
        blk->magic = kMagic;
    } else if (blk->magic != kMagic || blk->n_sources < 1 || blk->n_sources > kMaxSources ||
               bytes < ctrl_bytes(blk->n_sources)) {
        munmap(p, bytes);
        return TAP_ESYS;
    }
    tap_ctrl *c = (tap_ctrl *)calloc(1, sizeof(tap_ctrl));
    if (!c) { munmap(p, bytes); return TAP_ESYS; }
    c->blk = blk;
    c->bytes = bytes;
    strncpy(c->name, name, sizeof(c->name) - 1);
    *out = c;
    return TAP_OK;
}

extern "C" int tap_ctrl_create(const char *name, int n_sources, uint64_t slot_bytes, tap_ctrl_t **out) {
    return map_block(name, true, n_sources, slot_bytes, out);
}

extern "C" int tap_ctrl_attach(const char *name, tap_ctrl_t **out) { return map_block(name, false, 0, 0, out); }

extern "C" int tap_ctrl_close(tap_ctrl_t *ctrl, int unlink) {
    if (!ctrl) return TAP_EINVAL;
    munmap(ctrl->blk, ctrl->bytes);
    if (unlink) shm_unlink(ctrl->name);
    free(ctrl);
    return TAP_OK;
}

extern "C" int tap_ctrl_sources(const tap_ctrl_t *ctrl) { return ctrl ? ctrl->blk->n_sources : TAP_EINVAL; }
extern "C" uint64_t tap_ctrl_slot_bytes(const tap_ctrl_t *ctrl) { return ctrl ? ctrl->blk->slot_bytes : 0; }

static inline bool source_ok(const tap_ctrl *c, int source) {
    return c && source >= 0 && source < c->blk->n_sources;
}

extern "C" uint64_t tap_ctrl_stamp(const tap_ctrl_t *ctrl, int source) {
    if (!source_ok(ctrl, source)) return ~0ull;
    return ctrl->blk->slot[source].stamp.load(std::memory_order_acquire);
}

extern "C" int tap_ctrl_publish(tap_ctrl_t *ctrl, int source, uint64_t seq, uint64_t bytes) {
    if (!source_ok(ctrl, source) || seq == 0 || (seq >> 63) || bytes > ctrl->blk->slot_bytes) return TAP_EINVAL;
    SlotCtrl &s = ctrl->blk->slot[source];
    s.bytes.store(bytes, std::memory_order_relaxed);
    uint64_t expect = 0;
    if (!s.stamp.compare_exchange_strong(expect, seq, std::memory_order_release, std::memory_order_relaxed))
        return TAP_ESTATE;
    return TAP_OK;
}

// Two-step publication for asynchronous writers: the slot is taken on the host when the copy is
// queued (so that a second send cannot slip in before the first has landed), and becomes
// readable when the copy has finished.
constexpr uint64_t kReserved = 1ull << 63;

extern "C" int tap_ctrl_reserve(tap_ctrl_t *ctrl, int source, uint64_t seq) {
    if (!source_ok(ctrl, source) || seq == 0 || (seq & kReserved)) return TAP_EINVAL;
    uint64_t expect = 0;
    if (!ctrl->blk->slot[source].stamp.compare_exchange_strong(expect, seq | kReserved, std::memory_order_acq_rel,
                                                               std::memory_order_relaxed))
        return TAP_ESTATE;
    return TAP_OK;
}

extern "C" int tap_ctrl_commit(tap_ctrl_t *ctrl, int source, uint64_t seq, uint64_t bytes) {
    if (!source_ok(ctrl, source) || seq == 0 || (seq & kReserved) || bytes > ctrl->blk->slot_bytes) return TAP_EINVAL;
    SlotCtrl &s = ctrl->blk->slot[source];
    s.bytes.store(bytes, std::memory_order_relaxed);
    uint64_t expect = seq | kReserved;
    if (!s.stamp.compare_exchange_strong(expect, seq, std::memory_order_release, std::memory_order_relaxed))
        return TAP_ESTATE;
    return TAP_OK;
}

extern "C" int tap_ctrl_wait(tap_ctrl_t *ctrl, int source, uint64_t want, double timeout_s, uint64_t *bytes_out) {
    if (!source_ok(ctrl, source) || !(timeout_s >= 0.0)) return TAP_EINVAL;
    SlotCtrl &s = ctrl->blk->slot[source];
    const auto t0 = std::chrono::steady_clock::now();
    for (unsigned spins = 0;; ++spins) {
        if (s.stamp.load(std::memory_order_acquire) == want) {
            if (bytes_out) *bytes_out = s.bytes.load(std::memory_order_relaxed);
            return TAP_OK;
        }
        const double waited = std::chrono::duration<double>(std::chrono::steady_clock::now() - t0).count();
        if (waited >= timeout_s) return TAP_ETIMEOUT;
        if (spins < 200) std::this_thread::yield();
        else std::this_thread::sleep_for(std::chrono::microseconds(50));
    }
}

extern "C" int tap_ctrl_clear(tap_ctrl_t *ctrl, int source, uint64_t seq) {
    if (!source_ok(ctrl, source) || seq == 0) return TAP_EINVAL;
    uint64_t expect = seq;
    if (!ctrl->blk->slot[source].stamp.compare_exchange_strong(expect, 0, std::memory_order_release,
                                                               std::memory_order_relaxed))
        return TAP_ESTATE;
    return TAP_OK;
}

// ---------------------------------------------------------------------- draft side

extern "C" int tap_mailbox_create(const char *name, int n_sources, uint64_t slot_bytes, tap_mailbox_t **out) {
    if (!out) return TAP_EINVAL;
    *out = nullptr;
    if (slot_bytes == 0 || n_sources < 1 || n_sources > kMaxSources) return TAP_EINVAL;
    const uint64_t rounded = (slot_bytes + 255) / 256 * 256;
    tap_ctrl *ctrl = nullptr;
    int rc = tap_ctrl_create(name, n_sources, rounded, &ctrl);
    if (rc != TAP_OK) return rc;
    void *slots = nullptr;
    cudaError_t e = cudaMalloc(&slots, (size_t)rounded * n_sources);   // set-up time: the mailbox's slots
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        tap_ctrl_close(ctrl, 1);
        return TAP_ECUDA;
    }
    tap_mailbox *mb = (tap_mailbox *)calloc(1, sizeof(tap_mailbox));
    if (!mb) { cudaFree(slots); tap_ctrl_close(ctrl, 1); return TAP_ESYS; }
    mb->ctrl = ctrl;
    mb->slots = (char *)slots;
    mb->slot_bytes = rounded;
    mb->n_sources = n_sources;
    *out = mb;
    return TAP_OK;
}

extern "C" int tap_mailbox_ipc_handle(tap_mailbox_t *mb, void *handle_64_bytes) {
    if (!mb || !handle_64_bytes) return TAP_EINVAL;
    static_assert(sizeof(cudaIpcMemHandle_t) == 64, "IPC handle size");
    cudaIpcMemHandle_t h;
    TAP_CUDA_CHECK(cudaIpcGetMemHandle(&h, mb->slots));
    memcpy(handle_64_bytes, &h, sizeof h);
    return TAP_OK;
}

extern "C" void *tap_mailbox_slot(tap_mailbox_t *mb, int source) {
    if (!mb || source < 0 || source >= mb->n_sources) return nullptr;
    return mb->slots + (size_t)source * mb->slot_bytes;
}

extern "C" uint64_t tap_mailbox_slot_bytes(const tap_mailbox_t *mb) { return mb ? mb->slot_bytes : 0; }

extern "C" int tap_mailbox_wait(tap_mailbox_t *mb, int source, uint64_t seq, double timeout_s, uint64_t *bytes_out) {
    if (!mb || seq == 0) return TAP_EINVAL;
    return tap_ctrl_wait(mb->ctrl, source, seq, timeout_s, bytes_out);
}

namespace {
struct StampJob {
    tap_ctrl *ctrl;
    int source;
    uint64_t seq, bytes;
    bool publish;   // else clear
};
// Runs on a CUDA-internal thread once everything queued before it on the stream has finished.
// Only touches the stamp (host functions must not call CUDA).
void CUDART_CB stamp_job(void *arg) {
    StampJob *j = (StampJob *)arg;
    if (j->publish) tap_ctrl_commit(j->ctrl, j->source, j->seq, j->bytes);
    else tap_ctrl_clear(j->ctrl, j->source, j->seq);
    delete j;
}
}  // namespace

extern "C" int tap_mailbox_release(tap_mailbox_t *mb, int source, uint64_t seq, void *stream) {
    if (!mb || source < 0 || source >= mb->n_sources || seq == 0) return TAP_EINVAL;
    if (tap_ctrl_stamp(mb->ctrl, source) != seq) return TAP_ESTATE;   // nothing of that sequence to hand back
    StampJob *j = new (std::nothrow) StampJob{mb->ctrl, source, seq, 0, false};
    if (!j) return TAP_ESYS;
    cudaError_t e = cudaLaunchHostFunc((cudaStream_t)stream, stamp_job, j);
    if (e != cudaSuccess) { delete j; g_last_cuda_error = (int)e; return TAP_ECUDA; }
    return TAP_OK;
}

extern "C" int tap_mailbox_destroy(tap_mailbox_t *mb) {
    if (!mb) return TAP_EINVAL;
    cudaDeviceSynchronize();   // queued stamp jobs refer to the control block
    cudaFree(mb->slots);
    tap_ctrl_close(mb->ctrl, 1);
    free(mb);
    return TAP_OK;
}

// --------------------------------------------------------------------- source side

extern "C" int tap_source_open(const char *name, int source, const void *ipc_handle_64_bytes, void *local_slots,
                               tap_source_t **out) {
    if (!out) return TAP_EINVAL;
    *out = nullptr;
    if (!ipc_handle_64_bytes && !local_slots) return TAP_EINVAL;
    tap_ctrl *ctrl = nullptr;
    int rc = tap_ctrl_attach(name, &ctrl);
    if (rc != TAP_OK) return rc;
    if (source < 0 || source >= ctrl->blk->n_sources) { tap_ctrl_close(ctrl, 0); return TAP_EINVAL; }
    void *slots = local_slots;
    if (ipc_handle_64_bytes) {
        cudaIpcMemHandle_t h;
        memcpy(&h, ipc_handle_64_bytes, sizeof h);
        cudaError_t e = cudaIpcOpenMemHandle(&slots, h, cudaIpcMemLazyEnablePeerAccess);
        if (e != cudaSuccess) { g_last_cuda_error = (int)e; tap_ctrl_close(ctrl, 0); return TAP_ECUDA; }
    }
    tap_source *s = (tap_source *)calloc(1, sizeof(tap_source));
    if (!s) { if (ipc_handle_64_bytes) cudaIpcCloseMemHandle(slots); tap_ctrl_close(ctrl, 0); return TAP_ESYS; }
    s->ctrl = ctrl;
    s->slots = (char *)slots;
    s->mapped_by_ipc = ipc_handle_64_bytes != nullptr;
    s->source = source;
    *out = s;
    return TAP_OK;
}

extern "C" int tap_source_send(tap_source_t *src, const void *taps, uint64_t bytes, uint64_t seq, void *stream,
                               double timeout_s) {
    if (!src || !taps || seq == 0 || bytes == 0 || bytes > src->ctrl->blk->slot_bytes) return TAP_EINVAL;
    // the slot is mine again only once the draft has read the previous taps (stamp back to 0)
    int rc = tap_ctrl_wait(src->ctrl, src->source, 0, timeout_s, nullptr);
    if (rc != TAP_OK) return rc;
    if ((rc = tap_ctrl_reserve(src->ctrl, src->source, seq)) != TAP_OK) return rc;   // mine until the draft clears it
    char *dst = src->slots + (size_t)src->source * src->ctrl->blk->slot_bytes;
    cudaStream_t st = (cudaStream_t)stream;
    StampJob *j = new (std::nothrow) StampJob{src->ctrl, src->source, seq, bytes, true};
    cudaError_t e = j ? cudaMemcpyAsync(dst, taps, (size_t)bytes, cudaMemcpyDeviceToDevice, st) : cudaErrorMemoryAllocation;
    if (e == cudaSuccess) e = cudaLaunchHostFunc(st, stamp_job, j);   // publish once the copy has landed
    if (e != cudaSuccess) {     // nothing will publish: give the slot back
        delete j;
        src->ctrl->blk->slot[src->source].stamp.store(0, std::memory_order_release);
        g_last_cuda_error = (int)e;
        return TAP_ECUDA;
    }
    return TAP_OK;
}

extern "C" int tap_source_close(tap_source_t *src) {
    if (!src) return TAP_EINVAL;
    cudaDeviceSynchronize();   // queued stamp jobs refer to the control block
    if (src->mapped_by_ipc) cudaIpcCloseMemHandle(src->slots);
    tap_ctrl_close(src->ctrl, 0);
    free(src);
    return TAP_OK;
}
