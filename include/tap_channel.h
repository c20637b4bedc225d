/*
 * tap_channel.h -- C ABI of TapChannel: the side path that carries target features
 * ("taps") from the pipeline stages that produce them to the draft stage.
 *
 * Paper Section 3.3 ("TapChannel under Pipeline Parallelism"): the draft stage owns a
 * mailbox with one pre-allocated slot per source stage.  A source writes the taps of a
 * microbatch into its slot after its own forward; the draft reads the slot right before
 * its forward for the same microbatch.  Each slot carries a sequence stamp that orders
 * the two sides; for co-located sources (CUDA IPC) the draft clears the stamp after
 * reading, which hands the slot back to the source.  The payload per microbatch is
 * V_Tap = b n sum_s d_s bytes (Eq. tap-comm); every feature crosses once.
 *
 * This build covers the co-located form: slots in the draft process's device memory,
 * mapped into the source processes through CUDA IPC; stamps in a host shared-memory
 * block that every process maps.  All waiting happens on the HOST and is bounded
 * (a timeout returns TAP_ETIMEOUT); no kernel ever waits for another process.
 *   stamp 0      : slot empty, the source may write
 *   stamp s > 0  : the taps of microbatch sequence number s are complete in the slot
 * Source:  wait (bounded) for stamp 0 -> device copy into the slot on its stream -> the
 *          stamp is set to s by a host function queued behind the copy.
 * Draft:   wait (bounded) for stamp s -> queue its reads of the slot on its stream ->
 *          tap_mailbox_release queues a host function behind them that resets the
 *          stamp to 0.
 * The cross-node form of the paper (dedicated NCCL communicator, GPUDirect RDMA) is
 * not built.
 *
 * Every function returns TAP_OK (0) or a negative tap_status; nothing throws.
 */
#ifndef TAP_CHANNEL_H_
#define TAP_CHANNEL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum tap_status {
    TAP_OK = 0,
    TAP_EINVAL = -1,    /* bad argument */
    TAP_ESYS = -2,      /* shared memory could not be created / mapped */
    TAP_ECUDA = -3,     /* a CUDA runtime call failed; see tap_last_cuda_error */
    TAP_ETIMEOUT = -4,  /* a bounded wait ran out */
    TAP_ESTATE = -5     /* the handshake was violated (slot not empty / wrong stamp) */
} tap_status;

const char *tap_status_string(int status);
int tap_last_cuda_error(void);

/* Eq. (tap-comm): bytes delivered per microbatch, b * n * sum_s d_s. */
uint64_t tap_payload_bytes(uint64_t n_rows, const uint32_t *feature_dims, int n_sources, uint32_t elem_bytes);

/* ---- control block: the stamps, in host shared memory (no CUDA involved) ----------
 * tap_ctrl_create   (draft side) creates and zeroes the block `name` ("/something").
 * tap_ctrl_attach   (source side) maps an existing block.
 * tap_ctrl_close    unmaps; unlink != 0 also removes the name (creator only).
 * tap_ctrl_publish  stamp 0 -> seq with the payload size; TAP_ESTATE if the slot is not empty.
 * tap_ctrl_reserve / tap_ctrl_commit  the same in two steps for asynchronous writers:
 *                   reserve takes the empty slot for `seq` at once (TAP_ESTATE if not empty;
 *                   readers do not see the taps yet), commit makes them readable.
 * tap_ctrl_wait     waits at most timeout_s seconds until the stamp equals `want`
 *                   (want = 0: until the slot is empty); *bytes_out (may be NULL) receives
 *                   the published payload size.
 * tap_ctrl_clear    stamp seq -> 0; TAP_ESTATE if the stamp is not seq.
 */
typedef struct tap_ctrl tap_ctrl_t;
int tap_ctrl_create(const char *name, int n_sources, uint64_t slot_bytes, tap_ctrl_t **out);
int tap_ctrl_attach(const char *name, tap_ctrl_t **out);
int tap_ctrl_close(tap_ctrl_t *ctrl, int unlink);
int tap_ctrl_sources(const tap_ctrl_t *ctrl);
uint64_t tap_ctrl_slot_bytes(const tap_ctrl_t *ctrl);
uint64_t tap_ctrl_stamp(const tap_ctrl_t *ctrl, int source);
int tap_ctrl_publish(tap_ctrl_t *ctrl, int source, uint64_t seq, uint64_t bytes);
int tap_ctrl_reserve(tap_ctrl_t *ctrl, int source, uint64_t seq);
int tap_ctrl_commit(tap_ctrl_t *ctrl, int source, uint64_t seq, uint64_t bytes);
int tap_ctrl_wait(tap_ctrl_t *ctrl, int source, uint64_t want, double timeout_s, uint64_t *bytes_out);
int tap_ctrl_clear(tap_ctrl_t *ctrl, int source, uint64_t seq);

/* ---- draft side: the mailbox -------------------------------------------------------
 * tap_mailbox_create allocates n_sources slots of slot_bytes (rounded up to 256) in the
 *   current device's memory (set-up time; the only allocation) and creates the control
 *   block `name`.
 * tap_mailbox_ipc_handle writes the 64-byte CUDA IPC handle of the slot memory, to be
 *   passed to the source processes by any host channel.
 * tap_mailbox_slot   device pointer of a source's slot (valid in the draft process).
 * tap_mailbox_wait   bounded host wait until the taps of sequence `seq` are complete.
 * tap_mailbox_release queues, on `stream`, the hand-back of the slot: once the work
 *   queued on `stream` so far (the draft's reads) has finished, the stamp returns to 0.
 */
typedef struct tap_mailbox tap_mailbox_t;
int tap_mailbox_create(const char *name, int n_sources, uint64_t slot_bytes, tap_mailbox_t **out);
int tap_mailbox_ipc_handle(tap_mailbox_t *mb, void *handle_64_bytes);
void *tap_mailbox_slot(tap_mailbox_t *mb, int source);
uint64_t tap_mailbox_slot_bytes(const tap_mailbox_t *mb);
int tap_mailbox_wait(tap_mailbox_t *mb, int source, uint64_t seq, double timeout_s, uint64_t *bytes_out);
int tap_mailbox_release(tap_mailbox_t *mb, int source, uint64_t seq, void *stream);
int tap_mailbox_destroy(tap_mailbox_t *mb);

/* ---- source side --------------------------------------------------------------------
 * tap_source_open maps the mailbox: through its IPC handle (another process on the same
 *   node), or, with ipc_handle NULL, through `local_slots` = tap_mailbox_slot(mb, 0) when
 *   source and draft share a process.
 * tap_source_send waits (bounded) until the slot is empty, queues the device copy of
 *   `bytes` (<= slot_bytes) from `taps` into the slot on `stream`, and queues behind it
 *   the host function that publishes `seq` (> 0).  Returns without waiting for the copy.
 */
typedef struct tap_source tap_source_t;
int tap_source_open(const char *name, int source, const void *ipc_handle_64_bytes, void *local_slots,
                    tap_source_t **out);
int tap_source_send(tap_source_t *src, const void *taps, uint64_t bytes, uint64_t seq, void *stream,
                    double timeout_s);
int tap_source_close(tap_source_t *src);

#ifdef __cplusplus
}
#endif
#endif /* TAP_CHANNEL_H_ */
