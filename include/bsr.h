/*
 * bsr.h -- C interface of the bounded-state restoration (BSR) library for NVIDIA B200.
 *
 * The library restores a complete reusable KV-cache prefix from an external host tier into an
 * engine's paged KV cache through a staging window of at most W chunks, following the paper's
 * three-phase protocol (Section 3 "Protocol: Probe, Install, Commit"):
 *
 *     bsr_probe      complete candidate hit H(S) as knowledge, not residency
 *     bsr_restore    bounded installation: |L(t)| <= W live staged chunks (Eq. 3, Eq. 4)
 *     bsr_commit     expose the advertised prefix only if Q(S) = AND_r AND_g q_{r,g} = 1 (Eq. 6)
 *     bsr_invalidate whole-prefix invalidation on any failure (Proposition 2)
 *
 * Conventions
 *   - Every function returns an int status: BSR_OK (0) or a negative BSR_ERR_* code.  Nothing
 *     throws, aborts or exits.  Out-parameters are written only on BSR_OK unless stated.
 *   - "host" pointers are ordinary CPU addresses; "device" pointers are CUDA device addresses of
 *     the context's GPU.  The library never frees memory it did not allocate.
 *   - Handles (bsr_ctx, bsr_req) are opaque.  A context is bound to one GPU.  Calls on one context
 *     may come from any thread; restores on one context are serialised by a context-wide lock
 *     (Section 3 "Install locally": concurrent requests must not multiply the staging budget)
 *     unless bsr_config.budget_slots sets a shared admission budget for concurrent restores.
 *   - All integer arithmetic of the method is unsigned, modulo 2^64.
 *
 * Functions the paper leaves open and this library defines (documented at each call): the chunk
 * digest and prefix-key chain, the per-(rank, chunk, group) checksum, the chunk byte layout, the
 * paged layout and the validity-bitmap layout.
 */
#ifndef BSR_H_
#define BSR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define BSR_CHUNK_TOKENS 256u /* Section 4 "System topology": the chunk is 256 tokens        */
#define BSR_MAX_GROUPS 8u     /* allocator groups per registration                             */
#define BSR_MAX_RANKS 8u      /* TP rank slices per context                                    */
#define BSR_MAX_TIERS 4u      /* reusable tiers in priority order: 0 first (e.g. remote DRAM),
                                 then lower tiers (e.g. local SSD)                              */

enum {
  BSR_OK = 0,
  BSR_ERR_INVALID = -1,  /* bad argument, W = 0, unknown handle                                */
  BSR_ERR_MISSING = -2,  /* a chunk of the advertised prefix is not in the tier                */
  BSR_ERR_CHECKSUM = -3, /* a staged group segment does not match its stored checksum          */
  BSR_ERR_TIMEOUT = -4,  /* a fill, copy or install did not finish within timeout_ms           */
  BSR_ERR_TRANSFER = -5, /* the tier read or the host-to-device copy reported an error         */
  BSR_ERR_NOMEM = -6,    /* a host or device allocation failed                                 */
  BSR_ERR_ALIGN = -7,    /* bytes_per_token not a multiple of 16, or a pointer not 16-B aligned */
  BSR_ERR_STATE = -8,    /* call not legal in this state (e.g. register after first restore)   */
  BSR_ERR_CUDA = -9      /* a CUDA runtime call failed; see bsr_last_error                     */
};

typedef struct bsr_ctx bsr_ctx;
typedef struct bsr_req bsr_req;

/* Where a tier object's bytes live. */
enum {
  BSR_LOC_HOST = 0,  /* pageable or pinned host memory: restored through the pinned ring       */
  BSR_LOC_DEVICE = 1 /* already in this GPU's memory: installed in place, no staging is used   */
};

/* Which install kernel bsr_restore launches. */
enum { BSR_INSTALL_AUTO = 0, BSR_INSTALL_VECTOR = 1, BSR_INSTALL_BULK = 2 };

typedef struct bsr_config {
  uint32_t window_chunks;     /* W >= 1: pinned staging slots per rank (Eq. 3).  W = 0, the paper's
                                 legacy whole-plan mode (Table 1), is rejected                  */
  uint32_t n_ranks;           /* R: TP rank slices restored by this context, 1..BSR_MAX_RANKS   */
  uint32_t chunk_tokens;      /* must be BSR_CHUNK_TOKENS                                        */
  uint32_t load_concurrency;  /* threads copying tier objects into staging slots (Table 1 "FS
                                 load concurrency": changes throughput, never W or the peak)     */
  uint32_t dev_staging_depth; /* D >= 1 device staging buffers per rank (bounded auxiliary state,
                                 M_aux of Eq. 4; independent of the prefix length); 0 = what
                                 one install launch takes per rank (install_batch / R, at least
                                 16: 32 for the defaults at R = 2); values above 64 are taken as 64 */
  uint32_t timeout_ms;        /* deadline of one bsr_restore call; 0 = 30,000                    */
  uint32_t slot_align;        /* staging slot size = chunk bytes rounded up to this; 0 = 4096    */
  int32_t device;             /* CUDA device ordinal                                             */
  uint64_t reg_id;            /* registration identity mixed into every prefix key               */
  uint32_t install_variant;   /* BSR_INSTALL_*                                                   */
  uint32_t time_kernels;      /* nonzero: bracket every install launch with CUDA events and accumulate
                                 bsr_stats.install_kernel_ms; the kernels also note their own span
                                 (first CTA's start to the last CTA's end, one atomic per CTA) in
                                 bsr_stats.install_span_ms                                        */
  uint32_t direct_install;    /* nonzero: no device staging and no copy-engine transfer; the install
                                 kernel reads the pinned slots over the host link itself (the
                                 staging-free design point of the paper's "Avoiding staging"
                                 discussion): HBM sees each payload byte once instead of three times */
  uint32_t budget_slots;      /* 0: restores on this context are serialised by a lock and each owns W
                                 slots per rank (the paper's prototype).  B > 0: a global admission
                                 budget (Section 7 "Current concurrency is conservative"): restores
                                 run concurrently and share a pool of B slots per rank; each holds
                                 at most W, together never more than B                            */
  uint32_t install_batch;     /* chunk descriptors (chunk x rank) one install launch takes on the
                                 path through the slot pool; 0 = 64.  A launch waits until that many
                                 chunks have been queued for copying: never more per rank than D,
                                 never fewer than one chunk of every rank, and never while nothing
                                 else could make progress.  It does not depend on W: a pinned slot
                                 returns to the pool when its copy into device staging has been
                                 observed complete, not when its launch has (with direct_install
                                 the kernel reads the slots itself: one chunk per launch, slot held
                                 until the launch is done).  Larger launches run the kernel nearer
                                 device-copy speed.  Changes throughput only, never W or the peak */
  uint32_t numa_bind;         /* BSR_NUMA_*: placement of the fill threads and the pinned pool      */
} bsr_config;

/* Host placement.  AUTO: on a host with more than one NUMA node, the fill threads are bound to the
 * CPUs of the node the context's GPU hangs off (as far as the process' own affinity mask allows)
 * and the pinned pool is allocated from a thread bound the same way, so that fills and the GPU's
 * DMA reads stay on one memory controller; a single-node host, or an unknown node, is left alone.
 * OFF: never bind.  ALWAYS: bind whenever the GPU's node is known.  Only thread affinity and page
 * placement of this process are touched, never a setting of the GPU or the driver. */
enum { BSR_NUMA_AUTO = 0, BSR_NUMA_OFF = 1, BSR_NUMA_ALWAYS = 2 };

typedef struct bsr_group_desc {
  uint32_t block_tokens;    /* tokens per paged block; must divide 256                           */
  uint32_t num_phys_blocks; /* size of the group's physical block pool                           */
} bsr_group_desc;

typedef struct bsr_tensor_desc {
  uint32_t group;           /* allocator group of this tensor                                    */
  uint32_t bytes_per_token; /* multiple of 16                                                    */
  void *dev_base;           /* device, caller-owned, 16-byte aligned, at least
                               num_phys_blocks * block_tokens * bytes_per_token bytes            */
} bsr_tensor_desc;

typedef struct bsr_stats {
  uint64_t peak_staging_bytes[BSR_MAX_RANKS];   /* max over time of live slots x slot bytes (Eq. 1) */
  uint64_t ring_bytes_allocated[BSR_MAX_RANKS]; /* pinned pool: W (or budget B) x slot bytes         */
  uint64_t bytes_filled[BSR_MAX_RANKS];         /* tier -> slot                                      */
  uint64_t bytes_h2d[BSR_MAX_RANKS];            /* slot -> device staging                            */
  uint64_t bytes_installed[BSR_MAX_RANKS];      /* verified and scattered                            */
  uint64_t slot_bytes;                          /* staging footprint of one chunk                    */
  uint64_t dev_aux_bytes;                       /* device staging + kernel scratch, all ranks        */
  uint64_t windows;                             /* passes over the ring: K = ceil(N / W)             */
  uint64_t tier_bytes_read_by_probe;            /* stays 0: probe touches the index only             */
  uint64_t kernel_launches;                     /* kernels of this library launched                  */
  uint64_t h2d_copies;                          /* cudaMemcpyAsync calls issued                      */
  uint64_t install_launches;                    /* install kernel launches                           */
  uint64_t bytes_restored_by_tier[BSR_MAX_TIERS]; /* verified and installed, by source tier          */
  double install_kernel_ms;                     /* sum of their device durations (time_kernels)      */
  double last_restore_ms;                       /* host wall time of the last bsr_restore            */
  uint64_t install_descriptors;                 /* chunk descriptors those install launches carried  */
  int64_t fill_numa_node;                       /* node the fill threads and the pool are bound to,
                                                   -1 = not bound (see bsr_config.numa_bind)          */
  double install_span_ms;                       /* sum of the launches' in-kernel spans (time_kernels):
                                                   install_kernel_ms minus launch and completion
                                                   latency; a restore of device-resident objects that
                                                   needs more than 8 launches adds nothing here       */
} bsr_stats;

/* ---- context ------------------------------------------------------------------------------- */

/* Creates a context on cfg->device.  Allocates nothing proportional to a prefix; the pinned slot
 * pool (W slots per rank, or B with an admission budget) and the device staging buffers are
 * allocated at the first restore, when the chunk size is known.
 * Errors: INVALID (W = 0, ranks out of range, chunk_tokens != 256), CUDA (no usable device). */
int bsr_ctx_create(const bsr_config *cfg, bsr_ctx **out);

/* Destroys the context, its slot pool, staging and index.  Release every request of the context
 * first (bsr_req_release) and let no call be in flight on it. */
int bsr_ctx_destroy(bsr_ctx *ctx);

/* Text of the last CUDA or argument error seen by this context (never NULL).  The returned string
 * is a copy that belongs to the calling thread and stays valid until that thread calls
 * bsr_last_error again; calls running on other threads cannot invalidate it.  With several
 * threads failing on one context the text is that of whichever failed last. */
const char *bsr_last_error(bsr_ctx *ctx);

/* ---- registration (Section 4: registered tensors in allocator groups, per TP rank) -------- */

/* Registers rank's paged pools.  groups[G] and tensors[L] are host arrays, copied.  Tensors must
 * be listed group-major (all of group 0, then group 1, ...).  All ranks must register the same
 * geometry; only dev_base differs.  Every group 0..n_groups-1 must own at least one tensor.
 *
 * Chunk byte layout (defined here, the paper only says a chunk "spans the registered per-rank state
 * of its token range"): groups in order; inside a group its tensors in registration order; per
 * tensor 256 tokens x bytes_per_token, token-major.
 * Paged layout: tensor l is an array [num_phys_blocks][block_tokens][bytes_per_token]; logical block
 * j of the request maps to physical block table[j] of the tensor's group.
 * Errors: INVALID, ALIGN, STATE (after the first restore). */
int bsr_register(bsr_ctx *ctx, uint32_t rank, const bsr_group_desc *groups, uint32_t n_groups,
                 const bsr_tensor_desc *tensors, uint32_t n_tensors);

/* Which install kernel the context launches for sources in device memory: BSR_INSTALL_BULK or
 * BSR_INSTALL_VECTOR.  BSR_INSTALL_AUTO means the bulk-copy kernel (level with or ahead of the vector
 * kernel on every registration measured); direct_install always reads host slots with the vector
 * kernel.  Errors: STATE (not every rank registered yet), CUDA. */
int bsr_install_kernel_in_use(bsr_ctx *ctx, int *variant);

/* Bytes of one chunk and of one staging slot under the current registration. */
int bsr_chunk_bytes(bsr_ctx *ctx, uint64_t *chunk_bytes, uint64_t *slot_bytes);

/* ---- external tier + chunk index ---------------------------------------------------------- */

/* Adds (or replaces) the object `key` of `rank`.  `data` (host or device per `location`) is
 * BORROWED: the caller keeps it alive and unmodified for as long as the key is present (tests
 * corrupt it on purpose).  len must equal the chunk bytes.  group_ck[G] (host) are the checksums
 * of the G group segments; NULL makes the library compute them now on the GPU (store path).
 *
 * Checksum (defined here; Table 1 says "verify" without a formula): over the little-endian 32-bit
 * words w_k of a group's segment, k from the segment start, CK = sum_k w_k * (2k + 1) mod 2^64.
 * Errors: INVALID, STATE (no registration), CUDA. */
int bsr_tier_put(bsr_ctx *ctx, uint32_t rank, uint64_t key, const void *data, size_t len,
                 const uint64_t *group_ck, int location);

/* Removes a key (no error if absent).  A chunk may vanish between probe and restore; the restore
 * then fails closed with BSR_ERR_MISSING. */
int bsr_tier_remove(bsr_ctx *ctx, uint32_t rank, uint64_t key);

/* Reads back the stored checksums of a key into out[G] (host).  MISSING if absent. */
int bsr_tier_checksums(bsr_ctx *ctx, uint32_t rank, uint64_t key, uint64_t *out);

/* ---- probe (Section 3 "Probe globally") ---------------------------------------------------- */

/* Computes, on the GPU, one digest per full 256-token chunk and chains them into prefix keys, then
 * looks every key up in the chunk index of every rank.
 *
 *   mix64(x): x += PHI; x = (x ^ x>>32) * PHI; x = (x ^ x>>29) * PHI; return x ^ x>>32
 *             with PHI = 0x9E3779B97F4A7C15
 *   d_i  = sum_{j<256} mix64( ((u64)(u32)tok[256 i + j] << 32 | j) ^ salt )
 *   k_-1 = mix64(salt ^ mix64(reg_id)),   k_i = mix64(k_{i-1} ^ d_i)
 *
 * tok: n_tok int32 ids, host or device per tok_on_device; the trailing n_tok % 256 are ignored.
 * keys_out[N] (host, may be NULL), hit_bitmap_out[ceil(N/64)] (host, may be NULL; bit i = every
 * rank holds key i), n_hit_chunks = length of the longest all-hit prefix.  N = n_tok / 256.
 * Probe reads no payload byte, takes no staging slot and keeps no lock or reference after return.
 * Errors: INVALID, STATE, CUDA. */
int bsr_probe(bsr_ctx *ctx, const int32_t *tok, size_t n_tok, int tok_on_device, uint64_t salt,
              uint64_t *keys_out, uint64_t *hit_bitmap_out, uint32_t *n_hit_chunks);

/* ---- request: advertised prefix and destination blocks (Fig. 2, second box) -------------- */

/* The caller plays the scheduler: it advertises the first n_adv_chunks keys and has allocated the
 * destination blocks.  block_tables is a host array of R*G host pointers, entry r*G+g pointing at
 * n_adv_chunks * 256 / block_tokens[g] int32 physical block ids.  Tables are validated (ids in
 * range, no duplicates within a table) and copied to the device.  Errors: INVALID, NOMEM, CUDA. */
int bsr_req_create(bsr_ctx *ctx, const uint64_t *keys, uint32_t n_adv_chunks,
                   const int32_t *const *block_tables, bsr_req **out);

/* Frees the request and its device-side tables (waits for a call in flight on it).  Nothing the
 * caller passed at creation is referenced afterwards: keys and tables were copied. */
int bsr_req_release(bsr_ctx *ctx, bsr_req *req);

/* ---- restore (Section 2 "Bounded installation", Section 3 "Install locally") -------------- */

/* Installs the advertised prefix of every rank.  Chunk i of rank r is copied from the tier into
 * a free pinned slot of r's pool (this restore holds at most W slots per rank; a slot is live from
 * its admission, before the fill, until its copy into device staging has been observed complete:
 * Eq. 3 bounds the pinned pool, the D staging buffers per rank are the bounded auxiliary state of
 * Eq. 4), copied to a device staging buffer on the library's copy stream, then verified and
 * scattered through the block tables by the install kernel on `cuda_stream` (a cudaStream_t, or
 * NULL for a stream owned by the library).  One install launch takes the chunks queued since the
 * previous one (see bsr_config.install_batch); a staging buffer is reused once the launch that read
 * it has been observed complete.  With direct_install there is no device staging: the kernel reads
 * the slot, which stays live until that launch is done.  Objects that live in device memory are
 * installed in place.  The first
 * missing key, checksum mismatch, transfer error or deadline overrun stops admission, drains what
 * is in flight, invalidates the whole request and is returned.  Blocking; on return no slot is
 * live and every kernel of the call has finished.
 * Returns BSR_OK iff every (rank, group, chunk) was verified and installed. */
int bsr_restore(bsr_ctx *ctx, bsr_req *req, void *cuda_stream);

/* Asynchronous form (Section 3 speaks of "a failed asynchronous restore"): bsr_restore_async starts
 * the same restore on a thread of the library and returns at once; bsr_restore_wait blocks until it
 * has finished and stores its status (the value bsr_restore would have returned) in
 * *restore_status.  One restore per request at a time (STATE otherwise); commit, invalidate and
 * the observability calls on the request wait for it.  Without an admission budget the restores
 * of one context still run one after the other. */
int bsr_restore_async(bsr_ctx *ctx, bsr_req *req, void *cuda_stream);
int bsr_restore_wait(bsr_ctx *ctx, bsr_req *req, int *restore_status);

/* Calibration of the host side of a restore (Section 6.5 keeps throughput apart from the capacity
 * bound: this is the throughput side).  Runs the request's chunks through the same slot pool with
 * the same fill threads, piece size and admission rule as bsr_restore, but stops early:
 *   BSR_CAL_FILL      tier -> pinned slot only; a slot is released as soon as it is full
 *   BSR_CAL_FILL_H2D  ... and slot -> device staging on the copy stream; released when copied
 * No kernel is launched, so the paged cache, the request's bitmap and its commit state are left as
 * they are; byte counters are not advanced (the peak meter is: slots were live).  *seconds = host
 * wall time of the pass.  Comparing request bytes / seconds of the two forms with the link rate
 * and with a full restore tells which stage bounds a restore on this host.
 * Errors: INVALID, STATE (BSR_CAL_FILL_H2D on a direct_install context, which has no device staging),
 * and whatever a restore can return for a missing key or a failed copy. */
enum { BSR_CAL_FILL = 1, BSR_CAL_FILL_H2D = 2 };
int bsr_restore_calibrate(bsr_ctx *ctx, bsr_req *req, int stages, double *seconds);

/* ---- commit / invalidate (Section 3 "Commit at request semantics", Eq. 6, Proposition 2) -- */

/* exposed_chunks = n_adv_chunks iff a restore of the request completed and all validity bits are
 * set; otherwise the request is invalidated and 0 is exposed (a zero-reuse outcome is an answer,
 * not an API error).  Idempotent. */
int bsr_commit(bsr_ctx *ctx, bsr_req *req, uint32_t *exposed_chunks);

#define BSR_SCRUB 1u /* also zero-fill every destination block of the request, all groups/ranks */

/* Clears the whole validity bitmap (healthy ranks and groups included); afterwards commit yields
 * 0.  Idempotent. */
int bsr_invalidate(bsr_ctx *ctx, bsr_req *req, unsigned flags);

/* ---- observability ------------------------------------------------------------------------ */

/* Validity bitmap: bit (r, g, i) lives in word (r*G + g) * ceil(n_adv/64) + i/64 at position
 * i % 64.  `words` must be at least R*G*ceil(n_adv/64). */
int bsr_req_bitmap(bsr_ctx *ctx, bsr_req *req, uint64_t *out, size_t words);

/* The destination blocks an engine must treat as erroneous (Section 4 "vLLM failure integration":
 * a failed retrieve can already have copied a subset of its blocks, so ALL its destination block
 * ids are recorded).  *count = number of ids of (rank, group): every block of the request's table
 * once the request has failed or been invalidated, 0 while it is healthy; the first
 * min(*count, capacity) ids are copied to out. */
int bsr_req_invalid_blocks(bsr_ctx *ctx, bsr_req *req, uint32_t rank, uint32_t group, int32_t *out,
                           size_t capacity, size_t *count);

/* Checksums the install kernel computed, out[(r*G + g) * n_adv + i]; 0 where not installed. */
int bsr_req_checksums(bsr_ctx *ctx, bsr_req *req, uint64_t *out, size_t count);

/* Copies the context's counters (Eq. 1 peak, byte counters of every stage, windows, launches).
 * bsr_reset_stats zeroes them, keeping only the sizes of what stays allocated (slot_bytes,
 * ring_bytes_allocated, dev_aux_bytes). */
int bsr_get_stats(bsr_ctx *ctx, bsr_stats *out);
int bsr_reset_stats(bsr_ctx *ctx);

/* Timeline of one chunk of one rank through the window: nanoseconds since the restore started. */
typedef struct bsr_trace_rec {
  uint32_t chunk, rank, slot, reserved;
  uint64_t t_admit_ns;  /* a slot was reserved for the chunk (it becomes live)                  */
  uint64_t t_filled_ns; /* the last piece of the tier object landed in the slot                 */
  uint64_t t_submit_ns; /* its copies were queued (its install launch follows when its group closes) */
  uint64_t t_done_ns;   /* the slot went back to the pool: the chunk's copy into device staging (with
                           direct_install: its install launch) was observed complete; 0 = never  */
} bsr_trace_rec;

/* Copies the timeline of the most recent restore that went through the slot pool (one record per
 * admitted (chunk, rank), in admission order) into out[capacity]; *count = records available. */
int bsr_get_trace(bsr_ctx *ctx, bsr_trace_rec *out, size_t capacity, size_t *count);

/* How the install kernels cut one chunk of a registration into the spans they move (pure host code, no
 * CUDA call; the same plan bsr_register's geometry gets at its first use).  A span is a contiguous
 * byte range of the chunk of at most 16 KiB: either a piece of ONE destination run (n_runs == 1: bytes
 * [dst_off, dst_off + bytes) of block `block` of tensor `tensor`), or n_runs whole runs of at most
 * 1 KiB each that lie back to back in the chunk (run j is block (block + j) mod blocks-per-chunk of
 * tensor `tensor` + (block + j) / blocks-per-chunk; all those tensors have the same bytes per token).
 * dev_base of the tensor descriptors is ignored.  *count = spans of the plan; the first
 * min(*count, capacity) are written to out.  Errors: INVALID, ALIGN as for bsr_register. */
typedef struct bsr_span_info {
  uint32_t src_off, bytes, dst_off, run_bytes;
  uint32_t tensor, group, block, n_runs;
} bsr_span_info;
int bsr_plan_spans(const bsr_group_desc *groups, uint32_t n_groups, const bsr_tensor_desc *tensors,
                   uint32_t n_tensors, bsr_span_info *out, size_t capacity, size_t *count);

/* How a restore of n_chunks chunks of chunk_bytes bytes on n_ranks rank slices is cut into the pieces
 * that its fill threads fetch (tier -> pinned slot, or the tier's fetch callback) and its copy stream
 * moves, in the order they are handed out (pure host code, no CUDA call; the plan bsr_restore uses
 * with fill_threads = load_concurrency).  Section 4 "Storage-side concurrency is orthogonal": the
 * pieces change when bytes arrive, never how many slots are live.  The pieces of a chunk tile it in
 * ascending offset order; 8 MiB in the body of a prefix, 1 MiB for the first chunk of every rank,
 * growing by 512 KiB per piece from there, 2 MiB for the last chunks (as many as fill_threads pieces of
 * 8 MiB cover), never under 256 KiB unless the chunk is.  *count = pieces of the plan; the first
 * min(*count, capacity) are written to out.  Errors: INVALID (a zero argument, a chunk of 4 GiB or
 * more, more than BSR_MAX_RANKS ranks, more than 2^24 items). */
typedef struct bsr_piece_info {
  uint32_t chunk, rank;   /* the chunk of the prefix and the rank slice the piece belongs to */
  uint32_t offset, bytes; /* bytes [offset, offset + bytes) of that chunk                     */
} bsr_piece_info;
int bsr_plan_pieces(uint64_t chunk_bytes, uint32_t n_chunks, uint32_t n_ranks, uint32_t fill_threads,
                    bsr_piece_info *out, size_t capacity, size_t *count);

/* Host topology helper behind BSR_NUMA_AUTO (pure host code, no CUDA call): reads
 * <sysfs_root>/bus/pci/devices/<pci_bus_id>/numa_node into *node (-1 = the platform does not say),
 * counts the nodes under <sysfs_root>/devices/system/node into *n_nodes (may be NULL) and copies the
 * node's CPU list ("0-15,32-47", empty when *node < 0) into cpulist[cpulist_cap] (may be NULL).
 * sysfs_root is "/sys" on a live system; pci_bus_id as cudaDeviceGetPCIBusId prints it (either case).
 * Errors: INVALID (NULL argument, unparsable file, list longer than the buffer), MISSING (no such
 * device or node directory). */
int bsr_numa_of_pci(const char *sysfs_root, const char *pci_bus_id, int *node, char *cpulist,
                    size_t cpulist_cap, int *n_nodes);

/* ---- host-side failure injection (tests) -------------------------------------------------- */

enum {
  BSR_INJECT_NONE = 0,
  BSR_INJECT_CORRUPT_SLOT = 1, /* flip one word of (rank, group, chunk) in the pinned slot after
                                  the fill, before the device copy                             */
  BSR_INJECT_FILL_ERROR = 2,   /* the tier read of (rank, chunk) reports a transfer error      */
  BSR_INJECT_FILL_STALL = 3,   /* the tier read of (rank, chunk) does not finish before the
                                  deadline                                                     */
  BSR_INJECT_KERNEL_WAIT = 4   /* in the install launch of (rank, chunk) one tile is never loaded and
                                  the kernel's waits are bounded at 50 ms: the waits run out, the
                                  kernel raises its error flag, drains and returns; the restore
                                  reports BSR_ERR_TIMEOUT and the context stays usable           */
};

/* Arms one fault for the next restore (one shot; BSR_INJECT_NONE disarms).  Kinds 1-3 act on host
 * memory and host threads only.  Kind 4 makes a bounded wait inside the kernel expire; nothing is
 * ever made to fault, trap or spin without a limit. */
int bsr_test_inject(bsr_ctx *ctx, int kind, uint32_t rank, uint32_t group, uint32_t chunk,
                    uint64_t seed);

/* ---- request-level recovery (Section 3 "Recover without re-entering the same fault";
 *      Section 6.4: lower valid tier when available, otherwise zero external reuse) ---------- */

/* bsr_tier_put / bsr_tier_remove act on tier 0.  These address any tier 0..BSR_MAX_TIERS-1. */
int bsr_tier_put_at(bsr_ctx *ctx, uint32_t tier, uint32_t rank, uint64_t key, const void *data,
                    size_t len, const uint64_t *group_ck, int location);
int bsr_tier_remove_at(bsr_ctx *ctx, uint32_t tier, uint32_t rank, uint64_t key);

/* Tier adapter (Section 4 "Storage-side concurrency is orthogonal": reads fill the same
 * preallocated window objects).  For a tier whose bytes are not in addressable memory (a file,
 * a remote store), register a fetch function and put the objects with data = NULL, BSR_LOC_HOST
 * and their checksums.  At restore time the library calls, from its fill threads and up to
 * load_concurrency at once,
 *     fn(user, tier, rank, key, offset, len, dst)
 * to deliver bytes [offset, offset + len) of the object straight into the pinned staging slot at
 * dst (pieces of 1 to 8 MiB that tile the object, in no particular order).  Return 0 on success; any other value
 * fails the restore closed with BSR_ERR_TRANSFER.  fn must be thread-safe and must not call back
 * into the context.  NULL removes the adapter. */
typedef int (*bsr_fetch_fn)(void *user, uint32_t tier, uint32_t rank, uint64_t key, uint64_t offset,
                            uint64_t len, void *dst);
int bsr_tier_set_fetch(bsr_ctx *ctx, uint32_t tier, bsr_fetch_fn fn, void *user);

/* Marks a tier reachable (default) or unreachable.  An unreachable tier is skipped by
 * bsr_probe_request, and a restore bound to it fails closed with BSR_ERR_TRANSFER. */
int bsr_tier_set_available(bsr_ctx *ctx, uint32_t tier, int available);

/* Request-scoped probe: same keys and bitmap semantics as bsr_probe, but
 *   - if request_id carries the force-local marker, zero external chunks are reported and no tier
 *     is consulted (tier_out = -1): the request re-enters local prefill;
 *   - otherwise every available tier is probed and ONE tier serves the request: the one with the
 *     longest complete prefix, the higher-priority (lower-numbered) tier on a tie.  hit_bitmap_out
 *     is that tier's raw hit bitmap; tier_out = -1 when nothing is reusable. */
int bsr_probe_request(bsr_ctx *ctx, uint64_t request_id, const int32_t *tok, size_t n_tok,
                      int tok_on_device, uint64_t salt, uint64_t *keys_out, uint64_t *hit_bitmap_out,
                      uint32_t *n_hit_chunks, int *tier_out);

/* Binds a request object to the engine's request identity and to the tier its probe chose.  A
 * bound request whose restore fails (any error) installs the force-local marker for request_id.
 * Unbound requests (the default) restore from tier 0 and leave no marker. */
int bsr_req_bind(bsr_ctx *ctx, bsr_req *req, uint64_t request_id, uint32_t tier);

/* Removes the marker: call after the request reached RUNNING admission or was torn down. */
int bsr_request_done(bsr_ctx *ctx, uint64_t request_id);

int bsr_request_is_force_local(bsr_ctx *ctx, uint64_t request_id, int *out);

/* ---- allocation-free prefix keys ----------------------------------------------------------- */

#define BSR_NOALLOC_MAX_CHUNKS 8192u /* 2,097,152 tokens; the fixed scratch is 64 KiB + 256 B per GPU */

/* The paper has no counterpart of this call; it exists for callers that cannot allocate.
 *
 * Who they are: an engine that has already given (nearly) all device memory to its KV block pool,
 * where a cudaMalloc made later can simply fail; and scheduler-side code running between model
 * steps, where the device-wide synchronisation hidden in cudaMalloc/cudaFree is not acceptable.
 * bsr_probe grows its scratch with cudaMalloc on demand, so such callers use this instead.
 *
 * Computes the same prefix keys as bsr_probe (same digest, same chain, same reg_id mixing) for the
 * n_tok / 256 full chunks of d_tok and writes them to d_keys_out, enqueued on `cuda_stream` (a
 * cudaStream_t, NULL = the default stream).  It does not consult any index and returns as soon as
 * the work is queued; the caller synchronises the stream before reading the keys.
 *   d_tok       device, int32[n_tok], 16-byte aligned, caller-owned
 *   d_keys_out  device, uint64[n_tok / 256], caller-owned
 * The kernel's scratch lives in a fixed array inside the library image, so the call performs no
 * cudaMalloc, cudaFree or other allocating routine.  Consequences the caller must know:
 *   - at most BSR_NOALLOC_MAX_CHUNKS chunks per call; more is rejected with BSR_ERR_INVALID and a
 *     message on stderr, nothing is launched;
 *   - the first call on each GPU looks up the array's device address (one-time set-up); make that
 *     first call outside any stream capture;
 *   - all calls on one GPU share the one array: two calls whose kernels can overlap on the GPU
 *     (different streams, no ordering between them) race and produce wrong keys.  Calls on one
 *     stream, or otherwise ordered, are safe; each call clears what it needs before use.
 * Errors: INVALID (device out of range, NULL pointer, too many chunks), ALIGN, CUDA. */
int bsr_probe_keys_noalloc(int device, const int32_t *d_tok, size_t n_tok, uint64_t salt,
                           uint64_t reg_id, uint64_t *d_keys_out, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* BSR_H_ */
