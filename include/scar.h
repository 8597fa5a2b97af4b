/*
 * scar.h - C ABI of the SCAR checkpoint-and-recover parameter pass on one GPU.
 *
 * The library keeps a running checkpoint z of a caller-owned parameter buffer
 * x in device memory and offers the two strategies of the paper's Section 4:
 *   - prioritized partial checkpoints (Section 4.2, protocol of Section 4.3):
 *     score every block by its distance to the saved copy, take the fraction
 *     r with the largest scores, refresh z on those blocks and emit them as a
 *     contiguous payload;
 *   - partial recovery (Section 4.1): restore only the lost blocks from z and
 *     report the perturbation ||z_S - x_S|| that the iteration-cost bound of
 *     Theorem 3.2 depends on.
 *
 * Terms.  An element is 4 bytes (float32 or int32).  A block is a contiguous
 * element range and is the unit of scoring, selection and loss (the paper's
 * "parameter": a row, a layer or a shard of a layer, Section 5.1).  A shard is
 * a contiguous range of blocks standing for one parameter-server node.
 *
 * Conventions for every call.
 *   - Return value: SCAR_OK (0) or a negative SCAR_ERR_* code; nothing throws.
 *     Arguments are validated before any GPU work is enqueued, so a call that
 *     fails validation leaves every buffer untouched.
 *   - Pointer names say where the memory lives: d_* device, h_* host.
 *   - All GPU work of a context runs on the CUDA stream given at init, in call
 *     order.  A call whose result pointer `out` is NULL only enqueues; with a
 *     non-NULL `out` it also waits for the stream and fills `out`.
 *     Enqueue-only calls use no host synchronisation and read no caller-owned
 *     host memory after they return, so they can be recorded by CUDA stream
 *     capture on the context's stream: saves, recoveries and norms with device
 *     block masks or with shard masks of up to 1024 shards (their flags travel
 *     in launch parameters; a replay uses the mask of the capture), and
 *     scar_ckpt_load.  A shard-mask call on a context with more than 1024
 *     shards waits for the stream and is not capturable.
 *   - One context serves one caller at a time (no internal locking).
 *   - There is no CPU fallback: without a usable CUDA device init fails.
 */
#ifndef SCAR_H
#define SCAR_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct scar_ctx scar_ctx; /* opaque; created by scar_ckpt_init, freed by scar_ckpt_destroy */

/* Element type.  SCAR_F32 scores blocks by the squared l2 distance (the norm of
 * the appendix proofs of Theorems 4.1/4.2); SCAR_I32 by the integer l1 distance
 * (twice the length-scaled total variation that Appendix C uses for LDA). */
typedef enum { SCAR_F32 = 0, SCAR_I32 = 1 } scar_dtype;

/* Which norm measures the distance of a block to its saved copy.  DEFAULT is the
 * one above for the element type.  L1 on SCAR_F32 data scores a block by
 * sum |x_i - z_i| in float32 and reports perturbations as the plain sum (no
 * square root): with per-block weights L_b / 2 this is the total variation of
 * each topic distribution scaled by its document's length, the norm Appendix C
 * uses for LDA.  On SCAR_I32 data L1 is the default already. */
typedef enum { SCAR_NORM_DEFAULT = 0, SCAR_NORM_L1 = 1 } scar_norm;

enum {
    SCAR_OK = 0,
    SCAR_ERR_INVALID_ARG = -1, /* NULL where not allowed, r outside [0,1], k > B, misaligned x ... */
    SCAR_ERR_LAYOUT = -2,      /* inconsistent block geometry */
    SCAR_ERR_ALLOC = -3,       /* device or host allocation failed */
    SCAR_ERR_CUDA = -4,        /* a CUDA runtime call or kernel launch failed */
    SCAR_ERR_STATE = -5,       /* call not valid in the context's current state */
    SCAR_ERR_TIMEOUT = -6,     /* a bounded device-side wait (of the selection, or of the norm reduction) gave
                                  up; the call's outputs are invalid, the context stays usable */
    SCAR_ERR_CAPACITY = -7,    /* problem larger than a fixed-size internal buffer */
    SCAR_ERR_IO = -8           /* a read or write of the stored checkpoint failed or came up short */
};

/* Block geometry of the flat buffer of n_elems elements.
 *   Implicit form (block_offsets == NULL): rows of row_elems elements
 *   (0 = one row of n_elems; otherwise n_elems % row_elems == 0), each cut into
 *   blocks of block_elems; the last block of a row may be shorter; blocks never
 *   cross a row end.  n_blocks is ignored.
 *   Explicit form: block_offsets is a HOST array of n_blocks + 1 non-decreasing
 *   element offsets with block_offsets[0] == 0 and block_offsets[n_blocks] ==
 *   n_elems; it is copied during init.  row_elems / block_elems are ignored.
 * n_shards >= 1; shard s owns blocks [floor(s*B/S), floor((s+1)*B/S)).
 * At most 2^32 - 1 blocks. */
typedef struct {
    uint64_t n_elems;
    uint64_t row_elems;
    uint32_t block_elems;
    uint32_t n_shards;
    const uint64_t *block_offsets;
    uint64_t n_blocks;
} scar_layout;

typedef struct {
    uint64_t k;                /* blocks saved */
    uint64_t payload_elems;    /* elements in the payload = poff[k] */
    uint64_t nonfinite_blocks; /* SCAR_F32: blocks whose score was NaN or +Inf (ranked first) */
} scar_save_info;

typedef struct {
    double l2;            /* SCAR_F32: ||z_S - x_S|| in the context's norm (l2 unless scar_ckpt_set_norm
                             chose another); 0 for SCAR_I32 */
    uint64_t l1;          /* SCAR_I32: sum_{i in S} |z_i - x_i| ; 0 for SCAR_F32 */
    uint64_t lost_blocks; /* |S| in blocks */
    uint64_t lost_elems;  /* |S| in elements */
} scar_norm_info;

/* Creates a context over the caller's device buffer d_x (n_elems elements of
 * type dt, 16-byte aligned, owned by the caller, must stay valid and in place
 * until destroy) and initialises the running checkpoint z := x (Section 4.2:
 * the running checkpoint starts from the initial parameter values).  Allocates
 * z, the score/selection arrays and a payload buffer of n_elems elements on the
 * current CUDA device.  cuda_stream is a cudaStream_t (NULL = default stream).
 * Waits for the stream before returning.  On error *out is NULL. */
int scar_ckpt_init(scar_ctx **out, void *d_x, scar_dtype dt, const scar_layout *layout, void *cuda_stream);

/* Chooses the norm and optional per-block weights for all later scoring,
 * selection and perturbation results of this context.  h_block_weights: HOST
 * array of B finite floats >= 0 (copied before the call returns), or NULL for
 * no weights; SCAR_F32 only (SCAR_ERR_INVALID_ARG with SCAR_I32: integer scores
 * stay exact integers, and for count rows of fixed total the length-scaled
 * total variation is half the plain l1 anyway).  With weights w a block scores
 * w_b * dist(x_b, z_b) (dist = squared l2, or l1), and a perturbation is
 * sqrt(sum_b w_b ||d_b||^2) or sum_b w_b ||d_b||_1, reported in the l2 field of
 * scar_norm_info: a positive combination of block norms, hence a norm
 * (Appendix C).  Waits for the stream. */
int scar_ckpt_set_norm(scar_ctx *ctx, scar_norm norm, const float *h_block_weights);

/* Checkpoint step 1 of Section 4.3 alone: recomputes score_b = dist(x_b, z_b)
 * for every block into the context's score array (float32 squared l2, or
 * uint64 l1).  Enqueue only. */
int scar_ckpt_block_scores(scar_ctx *ctx);

/* One prioritized partial checkpoint (Section 4.2; steps 1, 3, 4 of the
 * checkpoint protocol in Section 4.3): scores all blocks, selects the
 * k = round(r*B) highest (halves away from zero; at least 1 if r > 0; ties to
 * the lowest block id; NaN/Inf scores rank first), writes their ids ascending to
 * sel[k], their payload offsets to poff[k+1], copies x over them into the
 * payload in that order and refreshes z_b := x_b on them.  r = 1 is the
 * traditional full checkpoint.  r outside [0,1] or NaN: SCAR_ERR_INVALID_ARG. */
int scar_ckpt_priority_save(scar_ctx *ctx, double r, scar_save_info *out);

/* The rule that turns the fraction r of Section 4.2 into a block count, as
 * scar_ckpt_priority_save applies it: k = round(r * n_blocks), halves away from
 * zero, at least 1 when r > 0 and n_blocks > 0, at most n_blocks.  For callers
 * that schedule saves themselves (the baseline selectors take k, not r).  Host
 * only.  SCAR_ERR_INVALID_ARG for r outside [0,1], NaN, or k == NULL. */
int scar_k_from_r(double r, uint64_t n_blocks, uint64_t *k);

/* Same with the block count given directly (0 <= k <= B). */
int scar_ckpt_priority_save_k(scar_ctx *ctx, uint64_t k, scar_save_info *out);

/* The multi-GPU form of a prioritized save: the checkpoint protocol of Section
 * 4.3 the way the paper runs it, with one GPU per parameter-server node.  Every
 * node scores its own partition (step 1: scar_ckpt_block_scores), the scores of
 * all nodes are made known to all (step 2: the caller's exchange, e.g. an NCCL
 * all-gather of the score arrays; the library itself has no communication), and
 * every node selects the same global fraction and saves what it owns (steps 3
 * and 4: this call).  Payloads never leave their GPU; recovery stays a local
 * call on whichever context owns the lost blocks.
 *
 * The context covers this rank's partition: its B blocks are blocks
 * [first_block, first_block + B) of a global layout of n_global_blocks blocks.
 *   d_global_scores  DEVICE array of n_global_blocks scores in global block
 *                    order, of the context's score type (float32 / uint64), as
 *                    scar_ckpt_view returns them per rank; read when the
 *                    enqueued work runs
 *   k_global         blocks to save over all ranks (e.g. scar_k_from_r(r,
 *                    n_global_blocks)), 0 <= k_global <= n_global_blocks
 * The k_global highest global scores are selected, ties to the lowest global
 * id; the ones in this rank's range are packed and refreshed exactly as by a
 * single-GPU save: sel holds LOCAL block ids, ascending, out->k is this rank's
 * count, out->nonfinite_blocks counts over all ranks.  The union over ranks of
 * the saved blocks (local id + first_block) is what one context over the
 * concatenated buffer would have saved.  Always waits for the stream (the
 * rank's count crosses to the host once), so `out` must not be NULL and the
 * call cannot be captured. */
int scar_ckpt_priority_save_sharded(scar_ctx *ctx, const void *d_global_scores, uint64_t n_global_blocks,
                                    uint64_t first_block, uint64_t k_global, scar_save_info *out);

/* The two baseline selectors the paper compares the prioritized checkpoint with
 * (Section 5.4).  Both skip the scoring pass (the score array keeps the values
 * of the last scoring) and then pack the chosen blocks and refresh z on them
 * exactly as a prioritized save does: same sel / poff / payload outputs, ids
 * ascending.
 *   round:  "selected in a round-robin manner": the k blocks that follow the
 *           context's cursor, wrapping at the end of the buffer; the cursor
 *           then advances by k (mod B).  It starts at block 0.
 *   random: "selected uniformly at random".  The randomness is the caller's:
 *           d_priorities is a DEVICE array of B uint32 values drawn
 *           independently and uniformly by the caller; the k largest are taken,
 *           ties to the lowest id, which is a uniform k-subset up to those ties.
 *           Read when the enqueued work runs.
 * 0 <= k <= B, otherwise SCAR_ERR_INVALID_ARG. */
int scar_ckpt_save_round(scar_ctx *ctx, uint64_t k, scar_save_info *out);
int scar_ckpt_save_random(scar_ctx *ctx, uint64_t k, const uint32_t *d_priorities, scar_save_info *out);

/* Round-robin cursor: if set != NULL the cursor becomes *set (must be < B, or 0
 * when B == 0); if get != NULL it receives the cursor.  Host state only. */
int scar_ckpt_round_cursor(scar_ctx *ctx, const uint64_t *set, uint64_t *get);

/* Partial recovery (Section 4.1; recovery step 2 of Section 4.3): for every
 * block of every lost shard, accumulates the perturbation of the appendix proof
 * of Theorem 4.1, ||z_S - x_S||, from the values x still holds, then overwrites
 * x_b := z_b.  Blocks outside S and all of z are left untouched.
 * h_lost_shards: HOST array of n_shards bytes, 0 = alive, non-zero = lost. */
int scar_recover_partial(scar_ctx *ctx, const uint8_t *h_lost_shards, scar_norm_info *out);

/* Same with an arbitrary lost set: d_lost_blocks is a DEVICE array of B bytes
 * (0 alive, non-zero lost), read when the enqueued work runs. */
int scar_recover_partial_blocks(scar_ctx *ctx, const uint8_t *d_lost_blocks, scar_norm_info *out);

/* The perturbation a recovery of the given lost set would cause, without
 * writing anything.  NULL mask = every block lost = full recovery, whose
 * perturbation is x^(T) - x^(C) (Example 2.3). */
int scar_perturbation_norm(scar_ctx *ctx, const uint8_t *h_lost_shards, scar_norm_info *out);
int scar_perturbation_norm_blocks(scar_ctx *ctx, const uint8_t *d_lost_blocks, scar_norm_info *out);

/* Perturbation norm without any allocation.  (The paper has no counterpart: it
 * is the same quantity as scar_perturbation_norm_blocks, offered for callers
 * that cannot allocate.)
 *
 * Some callers cannot create a context, because scar_ckpt_init calls cudaMalloc:
 * a failure handler running while memory is exhausted, a latency-critical loop
 * that cannot take the device-wide synchronisation an allocation implies, or a
 * plug-in whose host forbids it to grow its memory.  This call needs no
 * context and calls no cudaMalloc / cudaFree or other allocating routine.  Its
 * partial sums live in a fixed array of about 0.3 MiB inside the library's
 * device image (every GPU that loads the library holds it until the process
 * exits), which caps the problem at SCAR_STATIC_MAX_BLOCKS blocks; larger
 * layouts return SCAR_ERR_CAPACITY and nothing is enqueued.
 *
 *   d_x, d_z       DEVICE buffers of layout->n_elems elements of type dt, both
 *                  16-byte aligned, read only; z is the checkpoint to compare with
 *   layout         implicit form only (block_offsets must be NULL); n_shards ignored
 *   d_lost_blocks  DEVICE array of B bytes, 0 alive / non-zero lost; NULL = all lost
 *   d_out          DEVICE scar_norm_info written by the enqueued work (caller-owned)
 *   cuda_stream    cudaStream_t to enqueue on; the call does not wait
 *
 * The first call on each device looks up the array's device address (once, with
 * that device current), and with CUDA's lazy module loading it is also what
 * brings the array and this call's kernels onto the device, which itself needs
 * a little device memory.  So make the first call at start-up, before memory
 * can run short and before any stream capture: a call with n_elems == 0 does the
 * look-up, one tiny real call loads the kernels.  All calls on a device share
 * the one array (each call first empties the part it uses): calls whose GPU
 * work overlaps (different streams, or different threads) race and give wrong
 * results; calls ordered on one stream are fine.  Results are bit-identical to
 * scar_perturbation_norm_blocks. */
#define SCAR_STATIC_MAX_BLOCKS (1ull << 20)
int scar_perturbation_norm_static(const void *d_x, const void *d_z, scar_dtype dt, const scar_layout *layout,
                                  const uint8_t *d_lost_blocks, scar_norm_info *d_out, void *cuda_stream);

/* Host-buffer forms for callers whose parameters live in host memory.
 * save_host: copies n_elems elements from h_x into the context's x, runs the
 * save, then copies back payload_elems elements to h_payload (capacity n_elems
 * elements), k ids to h_sel (capacity k) and k+1 offsets to h_poff.  Always
 * waits for completion; `out` must not be NULL.
 * recover_host: copies the lost shards' element ranges of h_x (the values the
 * failed nodes last held) into x, runs the recovery, and copies the recovered
 * ranges back into h_x; other ranges of h_x are neither read nor written. */
int scar_ckpt_priority_save_host(scar_ctx *ctx, const void *h_x, double r, void *h_payload, uint32_t *h_sel,
                                 uint64_t *h_poff, scar_save_info *out);
int scar_recover_partial_host(scar_ctx *ctx, void *h_x, const uint8_t *h_lost_shards, scar_norm_info *out);

/* ---- Asynchronous drain of a save's output (Section 4.3) --------------------
 * In the paper's protocol training resumes as soon as the in-memory cache (z)
 * is refreshed, while the saved parameters go to persistent storage in the
 * background, so the checkpoint overhead T_dump is only the prioritisation and
 * the cache refresh.  Here: a save runs on the context's stream as always;
 * scar_ckpt_drain_enqueue then copies that save's ids, offsets and payload to
 * pinned host memory on a second, library-owned stream, ordered after the save
 * by an event, and returns at once.  Two slots alternate, so the next save can
 * run while the previous one is still being copied out.
 *
 *   drain_init     switches the context to drain mode and allocates the second
 *                  device output set plus two pinned host mirrors.  From then
 *                  on every save is limited to max_k blocks and to layouts whose
 *                  k longest blocks together hold at most max_payload_elems
 *                  elements (whatever the save then selects fits; otherwise
 *                  SCAR_ERR_CAPACITY, nothing enqueued).  Waits for
 *                  the context's stream.  Once per context.
 *   drain_enqueue  hands the most recent save (there must be one that was not
 *                  handed over yet: SCAR_ERR_STATE otherwise) to the drain
 *                  stream; *ticket identifies it.  The next save writes to the
 *                  other slot, and fails with SCAR_ERR_STATE, nothing enqueued,
 *                  while that slot's ticket has not been released: at most two
 *                  tickets are out at any time.  Does not wait.
 *   drain_done     1 if the copy of that ticket has finished, 0 if not yet.
 *   drain_wait     waits for the copy and fills *out with HOST pointers into
 *                  the slot's pinned mirror: valid until drain_release.
 *   drain_release  gives the slot back to the library (waits for the copy if it
 *                  is still running).
 * scar_ckpt_view keeps returning the device buffers of the most recent save.
 * A save called with a non-NULL `out` fetches its result record over the same
 * device-to-host path and can queue behind a running drain; to overlap, enqueue
 * saves with out == NULL and read the record from the drained view. */
typedef struct {
    scar_save_info info;
    const uint32_t *h_sel;  /* info.k ids, ascending */
    const uint64_t *h_poff; /* info.k + 1 element offsets */
    const void *h_payload;  /* info.payload_elems elements */
} scar_drain_view;
int scar_ckpt_drain_init(scar_ctx *ctx, uint64_t max_k, uint64_t max_payload_elems);
int scar_ckpt_drain_enqueue(scar_ctx *ctx, uint64_t *ticket);
int scar_ckpt_drain_done(scar_ctx *ctx, uint64_t ticket);
int scar_ckpt_drain_wait(scar_ctx *ctx, uint64_t ticket, scar_drain_view *out);
int scar_ckpt_drain_release(scar_ctx *ctx, uint64_t ticket);

/* ---- The running checkpoint in persistent storage (Sections 4.2, 4.3) --------
 * The paper keeps the running checkpoint in shared persistent storage and z is
 * only the in-memory cache of it: step 4 of a checkpoint saves the selected
 * parameters there, and a recovery re-loads parameters from it.  Here the
 * stored checkpoint is a plain file of n_elems * 4 bytes in element order, given
 * as an open POSIX file descriptor (the caller opens, syncs and closes it); after
 * every store it holds exactly the bytes of z.
 *   store_full     writes all of z (the initial checkpoint x^(0), or after
 *                  scar_ckpt_load).  Waits for the stream.
 *   store_drained  waits for the drain of `ticket` and writes each saved block
 *                  from the pinned host mirror to its place in the file (one
 *                  write per run of consecutive blocks).  The ticket stays
 *                  valid; release it afterwards.  Host work only.
 *   load_stored    z := the file (a restart that lost the in-memory cache, or a
 *                  recovery from storage: follow it with scar_recover_partial).
 *                  Waits for the stream.
 * SCAR_ERR_IO on a failed or short read / write; the file or z may then be
 * partly updated. */
int scar_ckpt_store_full(scar_ctx *ctx, int fd);
int scar_ckpt_store_drained(scar_ctx *ctx, uint64_t ticket, int fd);
int scar_ckpt_load_stored(scar_ctx *ctx, int fd);

/* Replaces the running checkpoint by n_elems elements read from the device
 * buffer d_z_src (e.g. a checkpoint read back from storage).  Enqueue only. */
int scar_ckpt_load(scar_ctx *ctx, const void *d_z_src);

/* Waits for the stream and returns the results of the most recent save and the
 * most recent recover/norm call (either pointer may be NULL). */
int scar_ckpt_last_info(scar_ctx *ctx, scar_save_info *save, scar_norm_info *norm);

/* Borrowed device pointers (any may be NULL to skip): z (n_elems elements),
 * scores (B float32 for SCAR_F32, B uint64 for SCAR_I32; as of the last
 * scoring), sel (k uint32), poff (k+1 uint64), payload.  Valid until destroy;
 * contents change with the next save. */
int scar_ckpt_view(scar_ctx *ctx, const void **d_z, const void **d_scores, const uint32_t **d_sel,
                   const uint64_t **d_poff, const void **d_payload);

/* Geometry as the library resolved it. */
uint64_t scar_ckpt_n_blocks(const scar_ctx *ctx);

/* Kernels this context has launched so far (its own kernels only). */
uint64_t scar_ckpt_launch_count(const scar_ctx *ctx);

/* Optional per-phase device timing.  With enable != 0 every later call brackets
 * its phases with CUDA events on the context's stream.  phase_ms receives the
 * duration of the most recent call's phases, in milliseconds, after waiting for
 * the stream: [0] block scores, [1] selection, [2] pack + cache refresh,
 * [3] restore / norm pass including its reduction (one kernel), [4] the
 * reduction as a kernel of its own (layouts cut into segments only, else 0);
 * phases a call did not run read 0. */
int scar_ckpt_profile(scar_ctx *ctx, int enable);
int scar_ckpt_profile_read(scar_ctx *ctx, float phase_ms[5]);

/* ---- Iteration-cost arithmetic of Section 3 (host only, no GPU work) --------
 * c is the linear convergence rate of the training algorithm, 0 < c < 1
 * (Eq. 5/6); dist0 = ||x^(0) - x*|| > 0.  Every function returns NaN when an
 * argument is outside its domain.
 *
 * baseline_iterations: kappa(x, eps) = log(dist0 / eps) / log(1 / c), the
 *   iterations the unperturbed sequence needs to come within eps (Section 3.1).
 * discounted_perturbation: Delta_T = sum_i c^(-iters[i]) * norms[i] of
 *   Theorem 3.2, for n perturbations of size norms[i] >= 0 met at iteration
 *   iters[i] (HOST arrays).  A single recovery at iteration T with
 *   perturbation norm p gives c^(-T) * p.
 * iteration_cost_bound: Theorem 3.2, log(1 + Delta_T / dist0) / log(1 / c):
 *   the most extra iterations the perturbations can cost.
 * irreducible_error: (c / (1 - c)) * delta_max, the accuracy floor when every
 *   iteration may be perturbed by up to delta_max (Example 3.3, infinite
 *   perturbations). */
double scar_baseline_iterations(double dist0, double eps, double c);
double scar_discounted_perturbation(const double *norms, const uint64_t *iters, uint64_t n, double c);
double scar_iteration_cost_bound(double delta_T, double dist0, double c);
double scar_irreducible_error(double delta_max, double c);

/* Self-test hook for the bounded device-side wait.  The selection kernel's
 * CTAs meet at a few points whose wait gives up after a fixed number of polls
 * (2^19 to 2^20: a quarter of a second at the earliest, about a second in
 * practice) instead of hanging.  This call makes the NEXT prioritized or
 * random save wait for one key, one record or one arrival more than its
 * selection has (host state only), so that its first wait can never
 * complete: that save takes up to about a second,
 * selects and copies nothing, leaves z untouched, and returns SCAR_ERR_TIMEOUT
 * from the call that reads its result (the save itself with a non-NULL out, or
 * scar_ckpt_last_info).  The save after that one works normally.
 * SCAR_ERR_STATE on an empty buffer. */
int scar_ckpt_selftest_arm_timeout(scar_ctx *ctx);

/* ---- Guard bands (debugging aid; no counterpart in the paper) ------------------
 * scar_ckpt_init_guarded is scar_ckpt_init for a context whose every device
 * buffer (running checkpoint, payload, scores, id and offset lists, masks,
 * selection and reduction scratch, segment tables, drain and sharding buffers
 * allocated later) sits between two bands of 256 bytes holding a known pattern,
 * the second band starting at the first byte behind the buffer.
 * scar_ckpt_debug_check_guards waits for the stream and counts, on the device,
 * the band bytes that no longer hold the pattern: any write of the library's
 * kernels just outside one of its buffers shows up as a non-zero count.
 * SCAR_ERR_STATE on a context that was not created guarded.
 * scar_static_debug_check_guard does the same for the band behind the fixed
 * array of scar_perturbation_norm_static on the current device (waits for the
 * device; SCAR_ERR_STATE before that call was ever used there). */
int scar_ckpt_init_guarded(scar_ctx **out, void *d_x, scar_dtype dt, const scar_layout *layout, void *cuda_stream);
int scar_ckpt_debug_check_guards(scar_ctx *ctx, uint64_t *bad_bytes);
int scar_static_debug_check_guard(uint64_t *bad_bytes);

/* Diagnostic builds only (library compiled with -DSCAR_SELECT_STAMPS; otherwise
 * SCAR_ERR_STATE).  Waits for the stream and copies the 32 time stamps of the
 * most recent selection kernel: SM clock cycles of its first CTA at
 *   [0] start, [1] keys loaded, then for digit pass p = 0..5
 *   [2+4p] shared histogram built, [3+4p] flushed to the global histogram
 *   (a selection that one CTA does alone flushes nothing), [4+4p] every CTA
 *   has arrived (only selections with several tiles per CTA meet at a
 *   counter; otherwise the same point as [3+4p]), [5+4p] global histogram
 *   complete and digit resolved,
 *   [26] own counts known, [27] every CTA's record read, [28] output bases
 *   known, [29] ids and offsets written.
 * Stamps of passes that did not run keep the value of an earlier selection (or
 * zero).  No counterpart in the paper: it shows where the selection of
 * checkpoint step 3 spends its time. */
int scar_ckpt_debug_select_stamps(scar_ctx *ctx, int64_t stamps[32]);

/* Waits for the stream, frees everything the context owns (never x). */
int scar_ckpt_destroy(scar_ctx *ctx);

/* Static description of an error code. */
const char *scar_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* SCAR_H */
