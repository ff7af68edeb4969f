/*
 * lora_mixed_linear.h — C ABI of the B200 (sm_100a) mixed-adapter LoRA linear layer.
 *
 * The operation.  A batch of T tokens from several agents shares one frozen base weight W0
 * and every token is bound to one resident (adapter, version) entry of an adapter slot
 * table, or to none:
 *
 *     y[t][n] = sum_k x[t][k] W0[n][k]  +  scale_s * sum_j ( sum_k x[t][k] A_s[j][k] ) B_s[n][j]
 *
 * with s the entry of token t; a token bound to no adapter (slot -1) gets the first sum only.
 * Source of the problem statement: the paper's Section 2 ("LoRA adapters": low-rank modules
 * on a shared frozen base; requests routed to the correct adapter; updates published
 * atomically, never partially visible), Section 4.2 (inference binds the last committed
 * adapter version, staged state stays private until published), Section 5.1 (validity key:
 * the adapter names the LoRA slot, the adapter version the committed state) and Section 5.3
 * (an old version keeps serving while work for the newly trained version already runs, so
 * both are resident at once).  One physical slot of the table = one resident
 * (adapter_id, version) pair; two versions of one adapter occupy two slots.
 *
 * Conventions for every call below
 *   - All matrices are row-major bf16:  x[T][d_in], W0[d_out][d_in], A[rank][d_in],
 *     B[d_out][rank], y[T][d_out].  Accumulation is fp32; y is rounded once to bf16 (nearest
 *     even).  The shrink result u = scale*(x.A^T) is rounded to bf16 before the expand.
 *   - "device pointer" = memory of the table's CUDA device; "host pointer" = ordinary host
 *     memory.  Device pointers must be 16-byte aligned; d_in and d_out are multiples of 8.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - The library never allocates, frees or keeps x, W0, y or the workspace: the caller owns
 *     them and must keep them alive until the stream work has finished.  The table owns only
 *     its own packed copy of the registered adapters and a status word.
 *   - Errors are return codes; nothing throws, aborts or traps.  An error detected on the
 *     host returns before anything is launched and leaves the table unchanged.  Errors only
 *     visible on the device (an unknown or retired slot id in slot_ids, malformed
 *     seg_offsets, a perm entry outside [0,T), a bounded wait that ran out) set a sticky bit
 *     in the table's device status word; the affected tokens get the base output only
 *     (malformed seg_offsets: every token of that call), and the kernels finish normally.
 *   - lora_mixed_linear, lml_segment_tokens and lora_mixed_linear_host neither allocate nor
 *     synchronise nor read device memory from the host.
 *   - Calls that use the same workspace, or the same table from different streams without
 *     ordering between them, race; one table may be shared by ordered streams.
 *   - Same inputs give bitwise the same y on every run (no atomics touch y).
 */
#ifndef LORA_MIXED_LINEAR_H_
#define LORA_MIXED_LINEAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lml_table lml_table; /* adapter slot table of ONE linear site (fixed d_in, d_out) */

typedef enum {
    LML_OK = 0,
    LML_ERR_INVALID_ARG = 1, /* null / misaligned pointer, negative size, rank outside [1,64], ... */
    LML_ERR_BAD_SLOT = 2,
    LML_ERR_TABLE_FULL = 3,
    LML_ERR_DUPLICATE = 4,   /* (adapter_id, version) already resident */
    LML_ERR_NOT_FOUND = 5,
    LML_ERR_UNSUPPORTED = 6, /* device is not sm_100 */
    LML_ERR_CUDA = 7,        /* a CUDA runtime / driver call failed */
    LML_ERR_TIMEOUT = 8,
    LML_ERR_WORKSPACE = 9,   /* workspace missing, misaligned or smaller than lml_workspace_bytes */
    LML_ERR_TOO_LARGE = 10   /* the call is larger than a fixed-capacity entry point can take */
} lml_status;

/* bits of the device status word (lml_device_status) */
#define LML_FLAG_BAD_SLOT 1u    /* slot id >= max_slots or not live: tokens got base output only  */
#define LML_FLAG_BAD_OFFSETS 2u /* seg_offsets not 0-based / monotone / ending at T: base only     */
#define LML_FLAG_BAD_PERM 4u    /* perm entry outside [0,T): that position was skipped             */
#define LML_FLAG_TIMEOUT 8u     /* a bounded in-kernel wait gave up                                */

#define LML_MAX_SLOTS 64  /* upper bound for max_slots */
#define LML_MAX_RANK 64   /* upper bound for an adapter's rank */
#define LML_MAX_ADAPTER_IDS 4096 /* adapter ids 0 .. this-1 can be published and resolved on the device */
#define LML_DECODE_MAX_TOKENS 16 /* T <= this takes the bandwidth-bound decode kernel */
#define LML_MAX_PROJECTIONS 4 /* projections one lora_mixed_linear_multi call can take */

const char* lml_status_string(lml_status s);

/*
 * Create the slot table of one linear site on CUDA device `device`.
 * Allocates (once, here) the packed adapter arena: max_slots * 64 * (d_in + d_out) bf16, plus
 * a few hundred bytes.  1 <= max_slots <= LML_MAX_SLOTS; d_in, d_out > 0 and multiples of 8.
 * Errors: INVALID_ARG, UNSUPPORTED (not compute capability 10.x), CUDA.
 */
lml_status lml_table_create(lml_table** out, int device, int d_in, int d_out, int max_slots);

/* Free the table and its arena.  The caller makes sure no enqueued work still uses it. */
lml_status lml_table_destroy(lml_table* t);

/*
 * register_adapter — make (adapter_id, version) resident (the paper's "publish a staged
 * version": Section 4.2 / 5.3; a newer version is registered while the older one still
 * serves).  A: device bf16 [rank][d_in]; B: device bf16 [d_out][rank]; 1 <= rank <= 64;
 * scale is the final multiplier (the library never divides by rank).  The adapter is copied
 * into the table's arena in the layout the kernels read (rows zero-padded to rank 64) by a
 * small kernel enqueued on `stream`; A and B may be released once that stream work is done.
 * The new entry is visible to calls issued after this returns; work on OTHER streams must be
 * ordered after `stream` by the caller.  *slot_out receives the physical slot index to use in
 * slot_ids / token_slots (lowest free index).  A rejected call changes nothing: no
 * half-registered entry is ever visible.  (`stream` is this library's addition to the call: the copy
 * into the arena is a kernel, and the caller says where it runs.)
 * Errors: INVALID_ARG, DUPLICATE, TABLE_FULL, CUDA.
 */
lml_status register_adapter(lml_table* t, int adapter_id, int version, const void* A, const void* B,
                            int rank, float scale, void* stream, int* slot_out);

/*
 * retire_version / retire_version_on — drop a resident (adapter_id, version) entry (Section 5.3: the
 * old version goes away once in-flight work bound to it is done).  On the host the entry is gone for
 * every later call; work already enqueued keeps the slot description it was launched with, but the
 * slot's arena space may be reused by the next register_adapter, so retire only after work bound to
 * that slot has been ordered before the registering stream.  Other slots keep their indices.  A pinned
 * entry only becomes RETIRING (see lml_pin).
 * Retiring the SERVING version of an adapter also takes it out of the device map that the *_adapters
 * calls resolve through: a one-thread kernel, enqueued on `stream`, clears the adapter's word if it still
 * names this entry.  Pass the stream the entry was published on (or one ordered behind it), so that the
 * clear cannot overtake the publish.  retire_version is retire_version_on with the legacy default stream,
 * which orders against blocking streams only.  Every later register_adapter makes its stream wait for the
 * clear before it overwrites a slot.  Independently of all ordering, a word of the map names the
 * registration it was published for: once that entry is retired, or its slot holds another registration,
 * the word resolves to "no serving version" (base output, LML_FLAG_BAD_SLOT), never to the slot's new
 * tenant.  Neither call may be made while `stream` is being captured.
 * Errors: INVALID_ARG, NOT_FOUND, CUDA (the clear could not be enqueued; the entry stays).
 */
lml_status retire_version(lml_table* t, int adapter_id, int version);
lml_status retire_version_on(lml_table* t, int adapter_id, int version, void* stream);

/* Slot index of a resident (adapter_id, version).  Errors: INVALID_ARG, NOT_FOUND. */
lml_status lml_lookup(const lml_table* t, int adapter_id, int version, int* slot_out);

/* rank / scale / (adapter_id, version) of a slot; any out pointer may be NULL.
 * Errors: INVALID_ARG, BAD_SLOT (index out of range or slot free). */
lml_status lml_slot_info(const lml_table* t, int slot, int* adapter_id, int* version, int* rank,
                         float* scale);

/*
 * Bytes of device workspace (256-byte aligned) lora_mixed_linear needs for T <= max_tokens and G <= max_segments
 * (with or without perm).  Contents need no initialisation and carry nothing between calls.
 * Returns 0 on invalid arguments.
 */
size_t lml_workspace_bytes(const lml_table* t, int max_tokens, int max_segments);

/*
 * Publication (Section 4.2: requests bind to the last committed adapter; Section 5.3: a staged
 * version runs privately while the old one serves, and becomes visible at one controlled point).
 *
 * An entry made by register_adapter is RESIDENT: usable by whoever names its slot (that is how a
 * staged version is exercised before it is published), invisible to calls that name adapters.
 * lml_publish makes (adapter_id, version), which must be resident, the SERVING version of the
 * adapter: from that point of `stream` on, calls that name the adapter (the *_adapters forms
 * below) resolve to its slot; calls enqueued on `stream` earlier still resolve to the version
 * that served before.  The switch is a single 4-byte store on the device, so no call sees a
 * mixture.  The version that served before becomes RETIRING: it stays resident while work is
 * pinned to it and is retired (slot free again) by the unpin that brings its count to zero, or at
 * once if nothing is pinned.  So work that spans two calls and must see one version (ids resolved by
 * lml_segment_tokens_adapters, the layer run later by lora_mixed_linear) pins the slot it resolved to,
 * or does not straddle a publish: without the pin the old slot is free by the time the second call
 * takes its snapshot, and its tokens get base output and LML_FLAG_BAD_SLOT.
 * previous_version_out (may be NULL) receives that version, or -1.
 * 0 <= adapter_id < LML_MAX_ADAPTER_IDS.  Errors: INVALID_ARG, NOT_FOUND, CUDA.
 *
 * lml_pin / lml_unpin count work in flight that is bound to a slot (a request that started under
 * a version keeps it until it ends).  retire_version on a pinned entry likewise only marks it
 * RETIRING.  Errors: INVALID_ARG, BAD_SLOT (slot free), and for unpin INVALID_ARG if not pinned.
 *
 * lml_resolve: serving slot and version of an adapter on the host (NOT_FOUND if none).
 * lml_slot_state: state (LML_STATE_*) and pin count of a live slot; out pointers may be NULL.
 */
#define LML_STATE_RESIDENT 0
#define LML_STATE_SERVING 1
#define LML_STATE_RETIRING 2
lml_status lml_publish(lml_table* t, int adapter_id, int version, void* stream, int* previous_version_out);
lml_status lml_pin(lml_table* t, int slot);
lml_status lml_unpin(lml_table* t, int slot);
lml_status lml_resolve(const lml_table* t, int adapter_id, int* slot_out, int* version_out);
lml_status lml_slot_state(const lml_table* t, int slot, int* state_out, int* pins_out);

/*
 * lml_segment_tokens — the token-segmentation pass: group T tokens by slot.
 * token_slots: device int32[T], physical slot per token or -1 (no adapter).
 * Outputs (device): perm int32[T] (position -> token row); seg_offsets int32[max_slots + 2];
 * seg_slot_ids int32[max_slots + 1].  Always exactly G = max_slots + 1 segments are produced:
 * segment i < max_slots holds the tokens of slot i (possibly none), the last segment holds
 * the -1 tokens; so G is known on the host without reading device memory.  The grouping is
 * stable: tokens keep their relative order inside a segment.  Ids outside [-1, max_slots)
 * or naming a free slot go to the -1 group and set LML_FLAG_BAD_SLOT.
 * T == 0 is valid (all offsets 0).  Errors: INVALID_ARG, CUDA.
 */
lml_status lml_segment_tokens(lml_table* t, const int32_t* token_slots, int T, int32_t* perm,
                              int32_t* seg_offsets, int32_t* seg_slot_ids, void* stream);

/*
 * lora_mixed_linear — the layer.  x: device bf16 [T][d_in]; W0: device bf16 [d_out][d_in];
 * y: device bf16 [T][d_out], overwritten.  seg_offsets: device int32[G+1] with
 * seg_offsets[0] = 0 <= ... <= seg_offsets[G] = T; slot_ids: device int32[G], physical slot
 * or -1 per segment (repeated slots, empty segments and any order are fine; a non-empty
 * segment whose slot holds no live adapter gets base output and sets LML_FLAG_BAD_SLOT).  Segment g
 * covers positions [seg_offsets[g], seg_offsets[g+1]); position p is row perm[p] of x and y
 * if perm (device int32[T], a permutation) is given, else row p.  G == 0 means "no adapter
 * anywhere": the base product is still computed and y written (one launch).  T == 0 returns LML_OK
 * without launching.
 * T <= 16 runs the bandwidth-bound decode kernel (W0 read once through a bulk-copy ring; with
 * segments its CTAs hand one another their share of the shrink result and count themselves in
 * a small exchange block that belongs to the table, so two decode calls on the SAME table must not overlap on the GPU:
 * put them on one stream or order them; a CTA whose peers are late computes their share itself,
 * so the call completes even when the grid cannot be resident all at once); larger T runs the
 * TMA / tcgen05 GEMM with the LoRA expand as extra tensor-core K-steps.
 * W0 is the frozen base weight: it must not be written by the operation that immediately precedes
 * the call on `stream` (the decode kernel starts fetching W0 while the kernel before it is still
 * draining; x, the segment arrays and the adapters are read only after that kernel has finished).
 * Errors: INVALID_ARG, WORKSPACE, CUDA.
 */
lml_status lora_mixed_linear(lml_table* t, const void* x, const void* W0, int T,
                             const int32_t* seg_offsets, const int32_t* slot_ids, int G,
                             const int32_t* perm, void* y, void* workspace, size_t workspace_bytes,
                             void* stream);

/*
 * lora_mixed_linear_dual — the same tokens under two bindings in one call (Section 5.3: hot prefixes
 * are recomputed under the staged version while the old one still serves).  slot_ids_a / slot_ids_b:
 * device int32[G], the slot of every segment under the first and under the second binding (-1 = no
 * adapter, either side).  y_a = x.W0 + delta_a, y_b = x.W0 + delta_b, both device bf16 [T][d_out],
 * distinct buffers.  For T > 16 the base product x.W0 is computed once: y_a is read out of the
 * accumulator, then (delta_b - delta_a) is added to it with a few more tensor-core steps and y_b is
 * read out, so y_a agrees with lora_mixed_linear with slot_ids_a to the bf16 rounding of u (bit for
 * bit when that call takes u from the same shrink kernel) and y_b with lora_mixed_linear with
 * slot_ids_b to fp32 rounding of the accumulator as well.  For T <= 16 the call is one launch of
 * the decode kernel with half of its CTAs per binding (the two halves walk W0 together, so it
 * leaves HBM once); y_a and y_b are bit for bit those of two lora_mixed_linear calls.  G >= 1.  workspace: at least lml_dual_workspace_bytes(t, T, G).  Other arguments,
 * flags and errors as lora_mixed_linear.
 */
size_t lml_dual_workspace_bytes(const lml_table* t, int max_tokens, int max_segments);
lml_status lora_mixed_linear_dual(lml_table* t, const void* x, const void* W0, int T,
                                  const int32_t* seg_offsets, const int32_t* slot_ids_a,
                                  const int32_t* slot_ids_b, int G, const int32_t* perm, void* y_a, void* y_b,
                                  void* workspace, size_t workspace_bytes, void* stream);

/*
 * Backward pass of the layer, for the training task that shares the GPU with inference (Section 2.2:
 * adapters are updated online in the background; Section 4.1: the task model's training task).
 * With y = x.W0^T + s (x.A^T).B^T per segment and an upstream gradient dy [T][d_out]:
 *
 *   dx = dy.W0 + s (dy.B).A  is the layer itself on the transposed problem: a second table t_T with
 *   d_in = d_out(t), d_out = d_in(t), the caller's W0^T [d_in][d_out] as base weight and every adapter
 *   registered with register_adapter_transposed (which stores B^T as "A" and A^T as "B").  Call
 *   lora_mixed_linear(t_T, dy, W0T, ...) with the slots of t_T: same kernels, same accuracy.
 *
 *   lora_mixed_linear_backward_adapters adds the adapter gradients of one batch onto dA and dB:
 *     dA[slot][j][k] += s sum_t (dy.B)[t][j] x[t][k],  float32 [max_slots(t)][64][d_in], rows j >= rank untouched
 *     dB[slot][n][j] += s sum_t dy[t][n] (x.A^T)[t][j], float32 [max_slots(t)][d_out][64], columns j >= rank untouched
 *   over the tokens t of the segments bound to the slot (slot numbering of t).  The two small
 *   products (x.A^T and dy.B) go through the shrink kernels and are rounded to bf16 before the
 *   sums, which run in fp32 in a fixed order.  x, dy: device bf16, rows in segment order (no perm).
 *   slot_ids / slot_ids_T: device int32[G], the slot of every segment in t and in t_T (-1 = none,
 *   both).  The caller zeroes dA and dB at the start of a step; several calls accumulate.
 *   workspace: lml_backward_workspace_bytes(t, T, G).  Errors: INVALID_ARG, WORKSPACE, CUDA.
 */
lml_status register_adapter_transposed(lml_table* t_T, int adapter_id, int version, const void* A, const void* B,
                                       int rank, float scale, void* stream, int* slot_out);
size_t lml_backward_workspace_bytes(const lml_table* t, int max_tokens, int max_segments);
lml_status lora_mixed_linear_backward_adapters(lml_table* t, lml_table* t_T, const void* x, const void* dy, int T,
                                               const int32_t* seg_offsets, const int32_t* slot_ids,
                                               const int32_t* slot_ids_T, int G, float* dA, float* dB,
                                               void* workspace, size_t workspace_bytes, void* stream);

/*
 * lora_mixed_linear_tokens — segmentation and layer in one call, for callers that hold one slot id
 * per token (what a scheduler hands a decode step).  token_slots: device int32[T], physical slot
 * per row of x or -1; ids outside [-1, max_slots) or naming a free slot count as -1 and set
 * LML_FLAG_BAD_SLOT, exactly as in lml_segment_tokens.  x, W0, y as in lora_mixed_linear.
 * T <= 16: one launch; the decode kernel treats every row on its own and reads the ids itself, no
 * grouping is computed.  A few blocks of 16 tokens (T <= 48 where d_in * d_out <= 2^24; else T <= 32 where d_in > 4096) are
 * one launch of the same kernel, an equal share of its CTAs per block: every block's rows are bit for
 * bit those of a decode call on that block, and W0 still leaves HBM once.  Beyond that, up to one
 * row tile (T <= 128; two tiles, T <= 256, where d_in <= 4096): two launches, the tokens staying in
 * their order; the first binds them and writes, per row tile and distinct slot, the slot's rows of
 * the shrink result, the GEMM adds them slot by slot.  Larger T: the segmentation pass runs into the
 * tail of the workspace and the perm form of lora_mixed_linear follows on the same stream; results
 * are then identical to lml_segment_tokens followed by lora_mixed_linear (on the other paths they
 * agree with it to fp32 summation order and the bf16 rounding of u).  workspace: device, 256-byte aligned, at least
 * lml_tokens_workspace_bytes(t, T) bytes.  Errors: INVALID_ARG, WORKSPACE, CUDA.
 */
size_t lml_tokens_workspace_bytes(const lml_table* t, int max_tokens);
lml_status lora_mixed_linear_tokens(lml_table* t, const void* x, const void* W0, int T,
                                    const int32_t* token_slots, void* y, void* workspace,
                                    size_t workspace_bytes, void* stream);

/*
 * lora_mixed_linear_multi — several projections that read the same x in one call: q / k / v of an
 * attention block, gate / up of an MLP (a decoder layer runs all of its projections at every step;
 * the paper's runtime replays decode steps from CUDA graphs, Section 7.7).  Projection p has its own
 * table tables[p] (its own adapters, ranks, scales), base weight W0[p] (device bf16
 * [d_out_p][d_in]), per-token binding token_slots[p] (device int32[T]: slot of tables[p] per row of
 * x, or -1; the pointers may be equal when the tables were filled in the same order) and output
 * y[p] (device bf16 [T][d_out_p], distinct buffers).  tables, W0, token_slots and y are HOST arrays of
 * P pointers, 1 <= P <= LML_MAX_PROJECTIONS; all tables share d_in and the device.
 * T <= 16: ONE launch of the decode kernel for all projections.  Its CTAs are dealt out over the projections in
 * proportion to their rows; each works on its projection exactly as in a call of its own, so results per
 * projection are bit for bit those of lora_mixed_linear_tokens on that projection, and the fixed cost of a
 * call (the wait for the preceding work, the fetch of x, the tail) is paid once.  A single projection, or a
 * table named twice, runs as one decode call per projection.
 * T > 16: the projections run one after the other on `stream`, each exactly as
 * lora_mixed_linear_tokens(tables[p], ...).
 * Every projection's CTAs count themselves in that table's exchange block, as in a decode call: two calls
 * that share a table must not overlap on the GPU.  Device-detected errors set the flags of the table they
 * concern.
 * workspace: device, 256-byte aligned, at least lml_multi_workspace_bytes(tables, P, T).
 * Errors: INVALID_ARG, WORKSPACE, CUDA.
 */
size_t lml_multi_workspace_bytes(lml_table* const* tables, int P, int max_tokens);
lml_status lora_mixed_linear_multi(lml_table* const* tables, int P, const void* x, const void* const* W0, int T,
                                   const int32_t* const* token_slots, void* const* y, void* workspace,
                                   size_t workspace_bytes, void* stream);

/*
 * The same two calls for callers that hold ADAPTER ids per token instead of slots: every id is
 * resolved on the device to the adapter's serving slot at the moment the call runs in stream
 * order (see lml_publish).  -1 means no adapter; an id without a serving version counts as -1 and
 * sets LML_FLAG_BAD_SLOT.  Otherwise identical to lml_segment_tokens / lora_mixed_linear_tokens.
 */
lml_status lml_segment_tokens_adapters(lml_table* t, const int32_t* token_adapter_ids, int T, int32_t* perm,
                                       int32_t* seg_offsets, int32_t* seg_slot_ids, void* stream);
lml_status lora_mixed_linear_adapters(lml_table* t, const void* x, const void* W0, int T,
                                      const int32_t* token_adapter_ids, void* y, void* workspace,
                                      size_t workspace_bytes, void* stream);

/*
 * Host-buffer form of the same call, for callers whose activations live in host memory.
 * x_host, seg_offsets_host, slot_ids_host, perm_host (may be NULL), y_host are HOST pointers
 * (pinned memory makes the copies asynchronous); W0 stays a device pointer (resident
 * weight).  The call enqueues on `stream`: copies in, the layer, the copy of y out.  The
 * device staging lives in `workspace`, which must hold lml_host_workspace_bytes().  y_host
 * is valid once the stream has been synchronised.  Errors as lora_mixed_linear.
 * Up to LML_DECODE_MAX_TOKENS tokens, when every host buffer is pinned (cudaHostAlloc /
 * cudaHostRegister; x_host and y_host 16-byte aligned), no copy is enqueued at all: one kernel
 * reads the inputs out of host memory into the staging and the decode kernel writes y straight
 * into y_host (two launches).  Pageable buffers, and larger calls, take the copies.
 * From 2048 tokens on, with pinned x_host and y_host and no perm, the call runs in eight chunks of
 * whole 128-row tiles: the copy of the next chunk's x, the layer on this chunk and the copy of the
 * last chunk's y proceed side by side on the caller's stream and two streams that belong to the
 * table (created with it; the call creates nothing), and the caller's stream is made to wait for
 * the last copy, so stream order is what the caller sees.  Results are those of lora_mixed_linear
 * on the same rows.
 */
size_t lml_host_workspace_bytes(const lml_table* t, int max_tokens, int max_segments);
lml_status lora_mixed_linear_host(lml_table* t, const void* x_host, const void* W0, int T,
                                  const int32_t* seg_offsets_host, const int32_t* slot_ids_host,
                                  int G, const int32_t* perm_host, void* y_host, void* workspace,
                                  size_t workspace_bytes, void* stream);

/*
 * lora_mixed_linear_decode_static — the decode form of lora_mixed_linear (T <= 16) for callers
 * that cannot give the library a workspace.  (The paper has no counterpart; this entry point
 * exists for integration only.)
 *
 * Who needs it: code that runs where device memory cannot be obtained — a plug-in or callback
 * invoked by a host runtime that owns all allocations and forbids cudaMalloc from inside the
 * callback, a real-time loop that must not touch the allocator, a process whose memory budget
 * was handed out completely at start-up.  Such a caller still passes its inputs and the output
 * (x, W0, seg_offsets, slot_ids, perm, y: same meaning, layout and alignment as in
 * lora_mixed_linear), but no workspace: the scratch the decode kernel needs between its two
 * phases (the scaled shrink result, 16 x 64 fp32, each value beside the mark of the launch that
 * wrote it, and three counters) lives in an 8448-byte array inside the library image.  Every GPU that loads the library holds that array until the
 * process exits.  The call allocates and frees nothing, and calls no allocating routine.
 *
 * Limits and rules
 *   - T <= LML_DECODE_MAX_TOKENS (16).  A larger T is refused with LML_ERR_TOO_LARGE before
 *     anything is launched; use lora_mixed_linear with a workspace for it.
 *   - Every call looks up the array's device address (cudaGetSymbolAddress, with the table's device
 *     current; no allocation).  The first call on a device may load the library's device code:
 *     make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps the previous call's contents:
 *     it starts as zeros (a file-scope object), and its own launch counter tells a call's values
 *     from those of earlier calls, whichever table they were for.  Two calls that overlap on the GPU (different streams without ordering, or concurrent
 *     graph branches) race on the array: order them.
 *   - Results are identical to lora_mixed_linear on the same inputs.
 * Errors: INVALID_ARG, TOO_LARGE, CUDA.
 */
lml_status lora_mixed_linear_decode_static(lml_table* t, const void* x, const void* W0, int T,
                                           const int32_t* seg_offsets, const int32_t* slot_ids, int G,
                                           const int32_t* perm, void* y, void* stream);

/*
 * Read and clear the sticky device status word (LML_FLAG_* bits).  Synchronises `stream`.
 * When the word carries LML_FLAG_TIMEOUT (a launch gave up on a wait), the table's decode exchange blocks
 * (values, marks, counters) are put back to zero as well; no decode call on the table may be in flight then.
 * Errors: INVALID_ARG, CUDA.
 */
lml_status lml_device_status(lml_table* t, uint32_t* flags_out, void* stream);

/* Number of kernels the last lora_mixed_linear / lml_segment_tokens call on this table
 * launched (for launch accounting in benchmarks). */
int lml_last_launch_count(const lml_table* t);

#ifdef __cplusplus
}
#endif
#endif /* LORA_MIXED_LINEAR_H_ */
