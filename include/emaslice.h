/* emaslice.h — C ABI of libemaslice.so: the memory-slice hot path on one B200 (sm_100a).
 *
 * A memory slice (paper, Section 4) is a segment shared by two GPUs; a user's data may sit in its
 * own part ("local") or in the part the peer contributed ("lent"). Before a layer runs, the slice
 * side prepares a directly accessible address and prefetches the data (Section 5.1), inside the
 * latency window between two uses of the same layer (Section 2.3); the lender can take its memory
 * back at any time (Section 4.1). On one GPU the lent part is a separate arena that only the
 * prefetch, write-back, append and reclaim kernels touch; attention reads the local arena and the
 * staging ring only.
 *
 * Conventions
 *   - No exception, abort or print crosses this boundary. Every call returns a status code
 *     (0 = OK, negative = error, see slice_strerror). A failing call leaves tables, free lists and
 *     capacities unchanged.
 *   - "device pointer": memory the GPU can address (HBM; for the lent arena optionally mapped
 *     pinned host memory). "host pointer": ordinary host memory. The caller owns every buffer it
 *     passes; arenas and staging must outlive the slice and be 256-byte aligned.
 *   - Streams are cudaStream_t values passed as void*. prefetch_layer, paged_decode,
 *     slice_append_kv, slice_writeback_layer and slice_reclaim enqueue work and return; the
 *     library orders them with its own events (attention of a layer waits for that layer's
 *     prefetch; a prefetch into a ring slot waits for the attention that last read the slot;
 *     reclaim waits for everything outstanding and invalidates what is staged).
 *   - One caller thread per slice.
 *
 * Data layout
 *   block      = K plane [block_tokens][num_kv_heads][head_dim] bf16, then the V plane of the
 *                same shape: 2*16*8*128*2 = 65 536 bytes for the shapes used here.
 *                Storage order inside a token row: within every aligned 128 bytes of row r, the
 *                16-byte unit u (8 bf16) is stored at unit u ^ (r & 7). The permutation is its own
 *                inverse; slice_append_kv writes it, paged_decode reads it, and the copy paths
 *                (prefetch, write-back, reclaim) move whole blocks and never look inside. It lets a
 *                plane go from HBM to shared memory as ONE linear bulk copy and still be read by
 *                ldmatrix without bank conflicts. A caller that fills blocks itself applies the
 *                same permutation (the Python binding has kv_block_swizzle for it).
 *   arena      = [layer][block id][block]; byte address = base + layer*layer_stride
 *                + id*block_stride (strides 0 select the dense default).
 *   staging    = [ring slot][position][block], dense.
 *   table entry (int32): e >= 0 is local id e; e < 0 is lent id ~e. Block ids are the same for
 *                every layer (Section 4.2.1: allocation "applied uniformly across all layers").
 *   resolved entry (int32): e >= 0 is local id e; e < 0 is staging position ~e.
 *   Supported shapes: head_dim 128, block_tokens 16, num_kv_heads 1..8, bf16,
 *   num_q_heads = G * num_kv_heads with G in 1..8.
 */
#ifndef EMASLICE_H_
#define EMASLICE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ema_slice slice_t; /* opaque; the library owns metadata, events and work lists */

enum {
  SLICE_OK = 0,
  SLICE_EINVAL = -1,   /* bad id, shape, pointer or argument                                   */
  SLICE_ENOSPC = -2,   /* not enough free blocks: capacity beyond the local part is not
                          guaranteed (Section 5.1); the caller preempts and retries             */
  SLICE_ESTAGING = -3, /* the batch's lent blocks exceed a ring slot                            */
  SLICE_ESTALE = -4,   /* paged_decode of a layer whose prefetch for this batch is not valid     */
  SLICE_ECUDA = -5,    /* a CUDA call failed; slice_stats reports the code                       */
  SLICE_ETIMEOUT = -6, /* a bounded device-side wait expired (reported through slice_stats)      */
  SLICE_ESTATE = -7,   /* unknown sequence, double free                                          */
  SLICE_ESCRATCH = -8, /* paged_decode_noalloc: the batch needs more than the static scratch array */
  SLICE_ECAPPED = -9   /* slice_alloc_blocks: a cap set by an earlier preemption still holds
                          (Section 5.3); the request waits, nobody is preempted for it          */
};

enum { SLICE_TIER_AUTO = 0, SLICE_TIER_LOCAL = 1, SLICE_TIER_LENT = 2 };

enum {
  SLICE_FLAG_PROFILE = 1u,     /* record timing events around the kernels (slice_layer_times)     */
  SLICE_FLAG_TRACE = 2u,       /* per-CTA device-timer traces (slice_cta_trace)                    */
  SLICE_FLAG_NULL_DEVICE = 4u  /* tables only: no CUDA call is made, no kernel is launched       */
};

/* TEST HOOKS, not for callers: further bits of slice_config_t.flags with which the library's own
 * tests make a failure happen on the host side, without faulting anything on the GPU. */
enum {
  SLICE_FLAG_TEST_WITHHOLD_Q = 8u, /* bounded waits: queries streamed in from pinned host memory
                                      arrive, their arrival flags are never written, so the kernel's
                                      wait for them runs out (about two seconds) and it returns with
                                      SLICE_ETIMEOUT in slice_stats().device_status               */
  SLICE_FLAG_TEST_FAIL_COPY = 16u  /* slice_reclaim / slice_reclaim_preempt: the step that enqueues
                                      the migration reports failure like a failed CUDA call
                                      (SLICE_ECUDA); the state must be left as it was              */
};

typedef struct {
  uint32_t num_layers, num_kv_heads, head_dim, block_tokens;
  uint32_t dtype;                 /* 0 = bf16 */
  uint32_t local_blocks;          /* local capacity in block ids                                 */
  uint32_t lent_blocks;           /* lent capacity now; changes with slice_reclaim / slice_lend  */
  uint32_t lent_blocks_physical;  /* size of the lent arena in block ids (>= lent_blocks)        */
  uint32_t ring_slots;            /* staging ring depth R >= 1; layer l uses slot l mod R        */
  uint32_t staging_blocks_per_slot;
  uint32_t max_seqs, max_blocks_per_seq;
  uint32_t lent_kind;             /* 0 = device HBM arena, 1 = mapped pinned-host arena (a slow link:
                                     in the fused pipelines only a few SMs then copy; copy_ctas, if
                                     set, says how many)                                          */
  uint32_t flags;                 /* SLICE_FLAG_*                                                */
  void* local_base;               /* device pointers, caller-owned (may be NULL with NULL_DEVICE) */
  void* lent_base;
  void* staging_base;
  uint64_t local_layer_stride, local_block_stride; /* bytes; 0 = dense                          */
  uint64_t lent_layer_stride, lent_block_stride;
  const uint32_t* local_free_order; /* host; optional pop order of local ids (a permutation of
                                       0..local_blocks-1); NULL = ascending                      */
  const uint32_t* lent_free_order;  /* host; optional permutation of 0..lent_blocks_physical-1;
                                       ids >= lent_blocks are skipped at creation                */
  uint32_t decode_ctas;           /* 0 = one per SM; CTAs of the layer (attention) kernel        */
  uint32_t copy_ctas;             /* 0 = default; CTAs of the stand-alone gather / migration kernel */
  uint32_t copy_kind;             /* stand-alone gather, write-back and migration kernel: 0 = default (gather
                                     and write-back: 3; migration: 2), 1 = vector load/store kernel, 2 =
                                     bulk-copy ring of 8 x 16 KB per CTA (fastest alone), 3 = the same
                                     with 6 stages: a CTA of it fits on an SM beside a CTA of the
                                     attention kernel, so a gather on a second stream runs WHILE the
                                     attention does instead of taking turns with it                 */
  uint32_t pipeline_mode;         /* slice_decode_step: 0 = one persistent launch for the whole pass
                                     (attention of layer l overlapped with the gather of layer l+1,
                                     soft layer boundaries; falls back to 2 when the shape does not
                                     allow it), 1 = two kernels on two streams ordered by events,
                                     2 = one fused launch per layer, the stream ordering the layers,
                                     3 = a chain of fused launches, one per layer, in which each
                                     launch starts while the one before it still runs (programmatic
                                     dependent launch): its CTAs take the SMs that the earlier
                                     launch's CTAs leave and the layers order themselves through the
                                     same flags and counters as inside the single launch of mode 0.
                                     Same fall-back as mode 0. Nothing else may be enqueued on
                                     `stream` by other threads while slice_decode_step enqueues a
                                     chain                                                        */
  uint32_t static_split;          /* attention work split: 0 = each CTA owns a range of blocks and idle
                                     CTAs steal from the ranges with most left (default); 1 = static
                                     ranges only                                                  */
  uint32_t claim_blocks;          /* most KV blocks a CTA claims from its own range at a time
                                     (0 = default 16, at most 32); smaller claims leave more for idle
                                     CTAs to steal, larger ones cost fewer atomics               */
  uint32_t steal_floor;           /* persistent pass (pipeline_mode 0): before the last layer an idle
                                     CTA steals only from a range with at least this many blocks
                                     left, and otherwise starts on the next layer. 0 = default (a
                                     third of a range; 8 blocks in the last layer of a launch and
                                     in single-layer launches); 1 = steal down to the last block, which
                                     keeps all CTAs in step: almost no CTA ever waits for
                                     prefetched data, at a lower overall rate                    */
  uint32_t prefetch_priority;     /* one launch per pass: 0 = default, the layers take turns with four
                                     buffers of split-KV partials, so a CTA may run up to three
                                     layers ahead of the slowest merge; attention follows the
                                     prefetch closely, waits for it part of the time and reads
                                     staged blocks out of L2 (highest tokens/s); 1 = two buffers:
                                     the CTAs stay within a layer of one another, the prefetch is
                                     far ahead of all of them, attention (almost) never waits for
                                     it, staged blocks come from DRAM and the pass is slower.
                                     (Layer-dependent passes, slice_step_begin, have a hard boundary
                                     after every layer: the setting changes little there)          */
  uint32_t slab_blocks;           /* Section 4.2.1: 0 = blocks are handed out one by one from free stacks
                                     (the seeded orders); S > 0 = slab allocator: the ids of each part
                                     form slabs of S consecutive ids (the paper's default is 10,
                                     Section 6.7), a slab belongs to the user while one of its blocks
                                     is in use, and the next id is the lowest free id in a slab the
                                     user holds, else the lowest free id of all (a new slab). The
                                     free orders must then be NULL                                 */
  uint32_t layer_group;           /* Section 4.2.2: layers per layer group, the unit of a swap (0 or 1 =
                                     single layers; the paper's default is 4). A ring slot holds one
                                     group: staging is [ring_slots][layer_group][staging_blocks_per_slot]
                                     blocks, layer l is staged in layer slot l mod (ring_slots *
                                     layer_group), and the pipelines fetch layer l + layer_group
                                     while layer l is attended to (a group's transfer is issued as
                                     one piece per layer, at the start of each layer of the group
                                     before; buffer and latency window are those of a group)       */
  uint32_t layout;                /* Sections 4.2.1-4.2.3, order of the blocks in BOTH arenas (bytes;
                                     bb = block bytes, S = slab_blocks, k = layer_group, N = ids of
                                     the arena, L = layers): 0 layer-major [layer][id] (strides may
                                     override it); 1 slab-major [slab][layer][block in slab];
                                     2 layer-group-major [group][slab][layer in group][block in slab].
                                     1 and 2 need S > 0, N a multiple of S for both arenas, L a
                                     multiple of k, and zero strides                               */
  uint32_t split_layer;           /* Section 4.1, the paper's own placement (expansion ratio 2 when it is
                                     half the layers): 0 = off, blocks are placed local or lent one
                                     by one; s in 1..L-1 = every block keeps layers 0..s-1 in the
                                     local arena and layers s..L-1 in the lent arena, under the same
                                     block id. The local arena then holds s layers, the lent arena
                                     L - s (its first layer is layer s) with at least local_blocks
                                     ids, ids come from the local list only (hint LENT is EINVAL),
                                     layers below s are attended to in place, layers from s on are
                                     prefetched whole (every block of the batch, staging position =
                                     position of the block in the batch), and slice_reclaim does not
                                     apply (EINVAL): the lender regains memory by preemption. Needs
                                     layout 0                                                       */
  uint32_t swap_out;              /* Section 2.3 (layers are swapped in AND out, cyclically; what comes in
                                     must be matched by what goes out): 0 = the ring holds read-only
                                     copies and slice_append_kv writes a new row to the home block and
                                     to the staged copy; 1 = write-back: slice_append_kv writes a row
                                     whose block is staged to the staged copy only, and every pass of
                                     slice_decode_step writes each staged layer back to the lent
                                     arena (all its staged blocks) while that layer is attended to and
                                     the next transfer comes in; a slot is refilled only after its
                                     write-back. With pipeline_mode 0 the copy threads of the pass's
                                     one launch do it; with the other pipelines the pass runs one
                                     launch per layer and the write-back goes on a stream of the
                                     library's own. 2 = the same, but a pass writes back only the
                                     blocks that can have changed since they were fetched: the staged
                                     tail block of every sequence of the batch (rows are appended
                                     nowhere else), a few MB per layer instead of the layer's whole
                                     lent part (slice_writeback_layer still writes the whole layer).
                                     After an append, run a pass (or
                                     slice_writeback_layer for the staged layers) before the tables
                                     change again, or the appended rows of staged blocks are lost   */
} slice_config_t;

typedef struct {
  uint32_t local_used, local_free, lent_used, lent_free, lent_capacity, num_seqs;
  uint64_t prefetch_calls, prefetched_blocks, prefetched_bytes;
  uint64_t decode_calls, decode_tokens;
  uint64_t reclaims, migrated_blocks, migrated_bytes;
  uint64_t plans_built;          /* how often tables were re-resolved for a batch               */
  uint64_t kernel_launches;      /* kernels of this library launched so far                     */
  int32_t last_cuda_error;       /* cudaError_t of the last failed CUDA call, 0 if none         */
  int32_t device_status;         /* 0, or SLICE_ETIMEOUT if a kernel gave up a bounded wait (a word in
                                    mapped host memory that the kernels write: reading it makes no
                                    CUDA call and waits for nothing)                            */
} slice_stats_t;

/* Section 4 (memory slice with a mapping table per user). Creates the allocator state and the
 * device-side work lists. cfg and the free orders are host pointers, read during the call only.
 * out receives the handle. Errors: EINVAL (shape unsupported, NULL arena without NULL_DEVICE,
 * lent_blocks > lent_blocks_physical, ring_slots == 0), ECUDA. */
int slice_create(const slice_config_t* cfg, slice_t** out);

/* Frees what slice_create made after waiting for the slice's outstanding work. */
int slice_destroy(slice_t* s);

/* Section 4.1 (allocation tries the user's own free memory before anything else): appends n
 * logical blocks to sequence seq (created when absent). AUTO takes free local ids first and the
 * lent part only when local memory is exhausted; LOCAL / LENT force a tier (seeded placements). out_entries (host, n
 * entries, may be NULL) receives the new table entries. Errors: ENOSPC (nothing changes), EINVAL
 * (negative seq, bad hint, more than max_seqs sequences or max_blocks_per_seq blocks), ECAPPED
 * (n > 0 and a cap from an earlier preemption holds, see slice_preempt_seq; nothing changes). */
int slice_alloc_blocks(slice_t* s, int32_t seq, uint32_t n, int32_t tier_hint, int32_t* out_entries);

/* Sets the number of valid tokens of seq; len <= block_tokens * allocated blocks.
 * Errors: ESTATE (unknown seq), EINVAL. */
int slice_set_seq_len(slice_t* s, int32_t seq, uint32_t len);

/* Completion or preemption of a request (Section 4.1): its blocks return to the free lists, in
 * descending logical order. Errors: ESTATE. */
int slice_free_seq(slice_t* s, int32_t seq);

/* Copies the block table of seq to out (host, cap entries; may be NULL to query). n and len
 * (host, may be NULL) receive the number of blocks and tokens. Errors: ESTATE, EINVAL (cap). */
int slice_get_block_table(slice_t* s, int32_t seq, int32_t* out, uint32_t cap, uint32_t* n, uint32_t* len);

/* Test hook: free list of a tier (1 local, 2 lent) in pop order. */
int slice_get_free_stack(slice_t* s, int32_t tier, int32_t* out, uint32_t cap, uint32_t* n);

/* Sections 2.3, 4.2.1, 5.1: prefetch before use. For layer `layer` and the batch seqs[0..nseq)
 * (host array of distinct sequence ids), every in-use lent block is copied, in batch order then
 * logical order, from the lent arena into ring slot (layer mod R) at consecutive positions; the
 * batch's resolved table maps each lent block to its position. Enqueued on side_stream after the
 * attention that last read the slot. Errors: EINVAL, ESTATE, ESTAGING (before any copy), ECUDA. */
int prefetch_layer(slice_t* s, uint32_t layer, const int32_t* seqs, uint32_t nseq, void* side_stream);

/* The consumer of the prepared addresses (Section 5.1); the paper takes the attention kernel from
 * its serving engine (Section 6.1) and does not define it. Computes, for each sequence i of the
 * batch and query head h (KV head h / G): out = softmax(sm_scale * q K^T) V over tokens
 * 0..len-1, read through the resolved table from the local arena and the ring slot of `layer`.
 *   q, out  device, [nseq][num_q_heads][128] bf16;  lse_or_null device, [nseq][num_q_heads] f32
 *           (natural-log sum of exponentials of the scaled scores).
 * Arithmetic: bf16 products, f32 accumulation and softmax, bf16 result (nearest even).
 * The split-KV partials are merged inside the same launch. Calls on one slice must not overlap on
 * the GPU (they share the partial buffers): issue them on one stream or order them.
 * Enqueued on stream after the layer's prefetch. Errors: EINVAL (shape, zero-length sequence,
 * G > 8), ESTATE, ESTALE (batch has lent blocks and the slot does not hold a valid prefetch of
 * this layer for this batch and table state), ECUDA. */
int paged_decode(slice_t* s, uint32_t layer, const int32_t* seqs, uint32_t nseq, const void* q,
                 uint32_t num_q_heads, float sm_scale, void* out, float* lse_or_null, void* stream);

/* The paper has no counterpart to this entry point; it exists for callers that must not cause a
 * device memory allocation when they run attention. paged_decode obtains its split-KV scratch from
 * cudaMalloc on its first call (and again if a later call needs more). That is unusable for a server
 * that gave every byte of the GPU to its KV-cache pool at start-up, for a decode loop that cannot
 * tolerate the device-wide synchronisation an allocation brings, and under rules that forbid
 * allocator calls once initialisation is over. paged_decode_noalloc takes the same arguments,
 * computes the same result and orders itself on the streams the same way, but keeps the scratch in a
 * static device array built into the library: 8 MiB on every GPU on which a slice has been created
 * (or this entry point called), held until the process exits. The call itself makes no cudaMalloc,
 * cudaFree or other allocating call.
 *   Set-up: slice_create (without SLICE_FLAG_NULL_DEVICE) does everything that has to happen once
 *   per device, with that device current: it loads the part of the library that holds the array
 *   (under CUDA's lazy loading this is the moment the 8 MiB are reserved), looks up the array's
 *   device address and runs the attention kernels once on an empty batch. A first decode call
 *   therefore finds nothing left to set up. Should the look-up not have happened for the current
 *   device, the first call here does it; create slices, and make such a first call, outside any
 *   stream capture.
 *   Device: the call must be made with the slice's device current (the device that was current in
 *   slice_create); otherwise it returns SLICE_EINVAL and launches nothing.
 *   Limit: this entry point splits the work statically (no stealing between CTAs), which needs one
 *   partial slot per (sequence, CTA range it touches) plus one per sequence, i.e. at most
 *   2 * nseq + CTAs slots; slots * num_q_heads * 528 bytes plus about 8 bytes per (sequence, KV head)
 *   and 8 per CTA must fit in 8 MiB; larger requests return SLICE_ESCRATCH
 *   and change nothing.
 *   Sharing: all calls, from every slice in the process, use the one array, and it keeps the last
 *   call's contents (its counters are cleared on the stream before every launch; the partial rows
 *   need no clearing: each call overwrites what it later reads). Two
 *   calls whose kernels may overlap on the GPU (different streams without an ordering between them)
 *   race on it; issue them on one stream or order them with events.
 * Errors: as paged_decode, plus SLICE_ESCRATCH and SLICE_EINVAL (other device current). */
int paged_decode_noalloc(slice_t* s, uint32_t layer, const int32_t* seqs, uint32_t nseq, const void* q,
                         uint32_t num_q_heads, float sm_scale, void* out, float* lse_or_null, void* stream);

/* Section 4.1: the lender regains capacity immediately. The paper reclaims by preempting the
 * borrower's requests; this entry migrates instead. The top `take_blocks` ids of the lent range
 * (UINT32_MAX = all) leave the slice; in-use blocks there move, for every layer, to free local ids
 * first and then to the smallest free lent ids below the cut; tables and free lists are rewritten
 * and everything staged becomes invalid. out_n_migrated (host, may be NULL) receives the number of
 * block ids moved. The copy is enqueued on stream after all outstanding work of the slice; later
 * calls on other streams wait for it. Errors: ENOSPC (no room; nothing changes), ECUDA. */
int slice_reclaim(slice_t* s, uint32_t take_blocks, uint64_t* out_n_migrated, void* stream);

/* Section 4.1 as the paper states it: where the migration of slice_reclaim has no room, requests of
 * the borrower are preempted until it has. Section 4.2.1 gives the choice: the slab with the fewest
 * active requests. Slabs are runs of slab_blocks consecutive lent ids (the paper's default is 10;
 * the last slab may be short). While the in-use blocks of the reclaimed range outnumber the free
 * places (local, or lent below the cut), the slab of the lent range that holds blocks of the
 * fewest distinct requests (at least one; among equals the highest slab, which lies nearest the
 * reclaimed range) loses all its requests, in ascending id order: they are freed as by
 * slice_free_seq and the caller re-queues them. What then remains in the range migrates as in
 * slice_reclaim (same stream ordering). The call never fails for lack of room.
 *   victims     host, cap entries: the preempted sequence ids in eviction order; n_victims (host,
 *               may be NULL) their number; out_n_migrated as in slice_reclaim.
 * Every victim counts as a preemption by reclamation and, as in slice_preempt_seq, can set the cap.
 * Errors: EINVAL (slab_blocks == 0, or cap smaller than the number of victims), ECUDA (the
 * migration could not be enqueued). After an error nothing has changed: no request was evicted, no
 * counter moved, no cap was set. */
int slice_reclaim_preempt(slice_t* s, uint32_t take_blocks, uint32_t slab_blocks, int32_t* victims, uint32_t cap,
                          uint32_t* n_victims, uint64_t* out_n_migrated, void* stream);

/* A preemption the serving engine chose itself: frees seq like slice_free_seq and counts it by
 * cause (Section 5.2 names the two, Section 6.6 reports them): SLICE_PREEMPT_OOM, the user's own
 * requests give way because capacity is exhausted, or SLICE_PREEMPT_RECLAIM, the lender took
 * memory back. Section 5.3, against back-and-forth preemption under bursty load: a user preempted
 * by reclamation while it holds more than its static share (the local part of the slice, half of a
 * symmetric slice) may afterwards not grow beyond the level it was preempted to, for a window of
 * length T; a later such preemption inside the window can only lower the level and restarts the
 * window; once T has passed without one the cap is lifted. While the cap holds,
 * slice_alloc_blocks returns SLICE_ECAPPED for a request that would pass the level.
 * Errors: EINVAL (cause), ESTATE (unknown seq). */
enum { SLICE_PREEMPT_OOM = 1, SLICE_PREEMPT_RECLAIM = 2 };
int slice_preempt_seq(slice_t* s, int32_t seq, int32_t cause);

/* Section 5.3 leaves T and its unit open: the caller sets the window (0, the default, = no cap is
 * ever set) and reports the time in the same unit (steps, milliseconds, ...); time must not run
 * backwards (EINVAL). */
int slice_set_preempt_window(slice_t* s, uint64_t window);
int slice_set_time(slice_t* s, uint64_t now);

typedef struct {
  uint64_t preempt_oom, preempt_reclaim; /* requests preempted so far, by cause                    */
  uint64_t now, window;
  uint64_t cap_until;                    /* the cap holds while now < cap_until; 0 when none holds */
  uint64_t cap_level;                    /* blocks the user may hold while it holds; 0 when none   */
} slice_preempt_stats_t;
int slice_preempt_stats(slice_t* s, slice_preempt_stats_t* out);

/* Section 5.2: a process with several slices (one per peer, Section 5.1) sends each request to the
 * slice k with the smallest util_{k,i} + util_{k,j} (Greedy-Least-Loaded; Appendix C bounds its peak
 * utilisation by (m + 3) / 2 times the offline optimum for m GPUs). A slice's capacity is all its
 * block ids, local part plus the peer's whole arena; util_{k,i} = blocks this user holds / capacity;
 * util_{k,j} = blocks the peer itself holds / capacity, which only the peer knows: its side reports
 * the number with slice_set_peer_used (0 until then). Errors: EINVAL (more than the peer's arena). */
int slice_set_peer_used(slice_t* s, uint32_t peer_blocks);

/* Picks among slices[0..n) (host array of handles) by the rule above, compared exactly (as
 * fractions, not in floating point); among equals the first. out_index (host) receives the choice.
 * Nothing is allocated: the caller then calls slice_alloc_blocks on that slice. Errors: EINVAL
 * (n == 0, NULL handle). */
int slice_schedule_gll(slice_t* const* slices, uint32_t n, uint32_t* out_index);

/* The lender offers n more block ids (the share of a slice is renegotiated at run time,
 * Section 1 / 4.1). New ids are handed out in ascending order. Errors: EINVAL (beyond arena). */
int slice_lend(slice_t* s, uint32_t n_blocks);

/* One new token per sequence (the caller has already grown len and allocated a block where
 * needed): writes K and V rows of token len-1 for `layer` into the home block and, when the home is
 * lent and the layer is validly staged for this batch, into the staged copy too.
 *   k_new, v_new  device, [nseq][num_kv_heads][128] bf16 (canonical order; the call applies the block
 *                 format's swizzle).
 *   layer == SLICE_ALL_LAYERS appends to every layer in one launch (at most 128 layers):
 *                 k_new, v_new are then [num_layers][nseq][num_kv_heads][128]. */
#define SLICE_ALL_LAYERS 0xFFFFFFFFu
int slice_append_kv(slice_t* s, uint32_t layer, const int32_t* seqs, uint32_t nseq, const void* k_new,
                    const void* v_new, void* stream);

/* The way back (swap-out direction of Section 4): every staged block of the batch's layer is
 * written from its ring slot to its home in the lent arena. Requires a valid prefetch of the
 * layer for this batch (ESTALE otherwise). */
int slice_writeback_layer(slice_t* s, uint32_t layer, const int32_t* seqs, uint32_t nseq, void* stream);

/* One pass of the whole path over a batch: for every layer, the prefetch of layer l+1 overlapped
 * with the attention of layer l (cyclic: the last layer's attention overlaps the prefetch of layer 0
 * for the next pass when wrap_prefetch != 0). With pipeline_mode 0, 2 or 3 and a ring of at least two
 * slots both run inside the same kernel on `stream` (side_stream is not used): one launch for the
 * whole pass (mode 0) or one per layer (mode 2; mode 3, in which the launches overlap); with
 * pipeline_mode 1 the gather kernel runs on side_stream and the attention kernel on stream, ordered
 * by events, the two sharing the SMs.
 *   q, out: [num_layers][nseq][num_q_heads][128] bf16; device pointers when io_on_host == 0.
 *   With io_on_host != 0 they are host pointers. Pageable memory: q is copied to the device and out
 *   back to the host on `stream`, inside the call's enqueued work, through device buffers the
 *   library allocates on first use. Pinned memory: the kernels write out straight into it (every
 *   finished row goes to the host while the pass goes on; complete when the work enqueued on
 *   `stream` is), and when one launch covers the pass q is brought in behind the running kernel on
 *   a copy stream of the library's own, a few layers per copy, each copy followed by an arrival
 *   flag that the kernel checks (bounded wait, SLICE_ETIMEOUT through slice_stats) before it reads
 *   that layer's rows. The caller must not change q before the work enqueued on `stream` is done. */
int slice_decode_step(slice_t* s, const int32_t* seqs, uint32_t nseq, const void* q, uint32_t num_q_heads,
                      float sm_scale, void* out, int32_t io_on_host, int32_t wrap_prefetch,
                      void* stream, void* side_stream);

/* Sections 2.3 and 5.1: the layer-dependent form of the one-launch pass. In a decoder the queries of
 * layer l+1 exist only after layer l's output has gone through the rest of the block; the latency
 * window in which the prefetch of a layer hides is exactly that time. slice_step_begin enqueues
 * the same persistent launch as slice_decode_step (pipeline_mode 0, device q and out, same layout),
 * except that the attention of EVERY layer l first waits, bounded, for the arrival of q[l], and that
 * the merge which completes out[l] announces it. The gathers do not wait for queries: while a
 * layer's attention waits for its q, the copy threads go on prefetching.
 *   slice_step_begin      enqueues the pass on `stream` and returns. No layer's queries count as
 *                         arrived yet, layer 0 included.
 *   slice_step_submit_q   enqueues on caller_stream, behind the work already enqueued there (which
 *                         wrote q[layer]), a write of layer's arrival word.
 *   slice_step_wait_out   makes caller_stream wait until out[layer] is complete.
 *   slice_step_flags      for callers whose own kernels do the signalling instead: device addresses
 *                         of the two arrays of 32-bit words (one word per layer) and the epoch of
 *                         the pass. q[l] has arrived when q_ready[l] >= epoch (write q, fence, then
 *                         the word); out[l] is complete once out_ready[l] >= epoch (acquire).
 * submit / wait / flags refer to the pass begun last; begin the next pass only after all of them
 * have been enqueued for this one. caller_stream must differ from `stream` (which the running
 * launch occupies). The launch holds every SM it runs on for the whole pass, with nearly all of
 * their shared memory: kernels of the caller that are to run meanwhile (device-to-device copies are
 * kernels in this sense) need SMs of their own, i.e. decode_ctas below the SM count, and must have
 * run once before the pass begins (a kernel's first launch loads its code, which does not finish
 * while the pass runs); the two calls above need neither. A q that does not
 * arrive within the kernel's bounded wait (about two seconds) ends the launch with SLICE_ETIMEOUT in
 * slice_stats().device_status.
 * Errors: EINVAL (pipeline_mode other than 0, a ring of one slot, fewer than 2 or more than 128
 * layers, more CTAs than SMs; submit / wait / flags without a pass begun by slice_step_begin),
 * ECUDA (the driver offers no stream memory operations), and those of slice_decode_step. */
int slice_step_begin(slice_t* s, const int32_t* seqs, uint32_t nseq, const void* q, uint32_t num_q_heads,
                     float sm_scale, void* out, int32_t wrap_prefetch, void* stream);
int slice_step_submit_q(slice_t* s, uint32_t layer, void* caller_stream);
int slice_step_wait_out(slice_t* s, uint32_t layer, void* caller_stream);
int slice_step_flags(slice_t* s, uint32_t** q_ready, uint32_t** out_ready, uint32_t* epoch);

/* Measurement and test utility for the calls above (the paper has no counterpart): enqueues on
 * caller_stream a one-thread kernel that plays the rest of a decoder whose work between two
 * attention layers takes no time. It releases q[0] at once and q[l+1] as soon as out[l] is announced,
 * through the device words of slice_step_flags (about a microsecond per hand-over; the stream-ordered
 * slice_step_wait_out + slice_step_submit_q pair costs tens of microseconds per layer). The caller
 * must have put q[l+1] where out[l] is written (q = X, out = X + one layer) or not care what the
 * later layers attend to. Needs an SM the pass leaves free: EINVAL unless decode_ctas is below the
 * SM count, or without a pass begun by slice_step_begin. Bounded waits as everywhere. */
int slice_step_relay(slice_t* s, void* caller_stream);

/* Counters and capacities (host struct). */
int slice_stats(slice_t* s, slice_stats_t* out);

/* Test hook: resolved table of the batch, as [nseq][max_blocks_per_seq] int32 on the host (entries
 * past a sequence's in-use blocks are left untouched); k receives the number of staged blocks. */
int slice_get_resolved(slice_t* s, const int32_t* seqs, uint32_t nseq, int32_t* out, uint32_t cap, uint32_t* k);

/* With SLICE_FLAG_PROFILE: after synchronising, returns for each layer of the most recent pass
 * five times in microseconds relative to the pass's first event: prefetch start, prefetch end,
 * attention start, attention end (after the merge), end of the attention kernel proper (before the
 * merge) (host, [num_layers][5] floats; NaN where not recorded). A pass done in one launch records
 * only the attention start of layer 0 and the two end times of the last layer. */
int slice_layer_times(slice_t* s, float* out, uint32_t cap_layers);

/* With SLICE_FLAG_PROFILE: per-CTA times (GPU nanosecond timer) of the most recent launch of each
 * layer's kernel, as [num_layers][ctas_per_layer][words_per_cta] uint64 on the host; unused entries
 * are 0. which = 0: layer kernel, 8 words (time the CTA started on the layer, nanoseconds its
 * attention waited for the layer's prefetched blocks, end of the copy work it did during the layer,
 * SM id | runs << 16 | claims << 32, time its producer had issued the layer's last block, time its
 * first consumer warp finished its last run of the layer, nanoseconds that warp waited for the
 * layer's queries, time it first had them: the last two only where queries arrive while the launch
 * runs); which = 1: stand-alone gather kernel, 2 words (start, end). out may be NULL to query
 * the two sizes. Synchronises the device. */
int slice_cta_trace(slice_t* s, int32_t which, uint64_t* out, uint64_t cap_entries, uint32_t* ctas_per_layer,
                    uint32_t* words_per_cta);

/* Low-level copy used by the prefetch microbenchmark: n blocks of block_bytes (a multiple of 16
 * bytes, 16-byte aligned addresses) are copied dst_base + dst_idx[i]*block_bytes <-
 * src_base + src_idx[i]*block_bytes. Index arrays and bases are device pointers; dst_idx or src_idx
 * may be NULL for the identity. kind: 0 default (vector), 1 vector load/store, 2 bulk-copy ring,
 * 3 bulk-copy ring of 6 stages. */
int slice_copy_blocks(void* dst_base, const int32_t* dst_idx, const void* src_base, const int32_t* src_idx,
                      uint32_t n, uint64_t block_bytes, uint32_t kind, uint32_t ctas, void* stream);

/* The prefetch / migration microbenchmark's inner loop, so that launches of a few blocks are not
 * timed through a scripting language: blocks idx[0 .. n_total) (device array of ids into arena_base)
 * are gathered in launches of per_launch blocks into a ring of ring_slots staging slots of
 * slot_bytes each (launch j fills slot j mod ring_slots from position 0), or, with scatter != 0,
 * written from the slots back to those ids. n_total / per_launch launches are enqueued on stream;
 * a remainder is left out. Same kinds and alignment rules as slice_copy_blocks. */
int slice_copy_blocks_series(void* ring_base, uint32_t ring_slots, uint64_t slot_bytes, void* arena_base, const int32_t* idx,
                             uint64_t n_total, uint32_t per_launch, uint64_t block_bytes, int32_t scatter, uint32_t kind,
                             uint32_t ctas, void* stream);

const char* slice_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* EMASLICE_H_ */
