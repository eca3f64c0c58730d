// kernels.h — launch interface between the host side of libemaslice (slice.cpp) and its CUDA
// kernels (copy_kernels.cu, layer_kernel.cu, noalloc.cu). Internal to the library; not part of the
// C ABI.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace ema {

// Value written to the device status word when a bounded wait expires.
constexpr int kDevTimeout = -6;

// One batched block copy: item i moves block_bytes from src(entry src_entry[i]) to
// dst(entry dst_entry[i]) for each of nlayers layers. An entry e >= 0 addresses id e of base[0],
// e < 0 addresses id ~e of base[1]. A NULL entry array means entry i = i.
// Byte offset of layer l in an arena whose layers come in groups of k: group l / k starts at a
// multiple of group_stride, layer l % k of the group at a multiple of layer_stride (k = 1 and
// group_stride = layer_stride give the plain [layer] order).
__host__ __device__ inline uint64_t layer_offset(uint32_t l, uint32_t k, uint64_t group_stride, uint64_t layer_stride) {
  return static_cast<uint64_t>(l / k) * group_stride + static_cast<uint64_t>(l % k) * layer_stride;
}

struct CopyDesc {
  const uint8_t* src_base[2];
  uint8_t* dst_base[2];
  uint64_t src_block_stride[2];
  uint64_t dst_block_stride[2];
  uint64_t src_layer_stride[2];
  uint64_t dst_layer_stride[2];
  uint64_t src_group_stride[2];  // used when layer_group > 1 (see layer_offset)
  uint64_t dst_group_stride[2];
  uint32_t layer_group;          // 0 or 1: layers are src/dst_layer_stride apart
  const int32_t* src_entry;
  const int32_t* dst_entry;
  uint32_t n;
  uint32_t nlayers;
  uint64_t block_bytes;  // multiple of 16
  int* status;
  unsigned long long* trace;  // optional [grid][2] start/end %globaltimer per CTA (profiling)
};

// kCopyBulkShared: the bulk-copy ring with 6 instead of 8 stages (96 KB), small enough for a CTA of it
// to share an SM with a CTA of the layer kernel that gathers nothing itself.
enum CopyKind : uint32_t { kCopyDefault = 0, kCopyVector = 1, kCopyBulk = 2, kCopyBulkShared = 3 };

// Launches one copy kernel on `stream`. ctas == 0 picks a default grid. Returns the CUDA error.
cudaError_t launch_copy(const CopyDesc& d, uint32_t kind, uint32_t ctas, int num_sms, cudaStream_t stream);

// Device counters of ONE layer inside a layer-kernel launch; the whole block must be zero when the
// kernel starts. Layout in uint32 words:
//   [0, 32)                 launch words: [1] next copy unit of the gather issued during this layer,
//                           [2] attention work finished (blocks x KV heads); in a cache line of
//                           their own, which idle merge warps poll, [16] merge requests published,
//                           [17] merge requests taken, [18] query heads merged
//   [32, 32 + 2*ncta)       one 64-bit claim word per CTA range: blocks claimed from the front (low
//                           half, by the owner) and from the back (high half, by thieves)
//   [.., + nseq)            partial slots handed out per sequence
//   [.., + nseq*Hkv)        blocks finished per (sequence, KV head)
//   [.., + 8*nseq*Hkv)      merge requests in the order they were published:
//                           1 + 16*(sequence*Hkv + KV head) + (8 + query head of the group, for a
//                           request that covers one query head only, else 0)
constexpr uint32_t kLaunchCounters = 32;
constexpr uint32_t kCntCopyTicket = 1, kCntAttnDone = 2, kCntWbTicket = 3, kCntWbDone = 4, kCntMergePub = 16, kCntMergeTaken = 17,
                   kCntMerged = 18;
constexpr uint32_t kMaxStepLayers = 128;
// Consumer warps per KV head in the layer kernel, each leaving a partial of its own in every partial
// slot: with 1 to 4 KV heads the blocks of a unit are dealt to 8 / Hkv (8, 4, 2, 2) warps per head.
__host__ __device__ constexpr uint32_t partials_per_slot(uint32_t Hkv) { return Hkv <= 4 ? 8u / Hkv : 1u; }
// Words of the per-CTA, per-layer trace of the layer kernel: [0] time the CTA started on the layer,
// [1] ns its attention waited for prefetched blocks, [2] end of the copy work it did during the
// layer, [3] SM id | runs << 16 | claims << 32, [4] time its producer had issued the layer's last
// block, [5] time the first consumer warp finished its last run of the layer, [6] ns that warp
// waited for the layer's queries, [7] time it first had them.
constexpr uint32_t kTraceWords = 8;
constexpr uint32_t kSharedMergeMin = 12;  // partials from which a merge is offered to every CTA
constexpr uint32_t kSplitMergeMin = 48;   // partials from which it is offered one query head at a time
inline size_t layer_counter_words(uint32_t ncta, uint32_t nseq, uint32_t Hkv) {
  return kLaunchCounters + 2 * static_cast<size_t>(ncta) + nseq + 9 * static_cast<size_t>(nseq) * Hkv;
}

// Parameters of one launch of the layer kernel. It covers layers first_layer .. first_layer +
// num_layers - 1 of one batch; pointers refer to first_layer and the strides lead to the next layer.
struct LayerParams {
  const uint8_t* local_base;    // local arena; layer l starts at layer_offset(l, layer_group, local_group_stride,
  uint64_t local_group_stride;  //   local_layer_stride), and an entry e >= 0 addresses e * local_block_stride
  uint64_t local_layer_stride;  //   from there (entries are physical indices: the host has applied the layout)
  uint64_t local_block_stride;
  uint32_t layer_group;         // layers per group of the arenas' layout (>= 1)
  uint32_t prefetch_distance;   // the gather issued during launch layer i fetches layer i + prefetch_distance
  uint32_t split_layer;         // layer-split placement: from this layer on EVERY block of the batch is read from
                                //   the ring slot, at the position equal to its flat index (0xFFFFFFFF: no split;
                                //   then the resolved table says where each block is)
  const uint8_t* staging_base;  // ring: layer l is staged in slot l % ring_slots
  uint64_t slot_bytes;
  uint32_t ring_slots;
  uint32_t first_layer, num_layers;
  uint32_t li_begin, li_end;    // the layers first_layer + [li_begin, li_end) are what THIS launch runs. A pass may be
                                //   one launch (0, num_layers) or a chain of launches over the same parameter
                                //   block, each taking a slice of the layers (see `chained`)
  uint32_t chained;             // 0: a launch of its own. 1, 2: a link of a chain of launches in one stream, every
                                //   link lets its successor start as soon as all its own CTAs have started
                                //   (programmatic dependent launch; 2 = launched as such a successor). The
                                //   links order themselves through the same flags and counters as the layers
                                //   of a single launch, and a link ends only after its predecessor has ended
  uint64_t block_bytes;
  const int32_t* resolved;      // flat resolved table of the batch (batch order, then block order)
  const uint32_t* lens;         // [nseq] tokens
  const uint32_t* blk_seq;      // [total_blocks] batch position of each flat block
  const uint32_t* blk_off;      // [nseq + 1] first flat block of each sequence
  const uint32_t* seq_slot_base;// [nseq + 1] first partial slot of each sequence
  uint32_t total_blocks;
  uint32_t per;                 // blocks per CTA range; range c = [c*per, min((c+1)*per, total))
  uint32_t used_cta;            // number of non-empty ranges
  uint32_t allow_steal;         // 0: every range is processed by its owner only
  uint32_t own_chunk;           // most blocks an owner claims at a time
  uint32_t steal_floor;         // before the launch's last layer: least a range must have left to be stolen from
  uint32_t steal_floor_last;    // the same in the launch's last layer
  uint32_t merge_inline;        // 1: the warp that completes a (sequence, KV head) merges it itself
  uint32_t shared_merges;       // 1: merges of kSharedMergeMin partials or more are published for every CTA to take
  uint32_t copy_loads_ahead;    // 16 KB loads the copy thread keeps in flight: 3 or 4 (the host sets 4)
  uint32_t copy_sms;            // 0: every CTA's copy thread takes part in the gather; else only the first copy_sms
  const void* q;                // first_layer's [nseq][Hq][128] bf16
  void* out;
  uint64_t io_layer_stride;     // bytes from one layer's q / out to the next
  const uint32_t* q_ready;      // optional: q arrives while the launch runs; layer l's rows may be read once
  uint32_t q_ready_epoch;       //   q_ready[l / q_ready_layers] >= q_ready_epoch (written after the rows themselves)
  uint32_t q_ready_layers;
  uint32_t* out_ready;          // optional: out_ready[l] = out_ready_epoch once every row of layer l's output is written
  uint32_t out_ready_epoch;
  float* lse;                   // [nseq][Hq] or NULL (single-layer launches only)
  float* part_o;                // [slots][Hq][128] unnormalised partial outputs; layers alternate
  float* part_ml;               // [slots][Hq][4]   between part_buffers such buffers (stride below)
  uint64_t part_o_stride, part_ml_stride;  // floats between the buffers (0: single layer)
  uint32_t part_buffers;        // buffers the layers of a launch take turns with (1, 2 or 4)
  uint32_t* counters;           // first_layer's layer_counter_words(), all zeroed before the launch
  uint64_t counters_stride;     // words from one layer's counters to the next
  uint32_t nseq, ncta;
  uint32_t Hq, Hkv, G;
  float scale_log2;             // sm_scale * log2(e)
  // Gather issued while layer first_layer + i is attended to: target layer (or -1), and the layer of
  // this launch whose attention must be complete before the target's ring slot may be overwritten
  // (-1: ordered by the stream already).
  const uint8_t* lent_base;     // lent arena (same addressing as the local one)
  uint64_t lent_group_stride, lent_layer_stride, lent_block_stride;
  const int32_t* copy_src;      // lent entries (~physical index) by staging position
  const uint32_t* copy_order;   // [copy_n] copy units in the order they are gathered: first staging position
                                //   (low 24 bits) and blocks - 1 (high 8 bits) of a run of blocks that
                                //   are neighbours in the lent arena and in the slot
  uint32_t copy_n;
  uint32_t writeback;           // swap-out pass (0 when wb_n is 0): while layer l >= writeback_from is attended to,
  uint32_t writeback_from;      //   the copy threads also write the units wb_order[0 .. wb_n) back from its ring
  const uint32_t* wb_order;     //   slot to the lent arena (units as in copy_order: all of them, or only the
  uint32_t wb_n;                //   blocks that can have changed), and a slot is refilled only after the
                                //   write-back of the layer it held
  uint32_t* ready;              // [ring_slots][ready_stride] per staged position: epoch of the layer
  uint32_t ready_stride;        //   whose block has landed there (multi-layer launches)
  uint32_t epoch_base;          // epoch of first_layer; layer l has epoch_base + (l - first_layer)
  int16_t gather_target[kMaxStepLayers];
  int16_t gather_after[kMaxStepLayers];
  int* status;
  unsigned long long* trace;    // optional, per layer [ncta][kTraceWords]
  uint64_t trace_stride;        // words from one layer's trace to the next
};

// Shared memory the layer kernel needs for Hkv KV heads (0 if unsupported).
size_t layer_smem_bytes(uint32_t Hkv);
// One-time per-process opt-in to large dynamic shared memory.
cudaError_t layer_setup();
// Attention (+ fused gather, + merges) of the layers [li_begin, li_end) of p: ONE launch. A launch
// that spans several layers contains bounded waits between its CTAs and is therefore launched
// cooperatively (all CTAs resident); a link of a chain spans one layer and waits only for CTAs of
// earlier links, which have all started before its first CTA does.
cudaError_t launch_layer(const LayerParams& p, cudaStream_t stream);

// A one-thread kernel that releases q_ready[l + 1] as soon as out_ready[l] shows `epoch` (and
// q_ready[0] at once): the rest of a decoder, taking no time (measurements and tests).
cudaError_t launch_step_relay(const uint32_t* out_ready, uint32_t* q_ready, uint32_t layers, uint32_t epoch, int* status,
                              cudaStream_t stream);

// noalloc.cu: the same launch with partials and counters in a static device array (part_o,
// part_ml, counters of p are ignored). static_scratch_needed() > static_scratch_bytes() must be
// rejected by the caller.
// static_scratch_setup(): initialisation-time set-up on the current device (module load = the
// array's reservation, address look-up, one empty launch of the kernel variant for G).
size_t static_scratch_bytes();
cudaError_t static_scratch_setup(uint32_t Hkv, uint32_t G, uint32_t ncta);
size_t static_scratch_needed(uint32_t slots, uint32_t Hq, uint32_t nseq, uint32_t Hkv, uint32_t ncta);
cudaError_t launch_layer_static(LayerParams p, uint32_t slots, cudaStream_t stream);

struct AppendParams {
  uint8_t* local_base;         // arenas; layer first_layer + y of the launch at layer_offset(...) from there
  uint64_t local_block_stride;
  uint8_t* lent_base;
  uint64_t lent_block_stride;
  uint32_t layer_group;
  uint64_t local_group_stride, lent_group_stride;
  uint32_t staged_only;        // 1: a row whose block is staged goes to the staged copy only (it is written back later)
  uint32_t split_layer;        // layers from here on have their home in the lent arena, at the id the entry names
                               //   (0xFFFFFFFF: no split; the entry's sign names the arena)
  uint8_t* slot_base;          // one layer: ring slot holding the layer, or NULL when not staged
  // several layers in one launch (grid.y = layer): strides to the next layer, and which layers are staged
  uint32_t num_layers, first_layer, ring_slots;
  uint64_t local_layer_stride, lent_layer_stride, io_layer_stride, slot_bytes;
  uint8_t* staging_base;
  uint32_t staged_mask[4];     // bit l: layer first_layer + l is validly staged for this batch
  uint64_t block_bytes;
  const int32_t* home_entry;   // [nseq] entry (physical index) of the block holding token len-1
  const int32_t* stage_pos;    // [nseq] staging position of that block, or -1
  const uint32_t* lens;        // [nseq]
  const void* k_new;           // [nseq][Hkv][128] bf16
  const void* v_new;
  uint32_t nseq;
  uint32_t row_bytes;          // Hkv * 128 * 2
  uint32_t block_tokens;
};
cudaError_t launch_append(const AppendParams& p, cudaStream_t stream);

}  // namespace ema
