// slice.cpp — host side of libemaslice: the slice arena allocator (block tables, free lists,
// local/lent split), batch plans (resolved tables, copy lists, attention work items), the layer
// pipeline (fused: attention of layer l and gather of layer l+1 in one launch; or two streams with
// events), the reclaim planner, and the C ABI declared in include/emaslice.h.
#include "../../include/emaslice.h"
#include "kernels.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <limits>
#include <new>
#include <unordered_map>
#include <vector>

namespace {

constexpr int kNumPlans = 4;
constexpr int kMaxGuards = 4;
constexpr uint32_t kBlockTokens = 16;
constexpr uint32_t kHeadDim = 128;
constexpr uint32_t kTraceCopyCtas = 2048;
constexpr uint32_t kStealMin = 2;  // smallest unclipped steal, in blocks (must match the kernel)
constexpr uint32_t kStealFloorMin = 4;  // default steal floor: a third of a range, at least this
constexpr uint32_t kStealFloorLast = 8; // default steal floor in the last layer of a launch
constexpr uint32_t kInlineMergePer = 48; // ranges up to this many blocks: consumer warps merge in line
constexpr uint32_t kSlowLinkCopySms = 8;  // copy threads that take part in the gather over a slow link
constexpr uint32_t kMinPer = 8;           // least blocks per CTA range: fewer CTAs rather than more partials
constexpr uint32_t kOwnChunk = 16;  // most blocks a CTA claims from its own range at a time

struct Seq {
  std::vector<int32_t> table;
  uint32_t len = 0;
};

struct Owner {
  int32_t seq = -1;
  int32_t logical = -1;
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// A batch plan: everything about a batch that does not depend on the layer.
struct Plan {
  bool valid = false;
  uint64_t serial = 0;   // unique id of this plan
  uint64_t version = 0;  // table version it was built from
  std::vector<int32_t> seqs;
  uint32_t nseq = 0, total_blocks = 0, k = 0;
  uint32_t units = 0;                    // copy units of the fused gather (runs of neighbouring staged blocks)
  uint32_t tail_units = 0;               // staged tail blocks of the batch (the only staged blocks an append changes)
  uint32_t per = 1, used_cta = 0;        // attention ranges: range c = [c*per, min((c+1)*per, total))
  uint32_t slots = 0, slots_static = 0;  // partial slots with / without work stealing
  uint64_t tokens = 0;
  // byte offsets inside the plan buffer
  size_t off_resolved = 0, off_blk_seq = 0, off_lens = 0, off_copy_src = 0, off_copy_order = 0, off_blk_off = 0, off_slot_base = 0,
         off_slot_base_static = 0, off_home = 0, off_stage_pos = 0, off_tail_order = 0, off_tail_dst = 0, bytes = 0;
  std::vector<uint32_t> blk_off;  // host copy for the test hook
  std::vector<int32_t> resolved_ids;  // resolved table in block ids (the device copy holds physical indices)
  uint8_t* host = nullptr;        // pinned (plain memory in tables-only mode)
  uint8_t* dev = nullptr;
  size_t cap = 0;
  bool uploaded = false;
  cudaEvent_t ev_uploaded = nullptr;
  cudaStream_t upload_stream = nullptr;
  // Guards of the device buffer: recorded on every known stream when the plan can no longer be
  // used; the next upload into the buffer waits for them.
  cudaEvent_t guard[kMaxGuards] = {};
  int n_guard = 0;
  bool guarded = true;
};

struct SlotState {
  bool valid = false;
  uint32_t layer = 0;
  uint64_t plan_serial = 0;
  bool pref_recorded = false, attn_recorded = false, wb_recorded = false;
  cudaStream_t pref_stream = nullptr, attn_stream = nullptr, wb_stream = nullptr;
  cudaEvent_t pref_done = nullptr, attn_done = nullptr;
  cudaEvent_t wb_done = nullptr;  // swap-out passes: the slot's last write-back to the lent arena
};

struct StreamEpoch {
  cudaStream_t stream;
  uint64_t epoch;
};

}  // namespace

struct ema_slice {
  slice_config_t cfg{};
  bool null_dev = false, profile = false, trace = false;
  uint64_t block_bytes = 0;
  uint64_t local_ls = 0, local_bs = 0, lent_ls = 0, lent_bs = 0, slot_bytes = 0;
  // Layout of the arenas (Section 4.2): layers in groups of `group` (layer l of an arena starts at
  // (l / group) * gs + (l % group) * ls), block ids in slabs of `slab` (physical index of id b within
  // a layer: (b / slab) * W + b % slab; W = slab for the layer-major order, where it equals b).
  uint32_t group = 1, slab = 0, layout = 0;
  uint64_t local_gs = 0, lent_gs = 0;
  uint32_t local_W = 0, lent_W = 0;
  uint32_t layer_slots = 1;  // ring slots in layers: ring_slots groups of `group` layers
  // Layer-split placement (Section 4.1): layers [0, split) of every block live in the local arena,
  // layers [split, L) in the lent arena under the same block id; 0 = blocks are split instead.
  uint32_t split = 0;
  std::vector<uint32_t> slab_used_local, slab_used_lent;  // blocks in use per slab (slab allocator)
  int device = -1;  // the CUDA device the slice was created on
  int num_sms = 148;
  uint32_t ncta = 148;
  bool steal = true;
  size_t cnt_stride = 0;  // uint32 words of device counters per layer
  // allocator
  std::vector<int32_t> free_local, free_lent;  // back() pops next
  std::unordered_map<int32_t, Seq> seqs;
  std::vector<Owner> owner_local, owner_lent;
  uint32_t lent_cap = 0;
  uint64_t version = 1;
  // preemption control: caller's clock, window T, the cap in force while now < cap_until
  uint64_t now = 0, preempt_window = 0, cap_until = 0;
  uint32_t cap_level = 0;
  uint64_t preempt_oom = 0, preempt_reclaim = 0;
  uint32_t peer_used = 0;  // blocks the peer holds in this slice, as last reported
  // plans and slots
  Plan plans[kNumPlans];
  int next_plan = 0;
  uint64_t plan_serial = 0;
  std::vector<SlotState> slots;
  // device scratch
  float* part_o = nullptr;
  float* part_ml = nullptr;
  size_t part_rows = 0;         // partial rows (segments * query heads) currently allocated
  uint32_t* cnt_dev = nullptr;  // [num_layers][cnt_stride] device counters of the layer kernel
  uint32_t* ready_dev = nullptr;  // [ring_slots][staging_blocks_per_slot] ready flags (epochs)
  uint32_t epoch = 1;
  int* dev_status = nullptr;  // mapped pinned host word: kernels record a failed bounded wait, the host reads it
  // reclaim
  int32_t* reclaim_host = nullptr;
  int32_t* reclaim_dev = nullptr;
  cudaEvent_t reclaim_done = nullptr;
  bool reclaim_recorded = false;
  uint64_t reclaim_epoch = 0;
  std::vector<StreamEpoch> streams;
  cudaEvent_t append_done = nullptr;
  bool append_pending = false;
  bool in_pass = false;  // a write-back is being enqueued by slice_decode_step, not by slice_writeback_layer
  cudaStream_t append_stream = nullptr;
  cudaEvent_t ev_tmp = nullptr;
  // host io staging for slice_decode_step
  void* io_q = nullptr;
  void* io_out = nullptr;
  size_t io_bytes = 0;
  // q streamed in behind a running pass: copy stream, per-chunk arrival flags, their epoch (pinned
  // host word the flag copies read), and the event after which io_q may be overwritten.
  cudaStream_t io_stream = nullptr;
  cudaStream_t swap_stream = nullptr;  // swap-out passes: the write-backs run here, beside gather and attention
  uint32_t* q_flags_dev = nullptr;
  uint32_t* q_epoch_host = nullptr;
  uint32_t q_epoch = 0;
  cudaEvent_t io_q_free = nullptr;
  bool io_q_busy = false;
  const uint32_t* step_q_ready = nullptr;  // set for the pass being enqueued
  uint32_t step_q_layers = 0;
  // layer-dependent passes (slice_step_begin): out_flags_dev[l] = epoch once layer l's output is complete
  uint32_t* out_flags_dev = nullptr;
  uint32_t* step_out_ready = nullptr;      // set for the pass being enqueued
  // After the launch of a layer-dependent pass, in stream order, every out-ready word is set once
  // more from pinned host memory: whatever happened inside the kernel (a bounded wait that ran out),
  // a caller's stream that waits for an output is released when the launch has ended.
  static constexpr int kFillSlots = 8;
  uint32_t* out_fill_host = nullptr;       // [kFillSlots][kMaxStepLayers]
  cudaEvent_t fill_done[kFillSlots] = {};
  bool fill_busy[kFillSlots] = {};
  bool dependent_pass = false;             // a pass begun by slice_step_begin is the most recent one
  // profiling
  std::vector<cudaEvent_t> prof;  // [layer][5]
  std::vector<uint8_t> prof_set;
  cudaEvent_t prof_base = nullptr;
  bool prof_base_set = false;
  unsigned long long* trace_layer = nullptr;  // [layer][ncta][kTraceWords]
  unsigned long long* trace_copy = nullptr;   // [layer][kTraceCopyCtas][2]
  slice_stats_t st{};
};

namespace {

#define CU(s, call)                                    \
  do {                                                 \
    cudaError_t e__ = (call);                          \
    if (e__ != cudaSuccess) {                          \
      (s)->st.last_cuda_error = static_cast<int>(e__); \
      return SLICE_ECUDA;                              \
    }                                                  \
  } while (0)

inline uint32_t blocks_for(uint32_t len) { return (len + kBlockTokens - 1) / kBlockTokens; }

inline bool multi_stream(const ema_slice* s) { return s->streams.size() > 1; }

inline uint64_t local_off(const ema_slice* s, uint32_t l) { return ema::layer_offset(l, s->group, s->local_gs, s->local_ls); }
// With the layer split the lent arena holds layers split .. L-1 only (layer-major, so the offset is linear).
inline uint64_t lent_off(const ema_slice* s, uint32_t l) { return ema::layer_offset(l - s->split, s->group, s->lent_gs, s->lent_ls); }

// Does `layer` read from its ring slot for this batch?
inline bool needs_staging(const ema_slice* s, uint32_t layer, uint32_t k) { return k > 0 && (!s->split || layer >= s->split); }

// Table entry -> what the kernels index with: the block's physical index inside a layer of its
// arena (the id itself in the layer-major order), lent entries staying negative (~index).
inline int32_t phys_entry(const ema_slice* s, int32_t e) {
  if (!s->layout) return e;
  const uint32_t id = e >= 0 ? static_cast<uint32_t>(e) : static_cast<uint32_t>(~e);
  const uint32_t W = e >= 0 ? s->local_W : s->lent_W;
  const int32_t ph = static_cast<int32_t>(id / s->slab * W + id % s->slab);
  return e >= 0 ? ph : ~ph;
}

// Slab allocator (Section 4.2.1): the next id of a part of the slice among the ids below `cap` that
// are neither in use nor marked in `taken`: the lowest one lying in a slab of which `used` says
// that it holds blocks already (the user fills the slabs it has), else the lowest one of all (it
// opens the lowest free slab). -1 when there is none. `used` counts blocks per slab, those marked
// taken included.
int32_t slab_choose(const std::vector<Owner>& own, const std::vector<uint32_t>& used, const std::vector<char>* taken,
                    uint32_t S, uint32_t cap) {
  const uint32_t nslabs = (cap + S - 1) / S;
  int32_t fresh = -1;
  for (uint32_t sl = 0; sl < nslabs; ++sl) {
    const uint32_t first = sl * S, avail = std::min(S, cap - first);
    if (used[sl] >= S) continue;                // full
    if (used[sl] == 0) {                        // a free slab: remembered, taken only if no slab in use has room
      if (fresh < 0) fresh = static_cast<int32_t>(first);
      continue;
    }
    // In use (possibly only by ids at or above cap, which count but cannot be handed out).
    for (uint32_t id = first; id < first + avail; ++id)
      if (own[id].seq < 0 && !(taken && (*taken)[id])) return static_cast<int32_t>(id);
  }
  return fresh;
}

void recount_slabs(ema_slice* s) {
  if (!s->slab) return;
  std::fill(s->slab_used_local.begin(), s->slab_used_local.end(), 0u);
  std::fill(s->slab_used_lent.begin(), s->slab_used_lent.end(), 0u);
  for (size_t id = 0; id < s->owner_local.size(); ++id) s->slab_used_local[id / s->slab] += s->owner_local[id].seq >= 0;
  for (size_t id = 0; id < s->owner_lent.size(); ++id) s->slab_used_lent[id / s->slab] += s->owner_lent[id].seq >= 0;
}

// Takes the next free id of a tier: the top of the free stack, or the slab rule's choice.
int32_t take_free(ema_slice* s, bool local) {
  std::vector<int32_t>& stack = local ? s->free_local : s->free_lent;
  if (!s->slab) {
    const int32_t id = stack.back();
    stack.pop_back();
    return id;
  }
  const int32_t id = slab_choose(local ? s->owner_local : s->owner_lent, local ? s->slab_used_local : s->slab_used_lent,
                                 nullptr, s->slab, local ? s->cfg.local_blocks : s->lent_cap);
  stack.erase(std::find(stack.begin(), stack.end(), id));
  return id;
}

// Blocks the user holds in both parts of the slice.
inline uint32_t blocks_held(const ema_slice* s) {
  return static_cast<uint32_t>(s->cfg.local_blocks - s->free_local.size() + s->lent_cap - s->free_lent.size());
}

inline bool cap_in_force(const ema_slice* s) { return s->preempt_window != 0 && s->now < s->cap_until; }

// Bursty-workload control: a preemption by reclamation above the static share (the local part)
// limits the user to the level it fell to; inside the window the level only goes down, and every
// such preemption restarts the window.
inline void cap_after_reclaim_preemption(ema_slice* s, uint32_t held_before) {
  if (s->preempt_window == 0 || held_before <= s->cfg.local_blocks) return;
  const uint32_t level = blocks_held(s);
  s->cap_level = cap_in_force(s) ? std::min(s->cap_level, level) : level;
  s->cap_until = s->now + s->preempt_window;
}

// Registers a stream with the slice. A stream seen for the first time waits for everything the
// slice has enqueued on the streams it already knows (from then on per-operation events order the
// streams); every stream waits once for the latest reclaim.
int ensure_stream(ema_slice* s, cudaStream_t stream) {
  if (s->null_dev) return SLICE_OK;
  for (auto& se : s->streams) {
    if (se.stream == stream) {
      if (se.epoch < s->reclaim_epoch) {
        CU(s, cudaStreamWaitEvent(stream, s->reclaim_done, 0));
        se.epoch = s->reclaim_epoch;
      }
      return SLICE_OK;
    }
  }
  for (auto& se : s->streams) {
    CU(s, cudaEventRecord(s->ev_tmp, se.stream));
    CU(s, cudaStreamWaitEvent(stream, s->ev_tmp, 0));
  }
  if (s->reclaim_recorded) CU(s, cudaStreamWaitEvent(stream, s->reclaim_done, 0));
  s->streams.push_back(StreamEpoch{stream, s->reclaim_epoch});
  return SLICE_OK;
}

size_t plan_capacity(const ema_slice* s) {
  const slice_config_t& c = s->cfg;
  size_t b = 0;
  b += 2 * align_up(static_cast<size_t>(c.max_seqs) * c.max_blocks_per_seq * 4, 256);  // resolved, blk_seq (upper bound)
  b += align_up(static_cast<size_t>(c.max_seqs) * 4, 256);                              // lens
  b += 2 * align_up(static_cast<size_t>(c.staging_blocks_per_slot) * 4, 256);           // copy_src, copy_order
  b += 3 * align_up((static_cast<size_t>(c.max_seqs) + 1) * 4, 256);                    // blk_off, slot bases
  b += 4 * align_up(static_cast<size_t>(c.max_seqs) * 4, 256);                          // home, stage_pos, staged tail blocks (positions, homes)
  return b;
}

// Validates a batch: known, distinct sequences. Returns OK or the error.
int check_batch(ema_slice* s, const int32_t* seqs, uint32_t nseq) {
  if (nseq == 0 || nseq > s->cfg.max_seqs) return SLICE_EINVAL;
  for (uint32_t i = 0; i < nseq; ++i)
    if (s->seqs.find(seqs[i]) == s->seqs.end()) return SLICE_ESTATE;
  if (nseq > 1) {
    std::vector<int32_t> tmp(seqs, seqs + nseq);
    std::sort(tmp.begin(), tmp.end());
    if (std::adjacent_find(tmp.begin(), tmp.end()) != tmp.end()) return SLICE_EINVAL;
  }
  return SLICE_OK;
}

// Records the guards of a plan's device buffer on every known stream: all uses of the plan have
// been enqueued by now, so a later upload into the buffer only has to wait for these events.
int guard_plan(ema_slice* s, Plan& p) {
  if (s->null_dev || p.guarded) return SLICE_OK;
  p.n_guard = 0;
  if (s->streams.size() > static_cast<size_t>(kMaxGuards)) {
    CU(s, cudaDeviceSynchronize());
  } else {
    for (auto& se : s->streams) {
      CU(s, cudaEventRecord(p.guard[p.n_guard], se.stream));
      ++p.n_guard;
    }
  }
  p.guarded = true;
  return SLICE_OK;
}

// Finds or builds the plan of a batch for the current table version.
int get_plan(ema_slice* s, const int32_t* seqs, uint32_t nseq, Plan** out) {
  if (!seqs || nseq == 0) return SLICE_EINVAL;
  for (Plan& p : s->plans) {
    if (p.valid && p.version == s->version && p.nseq == nseq &&
        std::memcmp(p.seqs.data(), seqs, nseq * sizeof(int32_t)) == 0) {
      *out = &p;
      return SLICE_OK;
    }
  }
  int rc = check_batch(s, seqs, nseq);
  if (rc != SLICE_OK) return rc;
  // Size the batch before touching a plan buffer.
  uint64_t total_blocks = 0, k = 0, tokens = 0;
  for (uint32_t i = 0; i < nseq; ++i) {
    const Seq& q = s->seqs[seqs[i]];
    const uint32_t nb = blocks_for(q.len);
    total_blocks += nb;
    tokens += q.len;
    for (uint32_t b = 0; b < nb; ++b)
      if (q.table[b] < 0) ++k;
  }
  if (s->split) k = total_blocks;  // layer split: the layers of the lent half stage every block
  if (k > s->cfg.staging_blocks_per_slot) return SLICE_ESTAGING;

  // Plans of older table versions can never be used again: guard their buffers now.
  for (Plan& old : s->plans)
    if (old.valid && old.version != s->version) {
      rc = guard_plan(s, old);
      if (rc) return rc;
      old.valid = false;
    }
  Plan& p = s->plans[s->next_plan];
  s->next_plan = (s->next_plan + 1) % kNumPlans;
  rc = guard_plan(s, p);  // still current (same version, other batch): guard at recycling time
  if (rc) return rc;
  if (!s->null_dev && p.uploaded) CU(s, cudaEventSynchronize(p.ev_uploaded));  // host buffer is free again
  p.valid = false;
  p.serial = ++s->plan_serial;
  p.version = s->version;
  p.seqs.assign(seqs, seqs + nseq);
  p.nseq = nseq;
  p.total_blocks = static_cast<uint32_t>(total_blocks);
  p.k = static_cast<uint32_t>(k);
  p.tokens = tokens;
  p.uploaded = false;

  // Attention work: the flat block list (batch order) is cut into one contiguous range per CTA.
  // Inside the kernel a CTA claims blocks from the front of its range and, once that is used up,
  // steals from the back of other ranges; a run of claims within one sequence yields one partial.
  // Partial slots per sequence are sized for the worst case: every steal takes at least kStealMin
  // blocks, except one clipped steal and one clipped owner claim per range.
  const uint32_t ncta = s->ncta;
  const uint32_t total = p.total_blocks;
  uint32_t per = std::max((total + ncta - 1) / ncta, kMinPer);
  p.per = per;
  p.used_cta = (total + per - 1) / per;

  size_t off = 0;
  p.off_resolved = off;
  off += align_up(static_cast<size_t>(total) * 4, 256);
  p.off_blk_seq = off;
  off += align_up(static_cast<size_t>(total) * 4, 256);
  p.off_lens = off;
  off += align_up(static_cast<size_t>(nseq) * 4, 256);
  p.off_copy_src = off;
  off += align_up(static_cast<size_t>(k) * 4, 256);
  p.off_copy_order = off;
  off += align_up(static_cast<size_t>(k) * 4, 256);
  p.off_blk_off = off;
  off += align_up((static_cast<size_t>(nseq) + 1) * 4, 256);
  p.off_slot_base = off;
  off += align_up((static_cast<size_t>(nseq) + 1) * 4, 256);
  p.off_slot_base_static = off;
  off += align_up((static_cast<size_t>(nseq) + 1) * 4, 256);
  p.off_home = off;
  off += align_up(static_cast<size_t>(nseq) * 4, 256);
  p.off_stage_pos = off;
  off += align_up(static_cast<size_t>(nseq) * 4, 256);
  p.off_tail_order = off;
  off += align_up(static_cast<size_t>(nseq) * 4, 256);
  p.off_tail_dst = off;
  off += align_up(static_cast<size_t>(nseq) * 4, 256);
  p.bytes = off;
  if (off > p.cap) return SLICE_EINVAL;  // cannot happen: capacity is sized from the maxima

  int32_t* resolved = reinterpret_cast<int32_t*>(p.host + p.off_resolved);
  uint32_t* blk_seq = reinterpret_cast<uint32_t*>(p.host + p.off_blk_seq);
  uint32_t* lens = reinterpret_cast<uint32_t*>(p.host + p.off_lens);
  int32_t* copy_src = reinterpret_cast<int32_t*>(p.host + p.off_copy_src);
  uint32_t* copy_order = reinterpret_cast<uint32_t*>(p.host + p.off_copy_order);
  uint32_t* blk_off = reinterpret_cast<uint32_t*>(p.host + p.off_blk_off);
  std::vector<uint32_t> pos_range(k), pos_rank(k), range_staged(p.used_cta + 1, 0);
  uint32_t* slot_base = reinterpret_cast<uint32_t*>(p.host + p.off_slot_base);
  uint32_t* slot_base_static = reinterpret_cast<uint32_t*>(p.host + p.off_slot_base_static);
  int32_t* home = reinterpret_cast<int32_t*>(p.host + p.off_home);
  int32_t* stage_pos = reinterpret_cast<int32_t*>(p.host + p.off_stage_pos);

  p.blk_off.resize(nseq + 1);
  p.resolved_ids.resize(total);
  uint32_t flat = 0, kk = 0, slots = 0, slots_static = 0;
  for (uint32_t i = 0; i < nseq; ++i) {
    const Seq& q = s->seqs[seqs[i]];
    const uint32_t nb = blocks_for(q.len);
    p.blk_off[i] = blk_off[i] = flat;
    lens[i] = q.len;
    slot_base[i] = slots;
    slot_base_static[i] = slots_static;
    if (nb) {
      const uint32_t ranges = (flat + nb - 1) / per - flat / per + 1;
      slots += nb / kStealMin + 2 * ranges + 2;
      slots_static += ranges + 1;
    }
    home[i] = 0;
    stage_pos[i] = -1;
    const uint32_t last_b = q.len ? (q.len - 1) / kBlockTokens : 0;
    for (uint32_t b = 0; b < nb; ++b) {
      const int32_t e = q.table[b];
      int32_t r = phys_entry(s, e);
      p.resolved_ids[flat] = e;
      if (s->split) {
        // Layer split: the resolved table serves the local half; for the lent half the kernel reads
        // block `flat` at staging position `flat`, and the gather brings it there from the same id.
        copy_src[kk] = ~e;
        pos_range[kk] = flat / per;
        pos_rank[kk] = range_staged[flat / per]++;
        ++kk;
      } else if (e < 0) {
        copy_src[kk] = r;  // negative entry: tier 1 (lent arena), physical index ~r
        r = ~static_cast<int32_t>(kk);
        p.resolved_ids[flat] = r;
        pos_range[kk] = flat / per;
        pos_rank[kk] = range_staged[flat / per]++;
        ++kk;
      }
      resolved[flat] = r;
      blk_seq[flat] = i;
      if (b == last_b) {
        home[i] = phys_entry(s, e);
        stage_pos[i] = s->split ? static_cast<int32_t>(flat) : e < 0 ? ~r : -1;
      }
      ++flat;
    }
  }
  p.blk_off[nseq] = blk_off[nseq] = flat;
  slot_base[nseq] = slots;
  slot_base_static[nseq] = slots_static;
  p.slots = std::max(slots, 1u);
  p.slots_static = std::max(slots_static, 1u);
  // Order in which the fused kernel gathers the staged positions: the first staged block of every
  // CTA range, then the second of every range, ... A CTA reads its range front to back, so what it
  // needs first lands first and what lands last is needed last.
  // Blocks smaller than 64 KB (fewer KV heads) are gathered several at a time where they are
  // neighbours both in the lent arena and in the slot, which the slab allocator brings about
  // (Section 4.2: transfers in large pieces): a unit is such a run within one CTA range, at most
  // 64 KB and 8 blocks. With 64 KB blocks every unit is one block.
  {
    const uint32_t max_n = s->lent_bs == s->block_bytes ? static_cast<uint32_t>(std::min<uint64_t>(8, std::max<uint64_t>(1, 65536 / s->block_bytes))) : 1u;
    std::vector<uint32_t> unit_first, unit_len;
    for (uint32_t j = 0; j < kk; ++j) {
      const bool joins = j > 0 && unit_len.back() < max_n && pos_range[j] == pos_range[j - 1] &&
                         ~copy_src[j] == ~copy_src[j - 1] + 1;
      if (joins) {
        ++unit_len.back();
      } else {
        unit_first.push_back(j);
        unit_len.push_back(1);
      }
    }
    p.units = static_cast<uint32_t>(unit_first.size());
    uint32_t max_rank = 0;
    for (uint32_t c = 0; c < p.used_cta; ++c) max_rank = std::max(max_rank, range_staged[c]);
    std::vector<uint32_t> start(max_rank + 1, 0);
    for (uint32_t u = 0; u < p.units; ++u) ++start[pos_rank[unit_first[u]] + 1];
    for (uint32_t r = 0; r < max_rank; ++r) start[r + 1] += start[r];
    for (uint32_t u = 0; u < p.units; ++u)  // positions ascend within a rank
      copy_order[start[pos_rank[unit_first[u]]]++] = unit_first[u] | ((unit_len[u] - 1) << 24);
  }
  // The staged tail blocks, as copy units of one block each: what a swap-out pass that writes back
  // only what can have changed has to move (rows are appended to tail blocks and nowhere else).
  {
    uint32_t* tail_order = reinterpret_cast<uint32_t*>(p.host + p.off_tail_order);
    int32_t* tail_dst = reinterpret_cast<int32_t*>(p.host + p.off_tail_dst);  // their homes, for the stand-alone copy kernel
    p.tail_units = 0;
    for (uint32_t i = 0; i < nseq; ++i)
      if (stage_pos[i] >= 0) {
        tail_dst[p.tail_units] = copy_src[stage_pos[i]];
        tail_order[p.tail_units++] = static_cast<uint32_t>(stage_pos[i]);
      }
  }
  p.guarded = false;
  p.valid = true;
  s->st.plans_built++;
  *out = &p;
  return SLICE_OK;
}

// Uploads the plan on `stream` if nobody has yet; otherwise makes `stream` wait for the upload.
int plan_on_stream(ema_slice* s, Plan* p, cudaStream_t stream) {
  if (s->null_dev) return SLICE_OK;
  if (!p->uploaded) {
    for (int g = 0; g < p->n_guard; ++g) CU(s, cudaStreamWaitEvent(stream, p->guard[g], 0));
    p->n_guard = 0;
    CU(s, cudaMemcpyAsync(p->dev, p->host, p->bytes, cudaMemcpyHostToDevice, stream));
    CU(s, cudaEventRecord(p->ev_uploaded, stream));
    p->uploaded = true;
    p->upload_stream = stream;
  } else if (p->upload_stream != stream) {
    CU(s, cudaStreamWaitEvent(stream, p->ev_uploaded, 0));
  }
  return SLICE_OK;
}

int do_writeback(ema_slice* s, uint32_t layer, Plan* p, cudaStream_t stream);

void invalidate_staged(ema_slice* s) {
  for (auto& sl : s->slots) sl.valid = false;
}

void bump_version(ema_slice* s) { ++s->version; }

int prof_record(ema_slice* s, uint32_t layer, int which, cudaStream_t stream) {
  if (!s->profile || s->null_dev) return SLICE_OK;
  CU(s, cudaEventRecord(s->prof[layer * 5 + which], stream));
  s->prof_set[layer * 5 + which] = 1;
  return SLICE_OK;
}

bool staged(const ema_slice* s, uint32_t layer, const Plan* p) {
  const SlotState& sl = s->slots[layer % s->layer_slots];
  return sl.valid && sl.layer == layer && sl.plan_serial == p->serial;
}

// Describes the gather of `layer`'s lent blocks into its ring slot.
void fill_gather(const ema_slice* s, uint32_t layer, const Plan* p, ema::CopyDesc& d) {
  const uint32_t slot = layer % s->layer_slots;
  d = ema::CopyDesc{};
  d.src_base[0] = d.src_base[1] = static_cast<const uint8_t*>(s->cfg.lent_base) + lent_off(s, layer);
  d.src_block_stride[0] = d.src_block_stride[1] = s->lent_bs;
  d.dst_base[0] = d.dst_base[1] = static_cast<uint8_t*>(s->cfg.staging_base) + slot * s->slot_bytes;
  d.dst_block_stride[0] = d.dst_block_stride[1] = s->block_bytes;
  d.src_entry = reinterpret_cast<const int32_t*>(p->dev + p->off_copy_src);
  d.dst_entry = nullptr;
  d.n = p->k;
  d.nlayers = 1;
  d.block_bytes = s->block_bytes;
  d.status = s->dev_status;
}

// Ordering before a write into ring slot `sl` on `stream`: after the attention that last read
// it, and after the last append / write-back (which may have written the blocks to be read).
int order_before_slot_write(ema_slice* s, SlotState& sl, cudaStream_t stream) {
  if (sl.attn_recorded && sl.attn_stream != stream) CU(s, cudaStreamWaitEvent(stream, sl.attn_done, 0));
  if (s->append_pending && s->append_stream != stream) CU(s, cudaStreamWaitEvent(stream, s->append_done, 0));
  // Swap-out: the slot is refilled only when its content has been written back, and a gather of the
  // same layer later on reads the lent arena only after that write.
  if (sl.wb_recorded && sl.wb_stream != stream) CU(s, cudaStreamWaitEvent(stream, sl.wb_done, 0));
  return SLICE_OK;
}

int note_slot_written(ema_slice* s, SlotState& sl, uint32_t layer, const Plan* p, cudaStream_t stream) {
  if (!s->null_dev) {
    if (multi_stream(s)) {
      CU(s, cudaEventRecord(sl.pref_done, stream));
      sl.pref_recorded = true;
    }
    sl.pref_stream = stream;
  }
  sl.valid = true;
  sl.layer = layer;
  sl.plan_serial = p->serial;
  s->st.prefetch_calls++;
  s->st.prefetched_blocks += p->k;
  s->st.prefetched_bytes += static_cast<uint64_t>(p->k) * s->block_bytes;
  return SLICE_OK;
}

// Stand-alone gather of one layer (the copy kernel), used by prefetch_layer and to prime the ring.
int do_prefetch(ema_slice* s, uint32_t layer, Plan* p, cudaStream_t side) {
  if (s->split && layer < s->split) return SLICE_OK;  // a layer of the local half: read in place, nothing to fetch
  int rc = ensure_stream(s, side);
  if (rc) return rc;
  rc = plan_on_stream(s, p, side);
  if (rc) return rc;
  SlotState& sl = s->slots[layer % s->layer_slots];
  if (!s->null_dev) {
    rc = order_before_slot_write(s, sl, side);
    if (rc) return rc;
    rc = prof_record(s, layer, 0, side);
    if (rc) return rc;
    if (p->k) {
      ema::CopyDesc d;
      fill_gather(s, layer, p, d);
      if (s->trace_copy && (s->cfg.copy_ctas ? s->cfg.copy_ctas : s->num_sms * 8u) <= kTraceCopyCtas)
        d.trace = s->trace_copy + static_cast<size_t>(layer) * kTraceCopyCtas * 2;
      // Default: the bulk-copy ring in the form that shares an SM with an attention CTA, so that a
      // gather on a second stream runs while the attention does (the vector kernel needs no shared
      // memory, but beside the layer kernel's 352 threads there are not the registers for its CTAs:
      // the two took turns instead of overlapping).
      uint32_t kind = s->cfg.lent_kind == 1 ? ema::kCopyVector : s->cfg.copy_kind;
      if (kind == ema::kCopyDefault) kind = ema::kCopyBulkShared;
      CU(s, ema::launch_copy(d, kind, s->cfg.copy_ctas, s->num_sms, side));
      s->st.kernel_launches++;
    }
    rc = prof_record(s, layer, 1, side);
    if (rc) return rc;
  }
  return note_slot_written(s, sl, layer, p, side);
}

// Room for `buffers` partial buffers of slots * Hq rows each (a pass over all layers alternates
// between two).
int ensure_partials(ema_slice* s, uint32_t Hq, uint32_t slots, uint32_t buffers = 1) {
  // (a slot holds one partial per consumer warp of a KV head)
  const size_t rows = static_cast<size_t>(slots) * ema::partials_per_slot(s->cfg.num_kv_heads) * Hq * buffers;
  if (s->null_dev || rows <= s->part_rows) return SLICE_OK;
  if (s->part_o) {
    CU(s, cudaDeviceSynchronize());
    cudaFree(s->part_o);
    cudaFree(s->part_ml);
    s->part_o = s->part_ml = nullptr;
    s->part_rows = 0;
  }
  const size_t want = rows + rows / 4 + 64;  // head room: lengths grow from step to step
  CU(s, cudaMalloc(&s->part_o, want * kHeadDim * sizeof(float)));
  CU(s, cudaMalloc(&s->part_ml, want * 4 * sizeof(float)));
  s->part_rows = want;
  return SLICE_OK;
}

// Fields of the layer kernel's parameters that do not depend on how many layers a launch spans.
void fill_common(const ema_slice* s, const Plan* p, ema::LayerParams& d, uint32_t first_layer, uint32_t num_layers,
                 const void* q, void* out, uint32_t Hq, float sm_scale, bool steal) {
  const uint32_t Hkv = s->cfg.num_kv_heads;
  d.local_base = static_cast<const uint8_t*>(s->cfg.local_base);
  d.local_group_stride = s->local_gs;
  d.local_layer_stride = s->local_ls;
  d.local_block_stride = s->local_bs;
  d.layer_group = s->group;
  d.prefetch_distance = s->group;
  d.split_layer = s->split ? s->split : 0xFFFFFFFFu;
  d.staging_base = static_cast<const uint8_t*>(s->cfg.staging_base);
  d.slot_bytes = s->slot_bytes;
  d.ring_slots = s->layer_slots;
  d.first_layer = first_layer;
  d.num_layers = num_layers;
  d.li_begin = 0;
  d.li_end = num_layers;
  d.chained = 0;
  d.block_bytes = s->block_bytes;
  d.resolved = reinterpret_cast<const int32_t*>(p->dev + p->off_resolved);
  d.lens = reinterpret_cast<const uint32_t*>(p->dev + p->off_lens);
  d.blk_seq = reinterpret_cast<const uint32_t*>(p->dev + p->off_blk_seq);
  d.blk_off = reinterpret_cast<const uint32_t*>(p->dev + p->off_blk_off);
  // Without stealing a sequence needs one slot per range it touches: the compact layout.
  d.seq_slot_base = reinterpret_cast<const uint32_t*>(p->dev + (steal ? p->off_slot_base : p->off_slot_base_static));
  d.total_blocks = p->total_blocks;
  d.per = p->per;
  d.used_cta = p->used_cta;
  d.allow_steal = steal ? 1u : 0u;
  d.own_chunk = s->cfg.claim_blocks ? s->cfg.claim_blocks : kOwnChunk;
  d.steal_floor = s->cfg.steal_floor ? s->cfg.steal_floor : std::max(kStealFloorMin, p->per / 3);
  d.steal_floor_last = s->cfg.steal_floor ? std::min(s->cfg.steal_floor, kStealFloorLast) : kStealFloorLast;
  // A layer of a few dozen blocks per CTA lasts less than the merges of one sequence done in a row.
  d.merge_inline = p->per <= kInlineMergePer ? 1u : 0u;
  // Few, long sequences: a sequence is cut into many partials and its merges are worth sharing
  // between the CTAs (stealing adds a few partials to the count the even split gives).
  uint32_t longest = 0;
  for (uint32_t i = 0; i < p->nseq; ++i) longest = std::max(longest, p->blk_off[i + 1] - p->blk_off[i]);
  d.shared_merges = longest / p->per + 4 >= ema::kSharedMergeMin ? 1u : 0u;
  d.copy_loads_ahead = 4;  // with four partial buffers 4 loads in flight measure 2 % faster than 3
  // Lent arena behind a slow link (pinned host memory): a few copy threads saturate it.
  d.copy_sms = s->cfg.lent_kind == 1 ? (s->cfg.copy_ctas ? std::min(s->cfg.copy_ctas, s->ncta) : std::min(kSlowLinkCopySms, s->ncta)) : 0u;
  d.q = q;
  d.out = out;
  d.io_layer_stride = static_cast<uint64_t>(p->nseq) * Hq * kHeadDim * 2;
  d.lse = nullptr;
  d.part_o = s->part_o;
  d.part_ml = s->part_ml;
  d.part_o_stride = d.part_ml_stride = 0;
  d.part_buffers = 1;
  d.counters_stride = s->cnt_stride;
  d.nseq = p->nseq;
  d.ncta = s->ncta;
  d.Hq = Hq;
  d.Hkv = Hkv;
  d.G = Hq / Hkv;
  d.scale_log2 = sm_scale * 1.4426950408889634f;
  // (with the layer split the lent arena starts at layer `split`: the kernel indexes it by layer)
  d.lent_base = static_cast<const uint8_t*>(s->cfg.lent_base) - ema::layer_offset(s->split, s->group, s->lent_gs, s->lent_ls);
  d.lent_group_stride = s->lent_gs;
  d.lent_layer_stride = s->lent_ls;
  d.lent_block_stride = s->lent_bs;
  d.copy_src = reinterpret_cast<const int32_t*>(p->dev + p->off_copy_src);
  d.copy_order = reinterpret_cast<const uint32_t*>(p->dev + p->off_copy_order);
  d.copy_n = p->units;
  d.writeback = 0;
  d.writeback_from = s->split;
  d.wb_order = nullptr;
  d.wb_n = 0;
  d.ready = s->ready_dev;
  d.ready_stride = s->cfg.staging_blocks_per_slot;
  d.epoch_base = 0;
  for (uint32_t i = 0; i < ema::kMaxStepLayers; ++i) d.gather_target[i] = d.gather_after[i] = -1;
  d.status = s->dev_status;
  d.trace = s->trace_layer ? s->trace_layer + static_cast<size_t>(first_layer) * s->ncta * ema::kTraceWords : nullptr;
  d.trace_stride = static_cast<uint64_t>(s->ncta) * ema::kTraceWords;
}

// One launch of the layer kernel: attention of `layer` and, when next_layer >= 0, the gather of
// next_layer's lent blocks into its ring slot (which must differ from layer's slot).
int do_layer(ema_slice* s, uint32_t layer, Plan* p, const void* q, uint32_t Hq, float sm_scale, void* out, float* lse,
             cudaStream_t stream, int next_layer, bool static_scratch, bool counters_zeroed) {
  const uint32_t Hkv = s->cfg.num_kv_heads;
  const uint32_t R = s->layer_slots;
  if (Hq == 0 || Hq % Hkv != 0 || Hq / Hkv > 8) return SLICE_EINVAL;
  if (!s->null_dev && (!q || !out)) return SLICE_EINVAL;
  const uint32_t* lens = reinterpret_cast<const uint32_t*>(p->host + p->off_lens);
  for (uint32_t i = 0; i < p->nseq; ++i)
    if (lens[i] == 0) return SLICE_EINVAL;
  if (static_scratch) {
    if (ema::static_scratch_needed(p->slots_static * ema::partials_per_slot(Hkv), Hq, p->nseq, Hkv, s->ncta) > ema::static_scratch_bytes())
      return SLICE_ESCRATCH;
    // The array's address belongs to the device the slice lives on; with another device current the
    // launch would be given another GPU's array.
    int cur = -1;
    if (!s->null_dev && (cudaGetDevice(&cur) != cudaSuccess || cur != s->device)) return SLICE_EINVAL;
  }
  const uint32_t slot = layer % R;
  SlotState& sl = s->slots[slot];
  if (needs_staging(s, layer, p->k) && !staged(s, layer, p)) return SLICE_ESTALE;
  const bool gather = next_layer >= 0 && needs_staging(s, static_cast<uint32_t>(next_layer), p->k);
  if (next_layer >= 0 && static_cast<uint32_t>(next_layer) % R == slot) return SLICE_EINVAL;
  int rc = ensure_stream(s, stream);
  if (rc) return rc;
  if (!static_scratch) {
    rc = ensure_partials(s, Hq, p->slots);
    if (rc) return rc;
  }
  rc = plan_on_stream(s, p, stream);
  if (rc) return rc;
  SlotState* nsl = next_layer >= 0 ? &s->slots[static_cast<uint32_t>(next_layer) % R] : nullptr;
  if (!s->null_dev) {
    if (needs_staging(s, layer, p->k) && sl.pref_recorded && sl.pref_stream != stream) CU(s, cudaStreamWaitEvent(stream, sl.pref_done, 0));
    if (gather) {
      rc = order_before_slot_write(s, *nsl, stream);
      if (rc) return rc;
    }
    uint32_t* counters = s->cnt_dev + static_cast<size_t>(layer) * s->cnt_stride;
    if (!static_scratch && !counters_zeroed)
      CU(s, cudaMemsetAsync(counters, 0, s->cnt_stride * sizeof(uint32_t), stream));
    rc = prof_record(s, layer, 2, stream);
    if (rc) return rc;
    ema::LayerParams d{};
    fill_common(s, p, d, layer, 1, q, out, Hq, sm_scale, s->steal && !static_scratch);
    // A launch of one layer ends with its merges: in line, the warps that finish a sequence together
    // merge side by side instead of queueing behind the CTA's merge warp (1-2 % per layer measured).
    d.merge_inline = 1;
    d.lse = lse;
    d.counters = counters;
    d.gather_target[0] = gather ? static_cast<int16_t>(next_layer) : static_cast<int16_t>(-1);
    d.gather_after[0] = -1;  // the slot's last reader precedes this launch in stream order
    if (static_scratch)
      CU(s, ema::launch_layer_static(d, p->slots_static * ema::partials_per_slot(Hkv), stream));
    else
      CU(s, ema::launch_layer(d, stream));
    s->st.kernel_launches++;
    rc = prof_record(s, layer, 4, stream);
    if (rc) return rc;
    rc = prof_record(s, layer, 3, stream);
    if (rc) return rc;
    // The slot may be refilled once this attention has read it.
    if (multi_stream(s)) {
      CU(s, cudaEventRecord(sl.attn_done, stream));
      sl.attn_recorded = true;
    }
    sl.attn_stream = stream;
  }
  s->st.decode_calls++;
  s->st.decode_tokens += p->tokens;
  if (gather) return note_slot_written(s, *nsl, static_cast<uint32_t>(next_layer), p, stream);
  return SLICE_OK;
}

// One launch for a whole pass: attention of every layer, each overlapped with the gather of the next
// layer's lent blocks, layer boundaries soft (see layer_kernel.cu). The caller has primed layer 0.
int do_step(ema_slice* s, Plan* p, const void* q, uint32_t Hq, float sm_scale, void* out, cudaStream_t stream,
            bool wrap) {
  const uint32_t Hkv = s->cfg.num_kv_heads, L = s->cfg.num_layers, R = s->layer_slots, K = s->group;
  if (Hq == 0 || Hq % Hkv != 0 || Hq / Hkv > 8) return SLICE_EINVAL;
  if (!s->null_dev && (!q || !out)) return SLICE_EINVAL;
  const uint32_t* lens = reinterpret_cast<const uint32_t*>(p->host + p->off_lens);
  for (uint32_t i = 0; i < p->nseq; ++i)
    if (lens[i] == 0) return SLICE_EINVAL;
  // The first layer group is staged before the launch; inside it, the gather issued during layer l
  // fetches layer l + K (the same layer of the next group).
  for (uint32_t l = 0; l < std::min(K, L); ++l)
    if (needs_staging(s, l, p->k) && !staged(s, l, p)) return SLICE_ESTALE;
  // Plan the gathers by following what each ring slot will hold.
  std::vector<int64_t> holds(R, -1);
  for (uint32_t r = 0; r < R; ++r)
    if (s->slots[r].valid && s->slots[r].plan_serial == p->serial) holds[r] = s->slots[r].layer;
  int16_t target[ema::kMaxStepLayers], after[ema::kMaxStepLayers];
  uint32_t n_gathers = 0;
  for (uint32_t l = 0; l < L; ++l) {
    target[l] = after[l] = -1;
    if (!p->k) continue;
    int64_t t = -1;
    if (l + K < L) {
      t = l + K;
    } else if (wrap && L > 1) {
      // A layer of the next pass's first group, unless its slot still serves a layer of this pass.
      t = static_cast<int64_t>(l) + K - L;
      for (uint32_t j = l; j < L; ++j)
        if (j % R == t % R) t = -1;
    }
    if (t >= 0 && !needs_staging(s, static_cast<uint32_t>(t), p->k)) t = -1;  // a layer of the local half
    if (t < 0 || holds[t % R] == t) continue;  // nothing to fetch, or the slot still holds that layer
    target[l] = static_cast<int16_t>(t);
    for (int64_t j = static_cast<int64_t>(l) - 1; j >= 0; --j)
      if (j % R == t % R) {
        after[l] = static_cast<int16_t>(j);
        break;
      }
    holds[t % R] = t;
    ++n_gathers;
  }
  int rc = ensure_stream(s, stream);
  if (rc) return rc;
  // A partial buffer is reused only when the merges of the layer that used it last are done. With
  // two buffers that left them one layer's time and the start of every layer waited for the slowest
  // merge of the layer before last; with four they have three layers (measured: 4.64 -> 4.44 ms per
  // pass on the 8B shapes, small batches up to 30 % faster; 8 or 16 buffers are no faster).
  // prefetch_priority: two buffers keep the CTAs within a layer of one another, the gather is then
  // far ahead of all of them and no CTA waits for prefetched blocks (at a lower overall rate).
  const uint32_t nbuf = s->cfg.prefetch_priority ? 2u : 4u;
  rc = ensure_partials(s, Hq, p->slots, nbuf);
  if (rc) return rc;
  rc = plan_on_stream(s, p, stream);
  if (rc) return rc;
  if (!s->null_dev) {
    for (uint32_t r = 0; r < R; ++r) {
      SlotState& sl = s->slots[r];
      if (p->k && sl.pref_recorded && sl.pref_stream != stream) CU(s, cudaStreamWaitEvent(stream, sl.pref_done, 0));
      rc = order_before_slot_write(s, sl, stream);
      if (rc) return rc;
    }
    rc = prof_record(s, 0, 2, stream);  // the launch spans the pass: start of layer 0 ...
    if (rc) return rc;
    ema::LayerParams d{};
    fill_common(s, p, d, 0, L, q, out, Hq, sm_scale, s->steal);
    d.counters = s->cnt_dev;
    d.q_ready = s->step_q_ready;
    d.q_ready_epoch = s->q_epoch;
    d.q_ready_layers = s->step_q_layers ? s->step_q_layers : 1;
    d.out_ready = s->step_out_ready;
    d.out_ready_epoch = s->q_epoch;
    // A layer-dependent pass has a hard boundary after every layer, and what stands between the
    // last block of a layer and the next layer's queries is the merges. Queued to the CTA's merge
    // warp, the merges of the KV heads of a sequence run one after the other (measured: 90 us from
    // the last block to the announcement of the output); in line, the warps that finish a sequence
    // together merge side by side, and the ring they stall has nothing to stream for long anyway.
    if (s->step_out_ready) d.merge_inline = 1;
    // (Layer-dependent passes gather in the same order as the others. The reverse order — what a
    // CTA reads first lands last and is still in the L2 when the layer starts — was tried: 2 % faster
    // on the 8B shapes in some runs and 2 % slower in others, 10 % slower on the 70B shapes, where the
    // start of every layer waited 86 us for those last blocks.)
    // Swap-out pass: the write-back of every staged layer is part of the launch (the copy threads do it
    // while the layer is attended to; the gathers wait for it where they must).
    if (s->cfg.swap_out == 2) {  // only the blocks that can have changed
      d.wb_order = reinterpret_cast<const uint32_t*>(p->dev + p->off_tail_order);
      d.wb_n = p->tail_units;
    } else if (s->cfg.swap_out) {
      d.wb_order = d.copy_order;
      d.wb_n = p->units;
    }
    d.writeback = d.wb_n ? 1u : 0u;
    d.epoch_base = s->epoch;
    s->epoch += L;  // one epoch per layer of every pass: a ready flag never matches a later layer
    const size_t rows = s->part_rows / nbuf;
    d.part_o_stride = rows * kHeadDim;
    d.part_ml_stride = rows * 4;
    d.part_buffers = nbuf;
    for (uint32_t l = 0; l < L; ++l) {
      d.gather_target[l] = target[l];
      d.gather_after[l] = after[l];
    }
    if (s->cfg.pipeline_mode == 3) {
      // A chain of launches, one per layer, over the one parameter block: each link starts as soon as
      // every CTA of the link before it has started, on the SMs that link's CTAs leave, and the links
      // order themselves through the flags and counters that order the layers of a single launch.
      // Nothing else may be enqueued between two links.
      d.merge_inline = 1;  // a link's CTA leaves when its merges are done: side by side, not queued
      for (uint32_t l = 0; l < L; ++l) {
        d.li_begin = l;
        d.li_end = l + 1;
        d.chained = l == 0 ? 1u : 2u;
        CU(s, ema::launch_layer(d, stream));
        s->st.kernel_launches++;
      }
    } else {
      CU(s, ema::launch_layer(d, stream));
      s->st.kernel_launches++;
    }
    rc = prof_record(s, L - 1, 4, stream);  // ... and end of the last layer
    if (rc) return rc;
    rc = prof_record(s, L - 1, 3, stream);
    if (rc) return rc;
  }
  for (uint32_t r = 0; r < R; ++r) {
    SlotState& sl = s->slots[r];
    if (!s->null_dev) {
      if (multi_stream(s)) {
        CU(s, cudaEventRecord(sl.attn_done, stream));
        CU(s, cudaEventRecord(sl.pref_done, stream));
        sl.attn_recorded = sl.pref_recorded = true;
        if (s->cfg.swap_out) {
          CU(s, cudaEventRecord(sl.wb_done, stream));
          sl.wb_recorded = true;
        }
      }
      sl.attn_stream = sl.pref_stream = stream;
      if (s->cfg.swap_out) sl.wb_stream = stream;
    }
    if (holds[r] >= 0) {
      sl.valid = true;
      sl.layer = static_cast<uint32_t>(holds[r]);
      sl.plan_serial = p->serial;
    }
  }
  s->st.decode_calls += L;
  s->st.decode_tokens += p->tokens * L;
  s->st.prefetch_calls += n_gathers;
  s->st.prefetched_blocks += static_cast<uint64_t>(n_gathers) * p->k;
  s->st.prefetched_bytes += static_cast<uint64_t>(n_gathers) * p->k * s->block_bytes;
  return SLICE_OK;
}

void destroy_impl(ema_slice* s) {
  if (!s->null_dev) {
    cudaDeviceSynchronize();
    for (Plan& p : s->plans) {
      if (p.host) cudaFreeHost(p.host);
      if (p.dev) cudaFree(p.dev);
      if (p.ev_uploaded) cudaEventDestroy(p.ev_uploaded);
      for (auto g : p.guard)
        if (g) cudaEventDestroy(g);
    }
    for (auto& sl : s->slots) {
      if (sl.pref_done) cudaEventDestroy(sl.pref_done);
      if (sl.attn_done) cudaEventDestroy(sl.attn_done);
      if (sl.wb_done) cudaEventDestroy(sl.wb_done);
    }
    for (auto e : s->prof)
      if (e) cudaEventDestroy(e);
    if (s->prof_base) cudaEventDestroy(s->prof_base);
    if (s->trace_layer) cudaFree(s->trace_layer);
    if (s->trace_copy) cudaFree(s->trace_copy);
    if (s->part_o) cudaFree(s->part_o);
    if (s->part_ml) cudaFree(s->part_ml);
    if (s->cnt_dev) cudaFree(s->cnt_dev);
    if (s->ready_dev) cudaFree(s->ready_dev);
    if (s->dev_status) cudaFreeHost(s->dev_status);
    if (s->reclaim_host) cudaFreeHost(s->reclaim_host);
    if (s->reclaim_dev) cudaFree(s->reclaim_dev);
    if (s->reclaim_done) cudaEventDestroy(s->reclaim_done);
    if (s->append_done) cudaEventDestroy(s->append_done);
    if (s->ev_tmp) cudaEventDestroy(s->ev_tmp);
    if (s->io_q) cudaFree(s->io_q);
    if (s->io_out) cudaFree(s->io_out);
    if (s->q_flags_dev) cudaFree(s->q_flags_dev);
    if (s->out_flags_dev) cudaFree(s->out_flags_dev);
    if (s->out_fill_host) cudaFreeHost(s->out_fill_host);
    for (auto e : s->fill_done)
      if (e) cudaEventDestroy(e);
    if (s->q_epoch_host) cudaFreeHost(s->q_epoch_host);
    if (s->io_q_free) cudaEventDestroy(s->io_q_free);
    if (s->io_stream) cudaStreamDestroy(s->io_stream);
    if (s->swap_stream) cudaStreamDestroy(s->swap_stream);
  } else {
    for (Plan& p : s->plans) delete[] p.host;
  }
  delete s;
}

}  // namespace

extern "C" {

int slice_create(const slice_config_t* cfg, slice_t** out) {
  if (!cfg || !out) return SLICE_EINVAL;
  *out = nullptr;
  const bool null_dev = (cfg->flags & SLICE_FLAG_NULL_DEVICE) != 0;
  if (cfg->head_dim != kHeadDim || cfg->block_tokens != kBlockTokens || cfg->dtype != 0) return SLICE_EINVAL;
  if (cfg->num_kv_heads == 0 || cfg->num_kv_heads > 8 || cfg->num_layers == 0) return SLICE_EINVAL;
  if (cfg->ring_slots == 0 || cfg->lent_blocks > cfg->lent_blocks_physical) return SLICE_EINVAL;
  if (cfg->max_seqs == 0 || cfg->max_blocks_per_seq == 0 || cfg->lent_kind > 1 || cfg->copy_kind > 3) return SLICE_EINVAL;
  if (cfg->pipeline_mode > 3 || cfg->static_split > 1 || cfg->prefetch_priority > 1 || cfg->swap_out > 2) return SLICE_EINVAL;
  // Section 4.2: slabs, layer groups, layouts.
  const uint32_t group = cfg->layer_group ? cfg->layer_group : 1u, slab = cfg->slab_blocks;
  if (cfg->layout > 2 || group > cfg->num_layers) return SLICE_EINVAL;
  if (slab && (cfg->local_free_order || cfg->lent_free_order)) return SLICE_EINVAL;  // the slab rule fixes the order
  if (cfg->layout != 0) {
    // The slab-major and layer-group-major orders are defined over whole slabs and whole groups,
    // and exclude caller-chosen strides.
    if (!slab || cfg->local_blocks % slab || cfg->lent_blocks_physical % slab || cfg->num_layers % group) return SLICE_EINVAL;
    if (cfg->local_layer_stride || cfg->local_block_stride || cfg->lent_layer_stride || cfg->lent_block_stride)
      return SLICE_EINVAL;
  }
  if (static_cast<uint64_t>(cfg->ring_slots) * group > 4096 || cfg->staging_blocks_per_slot >= (1u << 24)) return SLICE_EINVAL;
  // Layer split: the same ids in both arenas, plain layer-major order, no block-level lending.
  if (cfg->split_layer && (cfg->split_layer >= cfg->num_layers || cfg->layout != 0 || cfg->lent_blocks_physical < cfg->local_blocks ||
                           cfg->lent_layer_stride || cfg->lent_block_stride))
    return SLICE_EINVAL;
  if (!null_dev && (!cfg->local_base || !cfg->staging_base || (cfg->lent_blocks_physical && !cfg->lent_base)))
    return SLICE_EINVAL;
  const uint64_t bb = 2ull * kBlockTokens * cfg->num_kv_heads * kHeadDim * 2;
  if (!null_dev) {
    const uintptr_t a = reinterpret_cast<uintptr_t>(cfg->local_base) | reinterpret_cast<uintptr_t>(cfg->lent_base) |
                        reinterpret_cast<uintptr_t>(cfg->staging_base);
    if (a & 255u) return SLICE_EINVAL;
  }
  const uint64_t strides[4] = {cfg->local_layer_stride, cfg->local_block_stride, cfg->lent_layer_stride,
                               cfg->lent_block_stride};
  for (uint64_t v : strides)
    if (v & 255u) return SLICE_EINVAL;
  // free orders must be permutations
  auto is_perm = [](const uint32_t* o, uint32_t n) {
    if (!o) return true;
    std::vector<uint8_t> seen(n, 0);
    for (uint32_t k = 0; k < n; ++k) {
      if (o[k] >= n || seen[o[k]]) return false;
      seen[o[k]] = 1;
    }
    return true;
  };
  if (!is_perm(cfg->local_free_order, cfg->local_blocks) || !is_perm(cfg->lent_free_order, cfg->lent_blocks_physical))
    return SLICE_EINVAL;

  ema_slice* s = new (std::nothrow) ema_slice();
  if (!s) return SLICE_EINVAL;
  s->cfg = *cfg;
  s->cfg.local_free_order = s->cfg.lent_free_order = nullptr;
  s->null_dev = null_dev;
  s->profile = (cfg->flags & SLICE_FLAG_PROFILE) != 0;
  s->trace = (cfg->flags & SLICE_FLAG_TRACE) != 0;
  s->steal = cfg->static_split == 0;
  s->block_bytes = bb;
  s->local_bs = cfg->local_block_stride ? cfg->local_block_stride : bb;
  s->local_ls = cfg->local_layer_stride ? cfg->local_layer_stride : bb * cfg->local_blocks;
  s->lent_bs = cfg->lent_block_stride ? cfg->lent_block_stride : bb;
  s->lent_ls = cfg->lent_layer_stride ? cfg->lent_layer_stride : bb * cfg->lent_blocks_physical;
  s->slot_bytes = bb * cfg->staging_blocks_per_slot;
  s->group = group;
  s->split = cfg->split_layer;
  s->slab = slab;
  s->layout = cfg->layout;
  s->layer_slots = cfg->ring_slots * group;
  if (cfg->layout == 0) {          // [layer][id]: groups are just runs of layers
    s->local_gs = group * s->local_ls;
    s->lent_gs = group * s->lent_ls;
    s->local_W = s->lent_W = slab;
  } else if (cfg->layout == 1) {   // slab-major [slab][layer][block in slab]
    s->local_ls = s->lent_ls = bb * slab;
    s->local_gs = s->lent_gs = bb * slab * group;
    s->local_W = s->lent_W = cfg->num_layers * slab;
  } else {                         // layer-group-major [group][slab][layer in group][block in slab]
    s->local_ls = s->lent_ls = bb * slab;
    s->local_gs = bb * slab * group * (cfg->local_blocks / slab);
    s->lent_gs = bb * slab * group * (cfg->lent_blocks_physical / slab);
    s->local_W = s->lent_W = group * slab;
  }
  if (slab) {
    s->slab_used_local.assign((cfg->local_blocks + slab - 1) / slab, 0u);
    s->slab_used_lent.assign((cfg->lent_blocks_physical + slab - 1) / slab, 0u);
  }
  s->lent_cap = cfg->lent_blocks;
  s->owner_local.assign(cfg->local_blocks, Owner());
  s->owner_lent.assign(cfg->lent_blocks_physical, Owner());
  for (uint32_t k = cfg->local_blocks; k-- > 0;)
    s->free_local.push_back(static_cast<int32_t>(cfg->local_free_order ? cfg->local_free_order[k] : k));
  for (uint32_t k = cfg->lent_blocks_physical; k-- > 0;) {
    const uint32_t id = cfg->lent_free_order ? cfg->lent_free_order[k] : k;
    if (id < cfg->lent_blocks) s->free_lent.push_back(static_cast<int32_t>(id));
  }
  s->slots.resize(s->layer_slots);

  auto fail = [&](int code) {
    destroy_impl(s);
    return code;
  };
  if (!null_dev) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&s->num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
      return fail(SLICE_ECUDA);
    s->device = dev;
    if (ema::layer_setup() != cudaSuccess) return fail(SLICE_ECUDA);
  }
  s->ncta = cfg->decode_ctas ? cfg->decode_ctas : static_cast<uint32_t>(s->num_sms);
  if (!null_dev) {
    // paged_decode_noalloc must find nothing left to set up when it is first called: load its module
    // (which reserves the static scratch array on this device), look the array up and run both
    // variants of the attention kernel once, empty.
    const uint32_t warm_ctas = std::min(s->ncta, static_cast<uint32_t>(s->num_sms));
    if (ema::static_scratch_setup(cfg->num_kv_heads, 1, warm_ctas) != cudaSuccess ||
        ema::static_scratch_setup(cfg->num_kv_heads, 2, warm_ctas) != cudaSuccess)
      return fail(SLICE_ECUDA);
  }
  const size_t cap = plan_capacity(s);
  for (Plan& p : s->plans) {
    p.cap = cap;
    if (null_dev) {
      p.host = new (std::nothrow) uint8_t[cap];
      if (!p.host) return fail(SLICE_EINVAL);
    } else {
      if (cudaMallocHost(reinterpret_cast<void**>(&p.host), cap) != cudaSuccess) return fail(SLICE_ECUDA);
      if (cudaMalloc(reinterpret_cast<void**>(&p.dev), cap) != cudaSuccess) return fail(SLICE_ECUDA);
      if (cudaEventCreateWithFlags(&p.ev_uploaded, cudaEventDisableTiming) != cudaSuccess) return fail(SLICE_ECUDA);
      for (auto& g : p.guard)
        if (cudaEventCreateWithFlags(&g, cudaEventDisableTiming) != cudaSuccess) return fail(SLICE_ECUDA);
    }
  }
  if (!null_dev) {
    for (auto& sl : s->slots) {
      if (cudaEventCreateWithFlags(&sl.pref_done, cudaEventDisableTiming) != cudaSuccess ||
          cudaEventCreateWithFlags(&sl.attn_done, cudaEventDisableTiming) != cudaSuccess ||
          cudaEventCreateWithFlags(&sl.wb_done, cudaEventDisableTiming) != cudaSuccess)
        return fail(SLICE_ECUDA);
    }
    if (cudaHostAlloc(reinterpret_cast<void**>(&s->dev_status), 256, cudaHostAllocMapped) != cudaSuccess) return fail(SLICE_ECUDA);
    std::memset(s->dev_status, 0, 256);
    s->cnt_stride = align_up(ema::layer_counter_words(s->ncta, cfg->max_seqs, cfg->num_kv_heads), 64);
    const size_t cnt_words = static_cast<size_t>(cfg->num_layers) * s->cnt_stride;
    if (cudaMalloc(reinterpret_cast<void**>(&s->cnt_dev), cnt_words * sizeof(uint32_t)) != cudaSuccess ||
        cudaMemset(s->cnt_dev, 0, cnt_words * sizeof(uint32_t)) != cudaSuccess)
      return fail(SLICE_ECUDA);
    const size_t rd = static_cast<size_t>(s->layer_slots) * std::max(cfg->staging_blocks_per_slot, 1u) * sizeof(uint32_t);
    if (cudaMalloc(reinterpret_cast<void**>(&s->ready_dev), rd) != cudaSuccess || cudaMemset(s->ready_dev, 0, rd) != cudaSuccess)
      return fail(SLICE_ECUDA);
    if (cudaMalloc(reinterpret_cast<void**>(&s->q_flags_dev), ema::kMaxStepLayers * sizeof(uint32_t)) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&s->out_flags_dev), ema::kMaxStepLayers * sizeof(uint32_t)) != cudaSuccess ||
        cudaMemset(s->q_flags_dev, 0, ema::kMaxStepLayers * sizeof(uint32_t)) != cudaSuccess ||
        cudaMemset(s->out_flags_dev, 0, ema::kMaxStepLayers * sizeof(uint32_t)) != cudaSuccess)
      return fail(SLICE_ECUDA);
    if (cudaMallocHost(reinterpret_cast<void**>(&s->out_fill_host),
                       ema_slice::kFillSlots * ema::kMaxStepLayers * sizeof(uint32_t)) != cudaSuccess)
      return fail(SLICE_ECUDA);
    for (auto& e : s->fill_done)
      if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return fail(SLICE_ECUDA);
    // The relay kernel is launched beside a running pass, where a kernel's first launch (which loads
    // its code) would not get through: launch it once now, over no layers.
    if (ema::launch_step_relay(s->out_flags_dev, s->q_flags_dev, 0, 0, nullptr, nullptr) != cudaSuccess ||
        cudaStreamSynchronize(nullptr) != cudaSuccess)
      return fail(SLICE_ECUDA);
    const size_t rl = static_cast<size_t>(std::max(cfg->lent_blocks_physical, 1u)) * 2 * sizeof(int32_t);
    if (cudaMallocHost(reinterpret_cast<void**>(&s->reclaim_host), rl) != cudaSuccess) return fail(SLICE_ECUDA);
    if (cudaMalloc(reinterpret_cast<void**>(&s->reclaim_dev), rl) != cudaSuccess) return fail(SLICE_ECUDA);
    if (cudaEventCreateWithFlags(&s->reclaim_done, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&s->append_done, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&s->ev_tmp, cudaEventDisableTiming) != cudaSuccess)
      return fail(SLICE_ECUDA);
    if (s->profile) {
      s->prof.assign(static_cast<size_t>(cfg->num_layers) * 5, nullptr);
      s->prof_set.assign(static_cast<size_t>(cfg->num_layers) * 5, 0);
      for (auto& e : s->prof)
        if (cudaEventCreate(&e) != cudaSuccess) return fail(SLICE_ECUDA);
      if (cudaEventCreate(&s->prof_base) != cudaSuccess) return fail(SLICE_ECUDA);
    }
    if (s->trace) {
      const size_t tl = static_cast<size_t>(cfg->num_layers) * s->ncta * ema::kTraceWords * sizeof(unsigned long long);
      const size_t tc = static_cast<size_t>(cfg->num_layers) * kTraceCopyCtas * 2 * sizeof(unsigned long long);
      if (cudaMalloc(reinterpret_cast<void**>(&s->trace_layer), tl) != cudaSuccess ||
          cudaMalloc(reinterpret_cast<void**>(&s->trace_copy), tc) != cudaSuccess ||
          cudaMemset(s->trace_layer, 0, tl) != cudaSuccess || cudaMemset(s->trace_copy, 0, tc) != cudaSuccess)
        return fail(SLICE_ECUDA);
    }
  }
  *out = s;
  return SLICE_OK;
}

int slice_destroy(slice_t* s) {
  if (!s) return SLICE_EINVAL;
  destroy_impl(s);
  return SLICE_OK;
}

int slice_alloc_blocks(slice_t* s, int32_t seq, uint32_t n, int32_t hint, int32_t* out_entries) {
  if (!s || seq < 0 || hint < SLICE_TIER_AUTO || hint > SLICE_TIER_LENT) return SLICE_EINVAL;
  if (s->split) {  // layer split: an id names a block's place in both arenas; ids come from the local list only
    if (hint == SLICE_TIER_LENT) return SLICE_EINVAL;
    hint = SLICE_TIER_LOCAL;
  }
  auto it = s->seqs.find(seq);
  const bool exists = it != s->seqs.end();
  if (!exists && s->seqs.size() >= s->cfg.max_seqs) return SLICE_EINVAL;
  const size_t have = exists ? it->second.table.size() : 0;
  if (have + n > s->cfg.max_blocks_per_seq) return SLICE_EINVAL;
  if (n > 0 && cap_in_force(s) && static_cast<uint64_t>(blocks_held(s)) + n > s->cap_level) return SLICE_ECAPPED;
  const size_t fl = s->free_local.size(), fr = s->free_lent.size();
  if (hint == SLICE_TIER_AUTO && n > fl + fr) return SLICE_ENOSPC;
  if (hint == SLICE_TIER_LOCAL && n > fl) return SLICE_ENOSPC;
  if (hint == SLICE_TIER_LENT && n > fr) return SLICE_ENOSPC;
  Seq& q = s->seqs[seq];
  for (uint32_t k = 0; k < n; ++k) {
    const bool local = hint == SLICE_TIER_LOCAL || (hint == SLICE_TIER_AUTO && !s->free_local.empty());
    const int32_t id = take_free(s, local);
    (local ? s->owner_local : s->owner_lent)[id] = Owner{seq, static_cast<int32_t>(q.table.size())};
    if (s->slab) ++(local ? s->slab_used_local : s->slab_used_lent)[id / s->slab];
    const int32_t entry = local ? id : ~id;
    q.table.push_back(entry);
    if (out_entries) out_entries[k] = entry;
  }
  bump_version(s);
  return SLICE_OK;
}

int slice_set_seq_len(slice_t* s, int32_t seq, uint32_t len) {
  if (!s) return SLICE_EINVAL;
  auto it = s->seqs.find(seq);
  if (it == s->seqs.end()) return SLICE_ESTATE;
  if (len > static_cast<uint64_t>(it->second.table.size()) * kBlockTokens) return SLICE_EINVAL;
  if (it->second.len != len) {
    it->second.len = len;
    bump_version(s);
  }
  return SLICE_OK;
}

int slice_free_seq(slice_t* s, int32_t seq) {
  if (!s) return SLICE_EINVAL;
  auto it = s->seqs.find(seq);
  if (it == s->seqs.end()) return SLICE_ESTATE;
  const std::vector<int32_t>& t = it->second.table;
  for (size_t b = t.size(); b-- > 0;) {
    const int32_t e = t[b];
    if (e >= 0) {
      s->free_local.push_back(e);
      s->owner_local[e] = Owner();
      if (s->slab) --s->slab_used_local[e / s->slab];
    } else {
      s->free_lent.push_back(~e);
      s->owner_lent[~e] = Owner();
      if (s->slab) --s->slab_used_lent[~e / s->slab];
    }
  }
  s->seqs.erase(it);
  bump_version(s);
  return SLICE_OK;
}

int slice_get_block_table(slice_t* s, int32_t seq, int32_t* out, uint32_t cap, uint32_t* n, uint32_t* len) {
  if (!s) return SLICE_EINVAL;
  auto it = s->seqs.find(seq);
  if (it == s->seqs.end()) return SLICE_ESTATE;
  const std::vector<int32_t>& t = it->second.table;
  if (n) *n = static_cast<uint32_t>(t.size());
  if (len) *len = it->second.len;
  if (out) {
    if (cap < t.size()) return SLICE_EINVAL;
    std::copy(t.begin(), t.end(), out);
  }
  return SLICE_OK;
}

int slice_get_free_stack(slice_t* s, int32_t tier, int32_t* out, uint32_t cap, uint32_t* n) {
  if (!s || (tier != SLICE_TIER_LOCAL && tier != SLICE_TIER_LENT)) return SLICE_EINVAL;
  const std::vector<int32_t>& st = tier == SLICE_TIER_LOCAL ? s->free_local : s->free_lent;
  if (n) *n = static_cast<uint32_t>(st.size());
  if (out) {
    if (cap < st.size()) return SLICE_EINVAL;
    for (size_t k = 0; k < st.size(); ++k) out[k] = st[st.size() - 1 - k];
  }
  return SLICE_OK;
}

int prefetch_layer(slice_t* s, uint32_t layer, const int32_t* seqs, uint32_t nseq, void* side_stream) {
  if (!s || layer >= s->cfg.num_layers) return SLICE_EINVAL;
  Plan* p = nullptr;
  int rc = get_plan(s, seqs, nseq, &p);
  if (rc) return rc;
  return do_prefetch(s, layer, p, static_cast<cudaStream_t>(side_stream));
}

int paged_decode(slice_t* s, uint32_t layer, const int32_t* seqs, uint32_t nseq, const void* q, uint32_t num_q_heads,
                 float sm_scale, void* out, float* lse_or_null, void* stream) {
  if (!s || layer >= s->cfg.num_layers) return SLICE_EINVAL;
  Plan* p = nullptr;
  int rc = get_plan(s, seqs, nseq, &p);
  if (rc) return rc;
  return do_layer(s, layer, p, q, num_q_heads, sm_scale, out, lse_or_null, static_cast<cudaStream_t>(stream), -1, false,
                  false);
}

int paged_decode_noalloc(slice_t* s, uint32_t layer, const int32_t* seqs, uint32_t nseq, const void* q,
                         uint32_t num_q_heads, float sm_scale, void* out, float* lse_or_null, void* stream) {
  if (!s || layer >= s->cfg.num_layers) return SLICE_EINVAL;
  Plan* p = nullptr;
  int rc = get_plan(s, seqs, nseq, &p);
  if (rc) return rc;
  return do_layer(s, layer, p, q, num_q_heads, sm_scale, out, lse_or_null, static_cast<cudaStream_t>(stream), -1, true,
                  false);
}

int slice_reclaim(slice_t* s, uint32_t take, uint64_t* out_n_migrated, void* stream_v) {
  if (!s) return SLICE_EINVAL;
  // With the layer split a request's layers sit half here, half there: nothing can migrate; the
  // lender gets memory back by preemption (slice_preempt_seq), as in Section 4.1.
  if (s->split) return SLICE_EINVAL;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  if (take > s->lent_cap) take = s->lent_cap;
  const uint32_t cut = s->lent_cap - take;
  std::vector<int32_t> victims;
  for (uint32_t id = cut; id < s->lent_cap; ++id)
    if (s->owner_lent[id].seq >= 0) victims.push_back(static_cast<int32_t>(id));
  std::vector<int32_t> below;  // free lent ids under the cut
  for (int32_t id : s->free_lent)
    if (static_cast<uint32_t>(id) < cut) below.push_back(id);
  if (victims.size() > s->free_local.size() + below.size()) return SLICE_ENOSPC;

  // Plan first: destinations in ascending victim order, local ids before lent ids.
  const size_t n_local = std::min(victims.size(), s->free_local.size());
  const size_t n_lent = victims.size() - n_local;
  std::vector<int32_t> dst(victims.size());
  if (!s->slab) {
    std::vector<int32_t> sorted_below(below);
    std::sort(sorted_below.begin(), sorted_below.end());
    for (size_t k = 0; k < n_local; ++k) dst[k] = s->free_local[s->free_local.size() - 1 - k];
    for (size_t k = 0; k < n_lent; ++k) dst[n_local + k] = ~sorted_below[k];
  } else {
    // Slab allocator: every victim goes where the next allocation would go, each choice seeing the
    // ones before it (scratch copies; nothing is committed yet).
    std::vector<uint32_t> used_l(s->slab_used_local), used_r(s->slab_used_lent);
    std::vector<char> taken_l(s->owner_local.size(), 0), taken_r(s->owner_lent.size(), 0);
    for (size_t k = 0; k < victims.size(); ++k) {
      if (k < n_local) {
        const int32_t id = slab_choose(s->owner_local, used_l, &taken_l, s->slab, s->cfg.local_blocks);
        taken_l[id] = 1;
        ++used_l[id / s->slab];
        dst[k] = id;
      } else {
        const int32_t id = slab_choose(s->owner_lent, used_r, &taken_r, s->slab, cut);
        taken_r[id] = 1;
        ++used_r[id / s->slab];
        dst[k] = ~id;
      }
      --used_r[victims[k] / s->slab];  // this victim has left its slab before the next one is placed
    }
  }

  // Test hook: the step that enqueues the migration fails, as a CUDA call might; nothing is committed.
  if ((s->cfg.flags & SLICE_FLAG_TEST_FAIL_COPY) && !victims.empty()) {
    s->st.last_cuda_error = static_cast<int>(cudaErrorUnknown);
    return SLICE_ECUDA;
  }
  if (!s->null_dev && !victims.empty()) {
    // Everything outstanding on the slice's streams must finish before blocks move.
    int rc = ensure_stream(s, stream);
    if (rc) return rc;
    if (s->reclaim_recorded) CU(s, cudaEventSynchronize(s->reclaim_done));  // list buffer reuse
    for (auto& se : s->streams) {
      if (se.stream == stream) continue;
      CU(s, cudaEventRecord(s->ev_tmp, se.stream));
      CU(s, cudaStreamWaitEvent(stream, s->ev_tmp, 0));
    }
    const size_t n = victims.size();
    for (size_t k = 0; k < n; ++k) {  // physical indices for the kernel
      s->reclaim_host[k] = phys_entry(s, ~victims[k]);
      s->reclaim_host[n + k] = phys_entry(s, dst[k]);
    }
    CU(s, cudaMemcpyAsync(s->reclaim_dev, s->reclaim_host, 2 * n * sizeof(int32_t), cudaMemcpyHostToDevice, stream));
    ema::CopyDesc d{};
    d.src_base[0] = d.src_base[1] = static_cast<const uint8_t*>(s->cfg.lent_base);
    d.src_block_stride[0] = d.src_block_stride[1] = s->lent_bs;
    d.src_layer_stride[0] = d.src_layer_stride[1] = s->lent_ls;
    d.dst_base[0] = static_cast<uint8_t*>(s->cfg.local_base);
    d.dst_block_stride[0] = s->local_bs;
    d.dst_layer_stride[0] = s->local_ls;
    d.dst_base[1] = static_cast<uint8_t*>(s->cfg.lent_base);
    d.dst_block_stride[1] = s->lent_bs;
    d.dst_layer_stride[1] = s->lent_ls;
    d.layer_group = s->group;
    d.src_group_stride[0] = d.src_group_stride[1] = d.dst_group_stride[1] = s->lent_gs;
    d.dst_group_stride[0] = s->local_gs;
    d.src_entry = s->reclaim_dev;
    d.dst_entry = s->reclaim_dev + n;
    d.n = static_cast<uint32_t>(n);
    d.nlayers = s->cfg.num_layers;
    d.block_bytes = s->block_bytes;
    d.status = s->dev_status;
    // Nothing else runs during a migration, so the ring kernel (6.4 TB/s against the vector kernel's
    // 5.9-6.0) can have the shared memory it needs on every SM.
    uint32_t kind = s->cfg.lent_kind == 1 ? ema::kCopyVector : s->cfg.copy_kind;
    if (kind == ema::kCopyDefault) kind = ema::kCopyBulk;
    CU(s, ema::launch_copy(d, kind, 0, s->num_sms, stream));
    s->st.kernel_launches++;
    CU(s, cudaEventRecord(s->reclaim_done, stream));
    s->reclaim_recorded = true;
    ++s->reclaim_epoch;
    for (auto& se : s->streams)
      if (se.stream == stream) se.epoch = s->reclaim_epoch;
  }

  // Commit the integer state.
  std::vector<int32_t> kept;
  for (int32_t id : s->free_lent)
    if (static_cast<uint32_t>(id) < cut) kept.push_back(id);
  s->free_lent.swap(kept);
  for (size_t k = 0; k < victims.size(); ++k) {
    const int32_t v = victims[k];
    const Owner own = s->owner_lent[v];
    if (k < n_local) {
      if (s->slab)
        s->free_local.erase(std::find(s->free_local.begin(), s->free_local.end(), dst[k]));
      else
        s->free_local.pop_back();
      s->owner_local[dst[k]] = own;
    } else {
      const int32_t id = ~dst[k];
      s->free_lent.erase(std::find(s->free_lent.begin(), s->free_lent.end(), id));
      s->owner_lent[id] = own;
    }
    s->seqs[own.seq].table[own.logical] = dst[k];
    s->owner_lent[v] = Owner();
  }
  recount_slabs(s);
  s->lent_cap = cut;
  bump_version(s);
  invalidate_staged(s);
  s->st.reclaims++;
  s->st.migrated_blocks += victims.size();
  s->st.migrated_bytes += static_cast<uint64_t>(victims.size()) * s->block_bytes * s->cfg.num_layers;
  if (out_n_migrated) *out_n_migrated = victims.size();
  return SLICE_OK;
}

int slice_set_preempt_window(slice_t* s, uint64_t window) {
  if (!s) return SLICE_EINVAL;
  s->preempt_window = window;
  return SLICE_OK;
}

int slice_set_time(slice_t* s, uint64_t now) {
  if (!s || now < s->now) return SLICE_EINVAL;
  s->now = now;
  return SLICE_OK;
}

int slice_preempt_seq(slice_t* s, int32_t seq, int32_t cause) {
  if (!s || (cause != SLICE_PREEMPT_OOM && cause != SLICE_PREEMPT_RECLAIM)) return SLICE_EINVAL;
  const uint32_t held = blocks_held(s);
  const int rc = slice_free_seq(s, seq);
  if (rc) return rc;
  if (cause == SLICE_PREEMPT_OOM) {
    ++s->preempt_oom;
  } else {
    ++s->preempt_reclaim;
    cap_after_reclaim_preemption(s, held);
  }
  return SLICE_OK;
}

int slice_reclaim_preempt(slice_t* s, uint32_t take, uint32_t slab_blocks, int32_t* victims, uint32_t cap,
                          uint32_t* n_victims, uint64_t* out_n_migrated, void* stream) {
  if (!s || slab_blocks == 0) return SLICE_EINVAL;
  if (take > s->lent_cap) take = s->lent_cap;
  const uint32_t cut = s->lent_cap - take;
  // What has to leave the range and the places it can go to, kept up to date as requests are marked.
  int64_t must_move = 0, room = static_cast<int64_t>(s->free_local.size());
  for (uint32_t id = cut; id < s->lent_cap; ++id) must_move += s->owner_lent[id].seq >= 0;
  for (int32_t id : s->free_lent) room += static_cast<uint32_t>(id) < cut;
  std::vector<int32_t> order;  // marked requests, in eviction order
  if (must_move > room) {
    // Dense request numbers for the lent ids, so that the rounds below touch arrays only.
    std::unordered_map<int32_t, uint32_t> number;
    std::vector<int32_t> id_of;
    std::vector<uint32_t> req(s->lent_cap, UINT32_MAX);
    for (uint32_t id = 0; id < s->lent_cap; ++id) {
      const int32_t q = s->owner_lent[id].seq;
      if (q < 0) continue;
      auto ins = number.emplace(q, static_cast<uint32_t>(id_of.size()));
      if (ins.second) id_of.push_back(q);
      req[id] = ins.first->second;
    }
    std::vector<uint32_t> stamp(id_of.size(), 0);  // 1 + slab a request was last counted in
    std::vector<char> marked(id_of.size(), 0);
    const uint32_t nslabs = (s->lent_cap + slab_blocks - 1) / slab_blocks;
    while (must_move > room) {
      // Requests per slab, each counted once per slab (the ids of a slab are consecutive).
      uint32_t best = UINT32_MAX, best_n = UINT32_MAX;
      std::fill(stamp.begin(), stamp.end(), 0u);
      for (uint32_t sl = 0; sl < nslabs; ++sl) {
        uint32_t n = 0;
        const uint32_t end = std::min(s->lent_cap, (sl + 1) * slab_blocks);
        for (uint32_t id = sl * slab_blocks; id < end; ++id) {
          const uint32_t r = req[id];
          if (r == UINT32_MAX || marked[r] || stamp[r] == sl + 1) continue;
          stamp[r] = sl + 1;
          ++n;
        }
        if (n && n <= best_n) {  // <=: among equals the highest slab
          best_n = n;
          best = sl;
        }
      }
      if (best == UINT32_MAX) break;  // nothing in use: cannot happen while must_move > 0
      std::vector<int32_t> grp;
      const uint32_t end = std::min(s->lent_cap, (best + 1) * slab_blocks);
      for (uint32_t id = best * slab_blocks; id < end; ++id) {
        const uint32_t r = req[id];
        if (r == UINT32_MAX || marked[r]) continue;
        marked[r] = 1;
        grp.push_back(id_of[r]);
      }
      std::sort(grp.begin(), grp.end());
      for (int32_t q : grp) {
        order.push_back(q);
        for (int32_t e : s->seqs[q].table) {
          if (e < 0 && static_cast<uint32_t>(~e) >= cut) --must_move;
          else ++room;
        }
      }
    }
  }
  if (order.size() > cap || (!order.empty() && !victims)) return SLICE_EINVAL;
  const uint32_t held = blocks_held(s);
  // The migration plans its destinations on the state the evictions leave, and its enqueue can still
  // fail (a CUDA error): the evictions are therefore made on the live state with everything they
  // touch kept aside, and put back if the migration does not go through. Nothing is reported to the
  // caller, counted or capped before it has.
  struct Saved {
    std::vector<int32_t> free_local, free_lent;
    std::vector<std::pair<int32_t, Seq>> seqs;
    uint64_t version;
  } keep;
  if (!order.empty()) {
    keep.free_local = s->free_local;
    keep.free_lent = s->free_lent;
    keep.version = s->version;
    for (int32_t q : order) keep.seqs.emplace_back(q, s->seqs[q]);
    for (int32_t q : order) slice_free_seq(s, q);
  }
  const int rc = slice_reclaim(s, take, out_n_migrated, stream);
  if (rc != SLICE_OK) {
    if (!order.empty()) {
      s->free_local.swap(keep.free_local);
      s->free_lent.swap(keep.free_lent);
      for (auto& kv : keep.seqs) {
        const std::vector<int32_t>& t = kv.second.table;
        for (size_t b = 0; b < t.size(); ++b) {
          const int32_t e = t[b];
          (e >= 0 ? s->owner_local[e] : s->owner_lent[~e]) = Owner{kv.first, static_cast<int32_t>(b)};
        }
        s->seqs[kv.first] = std::move(kv.second);
      }
      recount_slabs(s);
      // The plans built meanwhile saw none of this; a new version keeps them from being reused.
      s->version = keep.version;
      bump_version(s);
    }
    return rc;
  }
  for (size_t k = 0; k < order.size(); ++k) victims[k] = order[k];
  s->preempt_reclaim += order.size();
  if (n_victims) *n_victims = static_cast<uint32_t>(order.size());
  if (!order.empty()) cap_after_reclaim_preemption(s, held);
  return SLICE_OK;
}

int slice_preempt_stats(slice_t* s, slice_preempt_stats_t* out) {
  if (!s || !out) return SLICE_EINVAL;
  out->preempt_oom = s->preempt_oom;
  out->preempt_reclaim = s->preempt_reclaim;
  out->now = s->now;
  out->window = s->preempt_window;
  out->cap_until = cap_in_force(s) ? s->cap_until : 0;
  out->cap_level = cap_in_force(s) ? s->cap_level : 0;
  return SLICE_OK;
}

int slice_set_peer_used(slice_t* s, uint32_t peer_blocks) {
  if (!s || peer_blocks > s->cfg.lent_blocks_physical) return SLICE_EINVAL;
  s->peer_used = peer_blocks;
  return SLICE_OK;
}

int slice_schedule_gll(slice_t* const* slices, uint32_t n, uint32_t* out_index) {
  if (!slices || !out_index || n == 0) return SLICE_EINVAL;
  for (uint32_t k = 0; k < n; ++k)
    if (!slices[k]) return SLICE_EINVAL;
  // used_k / cap_k compared by cross-multiplication: both factors are below 2^33.
  uint32_t best = 0;
  uint64_t best_used = 0, best_cap = 1;
  for (uint32_t k = 0; k < n; ++k) {
    const ema_slice* s = slices[k];
    const uint64_t used = static_cast<uint64_t>(blocks_held(s)) + s->peer_used;
    const uint64_t cap = static_cast<uint64_t>(s->cfg.local_blocks) + s->cfg.lent_blocks_physical;
    if (k == 0 || used * best_cap < best_used * cap) {
      best = k;
      best_used = used;
      best_cap = cap;
    }
  }
  *out_index = best;
  return SLICE_OK;
}

int slice_lend(slice_t* s, uint32_t n) {
  if (!s) return SLICE_EINVAL;
  if (static_cast<uint64_t>(s->lent_cap) + n > s->cfg.lent_blocks_physical) return SLICE_EINVAL;
  for (uint32_t k = n; k-- > 0;) s->free_lent.push_back(static_cast<int32_t>(s->lent_cap + k));
  s->lent_cap += n;
  return SLICE_OK;
}

int slice_append_kv(slice_t* s, uint32_t layer, const int32_t* seqs, uint32_t nseq, const void* k_new,
                    const void* v_new, void* stream_v) {
  const bool all = layer == SLICE_ALL_LAYERS;
  if (!s || (!all && layer >= s->cfg.num_layers)) return SLICE_EINVAL;
  if (all && s->cfg.num_layers > 128) return SLICE_EINVAL;
  if (!s->null_dev && (!k_new || !v_new)) return SLICE_EINVAL;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  Plan* p = nullptr;
  int rc = get_plan(s, seqs, nseq, &p);
  if (rc) return rc;
  const uint32_t* lens = reinterpret_cast<const uint32_t*>(p->host + p->off_lens);
  for (uint32_t i = 0; i < nseq; ++i)
    if (lens[i] == 0) return SLICE_EINVAL;
  if (s->null_dev) return SLICE_OK;
  rc = ensure_stream(s, stream);
  if (rc) return rc;
  rc = plan_on_stream(s, p, stream);
  if (rc) return rc;
  const uint32_t first = all ? 0 : layer, count = all ? s->cfg.num_layers : 1;
  ema::AppendParams a{};
  bool one_staged = false;
  for (uint32_t l = first; l < first + count; ++l) {
    SlotState& sl = s->slots[l % s->layer_slots];
    if (!needs_staging(s, l, p->k) || !staged(s, l, p)) continue;
    if (sl.pref_recorded && sl.pref_stream != stream) CU(s, cudaStreamWaitEvent(stream, sl.pref_done, 0));
    a.staged_mask[(l - first) >> 5] |= 1u << ((l - first) & 31u);
    one_staged = true;
  }
  a.local_base = static_cast<uint8_t*>(s->cfg.local_base);
  a.local_block_stride = s->local_bs;
  a.lent_base = static_cast<uint8_t*>(s->cfg.lent_base) - ema::layer_offset(s->split, s->group, s->lent_gs, s->lent_ls);
  a.lent_block_stride = s->lent_bs;
  a.split_layer = s->split ? s->split : 0xFFFFFFFFu;
  a.staged_only = s->cfg.swap_out;
  a.layer_group = s->group;
  a.local_group_stride = s->local_gs;
  a.lent_group_stride = s->lent_gs;
  a.slot_base = (count == 1 && one_staged) ? static_cast<uint8_t*>(s->cfg.staging_base) + (first % s->layer_slots) * s->slot_bytes : nullptr;
  a.num_layers = count;
  a.first_layer = first;
  a.ring_slots = s->layer_slots;
  a.local_layer_stride = s->local_ls;
  a.lent_layer_stride = s->lent_ls;
  a.io_layer_stride = static_cast<uint64_t>(nseq) * s->cfg.num_kv_heads * kHeadDim * 2;
  a.slot_bytes = s->slot_bytes;
  a.staging_base = static_cast<uint8_t*>(s->cfg.staging_base);
  a.block_bytes = s->block_bytes;
  a.home_entry = reinterpret_cast<const int32_t*>(p->dev + p->off_home);
  a.stage_pos = reinterpret_cast<const int32_t*>(p->dev + p->off_stage_pos);
  a.lens = reinterpret_cast<const uint32_t*>(p->dev + p->off_lens);
  a.k_new = k_new;
  a.v_new = v_new;
  a.nseq = nseq;
  a.row_bytes = s->cfg.num_kv_heads * kHeadDim * 2;
  a.block_tokens = kBlockTokens;
  CU(s, ema::launch_append(a, stream));
  s->st.kernel_launches++;
  if (multi_stream(s)) CU(s, cudaEventRecord(s->append_done, stream));
  s->append_pending = multi_stream(s);
  s->append_stream = stream;
  return SLICE_OK;
}

int slice_writeback_layer(slice_t* s, uint32_t layer, const int32_t* seqs, uint32_t nseq, void* stream_v) {
  if (!s || layer >= s->cfg.num_layers) return SLICE_EINVAL;
  Plan* p = nullptr;
  int rc = get_plan(s, seqs, nseq, &p);
  if (rc) return rc;
  return do_writeback(s, layer, p, static_cast<cudaStream_t>(stream_v));
}

}  // extern "C"

namespace {

// Every staged block of `layer` goes from its ring slot back to its home in the lent arena.
int do_writeback(ema_slice* s, uint32_t layer, Plan* p, cudaStream_t stream) {
  int rc = SLICE_OK;
  const uint32_t slot = layer % s->layer_slots;
  SlotState& sl = s->slots[slot];
  if (s->split && layer < s->split) return SLICE_EINVAL;  // a layer of the local half is never staged
  if (!staged(s, layer, p)) return SLICE_ESTALE;
  if (s->null_dev || p->k == 0) return SLICE_OK;
  rc = ensure_stream(s, stream);
  if (rc) return rc;
  rc = plan_on_stream(s, p, stream);
  if (rc) return rc;
  if (sl.pref_recorded && sl.pref_stream != stream) CU(s, cudaStreamWaitEvent(stream, sl.pref_done, 0));
  // rows appended to the staged copy (on the caller's stream) must be in it
  if (s->append_pending && s->append_stream != stream) CU(s, cudaStreamWaitEvent(stream, s->append_done, 0));
  ema::CopyDesc d{};
  d.src_base[0] = d.src_base[1] = static_cast<const uint8_t*>(s->cfg.staging_base) + slot * s->slot_bytes;
  d.src_block_stride[0] = d.src_block_stride[1] = s->block_bytes;
  d.dst_base[0] = d.dst_base[1] = static_cast<uint8_t*>(s->cfg.lent_base) + lent_off(s, layer);
  d.dst_block_stride[0] = d.dst_block_stride[1] = s->lent_bs;
  d.src_entry = nullptr;
  d.dst_entry = reinterpret_cast<const int32_t*>(p->dev + p->off_copy_src);
  d.n = p->k;
  if (s->cfg.swap_out == 2 && s->in_pass) {
    // Inside a pass only the staged tail blocks can differ from their homes (the explicit
    // slice_writeback_layer call still writes the whole layer).
    if (p->tail_units == 0) return SLICE_OK;
    d.src_entry = reinterpret_cast<const int32_t*>(p->dev + p->off_tail_order);
    d.dst_entry = reinterpret_cast<const int32_t*>(p->dev + p->off_tail_dst);
    d.n = p->tail_units;
  }
  d.nlayers = 1;
  d.block_bytes = s->block_bytes;
  d.status = s->dev_status;
  uint32_t kind = s->cfg.lent_kind == 1 ? ema::kCopyVector : s->cfg.copy_kind;
  if (kind == ema::kCopyDefault) kind = ema::kCopyBulkShared;  // runs beside the attention, like the gather
  CU(s, ema::launch_copy(d, kind, s->cfg.copy_ctas, s->num_sms, stream));
  s->st.kernel_launches++;
  // A later prefetch into this slot (of this layer again, which reads the lent arena, or of another
  // layer, which overwrites the slot) must come after the written blocks.
  if (multi_stream(s)) {
    CU(s, cudaEventRecord(sl.wb_done, stream));
    sl.wb_recorded = true;
  }
  sl.wb_stream = stream;
  return SLICE_OK;
}

// Stream memory operations of the driver (a stream-ordered 32-bit write; a stream-ordered wait until
// a 32-bit word has reached a value), looked up through the runtime so that the library does not
// link against the driver library. Both take (stream, device address, value, flags).
typedef int (*StreamValue32Fn)(cudaStream_t, unsigned long long, unsigned int, unsigned int);
struct StreamOps {
  StreamValue32Fn write = nullptr, wait = nullptr;
  bool tried = false;
};
StreamOps g_stream_ops;

bool stream_ops_ready() {
  if (!g_stream_ops.tried) {
    g_stream_ops.tried = true;
    void *w = nullptr, *v = nullptr;
    cudaDriverEntryPointQueryResult qw, qv;
    if (cudaGetDriverEntryPoint("cuStreamWriteValue32", &w, cudaEnableDefault, &qw) == cudaSuccess &&
        cudaGetDriverEntryPoint("cuStreamWaitValue32", &v, cudaEnableDefault, &qv) == cudaSuccess &&
        qw == cudaDriverEntryPointSuccess && qv == cudaDriverEntryPointSuccess) {
      g_stream_ops.write = reinterpret_cast<StreamValue32Fn>(w);
      g_stream_ops.wait = reinterpret_cast<StreamValue32Fn>(v);
    } else {
      cudaGetLastError();
    }
  }
  return g_stream_ops.write && g_stream_ops.wait;
}

// One pass over all layers (slice_decode_step), or the same pass in its layer-dependent form
// (slice_step_begin): every layer's queries are waited for and every layer's output is announced.
int decode_step_impl(ema_slice* s, const int32_t* seqs, uint32_t nseq, const void* q, uint32_t Hq, float sm_scale,
                     void* out, int32_t io_on_host, int32_t wrap, void* stream_v, void* side_v, bool dependent) {
  if (!s) return SLICE_EINVAL;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v), side = static_cast<cudaStream_t>(side_v);
  Plan* p = nullptr;
  int rc = get_plan(s, seqs, nseq, &p);
  if (rc) return rc;
  const uint32_t L = s->cfg.num_layers, R = s->layer_slots, K = s->group;
  // Mode 0: one launch for the whole pass when the shape allows it, else one launch per layer.
  // (Swap-out passes run layer by layer: the write-back of a layer goes on a stream of its own.)
  const bool step = (s->cfg.pipeline_mode == 0 || s->cfg.pipeline_mode == 3) && s->cfg.ring_slots >= 2 && L >= 2 &&
                    L <= ema::kMaxStepLayers &&
                    s->ncta <= static_cast<uint32_t>(s->num_sms) && !(s->cfg.swap_out && s->cfg.pipeline_mode == 3);
  const bool fused = s->cfg.pipeline_mode != 1 && s->cfg.ring_slots >= 2;
  if (fused) side = stream;
  const size_t per_layer = static_cast<size_t>(nseq) * Hq * kHeadDim * 2;
  const uint8_t* qd = static_cast<const uint8_t*>(q);
  uint8_t* od = static_cast<uint8_t*>(out);
  bool out_mapped = false, streamed_q = false;
  s->step_q_ready = nullptr;
  s->step_out_ready = nullptr;
  if (dependent) {
    // Only the one-launch pass has anything to feed: with the other pipelines the caller drives the
    // layers itself and the stream already orders a layer's attention after its queries.
    if (io_on_host || !step || s->cfg.pipeline_mode != 0) return SLICE_EINVAL;
    for (uint32_t i = 0; i < nseq; ++i)
      if (s->seqs[seqs[i]].len == 0) return SLICE_EINVAL;  // before the epoch moves
    if (!s->null_dev && !stream_ops_ready()) {
      s->st.last_cuda_error = static_cast<int>(cudaErrorNotSupported);
      return SLICE_ECUDA;
    }
    ++s->q_epoch;
    s->step_q_ready = s->q_flags_dev;
    s->step_q_layers = 1;
    s->step_out_ready = s->out_flags_dev;
  }
  if (!s->null_dev) {
    rc = ensure_stream(s, stream);
    if (rc) return rc;
  }
  if (s->profile && !s->null_dev) {
    std::fill(s->prof_set.begin(), s->prof_set.end(), 0);
    CU(s, cudaEventRecord(s->prof_base, stream));
    s->prof_base_set = true;
  }
  if (io_on_host && !s->null_dev) {
    if (!q || !out) return SLICE_EINVAL;
    const size_t need = per_layer * L;
    if (need > s->io_bytes) {
      CU(s, cudaDeviceSynchronize());
      if (s->io_q) cudaFree(s->io_q);
      if (s->io_out) cudaFree(s->io_out);
      s->io_q = s->io_out = nullptr;
      s->io_bytes = 0;
      CU(s, cudaMalloc(&s->io_q, need));
      CU(s, cudaMalloc(&s->io_out, need));
      s->io_bytes = need;
    }
    qd = static_cast<const uint8_t*>(s->io_q);
    od = static_cast<uint8_t*>(s->io_out);
    cudaPointerAttributes aq{};
    const bool q_pinned = cudaPointerGetAttributes(&aq, q) == cudaSuccess && aq.type == cudaMemoryTypeHost;
    if (!q_pinned) cudaGetLastError();
    if (step && q_pinned) {
      // One launch covers the pass: bring q in behind it, a few layers per copy on a stream of its
      // own, each copy followed by a 4-byte copy that sets the chunk's arrival flag; the kernel
      // reads a layer's rows only after its flag shows this pass's epoch (bounded wait).
      if (!s->io_stream) {
        CU(s, cudaStreamCreateWithFlags(&s->io_stream, cudaStreamNonBlocking));
        CU(s, cudaMallocHost(reinterpret_cast<void**>(&s->q_epoch_host), 64 * sizeof(uint32_t)));
        CU(s, cudaEventCreateWithFlags(&s->io_q_free, cudaEventDisableTiming));
      }
      if (s->io_q_busy) CU(s, cudaStreamWaitEvent(s->io_stream, s->io_q_free, 0));
      // everything enqueued on `stream` so far (earlier passes, the reallocation above) comes first
      CU(s, cudaEventRecord(s->ev_tmp, stream));
      CU(s, cudaStreamWaitEvent(s->io_stream, s->ev_tmp, 0));
      const uint32_t per_flag = 4;
      ++s->q_epoch;
      // The flag copies read this word when they execute; epochs only grow and the kernel waits for
      // "at least its own", so a word overwritten by a later pass that is enqueued far ahead still
      // says what it must: this pass's chunk has arrived (its copy precedes the flag copy).
      uint32_t* epoch_word = s->q_epoch_host + (s->q_epoch % 64);
      *epoch_word = s->q_epoch;
      for (uint32_t l0 = 0; l0 < L; l0 += per_flag) {
        const size_t bytes = per_layer * std::min(per_flag, L - l0);
        CU(s, cudaMemcpyAsync(static_cast<uint8_t*>(s->io_q) + l0 * per_layer, static_cast<const uint8_t*>(q) + l0 * per_layer, bytes,
                              cudaMemcpyHostToDevice, s->io_stream));
        if (!(s->cfg.flags & SLICE_FLAG_TEST_WITHHOLD_Q))
          CU(s, cudaMemcpyAsync(s->q_flags_dev + l0 / per_flag, epoch_word, sizeof(uint32_t), cudaMemcpyHostToDevice, s->io_stream));
      }
      s->step_q_ready = s->q_flags_dev;
      s->step_q_layers = per_flag;
      streamed_q = true;
    } else {
      CU(s, cudaMemcpyAsync(s->io_q, q, need, cudaMemcpyHostToDevice, stream));
    }
    // Pinned (mapped) host memory can be written by the kernels themselves: the merges then store
    // each finished row straight to the host while the pass goes on, and no copy follows the pass.
    cudaPointerAttributes attr{};
    if (cudaPointerGetAttributes(&attr, out) == cudaSuccess && attr.type == cudaMemoryTypeHost && attr.devicePointer) {
      od = static_cast<uint8_t*>(attr.devicePointer);
      out_mapped = true;
    } else {
      cudaGetLastError();  // a pageable pointer is not an error here
    }
  }
  if (!s->null_dev)  // the work counters of all layers, cleared once per pass
    CU(s, cudaMemsetAsync(s->cnt_dev, 0, static_cast<size_t>(L) * s->cnt_stride * sizeof(uint32_t), stream));
  for (uint32_t l = 0; l < std::min(K, L); ++l) {  // the first layer group
    if (!needs_staging(s, l, p->k) || staged(s, l, p)) continue;
    rc = do_prefetch(s, l, p, side);
    if (rc) return rc;
  }
  if (step) {
    rc = do_step(s, p, qd, Hq, sm_scale, od, stream, wrap != 0);
    if (rc) return rc;
    if (dependent && !s->null_dev) {
      const int slot = static_cast<int>(s->q_epoch % ema_slice::kFillSlots);
      if (s->fill_busy[slot]) CU(s, cudaEventSynchronize(s->fill_done[slot]));  // the words of 8 passes ago
      uint32_t* words = s->out_fill_host + static_cast<size_t>(slot) * ema::kMaxStepLayers;
      for (uint32_t l = 0; l < L; ++l) words[l] = s->q_epoch;
      CU(s, cudaMemcpyAsync(s->out_flags_dev, words, L * sizeof(uint32_t), cudaMemcpyHostToDevice, stream));
      CU(s, cudaEventRecord(s->fill_done[slot], stream));
      s->fill_busy[slot] = true;
    }
  }
  if (s->cfg.swap_out && !s->null_dev && !s->swap_stream)
    CU(s, cudaStreamCreateWithFlags(&s->swap_stream, cudaStreamNonBlocking));
  for (uint32_t l = 0; l < L && !step; ++l) {
    // Swap-out (Section 2.3: layers are swapped in and out cyclically; as much leaves as comes in):
    // the layer's staged blocks go back to the lent arena, on a third stream, while the layer is
    // attended to and the next transfer comes in. The slot is refilled only after that write.
    if (s->cfg.swap_out && needs_staging(s, l, p->k) && staged(s, l, p)) {
      s->in_pass = true;
      rc = do_writeback(s, l, p, s->swap_stream);
      s->in_pass = false;
      if (rc) return rc;
    }
    // Layer-boundary check (Section 4.2.2): decide the next transfer before computing this layer.
    int next = -1;
    if (p->k) {
      if (l + K < L) {
        next = static_cast<int>(l + K);
      } else if (wrap && L > 1) {
        next = static_cast<int>(l + K - L);
        for (uint32_t j = l; j < L; ++j)
          if (j % R == static_cast<uint32_t>(next) % R) next = -1;  // its slot still serves this pass
      }
      if (next >= 0 && (!needs_staging(s, static_cast<uint32_t>(next), p->k) || staged(s, static_cast<uint32_t>(next), p))) next = -1;
    }
    if (fused) {
      rc = do_layer(s, l, p, qd + l * per_layer, Hq, sm_scale, od + l * per_layer, nullptr, stream, next, false, true);
      if (rc) return rc;
    } else {
      // A ring of one slot: the next layer's data goes where this layer's is, so the prefetch can
      // only follow the attention (no overlap; the slot-reuse event orders the two streams).
      const bool same_slot = next >= 0 && static_cast<uint32_t>(next) % R == l % R;
      if (next >= 0 && !same_slot) {
        rc = do_prefetch(s, static_cast<uint32_t>(next), p, side);
        if (rc) return rc;
      }
      rc = do_layer(s, l, p, qd + l * per_layer, Hq, sm_scale, od + l * per_layer, nullptr, stream, -1, false, true);
      if (rc) return rc;
      if (same_slot) {
        rc = do_prefetch(s, static_cast<uint32_t>(next), p, side);
        if (rc) return rc;
      }
    }
  }
  for (uint32_t l = 0; wrap && L > 1 && l < std::min(K, L); ++l) {
    // Layers of the next pass's first group whose ring slot served a layer of this pass to the end:
    // refilled only after that attention.
    if (!needs_staging(s, l, p->k) || staged(s, l, p)) continue;
    rc = do_prefetch(s, l, p, side);
    if (rc) return rc;
  }
  if (streamed_q) {
    // io_q may be overwritten once this pass is done; a later non-streamed use of io_q on `stream`
    // is ordered by the stream itself.
    CU(s, cudaEventRecord(s->io_q_free, stream));
    s->io_q_busy = true;
  }
  s->step_q_ready = nullptr;
  s->step_out_ready = nullptr;
  s->dependent_pass = dependent;
  if (io_on_host && !s->null_dev && !out_mapped)
    CU(s, cudaMemcpyAsync(out, s->io_out, per_layer * L, cudaMemcpyDeviceToHost, stream));
  return SLICE_OK;
}

}  // namespace

extern "C" {

int slice_decode_step(slice_t* s, const int32_t* seqs, uint32_t nseq, const void* q, uint32_t Hq, float sm_scale,
                      void* out, int32_t io_on_host, int32_t wrap, void* stream_v, void* side_v) {
  return decode_step_impl(s, seqs, nseq, q, Hq, sm_scale, out, io_on_host, wrap, stream_v, side_v, false);
}

int slice_step_begin(slice_t* s, const int32_t* seqs, uint32_t nseq, const void* q, uint32_t Hq, float sm_scale,
                     void* out, int32_t wrap, void* stream_v) {
  return decode_step_impl(s, seqs, nseq, q, Hq, sm_scale, out, 0, wrap, stream_v, stream_v, true);
}

int slice_step_submit_q(slice_t* s, uint32_t layer, void* caller_stream) {
  if (!s || layer >= s->cfg.num_layers || !s->dependent_pass) return SLICE_EINVAL;
  if (s->null_dev) return SLICE_OK;
  if (!stream_ops_ready()) return SLICE_ECUDA;
  const int r = g_stream_ops.write(static_cast<cudaStream_t>(caller_stream),
                                   reinterpret_cast<unsigned long long>(s->q_flags_dev + layer), s->q_epoch, 0u);
  if (r != 0) {
    s->st.last_cuda_error = r;
    return SLICE_ECUDA;
  }
  return SLICE_OK;
}

int slice_step_wait_out(slice_t* s, uint32_t layer, void* caller_stream) {
  if (!s || layer >= s->cfg.num_layers || !s->dependent_pass) return SLICE_EINVAL;
  if (s->null_dev) return SLICE_OK;
  if (!stream_ops_ready()) return SLICE_ECUDA;
  const int r = g_stream_ops.wait(static_cast<cudaStream_t>(caller_stream),
                                  reinterpret_cast<unsigned long long>(s->out_flags_dev + layer), s->q_epoch,
                                  0u /* wait until the word is >= the value (epochs only grow) */);
  if (r != 0) {
    s->st.last_cuda_error = r;
    return SLICE_ECUDA;
  }
  return SLICE_OK;
}

int slice_step_relay(slice_t* s, void* caller_stream) {
  if (!s || !s->dependent_pass) return SLICE_EINVAL;
  if (s->null_dev) return SLICE_OK;
  // The relay has to run beside the pass: it needs an SM that the pass leaves free.
  if (s->ncta >= static_cast<uint32_t>(s->num_sms)) return SLICE_EINVAL;
  CU(s, ema::launch_step_relay(s->out_flags_dev, s->q_flags_dev, s->cfg.num_layers, s->q_epoch, s->dev_status,
                               static_cast<cudaStream_t>(caller_stream)));
  s->st.kernel_launches++;
  return SLICE_OK;
}

int slice_step_flags(slice_t* s, uint32_t** q_ready, uint32_t** out_ready, uint32_t* epoch) {
  if (!s || !s->dependent_pass) return SLICE_EINVAL;
  if (q_ready) *q_ready = s->q_flags_dev;
  if (out_ready) *out_ready = s->out_flags_dev;
  if (epoch) *epoch = s->q_epoch;
  return SLICE_OK;
}

int slice_stats(slice_t* s, slice_stats_t* out) {
  if (!s || !out) return SLICE_EINVAL;
  s->st.local_free = static_cast<uint32_t>(s->free_local.size());
  s->st.local_used = s->cfg.local_blocks - s->st.local_free;
  s->st.lent_free = static_cast<uint32_t>(s->free_lent.size());
  s->st.lent_used = s->lent_cap - s->st.lent_free;
  s->st.lent_capacity = s->lent_cap;
  s->st.num_seqs = static_cast<uint32_t>(s->seqs.size());
  // The status word lives in mapped host memory: reading it costs no CUDA call and waits for nothing.
  if (!s->null_dev && s->dev_status) s->st.device_status = *static_cast<volatile int*>(s->dev_status);
  *out = s->st;
  return SLICE_OK;
}

int slice_get_resolved(slice_t* s, const int32_t* seqs, uint32_t nseq, int32_t* out, uint32_t cap, uint32_t* k) {
  if (!s) return SLICE_EINVAL;
  Plan* p = nullptr;
  int rc = get_plan(s, seqs, nseq, &p);
  if (rc) return rc;
  if (k) *k = p->k;
  if (out) {
    const uint32_t stride = s->cfg.max_blocks_per_seq;
    if (static_cast<uint64_t>(cap) < static_cast<uint64_t>(nseq) * stride) return SLICE_EINVAL;
    for (uint32_t i = 0; i < nseq; ++i)
      for (uint32_t f = p->blk_off[i]; f < p->blk_off[i + 1]; ++f)
        out[static_cast<size_t>(i) * stride + (f - p->blk_off[i])] = p->resolved_ids[f];
  }
  return SLICE_OK;
}

int slice_cta_trace(slice_t* s, int32_t which, uint64_t* out, uint64_t cap_entries, uint32_t* ctas_per_layer,
                    uint32_t* words_per_cta) {
  if (!s || !s->trace || s->null_dev || (which != 0 && which != 1)) return SLICE_EINVAL;
  const uint32_t per = which == 0 ? s->ncta : kTraceCopyCtas;
  const uint32_t words = which == 0 ? ema::kTraceWords : 2;
  if (ctas_per_layer) *ctas_per_layer = per;
  if (words_per_cta) *words_per_cta = words;
  if (!out) return SLICE_OK;
  const uint64_t n = static_cast<uint64_t>(s->cfg.num_layers) * per * words;
  if (cap_entries < n) return SLICE_EINVAL;
  CU(s, cudaDeviceSynchronize());
  CU(s, cudaMemcpy(out, which == 0 ? s->trace_layer : s->trace_copy, n * sizeof(uint64_t), cudaMemcpyDeviceToHost));
  return SLICE_OK;
}

int slice_layer_times(slice_t* s, float* out, uint32_t cap_layers) {
  if (!s || !out || !s->profile || s->null_dev || !s->prof_base_set) return SLICE_EINVAL;
  if (cap_layers < s->cfg.num_layers) return SLICE_EINVAL;
  CU(s, cudaDeviceSynchronize());
  for (uint32_t i = 0; i < s->cfg.num_layers * 5; ++i) {
    out[i] = std::numeric_limits<float>::quiet_NaN();
    if (!s->prof_set[i]) continue;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, s->prof_base, s->prof[i]) == cudaSuccess) out[i] = ms * 1000.f;
  }
  return SLICE_OK;
}

int slice_copy_blocks(void* dst_base, const int32_t* dst_idx, const void* src_base, const int32_t* src_idx, uint32_t n,
                      uint64_t block_bytes, uint32_t kind, uint32_t ctas, void* stream) {
  if (!dst_base || !src_base || (block_bytes & 15u) || block_bytes == 0 || kind > 3) return SLICE_EINVAL;
  if ((reinterpret_cast<uintptr_t>(dst_base) | reinterpret_cast<uintptr_t>(src_base)) & 15u) return SLICE_EINVAL;
  static int sms_of[64] = {};  // per device
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SLICE_ECUDA;
  if (!sms_of[dev] && cudaDeviceGetAttribute(&sms_of[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return SLICE_ECUDA;
  const int sms = sms_of[dev];
  ema::CopyDesc d{};
  d.src_base[0] = d.src_base[1] = static_cast<const uint8_t*>(src_base);
  d.dst_base[0] = d.dst_base[1] = static_cast<uint8_t*>(dst_base);
  d.src_block_stride[0] = d.src_block_stride[1] = block_bytes;
  d.dst_block_stride[0] = d.dst_block_stride[1] = block_bytes;
  d.src_entry = src_idx;
  d.dst_entry = dst_idx;
  d.n = n;
  d.nlayers = 1;
  d.block_bytes = block_bytes;
  d.status = nullptr;
  return ema::launch_copy(d, kind, ctas, sms, static_cast<cudaStream_t>(stream)) == cudaSuccess ? SLICE_OK : SLICE_ECUDA;
}

int slice_copy_blocks_series(void* ring_base, uint32_t ring_slots, uint64_t slot_bytes, void* arena_base, const int32_t* idx,
                             uint64_t n_total, uint32_t per_launch, uint64_t block_bytes, int32_t scatter, uint32_t kind,
                             uint32_t ctas, void* stream) {
  if (!ring_base || !arena_base || !idx || ring_slots == 0 || per_launch == 0 || (block_bytes & 15u) || block_bytes == 0 || kind > 2)
    return SLICE_EINVAL;
  if (static_cast<uint64_t>(per_launch) * block_bytes > slot_bytes) return SLICE_EINVAL;
  if ((reinterpret_cast<uintptr_t>(ring_base) | reinterpret_cast<uintptr_t>(arena_base) | slot_bytes) & 15u) return SLICE_EINVAL;
  const uint64_t launches = n_total / per_launch;
  for (uint64_t j = 0; j < launches; ++j) {
    uint8_t* slot = static_cast<uint8_t*>(ring_base) + (j % ring_slots) * slot_bytes;
    const int32_t* sel = idx + j * per_launch;
    const int rc = scatter ? slice_copy_blocks(arena_base, sel, slot, nullptr, per_launch, block_bytes, kind, ctas, stream)
                           : slice_copy_blocks(slot, nullptr, arena_base, sel, per_launch, block_bytes, kind, ctas, stream);
    if (rc) return rc;
  }
  return SLICE_OK;
}

const char* slice_strerror(int code) {
  switch (code) {
    case SLICE_OK: return "ok";
    case SLICE_EINVAL: return "invalid argument";
    case SLICE_ENOSPC: return "not enough free blocks";
    case SLICE_ESTAGING: return "batch exceeds the staging slot";
    case SLICE_ESTALE: return "layer is not validly staged for this batch";
    case SLICE_ECUDA: return "CUDA call failed";
    case SLICE_ETIMEOUT: return "bounded device wait expired";
    case SLICE_ESTATE: return "unknown sequence or bad state";
    case SLICE_ECAPPED: return "a cap set by an earlier preemption holds";
    case SLICE_ESCRATCH: return "request exceeds the static scratch array";
    default: return "unknown status";
  }
}

}  // extern "C"
