// layer_kernel.cu — the fused kernel of the memory-slice hot path. One persistent launch (one CTA
// per SM) covers one layer or a whole pass over all layers of a batch:
//   paged GQA decode attention of layer l  (split-KV flash decoding, merge included)
//   + prefetch gather of layer l+1's lent blocks into the other ring slot,
// so the two streams of HBM traffic share every SM for the whole duration of a layer, with no second
// kernel to co-schedule, no merge launch and no cross-stream event. When the launch spans several
// layers, layer boundaries are soft: a CTA that runs out of work in layer l moves on to layer l+1
// while others finish l, so tails, merges and ramp-up overlap with streaming instead of leaving HBM
// idle once per layer.
//
// Work distribution. The batch's blocks, flattened in batch order, are cut into one contiguous range
// per CTA (the same for every layer). A CTA claims blocks from the FRONT of its own range; a CTA
// whose range is used up steals from the BACK of the range with the most unclaimed blocks, provided
// that range is well behind (steal floor), and otherwise moves on to the next layer. Both kinds of
// claim are one atomicAdd on the range's packed 64-bit word (front count | back count), so they can
// never overlap. SMs stream at visibly different rates (position on the die, mixed read/write
// traffic). A CTA keeps one running softmax state per "run" = consecutive claims within one
// sequence, so partial results stay few.
//
// Roles inside a CTA (warps):
//   * producer warp: claims work and streams KV blocks into a shared-memory ring of half blocks
//     (K plane / V plane, 16 token rows of Hkv*256 B) with ONE untiled TMA bulk copy per plane
//     (cp.async.bulk, 32 KB for 8 KV heads: small copies cap the rate an SM can stream at),
//     completion by mbarrier expect-tx; the block format stores the 16-byte units of a row swizzled,
//     so the linear copy leaves a layout that ldmatrix reads without bank conflicts. A small
//     descriptor queue tells the consumers what each unit is.
//   * one consumer warp per KV head: tile products on tensor cores when the GQA group is >= 2
//     (mma.sync m16n8k16 bf16, swapped form), f32 FMAs when G == 1; online softmax with warp
//     shuffles. A finished run writes (max, sums, unnormalised output) to a partial slot and adds its
//     block count to the (sequence, KV head) counter; the warp whose addition completes the sequence
//     queues a merge request (the ring is shared by all consumer warps, so a warp that stopped to
//     merge would stall the whole CTA) or, when layers are short, merges in line (then the merges
//     of a sequence's KV heads run side by side instead of one after the other).
//   * merge warp: serves the CTA's merge queue, then merge requests that any CTA has published for
//     all: the KV heads of a sequence finish together in one CTA, and with few long sequences their
//     merges, of a hundred and more partials each, would queue up behind one warp (a layer of one
//     128k-token sequence took 155 us that way and takes 87 us now). Consumer warps join once their
//     streaming is over. Nobody waits for a request that is not yet published, so a CTA never stays
//     behind for work of CTAs that are not resident yet.
//   * copy warp: one thread moves 16 KB pieces lent arena -> shared ring -> staging slot with TMA
//     bulk copies (global->shared on an mbarrier, shared->global in bulk async-groups), pulling
//     64 KB units from an atomic counter. No SM lane touches the copied bytes.
//
// Waits. Inside a CTA everything is mbarriers. Between CTAs there are three waits, only in launches
// that span several layers (which are launched cooperatively, so every CTA is resident): a staged
// block of layer l is read only after its ready flag shows that the gather has landed it; a ring
// slot is overwritten only after the attention of the layer that last used it is complete; a partial
// buffer (four take turns) is reused only after the merges of the layer that used it last are done. They
// wait on what earlier layers' work produces, never on later work, and a run left open at the end of
// a layer is closed at once (a CTA may find nothing to claim in later layers), so they cannot form a
// cycle. A fourth, optional wait is for queries that arrive from the host while the launch runs. Every wait, mbarrier or counter, is bounded (about two seconds): on expiry the role records
// SLICE_ETIMEOUT in the status word, gives its own copies in flight a bounded chance to land and
// returns.
// HBM-bound: algorithmic bytes per layer = sum_s len_s * 2*Hkv*128*2 (+ q, out, table)
// + 2 * block_bytes per gathered block.
#include "attention_tiles.cuh"
#include "kernels.h"

#include <cooperative_groups.h>
#include <cuda_bf16.h>

namespace ema {

namespace {

constexpr uint32_t kNAFused = 4;           // attention ring (stages of up to 32 KB) beside a copy ring
constexpr uint32_t kNAAlone = 3;           // ... and when the launch gathers nothing. With one 32 KB request per
                                           // stage a deeper ring only queues more reads in the memory
                                           // system and measures slower (3: 6.1 TB/s, 6: 5.3 TB/s).
                                           // With 1 or 2 KV heads a plane is small (4 KB per head): a stage
                                           // then holds the planes of 8 / Hkv consecutive blocks, each with
                                           // consumer warps of its own (see blocks_per_stage); with 3 or 4
                                           // the ring has twice as many, smaller stages.
constexpr uint32_t kNAMax = 8;
constexpr int kNC = 6;                     // copy ring: 16 KB stages
constexpr uint32_t kCopyLoadsDefault = 3;  // loads in flight (LayerParams::copy_loads_ahead, 3 or 4) ...
constexpr int kStoresOpen = 2;             // ... and stores not yet known complete; 4 + 2 = kNC
constexpr uint32_t kCopyChunk = 16384;
constexpr int kQueue = 12;                 // unit descriptors in flight (> kNAMax / 2 + 1, plus a flush and the end marker)
constexpr uint32_t kSentinel = 0xFFFFFFFFu;
constexpr uint32_t kFlush = 0xFFFFFFFEu;   // descriptor without data: close the open run now
constexpr uint32_t kNewRun = 0x80000000u;
constexpr uint32_t kRingAlign = 128;
constexpr uint32_t kStealMin = 2, kStealMax = 16;
constexpr uint64_t kWaitNs = 2000000000ull;
constexpr uint32_t kMq = 32;               // merge requests queued per CTA
constexpr uint32_t kMqEmpty = 0xFFFFFFFFu;
constexpr uint32_t kMqTail = kMq, kMqHead = kMq + 1, kMqDone = kMq + 2;
constexpr uint32_t kMqWind = kMq + 3;      // set by the producer when it streams the launch's last claim
constexpr uint32_t kOwnCache = 352;        // resolved entries of the own range kept in shared memory

__host__ __device__ constexpr uint32_t row_bytes(uint32_t Hkv) { return Hkv * kD * 2; }
__host__ __device__ constexpr uint32_t half_stage_bytes(uint32_t Hkv) { return kT * row_bytes(Hkv); }

// A unit: blocks [blk_begin, blk_end) of batch position seq_idx in layer `layer`. slot carries the
// run's partial slot and the kNewRun flag when the unit starts a new run.
struct UnitDesc {
  uint32_t seq_idx, blk_begin, blk_end, slot, layer, pad0, pad1, pad2;
};

// Position in the attention ring: stage index and the parity of its current use, advanced without
// divisions (the ring depth is a run-time value).
struct RingPos {
  uint32_t stg = 0, phase = 0;
  __device__ __forceinline__ void advance(uint32_t na) {
    if (++stg == na) {
      stg = 0;
      phase ^= 1u;
    }
  }
};

struct Claim {
  uint32_t b, e;  // flat blocks [b, e); empty when b >= e
};

// The sequence the producer is in: batch position, its flat blocks [lo, hi), and the end of the
// next sequence's blocks (fetched ahead).
struct Cursor {
  uint32_t seq, lo, hi, nhi;
};

struct Smem {
  uint32_t na;          // attention ring stages in use
  uint8_t* att_ring;
  uint8_t* copy_ring;
  uint64_t* att_full;   // [kNAMax]
  uint64_t* att_empty;  // [kNAMax]
  uint64_t* copy_full;  // [kNC]
  UnitDesc* queue;      // [kQueue]
  uint8_t** copy_dst;   // [kNC]
  uint32_t* copy_len;   // [kNC]
  uint32_t* mq;         // merge queue of the CTA: [kMq] entries, then tail, head, consumer warps done
  uint32_t* head_runs;  // [8] per KV head: partials written by its consumer warps (runs x warps of the head)
  int32_t* own_res;     // [kOwnCache] resolved entries of the CTA's own range
};

// Bookkeeping area behind the two rings; every part 16-byte aligned.
constexpr size_t kBarBytes = 70 * sizeof(uint64_t);
constexpr size_t kQueueBytes = kQueue * sizeof(UnitDesc);
constexpr size_t kCopyDstBytes = 8 * sizeof(uint8_t*);
constexpr size_t kCopyLenBytes = 8 * sizeof(uint32_t);
constexpr size_t kMqBytes = (kMq + 4 + 8) * sizeof(uint32_t);
constexpr size_t kOwnBytes = kOwnCache * sizeof(int32_t);
static_assert(2 * kNAMax + kNC <= 70 && kNC <= 8 && kQueue > kNAMax / 2 + 1, "bookkeeping area too small");
static_assert(kNAFused * 32768 + kNC * 16384 >= kNAAlone * 32768, "the deeper ring must fit in the fused layout");

// Blocks that share a stage: with few KV heads a plane is small (4 KB per head), and one warp per
// KV head taking the blocks one by one, behind one producer lane issuing them one by one, is bound
// by the per-block latencies of both (2.1 TB/s at 1 KV head, 4.2 at 2). A stage therefore holds the
// planes of V = 8 / Hkv consecutive blocks of a unit, copied by V lanes of the producer at once, and
// every KV head has V consumer warps, warp v taking block v of each group of V with a softmax state
// and a partial of its own (the merge adds them up like any other partials).
// Measured (64 sequences of 2k..8k tokens, nothing lent, KV read rate): 1 KV head 2.08 -> 4.46 TB/s,
// 2 KV heads 4.17 -> 6.02, 3 KV heads (two warps per head, six in all) 5.80 -> 6.52, 4 KV heads
// 6.49 -> 6.79 (3 and 4 heads: the same as one block per stage when the launch also gathers).
__host__ __device__ constexpr uint32_t blocks_per_stage(uint32_t Hkv) { return partials_per_slot(Hkv); }
// A shared stage holds the V blocks whole (K plane and V plane are neighbours in memory: one request
// of 8 or 16 KB per block instead of two of 4 or 8 KB), 64 KB per stage, two stages.
__host__ __device__ constexpr uint32_t stage_bytes(uint32_t Hkv) {
  return blocks_per_stage(Hkv) > 1 ? blocks_per_stage(Hkv) * 2 * half_stage_bytes(Hkv) : half_stage_bytes(Hkv);
}
constexpr uint32_t kGroupedStages = 2;     // beside a copy ring; 3 when the launch gathers nothing (4-5 % faster there)

static_assert(kRingAlign + kNAFused * 32768 + kNC * kCopyChunk + kBarBytes + kQueueBytes + kCopyDstBytes + kCopyLenBytes + kMqBytes +
                      kOwnBytes <= 232448,
              "more shared memory than a CTA can have (227 KB)");

__host__ __device__ constexpr size_t smem_total(uint32_t Hkv) {
  return kRingAlign + static_cast<size_t>(blocks_per_stage(Hkv) > 1 ? kGroupedStages : kNAFused) * stage_bytes(Hkv) +
         static_cast<size_t>(kNC) * kCopyChunk + kBarBytes +
         kQueueBytes + kCopyDstBytes + kCopyLenBytes + kMqBytes + kOwnBytes;
}

// Attention stages of a launch: beside a copy ring, or alone (the launch gathers nothing).
__host__ __device__ constexpr uint32_t attention_stages(uint32_t Hkv, bool gathers) {
  return blocks_per_stage(Hkv) > 1 ? (gathers ? kGroupedStages : 3u) : (gathers ? kNAFused : kNAAlone);
}
// A launch that gathers nothing has no copy ring: the bookkeeping follows the attention ring, and with
// 5 to 8 KV heads the CTA takes 100 KB, which leaves room on its SM for a CTA of the shared form of
// the gather kernel (a gather on a second stream then really runs beside the attention).
__host__ __device__ constexpr size_t smem_needed(uint32_t Hkv, bool gathers) {
  return kRingAlign + static_cast<size_t>(attention_stages(Hkv, gathers)) * stage_bytes(Hkv) +
         (gathers ? static_cast<size_t>(kNC) * kCopyChunk : 0) + kBarBytes + kQueueBytes + kCopyDstBytes + kCopyLenBytes + kMqBytes +
         kOwnBytes;
}

__device__ __forceinline__ Smem carve(uint8_t* base, uint32_t Hkv, bool gathers) {
  Smem s;
  s.na = attention_stages(Hkv, gathers);
  base += (kRingAlign - (ptx::smem_u32(base) & (kRingAlign - 1))) & (kRingAlign - 1);
  s.att_ring = base;
  s.copy_ring = base + static_cast<size_t>(s.na) * stage_bytes(Hkv);
  uint8_t* p = s.copy_ring + (gathers ? static_cast<size_t>(kNC) * kCopyChunk : 0);
  s.att_full = reinterpret_cast<uint64_t*>(p);
  s.att_empty = s.att_full + kNAMax;
  s.copy_full = s.att_empty + kNAMax;
  s.queue = reinterpret_cast<UnitDesc*>(p + kBarBytes);
  s.copy_dst = reinterpret_cast<uint8_t**>(p + kBarBytes + kQueueBytes);
  s.copy_len = reinterpret_cast<uint32_t*>(p + kBarBytes + kQueueBytes + kCopyDstBytes);
  s.mq = reinterpret_cast<uint32_t*>(p + kBarBytes + kQueueBytes + kCopyDstBytes + kCopyLenBytes);
  s.head_runs = s.mq + kMq + 4;
  s.own_res = reinterpret_cast<int32_t*>(p + kBarBytes + kQueueBytes + kCopyDstBytes + kCopyLenBytes + kMqBytes);
  return s;
}

// Per-layer pieces of the parameter block; li = layer - first_layer.
__device__ __forceinline__ uint32_t* layer_counters(const LayerParams& p, uint32_t li) {
  return p.counters + li * p.counters_stride;
}
__device__ __forceinline__ unsigned long long* range_words(const LayerParams& p, uint32_t li) {
  return reinterpret_cast<unsigned long long*>(layer_counters(p, li) + kLaunchCounters);
}
__device__ __forceinline__ uint32_t* seq_counts(const LayerParams& p, uint32_t li) {
  return layer_counters(p, li) + kLaunchCounters + 2 * p.ncta;
}
__device__ __forceinline__ uint32_t* merge_counts(const LayerParams& p, uint32_t li) { return seq_counts(p, li) + p.nseq; }
__device__ __forceinline__ uint32_t* merge_requests(const LayerParams& p, uint32_t li) {
  return merge_counts(p, li) + p.nseq * p.Hkv;
}
__device__ __forceinline__ float* part_o_of(const LayerParams& p, uint32_t li) {
  return p.part_o + (li & (p.part_buffers - 1u)) * p.part_o_stride;
}
__device__ __forceinline__ float* part_ml_of(const LayerParams& p, uint32_t li) {
  return p.part_ml + (li & (p.part_buffers - 1u)) * p.part_ml_stride;
}

// Bounded wait until a device word written by another CTA equals `value`. The reads are acquires:
// what the writer did before its release of the word is visible after a successful wait.
__device__ __forceinline__ bool wait_counter_eq(const uint32_t* word, uint32_t value, int* status) {
  if (ptx::ld_acquire_gpu(word) == value) return true;
  const uint64_t t0 = ptx::global_timer_ns();
  while (ptx::ld_acquire_gpu(word) != value) {
    if (ptx::global_timer_ns() - t0 > kWaitNs) {
      ptx::report_status(status, kDevTimeout);
      return false;
    }
    __nanosleep(64);
  }
  return true;
}

// Bounded wait until a device counter written by other CTAs reaches `target`.
__device__ __forceinline__ bool wait_counter(const uint32_t* cnt, uint32_t target, int* status) {
  if (ptx::ld_acquire_gpu(cnt) >= target) return true;
  const uint64_t t0 = ptx::global_timer_ns();
  while (ptx::ld_acquire_gpu(cnt) < target) {
    if (ptx::global_timer_ns() - t0 > kWaitNs) {
      ptx::report_status(status, kDevTimeout);
      return false;
    }
    __nanosleep(128);
  }
  return true;
}

// ---------------------------------------------------------------------------------------------
// producer warp
// ---------------------------------------------------------------------------------------------
template <bool kGrouped>
__device__ void producer_role(const LayerParams& p, const Smem& sm) {
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t Hkv = p.Hkv;
  const uint32_t hsb = half_stage_bytes(Hkv);
  const uint32_t plane_bytes = hsb;
  const uint32_t V = kGrouped ? blocks_per_stage(Hkv) : 1u, sbytes = kGrouped ? stage_bytes(Hkv) : hsb;
  const uint32_t ring = ptx::smem_u32(sm.att_ring);
  uint32_t hs = 0, nq = 0;
  RingPos pos;
  bool ok = true;

  // Every KV byte is read once per pass: its L2 lines are the first to go, which leaves the L2 to
  // the staged blocks the gather has just written (they are read one layer later).
  const uint64_t pol_stream = ptx::policy_evict_first();
  // What is the same in every layer of the launch: the own range, its resolved entries (copied to
  // shared memory as far as they fit) and the sequence its first block belongs to.
  const bool owner = blockIdx.x < p.used_cta;
  const uint32_t r0 = owner ? blockIdx.x * p.per : 0;
  const uint32_t r1 = owner ? min(r0 + p.per, p.total_blocks) : 0;
  const uint32_t ncache = min(r1 - r0, kOwnCache);
  const uint32_t own_chunk = min(p.own_chunk, 32u);
  for (uint32_t i = lane; i < ncache; i += 32) sm.own_res[i] = p.resolved[r0 + i];
  __syncwarp();
  Cursor first{kSentinel, 0, 0, 0};
  if (owner) {
    first.seq = p.blk_seq[r0];
    first.lo = p.blk_off[first.seq];
    first.hi = p.blk_off[first.seq + 1];
    first.nhi = p.blk_off[min(first.seq + 2, p.nseq)];
  }

  for (uint32_t li = p.li_begin; li < p.li_end && ok; ++li) {
    const uint32_t layer = p.first_layer + li;
    const uint8_t* local_layer = p.local_base + layer_offset(layer, p.layer_group, p.local_group_stride, p.local_layer_stride);
    const uint8_t* slot_base = p.staging_base + (layer % p.ring_slots) * p.slot_bytes;
    unsigned long long* rw = range_words(p, li);
    uint32_t* seq_count = seq_counts(p, li);
    uint32_t cur_seq = kSentinel, nruns = 0, nclaims = 0;
    Cursor cur = first;
    // A staged block of this layer may be read once the gather issued during the previous layer of
    // this launch (prefetch_distance layers ahead of it) has landed it (per-position ready flags
    // carrying the layer's epoch); the first layers' gathers precede the launch in stream order, as
    // does any gather the host skipped.
    const bool check_ready = li >= p.prefetch_distance && p.gather_target[li - p.prefetch_distance] == static_cast<int16_t>(layer);
    const uint32_t* ready = p.ready + static_cast<size_t>(layer % p.ring_slots) * p.ready_stride;
    const uint32_t epoch = p.epoch_base + li;
    // Layer-split placement: this layer's blocks all come from the ring slot, in flat order.
    const bool all_staged = layer >= p.split_layer;
    uint64_t waited_ns = 0;
    if (p.trace && lane == 0) {
      p.trace[li * p.trace_stride + kTraceWords * blockIdx.x] = ptx::global_timer_ns();
      p.trace[li * p.trace_stride + kTraceWords * blockIdx.x + 1] = 0;
    }
    // The partial buffer of this layer was last used part_buffers layers ago: its merges must be done.
    if (li >= p.part_buffers) {
      ok = wait_counter(layer_counters(p, li - p.part_buffers) + kCntMerged, p.nseq * p.Hq, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
    }

    // Moves the sequence cursor to the sequence that holds flat block `at`. Walking into the next
    // sequence costs no load that is waited for (its end was fetched when the cursor last moved);
    // anywhere else (a stolen claim) the sequence is looked up, `hint` being blk_seq[at] if the
    // caller has fetched it already.
    auto seek = [&](uint32_t at, uint32_t hint) {
      if (at >= cur.lo && at < cur.hi) return;
      if (at == cur.hi && cur.seq != kSentinel && cur.seq + 1 < p.nseq && at < cur.nhi) {
        ++cur.seq;
        cur.lo = cur.hi;
        cur.hi = cur.nhi;
        cur.nhi = p.blk_off[min(cur.seq + 2, p.nseq)];
        return;
      }
      cur.seq = hint != kSentinel ? hint : p.blk_seq[at];
      cur.lo = p.blk_off[cur.seq];
      cur.hi = p.blk_off[cur.seq + 1];
      cur.nhi = p.blk_off[min(cur.seq + 2, p.nseq)];
    };

    // Streams a claim of at most 32 flat blocks, one unit per sequence it touches. Lane j holds the
    // resolved entry of block c.b + j in `my` and, when have_rdy, the ready flag it read for it. A
    // unit of another sequence than the previous one starts a new run and takes the next partial
    // slot of its sequence.
    auto stream_claim = [&](Claim c, int32_t my, uint32_t rdy, bool have_rdy, uint32_t hint) {
      ++nclaims;
      if (!have_rdy) {
        rdy = epoch;
        if (check_ready && lane < c.e - c.b && my < 0) rdy = ptx::ld_acquire_gpu(ready + static_cast<uint32_t>(~my));
      }
      // The flags were read (acquired) one per lane and lane 0 issues the copies: the warp barrier
      // carries every lane's acquire over to it.
      __syncwarp();
      uint32_t at = c.b;
      while (at < c.e && ok) {
        seek(at, at == c.b ? hint : kSentinel);
        const uint32_t seq = cur.seq, seq_lo = cur.lo;
        const uint32_t ue = min(c.e, cur.hi);
        uint32_t slot_flag = 0;
        if (seq != cur_seq) {
          // With stealing, slots are handed out in arrival order; with the static split a
          // sequence's slot is the index of the range among those it touches, so the merge order,
          // and with it every bit of the result, is the same from run to run.
          uint32_t k = 0;
          if (p.allow_steal) {
            if (lane == 0) k = atomicAdd(&seq_count[seq], 1u);
            k = __shfl_sync(0xffffffffu, k, 0);
          } else {
            k = blockIdx.x - seq_lo / p.per;
          }
          const uint32_t base = p.seq_slot_base[seq], cap = p.seq_slot_base[seq + 1] - base;
          if (k >= cap) {  // cannot happen with the host's sizing; never write outside the slots
            if (lane == 0) ptx::report_status(p.status, kDevTimeout - 1);
            k = cap - 1;
          }
          slot_flag = (base + k) | kNewRun;
          cur_seq = seq;
          ++nruns;
        }
        if constexpr (!kGrouped) {
          // One block at a time, one stage per plane (5 to 8 KV heads: a plane is 20 to 32 KB).
          for (uint32_t blk = at; blk < ue && ok; ++blk) {
            const uint32_t j = blk - c.b;
            const int32_t e = __shfl_sync(0xffffffffu, my, j);
            if (check_ready && e < 0 && __shfl_sync(0xffffffffu, rdy, j) != epoch) {
              const uint64_t w0 = ptx::global_timer_ns();
              ok = wait_counter_eq(ready + static_cast<uint32_t>(~e), epoch, p.status);
              ok = __all_sync(0xffffffffu, ok);
              if (!ok) return;
              waited_ns += ptx::global_timer_ns() - w0;  // the attention sat waiting for prefetched data
            }
            const uint8_t* src = e >= 0 ? local_layer + static_cast<uint64_t>(e) * p.local_block_stride
                                        : slot_base + static_cast<uint64_t>(~e) * p.block_bytes;
  #pragma unroll
            for (uint32_t plane = 0; plane < 2; ++plane, ++hs, pos.advance(sm.na)) {
              const uint32_t stg = pos.stg;
              ok = ptx::mbar_wait(ptx::smem_u32(&sm.att_empty[stg]), pos.phase ^ 1u, p.status, kDevTimeout);
              ok = __all_sync(0xffffffffu, ok);
              if (!ok) return;
              const uint32_t full = ptx::smem_u32(&sm.att_full[stg]);
              if (lane == 0) {
                if (blk == at && plane == 0) {
                  sm.queue[nq % kQueue] = UnitDesc{seq, at - seq_lo, ue - seq_lo, slot_flag, li, 0, 0, 0};
                  ++nq;
                }
                // The stage was last read through the generic proxy (ldmatrix / ld.shared of the
                // consumer warps, ordered before this point by the empty barrier); the bulk copy writes
                // it through the asynchronous proxy. Without this fence the copy can overtake those
                // reads: seen as rare wrong V tiles in launches spanning several layers.
                ptx::fence_proxy_async();
                // A staged block was written by another CTA's bulk stores and announced through its
                // ready flag (release / acquire above): the bulk load reads it through the
                // asynchronous proxy, which the acquire alone does not cover.
                if (check_ready && e < 0 && plane == 0) ptx::fence_proxy_async_global();
                ptx::mbar_arrive_expect_tx(full, plane_bytes);
                // One request per plane: an SM streams far faster through few large bulk copies than
                // through many small ones.
                ptx::bulk_g2s_hint(ring + stg * hsb, src + plane * plane_bytes, plane_bytes, full, pol_stream);
              }
            }
          }
        } else {
          // Groups of V consecutive blocks of the unit share a stage: lane t takes block blk + t.
          for (uint32_t blk = at; blk < ue && ok; blk += V) {
            const uint32_t j0 = blk - c.b, np = min(V, ue - blk);
            const int32_t e = __shfl_sync(0xffffffffu, my, (j0 + lane) & 31u);
            const uint32_t r = __shfl_sync(0xffffffffu, rdy, (j0 + lane) & 31u);
            const bool mine = lane < np;
            const bool staged_blk = check_ready && mine && e < 0;
            if (__any_sync(0xffffffffu, staged_blk && r != epoch)) {
              const uint64_t w0 = ptx::global_timer_ns();
              bool landed = true;
              if (staged_blk && r != epoch) landed = wait_counter_eq(ready + static_cast<uint32_t>(~e), epoch, p.status);
              ok = __all_sync(0xffffffffu, landed);
              if (!ok) return;
              waited_ns += ptx::global_timer_ns() - w0;  // the attention sat waiting for prefetched data
            }
            const uint8_t* src = e >= 0 ? local_layer + static_cast<uint64_t>(e) * p.local_block_stride
                                        : slot_base + static_cast<uint64_t>(~e) * p.block_bytes;
            const uint32_t stg = pos.stg;
            ok = ptx::mbar_wait(ptx::smem_u32(&sm.att_empty[stg]), pos.phase ^ 1u, p.status, kDevTimeout);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) return;
            const uint32_t full = ptx::smem_u32(&sm.att_full[stg]);
            if (lane == 0) {
              if (blk == at) {
                sm.queue[nq % kQueue] = UnitDesc{seq, at - seq_lo, ue - seq_lo, slot_flag, li, 0, 0, 0};
                ++nq;
              }
              ptx::mbar_arrive_expect_tx(full, np * 2 * plane_bytes);
            }
            __syncwarp();
            if (mine) {
              // The stage was last read through the generic proxy (ldmatrix / ld.shared of the
              // consumer warps, ordered before this point by the empty barrier); the bulk copy writes
              // it through the asynchronous proxy: fence between the two.
              ptx::fence_proxy_async();
              // A staged block was written by another CTA's bulk stores and announced through its
              // ready flag (release / acquire above): the bulk load reads it through the
              // asynchronous proxy, which the acquire alone does not cover.
              if (staged_blk) ptx::fence_proxy_async_global();
              // One request per block: its K plane and V plane are neighbours in memory.
              ptx::bulk_g2s_hint(ring + stg * sbytes + lane * 2 * hsb, src, 2 * plane_bytes, full, pol_stream);
            }
            ++hs;
            pos.advance(sm.na);
          }
        }
        at = ue;
      }
    };

    auto range_len = [&](uint32_t c) { return min(p.per, p.total_blocks - c * p.per); };

    // Claims from the front of the own range are split in two: the atomic is issued before the
    // current claim is streamed and its answer is read afterwards, so its latency costs nothing.
    // Claims shrink as the range runs out (a quarter of what the last claim saw left), so that
    // little claimed-but-unprocessed work is hidden from thieves near the end.
    uint32_t own_left = 0xFFFFFFFFu, pend_want = 0;
    unsigned long long pend_old = 0;
    auto issue_front = [&]() {
      pend_want = min(own_chunk, max(1u, own_left / 4));
      if (lane == 0) pend_old = atomicAdd(&rw[blockIdx.x], static_cast<unsigned long long>(pend_want));
    };
    auto resolve_front = [&]() -> Claim {
      const unsigned long long old = __shfl_sync(0xffffffffu, pend_old, 0);
      const uint32_t f = static_cast<uint32_t>(old), b = static_cast<uint32_t>(old >> 32);
      const uint32_t len = r1 - r0;
      const uint32_t avail_end = b < len ? len - b : 0;
      if (f >= avail_end) return Claim{0, 0};
      const uint32_t e = min(f + pend_want, avail_end);
      own_left = avail_end - e;
      return Claim{r0 + f, r0 + e};
    };
    // Entries of n own blocks from flat block b on and, when they come from the shared-memory copy
    // (no load to wait for), their ready flags as well.
    auto prefetch_own = [&](uint32_t b, uint32_t n, int32_t& my, uint32_t& rdy, bool& have) {
      have = all_staged || b + n - r0 <= ncache;
      my = 0;
      if (lane < n) my = all_staged ? ~static_cast<int32_t>(b + lane) : have ? sm.own_res[b + lane - r0] : p.resolved[b + lane];
      rdy = epoch;
      if (have && check_ready && lane < n && my < 0) rdy = ptx::ld_acquire_gpu(ready + static_cast<uint32_t>(~my));
    };

    // Before the last layer of a launch a CTA that is out of own work does better to start on the
    // next layer than to compete for another range's last blocks: it steals only from ranges that
    // are well behind. In the last layer the floor is lower but not 1: stealing the last few blocks
    // of a range costs more (latency of the claim, one more partial and a longer merge at the very
    // end of the launch) than the slower SM needs to finish them.
    // Keeping all CTAs in step would cost more (every layer would end in a scramble for crumbs,
    // with the rings running dry) than the lead it takes away.
    const uint32_t steal_floor = max(li + 1 < p.num_layers ? p.steal_floor : p.steal_floor_last, 1u);
    auto steal = [&]() -> Claim {
      for (int attempt = 0; attempt < 16; ++attempt) {
        uint32_t best_rem = 0, best_v = 0;
        for (uint32_t v = lane; v < p.used_cta; v += 32) {
          const unsigned long long w = __ldcg(&rw[v]);
          const uint32_t f = static_cast<uint32_t>(w), b = static_cast<uint32_t>(w >> 32);
          const uint32_t len = range_len(v);
          const uint32_t rem = f + b < len ? len - f - b : 0;
          if (rem > best_rem) {
            best_rem = rem;
            best_v = v;
          }
        }
#pragma unroll
        for (int sh = 16; sh >= 1; sh >>= 1) {
          const uint32_t r = __shfl_xor_sync(0xffffffffu, best_rem, sh);
          const uint32_t vv = __shfl_xor_sync(0xffffffffu, best_v, sh);
          if (r > best_rem || (r == best_rem && vv < best_v)) {
            best_rem = r;
            best_v = vv;
          }
        }
        if (best_rem < steal_floor) return Claim{0, 0};
        const uint32_t amount = min(kStealMax, max(kStealMin, best_rem / 4));
        unsigned long long old = 0;
        if (lane == 0) old = atomicAdd(&rw[best_v], static_cast<unsigned long long>(amount) << 32);
        old = __shfl_sync(0xffffffffu, old, 0);
        const uint32_t f = static_cast<uint32_t>(old), b = static_cast<uint32_t>(old >> 32);
        const uint32_t len = range_len(best_v);
        const uint32_t hi = b < len ? len - b : 0;  // end of what was unclaimed before this steal
        const uint32_t lo_avail = min(f, hi);
        if (hi > lo_avail) {
          const uint32_t lo = hi - lo_avail > amount ? hi - amount : lo_avail;
          return Claim{best_v * p.per + lo, best_v * p.per + hi};
        }
      }
      return Claim{0, 0};
    };

    // Own range first. While a claim is streamed, the next claim's atomic is in flight and the
    // entries and ready flags of the blocks it will start with (it begins where this one ends)
    // are fetched, so a new claim does not leave the ring dry.
    if (owner) {
      issue_front();
      Claim c = resolve_front();
      int32_t my = 0;
      uint32_t rdy = 0;
      bool have = false;
      if (c.b < c.e) prefetch_own(c.b, c.e - c.b, my, rdy, have);
      while (c.b < c.e && ok) {
        issue_front();
        int32_t my_n = 0;
        uint32_t rdy_n = 0;
        bool have_n = false;
        prefetch_own(c.e, min(pend_want, r1 - c.e), my_n, rdy_n, have_n);
        stream_claim(c, my, rdy, have, kSentinel);
        c = resolve_front();
        my = my_n;
        rdy = rdy_n;
        have = have_n;
      }
    }
    // ... then the back of whichever range has most left (the next steal, its entries and its
    // sequence are fetched before the current one is streamed).
    if (ok && p.allow_steal) {
      Claim c = steal();
      while (c.b < c.e && ok) {
        const int32_t my = lane >= c.e - c.b ? 0 : all_staged ? ~static_cast<int32_t>(c.b + lane) : p.resolved[c.b + lane];
        const uint32_t hint = p.blk_seq[c.b];
        const Claim nxt = steal();
        // The last claim of a link of a chain: its copy thread takes no more units from here on, so
        // that its last copies land while the last blocks are attended to, not after them.
        if (nxt.b >= nxt.e && li + 1 == p.li_end && lane == 0) *reinterpret_cast<volatile uint32_t*>(sm.mq + kMqWind) = 1u;
        stream_claim(c, my, 0, false, hint);
        c = nxt;
      }
    }
    if (li + 1 == p.li_end && lane == 0) *reinterpret_cast<volatile uint32_t*>(sm.mq + kMqWind) = 1u;
    // A run left open at the end of a layer would be closed only by this CTA's next unit, and a CTA
    // may find nothing to claim in the following layers while every CTA waits for this layer's
    // merges: close it now with a descriptor that has no data behind it.
    if (ok && cur_seq != kSentinel && li + 1 < p.li_end) {
      const uint32_t stg = pos.stg;
      ok = ptx::mbar_wait(ptx::smem_u32(&sm.att_empty[stg]), pos.phase ^ 1u, p.status, kDevTimeout);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        if (lane == 0) {
          sm.queue[nq % kQueue] = UnitDesc{kFlush, 0, 0, 0, li, 0, 0, 0};
          ++nq;
          ptx::mbar_arrive(ptx::smem_u32(&sm.att_full[stg]));
        }
        ++hs;
        pos.advance(sm.na);
      }
    }
    if (p.trace && lane == 0) {
      p.trace[li * p.trace_stride + kTraceWords * blockIdx.x + 4] = ptx::global_timer_ns();
      uint32_t smid;
      asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
      p.trace[li * p.trace_stride + kTraceWords * blockIdx.x + 1] = waited_ns;
      p.trace[li * p.trace_stride + kTraceWords * blockIdx.x + 3] =
          smid | (static_cast<unsigned long long>(nruns) << 16) | (static_cast<unsigned long long>(nclaims) << 32);
    }
  }
  if (ok) {
    // End marker: a descriptor with no data behind it.
    const uint32_t stg = pos.stg;
    ok = ptx::mbar_wait(ptx::smem_u32(&sm.att_empty[stg]), pos.phase ^ 1u, p.status, kDevTimeout);
    ok = __all_sync(0xffffffffu, ok);
    if (ok && lane == 0) {
      sm.queue[nq % kQueue] = UnitDesc{kSentinel, 0, 0, 0, 0, 0, 0, 0};
      ptx::mbar_arrive(ptx::smem_u32(&sm.att_full[stg]));
    }
  }
  if (!ok) {
    // Bounded second chance for copies already issued, so that none lands after the CTA is gone.
    const uint32_t from = hs > sm.na ? hs - sm.na : 0;
    for (uint32_t k = from; k < hs; ++k)
      ptx::mbar_wait(ptx::smem_u32(&sm.att_full[k % sm.na]), (k / sm.na) & 1u, nullptr, 0);
  }
}

// ---------------------------------------------------------------------------------------------
// merge of a (layer, sequence, KV head): n partial slots starting at s0, all kG query heads at
// once. Lane groups of 32/kG lanes own one head each; a lane owns 4*kG consecutive dims.
// ---------------------------------------------------------------------------------------------
struct MergeCtx {
  const float* part_o;
  const float* part_ml;
  void* out;
  float* lse;
};

template <int kG>
__device__ __forceinline__ void merge_heads(const LayerParams& p, const MergeCtx& c, uint32_t seq, uint32_t g,
                                            uint32_t s0, uint32_t n) {
  constexpr uint32_t kLph = 32 / kG;  // lanes per head
  constexpr int kU = 16 / kG;         // partials in flight per round (16 float4 loads per lane)
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t hh = lane / kLph, j = lane % kLph;
  const uint32_t h = g * kG + hh;
  const float* mlh = c.part_ml + (static_cast<uint64_t>(s0) * p.Hq + h) * 4;
  const float* poh = c.part_o + (static_cast<uint64_t>(s0) * p.Hq + h) * kD + j * 4 * kG;
  const uint64_t ml_step = static_cast<uint64_t>(p.Hq) * 4, po_step = static_cast<uint64_t>(p.Hq) * kD;
  float M = kNegInf;
  for (uint32_t s = j; s < n; s += kLph) M = fmaxf(M, __ldcg(mlh + s * ml_step));
#pragma unroll
  for (uint32_t sh = 1; sh < kLph; sh <<= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, sh));
  float l = 0.f, le = 0.f;
  for (uint32_t s = j; s < n; s += kLph) {
    const float4 ml = __ldcg(reinterpret_cast<const float4*>(mlh + s * ml_step));
    const float w = ptx::exp2_approx(ml.x - M);
    l += ml.y * w;
    le += ml.z * w;
  }
#pragma unroll
  for (uint32_t sh = 1; sh < kLph; sh <<= 1) {
    l += __shfl_xor_sync(0xffffffffu, l, sh);
    le += __shfl_xor_sync(0xffffffffu, le, sh);
  }
  float4 acc[kG];
#pragma unroll
  for (int k = 0; k < kG; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
  for (uint32_t sb = 0; sb < n; sb += kU) {
    float4 v[kU][kG];
    float m[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const bool in = sb + u < n;
      m[u] = in ? __ldcg(mlh + (sb + u) * ml_step) : kNegInf;
#pragma unroll
      for (int k = 0; k < kG; ++k)
        v[u][k] = in ? __ldcg(reinterpret_cast<const float4*>(poh + (sb + u) * po_step + 4 * k)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      const float w = ptx::exp2_approx(m[u] - M);
#pragma unroll
      for (int k = 0; k < kG; ++k) {
        acc[k].x = fmaf(v[u][k].x, w, acc[k].x);
        acc[k].y = fmaf(v[u][k].y, w, acc[k].y);
        acc[k].z = fmaf(v[u][k].z, w, acc[k].z);
        acc[k].w = fmaf(v[u][k].w, w, acc[k].w);
      }
    }
  }
  const float inv = 1.f / l;
  uint2* dst = reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(c.out) + (static_cast<uint64_t>(seq) * p.Hq + h) * kD +
                                        j * 4 * kG);
#pragma unroll
  for (int k = 0; k < kG; ++k)
    dst[k] = make_uint2(ptx::pack_bf16x2(acc[k].x * inv, acc[k].y * inv), ptx::pack_bf16x2(acc[k].z * inv, acc[k].w * inv));
  if (c.lse && j == 0) c.lse[static_cast<uint64_t>(seq) * p.Hq + h] = (M + log2f(le)) * 0.6931471805599453f;
}

// The same for any group size, one head after the other (group sizes that are not a power of two).
__device__ __forceinline__ void merge_heads_serial(const LayerParams& p, const MergeCtx& c, uint32_t seq, uint32_t g,
                                                   uint32_t s0, uint32_t n) {
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t G = p.G;
  for (uint32_t hh = 0; hh < G; ++hh) {
    const uint32_t h = g * G + hh;
    const float* mlh = c.part_ml + (static_cast<uint64_t>(s0) * p.Hq + h) * 4;
    const float* poh = c.part_o + (static_cast<uint64_t>(s0) * p.Hq + h) * kD + lane * 4;
    const uint64_t ml_step = static_cast<uint64_t>(p.Hq) * 4, po_step = static_cast<uint64_t>(p.Hq) * kD;
    float M = kNegInf, l = 0.f, le = 0.f;
    for (uint32_t s = lane; s < n; s += 32) M = fmaxf(M, __ldcg(mlh + s * ml_step));
#pragma unroll
    for (int sh = 1; sh <= 16; sh <<= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, sh));
    for (uint32_t s = lane; s < n; s += 32) {
      const float4 ml = __ldcg(reinterpret_cast<const float4*>(mlh + s * ml_step));
      const float w = ptx::exp2_approx(ml.x - M);
      l += ml.y * w;
      le += ml.z * w;
    }
#pragma unroll
    for (int sh = 1; sh <= 16; sh <<= 1) {
      l += __shfl_xor_sync(0xffffffffu, l, sh);
      le += __shfl_xor_sync(0xffffffffu, le, sh);
    }
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (uint32_t s = 0; s < n; ++s) {
      const float w = ptx::exp2_approx(__ldcg(mlh + s * ml_step) - M);
      const float4 v = __ldcg(reinterpret_cast<const float4*>(poh + s * po_step));
      acc.x = fmaf(v.x, w, acc.x);
      acc.y = fmaf(v.y, w, acc.y);
      acc.z = fmaf(v.z, w, acc.z);
      acc.w = fmaf(v.w, w, acc.w);
    }
    const float inv = 1.f / l;
    uint2* dst = reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(c.out) + (static_cast<uint64_t>(seq) * p.Hq + h) * kD +
                                          lane * 4);
    *dst = make_uint2(ptx::pack_bf16x2(acc.x * inv, acc.y * inv), ptx::pack_bf16x2(acc.z * inv, acc.w * inv));
    if (c.lse && lane == 0) c.lse[static_cast<uint64_t>(seq) * p.Hq + h] = (M + log2f(le)) * 0.6931471805599453f;
  }
}

// sub = 0: all query heads of KV head g; sub = 8 + hh: query head hh of the group only.
__device__ __forceinline__ void merge_one(const LayerParams& p, uint32_t li, uint32_t seq, uint32_t g, uint32_t sub = 0) {
  MergeCtx c;
  c.part_o = part_o_of(p, li);
  c.part_ml = part_ml_of(p, li);
  c.out = static_cast<uint8_t*>(p.out) + li * p.io_layer_stride;
  c.lse = p.lse;
  // Every run of the sequence left one partial per consumer warp of the KV head: V per slot.
  const uint32_t V = blocks_per_stage(p.Hkv);
  const uint32_t s0 = p.seq_slot_base[seq] * V;
  const uint32_t n = (p.allow_steal ? __ldcg(&seq_counts(p, li)[seq])
                                    : (p.blk_off[seq + 1] - 1) / p.per - p.blk_off[seq] / p.per + 1) * V;
  switch (sub ? 0u : p.G) {
    case 0: merge_heads<1>(p, c, seq, g * p.G + (sub & 7u), s0, n); break;  // one head: 16 partials in flight
    case 1: merge_heads<1>(p, c, seq, g, s0, n); break;
    case 2: merge_heads<2>(p, c, seq, g, s0, n); break;
    case 4: merge_heads<4>(p, c, seq, g, s0, n); break;
    case 8: merge_heads<8>(p, c, seq, g, s0, n); break;
    default: merge_heads_serial(p, c, seq, g, s0, n); break;
  }
  __syncwarp();
  if ((threadIdx.x & 31u) == 0) {
    __threadfence();
    const uint32_t add = sub ? 1u : p.G;
    const uint32_t old = atomicAdd(layer_counters(p, li) + kCntMerged, add);
    // The merge that completes the layer announces its output to whoever computes the next layer's
    // queries from it (another stream of the caller, waiting on this word). Every merging warp
    // fenced before its addition and this one fences after it, so all rows are visible first.
    if (p.out_ready && old + add == p.nseq * p.Hq) {
      __threadfence_system();
      *reinterpret_cast<volatile uint32_t*>(p.out_ready + li) = p.out_ready_epoch;
    }
  }
}

// End of a run: count its blocks; the warp that completes a (sequence, KV head) queues the merge
// for the merge warp, and merges itself only when the queue is nearly full.
__device__ __forceinline__ void finish_run(const LayerParams& p, const Smem& sm, uint32_t li, uint32_t seq, uint32_t g,
                                           uint32_t blocks) {
  const uint32_t lane = threadIdx.x & 31u;
  __threadfence();
  __syncwarp();
  uint32_t old = 0;
  if (lane == 0) {
    old = atomicAdd(&merge_counts(p, li)[seq * p.Hkv + g], blocks);
    atomicAdd(layer_counters(p, li) + kCntAttnDone, blocks);
  }
  old = __shfl_sync(0xffffffffu, old, 0);
  if (old + blocks != p.blk_off[seq + 1] - p.blk_off[seq]) return;
  __threadfence();
  // A sequence cut into many partials (few, long sequences) has long merges, and those of its KV
  // heads all become due in this CTA at the same time: they are published for any CTA's merge warp
  // to take. Other merges are done in line when a layer is short (they are the critical path then:
  // the Hkv warps that finish a sequence together merge side by side), else they go to the CTA's
  // own queue, which costs no global atomics and does not hold up the ring.
  uint32_t n = 0;  // partials of the sequence; only looked up where merges can be shared at all
  if (p.shared_merges)
    n = p.allow_steal ? __ldcg(&seq_counts(p, li)[seq]) : (p.blk_off[seq + 1] - 1) / p.per - p.blk_off[seq] / p.per + 1;
  const bool shared = n >= kSharedMergeMin;
  if (p.merge_inline && !shared) {
    merge_one(p, li, seq, g);
    return;
  }
  volatile uint32_t* mq = sm.mq;
  uint32_t queued = 0;
  if (lane == 0) {
    if (shared) {
      // A very long merge goes out one query head at a time: more warps, and each keeps four times
      // as many partials in flight.
      const uint32_t parts = n >= kSplitMergeMin && p.G > 1 ? p.G : 1u;
      const uint32_t slot = atomicAdd(layer_counters(p, li) + kCntMergePub, parts);
      for (uint32_t hh = 0; hh < parts; ++hh)
        ptx::st_release_gpu(merge_requests(p, li) + slot + hh, 1u + 16u * (seq * p.Hkv + g) + (parts > 1 ? 8u + hh : 0u));
      queued = 1;
    } else if (static_cast<int32_t>(mq[kMqTail] - mq[kMqHead]) < static_cast<int32_t>(kMq - 8)) {
      // Up to Hkv warps may pass this check at once, hence the margin.
      const uint32_t t = atomicAdd(&sm.mq[kMqTail], 1u);
      const uint64_t t0 = ptx::global_timer_ns();
      bool slot_free = true;
      while (mq[t % kMq] != kMqEmpty) {
        if (ptx::global_timer_ns() - t0 > kWaitNs) {  // the merge warp is gone or stuck: report, merge in line
          ptx::report_status(p.status, kDevTimeout);
          slot_free = false;
          break;
        }
        __nanosleep(64);
      }
      // The ticket is spent either way; a merge warp that draws it finds the slot still holding the
      // older request (or nothing) and this warp does the merge itself.
      if (slot_free) {
        mq[t % kMq] = (li << 24) | (seq << 4) | g;
        queued = 1;
      }
    }
  }
  queued = __shfl_sync(0xffffffffu, queued, 0);
  if (!queued) merge_one(p, li, seq, g);
}

// Serves merge requests: first those of the CTA's own queue, then requests that any CTA has
// published for all. Run by the merge warp from the start and by each consumer warp once its
// streaming is over. A warp leaves when its CTA queues nothing more (a consumer warp: at once), its
// queue is empty and nothing published is left untaken; a published request is therefore taken at
// the latest by the warp that published it. Nobody waits for a request that is not yet published, so
// a CTA never stays behind for work of CTAs that are not resident yet.
// The CTA's own queue only (launches in which no merge is shared): every warp draws a ticket and
// waits for the request that gets it, or until no request can get it any more.
__device__ void merge_role_local(const LayerParams& p, const Smem& sm) {
  const uint32_t lane = threadIdx.x & 31u;
  volatile uint32_t* mq = sm.mq;
  for (;;) {
    uint32_t v = kMqEmpty;
    if (lane == 0) {
      const uint32_t h = atomicAdd(&sm.mq[kMqHead], 1u);
      const uint64_t t0 = ptx::global_timer_ns();
      for (;;) {
        v = mq[h % kMq];
        if (v != kMqEmpty) {
          mq[h % kMq] = kMqEmpty;
          break;
        }
        // No request will ever get this ticket once all consumers are done and the tail is behind it.
        if (mq[kMqDone] == p.Hkv * blocks_per_stage(p.Hkv) && static_cast<int32_t>(mq[kMqTail] - h) <= 0) break;
        if (ptx::global_timer_ns() - t0 > 2 * kWaitNs) break;  // a consumer that gave up never reports in
        __nanosleep(128);
      }
    }
    v = __shfl_sync(0xffffffffu, v, 0);
    if (v == kMqEmpty) return;
    __threadfence();
    merge_one(p, v >> 24, (v >> 4) & 0xFFFFFu, v & 15u);
  }
}

__device__ __forceinline__ void merge_role(const LayerParams& p, const Smem& sm, bool is_consumer) {
  if (!p.shared_merges) {
    if (!p.merge_inline) merge_role_local(p, sm);
    return;
  }
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t total = p.nseq * p.Hq;  // query heads to merge per layer
  volatile uint32_t* mq = sm.mq;
  uint32_t gli = p.li_begin, idle = 0;  // idle: looks at the own queue since the last request
  for (;;) {
    uint32_t v = kMqEmpty, sub = 0;  // a request in the CTA queue's format; one query head only?
    bool leave = false;
    if (lane == 0) {
      for (;;) {
        // 1. the CTA's own queue
        const uint32_t hd = mq[kMqHead];
        if (static_cast<int32_t>(mq[kMqTail] - hd) > 0) {
          if (atomicCAS(&sm.mq[kMqHead], hd, hd + 1) != hd) continue;
          const uint64_t t0 = ptx::global_timer_ns();
          while ((v = mq[hd % kMq]) == kMqEmpty) {  // its writer holds the ticket already
            if (ptx::global_timer_ns() - t0 > kWaitNs) {
              ptx::report_status(p.status, kDevTimeout);
              leave = true;
              break;
            }
          }
          if (!leave) mq[hd % kMq] = kMqEmpty;
          break;
        }
        // 2. requests published for all: the oldest layer not yet merged completely, and the next.
        // The own queue (shared memory) is looked at every 128 ns, the list in device memory at
        // once when the warp falls idle and then every eighth time, about once a microsecond.
        const bool look = (idle & 7u) == 0;
        ++idle;
        if (look)
          while (gli < p.li_end && __ldcg(layer_counters(p, gli) + kCntMerged) >= total) ++gli;
        for (uint32_t l = gli; look && l < p.li_end && l < gli + 2 && v == kMqEmpty && !leave; ++l) {
          uint32_t* cnt = layer_counters(p, l);
          uint32_t pub = __ldcg(cnt + kCntMergePub);
          uint32_t taken = __ldcg(cnt + kCntMergeTaken);
          if (taken < pub) {
            // Every idle merge warp of the GPU sees a new request within a microsecond or two. They
            // come forward in sixteen groups, 128 ns apart, so that a handful of them compete for
            // it and the rest find it gone without touching the counter.
            const uint32_t turn = (blockIdx.x + taken) & 15u;
            if (turn) {
              __nanosleep(turn * 128);
              pub = __ldcg(cnt + kCntMergePub);
              taken = __ldcg(cnt + kCntMergeTaken);
            }
          }
          while (taken < pub) {
            const uint32_t old = atomicCAS(cnt + kCntMergeTaken, taken, taken + 1);
            if (old != taken) {
              taken = old;
              continue;
            }
            // The publisher bumps the count before it writes the entry: a short, bounded wait.
            const uint32_t* e = merge_requests(p, l) + taken;
            uint32_t job;
            const uint64_t t0 = ptx::global_timer_ns();
            while ((job = ptx::ld_acquire_gpu(e)) == 0) {
              if (ptx::global_timer_ns() - t0 > kWaitNs) {
                ptx::report_status(p.status, kDevTimeout);
                leave = true;
                break;
              }
            }
            if (!leave) {
              const uint32_t sg = (job - 1) >> 4;
              v = (l << 24) | ((sg / p.Hkv) << 4) | (sg % p.Hkv);
              sub = (job - 1) & 15u;
            }
            break;
          }
        }
        if (v != kMqEmpty || leave) break;
        // 3. nothing to do: leave, or look again a little later
        if (is_consumer || mq[kMqDone] == p.Hkv * blocks_per_stage(p.Hkv)) {
          bool pending = static_cast<int32_t>(mq[kMqTail] - mq[kMqHead]) > 0;
          for (uint32_t l = gli; l < p.li_end && !pending; ++l) {
            const uint32_t* cnt = layer_counters(p, l);
            pending = __ldcg(cnt + kCntMergeTaken) < __ldcg(cnt + kCntMergePub);
          }
          if (!pending) {
            leave = true;
            break;
          }
          continue;
        }
        __nanosleep(128);
      }
    }
    leave = __shfl_sync(0xffffffffu, leave, 0);
    v = __shfl_sync(0xffffffffu, v, 0);
    sub = __shfl_sync(0xffffffffu, sub, 0);
    if (v != kMqEmpty) {
      idle = 0;
      __threadfence();
      merge_one(p, v >> 24, (v >> 4) & 0xFFFFFu, v & 15u, sub);
    }
    if (leave) return;
  }
}

// Waits for the next half-stage; false when the bounded wait expired anywhere in the warp.
__device__ __forceinline__ bool wait_stage(const LayerParams& p, const Smem& sm, const RingPos& pos) {
  const bool ok = ptx::mbar_wait(ptx::smem_u32(&sm.att_full[pos.stg]), pos.phase, p.status, kDevTimeout);
  return __all_sync(0xffffffffu, ok);
}

__device__ __forceinline__ void release_stage(const Smem& sm, const RingPos& pos) {
  __syncwarp();
  if ((threadIdx.x & 31u) == 0) ptx::mbar_arrive(ptx::smem_u32(&sm.att_empty[pos.stg]));
}

// ---------------------------------------------------------------------------------------------
// consumer warp (= KV head g), tensor-core tiles, one block per stage (5 to 8 KV heads)
// ---------------------------------------------------------------------------------------------
__device__ void consumer_mma_single(const LayerParams& p, const Smem& sm, uint32_t g) {
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t Hkv = p.Hkv, G = p.G;
  const uint32_t hsb = half_stage_bytes(Hkv), rb = row_bytes(Hkv);
  const uint32_t head_off = g * kD * 2;
  const uint32_t ring = ptx::smem_u32(sm.att_ring);
  const uint32_t n = lane >> 2, tig = lane & 3u, r0 = lane >> 2;
  uint32_t nunit = 0;
  RingPos pos;
  bool have_run = false;
  uint32_t run_seq = 0, run_slot = 0, run_blocks = 0, run_li = 0, len = 0, q_upto = 0;
  SegState st{kNegInf, kNegInf, 0.f, 0.f, 0.f, 0.f};
  uint32_t qf[8][2];
  float o[8][4];

  auto emit = [&]() {
#pragma unroll
    for (int sh = 4; sh <= 16; sh <<= 1) {
      st.l0 += __shfl_xor_sync(0xffffffffu, st.l0, sh);
      st.l1 += __shfl_xor_sync(0xffffffffu, st.l1, sh);
      st.e0 += __shfl_xor_sync(0xffffffffu, st.e0, sh);
      st.e1 += __shfl_xor_sync(0xffffffffu, st.e1, sh);
    }
    const uint32_t h0 = 2 * tig, h1 = h0 + 1;
    float* po = part_o_of(p, run_li) + (static_cast<uint64_t>(run_slot) * p.Hq + g * G) * kD;
    float* pml = part_ml_of(p, run_li) + (static_cast<uint64_t>(run_slot) * p.Hq + g * G) * 4;
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
      const uint32_t d = mt * 16 + r0;
      if (h0 < G) {
        po[h0 * kD + d] = o[mt][0];
        po[h0 * kD + d + 8] = o[mt][2];
      }
      if (h1 < G) {
        po[h1 * kD + d] = o[mt][1];
        po[h1 * kD + d + 8] = o[mt][3];
      }
    }
    if (r0 == 0) {
      if (h0 < G) *reinterpret_cast<float4*>(pml + h0 * 4) = make_float4(st.m0, st.l0, st.e0, 0.f);
      if (h1 < G) *reinterpret_cast<float4*>(pml + h1 * 4) = make_float4(st.m1, st.l1, st.e1, 0.f);
    }
    if (p.trace && g == 0 && lane == 0)
      p.trace[run_li * p.trace_stride + kTraceWords * blockIdx.x + 5] = ptx::global_timer_ns();
    finish_run(p, sm, run_li, run_seq, g, run_blocks);
  };

  for (;;) {
    if (!wait_stage(p, sm, pos)) return;
    const UnitDesc it = sm.queue[nunit % kQueue];
    if (it.seq_idx == kFlush) {
      if (have_run) emit();
      have_run = false;
      ++nunit;
      release_stage(sm, pos);
      pos.advance(sm.na);
      continue;
    }
    const bool end = it.seq_idx == kSentinel;
    if (end || (it.slot & kNewRun)) {
      if (have_run) emit();
      if (end) break;
      have_run = true;
      run_seq = it.seq_idx;
      run_slot = it.slot & ~kNewRun;
      run_li = it.layer;
      run_blocks = 0;
      len = p.lens[run_seq];
      st = SegState{kNegInf, kNegInf, 0.f, 0.f, 0.f, 0.f};
      if (run_li >= q_upto) {  // q may still be on its way: wait for this layer's rows (or chunk of layers)
        const uint64_t w0 = p.trace && p.q_ready ? ptx::global_timer_ns() : 0;
        if (p.q_ready && !wait_counter(p.q_ready + run_li / p.q_ready_layers, p.q_ready_epoch, p.status)) return;
        q_upto = p.q_ready ? (run_li / p.q_ready_layers + 1) * p.q_ready_layers : 0xFFFFFFFFu;
        if (p.trace && p.q_ready && g == 0 && lane == 0) {
          const uint64_t w1 = ptx::global_timer_ns();
          p.trace[run_li * p.trace_stride + kTraceWords * blockIdx.x + 6] = w1 - w0;
          p.trace[run_li * p.trace_stride + kTraceWords * blockIdx.x + 7] = w1;
        }
      }
      // Q^T fragments (B operand): head n = lane/4 of the group, dims ks*16 + 2*(lane%4) (+8).
      const __nv_bfloat16* qg =
          reinterpret_cast<const __nv_bfloat16*>(static_cast<const uint8_t*>(p.q) + run_li * p.io_layer_stride);
      const uint32_t* qrow =
          reinterpret_cast<const uint32_t*>(qg + (static_cast<uint64_t>(run_seq) * p.Hq + g * G + (n < G ? n : 0)) * kD);
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        qf[ks][0] = n < G ? __ldcg(qrow + ks * 8 + tig) : 0u;
        qf[ks][1] = n < G ? __ldcg(qrow + ks * 8 + tig + 4) : 0u;
      }
#pragma unroll
      for (int mt = 0; mt < 8; ++mt) o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f;
    }
    ++nunit;
    for (uint32_t b = it.blk_begin; b < it.blk_end; ++b) {
      if (b != it.blk_begin && !wait_stage(p, sm, pos)) return;
      const uint32_t valid = min(kT, len - b * kT);
      uint32_t pb0, pb1;
      float al0, al1;
      tile_mma_scores(ring + pos.stg * hsb + head_off, rb, valid, qf, p.scale_log2, st, pb0, pb1, al0, al1);
      release_stage(sm, pos);
      pos.advance(sm.na);
      if (!wait_stage(p, sm, pos)) return;
      tile_mma_pv(ring + pos.stg * hsb + head_off, rb, valid, pb0, pb1, al0, al1, o);
      release_stage(sm, pos);
      pos.advance(sm.na);
    }
    run_blocks += it.blk_end - it.blk_begin;
  }
}

// ---------------------------------------------------------------------------------------------
// consumer warp (= KV head = query head g), f32 tiles for G == 1, one block per stage (5 to 8 KV heads)
// ---------------------------------------------------------------------------------------------
__device__ void consumer_alu_single(const LayerParams& p, const Smem& sm, uint32_t g) {
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t Hkv = p.Hkv;
  const uint32_t hsb = half_stage_bytes(Hkv), rb = row_bytes(Hkv);
  const uint32_t head_off = g * kD * 2;
  const uint32_t half = lane & 1u;
  uint32_t nunit = 0;
  RingPos pos;
  bool have_run = false;
  uint32_t run_seq = 0, run_slot = 0, run_blocks = 0, run_li = 0, len = 0, q_upto = 0;
  SegState st{kNegInf, kNegInf, 0.f, 0.f, 0.f, 0.f};
  float qh[64];  // this lane's half (64 dims) of q as f32
  float o[4] = {0.f, 0.f, 0.f, 0.f};

  auto emit = [&]() __attribute__((always_inline)) {
#pragma unroll
    for (int sh = 1; sh <= 16; sh <<= 1) st.l0 += __shfl_xor_sync(0xffffffffu, st.l0, sh);
    float* po = part_o_of(p, run_li) + (static_cast<uint64_t>(run_slot) * p.Hq + g) * kD;
    *reinterpret_cast<float4*>(po + lane * 4) = make_float4(o[0], o[1], o[2], o[3]);
    if (lane == 0)
      *reinterpret_cast<float4*>(part_ml_of(p, run_li) + (static_cast<uint64_t>(run_slot) * p.Hq + g) * 4) =
          make_float4(st.m0, st.l0, st.l0, 0.f);
    if (p.trace && g == 0 && lane == 0)
      p.trace[run_li * p.trace_stride + kTraceWords * blockIdx.x + 5] = ptx::global_timer_ns();
    finish_run(p, sm, run_li, run_seq, g, run_blocks);
  };

  for (;;) {
    if (!wait_stage(p, sm, pos)) return;
    const UnitDesc it = sm.queue[nunit % kQueue];
    if (it.seq_idx == kFlush) {
      if (have_run) emit();
      have_run = false;
      ++nunit;
      release_stage(sm, pos);
      pos.advance(sm.na);
      continue;
    }
    const bool end = it.seq_idx == kSentinel;
    if (end || (it.slot & kNewRun)) {
      if (have_run) emit();
      if (end) break;
      have_run = true;
      run_seq = it.seq_idx;
      run_slot = it.slot & ~kNewRun;
      run_li = it.layer;
      run_blocks = 0;
      len = p.lens[run_seq];
      st = SegState{kNegInf, kNegInf, 0.f, 0.f, 0.f, 0.f};
      if (run_li >= q_upto) {  // q may still be on its way: wait for this layer's rows (or chunk of layers)
        const uint64_t w0 = p.trace && p.q_ready ? ptx::global_timer_ns() : 0;
        if (p.q_ready && !wait_counter(p.q_ready + run_li / p.q_ready_layers, p.q_ready_epoch, p.status)) return;
        q_upto = p.q_ready ? (run_li / p.q_ready_layers + 1) * p.q_ready_layers : 0xFFFFFFFFu;
        if (p.trace && p.q_ready && g == 0 && lane == 0) {
          const uint64_t w1 = ptx::global_timer_ns();
          p.trace[run_li * p.trace_stride + kTraceWords * blockIdx.x + 6] = w1 - w0;
          p.trace[run_li * p.trace_stride + kTraceWords * blockIdx.x + 7] = w1;
        }
      }
      const __nv_bfloat16* qg =
          reinterpret_cast<const __nv_bfloat16*>(static_cast<const uint8_t*>(p.q) + run_li * p.io_layer_stride);
      const uint4* qrow =
          reinterpret_cast<const uint4*>(qg + (static_cast<uint64_t>(run_seq) * p.Hq + g) * kD + half * 64);
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const uint4 v = __ldcg(qrow + c);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          qh[c * 8 + 2 * e] = __uint_as_float(w[e] << 16);
          qh[c * 8 + 2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
        }
      }
      o[0] = o[1] = o[2] = o[3] = 0.f;
    }
    ++nunit;
    for (uint32_t b = it.blk_begin; b < it.blk_end; ++b) {
      if (b != it.blk_begin && !wait_stage(p, sm, pos)) return;
      const uint32_t valid = min(kT, len - b * kT);
      float pw, al;
      tile_alu_scores(sm.att_ring + pos.stg * hsb + head_off, rb, valid, qh, p.scale_log2, st, pw, al);
      release_stage(sm, pos);
      pos.advance(sm.na);
      if (!wait_stage(p, sm, pos)) return;
      tile_alu_pv(sm.att_ring + pos.stg * hsb + head_off, rb, valid, pw, al, o);
      release_stage(sm, pos);
      pos.advance(sm.na);
    }
    run_blocks += it.blk_end - it.blk_begin;
  }
}

// End of a run for consumer warp v of KV head g, its partial written: warp 0 of the head counts the
// run's blocks (and merges or queues the merge when they complete a sequence) once the other warps
// of the head have written theirs. They process the same stages in step, so the wait is short; it
// is bounded like every other wait.
__device__ __forceinline__ void close_run(const LayerParams& p, const Smem& sm, uint32_t li, uint32_t seq, uint32_t g,
                                          uint32_t v, uint32_t blocks, uint32_t& runs_closed) {
  const uint32_t V = blocks_per_stage(p.Hkv);
  ++runs_closed;
  if (V == 1) {
    finish_run(p, sm, li, seq, g, blocks);
    return;
  }
  __threadfence();
  __syncwarp();
  if ((threadIdx.x & 31u) == 0) atomicAdd(&sm.head_runs[g], 1u);
  if (v != 0) return;
  volatile uint32_t* cnt = sm.head_runs + g;
  const uint32_t target = runs_closed * V;
  if (*cnt < target) {
    const uint64_t t0 = ptx::global_timer_ns();
    while (*cnt < target) {
      if (ptx::global_timer_ns() - t0 > kWaitNs) {
        ptx::report_status(p.status, kDevTimeout);
        break;
      }
    }
  }
  finish_run(p, sm, li, seq, g, blocks);
}

// ---------------------------------------------------------------------------------------------
// consumer warp v of KV head g, tensor-core tiles
// ---------------------------------------------------------------------------------------------
template <bool kGrouped>
__device__ void consumer_mma(const LayerParams& p, const Smem& sm, uint32_t g, uint32_t v) {
  if constexpr (!kGrouped) {
    consumer_mma_single(p, sm, g);
    return;
  }
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t Hkv = p.Hkv, G = p.G;
  const uint32_t hsb = half_stage_bytes(Hkv), rb = row_bytes(Hkv);
  const uint32_t V = kGrouped ? blocks_per_stage(Hkv) : 1u, sbytes = kGrouped ? stage_bytes(Hkv) : hsb;
  const uint32_t head_off = v * 2 * hsb + g * kD * 2;  // this warp's block of a stage (K plane, then V plane), this head's columns
  const uint32_t ring = ptx::smem_u32(sm.att_ring);
  const uint32_t n = lane >> 2, tig = lane & 3u, r0 = lane >> 2;
  uint32_t nunit = 0, runs_closed = 0;
  RingPos pos;
  bool have_run = false;
  uint32_t run_seq = 0, run_slot = 0, run_blocks = 0, run_li = 0, len = 0, q_upto = 0;
  SegState st{kNegInf, kNegInf, 0.f, 0.f, 0.f, 0.f};
  uint32_t qf[8][2];
  float o[8][4];

  auto emit = [&]() {
#pragma unroll
    for (int sh = 4; sh <= 16; sh <<= 1) {
      st.l0 += __shfl_xor_sync(0xffffffffu, st.l0, sh);
      st.l1 += __shfl_xor_sync(0xffffffffu, st.l1, sh);
      st.e0 += __shfl_xor_sync(0xffffffffu, st.e0, sh);
      st.e1 += __shfl_xor_sync(0xffffffffu, st.e1, sh);
    }
    const uint32_t h0 = 2 * tig, h1 = h0 + 1;
    float* po = part_o_of(p, run_li) + ((static_cast<uint64_t>(run_slot) * V + v) * p.Hq + g * G) * kD;
    float* pml = part_ml_of(p, run_li) + ((static_cast<uint64_t>(run_slot) * V + v) * p.Hq + g * G) * 4;
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
      const uint32_t d = mt * 16 + r0;
      if (h0 < G) {
        po[h0 * kD + d] = o[mt][0];
        po[h0 * kD + d + 8] = o[mt][2];
      }
      if (h1 < G) {
        po[h1 * kD + d] = o[mt][1];
        po[h1 * kD + d + 8] = o[mt][3];
      }
    }
    if (r0 == 0) {
      if (h0 < G) *reinterpret_cast<float4*>(pml + h0 * 4) = make_float4(st.m0, st.l0, st.e0, 0.f);
      if (h1 < G) *reinterpret_cast<float4*>(pml + h1 * 4) = make_float4(st.m1, st.l1, st.e1, 0.f);
    }
    if (p.trace && g == 0 && v == 0 && lane == 0)
      p.trace[run_li * p.trace_stride + kTraceWords * blockIdx.x + 5] = ptx::global_timer_ns();
    close_run(p, sm, run_li, run_seq, g, v, run_blocks, runs_closed);
  };

  for (;;) {
    if (!wait_stage(p, sm, pos)) return;
    const UnitDesc it = sm.queue[nunit % kQueue];
    if (it.seq_idx == kFlush) {
      if (have_run) emit();
      have_run = false;
      ++nunit;
      release_stage(sm, pos);
      pos.advance(sm.na);
      continue;
    }
    const bool end = it.seq_idx == kSentinel;
    if (end || (it.slot & kNewRun)) {
      if (have_run) emit();
      if (end) break;
      have_run = true;
      run_seq = it.seq_idx;
      run_slot = it.slot & ~kNewRun;
      run_li = it.layer;
      run_blocks = 0;
      len = p.lens[run_seq];
      st = SegState{kNegInf, kNegInf, 0.f, 0.f, 0.f, 0.f};
      if (run_li >= q_upto) {  // q may still be on its way: wait for this layer's rows (or chunk of layers)
        const uint64_t w0 = p.trace && p.q_ready ? ptx::global_timer_ns() : 0;
        if (p.q_ready && !wait_counter(p.q_ready + run_li / p.q_ready_layers, p.q_ready_epoch, p.status)) return;
        q_upto = p.q_ready ? (run_li / p.q_ready_layers + 1) * p.q_ready_layers : 0xFFFFFFFFu;
        if (p.trace && p.q_ready && g == 0 && v == 0 && lane == 0) {
          const uint64_t w1 = ptx::global_timer_ns();
          p.trace[run_li * p.trace_stride + kTraceWords * blockIdx.x + 6] = w1 - w0;
          p.trace[run_li * p.trace_stride + kTraceWords * blockIdx.x + 7] = w1;
        }
      }
      // Q^T fragments (B operand): head n = lane/4 of the group, dims ks*16 + 2*(lane%4) (+8).
      const __nv_bfloat16* qg =
          reinterpret_cast<const __nv_bfloat16*>(static_cast<const uint8_t*>(p.q) + run_li * p.io_layer_stride);
      const uint32_t* qrow =
          reinterpret_cast<const uint32_t*>(qg + (static_cast<uint64_t>(run_seq) * p.Hq + g * G + (n < G ? n : 0)) * kD);
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        qf[ks][0] = n < G ? __ldcg(qrow + ks * 8 + tig) : 0u;
        qf[ks][1] = n < G ? __ldcg(qrow + ks * 8 + tig + 4) : 0u;
      }
#pragma unroll
      for (int mt = 0; mt < 8; ++mt) o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f;
    }
    ++nunit;
    // Groups of V blocks share a stage; this warp takes block v of each group (none in a short one).
    for (uint32_t gb = it.blk_begin; gb < it.blk_end; gb += V) {
      if (gb != it.blk_begin && !wait_stage(p, sm, pos)) return;
      const uint32_t b = gb + v;
      const bool mine = !kGrouped || b < it.blk_end;
      const uint32_t valid = mine ? min(kT, len - b * kT) : 0u;
      uint32_t pb0 = 0, pb1 = 0;
      float al0 = 1.f, al1 = 1.f;
      if (mine) {
        tile_mma_scores(ring + pos.stg * sbytes + head_off, rb, valid, qf, p.scale_log2, st, pb0, pb1, al0, al1);
        tile_mma_pv(ring + pos.stg * sbytes + head_off + hsb, rb, valid, pb0, pb1, al0, al1, o);
      }
      release_stage(sm, pos);
      pos.advance(sm.na);
    }
    run_blocks += it.blk_end - it.blk_begin;  // the run's blocks, whichever warp of the head took them
  }
}

// ---------------------------------------------------------------------------------------------
// consumer warp v of KV head (= query head) g, f32 tiles for G == 1
// ---------------------------------------------------------------------------------------------
template <bool kGrouped>
__device__ void consumer_alu(const LayerParams& p, const Smem& sm, uint32_t g, uint32_t v) {
  if constexpr (!kGrouped) {
    consumer_alu_single(p, sm, g);
    return;
  }
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t Hkv = p.Hkv;
  const uint32_t hsb = half_stage_bytes(Hkv), rb = row_bytes(Hkv);
  const uint32_t V = kGrouped ? blocks_per_stage(Hkv) : 1u, sbytes = kGrouped ? stage_bytes(Hkv) : hsb;
  const uint32_t head_off = v * 2 * hsb + g * kD * 2;
  const uint32_t half = lane & 1u;
  uint32_t nunit = 0, runs_closed = 0;
  RingPos pos;
  bool have_run = false;
  uint32_t run_seq = 0, run_slot = 0, run_blocks = 0, run_li = 0, len = 0, q_upto = 0;
  SegState st{kNegInf, kNegInf, 0.f, 0.f, 0.f, 0.f};
  float qh[64];  // this lane's half (64 dims) of q as f32
  float o[4] = {0.f, 0.f, 0.f, 0.f};

  auto emit = [&]() __attribute__((always_inline)) {
#pragma unroll
    for (int sh = 1; sh <= 16; sh <<= 1) st.l0 += __shfl_xor_sync(0xffffffffu, st.l0, sh);
    float* po = part_o_of(p, run_li) + ((static_cast<uint64_t>(run_slot) * V + v) * p.Hq + g) * kD;
    *reinterpret_cast<float4*>(po + lane * 4) = make_float4(o[0], o[1], o[2], o[3]);
    if (lane == 0)
      *reinterpret_cast<float4*>(part_ml_of(p, run_li) + ((static_cast<uint64_t>(run_slot) * V + v) * p.Hq + g) * 4) =
          make_float4(st.m0, st.l0, st.l0, 0.f);
    if (p.trace && g == 0 && v == 0 && lane == 0)
      p.trace[run_li * p.trace_stride + kTraceWords * blockIdx.x + 5] = ptx::global_timer_ns();
    close_run(p, sm, run_li, run_seq, g, v, run_blocks, runs_closed);
  };

  for (;;) {
    if (!wait_stage(p, sm, pos)) return;
    const UnitDesc it = sm.queue[nunit % kQueue];
    if (it.seq_idx == kFlush) {
      if (have_run) emit();
      have_run = false;
      ++nunit;
      release_stage(sm, pos);
      pos.advance(sm.na);
      continue;
    }
    const bool end = it.seq_idx == kSentinel;
    if (end || (it.slot & kNewRun)) {
      if (have_run) emit();
      if (end) break;
      have_run = true;
      run_seq = it.seq_idx;
      run_slot = it.slot & ~kNewRun;
      run_li = it.layer;
      run_blocks = 0;
      len = p.lens[run_seq];
      st = SegState{kNegInf, kNegInf, 0.f, 0.f, 0.f, 0.f};
      if (run_li >= q_upto) {  // q may still be on its way: wait for this layer's rows (or chunk of layers)
        const uint64_t w0 = p.trace && p.q_ready ? ptx::global_timer_ns() : 0;
        if (p.q_ready && !wait_counter(p.q_ready + run_li / p.q_ready_layers, p.q_ready_epoch, p.status)) return;
        q_upto = p.q_ready ? (run_li / p.q_ready_layers + 1) * p.q_ready_layers : 0xFFFFFFFFu;
        if (p.trace && p.q_ready && g == 0 && v == 0 && lane == 0) {
          const uint64_t w1 = ptx::global_timer_ns();
          p.trace[run_li * p.trace_stride + kTraceWords * blockIdx.x + 6] = w1 - w0;
          p.trace[run_li * p.trace_stride + kTraceWords * blockIdx.x + 7] = w1;
        }
      }
      const __nv_bfloat16* qg =
          reinterpret_cast<const __nv_bfloat16*>(static_cast<const uint8_t*>(p.q) + run_li * p.io_layer_stride);
      const uint4* qrow =
          reinterpret_cast<const uint4*>(qg + (static_cast<uint64_t>(run_seq) * p.Hq + g) * kD + half * 64);
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const uint4 v = __ldcg(qrow + c);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          qh[c * 8 + 2 * e] = __uint_as_float(w[e] << 16);
          qh[c * 8 + 2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
        }
      }
      o[0] = o[1] = o[2] = o[3] = 0.f;
    }
    ++nunit;
    for (uint32_t gb = it.blk_begin; gb < it.blk_end; gb += V) {
      if (gb != it.blk_begin && !wait_stage(p, sm, pos)) return;
      const uint32_t b = gb + v;
      const bool mine = !kGrouped || b < it.blk_end;
      const uint32_t valid = mine ? min(kT, len - b * kT) : 0u;
      float pw = 0.f, al = 1.f;
      if (mine) {
        tile_alu_scores(sm.att_ring + pos.stg * sbytes + head_off, rb, valid, qh, p.scale_log2, st, pw, al);
        tile_alu_pv(sm.att_ring + pos.stg * sbytes + head_off + hsb, rb, valid, pw, al, o);
      }
      release_stage(sm, pos);
      pos.advance(sm.na);
    }
    run_blocks += it.blk_end - it.blk_begin;
  }
}

// ---------------------------------------------------------------------------------------------
// copy warp (one thread): the gathers issued during each layer of the launch
// ---------------------------------------------------------------------------------------------
__device__ void copy_role(const LayerParams& p, const Smem& sm) {
  const uint32_t ring = ptx::smem_u32(sm.copy_ring);
  const uint64_t pol = ptx::policy_evict_first();
  const uint64_t pol_keep = ptx::policy_evict_last();  // staged lines: wanted again within a layer's time
  const uint32_t loads_ahead = p.copy_loads_ahead == 4 ? 4u : kCopyLoadsDefault;
  uint32_t issued = 0, done = 0;  // pieces over the whole launch: stages and barrier phases continue
  bool ok = true;
  // Over a slow link only a few SMs copy: a handful of them keeps the link full, and an SM whose
  // copy engine is queued up with slow loads also delays its own attention loads.
  if (p.copy_sms && blockIdx.x >= p.copy_sms) return;
  // A link of a chain of launches must not keep its SM until the last unit of its layer's gather has
  // landed: its successor's CTA is waiting for that SM. Once the CTA's attention is done the copy
  // thread takes no more units (before the pass's last layer), and the copy thread of a link
  // starts with what is left of the gather of the layer before.
  const uint32_t li_first = p.chained && p.li_begin > 0 ? p.li_begin - 1 : p.li_begin;
  volatile uint32_t* winding_down = sm.mq + kMqWind;

  // Moves the copy units of one layer between the lent arena and the layer's ring slot, in one
  // direction: in (the gather: lent arena -> slot, landed positions announced through `ready`) or
  // out (the write-back of a swap-out pass: slot -> lent arena). Units are drawn by ticket from
  // `ticket`; returns the number of units this thread moved, all of them complete in global memory.
  // A unit is a run of blocks that are neighbours both in the lent arena and in the slot (one block
  // when blocks are 64 KB; up to 64 KB worth of smaller blocks that the slab allocator kept together).
  // `ready` / `epoch`: on the way in, the flags to set for what has landed (or null); on the way out,
  // the flags to wait for before a position is read (or null when the layer was staged before the
  // launch): the slot may still be filling, by other CTAs' copy threads, when a write-back starts.
  auto transfer = [&](uint32_t layer, bool out, uint32_t* ticket, const uint32_t* order, uint32_t count, uint32_t* ready,
                      uint32_t epoch, bool may_leave, uint32_t li_trace) -> uint32_t {
    uint8_t* lent_layer = const_cast<uint8_t*>(p.lent_base) + layer_offset(layer, p.layer_group, p.lent_group_stride, p.lent_layer_stride);
    uint8_t* slot = const_cast<uint8_t*>(p.staging_base) + (layer % p.ring_slots) * p.slot_bytes;
    uint32_t my_pos[16], my_n[16], my_end[16];  // this thread's most recent units: first position, blocks,
                                                // and this layer's piece count once the unit is fully issued
    uint32_t my_units = 0;                // units of this layer taken by this thread
    // Small blocks: tickets are drawn four at a time and the four units' descriptors fetched together.
    // A unit costs an atomic and two dependent loads before its first byte can be requested, about
    // 2.5 us that nothing overlaps; with 8 KB units that, not the bytes, was the gather's time.
    const uint32_t batch = p.block_bytes <= 16384 ? 4u : 1u;
    uint32_t bat_v[4], bat_e[4], bat_i = 0, bat_n = 0;
    uint32_t piece = 0, pieces = 0;       // equal: forces a unit fetch
    uint64_t unit_bytes = 0;
    const uint8_t* src_blk = nullptr;
    uint8_t* dst_blk = nullptr;
    const uint32_t first_piece = issued;  // this layer's pieces are [first_piece, issued)
    uint32_t reported = 0;                // units of this layer already reported as landed
    bool more = true;

    // Issues the load of the next 16 KB piece, pulling a new unit when the current one is used up.
    auto issue_next = [&]() -> bool {
      if (piece == pieces) {
        if (bat_i == bat_n) {
          if (may_leave && *winding_down) return false;
          const uint32_t first = atomicAdd(ticket, batch);
          if (first >= count) return false;
          bat_n = min(batch, count - first);
          bat_i = 0;
#pragma unroll
          for (uint32_t i = 0; i < 4; ++i)
            if (i < bat_n) bat_v[i] = order[first + i];
#pragma unroll
          for (uint32_t i = 0; i < 4; ++i)
            if (i < bat_n) bat_e[i] = static_cast<uint32_t>(p.copy_src[bat_v[i] & 0xFFFFFFu]);
        }
        const uint32_t v = bat_v[bat_i];
        const int32_t e = static_cast<int32_t>(bat_e[bat_i]);
        ++bat_i;
        const uint32_t pos = v & 0xFFFFFFu, n = (v >> 24) + 1u;
        if (out && ready) {
          for (uint32_t i = 0; i < n && ok; ++i) ok = wait_counter_eq(ready + pos + i, epoch, p.status);
          if (!ok) return false;
          ptx::fence_proxy_async_global();  // the flags were acquired; the bulk loads read through the asynchronous proxy
        }
        uint8_t* in_arena = lent_layer + static_cast<uint64_t>(static_cast<uint32_t>(~e)) * p.lent_block_stride;
        uint8_t* in_slot = slot + static_cast<uint64_t>(pos) * p.block_bytes;
        src_blk = out ? in_slot : in_arena;
        dst_blk = out ? in_arena : in_slot;
        unit_bytes = static_cast<uint64_t>(n) * p.block_bytes;
        pieces = static_cast<uint32_t>((unit_bytes + kCopyChunk - 1) / kCopyChunk);
        my_pos[my_units % 16] = pos;
        my_n[my_units % 16] = n;
        my_end[my_units % 16] = issued - first_piece + pieces;
        ++my_units;
        piece = 0;
      }
      const uint64_t off = static_cast<uint64_t>(piece) * kCopyChunk;
      const uint64_t left = unit_bytes - off;
      const uint32_t bytes = left < kCopyChunk ? static_cast<uint32_t>(left) : kCopyChunk;
      const uint32_t stg = issued % kNC;
      sm.copy_dst[stg] = dst_blk + off;
      sm.copy_len[stg] = bytes;
      const uint32_t bar = ptx::smem_u32(&sm.copy_full[stg]);
      ptx::mbar_arrive_expect_tx(bar, bytes);
      ptx::bulk_g2s_hint(ring + stg * kCopyChunk, src_blk + off, bytes, bar, pol);
      ++piece;
      ++issued;
      return true;
    };
    // Reports the units all of whose pieces are among the first `complete` stored pieces of this layer.
    auto report_landed = [&](uint32_t complete) {
      if (out || !ready || reported == my_units || my_end[reported % 16] > complete) return;
      // The units' bulk stores are complete (wait_group); they went through the asynchronous proxy,
      // the flags go through the generic one: order the two, then publish with a release.
      ptx::fence_proxy_async_global();
      for (; reported < my_units && my_end[reported % 16] <= complete; ++reported)
        for (uint32_t i = 0; i < my_n[reported % 16]; ++i) ptx::st_release_gpu(ready + my_pos[reported % 16] + i, epoch);
    };

    while (issued - done < loads_ahead && more) more = issue_next();
    while (done < issued) {
      const uint32_t stg = done % kNC;
      ok = ptx::mbar_wait(ptx::smem_u32(&sm.copy_full[stg]), (done / kNC) & 1u, p.status, kDevTimeout);
      if (!ok) break;
      // (what goes out to the lent arena is not read again before the next pass)
      ptx::bulk_s2g_hint(sm.copy_dst[stg], ring + stg * kCopyChunk, sm.copy_len[stg], out ? pol : pol_keep);
      ptx::bulk_commit();
      ++done;
      // All but the newest kStoresOpen stores are complete after this wait: their stages may be
      // refilled and their bytes are in global memory. (Three open stores measured 4 % slower.)
      ptx::bulk_wait_all<kStoresOpen>();
      const uint32_t stored = done - first_piece;
      report_landed(stored > kStoresOpen ? stored - kStoresOpen : 0);
      if (more) more = issue_next();
    }
    ptx::bulk_wait_all<0>();
    if (ok) report_landed(done - first_piece);
    if (p.trace && !out) p.trace[li_trace * p.trace_stride + kTraceWords * blockIdx.x + 2] = ptx::global_timer_ns();
    return my_units;
  };

  for (uint32_t li = li_first; li < p.li_end && ok; ++li) {
    const uint32_t layer = p.first_layer + li;
    const int32_t target = p.gather_target[li];
    if (target >= 0 && p.copy_n != 0) {
      const bool may_leave = p.chained && li >= p.li_begin && li + 1 < p.num_layers;
      // The target's ring slot was last read by an earlier layer of this launch: wait for its attention
      // and, in a swap-out pass, for its write-back (the slot's content is then safe in the lent arena).
      const int32_t after = p.gather_after[li];
      if (after >= 0) {
        uint32_t* cnt = layer_counters(p, static_cast<uint32_t>(after) - p.first_layer);
        ok = wait_counter(cnt + kCntAttnDone, p.total_blocks * p.Hkv, p.status);
        if (ok && p.writeback && static_cast<uint32_t>(after) >= p.writeback_from) ok = wait_counter(cnt + kCntWbDone, p.wb_n, p.status);
        if (!ok) break;
      }
      // A layer of the next pass (gathered at the end of this one) is read from the lent arena only
      // after this pass has written it back.
      if (p.writeback && static_cast<uint32_t>(target) < layer && static_cast<uint32_t>(target) >= p.writeback_from &&
          static_cast<uint32_t>(target) >= p.first_layer) {
        ok = wait_counter(layer_counters(p, static_cast<uint32_t>(target) - p.first_layer) + kCntWbDone, p.wb_n, p.status);
        if (!ok) break;
      }
      // (the waits above were acquires of counters that bulk copies' completions were released to)
      if (p.writeback) ptx::fence_proxy_async_global();
      // A landed block is announced by writing the target layer's epoch to its position's ready flag
      // (only when the target is attended to later in this launch).
      const bool report = static_cast<uint32_t>(target) > layer && static_cast<uint32_t>(target) < p.first_layer + p.num_layers;
      uint32_t* ready = report ? p.ready + static_cast<size_t>(static_cast<uint32_t>(target) % p.ring_slots) * p.ready_stride : nullptr;
      const uint32_t epoch = p.epoch_base + (static_cast<uint32_t>(target) - p.first_layer);
      transfer(static_cast<uint32_t>(target), false, layer_counters(p, li) + kCntCopyTicket, p.copy_order, p.copy_n, ready, epoch,
               may_leave, li);
      if (!ok) break;
    }
    // Swap-out pass (Section 2.3: what comes in is matched by what goes out): while this layer is attended
    // to, its staged blocks, rows appended since they were fetched included, go back to the lent
    // arena. The attention only reads the slot; nothing writes it before the gather that waits above.
    if (p.writeback && li >= p.li_begin && layer >= p.writeback_from) {
      // (the same test as the attention's: was this layer gathered inside this launch?)
      const bool filling = li >= p.prefetch_distance && p.gather_target[li - p.prefetch_distance] == static_cast<int16_t>(layer);
      uint32_t* landed = filling ? p.ready + static_cast<size_t>(layer % p.ring_slots) * p.ready_stride : nullptr;
      const uint32_t moved = transfer(layer, true, layer_counters(p, li) + kCntWbTicket, p.wb_order, p.wb_n, landed,
                                      p.epoch_base + li, false, li);
      if (!ok) break;
      if (moved) {
        // every store of this thread is complete (bulk_wait_all<0>); they went through the
        // asynchronous proxy, the counter goes through the generic one
        ptx::fence_proxy_async_global();
        __threadfence();
        atomicAdd(layer_counters(p, li) + kCntWbDone, moved);
      }
    }
  }
  if (!ok) {
    for (uint32_t k = done; k < issued; ++k)
      ptx::mbar_wait(ptx::smem_u32(&sm.copy_full[k % kNC]), (k / kNC) & 1u, nullptr, 0);
    ptx::bulk_wait_all<0>();
  }
}

template <bool kMma, bool kGrouped>
__global__ void __launch_bounds__(352, 1) slice_layer_kernel(const LayerParams p) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  bool gathers = false;
  if (p.copy_n)
    for (uint32_t li = p.chained && p.li_begin > 0 ? p.li_begin - 1 : p.li_begin; li < p.li_end; ++li)
      gathers |= p.gather_target[li] >= 0 || p.writeback != 0;
  // A link of a chain of launches: the next link may start as soon as every CTA of this one has (it
  // takes the SMs that CTAs of this link leave, and waits for nothing but flags and counters).
  if (p.chained) ptx::launch_dependents();
  const Smem sm = carve(smem_raw, p.Hkv, gathers);
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
  const uint32_t ncons = p.Hkv * blocks_per_stage(p.Hkv);  // consumer warps: blocks_per_stage per KV head
  if (threadIdx.x == 0) {
    for (uint32_t s = 0; s < sm.na; ++s) {
      ptx::mbar_init(ptx::smem_u32(&sm.att_full[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&sm.att_empty[s]), ncons);
    }
    for (uint32_t g = 0; g < 8; ++g) sm.head_runs[g] = 0;
    for (int s = 0; s < kNC; ++s) ptx::mbar_init(ptx::smem_u32(&sm.copy_full[s]), 1);
    for (uint32_t s = 0; s < kMq; ++s) sm.mq[s] = kMqEmpty;
    sm.mq[kMqTail] = sm.mq[kMqHead] = sm.mq[kMqDone] = sm.mq[kMqWind] = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  if (warp < ncons) {
    if constexpr (kMma)
      consumer_mma<kGrouped>(p, sm, warp % p.Hkv, warp / p.Hkv);
    else
      consumer_alu<kGrouped>(p, sm, warp % p.Hkv, warp / p.Hkv);
    __syncwarp();
    if (lane == 0) {
      __threadfence_block();
      atomicAdd(&sm.mq[kMqDone], 1u);  // this consumer warp queues no more merges
    }
    __syncwarp();
    merge_role(p, sm, true);
  } else if (warp == ncons) {
    producer_role<kGrouped>(p, sm);
  } else if (warp == ncons + 1) {
    if (lane == 0) {
      copy_role(p, sm);
      // Links end in order: the stream's next operation, which waits for the last link only, then
      // finds the whole chain complete (no wait at all in a kernel that is no dependent).
      if (p.chained) ptx::grid_dependency_wait();
    }
  } else if (warp == ncons + 2) {
    merge_role(p, sm, false);
  }
}

// One CTA per (sequence, layer): the new token's K and V rows go to the home block and the staged copy.
__global__ void __launch_bounds__(128) append_kv_kernel(const AppendParams p) {
  const uint32_t i = blockIdx.x;
  if (i >= p.nseq) return;
  const uint32_t len = p.lens[i];
  if (len == 0) return;
  const uint32_t r = (len - 1) % p.block_tokens;
  const int32_t e = p.home_entry[i];
  const uint32_t y = blockIdx.y;  // layer within the launch
  const uint32_t layer = p.first_layer + y;
  const bool lent_home = p.split_layer == 0xFFFFFFFFu ? e < 0 : layer >= p.split_layer;
  const uint32_t id = e >= 0 ? static_cast<uint32_t>(e) : static_cast<uint32_t>(~e);
  uint8_t* home = !lent_home ? p.local_base + layer_offset(layer, p.layer_group, p.local_group_stride, p.local_layer_stride) +
                               static_cast<uint64_t>(id) * p.local_block_stride
                         : p.lent_base + layer_offset(layer, p.layer_group, p.lent_group_stride, p.lent_layer_stride) +
                               static_cast<uint64_t>(id) * p.lent_block_stride;
  const int32_t sp = p.stage_pos[i];
  uint8_t* slot = p.slot_base;
  if (p.num_layers > 1)
    slot = (p.staged_mask[y >> 5] >> (y & 31u)) & 1u ? p.staging_base + ((p.first_layer + y) % p.ring_slots) * p.slot_bytes : nullptr;
  uint8_t* staged = (slot && sp >= 0) ? slot + static_cast<uint64_t>(sp) * p.block_bytes : nullptr;
  const uint32_t plane = p.block_tokens * p.row_bytes;
  const uint32_t vecs = p.row_bytes >> 4;
  const uint4* ks = reinterpret_cast<const uint4*>(static_cast<const uint8_t*>(p.k_new) + y * p.io_layer_stride + static_cast<uint64_t>(i) * p.row_bytes);
  const uint4* vs = reinterpret_cast<const uint4*>(static_cast<const uint8_t*>(p.v_new) + y * p.io_layer_stride + static_cast<uint64_t>(i) * p.row_bytes);
  for (uint32_t v = threadIdx.x; v < vecs; v += blockDim.x) {
    const uint4 kv = ks[v], vv = vs[v];
    const uint32_t w = (v & ~7u) | ((v & 7u) ^ (r & 7u));  // the block format's swizzle of 16-byte units
    if (!(staged && p.staged_only)) {
      reinterpret_cast<uint4*>(home + r * p.row_bytes)[w] = kv;
      reinterpret_cast<uint4*>(home + plane + r * p.row_bytes)[w] = vv;
    }
    if (staged) {
      reinterpret_cast<uint4*>(staged + r * p.row_bytes)[w] = kv;
      reinterpret_cast<uint4*>(staged + plane + r * p.row_bytes)[w] = vv;
    }
  }
}

// One thread stands in for the rest of a decoder whose work between two attention layers takes no
// time: it releases the queries of layer 0 and then, as soon as the output of layer l is announced,
// those of layer l+1. It gives up at the first bounded wait that runs out.
__global__ void __launch_bounds__(32) step_relay_kernel(const uint32_t* out_ready, uint32_t* q_ready, uint32_t layers,
                                                        uint32_t epoch, int* status) {
  if (threadIdx.x != 0) return;
  ptx::st_release_gpu(q_ready, epoch);
  for (uint32_t l = 0; l + 1 < layers; ++l) {
    if (!wait_counter(out_ready + l, epoch, status)) return;
    ptx::st_release_gpu(q_ready + l + 1, epoch);
  }
}

}  // namespace

cudaError_t launch_step_relay(const uint32_t* out_ready, uint32_t* q_ready, uint32_t layers, uint32_t epoch, int* status,
                              cudaStream_t stream) {
  step_relay_kernel<<<1, 32, 0, stream>>>(out_ready, q_ready, layers, epoch, status);
  return cudaGetLastError();
}

size_t layer_smem_bytes(uint32_t Hkv) {
  if (Hkv == 0 || Hkv > 8) return 0;
  return smem_total(Hkv);
}

namespace {
// The four instantiations: tensor-core or f32 tiles, one block per stage (5..8 KV heads) or groups of
// 8 / Hkv blocks per stage (1 to 4 KV heads).
const void* layer_kernel_for(uint32_t Hkv, uint32_t G) {
  const bool grouped = blocks_per_stage(Hkv) > 1;
  if (G == 1)
    return grouped ? reinterpret_cast<const void*>(slice_layer_kernel<false, true>)
                   : reinterpret_cast<const void*>(slice_layer_kernel<false, false>);
  return grouped ? reinterpret_cast<const void*>(slice_layer_kernel<true, true>)
                 : reinterpret_cast<const void*>(slice_layer_kernel<true, false>);
}
}  // namespace

cudaError_t layer_setup() {
  const int smem = static_cast<int>(layer_smem_bytes(8));
  for (uint32_t Hkv : {8u, 1u})
    for (uint32_t G : {1u, 2u}) {
      cudaError_t e = cudaFuncSetAttribute(layer_kernel_for(Hkv, G), cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
      if (e != cudaSuccess) return e;
      // A launch that gathers nothing takes 100 KB; the SM keeps its largest shared-memory split all
      // the same, so that a CTA of the gather kernel can join it (and leave) without the split changing.
      e = cudaFuncSetAttribute(layer_kernel_for(Hkv, G), cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
      if (e != cudaSuccess) return e;
    }
  return cudaSuccess;
}

cudaError_t launch_layer(const LayerParams& p, cudaStream_t stream) {
  // The same test as in the kernel: does any layer this launch works on gather?
  bool gathers = false;
  if (p.copy_n)
    for (uint32_t li = p.chained && p.li_begin > 0 ? p.li_begin - 1 : p.li_begin; li < p.li_end; ++li)
      gathers |= p.gather_target[li] >= 0 || p.writeback != 0;
  const size_t smem = smem_needed(p.Hkv, gathers);
  const unsigned threads = (p.Hkv * blocks_per_stage(p.Hkv) + 3) * 32;
  void* args[] = {const_cast<LayerParams*>(&p)};
  const void* fn = layer_kernel_for(p.Hkv, p.G);
  // CTAs of a launch that spans several layers wait for one another: all of them must be resident.
  if (p.li_end - p.li_begin > 1) return cudaLaunchCooperativeKernel(fn, dim3(p.ncta), dim3(threads), args, smem, stream);
  if (p.chained == 2) {
    // A later link of a chain: it may start while its predecessor still runs.
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(p.ncta);
    cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelExC(&cfg, fn, args);
  }
  return cudaLaunchKernel(fn, dim3(p.ncta), dim3(threads), args, smem, stream);
}

cudaError_t launch_append(const AppendParams& p, cudaStream_t stream) {
  if (p.nseq == 0) return cudaSuccess;
  append_kv_kernel<<<dim3(p.nseq, p.num_layers ? p.num_layers : 1), 128, 0, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace ema
