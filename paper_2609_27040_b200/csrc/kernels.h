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
struct CopyDesc {
  const uint8_t* src_base[2];
  uint8_t* dst_base[2];
  uint64_t src_block_stride[2];
  uint64_t dst_block_stride[2];
  uint64_t src_layer_stride[2];
  uint64_t dst_layer_stride[2];
  const int32_t* src_entry;
  const int32_t* dst_entry;
  uint32_t n;
  uint32_t nlayers;
  uint64_t block_bytes;  // multiple of 16
  int* status;
  unsigned long long* trace;  // optional [grid][2] start/end %globaltimer per CTA (profiling)
};

enum CopyKind : uint32_t { kCopyDefault = 0, kCopyVector = 1, kCopyBulk = 2 };

// Launches one copy kernel on `stream`. ctas == 0 picks a default grid. Returns the CUDA error.
cudaError_t launch_copy(const CopyDesc& d, uint32_t kind, uint32_t ctas, int num_sms, cudaStream_t stream);

// One unit of attention work: blocks [blk_begin, blk_end) of batch position seq_idx. Its partial
// result goes to slot seg_id (slots of one sequence are contiguous).
struct WorkItem {
  uint32_t seq_idx;
  uint32_t blk_begin;
  uint32_t blk_end;
  uint32_t flat_begin;  // index of blk_begin in the batch's flat resolved table
  uint32_t seg_id;
  uint32_t pad[3];
};

// Device counters of one layer-kernel launch (must be zero when the kernel starts).
//   [0] next dynamic attention item, [1] next copy unit; merge_cnt[seq * Hkv + g] counts the
//   finished segments of a (sequence, KV head) and is reset by the warp that merges.
constexpr uint32_t kLaunchCounters = 16;  // uint32 words reserved per launch for [0], [1]

struct LayerParams {
  // attention of one layer over one batch
  const uint8_t* local_layer;   // base of this layer's local arena
  uint64_t local_block_stride;
  const uint8_t* slot_base;     // ring slot that holds this layer's staged blocks
  uint64_t block_bytes;
  const int32_t* resolved;      // flat resolved table of the batch
  const uint32_t* lens;         // [nseq] tokens
  const WorkItem* items;        // static items grouped by CTA, then the dynamic items
  const uint32_t* cta_item_off; // [ncta + 1] static items of each CTA
  uint32_t dyn_begin, n_dyn;    // dynamic items: items[dyn_begin .. dyn_begin + n_dyn)
  const uint32_t* seq_seg_off;  // [nseq + 1] partial slots of each sequence
  const void* q;                // [nseq][Hq][128] bf16
  void* out;                    // [nseq][Hq][128] bf16
  float* lse;                   // [nseq][Hq] or NULL
  float* part_o;                // [nsegs][Hq][128] unnormalised partial outputs
  float* part_ml;               // [nsegs][Hq][4]   max (log2 domain), sum as used, exact sum, pad
  uint32_t* launch_cnt;         // [kLaunchCounters] zeroed before the launch
  uint32_t* merge_cnt;          // [nseq * Hkv] zero between launches
  uint32_t nseq, nsegs, ncta;
  uint32_t Hq, Hkv, G;
  float scale_log2;             // sm_scale * log2(e)
  uint32_t has_attention;       // 0: copy work only
  // optional gather of another layer's lent blocks in the same launch (copy.n == 0: none)
  CopyDesc copy;
  int* status;
  unsigned long long* trace;    // optional [ncta][4]: start, attention end, copy end, SM id
};

// Shared memory the layer kernel needs for Hkv KV heads (0 if unsupported).
size_t layer_smem_bytes(uint32_t Hkv);
// One-time per-process opt-in to large dynamic shared memory.
cudaError_t layer_setup();
// Attention (+ fused gather, + merge by the last-arriving warp): ONE launch.
cudaError_t launch_layer(const LayerParams& p, cudaStream_t stream);

// noalloc.cu: the same launch with partials and counters in a static device array (part_o,
// part_ml, launch_cnt, merge_cnt of p are ignored). static_scratch_needed() >
// static_scratch_bytes() must be rejected by the caller.
size_t static_scratch_bytes();
size_t static_scratch_needed(uint32_t nsegs, uint32_t Hq, uint32_t nseq, uint32_t Hkv);
cudaError_t launch_layer_static(LayerParams p, cudaStream_t stream);

struct AppendParams {
  uint8_t* local_layer;        // this layer's local arena
  uint64_t local_block_stride;
  uint8_t* lent_layer;         // this layer's lent arena
  uint64_t lent_block_stride;
  uint8_t* slot_base;          // ring slot holding the layer, or NULL when not staged
  uint64_t block_bytes;
  const int32_t* home_entry;   // [nseq] table entry of the block holding token len-1
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
