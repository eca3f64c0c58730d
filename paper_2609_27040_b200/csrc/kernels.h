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

// Device counters of one layer-kernel launch; the whole block must be zero when the kernel
// starts. Layout in uint32 words:
//   [0, 16)                         launch words: [1] = next copy unit
//   [16, 16 + 2*ncta)               one 64-bit claim word per CTA range: blocks claimed from the front
//                                   (low half, by the owner) and from the back (high half, by thieves)
//   [.., + nseq)                    partial slots handed out per sequence
//   [.., + nseq*Hkv)                blocks finished per (sequence, KV head)
constexpr uint32_t kLaunchCounters = 16;
inline size_t layer_counter_words(uint32_t ncta, uint32_t nseq, uint32_t Hkv) {
  return kLaunchCounters + 2 * static_cast<size_t>(ncta) + nseq + static_cast<size_t>(nseq) * Hkv;
}

struct LayerParams {
  // attention of one layer over one batch
  const uint8_t* local_layer;   // base of this layer's local arena
  uint64_t local_block_stride;
  const uint8_t* slot_base;     // ring slot that holds this layer's staged blocks
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
  const void* q;                // [nseq][Hq][128] bf16
  void* out;                    // [nseq][Hq][128] bf16
  float* lse;                   // [nseq][Hq] or NULL
  float* part_o;                // [slots][Hq][128] unnormalised partial outputs
  float* part_ml;               // [slots][Hq][4]   max (log2 domain), sum as used, exact sum, pad
  uint32_t* counters;           // layer_counter_words(), zeroed before the launch
  uint32_t nseq, ncta;
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
// part_ml, counters of p are ignored). static_scratch_needed() > static_scratch_bytes() must be
// rejected by the caller.
size_t static_scratch_bytes();
size_t static_scratch_needed(uint32_t slots, uint32_t Hq, uint32_t nseq, uint32_t Hkv, uint32_t ncta);
cudaError_t launch_layer_static(LayerParams p, uint32_t slots, cudaStream_t stream);

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
