// copy_kernels.cu — block-table-indexed block copies: the prefetch gather (lent arena -> staging
// ring slot), the write-back scatter, and the reclaim migration (lent -> local / lower lent ids,
// all layers). Two kernels over the same descriptor:
//   * vector kernel: 128-bit coalesced loads/stores through registers; needs no shared memory, so
//     its CTAs can share an SM with the attention kernel while layers are pipelined;
//   * bulk ring kernel: one thread per CTA drives untiled TMA bulk copies global -> shared ->
//     global through a shared-memory ring; no SM lanes touch the data.
// HBM-bound: algorithmic bytes = 2 * block_bytes per block per layer (read + write).
#include "kernels.h"
#include "ptx.cuh"

namespace ema {

namespace {

constexpr uint32_t kVecThreads = 256;
constexpr uint32_t kVecPerThread = 4;
constexpr uint32_t kPieceVecs = kVecThreads * kVecPerThread;  // 1024 x 16 B = 16 KB per piece

__device__ __forceinline__ const uint8_t* src_addr(const CopyDesc& d, uint32_t i, uint32_t layer) {
  int32_t e = d.src_entry ? d.src_entry[i] : static_cast<int32_t>(i);
  int t = e < 0;
  uint32_t id = t ? static_cast<uint32_t>(~e) : static_cast<uint32_t>(e);
  const uint64_t lo = d.layer_group > 1 ? layer_offset(layer, d.layer_group, d.src_group_stride[t], d.src_layer_stride[t])
                                        : layer * d.src_layer_stride[t];
  return d.src_base[t] + lo + id * d.src_block_stride[t];
}

__device__ __forceinline__ uint8_t* dst_addr(const CopyDesc& d, uint32_t i, uint32_t layer) {
  int32_t e = d.dst_entry ? d.dst_entry[i] : static_cast<int32_t>(i);
  int t = e < 0;
  uint32_t id = t ? static_cast<uint32_t>(~e) : static_cast<uint32_t>(e);
  const uint64_t lo = d.layer_group > 1 ? layer_offset(layer, d.layer_group, d.dst_group_stride[t], d.dst_layer_stride[t])
                                        : layer * d.dst_layer_stride[t];
  return d.dst_base[t] + lo + id * d.dst_block_stride[t];
}

__global__ void __launch_bounds__(kVecThreads) copy_blocks_vector(const CopyDesc d) {
  const uint32_t vecs = static_cast<uint32_t>(d.block_bytes >> 4);
  const uint32_t pieces = (vecs + kPieceVecs - 1) / kPieceVecs;
  const uint64_t total = static_cast<uint64_t>(d.n) * d.nlayers * pieces;
  if (d.trace && threadIdx.x == 0) d.trace[2 * blockIdx.x] = ptx::global_timer_ns();
  for (uint64_t w = blockIdx.x; w < total; w += gridDim.x) {
    const uint32_t piece = static_cast<uint32_t>(w % pieces);
    const uint64_t bi = w / pieces;
    const uint32_t i = static_cast<uint32_t>(bi % d.n);
    const uint32_t layer = static_cast<uint32_t>(bi / d.n);
    const uint4* src = reinterpret_cast<const uint4*>(src_addr(d, i, layer));
    uint4* dst = reinterpret_cast<uint4*>(dst_addr(d, i, layer));
    const uint32_t v0 = piece * kPieceVecs + threadIdx.x;
    uint4 r[kVecPerThread];
#pragma unroll
    for (uint32_t j = 0; j < kVecPerThread; ++j) {
      const uint32_t v = v0 + j * kVecThreads;
      if (v < vecs) r[j] = ptx::ld_stream_v4(src + v);
    }
#pragma unroll
    for (uint32_t j = 0; j < kVecPerThread; ++j) {
      const uint32_t v = v0 + j * kVecThreads;
      if (v < vecs) dst[v] = r[j];
    }
  }
  if (d.trace && threadIdx.x == 0) d.trace[2 * blockIdx.x + 1] = ptx::global_timer_ns();
}

// Bulk ring: stage = 16 KB; kLoadsAhead loads in flight, the remaining stages drain as stores.
// Measured on 100 000 blocks: 8 stages with 4 loads ahead 6.40 TB/s; 12 with 8 ahead 6.00; 6 with 3
// ahead 6.04; 32 KB stages 6.27-6.35: more bytes in flight only queue in the memory system.
// With 6 stages (kCopyBulkShared) a CTA needs 96 KB and fits beside a CTA of the layer kernel that
// only attends, so that a gather on a second stream really runs while the attention does.
constexpr uint32_t kChunk = 16384;
constexpr int kLoadsAhead = 4;

struct ChunkRef {
  const uint8_t* src;
  uint8_t* dst;
  uint32_t bytes;
};

__device__ __forceinline__ ChunkRef chunk_ref(const CopyDesc& d, uint64_t w, uint32_t pieces) {
  const uint32_t piece = static_cast<uint32_t>(w % pieces);
  const uint64_t bi = w / pieces;
  const uint32_t i = static_cast<uint32_t>(bi % d.n);
  const uint32_t layer = static_cast<uint32_t>(bi / d.n);
  const uint64_t off = static_cast<uint64_t>(piece) * kChunk;
  const uint64_t left = d.block_bytes - off;
  ChunkRef c;
  c.src = src_addr(d, i, layer) + off;
  c.dst = dst_addr(d, i, layer) + off;
  c.bytes = left < kChunk ? static_cast<uint32_t>(left) : kChunk;
  return c;
}

template <int kStages>
__global__ void __launch_bounds__(32) copy_blocks_bulk(const CopyDesc d) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ __align__(8) uint64_t bars[kStages];
  if (threadIdx.x != 0) return;
  const uint32_t pieces = static_cast<uint32_t>((d.block_bytes + kChunk - 1) / kChunk);
  const uint64_t total = static_cast<uint64_t>(d.n) * d.nlayers * pieces;
  const uint64_t per = (total + gridDim.x - 1) / gridDim.x;
  const uint64_t w0 = blockIdx.x * per;
  if (w0 >= total) return;
  const uint64_t w1 = w0 + per < total ? w0 + per : total;
  const uint32_t cnt = static_cast<uint32_t>(w1 - w0);
  for (int s = 0; s < kStages; ++s) ptx::mbar_init(ptx::smem_u32(&bars[s]), 1);
  ptx::fence_barrier_init();
  const uint32_t base = ptx::smem_u32(smem);
  const uint64_t pol = ptx::policy_evict_first();
  const uint64_t pol_keep = ptx::policy_evict_last();  // the shared form gathers: staged blocks are read within a layer's time
  uint32_t issued = 0;
  for (; issued < cnt && issued < static_cast<uint32_t>(kLoadsAhead); ++issued) {
    ChunkRef c = chunk_ref(d, w0 + issued, pieces);
    const uint32_t bar = ptx::smem_u32(&bars[issued % kStages]);
    ptx::mbar_arrive_expect_tx(bar, c.bytes);
    ptx::bulk_g2s_hint(base + (issued % kStages) * kChunk, c.src, c.bytes, bar, pol);
  }
  bool ok = true;
  uint32_t j = 0;
  for (; j < cnt; ++j) {
    const uint32_t st = j % kStages;
    ok = ptx::mbar_wait(ptx::smem_u32(&bars[st]), (j / kStages) & 1u, d.status, kDevTimeout);
    if (!ok) break;
    ChunkRef c = chunk_ref(d, w0 + j, pieces);
    if constexpr (kStages == 6)
      ptx::bulk_s2g_hint(c.dst, base + st * kChunk, c.bytes, pol_keep);
    else
      ptx::bulk_s2g(c.dst, base + st * kChunk, c.bytes);
    ptx::bulk_commit();
    if (issued < cnt) {
      // The stage about to be refilled was last read by the store of chunk issued - kStages.
      ptx::bulk_wait_read<kStages - kLoadsAhead>();
      ChunkRef n = chunk_ref(d, w0 + issued, pieces);
      const uint32_t bar = ptx::smem_u32(&bars[issued % kStages]);
      ptx::mbar_arrive_expect_tx(bar, n.bytes);
      ptx::bulk_g2s_hint(base + (issued % kStages) * kChunk, n.src, n.bytes, bar, pol);
      ++issued;
    }
  }
  if (!ok) {
    // Give the loads still in flight a bounded chance to land before shared memory is released.
    for (uint32_t k = j; k < issued; ++k)
      ptx::mbar_wait(ptx::smem_u32(&bars[k % kStages]), (k / kStages) & 1u, nullptr, 0);
  }
  ptx::bulk_wait_all<0>();
}

}  // namespace

cudaError_t launch_copy(const CopyDesc& d, uint32_t kind, uint32_t ctas, int num_sms, cudaStream_t stream) {
  if (d.n == 0 || d.nlayers == 0) return cudaSuccess;
  if (kind == kCopyDefault) kind = kCopyVector;
  if (kind == kCopyBulk || kind == kCopyBulkShared) {
    static bool attr_set[64] = {};  // the attribute is a property of the function on one device
    const int stages = kind == kCopyBulk ? 8 : 6;
    const size_t smem = static_cast<size_t>(stages) * kChunk;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_set[dev]) {
      e = cudaFuncSetAttribute(copy_blocks_bulk<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 8 * static_cast<int>(kChunk));
      if (e != cudaSuccess) return e;
      e = cudaFuncSetAttribute(copy_blocks_bulk<6>, cudaFuncAttributeMaxDynamicSharedMemorySize, 6 * static_cast<int>(kChunk));
      if (e != cudaSuccess) return e;
      // Two kernels share an SM only under one split of its L1 / shared memory: both ask for the
      // largest shared part (as does the layer kernel), whatever they need themselves.
      e = cudaFuncSetAttribute(copy_blocks_bulk<6>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
      if (e != cudaSuccess) return e;
      attr_set[dev] = true;
    }
    const uint64_t pieces = (d.block_bytes + kChunk - 1) / kChunk;
    const uint64_t total = static_cast<uint64_t>(d.n) * d.nlayers * pieces;
    uint64_t grid = ctas ? ctas : static_cast<uint64_t>(num_sms);
    if (grid > total) grid = total;
    if (kind == kCopyBulk)
      copy_blocks_bulk<8><<<static_cast<unsigned>(grid), 32, smem, stream>>>(d);
    else
      copy_blocks_bulk<6><<<static_cast<unsigned>(grid), 32, smem, stream>>>(d);
  } else {
    const uint64_t vecs = d.block_bytes >> 4;
    const uint64_t pieces = (vecs + kPieceVecs - 1) / kPieceVecs;
    const uint64_t total = static_cast<uint64_t>(d.n) * d.nlayers * pieces;
    uint64_t grid = ctas ? ctas : static_cast<uint64_t>(num_sms) * 8;
    if (grid > total) grid = total;
    copy_blocks_vector<<<static_cast<unsigned>(grid), kVecThreads, 0, stream>>>(d);
  }
  return cudaGetLastError();
}

}  // namespace ema
