// layer_kernel.cu — the fused per-layer kernel of the memory-slice hot path:
//   paged GQA decode attention of layer l  (split-KV flash decoding, merge included)
//   + prefetch gather of layer l+1's lent blocks into the other ring slot
// in ONE persistent launch (one CTA per SM), so the two streams of HBM traffic share every SM and
// overlap for the whole duration of the layer, with no second kernel to co-schedule, no merge launch
// and no cross-stream event between layers. With copy.n == 0 it is the plain attention kernel.
//
// Roles inside a CTA (warps):
//   * producer warp: streams KV blocks of the CTA's work items into a shared-memory ring of half
//     blocks (K plane / V plane, 16 token rows of Hkv*256 B, each row padded by 16 B so ldmatrix is
//     bank-conflict free) with untiled TMA bulk copies (cp.async.bulk, one row per lane), completion
//     by mbarrier expect-tx. Work items: a static share per CTA, then items pulled from a shared
//     dynamic pool (atomic counter), which evens out SMs that stream at different rates.
//   * one consumer warp per KV head: tile products on tensor cores when the GQA group is >= 2
//     (mma.sync m16n8k16 bf16, swapped form), f32 FMAs when G == 1; online softmax with warp
//     shuffles. Each item emits a partial (max, sums, unnormalised output); the warp that
//     delivers the last partial of a (sequence, KV head) merges them and writes bf16 (no waiting:
//     a per-(sequence, head) arrival counter decides).
//   * copy warp: one thread moves 16 KB pieces lent arena -> shared ring -> staging slot with TMA
//     bulk copies (global->shared on an mbarrier, shared->global in bulk async-groups), pulling
//     64 KB units from a second atomic counter. No SM lane touches the copied bytes.
// Every mbarrier wait is bounded; on expiry the role records SLICE_ETIMEOUT in the status word,
// gives its own copies in flight a bounded chance to land and returns.
// HBM-bound: algorithmic bytes per launch = sum_s len_s * 2*Hkv*128*2 (+ q, out, table)
// + 2 * block_bytes per gathered block.
#include "attention_tiles.cuh"
#include "kernels.h"

#include <cuda_bf16.h>

namespace ema {

namespace {

constexpr int kNA = 4;                     // attention ring: half-block stages
constexpr int kNC = 5;                     // copy ring: 16 KB stages
constexpr int kCopyLoadsAhead = 3;         // loads in flight; the other stages drain as stores
constexpr uint32_t kCopyChunk = 16384;
constexpr int kQueue = 8;                  // item descriptors in flight (> kNA / 2 + 1)
constexpr uint32_t kSentinel = 0xFFFFFFFFu;
constexpr uint32_t kRowPad = 16;

__host__ __device__ constexpr uint32_t row_bytes(uint32_t Hkv) { return Hkv * kD * 2; }
__host__ __device__ constexpr uint32_t row_pitch(uint32_t Hkv) { return row_bytes(Hkv) + kRowPad; }
__host__ __device__ constexpr uint32_t half_stage_bytes(uint32_t Hkv) { return kT * row_pitch(Hkv); }

struct ItemDesc {
  uint32_t seq_idx, blk_begin, blk_end, seg_id;
};

struct Smem {
  uint8_t* att_ring;
  uint8_t* copy_ring;
  uint64_t* att_full;   // [kNA]
  uint64_t* att_empty;  // [kNA]
  uint64_t* copy_full;  // [kNC]
  ItemDesc* queue;      // [kQueue]
  uint8_t** copy_dst;   // [kNC]
  uint32_t* copy_len;   // [kNC]
};

// Bookkeeping area behind the two rings: 16 mbarrier slots, the item queue, the copy ring's
// destination pointers and lengths; every part 16-byte aligned.
constexpr size_t kBarBytes = 16 * sizeof(uint64_t);
constexpr size_t kQueueBytes = kQueue * sizeof(ItemDesc);
constexpr size_t kCopyDstBytes = 8 * sizeof(uint8_t*);
constexpr size_t kCopyLenBytes = 8 * sizeof(uint32_t);
static_assert(2 * kNA + kNC <= 16 && kNC <= 8, "bookkeeping area too small");

__host__ __device__ constexpr size_t smem_total(uint32_t Hkv) {
  return static_cast<size_t>(kNA) * half_stage_bytes(Hkv) + static_cast<size_t>(kNC) * kCopyChunk + kBarBytes +
         kQueueBytes + kCopyDstBytes + kCopyLenBytes;
}

__device__ __forceinline__ Smem carve(uint8_t* base, uint32_t Hkv) {
  Smem s;
  s.att_ring = base;
  s.copy_ring = base + static_cast<size_t>(kNA) * half_stage_bytes(Hkv);
  uint8_t* p = s.copy_ring + static_cast<size_t>(kNC) * kCopyChunk;
  s.att_full = reinterpret_cast<uint64_t*>(p);
  s.att_empty = s.att_full + kNA;
  s.copy_full = s.att_empty + kNA;
  s.queue = reinterpret_cast<ItemDesc*>(p + kBarBytes);
  s.copy_dst = reinterpret_cast<uint8_t**>(p + kBarBytes + kQueueBytes);
  s.copy_len = reinterpret_cast<uint32_t*>(p + kBarBytes + kQueueBytes + kCopyDstBytes);
  return s;
}

__device__ __forceinline__ const uint8_t* copy_src(const CopyDesc& d, uint32_t i, uint32_t layer) {
  const int32_t e = d.src_entry ? d.src_entry[i] : static_cast<int32_t>(i);
  const int t = e < 0;
  const uint32_t id = t ? static_cast<uint32_t>(~e) : static_cast<uint32_t>(e);
  return d.src_base[t] + layer * d.src_layer_stride[t] + id * d.src_block_stride[t];
}

__device__ __forceinline__ uint8_t* copy_dst(const CopyDesc& d, uint32_t i, uint32_t layer) {
  const int32_t e = d.dst_entry ? d.dst_entry[i] : static_cast<int32_t>(i);
  const int t = e < 0;
  const uint32_t id = t ? static_cast<uint32_t>(~e) : static_cast<uint32_t>(e);
  return d.dst_base[t] + layer * d.dst_layer_stride[t] + id * d.dst_block_stride[t];
}

// ---------------------------------------------------------------------------------------------
// producer warp
// ---------------------------------------------------------------------------------------------
__device__ void producer_role(const LayerParams& p, const Smem& sm) {
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t Hkv = p.Hkv;
  const uint32_t rb = row_bytes(Hkv), pitch = row_pitch(Hkv), hsb = half_stage_bytes(Hkv);
  const uint32_t plane_bytes = kT * rb;
  const uint32_t ring = ptx::smem_u32(sm.att_ring);
  uint32_t hs = 0, nq = 0;
  bool ok = true;

  auto stream_item = [&](const WorkItem& it) {
    const uint32_t nb = it.blk_end - it.blk_begin;
    for (uint32_t b0 = 0; b0 < nb && ok; b0 += 32) {
      const uint32_t cnt = min(32u, nb - b0);
      const int32_t my = lane < cnt ? p.resolved[it.flat_begin + b0 + lane] : 0;
      for (uint32_t j = 0; j < cnt && ok; ++j) {
        const int32_t e = __shfl_sync(0xffffffffu, my, j);
        const uint8_t* src = e >= 0 ? p.local_layer + static_cast<uint64_t>(e) * p.local_block_stride
                                    : p.slot_base + static_cast<uint64_t>(~e) * p.block_bytes;
#pragma unroll
        for (uint32_t plane = 0; plane < 2; ++plane, ++hs) {
          const uint32_t stg = hs % kNA;
          ok = ptx::mbar_wait(ptx::smem_u32(&sm.att_empty[stg]), ((hs / kNA) & 1u) ^ 1u, p.status, kDevTimeout);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) return;
          const uint32_t full = ptx::smem_u32(&sm.att_full[stg]);
          if (lane == 0) {
            if (b0 + j == 0 && plane == 0) {
              sm.queue[nq % kQueue] = ItemDesc{it.seq_idx, it.blk_begin, it.blk_end, it.seg_id};
              ++nq;
            }
            ptx::mbar_arrive_expect_tx(full, plane_bytes);
          }
          __syncwarp();
          if (lane < kT)
            ptx::bulk_g2s(ring + stg * hsb + lane * pitch, src + plane * plane_bytes + static_cast<uint64_t>(lane) * rb,
                          rb, full);
        }
      }
    }
  };

  auto fetch_dynamic = [&]() -> uint32_t {
    uint32_t j = 0;
    if (lane == 0) j = atomicAdd(&p.launch_cnt[0], 1u);
    return __shfl_sync(0xffffffffu, j, 0);
  };

  const uint32_t s0 = p.cta_item_off[blockIdx.x], s1 = p.cta_item_off[blockIdx.x + 1];
  for (uint32_t i = s0; i < s1 && ok; ++i) stream_item(p.items[i]);
  if (ok && p.n_dyn) {
    uint32_t next = fetch_dynamic();
    while (ok && next < p.n_dyn) {
      const WorkItem cur = p.items[p.dyn_begin + next];
      next = fetch_dynamic();  // one ahead: the atomic's latency hides behind this item's blocks
      stream_item(cur);
    }
  }
  if (ok) {
    // End marker: a descriptor with no data behind it.
    const uint32_t stg = hs % kNA;
    ok = ptx::mbar_wait(ptx::smem_u32(&sm.att_empty[stg]), ((hs / kNA) & 1u) ^ 1u, p.status, kDevTimeout);
    ok = __all_sync(0xffffffffu, ok);
    if (ok && lane == 0) {
      sm.queue[nq % kQueue] = ItemDesc{kSentinel, 0, 0, 0};
      ptx::mbar_arrive(ptx::smem_u32(&sm.att_full[stg]));
    }
  }
  if (!ok) {
    // Bounded second chance for copies already issued, so that none lands after the CTA is gone.
    const uint32_t from = hs > static_cast<uint32_t>(kNA) ? hs - kNA : 0;
    for (uint32_t k = from; k < hs; ++k)
      ptx::mbar_wait(ptx::smem_u32(&sm.att_full[k % kNA]), (k / kNA) & 1u, nullptr, 0);
  }
}

// ---------------------------------------------------------------------------------------------
// merge by the last-arriving warp of a (sequence, KV head)
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void finish_segment(const LayerParams& p, uint32_t seq, uint32_t g) {
  const uint32_t lane = threadIdx.x & 31u;
  __threadfence();
  __syncwarp();
  uint32_t old = 0;
  if (lane == 0) old = atomicAdd(&p.merge_cnt[seq * p.Hkv + g], 1u);
  old = __shfl_sync(0xffffffffu, old, 0);
  const uint32_t s0 = p.seq_seg_off[seq], s1 = p.seq_seg_off[seq + 1];
  if (old + 1 != s1 - s0) return;
  __threadfence();
  const uint32_t G = p.G;
  for (uint32_t hh = 0; hh < G; ++hh) {
    const uint32_t h = g * G + hh;
    float M = kNegInf;
    for (uint32_t s = s0; s < s1; ++s) M = fmaxf(M, __ldcg(p.part_ml + (static_cast<uint64_t>(s) * p.Hq + h) * 4));
    float l = 0.f, le = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (uint32_t s = s0; s < s1; ++s) {
      const float4 ml = __ldcg(reinterpret_cast<const float4*>(p.part_ml + (static_cast<uint64_t>(s) * p.Hq + h) * 4));
      const float wgt = ptx::exp2_approx(ml.x - M);
      l += ml.y * wgt;
      le += ml.z * wgt;
      const float4 v =
          __ldcg(reinterpret_cast<const float4*>(p.part_o + (static_cast<uint64_t>(s) * p.Hq + h) * kD + lane * 4));
      acc.x = fmaf(v.x, wgt, acc.x);
      acc.y = fmaf(v.y, wgt, acc.y);
      acc.z = fmaf(v.z, wgt, acc.z);
      acc.w = fmaf(v.w, wgt, acc.w);
    }
    const float inv = 1.f / l;
    const uint32_t lo = ptx::pack_bf16x2(acc.x * inv, acc.y * inv);
    const uint32_t hi = ptx::pack_bf16x2(acc.z * inv, acc.w * inv);
    uint2* dst = reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(p.out) + (static_cast<uint64_t>(seq) * p.Hq + h) * kD +
                                          lane * 4);
    *dst = make_uint2(lo, hi);
    if (p.lse && lane == 0) p.lse[static_cast<uint64_t>(seq) * p.Hq + h] = (M + log2f(le)) * 0.6931471805599453f;
  }
  if (lane == 0) p.merge_cnt[seq * p.Hkv + g] = 0;  // ready for the next launch
}

// ---------------------------------------------------------------------------------------------
// consumer warp (= KV head g)
// ---------------------------------------------------------------------------------------------
template <bool kMma>
__device__ void consumer_role(const LayerParams& p, const Smem& sm, uint32_t g) {
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t Hkv = p.Hkv, G = p.G;
  const uint32_t pitch = row_pitch(Hkv), hsb = half_stage_bytes(Hkv);
  const uint32_t head_off = g * kD * 2;
  const uint32_t ring = ptx::smem_u32(sm.att_ring);
  const __nv_bfloat16* qg = static_cast<const __nv_bfloat16*>(p.q);
  uint32_t hs = 0, nseg = 0;
  for (;;) {
    {
      const uint32_t stg = hs % kNA;
      const bool ok = ptx::mbar_wait(ptx::smem_u32(&sm.att_full[stg]), (hs / kNA) & 1u, p.status, kDevTimeout);
      if (!__all_sync(0xffffffffu, ok)) return;
    }
    const ItemDesc it = sm.queue[nseg % kQueue];
    if (it.seq_idx == kSentinel) break;
    ++nseg;
    const uint32_t len = p.lens[it.seq_idx];
    SegState st{kNegInf, kNegInf, 0.f, 0.f, 0.f, 0.f};
    if constexpr (kMma) {
      // Q^T fragments (B operand): head n = lane/4 of the group, dims ks*16 + 2*(lane%4) (+8).
      uint32_t qf[8][2];
      const uint32_t n = lane >> 2, tig = lane & 3u;
      const uint32_t* qrow =
          reinterpret_cast<const uint32_t*>(qg + (static_cast<uint64_t>(it.seq_idx) * p.Hq + g * G + (n < G ? n : 0)) * kD);
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        qf[ks][0] = n < G ? qrow[ks * 8 + tig] : 0u;
        qf[ks][1] = n < G ? qrow[ks * 8 + tig + 4] : 0u;
      }
      float o[8][4];
#pragma unroll
      for (int mt = 0; mt < 8; ++mt) o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f;
      for (uint32_t b = it.blk_begin; b < it.blk_end; ++b) {
        uint32_t stg = hs % kNA;
        if (b != it.blk_begin) {
          const bool ok = ptx::mbar_wait(ptx::smem_u32(&sm.att_full[stg]), (hs / kNA) & 1u, p.status, kDevTimeout);
          if (!__all_sync(0xffffffffu, ok)) return;
        }
        const uint32_t valid = min(kT, len - b * kT);
        uint32_t pb0, pb1;
        float al0, al1;
        tile_mma_scores(ring + stg * hsb, pitch, head_off, valid, qf, p.scale_log2, st, pb0, pb1, al0, al1);
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sm.att_empty[stg]));
        ++hs;
        stg = hs % kNA;
        {
          const bool ok = ptx::mbar_wait(ptx::smem_u32(&sm.att_full[stg]), (hs / kNA) & 1u, p.status, kDevTimeout);
          if (!__all_sync(0xffffffffu, ok)) return;
        }
        tile_mma_pv(ring + stg * hsb, pitch, head_off, valid, pb0, pb1, al0, al1, o);
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sm.att_empty[stg]));
        ++hs;
      }
#pragma unroll
      for (int sh = 4; sh <= 16; sh <<= 1) {
        st.l0 += __shfl_xor_sync(0xffffffffu, st.l0, sh);
        st.l1 += __shfl_xor_sync(0xffffffffu, st.l1, sh);
        st.e0 += __shfl_xor_sync(0xffffffffu, st.e0, sh);
        st.e1 += __shfl_xor_sync(0xffffffffu, st.e1, sh);
      }
      const uint32_t r0 = lane >> 2;
      const uint32_t h0 = 2 * tig, h1 = h0 + 1;
      float* po = p.part_o + (static_cast<uint64_t>(it.seg_id) * p.Hq + g * G) * kD;
      float* pml = p.part_ml + (static_cast<uint64_t>(it.seg_id) * p.Hq + g * G) * 4;
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
    } else {
      // G == 1: query head = KV head. Lane keeps its half (64 dims) of q in registers as f32.
      float qh[64];
      const uint32_t half = lane & 1u;
      const uint4* qrow =
          reinterpret_cast<const uint4*>(qg + (static_cast<uint64_t>(it.seq_idx) * p.Hq + g) * kD + half * 64);
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const uint4 v = qrow[c];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          qh[c * 8 + 2 * e] = __uint_as_float(w[e] << 16);
          qh[c * 8 + 2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
        }
      }
      float o[4] = {0.f, 0.f, 0.f, 0.f};
      for (uint32_t b = it.blk_begin; b < it.blk_end; ++b) {
        uint32_t stg = hs % kNA;
        if (b != it.blk_begin) {
          const bool ok = ptx::mbar_wait(ptx::smem_u32(&sm.att_full[stg]), (hs / kNA) & 1u, p.status, kDevTimeout);
          if (!__all_sync(0xffffffffu, ok)) return;
        }
        const uint32_t valid = min(kT, len - b * kT);
        float pw, al;
        tile_alu_scores(sm.att_ring + stg * hsb, pitch, head_off, valid, qh, p.scale_log2, st, pw, al);
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sm.att_empty[stg]));
        ++hs;
        stg = hs % kNA;
        {
          const bool ok = ptx::mbar_wait(ptx::smem_u32(&sm.att_full[stg]), (hs / kNA) & 1u, p.status, kDevTimeout);
          if (!__all_sync(0xffffffffu, ok)) return;
        }
        tile_alu_pv(sm.att_ring + stg * hsb, pitch, head_off, valid, pw, al, o);
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sm.att_empty[stg]));
        ++hs;
      }
#pragma unroll
      for (int sh = 1; sh <= 16; sh <<= 1) st.l0 += __shfl_xor_sync(0xffffffffu, st.l0, sh);
      float* po = p.part_o + (static_cast<uint64_t>(it.seg_id) * p.Hq + g) * kD;
      *reinterpret_cast<float4*>(po + lane * 4) = make_float4(o[0], o[1], o[2], o[3]);
      if (lane == 0)
        *reinterpret_cast<float4*>(p.part_ml + (static_cast<uint64_t>(it.seg_id) * p.Hq + g) * 4) =
            make_float4(st.m0, st.l0, st.l0, 0.f);
    }
    finish_segment(p, it.seq_idx, g);
  }
}

// ---------------------------------------------------------------------------------------------
// copy warp (one thread)
// ---------------------------------------------------------------------------------------------
__device__ void copy_role(const LayerParams& p, const Smem& sm) {
  const CopyDesc& d = p.copy;
  const uint32_t n_units = d.n * d.nlayers;
  const uint32_t pieces = static_cast<uint32_t>((d.block_bytes + kCopyChunk - 1) / kCopyChunk);
  const uint32_t ring = ptx::smem_u32(sm.copy_ring);
  const uint64_t pol = ptx::policy_evict_first();
  uint32_t piece = pieces;  // forces a unit fetch
  const uint8_t* src_blk = nullptr;
  uint8_t* dst_blk = nullptr;
  uint32_t issued = 0, done = 0;
  bool more = true, ok = true;

  // Issues the load of the next 16 KB piece, pulling a new 64 KB unit when the current one is used up.
  auto issue_next = [&]() -> bool {
    if (piece == pieces) {
      const uint32_t unit = atomicAdd(&p.launch_cnt[1], 1u);
      if (unit >= n_units) return false;
      const uint32_t i = unit % d.n, layer = unit / d.n;
      src_blk = copy_src(d, i, layer);
      dst_blk = copy_dst(d, i, layer);
      piece = 0;
    }
    const uint64_t off = static_cast<uint64_t>(piece) * kCopyChunk;
    const uint64_t left = d.block_bytes - off;
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

  while (issued < static_cast<uint32_t>(kCopyLoadsAhead) && more) more = issue_next();
  while (done < issued) {
    const uint32_t stg = done % kNC;
    ok = ptx::mbar_wait(ptx::smem_u32(&sm.copy_full[stg]), (done / kNC) & 1u, p.status, kDevTimeout);
    if (!ok) break;
    ptx::bulk_s2g(sm.copy_dst[stg], ring + stg * kCopyChunk, sm.copy_len[stg]);
    ptx::bulk_commit();
    ++done;
    if (more) {
      // The stage about to be refilled was last read by the store of piece issued - kNC.
      ptx::bulk_wait_read<kNC - kCopyLoadsAhead>();
      more = issue_next();
    }
  }
  if (!ok) {
    for (uint32_t k = done; k < issued; ++k)
      ptx::mbar_wait(ptx::smem_u32(&sm.copy_full[k % kNC]), (k / kNC) & 1u, nullptr, 0);
  }
  ptx::bulk_wait_all<0>();
}

template <bool kMma>
__global__ void __launch_bounds__(320, 1) slice_layer_kernel(const LayerParams p) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  const Smem sm = carve(smem_raw, p.Hkv);
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
  if (threadIdx.x == 0) {
    if (p.trace) {
      uint32_t smid;
      asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
      p.trace[4 * blockIdx.x] = ptx::global_timer_ns();
      p.trace[4 * blockIdx.x + 1] = 0;
      p.trace[4 * blockIdx.x + 2] = 0;
      p.trace[4 * blockIdx.x + 3] = smid;
    }
    for (int s = 0; s < kNA; ++s) {
      ptx::mbar_init(ptx::smem_u32(&sm.att_full[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&sm.att_empty[s]), p.Hkv);
    }
    for (int s = 0; s < kNC; ++s) ptx::mbar_init(ptx::smem_u32(&sm.copy_full[s]), 1);
    ptx::fence_barrier_init();
  }
  __syncthreads();
  if (warp < p.Hkv) {
    if (p.has_attention) consumer_role<kMma>(p, sm, warp);
    if (p.trace && warp == 0 && lane == 0) p.trace[4 * blockIdx.x + 1] = ptx::global_timer_ns();
  } else if (warp == p.Hkv) {
    if (p.has_attention) producer_role(p, sm);
  } else if (warp == p.Hkv + 1) {
    if (lane == 0 && p.copy.n) {
      copy_role(p, sm);
      if (p.trace) p.trace[4 * blockIdx.x + 2] = ptx::global_timer_ns();
    }
  }
}

// One CTA per sequence: the new token's K and V rows go to the home block and the staged copy.
__global__ void __launch_bounds__(128) append_kv_kernel(const AppendParams p) {
  const uint32_t i = blockIdx.x;
  if (i >= p.nseq) return;
  const uint32_t len = p.lens[i];
  if (len == 0) return;
  const uint32_t r = (len - 1) % p.block_tokens;
  const int32_t e = p.home_entry[i];
  uint8_t* home = e >= 0 ? p.local_layer + static_cast<uint64_t>(e) * p.local_block_stride
                         : p.lent_layer + static_cast<uint64_t>(~e) * p.lent_block_stride;
  const int32_t sp = p.stage_pos[i];
  uint8_t* staged = (p.slot_base && sp >= 0) ? p.slot_base + static_cast<uint64_t>(sp) * p.block_bytes : nullptr;
  const uint32_t plane = p.block_tokens * p.row_bytes;
  const uint32_t vecs = p.row_bytes >> 4;
  const uint4* ks = reinterpret_cast<const uint4*>(static_cast<const uint8_t*>(p.k_new) + static_cast<uint64_t>(i) * p.row_bytes);
  const uint4* vs = reinterpret_cast<const uint4*>(static_cast<const uint8_t*>(p.v_new) + static_cast<uint64_t>(i) * p.row_bytes);
  for (uint32_t v = threadIdx.x; v < vecs; v += blockDim.x) {
    const uint4 kv = ks[v], vv = vs[v];
    reinterpret_cast<uint4*>(home + r * p.row_bytes)[v] = kv;
    reinterpret_cast<uint4*>(home + plane + r * p.row_bytes)[v] = vv;
    if (staged) {
      reinterpret_cast<uint4*>(staged + r * p.row_bytes)[v] = kv;
      reinterpret_cast<uint4*>(staged + plane + r * p.row_bytes)[v] = vv;
    }
  }
}

}  // namespace

size_t layer_smem_bytes(uint32_t Hkv) {
  if (Hkv == 0 || Hkv > 8) return 0;
  return smem_total(Hkv);
}

cudaError_t layer_setup() {
  const int smem = static_cast<int>(layer_smem_bytes(8));
  cudaError_t e = cudaFuncSetAttribute(slice_layer_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(slice_layer_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
}

cudaError_t launch_layer(const LayerParams& p, cudaStream_t stream) {
  const size_t smem = layer_smem_bytes(p.Hkv);
  const unsigned threads = (p.Hkv + 2) * 32;
  if (p.G == 1)
    slice_layer_kernel<false><<<p.ncta, threads, smem, stream>>>(p);
  else
    slice_layer_kernel<true><<<p.ncta, threads, smem, stream>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_append(const AppendParams& p, cudaStream_t stream) {
  if (p.nseq == 0) return cudaSuccess;
  append_kv_kernel<<<p.nseq, 128, 0, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace ema
