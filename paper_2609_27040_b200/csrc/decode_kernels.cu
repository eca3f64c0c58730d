// decode_kernels.cu — paged GQA decode attention (split-KV flash decoding) over the local arena
// and a staging-ring slot, plus the merge of the split partials and the KV append.
//
// Shape of the attention kernel
//   * Persistent CTAs (one per SM). The batch's blocks, flattened in batch order, are cut into
//     equal contiguous ranges, one per CTA; a range is a list of segments (sequence, blocks).
//   * A producer warp streams whole 64 KB blocks (all KV heads, K plane then V plane) into a
//     shared-memory ring with untiled TMA bulk copies, one 2 KB token row per lane, each row
//     padded by 16 B so that ldmatrix over eight token rows is bank-conflict free. Completion is
//     tracked by mbarriers (expect-tx); every wait is bounded.
//   * One consumer warp per KV head. With a GQA group G >= 2 the tile products run on tensor
//     cores in swapped form: S^T[16 tokens x 8 heads] = K[16 x 128] Q^T, O^T[128 x 8] += V^T P^T
//     (mma.sync m16n8k16 bf16, f32 accumulate; heads padded to 8). With G == 1 there is no dense
//     tile and the warp uses f32 FMAs. Softmax is online, in the log2 domain, with warp-shuffle
//     reductions; tokens past the sequence length get -inf scores and their V rows are zeroed.
//   * Each segment emits (max, sum, unnormalised output); a second kernel merges a sequence's
//     partials and writes bf16.
// HBM-bound: algorithmic bytes per layer = sum over sequences of len * 2 * Hkv * 128 * 2.
#include "kernels.h"
#include "ptx.cuh"

#include <cuda_bf16.h>

namespace ema {

namespace {

constexpr uint32_t kD = 128;
constexpr uint32_t kT = 16;
constexpr int kRing = 3;               // blocks in flight / in use per CTA
constexpr uint32_t kRowPad = 16;       // bytes added to every token row in shared memory
constexpr float kNegInf = -INFINITY;

__host__ __device__ constexpr uint32_t row_bytes(uint32_t Hkv) { return Hkv * kD * 2; }
__host__ __device__ constexpr uint32_t row_pitch(uint32_t Hkv) { return row_bytes(Hkv) + kRowPad; }
__host__ __device__ constexpr uint32_t stage_bytes(uint32_t Hkv) { return 2 * kT * row_pitch(Hkv); }

struct SegState {
  float m0, m1;  // running max of the two heads this thread owns (MMA path) / of the head (ALU path)
  float l0, l1;  // running sums of the weights as used in P*V (per-thread partial)
  float e0, e1;  // running sums of the unrounded weights, for the log-sum-exp
};

// ------------------------------------------------------------------------------------------
// Tensor-core tile: one KV head, one block of up to 16 tokens, heads of the group on the N axis.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void tile_mma(uint32_t stage_addr, uint32_t pitch, uint32_t head_off, uint32_t valid,
                                         const uint32_t (&qf)[8][2], float scale_log2, SegState& st,
                                         float (&o)[8][4]) {
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t mj = lane >> 3, mr = lane & 7u;
  // K fragment addresses: matrix mj covers tokens (mj&1)*8.., dims (mj>>1)*8..
  const uint32_t k_addr = stage_addr + ((mj & 1u) * 8 + mr) * pitch + head_off + (mj >> 1) * 16;
  float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int ks = 0; ks < 8; ks += 2) {
    uint32_t a[4], b[4];
    ptx::ldmatrix_x4(a, k_addr + ks * 32);
    ptx::ldmatrix_x4(b, k_addr + (ks + 1) * 32);
    ptx::mma_bf16_16816(sa, a, qf[ks][0], qf[ks][1]);
    ptx::mma_bf16_16816(sb, b, qf[ks + 1][0], qf[ks + 1][1]);
  }
  const uint32_t r0 = lane >> 2, tig = lane & 3u;
  float s0 = (sa[0] + sb[0]) * scale_log2, s1 = (sa[1] + sb[1]) * scale_log2;
  float s2 = (sa[2] + sb[2]) * scale_log2, s3 = (sa[3] + sb[3]) * scale_log2;
  if (valid < kT) {
    if (r0 >= valid) s0 = s1 = kNegInf;
    if (r0 + 8 >= valid) s2 = s3 = kNegInf;
  }
  float mx0 = fmaxf(s0, s2), mx1 = fmaxf(s1, s3);
#pragma unroll
  for (int sh = 4; sh <= 16; sh <<= 1) {
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, sh));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, sh));
  }
  const float mn0 = fmaxf(st.m0, mx0), mn1 = fmaxf(st.m1, mx1);
  const float al0 = ptx::exp2_approx(st.m0 - mn0), al1 = ptx::exp2_approx(st.m1 - mn1);
  st.m0 = mn0;
  st.m1 = mn1;
  const float p0 = ptx::exp2_approx(s0 - mn0), p1 = ptx::exp2_approx(s1 - mn1);
  const float p2 = ptx::exp2_approx(s2 - mn0), p3 = ptx::exp2_approx(s3 - mn1);
  const uint32_t p01 = ptx::pack_bf16x2(p0, p1), p23 = ptx::pack_bf16x2(p2, p3);
  // The sums use the rounded weights, so the result stays a convex combination of V rows.
  st.l0 = st.l0 * al0 + __uint_as_float(p01 << 16) + __uint_as_float(p23 << 16);
  st.l1 = st.l1 * al1 + __uint_as_float(p01 & 0xffff0000u) + __uint_as_float(p23 & 0xffff0000u);
  st.e0 = st.e0 * al0 + (p0 + p2);
  st.e1 = st.e1 * al1 + (p1 + p3);
  const uint32_t pb0 = ptx::movmatrix_trans(p01);  // P^T rows = tokens 0..7
  const uint32_t pb1 = ptx::movmatrix_trans(p23);  // tokens 8..15
  // V^T fragment addresses: matrix mj covers tokens (mj>>1)*8.., dims (mj&1)*8..
  const uint32_t v_addr = stage_addr + (kT + (mj >> 1) * 8 + mr) * pitch + head_off + (mj & 1u) * 16;
  uint32_t keep_lo = 0xffffffffu, keep_hi = 0xffffffffu;  // masks for token pairs (2tig,2tig+1), (+8,+9)
  if (valid < kT) {
    const uint32_t t = 2 * tig;
    keep_lo = (t < valid ? 0x0000ffffu : 0u) | (t + 1 < valid ? 0xffff0000u : 0u);
    keep_hi = (t + 8 < valid ? 0x0000ffffu : 0u) | (t + 9 < valid ? 0xffff0000u : 0u);
  }
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) {
    uint32_t a[4];
    ptx::ldmatrix_x4_trans(a, v_addr + mt * 32);
    if (valid < kT) {
      a[0] &= keep_lo;
      a[1] &= keep_lo;
      a[2] &= keep_hi;
      a[3] &= keep_hi;
    }
    o[mt][0] *= al0;
    o[mt][1] *= al1;
    o[mt][2] *= al0;
    o[mt][3] *= al1;
    ptx::mma_bf16_16816(o[mt], a, pb0, pb1);
  }
}

// ------------------------------------------------------------------------------------------
// f32 tile for G == 1: lane pair (2t, 2t+1) scores token t; lane l owns output dims 4l..4l+3.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void tile_alu(const uint8_t* stage, uint32_t pitch, uint32_t head_off, uint32_t valid,
                                         const float (&qh)[64], float scale_log2, SegState& st, float (&o)[4]) {
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t t = lane >> 1, half = lane & 1u;
  const uint4* krow = reinterpret_cast<const uint4*>(stage + t * pitch + head_off + half * 128);
  float acc = 0.f;
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    const uint4 v = krow[c];
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      acc = fmaf(qh[c * 8 + 2 * e], __uint_as_float(w[e] << 16), acc);
      acc = fmaf(qh[c * 8 + 2 * e + 1], __uint_as_float(w[e] & 0xffff0000u), acc);
    }
  }
  acc += __shfl_xor_sync(0xffffffffu, acc, 1);
  float s = t < valid ? acc * scale_log2 : kNegInf;
  float mx = s;
#pragma unroll
  for (int sh = 2; sh <= 16; sh <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, sh));
  const float mn = fmaxf(st.m0, mx);
  const float al = ptx::exp2_approx(st.m0 - mn);
  st.m0 = mn;
  const float p = ptx::exp2_approx(s - mn);
  st.l0 = st.l0 * al + (half == 0 ? p : 0.f);
#pragma unroll
  for (int e = 0; e < 4; ++e) o[e] *= al;
  const uint8_t* vbase = stage + kT * pitch + head_off + lane * 8;
  for (uint32_t tt = 0; tt < valid; ++tt) {
    const float pt = __shfl_sync(0xffffffffu, p, 2 * tt);
    const uint2 v = *reinterpret_cast<const uint2*>(vbase + tt * pitch);
    o[0] = fmaf(pt, __uint_as_float(v.x << 16), o[0]);
    o[1] = fmaf(pt, __uint_as_float(v.x & 0xffff0000u), o[1]);
    o[2] = fmaf(pt, __uint_as_float(v.y << 16), o[2]);
    o[3] = fmaf(pt, __uint_as_float(v.y & 0xffff0000u), o[3]);
  }
}

template <bool kMma>
__global__ void __launch_bounds__(288, 1) paged_decode_kernel(const DecodeParams p) {
  extern __shared__ __align__(128) uint8_t smem[];
  const uint32_t Hkv = p.Hkv;
  const uint32_t pitch = row_pitch(Hkv);
  const uint32_t sbytes = stage_bytes(Hkv);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kRing * sbytes);  // full[kRing], empty[kRing]
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
  const uint32_t seg0 = p.cta_seg_off[blockIdx.x], seg1 = p.cta_seg_off[blockIdx.x + 1];
  if (seg0 >= seg1) return;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kRing; ++s) {
      ptx::mbar_init(ptx::smem_u32(&bars[s]), 1);
      ptx::mbar_init(ptx::smem_u32(&bars[kRing + s]), Hkv);
    }
    ptx::fence_barrier_init();
  }
  __syncthreads();
  const uint32_t smem_base = ptx::smem_u32(smem);

  if (warp == Hkv) {
    // ---------------- producer: one block per ring stage, one token row per lane ----------------
    const Segment first = p.segs[seg0], last = p.segs[seg1 - 1];
    const uint32_t f0 = first.flat_begin, f1 = last.flat_begin + (last.blk_end - last.blk_begin);
    const uint32_t rb = row_bytes(Hkv);
    uint32_t it = 0;
    bool ok = true;
    for (uint32_t fb = f0; fb < f1 && ok; fb += 32) {
      const uint32_t nb = min(32u, f1 - fb);
      const int32_t my = lane < nb ? p.resolved[fb + lane] : 0;
      for (uint32_t j = 0; j < nb; ++j, ++it) {
        const int32_t e = __shfl_sync(0xffffffffu, my, j);
        const uint32_t stg = it % kRing;
        ok = ptx::mbar_wait(ptx::smem_u32(&bars[kRing + stg]), ((it / kRing) & 1u) ^ 1u, p.status, kDevTimeout);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const uint8_t* src = e >= 0 ? p.local_layer + static_cast<uint64_t>(e) * p.local_block_stride
                                    : p.slot_base + static_cast<uint64_t>(~e) * p.block_bytes;
        const uint32_t full = ptx::smem_u32(&bars[stg]);
        if (lane == 0) ptx::mbar_arrive_expect_tx(full, 2 * kT * rb);
        __syncwarp();
        ptx::bulk_g2s(smem_base + stg * sbytes + lane * pitch, src + static_cast<uint64_t>(lane) * rb, rb, full);
      }
    }
    if (!ok) {
      // Bounded second chance for copies already issued, so none lands after the CTA is gone.
      const uint32_t from = it > static_cast<uint32_t>(kRing) ? it - kRing : 0;
      for (uint32_t k = from; k < it; ++k)
        ptx::mbar_wait(ptx::smem_u32(&bars[k % kRing]), (k / kRing) & 1u, nullptr, 0);
    }
    return;
  }
  if (warp > Hkv) return;

  // ---------------- consumers: warp = KV head ----------------
  const uint32_t g = warp;
  const uint32_t head_off = g * kD * 2;
  const uint32_t G = p.G;
  const __nv_bfloat16* qg = static_cast<const __nv_bfloat16*>(p.q);
  uint32_t it = 0;
  for (uint32_t sgi = seg0; sgi < seg1; ++sgi) {
    const Segment sg = p.segs[sgi];
    const uint32_t len = p.lens[sg.seq_idx];
    SegState st{kNegInf, kNegInf, 0.f, 0.f, 0.f, 0.f};
    bool ok = true;
    if constexpr (kMma) {
      // Q^T fragments (B operand): head n = lane/4 of the group, dims ks*16 + 2*(lane%4) (+8).
      uint32_t qf[8][2];
      const uint32_t n = lane >> 2, tig = lane & 3u;
      const uint32_t* qrow =
          reinterpret_cast<const uint32_t*>(qg + (static_cast<uint64_t>(sg.seq_idx) * p.Hq + g * G + n) * kD);
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        qf[ks][0] = n < G ? qrow[ks * 8 + tig] : 0u;
        qf[ks][1] = n < G ? qrow[ks * 8 + tig + 4] : 0u;
      }
      float o[8][4];
#pragma unroll
      for (int mt = 0; mt < 8; ++mt) o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f;
      for (uint32_t b = sg.blk_begin; b < sg.blk_end; ++b, ++it) {
        const uint32_t stg = it % kRing;
        ok = ptx::mbar_wait(ptx::smem_u32(&bars[stg]), (it / kRing) & 1u, p.status, kDevTimeout);
        if (!__all_sync(0xffffffffu, ok)) return;
        const uint32_t valid = min(kT, len - b * kT);
        tile_mma(smem_base + stg * sbytes, pitch, head_off, valid, qf, p.scale_log2, st, o);
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&bars[kRing + stg]));
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
      float* po = p.part_o + (static_cast<uint64_t>(sgi) * p.Hq + g * G) * kD;
      float* pml = p.part_ml + (static_cast<uint64_t>(sgi) * p.Hq + g * G) * 4;
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
        if (h0 < G) {
          pml[h0 * 4] = st.m0;
          pml[h0 * 4 + 1] = st.l0;
          pml[h0 * 4 + 2] = st.e0;
        }
        if (h1 < G) {
          pml[h1 * 4] = st.m1;
          pml[h1 * 4 + 1] = st.l1;
          pml[h1 * 4 + 2] = st.e1;
        }
      }
    } else {
      // G == 1: query head = KV head. Lane keeps its half (64 dims) of q in registers as f32.
      float qh[64];
      const uint32_t half = lane & 1u;
      const uint4* qrow = reinterpret_cast<const uint4*>(qg + (static_cast<uint64_t>(sg.seq_idx) * p.Hq + g) * kD +
                                                         half * 64);
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
      for (uint32_t b = sg.blk_begin; b < sg.blk_end; ++b, ++it) {
        const uint32_t stg = it % kRing;
        ok = ptx::mbar_wait(ptx::smem_u32(&bars[stg]), (it / kRing) & 1u, p.status, kDevTimeout);
        if (!__all_sync(0xffffffffu, ok)) return;
        const uint32_t valid = min(kT, len - b * kT);
        tile_alu(smem + stg * sbytes, pitch, head_off, valid, qh, p.scale_log2, st, o);
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&bars[kRing + stg]));
      }
#pragma unroll
      for (int sh = 1; sh <= 16; sh <<= 1) st.l0 += __shfl_xor_sync(0xffffffffu, st.l0, sh);
      float* po = p.part_o + (static_cast<uint64_t>(sgi) * p.Hq + g) * kD;
      *reinterpret_cast<float4*>(po + lane * 4) = make_float4(o[0], o[1], o[2], o[3]);
      if (lane == 0) {
        float* pml = p.part_ml + (static_cast<uint64_t>(sgi) * p.Hq + g) * 4;
        pml[0] = st.m0;
        pml[1] = st.l0;
        pml[2] = st.l0;
      }
    }
  }
}

// One warp per (sequence, query head): combine the sequence's partials and write bf16.
__global__ void __launch_bounds__(128) merge_partials_kernel(const DecodeParams p) {
  const uint32_t w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const uint32_t lane = threadIdx.x & 31u;
  if (w >= p.nseq * p.Hq) return;
  const uint32_t i = w / p.Hq, h = w % p.Hq;
  const uint32_t s0 = p.seq_seg_off[i], s1 = p.seq_seg_off[i + 1];
  float M = kNegInf;
  for (uint32_t s = s0; s < s1; ++s) M = fmaxf(M, p.part_ml[(static_cast<uint64_t>(s) * p.Hq + h) * 4]);
  float l = 0.f, le = 0.f;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (uint32_t s = s0; s < s1; ++s) {
    const float* ml = p.part_ml + (static_cast<uint64_t>(s) * p.Hq + h) * 4;
    const float wgt = ptx::exp2_approx(ml[0] - M);
    l += ml[1] * wgt;
    le += ml[2] * wgt;
    const float4 v = *reinterpret_cast<const float4*>(p.part_o + (static_cast<uint64_t>(s) * p.Hq + h) * kD + lane * 4);
    acc.x = fmaf(v.x, wgt, acc.x);
    acc.y = fmaf(v.y, wgt, acc.y);
    acc.z = fmaf(v.z, wgt, acc.z);
    acc.w = fmaf(v.w, wgt, acc.w);
  }
  const float inv = 1.f / l;
  const uint32_t lo = ptx::pack_bf16x2(acc.x * inv, acc.y * inv);
  const uint32_t hi = ptx::pack_bf16x2(acc.z * inv, acc.w * inv);
  uint2* dst = reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(p.out) + (static_cast<uint64_t>(i) * p.Hq + h) * kD +
                                        lane * 4);
  *dst = make_uint2(lo, hi);
  if (p.lse && lane == 0) p.lse[static_cast<uint64_t>(i) * p.Hq + h] = (M + log2f(le)) * 0.6931471805599453f;
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

size_t decode_smem_bytes(uint32_t Hkv) {
  if (Hkv == 0 || Hkv > 8) return 0;
  return static_cast<size_t>(kRing) * stage_bytes(Hkv) + 2 * kRing * sizeof(uint64_t);
}

cudaError_t decode_setup() {
  const int smem = static_cast<int>(decode_smem_bytes(8));
  cudaError_t e = cudaFuncSetAttribute(paged_decode_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(paged_decode_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
}

cudaError_t launch_decode(const DecodeParams& p, cudaStream_t stream) {
  const size_t smem = decode_smem_bytes(p.Hkv);
  const unsigned threads = (p.Hkv + 1) * 32;
  if (p.G == 1)
    paged_decode_kernel<false><<<p.ncta, threads, smem, stream>>>(p);
  else
    paged_decode_kernel<true><<<p.ncta, threads, smem, stream>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_merge(const DecodeParams& p, cudaStream_t stream) {
  const unsigned warps = p.nseq * p.Hq;
  merge_partials_kernel<<<(warps + 3) / 4, 128, 0, stream>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_append(const AppendParams& p, cudaStream_t stream) {
  if (p.nseq == 0) return cudaSuccess;
  append_kv_kernel<<<p.nseq, 128, 0, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace ema
