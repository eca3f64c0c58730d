// attention_tiles.cuh — per-warp tile arithmetic of the paged decode attention: one KV head, one
// block of up to 16 tokens held in shared memory as a K half-stage and a V half-stage. A half-stage
// is a byte copy of one plane of a KV block as it lies in HBM: [16 token rows][Hkv * 256 B], where
// within every 128 bytes of a row the 16-byte unit u is stored at unit u ^ (row & 7). The block
// format carries this swizzle so that ONE linear bulk copy per plane fills the stage (small copies
// cap the rate an SM can stream at) and the same unit of 8 consecutive tokens, which is what
// ldmatrix fetches, still lies in 8 different bank groups.
//   * G >= 2: tensor-core tiles in swapped form, S^T[16 tokens x 8 heads] = K Q^T and
//     O^T[128 x 8] += V^T P^T (mma.sync m16n8k16 bf16, f32 accumulate), heads padded to 8;
//   * G == 1: f32 FMAs (no dense tile to feed a tensor core).
// Online softmax in the log2 domain; tokens past the sequence length get -inf scores and their V
// rows are zeroed, so NaN bit patterns in block tails cannot reach the output.
#pragma once

#include "ptx.cuh"

namespace ema {

constexpr uint32_t kD = 128;
constexpr uint32_t kT = 16;
constexpr float kNegInf = -INFINITY;

// Offset, from the start of a KV head's 256 bytes in token row 0, of 16-byte unit j (0..15) of the
// head in token row r; rb = bytes per token row.
__device__ __forceinline__ uint32_t swz(uint32_t r, uint32_t j, uint32_t rb) {
  return r * rb + (j >> 3) * 128 + (((j & 7u) ^ (r & 7u)) << 4);
}

struct SegState {
  float m0, m1;  // running max of the two heads this thread owns (MMA path) / of the head (ALU path)
  float l0, l1;  // running sums of the weights as used in P*V (per-thread partial)
  float e0, e1;  // running sums of the unrounded weights, for the log-sum-exp
};

// Scores and softmax of one tile (K half-stage). Leaves the bf16 weights P^T for the P*V product in
// pb0 (tokens 0..7) and pb1 (tokens 8..15) and the rescale factors of the two owned heads in al0/al1.
__device__ __forceinline__ void tile_mma_scores(uint32_t k_head, uint32_t rb, uint32_t valid,
                                                const uint32_t (&qf)[8][2], float scale_log2, SegState& st,
                                                uint32_t& pb0, uint32_t& pb1, float& al0, float& al1) {
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t mj = lane >> 3, mr = lane & 7u;
  // K fragment rows: matrix mj covers tokens (mj&1)*8.., dims (mj>>1)*8.. of each 16-dim step.
  const uint32_t row = (mj & 1u) * 8 + mr, unit = mj >> 1;
  float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int ks = 0; ks < 8; ks += 2) {
    uint32_t a[4], b[4];
    ptx::ldmatrix_x4(a, k_head + swz(row, 2 * ks + unit, rb));
    ptx::ldmatrix_x4(b, k_head + swz(row, 2 * ks + 2 + unit, rb));
    ptx::mma_bf16_16816(sa, a, qf[ks][0], qf[ks][1]);
    ptx::mma_bf16_16816(sb, b, qf[ks + 1][0], qf[ks + 1][1]);
  }
  const uint32_t r0 = lane >> 2;
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
  al0 = ptx::exp2_approx(st.m0 - mn0);
  al1 = ptx::exp2_approx(st.m1 - mn1);
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
  pb0 = ptx::movmatrix_trans(p01);
  pb1 = ptx::movmatrix_trans(p23);
}

// O^T += V^T P^T for one tile (V half-stage), after rescaling O by the factors of tile_mma_scores.
__device__ __forceinline__ void tile_mma_pv(uint32_t v_head, uint32_t rb, uint32_t valid,
                                            uint32_t pb0, uint32_t pb1, float al0, float al1, float (&o)[8][4]) {
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t mj = lane >> 3, mr = lane & 7u, tig = lane & 3u;
  // V^T fragment rows: matrix mj covers tokens (mj>>1)*8.., dims (mj&1)*8.. of each 16-dim step.
  const uint32_t row = (mj >> 1) * 8 + mr, unit = mj & 1u;
  uint32_t keep_lo = 0xffffffffu, keep_hi = 0xffffffffu;  // token pairs (2tig, 2tig+1) and (+8, +9)
  if (valid < kT) {
    const uint32_t t = 2 * tig;
    keep_lo = (t < valid ? 0x0000ffffu : 0u) | (t + 1 < valid ? 0xffff0000u : 0u);
    keep_hi = (t + 8 < valid ? 0x0000ffffu : 0u) | (t + 9 < valid ? 0xffff0000u : 0u);
  }
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) {
    uint32_t a[4];
    ptx::ldmatrix_x4_trans(a, v_head + swz(row, 2 * mt + unit, rb));
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

// f32 scores for G == 1: lane pair (2t, 2t+1) scores token t. Returns this lane's weight p (the
// weight of token lane/2) and the rescale factor al.
__device__ __forceinline__ void tile_alu_scores(const uint8_t* k_head, uint32_t rb, uint32_t valid, const float (&qh)[64],
                                                float scale_log2,
                                                SegState& st, float& p, float& al) {
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t t = lane >> 1, half = lane & 1u;
  float acc = 0.f;
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    const uint4 v = *reinterpret_cast<const uint4*>(k_head + swz(t, half * 8 + c, rb));
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      acc = fmaf(qh[c * 8 + 2 * e], __uint_as_float(w[e] << 16), acc);
      acc = fmaf(qh[c * 8 + 2 * e + 1], __uint_as_float(w[e] & 0xffff0000u), acc);
    }
  }
  acc += __shfl_xor_sync(0xffffffffu, acc, 1);
  const float s = t < valid ? acc * scale_log2 : kNegInf;
  float mx = s;
#pragma unroll
  for (int sh = 2; sh <= 16; sh <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, sh));
  const float mn = fmaxf(st.m0, mx);
  al = ptx::exp2_approx(st.m0 - mn);
  st.m0 = mn;
  p = ptx::exp2_approx(s - mn);
  st.l0 = st.l0 * al + (half == 0 ? p : 0.f);
}

// f32 P*V for G == 1: lane l owns output dims 4l..4l+3.
__device__ __forceinline__ void tile_alu_pv(const uint8_t* v_head, uint32_t rb, uint32_t valid, float p, float al,
                                            float (&o)[4]) {
  const uint32_t lane = threadIdx.x & 31u;
#pragma unroll
  for (int e = 0; e < 4; ++e) o[e] *= al;
  for (uint32_t tt = 0; tt < valid; ++tt) {
    const float pt = __shfl_sync(0xffffffffu, p, 2 * tt);
    const uint2 v = *reinterpret_cast<const uint2*>(v_head + swz(tt, lane >> 1, rb) + (lane & 1u) * 8);
    o[0] = fmaf(pt, __uint_as_float(v.x << 16), o[0]);
    o[1] = fmaf(pt, __uint_as_float(v.x & 0xffff0000u), o[1]);
    o[2] = fmaf(pt, __uint_as_float(v.y << 16), o[2]);
    o[3] = fmaf(pt, __uint_as_float(v.y & 0xffff0000u), o[3]);
  }
}

}  // namespace ema
