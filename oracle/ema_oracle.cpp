// ema_oracle.cpp — plain CPU oracle for the memory-slice hot path.
//
// TEST INFRASTRUCTURE ONLY. This file is the slow, obviously-correct statement of what the
// CUDA path must compute. It shares no code, header, table or helper with the CUDA library,
// and the product never calls it: only the tests, the smoke check and the benchmark's CPU
// baseline load it.
//
// What it states, and the passage of the paper each part follows:
//   * O-alloc   — a memory slice keeps a mapping table per user and hands out capacity from
//                 free memory first (Section 4, "Memory Slice", and Section 4.1: "first attempts
//                 to allocate from free memory"); block ids apply uniformly to every layer
//                 (Section 4.2.1, layer-major allocation).
//   * O-gather  — data that lives in the peer's part of the slice is copied into a buffer of
//                 one transferred chunk before the layer that reads it runs (Section 2.3 latency
//                 window; Section 4.2.1 "prefetched in time"; Section 4.2.2 swap buffer;
//                 Section 5.1 "prepares a directly accessible address").
//   * O-attn    — the consumer of the prepared addresses: decode attention over a paged KV
//                 cache. The paper inherits it from its serving engine (Section 6.1) and does
//                 not define it; the definition used is softmax(scale * q K^T) V per query head,
//                 with grouped-query head mapping g = h / (Hq / Hkv), in fp64.
//   * O-reclaim — the lender regains capacity at once (Section 4.1, static-dynamic symmetry).
//                 The paper does it by preempting the borrower; this build migrates the lent
//                 blocks instead and rewrites the mapping tables (the variant the task fixes).
//   * O-append  — one new token's K/V row written to its home block and to the staged copy.
//   * O-preempt — the paper's own reclaim (Section 4.1): when the lender wants capacity back and
//                 the borrower has no room to keep the data, requests of the borrower are evicted
//                 until it has; the allocator picks "a slab ... that contains the fewest number
//                 of active requests" (Section 4.2.1); after a preemption above the static share
//                 the user's allocations are capped for a window T (Section 5.3, bursty workload
//                 preemption control); preemptions are counted by cause (Section 6.6).
//   * O-slab    — Section 4.2.1: the slice hands out slabs, runs of consecutive block ids that belong
//                 to one user as a whole (a slab returns to the slice only when its last block is
//                 freed); Sections 4.2.1-4.2.3: the three memory layouts (layer-major, slab-major,
//                 layer-group-major) as address maps, the layer group as the unit of a swap, and
//                 the sizes of the contiguous pieces a swap of one layer group moves (S..mS, kS,
//                 kS..mkS), found by brute force over the address map.
//   * O-schedule — the choice among several slices (Section 5.2, Greedy-Least-Loaded) is stated in
//                 the Python front end (gll_choose, exact rationals); pins in
//                 tests/test_oracle_schedule.py.
//
// Parity pins (tests/test_oracle_*.py): paged == dense brute force; softmax row sums; closed
// forms (n=1, equal keys, constant V, dominant key, score shift, token permutation); fp64
// library attention; NaN-poisoned tails; tag round trips for gather; byte/logical-order
// preservation for migration; allocator invariants under random operation sequences; for
// O-preempt hand-worked victim choices and cap time lines, twin states that reclaim without
// preemption, a brute-force request count per slab, and the back-and-forth scenario of
// Section 5.3 with and without the cap (tests/test_oracle_preempt.py).
// Bit-level agreement of the GPU attention with this file is "parity unpinned" beyond the
// stated tolerance, by design: any result within tolerance is correct.
//
// Block layout (bytes): K plane [T][Hkv][D] bf16, then V plane [T][Hkv][D] bf16.
// Arena layout: [layer][block id][block bytes].
// Block-table entry (int32): e >= 0 -> local id e; e < 0 -> lent id ~e.
// Resolved entry (int32):    e >= 0 -> local id e; e < 0 -> staging position ~e.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <map>
#include <utility>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

enum Status : int {
  OK = 0,
  E_INVAL = -1,
  E_NOSPC = -2,
  E_STAGING = -3,
  E_STATE = -7,
  E_CAPPED = -9,
};

enum Tier : int { AUTO = 0, LOCAL = 1, LENT = 2 };

struct Seq {
  std::vector<int32_t> table;  // logical block -> entry
  uint32_t len = 0;            // tokens
};

struct Owner {
  int32_t seq = -1;
  int32_t logical = -1;
};

struct State {
  uint32_t num_layers = 0;
  uint32_t block_tokens = 0;
  uint64_t block_bytes = 0;
  uint32_t local_blocks = 0;
  uint32_t lent_cap = 0;   // current lent capacity (ids < lent_cap may be used)
  uint32_t lent_phys = 0;  // physical size of the lent arena, in block ids
  uint32_t ring_slots = 0;
  uint32_t staging_cap = 0;  // blocks per ring slot
  uint32_t max_seqs = 0;
  uint32_t max_blocks_per_seq = 0;
  // Free stacks: back() is the next id popped.
  std::vector<int32_t> free_local;
  std::vector<int32_t> free_lent;
  // Order in which never-yet-lent ids are revealed is irrelevant: lend() pushes explicit ids.
  std::map<int32_t, Seq> seqs;
  std::vector<Owner> owner_local;
  std::vector<Owner> owner_lent;
  // Preemption control (O-preempt). Time is a number the caller sets; the window is in its unit.
  uint64_t now = 0;
  uint64_t window = 0;      // T; 0 = no cap is ever set
  uint64_t cap_until = 0;   // a cap holds while now < cap_until
  uint32_t cap_level = 0;   // blocks the user may hold while the cap holds
  uint64_t preempt_oom = 0, preempt_reclaim = 0;
  // O-slab: blocks per slab; 0 = block-granular free stacks (the seeded orders), no slabs.
  uint32_t slab = 0;
};

inline uint32_t used_blocks(const State* s) {
  uint32_t u = 0;
  for (const auto& kv : s->seqs) u += static_cast<uint32_t>(kv.second.table.size());
  return u;
}
inline bool cap_holds(const State* s) { return s->window > 0 && s->now < s->cap_until; }

inline double bf16_to_double(uint16_t b) {
  uint32_t u = static_cast<uint32_t>(b) << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return static_cast<double>(f);
}

// Round-to-nearest-even conversion double -> bf16, through float.
inline uint16_t double_to_bf16_rne(double x) {
  float f = static_cast<float>(x);
  uint32_t u;
  std::memcpy(&u, &f, 4);
  if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu)) return static_cast<uint16_t>((u >> 16) | 0x40);
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb;
  return static_cast<uint16_t>(u >> 16);
}

inline uint32_t blocks_for(uint32_t len, uint32_t block_tokens) {
  return (len + block_tokens - 1) / block_tokens;
}

// The next free id of a part of the slice. Without slabs: the top of the free stack. With slabs
// (Section 4.2.1): a slab belongs to the user as long as one of its blocks is in use, and the
// user fills the slabs it already has before it asks the slice for another one: the lowest free
// id that lies in a slab holding a block in use; failing that the lowest free id of all, which
// opens the lowest free slab. The caller has checked that a free id exists.
int32_t take_free(State* s, bool local) {
  std::vector<int32_t>& fr = local ? s->free_local : s->free_lent;
  if (s->slab == 0) {
    const int32_t id = fr.back();
    fr.pop_back();
    return id;
  }
  const std::vector<Owner>& own = local ? s->owner_local : s->owner_lent;
  int32_t in_open_slab = -1, any = -1;
  for (int32_t f : fr) {
    if (any < 0 || f < any) any = f;
    const uint32_t first = static_cast<uint32_t>(f) / s->slab * s->slab;
    bool in_use = false;
    for (uint32_t id = first; id < first + s->slab && id < own.size(); ++id) in_use = in_use || own[id].seq >= 0;
    if (in_use && (in_open_slab < 0 || f < in_open_slab)) in_open_slab = f;
  }
  const int32_t id = in_open_slab >= 0 ? in_open_slab : any;
  fr.erase(std::find(fr.begin(), fr.end(), id));
  return id;
}

}  // namespace

extern "C" {

// ------------------------------------------------------------------------------------------
// O-alloc
// ------------------------------------------------------------------------------------------

// free orders: local_free_order has local_blocks ids, lent_free_order has lent_phys ids (a
// permutation of the arena); NULL means identity. Pops return order[0], order[1], ...; the lent
// stack initially holds only the ids < lent_blocks, in that order.
void* oracle_create(uint32_t num_layers, uint32_t block_tokens, uint64_t block_bytes,
                    uint32_t local_blocks, uint32_t lent_blocks, uint32_t lent_phys,
                    uint32_t ring_slots, uint32_t staging_cap, uint32_t max_seqs,
                    uint32_t max_blocks_per_seq, const uint32_t* local_free_order,
                    const uint32_t* lent_free_order) {
  if (lent_blocks > lent_phys || ring_slots == 0 || block_tokens == 0) return nullptr;
  State* s = new State();
  s->num_layers = num_layers;
  s->block_tokens = block_tokens;
  s->block_bytes = block_bytes;
  s->local_blocks = local_blocks;
  s->lent_cap = lent_blocks;
  s->lent_phys = lent_phys;
  s->ring_slots = ring_slots;
  s->staging_cap = staging_cap;
  s->max_seqs = max_seqs;
  s->max_blocks_per_seq = max_blocks_per_seq;
  s->owner_local.assign(local_blocks, Owner());
  s->owner_lent.assign(lent_phys, Owner());
  for (uint32_t k = local_blocks; k-- > 0;) {
    s->free_local.push_back(static_cast<int32_t>(local_free_order ? local_free_order[k] : k));
  }
  for (uint32_t k = lent_phys; k-- > 0;) {
    uint32_t id = lent_free_order ? lent_free_order[k] : k;
    if (id < lent_blocks) s->free_lent.push_back(static_cast<int32_t>(id));
  }
  return s;
}

void oracle_destroy(void* h) { delete static_cast<State*>(h); }

// O-slab: turns the slab allocator on (blocks per slab; the paper's default is 10, Section 6.7).
// To be called before the first allocation; capacities need not be multiples of the slab (the
// last slab of a part is then short).
int oracle_set_slab_blocks(void* h, uint32_t slab_blocks) {
  State* s = static_cast<State*>(h);
  if (!s->seqs.empty()) return E_STATE;
  s->slab = slab_blocks;
  return OK;
}

int oracle_alloc_blocks(void* h, int32_t seq, uint32_t n, int32_t hint, int32_t* out_entries) {
  State* s = static_cast<State*>(h);
  if (seq < 0 || hint < AUTO || hint > LENT) return E_INVAL;
  auto it = s->seqs.find(seq);
  const bool exists = it != s->seqs.end();
  if (!exists && s->seqs.size() >= s->max_seqs) return E_INVAL;
  const size_t have = exists ? it->second.table.size() : 0;
  if (have + n > s->max_blocks_per_seq) return E_INVAL;
  // Section 5.3: while a cap from an earlier preemption holds, the user may not grow past it.
  if (n > 0 && cap_holds(s) && used_blocks(s) + n > s->cap_level) return E_CAPPED;
  const size_t fl = s->free_local.size(), fr = s->free_lent.size();
  if (hint == AUTO && n > fl + fr) return E_NOSPC;
  if (hint == LOCAL && n > fl) return E_NOSPC;
  if (hint == LENT && n > fr) return E_NOSPC;
  Seq& q = s->seqs[seq];  // creates when absent
  for (uint32_t k = 0; k < n; ++k) {
    bool take_local = hint == LOCAL || (hint == AUTO && !s->free_local.empty());
    int32_t entry;
    if (take_local) {
      int32_t id = take_free(s, true);
      s->owner_local[id] = Owner{seq, static_cast<int32_t>(q.table.size())};
      entry = id;
    } else {
      int32_t id = take_free(s, false);
      s->owner_lent[id] = Owner{seq, static_cast<int32_t>(q.table.size())};
      entry = ~id;
    }
    q.table.push_back(entry);
    if (out_entries) out_entries[k] = entry;
  }
  return OK;
}

int oracle_set_seq_len(void* h, int32_t seq, uint32_t len) {
  State* s = static_cast<State*>(h);
  auto it = s->seqs.find(seq);
  if (it == s->seqs.end()) return E_STATE;
  if (len > static_cast<uint64_t>(it->second.table.size()) * s->block_tokens) return E_INVAL;
  it->second.len = len;
  return OK;
}

int oracle_free_seq(void* h, int32_t seq) {
  State* s = static_cast<State*>(h);
  auto it = s->seqs.find(seq);
  if (it == s->seqs.end()) return E_STATE;
  const std::vector<int32_t>& t = it->second.table;
  for (size_t b = t.size(); b-- > 0;) {  // descending logical order
    int32_t e = t[b];
    if (e >= 0) {
      s->free_local.push_back(e);
      s->owner_local[e] = Owner();
    } else {
      s->free_lent.push_back(~e);
      s->owner_lent[~e] = Owner();
    }
  }
  s->seqs.erase(it);
  return OK;
}

int oracle_get_block_table(void* h, int32_t seq, int32_t* out, uint32_t cap, uint32_t* n,
                           uint32_t* len) {
  State* s = static_cast<State*>(h);
  auto it = s->seqs.find(seq);
  if (it == s->seqs.end()) return E_STATE;
  const std::vector<int32_t>& t = it->second.table;
  if (n) *n = static_cast<uint32_t>(t.size());
  if (len) *len = it->second.len;
  if (out) {
    if (cap < t.size()) return E_INVAL;
    std::copy(t.begin(), t.end(), out);
  }
  return OK;
}

// Free stacks in pop order (first element = next id popped). which: 1 local, 2 lent.
int oracle_get_free_stack(void* h, int32_t which, int32_t* out, uint32_t cap, uint32_t* n) {
  State* s = static_cast<State*>(h);
  const std::vector<int32_t>& st = which == LOCAL ? s->free_local : s->free_lent;
  if (n) *n = static_cast<uint32_t>(st.size());
  if (out) {
    if (cap < st.size()) return E_INVAL;
    for (size_t k = 0; k < st.size(); ++k) out[k] = st[st.size() - 1 - k];
  }
  return OK;
}

uint32_t oracle_lent_capacity(void* h) { return static_cast<State*>(h)->lent_cap; }
uint32_t oracle_num_seqs(void* h) { return static_cast<uint32_t>(static_cast<State*>(h)->seqs.size()); }

// ------------------------------------------------------------------------------------------
// O-gather: resolve a batch's tables and copy every in-use lent block of `layer` into ring
// slot (layer mod R), in canonical order: batch position, then logical index.
// resolved is [nseq][max_blocks_per_seq] (entries past a sequence's in-use blocks are left as is).
// lent_arena / staging may be NULL: then only the integer results are produced.
// ------------------------------------------------------------------------------------------
int oracle_gather(void* h, uint32_t layer, const int32_t* seqs, uint32_t nseq,
                  const uint8_t* lent_arena, uint8_t* staging, int32_t* resolved, uint32_t* k_out) {
  State* s = static_cast<State*>(h);
  if (layer >= s->num_layers) return E_INVAL;
  for (uint32_t i = 0; i < nseq; ++i) {
    if (s->seqs.find(seqs[i]) == s->seqs.end()) return E_STATE;
    for (uint32_t j = 0; j < i; ++j)
      if (seqs[j] == seqs[i]) return E_INVAL;
  }
  // Count first, so that an overflow is reported before any byte moves.
  uint64_t total = 0;
  for (uint32_t i = 0; i < nseq; ++i) {
    const Seq& q = s->seqs[seqs[i]];
    uint32_t nb = blocks_for(q.len, s->block_tokens);
    for (uint32_t b = 0; b < nb; ++b)
      if (q.table[b] < 0) ++total;
  }
  if (total > s->staging_cap) return E_STAGING;
  const uint64_t bb = s->block_bytes;
  const uint64_t lent_layer = static_cast<uint64_t>(s->lent_phys) * bb;
  const uint64_t slot_bytes = static_cast<uint64_t>(s->staging_cap) * bb;
  const uint32_t slot = layer % s->ring_slots;
  uint32_t k = 0;
  for (uint32_t i = 0; i < nseq; ++i) {
    const Seq& q = s->seqs[seqs[i]];
    uint32_t nb = blocks_for(q.len, s->block_tokens);
    for (uint32_t b = 0; b < nb; ++b) {
      int32_t e = q.table[b];
      int32_t r;
      if (e >= 0) {
        r = e;
      } else {
        if (lent_arena && staging) {
          const uint8_t* src = lent_arena + layer * lent_layer + static_cast<uint64_t>(~e) * bb;
          uint8_t* dst = staging + slot * slot_bytes + static_cast<uint64_t>(k) * bb;
          std::memcpy(dst, src, bb);
        }
        r = ~static_cast<int32_t>(k);
        ++k;
      }
      if (resolved) resolved[static_cast<uint64_t>(i) * s->max_blocks_per_seq + b] = r;
    }
  }
  if (k_out) *k_out = k;
  return OK;
}

// The way back: every staged block of the batch is written to its home in the lent arena.
int oracle_scatter(void* h, uint32_t layer, const int32_t* seqs, uint32_t nseq,
                   const uint8_t* staging, uint8_t* lent_arena) {
  State* s = static_cast<State*>(h);
  if (layer >= s->num_layers) return E_INVAL;
  const uint64_t bb = s->block_bytes;
  const uint64_t lent_layer = static_cast<uint64_t>(s->lent_phys) * bb;
  const uint64_t slot_bytes = static_cast<uint64_t>(s->staging_cap) * bb;
  const uint32_t slot = layer % s->ring_slots;
  uint32_t k = 0;
  for (uint32_t i = 0; i < nseq; ++i) {
    auto it = s->seqs.find(seqs[i]);
    if (it == s->seqs.end()) return E_STATE;
    const Seq& q = it->second;
    uint32_t nb = blocks_for(q.len, s->block_tokens);
    for (uint32_t b = 0; b < nb; ++b) {
      int32_t e = q.table[b];
      if (e >= 0) continue;
      std::memcpy(lent_arena + layer * lent_layer + static_cast<uint64_t>(~e) * bb,
                  staging + slot * slot_bytes + static_cast<uint64_t>(k) * bb, bb);
      ++k;
    }
  }
  return OK;
}

// ------------------------------------------------------------------------------------------
// O-attn: decode attention read through resolved tables, fp64.
//   q        [nseq][Hq][D] bf16 bit patterns
//   local    base of this layer's local arena  [id][2][T][Hkv][D] bf16
//   staging  base of this layer's ring slot    [pos][2][T][Hkv][D] bf16
//   resolved [nseq][table_stride] ; lens [nseq]
//   out      [nseq][Hq][D] double ; lse [nseq][Hq] double (may be NULL)
// Tokens t >= len are excluded, not multiplied by zero.
// ------------------------------------------------------------------------------------------
int oracle_paged_attention(const uint16_t* q, const uint16_t* local, const uint16_t* staging,
                           const int32_t* resolved, uint32_t table_stride, const uint32_t* lens,
                           uint32_t nseq, uint32_t Hq, uint32_t Hkv, uint32_t D, uint32_t T,
                           double sm_scale, double* out, double* lse) {
  if (Hkv == 0 || Hq % Hkv != 0) return E_INVAL;
  for (uint32_t i = 0; i < nseq; ++i)
    if (lens[i] == 0) return E_INVAL;
  const uint32_t G = Hq / Hkv;
  const uint64_t plane = static_cast<uint64_t>(T) * Hkv * D;  // elements
  const uint64_t block_elems = 2 * plane;
  const int64_t npairs = static_cast<int64_t>(nseq) * Hq;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t pair = 0; pair < npairs; ++pair) {
    const uint32_t i = static_cast<uint32_t>(pair / Hq);
    const uint32_t hq = static_cast<uint32_t>(pair % Hq);
    const uint32_t g = hq / G;
    const uint32_t n = lens[i];
    const uint16_t* qv = q + (static_cast<uint64_t>(i) * Hq + hq) * D;
    std::vector<double> sc(n);
    double m = -std::numeric_limits<double>::infinity();
    for (uint32_t t = 0; t < n; ++t) {
      int32_t e = resolved[static_cast<uint64_t>(i) * table_stride + t / T];
      const uint16_t* blk = e >= 0 ? local + static_cast<uint64_t>(e) * block_elems
                                   : staging + static_cast<uint64_t>(~e) * block_elems;
      const uint16_t* krow = blk + (static_cast<uint64_t>(t % T) * Hkv + g) * D;
      double acc = 0.0;
      for (uint32_t d = 0; d < D; ++d) acc += bf16_to_double(qv[d]) * bf16_to_double(krow[d]);
      sc[t] = sm_scale * acc;
      if (sc[t] > m) m = sc[t];
    }
    double l = 0.0;
    std::vector<double> o(D, 0.0);
    for (uint32_t t = 0; t < n; ++t) {
      int32_t e = resolved[static_cast<uint64_t>(i) * table_stride + t / T];
      const uint16_t* blk = e >= 0 ? local + static_cast<uint64_t>(e) * block_elems
                                   : staging + static_cast<uint64_t>(~e) * block_elems;
      const uint16_t* vrow = blk + plane + (static_cast<uint64_t>(t % T) * Hkv + g) * D;
      double p = std::exp(sc[t] - m);
      l += p;
      for (uint32_t d = 0; d < D; ++d) o[d] += p * bf16_to_double(vrow[d]);
    }
    double* od = out + (static_cast<uint64_t>(i) * Hq + hq) * D;
    for (uint32_t d = 0; d < D; ++d) od[d] = o[d] / l;
    if (lse) lse[static_cast<uint64_t>(i) * Hq + hq] = m + std::log(l);
  }
  return OK;
}

// Brute force on a dense, contiguous cache: K, V are [n][Hkv][D] bf16 for ONE sequence.
// Also returns the normalised probabilities (probs [Hq][n], may be NULL) for the row-sum pin.
int oracle_dense_attention(const uint16_t* q, const uint16_t* K, const uint16_t* V, uint32_t n,
                           uint32_t Hq, uint32_t Hkv, uint32_t D, double sm_scale, double* out,
                           double* lse, double* probs) {
  if (n == 0 || Hkv == 0 || Hq % Hkv != 0) return E_INVAL;
  const uint32_t G = Hq / Hkv;
  for (uint32_t hq = 0; hq < Hq; ++hq) {
    const uint32_t g = hq / G;
    std::vector<double> sc(n);
    double m = -std::numeric_limits<double>::infinity();
    for (uint32_t t = 0; t < n; ++t) {
      const uint16_t* krow = K + (static_cast<uint64_t>(t) * Hkv + g) * D;
      double acc = 0.0;
      for (uint32_t d = 0; d < D; ++d) acc += bf16_to_double(q[hq * D + d]) * bf16_to_double(krow[d]);
      sc[t] = sm_scale * acc;
      m = std::max(m, sc[t]);
    }
    double l = 0.0;
    std::vector<double> o(D, 0.0);
    for (uint32_t t = 0; t < n; ++t) {
      const uint16_t* vrow = V + (static_cast<uint64_t>(t) * Hkv + g) * D;
      double p = std::exp(sc[t] - m);
      l += p;
      for (uint32_t d = 0; d < D; ++d) o[d] += p * bf16_to_double(vrow[d]);
    }
    for (uint32_t d = 0; d < D; ++d) out[static_cast<uint64_t>(hq) * D + d] = o[d] / l;
    if (lse) lse[hq] = m + std::log(l);
    if (probs)
      for (uint32_t t = 0; t < n; ++t) probs[static_cast<uint64_t>(hq) * n + t] = std::exp(sc[t] - m) / l;
  }
  return OK;
}

// Elementwise double -> bf16 (round to nearest even), for reporting.
void oracle_to_bf16(const double* x, uint16_t* y, uint64_t n) {
  for (uint64_t k = 0; k < n; ++k) y[k] = double_to_bf16_rne(x[k]);
}

// ------------------------------------------------------------------------------------------
// O-reclaim: the lender takes the top `take` ids of the lent range; in-use blocks there move,
// for every layer, to free local ids first and then to the smallest free lent id below the cut.
// Arenas may be NULL (integer state only).
// ------------------------------------------------------------------------------------------
int oracle_reclaim(void* h, uint32_t take, uint8_t* local_arena, uint8_t* lent_arena,
                   uint64_t* out_migrated) {
  State* s = static_cast<State*>(h);
  if (take > s->lent_cap) take = s->lent_cap;
  const uint32_t cut = s->lent_cap - take;
  std::vector<int32_t> victims;
  for (uint32_t id = cut; id < s->lent_cap; ++id)
    if (s->owner_lent[id].seq >= 0) victims.push_back(static_cast<int32_t>(id));
  size_t free_below = 0;
  for (int32_t id : s->free_lent)
    if (static_cast<uint32_t>(id) < cut) ++free_below;
  if (victims.size() > s->free_local.size() + free_below) return E_NOSPC;
  // Free ids at or above the cut leave the stack; the others keep their relative order.
  std::vector<int32_t> kept;
  for (int32_t id : s->free_lent)
    if (static_cast<uint32_t>(id) < cut) kept.push_back(id);
  s->free_lent.swap(kept);
  const uint64_t bb = s->block_bytes;
  const uint64_t local_layer = static_cast<uint64_t>(s->local_blocks) * bb;
  const uint64_t lent_layer = static_cast<uint64_t>(s->lent_phys) * bb;
  for (int32_t v : victims) {
    Owner own = s->owner_lent[v];
    bool to_local = !s->free_local.empty();
    int32_t dst;
    if (to_local) {
      dst = take_free(s, true);
    } else if (s->slab) {
      dst = take_free(s, false);  // what is left of the lent list lies below the cut
    } else {
      auto mn = std::min_element(s->free_lent.begin(), s->free_lent.end());
      dst = *mn;
      s->free_lent.erase(mn);
    }
    if (local_arena && lent_arena) {
      for (uint32_t l = 0; l < s->num_layers; ++l) {
        const uint8_t* src = lent_arena + l * lent_layer + static_cast<uint64_t>(v) * bb;
        uint8_t* d = to_local ? local_arena + l * local_layer + static_cast<uint64_t>(dst) * bb
                              : lent_arena + l * lent_layer + static_cast<uint64_t>(dst) * bb;
        std::memcpy(d, src, bb);
      }
    }
    s->seqs[own.seq].table[own.logical] = to_local ? dst : ~dst;
    if (to_local) s->owner_local[dst] = own; else s->owner_lent[dst] = own;
    s->owner_lent[v] = Owner();
  }
  s->lent_cap = cut;
  if (out_migrated) *out_migrated = victims.size();
  return OK;
}

// ------------------------------------------------------------------------------------------
// O-preempt: reclaim by preemption, the cap that follows it, and the counters.
// ------------------------------------------------------------------------------------------

// Time and window T of the preemption cap (Section 5.3). The paper gives T no unit: the caller
// chooses one and reports the time in it; time never runs backwards.
int oracle_set_preempt_window(void* h, uint64_t window) {
  static_cast<State*>(h)->window = window;
  return OK;
}

int oracle_set_time(void* h, uint64_t now) {
  State* s = static_cast<State*>(h);
  if (now < s->now) return E_INVAL;
  s->now = now;
  return OK;
}

namespace {
// Section 5.3: a user preempted while it holds more than its static share (its own, local part of
// the slice: half of a symmetric slice) is limited to the level it was preempted to; a later
// preemption inside the window can only lower the level, and every one restarts the window.
void note_reclaim_preemption(State* s, uint32_t used_before, uint32_t used_after) {
  if (s->window == 0 || used_before <= s->local_blocks) return;
  s->cap_level = cap_holds(s) ? std::min(s->cap_level, used_after) : used_after;
  s->cap_until = s->now + s->window;
}
}  // namespace

// One request is preempted by the engine's own choice. cause: 1 = out of memory (the user's own
// requests give way because capacity is exhausted), 2 = reclamation by the lender (Section 5.2
// names the two causes, Section 6.6 counts them). Only cause 2 can set the cap.
int oracle_preempt_seq(void* h, int32_t seq, int32_t cause) {
  State* s = static_cast<State*>(h);
  if (cause != 1 && cause != 2) return E_INVAL;
  if (s->seqs.find(seq) == s->seqs.end()) return E_STATE;
  const uint32_t before = used_blocks(s);
  oracle_free_seq(h, seq);
  if (cause == 1) {
    ++s->preempt_oom;
  } else {
    ++s->preempt_reclaim;
    note_reclaim_preemption(s, before, used_blocks(s));
  }
  return OK;
}

// The lender takes the top `take` ids back and the borrower may have no room for what is stored
// there. Section 4.1: requests of the borrower are evicted "until" enough is reclaimed; Section
// 4.2.1: the allocator takes the slab with the fewest active requests. Slabs are runs of
// slab_blocks consecutive lent ids (the last one may be short). While the blocks that must leave
// the reclaimed range outnumber the free places (local, or lent below the cut), the slab of the
// lent range that holds blocks of the fewest distinct requests (at least one; ties: the highest
// slab) loses all its requests, in ascending id order. What then remains in the range migrates as
// in O-reclaim. victims (cap entries) receives the evicted ids in eviction order.
// Returns E_INVAL, with nothing changed, when slab_blocks is 0 or cap is too small.
int oracle_reclaim_preempt(void* h, uint32_t take, uint32_t slab_blocks, uint8_t* local_arena,
                           uint8_t* lent_arena, int32_t* victims, uint32_t cap,
                           uint32_t* n_victims, uint64_t* out_migrated) {
  State* s = static_cast<State*>(h);
  if (slab_blocks == 0) return E_INVAL;
  if (take > s->lent_cap) take = s->lent_cap;
  const uint32_t cut = s->lent_cap - take;
  // Choose first (nothing changes if the caller's array is too small), on a copy of the owners.
  std::vector<int32_t> chosen;
  auto gone = [&](int32_t seq) {
    return std::find(chosen.begin(), chosen.end(), seq) != chosen.end();
  };
  for (;;) {
    size_t must_move = 0, room = s->free_local.size();
    for (uint32_t id = cut; id < s->lent_cap; ++id)
      if (s->owner_lent[id].seq >= 0 && !gone(s->owner_lent[id].seq)) ++must_move;
    for (int32_t id : s->free_lent)
      if (static_cast<uint32_t>(id) < cut) ++room;
    for (uint32_t id = 0; id < s->local_blocks; ++id)
      if (s->owner_local[id].seq >= 0 && gone(s->owner_local[id].seq)) ++room;
    for (uint32_t id = 0; id < cut; ++id)
      if (s->owner_lent[id].seq >= 0 && gone(s->owner_lent[id].seq)) ++room;
    if (must_move <= room) break;
    const uint32_t nslabs = (s->lent_cap + slab_blocks - 1) / slab_blocks;
    int64_t best = -1;
    size_t best_count = 0;
    std::vector<int32_t> best_set;
    for (uint32_t sl = 0; sl < nslabs; ++sl) {
      std::vector<int32_t> in_slab;
      const uint32_t hi = std::min(s->lent_cap, (sl + 1) * slab_blocks);
      for (uint32_t id = sl * slab_blocks; id < hi; ++id) {
        const int32_t q = s->owner_lent[id].seq;
        if (q >= 0 && !gone(q) && std::find(in_slab.begin(), in_slab.end(), q) == in_slab.end())
          in_slab.push_back(q);
      }
      if (in_slab.empty()) continue;
      if (best < 0 || in_slab.size() <= best_count) {  // <= : the highest slab wins a tie
        best = sl;
        best_count = in_slab.size();
        best_set = in_slab;
      }
    }
    std::sort(best_set.begin(), best_set.end());
    for (int32_t q : best_set) chosen.push_back(q);
  }
  if (chosen.size() > cap) return E_INVAL;
  const uint32_t before = used_blocks(s);
  for (size_t k = 0; k < chosen.size(); ++k) {
    oracle_free_seq(h, chosen[k]);
    if (victims) victims[k] = chosen[k];
    ++s->preempt_reclaim;
  }
  if (n_victims) *n_victims = static_cast<uint32_t>(chosen.size());
  const int rc = oracle_reclaim(h, take, local_arena, lent_arena, out_migrated);
  if (!chosen.empty()) note_reclaim_preemption(s, before, used_blocks(s));
  return rc;
}

// out[0..6) = preemptions by out-of-memory, preemptions by reclamation, now, window, cap_until,
// cap level in blocks (0 when no cap holds).
void oracle_preempt_state(void* h, uint64_t* out) {
  State* s = static_cast<State*>(h);
  out[0] = s->preempt_oom;
  out[1] = s->preempt_reclaim;
  out[2] = s->now;
  out[3] = s->window;
  out[4] = cap_holds(s) ? s->cap_until : 0;
  out[5] = cap_holds(s) ? s->cap_level : 0;
}

// The lender offers n more block ids: capacity grows, new ids pop in ascending order.
int oracle_lend(void* h, uint32_t n) {
  State* s = static_cast<State*>(h);
  if (static_cast<uint64_t>(s->lent_cap) + n > s->lent_phys) return E_INVAL;
  for (uint32_t k = n; k-- > 0;) s->free_lent.push_back(static_cast<int32_t>(s->lent_cap + k));
  s->lent_cap += n;
  return OK;
}

// ------------------------------------------------------------------------------------------
// O-append: token (len-1) of each sequence gets its K and V rows ([nseq][Hkv][D] bf16 each).
// staging_slot, when not NULL, is the ring slot that currently holds `layer` for this batch:
// rows whose home block is lent are written there too (position taken from the canonical order).
// ------------------------------------------------------------------------------------------
int oracle_append_kv(void* h, uint32_t layer, const int32_t* seqs, uint32_t nseq,
                     const uint16_t* k_new, const uint16_t* v_new, uint32_t Hkv, uint32_t D,
                     uint8_t* local_arena, uint8_t* lent_arena, uint8_t* staging_slot) {
  State* s = static_cast<State*>(h);
  if (layer >= s->num_layers) return E_INVAL;
  const uint64_t bb = s->block_bytes;
  const uint64_t row = static_cast<uint64_t>(Hkv) * D * 2;  // bytes of one token's K (or V) row
  const uint64_t plane = static_cast<uint64_t>(s->block_tokens) * row;
  if (2 * plane != bb) return E_INVAL;
  const uint64_t local_layer = static_cast<uint64_t>(s->local_blocks) * bb;
  const uint64_t lent_layer = static_cast<uint64_t>(s->lent_phys) * bb;
  uint32_t k = 0;  // staging position counter, canonical order
  for (uint32_t i = 0; i < nseq; ++i) {
    auto it = s->seqs.find(seqs[i]);
    if (it == s->seqs.end()) return E_STATE;
    const Seq& q = it->second;
    if (q.len == 0) return E_INVAL;
    const uint32_t nb = blocks_for(q.len, s->block_tokens);
    const uint32_t t = q.len - 1, b = t / s->block_tokens, r = t % s->block_tokens;
    const uint8_t* ks = reinterpret_cast<const uint8_t*>(k_new) + i * row;
    const uint8_t* vs = reinterpret_cast<const uint8_t*>(v_new) + i * row;
    for (uint32_t bi = 0; bi < nb; ++bi) {
      int32_t e = q.table[bi];
      if (bi == b) {
        uint8_t* home = e >= 0 ? local_arena + layer * local_layer + static_cast<uint64_t>(e) * bb
                               : lent_arena + layer * lent_layer + static_cast<uint64_t>(~e) * bb;
        std::memcpy(home + r * row, ks, row);
        std::memcpy(home + plane + r * row, vs, row);
        if (e < 0 && staging_slot) {
          uint8_t* st = staging_slot + static_cast<uint64_t>(k) * bb;
          std::memcpy(st + r * row, ks, row);
          std::memcpy(st + plane + r * row, vs, row);
        }
      }
      if (e < 0) ++k;
    }
  }
  return OK;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

// ------------------------------------------------------------------------------------------
// O-slab: memory layouts of Section 4.2 as address maps. An arena holds n_blocks block ids (a
// whole number of slabs of S ids) for each of L layers; a layer group is k consecutive layers
// (group g = layers g*k .. g*k + k - 1; L a multiple of k). The byte offset of block `id` of
// `layer` is the position of that block in the nested array the figure of each layout draws:
//   0 layer-major        [layer][id]                              (Section 4.2.1)
//   1 slab-major         [slab][layer][block in slab]             (Section 4.2.2: all layers of a
//                                                                  slab together)
//   2 layer-group-major  [group][slab][layer in group][block in slab]   (Section 4.2.3: slab i+1
//                                                                  of the same group follows slab i)
// ------------------------------------------------------------------------------------------
uint64_t oracle_layout_offset(uint32_t layout, uint32_t L, uint32_t n_blocks, uint32_t S, uint32_t k,
                              uint64_t block_bytes, uint32_t layer, uint32_t id) {
  const uint64_t slabs = n_blocks / S, slab = id / S, in_slab = id % S;
  uint64_t index = 0;  // in blocks
  if (layout == 0) {
    index = static_cast<uint64_t>(layer) * n_blocks + id;
  } else if (layout == 1) {
    index = (slab * L + layer) * S + in_slab;
  } else {
    const uint64_t group = layer / k, in_group = layer % k;
    index = ((group * slabs + slab) * k + in_group) * S + in_slab;
  }
  return index * block_bytes;
}

// The contiguous pieces that a swap of layer group `group` moves for a user who owns the listed
// slabs (Section 4.2.3 compares their sizes across the layouts), by brute force: the byte interval
// of every block of every listed slab in every layer of the group is laid on the address line,
// touching intervals are joined, and the lengths of the joined pieces are returned in ascending
// address order. Returns the number of pieces (out may be NULL to count).
uint32_t oracle_swap_pieces(uint32_t layout, uint32_t L, uint32_t n_blocks, uint32_t S, uint32_t k,
                            uint64_t block_bytes, uint32_t group, const uint32_t* slabs, uint32_t nslabs,
                            uint64_t* out_bytes, uint32_t cap) {
  std::vector<std::pair<uint64_t, uint64_t>> iv;
  for (uint32_t layer = group * k; layer < (group + 1) * k && layer < L; ++layer)
    for (uint32_t j = 0; j < nslabs; ++j)
      for (uint32_t b = 0; b < S; ++b) {
        const uint64_t off = oracle_layout_offset(layout, L, n_blocks, S, k, block_bytes, layer, slabs[j] * S + b);
        iv.emplace_back(off, off + block_bytes);
      }
  std::sort(iv.begin(), iv.end());
  uint32_t n = 0;
  size_t i = 0;
  while (i < iv.size()) {
    uint64_t lo = iv[i].first, hi = iv[i].second;
    size_t j = i + 1;
    while (j < iv.size() && iv[j].first <= hi) hi = std::max(hi, iv[j++].second);
    if (out_bytes && n < cap) out_bytes[n] = hi - lo;
    ++n;
    i = j;
  }
  return n;
}

}  // extern "C"
