// noalloc.cu — attention launch whose split-KV scratch lives in a static device array.
//
// paged_decode keeps the partial results of its split-KV segments in a buffer that it obtains from
// cudaMalloc the first time it is called (and again when a later call needs a larger one). Some
// callers must not trigger a device allocation at that point: a serving engine that has handed
// all of the GPU's memory to its KV-cache pool at start-up (a late cudaMalloc would fail), a
// latency-critical decode loop that cannot afford the device-wide synchronisation an allocation
// implies, or code running under a policy that forbids allocator calls after initialisation.
// For them this file provides the same two launches with the scratch placed in a file-scope
// `static __device__` array of fixed size.
//
// The array occupies kStaticScratchBytes on every GPU on which this part of the library has been
// loaded, until the process exits. With CUDA's lazy module loading (the default) that load, and
// with it the reservation of the array, happens at the first use of a symbol of this file on the
// device; slice_create does that use (static_scratch_setup below), so that it falls into
// initialisation and not into the first decode call. In host code the array's name is only a
// host-side stand-in, not a device address, so the address handed to the kernels is looked up with
// cudaGetSymbolAddress: once per device, with that device current. All calls share the one array
// and it keeps whatever the last call left in it; two calls whose kernels overlap on the GPU would
// race on it.
#include "kernels.h"

namespace {

constexpr size_t kStaticScratchBytes = 8u << 20;  // 8 MiB per GPU
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device addresses of g_static_scratch, filled in once per device.
void* g_scratch_addr[kMaxDevices] = {};
bool g_warmed[kMaxDevices][2] = {};  // [device][tensor-core variant]: an empty launch has been made

inline size_t align256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

}  // namespace

namespace ema {

size_t static_scratch_bytes() { return kStaticScratchBytes; }

size_t static_scratch_needed(uint32_t slots, uint32_t Hq, uint32_t nseq, uint32_t Hkv, uint32_t ncta) {
  const size_t o_bytes = static_cast<size_t>(slots) * Hq * 128 * sizeof(float);
  const size_t ml_bytes = static_cast<size_t>(slots) * Hq * 4 * sizeof(float);
  const size_t cnt_bytes = layer_counter_words(ncta, nseq, Hkv) * sizeof(uint32_t);
  return align256(o_bytes) + align256(ml_bytes) + align256(cnt_bytes);
}

// Set-up for the device that is current: resolves and caches the array's device address.
cudaError_t static_scratch_address(void** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

// Initialisation-time set-up for the device that is current (called by slice_create): loads this
// module on the device, which is what reserves the array, resolves the array's address, and makes
// one empty launch of the attention kernel variant that serves `G` query heads per KV head, so that
// whatever the driver sets up at a kernel's first launch (its code, the thread stacks) is in place
// before the first decode call rather than inside it.
cudaError_t static_scratch_setup(uint32_t Hkv, uint32_t G, uint32_t ncta) {
  void* base = nullptr;
  cudaError_t e = static_scratch_address(&base);
  if (e != cudaSuccess) return e;
  int dev = 0;
  e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const int variant = G == 1 ? 0 : 1;
  if (g_warmed[dev][variant]) return cudaSuccess;
  LayerParams p{};  // no blocks, no sequences, no gather: every role finds nothing to do and returns
  p.num_layers = 1;
  p.li_end = 1;
  p.ring_slots = 1;
  p.layer_group = 1;
  p.prefetch_distance = 1;
  p.split_layer = 0xFFFFFFFFu;
  p.per = 1;
  p.merge_inline = 1;
  p.part_buffers = 1;
  p.ncta = ncta;
  p.Hkv = Hkv;
  p.G = G;
  p.Hq = Hkv * G;
  p.counters = static_cast<uint32_t*>(base);
  for (uint32_t i = 0; i < kMaxStepLayers; ++i) p.gather_target[i] = p.gather_after[i] = -1;
  e = launch_layer(p, nullptr);
  if (e != cudaSuccess) return e;
  e = cudaStreamSynchronize(nullptr);
  if (e != cudaSuccess) return e;
  g_warmed[dev][variant] = true;
  return cudaSuccess;
}

// The layer kernel with its partials and counters in the static array. The partial rows need no
// clearing (every work item writes its row before the merging warp reads it, and only this
// launch's rows are read); the work and arrival counters must start at zero and may hold anything
// after an earlier call that failed, so they are cleared on the stream before every launch.
cudaError_t launch_layer_static(LayerParams p, uint32_t slots, cudaStream_t stream) {
  void* base = nullptr;
  cudaError_t e = static_scratch_address(&base);
  if (e != cudaSuccess) return e;
  if (static_scratch_needed(slots, p.Hq, p.nseq, p.Hkv, p.ncta) > kStaticScratchBytes) return cudaErrorInvalidValue;
  const size_t o_bytes = align256(static_cast<size_t>(slots) * p.Hq * 128 * sizeof(float));
  const size_t ml_bytes = align256(static_cast<size_t>(slots) * p.Hq * 4 * sizeof(float));
  const size_t cnt_bytes = layer_counter_words(p.ncta, p.nseq, p.Hkv) * sizeof(uint32_t);
  unsigned char* b = static_cast<unsigned char*>(base);
  p.part_o = reinterpret_cast<float*>(b);
  p.part_ml = reinterpret_cast<float*>(b + o_bytes);
  p.counters = reinterpret_cast<uint32_t*>(b + o_bytes + ml_bytes);
  e = cudaMemsetAsync(p.counters, 0, cnt_bytes, stream);
  if (e != cudaSuccess) return e;
  return launch_layer(p, stream);
}

}  // namespace ema
