// balancekv_decode_attn_static: weighted decode attention that allocates nothing.
//
// Some callers are not allowed to allocate device memory: code that runs inside a latency
// critical serving loop where cudaMalloc's implicit device synchronisation is forbidden,
// plugins that are handed buffers by a host framework and must not touch the allocator, or
// processes whose memory pool was sized up front and is fully committed.  They cannot create
// a balancekv context either, because creating one allocates the cache.  This entry point
// serves them: the caller owns the cache rows, the queries and the outputs, and the split-K
// scratch (per-split partial sums, the ticket counters, the small segment table and a status
// word) lives in a fixed array that is part of the library image.
//
// The array is a file-scope __device__ array, so every GPU that loads the library holds its
// kStaticBytes until the process exits.  In host code the array's name is only a handle; the
// device address is obtained once per device with cudaGetSymbolAddress.
#include <cstdio>
#include <mutex>

#include "../../include/balancekv.h"
#include "common.cuh"

namespace bkv {

namespace {

constexpr size_t kStaticBytes = (size_t)8 << 20;   // 8 MiB per GPU
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
unsigned char* g_scratch_addr[kMaxDevices] = {};    // device address of the array, per device
int g_sm_count[kMaxDevices] = {};
std::once_flag g_setup_once[kMaxDevices];           // the per-device set-up runs once, whichever host thread comes first
cudaError_t g_setup_err[kMaxDevices] = {};

// Layout inside the array: [status word, 256 B][segment table][tickets + partials].  The status word
// is left alone here: it keeps the first failure until balancekv_decode_attn_static_status reads it.
__global__ void static_setup_kernel(unsigned char* base, int n_streams, int T, int n_heavy, int n_tail,
                                    size_t seg_off, size_t scratch_off) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n_streams) {
    Seg* seg = reinterpret_cast<Seg*>(base + seg_off) + (size_t)i * (T + 1);
    for (int l = 0; l <= T; ++l) seg[l] = Seg{0, 0};
    seg[T] = Seg{0, n_heavy};
    if (T > 0) seg[0] = Seg{0, n_tail};
    else seg[0] = Seg{0, n_heavy + n_tail};
    reinterpret_cast<unsigned*>(base + scratch_off)[i] = 0u;   // ticket counter of the stream
  }
}

// Once per device, with that device current: resolve the array's device address (in host code the
// array's name is only a handle) and clear the status word.  The array is not otherwise initialised:
// every call sets up the part it uses.
void static_setup_device(int dev) {
  void* p = nullptr;
  cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
  if (e == cudaSuccess && !p) e = cudaErrorInvalidSymbol;
  int sms = 0;
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e == cudaSuccess && sms < 1) e = cudaErrorInvalidValue;
  if (e == cudaSuccess) e = cudaMemset(p, 0, 256);
  g_setup_err[dev] = e;
  if (e != cudaSuccess) return;
  g_sm_count[dev] = sms;
  g_scratch_addr[dev] = static_cast<unsigned char*>(p);
}

// 0 on success, with the current device's index in *dev_out.
int static_device(int* dev_out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return BALANCEKV_E_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return BALANCEKV_E_INVAL;
  std::call_once(g_setup_once[dev], static_setup_device, dev);
  if (g_setup_err[dev] != cudaSuccess || !g_scratch_addr[dev]) {
    std::fprintf(stderr, "balancekv_decode_attn_static: set-up of the built-in scratch array failed: %s\n",
                 cudaGetErrorString(g_setup_err[dev]));
    return BALANCEKV_E_CUDA;
  }
  *dev_out = dev;
  return BALANCEKV_OK;
}

}  // namespace

}  // namespace bkv

using namespace bkv;

extern "C" int balancekv_decode_attn_static(const void* K, const void* V, int n_streams, int cache_len, int n_heavy,
                                            int level, const void* q, void* out, int group, int head_dim, int dtype,
                                            void* stream) {
  if (!K || !V || !q || !out) return BALANCEKV_E_INVAL;
  if (n_streams < 1 || cache_len < 0 || n_heavy < 0 || n_heavy > cache_len) return BALANCEKV_E_INVAL;
  if (level < 0 || level > kMaxLevels || group < 1 || group > kMaxGroup) return BALANCEKV_E_INVAL;
  if ((head_dim != 64 && head_dim != 128) || (dtype != 0 && dtype != 1)) return BALANCEKV_E_INVAL;
  const uintptr_t align = reinterpret_cast<uintptr_t>(K) | reinterpret_cast<uintptr_t>(V) |
                          reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out);
  if (align & 15) return BALANCEKV_E_INVAL;
  int dev = 0;
  if (int rc = static_device(&dev)) return rc;
  unsigned char* base = g_scratch_addr[dev];
  const int esz = dtype ? 2 : 4;
  const int T = level;
  const int n_tail = cache_len - n_heavy;

  Geom G{};
  G.d = head_dim; G.t = 64; G.T = T; G.H = 1; G.L = 1; G.B = n_streams; G.g = group;
  G.is_bf16 = dtype;
  G.rows_per_stream = cache_len;
  for (int l = 0; l <= kMaxLevels; ++l) G.region_off[l] = 0;
  if (T > 0) G.region_off[0] = n_heavy;
  G.inv_sqrt_d = (float)(1.0 / sqrt((double)head_dim));

  const int tile_tokens = 16384 / (head_dim * esz);
  const int64_t tiles = (cache_len + tile_tokens - 1) / tile_tokens + 1;
  int splits = (2 * g_sm_count[dev] + n_streams - 1) / n_streams;
  splits = (int)std::max<int64_t>(1, std::min<int64_t>(std::min(64, splits), (tiles + 1) / 2));
  const size_t seg_off = 256;
  const size_t seg_bytes = ((size_t)n_streams * (T + 1) * sizeof(Seg) + 255) & ~(size_t)255;
  const size_t scratch_off = seg_off + seg_bytes;
  const size_t need = scratch_off + decode_scratch_bytes(G, splits);
  if (need > kStaticBytes) {
    std::fprintf(stderr,
                 "balancekv_decode_attn_static: needs %zu bytes of scratch for %d streams x %d splits x %d heads, "
                 "the built-in array holds %zu; use balancekv_decode_attn with a context instead\n",
                 need, n_streams, splits, group, kStaticBytes);
    return BALANCEKV_E_NOMEM;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  static_setup_kernel<<<(n_streams + 255) / 256, 256, 0, st>>>(base, n_streams, T, n_heavy, n_tail, seg_off, scratch_off);
  if (cudaGetLastError() != cudaSuccess) return BALANCEKV_E_CUDA;
  Arena A{};
  A.K = const_cast<void*>(K);
  A.V = const_cast<void*>(V);
  A.idx = nullptr;
  A.seg = reinterpret_cast<Seg*>(base + seg_off);
  cudaError_t e = launch_decode(G, A, 0, q, out, reinterpret_cast<float*>(base + scratch_off), splits,
                                reinterpret_cast<int*>(base), st);
  if (e != cudaSuccess) {
    std::fprintf(stderr, "balancekv_decode_attn_static: launch failed: %s\n", cudaGetErrorString(e));
    return BALANCEKV_E_CUDA;
  }
  return BALANCEKV_OK;
}

extern "C" int balancekv_decode_attn_static_status(int* status_host, void* stream) {
  if (!status_host) return BALANCEKV_E_INVAL;
  int dev = 0;
  if (int rc = static_device(&dev)) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int v = 0;
  // read, then clear, in stream order behind the launches issued so far on `stream`
  if (cudaMemcpyAsync(&v, g_scratch_addr[dev], sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return BALANCEKV_E_CUDA;
  if (cudaMemsetAsync(g_scratch_addr[dev], 0, sizeof(int), st) != cudaSuccess) return BALANCEKV_E_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return BALANCEKV_E_CUDA;
  *status_host = v;
  return BALANCEKV_OK;
}
