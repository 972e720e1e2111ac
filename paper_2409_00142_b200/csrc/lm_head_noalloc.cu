// ddd_lm_head_topk_noalloc: one LM-head pass (logits, log-softmax, per-row top-k) for callers
// that cannot allocate device memory.
//
// The other entry points keep their scratch (the per-block partial results that a second
// kernel merges) in a workspace the caller allocates.  Some callers have no allocator to
// ask: code that runs inside another library's callback or plug-in interface and is handed
// fixed buffers and nothing else, a process whose device memory belongs to a framework pool
// it must not call back into, or a real-time loop where cudaMalloc (which may synchronise
// the whole device) is not acceptable.  For them the scratch lives here, in a file-scope
// __device__ array that is part of the loaded module: every GPU that loads the library holds
// these 2,162,688 bytes until the process exits, and nothing is allocated or freed at call
// time.  All calls share that one array, so two calls that overlap on the GPU race.
#include <mutex>

#include "ddd_common.cuh"

namespace {

using namespace ddd;

constexpr int kNaMaxRows = 32;      // beam rows per call
constexpr int kNaMaxK = 32;         // list width per row (one key per lane)
constexpr int kNaMaxBlocks = 256;   // thread blocks of the first kernel
constexpr int kNaThreads = 256;
constexpr int kNaWarps = kNaThreads / 32;
constexpr int kNaRowChunk = 8;
constexpr int kNaMaxDevices = 64;

// Scratch layout: keys [block][row][k] (8 bytes each), then (max, sum) [block][row].
constexpr size_t kNaKeyBytes = (size_t)kNaMaxBlocks * kNaMaxRows * kNaMaxK * sizeof(unsigned long long);
constexpr size_t kNaMsBytes = (size_t)kNaMaxBlocks * kNaMaxRows * sizeof(float2);
constexpr size_t kNoAllocScratchBytes = kNaKeyBytes + kNaMsBytes;   // 2,162,688 bytes

// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

template <typename T>
struct NaVec;
template <>
struct NaVec<float> {
  static constexpr int N = 4;
  __device__ static void load(const float* p, float (&v)[4]) {
    const float4 q = *reinterpret_cast<const float4*>(p);
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
  }
};
template <>
struct NaVec<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static void load(const __nv_bfloat16* p, float (&v)[8]) {
    const uint4 q = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
};

// First kernel: every block walks tiles of kTile vocab rows and leaves, per beam row, its
// (max, sum-exp) and its k best (logit, token) keys in the scratch array.  Every slot the
// second kernel reads is written here on every call, so stale contents never matter.
template <typename T>
__global__ void __launch_bounds__(kNaThreads)
noalloc_partials_kernel(const T* __restrict__ W, const float* __restrict__ bias, const T* __restrict__ H,
                        int rows, int hidden, int vocab, int k, float scale, unsigned char* scratch) {
  __shared__ __align__(16) float zt[kNaMaxRows * kTile];
  __shared__ unsigned long long st_key[kNaMaxRows * 32];
  __shared__ float2 st_ms[kNaMaxRows];
  unsigned long long* part_key = reinterpret_cast<unsigned long long*>(scratch);
  float2* part_ms = reinterpret_cast<float2*>(scratch + kNaKeyBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int VEC = NaVec<T>::N;
  const int n_tiles = (vocab + kTile - 1) / kTile;
  for (int r = warp; r < rows; r += kNaWarps) {
    st_key[r * 32 + lane] = 0ull;
    if (lane == 0) st_ms[r] = make_float2(neg_inf(), 0.f);
  }
  __syncthreads();

  for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const int v0 = tile * kTile;
    for (int vl = warp; vl < kTile; vl += kNaWarps) {
      const int v = v0 + vl;
      const bool v_ok = v < vocab;
      const float b = (v_ok && bias) ? bias[v] : 0.f;
      for (int r0 = 0; r0 < rows; r0 += kNaRowChunk) {
        float acc[kNaRowChunk];
#pragma unroll
        for (int rc = 0; rc < kNaRowChunk; ++rc) acc[rc] = 0.f;
        if (v_ok) {
          const T* wrow = W + (size_t)v * hidden;
          for (int j = lane * VEC; j < hidden; j += 32 * VEC) {
            float w[VEC];
            NaVec<T>::load(wrow + j, w);
#pragma unroll
            for (int rc = 0; rc < kNaRowChunk; ++rc) {
              if (r0 + rc >= rows) continue;
              float h[VEC];
              NaVec<T>::load(H + (size_t)(r0 + rc) * hidden + j, h);
#pragma unroll
              for (int e = 0; e < VEC; ++e) acc[rc] = fmaf(w[e], h[e], acc[rc]);
            }
          }
        }
#pragma unroll
        for (int rc = 0; rc < kNaRowChunk; ++rc) {
          if (r0 + rc >= rows) continue;
          const float sum = warp_sum(acc[rc]);
          if (lane == rc) zt[(r0 + rc) * kTile + vl] = v_ok ? fmaf(sum, scale, b) : neg_inf();
        }
      }
    }
    __syncthreads();
    for (int r = warp; r < rows; r += kNaWarps) {
      float2 ms = st_ms[r];
      unsigned long long key = st_key[r * 32 + lane];
      row_tile_update(zt + r * kTile, v0, k, ms.x, ms.y, key);
      st_key[r * 32 + lane] = key;
      if (lane == 0) st_ms[r] = ms;
    }
    __syncthreads();
  }
  for (int r = warp; r < rows; r += kNaWarps) {
    const size_t slot = (size_t)blockIdx.x * rows + r;
    if (lane < k) part_key[slot * k + lane] = st_key[r * 32 + lane];
    if (lane == 0) part_ms[slot] = st_ms[r];
  }
}

// Second kernel: one warp per beam row merges the partials of all blocks, in a fixed order,
// into the row's logsumexp and its k best tokens with their log-probabilities.
__global__ void __launch_bounds__(32 * kNaMaxRows)
noalloc_merge_kernel(const unsigned char* __restrict__ scratch, int blocks, int rows, int k,
                     int* __restrict__ out_token, float* __restrict__ out_logprob, float* __restrict__ out_lse) {
  const unsigned long long* part_key = reinterpret_cast<const unsigned long long*>(scratch);
  const float2* part_ms = reinterpret_cast<const float2*>(scratch + kNaKeyBytes);
  const int r = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (r >= rows) return;
  float M = neg_inf();
  for (int c = lane; c < blocks; c += 32) M = fmaxf(M, part_ms[(size_t)c * rows + r].x);
  M = ordered_to_float(__reduce_max_sync(kFullMask, float_to_ordered(M)));
  float S = 0.f;
  for (int c = lane; c < blocks; c += 32) {
    const float2 ms = part_ms[(size_t)c * rows + r];
    if (ms.y > 0.f) S += ms.y * expf(ms.x - M);
  }
  S = warp_sum(S);
  const float lse = M + logf(S);
  // keys are unique, so the j-th best is the largest key below the (j-1)-th best
  unsigned long long prev = ~0ull, mine = 0ull;
  const int n_keys = blocks * k;
  for (int j = 0; j < k; ++j) {
    unsigned long long best = 0ull;
    for (int e = lane; e < n_keys; e += 32) {
      const int c = e / k, q = e - c * k;
      const unsigned long long key = part_key[((size_t)c * rows + r) * k + q];
      if (key < prev && key > best) best = key;
    }
    const unsigned long long wk = warp_max_key(best);
    if (lane == j) mine = wk;
    prev = wk;
  }
  if (lane < k) {
    out_token[r * k + lane] = mine ? (int)key_index(mine) : -1;
    out_logprob[r * k + lane] = mine ? fminf(key_value(mine) - lse, 0.f) : neg_inf();
  }
  if (lane == 0) out_lse[r] = lse;
}

// Device address of the scratch array, looked up once per device.
std::mutex g_na_mutex;
unsigned char* g_na_scratch_ptr[kNaMaxDevices] = {};

int noalloc_scratch_for_current_device(unsigned char** ptr) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNaMaxDevices) return DDD_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_na_mutex);
  if (!g_na_scratch_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return DDD_ERR_CUDA;
    }
    g_na_scratch_ptr[dev] = static_cast<unsigned char*>(p);
  }
  *ptr = g_na_scratch_ptr[dev];
  return DDD_OK;
}

}  // namespace

extern "C" int ddd_lm_head_topk_noalloc(const void* W, const float* bias, const void* hidden_rows, int32_t dtype,
                                        int32_t rows, int32_t hidden, int32_t vocab, int32_t k, float logit_scale,
                                        int32_t* out_token, float* out_logprob, float* out_lse,
                                        void* cuda_stream) {
  if (!W || !hidden_rows || !out_token || !out_logprob || !out_lse) return DDD_ERR_INVALID_ARG;
  if (dtype != DDD_DTYPE_FP32 && dtype != DDD_DTYPE_BF16) return DDD_ERR_INVALID_ARG;
  if (rows < 1 || rows > kNaMaxRows || k < 1 || k > kNaMaxK) return DDD_ERR_INVALID_ARG;   // beyond the scratch
  if (hidden < 8 || hidden % 8 != 0 || vocab <= k) return DDD_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(W) & 15u) || (reinterpret_cast<uintptr_t>(hidden_rows) & 15u))
    return DDD_ERR_ALIGNMENT;
  unsigned char* scratch = nullptr;
  const int rc = noalloc_scratch_for_current_device(&scratch);
  if (rc != DDD_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int n_tiles = (vocab + kTile - 1) / kTile;
  const int blocks = n_tiles < kNaMaxBlocks ? n_tiles : kNaMaxBlocks;
  if (dtype == DDD_DTYPE_FP32)
    noalloc_partials_kernel<float><<<blocks, kNaThreads, 0, st>>>(
        static_cast<const float*>(W), bias, static_cast<const float*>(hidden_rows), rows, hidden, vocab, k,
        logit_scale, scratch);
  else
    noalloc_partials_kernel<__nv_bfloat16><<<blocks, kNaThreads, 0, st>>>(
        static_cast<const __nv_bfloat16*>(W), bias, static_cast<const __nv_bfloat16*>(hidden_rows), rows, hidden,
        vocab, k, logit_scale, scratch);
  if (cudaGetLastError() != cudaSuccess) return DDD_ERR_CUDA;
  noalloc_merge_kernel<<<1, 32 * rows, 0, st>>>(scratch, blocks, rows, k, out_token, out_logprob, out_lse);
  if (cudaGetLastError() != cudaSuccess) return DDD_ERR_CUDA;
  return DDD_OK;
}
