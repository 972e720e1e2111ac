// LM-head pass on CUDA cores: logits = s * h W^T + bias for the beam rows, with the
// log-softmax statistics and the per-row top-k folded in, so logits never reach HBM.
// This is the fp32 kernel (tensor cores have no fp32 path and TF32 would cost the
// 2e-3 logprob tolerance); it also accepts bf16 storage so it can cross-check the
// tensor-core kernel.  Each thread block walks tiles of kTile vocab rows; a warp
// computes one vocab row at a time against all live beam rows.
#include "ddd_common.cuh"

namespace ddd {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kRowChunk = 8;   // beam rows accumulated together per sweep over Hd

template <typename T>
struct Vec;
template <>
struct Vec<float> {
  static constexpr int N = 4;
  __device__ static void load(const float* p, float (&v)[4]) {
    const float4 q = *reinterpret_cast<const float4*>(p);
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
  }
};
template <>
struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static void load(const __nv_bfloat16* p, float (&v)[8]) {
    const uint4 q = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);          // low half = even element
      v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
};

// Shared memory: logits of the current tile, transposed to [row][kTile], then the running
// state of every beam row: top-k keys [row][32] and (max, sum) [row].
template <typename T>
__global__ void __launch_bounds__(kThreads) lm_head_simt_kernel(const Params p, const int d,
                                                                const int force_all) {
  if (!force_all && *p.n_active == 0) return;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* zt = reinterpret_cast<float*>(smem_raw);
  unsigned long long* st_key = reinterpret_cast<unsigned long long*>(zt + (size_t)p.R * kTile);
  const int kst = p.k <= kNarrowK ? 32 : kWideK;     // keys kept per row: one or four per lane
  float2* st_ms = reinterpret_cast<float2*>(st_key + (size_t)p.R * kst);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int VEC = Vec<T>::N;
  const T* W = static_cast<const T*>(p.W);
  const T* H = static_cast<const T*>(p.hbuf[(d - 1) & 1]);
  const int n_tiles = (p.Vl + kTile - 1) / kTile;   // W, bias: local rows; tokens: v0 + local row

  for (int r = warp; r < p.R; r += kWarps) {
    for (int e = lane; e < kst; e += 32) st_key[r * kst + e] = 0ull;
    if (lane == 0) st_ms[r] = make_float2(neg_inf(), 0.f);
  }
  __syncthreads();

  for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const int v0 = tile * kTile;
    // ---- logits of this tile
    for (int vl = warp; vl < kTile; vl += kWarps) {
      const int v = v0 + vl;
      const bool v_ok = v < p.Vl;
      const float bias = (v_ok && p.bias) ? p.bias[v] : 0.f;
      for (int r0 = 0; r0 < p.R; r0 += kRowChunk) {
        float acc[kRowChunk];
        bool live[kRowChunk];
        bool any_live = false;
#pragma unroll
        for (int rc = 0; rc < kRowChunk; ++rc) {
          acc[rc] = 0.f;
          live[rc] = (r0 + rc < p.R) && row_live(p, r0 + rc, d, force_all);
          any_live |= live[rc];
        }
        if (v_ok && any_live) {
          const T* wrow = W + (size_t)v * p.Hd;
          for (int j = lane * VEC; j < p.Hd; j += 32 * VEC) {
            float w[VEC];
            Vec<T>::load(wrow + j, w);
#pragma unroll
            for (int rc = 0; rc < kRowChunk; ++rc) {
              if (!live[rc]) continue;
              float h[VEC];
              Vec<T>::load(H + (size_t)(r0 + rc) * p.Hd + j, h);
#pragma unroll
              for (int e = 0; e < VEC; ++e) acc[rc] = fmaf(w[e], h[e], acc[rc]);
            }
          }
        }
#pragma unroll
        for (int rc = 0; rc < kRowChunk; ++rc) {
          if (r0 + rc >= p.R) continue;
          const float sum = warp_sum(acc[rc]);
          if (lane == rc) {
            const int r = r0 + rc;
            float z = neg_inf();
            if (v_ok && live[rc] && p.row_plant[r] != v + p.v0) z = fmaf(sum, p.s, bias);
            zt[(size_t)r * kTile + vl] = z;
          }
        }
      }
    }
    __syncthreads();
    // ---- fold the tile into every live row's running state
    for (int r = warp; r < p.R; r += kWarps) {
      if (!row_live(p, r, d, force_all)) continue;
      float2 ms = st_ms[r];
      if (p.k <= kNarrowK) {
        unsigned long long key = st_key[r * 32 + lane];
        row_tile_update(zt + (size_t)r * kTile, v0 + p.v0, p.k, ms.x, ms.y, key);
        st_key[r * 32 + lane] = key;
      } else {
        unsigned long long list[4];
        wide_load(list, st_key + (size_t)r * kWideK, kWideK);
        row_tile_update_wide(zt + (size_t)r * kTile, v0 + p.v0, p.k, ms.x, ms.y, list);
        wide_store(list, st_key + (size_t)r * kWideK, kWideK);
      }
      if (lane == 0) st_ms[r] = ms;
    }
    __syncthreads();
  }

  // ---- publish this block's partial results
  for (int r = warp; r < p.R; r += kWarps) {
    if (!row_live(p, r, d, force_all)) continue;
    const size_t slot = (size_t)blockIdx.x * p.R + r;
    for (int e = lane; e < p.k; e += 32) p.part_key[slot * p.k + e] = st_key[r * kst + e];
    if (lane == 0) p.part_ms[slot] = st_ms[r];
  }
}

size_t simt_smem(const Params& p) {
  const size_t kst = p.k <= kNarrowK ? 32 : kWideK;
  return (size_t)p.R * kTile * sizeof(float) + (size_t)p.R * kst * sizeof(unsigned long long) +
         (size_t)p.R * sizeof(float2);
}

}  // namespace

cudaError_t prepare_simt(const Params& p) {
  if (simt_smem(p) > 200 * 1024) return cudaErrorInvalidValue;
  cudaError_t e = allow_max_dynamic_smem(lm_head_simt_kernel<float>);
  if (e != cudaSuccess) return e;
  return allow_max_dynamic_smem(lm_head_simt_kernel<__nv_bfloat16>);
}

cudaError_t launch_lm_head_simt(const Params& p, int d, int force_all, int ctas, cudaStream_t st) {
  const size_t smem = simt_smem(p);
  if (p.dtype == DDD_DTYPE_FP32)
    lm_head_simt_kernel<float><<<ctas, kThreads, smem, st>>>(p, d, force_all);
  else
    lm_head_simt_kernel<__nv_bfloat16><<<ctas, kThreads, smem, st>>>(p, d, force_all);
  return cudaGetLastError();
}

}  // namespace ddd
