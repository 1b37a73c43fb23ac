// Stacked learnable hashing predictor, inference (Section 3.3.1 - 3.3.3 of the paper): an alternative to the linear
// predictor for ranking a layer's neurons.  y_k = T_k[phi_tau(sign(x_k (*) W_k))]: the first layer hashes the PCA-projected
// feature with real hyperplanes (fp64, so that the sign is decided in the oracle's precision), every later layer is binary:
// sign vectors are packed one bit per component (+1 -> 1, component c at bit c % 32 of word c / 32) and an inner product
// is d - 2 * popcount(x XOR w).  A neuron's priority is the inner product of the last layer's output with the neuron's
// binary code: an integer, so the ranking is exact by construction (equal priorities: lower index first).
#pragma once
#include "ls_common.cuh"

namespace ls {

constexpr int HASH_MAX_WORDS = 32;   // d_code <= 1024
constexpr int HASH_MAX_TAU = 16;
constexpr int HASH_MAX_LAYERS = 16;

// One CTA: all layers.  z [rank] fp64 (the projected feature), w1 [rank][tau] float, w [(L-1)][tau][words],
// tables [L][2^tau][words]; y_out [words] the last layer's output, idx_out [L] (nullable) every layer's bucket.
__global__ void __launch_bounds__(256) ls_hash_layers_kernel(const double* __restrict__ z, const float* __restrict__ w1, int rank, int tau,
                                                            int words, int n_layers, const uint32_t* __restrict__ w,
                                                            const uint32_t* __restrict__ tables, uint32_t* y_out, int32_t* idx_out) {
  __shared__ double s_part[HASH_MAX_TAU][16];
  __shared__ uint32_t s_y[HASH_MAX_WORDS];
  __shared__ int s_bits[HASH_MAX_TAU];
  __shared__ int s_idx;
  const int tid = threadIdx.x;
  // first layer: tau real inner products of length rank; 16 threads per hyperplane, each a contiguous part, summed in order
  {
    const int t = tid >> 4, part = tid & 15;
    if (t < tau) {
      const int per = (rank + 15) / 16, j0 = part * per, j1 = min(rank, j0 + per);
      double a = 0.0;
      for (int j = j0; j < j1; ++j) a = fma(z[j], (double)w1[j * tau + t], a);
      s_part[t][part] = a;
    }
  }
  __syncthreads();
  if (tid < tau) {
    double a = 0.0;
    for (int p = 0; p < 16; ++p) a += s_part[tid][p];
    s_bits[tid] = a >= 0.0 ? 1 : 0;
  }
  __syncthreads();
  const int d_code = words * 32;
  for (int k = 0; k < n_layers; ++k) {
    if (tid == 0) {
      int idx = 0;
      for (int t = 0; t < tau; ++t) idx = (idx << 1) | s_bits[t];  // first component = most significant bit
      s_idx = idx;
      if (idx_out) idx_out[k] = idx;
    }
    __syncthreads();
    if (tid < words) s_y[tid] = tables[((size_t)k * ((size_t)1 << tau) + s_idx) * words + tid];
    __syncthreads();
    if (k + 1 < n_layers && tid < tau) {
      const uint32_t* wk = w + ((size_t)k * tau + tid) * words;
      int diff = 0;
      for (int q = 0; q < words; ++q) diff += __popc(s_y[q] ^ wk[q]);
      s_bits[tid] = (d_code - 2 * diff) >= 0 ? 1 : 0;
    }
    __syncthreads();
  }
  if (tid < words) y_out[tid] = s_y[tid];
}

// Priorities: s_i = d - 2 * popcount(y XOR codes[i]) for every neuron (to scores_user, nullable).  The priorities are
// small integers with hundreds of neurons per value; the ranking key written to `keys` is s_i * F + (F - 1 - i), an exact
// integer in fp64 whose order is the library's total order (priority descending, index ascending) without any ties, so
// the binned top-k that follows meets evenly filled bins instead of a few huge ones.
__global__ void __launch_bounds__(256) ls_hash_scores_kernel(const uint32_t* __restrict__ y, const uint32_t* __restrict__ codes, int words, int F,
                                                            double* __restrict__ keys, double* __restrict__ scores_user) {
  __shared__ uint32_t s_y[HASH_MAX_WORDS];
  if (threadIdx.x < words) s_y[threadIdx.x] = y[threadIdx.x];
  __syncthreads();
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < F; i += gridDim.x * blockDim.x) {
    const uint32_t* c = codes + (size_t)i * words;
    int diff = 0;
    if ((words & 3) == 0) {
      for (int q = 0; q < words; q += 4) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(c + q));
        diff += __popc(v.x ^ s_y[q]) + __popc(v.y ^ s_y[q + 1]) + __popc(v.z ^ s_y[q + 2]) + __popc(v.w ^ s_y[q + 3]);
      }
    } else {
      for (int q = 0; q < words; ++q) diff += __popc(__ldg(c + q) ^ s_y[q]);
    }
    const double s = (double)(words * 32 - 2 * diff);
    keys[i] = s * (double)F + (double)(F - 1 - i);
    if (scores_user) scores_user[i] = s;
  }
}

}  // namespace ls
