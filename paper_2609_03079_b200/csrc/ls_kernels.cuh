// Kernels of the stage-by-stage (one launch per operation) path.
//   speculate / refine : ls_latent_kernel -> ls_scores_kernel -> ls_topk_kernel
//   stage c of K       : ls_gateup_kernel -> ls_down_kernel -> ls_stage_finalize_kernel
#pragma once
#include "ls_common.cuh"
#include "ls_topk.cuh"

namespace ls {

// ------------------------------------------------------------------------------------------------------------------
// Step set-up: xin <- x (the MLP input source, kept because x_out may alias x), xt <- x (+ b_down) = x~^(0).
// ------------------------------------------------------------------------------------------------------------------
__global__ void ls_step_init_kernel(const float* __restrict__ x, const float* __restrict__ b_down, float* xin, float* xt,
                                    float* trace0, int B, int d, uint32_t* survive, int nwords, uint32_t* survive_trace) {
  const int n = B * d;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    const float v = x[i];
    xin[i] = v;
    const float t = b_down ? v + b_down[i % d] : v;
    xt[i] = t;
    if (trace0) trace0[i] = t;
  }
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < nwords; i += gridDim.x * blockDim.x) {
    survive[i] = 0u;
    if (survive_trace) survive_trace[i] = 0u;
  }
}

// ------------------------------------------------------------------------------------------------------------------
// Predictor latent, un-normalised: z[b][j] = sum_i A[i][j] * v[b][i] in fp64 (A stored transposed, one row per j),
// plus sum of squares of the feature (the RMS norm is a scalar applied by the scores kernel).
// FOUR warps per latent row (a launch of r / 2 blocks keeps more loads in flight than one warp per row did: the kernel is
// bound by the latency of its row loads): warp q of a row takes the 8-column chunks q, q + 4, ...; the four partial sums
// are added in a fixed order.
// ------------------------------------------------------------------------------------------------------------------
template <int WD>
__global__ void __launch_bounds__(256) ls_latent_kernel(const uint16_t* __restrict__ At, const float* __restrict__ v, int d,
                                                        int r, int B, double* __restrict__ z, double* __restrict__ sumsq) {
  __shared__ double s_part[2][4], s_sq[4];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int jr = warp >> 2, q = warp & 3;  // row of this block, quarter of the row
  const int j = blockIdx.x * 2 + jr;
  const int nch = d >> 3;
  const uint16_t* row = At + (size_t)min(j, r - 1) * d;
  for (int b = 0; b < B; ++b) {
    const float* vb = v + (size_t)b * d;
    double acc = 0.0, sq = 0.0;
    if (j < r) {
#pragma unroll 2
      for (int ch = q * 32 + lane; ch < nch; ch += 128) {
        float w[8];
        unpack8<WD>(ldg128(row + ch * 8), w);
        const float4 x0 = __ldg(reinterpret_cast<const float4*>(vb + ch * 8));
        const float4 x1 = __ldg(reinterpret_cast<const float4*>(vb + ch * 8 + 4));
        const float xs[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
#pragma unroll
        for (int e = 0; e < 8; ++e) acc = fma((double)w[e], (double)xs[e], acc);
        if (j == 0) {
#pragma unroll
          for (int e = 0; e < 8; ++e) sq = fma((double)xs[e], (double)xs[e], sq);
        }
      }
    }
    acc = warp_sum(acc);
    sq = warp_sum(sq);
    __syncthreads();
    if (lane == 0) {
      s_part[jr][q] = acc;
      if (j == 0) s_sq[q] = sq;
    }
    __syncthreads();
    if (q == 0 && lane == 0 && j < r) {
      z[(size_t)b * r + j] = (s_part[jr][0] + s_part[jr][1]) + (s_part[jr][2] + s_part[jr][3]);
      if (j == 0) sumsq[b] = (s_sq[0] + s_sq[1]) + (s_sq[2] + s_sq[3]);
    }
  }
}

// ------------------------------------------------------------------------------------------------------------------
// Predictor scores: s[b][i] = sum_j B[j][i] * z[b][j] * inv_rms[b] + c[i], fp64; prio[i] = max_b s[b][i].
// B stored transposed ([F][r], one row per neuron); one warp per neuron, every neuron reduced in the same order,
// so equal predictor columns give bit-equal scores.  At batch 1 with r <= 512 a lane's (at most two) chunks of the
// normalised latents stay in registers for all its neurons (the shared-memory reads of z were what the kernel waited for).
// ------------------------------------------------------------------------------------------------------------------
template <int WD>
__global__ void __launch_bounds__(256) ls_scores_kernel(const uint16_t* __restrict__ Bt, const float* __restrict__ c,
                                                        const double* __restrict__ z, const double* __restrict__ sumsq, int d,
                                                        int r, int F, int B, int norm, float eps, double* __restrict__ scores,
                                                        double* __restrict__ prio, double* __restrict__ prio_user) {
  extern __shared__ double zs[];  // [B][r], normalised
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int wpb = blockDim.x >> 5;
  const int nch = r >> 3;
  if (B == 1 && nch <= 64) {
    const double inv = norm == 0 ? 1.0 / sqrt(sumsq[0] / (double)d + (double)eps) : 1.0;
    double z0[8], z1[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      z0[e] = lane < nch ? z[lane * 8 + e] * inv : 0.0;
      z1[e] = lane + 32 < nch ? z[(lane + 32) * 8 + e] * inv : 0.0;
    }
    for (int i = blockIdx.x * wpb + warp; i < F; i += gridDim.x * wpb) {
      const uint16_t* row = Bt + (size_t)i * r;
      double acc = 0.0;
      if (lane < nch) {
        float w[8];
        unpack8<WD>(ldg128(row + lane * 8), w);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc = fma((double)w[e], z0[e], acc);
      }
      if (lane + 32 < nch) {
        float w[8];
        unpack8<WD>(ldg128(row + (lane + 32) * 8), w);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc = fma((double)w[e], z1[e], acc);
      }
      acc = warp_sum(acc);
      const double s = canonical_score(acc + (c ? (double)c[i] : 0.0));
      if (lane == 0) {
        prio[i] = s;
        if (prio_user) prio_user[i] = s;
      }
    }
    return;
  }
  for (int t = threadIdx.x; t < B * r; t += blockDim.x) {
    const int b = t / r;
    const double inv = norm == 0 ? 1.0 / sqrt(sumsq[b] / (double)d + (double)eps) : 1.0;
    zs[t] = z[t] * inv;
  }
  __syncthreads();
  for (int i = blockIdx.x * wpb + warp; i < F; i += gridDim.x * wpb) {
    const uint16_t* row = Bt + (size_t)i * r;
    double best = 0.0;
    for (int b = 0; b < B; ++b) {
      double acc = 0.0;
      for (int ch = lane; ch < nch; ch += 32) {
        float w[8];
        unpack8<WD>(ldg128(row + ch * 8), w);
        const double* zb = zs + b * r + ch * 8;
#pragma unroll
        for (int e = 0; e < 8; ++e) acc = fma((double)w[e], zb[e], acc);
      }
      acc = warp_sum(acc);
      const double s = canonical_score(acc + (c ? (double)c[i] : 0.0));
      if (lane == 0 && B > 1) scores[(size_t)b * F + i] = s;
      best = (b == 0 || s > best) ? s : best;
    }
    if (lane == 0) {
      prio[i] = best;
      if (prio_user) prio_user[i] = best;
    }
  }
}

// ------------------------------------------------------------------------------------------------------------------
// Stage c, part 1: gate/up gather-GEMV and activation for the neurons of the stage (Eq. 1, the bracket).
// FOUR warps per neuron (two neurons per block of eight warps): a stage is a few hundred neurons, and with one warp per
// neuron the launch was a few dozen blocks waiting for their own row loads.  Warp q of a neuron takes the 8-column chunks
// q, q + 4, ... of the gate and up rows; 128-bit row loads, fp32 accumulation, warp-shuffle reduction, the four partial
// sums added in a fixed order.
// a[b][p] = act(inv_rms_b * (w_gate[i] . x_b) + b_i) * (inv_rms_b * (w_up[i] . x_b)), p = rank position of neuron i.
// ------------------------------------------------------------------------------------------------------------------
template <int WD, int BT>
__global__ void __launch_bounds__(256)
    ls_gateup_kernel(const uint16_t* __restrict__ bundles, int n_mat, int gated, int act_kind, const int32_t* __restrict__ slot_of,
                     const float* __restrict__ b_gate, const float* __restrict__ xin, int B, int d, int norm, float eps,
                     const int32_t* __restrict__ exec_idx, const int32_t* __restrict__ count_ptr, int K, int c, int F,
                     float* __restrict__ act, int act_stride, uint32_t* survive, int* status, const unsigned* landed, unsigned need_seq,
                     const int32_t* list_hdr) {
  extern __shared__ __align__(16) float xs[];  // [B][d]
  __shared__ float s_inv[8];
  __shared__ double s_red[8][8];
  __shared__ float s_acc[2][4][BT][2];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int lo, hi;
  stage_bounds(*count_ptr, K, c, lo, hi);
  if (lo + (int)blockIdx.x * 2 >= hi) return;
  // Cached layer: the residents come first in the execution order; a stage that reaches into the misses waits (bounded)
  // until the rows of the layer's request have landed in their slots.
  if (landed && threadIdx.x == 0 && hi > list_hdr[1]) {
    const long long t0 = clock64();
    while (*reinterpret_cast<const volatile unsigned*>(landed) < need_seq) {
      if (clock64() - t0 > 4000LL * 1000 * 1000) { set_status(status, ST_TIMEOUT); break; }
    }
    __threadfence();
  }

  for (int b = 0; b < B; ++b) {
    double sq = 0.0;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
      const float v = xin[(size_t)b * d + i];
      xs[b * d + i] = v;
      sq = fma((double)v, (double)v, sq);
    }
    sq = warp_sum(sq);
    if (lane == 0) s_red[b][warp] = sq;
  }
  __syncthreads();
  if (threadIdx.x < B) {
    double t = 0.0;
    for (int w = 0; w < 8; ++w) t += s_red[threadIdx.x][w];
    s_inv[threadIdx.x] = norm == 0 ? (float)(1.0 / sqrt(t / (double)d + (double)eps)) : 1.0f;
  }
  __syncthreads();

  const int nch = d >> 3;
  const int jr = warp >> 2, q = warp & 3;  // neuron of this block, quarter of its rows
  for (int p0 = lo + blockIdx.x * 2; p0 < hi; p0 += gridDim.x * 2) {
    const int p = p0 + jr;
    const bool live = p < hi;
    const int i = live ? exec_idx[p] : 0;
    const bool in_range = live && (unsigned)i < (unsigned)F;  // never dereference a bad index
    const int slot = in_range ? (slot_of ? slot_of[i] : i) : -1;
    const bool ok = in_range && slot >= 0;
    float ag[BT], au[BT];
#pragma unroll
    for (int b = 0; b < BT; ++b) { ag[b] = 0.f; au[b] = 0.f; }
    if (ok) {
      const uint16_t* grow = bundles + (size_t)slot * n_mat * d;
      const uint16_t* urow = grow + d;
#pragma unroll 4
      for (int ch = q * 32 + lane; ch < nch; ch += 128) {
        float wg[8], wu[8];
        unpack8<WD>(ld_stream128(grow + ch * 8), wg);
        if (gated) unpack8<WD>(ld_stream128(urow + ch * 8), wu);
#pragma unroll
        for (int b = 0; b < BT; ++b) {
          if (b < B) {
            const float4 x0 = *reinterpret_cast<const float4*>(xs + b * d + ch * 8);
            const float4 x1 = *reinterpret_cast<const float4*>(xs + b * d + ch * 8 + 4);
            const float xv[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              ag[b] = fmaf(wg[e], xv[e], ag[b]);
              if (gated) au[b] = fmaf(wu[e], xv[e], au[b]);
            }
          }
        }
      }
    }
#pragma unroll
    for (int b = 0; b < BT; ++b) {
      if (b < B) {
        const float g = warp_sum(ag[b]), u = gated ? warp_sum(au[b]) : 0.f;
        if (lane == 0) { s_acc[jr][q][b][0] = g; s_acc[jr][q][b][1] = u; }
      }
    }
    __syncthreads();
    if (q == 0 && lane == 0 && live) {
      if (!ok) {
        set_status(status, ST_BAD_INDEX);
        for (int b = 0; b < B; ++b) act[(size_t)b * act_stride + p] = 0.f;
      } else {
        bool any = false;
#pragma unroll
        for (int b = 0; b < BT; ++b) {
          if (b < B) {
            const float gs = (s_acc[jr][0][b][0] + s_acc[jr][1][b][0]) + (s_acc[jr][2][b][0] + s_acc[jr][3][b][0]);
            const float g = gs * s_inv[b] + (b_gate ? b_gate[i] : 0.f);
            float a = act_kind == 0 ? fmaxf(g, 0.f) : g / (1.f + expf(-g));  // ReLU, or SiLU as Eq. 1 prints it
            if (gated) a *= ((s_acc[jr][0][b][1] + s_acc[jr][1][b][1]) + (s_acc[jr][2][b][1] + s_acc[jr][3][b][1])) * s_inv[b];
            act[(size_t)b * act_stride + p] = a;
            any |= (a != 0.f);
          }
        }
        if (any) atomicOr(&survive[i >> 5], 1u << (i & 31));
      }
    }
    __syncthreads();
  }
}

// ------------------------------------------------------------------------------------------------------------------
// Stage c, part 2: sparse down projection, partial sums.  Block (tile, split): 2048 columns x every `nsplit`-th
// neuron of the stage; rows of neurons whose activation is zero for every token are not read.
// ------------------------------------------------------------------------------------------------------------------
template <int WD, int BT>
__global__ void __launch_bounds__(256)
    ls_down_kernel(const uint16_t* __restrict__ bundles, int n_mat, const int32_t* __restrict__ slot_of,
                   const int32_t* __restrict__ exec_idx, const int32_t* __restrict__ count_ptr, int K, int c,
                   const float* __restrict__ act, int act_stride, int B, int d, int F, float* __restrict__ ypart) {
  const int ch = blockIdx.x * blockDim.x + threadIdx.x;  // 8-column chunk
  const int split = blockIdx.y, nsplit = gridDim.y;
  int lo, hi;
  stage_bounds(*count_ptr, K, c, lo, hi);
  float acc[BT][8];
#pragma unroll
  for (int b = 0; b < BT; ++b)
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[b][e] = 0.f;
  const bool live = ch < (d >> 3);
  const int down_off = (n_mat - 1) * d;
  for (int p = lo + split; p < hi; p += nsplit) {
    float a[BT];
    bool any = false;
#pragma unroll
    for (int b = 0; b < BT; ++b) {
      a[b] = b < B ? act[(size_t)b * act_stride + p] : 0.f;
      any |= (a[b] != 0.f);
    }
    if (!any || !live) continue;
    const int i = exec_idx[p];
    if ((unsigned)i >= (unsigned)F) continue;
    const int slot = slot_of ? slot_of[i] : i;
    if (slot < 0) continue;
    float w[8];
    unpack8<WD>(ld_stream128(bundles + (size_t)slot * n_mat * d + down_off + ch * 8), w);
#pragma unroll
    for (int b = 0; b < BT; ++b)
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[b][e] = fmaf(a[b], w[e], acc[b][e]);
  }
  if (!live) return;
#pragma unroll
  for (int b = 0; b < BT; ++b) {
    if (b < B) {
      float4* dst = reinterpret_cast<float4*>(ypart + ((size_t)split * B + b) * d + ch * 8);
      dst[0] = make_float4(acc[b][0], acc[b][1], acc[b][2], acc[b][3]);
      dst[1] = make_float4(acc[b][4], acc[b][5], acc[b][6], acc[b][7]);
    }
  }
}

// x~^(c+1) = x~^(c) + sum over splits (fixed order: deterministic); optional copies to the trace and to x_out.
// Eight threads per element (the splits dealt over them, their partial sums added by a fixed tree): with one thread per
// element the kernel was a handful of blocks each waiting for its own chain of loads.  blockDim.x a multiple of 32.
__global__ void ls_stage_finalize_kernel(const float* __restrict__ ypart, int nsplit, int B, int d, float* xt, float* trace_out,
                                         float* x_out) {
  const int n = B * d;
  const int part = threadIdx.x & 7;
  const int per_block = blockDim.x >> 3;
  for (int i0 = blockIdx.x * per_block; i0 < n; i0 += gridDim.x * per_block) {  // (uniform over the block: shuffles below)
    const int i = i0 + (threadIdx.x >> 3);
    float s = 0.f;
    if (i < n)
      for (int sp = part; sp < nsplit; sp += 8) s += ypart[(size_t)sp * n + i];
    s += __shfl_xor_sync(0xffffffffu, s, 1);
    s += __shfl_xor_sync(0xffffffffu, s, 2);
    s += __shfl_xor_sync(0xffffffffu, s, 4);
    if (part == 0 && i < n) {
      const float v = xt[i] + s;
      xt[i] = v;
      if (trace_out) trace_out[i] = v;
      if (x_out) x_out[i] = v;
    }
  }
}

__global__ void ls_copy_f32_kernel(const float* __restrict__ src, float* dst, int n) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) dst[i] = src[i];
}
__global__ void ls_copy_u32_kernel(const uint32_t* __restrict__ src, uint32_t* dst, int n) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) dst[i] = src[i];
}
__global__ void ls_fill_u32_kernel(uint32_t* dst, uint32_t v, int n) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) dst[i] = v;
}

}  // namespace ls
