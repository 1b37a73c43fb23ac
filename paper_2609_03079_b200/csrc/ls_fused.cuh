// One kernel per layer step for the all-resident, batch-1 case (the decode hot path).
//
// One CTA per SM, cooperative launch (all CTAs co-resident), two warp-specialised roles per CTA:
//
//   stream role  (warps 0..7)  walks the CTA's share of the selected neurons in execution order without ever waiting
//                              for the predictor: gate+up rows arrive by 1-D TMA bulk copies into a shared-memory ring,
//                              the block reduces the two dot products, surviving neurons fetch their down row into a
//                              second ring, partial outputs are kept in registers per stage and flushed to the stage
//                              accumulator with vector reductions; then the CTA arrives on the stage counter.
//   predict role (warps 8..15) holds its share of the next layer's predictor (rows of A^T and B^T, expanded once to
//                              the high words of their fp64 values) in shared memory and runs the K+1 refinement
//                              evaluations as a three-deep software pipeline  Z_j | S_{j-1} | R_{j-2}  (latent, scores +
//                              histogram + bucket insert, exact ranks), separated by barriers among the predict roles.
//
// The coordination is asymmetric: stream roles only signal (arrive on stage counters), predict roles wait (bounded spins).
// Everything a launch dirties in the per-layer scratch is zero again when it ends (the last CTA to finish cleans).
#pragma once
#include "ls_common.cuh"

namespace ls {

constexpr int FZ_STREAM_THREADS = 256;
constexpr int FZ_PRED_THREADS = 256;
constexpr int FZ_THREADS = FZ_STREAM_THREADS + FZ_PRED_THREADS;
constexpr int FZ_NB = 4096;    // score bins
constexpr int FZ_CNT_STRIDE = FZ_NB + 4;  // bin counts + overflow count, padded so every set stays 16-byte aligned
constexpr int FZ_CAPB = 16;    // bucket capacity per bin; the rest goes to the overflow list
constexpr int FZ_MAXK = 16;    // stages supported by the fused path
constexpr int FZ_GU_DEPTH = 3; // gate/up ring stages
constexpr int FZ_DN_DEPTH = 3; // down-row ring stages
constexpr long long FZ_SPIN_LIMIT = 40LL * 1000 * 1000;

struct FusedArgs {
  // layer being executed
  const uint16_t* bundles; int n_mat; int gated; const float* b_gate; const float* b_down;
  int d, F, norm; float eps;
  const float* x; float* x_out;
  const int32_t* sel_idx; const int32_t* sel_count; int sel_cap; int K;
  float* dacc;            // [FZ_MAXK][d] stage accumulators, zero on entry and on exit
  unsigned* stage_done;   // [FZ_MAXK] arrivals per stage, zero on entry and on exit
  unsigned* fin;          // [1] CTAs finished, zero on entry and on exit
  int* status;
  // next layer's predictor (has_next == 0: no refinement)
  int has_next;
  const uint16_t* At; const uint16_t* Bt; const float* pc;
  int r, Fn, norm_n; float eps_n; int k_next;
  double* z;              // [2][r]
  double* sumsq;          // [2]
  unsigned* cnt;          // [3][FZ_CNT_STRIDE] bin counts (+ overflow count at FZ_NB), zero on entry and on exit
  unsigned long long* bkey;  // [3][FZ_NB * FZ_CAPB]
  int32_t* bidx;             // [3][FZ_NB * FZ_CAPB]
  unsigned long long* okey;  // [3][Fn] overflow entries
  int32_t* oidx;             // [3][Fn]
  int32_t* obin;             // [3][Fn]
  double* range;          // [4]: lo, hi used for binning; lo, hi observed by the last evaluation (for the next launch)
  unsigned long long* range_obs;  // [2] ordered keys: min, max observed in the final evaluation
  unsigned* bar_count; unsigned* bar_gen;
  int32_t* tmp_idx;       // [max_sel] list of an intermediate evaluation (not returned)
  // outputs for the next layer
  int32_t* next_idx; int32_t* next_count; uint32_t* next_mask; double* next_scores; double* next_prio; int next_cap;
  // trace (all nullable)
  float* tr_xtilde; uint32_t* tr_masks; int32_t* tr_counts; uint32_t* tr_survive;
};

// ---- PTX helpers ---------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after a fixed number of polls and records a timeout instead of hanging.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, int* status) {
  for (long long it = 0; it < FZ_SPIN_LIMIT; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  set_status(status, ST_TIMEOUT);
  return false;
}
// 1-D bulk copy global -> shared, completion counted in bytes on an mbarrier (no multicast).
__device__ __forceinline__ void tma_load_1d(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
  asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ float4 ld_cg_f4(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }

// Waits (bounded) until *ctr >= target; one thread calls it.
__device__ __forceinline__ bool spin_until_ge(const unsigned* ctr, unsigned target, int* status) {
  for (long long it = 0; it < FZ_SPIN_LIMIT; ++it) {
    if (ld_acquire_u32(ctr) >= target) return true;
    if (it > 64) __nanosleep(32);
  }
  set_status(status, ST_TIMEOUT);
  return false;
}

// Barrier among the predict roles of all CTAs (self-resetting counter + generation).
__device__ __forceinline__ void predict_grid_barrier(const FusedArgs& A, int G, int ptid) {
  named_bar_sync(2, FZ_PRED_THREADS);
  if (ptid == 0) {
    const unsigned my = ld_acquire_u32(A.bar_gen);
    __threadfence();
    const unsigned old = atomicAdd(A.bar_count, 1u);
    if (old == (unsigned)G - 1u) {
      atomicExch(A.bar_count, 0u);
      __threadfence();
      atomicAdd(A.bar_gen, 1u);
    } else {
      bool ok = false;
      for (long long it = 0; it < FZ_SPIN_LIMIT; ++it) {
        if (ld_acquire_u32(A.bar_gen) != my) { ok = true; break; }
        if (it > 16) __nanosleep(20);
      }
      if (!ok) set_status(A.status, ST_TIMEOUT);
    }
    __threadfence();
  }
  named_bar_sync(2, FZ_PRED_THREADS);
}

// High 32 bits of the fp64 value of a 16-bit weight (its low word is zero): exact widening done once per layer.
template <int WD>
__device__ __forceinline__ uint32_t w16_to_f64hi(uint16_t b) {
  float f;
  if (WD == WD_BF16) f = __uint_as_float((uint32_t)b << 16);
  else f = __half2float(__ushort_as_half(b));
  return (uint32_t)__double2hiint((double)f);
}

struct FusedSmemLayout {
  size_t gu_off, dn_off, bar_off, red_off, a_off, b_off, xt_off, zs_off, base_off, own_off, misc_off, total;
  int per, nA;
};

__host__ __device__ inline FusedSmemLayout fused_layout(int d, int n_in, int r, int Fn, int G, int has_next) {
  FusedSmemLayout L{};
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o += (bytes + 127) & ~(size_t)127; return at; };
  L.gu_off = take((size_t)FZ_GU_DEPTH * n_in * d * 2);
  L.dn_off = take((size_t)FZ_DN_DEPTH * d * 2);
  L.bar_off = take(16 * 8);
  L.red_off = take(2 * 8 * 2 * 4 + 64 * 8);      // stream dot partials (double-buffered) + predict fp64 partials
  L.per = has_next ? (Fn + G - 1) / G : 0;
  L.nA = has_next ? (r + G - 1) / G : 0;
  L.a_off = take((size_t)L.nA * d * 4);
  L.b_off = take((size_t)L.per * r * 4);
  L.xt_off = take((size_t)d * 4);
  L.zs_off = take((size_t)(has_next ? r : 0) * 8);
  L.base_off = take(has_next ? (size_t)(FZ_NB + 1) * 4 : 0);
  L.own_off = take((size_t)L.per * (8 + 4) * 2);  // own scores and bins, double-buffered by evaluation parity
  L.misc_off = take(256);
  L.total = o;
  return L;
}

// =====================================================================================================================
template <int WD, int CPT>
__global__ void __launch_bounds__(FZ_THREADS, 1) ls_fused_step_kernel(const __grid_constant__ FusedArgs A) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int G = gridDim.x, cta = blockIdx.x, tid = threadIdx.x;
  const int d = A.d, K = A.K, nchunk = A.d >> 3;
  const int n_in = A.gated ? 2 : 1;
  const FusedSmemLayout lay = fused_layout(d, n_in, A.r, A.Fn, G, A.has_next);
  uint16_t* s_gu = reinterpret_cast<uint16_t*>(smem + lay.gu_off);
  uint16_t* s_dn = reinterpret_cast<uint16_t*>(smem + lay.dn_off);
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(smem + lay.bar_off);  // [0..GU) gate/up full, [8..8+DN) down full
  float* s_red = reinterpret_cast<float*>(smem + lay.red_off);        // [2][8][2]
  double* s_redd = reinterpret_cast<double*>(smem + lay.red_off + 2 * 8 * 2 * 4);  // [64]

  if (tid == 0) {
    for (int i = 0; i < FZ_GU_DEPTH; ++i) mbar_init(&s_bar[i], 1);
    for (int i = 0; i < FZ_DN_DEPTH; ++i) mbar_init(&s_bar[8 + i], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  const int count = max(0, min(*A.sel_count, A.sel_cap));
  const int m = count > 0 ? (count + K - 1) / K : 1;

  if (tid < FZ_STREAM_THREADS) {
    // ================================================= stream role =================================================
    const int lane = tid & 31, warp = tid >> 5;
    float xr[CPT][8];
    double sq = 0.0;
#pragma unroll
    for (int q = 0; q < CPT; ++q) {
      const int ch = tid + q * FZ_STREAM_THREADS;
      if (ch < nchunk) {
        const float4 a0 = __ldg(reinterpret_cast<const float4*>(A.x + ch * 8));
        const float4 a1 = __ldg(reinterpret_cast<const float4*>(A.x + ch * 8 + 4));
        xr[q][0] = a0.x; xr[q][1] = a0.y; xr[q][2] = a0.z; xr[q][3] = a0.w;
        xr[q][4] = a1.x; xr[q][5] = a1.y; xr[q][6] = a1.z; xr[q][7] = a1.w;
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) xr[q][e] = 0.f;
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) sq = fma((double)xr[q][e], (double)xr[q][e], sq);
    }
    sq = warp_sum(sq);
    if (lane == 0) s_redd[warp] = sq;
    named_bar_sync(1, FZ_STREAM_THREADS);
    double tot = 0.0;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += s_redd[w];
    const float inv_rms = A.norm == 0 ? (float)(1.0 / sqrt(tot / (double)d + (double)A.eps)) : 1.0f;

    const uint32_t gu_bytes = (uint32_t)n_in * d * 2, dn_bytes = (uint32_t)d * 2;
    const size_t bundle_elems = (size_t)A.n_mat * d;
    const int n_mine = cta < count ? (count - cta + G - 1) / G : 0;

    auto issue_gu = [&](int it) {  // thread 0 only
      const int p = cta + it * G;
      int i = A.sel_idx[p];
      if ((unsigned)i >= (unsigned)A.F) { set_status(A.status, ST_BAD_INDEX); i = 0; }
      uint64_t* bar = &s_bar[it % FZ_GU_DEPTH];
      mbar_expect_tx(bar, gu_bytes);
      tma_load_1d(s_gu + (size_t)(it % FZ_GU_DEPTH) * n_in * d, A.bundles + (size_t)i * bundle_elems, gu_bytes, bar);
    };
    if (tid == 0)
      for (int it = 0; it < min(n_mine, FZ_GU_DEPTH); ++it) issue_gu(it);

    // pending down rows: FIFO over the down ring (entries hold the activation and the stage parity)
    __shared__ float dq_a[FZ_DN_DEPTH];
    __shared__ int dq_par[FZ_DN_DEPTH];
    int dq_head = 0, dq_tail = 0;  // uniform across the stream threads
    float yacc[2][CPT][8];
#pragma unroll
    for (int s = 0; s < 2; ++s)
#pragma unroll
      for (int q = 0; q < CPT; ++q)
#pragma unroll
        for (int e = 0; e < 8; ++e) yacc[s][q][e] = 0.f;
    int open_lo = 0;  // stages < open_lo have been flushed and arrived
    bool dirty0 = false, dirty1 = false;  // accumulator sets that hold something

    auto consume_one = [&]() {  // consume the head of the down FIFO into the accumulator of its stage parity
      const int slot = dq_head % FZ_DN_DEPTH;
      mbar_wait(&s_bar[8 + slot], (uint32_t)((dq_head / FZ_DN_DEPTH) & 1), A.status);
      const float a = dq_a[slot];
      const int par = dq_par[slot] & 1;
      if (par == 0) dirty0 = true; else dirty1 = true;
      const uint16_t* row = s_dn + (size_t)slot * d;
#pragma unroll
      for (int q = 0; q < CPT; ++q) {
        const int ch = tid + q * FZ_STREAM_THREADS;
        if (ch < nchunk) {
          float w[8];
          unpack8<WD>(*reinterpret_cast<const uint4*>(row + ch * 8), w);
          if (par == 0) {
#pragma unroll
            for (int e = 0; e < 8; ++e) yacc[0][q][e] = fmaf(a, w[e], yacc[0][q][e]);
          } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) yacc[1][q][e] = fmaf(a, w[e], yacc[1][q][e]);
          }
        }
      }
      ++dq_head;
    };
    auto flush_stage = [&](int s) {  // add this CTA's partial of stage s to the stage accumulator, then arrive
      float* dst = A.dacc + (size_t)s * d;
      const bool dirty = (s & 1) ? dirty1 : dirty0;
      if ((s & 1) == 0) dirty0 = false; else dirty1 = false;
#pragma unroll
      for (int q = 0; q < CPT; ++q) {
        const int ch = tid + q * FZ_STREAM_THREADS;
        if (dirty && ch < nchunk) {
          if ((s & 1) == 0) {
            red_add_v4(dst + ch * 8, yacc[0][q][0], yacc[0][q][1], yacc[0][q][2], yacc[0][q][3]);
            red_add_v4(dst + ch * 8 + 4, yacc[0][q][4], yacc[0][q][5], yacc[0][q][6], yacc[0][q][7]);
#pragma unroll
            for (int e = 0; e < 8; ++e) yacc[0][q][e] = 0.f;
          } else {
            red_add_v4(dst + ch * 8, yacc[1][q][0], yacc[1][q][1], yacc[1][q][2], yacc[1][q][3]);
            red_add_v4(dst + ch * 8 + 4, yacc[1][q][4], yacc[1][q][5], yacc[1][q][6], yacc[1][q][7]);
#pragma unroll
            for (int e = 0; e < 8; ++e) yacc[1][q][e] = 0.f;
          }
        }
      }
      named_bar_sync(1, FZ_STREAM_THREADS);
      if (tid == 0) {
        __threadfence();
        atomicAdd(&A.stage_done[s], 1u);
      }
    };
    // close every stage below `upto`: their pending down rows are consumed first (FIFO order = stage order)
    auto close_stages = [&](int upto, bool had_data_hint) {
      (void)had_data_hint;
      while (open_lo < upto) {
        while (dq_head < dq_tail && (dq_par[dq_head % FZ_DN_DEPTH] >> 8) <= open_lo) consume_one();
        flush_stage(open_lo);
        ++open_lo;
      }
    };

    for (int it = 0; it < n_mine; ++it) {
      const int p = cta + it * G;
      const int stage = min(p / m, K - 1);
      // a stage may stay open while the next one runs (two accumulator sets); anything older is closed now
      if (stage - 1 > open_lo) close_stages(stage - 1, true);
      const int slot = it % FZ_GU_DEPTH;
      mbar_wait(&s_bar[slot], (uint32_t)((it / FZ_GU_DEPTH) & 1), A.status);
      const uint16_t* grow = s_gu + (size_t)slot * n_in * d;
      float pg = 0.f, pu = 0.f;
#pragma unroll
      for (int q = 0; q < CPT; ++q) {
        const int ch = tid + q * FZ_STREAM_THREADS;
        if (ch < nchunk) {
          float w[8];
          unpack8<WD>(*reinterpret_cast<const uint4*>(grow + ch * 8), w);
#pragma unroll
          for (int e = 0; e < 8; ++e) pg = fmaf(w[e], xr[q][e], pg);
          if (A.gated) {
            unpack8<WD>(*reinterpret_cast<const uint4*>(grow + d + ch * 8), w);
#pragma unroll
            for (int e = 0; e < 8; ++e) pu = fmaf(w[e], xr[q][e], pu);
          }
        }
      }
      pg = warp_sum(pg);
      pu = warp_sum(pu);
      float* red = s_red + (it & 1) * 16;
      if (lane == 0) { red[warp * 2] = pg; red[warp * 2 + 1] = pu; }
      named_bar_sync(1, FZ_STREAM_THREADS);  // also: every thread has finished reading ring slot `slot`
      float g = 0.f, u = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) { g += red[w * 2]; u += red[w * 2 + 1]; }
      int i = A.sel_idx[p];
      if ((unsigned)i >= (unsigned)A.F) i = -1;
      g = g * inv_rms + ((A.b_gate && i >= 0) ? A.b_gate[i] : 0.f);
      float a = fmaxf(g, 0.f);
      if (A.gated) a *= u * inv_rms;
      if (i < 0) a = 0.f;
      if (tid == 0 && it + FZ_GU_DEPTH < n_mine) issue_gu(it + FZ_GU_DEPTH);
      if (a != 0.f) {
        if (dq_tail - dq_head == FZ_DN_DEPTH) consume_one();  // ring full: make room
        named_bar_sync(1, FZ_STREAM_THREADS);                 // everyone is past its reads of the slot being refilled
        const int ds = dq_tail % FZ_DN_DEPTH;
        if (tid == 0) {
          dq_a[ds] = a;
          dq_par[ds] = (stage & 1) | (stage << 8);
          uint64_t* bar = &s_bar[8 + ds];
          mbar_expect_tx(bar, dn_bytes);
          tma_load_1d(s_dn + (size_t)ds * d, A.bundles + (size_t)i * bundle_elems + (size_t)(A.n_mat - 1) * d, dn_bytes, bar);
          if (A.tr_survive) atomicOr(&A.tr_survive[i >> 5], 1u << (i & 31));
        }
        ++dq_tail;
        named_bar_sync(1, FZ_STREAM_THREADS);  // dq_a / dq_par visible to every stream thread
      }
      // keep at most two rows in flight behind the gate/up front
      while (dq_tail - dq_head > 2) consume_one();
    }
    close_stages(K, false);
    // (dq_par: low bit selects the accumulator set, bits 8.. carry the stage for close_stages)
  } else {
    // ================================================= predict role ================================================
    const int ptid = tid - FZ_STREAM_THREADS, lane = ptid & 31, warp = ptid >> 5;
    float* s_xt = reinterpret_cast<float*>(smem + lay.xt_off);
    uint32_t* s_A = reinterpret_cast<uint32_t*>(smem + lay.a_off);
    uint32_t* s_B = reinterpret_cast<uint32_t*>(smem + lay.b_off);
    double* s_zs = reinterpret_cast<double*>(smem + lay.zs_off);
    unsigned* s_base = reinterpret_cast<unsigned*>(smem + lay.base_off);
    double* s_own = reinterpret_cast<double*>(smem + lay.own_off);          // [2][per]
    int* s_ownbin = reinterpret_cast<int*>(s_own + 2 * lay.per);            // [2][per]
    int* s_misc = reinterpret_cast<int*>(smem + lay.misc_off);
    const int per = lay.per, r = A.r, Fn = A.Fn;
    const int i_lo = cta * per, i_hi = min(Fn, i_lo + per);

    const bool active = A.has_next || cta == 0;  // without a next layer only CTA 0 tracks x~ (to write x_out and the trace)
    // x~^(0) = x (+ b_down)
    if (active)
      for (int c = ptid; c < d; c += FZ_PRED_THREADS) s_xt[c] = A.x[c] + (A.b_down ? A.b_down[c] : 0.f);
    if (A.has_next) {
      // this CTA's rows of A^T and B^T, widened once to fp64 high words
      for (int a = 0; a < lay.nA; ++a) {
        const int j = cta + a * G;
        if (j < r)
          for (int c = ptid; c < d; c += FZ_PRED_THREADS) s_A[a * d + c] = w16_to_f64hi<WD>(A.At[(size_t)j * d + c]);
      }
      const int nB = max(0, i_hi - i_lo) * r;
      const uint16_t* bsrc = A.Bt + (size_t)i_lo * r;
      for (int t = ptid; t < nB; t += FZ_PRED_THREADS) s_B[t] = w16_to_f64hi<WD>(bsrc[t]);
    }
    named_bar_sync(2, FZ_PRED_THREADS);
    if (cta == 0 && A.tr_xtilde)
      for (int c = ptid; c < d; c += FZ_PRED_THREADS) A.tr_xtilde[c] = s_xt[c];

    const double bin_lo = A.has_next ? __ldcg(&A.range[0]) : 0.0;
    const double bin_hi = A.has_next ? __ldcg(&A.range[1]) : 0.0;
    const double INF = __longlong_as_double(0x7ff0000000000000LL);
    const double brange = bin_hi - bin_lo;
    const double bscale = (brange > 0.0 && brange < INF) ? (double)FZ_NB / brange : 0.0;
    const int keff = min(A.k_next, Fn);
    const int n_phase = A.has_next ? K + 3 : (active ? K + 1 : 0);

    for (int ph = 0; ph < n_phase; ++ph) {
      // ---------------- feature update (ph >= 1) and latent Z_ph
      if (ph >= 1 && ph <= K) {
        if (ptid == 0) spin_until_ge(&A.stage_done[ph - 1], (unsigned)G, A.status);
        named_bar_sync(2, FZ_PRED_THREADS);
        const float* acc = A.dacc + (size_t)(ph - 1) * d;
        for (int c4 = ptid; c4 < (d >> 2); c4 += FZ_PRED_THREADS) {
          const float4 v = ld_cg_f4(acc + c4 * 4);
          float4 t = *reinterpret_cast<float4*>(s_xt + c4 * 4);
          t.x += v.x; t.y += v.y; t.z += v.z; t.w += v.w;
          *reinterpret_cast<float4*>(s_xt + c4 * 4) = t;
          if (cta == 0) {
            if (A.tr_xtilde) *reinterpret_cast<float4*>(A.tr_xtilde + (size_t)ph * d + c4 * 4) = t;
            if (ph == K) *reinterpret_cast<float4*>(A.x_out + c4 * 4) = t;
          }
        }
        named_bar_sync(2, FZ_PRED_THREADS);
      }
      if (!A.has_next) continue;

      if (ph <= K) {
        // Z_ph: this CTA's latent rows (un-normalised) and, on CTA 0, the sum of squares
        double part[3] = {0.0, 0.0, 0.0};
        for (int c = ptid; c < d; c += FZ_PRED_THREADS) {
          const double xv = (double)s_xt[c];
          if (lay.nA > 0) part[0] = fma(__hiloint2double((int)s_A[c], 0), xv, part[0]);
          if (lay.nA > 1) part[1] = fma(__hiloint2double((int)s_A[d + c], 0), xv, part[1]);
          part[2] = fma(xv, xv, part[2]);
        }
        // rows beyond two (large ranks on few SMs) are handled one by one
        for (int e = 0; e < 3; ++e) {
          part[e] = warp_sum(part[e]);
          if (lane == 0) s_redd[8 + e * 8 + warp] = part[e];
        }
        named_bar_sync(2, FZ_PRED_THREADS);
        if (ptid < 3) {
          double t = 0.0;
          for (int w = 0; w < 8; ++w) t += s_redd[8 + ptid * 8 + w];
          if (ptid < 2) {
            const int j = cta + ptid * G;
            if (ptid < lay.nA && j < r) A.z[(size_t)(ph & 1) * r + j] = t;
          } else if (cta == 0) {
            A.sumsq[ph & 1] = t;
          }
        }
        for (int a = 2; a < lay.nA; ++a) {
          const int j = cta + a * G;
          double pa = 0.0;
          for (int c = ptid; c < d; c += FZ_PRED_THREADS) pa = fma(__hiloint2double((int)s_A[a * d + c], 0), (double)s_xt[c], pa);
          pa = warp_sum(pa);
          named_bar_sync(2, FZ_PRED_THREADS);
          if (lane == 0) s_redd[8 + warp] = pa;
          named_bar_sync(2, FZ_PRED_THREADS);
          if (ptid == 0 && j < r) {
            double t = 0.0;
            for (int w = 0; w < 8; ++w) t += s_redd[8 + w];
            A.z[(size_t)(ph & 1) * r + j] = t;
          }
        }
      }

      // ---------------- S_{ph-1}: scores of this CTA's neurons, histogram, bucket insert
      if (ph >= 1 && ph <= K + 1) {
        const int e = ph - 1, es = e % 3, ep = e & 1;
        const double inv = A.norm_n == 0 ? 1.0 / sqrt(__ldcg(&A.sumsq[ep]) / (double)d + (double)A.eps_n) : 1.0;
        for (int j = ptid; j < r; j += FZ_PRED_THREADS) s_zs[j] = __ldcg(&A.z[(size_t)ep * r + j]) * inv;
        named_bar_sync(2, FZ_PRED_THREADS);
        unsigned* cnt = A.cnt + (size_t)es * FZ_CNT_STRIDE;
        for (int li = warp; li < i_hi - i_lo; li += FZ_PRED_THREADS / 32) {
          const uint32_t* brow = s_B + (size_t)li * r;
          double acc = 0.0;
          for (int j = lane; j < r; j += 32) acc = fma(__hiloint2double((int)brow[j], 0), s_zs[j], acc);
          acc = warp_sum(acc);
          if (lane == 0) {
            const int i = i_lo + li;
            const double s = canonical_score(acc + (A.pc ? (double)A.pc[i] : 0.0));
            const double sc = fmin(fmax(s, -1.7976931348623157e308), 1.7976931348623157e308);
            int b = (int)((bin_hi - sc) * bscale);
            b = max(0, min(FZ_NB - 1, b));
            const unsigned slot = atomicAdd(&cnt[b], 1u);
            const unsigned long long key = ordered_key(s);
            if (slot < (unsigned)FZ_CAPB) {
              A.bkey[((size_t)es * FZ_NB + b) * FZ_CAPB + slot] = key;
              A.bidx[((size_t)es * FZ_NB + b) * FZ_CAPB + slot] = i;
            } else {
              const unsigned o = atomicAdd(&cnt[FZ_NB], 1u);
              A.okey[(size_t)es * Fn + o] = key;
              A.oidx[(size_t)es * Fn + o] = i;
              A.obin[(size_t)es * Fn + o] = b;
            }
            s_own[ep * per + li] = s;
            s_ownbin[ep * per + li] = b;
            if (e == K) {
              if (A.next_prio) A.next_prio[i] = s;
              if (A.next_scores) A.next_scores[i] = s;
              atomicMin(&A.range_obs[0], key);
              atomicMax(&A.range_obs[1], key);
            }
          }
        }
      }

      // ---------------- R_{ph-2}: exact ranks of this CTA's neurons from the global histogram and buckets
      if (ph >= 2) {
        const int e = ph - 2, es = e % 3, ep = e & 1;
        const unsigned* cnt = A.cnt + (size_t)es * FZ_CNT_STRIDE;
        // exclusive prefix over the bins: 16 bins per thread
        unsigned c16[16], run = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint4 v = __ldcg(reinterpret_cast<const uint4*>(cnt + ptid * 16 + q * 4));
          c16[q * 4] = v.x; c16[q * 4 + 1] = v.y; c16[q * 4 + 2] = v.z; c16[q * 4 + 3] = v.w;
          run += v.x + v.y + v.z + v.w;
        }
        unsigned incl = run;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += t;
        }
        if (lane == 31) s_misc[warp] = (int)incl;
        named_bar_sync(2, FZ_PRED_THREADS);
        unsigned woff = 0;
        for (int w = 0; w < warp; ++w) woff += (unsigned)s_misc[w];
        unsigned base = woff + incl - run;
#pragma unroll
        for (int q = 0; q < 16; ++q) { s_base[ptid * 16 + q] = base; base += c16[q]; }
        const unsigned novf = __ldcg(&cnt[FZ_NB]);
        named_bar_sync(2, FZ_PRED_THREADS);
        int32_t* idx_out = (e == K) ? A.next_idx : A.tmp_idx;
        const int cap = (e == K) ? A.next_cap : 0x7fffffff;
        uint32_t* mask_out = A.tr_masks ? A.tr_masks + (size_t)e * ((Fn + 31) >> 5) : nullptr;
        for (int li = ptid; li < i_hi - i_lo; li += FZ_PRED_THREADS) {
          const int b = s_ownbin[ep * per + li];
          const unsigned b0 = s_base[b];
          if ((int)b0 >= keff) continue;
          const int i = i_lo + li;
          const unsigned long long kp = ordered_key(s_own[ep * per + li]);
          const unsigned nb = min(__ldcg(&cnt[b]), (unsigned)FZ_CAPB);
          int before = 0;
          const size_t bo = ((size_t)es * FZ_NB + b) * FZ_CAPB;
          for (unsigned q = 0; q < nb; ++q) {
            const unsigned long long kq = __ldcg(&A.bkey[bo + q]);
            const int iq = __ldcg(&A.bidx[bo + q]);
            before += (kq > kp) || (kq == kp && iq < i);
          }
          for (unsigned q = 0; q < novf; ++q) {
            if (__ldcg(&A.obin[(size_t)es * Fn + q]) != b) continue;
            const unsigned long long kq = __ldcg(&A.okey[(size_t)es * Fn + q]);
            const int iq = __ldcg(&A.oidx[(size_t)es * Fn + q]);
            before += (kq > kp) || (kq == kp && iq < i);
          }
          const int rank = (int)b0 + before;
          if (rank < keff) {
            if (rank < cap) idx_out[rank] = i;
            if (mask_out) atomicOr(&mask_out[i >> 5], 1u << (i & 31));
            if (e == K && A.next_mask) atomicOr(&A.next_mask[i >> 5], 1u << (i & 31));
          }
        }
        if (cta == 0 && ptid == 0) {
          if (A.tr_counts) A.tr_counts[e] = keff;
          if (e == K) {
            *A.next_count = min(keff, A.next_cap);
            if (keff > A.next_cap) set_status(A.status, ST_CAPACITY);
          }
        }
      }
      if (ph + 1 < n_phase) {
        predict_grid_barrier(A, G, ptid);
        // the bin counts read in this phase (evaluation ph-2) are free now: clear this CTA's slice for their next use
        if (ph >= 2) {
          unsigned* cz = A.cnt + (size_t)((ph - 2) % 3) * FZ_CNT_STRIDE;
          for (int t = cta * FZ_PRED_THREADS + ptid; t < FZ_NB + 1; t += G * FZ_PRED_THREADS) cz[t] = 0u;
        }
      }
    }
  }

  // ---- the last CTA to finish restores the zero-on-entry invariants of the per-layer scratch
  __syncthreads();
  __shared__ int s_last;
  if (tid == 0) {
    __threadfence();
    s_last = (atomicAdd(A.fin, 1u) == (unsigned)G - 1u) ? 1 : 0;
  }
  __syncthreads();
  if (s_last) {
    __threadfence();
    for (int t = tid; t < K * d; t += FZ_THREADS) A.dacc[t] = 0.f;
    for (int t = tid; t < FZ_MAXK; t += FZ_THREADS) A.stage_done[t] = 0u;
    if (A.has_next) {
      for (int t = tid; t < 3 * FZ_CNT_STRIDE; t += FZ_THREADS) A.cnt[t] = 0u;
      if (tid == 0) {
        // binning range for the next launch: what the final evaluation observed, widened by 5 % on each side
        const unsigned long long kmin = A.range_obs[0], kmax = A.range_obs[1];
        if (kmin <= kmax) {
          auto unkey = [](unsigned long long k) {
            const unsigned long long b = (k >> 63) ? (k & 0x7fffffffffffffffULL) : ~k;
            return __longlong_as_double((long long)b);
          };
          double lo = unkey(kmin), hi = unkey(kmax);
          lo = fmax(lo, -1.0e300);
          hi = fmin(hi, 1.0e300);
          const double pad = 0.05 * (hi - lo);
          A.range[0] = lo - pad;
          A.range[1] = hi + pad;
        }
        A.range_obs[0] = 0xffffffffffffffffULL;
        A.range_obs[1] = 0ULL;
      }
    }
    if (tid == 0) *A.fin = 0u;
  }
}

}  // namespace ls
