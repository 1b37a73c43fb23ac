// One kernel per layer step for the all-resident, batch-1 case (the decode hot path).
//
// Grid barriers cost far more on this machine than any of the small predictor phases, so the step is organised to need
// only three of them, whatever the number of stages K:
//
//   1. stream   The K priority stages of the layer (Eq. 1) run CONCURRENTLY on K disjoint groups of CTAs (the output is
//               a sum over hidden neurons, so stage order in time is free; only stage membership defines the partial
//               features).  Inside a CTA the stream warps take two neurons per round: gate+up rows arrive by 1-D TMA
//               bulk copies into a shared-memory ring, the block reduces the dot products, surviving neurons fetch
//               their down row into a second ring, and the CTA's whole contribution to its stage is kept in registers
//               and added once to the stage accumulator (vector reductions).  Meanwhile the loader warps bring this
//               CTA's share of the next layer's predictor (rows of A^T and of B^T) into shared memory.
//      -- barrier --
//   2. latent   Every partial residual feature x~^(j) = x + sum_{c<j} dm^(c), j = 0..K (Eq. 2), is rebuilt on the fly
//               from the stage accumulators, and this CTA's rows of all K+1 latents z^(j) = A^T x~^(j) are formed in one
//               pass (fp64), each weight converted once and used K+1 times.
//      -- barrier --
//   3. scores   All K+1 score vectors of this CTA's neurons (fp64), histogram + bucket insert per evaluation.
//      -- barrier --
//   4. ranks    Exact rank of every neuron that can be inside the first k ranks, for every evaluation: coarse prefix,
//               fine prefix inside one coarse bin, comparison inside the neuron's bucket.
//
// Everything a launch dirties in the per-layer scratch is zero again when it ends (the last CTA to finish cleans).
#pragma once
#include "ls_common.cuh"

namespace ls {

constexpr int FZ_STREAM_THREADS = 256;
constexpr int FZ_THREADS = 512;
constexpr int FZ_NG = 2;          // neurons the stream warps process per round
constexpr int FZ_NB = 4096;       // fine score bins per evaluation
constexpr int FZ_NC = 64;         // coarse bins (FZ_NB / FZ_NC fine bins each)
constexpr int FZ_CNT_STRIDE = FZ_NB + FZ_NC + 4;  // fine counts, coarse counts, overflow count (+ padding to 16 bytes)
constexpr int FZ_CAPB = 16;       // bucket capacity per fine bin; the rest goes to the overflow list
constexpr int FZ_MAXK = 16;       // stages supported by the fused path
constexpr int FZ_MAXE = FZ_MAXK + 1;  // evaluations j = 0..K
constexpr int FZ_BPAD = 8;        // padding (elements) of a predictor row in shared memory: eight rows on distinct banks
constexpr int FZ_ZPAD = 4;        // padding (doubles) of a latent row in shared memory
constexpr int FZ_MAX_DEPTH = 8;   // most ring stages; the depths are chosen per launch from the shared memory left
constexpr int FZ_MAX_MINE = 256;  // neurons one CTA may own in one step
constexpr long long FZ_SPIN_CYCLES = 4000LL * 1000 * 1000;  // every wait gives up after about two seconds of SM clocks

struct FusedArgs {
  // layer being executed
  const uint16_t* bundles; int n_mat; int gated; const float* b_gate; const float* b_down;
  int d, F, norm; float eps;
  const float* x; float* x_out;
  const int32_t* sel_idx; const int32_t* sel_count; int sel_cap; int K;
  int gu_depth, dn_depth; // ring stages (host: as many as fit)
  float* dacc;            // [FZ_MAXK][d] stage accumulators, zero on entry and on exit
  unsigned* fin;          // [1] CTAs finished, zero on entry and on exit
  unsigned long long* bar_count;  // [1] barrier arrivals since the layer was created (monotonic)
  int* status;
  // next layer's predictor (has_next == 0: no refinement)
  int has_next;
  const uint16_t* At; const uint16_t* Bt; const float* pc;
  int r, Fn, norm_n; float eps_n; int k_next;
  double* z;              // [FZ_MAXE][r] un-normalised latents
  double* sumsq;          // [FZ_MAXE]
  unsigned* cnt;          // [FZ_MAXE][FZ_CNT_STRIDE], zero on entry and on exit
  unsigned long long* bkey;  // [FZ_MAXE][FZ_NB * FZ_CAPB]
  int32_t* bidx;             // [FZ_MAXE][FZ_NB * FZ_CAPB]
  unsigned long long* okey;  // [FZ_MAXE][Fn] overflow entries
  int32_t* oidx;             // [FZ_MAXE][Fn]
  int32_t* obin;             // [FZ_MAXE][Fn]
  double* range;          // [2] lo, hi used for binning (observed by the previous launch on this layer)
  unsigned long long* range_obs;  // [2] ordered keys: min, max observed in the final evaluation
  int32_t* tmp_idx;       // [max_sel] rank list of the intermediate evaluations (not returned)
  // outputs for the next layer
  int32_t* next_idx; int32_t* next_count; uint32_t* next_mask; double* next_scores; double* next_prio; int next_cap;
  // trace (all nullable)
  float* tr_xtilde; uint32_t* tr_masks; int32_t* tr_counts; uint32_t* tr_survive;
};

#ifdef LS_FZ_TIMING
// Development aid (not compiled into the library): cycle stamps of CTA 0 at points of interest.
__device__ long long g_fz_timing[2][512];
#define FZ_STAMP(role, slot)                                                      \
  do {                                                                            \
    if (blockIdx.x == 0 && (slot) < 512) g_fz_timing[role][slot] = clock64();     \
  } while (0)
#else
#define FZ_STAMP(role, slot) do { } while (0)
#endif

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
// Bounded wait: gives up after a fixed number of SM clocks and records a timeout instead of hanging.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, int* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (clock64() - t0 < FZ_SPIN_CYCLES)
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
__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
  asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

// Barrier among all CTAs of the (cooperatively launched, co-resident) grid: one monotonically increasing 64-bit counter,
// never reset.  Arrival is a release, the poll an acquire, so what a CTA wrote before the barrier is visible to all
// after it.  Every thread of the block calls it.
__device__ __forceinline__ void grid_barrier(const FusedArgs& A, int G) {
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long old;
    asm volatile("atom.add.release.gpu.global.u64 %0, [%1], 1;" : "=l"(old) : "l"(A.bar_count) : "memory");
    const unsigned long long target = (old / (unsigned long long)G + 1ULL) * (unsigned long long)G;
    bool ok = false;
    const long long t0 = clock64();
    do {
      unsigned long long v;
      asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(A.bar_count) : "memory");
      if (v >= target) { ok = true; break; }
    } while (clock64() - t0 < FZ_SPIN_CYCLES);
    if (!ok) set_status(A.status, ST_TIMEOUT);
  }
  __syncthreads();
}

template <int WD>
__device__ __forceinline__ double w16_to_double(uint16_t b) {
  if (WD == WD_BF16) return (double)__uint_as_float((uint32_t)b << 16);
  return (double)__half2float(__ushort_as_half(b));
}

// Stage c of K runs on the CTAs [c*G/K, (c+1)*G/K).
__host__ __device__ inline int fz_group_lo(int c, int G, int K) { return (int)(((long long)c * G) / K); }
__host__ __device__ inline int fz_stage_of_cta(int cta, int G, int K) {
  int c = (int)(((long long)cta * K) / G);
  while (c + 1 < K && fz_group_lo(c + 1, G, K) <= cta) ++c;
  while (c > 0 && fz_group_lo(c, G, K) > cta) --c;
  return c;
}

struct FusedSmemLayout {
  size_t gu_off, dn_off, bar_off, red_off, redd_off, mine_off, a_off, b_off, pc_off, zs_off, own_off, bin_off, coarse_off, total;
  int per, nA, gu_depth, dn_depth;
};

__host__ __device__ inline FusedSmemLayout fused_layout(int d, int n_in, int r, int Fn, int G, int has_next, int gu_depth, int dn_depth) {
  FusedSmemLayout L{};
  L.gu_depth = gu_depth;
  L.dn_depth = dn_depth;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o += (bytes + 127) & ~(size_t)127; return at; };
  L.gu_off = take((size_t)gu_depth * n_in * d * 2);
  L.dn_off = take((size_t)dn_depth * d * 2);
  L.bar_off = take(2 * FZ_MAX_DEPTH * 8);
  L.red_off = take(2 * 8 * 4 * 4);                   // stream dot partials, double-buffered
  L.redd_off = take((size_t)FZ_MAXE * 3 * 16 * 8);   // fp64 partials of the latent phase: [evaluation][row0,row1,sumsq][warp]
  L.mine_off = take((size_t)FZ_MAX_MINE * 8);        // this CTA's neuron indices and gate biases
  L.per = has_next ? (Fn + G - 1) / G : 0;
  L.nA = has_next ? (r + G - 1) / G : 0;
  L.a_off = take((size_t)L.nA * d * 2);
  L.b_off = take((size_t)((L.per + 7) / 8 * 8) * (r + FZ_BPAD) * 2);
  L.pc_off = take((size_t)L.per * 4);
  L.zs_off = take((size_t)(has_next ? 8 * (r + FZ_ZPAD) : 0) * 8);
  L.own_off = take((size_t)FZ_MAXE * L.per * 8);     // this CTA's scores, every evaluation
  L.bin_off = take((size_t)FZ_MAXE * L.per * 2);     // and their fine bins
  L.coarse_off = take(has_next ? (size_t)FZ_MAXE * (FZ_NC + 1) * 4 : 0);
  L.total = o;
  return L;
}

// =====================================================================================================================
template <int WD, int CPT>
__global__ void __launch_bounds__(FZ_THREADS, 1) ls_fused_step_kernel(const __grid_constant__ FusedArgs A) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int G = gridDim.x, cta = blockIdx.x, tid = threadIdx.x;
  const int lane = tid & 31, warp = tid >> 5;
  const int d = A.d, K = A.K, nchunk = A.d >> 3;
  const int n_in = A.gated ? 2 : 1;
  const FusedSmemLayout lay = fused_layout(d, n_in, A.r, A.Fn, G, A.has_next, A.gu_depth, A.dn_depth);
  const int GU = A.gu_depth, DN = A.dn_depth;
  uint16_t* s_gu = reinterpret_cast<uint16_t*>(smem + lay.gu_off);
  uint16_t* s_dn = reinterpret_cast<uint16_t*>(smem + lay.dn_off);
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(smem + lay.bar_off);  // [0..GU) gate/up full, [FZ_MAX_DEPTH..+DN) down full
  float* s_red = reinterpret_cast<float*>(smem + lay.red_off);        // [2][8 warps][4]
  double* s_redd = reinterpret_cast<double*>(smem + lay.redd_off);
  uint16_t* s_A = reinterpret_cast<uint16_t*>(smem + lay.a_off);      // [nA][d]
  uint16_t* s_B = reinterpret_cast<uint16_t*>(smem + lay.b_off);      // [per][r]
  float* s_pc = reinterpret_cast<float*>(smem + lay.pc_off);
  __shared__ int s_last;

  if (tid == 0) {
    for (int i = 0; i < GU; ++i) mbar_init(&s_bar[i], 1);
    for (int i = 0; i < DN; ++i) mbar_init(&s_bar[FZ_MAX_DEPTH + i], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  const int per = lay.per, r = A.r, Fn = A.Fn;
  const int i_lo = cta * per, i_hi = min(Fn, i_lo + per);
  const int n_own = max(0, i_hi - i_lo);
  const bool feat_writer = (cta == 0);

  if (tid < FZ_STREAM_THREADS) {
    // ================================================= stream warps ================================================
    // this CTA serves one stage: the ranks [lo, hi) of the selection, every gsize-th neuron starting at its own offset
    const int count = max(0, min(*A.sel_count, A.sel_cap));
    const int m = count > 0 ? (count + K - 1) / K : 0;
    const int stage = fz_stage_of_cta(cta, G, K);
    const int g_lo = fz_group_lo(stage, G, K), gsize = fz_group_lo(stage + 1, G, K) - g_lo;
    const int lo = min(count, stage * m), hi = min(count, (stage + 1) * m);
    const int first = lo + (cta - g_lo);
    const int n_mine = first < hi ? (hi - first + gsize - 1) / gsize : 0;

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
    const uint32_t gu_bytes = (uint32_t)n_in * d * 2, dn_bytes = (uint32_t)d * 2;
    const size_t bundle_elems = (size_t)A.n_mat * d;

    // this CTA's neurons and their gate biases, fetched once (two dependent reads, all entries in parallel)
    int* s_myidx = reinterpret_cast<int*>(smem + lay.mine_off);
    float* s_mybias = reinterpret_cast<float*>(s_myidx + FZ_MAX_MINE);
    for (int t = tid; t < n_mine; t += FZ_STREAM_THREADS) {
      int i = A.sel_idx[first + t * gsize];
      if ((unsigned)i >= (unsigned)A.F) { set_status(A.status, ST_BAD_INDEX); i = -1; }
      s_myidx[t] = i;
      s_mybias[t] = (A.b_gate && i >= 0) ? A.b_gate[i] : 0.f;
    }
    sq = warp_sum(sq);
    if (lane == 0) s_redd[warp] = sq;
    named_bar_sync(1, FZ_STREAM_THREADS);
    double tot = 0.0;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += s_redd[w];
    const float inv_rms = A.norm == 0 ? (float)(1.0 / sqrt(tot / (double)d + (double)A.eps)) : 1.0f;

    auto issue_gu = [&](int it) {  // thread 0 only
      int i = s_myidx[it];
      if (i < 0) i = 0;  // a rejected index: read row 0, the result is discarded
      uint64_t* bar = &s_bar[it % GU];
      mbar_expect_tx(bar, gu_bytes);
      tma_load_1d(s_gu + (size_t)(it % GU) * n_in * d, A.bundles + (size_t)i * bundle_elems, gu_bytes, bar);
    };
    if (tid == 0)
      for (int it = 0; it < min(n_mine, GU); ++it) issue_gu(it);

    // pending down rows: FIFO over the down ring; every stream thread tracks the same activations in registers
    float qa[4] = {0.f, 0.f, 0.f, 0.f};
    int dq_head = 0, dq_tail = 0;
    float yacc[CPT][8];
#pragma unroll
    for (int q = 0; q < CPT; ++q)
#pragma unroll
      for (int e = 0; e < 8; ++e) yacc[q][e] = 0.f;
    bool dirty = false;
    if (tid == 0) FZ_STAMP(0, 0);

    auto consume_one = [&]() {  // the oldest pending down row, scaled, joins the CTA's partial output
      const int slot = dq_head % DN;
      mbar_wait(&s_bar[FZ_MAX_DEPTH + slot], (uint32_t)((dq_head / DN) & 1), A.status);
      float a = qa[0];
#pragma unroll
      for (int e = 1; e < 4; ++e)
        if (slot == e) a = qa[e];
      const uint16_t* row = s_dn + (size_t)slot * d;
#pragma unroll
      for (int q = 0; q < CPT; ++q) {
        const int ch = tid + q * FZ_STREAM_THREADS;
        if (ch < nchunk) {
          float w[8];
          unpack8<WD>(*reinterpret_cast<const uint4*>(row + ch * 8), w);
#pragma unroll
          for (int e = 0; e < 8; ++e) yacc[q][e] = fmaf(a, w[e], yacc[q][e]);
        }
      }
      dirty = true;
      ++dq_head;
    };

    const int n_rounds = (n_mine + FZ_NG - 1) / FZ_NG;
    for (int rd = 0; rd < n_rounds; ++rd) {
      const int it0 = rd * FZ_NG;
      const int nn = min(FZ_NG, n_mine - it0);
      if (tid == 0) FZ_STAMP(0, 1 + rd * 4);
      // (1) make room in the down ring for this round's survivors (reads of a slot end before the round barrier)
      while (dq_tail - dq_head > DN - FZ_NG) consume_one();
      // (2) partial dot products of the round's neurons
      float pg[FZ_NG], pu[FZ_NG];
#pragma unroll
      for (int e = 0; e < FZ_NG; ++e) {
        pg[e] = 0.f;
        pu[e] = 0.f;
        if (e < nn) {
          const int it = it0 + e, slot = it % GU;
          mbar_wait(&s_bar[slot], (uint32_t)((it / GU) & 1), A.status);
          const uint16_t* grow = s_gu + (size_t)slot * n_in * d;
#pragma unroll
          for (int q = 0; q < CPT; ++q) {
            const int ch = tid + q * FZ_STREAM_THREADS;
            if (ch < nchunk) {
              float w[8];
              unpack8<WD>(*reinterpret_cast<const uint4*>(grow + ch * 8), w);
#pragma unroll
              for (int t = 0; t < 8; ++t) pg[e] = fmaf(w[t], xr[q][t], pg[e]);
              if (A.gated) {
                unpack8<WD>(*reinterpret_cast<const uint4*>(grow + d + ch * 8), w);
#pragma unroll
                for (int t = 0; t < 8; ++t) pu[e] = fmaf(w[t], xr[q][t], pu[e]);
              }
            }
          }
        }
      }
      if (tid == 0) FZ_STAMP(0, 2 + rd * 4);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
        for (int e = 0; e < FZ_NG; ++e) {
          pg[e] += __shfl_xor_sync(0xffffffffu, pg[e], o);
          pu[e] += __shfl_xor_sync(0xffffffffu, pu[e], o);
        }
      }
      float* red = s_red + (rd & 1) * 32;
      if (lane == 0) *reinterpret_cast<float4*>(red + warp * 4) = make_float4(pg[0], pu[0], pg[1], pu[1]);
      named_bar_sync(1, FZ_STREAM_THREADS);  // partials visible; every thread is done with the round's ring slots
      float4 acc4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int w = 0; w < 8; ++w) {
        const float4 v = *reinterpret_cast<const float4*>(red + w * 4);
        acc4.x += v.x; acc4.y += v.y; acc4.z += v.z; acc4.w += v.w;
      }
      if (tid == 0) FZ_STAMP(0, 3 + rd * 4);
      // (3) activations; refill the ring slots; survivors queue their down row
      const float gs[FZ_NG] = {acc4.x, acc4.z}, us[FZ_NG] = {acc4.y, acc4.w};
#pragma unroll
      for (int e = 0; e < FZ_NG; ++e) {
        if (e < nn) {
          const int it = it0 + e;
          const int i = s_myidx[it];
          const float g = gs[e] * inv_rms + s_mybias[it];
          float a = fmaxf(g, 0.f);
          if (A.gated) a *= us[e] * inv_rms;
          if (i < 0) a = 0.f;
          if (tid == 0 && it + GU < n_mine) issue_gu(it + GU);
          if (a != 0.f) {
            const int ds = dq_tail % DN;
#pragma unroll
            for (int t = 0; t < 4; ++t)
              if (ds == t) qa[t] = a;
            if (tid == 0) {
              uint64_t* bar = &s_bar[FZ_MAX_DEPTH + ds];
              mbar_expect_tx(bar, dn_bytes);
              tma_load_1d(s_dn + (size_t)ds * d, A.bundles + (size_t)i * bundle_elems + (size_t)(A.n_mat - 1) * d, dn_bytes, bar);
              if (A.tr_survive) atomicOr(&A.tr_survive[i >> 5], 1u << (i & 31));
            }
            ++dq_tail;
          }
        }
      }
      if (tid == 0) FZ_STAMP(0, 4 + rd * 4);
    }
    if (tid == 0) FZ_STAMP(0, 500);
    while (dq_head < dq_tail) consume_one();
    // the CTA's whole contribution to its stage, added once (vector reductions; order across CTAs is not fixed)
    if (dirty) {
      float* dst = A.dacc + (size_t)stage * d;
#pragma unroll
      for (int q = 0; q < CPT; ++q) {
        const int ch = tid + q * FZ_STREAM_THREADS;
        if (ch < nchunk) {
          red_add_v4(dst + ch * 8, yacc[q][0], yacc[q][1], yacc[q][2], yacc[q][3]);
          red_add_v4(dst + ch * 8 + 4, yacc[q][4], yacc[q][5], yacc[q][6], yacc[q][7]);
        }
      }
    }
    if (tid == 0) FZ_STAMP(0, 501);
  } else if (A.has_next) {
    // ================================================= loader warps ================================================
    // this CTA's rows of A^T and of B^T, and the score biases of its neurons, as stored (128-bit loads)
    const int ltid = tid - FZ_STREAM_THREADS, LT = FZ_THREADS - FZ_STREAM_THREADS;
    for (int a = 0; a < lay.nA; ++a) {
      const int j = cta + a * G;
      if (j < r) {
#pragma unroll 4
        for (int c8 = ltid; c8 < (d >> 3); c8 += LT)
          *reinterpret_cast<uint4*>(s_A + (size_t)a * d + c8 * 8) = ldg128(A.At + (size_t)j * d + c8 * 8);
      }
    }
    for (int li = ltid; li < n_own; li += LT) s_pc[li] = A.pc ? A.pc[i_lo + li] : 0.f;
    const int r8 = r >> 3, nB8 = n_own * r8;  // r is a multiple of 8
    const uint16_t* bsrc = A.Bt + (size_t)i_lo * r;
#pragma unroll 4
    for (int t8 = ltid; t8 < nB8; t8 += LT) {
      const int li = t8 / r8, c8 = t8 - li * r8;
      *reinterpret_cast<uint4*>(s_B + (size_t)li * (r + FZ_BPAD) + c8 * 8) = ldg128(bsrc + (size_t)t8 * 8);
    }
  }

  // ------------------------------------------------------------------------------------------------ barrier 1 of 3
  if (tid == 0) FZ_STAMP(1, 0);
  grid_barrier(A, G);
  if (tid == 0) FZ_STAMP(1, 1);

  // ============================ phase 2: partial features x~^(j) and this CTA's latent rows ===========================
  // Each thread owns d/512 columns.  For every j = 0..K it rebuilds x~^(j) of its columns (x + the stage accumulators
  // below j) and accumulates the dot products with this CTA's rows of A^T; rows are taken two at a time.
  constexpr int XC = 4 * CPT;     // columns per thread (d <= 2048 * CPT)
  float xfin[XC];                 // x~^(K) of this thread's columns (kept by the CTA that writes x_out)
#pragma unroll
  for (int q = 0; q < XC; ++q) xfin[q] = 0.f;
  if (A.has_next || feat_writer) {
    constexpr int JG = 4;         // evaluations accumulated together
    const int npair = A.has_next ? max(1, (lay.nA + 1) / 2) : 1;
    for (int pr = 0; pr < npair; ++pr) {
      const int a0 = pr * 2;
      const bool one = A.has_next && a0 < lay.nA, two = A.has_next && a0 + 1 < lay.nA;
      float xs[XC];  // x~^(j) of this thread's columns, advanced stage by stage
#pragma unroll
      for (int q = 0; q < XC; ++q) {
        const int c = tid + q * FZ_THREADS;
        xs[q] = c < d ? A.x[c] + (A.b_down ? A.b_down[c] : 0.f) : 0.f;
      }
      for (int j0 = 0; j0 <= K; j0 += JG) {
        double p0[JG], p1[JG], sq[JG];
#pragma unroll
        for (int e = 0; e < JG; ++e) { p0[e] = 0.0; p1[e] = 0.0; sq[e] = 0.0; }
        // the stage accumulators this group needs, all fetched before anything is stored
        float dv[XC][JG];
#pragma unroll
        for (int q = 0; q < XC; ++q) {
          const int c = tid + q * FZ_THREADS;
#pragma unroll
          for (int e = 0; e < JG; ++e) dv[q][e] = (c < d && j0 + e < K) ? __ldcg(A.dacc + (size_t)(j0 + e) * d + c) : 0.f;
        }
#pragma unroll
        for (int q = 0; q < XC; ++q) {
          const int c = tid + q * FZ_THREADS;
          if (c < d) {
            const double w0 = one ? w16_to_double<WD>(s_A[(size_t)a0 * d + c]) : 0.0;
            const double w1 = two ? w16_to_double<WD>(s_A[(size_t)(a0 + 1) * d + c]) : 0.0;
            float xv = xs[q];
#pragma unroll
            for (int e = 0; e < JG; ++e) {
              const int j = j0 + e;
              if (j <= K) {
                const double xd = (double)xv;
                p0[e] = fma(w0, xd, p0[e]);
                p1[e] = fma(w1, xd, p1[e]);
                sq[e] = fma(xd, xd, sq[e]);
                if (feat_writer && pr == 0) {
                  if (A.tr_xtilde) A.tr_xtilde[(size_t)j * d + c] = xv;
                  if (j == K) xfin[q] = xv;
                }
                xv += dv[q][e];
              }
            }
            xs[q] = xv;
          }
        }
#pragma unroll
        for (int e = 0; e < JG; ++e) {
          const int j = j0 + e;
          if (j <= K) {
            double a = p0[e], b = p1[e], sv = sq[e];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
              a += __shfl_xor_sync(0xffffffffu, a, o);
              b += __shfl_xor_sync(0xffffffffu, b, o);
              sv += __shfl_xor_sync(0xffffffffu, sv, o);
            }
            if (lane == 0) {
              s_redd[(j * 3 + 0) * 16 + warp] = a;
              s_redd[(j * 3 + 1) * 16 + warp] = b;
              s_redd[(j * 3 + 2) * 16 + warp] = sv;
            }
          }
        }
      }
      __syncthreads();
      if (A.has_next) {
        for (int t = tid; t < (K + 1) * 3; t += FZ_THREADS) {
          const int j = t / 3, e = t - j * 3;
          double v = 0.0;
#pragma unroll
          for (int w = 0; w < 16; ++w) v += s_redd[t * 16 + w];
          if (e < 2) {
            const int row = cta + (a0 + e) * G;
            if (a0 + e < lay.nA && row < r) A.z[(size_t)j * r + row] = v;
          } else if (cta == 0 && pr == 0) {
            A.sumsq[j] = v;
          }
        }
      }
      __syncthreads();
    }
  }

  if (!A.has_next && feat_writer) {
#pragma unroll
    for (int q = 0; q < XC; ++q) {
      const int c = tid + q * FZ_THREADS;
      if (c < d) A.x_out[c] = xfin[q];
    }
  }
  if (A.has_next) {
    // ---------------------------------------------------------------------------------------------- barrier 2 of 3
    if (tid == 0) FZ_STAMP(1, 2);
    grid_barrier(A, G);
    if (tid == 0) FZ_STAMP(1, 3);
    if (feat_writer) {  // x_out may alias x, which every CTA was still reading before this barrier
#pragma unroll
      for (int q = 0; q < XC; ++q) {
        const int c = tid + q * FZ_THREADS;
        if (c < d) A.x_out[c] = xfin[q];
      }
    }

    // ============================ phase 3: scores of this CTA's neurons, every evaluation =============================
    double* s_zs = reinterpret_cast<double*>(smem + lay.zs_off);            // [8][r + FZ_ZPAD], normalised
    double* s_own = reinterpret_cast<double*>(smem + lay.own_off);          // [K+1][per]
    uint16_t* s_bin = reinterpret_cast<uint16_t*>(smem + lay.bin_off);      // [K+1][per]
    unsigned* s_coarse = reinterpret_cast<unsigned*>(smem + lay.coarse_off);  // [K+1][FZ_NC + 1] exclusive prefix
    const double bin_lo = __ldcg(&A.range[0]), bin_hi = __ldcg(&A.range[1]);
    const double INF = __longlong_as_double(0x7ff0000000000000LL);
    const double brange = bin_hi - bin_lo;
    const double bscale = (brange > 0.0 && brange < INF) ? (double)FZ_NB / brange : 0.0;
    const int keff = min(A.k_next, Fn);

    // C[neuron][evaluation] = B^T rows x latents, on the fp64 tensor cores (mma m8n8k4): a warp owns tiles of eight
    // neurons, the evaluations are taken eight at a time.  Every output element is accumulated over the columns in the
    // same order whatever its position in the tile, so equal predictor rows give bit-equal scores.
    const int RSB = r + FZ_BPAD, RSZ = r + FZ_ZPAD;
    const int n_mt = (n_own + 7) >> 3;
    for (int n0 = 0; n0 <= K; n0 += 8) {
      __syncthreads();  // the previous eight latents are no longer read
      for (int t = tid; t < 8 * r; t += FZ_THREADS) {
        const int e = t / r, jj = t - e * r, j = n0 + e;
        double v = 0.0;
        if (j <= K) {
          const double inv = A.norm_n == 0 ? 1.0 / sqrt(__ldcg(&A.sumsq[j]) / (double)d + (double)A.eps_n) : 1.0;
          v = __ldcg(&A.z[(size_t)j * r + jj]) * inv;
        }
        s_zs[e * RSZ + jj] = v;
      }
      __syncthreads();
      for (int mt = warp; mt < n_mt; mt += FZ_THREADS / 32) {
        const uint16_t* arow = s_B + (size_t)(mt * 8 + (lane >> 2)) * RSB + (lane & 3);
        const double* brow = s_zs + (size_t)(lane >> 2) * RSZ + (lane & 3);
        double c0 = 0.0, c1 = 0.0, e0 = 0.0, e1 = 0.0;  // two interleaved accumulator pairs (even / odd column steps)
        for (int k0 = 0; k0 < r; k0 += 8) {
          const double a0v = w16_to_double<WD>(arow[k0]), b0v = brow[k0];
          const double a1v = w16_to_double<WD>(arow[k0 + 4]), b1v = brow[k0 + 4];
          asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};" : "+d"(c0), "+d"(c1) : "d"(a0v), "d"(b0v));
          asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};" : "+d"(e0), "+d"(e1) : "d"(a1v), "d"(b1v));
        }
        const int li = mt * 8 + (lane >> 2);
        const int j = n0 + (lane & 3) * 2;
        if (li < n_own) {
          if (j <= K) s_own[(size_t)j * per + li] = canonical_score((c0 + e0) + (double)s_pc[li]);
          if (j + 1 <= K) s_own[(size_t)(j + 1) * per + li] = canonical_score((c1 + e1) + (double)s_pc[li]);
        }
      }
    }
    __syncthreads();
    // histogram (fine + coarse) and bucket insert: one thread per (evaluation, neuron), all atomics in flight together
    {
      unsigned long long kmin = 0xffffffffffffffffULL, kmax = 0ULL;
      for (int t = tid; t < (K + 1) * n_own; t += FZ_THREADS) {
        const int j = t / n_own, li = t - j * n_own, i = i_lo + li;
        const double sv = s_own[(size_t)j * per + li];
        const double sc = fmin(fmax(sv, -1.7976931348623157e308), 1.7976931348623157e308);
        int bb = (int)((bin_hi - sc) * bscale);
        bb = max(0, min(FZ_NB - 1, bb));
        unsigned* cnt = A.cnt + (size_t)j * FZ_CNT_STRIDE;
        const unsigned slot = atomicAdd(&cnt[bb], 1u);
        atomicAdd(&cnt[FZ_NB + bb / (FZ_NB / FZ_NC)], 1u);
        const unsigned long long key = ordered_key(sv);
        if (slot < (unsigned)FZ_CAPB) {
          A.bkey[((size_t)j * FZ_NB + bb) * FZ_CAPB + slot] = key;
          A.bidx[((size_t)j * FZ_NB + bb) * FZ_CAPB + slot] = i;
        } else {
          const unsigned o = atomicAdd(&cnt[FZ_NB + FZ_NC], 1u);
          A.okey[(size_t)j * Fn + o] = key;
          A.oidx[(size_t)j * Fn + o] = i;
          A.obin[(size_t)j * Fn + o] = bb;
        }
        s_bin[(size_t)j * per + li] = (uint16_t)bb;
        if (j == K) {
          if (A.next_prio) A.next_prio[i] = sv;
          if (A.next_scores) A.next_scores[i] = sv;
          kmin = min(kmin, key);
          kmax = max(kmax, key);
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
        kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
      }
      if (lane == 0 && kmin <= kmax) {  // observed score range of the final evaluation: one pair of atomics per warp
        atomicMin(&A.range_obs[0], kmin);
        atomicMax(&A.range_obs[1], kmax);
      }
    }

    // ---------------------------------------------------------------------------------------------- barrier 3 of 3
    if (tid == 0) FZ_STAMP(1, 4);
    grid_barrier(A, G);
    if (tid == 0) FZ_STAMP(1, 5);

    // ============================ phase 4: exact ranks, every evaluation ============================================
    // coarse exclusive prefix per evaluation: warp w handles evaluations w, w+16, ... (two coarse bins per lane)
    for (int j = warp; j <= K; j += FZ_THREADS / 32) {
      const unsigned* cc = A.cnt + (size_t)j * FZ_CNT_STRIDE + FZ_NB;
      const unsigned c0 = __ldcg(&cc[lane * 2]), c1 = __ldcg(&cc[lane * 2 + 1]);
      unsigned incl = c0 + c1;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      const unsigned ex = incl - (c0 + c1);
      s_coarse[j * (FZ_NC + 1) + lane * 2] = ex;
      s_coarse[j * (FZ_NC + 1) + lane * 2 + 1] = ex + c0;
      if (lane == 31) s_coarse[j * (FZ_NC + 1) + FZ_NC] = incl;
    }
    __syncthreads();
    constexpr int FPC = FZ_NB / FZ_NC;  // fine bins per coarse bin
    for (int t = tid; t < (K + 1) * n_own; t += FZ_THREADS) {
      const int j = t / n_own, li = t - j * n_own, i = i_lo + li;
      const int bb = s_bin[(size_t)j * per + li];
      const int cb = bb / FPC;
      const unsigned cbase = s_coarse[j * (FZ_NC + 1) + cb];
      if ((int)cbase >= keff) continue;  // every neuron of this coarse bin ranks behind the cut
      const unsigned* cnt = A.cnt + (size_t)j * FZ_CNT_STRIDE;
      // fine prefix inside the coarse bin: all its counts are fetched with independent 128-bit loads
      unsigned b0 = cbase, nb = 0;
#pragma unroll
      for (int q = 0; q < FPC; q += 4) {
        const uint4 v = __ldcg(reinterpret_cast<const uint4*>(cnt + cb * FPC + q));
        const unsigned cv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int fb = cb * FPC + q + u;
          b0 += fb < bb ? cv[u] : 0u;
          nb = fb == bb ? cv[u] : nb;
        }
      }
      if ((int)b0 >= keff) continue;
      const unsigned novf = nb > (unsigned)FZ_CAPB ? __ldcg(&cnt[FZ_NB + FZ_NC]) : 0u;
      nb = min(nb, (unsigned)FZ_CAPB);
      const unsigned long long kp = ordered_key(s_own[(size_t)j * per + li]);
      int before = 0;
      const size_t bo = ((size_t)j * FZ_NB + bb) * FZ_CAPB;
      {  // the whole bucket is fetched with independent 128-bit loads; entries beyond nb are ignored
        unsigned long long kq[FZ_CAPB];
        int iq[FZ_CAPB];
#pragma unroll
        for (int q = 0; q < FZ_CAPB; q += 2) {
          const uint4 v = __ldcg(reinterpret_cast<const uint4*>(A.bkey + bo + q));
          kq[q] = ((unsigned long long)v.y << 32) | v.x;
          kq[q + 1] = ((unsigned long long)v.w << 32) | v.z;
        }
#pragma unroll
        for (int q = 0; q < FZ_CAPB; q += 4) {
          const int4 v = __ldcg(reinterpret_cast<const int4*>(A.bidx + bo + q));
          iq[q] = v.x; iq[q + 1] = v.y; iq[q + 2] = v.z; iq[q + 3] = v.w;
        }
#pragma unroll
        for (int q = 0; q < FZ_CAPB; ++q)
          before += ((unsigned)q < nb) && ((kq[q] > kp) || (kq[q] == kp && iq[q] < i));
      }
      for (unsigned q = 0; q < novf; ++q) {  // only when this neuron's own bin overflowed its bucket
        if (__ldcg(&A.obin[(size_t)j * Fn + q]) != bb) continue;
        const unsigned long long kq = __ldcg(&A.okey[(size_t)j * Fn + q]);
        const int iq = __ldcg(&A.oidx[(size_t)j * Fn + q]);
        before += (kq > kp) || (kq == kp && iq < i);
      }
      const int rank = (int)b0 + before;
      if (rank < keff) {
        if (j == K) {
          if (rank < A.next_cap) A.next_idx[rank] = i;
          if (A.next_mask) atomicOr(&A.next_mask[i >> 5], 1u << (i & 31));
        } else {
          A.tmp_idx[rank] = i;
        }
        if (A.tr_masks) atomicOr(&A.tr_masks[(size_t)j * ((Fn + 31) >> 5) + (i >> 5)], 1u << (i & 31));
      }
    }
    if (cta == 0 && tid == 0) {
      if (A.tr_counts)
        for (int j = 0; j <= K; ++j) A.tr_counts[j] = keff;
      *A.next_count = min(keff, A.next_cap);
      if (keff > A.next_cap) set_status(A.status, ST_CAPACITY);
    }
    if (tid == 0) FZ_STAMP(1, 6);
  }

  // ---- the last CTA to finish restores the zero-on-entry invariants of the per-layer scratch
  __syncthreads();
  if (tid == 0) {
    __threadfence();
    s_last = (atomicAdd(A.fin, 1u) == (unsigned)G - 1u) ? 1 : 0;
  }
  __syncthreads();
  if (s_last) {
    __threadfence();
    for (int t = tid; t < K * d; t += FZ_THREADS) A.dacc[t] = 0.f;
    if (A.has_next) {
      for (int t = tid; t < (K + 1) * FZ_CNT_STRIDE; t += FZ_THREADS) A.cnt[t] = 0u;
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
