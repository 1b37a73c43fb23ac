// One kernel per layer step for the all-resident, batch-1 case (the decode hot path).
//
// One CTA per SM, cooperative launch (all CTAs co-resident), two warp-specialised roles per CTA:
//
//   stream role  (warps 0..7)  walks the CTA's share of the selected neurons in execution order, two at a time, without
//                              ever waiting for the predictor: gate+up rows arrive by 1-D TMA bulk copies into a
//                              shared-memory ring, the block reduces the dot products, surviving neurons fetch their
//                              down row into a second ring, and each arrived down row is scaled and added straight
//                              into the accumulator of its stage with vector reductions.
//   signal role  (warp 8)      one thread that publishes "this CTA has finished stage s" (fence + arrive on the stage
//                              counter), so that the stream warps never stall on a memory fence.
//   predict role (warps 9..16) holds its share of the next layer's predictor in shared memory (rows of A^T as stored,
//                              rows of B^T widened once to the high words of their fp64 values) and runs the K+1
//                              refinement evaluations as a three-deep software pipeline  Z_j | S_{j-1} | R_{j-2}
//                              (latent; scores + histogram + bucket insert; exact ranks), separated by barriers among
//                              the predict roles.
//
// The coordination is asymmetric: stream roles only signal (stage counters), predict roles wait (bounded spins).
// Everything a launch dirties in the per-layer scratch is zero again when it ends (the last CTA to finish cleans).
#pragma once
#include "ls_common.cuh"

namespace ls {

constexpr int FZ_STREAM_THREADS = 256;
constexpr int FZ_PRED_THREADS = 256;
constexpr int FZ_SIGNAL_THREADS = 32;
constexpr int FZ_PRED_BASE = FZ_STREAM_THREADS + FZ_SIGNAL_THREADS;
constexpr int FZ_THREADS = FZ_PRED_BASE + FZ_PRED_THREADS;
constexpr int FZ_NG = 2;       // neurons the stream role processes per round
constexpr int FZ_NB = 4096;    // score bins
constexpr int FZ_CNT_STRIDE = FZ_NB + 4;  // bin counts + overflow count, padded so every set stays 16-byte aligned
constexpr int FZ_CAPB = 32;    // bucket capacity per bin; the rest goes to the overflow list
constexpr int FZ_BPAD = 8;     // padding (words) of a predictor row in shared memory: keeps four rows on distinct banks
constexpr int FZ_MAXK = 16;    // stages supported by the fused path
constexpr int FZ_MAX_DEPTH = 8; // most ring stages (gate/up ring, down-row ring); the depths are chosen per launch from the shared memory left
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
  unsigned long long* bar_count;  // [1] barrier arrivals of the predict roles since the layer was created
  int32_t* tmp_idx;       // [max_sel] list of an intermediate evaluation (not returned)
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
// Bounded wait: gives up after a fixed number of polls and records a timeout instead of hanging.
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
  const long long t0 = clock64();
  do {
    if (ld_acquire_u32(ctr) >= target) return true;
  } while (clock64() - t0 < FZ_SPIN_CYCLES);
  set_status(status, ST_TIMEOUT);
  return false;
}

// Barrier among the predict roles of all CTAs: one monotonically increasing 64-bit counter (never reset).
// Arrival is a release, the poll an acquire, so what a CTA wrote before the barrier is visible to all after it.
__device__ __forceinline__ void predict_grid_barrier(const FusedArgs& A, int G, int ptid) {
  named_bar_sync(2, FZ_PRED_THREADS);
  if (ptid == 0) {
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
  size_t gu_off, dn_off, bar_off, red_off, mine_off, a_off, b_off, pc_off, xt_off, zs_off, base_off, own_off, misc_off, total;
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
  L.red_off = take(2 * 8 * 4 * 4 + 64 * 8);      // stream dot partials (double-buffered) + fp64 partials
  L.mine_off = take((size_t)FZ_MAX_MINE * 8);     // this CTA's neuron indices and gate biases
  L.per = has_next ? (Fn + G - 1) / G : 0;
  L.nA = has_next ? (r + G - 1) / G : 0;
  L.a_off = take((size_t)L.nA * d * 2);
  L.b_off = take((size_t)L.per * (r + FZ_BPAD) * 4);
  L.pc_off = take((size_t)L.per * 4);
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
  const FusedSmemLayout lay = fused_layout(d, n_in, A.r, A.Fn, G, A.has_next, A.gu_depth, A.dn_depth);
  const int GU = A.gu_depth, DN = A.dn_depth;
  uint16_t* s_gu = reinterpret_cast<uint16_t*>(smem + lay.gu_off);
  uint16_t* s_dn = reinterpret_cast<uint16_t*>(smem + lay.dn_off);
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(smem + lay.bar_off);  // [0..GU) gate/up full, [FZ_MAX_DEPTH..+DN) down full
  float* s_red = reinterpret_cast<float*>(smem + lay.red_off);        // [2][8 warps][4]
  double* s_redd = reinterpret_cast<double*>(smem + lay.red_off + 2 * 8 * 4 * 4);  // [64]
  __shared__ int s_mailbox;  // stages this CTA has completed (written by stream thread 0, read by the signal thread)
  __shared__ int s_last;

  if (tid == 0) {
    for (int i = 0; i < GU; ++i) mbar_init(&s_bar[i], 1);
    for (int i = 0; i < DN; ++i) mbar_init(&s_bar[FZ_MAX_DEPTH + i], 1);
    s_mailbox = 0;
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
    const uint32_t gu_bytes = (uint32_t)n_in * d * 2, dn_bytes = (uint32_t)d * 2;
    const size_t bundle_elems = (size_t)A.n_mat * d;
    const int n_mine = cta < count ? (count - cta + G - 1) / G : 0;

    // this CTA's neurons and their gate biases, fetched once (two dependent reads, all entries in parallel)
    int* s_myidx = reinterpret_cast<int*>(smem + lay.mine_off);
    float* s_mybias = reinterpret_cast<float*>(s_myidx + FZ_MAX_MINE);
    for (int t = tid; t < n_mine; t += FZ_STREAM_THREADS) {
      int i = A.sel_idx[cta + t * G];
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

    // pending down rows: FIFO over the down ring; every stream thread tracks the same metadata in registers
    float qa[4] = {0.f, 0.f, 0.f, 0.f};
    int qs[4] = {0, 0, 0, 0};
    int dq_head = 0, dq_tail = 0;
    int published = 0;  // stages already handed to the signal thread
    if (tid == 0) FZ_STAMP(0, 0);

    auto consume_one = [&]() {  // the oldest pending down row, scaled, goes straight into its stage accumulator
      const int slot = dq_head % DN;
      mbar_wait(&s_bar[FZ_MAX_DEPTH + slot], (uint32_t)((dq_head / DN) & 1), A.status);
      float a = qa[0];
      int st = qs[0];
#pragma unroll
      for (int e = 1; e < 4; ++e)
        if (slot == e) { a = qa[e]; st = qs[e]; }
      const uint16_t* row = s_dn + (size_t)slot * d;
      float* dst = A.dacc + (size_t)st * d;
#pragma unroll
      for (int q = 0; q < CPT; ++q) {
        const int ch = tid + q * FZ_STREAM_THREADS;
        if (ch < nchunk) {
          float w[8];
          unpack8<WD>(*reinterpret_cast<const uint4*>(row + ch * 8), w);
          red_add_v4(dst + ch * 8, a * w[0], a * w[1], a * w[2], a * w[3]);
          red_add_v4(dst + ch * 8 + 4, a * w[4], a * w[5], a * w[6], a * w[7]);
        }
      }
      ++dq_head;
    };
    // stages that are complete for this CTA: every neuron of the stage has been processed (the first neuron of the
    // coming round lies in a later stage) and no pending down row belongs to it
    auto complete_upto = [&](int next_it) {
      const int front = next_it < n_mine ? min((cta + next_it * G) / m, K - 1) : K;
      int oldest = K;
      if (dq_head < dq_tail) {
        const int slot = dq_head % DN;
        oldest = qs[0];
#pragma unroll
        for (int e = 1; e < 4; ++e)
          if (slot == e) oldest = qs[e];
      }
      return min(front, oldest);
    };

    const int n_rounds = (n_mine + FZ_NG - 1) / FZ_NG;
    for (int rd = 0; rd < n_rounds; ++rd) {
      const int it0 = rd * FZ_NG;
      const int nn = min(FZ_NG, n_mine - it0);
      if (tid == 0) FZ_STAMP(0, 1 + rd * 4);
      // (1) make room in the down ring for this round's survivors; these reds are ordered before the round barrier
      while (dq_tail - dq_head > DN - FZ_NG) consume_one();
      const int done = complete_upto(it0);
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
      // (3) stages whose last reds were issued before the barrier are handed to the signal thread
      if (tid == 0 && done > published) {
        asm volatile("st.release.cta.shared.s32 [%0], %1;" ::"r"(smem_u32(&s_mailbox)), "r"(done) : "memory");
      }
      published = max(published, done);
      // (4) activations; refill the ring slots; survivors queue their down row
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
            const int stage = min((cta + it * G) / m, K - 1);
#pragma unroll
            for (int t = 0; t < 4; ++t)
              if (ds == t) { qa[t] = a; qs[t] = stage; }
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
    named_bar_sync(1, FZ_STREAM_THREADS);
    if (tid == 0) asm volatile("st.release.cta.shared.s32 [%0], %1;" ::"r"(smem_u32(&s_mailbox)), "r"(K) : "memory");
    if (tid == 0) FZ_STAMP(0, 501);
  } else if (tid < FZ_PRED_BASE) {
    // ================================================= signal role =================================================
    if (tid == FZ_STREAM_THREADS) {
      int arrived = 0;
      const long long t0 = clock64();
      while (arrived < K && clock64() - t0 < FZ_SPIN_CYCLES) {
        int v;
        asm volatile("ld.acquire.cta.shared.s32 %0, [%1];" : "=r"(v) : "r"(smem_u32(&s_mailbox)) : "memory");
        if (v > arrived) {
          __threadfence();  // the stream warps' reductions of these stages are ordered before the arrivals
          for (int s = arrived; s < v; ++s) atomicAdd(&A.stage_done[s], 1u);
          arrived = v;
        } else {
          __nanosleep(64);
        }
      }
      if (arrived < K) set_status(A.status, ST_TIMEOUT);
    }
  } else {
    // ================================================= predict role ================================================
    const int ptid = tid - FZ_PRED_BASE, lane = ptid & 31, warp = ptid >> 5;
    float* s_xt = reinterpret_cast<float*>(smem + lay.xt_off);
    uint16_t* s_A = reinterpret_cast<uint16_t*>(smem + lay.a_off);
    uint32_t* s_B = reinterpret_cast<uint32_t*>(smem + lay.b_off);
    float* s_pc = reinterpret_cast<float*>(smem + lay.pc_off);
    double* s_zs = reinterpret_cast<double*>(smem + lay.zs_off);
    unsigned* s_base = reinterpret_cast<unsigned*>(smem + lay.base_off);
    double* s_own = reinterpret_cast<double*>(smem + lay.own_off);          // [2][per]
    int* s_ownbin = reinterpret_cast<int*>(s_own + 2 * lay.per);            // [2][per]
    int* s_misc = reinterpret_cast<int*>(smem + lay.misc_off);
    const int per = lay.per, r = A.r, Fn = A.Fn;
    const int RS = r + FZ_BPAD;  // row stride of s_B in words
    const int i_lo = cta * per, i_hi = min(Fn, i_lo + per);
    const int n_own = max(0, i_hi - i_lo);
    const bool active = A.has_next || cta == 0;  // without a next layer only CTA 0 tracks x~ (to write x_out and the trace)

    // x~^(0) = x (+ b_down)
    if (active)
      for (int c = ptid; c < d; c += FZ_PRED_THREADS) s_xt[c] = A.x[c] + (A.b_down ? A.b_down[c] : 0.f);
    if (A.has_next) {
      // this CTA's rows of A^T (as stored) and of B^T (widened once to fp64 high words), 128-bit loads
      for (int a = 0; a < lay.nA; ++a) {
        const int j = cta + a * G;
        if (j < r) {
#pragma unroll 4
          for (int c8 = ptid; c8 < (d >> 3); c8 += FZ_PRED_THREADS)
            *reinterpret_cast<uint4*>(s_A + (size_t)a * d + c8 * 8) = ldg128(A.At + (size_t)j * d + c8 * 8);
        }
      }
      for (int li = ptid; li < n_own; li += FZ_PRED_THREADS) s_pc[li] = A.pc ? A.pc[i_lo + li] : 0.f;
      const int r8 = r >> 3;  // r is a multiple of 8
      const int nB8 = n_own * r8;
      const uint16_t* bsrc = A.Bt + (size_t)i_lo * r;
#pragma unroll 4
      for (int t8 = ptid; t8 < nB8; t8 += FZ_PRED_THREADS) {
        const int li = t8 / r8, c8 = t8 - li * r8;
        const uint4 v = ldg128(bsrc + (size_t)t8 * 8);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        uint32_t o[8];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          o[2 * e] = w16_to_f64hi<WD>((uint16_t)(w[e] & 0xffffu));
          o[2 * e + 1] = w16_to_f64hi<WD>((uint16_t)(w[e] >> 16));
        }
        uint32_t* dst = s_B + (size_t)li * RS + c8 * 8;
        *reinterpret_cast<uint4*>(dst) = make_uint4(o[0], o[1], o[2], o[3]);
        *reinterpret_cast<uint4*>(dst + 4) = make_uint4(o[4], o[5], o[6], o[7]);
      }
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
    auto w16_to_double = [](uint16_t b) {
      if (WD == WD_BF16) return (double)__uint_as_float((uint32_t)b << 16);
      return (double)__half2float(__ushort_as_half(b));
    };

    if (ptid == 0) FZ_STAMP(1, 0);
    for (int ph = 0; ph < n_phase; ++ph) {
      if (ptid == 0) FZ_STAMP(1, 1 + ph * 8);
      const bool doS = A.has_next && ph >= 1 && ph <= K + 1;  // scores of evaluation ph-1
      const bool doR = A.has_next && ph >= 2;                 // ranks of evaluation ph-2
      const int eS = ph - 1, eR = ph - 2;

      // ---- every global read that only depends on the previous barrier is issued first
      double zreg[4] = {0.0, 0.0, 0.0, 0.0}, ssq = 1.0;
      unsigned c16[16];
      if (doS) {
        ssq = __ldcg(&A.sumsq[eS & 1]);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int j = ptid + q * FZ_PRED_THREADS;
          if (j < r) zreg[q] = __ldcg(&A.z[(size_t)(eS & 1) * r + j]);
        }
      }
      if (doR) {
        const unsigned* cnt = A.cnt + (size_t)(eR % 3) * FZ_CNT_STRIDE;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint4 v = __ldcg(reinterpret_cast<const uint4*>(cnt + ptid * 16 + q * 4));
          c16[q * 4] = v.x; c16[q * 4 + 1] = v.y; c16[q * 4 + 2] = v.z; c16[q * 4 + 3] = v.w;
        }
      }
      const unsigned novf = doR ? __ldcg(&A.cnt[(size_t)(eR % 3) * FZ_CNT_STRIDE + FZ_NB]) : 0u;

      if (ptid == 0) FZ_STAMP(1, 2 + ph * 8);
      // ---- S_{ph-1}, part 1: scores of this CTA's neurons (shared memory only); eight lanes per neuron, so a warp
      //      works on four neurons at once; every neuron is reduced in the same order (equal rows give equal scores)
      if (doS) {
        const double inv = A.norm_n == 0 ? 1.0 / sqrt(ssq / (double)d + (double)A.eps_n) : 1.0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int j = ptid + q * FZ_PRED_THREADS;
          if (j < r) s_zs[j] = zreg[q] * inv;
        }
        named_bar_sync(2, FZ_PRED_THREADS);
        const int l8 = lane & 7, sub = lane >> 3;
        for (int li0 = warp * 4; li0 < n_own; li0 += (FZ_PRED_THREADS / 32) * 4) {
          const int li = li0 + sub;
          const uint32_t* brow = s_B + (size_t)min(li, n_own - 1) * RS;
          double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
          int j = l8;
          for (; j + 24 < r; j += 32) {
            a0 = fma(__hiloint2double((int)brow[j], 0), s_zs[j], a0);
            a1 = fma(__hiloint2double((int)brow[j + 8], 0), s_zs[j + 8], a1);
            a2 = fma(__hiloint2double((int)brow[j + 16], 0), s_zs[j + 16], a2);
            a3 = fma(__hiloint2double((int)brow[j + 24], 0), s_zs[j + 24], a3);
          }
          for (; j < r; j += 8) a0 = fma(__hiloint2double((int)brow[j], 0), s_zs[j], a0);
          double acc = (a0 + a1) + (a2 + a3);
          acc += __shfl_xor_sync(0xffffffffu, acc, 4);
          acc += __shfl_xor_sync(0xffffffffu, acc, 2);
          acc += __shfl_xor_sync(0xffffffffu, acc, 1);
          if (l8 == 0 && li < n_own) s_own[(eS & 1) * per + li] = canonical_score(acc + (double)s_pc[li]);
        }
      }
      if (ptid == 0) FZ_STAMP(1, 3 + ph * 8);
      // ---- R_{ph-2}, part 1: exclusive prefix over the bins (16 bins per thread)
      if (doR) {
        unsigned run = 0;
#pragma unroll
        for (int q = 0; q < 16; ++q) run += c16[q];
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
        if (ptid == FZ_PRED_THREADS - 1) s_base[FZ_NB] = base;
      }
      if (doS || doR) named_bar_sync(2, FZ_PRED_THREADS);

      if (ptid == 0) FZ_STAMP(1, 4 + ph * 8);
      // ---- S part 2: histogram + bucket insert, one thread per neuron so that all atomics are in flight together
      if (doS) {
        const int es = eS % 3, ep = eS & 1;
        unsigned* cnt = A.cnt + (size_t)es * FZ_CNT_STRIDE;
        unsigned long long kmin = 0xffffffffffffffffULL, kmax = 0ULL;
        for (int li = ptid; li < n_own; li += FZ_PRED_THREADS) {
          const int i = i_lo + li;
          const double sv = s_own[ep * per + li];
          const double sc = fmin(fmax(sv, -1.7976931348623157e308), 1.7976931348623157e308);
          int bb = (int)((bin_hi - sc) * bscale);
          bb = max(0, min(FZ_NB - 1, bb));
          const unsigned slot = atomicAdd(&cnt[bb], 1u);
          const unsigned long long key = ordered_key(sv);
          if (slot < (unsigned)FZ_CAPB) {
            A.bkey[((size_t)es * FZ_NB + bb) * FZ_CAPB + slot] = key;
            A.bidx[((size_t)es * FZ_NB + bb) * FZ_CAPB + slot] = i;
          } else {
            const unsigned o = atomicAdd(&cnt[FZ_NB], 1u);
            A.okey[(size_t)es * Fn + o] = key;
            A.oidx[(size_t)es * Fn + o] = i;
            A.obin[(size_t)es * Fn + o] = bb;
          }
          s_ownbin[ep * per + li] = bb;
          if (eS == K) {
            if (A.next_prio) A.next_prio[i] = sv;
            if (A.next_scores) A.next_scores[i] = sv;
            kmin = min(kmin, key);
            kmax = max(kmax, key);
          }
        }
        if (eS == K) {  // observed score range, one pair of atomics per warp
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
            kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
          }
          if (lane == 0 && kmin <= kmax) {
            atomicMin(&A.range_obs[0], kmin);
            atomicMax(&A.range_obs[1], kmax);
          }
        }
      }
      if (ptid == 0) FZ_STAMP(1, 5 + ph * 8);
      // ---- R part 2: exact ranks of this CTA's neurons from the buckets
      if (doR) {
        const int es = eR % 3, ep = eR & 1;
        int32_t* idx_out = (eR == K) ? A.next_idx : A.tmp_idx;
        const int cap = (eR == K) ? A.next_cap : 0x7fffffff;
        uint32_t* mask_out = A.tr_masks ? A.tr_masks + (size_t)eR * ((Fn + 31) >> 5) : nullptr;
        for (int li = ptid; li < n_own; li += FZ_PRED_THREADS) {
          const int bb = s_ownbin[ep * per + li];
          const unsigned b0 = s_base[bb];
          if ((int)b0 >= keff) continue;
          const int i = i_lo + li;
          const unsigned long long kp = ordered_key(s_own[ep * per + li]);
          const unsigned nb = min(s_base[bb + 1] - b0, (unsigned)FZ_CAPB);
          int before = 0;
          const size_t bo = ((size_t)es * FZ_NB + bb) * FZ_CAPB;
          for (int h0 = 0; h0 < FZ_CAPB && (unsigned)h0 < nb; h0 += 16) {
            // sixteen bucket entries per pass, fetched with independent 128-bit loads; entries beyond nb are ignored
            unsigned long long kq[16];
            int iq[16];
#pragma unroll
            for (int q = 0; q < 16; q += 2) {
              const uint4 v = __ldcg(reinterpret_cast<const uint4*>(A.bkey + bo + h0 + q));
              kq[q] = ((unsigned long long)v.y << 32) | v.x;
              kq[q + 1] = ((unsigned long long)v.w << 32) | v.z;
            }
#pragma unroll
            for (int q = 0; q < 16; q += 4) {
              const int4 v = __ldcg(reinterpret_cast<const int4*>(A.bidx + bo + h0 + q));
              iq[q] = v.x; iq[q + 1] = v.y; iq[q + 2] = v.z; iq[q + 3] = v.w;
            }
#pragma unroll
            for (int q = 0; q < 16; ++q)
              before += ((unsigned)(h0 + q) < nb) && ((kq[q] > kp) || (kq[q] == kp && iq[q] < i));
          }
          for (unsigned q = 0; q < novf; ++q) {
            if (__ldcg(&A.obin[(size_t)es * Fn + q]) != bb) continue;
            const unsigned long long kq = __ldcg(&A.okey[(size_t)es * Fn + q]);
            const int iq = __ldcg(&A.oidx[(size_t)es * Fn + q]);
            before += (kq > kp) || (kq == kp && iq < i);
          }
          const int rank = (int)b0 + before;
          if (rank < keff) {
            if (rank < cap) idx_out[rank] = i;
            if (mask_out) atomicOr(&mask_out[i >> 5], 1u << (i & 31));
            if (eR == K && A.next_mask) atomicOr(&A.next_mask[i >> 5], 1u << (i & 31));
          }
        }
        if (cta == 0 && ptid == 0) {
          if (A.tr_counts) A.tr_counts[eR] = keff;
          if (eR == K) {
            *A.next_count = min(keff, A.next_cap);
            if (keff > A.next_cap) set_status(A.status, ST_CAPACITY);
          }
        }
      }

      if (ptid == 0) FZ_STAMP(1, 6 + ph * 8);
      // ---- feature update x~^(ph) = x~^(ph-1) + (stage ph-1 accumulator), then the latent Z_ph
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
      if (ptid == 0) FZ_STAMP(1, 7 + ph * 8);
      if (A.has_next && ph <= K) {
        // Z_ph: this CTA's latent rows (un-normalised, fp64) and, on CTA 0, the sum of squares
        for (int a0 = 0; a0 < lay.nA || a0 == 0; a0 += 2) {
          double p0a = 0.0, p0b = 0.0, p1a = 0.0, p1b = 0.0, sqa = 0.0;
          const bool two = a0 + 1 < lay.nA, one = a0 < lay.nA;
          const uint16_t* r0 = s_A + (size_t)a0 * d;
          const uint16_t* r1 = s_A + (size_t)(a0 + 1) * d;
          for (int c = ptid; c < d; c += 2 * FZ_PRED_THREADS) {
            const int c2 = c + FZ_PRED_THREADS;
            const double x0 = (double)s_xt[c];
            const double x1 = c2 < d ? (double)s_xt[c2] : 0.0;
            if (one) {
              p0a = fma(w16_to_double(r0[c]), x0, p0a);
              if (c2 < d) p0b = fma(w16_to_double(r0[c2]), x1, p0b);
            }
            if (two) {
              p1a = fma(w16_to_double(r1[c]), x0, p1a);
              if (c2 < d) p1b = fma(w16_to_double(r1[c2]), x1, p1b);
            }
            if (a0 == 0) sqa = fma(x0, x0, fma(x1, x1, sqa));
          }
          double part[3] = {p0a + p0b, p1a + p1b, sqa};
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
            for (int e = 0; e < 3; ++e) part[e] += __shfl_xor_sync(0xffffffffu, part[e], o);
          }
          named_bar_sync(2, FZ_PRED_THREADS);  // the previous use of the partial buffer is over
          if (lane == 0) {
#pragma unroll
            for (int e = 0; e < 3; ++e) s_redd[8 + e * 8 + warp] = part[e];
          }
          named_bar_sync(2, FZ_PRED_THREADS);
          if (ptid < 3) {
            double t = 0.0;
            for (int w = 0; w < 8; ++w) t += s_redd[8 + ptid * 8 + w];
            if (ptid < 2) {
              const int j = cta + (a0 + ptid) * G;
              if (a0 + ptid < lay.nA && j < r) A.z[(size_t)(ph & 1) * r + j] = t;
            } else if (cta == 0 && a0 == 0) {
              A.sumsq[ph & 1] = t;
            }
          }
        }
      }

      if (ptid == 0) FZ_STAMP(1, 8 + ph * 8);
      if (A.has_next && ph + 1 < n_phase) {
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
