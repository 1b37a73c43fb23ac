// One kernel per layer step (or per token: all layers of a resident stack) for the all-resident, batch-1 case: the
// decode hot path.  16 compute warps and one producer warp per CTA, one CTA per SM, cooperatively launched.
//
// A layer step has five phases separated by grid barriers (a barrier costs about 2,700 SM clocks here, more than most of
// the phases' arithmetic, so the phases are organised around needing as few as possible):
//
//   1. stream   The K priority stages of the layer (Eq. 1) run CONCURRENTLY on K disjoint groups of CTAs (the output is
//               a sum over hidden neurons, so stage order in time is free; only stage membership defines the partial
//               features).  Every bundle is [gate | up | down] rows of one neuron.  The producer warp brings the GATE
//               rows of the CTA's neurons into a first shared-memory ring by 1-D bulk copies (TMA), all at once when they
//               fit; the compute warps form the pre-activations; only the neurons that survive the ReLU have the rest of
//               their bundle (up and down rows) fetched into a second ring, their activation completed and their down
//               row, scaled, added to the CTA's partial output, which is kept in registers and written once to the
//               CTA's own row of a partial-output array (no floating-point atomics: every sum has a fixed order, the
//               kernel is bitwise repeatable).
//      -- barrier --
//   2. latent   The feature is cut into slices of 32 columns, one per CTA.  The owner rebuilds the K+1 partial residual
//               features x~^(j) = x + sum_{c<j} dm^(c) (Eq. 2) of its columns from the CTAs' partial outputs, writes
//               x_out = x~^(K), and multiplies them with its slice of the next layer's predictor matrix A on the fp64
//               tensor cores: per-slice partial latents.
//      -- barrier --
//   2b. sum     The slices' partials are added (fixed order) into the K+1 latents z^(j) and sums of squares.
//      -- barrier --
//   3. scores   Every CTA scores its share of the next layer's neurons for all K+1 evaluations (fp64 tensor cores; a
//               remainder of one or two evaluations on the ordinary fp64 pipe) and stores scores and their fine bins.
//      -- barrier --
//   4. select   One CTA per evaluation makes the exact top-k from the stored bins (histogram, scan, cut bin, exact
//               comparison inside the cut bin); the final evaluation, which also needs every member's exact rank, is
//               shared by 64 CTAs.  Meanwhile the other CTAs ask the next layer's likely rows into L2.
//
// Instruction fetch matters as much as arithmetic in phases that run once per layer: code that is not resident in the
// 16 KB per-scheduler instruction cache streams at 5 to 9 clocks per instruction, so loops are kept rolled unless the
// unrolling buys memory-level parallelism, and rare paths are out of line.
#pragma once
#include "ls_common.cuh"

namespace ls {

constexpr int FZ_THREADS = 512;        // compute threads (16 warps)
constexpr int FZ_BLOCK = FZ_THREADS + 32;  // plus the producer warp
constexpr int FZ_NG1 = 4;         // most neurons per round of the first ring
constexpr int FZ_NB2 = 8;         // most survivors per batch of the second ring
constexpr int FZ_NB = 4096;       // fine score bins per evaluation
constexpr int FZ_FIN_PARTS = 64;  // CTAs that share the ranking of the final evaluation
constexpr int FZ_CUTLIST = 1024;  // entries of the cut bin ranked in shared memory (a fuller bin falls back to global loops)
constexpr int FZ_CCAP = 4096;     // members grouped in shared memory (more: in the global scratch)
constexpr int FZ_MAXK = 16;       // stages supported by the fused path
constexpr int FZ_MAXE = FZ_MAXK + 1;  // evaluations j = 0..K
constexpr int FZ_MAX_G1 = 16;     // most slots of the first ring (first row of a bundle); depths are chosen per launch
constexpr int FZ_MAX_G2 = 16;     // most slots of the second ring (the rest of a survivor's bundle), carved slots included
constexpr int FZ_SL = 32;         // columns of the feature handled as one slice in the latent phase
constexpr int FZ_EPAD = 18;       // rows kept per evaluation-indexed buffer: at most two MMA tiles, or FZ_MAXE rows
constexpr int FZ_MAX_MINE = 256;  // neurons one CTA may own in one step
#ifdef LS_FZ_TIMING
constexpr long long FZ_SPIN_CYCLES = 40LL * 1000 * 1000;
#else
constexpr long long FZ_SPIN_CYCLES = 4000LL * 1000 * 1000;  // every wait gives up after about two seconds of SM clocks
#endif

// Shared-memory plan of a layer step (computed on the host, carried in the arguments).
struct FusedSmemLayout {
  // fixed regions
  unsigned bar_off, red_off, redd_off, mine_off, pc_off, xt_off, dv_off, a_off;
  // the stream's rings ...
  unsigned r1_off, r2_off;
  // ... and, in the same bytes once the rings have drained, the operands and results of the refinement
  unsigned b_off, zs_off, part_off, own_off, sel_off;
  unsigned total, free_lo;
  int per, ns_cta, a_alias, g1, g2, g2x;  // g2x: extra second-ring slots carved from the first ring once it is idle
};

struct alignas(16) FusedArgs {  // (an array of these is prefetched with 16-byte granularity)
  // layer being executed
  const uint16_t* bundles; int n_mat; int gated; const float* b_gate; const float* b_down;
  int d, F, norm; float eps;
  double inv_d;           // 1 / d
  const float* x; float* x_out;
  const int32_t* sel_idx; const int32_t* sel_count; int sel_cap; int K;
  FusedSmemLayout lay;    // where everything sits in dynamic shared memory
  float* ypart;           // [G][d] every CTA's partial output of its stage (no atomics: summed in a fixed order later)
  unsigned long long* bar_count;  // [1] barrier arrivals since the layer was created (monotonic)
  int* status;
  // next layer's predictor (has_next == 0: no refinement)
  int has_next;
  const uint16_t* At_sl;  // A of the next layer's predictor by column slices: [ceil(d / 32)][r][32], zero padded
  const uint16_t* Bt; const float* pc;
  int r, Fn, norm_n; float eps_n; int k_next;
  double* z;              // [FZ_MAXE][r] un-normalised latents
  double* sumsq;          // [FZ_MAXE]
  double* zpart;          // [slices][K + 1][r + 1] per-slice partial latents; entry r of a row: partial sum of squares
  double* sc;             // [K + 1][Fn] final scores of every evaluation (written by all CTAs, read by the selecting ones)
  uint16_t* sb;           // [K + 1][Fn] their fine bins
  uint4* bent;            // [Fn] members of the final evaluation grouped by bin: {key lo, key hi, neuron, fine bin}
  unsigned long long* kmm;  // [2 G] per CTA: smallest and largest ordered key it saw in the final evaluation
  double* range;          // [2] lo, hi used for binning (observed by the previous launch on this layer)
  // outputs for the next layer
  int32_t* next_idx; int32_t* next_count; uint32_t* next_mask; double* next_scores; double* next_prio; int next_cap;
  // what the layer after this one will read first (whole-token kernel): brought into L2 while this layer refines
  const void* pf_ptr[4]; unsigned pf_bytes[4];
  // big arrays the next layer gathers from: one line per 2 MB page is touched, so that its address translations are warm
  const void* pg_ptr[3]; unsigned long long pg_bytes[3];
  // speculation into L2: the next layer's bundles (first row of a neuron at spec_ptr + i * spec_stride, spec_bytes long)
  const char* spec_ptr; unsigned long long spec_stride; unsigned spec_bytes;
  // (whole-token kernel) the residual feature handed from layer to layer through shared memory: where this layer leaves
  // x_out for the next one, and where it finds its own x (byte offsets into the dynamic shared memory; -1: global memory)
  int xs_put, xs_get;
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
__device__ long long g_fz_cta[160][16];
__device__ int g_fz_fail[64];  // first failures: site, cta, tid, extra
__device__ int g_fz_nfail;
__device__ __forceinline__ void fz_fail(int site, int extra) {
  const int k = atomicAdd(&g_fz_nfail, 1);
  if (k < 16) { g_fz_fail[k * 4] = site; g_fz_fail[k * 4 + 1] = blockIdx.x; g_fz_fail[k * 4 + 2] = threadIdx.x; g_fz_fail[k * 4 + 3] = extra; }
}
#define FZ_FAIL(site, extra) fz_fail(site, extra)  // per-CTA wall-clock stamps (ns) and counters
__device__ __forceinline__ long long fz_now() { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return (long long)t; }
#define FZ_STAMP_DEP(role, slot, fval)                                           \
  do {                                                                            \
    long long c_;                                                                 \
    asm volatile("{ .reg .f32 t_; mov.f32 t_, %1; mov.u64 %0, %%clock64; }" : "=l"(c_) : "f"(fval)); \
    if (blockIdx.x == 0 && (slot) < 512) g_fz_timing[role][slot] = c_;            \
  } while (0)
#define FZ_STAMPB(slot) do { if (blockIdx.x == 1 && threadIdx.x == 0) g_fz_timing[0][(slot)] = clock64(); } while (0)
#define FZ_CSTAMP(slot) do { if (blockIdx.x < 160) g_fz_cta[blockIdx.x][slot] = fz_now(); } while (0)
#define FZ_CVAL(slot, v) do { if (blockIdx.x < 160) g_fz_cta[blockIdx.x][slot] = (v); } while (0)
#else
#define FZ_STAMP(role, slot) do { } while (0)
#define FZ_STAMP_DEP(role, slot, fval) do { } while (0)
#define FZ_FAIL(site, extra) do { } while (0)
#define FZ_STAMPB(slot) do { } while (0)
#define FZ_CSTAMP(slot) do { } while (0)
#define FZ_CVAL(slot, v) do { } while (0)
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
// Bounded wait: gives up after a fixed number of SM clocks and records a timeout instead of hanging.  The first probe is
// inline; the spinning part is a call, so that a wait costs a handful of instructions where it stands.
__device__ __noinline__ bool mbar_wait_slow(uint64_t* bar, uint32_t parity, int* status) {
  const long long t0 = clock64();
  while (clock64() - t0 < FZ_SPIN_CYCLES)
    if (mbar_try_wait(bar, parity)) return true;
  set_status(status, ST_TIMEOUT);
  return false;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, int* status) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, status);
}
// The producer's wait for the compute warps: s_round >= want (bounded like every other wait).
__device__ __noinline__ bool fz_wait_round(int* s_round, int want, int* status) {
  const long long t0 = clock64();
  do {
    int v;
    asm volatile("ld.acquire.cta.shared.s32 %0, [%1];" : "=r"(v) : "r"((uint32_t)__cvta_generic_to_shared(s_round)) : "memory");
    if (v >= want) return true;
    __nanosleep(128);  // the poll shares an instruction scheduler with four compute warps: leave them the issue slots
  } while (clock64() - t0 < FZ_SPIN_CYCLES);
  set_status(status, ST_TIMEOUT);
  return false;
}
// 1 / sqrt(a) in double precision from the hardware approximation and two Newton steps (relative error of a few ulp; a
// full-precision divide and square root would be over a hundred instructions where they stand).
__device__ __forceinline__ double fz_rsqrt(double a) {
  double y;
  asm("rsqrt.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(a));
  if (a > 0.0 && a < 1.0e300) {  // (zero, infinity and NaN keep what the approximation returns)
#pragma unroll
    for (int it = 0; it < 2; ++it) {
      const double h = 0.5 * a * y;
      y = fma(y, fma(-h, y, 0.5), y);
    }
  }
  return y;
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

// Barrier among all CTAs of the (cooperatively launched, co-resident) grid: one monotonically increasing 64-bit counter,
// never reset.  Arrival is a release, the poll an acquire, so what a CTA wrote before the barrier is visible to all
// after it.  Every compute thread of the block calls it (block barrier 1 spans the 512 compute threads; the producer
// warp has left by then).
__device__ __noinline__ void grid_barrier_thread0(const FusedArgs& A, int G) {
  {
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
    if (!ok) { set_status(A.status, ST_TIMEOUT); FZ_FAIL(6, (int)target); }
  }
}
__device__ __forceinline__ void grid_barrier(const FusedArgs& A, int G) {
  named_bar_sync(1, FZ_THREADS);
  if (threadIdx.x == 0) grid_barrier_thread0(A, G);
  named_bar_sync(1, FZ_THREADS);
}

template <int WD>
__device__ __forceinline__ double w16_to_double(uint16_t b) {
  if (WD == WD_BF16) return (double)__uint_as_float((uint32_t)b << 16);
  return (double)__half2float(__ushort_as_half(b));
}

// ---- fp64 tensor-core blocks ------------------------------------------------------------------------------------------
// Both predictor products (A^T x~ and B^T z) are cut into blocks of 32 columns, and the order of the columns INSIDE a
// block is permuted (the sum over a block does not depend on it): lane (g, t) of a warp, g = lane / 4, t = lane % 4,
// takes the eight consecutive columns 8t .. 8t+7, so that its eight weights are ONE 16-byte load, and the k-th MMA of the
// block pairs column 8t + k of the weights with the same column of the features.  Features are stored for that access:
// column c of a block sits at (c / 8) * 10 + c % 8 doubles (eight doubles, two of padding), which makes the 16-byte
// feature loads of a quarter-warp fall on distinct banks when the row stride is 16 words modulo 32.
constexpr int FZ_XBLK = 40;  // doubles a 32-column block of features occupies in shared memory
__host__ __device__ inline int fz_feat_pos(int c) { return (c >> 5) * FZ_XBLK + ((c >> 3) & 3) * 10 + (c & 7); }
// Row stride (doubles) of a feature array with `cols` columns: whole blocks, 16 words modulo 32.
__host__ __device__ inline int fz_feat_stride(int cols) {
  const int nb = (cols + 31) >> 5;
  return nb * FZ_XBLK + ((nb & 1) ? 0 : 8);
}
// Row stride (16-bit elements) of the B^T rows in shared memory: whole blocks, 64 bytes modulo 128.
__host__ __device__ inline int fz_brow_stride(int r) {
  const int c = ((r + 31) >> 5) << 5;
  return c + ((c & 63) == 32 ? 0 : 32);
}

template <int WD>
__device__ __forceinline__ void cvt8_to_double(const uint4 w, double a[8]) {
  const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    a[2 * q] = w16_to_double<WD>((uint16_t)(ww[q] & 0xffffu));
    a[2 * q + 1] = w16_to_double<WD>((uint16_t)(ww[q] >> 16));
  }
}
__device__ __forceinline__ void load8d(const double* p, double v[8]) {  // 16-byte aligned
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const double2 t = *reinterpret_cast<const double2*>(p + 2 * q);
    v[2 * q] = t.x;
    v[2 * q + 1] = t.y;
  }
}
// c (8 rows x 8 features, this lane's two elements) += one block: weights a[8] of this lane's row, features b[8]
__device__ __forceinline__ void mma_block(double (&c)[2], const double a[8], const double b[8]) {
#pragma unroll
  for (int k = 0; k < 8; ++k)
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                 : "+d"(c[0]), "+d"(c[1]) : "d"(a[k]), "d"(b[k]));
}
// sum over the four lanes of a row (fixed order)
__device__ __forceinline__ double quad_sum(double v) {
  v += __shfl_xor_sync(0xffffffffu, v, 1);
  v += __shfl_xor_sync(0xffffffffu, v, 2);
  return v;
}

// Shared-memory work area of the selection (see fz_select).
__host__ __device__ inline size_t fz_select_bytes(int Fn) {
  return (size_t)2 * FZ_NB * 4 + 128 + (size_t)((Fn + 7) & ~7) * 2 + (size_t)FZ_CUTLIST * 12 + (size_t)FZ_CCAP * 16;
}

// Bar indices: [0, FZ_MAX_G1) first-ring slots, [FZ_MAX_G1, +FZ_MAX_G2) second-ring slots, then the A slices, then B^T rows.
constexpr int FZ_BAR_R2 = FZ_MAX_G1, FZ_BAR_A = FZ_MAX_G1 + FZ_MAX_G2, FZ_BAR_B = FZ_BAR_A + 1, FZ_NBAR = FZ_BAR_B + 1;

// `a_alias` != 0 places the A slices inside the ring bytes too (they are then fetched only after the rings have drained).
inline FusedSmemLayout fused_layout(int d, int n_mat, int r, int Fn, int G, int has_next, int g1, int g2,
                                                        int a_alias) {
  FusedSmemLayout L{};
  L.g1 = g1;
  L.g2 = g2;
  {
    const long long extra = ((long long)g1 * d * 2) / ((long long)(n_mat - 1) * d * 2);
    L.g2x = (int)(extra < FZ_MAX_G2 - g2 ? extra : FZ_MAX_G2 - g2);
  }
  L.a_alias = a_alias;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o += (bytes + 127) & ~(size_t)127; return (unsigned)at; };
  const int nsl = (d + FZ_SL - 1) / FZ_SL;
  L.per = has_next ? (Fn + G - 1) / G : 0;
  L.ns_cta = (nsl + G - 1) / G;
  const size_t a_bytes = has_next ? (size_t)L.ns_cta * r * FZ_SL * 2 : 0;
  L.bar_off = take(FZ_NBAR * 8);
  L.red_off = take(2 * 16 * FZ_NG1 * 4 + 16 * FZ_NB2 * 4);  // stream dot partials: first ring [2][warp][FZ_NG1] (double-buffered), second ring [warp][FZ_NB2]
  L.redd_off = take(32 * 8);                         // fp64 partials of block reductions
  L.mine_off = take((size_t)FZ_MAX_MINE * 16);       // this CTA's neurons, their gate biases; the survivors, their activations
  L.pc_off = take((size_t)L.per * 4);
  L.xt_off = take((size_t)FZ_EPAD * FZ_XBLK * 8);  // x~^(j) of one slice, fp64, one padded block per row
  L.dv_off = take((size_t)(FZ_MAXK + FZ_THREADS / 32) * FZ_SL * 4);  // stage sums of one slice, and their partial sums
  if (!a_alias) L.a_off = take(a_bytes);
  const size_t base = o;
  L.r1_off = take((size_t)g1 * d * 2);
  L.r2_off = take((size_t)g2 * (n_mat - 1) * d * 2);
  const size_t end_stream = o;
  o = base;
  if (a_alias) L.a_off = take(a_bytes);
  const int per8 = (L.per + 7) / 8 * 8;
  L.b_off = take((size_t)per8 * fz_brow_stride(r) * 2);
  L.zs_off = take(has_next ? (size_t)FZ_EPAD * fz_feat_stride(r) * 8 : 0);
  {
    // partial sums of the score tiles: [slot][evaluation][neuron]; a tile's blocks are spread over at most `slots` warps
    const int n_mt = per8 / 8, nblk = (r + 31) / 32, nun = n_mt * nblk;
    const int U = nun > 0 ? (nun + 15) / 16 : 1;
    const int slots = (nblk + U - 1) / U + 1;
    L.part_off = take(has_next ? (size_t)slots * FZ_EPAD * per8 * 8 : 0);
  }
  L.own_off = take((size_t)L.per * 8);               // this CTA's scores of the final evaluation
  const size_t end_refine = o;
  o = base;  // the selection works when the score operands are dead: it shares their bytes
  L.sel_off = take(has_next ? fz_select_bytes(Fn) : 0);
  const size_t end_select = o;
  o = end_refine > end_select ? end_refine : end_select;
  L.free_lo = (unsigned)o;  // no phase after the stream uses shared memory from here on
  L.total = (unsigned)(o > end_stream ? o : end_stream);
  return L;
}

// =====================================================================================================================
// Block-shared state of a layer step (static shared memory of the kernels below).
struct FusedShared {
  FusedArgs args[2];                 // (whole-token kernel) this layer's arguments and, fetched meanwhile, the next layer's
  int round;                         // rounds the compute warps have finished (read by the producer)
  int stage, g_lo, gsize;            // this CTA's stage, the first CTA of the stage's group and the group's size
  unsigned phase[FZ_NBAR];           // phases every mbarrier has completed in earlier layers of the launch
  int nsurv, done;                   // survivors found so far / consumed so far (read by the producer)
  int b_hi, b_last;                  // the second ring's current batch ends before survivor b_hi; it is the last one
  double inv[FZ_EPAD + 32];          // 1 / rms per evaluation; behind them: partial-sum slots per score tile (ints)
  unsigned long long kmm[2 * 16];
};

// Inverse of ordered_key.
__device__ __forceinline__ double fz_unkey(unsigned long long k) {
  const unsigned long long b = (k >> 63) ? (k & 0x7fffffffffffffffULL) : ~k;
  return __longlong_as_double((long long)b);
}

// ---- exact top-k of one evaluation by one CTA ------------------------------------------------------------------------
// Inputs (global, written by all CTAs before the preceding grid barrier): sc[j][Fn] scores, sb[j][Fn] their fine bins
// (FZ_NB bins, descending score).  Shared-memory work area `wk` (see fz_select_bytes): the bins of all neurons, FZ_NB
// counters (then their exclusive prefix), FZ_NB fill counters, the entries of the cut bin, and the members grouped by
// bin.  Output: membership (trace mask) for j < K; for j == K the ranked index list, mask, count, and the observed score
// range for the layer's next launch.  Every evaluation checks that its set has exactly keff members.
// The final evaluation is shared by `nparts` CTAs: each builds the whole histogram (cheap), then ranks only the members
// of the bins whose first rank falls in its share of the ranks; nothing is exchanged between them.
template <int WD>
__device__ __noinline__ void fz_select(const FusedArgs& A, int j, int K, int keff, unsigned wk_off, int part, int nparts, bool fold) {
  // (the work area is addressed through the kernel's dynamic shared array, so that the compiler emits shared-memory
  // loads, stores and atomics: through a plain pointer argument they would be generic ones, several times slower)
  extern __shared__ __align__(128) unsigned char fz_dyn_smem[];
  unsigned char* const wk = fz_dyn_smem + wk_off;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int Fn = A.Fn, G = gridDim.x;
  uint4* s_cand = reinterpret_cast<uint4*>(wk);                               // [FZ_CCAP] {key lo, key hi, neuron, bin}
  unsigned long long* s_lkey = reinterpret_cast<unsigned long long*>(s_cand + FZ_CCAP);  // [FZ_CUTLIST]
  unsigned* s_cnt = reinterpret_cast<unsigned*>(s_lkey + FZ_CUTLIST);        // [FZ_NB] counts, then exclusive prefix
  unsigned* s_fill = s_cnt + FZ_NB;                                           // [FZ_NB]
  unsigned* s_wsum = s_fill + FZ_NB;                                          // [32] warp totals of the scan; [16..19] the cut; [20..] key ranges
  int* s_cutv = reinterpret_cast<int*>(s_wsum + 16);                          // cut fine bin, its first rank, its size; members counted
  int* s_list = reinterpret_cast<int*>(s_wsum + 32);                          // [FZ_CUTLIST] neurons of the cut bin
  uint16_t* s_ball = reinterpret_cast<uint16_t*>(s_list + FZ_CUTLIST);        // [Fn8] the bin of every neuron
  const double* sc = A.sc + (size_t)j * Fn;
  const uint16_t* sb = A.sb + (size_t)j * Fn;
  const bool fin = (j == K);
#pragma unroll 1
  for (int t = tid; t < 2 * FZ_NB / 4; t += FZ_THREADS) reinterpret_cast<uint4*>(s_cnt)[t] = make_uint4(0u, 0u, 0u, 0u);
  // (the CTA that folds the per-CTA score ranges: an early finisher, not one of the final evaluation's) they are fetched
  // now and folded at the end
  unsigned long long kmin = 0xffffffffffffffffULL, kmax = 0ULL;
  if (fold) {
#pragma unroll 1
    for (int c = tid; c < G; c += FZ_THREADS) { kmin = min(kmin, __ldcg(&A.kmm[2 * c])); kmax = max(kmax, __ldcg(&A.kmm[2 * c + 1])); }
  }
  if (tid == 0) { s_cutv[0] = -1; s_cutv[1] = 0; s_cutv[2] = 0; s_cutv[3] = 0; }
  named_bar_sync(1, FZ_THREADS);
  if (tid == 0) FZ_STAMP(1, 61);
  if (tid == 0) FZ_CSTAMP(12);
  FZ_STAMPB(300);
  // pass 1: the bins come to shared memory (eight neurons per 16-byte load when the row is aligned) and are counted
  if ((((size_t)j * Fn) & 7) == 0) {
    const uint4* sb8 = reinterpret_cast<const uint4*>(sb);
    const int n8 = Fn >> 3;
#pragma unroll 1
    for (int t0 = 0; t0 < n8; t0 += 4 * FZ_THREADS) {
      uint4 q[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int t = t0 + u * FZ_THREADS + tid;
        q[u] = t < n8 ? __ldcg(sb8 + t) : make_uint4(0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int t = t0 + u * FZ_THREADS + tid;
        if (t < n8) {
          reinterpret_cast<uint4*>(s_ball)[t] = q[u];
          const uint32_t w[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            atomicAdd(&s_cnt[w[e] & 0xffffu], 1u);
            atomicAdd(&s_cnt[w[e] >> 16], 1u);
          }
        }
      }
    }
#pragma unroll 1
    for (int t = (n8 << 3) + tid; t < Fn; t += FZ_THREADS) { const unsigned b = __ldcg(sb + t); s_ball[t] = (uint16_t)b; atomicAdd(&s_cnt[b], 1u); }
  } else {
#pragma unroll 1
    for (int t = tid; t < Fn; t += FZ_THREADS) { const unsigned b = __ldcg(sb + t); s_ball[t] = (uint16_t)b; atomicAdd(&s_cnt[b], 1u); }
  }
  named_bar_sync(1, FZ_THREADS);
  if (tid == 0) FZ_STAMP(1, 62);
  FZ_STAMPB(301);
  // exclusive scan of the FZ_NB counts (eight per thread), and the cut bin
  {
    constexpr int PT = FZ_NB / FZ_THREADS;
    static_assert(PT == 8, "a thread owns eight consecutive counters: two 16-byte accesses");
    unsigned c[PT], tot = 0;
    {  // (16-byte accesses: word accesses at a stride of eight would be eight-way bank conflicts)
      const uint4 c0 = reinterpret_cast<const uint4*>(s_cnt)[tid * 2], c1 = reinterpret_cast<const uint4*>(s_cnt)[tid * 2 + 1];
      c[0] = c0.x; c[1] = c0.y; c[2] = c0.z; c[3] = c0.w; c[4] = c1.x; c[5] = c1.y; c[6] = c1.z; c[7] = c1.w;
#pragma unroll
      for (int q = 0; q < PT; ++q) tot += c[q];
    }
    unsigned incl = tot;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) s_wsum[warp] = incl;
    named_bar_sync(1, FZ_THREADS);
    unsigned base = 0;
#pragma unroll 4
    for (int w = 0; w < FZ_THREADS / 32; ++w) base += w < warp ? s_wsum[w] : 0u;
    unsigned ex = base + incl - tot, pre[PT];
#pragma unroll
    for (int q = 0; q < PT; ++q) {
      pre[q] = ex;
      if (c[q] > 0 && (int)ex < keff && (int)(ex + c[q]) >= keff) { s_cutv[0] = tid * PT + q; s_cutv[1] = (int)ex; s_cutv[2] = (int)c[q]; }
      ex += c[q];
    }
    reinterpret_cast<uint4*>(s_cnt)[tid * 2] = make_uint4(pre[0], pre[1], pre[2], pre[3]);
    reinterpret_cast<uint4*>(s_cnt)[tid * 2 + 1] = make_uint4(pre[4], pre[5], pre[6], pre[7]);
  }
  named_bar_sync(1, FZ_THREADS);
  if (tid == 0) FZ_STAMP(1, 63);
  if (tid == 0) FZ_CSTAMP(13);
  FZ_STAMPB(302);
  const int cut_bin = s_cutv[0], cut_b0 = s_cutv[1], cut_nb = s_cutv[2];  // no cut bin (-1): keff == 0, nothing is selected
  const int need = keff - cut_b0;                                         // members inside the cut bin
  uint32_t* const trm = A.tr_masks ? A.tr_masks + (size_t)j * ((Fn + 31) >> 5) : nullptr;
  if (!fin) {
    // Intermediate evaluation: its refined set is now fixed by the cut (bins before the cut bin are in, the cut bin is
    // split by exact comparison: entry e is a member iff fewer than `need` entries of the bin precede it).  Nothing
    // consumes the set itself when every bundle is resident, so it is written out only when a trace asks for it.
    if (cut_bin >= 0 && trm) {
#pragma unroll 1
      for (int t = tid; t < Fn; t += FZ_THREADS) {
        const int b = s_ball[t];
        if (b < cut_bin) {
          if (trm) atomicOr(&trm[t >> 5], 1u << (t & 31));
        } else if (b == cut_bin) {
          const unsigned p = atomicAdd(&s_fill[b], 1u);
          if (p < (unsigned)FZ_CUTLIST) s_list[p] = t;
        }
      }
      named_bar_sync(1, FZ_THREADS);
      if (tid == 0) FZ_STAMP(1, 64);
      if (cut_nb <= FZ_CUTLIST) {
#pragma unroll 1
        for (int e = tid; e < cut_nb; e += FZ_THREADS) s_lkey[e] = ordered_key(__ldcg(sc + s_list[e]));
        named_bar_sync(1, FZ_THREADS);
#pragma unroll 1
        for (int e = tid; e < cut_nb; e += FZ_THREADS) {
          const int i = s_list[e];
          const unsigned long long kp = s_lkey[e];
          int before = 0;
#pragma unroll 1
          for (int q = 0; q < cut_nb; ++q) before += (s_lkey[q] > kp) || (s_lkey[q] == kp && s_list[q] < i);
          if (before < need) {
            atomicAdd(&s_cutv[3], 1);
            if (trm) atomicOr(&trm[i >> 5], 1u << (i & 31));
          }
        }
      } else {  // an overfull cut bin (degenerate score distributions): every neuron of the bin scans the whole row
#pragma unroll 1
        for (int i = tid; i < Fn; i += FZ_THREADS) {
          if ((int)s_ball[i] != cut_bin) continue;
          const unsigned long long kp = ordered_key(__ldcg(sc + i));
          int before = 0;
#pragma unroll 1
          for (int iq = 0; iq < Fn; ++iq) {
            if ((int)s_ball[iq] != cut_bin) continue;
            const unsigned long long kq = ordered_key(__ldcg(sc + iq));
            before += (kq > kp) || (kq == kp && iq < i);
          }
          if (before < need) {
            atomicAdd(&s_cutv[3], 1);
            if (trm) atomicOr(&trm[i >> 5], 1u << (i & 31));
          }
        }
      }
      named_bar_sync(1, FZ_THREADS);
      if (tid == 0 && cut_b0 + s_cutv[3] != keff) set_status(A.status, ST_INTERNAL);  // self-check of the set's size
    }
    if (!fold) return;
  } else {
  // final evaluation: the members of this CTA's share of the bins are scattered into `cand`, grouped by bin (position =
  // first rank of the bin + arrival order); a member's exact rank = first rank of its bin + entries of the bin before it
  const int ncand = cut_bin >= 0 ? cut_b0 + cut_nb : 0;
  const unsigned lo_r = (unsigned)(((long long)part * ncand) / nparts), hi_r = (unsigned)(((long long)(part + 1) * ncand) / nparts);
  uint4* const cand = ncand <= FZ_CCAP ? s_cand : A.bent;
  if (tid == 0) { s_cutv[4] = 0x7fffffff; s_cutv[5] = 0; }
  named_bar_sync(1, FZ_THREADS);
  if (cut_bin >= 0) {
    // (a) neuron and bin of every member, shared memory only
    unsigned pmin = 0x7fffffffu, pmax = 0u;
#pragma unroll 1
    for (int t0 = tid; t0 < Fn; t0 += 8 * FZ_THREADS) {
      int bb[8];
      unsigned pre[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {  // all the loads first: behind a store or an atomic they could not be moved up
        const int t = t0 + u * FZ_THREADS;
        bb[u] = t < Fn ? (int)s_ball[t] : FZ_NB;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) pre[u] = bb[u] <= cut_bin ? s_cnt[bb[u]] : 0xffffffffu;
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        if (pre[u] >= lo_r && pre[u] < hi_r) {
          const unsigned pos = pre[u] + atomicAdd(&s_fill[bb[u]], 1u);
          cand[pos] = make_uint4(0u, 0u, (unsigned)(t0 + u * FZ_THREADS), (unsigned)bb[u]);
          pmin = min(pmin, pos);
          pmax = max(pmax, pos + 1u);
        }
      }
    }
    pmin = __reduce_min_sync(0xffffffffu, pmin);
    pmax = __reduce_max_sync(0xffffffffu, pmax);
    if (lane == 0 && pmax > 0u) { atomicMin(&s_cutv[4], (int)pmin); atomicMax(&s_cutv[5], (int)pmax); }
  }
  named_bar_sync(1, FZ_THREADS);
  if (tid == 0) FZ_CSTAMP(14);
  FZ_STAMPB(303);
  const int pstart = min(s_cutv[4], s_cutv[5]), pend = s_cutv[5];  // this CTA's positions [pstart, pend)
  // (b) their keys: four score loads in flight per thread
#pragma unroll 1
  for (int p0 = pstart; p0 < pend; p0 += 4 * FZ_THREADS) {
    double v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int p = p0 + u * FZ_THREADS + tid;
      v[u] = p < pend ? __ldcg(sc + cand[p].z) : 0.0;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int p = p0 + u * FZ_THREADS + tid;
      if (p < pend) {
        const unsigned long long key = ordered_key(v[u]);
        cand[p].x = (unsigned)key;
        cand[p].y = (unsigned)(key >> 32);
      }
    }
  }
  named_bar_sync(1, FZ_THREADS);  // (also makes this CTA's writes to the global scratch visible to all its threads)
  if (tid == 0) FZ_CSTAMP(15);
  FZ_STAMPB(304);
  {
    int32_t* const nidx = A.next_idx;
    uint32_t* const nmask = A.next_mask;
    const int ncap = A.next_cap;
    int found = 0;
#pragma unroll 1
    for (int p = pstart + tid; p < pend; p += FZ_THREADS) {
      const uint4 me = cand[p];
      const int b = (int)me.w, i = (int)me.z;
      const unsigned long long kp = ((unsigned long long)me.y << 32) | me.x;
      const int b0 = (int)s_cnt[b], nb = (int)s_fill[b];
      int before = 0;
#pragma unroll 1
      for (int q = b0; nb > 1 && q < b0 + nb; ++q) {  // (a member alone in its bin has the bin's first rank)
        const uint4 o = cand[q];
        const unsigned long long kq = ((unsigned long long)o.y << 32) | o.x;
        before += (kq > kp) || (kq == kp && (int)o.z < i);
      }
      const int rank = b0 + before;
      if (rank < keff) {
        ++found;
        if (rank < ncap) nidx[rank] = i;
        if (nmask) atomicOr(&nmask[i >> 5], 1u << (i & 31));
        if (trm) atomicOr(&trm[i >> 5], 1u << (i & 31));
      }
    }
    FZ_STAMPB(305);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) found += __shfl_xor_sync(0xffffffffu, found, o);
    if (lane == 0 && found) atomicAdd(&s_cutv[3], found);
    FZ_STAMPB(306);
  }
  named_bar_sync(1, FZ_THREADS);
  if (tid == 0 && s_cutv[3] != max(0, min(keff, pend) - pstart)) set_status(A.status, ST_INTERNAL);  // self-check: one member per rank
  if (!fold) return;
  }
  named_bar_sync(1, FZ_THREADS);  // (the cut list's bytes are reused below)
  // the layer's binning range for its next launch: what all CTAs observed in this evaluation, widened by 5 % per side
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
    kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
  }
  unsigned long long* s_kmm2 = reinterpret_cast<unsigned long long*>(s_lkey);  // (the cut list is dead by now)
  if (lane == 0) { s_kmm2[warp] = kmin; s_kmm2[16 + warp] = kmax; }
  named_bar_sync(1, FZ_THREADS);
  if (tid == 0) {
#pragma unroll 1
    for (int w = 1; w < 16; ++w) { kmin = min(kmin, s_kmm2[w]); kmax = max(kmax, s_kmm2[16 + w]); }
    if (kmin <= kmax) {
      double lo = fmax(fz_unkey(kmin), -1.0e300), hi = fmin(fz_unkey(kmax), 1.0e300);
      const double pad = 0.05 * (hi - lo);
      A.range[0] = lo - pad;
      A.range[1] = hi + pad;
    }
    FZ_STAMPB(307);
    if (A.tr_counts)
#pragma unroll 1
      for (int jj = 0; jj <= K; ++jj) A.tr_counts[jj] = keff;
    *A.next_count = min(keff, A.next_cap);
    if (keff > A.next_cap) set_status(A.status, ST_CAPACITY);
  }
}

// The producer's copy of this CTA's column slices of the next layer's A (one mbarrier for all of them).
__device__ __noinline__ void fz_issue_a(const FusedArgs& A, uint16_t* s_A, uint64_t* abar, int cta, int G, int nsl) {
  const uint32_t sl_bytes = (uint32_t)A.r * FZ_SL * 2;
  int nmy = 0;
#pragma unroll 1
  for (int sl = cta; sl < nsl; sl += G) ++nmy;
  mbar_expect_tx(abar, (uint32_t)nmy * sl_bytes);
  int a = 0;
#pragma unroll 1
  for (int sl = cta; sl < nsl; sl += G, ++a)
    tma_load_1d(s_A + (size_t)a * A.r * FZ_SL, A.At_sl + (size_t)sl * A.r * FZ_SL, sl_bytes, abar);
}

// One layer step, executed by the whole block (16 compute warps + the producer warp).  The producer warp returns as
// soon as it has issued its last copy; the compute warps return when the layer's refined sets are written.
// `first_layer` says that this is the first layer of the launch (the mbarriers in shared memory are set up then);
// `known_count` >= 0 is the size of the selection when the caller knows it without reading it.
template <int WD, int CPT>
__device__ __forceinline__ void fused_layer(const FusedArgs& A, unsigned char* smem, FusedShared& sh, bool first_layer,
                                            int known_count) {
  const int G = gridDim.x, cta = blockIdx.x, tid = threadIdx.x;
  const int lane = tid & 31, warp = tid >> 5;
  const int d = A.d, K = A.K, nchunk = A.d >> 3;
  const FusedSmemLayout& lay = A.lay;
  const int G1 = lay.g1, G2 = lay.g2, G2T = lay.g2 + lay.g2x, NG1 = min(FZ_NG1, lay.g1);
  uint16_t* s_r1 = reinterpret_cast<uint16_t*>(smem + lay.r1_off);  // [G1][d]
  uint16_t* s_r2 = reinterpret_cast<uint16_t*>(smem + lay.r2_off);  // [G2][(n_mat - 1) d]
  uint64_t* s_bar = reinterpret_cast<uint64_t*>(smem + lay.bar_off);  // "full" barriers: gate/up slots, down slots, A, B^T
  float* s_red = reinterpret_cast<float*>(smem + lay.red_off);        // [2][16 warps][8]
  double* s_redd = reinterpret_cast<double*>(smem + lay.redd_off);
  uint16_t* s_A = reinterpret_cast<uint16_t*>(smem + lay.a_off);      // [ns_cta][r][32]
  uint16_t* s_B = reinterpret_cast<uint16_t*>(smem + lay.b_off);      // [per8][fz_brow_stride(r)]
  float* s_pc = reinterpret_cast<float*>(smem + lay.pc_off);
  double* s_xt = reinterpret_cast<double*>(smem + lay.xt_off);        // [K+1][32]
  int& s_round = sh.round;
  double* s_inv = sh.inv;
  unsigned long long* s_kmm = sh.kmm;

  if (tid == 0) FZ_CSTAMP(0);
  // The mbarriers are set up once per launch and keep running from layer to layer: sh.phase[b] counts the phases barrier
  // b has completed so far, so a wait for the t-th use of a barrier in this layer asks for parity (phase[b] + t) & 1.
  unsigned* s_phase = sh.phase;
  if (first_layer) {
    if (tid == 0) {
#pragma unroll 1
      for (int i = 0; i < FZ_NBAR; ++i) mbar_init(&s_bar[i], 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (tid < FZ_NBAR) s_phase[tid] = 0u;
    if (tid == 32) {  // stage c of K runs on the CTAs [c G / K, (c + 1) G / K)
      const int c = ((cta + 1) * K - 1) / G;
      sh.stage = c;
      sh.g_lo = c * G / K;
      sh.gsize = (c + 1) * G / K - sh.g_lo;
      s_round = 0; sh.nsurv = 0; sh.done = 0;  // (the whole-token kernel clears them again at every layer boundary)
    }
    __syncthreads();
  }
  if (tid == 0) FZ_STAMP(1, 20);

  const int per = lay.per, r = A.r, Fn = A.Fn;
  const int i_lo = cta * per, i_hi = min(Fn, i_lo + per);
  const int n_own = max(0, i_hi - i_lo);
  const int nsl = (d + FZ_SL - 1) / FZ_SL;  // column slices of the feature; this CTA takes slices cta, cta + G, ...
  int used_r1 = 0, used_r2 = 0;            // first-ring and second-ring copies this CTA waited for in this layer

  {
    // ================================================= stream: all warps ===========================================
    // this CTA serves one stage: the ranks [lo, hi) of the selection, every gsize-th neuron starting at its own offset
    const int count = max(0, min(known_count >= 0 ? known_count : __ldcg(A.sel_count), A.sel_cap));
    const int m = count > 0 ? (count + K - 1) / K : 0;
    const int stage = sh.stage, g_lo = sh.g_lo, gsize = sh.gsize;
    const int lo = min(count, stage * m), hi = min(count, (stage + 1) * m);
    const int first = lo + (cta - g_lo);
    const int n_mine = first < hi ? (hi - first + gsize - 1) / gsize : 0;
    const int n_rounds = (n_mine + NG1 - 1) / NG1;
    const uint32_t r1_bytes = (uint32_t)d * 2, r2_bytes = (uint32_t)(A.n_mat - 1) * d * 2;
    const size_t bundle_elems = (size_t)A.n_mat * d;
    const int up_off = A.gated ? 0 : -1, dn_off = A.gated ? d : 0;  // where the rows sit inside a second-ring slot

    int* s_myidx = reinterpret_cast<int*>(smem + lay.mine_off);
    float* s_mybias = reinterpret_cast<float*>(s_myidx + FZ_MAX_MINE);
    int* s_surv = s_myidx + 2 * FZ_MAX_MINE;                       // surviving neurons, in the order they were found
    float* s_qa = reinterpret_cast<float*>(s_myidx + 3 * FZ_MAX_MINE);  // their activations
    // The first ring is used in rounds of NG1 neurons: G1R rounds fit; the rows of a round complete one barrier together
    // (a wait costs a warp some two hundred clocks even when the data is there: one per round, not one per row).
    const int G1R = G1 / NG1;
    const int n_first = min(n_mine, G1R * NG1);  // rows requested in the prologue, by the compute warps
    float xr[CPT][8];
    {
      double sq = 0.0;
#pragma unroll
      for (int q = 0; q < CPT; ++q) {
        const int ch = tid + q * FZ_THREADS;
        if (ch < nchunk && warp < FZ_THREADS / 32) {
          // (x left in shared memory by the layer before: every CTA reading the same 16 KB of global memory at the same
          // moment, right after a grid barrier, holds up everything issued behind it)
          const float4* xsrc = A.xs_get >= 0 ? reinterpret_cast<const float4*>(smem + A.xs_get) + ch * 2 : nullptr;
          const float4 a0 = xsrc ? xsrc[0] : __ldcg(reinterpret_cast<const float4*>(A.x + ch * 8));
          const float4 a1 = xsrc ? xsrc[1] : __ldcg(reinterpret_cast<const float4*>(A.x + ch * 8 + 4));
          xr[q][0] = a0.x; xr[q][1] = a0.y; xr[q][2] = a0.z; xr[q][3] = a0.w;
          xr[q][4] = a1.x; xr[q][5] = a1.y; xr[q][6] = a1.z; xr[q][7] = a1.w;
        } else {
#pragma unroll
          for (int e = 0; e < 8; ++e) xr[q][e] = 0.f;
        }
      }
      // This CTA's neurons: warp w takes the neurons w, w + 16, ... of the CTA's list.  One lane fetches the index and,
      // at once, the gate bias (a small load issued after bulk copies would queue behind all of them); the row of the
      // first ring follows in four pieces from four lanes (several smaller copies from many warps land sooner than one
      // copy per row issued by one warp: a warp's bulk-copy instructions go out one lane after the other).
      if (warp < FZ_THREADS / 32) {
#ifdef LS_DBG_NP1
        const int np = 1;
#else
        const int np = (r1_bytes & 63u) == 0 ? 4 : 1;
#endif
        const uint32_t piece = r1_bytes / (uint32_t)np;
#pragma unroll 1
        for (int t = warp; t < n_mine; t += FZ_THREADS / 32) {
          int i = 0;
          float b = 0.f;
          if (lane == 0) {
            i = __ldcg(A.sel_idx + first + t * gsize);
            if ((unsigned)i >= (unsigned)A.F) { set_status(A.status, ST_BAD_INDEX); i = -1; }
            if (A.b_gate && i >= 0) b = A.b_gate[i];
            if (t < n_first && t % NG1 == 0) mbar_expect_tx(&s_bar[t / NG1], (uint32_t)min(NG1, n_mine - t) * r1_bytes);
          }
          i = __shfl_sync(0xffffffffu, i, 0);
          if (tid == 0) FZ_STAMP_DEP(1, 27, __int_as_float(i));
          if (t < n_first && lane < np)  // (a rejected index reads row 0; the result is discarded)
            tma_load_1d(s_r1 + (size_t)t * d + lane * (piece / 2), A.bundles + (size_t)max(i, 0) * bundle_elems + lane * (piece / 2), piece, &s_bar[t / NG1]);
          if (tid == 0) FZ_STAMP(1, 28);
          if (lane == 0) { s_myidx[t] = i; s_mybias[t] = b; }
          if (tid == 0) FZ_STAMP_DEP(1, 29, b);
        }
      }
#pragma unroll
      for (int q = 0; q < CPT; ++q)
#pragma unroll
        for (int e = 0; e < 8; ++e) sq = fma((double)xr[q][e], (double)xr[q][e], sq);
      sq = warp_sum(sq);
      if (tid == 0) FZ_STAMP_DEP(1, 31, (float)sq);
      if (lane == 0 && warp < FZ_THREADS / 32) s_redd[warp] = sq;
    }
    __syncthreads();  // indices and the sums of squares visible (the producer warp goes its own way from here)
    if (tid == 0) FZ_STAMP(1, 21);

    if (warp == FZ_THREADS / 32) {
      // ============================================= producer warp ================================================
      // After every round of the first ring it turns the compute warps' partial dot products into activations, keeps
      // the list of survivors, and issues every further bulk copy (lane l the l-th copy of a batch): the next rounds
      // of the first ring when more neurons than fit were assigned, and, for the survivors only, the rest of the bundle
      // (up and down rows) into the second ring as slots come free.  The compute warps never wait for any of this:
      // they signal a finished round on a named barrier without blocking and go on to the next round's rows.
      {
        float inv_rms_p = 1.0f;
        if (A.norm == 0) {
          double tot = 0.0;
#pragma unroll 4
          for (int w = 0; w < FZ_THREADS / 32; ++w) tot += s_redd[w];
          inv_rms_p = (float)fz_rsqrt(fma(tot, A.inv_d, (double)A.eps));
        }
        int issued2 = 0, nsurv = 0;
        bool ok = true;
        const long long t0 = clock64();
        // (after the rounds) survivors whose slot is free
        auto issue_survivors = [&](int done) {
          const int slot2 = issued2 % G2T;  // (survivor q goes to slot q % G2T)
          const int n_can = min(nsurv - issued2, G2T - (issued2 - done));
          if (lane < n_can) {
            int sl2 = slot2 + lane;
            if (sl2 >= G2T) sl2 -= G2T;
            const int i = s_surv[issued2 + lane];
            uint64_t* bar = &s_bar[FZ_BAR_R2 + sl2];
            uint16_t* dst = sl2 < G2 ? s_r2 + (size_t)sl2 * (A.n_mat - 1) * d : s_r1 + (size_t)(sl2 - G2) * (A.n_mat - 1) * d;
            mbar_expect_tx(bar, r2_bytes);
            tma_load_1d(dst, A.bundles + (size_t)i * bundle_elems + d, r2_bytes, bar);
            if (A.tr_survive) atomicOr(&A.tr_survive[i >> 5], 1u << (i & 31));
          }
          if (n_can > 0) issued2 += n_can;
        };
        if (!lay.a_alias && A.has_next && lane == 0) fz_issue_a(A, s_A, &s_bar[FZ_BAR_A], cta, G, nsl);  // A slices with a place of their own
#pragma unroll 1
        for (int rd = 0; rd < n_rounds; ++rd) {
          named_bar_sync(2 + (rd & 1), FZ_BLOCK);  // every compute warp has left its partial sums of round rd
          const int it0 = rd * NG1, nn = min(NG1, n_mine - it0);
          const float* red = s_red + (rd & 1) * (FZ_THREADS / 32) * FZ_NG1;  // [warp][FZ_NG1]
          float a = 0.f;
          int i = -1;
          {
            // lane l adds the partial sums of neuron l & 3 left by the warps 2 (l >> 2) and 2 (l >> 2) + 1; three
            // exchanges complete the sums (always in the same order)
            float v = red[(2 * (lane >> 2)) * FZ_NG1 + (lane & 3)] + red[(2 * (lane >> 2) + 1) * FZ_NG1 + (lane & 3)];
            v += __shfl_xor_sync(0xffffffffu, v, 4);
            v += __shfl_xor_sync(0xffffffffu, v, 8);
            v += __shfl_xor_sync(0xffffffffu, v, 16);
            if (lane < nn) {
              i = s_myidx[it0 + lane];
              a = fmaxf(v * inv_rms_p + s_mybias[it0 + lane], 0.f);
              if (i < 0) a = 0.f;
            }
          }
          const unsigned surv = __ballot_sync(0xffffffffu, a != 0.f);
          {
            // a survivor's lane requests the rest of its bundle at once when a slot is certainly free (nothing consumed yet)
            const int limit = rd + 1 == n_rounds ? G2T : G2;
            const bool direct = issued2 == nsurv;
            if (a != 0.f) {
              const int pos = nsurv + __popc(surv & ((1u << lane) - 1u));
              if (direct && pos < limit) {
                uint64_t* bar = &s_bar[FZ_BAR_R2 + pos];
                uint16_t* dst = pos < G2 ? s_r2 + (size_t)pos * (A.n_mat - 1) * d : s_r1 + (size_t)(pos - G2) * (A.n_mat - 1) * d;
                mbar_expect_tx(bar, r2_bytes);
                tma_load_1d(dst, A.bundles + (size_t)i * bundle_elems + d, r2_bytes, bar);
                if (A.tr_survive) atomicOr(&A.tr_survive[i >> 5], 1u << (i & 31));
              }
              s_surv[pos] = i;
              s_qa[pos] = a;
            }
            const int nnew = nsurv + __popc(surv);
            if (direct) issued2 = max(issued2, min(nnew, limit));
            nsurv = nnew;
          }
          __syncwarp();
          if (lane == 0) {
            sh.nsurv = nsurv;
            asm volatile("st.release.cta.shared.s32 [%0], %1;" ::"r"(smem_u32(&s_round)), "r"(rd + 1) : "memory");
          }
          // the round's slot is free: the round G1R ahead moves in
          const int rn = rd + G1R;
          if (rn < n_rounds) {
            const int t1 = rn * NG1, n1 = min(NG1, n_mine - t1), rs = rn % G1R;
            if (lane == 0) mbar_expect_tx(&s_bar[rs], (uint32_t)n1 * r1_bytes);
            __syncwarp();
            if (lane < n1) {
              int i1 = s_myidx[t1 + lane];
              if (i1 < 0) i1 = 0;  // a rejected index: read row 0, the result is discarded
              tma_load_1d(s_r1 + (size_t)(rs * NG1 + lane) * d, A.bundles + (size_t)i1 * bundle_elems, r1_bytes, &s_bar[rs]);
            }
          }
          if (tid == FZ_THREADS) FZ_STAMP(0, 3 + rd * 4);
        }
        // the remaining survivors (the first ring is idle now: every slot may be used), as the compute warps consume the second ring
        int done = 0;
#pragma unroll 1
        while (issued2 < nsurv) {
          issue_survivors(done);
          if (issued2 == nsurv) break;
          int dnow;
          while (true) {
            asm volatile("ld.acquire.cta.shared.s32 %0, [%1];" : "=r"(dnow) : "r"(smem_u32(&sh.done)) : "memory");
            dnow = __shfl_sync(0xffffffffu, dnow, 0);  // (one view for the whole warp)
            if (dnow > done) break;
            if (__shfl_sync(0xffffffffu, (int)(clock64() - t0 > FZ_SPIN_CYCLES), 0)) { ok = false; break; }
            __nanosleep(64);  // the poll shares an instruction scheduler with four compute warps
          }
          if (!ok) { if (lane == 0) set_status(A.status, ST_TIMEOUT); break; }
          done = dnow;
        }
        // The next layer's predictor operands that share bytes with the rings wait until the compute warps have drained them.
        if (A.has_next && ok) {
          int drained = 0;
          if (lane == 0) drained = fz_wait_round(&s_round, n_rounds + 1, A.status) ? 1 : 0;
          drained = __shfl_sync(0xffffffffu, drained, 0);
          if (drained) {
            uint64_t* bbar = &s_bar[FZ_BAR_B];  // rows of B^T: awaited before the score phase
            if (lane == 0) {
              if (lay.a_alias) fz_issue_a(A, s_A, &s_bar[FZ_BAR_A], cta, G, nsl);
              mbar_expect_tx(bbar, (uint32_t)n_own * (uint32_t)r * 2);
            }
            __syncwarp();
            const int rsb = fz_brow_stride(r);
#pragma unroll 1
            for (int li = lane; li < n_own; li += 32)
              tma_load_1d(s_B + (size_t)li * rsb, A.Bt + (size_t)(i_lo + li) * r, (uint32_t)r * 2, bbar);
          }
        }
      }
      return;  // an exited warp counts as arrived at every later block barrier
    }

    float inv_rms = 1.0f;
    if (A.norm == 0) {
      double tot = 0.0;
#pragma unroll 4
      for (int w = 0; w < FZ_THREADS / 32; ++w) tot += s_redd[w];
      inv_rms = (float)fz_rsqrt(fma(tot, A.inv_d, (double)A.eps));
    }
    if (tid == 0) FZ_STAMP(0, 0);
    if (tid == 0) { FZ_CSTAMP(1); FZ_CVAL(8, n_mine); FZ_CVAL(10, stage); }

    // ---- first ring: the dot products of every neuron's first row with x, a round of NG1 neurons at a time; each warp
    //      leaves its partial sums for the producer warp and moves on ---------------------------------------------------
    int rslot = 0;
    unsigned wrapr = 0;
#ifdef LS_FZ_TIMING
    unsigned tw[6] = {0, 0, 0, 0, 0, 0};
#endif
#pragma unroll 1
    for (int rd = 0; rd < n_rounds; ++rd) {
      const int it0 = rd * NG1;
      const int nn = min(NG1, n_mine - it0);
      if (tid == 0) FZ_STAMP(0, 1 + rd * 4);
#ifdef LS_FZ_TIMING
      if (rd == 1) tw[0] = clock();
      if (rd == 2) tw[5] = clock();
#endif
      // the partial sums and the named barrier of round rd - 2 are used again: the producer must be through with them
      if (rd >= 2) {
        if (lane == 0) fz_wait_round(&s_round, rd - 1, A.status);
        __syncwarp();
      }
      float* red = s_red + (rd & 1) * (FZ_THREADS / 32) * FZ_NG1;  // [warp][FZ_NG1]
      mbar_wait(&s_bar[rslot], (s_phase[rslot] + wrapr) & 1u, A.status);
      const uint16_t* g0 = s_r1 + (size_t)rslot * NG1 * d;
      if (++rslot == G1R) { rslot = 0; ++wrapr; }
#ifdef LS_FZ_TIMING
      if (rd == 1) tw[1] = clock();
#endif
      {  // up to four neurons: four independent chains of loads, FMAs and shuffles
        float pg[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int q = 0; q < CPT; ++q) {
          const int ch = tid + q * FZ_THREADS;
          if (ch < nchunk) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              if (u < nn) {
                float w[8];
                unpack8<WD>(*reinterpret_cast<const uint4*>(g0 + (size_t)u * d + ch * 8), w);
#pragma unroll
                for (int t = 0; t < 8; ++t) pg[u] = fmaf(w[t], xr[q][t], pg[u]);
              }
            }
          }
        }
#ifdef LS_FZ_TIMING
        if (rd == 1) asm volatile("{ .reg .f32 t_; add.f32 t_, %1, %2; mov.u32 %0, %%clock; }" : "=r"(tw[2]) : "f"(pg[0] + pg[1]), "f"(pg[2] + pg[3]));
#endif
        {  // four sums over the warp in six shuffles: at every step a lane hands over the half it does not keep
          const bool h16 = (lane & 16) != 0, h8 = (lane & 8) != 0;
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const float give = h16 ? pg[u] : pg[u + 2], keep = h16 ? pg[u + 2] : pg[u];
            pg[u] = keep + __shfl_xor_sync(0xffffffffu, give, 16);
          }
          const float give = h8 ? pg[0] : pg[1], keep = h8 ? pg[1] : pg[0];
          pg[0] = keep + __shfl_xor_sync(0xffffffffu, give, 8);
          pg[0] += __shfl_xor_sync(0xffffffffu, pg[0], 4);
          pg[0] += __shfl_xor_sync(0xffffffffu, pg[0], 2);
          pg[0] += __shfl_xor_sync(0xffffffffu, pg[0], 1);
        }
#ifdef LS_FZ_TIMING
        if (rd == 1) asm volatile("{ .reg .f32 t_; add.f32 t_, %1, %2; mov.u32 %0, %%clock; }" : "=r"(tw[3]) : "f"(pg[0]), "f"(pg[0]));
#endif
        if ((lane & 7) == 0) red[warp * FZ_NG1 + (lane >> 3)] = pg[0];  // lane 8 u holds the sum of neuron u
      }
      if (tid == 0) FZ_STAMP(0, 2 + rd * 4);
      __syncwarp();
      asm volatile("bar.arrive %0, %1;" ::"r"(2 + (rd & 1)), "r"(FZ_BLOCK) : "memory");  // (does not block)
#ifdef LS_FZ_TIMING
      if (rd == 1) tw[4] = clock();
#endif
    }
    if (tid == 0) FZ_STAMP(0, 500);
#ifdef LS_FZ_TIMING
    if (lane == 0 && blockIdx.x == 0)
      for (int i_ = 0; i_ < 6; ++i_) g_fz_timing[0][160 + warp * 6 + i_] = tw[i_];
#endif

    // ---- second ring: the survivors, in batches of up to FZ_NB2, as the producer finds them (a batch starts with whatever
    //      is known, so the survivors of the early rounds are worked on while the last round's rows are still in flight):
    //      (gated) their up rows complete the activations, then their down rows, scaled, join the CTA's partial output
    //      (kept in registers).  Survivor q sits in slot q % G2T and is the (q / G2T)-th use of that slot in this layer.
    float yacc[CPT][8];
#pragma unroll
    for (int q = 0; q < CPT; ++q)
#pragma unroll
      for (int e = 0; e < 8; ++e) yacc[q][e] = 0.f;
    float* red2 = s_red + 2 * (FZ_THREADS / 32) * FZ_NG1;  // [warp][FZ_NB2]
    const size_t r2_elems = (size_t)(A.n_mat - 1) * d;
    int q0 = 0, slot0 = 0;  // the batch starts at survivor q0, which sits in slot slot0 = q0 % G2T
    unsigned wrap0 = 0;     // q0 / G2T
#pragma unroll 1
    while (true) {
      if (warp == 0) {
        // what is known: survivors [q0, known) are listed; after round n_rounds the list is final
        int known = 0, fin = 0;
        if (lane == 0) {
          const long long t0 = clock64();
          while (true) {
            int rnow;
            asm volatile("ld.acquire.cta.shared.s32 %0, [%1];" : "=r"(rnow) : "r"(smem_u32(&s_round)) : "memory");
            known = *reinterpret_cast<volatile int*>(&sh.nsurv);
            fin = rnow >= n_rounds;
            if (known > q0 || fin) break;
            if (clock64() - t0 > FZ_SPIN_CYCLES) { set_status(A.status, ST_TIMEOUT); fin = 1; break; }
          }
        }
        known = __shfl_sync(0xffffffffu, known, 0);
        fin = __shfl_sync(0xffffffffu, fin, 0);
        const int hi = min(known, q0 + min(FZ_NB2, G2T));  // (a batch never needs more slots than there are)
        if (q0 + lane < hi) {  // the batch's rows: each lane waits for one
          int sl = slot0 + lane;
          unsigned wr = wrap0;
          if (sl >= G2T) { sl -= G2T; ++wr; }
          mbar_wait(&s_bar[FZ_BAR_R2 + sl], (s_phase[FZ_BAR_R2 + sl] + wr) & 1u, A.status);
        }
        __syncwarp();
        if (lane == 0) { sh.b_hi = hi; sh.b_last = (fin && hi == known) ? 1 : 0; }
      }
      named_bar_sync(1, FZ_THREADS);  // the batch is known to all, its rows have landed
      const int hi = *reinterpret_cast<volatile int*>(&sh.b_hi), last = *reinterpret_cast<volatile int*>(&sh.b_last);
      const int nb = hi - q0;
      if (nb > 0) {
        if (up_off >= 0) {
#pragma unroll 1
          for (int e0 = 0; e0 < nb; e0 += 4) {  // four up rows at a time: four independent chains of loads, FMAs and shuffles
            float pu[4] = {0.f, 0.f, 0.f, 0.f};
            const uint16_t* urow[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              int sl = slot0 + e0 + u;
              if (sl >= G2T) sl -= G2T;
              urow[u] = sl < G2 ? s_r2 + (size_t)sl * r2_elems : s_r1 + (size_t)(sl - G2) * r2_elems;
            }
#pragma unroll
            for (int q = 0; q < CPT; ++q) {
              const int ch = tid + q * FZ_THREADS;
              if (ch < nchunk) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                  if (e0 + u < nb) {
                    float w[8];
                    unpack8<WD>(*reinterpret_cast<const uint4*>(urow[u] + ch * 8), w);
#pragma unroll
                    for (int t = 0; t < 8; ++t) pu[u] = fmaf(w[t], xr[q][t], pu[u]);
                  }
                }
              }
            }
            // four sums over the warp in six shuffles: at every step a lane hands over the half it does not keep
            const bool h16 = (lane & 16) != 0, h8 = (lane & 8) != 0;
#pragma unroll
            for (int u = 0; u < 2; ++u) {
              const float give = h16 ? pu[u] : pu[u + 2], keep = h16 ? pu[u + 2] : pu[u];
              pu[u] = keep + __shfl_xor_sync(0xffffffffu, give, 16);
            }
            {
              const float give = h8 ? pu[0] : pu[1], keep = h8 ? pu[1] : pu[0];
              pu[0] = keep + __shfl_xor_sync(0xffffffffu, give, 8);
            }
            pu[0] += __shfl_xor_sync(0xffffffffu, pu[0], 4);
            pu[0] += __shfl_xor_sync(0xffffffffu, pu[0], 2);
            pu[0] += __shfl_xor_sync(0xffffffffu, pu[0], 1);
            if ((lane & 7) == 0) red2[warp * FZ_NB2 + e0 + (lane >> 3)] = pu[0];  // lane 8 u holds the sum of row e0 + u
          }
          named_bar_sync(1, FZ_THREADS);
          if (warp == 0) {  // lane l adds the partial sums of survivor l & 7 left by the warps 4 (l >> 3) .. 4 (l >> 3) + 3
            const int w4 = 4 * (lane >> 3), e = lane & 7;
            float v = (red2[w4 * FZ_NB2 + e] + red2[(w4 + 1) * FZ_NB2 + e]) + (red2[(w4 + 2) * FZ_NB2 + e] + red2[(w4 + 3) * FZ_NB2 + e]);
            v += __shfl_xor_sync(0xffffffffu, v, 8);
            v += __shfl_xor_sync(0xffffffffu, v, 16);
            if (lane < nb) s_qa[q0 + lane] *= v * inv_rms;
          }
          named_bar_sync(1, FZ_THREADS);
        }
#pragma unroll 1
        for (int e = 0; e < nb; ++e) {
          const float a = s_qa[q0 + e];
          int sl = slot0 + e;
          if (sl >= G2T) sl -= G2T;
          const uint16_t* row = (sl < G2 ? s_r2 + (size_t)sl * r2_elems : s_r1 + (size_t)(sl - G2) * r2_elems) + dn_off;
#pragma unroll
          for (int q = 0; q < CPT; ++q) {
            const int ch = tid + q * FZ_THREADS;
            if (ch < nchunk) {
              float w[8];
              unpack8<WD>(*reinterpret_cast<const uint4*>(row + ch * 8), w);
#pragma unroll
              for (int t = 0; t < 8; ++t) yacc[q][t] = fmaf(a, w[t], yacc[q][t]);
            }
          }
        }
        q0 = hi;
        slot0 += nb;
        if (slot0 >= G2T) { slot0 -= G2T; ++wrap0; }
        if (!last) {
          named_bar_sync(1, FZ_THREADS);  // every thread is done with the batch's slots: the producer may refill them
          if (tid == 0) asm volatile("st.release.cta.shared.s32 [%0], %1;" ::"r"(smem_u32(&sh.done)), "r"(q0) : "memory");
        }
      }
      if (last) break;
    }
    const int nsurv = q0;
    if (tid == 0) { FZ_CSTAMP(2); FZ_CVAL(9, nsurv); }
    used_r1 = n_rounds;
    used_r2 = nsurv;
    named_bar_sync(1, FZ_THREADS);  // nobody reads the rings any more: the producer may overwrite them
    if (tid == 0) asm volatile("st.release.cta.shared.s32 [%0], %1;" ::"r"(smem_u32(&s_round)), "r"(n_rounds + 1) : "memory");
    // the CTA's whole contribution to its stage (zeros when nothing survived) goes to its own row of ypart: the stage
    // sums are formed later in a fixed order, so the features do not depend on the order in which CTAs finish
    {
      float* dst = A.ypart + (size_t)cta * d;
#pragma unroll
      for (int q = 0; q < CPT; ++q) {
        const int ch = tid + q * FZ_THREADS;
        if (ch < nchunk) {
          *reinterpret_cast<float4*>(dst + ch * 8) = make_float4(yacc[q][0], yacc[q][1], yacc[q][2], yacc[q][3]);
          *reinterpret_cast<float4*>(dst + ch * 8 + 4) = make_float4(yacc[q][4], yacc[q][5], yacc[q][6], yacc[q][7]);
        }
      }
    }
    if (tid == 0) FZ_STAMP(0, 501);
    if (tid == 0) FZ_CSTAMP(3);
  }

  // ------------------------------------------------------------------------------------------------ barrier 1 of 5
  if (tid == 0) FZ_STAMP(1, 0);
  if (tid == 0) FZ_CSTAMP(4);
  grid_barrier(A, G);
  if (tid == 0) FZ_STAMP(1, 1);
  if (tid == 0) FZ_CSTAMP(5);
  if (A.has_next) {  // offsets of this CTA's share of the next layer's predictor (needed in the score phase)
#pragma unroll 1
    for (int li = tid; li < n_own; li += FZ_THREADS) s_pc[li] = A.pc ? A.pc[i_lo + li] : 0.f;
  }
  if (tid >= 64 && tid < 67) {  // one line of every 2 MB page of the next layer's weights and predictor (this CTA's share)
    const int i = tid - 64;
    const char* p = static_cast<const char*>(A.pg_ptr[i]);
    if (p) {
#pragma unroll 1
      for (unsigned long long off = (unsigned long long)cta << 21; off < A.pg_bytes[i]; off += (unsigned long long)G << 21)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(p + off));
    }
  }
  if (tid >= 32 && tid < 36) {  // HBM is idle now: this CTA's share of what the next layer reads first goes to L2
    const int i = tid - 32;
    const unsigned bytes = A.pf_bytes[i] & ~15u;
    const char* p = static_cast<const char*>(A.pf_ptr[i]);
    if (p && bytes && (reinterpret_cast<uintptr_t>(p) & 15) == 0) {
      const unsigned chunk = ((bytes + G - 1) / G + 127u) & ~127u, off = (unsigned)cta * chunk;
      if (off < bytes)
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p + off), "r"(min(chunk, bytes - off)) : "memory");
    }
  }

  // ============================ phase 2: partial features x~^(j), per-slice partial latents ==========================
  // The columns of the feature are cut into slices of 32; a CTA owns slices cta, cta + G, ...  For each it rebuilds
  // x~^(j), j = 0..K, of its columns (x + the stage accumulators below j, Eq. 2), writes x_out = x~^(K), and multiplies
  // the slice of A (r x 32, in shared memory) with the 32 x (K+1) block of features on the fp64 tensor cores.  The
  // partial latents (and the partial sums of squares, as row r) go to global memory, one block per slice.
  // Evaluations are taken eight at a time on the fp64 tensor cores; a remainder of one or two evaluations is cheaper on
  // the ordinary fp64 pipe (a padded tile would spend eight evaluations' worth of the same units).
  const int E = K + 1, RS = r + 1;
  int NTM = E >> 3, REM = E & 7;
  if (REM > 2) { ++NTM; REM = 0; }
  const int EM = NTM * 8;  // evaluations [0, EM) by MMA (rows past K are zero), [EM, E) by scalar code
  constexpr int XTS = FZ_XBLK;    // row stride (doubles) of s_xt: one block of features per row
  if (A.has_next && cta < nsl)
    mbar_wait(&s_bar[FZ_BAR_A], s_phase[FZ_BAR_A] & 1u, A.status);  // the A slices have landed
  if (tid == 0) FZ_STAMP(1, 10);
#pragma unroll 1
  for (int a = 0; cta + a * G < nsl; ++a) {
    const int sl = cta + a * G;
    if (a > 0) named_bar_sync(1, FZ_THREADS);  // the previous slice's features are no longer read
    float* s_dv = reinterpret_cast<float*>(smem + lay.dv_off);  // [K][32] stage sums dm^(c) of the slice's columns
    float* s_dvp = s_dv + FZ_MAXK * FZ_SL;                        // [16][32] partial sums of thread groups
    float xv = 0.f;
    {
      // Stage c is the sum of the partial outputs of the CTAs [c G / K, (c + 1) G / K).  The 16 groups of 32 threads
      // (one thread per column) share the stages: nh groups per stage, group h adds every nh-th CTA of the stage in
      // order, twelve loads in flight; the nh partial sums are then added in order: a fixed summation tree.
      const int col = tid & (FZ_SL - 1), u = tid >> 5, c = sl * FZ_SL + col;
      const int nh = max(1, (FZ_THREADS / 32) / K), cs = u / nh, h = u - cs * nh;
      float acc = 0.f;
      if (cs < K && c < d) {
        const int p_hi = (cs + 1) * G / K;
        const float* yp = A.ypart + c;
#pragma unroll 1
        for (int p = cs * G / K + h; p < p_hi; p += 12 * nh) {  // (148 CTAs: at most ten per thread, one batch)
          float q[12];
#pragma unroll
          for (int v = 0; v < 12; ++v) q[v] = p + v * nh < p_hi ? __ldcg(yp + (size_t)(p + v * nh) * d) : 0.f;
#pragma unroll
          for (int v = 0; v < 12; ++v) acc += q[v];
        }
      }
      s_dvp[tid] = acc;
    }
    if (tid < FZ_SL) {
      const int c = sl * FZ_SL + tid;
      if (c < d) xv = __ldcg(A.x + c) + (A.b_down ? A.b_down[c] : 0.f);
    }
    named_bar_sync(1, FZ_THREADS);
    if (tid < K * FZ_SL) {
      const int nh = max(1, (FZ_THREADS / 32) / K), cs = tid >> 5, col = tid & (FZ_SL - 1);
      float v = 0.f;
#pragma unroll 1
      for (int h = 0; h < nh; ++h) v += s_dvp[(cs * nh + h) * FZ_SL + col];
      s_dv[tid] = v;
    }
    named_bar_sync(1, FZ_THREADS);
    if (tid < FZ_SL) {
      const int c = sl * FZ_SL + tid;
      float* const trx = A.tr_xtilde;  // (the arguments live in shared memory: read them once, not after every store)
      float* const xo = A.x_out;
      const int rows = max(EM, E);
#pragma unroll 1
      for (int j = 0; j < rows; ++j) {
        s_xt[j * XTS + fz_feat_pos(tid)] = j <= K ? (double)xv : 0.0;
        if (j <= K && c < d) {
          if (trx) trx[(size_t)j * d + c] = xv;
          if (j == K) xo[c] = xv;  // may alias x: this thread is the only one that still needs x[c]
        }
        if (j < K) xv += s_dv[j * FZ_SL + tid];
      }
    }
    named_bar_sync(1, FZ_THREADS);
    if (tid == 0) FZ_STAMP(1, 11);
    if (A.has_next) {
      // 32 x (K+1) block of features times the slice of A: evaluations [0, EM) on the tensor cores, eight at a time,
      // evaluations [EM, E) (at most two) with ordinary FMAs on the same weights
      double* part = A.zpart + (size_t)sl * E * RS;
      const uint16_t* As = s_A + (size_t)a * r * FZ_SL;
      const int n_rt = (r + 7) >> 3;
      const int g = lane >> 2, t4 = lane & 3;
#pragma unroll 1
      for (int mt = warp; mt < n_rt; mt += FZ_THREADS / 32) {
        const int row = mt * 8 + g;
        double av[8];
        cvt8_to_double<WD>(*reinterpret_cast<const uint4*>(As + (size_t)min(row, r - 1) * FZ_SL + t4 * 8), av);
        double c[2][2] = {{0.0, 0.0}, {0.0, 0.0}}, rs[2] = {0.0, 0.0}, bv[8];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          if (nt < NTM) {
            load8d(s_xt + (size_t)(nt * 8 + g) * XTS + t4 * 10, bv);
            mma_block(c[nt], av, bv);
          }
        }
#pragma unroll
        for (int rm = 0; rm < 2; ++rm) {
          if (rm < REM) {
            load8d(s_xt + (size_t)(EM + rm) * XTS + t4 * 10, bv);
#pragma unroll
            for (int k = 0; k < 8; ++k) rs[rm] = fma(av[k], bv[k], rs[rm]);
            rs[rm] = quad_sum(rs[rm]);
          }
        }
        if (row < r) {
#pragma unroll
          for (int nt = 0; nt < 2; ++nt) {
            const int j = nt * 8 + t4 * 2;
            if (nt < NTM && j <= K) part[(size_t)j * RS + row] = c[nt][0];
            if (nt < NTM && j + 1 <= K) part[(size_t)(j + 1) * RS + row] = c[nt][1];
          }
          if (t4 < REM) part[(size_t)(EM + t4) * RS + row] = t4 == 0 ? rs[0] : rs[1];
        }
      }
      if (tid == 0) FZ_STAMP(1, 12);
      if (warp == FZ_THREADS / 32 - 1) {  // partial sums of squares of the slice, one evaluation per lane
#pragma unroll 1
        for (int j = lane; j <= K; j += 32) {
          double sq = 0.0;
#pragma unroll 8
          for (int c = 0; c < FZ_SL; ++c) { const double v = s_xt[j * XTS + fz_feat_pos(c)]; sq = fma(v, v, sq); }
          part[(size_t)j * RS + r] = sq;
        }
      }
    }
  }
  if (tid == 0) FZ_STAMP(1, 30);

  if (A.has_next) {
    // ---------------------------------------------------------------------------------------------- barrier 2 of 5
    if (tid == 0) FZ_STAMP(1, 2);
    if (tid == 0) FZ_CSTAMP(6);
    grid_barrier(A, G);
    if (tid == 0) FZ_STAMP(1, 3);

    // ============================ phase 2b: sum of the slices' partials, four values per warp =========================
    // A warp takes four consecutive values (one 32-byte sector per slice); lane (q, v), q = lane / 4, adds the slices
    // q, q + 8, ... of value v in order, the eight partial sums are combined by a butterfly: the result does not depend on
    // which warp of which CTA computes it, and every sector fetched is used whole.
    {
      const int V = E * RS;
      const int q8 = lane >> 2, v4 = lane & 3;
#pragma unroll 1
      for (int v0 = (warp * G + cta) * 4; v0 < V; v0 += G * (FZ_THREADS / 32) * 4) {  // tasks dealt round-robin over the CTAs
        const int v = v0 + v4;
        const double* zp = A.zpart + min(v, V - 1);
        double acc = 0.0;
#pragma unroll 1
        for (int s0 = 0; s0 < nsl; s0 += 64) {  // eight loads in flight per lane
          double q[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const int s2 = s0 + u * 8 + q8;
            q[u] = s2 < nsl ? __ldcg(zp + (size_t)s2 * V) : 0.0;
          }
#pragma unroll
          for (int u = 0; u < 8; ++u) acc += q[u];
        }
        acc += __shfl_xor_sync(0xffffffffu, acc, 4);
        acc += __shfl_xor_sync(0xffffffffu, acc, 8);
        acc += __shfl_xor_sync(0xffffffffu, acc, 16);
        if (q8 == 0 && v < V) {
          const int j = v / RS, row = v - j * RS;
          if (row < r) A.z[(size_t)j * r + row] = acc;
          else A.sumsq[j] = acc;
        }
      }
    }
    // ---------------------------------------------------------------------------------------------- barrier 3 of 5
    if (tid == 0) FZ_STAMP(1, 7);
    grid_barrier(A, G);
    if (tid == 0) FZ_STAMP(1, 8);

    // ============================ phase 3: scores of this CTA's neurons, every evaluation =============================
    double* s_zs = reinterpret_cast<double*>(smem + lay.zs_off);            // [max(EM, E)][fz_feat_stride(r)], un-normalised, blocked
    double* s_part = reinterpret_cast<double*>(smem + lay.part_off);        // [slot][prow][per8]
    double* s_own = reinterpret_cast<double*>(smem + lay.own_off);          // [per] scores of the final evaluation
    const double bin_lo = __ldcg(&A.range[0]), bin_hi = __ldcg(&A.range[1]);
    const double INF = __longlong_as_double(0x7ff0000000000000LL);
    const double brange = bin_hi - bin_lo;
    const double bscale = (brange > 0.0 && brange < INF) ? (double)FZ_NB / brange : 0.0;
    const int keff = min(A.k_next, Fn);
    const int RSB = fz_brow_stride(r), RSZ = fz_feat_stride(r);
    const int nblk = (r + 31) >> 5, cpad_b = nblk * 32;
    const int per8 = (per + 7) & ~7;

    // latents of every evaluation (un-normalised, in the blocked order the tensor-core loads want) and 1 / rms of every
    // feature; eight loads in flight per thread
    {
      const double* zg = A.z;
      const int nz = E * r;
      const unsigned rmagic = 0xffffffffu / (unsigned)r + 1u;  // t / r == umulhi(t, rmagic) for t < 2^16
#pragma unroll 1
      for (int t0 = 0; t0 < nz; t0 += 8 * FZ_THREADS) {
        double q[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int t = t0 + u * FZ_THREADS + tid;
          q[u] = (t < nz) ? __ldcg(zg + t) : 0.0;  // z is [evaluation][r], contiguous
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int t = t0 + u * FZ_THREADS + tid;
          if (t < nz) {
            const int e = (int)__umulhi((unsigned)t, rmagic);
            s_zs[e * RSZ + fz_feat_pos(t - e * r)] = q[u];
          }
        }
      }
      // rows of a padded tile past K, and the columns past r of a last partial block, must read as zero
      const int rows = max(EM, E), cpad = nblk * 32;
#pragma unroll 1
      for (int t = tid; t < (rows - E) * cpad; t += FZ_THREADS) s_zs[(E + t / cpad) * RSZ + fz_feat_pos(t % cpad)] = 0.0;
      if (cpad > r) {
#pragma unroll 1
        for (int t = tid; t < E * (cpad - r); t += FZ_THREADS)
          s_zs[(t / (cpad - r)) * RSZ + fz_feat_pos(r + t % (cpad - r))] = 0.0;
      }
    }
    if (tid < FZ_EPAD)
      s_inv[tid] = (tid <= K && A.norm_n == 0) ? fz_rsqrt(fma(__ldcg(&A.sumsq[tid]), A.inv_d, (double)A.eps_n)) : 1.0;
    mbar_wait(&s_bar[FZ_BAR_B], s_phase[FZ_BAR_B] & 1u, A.status);  // the rows of B^T have landed
    if (cpad_b > r) {  // (only when r is not a multiple of 32) the tail of the last block of every row reads as zero
#pragma unroll 1
      for (int t = tid; t < per8 * (cpad_b - r); t += FZ_THREADS)
        s_B[(size_t)(t / (cpad_b - r)) * RSB + r + t % (cpad_b - r)] = 0;
    }
    named_bar_sync(1, FZ_THREADS);
    if (tid == 0) FZ_STAMP(1, 40);

    // C[neuron][evaluation] = B^T rows x latents.  Evaluations [0, EM) go through the tensor cores, evaluations [EM, E)
    // (at most two) through ordinary FMAs on the same converted weights.  Within one evaluation every neuron's score is
    // accumulated in the same order whatever its position in a tile, so equal predictor rows give bit-equal scores.
    // Work units are (tile of eight neurons, 32-column block), in tile-major order, dealt evenly: warp w takes the units
    // [w U, (w + 1) U).  A warp's share of a tile goes to the partial-sum slot `w - first warp of the tile`; the slots
    // of a tile are added afterwards in order.
    const int n_mt = (n_own + 7) >> 3;
    const int prow = max(EM, E);                                   // rows of a slot of partial sums
    const int n_units = n_mt * nblk, U = max(1, (n_units + FZ_THREADS / 32 - 1) / (FZ_THREADS / 32));
    int* s_nslot = reinterpret_cast<int*>(s_inv + FZ_EPAD);  // [n_mt] slots per tile (n_mt <= 64: behind the scale factors)
#pragma unroll 1
    for (int m2 = tid; m2 < n_mt; m2 += FZ_THREADS) s_nslot[m2] = (m2 * nblk + nblk - 1) / U - (m2 * nblk) / U + 1;
    if (lane == 0) FZ_STAMP(1, 400 + warp * 4);
    {
      const int u_lo = warp * U, u_hi = min(n_units, u_lo + U);
      const int g = lane >> 2, t4 = lane & 3;
      const double* zrow = s_zs + (size_t)g * RSZ + t4 * 10;      // MMA tiles: evaluation nt * 8 + g
      const double* zrem = s_zs + (size_t)EM * RSZ + t4 * 10;     // remainder evaluations EM, EM + 1
      double c[2][2] = {{0.0, 0.0}, {0.0, 0.0}}, rs[2] = {0.0, 0.0};
      int mt = u_lo < u_hi ? u_lo / nblk : -1;
#pragma unroll 1
      for (int u = u_lo; u < u_hi; ++u) {
        const int b = u - mt * nblk;
        double av[8], bv[8];
        cvt8_to_double<WD>(*reinterpret_cast<const uint4*>(s_B + (size_t)(mt * 8 + g) * RSB + t4 * 8 + b * 32), av);
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          if (nt < NTM) {
            load8d(zrow + (size_t)nt * 8 * RSZ + b * FZ_XBLK, bv);
            mma_block(c[nt], av, bv);
          }
        }
#pragma unroll
        for (int rm = 0; rm < 2; ++rm) {
          if (rm < REM) {
            load8d(zrem + (size_t)rm * RSZ + b * FZ_XBLK, bv);
#pragma unroll
            for (int k = 0; k < 8; ++k) rs[rm] = fma(av[k], bv[k], rs[rm]);
          }
        }
        if (b == nblk - 1 || u == u_hi - 1) {  // the warp's share of this tile is complete: to its slot
          const int slot = warp - (mt * nblk) / U;
          double* outp = s_part + (size_t)slot * prow * per8 + mt * 8 + g;
#pragma unroll
          for (int nt = 0; nt < 2; ++nt) {
            if (nt < NTM) {
              const int j = nt * 8 + t4 * 2;
              outp[(size_t)j * per8] = c[nt][0];
              outp[(size_t)(j + 1) * per8] = c[nt][1];
              c[nt][0] = c[nt][1] = 0.0;
            }
          }
#pragma unroll
          for (int rm = 0; rm < 2; ++rm) {
            if (rm < REM) {
              const double v = quad_sum(rs[rm]);
              if (t4 == 0) outp[(size_t)(EM + rm) * per8] = v;
              rs[rm] = 0.0;
            }
          }
          ++mt;
        }
      }
    }
    if (lane == 0) FZ_STAMP(1, 402 + warp * 4);
    named_bar_sync(1, FZ_THREADS);
    if (tid == 0) FZ_STAMP(1, 41);
    // final scores of this CTA's neurons, every evaluation: to global memory with their fine bin (one thread per
    // (evaluation, neuron), no atomics); the exact selection is made per evaluation by ONE CTA after the next barrier
    {
      // (the observed range only steers the next launch's binning: the upper halves of the ordered keys, rounded outwards,
      // are enough, and 32-bit minima and maxima cross a warp in one instruction)
      unsigned kmin = 0xffffffffu, kmax = 0u;
      const int n_ent = E * n_own;
      double* const nprio = A.next_prio;
      double* const nscores = A.next_scores;
      double* const sc = A.sc;
      uint16_t* const sb = A.sb;
#pragma unroll 1
      for (int t = tid; t < n_ent; t += FZ_THREADS) {
        const int j = t / n_own, li = t - j * n_own, i = i_lo + li;
        double v = 0.0;
        {
          const int nsl2 = s_nslot[li >> 3];  // slots of this neuron's tile
#pragma unroll 1
          for (int sl2 = 0; sl2 < nsl2; ++sl2) v += s_part[((size_t)sl2 * prow + j) * per8 + li];
        }
        v = canonical_score(v * s_inv[j] + (double)s_pc[li]);
        const double scl = fmin(fmax(v, -1.7976931348623157e308), 1.7976931348623157e308);
        int b = (int)((bin_hi - scl) * bscale);
        b = max(0, min(FZ_NB - 1, b));
        sc[(size_t)j * Fn + i] = v;
        sb[(size_t)j * Fn + i] = (uint16_t)b;
        if (j == K) {
          s_own[li] = v;  // kept for the speculation below
          if (nprio) nprio[i] = v;
          if (nscores) nscores[i] = v;
          const unsigned kh = (unsigned)(ordered_key(v) >> 32);
          kmin = min(kmin, kh);
          kmax = max(kmax, kh);
        }
      }
      kmin = __reduce_min_sync(0xffffffffu, kmin);
      kmax = __reduce_max_sync(0xffffffffu, kmax);
      unsigned* s_kmm32 = reinterpret_cast<unsigned*>(s_kmm);
      if (lane == 0) { s_kmm32[warp] = kmin; s_kmm32[16 + warp] = kmax; }
      named_bar_sync(1, FZ_THREADS);
      if (warp == 0) {  // observed score range of the final evaluation, this CTA's part (no atomics: a selecting CTA folds them)
        kmin = __reduce_min_sync(0xffffffffu, lane < 16 ? s_kmm32[lane] : 0xffffffffu);
        kmax = __reduce_max_sync(0xffffffffu, lane < 16 ? s_kmm32[16 + lane] : 0u);
        if (lane == 0) {
          A.kmm[2 * cta] = (unsigned long long)kmin << 32;
          A.kmm[2 * cta + 1] = ((unsigned long long)kmax << 32) | 0xffffffffULL;
        }
      }
    }

    // ---------------------------------------------------------------------------------------------- barrier 4 of 5
    if (tid == 0) FZ_STAMP(1, 4);
    if (tid == 0) FZ_CSTAMP(7);
    // the exact selection is made per evaluation after the barrier: the final one by the first FZ_FIN_PARTS CTAs
    // together (each ranks its share of the members), every earlier one by one CTA of its own
    const int fparts = max(1, min(FZ_FIN_PARTS, G - K));
    const bool selects = cta < fparts + K;
    const int jme = cta < fparts ? K : cta - fparts;
    // Speculation into L2 (thread li of a group that holds, in s_own, the final scores of the n neurons from i_base on):
    // the neurons scored highest will most likely be in the refined set, whose exact ranks take another grid barrier to
    // establish; the first row of their bundles in the next layer is asked into L2 now, so that the next layer's ring
    // fill finds it there.  The score estimates the gate pre-activation (B is W_gate A, c the gate bias): a likely member
    // with a positive score will probably survive the ReLU too, so the rest of its bundle is asked for as well.  A wrong
    // guess costs bandwidth that is idle at this point, never correctness.
    // Called by whole warps: thread t of nthr; four threads share a neuron's comparisons.
    auto speculate = [&](int t, int nthr, int i_base, int n) {
      const int m_spec = (int)(((long long)keff * n * 3 / 2 + Fn - 1) / Fn) + 1;  // half again the fair share: a round waits for its slowest row
#pragma unroll 1
      for (int base = 0; base < n; base += nthr >> 2) {
        const int li = base + (t >> 2), p = t & 3;
        const bool mine = li < n;
        const double v = mine ? s_own[li] : 0.0;
        int above = 0;
        if (mine) {
#pragma unroll 4
          for (int l2 = p; l2 < n; l2 += 4) {
            const double o = s_own[l2];
            above += (o > v) || (o == v && l2 < li);
          }
        }
        above += __shfl_xor_sync(0xffffffffu, above, 1);
        above += __shfl_xor_sync(0xffffffffu, above, 2);
        if (mine && p == 0 && above < m_spec)
          asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(A.spec_ptr + (size_t)(i_base + li) * A.spec_stride),
                       "r"(v > 0.0 ? (unsigned)A.spec_stride : A.spec_bytes) : "memory");
      }
    };
    named_bar_sync(1, FZ_THREADS);
    if (tid == 0) {
      grid_barrier_thread0(A, G);
    } else {
      if (tid >= 32 && A.spec_ptr && !selects) speculate(tid - 32, FZ_THREADS - 32, i_lo, n_own);
      if (A.xs_put >= 0) {  // the next layer's x (complete since the second barrier) waits in shared memory for its start
        float4* xs = reinterpret_cast<float4*>(smem + A.xs_put);
#pragma unroll 1
        for (int c4 = tid - 1; c4 < (d >> 2); c4 += FZ_THREADS - 1) xs[c4] = __ldcg(reinterpret_cast<const float4*>(A.x_out) + c4);
      }
    }
    named_bar_sync(1, FZ_THREADS);
    if (tid == 0) FZ_STAMP(1, 5);
    {
      // the selecting CTAs have no time to speculate: the next CTAs do it for them, from the scores now in global memory
      const int nsel = fparts + K, c2 = cta - nsel;
      if (A.spec_ptr && c2 >= 0 && c2 < nsel) {
        const int i2 = c2 * per, n2 = max(0, min(Fn, i2 + per) - i2);
#pragma unroll 1
        for (int li = tid; li < n2; li += FZ_THREADS) s_own[li] = __ldcg(A.sc + (size_t)K * Fn + i2 + li);
        named_bar_sync(1, FZ_THREADS);
        speculate(tid, FZ_THREADS, i2, n2);
      }
    }

    // ============================ phase 4: the refined set of evaluation j, selected by one CTA =======================
    // Evaluation j belongs to CTA j * G / E.  The CTA histograms the fine bins of all Fn scores (shared-memory atomics),
    // scans them, finds the CUT bin (the one holding rank keff - 1): bins before it are in, bins after it are out, the
    // cut bin is split by exact comparison of its few entries.  The final evaluation also needs every member's exact
    // rank: members are scattered bin by bin into a scratch array and ranked against the other entries of their bin.
    // (what is written once per layer - the score range for the next launch, the counts - is left to the CTA of
    // evaluation 0, which finishes early; to the final evaluation's first CTA when there is no such CTA)
    if (selects) fz_select<WD>(A, jme, K, keff, lay.sel_off, cta < fparts ? cta : 0, cta < fparts ? fparts : 1, cta == (fparts < G ? fparts : 0));
    if (tid == 0) FZ_STAMP(1, 6);
    if (tid == 0) FZ_CSTAMP(11);
  }
  // phases completed in this layer (every wait above has returned)
  named_bar_sync(1, FZ_THREADS);
  if (tid < FZ_NBAR) {
    unsigned n = 0;
    if (tid < FZ_MAX_G1) n = used_r1 > tid ? (unsigned)((used_r1 - 1 - tid) / (G1 / NG1) + 1) : 0u;  // (rounds, one barrier per round-slot)
    else if (tid < FZ_BAR_A) { const int s2 = tid - FZ_BAR_R2; n = used_r2 > s2 ? (unsigned)((used_r2 - 1 - s2) / G2T + 1) : 0u; }
    else n = A.has_next ? 1u : 0u;
    s_phase[tid] += n;
  }
  // what this layer wrote to shared memory with ordinary stores is ordered before the next layer's bulk copies into it
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");

}

// ---- one launch per layer step ------------------------------------------------------------------------------------------
template <int WD, int CPT>
__global__ void __launch_bounds__(FZ_BLOCK, 1) ls_fused_step_kernel(const __grid_constant__ FusedArgs A) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ FusedShared sh;
  fused_layer<WD, CPT>(A, smem, sh, true, -1);
}

// ---- one launch per token: the layers of a resident stack run back to back inside one cooperative kernel ------------
// Per-call arguments of the whole-token kernel (the per-layer arguments live in a device array built at stack creation).
struct StackCall {
  const float* x_in; float* x_out;
  const int32_t* sel_idx; const int32_t* sel_count; int sel_cap;       // selection of the first layer
  int32_t* out_idx; int32_t* out_count; uint32_t* out_mask; double* out_scores; int out_cap;  // refined set of the last layer
  int K, k_next;
  float* tr_x;       // [n_layers + 1][d]      residual entering every layer and leaving the last (nullable)
  int32_t* tr_sel;   // [n_layers + 1][tr_cap] selection entering every layer, and the final refined one (nullable)
  int32_t* tr_cnt;   // [n_layers + 1]
  int tr_cap;
};

// Layer n reads x / selection buffers of parity n & 1 and writes those of the other parity; the device-wide scratch is
// overwritten by every layer, never accumulated into, so nothing has to be cleaned between layers.  A layer boundary
// costs one grid barrier instead of a launch.
template <int WD, int CPT>
__global__ void __launch_bounds__(FZ_BLOCK, 1)
    ls_fused_stack_kernel(const FusedArgs* __restrict__ g_args, int n_layers, const __grid_constant__ StackCall C) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ FusedShared sh;
  const int G = gridDim.x, cta = blockIdx.x, tid = threadIdx.x;
  constexpr int NW = sizeof(FusedArgs) / 4;
  int known_count = -1;
  // The arguments of layer m go to sh.args[m & 1]: layer 0's here, every later layer's by the producer warp while the
  // layer before it runs (that warp leaves the layer early), so a layer starts without a round trip to global memory.
  auto fetch_args = [&](int m, int t0, int nt) {
    FusedArgs& a = sh.args[m > 0];
#pragma unroll 1
    for (int w = t0; w < NW; w += nt) reinterpret_cast<uint32_t*>(&a)[w] = __ldcg(reinterpret_cast<const uint32_t*>(&g_args[m]) + w);
  };
  auto patch_args = [&](int m) {  // (one thread, after the copy is visible to it)
    FusedArgs& a = sh.args[m > 0];
    a.K = C.K;
    a.k_next = C.k_next;
    if (m == 0) { a.x = C.x_in; a.sel_idx = C.sel_idx; a.sel_count = C.sel_count; a.sel_cap = C.sel_cap; }
    if (m == n_layers - 1) {
      a.x_out = C.x_out;
      a.next_idx = C.out_idx; a.next_count = C.out_count; a.next_mask = C.out_mask; a.next_scores = C.out_scores; a.next_cap = C.out_cap;
    }
  };
  if (n_layers > 0) {
    if (tid == 0) FZ_STAMP(1, 24);
    fetch_args(0, tid, FZ_BLOCK);
    __syncthreads();
    if (tid == 0) patch_args(0);
    __syncthreads();
    if (tid == 0) FZ_STAMP(1, 25);
  }
#pragma unroll 1
  for (int n = 0; n < n_layers; ++n) {
    const FusedArgs& A = sh.args[0];
    if (n > 0) {  // fetched while the layer before ran
#pragma unroll 1
      for (int w = tid; w < NW; w += FZ_BLOCK) reinterpret_cast<uint32_t*>(&sh.args[0])[w] = reinterpret_cast<const uint32_t*>(&sh.args[1])[w];
      __syncthreads();
    }
    if (tid == 0) FZ_STAMP(1, 26);
    if (cta == G - 1 && C.tr_x && tid < FZ_THREADS) {  // what enters this layer (x_out may overwrite x)
#pragma unroll 1
      for (int c = tid; c < A.d; c += FZ_THREADS) C.tr_x[(size_t)n * A.d + c] = __ldcg(A.x + c);
      if (C.tr_sel) {
        const int cnt = max(0, min(__ldcg(A.sel_count), min(A.sel_cap, C.tr_cap)));
#pragma unroll 1
        for (int t = tid; t < cnt; t += FZ_THREADS) C.tr_sel[(size_t)n * C.tr_cap + t] = __ldcg(A.sel_idx + t);
        if (tid == 0) C.tr_cnt[n] = cnt;
      }
    }
    fused_layer<WD, CPT>(A, smem, sh, n == 0, known_count);
    known_count = A.has_next ? min(min(A.k_next, A.Fn), A.next_cap) : -1;  // what this layer wrote to *next_count
    if (tid >= FZ_THREADS && n + 1 < n_layers) {  // the producer warp is back early: the next layer's arguments
      fetch_args(n + 1, tid - FZ_THREADS, FZ_BLOCK - FZ_THREADS);
      __syncwarp();
      if (tid == FZ_THREADS) patch_args(n + 1);
    }
    if (tid < FZ_THREADS) {
      grid_barrier(A, G);                       // layer boundary: x_out and the refined selection are visible to all
#ifdef LS_FZ_TIMING
      if (tid == 0 && cta == 0 && n < 100) {
        unsigned long long gt;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt));
        g_fz_timing[1][200 + n] = clock64();
        g_fz_timing[1][300 + n] = (long long)gt;
      }
#endif
      if (tid == 0) { sh.round = 0; sh.nsurv = 0; sh.done = 0; }  // the stream phase's counters start every layer at zero
    }
    __syncthreads();
  }
  if (tid < FZ_THREADS && n_layers > 0) {
    const FusedArgs& A = sh.args[0];  // the last layer; every CTA is past its final barrier
    if (cta == G - 1 && C.tr_x) {
#pragma unroll 1
      for (int c = tid; c < A.d; c += FZ_THREADS) C.tr_x[(size_t)n_layers * A.d + c] = __ldcg(A.x_out + c);
      if (C.tr_sel && A.has_next) {
        const int cnt = max(0, min(__ldcg(A.next_count), min(A.next_cap, C.tr_cap)));
#pragma unroll 1
        for (int t = tid; t < cnt; t += FZ_THREADS) C.tr_sel[(size_t)n_layers * C.tr_cap + t] = __ldcg(A.next_idx + t);
        if (tid == 0) C.tr_cnt[n_layers] = cnt;
      }
    }
  }
}

}  // namespace ls
