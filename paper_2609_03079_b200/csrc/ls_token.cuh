// Whole-token kernel: every layer of a resident stack for one decode token in ONE cooperative launch (batch 1).
//
// Two costs shape it.  A grid barrier costs about 2,300 SM clocks on this GPU whatever its form (one L2 round trip to
// arrive, one to see the last arrival), as long as a layer's whole weight traffic takes at full HBM speed; and with one
// CTA of sixteen warps per SM every instruction on the path that all warps execute costs four to five clocks.  So a layer
// step has FOUR barriers, the fewest the data flow allows, every phase is a handful of small rolled loops, whatever can
// be computed once (on the host, or per launch) is, and rare paths (trace export, slow selection) are out of line.
//
//   S  stream    The K priority stages of the layer (Eq. 1) run concurrently on K groups of CTAs (the output is a sum over
//                hidden neurons, Section 3.2.2, so only stage MEMBERSHIP defines the partial features of Eq. 2).  A CTA
//                owns a contiguous slice of the ranks of one stage.  Rows travel global -> shared memory as bulk copies
//                (one instruction per row, completion on a transaction barrier): gate rows first (requested as soon as
//                the selection that lists them exists), then the up and down rows of the neurons that survive the
//                activation only.  Dot products run on the 16-bit tensor cores with x cut exactly into three 16-bit
//                terms.  The CTA's partial output goes to its own row of a scratch array.  CTAs without rows establish
//                the refined sets j < K of the layer before meanwhile.
//      -- barrier 1 --
//   P1 feature   The feature is cut into slices of 32 columns, one per CTA.  The owner adds the partial outputs of every
//                stage's CTAs in a fixed order, forms x~^(j) = x~^(j-1) + dm^(j), j = 0..K (Eq. 2), writes x_out = x~^(K)
//                and multiplies the K+1 features with its slice of the next layer's predictor matrix A (fp64).
//      -- barrier 2 --
//   P2 latent    The slices' partial latents are added in a fixed order: z^(j) = A^T x~^(j) and the sums of squares.
//                Every CTA also fetches x_out for the next layer's stream phase.
//      -- barrier 3 --
//   P3 scores    Every CTA scores its share of the next layer's neurons for all K+1 evaluations (fp64; its rows of B^T
//                were copied to shared memory asynchronously while the layer streamed), stores the scores and their bin
//                under a monotone linear map.
//      -- barrier 4 --
//   P4 select    EVERY CTA reads the bins of the final evaluation, builds the histogram and its prefix sum in shared
//                memory and finds by itself the neurons whose rank falls in ITS slice of the next layer's ranks: the bins
//                that cover the slice, their members, exact comparison of the members' keys.  Nothing is exchanged, so
//                the next layer's stream phase starts without a further barrier.  The refined sets of the evaluations
//                j < K are established by the same routine (the slice being the set's last rank) during the next layer's
//                stream phase on the CTAs that have no rows, or during its P1 on CTAs that own no slice of the feature.
//
// A selection whose bins are too full for this (ties, a score range that moved) takes a slower, equally exact route
// through one CTA and an extra barrier; the decision is taken from the same histogram by every CTA alike.
//
// Every sum has a fixed order: the kernel is bitwise repeatable.  Every wait is bounded; after a timeout the CTA stops
// waiting altogether, records LS_ERR_TIMEOUT and leaves.
#pragma once
#include "ls_common.cuh"
#include "ls_topk.cuh"

namespace ls {

constexpr int WT_THREADS = 512;
constexpr int WT_WARPS = WT_THREADS / 32;
constexpr int WT_NB = 4096;        // score bins of the selection
constexpr int WT_BPT = WT_NB / WT_THREADS;
constexpr int WT_MAXK = 16;        // stages
constexpr int WT_MAXE = WT_MAXK + 1;
constexpr int WT_MAXMINE = 256;    // neurons one CTA may own in a layer
constexpr int WT_BINCAP = 64;      // fast selection: no bin reaching into the first k ranks may hold more than this
constexpr int WT_CANDCAP = 1024;   // candidates a CTA compares exactly
constexpr int WT_SL = 32;          // columns of the feature one CTA owns in P1 (one slice)
constexpr int WT_XBLK = 40;        // doubles a 32-column block of features occupies in shared memory (see wt_feat_pos)
constexpr int WT_NSTAMP = 12;      // time stamps per CTA and layer (profiling export)
constexpr long long WT_SPIN_CLOCKS = 4000LL * 1000 * 1000;  // about two seconds

// ---- feature layout for the fp64 tensor-core blocks ---------------------------------------------------------------------
// Both predictor products (A^T x~ and B^T z) are cut into blocks of 32 columns.  Lane (g, t) of a warp, g = lane / 4,
// t = lane % 4, owns the eight consecutive columns 8t .. 8t+7 of a block (ONE 16-byte load of 16-bit weights); the k-th
// m8n8k4 MMA of the block pairs column 8t + k of the weights of row g with the same column of evaluation g.  Features
// are stored so that the lane's eight doubles are contiguous and a quarter-warp's 16-byte loads fall on distinct banks:
// column c of a block at (c / 8) * 10 + c % 8, rows 8 doubles apart modulo 16.
__host__ __device__ inline int wt_feat_stride(int cols) {
  const int nb = (cols + 31) >> 5;
  return nb * WT_XBLK + ((nb & 1) ? 0 : 8);
}
// Row stride (bytes) of the B^T rows in shared memory: whole 64-byte blocks, 64 bytes modulo 128.
__host__ __device__ inline int wt_brow_bytes(int r) {
  const int b = ((r + 31) >> 5) * 64;
  return b + ((b & 127) == 64 ? 0 : 64);
}
// evaluations handled by MMA tiles of eight, the rest (at most two) by plain FMAs
__host__ __device__ inline int wt_tiles(int E) { return E <= 2 ? 0 : (E <= 10 ? 1 : 2); }
__host__ __device__ inline int wt_plain(int E) { const int p = E - 8 * wt_tiles(E); return p > 0 ? p : 0; }
__host__ __device__ inline int wt_rows(int E) { return 8 * wt_tiles(E) + wt_plain(E); }

struct WtLayer {  // one per layer of the stack (device array)
  const uint16_t* bundles; const float* b_gate; const float* b_down;
  int n_mat, F, norm, act; float eps;  // act: 0 ReLU, 1 SiLU
  // predictor of the layer this one refines (the next layer; the last layer refines itself)
  const uint16_t* At_sl; const uint16_t* Bt_pad; const float* pc;  // Bt_pad: rows of wt_brow_bytes(r) bytes, zero padded
  int r, Fn, norm_n; float eps_n;
  int per;  // ceil(Fn / CTAs): the neurons of that predictor one CTA scores (computed on the host: no division on the device)
  double* range;  // [2] {hi, scale} of the score bins, refreshed by every launch for the next one
  int* status;
};

struct WtSmem {  // byte offsets into dynamic shared memory (computed on the host)
  unsigned x_off, xs_off, part_off, xt_off, dm_off, mine_off, bits_off, pc_off, hist_off, u_off;
  // region u: A slices | B^T rows | a slice of the partial outputs (P1) or latents (P3) | raw scores | selection lists.
  // While the layer streams the whole region is the ring of the rows in flight (the predictor operands are requested
  // when the stream is over); the general top-k also takes it from its start.
  unsigned b_off, yz_off, dot_off, w_off;
  unsigned bin_off, pref_off, ckey_off, cidx_off, cbin_off;  // (from the start of region u)
  unsigned total;
};

struct WtCall {
  double inv_d;  // 1 / d
  int n_layers, d, K, k_next, piece_len, gs, ring_bytes;  // gs: CTAs per stage; ring_bytes: room for rows in shared memory
  int mma;  // d is a multiple of 16: the dot products of the stream phase run on the 16-bit tensor cores
  const float* x_in; float* x_out;
  const int32_t* sel_idx; const int32_t* sel_count; int sel_cap;
  int32_t* out_idx; int32_t* out_count; uint32_t* out_mask; double* out_scores; int out_cap;
  // scratch shared by all layers
  float* xbuf;        // [2][d]
  float* ypart;       // [G][d]
  double* zpart;      // [slices][E][rz]
  double* z;          // [E][rz]
  double* sc;         // [E][Fn]
  uint16_t* sb;       // [E][Fs], Fs = Fn rounded up to 8
  unsigned long long* kmm;   // [2 G] smallest / largest finite key of the final evaluation per CTA
  unsigned long long* cuts;  // [n_layers][E] key of the last member of every refined set
  int32_t* sellist;   // [max_sel] ranked list of the slow selection
  unsigned long long* tk_key; int32_t* tk_idx;  // [F] global candidate lists of the top-k fallback
  unsigned* bar;      // barrier counter (zeroed before the launch)
  // trace (all nullable)
  float* tr_x; int32_t* tr_sel; int32_t* tr_cnt; int tr_cap;
  float* tr_xtilde; uint32_t* tr_masks; int tr_words; long long* tr_ns;
  uint32_t* tr_survive; int32_t* tr_counts;  // (single step) selected neurons with a nonzero activation; sizes of the refined sets
  WtSmem lay;
  WtLayer one;  // the layer of a single step (used when no table of layers is given)
};

struct WtShared {
  WtLayer L[2];
  unsigned long long mbar[3];  // transaction barriers of the bulk copies: rows into the ring, the A slices, the B^T rows
  int dead;               // a wait timed out: no more waiting
  int nmine, nsurv;
  int my_lo, my_hi, keff_shared;  // this CTA's ranks [my_lo, my_hi) of a selection of keff_shared neurons
  int wcnt[WT_WARPS];
  int blo, bhi, ncand, slow, found;
  float inv_x;            // 1 / rms of the layer's input
  unsigned long long kmin, kmax;  // key range of this CTA's final scores
  double bin_hi, bin_scale;       // the score bins of the refinement in progress (all its evaluations use the same)
  double pf_thr;                  // final scores from here on: the neuron's gate row is asked into L2 (speculation)
  const unsigned char* pf_base;   // first gate row of the next layer (nullptr: no speculation)
  unsigned pf_stride, pf_bytes;
  int b_valid;                    // the B^T rows in shared memory are intact (the general top-k borrows their place)
  double inv[WT_MAXE + 7];
  double redd[WT_WARPS];
  unsigned redu[WT_WARPS];
};

// ---- small helpers -----------------------------------------------------------------------------------------------------
template <int WD>
__device__ __forceinline__ void wt_cvt8(const uint4 w, double a[8]) {
  const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    if (WD == WD_BF16) {
      a[2 * q] = (double)__uint_as_float(ww[q] << 16);
      a[2 * q + 1] = (double)__uint_as_float(ww[q] & 0xffff0000u);
    } else {
      const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&ww[q]));
      a[2 * q] = (double)f.x;
      a[2 * q + 1] = (double)f.y;
    }
  }
}
__device__ __forceinline__ void wt_load8d(const double* p, double v[8]) {  // 16-byte aligned shared memory
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const double2 t = *reinterpret_cast<const double2*>(p + 2 * q);
    v[2 * q] = t.x;
    v[2 * q + 1] = t.y;
  }
}
// c (8 rows x 8 evaluations, this lane's two elements) += one 32-column block
__device__ __forceinline__ void wt_mma_block(double (&c)[2], const double a[8], const double b[8]) {
#pragma unroll
  for (int k = 0; k < 8; ++k)
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                 : "+d"(c[0]), "+d"(c[1]) : "d"(a[k]), "d"(b[k]));
}
__device__ __forceinline__ double wt_dot8(const double a[8], const double b[8], double acc) {
#pragma unroll
  for (int k = 0; k < 8; ++k) acc = fma(a[k], b[k], acc);
  return acc;
}
// 1 / sqrt(a) in double precision from the hardware approximation and two Newton steps (a few ulp; a full-precision
// divide and square root would be a few hundred instructions where they stand).
__device__ __forceinline__ double wt_rsqrt(double a) {
  double y;
  asm("rsqrt.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(a));
  if (a > 0.0 && a < 1.0e300) {
#pragma unroll
    for (int it = 0; it < 2; ++it) {
      const double h = 0.5 * a * y;
      y = fma(y, fma(-h, y, 0.5), y);
    }
  }
  return y;
}
__device__ __noinline__ void wt_stamp(const WtCall& C, int n, int slot) {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  C.tr_ns[((size_t)n * gridDim.x + blockIdx.x) * WT_NSTAMP + slot] = (long long)t;
}
__device__ __forceinline__ void wt_cp_async16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void wt_cp_async_wait() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// Barrier among all CTAs of the cooperatively launched grid.  The counter is zeroed before the launch and only grows:
// the e-th barrier completes when it reaches e * G.  Arrival is a release (a reduction: nothing comes back), the poll an
// acquire.
__device__ __noinline__ void wt_poll(const WtCall& C, WtShared& sh, unsigned target) {
  asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(C.bar) : "memory");
  const long long t0 = clock64();
  for (;;) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(C.bar) : "memory");
    if (v >= target) return;
    if (clock64() - t0 > WT_SPIN_CLOCKS) break;
  }
  sh.dead = 1;
  set_status(sh.L[0].status, ST_TIMEOUT);
}
__device__ __forceinline__ void wt_grid_sync(const WtCall& C, WtShared& sh, unsigned target) {
  __syncthreads();
  if (threadIdx.x == 0 && !sh.dead) wt_poll(C, sh, target);
  __syncthreads();
}

// This CTA's slice [lo, hi) of the ranks of a selection of `count` neurons run in K stages on groups of `gs` CTAs.
__device__ __forceinline__ void wt_share(int count, int K, int gs, int cta, int& lo, int& hi) {
  const int c = cta / gs;
  lo = hi = 0;
  if (c >= K || count <= 0) return;
  const int m = (count + K - 1) / K;
  const int s_lo = min(count, c * m), s_hi = min(count, (c + 1) * m);
  const int per = (m + gs - 1) / gs;
  lo = min(s_hi, s_lo + (cta - c * gs) * per);
  hi = min(s_hi, lo + per);
}

// ---- S: gate rows, survivors, up and down rows -----------------------------------------------------------------------
// Rows travel global -> shared memory as bulk copies (one instruction per row, issued by one lane; the copy engine moves
// the bytes and counts them off on a transaction barrier in shared memory), all in flight at once, no registers held;
// every computation is a small rolled loop over shared memory.
__device__ __forceinline__ uint32_t wt_saddr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void wt_mbar_init(unsigned long long* b, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(wt_saddr(b)), "r"(count) : "memory");
}
// One arrival that also announces `bytes` bytes of copies to come.
__device__ __forceinline__ void wt_mbar_expect(unsigned long long* b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(wt_saddr(b)), "r"(bytes) : "memory");
}
// Linear copy global -> shared memory (both 16-byte aligned, a multiple of 16 bytes, no multicast).
__device__ __forceinline__ void wt_bulk_load(void* dst, const void* src, uint32_t bytes, unsigned long long* b) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(wt_saddr(dst)), "l"(src),
               "r"(bytes), "r"(wt_saddr(b))
               : "memory");
}
// Shared memory that ordinary loads and stores touched is handed to the copy engine.
__device__ __forceinline__ void wt_fence_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// Wait (bounded) for the phase of parity `parity` to complete; on a timeout the CTA stops waiting for anything.
__device__ __noinline__ void wt_mbar_wait(WtShared& sh, unsigned long long* b, uint32_t parity) {
  if (sh.dead) return;
  const long long t0 = clock64();
  for (;;) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok)
                 : "r"(wt_saddr(b)), "r"(parity)
                 : "memory");
    if (ok) return;
    if (clock64() - t0 > WT_SPIN_CLOCKS) break;
  }
  sh.dead = 1;
  set_status(sh.L[0].status, ST_TIMEOUT);
}

// `nrow` rows of `bytes` bytes each, row i from src_of(i), to ring + i * stride: warp w's first lane issues
// the rows w, w + 16, ... and arrives once on the barrier (16 arrivals complete a phase) with the bytes it asked for.
template <class SrcFn>
__device__ __forceinline__ void wt_request_rows(unsigned long long* bar, unsigned char* ring, int stride, int nrow, int bytes, SrcFn src_of) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane != 0) return;
  uint32_t total = 0;
#pragma unroll 1
  for (int i = warp; i < nrow; i += WT_WARPS) total += src_of(i) != nullptr ? bytes : 0;
  wt_fence_async();
  wt_mbar_expect(bar, total);
#pragma unroll 1
  for (int i = warp; i < nrow; i += WT_WARPS) {
    const unsigned char* src = src_of(i);
    if (src != nullptr) wt_bulk_load(ring + (size_t)i * stride, src, bytes, bar);
  }
}

// Four consecutive 16-bit weights widened exactly to fp32.
template <int WD>
__device__ __forceinline__ void wt_unpack4(const uint2& v, float (&f)[4]) {
  if (WD == WD_BF16) {
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
  } else {
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&v.x)), b = __half22float2(*reinterpret_cast<const __half2*>(&v.y));
    f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y;
  }
}

// Dot products of `nrow` rows in the ring (row i at ring + i * stride) with x: out[4 i + p] = partial sum of quarter p of
// row i.  Warp (p, q) = (warp % 4, warp / 4) takes quarter p of the rows q, q + 4, ...; its part of x stays in registers
// across the rows (x is fp32, twice the bytes of a row: reading it once per row would double the shared-memory traffic).
// A lane owns columns 4 lane .. 4 lane + 3 of each run of 128 columns: every load is free of bank conflicts.
template <int WD>
__device__ __noinline__ void wt_ring_dots(const unsigned char* ring, int stride, int nrow, const float* s_x, int d, int piece_len, float* out) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int p = warp & 3, q = warp >> 2;
  const int c_lo = min(d, p * piece_len), c_hi = min(d, c_lo + piece_len);
  if (q >= nrow) return;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};  // rows r0, r0 + 4, r0 + 8, r0 + 12
#pragma unroll 1
  for (int r0 = q; r0 < nrow; r0 += 16) {
#pragma unroll 1
    for (int cb = c_lo + lane * 4; cb < c_hi; cb += 1024) {
      float4 xv[8];
#pragma unroll
      for (int it = 0; it < 8; ++it) {
        const int c = cb + it * 128;
        xv[it] = c < c_hi ? *reinterpret_cast<const float4*>(s_x + c) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int r = r0 + 4 * j;
        if (r < nrow) {
          const uint16_t* w = reinterpret_cast<const uint16_t*>(ring + (size_t)r * stride);
          float a0 = acc[j], a1 = 0.f;
#pragma unroll
          for (int it = 0; it < 8; it += 2) {
            const int c = cb + it * 128;
            float f[4], g[4];
            if (c < c_hi) {
              wt_unpack4<WD>(*reinterpret_cast<const uint2*>(w + c), f);
              a0 = fmaf(f[0], xv[it].x, a0); a0 = fmaf(f[1], xv[it].y, a0); a0 = fmaf(f[2], xv[it].z, a0); a0 = fmaf(f[3], xv[it].w, a0);
            }
            if (c + 128 < c_hi) {
              wt_unpack4<WD>(*reinterpret_cast<const uint2*>(w + c + 128), g);
              a1 = fmaf(g[0], xv[it + 1].x, a1); a1 = fmaf(g[1], xv[it + 1].y, a1); a1 = fmaf(g[2], xv[it + 1].z, a1); a1 = fmaf(g[3], xv[it + 1].w, a1);
            }
          }
          acc[j] = a0 + a1;
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int r = r0 + 4 * j;
      if (r < nrow) {  // (uniform over the warp)
        const float v = warp_sum(acc[j]);
        if (lane == 0) out[4 * r + p] = v;
      }
      acc[j] = 0.f;
    }
  }
}

// ---- the same dot products on the 16-bit tensor cores ---------------------------------------------------------------------
// A row-times-x product has one output column, but the kernel is bound by instructions, not by arithmetic, and one
// m16n8k16 MMA replaces 16 x 16 multiply-adds of 32 lanes.  Exactness: x (fp32) is cut into three 16-bit terms,
// x = t0 + 2^-S t1 + 2^-2S t2 (S = 8 for bf16, 11 for fp16; every cut is an exact fp32 subtraction), which become three
// columns of the B operand; products of 16-bit values are exact in the fp32 accumulator, so the result differs from the
// fp32 FMA loop only by the order and rounding of the additions.
constexpr int WT_MMA_ROWS = 32;  // rows per batch (two m-tiles)

template <int WD>
__device__ __forceinline__ uint32_t wt_to16(float v) {
  if (WD == WD_BF16) {
    unsigned short h;
    asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(h) : "f"(v));
    return (uint32_t)h;
  }
  return (uint32_t)__half_as_ushort(__float2half_rn(v));
}
template <int WD>
__device__ __forceinline__ float wt_from16(uint32_t h) {
  if (WD == WD_BF16) return __uint_as_float(h << 16);
  return __half2float(__ushort_as_half((unsigned short)h));
}
// Four consecutive components of x (c a multiple of 4) to the fp32 copy and to the three 16-bit terms, the latter in the
// order the MMA's B operand wants: [k-step of 16][term][t = 0..3][x[2t], x[2t+1], x[8+2t], x[8+2t+1]].
template <int WD>
__device__ __forceinline__ void wt_store_x4(float* s_x, uint16_t* s_xs, int c, const float4& v) {
  *reinterpret_cast<float4*>(s_x + c) = v;
  if (s_xs == nullptr) return;
  constexpr float SC = WD == WD_BF16 ? 256.f : 2048.f;
  const float x[4] = {v.x, v.y, v.z, v.w};
  uint32_t term[3][4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const uint32_t h0 = wt_to16<WD>(x[e]);
    const float r1 = (x[e] - wt_from16<WD>(h0)) * SC;
    const uint32_t h1 = wt_to16<WD>(r1);
    const float r2 = (r1 - wt_from16<WD>(h1)) * SC;
    term[0][e] = h0; term[1][e] = h1; term[2][e] = wt_to16<WD>(r2);
  }
  const int ks = c >> 4, w = c & 15, t0 = (w & 7) >> 1, j0 = (w >> 3) * 2;
#pragma unroll
  for (int g = 0; g < 3; ++g) {
    uint16_t* base = s_xs + ((ks * 3 + g) * 4 + t0) * 4 + j0;
    *reinterpret_cast<uint32_t*>(base) = term[g][0] | (term[g][1] << 16);
    *reinterpret_cast<uint32_t*>(base + 4) = term[g][2] | (term[g][3] << 16);
  }
}

// Dot products of `nrow` <= 32 rows in the ring (row i at ring + i * stride, stride = 16 mod 128 bytes so that the matrix
// loads are free of bank conflicts) with x: warp w takes the k-steps [w * per, (w + 1) * per) of every m-tile and leaves
// its partial sums in part[w][row]; the caller adds the sixteen partials in a fixed order.
template <int WD>
__device__ __noinline__ void wt_ring_mma(const unsigned char* ring, int stride, int nrow, const uint16_t* s_xs, int d, float* part) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, t = lane & 3;
  const int nks = d >> 4, per = (nks + WT_WARPS - 1) / WT_WARPS;
  const int k0 = min(nks, warp * per), k1 = min(nks, k0 + per);
  constexpr float M1 = WD == WD_BF16 ? 1.f / 256.f : 1.f / 2048.f;
  const int n_mt = (nrow + 15) >> 4;
#pragma unroll 1
  for (int mt = 0; mt < n_mt; ++mt) {
    // this lane's row of the four 8 x 8 matrices of an A tile: matrix lane / 8 = (rows 0-7 | 8-15) x (k 0-7 | 8-15)
    const int row = min(nrow - 1, mt * 16 + ((lane >> 3) & 1) * 8 + (lane & 7));
    uint32_t a_addr = wt_saddr(ring + (size_t)row * stride) + (uint32_t)(k0 * 32 + (lane >> 4) * 16);
    const uint16_t* xb = s_xs + ((k0 * 3 + g) * 4 + t) * 4;
    float c0 = 0.f, c1 = 0.f, c2 = 0.f, c3 = 0.f;
#pragma unroll 2
    for (int ks = k0; ks < k1; ++ks, a_addr += 32, xb += 48) {
      uint32_t a0, a1, a2, a3, b0 = 0u, b1 = 0u;
      asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3) : "r"(a_addr));
      if (g < 3) {
        const uint2 b = *reinterpret_cast<const uint2*>(xb);
        b0 = b.x; b1 = b.y;
      }
      if (WD == WD_BF16)
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c0), "+f"(c1), "+f"(c2), "+f"(c3) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
      else
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c0), "+f"(c1), "+f"(c2), "+f"(c3) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    }
    // columns 0, 1, 2 of the tile are the three terms: lane t = 0 holds columns 0 and 1, lane t = 1 column 2
    float lo8 = t == 0 ? c0 + M1 * c1 : (M1 * M1) * c0, hi8 = t == 0 ? c2 + M1 * c3 : (M1 * M1) * c2;
    lo8 += __shfl_down_sync(0xffffffffu, lo8, 1);
    hi8 += __shfl_down_sync(0xffffffffu, hi8, 1);
    if (t == 0) {
      part[warp * WT_MMA_ROWS + mt * 16 + g] = lo8;
      part[warp * WT_MMA_ROWS + mt * 16 + g + 8] = hi8;
    }
  }
}
// (after a __syncthreads) the sixteen partial sums of row i, added in a fixed order, as the first of the row's four places
__device__ __forceinline__ void wt_fold_parts(const float* part, int nrow, float* out) {
  const int i = threadIdx.x;
  if (i < nrow) {
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < WT_WARPS; ++w) v += part[w * WT_MMA_ROWS + i];
    *reinterpret_cast<float4*>(out + 4 * i) = make_float4(v, 0.f, 0.f, 0.f);
  }
}

// This CTA's slices of the next layer's predictor matrix A and its rows of B^T (stored padded, so both are plain linear
// copies: bulk copies by thread 0, each on a barrier of its own that completes exactly one phase per layer, also when
// there is nothing to copy) and its score offsets (4-byte asynchronous copies): needed in P1 and P3.  Called after a
// __syncthreads that ends the ring's use.
__device__ __forceinline__ void wt_fetch_predictor(const WtCall& C, WtShared& sh, const WtLayer& L, unsigned char* smem) {
  const int tid = threadIdx.x, G = gridDim.x, d = C.d;
  const int nsl = (d + 31) >> 5, slice_b = L.r * 64;  // bytes per slice: 32 columns of r 16-bit entries
  const int per = L.per, n0 = min(L.Fn, (int)blockIdx.x * per), n1 = min(L.Fn, n0 + per);
  if (tid == 0) {
    unsigned char* s_a = smem + C.lay.u_off;
    wt_fence_async();
    uint32_t a_bytes = 0;
#pragma unroll 1
    for (int s = blockIdx.x; s < nsl; s += G) a_bytes += slice_b;
    wt_mbar_expect(&sh.mbar[1], a_bytes);
    if (slice_b > 0) {
#pragma unroll 1
      for (int s = blockIdx.x, si = 0; s < nsl; s += G, ++si)
        wt_bulk_load(s_a + (size_t)si * slice_b, reinterpret_cast<const unsigned char*>(L.At_sl) + (size_t)s * slice_b, slice_b, &sh.mbar[1]);
    }
  }
  if (tid == 32) {  // (a thread of another warp: the two requests go out side by side)
    wt_fence_async();
    const int RB = wt_brow_bytes(L.r);
    const uint32_t b_bytes = (uint32_t)(((n1 - n0 + 7) >> 3) * 8) * RB;
    wt_mbar_expect(&sh.mbar[2], b_bytes);
    unsigned char* s_b = smem + C.lay.u_off + C.lay.b_off;
    const unsigned char* src = reinterpret_cast<const unsigned char*>(L.Bt_pad) + (size_t)n0 * RB;
#pragma unroll 1
    for (uint32_t o = 0; o < b_bytes; o += 32768u) wt_bulk_load(s_b + o, src + o, min(32768u, b_bytes - o), &sh.mbar[2]);
  }
  float* s_pc = reinterpret_cast<float*>(smem + C.lay.pc_off);
#pragma unroll 1
  for (int i = tid; i < n1 - n0; i += WT_THREADS) {
    if (L.pc) asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(s_pc + i)), "l"(L.pc + n0 + i) : "memory");
    else s_pc[i] = 0.f;
  }
}

// The same rows of B^T once more, by ordinary asynchronous copies (after a degenerate selection borrowed their place).
__device__ __noinline__ void wt_refetch_b(const WtCall& C, const WtLayer& L, unsigned char* smem) {
  const int per = L.per, n0 = min(L.Fn, (int)blockIdx.x * per), n1 = min(L.Fn, n0 + per);
  const int RB = wt_brow_bytes(L.r);
  const int npieces = (((n1 - n0 + 7) >> 3) * 8) * (RB >> 4);
  unsigned char* s_b = smem + C.lay.u_off + C.lay.b_off;
  const unsigned char* src = reinterpret_cast<const unsigned char*>(L.Bt_pad) + (size_t)n0 * RB;
#pragma unroll 1
  for (int i = threadIdx.x; i < npieces; i += WT_THREADS) wt_cp_async16(s_b + i * 16, src + (size_t)i * 16);
  wt_cp_async_wait();
}

template <int WD>
__device__ __noinline__ void wt_score_evals(const WtCall& C, WtShared& sh, const WtLayer& L, int e0, int ne, bool last);

// Requests the gate rows of this CTA's neurons g0, g0 + 1, ... (as many as a ring batch holds) of layer L.  Called by the
// stream phase, and for the first batch already at the end of the selection that produced the list, so that the rows
// travel while the layer's bookkeeping is done.
__device__ __forceinline__ void wt_request_gate(const WtCall& C, WtShared& sh, const WtLayer& L, unsigned char* smem, int g0, int nmine) {
  const int* s_mine = reinterpret_cast<const int*>(smem + C.lay.mine_off);
  const int row_b = C.d * 2, gstride = row_b + 16;
  const int cap_g = min(WT_MMA_ROWS, C.ring_bytes / gstride);
  const size_t bundle_b = (size_t)L.n_mat * row_b;
  const unsigned char* wbase = reinterpret_cast<const unsigned char*>(L.bundles);
  wt_request_rows(&sh.mbar[0], smem + C.lay.u_off, gstride, min(cap_g, nmine - g0), row_b, [&](int i) -> const unsigned char* {
    const int v = s_mine[g0 + i];
    return v >= 0 ? wbase + (size_t)v * bundle_b : nullptr;
  });
}

template <int WD>
__device__ __forceinline__ void wt_stream(const WtCall& C, WtShared& sh, const WtLayer& L, unsigned char* smem, bool active, uint32_t& ring_phase,
                                          bool first_requested) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int d = C.d;
  const float* s_x = reinterpret_cast<const float*>(smem + C.lay.x_off);
  int* s_mine = reinterpret_cast<int*>(smem + C.lay.mine_off);           // [256] neurons of this CTA, rank order
  float* s_gsum = reinterpret_cast<float*>(s_mine + WT_MAXMINE);         // [256][4] partial dot products
  int* s_sidx = reinterpret_cast<int*>(s_gsum + 4 * WT_MAXMINE);         // [256] survivors
  float* s_sact = reinterpret_cast<float*>(s_sidx + WT_MAXMINE);         // [256] their relu(g), then their activation
  unsigned char* ring = smem + C.lay.u_off;  // (nothing else in region u is alive while the layer streams)
  const int nmine = sh.nmine;
  const float inv = sh.inv_x;
  const int row_b = d * 2;
  const size_t bundle_b = (size_t)L.n_mat * row_b;
  const unsigned char* wbase = reinterpret_cast<const unsigned char*>(L.bundles);
  const bool gated = L.n_mat == 3;

  // gate bias of "my" neuron (used after the dot products; the load is in flight meanwhile)
  int my_idx = -1;
  float my_b = 0.f;
  if (tid < nmine) {
    my_idx = s_mine[tid];
    if (my_idx >= 0 && L.b_gate) my_b = __ldg(L.b_gate + my_idx);
  }
  const uint16_t* s_xs = reinterpret_cast<const uint16_t*>(smem + C.lay.xs_off);
  float* s_part = reinterpret_cast<float*>(smem + C.lay.part_off);
  // gate rows: as many at a time as the ring holds (all of them in the usual case); rows sit 16 bytes apart modulo 128
  const int gstride = row_b + 16;
  const int cap_g = min(WT_MMA_ROWS, C.ring_bytes / gstride);
#pragma unroll 1
  for (int g0 = 0; g0 < nmine; g0 += cap_g) {
    const int ng = min(cap_g, nmine - g0);
    if (g0 > 0 || !first_requested) wt_request_gate(C, sh, L, smem, g0, nmine);
    wt_mbar_wait(sh, &sh.mbar[0], ring_phase);
    ring_phase ^= 1u;
    if (C.mma) {
      wt_ring_mma<WD>(ring, gstride, ng, s_xs, d, s_part);
      __syncthreads();
      wt_fold_parts(s_part, ng, s_gsum + 4 * g0);
    } else {
      wt_ring_dots<WD>(ring, gstride, ng, s_x, d, C.piece_len, s_gsum + 4 * g0);
    }
    __syncthreads();
  }
  // activation of the gate branch and the ordered list of survivors (ReLU: a_i = relu(g_i) u_i, so g_i <= 0 needs no other
  // row; SiLU has no zeros: every selected neuron goes on)
  {
    float g = 0.f;
    bool sv = false;
    if (my_idx >= 0) {
      const float4 s4 = *reinterpret_cast<const float4*>(s_gsum + tid * 4);
      g = ((s4.x + s4.y) + (s4.z + s4.w)) * inv + my_b;
      sv = g > 0.f;
      if (L.act != 0) { g = g / (1.f + expf(-g)); sv = true; }
    }
    const unsigned m = __ballot_sync(0xffffffffu, sv);
    if (lane == 0) sh.wcnt[warp] = __popc(m);
    __syncthreads();
    int off = __popc(m & ((1u << lane) - 1u)), tot = 0;
#pragma unroll 1
    for (int w = 0; w < WT_MAXMINE / 32; ++w) {
      const int c = sh.wcnt[w];
      if (w < warp) off += c;
      tot += c;
    }
    if (sv) { s_sidx[off] = my_idx; s_sact[off] = g; }
    if (tid == 0) sh.nsurv = tot;
  }
  __syncthreads();
  const int nsurv = sh.nsurv;
  // survivors: the rest of their bundles (up and down rows are adjacent: one linear copy), as many as the ring holds
  const int rest_b = (L.n_mat - 1) * row_b;
  const int rstride = rest_b + 16;
  const int cap_s = min(WT_MMA_ROWS, C.ring_bytes / rstride);
  float acc8[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};  // (d <= 4096: one column group per thread; beyond: see below)
  float* yp = C.ypart + (size_t)blockIdx.x * d;
  const bool wide = d > WT_THREADS * 8;
  if (wide && active) {
#pragma unroll 1
    for (int c = tid * 4; c < d; c += WT_THREADS * 4) __stcg(reinterpret_cast<float4*>(yp + c), make_float4(0.f, 0.f, 0.f, 0.f));
  }
#pragma unroll 1
  for (int b0 = 0; b0 < nsurv; b0 += cap_s) {
    const int nb = min(cap_s, nsurv - b0);
    wt_request_rows(&sh.mbar[0], ring, rstride, nb, rest_b, [&](int i) -> const unsigned char* { return wbase + (size_t)s_sidx[b0 + i] * bundle_b + row_b; });
    wt_mbar_wait(sh, &sh.mbar[0], ring_phase);
    ring_phase ^= 1u;
    if (gated) {
      if (C.mma) {
        wt_ring_mma<WD>(ring, rstride, nb, s_xs, d, s_part);
        __syncthreads();
        wt_fold_parts(s_part, nb, s_gsum);
      } else {
        wt_ring_dots<WD>(ring, rstride, nb, s_x, d, C.piece_len, s_gsum);
      }
      __syncthreads();
      if (tid < nb) {
        const float4 u4 = *reinterpret_cast<const float4*>(s_gsum + tid * 4);
        s_sact[b0 + tid] *= ((u4.x + u4.y) + (u4.z + u4.w)) * inv;
      }
      __syncthreads();
    }
    if (C.tr_survive && tid < nb && s_sact[b0 + tid] != 0.f) atomicOr(C.tr_survive + (s_sidx[b0 + tid] >> 5), 1u << (s_sidx[b0 + tid] & 31));
    // down rows scaled into the partial output: every thread owns eight columns
    const unsigned char* dn = ring + (rest_b - row_b);
#pragma unroll 1
    for (int col = tid * 8; col < d; col += WT_THREADS * 8) {
      float a8[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) a8[e] = wide ? 0.f : acc8[e];
#pragma unroll 1
      for (int s0 = 0; s0 < nb; ++s0) {
        const float a = s_sact[b0 + s0];
        float f[8];
        unpack8<WD>(*reinterpret_cast<const uint4*>(dn + (size_t)s0 * rstride + col * 2), f);
#pragma unroll
        for (int e = 0; e < 8; ++e) a8[e] = fmaf(a, f[e], a8[e]);
      }
      if (wide) {  // (more than 4096 columns: the partial output is accumulated in its global row, which this CTA alone touches)
        if (active) {
          float4* o = reinterpret_cast<float4*>(yp + col);
          const float4 p0 = __ldcg(o), p1 = __ldcg(o + 1);
          __stcg(o, make_float4(p0.x + a8[0], p0.y + a8[1], p0.z + a8[2], p0.w + a8[3]));
          __stcg(o + 1, make_float4(p1.x + a8[4], p1.y + a8[5], p1.z + a8[6], p1.w + a8[7]));
        }
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) acc8[e] = a8[e];
      }
    }
    __syncthreads();
  }
  if (active && !wide && tid * 8 < d) {
    __stcg(reinterpret_cast<float4*>(yp + tid * 8), make_float4(acc8[0], acc8[1], acc8[2], acc8[3]));
    __stcg(reinterpret_cast<float4*>(yp + tid * 8 + 4), make_float4(acc8[4], acc8[5], acc8[6], acc8[7]));
  }
  wt_fetch_predictor(C, sh, L, smem);
}

// ---- P1: stage sums, partial residual features, x_out, partial latents of this CTA's slices ----------------------------
__device__ __noinline__ void wt_trace_feature(const WtCall& C, int n, int e, int E, int col, float xt) {
  C.tr_xtilde[((size_t)n * E + e) * C.d + col] = xt;
}
template <int WD>
__device__ __forceinline__ void wt_feature(const WtCall& C, WtShared& sh, const WtLayer& L, unsigned char* smem, int n, float* x_out,
                                           int E, int rz) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const int d = C.d, K = C.K, G = gridDim.x, r = L.r;
  const float* s_x = reinterpret_cast<const float*>(smem + C.lay.x_off);
  double* s_xt = reinterpret_cast<double*>(smem + C.lay.xt_off);  // [rows][WT_XBLK]
  float* s_dm = reinterpret_cast<float*>(smem + C.lay.dm_off);    // [16 warps][32] partial stage sums
  float* s_y = reinterpret_cast<float*>(smem + C.lay.u_off + C.lay.yz_off);  // [active CTAs][32] this slice of every partial output
  const uint16_t* s_a = reinterpret_cast<const uint16_t*>(smem + C.lay.u_off);
  const int nsl = (d + 31) >> 5, n_act = C.gs * K;
  const int ntile = wt_tiles(E), nplain = wt_plain(E), rows = wt_rows(E);
  const int pos = (lane >> 3) * 10 + (lane & 7);
  // warps per stage and the rows (CTAs) of a stage one warp adds
  const int wps = max(1, WT_WARPS / K), rpw = (C.gs + wps - 1) / wps;
#pragma unroll 1
  for (int s = blockIdx.x, si = 0; s < nsl; s += G, ++si) {
    const int col = 32 * s + lane;
    // this slice of every CTA's partial output: 128 bytes per CTA, eight lanes each
    if (lane < 8) {
      const float* yp = C.ypart + 32 * s + lane * 4;
#pragma unroll 1
      for (int row = warp; row < n_act; row += WT_WARPS) wt_cp_async16(s_y + row * 32 + lane * 4, yp + (size_t)row * d);
    }
    wt_cp_async_wait();
    wt_mbar_wait(sh, &sh.mbar[1], (uint32_t)n & 1u);  // (this CTA's slices of A, requested at the end of S)
    __syncthreads();
    {
      const int c = warp / wps, h = warp - c * wps;
      float a = 0.f;
      if (c < K) {
        const int g1 = min(C.gs, (h + 1) * rpw);
#pragma unroll 1
        for (int q = h * rpw; q < g1; ++q) a += s_y[(c * C.gs + q) * 32 + lane];
      }
      s_dm[warp * 32 + lane] = a;
    }
    __syncthreads();
    if (warp == 0) {
      // stage sums (fixed order), then x~^(e) = x~^(e-1) + dm^(e) (Eq. 2)
      float xt = 0.f;
      if (col < d) xt = s_x[col] + (L.b_down ? __ldg(L.b_down + col) : 0.f);
      s_xt[pos] = (double)xt;
#pragma unroll 1
      for (int c = 0; c < K; ++c) {
        float dm = 0.f;
#pragma unroll 1
        for (int h = 0; h < wps; ++h) dm += s_dm[(c * wps + h) * 32 + lane];
        xt += dm;
        s_xt[(c + 1) * WT_XBLK + pos] = (double)xt;
      }
#pragma unroll 1
      for (int e = E; e < rows; ++e) s_xt[e * WT_XBLK + pos] = 0.0;
      if (col < d) {
        __stcg(x_out + col, xt);
        if (C.tr_x) C.tr_x[(size_t)(n + 1) * d + col] = xt;
      }
    }
    __syncthreads();
    // sums of squares of every evaluation's slice (a warp each); trace
#pragma unroll 1
    for (int e = warp; e < E; e += WT_WARPS) {
      const double v = s_xt[e * WT_XBLK + pos];
      const double sq = warp_sum(v * v);
      if (lane == 0) __stcg(C.zpart + ((size_t)s * E + e) * rz + r, sq);
      if (C.tr_xtilde && col < d) wt_trace_feature(C, n, e, E, col, (float)v);
    }
    // partial latents: m-tiles of eight rows of A^T (the slice holds [r][32] 16-bit weights)
    const uint16_t* a_sl = s_a + (size_t)si * r * 32 + 8 * t;
    double f0[8], f1[8];
    wt_load8d(s_xt + g * WT_XBLK + t * 10, f0);
    if (ntile > 1) wt_load8d(s_xt + (8 + g) * WT_XBLK + t * 10, f1);
    double* zs = C.zpart + (size_t)s * E * rz;
#pragma unroll 1
    for (int mt = warp; mt < (r >> 3); mt += WT_WARPS) {
      const int l = 8 * mt + g;
      double a[8];
      wt_cvt8<WD>(*reinterpret_cast<const uint4*>(a_sl + l * 32), a);
      double* zp = zs + l;
      if (ntile > 0) {
        double c[2] = {0.0, 0.0};
        wt_mma_block(c, a, f0);
        if (2 * t < E) __stcg(zp + (2 * t) * rz, c[0]);
        if (2 * t + 1 < E) __stcg(zp + (2 * t + 1) * rz, c[1]);
      }
      if (ntile > 1) {
        double c[2] = {0.0, 0.0};
        wt_mma_block(c, a, f1);
        if (8 + 2 * t < E) __stcg(zp + (8 + 2 * t) * rz, c[0]);
        if (8 + 2 * t + 1 < E) __stcg(zp + (8 + 2 * t + 1) * rz, c[1]);
      }
#pragma unroll 1
      for (int q = 0; q < nplain; ++q) {
        const int e = 8 * ntile + q;
        double f[8];
        wt_load8d(s_xt + e * WT_XBLK + t * 10, f);
        double pa = wt_dot8(a, f, 0.0);
        pa += __shfl_xor_sync(0xffffffffu, pa, 1);
        pa += __shfl_xor_sync(0xffffffffu, pa, 2);
        if (t == 0) __stcg(zp + e * rz, pa);
      }
    }
    __syncthreads();
  }
}

// ---- P2: latents and sums of squares from the slices' partials ---------------------------------------------------------
__device__ __forceinline__ void wt_latent_sums(const WtCall& C, int r, int E, int rz) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, sg = lane >> 2, v = lane & 3;
  const int nsl = (C.d + 31) >> 5, ngrp = rz >> 2, units = E * ngrp, G = gridDim.x;
  const int step = E * rz;
#pragma unroll 1
  for (int u = warp * G + blockIdx.x; u < units; u += G * WT_WARPS) {  // (the units are dealt over all CTAs)
    const int e = u / ngrp, l = 4 * (u - e * ngrp) + v;
    double a = 0.0;
    if (l <= r) {
      const double* zp = C.zpart + e * rz + l + (size_t)sg * step;
#pragma unroll 1
      for (int s0 = sg; s0 < nsl; s0 += 128, zp += (size_t)128 * step) {  // sixteen partials in flight, added in order
        double v[16];
#pragma unroll
        for (int q = 0; q < 16; ++q) v[q] = s0 + 8 * q < nsl ? __ldcg(zp + (size_t)(8 * q) * step) : 0.0;
#pragma unroll
        for (int q = 0; q < 16; ++q) a += v[q];
      }
    }
    a += __shfl_xor_sync(0xffffffffu, a, 4);
    a += __shfl_xor_sync(0xffffffffu, a, 8);
    a += __shfl_xor_sync(0xffffffffu, a, 16);
    if (sg == 0 && l <= r) __stcg(C.z + e * rz + l, a);
  }
}

// ---- P3: scores of this CTA's share of the next layer's neurons, all evaluations ---------------------------------------
__device__ __forceinline__ int wt_bin_of(double s, double hi, double scale) {
  return (int)fmin(fmax((hi - s) * scale, 0.0), (double)(WT_NB - 1));
}

// Evaluations e0 .. e0 + ne - 1 of the refinement described by L: scores, bins (and, for the final evaluation, the key
// range this CTA saw).
template <int WD>
__device__ __noinline__ void wt_score_evals(const WtCall& C, WtShared& sh, const WtLayer& L, int e0, int ne, bool last) {
  extern __shared__ __align__(128) unsigned char wt_smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const int r = L.r, Fn = L.Fn, K = C.K;
  const int rz = (r + 4) & ~3;
  double* s_z = reinterpret_cast<double*>(wt_smem + C.lay.u_off + C.lay.yz_off);
  double* s_dot = reinterpret_cast<double*>(wt_smem + C.lay.u_off + C.lay.dot_off);  // [ne][per8] raw dot products
  const float* s_pc = reinterpret_cast<const float*>(wt_smem + C.lay.pc_off);
  const unsigned char* s_b = wt_smem + C.lay.u_off + C.lay.b_off;
  const int RS = wt_feat_stride(r), RB = wt_brow_bytes(r);
  const int ntile = wt_tiles(ne), nplain = wt_plain(ne), rows = wt_rows(ne);
  const int nblk = (r + 31) >> 5;
  const int per = L.per, n0 = min(Fn, (int)blockIdx.x * per), n1 = min(Fn, n0 + per);
  const int n_mt = (n1 - n0 + 7) >> 3, per8 = n_mt * 8;
  if (ne <= 0) return;
  {
    const int bv = sh.b_valid;
    __syncthreads();
    if (!bv) {  // (a general top-k borrowed the place of the B^T rows: fetch them again)
      wt_refetch_b(C, L, wt_smem);
      if (tid == 0) sh.b_valid = 1;
      __syncthreads();
    }
  }
  // latents to shared memory in the block layout, two at a time (pairs stay adjacent in it); 1 / rms of every evaluation
  if ((r & 31) || rows > ne) {  // (a rank that does not fill its last block, evaluations that do not fill their tile: zeros there)
#pragma unroll 1
    for (int i = tid; i < rows * RS; i += WT_THREADS) s_z[i] = 0.0;
    __syncthreads();
  }
  const double ss = tid < ne ? __ldcg(C.z + (e0 + tid) * rz + r) : 0.0;  // (requested before the latents: one round trip, not two)
#pragma unroll 1
  for (int e = warp; e < ne; e += WT_WARPS) {  // (plain loads: an asynchronous copy would also wait for the rows in flight)
    const double* zr = C.z + (e0 + e) * rz;
    double* zd = s_z + e * RS;
#pragma unroll 1
    for (int c0 = 2 * lane; c0 < r; c0 += 256) {
      double2 v[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) v[q] = c0 + 64 * q < r ? __ldcg(reinterpret_cast<const double2*>(zr + c0 + 64 * q)) : make_double2(0.0, 0.0);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int c = c0 + 64 * q;
        if (c < r) *reinterpret_cast<double2*>(zd + (c >> 5) * WT_XBLK + ((c >> 3) & 3) * 10 + (c & 7)) = v[q];
      }
    }
  }
  if (tid < ne) sh.inv[e0 + tid] = L.norm_n == 0 ? wt_rsqrt(ss * C.inv_d + (double)L.eps_n) : 1.0;
  if (tid == 0) { sh.kmin = 0xffffffffffffffffULL; sh.kmax = 0ULL; }
  __syncthreads();
  // raw dot products: a warp per m-tile of eight neurons, all blocks of the rank
#pragma unroll 1
  for (int mt = warp; mt < n_mt; mt += WT_WARPS) {
    const unsigned char* wrow = s_b + (8 * mt + g) * RB + 16 * t;
    const double* zb = s_z + t * 10;
    double c0[2] = {0.0, 0.0}, c1[2] = {0.0, 0.0}, pl[2] = {0.0, 0.0};
#pragma unroll 1
    for (int b = 0; b < nblk; ++b, wrow += 64, zb += WT_XBLK) {
      double a[8], f[8];
      wt_cvt8<WD>(*reinterpret_cast<const uint4*>(wrow), a);
      if (ntile > 0) { wt_load8d(zb + g * RS, f); wt_mma_block(c0, a, f); }
      if (ntile > 1) { wt_load8d(zb + (8 + g) * RS, f); wt_mma_block(c1, a, f); }
#pragma unroll 1
      for (int q = 0; q < nplain; ++q) {
        wt_load8d(zb + (8 * ntile + q) * RS, f);
        const double v = (a[0] * f[0] + a[1] * f[1]) + (a[2] * f[2] + a[3] * f[3]) + ((a[4] * f[4] + a[5] * f[5]) + (a[6] * f[6] + a[7] * f[7]));
        if (q == 0) pl[0] += v; else pl[1] += v;
      }
    }
    double* dp = s_dot + 8 * mt + g;
    if (ntile > 0) { dp[(2 * t) * per8] = c0[0]; dp[(2 * t + 1) * per8] = c0[1]; }
    if (ntile > 1) { dp[(8 + 2 * t) * per8] = c1[0]; dp[(8 + 2 * t + 1) * per8] = c1[1]; }
#pragma unroll
    for (int q = 0; q < 2; ++q)
      if (q < nplain) {
        double v = pl[q];
        v += __shfl_xor_sync(0xffffffffu, v, 1);
        v += __shfl_xor_sync(0xffffffffu, v, 2);
        if (t == 0) dp[(8 * ntile + q) * per8] = v;
      }
  }
  __syncthreads();
  // scores, bins, key range of the final evaluation: (evaluation, neuron) pairs dealt over the threads
  const double hi = sh.bin_hi, scale = sh.bin_scale;
  const int nown = n1 - n0;
  const int Fs = (Fn + 7) & ~7;
  unsigned long long kmin = 0xffffffffffffffffULL, kmax = 0ULL;
#pragma unroll 1
  for (int q = tid; q < ne * nown; q += WT_THREADS) {
    const int el = ne == 1 ? 0 : q / nown, i = q - el * nown, row = n0 + i, e = e0 + el;
    const double sv = canonical_score(s_dot[el * per8 + i] * sh.inv[e] + (double)s_pc[i]);
    __stcg(C.sc + (size_t)e * Fn + row, sv);
    C.sb[(size_t)e * Fs + row] = (uint16_t)wt_bin_of(sv, hi, scale);
    if (e == K) {
      if (last && C.out_scores) C.out_scores[row] = sv;
      // Speculation (beyond the paper's): the exact selection is two phases away, but a final score at or above the cut
      // the layer's previous token ended with (less a margin) almost certainly belongs to it, so its gate row is asked
      // into L2 now and travels while the selection is made.  A wrong guess costs idle bandwidth, never a result.
      if (sh.pf_base && sv >= sh.pf_thr)
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(sh.pf_base + (size_t)row * sh.pf_stride), "r"(sh.pf_bytes) : "memory");
      if (fabs(sv) <= 1.7976931348623157e308) {
        const unsigned long long key = ordered_key(sv);
        kmin = min(kmin, key);
        kmax = max(kmax, key);
      }
    }
  }
  if (n1 == Fn && nown > 0 && tid < ne * 8) {  // (entries that pad a row of bins to a multiple of eight: a bin of their own)
    const int e = e0 + (tid >> 3), i = Fn + (tid & 7);
    if (i < Fs) C.sb[(size_t)e * Fs + i] = (uint16_t)WT_NB;
  }
  if (e0 + ne > K) {
    if (kmax >= kmin) { atomicMin(&sh.kmin, kmin); atomicMax(&sh.kmax, kmax); }
    __syncthreads();
    if (tid == 0) { __stcg(C.kmm + 2 * blockIdx.x, sh.kmin); __stcg(C.kmm + 2 * blockIdx.x + 1, sh.kmax); }
  }
  __syncthreads();
}

// ---- P4: selection ---------------------------------------------------------------------------------------------------
// Members of the refined set of evaluation j whose rank falls in [lo, hi), by this CTA alone: bins of the evaluation to
// shared memory, histogram, prefix sum, the bins that cover the ranks, their members, exact comparison inside a bin.
// Found members go to out[rank - lo] (shared memory).  Returns false (to every thread, and alike in every CTA that asks
// about the same evaluation) when a bin that reaches into the first keff ranks is too full; the caller then takes the
// general route.  With want_mask the members of all ranks below hi are also marked in the shared bitmap (trace).
// (Shared memory is addressed through the kernel's dynamic array so that loads, stores and atomics are shared-space ones.)
__device__ __noinline__ bool wt_select(const WtCall& C, WtShared& sh, int j, int Fn, int keff, int lo, int hi, unsigned out_off,
                                       bool want_mask, unsigned long long* cut_out) {
  extern __shared__ __align__(128) unsigned char wt_smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  unsigned char* u = wt_smem + C.lay.u_off;
  unsigned* s_bin2 = reinterpret_cast<unsigned*>(u + C.lay.bin_off);  // two bins per word
  unsigned* s_hist = reinterpret_cast<unsigned*>(wt_smem + C.lay.hist_off);
  unsigned* s_pref = reinterpret_cast<unsigned*>(u + C.lay.pref_off);
  unsigned long long* s_ckey = reinterpret_cast<unsigned long long*>(u + C.lay.ckey_off);
  int* s_cidx = reinterpret_cast<int*>(u + C.lay.cidx_off);
  uint16_t* s_cbin = reinterpret_cast<uint16_t*>(u + C.lay.cbin_off);
  unsigned* s_bits = reinterpret_cast<unsigned*>(wt_smem + C.lay.bits_off);
  int* out = reinterpret_cast<int*>(wt_smem + out_off);
  const int Fs = (Fn + 7) & ~7, n2 = Fs >> 1;
  const unsigned char* sb = reinterpret_cast<const unsigned char*>(C.sb + (size_t)j * Fs);
  const double* sc = C.sc + (size_t)j * Fn;
  // the bins are requested first; the histogram is cleared while they are on their way
#pragma unroll 1
  for (int o = tid * 16; o < Fs * 2; o += WT_THREADS * 16) wt_cp_async16(reinterpret_cast<unsigned char*>(s_bin2) + o, sb + o);
  reinterpret_cast<uint4*>(s_hist)[tid] = make_uint4(0u, 0u, 0u, 0u);
  reinterpret_cast<uint4*>(s_hist)[tid + WT_THREADS] = make_uint4(0u, 0u, 0u, 0u);
  if (tid == 0) { sh.blo = WT_NB; sh.bhi = -1; sh.ncand = 0; sh.slow = 0; sh.found = 0; }
  wt_cp_async_wait();
  __syncthreads();
#pragma unroll 1
  for (int i = tid; i < n2; i += WT_THREADS) {  // (the entries that pad the row fall into a bin of their own)
    const unsigned w = s_bin2[i];
    atomicAdd(&s_hist[w & 0xffffu], 1u);
    atomicAdd(&s_hist[w >> 16], 1u);
  }
  __syncthreads();
  {
    // exclusive prefix sum over the bins (eight consecutive bins per thread, warp scans on two levels)
    const uint4 h0 = reinterpret_cast<const uint4*>(s_hist)[2 * tid], h1 = reinterpret_cast<const uint4*>(s_hist)[2 * tid + 1];
    const unsigned cnt[WT_BPT] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
    unsigned run = 0;
#pragma unroll
    for (int e = 0; e < WT_BPT; ++e) run += cnt[e];
    unsigned incl = run;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) sh.redu[warp] = incl;
    __syncthreads();
    unsigned wtot = lane < WT_WARPS ? sh.redu[lane] : 0u, wincl = wtot;
#pragma unroll
    for (int o = 1; o < WT_WARPS; o <<= 1) {
      const unsigned v = __shfl_up_sync(0xffffffffu, wincl, o);
      if (lane >= o) wincl += v;
    }
    int base = (int)(__shfl_sync(0xffffffffu, wincl - wtot, warp) + incl - run);
    int blo = WT_NB, bhi = -1, slow = 0;
    unsigned pre[WT_BPT];
#pragma unroll
    for (int e = 0; e < WT_BPT; ++e) {
      const int c = (int)cnt[e];
      pre[e] = (unsigned)base;
      if (c > 0) {
        if (base < keff && c > WT_BINCAP) slow = 1;
        if (base < hi && base + c > lo) { blo = min(blo, tid * WT_BPT + e); bhi = tid * WT_BPT + e; }
      }
      base += c;
    }
    reinterpret_cast<uint4*>(s_pref)[2 * tid] = make_uint4(pre[0], pre[1], pre[2], pre[3]);
    reinterpret_cast<uint4*>(s_pref)[2 * tid + 1] = make_uint4(pre[4], pre[5], pre[6], pre[7]);
    if (slow) sh.slow = 1;
    if (bhi >= 0) { atomicMin(&sh.blo, blo); atomicMax(&sh.bhi, bhi); }
  }
  __syncthreads();
  if (sh.slow) return false;
  const int blo = sh.blo, span = sh.bhi - blo;  // (span < 0: no bin covers the ranks)
  if (hi > lo || want_mask) {
    // the members of the covering bins
#pragma unroll 1
    for (int i = tid; i < n2; i += WT_THREADS) {
      const unsigned w = s_bin2[i];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int b = (int)(e ? w >> 16 : w & 0xffffu), idx = 2 * i + e;
        if ((unsigned)(b - blo) <= (unsigned)span && span >= 0) {
          const int pos = atomicAdd(&sh.ncand, 1);
          if (pos < WT_CANDCAP) { s_cidx[pos] = idx; s_cbin[pos] = (uint16_t)b; }
        } else if (want_mask && b < blo) {
          atomicOr(&s_bits[idx >> 5], 1u << (idx & 31));
        }
      }
    }
  }
  __syncthreads();
  const int ncand = min(sh.ncand, WT_CANDCAP);
#pragma unroll 1
  for (int q = tid; q < ncand; q += WT_THREADS) s_ckey[q] = ordered_key(__ldcg(sc + s_cidx[q]));
  __syncthreads();
  // exact rank of every candidate: a warp per candidate, the lanes share the comparisons
#pragma unroll 1
  for (int q = warp; q < ncand; q += WT_WARPS) {
    const unsigned long long kq = s_ckey[q];
    const int iq = s_cidx[q], bq = s_cbin[q];
    int before = 0;
#pragma unroll 1
    for (int w = lane; w < ncand; w += 32) {
      const unsigned long long kw = s_ckey[w];
      before += (s_cbin[w] == bq) && ((kw > kq) || (kw == kq && s_cidx[w] < iq));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xffffffffu, before, o);
    if (lane == 0) {
      const int rank = (int)s_pref[bq] + before;
      if (rank >= lo && rank < hi) {
        out[rank - lo] = iq;
        atomicAdd(&sh.found, 1);
      }
      if (want_mask && rank < hi) atomicOr(&s_bits[iq >> 5], 1u << (iq & 31));
      if (rank == keff - 1) __stcg(cut_out, kq);
    }
  }
  __syncthreads();
  if (tid == 0 && (sh.found != hi - lo || sh.ncand > WT_CANDCAP)) set_status(sh.L[0].status, ST_INTERNAL);
  return true;
}

// General route: exact top-k of evaluation j by ONE CTA for any input (all scores equal, a range that does not fit),
// only slower.  Writes the ranked list (when given), the shared bitmap (when asked) and the key of the last member.
__device__ __noinline__ void wt_select_general(const WtCall& C, WtShared& sh, unsigned char* smem, int j, int Fn, int keff, int32_t* ranked,
                                               bool want_mask, unsigned long long* cut_out) {
  unsigned* s_bits = reinterpret_cast<unsigned*>(smem + C.lay.bits_off);
  const double* sc = C.sc + (size_t)j * Fn;
  __syncthreads();
  if (keff <= 0) return;
  if (threadIdx.x == 0) sh.b_valid = 0;  // (the work area below covers this CTA's rows of B^T)
  TopkSmem sm = topk_carve(smem + C.lay.u_off);
  block_topk_nt<WT_THREADS>(
      Fn, keff,
      [&](int v, double& s) {
        s = __ldcg(sc + v);
        return true;
      },
      [&](int rank, int v) {
        if (ranked) ranked[rank] = v;
        if (want_mask) atomicOr(&s_bits[v >> 5], 1u << (v & 31));
        if (rank == keff - 1) *cut_out = ordered_key(canonical_score(__ldcg(sc + v)));
      },
      sm, C.tk_key, C.tk_idx);
}

// The refined set of an evaluation j < K by one CTA: its last member's key always, its mask when a trace asks for it.
__device__ __noinline__ void wt_refined_set(const WtCall& C, WtShared& sh, unsigned char* smem, int j, int Fn, int keff, uint32_t* mask_out,
                                            unsigned long long* cut_out) {
  const int tid = threadIdx.x;
  unsigned* s_bits = reinterpret_cast<unsigned*>(smem + C.lay.bits_off);
  const int nwords = (Fn + 31) >> 5;
  if (mask_out) {
    for (int w = tid; w < nwords; w += WT_THREADS) s_bits[w] = 0u;
    __syncthreads();
  }
  // (the member found goes to a word of scratch that is free during the selection)
  if (keff > 0 && !wt_select(C, sh, j, Fn, keff, keff - 1, keff, C.lay.dm_off, mask_out != nullptr, cut_out)) {
    if (mask_out) {
      __syncthreads();
      for (int w = tid; w < nwords; w += WT_THREADS) s_bits[w] = 0u;
    }
    wt_select_general(C, sh, smem, j, Fn, keff, nullptr, mask_out != nullptr, cut_out);
  }
  if (mask_out) {
    __syncthreads();
    for (int w = tid; w < nwords; w += WT_THREADS) mask_out[w] = s_bits[w];
  }
  __syncthreads();
}

// What leaves a layer besides x: the ranked list (trace, and the caller's list after the last layer), the masks.
__device__ __noinline__ void wt_export_selection(const WtCall& C, const int* s_mine, int n, int lo, int nmine, int keff, bool last) {
  const int tid = threadIdx.x, E = C.K + 1;
  if (tid < nmine) {
    const int v = s_mine[tid], rank = lo + tid;
    if (C.tr_sel && rank < C.tr_cap) C.tr_sel[(size_t)(n + 1) * C.tr_cap + rank] = v;
    if (C.tr_masks) atomicOr(C.tr_masks + ((size_t)n * E + C.K) * C.tr_words + (v >> 5), 1u << (v & 31));
    if (last) {
      if (rank < C.out_cap) C.out_idx[rank] = v;
      if (C.out_mask) atomicOr(C.out_mask + (v >> 5), 1u << (v & 31));
    }
  }
  if (blockIdx.x == 0 && tid == 0) {
    if (C.tr_cnt) C.tr_cnt[n + 1] = keff;
    if (last) *C.out_count = min(keff, C.out_cap);
  }
  if (blockIdx.x == 0 && C.tr_counts && tid < E) C.tr_counts[tid] = keff;
}

// New bin range of the layer's scores from what this launch observed (one warp; used by the next launch).
__device__ __noinline__ void wt_update_range(const WtCall& C, const WtLayer& L) {
  const int lane = threadIdx.x & 31, G = gridDim.x;
  unsigned long long kmin = 0xffffffffffffffffULL, kmax = 0ULL;
  for (int c = lane; c < G; c += 32) {
    kmin = min(kmin, __ldcg(C.kmm + 2 * c));
    kmax = max(kmax, __ldcg(C.kmm + 2 * c + 1));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
    kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
  }
  if (lane == 0 && kmax >= kmin) {
    auto unkey = [](unsigned long long k) {
      const unsigned long long b = (k >> 63) ? (k & 0x7fffffffffffffffULL) : ~k;
      return __longlong_as_double((long long)b);
    };
    const double lo = unkey(kmin), hi = unkey(kmax);
    const double w = hi - lo;
    if (w > 0.0 && w < 1.0e300) {
      L.range[0] = hi + 0.01 * w;
      L.range[1] = (double)WT_NB / (1.02 * w);
    }
  }
}

// =====================================================================================================================
template <int WD>
__global__ void __launch_bounds__(WT_THREADS, 1) ls_token_kernel(const WtLayer* __restrict__ g_layers, const __grid_constant__ WtCall C) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ WtShared sh;
  const int tid = threadIdx.x, cta = blockIdx.x, G = gridDim.x;
  const int d = C.d, K = C.K, E = K + 1;
  float* s_x = reinterpret_cast<float*>(smem + C.lay.x_off);
  uint16_t* s_xs = C.mma ? reinterpret_cast<uint16_t*>(smem + C.lay.xs_off) : nullptr;  // x as three 16-bit terms (tensor-core operand)
  int* s_mine = reinterpret_cast<int*>(smem + C.lay.mine_off);
  constexpr int NW = sizeof(WtLayer) / 4;
  const int n_act = C.gs * K;
  const bool active = cta < n_act;
  const bool stamps = C.tr_ns != nullptr && tid == 0;
  unsigned epoch = 0;

  // ---- prologue: arguments of layer 0, x, 1 / rms, this CTA's slice of the first selection
  if (tid < NW)
    reinterpret_cast<uint32_t*>(&sh.L[0])[tid] = g_layers ? reinterpret_cast<const uint32_t*>(&g_layers[0])[tid] : reinterpret_cast<const uint32_t*>(&C.one)[tid];
  if (tid == 0) {
    sh.dead = 0;
    sh.b_valid = 1;
    wt_mbar_init(&sh.mbar[0], WT_WARPS);  // rows into the ring: one arrival per warp and batch
    wt_mbar_init(&sh.mbar[1], 1);         // A slices, B^T rows: one phase per layer
    wt_mbar_init(&sh.mbar[2], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  uint32_t ring_phase = 0;
  {
    double sq = 0.0;
    for (int c = tid * 4; c < d; c += WT_THREADS * 4) {
      const float4 v = __ldcg(reinterpret_cast<const float4*>(C.x_in + c));
      wt_store_x4<WD>(s_x, s_xs, c, v);
      sq += (double)v.x * v.x + (double)v.y * v.y + (double)v.z * v.z + (double)v.w * v.w;
      if (C.tr_x && cta == 0) *reinterpret_cast<float4*>(C.tr_x + c) = v;
    }
    sq = warp_sum(sq);
    if ((tid & 31) == 0) sh.redd[tid >> 5] = sq;
  }
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int w = 0; w < WT_WARPS; ++w) t += sh.redd[w];
    sh.inv_x = sh.L[0].norm == 0 ? (float)wt_rsqrt(t / (double)d + (double)sh.L[0].eps) : 1.0f;
  }
  {
    const int count0 = max(0, min(__ldg(C.sel_count), C.sel_cap));
    int lo, hi;
    wt_share(count0, K, C.gs, cta, lo, hi);
    if (tid < hi - lo) {
      int v = __ldg(C.sel_idx + lo + tid);
      if ((unsigned)v >= (unsigned)sh.L[0].F) { v = -1; set_status(sh.L[0].status, ST_BAD_INDEX); }  // never dereferenced
      s_mine[tid] = v;
    }
    if (tid == 0) sh.nmine = hi - lo;
    if (C.tr_sel && cta == G - 1) {
      for (int i = tid; i < min(count0, C.tr_cap); i += WT_THREADS) C.tr_sel[i] = __ldg(C.sel_idx + i);
      if (tid == 0) C.tr_cnt[0] = count0;
    }
  }
  __syncthreads();

  // The refined sets of layer m's evaluations j < K (their scores are complete since layer m's last barrier).  `where` 0:
  // called at the start of the next layer's stream phase, 1: in its P1, 2: after the last layer.  The CTAs that have no
  // rows to stream take two evaluations each during the stream phase (it is long enough for two); what is left goes to
  // CTAs that own no slice of the feature, during P1 (or, when every CTA owns one, behind its slice).
  auto refined_sets = [&](int m, const WtLayer& Lm, int where) {
    const int n_idle = G - n_act, cap_s = min(K, 2 * n_idle);
    if ((where == 0 && cap_s == 0) || (where == 1 && cap_s == K)) return;
    const int nsl = (d + 31) >> 5, keff_m = min(C.k_next, Lm.Fn);
    const int j0 = where == 1 ? cap_s : 0, j1 = where == 0 ? cap_s : K;
    unsigned long long* cuts = C.cuts + (size_t)m * E;
#pragma unroll 1
    for (int j = j0; j < j1; ++j) {
      const int q = j - cap_s;
      const int owner = j < cap_s ? n_act + (j < n_idle ? j : j - n_idle) : (nsl + q < G ? nsl + q : G - 1 - (q % G));
      if (cta == owner) {
        // (in P1 this CTA's rows of B^T may still be on their way into the work area a degenerate selection borrows)
        if (where == 1) wt_mbar_wait(sh, &sh.mbar[2], (uint32_t)(m + 1) & 1u);
        wt_refined_set(C, sh, smem, j, Lm.Fn, keff_m, C.tr_masks ? C.tr_masks + ((size_t)m * E + j) * C.tr_words : nullptr, cuts + j);
      }
    }
  };

  if (tid == 0) sh.keff_shared = -1;  // (this CTA's ranks of the next selection are kept for as long as its size stays the same)
#pragma unroll 1
  for (int n = 0; n < C.n_layers; ++n) {
    const WtLayer& L = sh.L[n & 1];
    const bool last = n + 1 == C.n_layers;
    const int rz = (L.r + 4) & ~3;
    const int keff = min(C.k_next, L.Fn);
    if (stamps) wt_stamp(C, n, 0);
    // ---- S (and, on the CTAs without rows, the refined sets of the layer before)
    if (n > 0 && !active) refined_sets(n - 1, sh.L[(n - 1) & 1], 0);
    wt_stream<WD>(C, sh, L, smem, active, ring_phase, n > 0);
    if (stamps) wt_stamp(C, n, 1);
    wt_grid_sync(C, sh, ++epoch * G);
    if (sh.dead) return;
    if (stamps) wt_stamp(C, n, 2);
    // ---- P1 (and the refined sets of the layer before, whose scores are complete now)
    float* x_out = last ? C.x_out : C.xbuf + (size_t)((n + 1) & 1) * d;
    wt_feature<WD>(C, sh, L, smem, n, x_out, E, rz);
    if (n > 0) refined_sets(n - 1, sh.L[(n - 1) & 1], 1);
    if (stamps) wt_stamp(C, n, 3);
    // next layer's arguments (the layer before's are not needed any more)
    __syncthreads();
    if (!last && tid < NW) reinterpret_cast<uint32_t*>(&sh.L[(n + 1) & 1])[tid] = reinterpret_cast<const uint32_t*>(&g_layers[n + 1])[tid];
    wt_grid_sync(C, sh, ++epoch * G);
    if (sh.dead) return;
    if (stamps) wt_stamp(C, n, 4);
    // ---- P2
    // (the next layer's input is requested before the sums, so that the two round trips to L2 overlap)
    const int xc0 = tid * 4, xc1 = xc0 + WT_THREADS * 4;
    float4 xv0 = make_float4(0.f, 0.f, 0.f, 0.f), xv1 = xv0;
    if (!last && xc0 < d) xv0 = __ldcg(reinterpret_cast<const float4*>(x_out + xc0));
    if (!last && xc1 < d) xv1 = __ldcg(reinterpret_cast<const float4*>(x_out + xc1));
    wt_latent_sums(C, L.r, E, rz);
    if (!last) {
      if (xc0 < d) wt_store_x4<WD>(s_x, s_xs, xc0, xv0);
      if (xc1 < d) wt_store_x4<WD>(s_x, s_xs, xc1, xv1);
#pragma unroll 1
      for (int c = xc1 + WT_THREADS * 4; c < d; c += WT_THREADS * 4) wt_store_x4<WD>(s_x, s_xs, c, __ldcg(reinterpret_cast<const float4*>(x_out + c)));
    }
    if (tid == 32) {
      const double bh = L.range[0], bs = L.range[1];
      sh.bin_hi = bh; sh.bin_scale = bs;
      const unsigned long long ck = C.cuts[(size_t)n * E + K];  // (what the previous launch left: the previous token's cut)
      const WtLayer& Ln = sh.L[(n + 1) & 1];
      const bool spec = !last && ck != 0ULL && bs > 0.0 && ((d * 2) & 15) == 0;
      sh.pf_base = spec ? reinterpret_cast<const unsigned char*>(Ln.bundles) : nullptr;
      sh.pf_stride = (unsigned)Ln.n_mat * d * 2u;
      sh.pf_bytes = (unsigned)d * 2u;
      const unsigned long long cb = (ck >> 63) ? (ck & 0x7fffffffffffffffULL) : ~ck;
      sh.pf_thr = __longlong_as_double((long long)cb) - 48.0 / bs;  // (a margin of 48 of the 4096 bins)
    }
    if (stamps) wt_stamp(C, n, 5);
    wt_grid_sync(C, sh, ++epoch * G);
    if (sh.dead) return;
    if (stamps) wt_stamp(C, n, 6);
    // ---- P3
    wt_cp_async_wait();  // (this CTA's score offsets and rows of B^T, requested at the end of S)
    wt_mbar_wait(sh, &sh.mbar[2], (uint32_t)n & 1u);
    __syncthreads();
    wt_score_evals<WD>(C, sh, L, 0, E, last);
    if (stamps) wt_stamp(C, n, 7);
    wt_grid_sync(C, sh, ++epoch * G);
    if (sh.dead) return;
    if (stamps) wt_stamp(C, n, 8);
    // ---- P4
    if (keff != sh.keff_shared) {  // (three integer divisions: once per launch unless the layers differ in size)
      int l0, h0;
      wt_share(keff, K, C.gs, cta, l0, h0);
      __syncthreads();
      if (tid == 0) { sh.my_lo = l0; sh.my_hi = h0; sh.keff_shared = keff; }
      __syncthreads();
    }
    const int lo = sh.my_lo, hi = sh.my_hi;
    if (tid == 0) sh.inv_x = (float)sh.inv[K];
    unsigned long long* cuts = C.cuts + (size_t)n * E;  // the keys of the last members of this layer's refined sets
    if (!wt_select(C, sh, K, L.Fn, keff, lo, hi, C.lay.mine_off, false, cuts + K)) {
      if (cta == 0) wt_select_general(C, sh, smem, K, L.Fn, keff, C.sellist, false, cuts + K);
      wt_grid_sync(C, sh, ++epoch * G);
      if (sh.dead) return;
      if (tid < hi - lo) s_mine[tid] = __ldcg(C.sellist + lo + tid);
      __syncthreads();
    }
    if (stamps) wt_stamp(C, n, 9);
    if (!last && hi > lo) wt_request_gate(C, sh, sh.L[(n + 1) & 1], smem, 0, hi - lo);  // (the next layer's first gate rows: on their way)
    if (tid == 0) sh.nmine = hi - lo;
    if (last || C.tr_sel || C.tr_masks || C.tr_counts) wt_export_selection(C, s_mine, n, lo, hi - lo, keff, last);
    if (cta == 0 && tid < 32) wt_update_range(C, L);
    __syncthreads();
    if (stamps) wt_stamp(C, n, 10);
  }
  // ---- the last layer's refined sets
  refined_sets(C.n_layers - 1, sh.L[(C.n_layers - 1) & 1], 2);
}

}  // namespace ls
