// Whole-token kernel: every layer of a resident stack for one decode token in ONE cooperative launch (batch 1).
//
// Two costs shape it.  A grid barrier costs about 2,300 SM clocks on this GPU whatever its form (one L2 round trip to
// arrive, one to see the last arrival), as long as a layer's whole weight traffic takes at full HBM speed; and code that a
// layer executes once streams into the SM at about six clocks per instruction unless the layer's whole path fits the
// instruction cache (32 to 48 KB).  So a layer step has FOUR barriers, the fewest the data flow allows, and every phase is
// a handful of small rolled loops; rare paths (trace export, slow selection) are out of line.
//
//   S  stream    The K priority stages of the layer (Eq. 1) run concurrently on K groups of CTAs (the output is a sum over
//                hidden neurons, Section 3.2.2, so only stage MEMBERSHIP defines the partial features of Eq. 2).  A CTA
//                owns a contiguous slice of the ranks of one stage.  Rows go straight from global memory to registers with
//                128-bit loads, a dozen in flight per thread: gate rows first, then the up and down rows of the neurons
//                that survive the ReLU only.  The CTA's partial output goes to its own row of a scratch array.
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
//                j < K (Section 2.1: they steer fetching and retention, nothing on a resident stack waits for them) are
//                established by the same routine (the slice being the set's last rank) on CTAs with little to stream.
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
  int n_mat, F, norm; float eps;
  // predictor of the layer this one refines (the next layer; the last layer refines itself)
  const uint16_t* At_sl; const uint16_t* Bt_pad; const float* pc;  // Bt_pad: rows of wt_brow_bytes(r) bytes, zero padded
  int r, Fn, norm_n; float eps_n;
  double* range;  // [2] {hi, scale} of the score bins, refreshed by every launch for the next one
  int* status;
};

struct WtSmem {  // byte offsets into dynamic shared memory (computed on the host)
  unsigned x_off, xt_off, dm_off, mine_off, bits_off, pc_off, hist_off, u_off;
  // region u.  While a layer runs: A slices | B^T rows | partial outputs of a slice (P1), then latents and raw scores (P3).
  unsigned b_off, yz_off, dot_off;
  // region u during the selection (everything above is dead by then), or the general top-k's work area instead
  unsigned bin_off, pref_off, ckey_off, cidx_off, cbin_off;
  unsigned total;
};

struct WtCall {
  int n_layers, d, K, k_next, piece_len, gs;  // gs: CTAs per stage
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
  WtSmem lay;
};

struct WtShared {
  WtLayer L[2];
  int dead;               // a wait timed out: no more waiting
  int nmine, nsurv;
  int wcnt[WT_WARPS];
  int blo, bhi, ncand, slow, found;
  float inv_x;            // 1 / rms of the layer's input
  float act8[8];          // activations of a batch of survivors
  unsigned long long kmin, kmax;  // key range of this CTA's final scores
  double inv[WT_MAXE + 7];
  double redd[WT_WARPS];
  unsigned long long redk[2 * WT_WARPS];
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
// Dot products of up to three rows with x over one piece of the columns: r0..r2 and xs already point at this lane's first
// eight elements of the piece, `rem` is the length of the piece from there on (may be <= 0); four 16-byte loads per row,
// all issued before the first is used; the three sums are returned to every lane.
struct WtF3 { float a, b, c; };
template <int WD>
__device__ __noinline__ WtF3 wt_rows_dot(const uint16_t* r0, const uint16_t* r1, const uint16_t* r2, const float* xs, int rem, int nrows) {
  float acc[3] = {0.f, 0.f, 0.f};
  const uint16_t* rows[3] = {r0, r1, r2};
#pragma unroll 1
  for (int base = 0; base < rem; base += 1024) {
    uint4 w[3][4];
#pragma unroll
    for (int q = 0; q < 3; ++q)
#pragma unroll
      for (int it = 0; it < 4; ++it)
        w[q][it] = (q < nrows && base + it * 256 < rem) ? ld_stream128(rows[q] + base + it * 256) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      if (base + it * 256 < rem) {
        const float4 x0 = *reinterpret_cast<const float4*>(xs + base + it * 256);
        const float4 x1 = *reinterpret_cast<const float4*>(xs + base + it * 256 + 4);
        const float xv[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
#pragma unroll
        for (int q = 0; q < 3; ++q) {
          float f[8];
          unpack8<WD>(w[q][it], f);
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[q] = fmaf(f[e], xv[e], acc[q]);
        }
      }
    }
  }
  WtF3 o;
  o.a = warp_sum(acc[0]);
  o.b = warp_sum(acc[1]);
  o.c = warp_sum(acc[2]);
  return o;
}

// This CTA's slices of the next layer's predictor matrix A, its rows of B^T (stored padded, so both are plain linear
// copies) and its score offsets: asynchronously to shared memory; needed in P1 and P3.
__device__ __forceinline__ void wt_fetch_predictor(const WtCall& C, const WtLayer& L, unsigned char* smem) {
  const int tid = threadIdx.x, G = gridDim.x, d = C.d;
  const int nsl = (d + 31) >> 5, per_slice = L.r * 4;  // 16-byte pieces per slice
  unsigned char* s_a = smem + C.lay.u_off;
#pragma unroll 1
  for (int s = blockIdx.x, si = 0; s < nsl; s += G, ++si) {
    const unsigned char* src = reinterpret_cast<const unsigned char*>(L.At_sl) + (size_t)s * per_slice * 16;
#pragma unroll 1
    for (int i = tid; i < per_slice; i += WT_THREADS) wt_cp_async16(s_a + (si * per_slice + i) * 16, src + i * 16);
  }
  const int per = (L.Fn + G - 1) / G, n0 = min(L.Fn, (int)blockIdx.x * per), n1 = min(L.Fn, n0 + per);
  const int RB = wt_brow_bytes(L.r);
  const int npieces = (((n1 - n0 + 7) >> 3) * 8) * (RB >> 4);
  unsigned char* s_b = smem + C.lay.u_off + C.lay.b_off;
  const unsigned char* src = reinterpret_cast<const unsigned char*>(L.Bt_pad) + (size_t)n0 * RB;
#pragma unroll 1
  for (int i = tid; i < npieces; i += WT_THREADS) wt_cp_async16(s_b + i * 16, src + (size_t)i * 16);
  float* s_pc = reinterpret_cast<float*>(smem + C.lay.pc_off);
#pragma unroll 1
  for (int i = tid; i < n1 - n0; i += WT_THREADS) s_pc[i] = L.pc ? __ldg(L.pc + n0 + i) : 0.f;
}

template <int WD, int CPT>
__device__ __forceinline__ void wt_stream(const WtCall& C, WtShared& sh, const WtLayer& L, unsigned char* smem, bool active) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int d = C.d;
  const float* s_x = reinterpret_cast<const float*>(smem + C.lay.x_off);
  int* s_mine = reinterpret_cast<int*>(smem + C.lay.mine_off);           // [256] neurons of this CTA, rank order
  float* s_gsum = reinterpret_cast<float*>(s_mine + WT_MAXMINE);         // [256][4] partial gate dot products
  int* s_sidx = reinterpret_cast<int*>(s_gsum + 4 * WT_MAXMINE);         // [256] survivors
  float* s_sact = reinterpret_cast<float*>(s_sidx + WT_MAXMINE);         // [256] their relu(g)
  float* s_up = s_sact + WT_MAXMINE;                                     // [8][4] partial up dot products of a batch
  const int nmine = sh.nmine;
  const float inv = sh.inv_x;
  const unsigned bstride = (unsigned)L.n_mat * d;
  const int p = warp & 3, wq = warp >> 2;
  const int c_lo = min(d, p * C.piece_len);
  const int rem = min(d, c_lo + C.piece_len) - c_lo - lane * 8;
  const float* xs = s_x + c_lo + lane * 8;
  const uint16_t* wbase = L.bundles + c_lo + lane * 8;

  // gate bias of "my" neuron (used after the dot products; the load is in flight meanwhile)
  int my_idx = -1;
  float my_b = 0.f;
  if (tid < nmine) {
    my_idx = s_mine[tid];
    if (my_idx >= 0 && L.b_gate) my_b = __ldg(L.b_gate + my_idx);
  }
#pragma unroll 1
  for (int i0 = wq; i0 < nmine; i0 += 12) {
    const int nrows = min(3, (nmine - i0 + 3) >> 2);
    const uint16_t* r0 = wbase + (size_t)max(s_mine[i0], 0) * bstride;
    const uint16_t* r1 = nrows > 1 ? wbase + (size_t)max(s_mine[i0 + 4], 0) * bstride : r0;
    const uint16_t* r2 = nrows > 2 ? wbase + (size_t)max(s_mine[i0 + 8], 0) * bstride : r0;
    const WtF3 v = wt_rows_dot<WD>(r0, r1, r2, xs, rem, nrows);
    if (lane == 0) {
      s_gsum[i0 * 4 + p] = v.a;
      if (nrows > 1) s_gsum[(i0 + 4) * 4 + p] = v.b;
      if (nrows > 2) s_gsum[(i0 + 8) * 4 + p] = v.c;
    }
  }
  wt_fetch_predictor(C, L, smem);
  __syncthreads();
  // activation of the gate branch and the ordered list of survivors (a_i = relu(g_i) u_i: g_i <= 0 needs no other row)
  {
    float g = 0.f;
    if (my_idx >= 0) {
      const float4 s4 = *reinterpret_cast<const float4*>(s_gsum + tid * 4);
      g = ((s4.x + s4.y) + (s4.z + s4.w)) * inv + my_b;
    }
    const bool sv = g > 0.f;
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
  const bool gated = L.n_mat == 3;
  constexpr int NB = CPT == 1 ? 8 : 4;  // survivors per batch
  float acc8[CPT][8];
#pragma unroll
  for (int cp = 0; cp < CPT; ++cp)
#pragma unroll
    for (int e = 0; e < 8; ++e) acc8[cp][e] = 0.f;
  const uint16_t* dbase = L.bundles + (size_t)(L.n_mat - 1) * d + tid * 8;
#pragma unroll 1
  for (int b0 = 0; b0 < nsurv; b0 += NB) {
    const int nb = min(NB, nsurv - b0);
    uint4 dw[NB][CPT];
#pragma unroll
    for (int s = 0; s < NB; ++s)
#pragma unroll
      for (int cp = 0; cp < CPT; ++cp)
        dw[s][cp] = (s < nb && (tid + cp * WT_THREADS) * 8 < d) ? ld_stream128(dbase + (size_t)s_sidx[b0 + s] * bstride + cp * WT_THREADS * 8)
                                                                : make_uint4(0u, 0u, 0u, 0u);
    if (gated) {
      // up rows of the batch: warp (p, wq) takes piece p of the survivors wq and wq + 4
      if (wq < nb) {
        const int nrows = wq + 4 < nb ? 2 : 1;
        const uint16_t* r0 = wbase + d + (size_t)s_sidx[b0 + wq] * bstride;
        const uint16_t* r1 = nrows > 1 ? wbase + d + (size_t)s_sidx[b0 + wq + 4] * bstride : r0;
        const WtF3 v = wt_rows_dot<WD>(r0, r1, r0, xs, rem, nrows);
        if (lane == 0) {
          s_up[wq * 4 + p] = v.a;
          if (nrows > 1) s_up[(wq + 4) * 4 + p] = v.b;
        }
      }
      __syncthreads();
      if (tid < nb) {
        const float4 u4 = *reinterpret_cast<const float4*>(s_up + tid * 4);
        sh.act8[tid] = s_sact[b0 + tid] * (((u4.x + u4.y) + (u4.z + u4.w)) * inv);
      }
    } else if (tid < nb) {
      sh.act8[tid] = s_sact[b0 + tid];
    }
    __syncthreads();
#pragma unroll
    for (int s = 0; s < NB; ++s) {
      const float a = s < nb ? sh.act8[s] : 0.f;
#pragma unroll
      for (int cp = 0; cp < CPT; ++cp) {
        float f[8];
        unpack8<WD>(dw[s][cp], f);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc8[cp][e] = fmaf(a, f[e], acc8[cp][e]);
      }
    }
    __syncthreads();
  }
  if (active) {
    float* yp = C.ypart + (size_t)blockIdx.x * d + tid * 8;
#pragma unroll
    for (int cp = 0; cp < CPT; ++cp)
      if ((tid + cp * WT_THREADS) * 8 < d) {
        __stcg(reinterpret_cast<float4*>(yp + cp * WT_THREADS * 8), make_float4(acc8[cp][0], acc8[cp][1], acc8[cp][2], acc8[cp][3]));
        __stcg(reinterpret_cast<float4*>(yp + cp * WT_THREADS * 8 + 4), make_float4(acc8[cp][4], acc8[cp][5], acc8[cp][6], acc8[cp][7]));
      }
  }
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
  float* s_dm = reinterpret_cast<float*>(smem + C.lay.dm_off);    // [K][32] stage sums
  float* s_part = reinterpret_cast<float*>(smem + C.lay.u_off + C.lay.yz_off);  // [16 warps][32] partial stage sums
  const uint16_t* s_a = reinterpret_cast<const uint16_t*>(smem + C.lay.u_off);
  const int nsl = (d + 31) >> 5;
  const int ntile = wt_tiles(E), nplain = wt_plain(E), rows = wt_rows(E);
  const int pos = (lane >> 3) * 10 + (lane & 7);
  // warps per stage and the rows (CTAs) of a stage one warp adds: all loads of a warp are in flight together
  const int wps = max(1, WT_WARPS / K), rpw = (C.gs + wps - 1) / wps;
  wt_cp_async_wait();
#pragma unroll 1
  for (int s = blockIdx.x, si = 0; s < nsl; s += G, ++si) {
    const int col = 32 * s + lane;
    {
      const int c = warp / wps, h = warp - c * wps;
      float a = 0.f;
      if (c < K && col < d) {
        const int g0 = h * rpw, g1 = min(C.gs, g0 + rpw);
        const float* yp = C.ypart + (size_t)(c * C.gs + g0) * d + col;
#pragma unroll 1
        for (int q0 = g0; q0 < g1; q0 += 10, yp += (size_t)10 * d) {
          float v[10];
#pragma unroll
          for (int i = 0; i < 10; ++i) v[i] = q0 + i < g1 ? __ldcg(yp + (size_t)i * d) : 0.f;
#pragma unroll
          for (int i = 0; i < 10; ++i) a += v[i];
        }
      }
      s_part[warp * 32 + lane] = a;
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
        for (int h = 0; h < wps; ++h) dm += s_part[(c * wps + h) * 32 + lane];
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
  for (int u = blockIdx.x * WT_WARPS + warp; u < units; u += G * WT_WARPS) {
    const int e = u / ngrp, l = 4 * (u - e * ngrp) + v;
    double a = 0.0;
    if (l <= r) {
      const double* zp = C.zpart + e * rz + l + (size_t)sg * step;
#pragma unroll 4
      for (int s = sg; s < nsl; s += 8, zp += 8 * step) a += __ldcg(zp);
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

template <int WD>
__device__ __forceinline__ void wt_scores(const WtCall& C, WtShared& sh, const WtLayer& L, unsigned char* smem, int E, int rz, bool last) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const int r = L.r, Fn = L.Fn, G = gridDim.x, K = C.K;
  double* s_z = reinterpret_cast<double*>(smem + C.lay.u_off + C.lay.yz_off);
  double* s_dot = reinterpret_cast<double*>(smem + C.lay.u_off + C.lay.dot_off);  // [E][per8] raw dot products
  const float* s_pc = reinterpret_cast<const float*>(smem + C.lay.pc_off);
  const unsigned char* s_b = smem + C.lay.u_off + C.lay.b_off;
  const int RS = wt_feat_stride(r), RB = wt_brow_bytes(r);
  const int ntile = wt_tiles(E), nplain = wt_plain(E), rows = wt_rows(E);
  const int nblk = (r + 31) >> 5;
  const int per = (Fn + G - 1) / G, n0 = min(Fn, (int)blockIdx.x * per), n1 = min(Fn, n0 + per);
  const int n_mt = (n1 - n0 + 7) >> 3, per8 = n_mt * 8;
  // latents to shared memory in the block layout: thread (e, c) pairs, six loads in flight each; 1 / rms of every evaluation
  {
    const int ncol = nblk * 32, total = rows * ncol;
#pragma unroll 1
    for (int i0 = tid; i0 < total; i0 += 6 * WT_THREADS) {
      double v[6];
      int o[6];
#pragma unroll
      for (int q = 0; q < 6; ++q) {
        const int i = i0 + q * WT_THREADS;
        const int e = i / ncol, c = i - e * ncol;
        o[q] = i < total ? e * RS + (c >> 5) * WT_XBLK + ((c >> 3) & 3) * 10 + (c & 7) : -1;
        v[q] = (i < total && e < E && c < r) ? __ldcg(C.z + e * rz + c) : 0.0;
      }
#pragma unroll
      for (int q = 0; q < 6; ++q)
        if (o[q] >= 0) s_z[o[q]] = v[q];
    }
    if (tid < E) {
      const double ss = __ldcg(C.z + tid * rz + r);
      sh.inv[tid] = L.norm_n == 0 ? wt_rsqrt(ss / (double)C.d + (double)L.eps_n) : 1.0;
    }
    if (tid == 0) { sh.kmin = 0xffffffffffffffffULL; sh.kmax = 0ULL; }
  }
  __syncthreads();
  // raw dot products: a warp per m-tile of eight neurons, all blocks of the rank; two accumulator sets alternate between
  // the blocks so that consecutive MMAs do not wait for one another
#pragma unroll 1
  for (int mt = warp; mt < n_mt; mt += WT_WARPS) {
    const unsigned char* wrow = s_b + (8 * mt + g) * RB + 16 * t;
    const double* zb = s_z + t * 10;
    double c0[2][2] = {{0.0, 0.0}, {0.0, 0.0}}, c1[2][2] = {{0.0, 0.0}, {0.0, 0.0}}, pl[2] = {0.0, 0.0};
#pragma unroll 2
    for (int b = 0; b < nblk; ++b, wrow += 64, zb += WT_XBLK) {
      double a[8], f[8];
      wt_cvt8<WD>(*reinterpret_cast<const uint4*>(wrow), a);
      if (ntile > 0) { wt_load8d(zb + g * RS, f); wt_mma_block(c0[b & 1], a, f); }
      if (ntile > 1) { wt_load8d(zb + (8 + g) * RS, f); wt_mma_block(c1[b & 1], a, f); }
      if (nplain > 0) { wt_load8d(zb + (8 * ntile) * RS, f); pl[0] = wt_dot8(a, f, pl[0]); }
      if (nplain > 1) { wt_load8d(zb + (8 * ntile + 1) * RS, f); pl[1] = wt_dot8(a, f, pl[1]); }
    }
    double* dp = s_dot + 8 * mt + g;
    if (ntile > 0) { dp[(2 * t) * per8] = c0[0][0] + c0[1][0]; dp[(2 * t + 1) * per8] = c0[0][1] + c0[1][1]; }
    if (ntile > 1) { dp[(8 + 2 * t) * per8] = c1[0][0] + c1[1][0]; dp[(8 + 2 * t + 1) * per8] = c1[0][1] + c1[1][1]; }
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
  // scores, bins, key range of the final evaluation: thread (e, i) pairs
  const double hi = L.range[0], scale = L.range[1];
  const int nown = n1 - n0;
  const int Fs = (Fn + 7) & ~7;
  unsigned long long kmin = 0xffffffffffffffffULL, kmax = 0ULL;
#pragma unroll 1
  for (int q = tid; q < E * nown; q += WT_THREADS) {
    const int e = q / nown, i = q - e * nown, row = n0 + i;
    const double s = canonical_score(s_dot[e * per8 + i] * sh.inv[e] + (double)s_pc[i]);
    __stcg(C.sc + (size_t)e * Fn + row, s);
    C.sb[(size_t)e * Fs + row] = (uint16_t)wt_bin_of(s, hi, scale);
    if (e == K) {
      if (last && C.out_scores) C.out_scores[row] = s;
      if (fabs(s) <= 1.7976931348623157e308) {
        const unsigned long long key = ordered_key(s);
        kmin = min(kmin, key);
        kmax = max(kmax, key);
      }
    }
  }
  if (kmax >= kmin) { atomicMin(&sh.kmin, kmin); atomicMax(&sh.kmax, kmax); }
  __syncthreads();
  if (tid == 0) { __stcg(C.kmm + 2 * blockIdx.x, sh.kmin); __stcg(C.kmm + 2 * blockIdx.x + 1, sh.kmax); }
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
  uint4* s_bin8 = reinterpret_cast<uint4*>(u + C.lay.bin_off);
  unsigned* s_hist = reinterpret_cast<unsigned*>(wt_smem + C.lay.hist_off);
  unsigned* s_pref = reinterpret_cast<unsigned*>(u + C.lay.pref_off);
  unsigned long long* s_ckey = reinterpret_cast<unsigned long long*>(u + C.lay.ckey_off);
  int* s_cidx = reinterpret_cast<int*>(u + C.lay.cidx_off);
  uint16_t* s_cbin = reinterpret_cast<uint16_t*>(u + C.lay.cbin_off);
  unsigned* s_bits = reinterpret_cast<unsigned*>(wt_smem + C.lay.bits_off);
  int* out = reinterpret_cast<int*>(wt_smem + out_off);
  const int Fs = (Fn + 7) & ~7, n8 = Fs >> 3;
  const uint4* sb8 = reinterpret_cast<const uint4*>(C.sb + (size_t)j * Fs);
  const double* sc = C.sc + (size_t)j * Fn;
  // the bins are requested first; the histogram is cleared while they are on their way
  uint4 v[3];
#pragma unroll
  for (int q = 0; q < 3; ++q) v[q] = tid + q * WT_THREADS < n8 ? __ldcg(sb8 + tid + q * WT_THREADS) : make_uint4(0u, 0u, 0u, 0u);
  reinterpret_cast<uint4*>(s_hist)[tid] = make_uint4(0u, 0u, 0u, 0u);
  reinterpret_cast<uint4*>(s_hist)[tid + WT_THREADS] = make_uint4(0u, 0u, 0u, 0u);
  if (tid == 0) { sh.blo = WT_NB; sh.bhi = -1; sh.ncand = 0; sh.slow = 0; sh.found = 0; }
  __syncthreads();
#pragma unroll 1
  for (int i0 = 0; i0 < n8; i0 += 3 * WT_THREADS) {
#pragma unroll
    for (int q = 0; q < 3; ++q) {
      const int i = i0 + tid + q * WT_THREADS;
      if (i < n8) {
        const uint4 w = i0 == 0 ? v[q] : __ldcg(sb8 + i);
        s_bin8[i] = w;
        const unsigned ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (8 * i + 2 * e < Fn) atomicAdd(&s_hist[ww[e] & 0xffffu], 1u);
          if (8 * i + 2 * e + 1 < Fn) atomicAdd(&s_hist[ww[e] >> 16], 1u);
        }
      }
    }
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
      const unsigned t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) sh.redu[warp] = incl;
    __syncthreads();
    unsigned wtot = lane < WT_WARPS ? sh.redu[lane] : 0u, wincl = wtot;
#pragma unroll
    for (int o = 1; o < WT_WARPS; o <<= 1) {
      const unsigned t = __shfl_up_sync(0xffffffffu, wincl, o);
      if (lane >= o) wincl += t;
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
  const int blo = sh.blo, bhi = sh.bhi;
  if (hi > lo || want_mask) {
    // the members of the covering bins (the bins are read back from shared memory, eight at a time)
#pragma unroll 1
    for (int i = tid; i < n8; i += WT_THREADS) {
      const uint4 w = s_bin8[i];
      const unsigned ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int b = (int)((e & 1) ? ww[e >> 1] >> 16 : ww[e >> 1] & 0xffffu), idx = 8 * i + e;
        if (idx < Fn) {
          if (b >= blo && b <= bhi) {
            const int pos = atomicAdd(&sh.ncand, 1);
            if (pos < WT_CANDCAP) { s_cidx[pos] = idx; s_cbin[pos] = (uint16_t)b; }
          } else if (want_mask && b < blo) {
            atomicOr(&s_bits[idx >> 5], 1u << (idx & 31));
          }
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
__device__ __noinline__ void wt_select_general(const WtCall& C, unsigned char* smem, int j, int Fn, int keff, int32_t* ranked, bool want_mask,
                                               unsigned long long* cut_out) {
  unsigned* s_bits = reinterpret_cast<unsigned*>(smem + C.lay.bits_off);
  const double* sc = C.sc + (size_t)j * Fn;
  __syncthreads();
  if (keff <= 0) return;
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
    wt_select_general(C, smem, j, Fn, keff, nullptr, mask_out != nullptr, cut_out);
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
template <int WD, int CPT>
__global__ void __launch_bounds__(WT_THREADS, 1) ls_token_kernel(const WtLayer* __restrict__ g_layers, const __grid_constant__ WtCall C) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ WtShared sh;
  const int tid = threadIdx.x, cta = blockIdx.x, G = gridDim.x;
  const int d = C.d, K = C.K, E = K + 1;
  float* s_x = reinterpret_cast<float*>(smem + C.lay.x_off);
  int* s_mine = reinterpret_cast<int*>(smem + C.lay.mine_off);
  constexpr int NW = sizeof(WtLayer) / 4;
  const int n_act = C.gs * K;
  const bool active = cta < n_act;
  const bool stamps = C.tr_ns != nullptr && tid == 0;
  unsigned epoch = 0;

  // ---- prologue: arguments of layer 0, x, 1 / rms, this CTA's slice of the first selection
  if (tid < NW) reinterpret_cast<uint32_t*>(&sh.L[0])[tid] = reinterpret_cast<const uint32_t*>(&g_layers[0])[tid];
  if (tid == 0) sh.dead = 0;
  {
    double sq = 0.0;
    for (int c = tid * 4; c < d; c += WT_THREADS * 4) {
      const float4 v = __ldcg(reinterpret_cast<const float4*>(C.x_in + c));
      *reinterpret_cast<float4*>(s_x + c) = v;
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

#pragma unroll 1
  for (int n = 0; n < C.n_layers; ++n) {
    const WtLayer& L = sh.L[n & 1];
    const bool last = n + 1 == C.n_layers;
    const int rz = (L.r + 4) & ~3;
    const int keff = min(C.k_next, L.Fn);
    if (stamps) wt_stamp(C, n, 0);
    // next layer's arguments
    if (!last && tid >= WT_THREADS - NW)
      reinterpret_cast<uint32_t*>(&sh.L[(n + 1) & 1])[tid - (WT_THREADS - NW)] =
          reinterpret_cast<const uint32_t*>(&g_layers[n + 1])[tid - (WT_THREADS - NW)];
    // ---- S
    wt_stream<WD, CPT>(C, sh, L, smem, active);
    if (stamps) wt_stamp(C, n, 1);
    wt_grid_sync(C, sh, ++epoch * G);
    if (sh.dead) return;
    if (stamps) wt_stamp(C, n, 2);
    // ---- P1
    float* x_out = last ? C.x_out : C.xbuf + (size_t)((n + 1) & 1) * d;
    wt_feature<WD>(C, sh, L, smem, n, x_out, E, rz);
    if (stamps) wt_stamp(C, n, 3);
    wt_grid_sync(C, sh, ++epoch * G);
    if (sh.dead) return;
    if (stamps) wt_stamp(C, n, 4);
    // ---- P2
    wt_latent_sums(C, L.r, E, rz);
    if (!last) {
#pragma unroll 1
      for (int c = tid * 4; c < d; c += WT_THREADS * 4) *reinterpret_cast<float4*>(s_x + c) = __ldcg(reinterpret_cast<const float4*>(x_out + c));
    }
    if (stamps) wt_stamp(C, n, 5);
    wt_grid_sync(C, sh, ++epoch * G);
    if (sh.dead) return;
    if (stamps) wt_stamp(C, n, 6);
    // ---- P3
    wt_scores<WD>(C, sh, L, smem, E, rz, last);
    if (stamps) wt_stamp(C, n, 7);
    wt_grid_sync(C, sh, ++epoch * G);
    if (sh.dead) return;
    if (stamps) wt_stamp(C, n, 8);
    // ---- P4
    int lo, hi;
    wt_share(keff, K, C.gs, cta, lo, hi);
    if (tid == 0) sh.inv_x = (float)sh.inv[K];
    unsigned long long* cuts = C.cuts + (size_t)n * E;  // the keys of the last members of this layer's refined sets
    if (!wt_select(C, sh, K, L.Fn, keff, lo, hi, C.lay.mine_off, false, cuts + K)) {
      if (cta == 0) wt_select_general(C, smem, K, L.Fn, keff, C.sellist, false, cuts + K);
      wt_grid_sync(C, sh, ++epoch * G);
      if (sh.dead) return;
      if (tid < hi - lo) s_mine[tid] = __ldcg(C.sellist + lo + tid);
      __syncthreads();
    }
    if (stamps) wt_stamp(C, n, 9);
    if (tid == 0) sh.nmine = hi - lo;
    if (last || C.tr_sel || C.tr_masks) wt_export_selection(C, s_mine, n, lo, hi - lo, keff, last);
    if (cta == 0 && tid < 32) wt_update_range(C, L);
    // refined sets of the evaluations j < K, on the CTAs with no rows to stream (when there are some)
    {
      const int n_idle = G - n_act;
#pragma unroll 1
      for (int j = 0; j < K; ++j) {
        const int owner = n_idle > 0 ? n_act + (j % n_idle) : G - 1 - (j % G);
        if (cta == owner)
          wt_refined_set(C, sh, smem, j, L.Fn, keff, C.tr_masks ? C.tr_masks + ((size_t)n * E + j) * C.tr_words : nullptr, cuts + j);
      }
    }
    __syncthreads();
    if (stamps) wt_stamp(C, n, 10);
  }
}

}  // namespace ls
