// Whole-token kernel: every layer of a resident stack for one decode token in ONE cooperative launch (batch 1).
//
// A grid barrier costs about 2,300 SM clocks on this GPU whatever its form (one L2 round trip to arrive, one to see the
// last arrival), which is as long as a layer's whole weight traffic takes at full HBM speed.  The layer step is therefore
// organised around FOUR barriers, the fewest the data flow allows, and every phase between them is kept short:
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
//   P3 scores    Every CTA scores its share of the next layer's neurons for all K+1 evaluations (fp64), stores the scores
//                and their bin under a monotone linear map.
//      -- barrier 4 --
//   P4 select    EVERY CTA reads the bins of the final evaluation, builds the histogram and its prefix sum in shared
//                memory and finds by itself the neurons whose rank falls in ITS slice of the next layer's ranks: the bins
//                that cover the slice, their members, exact comparison of the members' keys.  Nothing is exchanged, so
//                the next layer's stream phase starts without a further barrier.  The refined sets of the evaluations
//                j < K (Section 2.1: they steer fetching and retention, nothing on a resident stack waits for them) are
//                established meanwhile by the CTAs that have no rows to stream.
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
__host__ __device__ inline int wt_feat_pos(int c) { return (c >> 5) * WT_XBLK + ((c >> 3) & 3) * 10 + (c & 7); }
__host__ __device__ inline int wt_feat_stride(int cols) {
  const int nb = (cols + 31) >> 5;
  return nb * WT_XBLK + ((nb & 1) ? 0 : 8);
}
// evaluations handled by MMA tiles of eight, the rest (at most two) by plain FMAs
__host__ __device__ inline int wt_tiles(int E) { return E <= 2 ? 0 : (E <= 10 ? 1 : 2); }
__host__ __device__ inline int wt_plain(int E) { const int p = E - 8 * wt_tiles(E); return p > 0 ? p : 0; }
__host__ __device__ inline int wt_rows(int E) { return 8 * wt_tiles(E) + wt_plain(E); }

struct WtLayer {  // one per layer of the stack (device array)
  const uint16_t* bundles; const float* b_gate; const float* b_down;
  int n_mat, F, norm; float eps;
  // predictor of the layer this one refines (the next layer; the last layer refines itself)
  const uint16_t* At_sl; const uint16_t* Bt; const float* pc;
  int r, Fn, norm_n; float eps_n;
  double* range;  // [2] {hi, scale} of the score bins, refreshed by every launch for the next one
  int* status;
};

struct WtSmem {  // byte offsets into dynamic shared memory (computed on the host)
  unsigned x_off, xt_off, dm_off, mine_off, bits_off, u_off;
  // inside the union region u (disjoint lifetimes): A slices [S..P1] | z rows [P3] | selection [P4] | top-k fallback
  unsigned bin_off, hist_off, pref_off, ckey_off, cidx_off;
  unsigned total;
};

struct WtCall {
  int n_layers, d, K, k_next, piece_len, gs;  // gs: CTAs per stage
  int rz_max;
  const float* x_in; float* x_out;
  const int32_t* sel_idx; const int32_t* sel_count; int sel_cap;
  int32_t* out_idx; int32_t* out_count; uint32_t* out_mask; double* out_scores; int out_cap;
  // scratch shared by all layers
  float* xbuf;        // [2][d]
  float* ypart;       // [G][d]
  double* zpart;      // [slices][E][rz]
  double* z;          // [E][rz]
  double* sc;         // [E][Fn]
  uint16_t* sb;       // [E][Fn]
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
  int nmine, lo, nsurv;
  int wcnt[WT_WARPS];
  int blo, bhi, ncand, slow, found;
  float inv_x;            // 1 / rms of the layer's input
  double inv[WT_MAXE + 7];
  double redd[2 * WT_WARPS];
  unsigned long long redk[2 * WT_WARPS];
  unsigned redu[WT_WARPS + 1];
};

// ---- small helpers -----------------------------------------------------------------------------------------------------
template <int WD>
__device__ __forceinline__ double wt_w16_to_double(uint16_t b) {
  if (WD == WD_BF16) return (double)__uint_as_float((uint32_t)b << 16);
  return (double)__half2float(__ushort_as_half(b));
}
template <int WD>
__device__ __forceinline__ void wt_cvt8(const uint4 w, double a[8]) {
  const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    a[2 * q] = wt_w16_to_double<WD>((uint16_t)(ww[q] & 0xffffu));
    a[2 * q + 1] = wt_w16_to_double<WD>((uint16_t)(ww[q] >> 16));
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
__device__ __forceinline__ long long wt_now_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return (long long)t;
}
__device__ __forceinline__ void wt_cp_async16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void wt_cp_async_wait() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ void wt_prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

// Barrier among all CTAs of the cooperatively launched grid.  The counter is zeroed before the launch and only grows:
// the e-th barrier completes when it reaches e * G.  Arrival is a release (reduction, nothing comes back), the poll an
// acquire.  Split in two so that work that needs nothing from the other CTAs can run between arriving and waiting.
__device__ __forceinline__ void wt_arrive(const WtCall& C, WtShared& sh) {
  __syncthreads();
  if (threadIdx.x == 0 && !sh.dead) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(C.bar) : "memory");
}
__device__ __noinline__ void wt_poll(const WtCall& C, WtShared& sh, unsigned target) {
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
__device__ __forceinline__ void wt_wait(const WtCall& C, WtShared& sh, unsigned target) {
  if (threadIdx.x == 0 && !sh.dead) wt_poll(C, sh, target);
  __syncthreads();
}

// This CTA's slice [lo, hi) of the ranks of a selection of `count` neurons run in K stages on groups of `gs` CTAs.
__device__ __forceinline__ void wt_share(int count, int K, int gs, int cta, int& lo, int& hi) {
  const int c = cta / gs;
  if (c >= K || count <= 0) { lo = hi = 0; return; }
  const int m = (count + K - 1) / K;
  const int s_lo = min(count, c * m), s_hi = min(count, (c + 1) * m);
  const int per = (m + gs - 1) / gs;
  lo = min(s_hi, s_lo + (cta - c * gs) * per);
  hi = min(s_hi, lo + per);
}

// ---- S: gate rows, survivors, up and down rows -----------------------------------------------------------------------
// Dot products of up to three rows with x: warp (p, q) = (warp % 4, warp / 4) takes piece p of the rows q, q + 4, q + 8 of
// the list, four 16-byte loads per row and lane, all issued before the first is used.
template <int WD>
__device__ __forceinline__ void wt_rows_dot(const uint16_t* const (&row)[3], const bool (&ok)[3], const float* s_x, int c_lo, int c_hi,
                                            int lane, float (&acc)[3]) {
  acc[0] = acc[1] = acc[2] = 0.f;
#pragma unroll 1
  for (int cb = c_lo; cb < c_hi; cb += 1024) {
    uint4 w[3][4];
#pragma unroll
    for (int q = 0; q < 3; ++q)
#pragma unroll
      for (int it = 0; it < 4; ++it) {
        const int c = cb + it * 256 + lane * 8;
        w[q][it] = (ok[q] && c < c_hi) ? ld_stream128(row[q] + c) : make_uint4(0u, 0u, 0u, 0u);
      }
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      const int c = cb + it * 256 + lane * 8;
      if (c < c_hi) {
        const float4 x0 = *reinterpret_cast<const float4*>(s_x + c);
        const float4 x1 = *reinterpret_cast<const float4*>(s_x + c + 4);
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
#pragma unroll
  for (int q = 0; q < 3; ++q) acc[q] = warp_sum(acc[q]);
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
  float* s_up = s_sact + WT_MAXMINE;                                     // [2][8][4] partial up dot products of a batch
  const int nmine = sh.nmine;
  const float inv = sh.inv_x;
  const size_t bstride = (size_t)L.n_mat * d;
  const int p = warp & 3, wq = warp >> 2;
  const int c_lo = min(d, p * C.piece_len), c_hi = min(d, c_lo + C.piece_len);

  // gate bias of "my" neuron (used after the dot products; the load is in flight meanwhile)
  int my_idx = -1;
  float my_b = 0.f;
  if (tid < nmine) {
    my_idx = s_mine[tid];
    if ((unsigned)my_idx >= (unsigned)L.F) { my_idx = -1; set_status(L.status, ST_BAD_INDEX); }
    else if (L.b_gate) my_b = __ldg(L.b_gate + my_idx);
  }
#pragma unroll 1
  for (int i0 = wq; i0 < nmine; i0 += 12) {
    const uint16_t* row[3];
    bool ok[3];
#pragma unroll
    for (int q = 0; q < 3; ++q) {
      const int i = i0 + 4 * q;
      const int v = i < nmine ? s_mine[i] : -1;
      ok[q] = (unsigned)v < (unsigned)L.F;
      row[q] = L.bundles + (size_t)(ok[q] ? v : 0) * bstride;
    }
    float acc[3];
    wt_rows_dot<WD>(row, ok, s_x, c_lo, c_hi, lane, acc);
    if (lane == 0) {
#pragma unroll
      for (int q = 0; q < 3; ++q)
        if (i0 + 4 * q < nmine) s_gsum[(i0 + 4 * q) * 4 + p] = acc[q];
    }
  }
  __syncthreads();
  // activation of the gate branch and the ordered list of survivors (a_i = relu(g_i) u_i: g_i <= 0 needs no other row)
  {
    float g = 0.f;
    if (my_idx >= 0) g = ((s_gsum[tid * 4] + s_gsum[tid * 4 + 1]) + (s_gsum[tid * 4 + 2] + s_gsum[tid * 4 + 3])) * inv + my_b;
    const bool sv = my_idx >= 0 && g > 0.f;
    const unsigned m = __ballot_sync(0xffffffffu, sv);
    if (lane == 0) sh.wcnt[warp] = __popc(m);
    __syncthreads();
    if (sv) {
      int off = __popc(m & ((1u << lane) - 1u));
      for (int w = 0; w < warp; ++w) off += sh.wcnt[w];
      s_sidx[off] = my_idx;
      s_sact[off] = g;
    }
    if (tid == 0) {
      int t = 0;
      for (int w = 0; w < WT_WARPS; ++w) t += sh.wcnt[w];
      sh.nsurv = t;
    }
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
  const size_t down_off = (size_t)(L.n_mat - 1) * d;
#pragma unroll 1
  for (int b0 = 0, bi = 0; b0 < nsurv; b0 += NB, ++bi) {
    const int nb = min(NB, nsurv - b0);
    uint4 dw[NB][CPT];
#pragma unroll
    for (int s = 0; s < NB; ++s)
#pragma unroll
      for (int cp = 0; cp < CPT; ++cp) {
        const int col = (tid + cp * WT_THREADS) * 8;
        dw[s][cp] = (s < nb && col < d) ? ld_stream128(L.bundles + (size_t)s_sidx[b0 + s] * bstride + down_off + col)
                                        : make_uint4(0u, 0u, 0u, 0u);
      }
    if (gated) {
      float* up = s_up + (bi & 1) * 32;
      const uint16_t* row[3];
      bool ok[3];
#pragma unroll
      for (int q = 0; q < 3; ++q) {
        const int s = wq + 4 * q;
        ok[q] = s < nb;
        row[q] = L.bundles + (size_t)(ok[q] ? s_sidx[b0 + s] : 0) * bstride + d;
      }
      float acc[3];
      wt_rows_dot<WD>(row, ok, s_x, c_lo, c_hi, lane, acc);
      if (lane == 0) {
#pragma unroll
        for (int q = 0; q < 2; ++q)
          if (wq + 4 * q < nb) up[(wq + 4 * q) * 4 + p] = acc[q];
      }
      __syncthreads();
    }
#pragma unroll
    for (int s = 0; s < NB; ++s) {
      if (s < nb) {
        float a = s_sact[b0 + s];
        if (gated) {
          const float* up = s_up + (bi & 1) * 32 + s * 4;
          a *= ((up[0] + up[1]) + (up[2] + up[3])) * inv;
        }
#pragma unroll
        for (int cp = 0; cp < CPT; ++cp) {
          float f[8];
          unpack8<WD>(dw[s][cp], f);
#pragma unroll
          for (int e = 0; e < 8; ++e) acc8[cp][e] = fmaf(a, f[e], acc8[cp][e]);
        }
      }
    }
  }
  if (active) {
    float* yp = C.ypart + (size_t)blockIdx.x * d;
#pragma unroll
    for (int cp = 0; cp < CPT; ++cp) {
      const int col = (tid + cp * WT_THREADS) * 8;
      if (col < d) {
        __stcg(reinterpret_cast<float4*>(yp + col), make_float4(acc8[cp][0], acc8[cp][1], acc8[cp][2], acc8[cp][3]));
        __stcg(reinterpret_cast<float4*>(yp + col + 4), make_float4(acc8[cp][4], acc8[cp][5], acc8[cp][6], acc8[cp][7]));
      }
    }
  }
}

// ---- P1: stage sums, partial residual features, x_out, partial latents of this CTA's slices ----------------------------
template <int WD>
__device__ __forceinline__ void wt_feature(const WtCall& C, WtShared& sh, const WtLayer& L, unsigned char* smem, int n, float* x_out,
                                           int E, int rz) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const int d = C.d, K = C.K, G = gridDim.x, r = L.r;
  const float* s_x = reinterpret_cast<const float*>(smem + C.lay.x_off);
  double* s_xt = reinterpret_cast<double*>(smem + C.lay.xt_off);  // [rows][WT_XBLK]
  float* s_dm = reinterpret_cast<float*>(smem + C.lay.dm_off);    // [K][32]
  const uint16_t* s_a = reinterpret_cast<const uint16_t*>(smem + C.lay.u_off);
  const int nsl = (d + 31) >> 5;
  const int ntile = wt_tiles(E), nplain = wt_plain(E), rows = wt_rows(E);
  wt_cp_async_wait();
  __syncthreads();
#pragma unroll 1
  for (int s = blockIdx.x, si = 0; s < nsl; s += G, ++si) {
    const int col = 32 * s + lane;
    if (warp < K) {
      float a = 0.f;
      if (col < d) {
        const float* yp = C.ypart + (size_t)warp * C.gs * d + col;
#pragma unroll 6
        for (int c = 0; c < C.gs; ++c) a += __ldcg(yp + (size_t)c * d);
      }
      s_dm[warp * 32 + lane] = a;
    }
    __syncthreads();
    if (warp == 0) {
      float xt = 0.f;
      if (col < d) xt = s_x[col] + (L.b_down ? __ldg(L.b_down + col) : 0.f);
      const int pos = wt_feat_pos(lane);
      double* zp = C.zpart + (size_t)s * E * rz + r;
#pragma unroll 1
      for (int e = 0; e <= K; ++e) {
        s_xt[e * WT_XBLK + pos] = (double)xt;
        if (C.tr_xtilde && col < d) C.tr_xtilde[((size_t)n * E + e) * d + col] = xt;
        const double sq = warp_sum((double)xt * (double)xt);
        if (lane == 0) __stcg(zp + (size_t)e * rz, sq);
        if (e < K) xt += s_dm[e * 32 + lane];
      }
      for (int e = E; e < rows; ++e) s_xt[e * WT_XBLK + pos] = 0.0;
      if (col < d) {
        __stcg(x_out + col, xt);
        if (C.tr_x) C.tr_x[(size_t)(n + 1) * d + col] = xt;
      }
    }
    __syncthreads();
    // partial latents: m-tiles of eight rows of A^T (the slice holds [r][32] 16-bit weights)
    const uint16_t* a_sl = s_a + (size_t)si * r * 32;
    double f0[8], f1[8];
    if (ntile > 0) wt_load8d(s_xt + g * WT_XBLK + t * 10, f0);
    if (ntile > 1) wt_load8d(s_xt + (8 + g) * WT_XBLK + t * 10, f1);
#pragma unroll 1
    for (int mt = warp; mt < (r >> 3); mt += WT_WARPS) {
      const int l = 8 * mt + g;
      double a[8];
      wt_cvt8<WD>(*reinterpret_cast<const uint4*>(a_sl + (size_t)l * 32 + 8 * t), a);
      double* zp = C.zpart + (size_t)s * E * rz + l;
      if (ntile > 0) {
        double c[2] = {0.0, 0.0};
        wt_mma_block(c, a, f0);
        if (2 * t < E) __stcg(zp + (size_t)(2 * t) * rz, c[0]);
        if (2 * t + 1 < E) __stcg(zp + (size_t)(2 * t + 1) * rz, c[1]);
      }
      if (ntile > 1) {
        double c[2] = {0.0, 0.0};
        wt_mma_block(c, a, f1);
        if (8 + 2 * t < E) __stcg(zp + (size_t)(8 + 2 * t) * rz, c[0]);
        if (8 + 2 * t + 1 < E) __stcg(zp + (size_t)(8 + 2 * t + 1) * rz, c[1]);
      }
#pragma unroll 1
      for (int q = 0; q < nplain; ++q) {
        const int e = 8 * ntile + q;
        double f[8];
        wt_load8d(s_xt + e * WT_XBLK + t * 10, f);
        double pa = 0.0;
#pragma unroll
        for (int k = 0; k < 8; ++k) pa = fma(a[k], f[k], pa);
        pa += __shfl_xor_sync(0xffffffffu, pa, 1);
        pa += __shfl_xor_sync(0xffffffffu, pa, 2);
        if (t == 0) __stcg(zp + (size_t)e * rz, pa);
      }
    }
    __syncthreads();
  }
}

// ---- P2: latents and sums of squares from the slices' partials ---------------------------------------------------------
__device__ __forceinline__ void wt_latent_sums(const WtCall& C, int r, int E, int rz) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, sg = lane >> 2, v = lane & 3;
  const int nsl = (C.d + 31) >> 5, ngrp = rz >> 2, units = E * ngrp, G = gridDim.x;
#pragma unroll 1
  for (int u = blockIdx.x * WT_WARPS + warp; u < units; u += G * WT_WARPS) {
    const int e = u / ngrp, l = 4 * (u - e * ngrp) + v;
    double a = 0.0;
    if (l <= r) {
      const double* zp = C.zpart + (size_t)e * rz + l;
#pragma unroll 4
      for (int s = sg; s < nsl; s += 8) a += __ldcg(zp + (size_t)s * E * rz);
    }
    a += __shfl_xor_sync(0xffffffffu, a, 4);
    a += __shfl_xor_sync(0xffffffffu, a, 8);
    a += __shfl_xor_sync(0xffffffffu, a, 16);
    if (sg == 0 && l <= r) __stcg(C.z + (size_t)e * rz + l, a);
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
  double* s_z = reinterpret_cast<double*>(smem + C.lay.u_off);
  const int RS = wt_feat_stride(r);
  const int ntile = wt_tiles(E), nplain = wt_plain(E), rows = wt_rows(E);
  const int nblk = (r + 31) >> 5;
  // latents to shared memory in the block layout; 1 / rms of every evaluation
  for (int i = tid; i < rows * RS; i += WT_THREADS) s_z[i] = 0.0;
  __syncthreads();
  for (int i = tid; i < E * r; i += WT_THREADS) {
    const int e = i / r, c = i - e * r;
    s_z[e * RS + wt_feat_pos(c)] = __ldcg(C.z + (size_t)e * rz + c);
  }
  if (tid < E) {
    const double ss = __ldcg(C.z + (size_t)tid * rz + r);
    sh.inv[tid] = L.norm_n == 0 ? 1.0 / sqrt(ss / (double)C.d + (double)L.eps_n) : 1.0;
  }
  const double hi = L.range[0], scale = L.range[1];
  __syncthreads();
  const int per = (Fn + G - 1) / G, n0 = min(Fn, (int)blockIdx.x * per), n1 = min(Fn, n0 + per);
  const int n_mt = (n1 - n0 + 7) >> 3;
  unsigned long long kmin = 0xffffffffffffffffULL, kmax = 0ULL;
#pragma unroll 1
  for (int mt = warp; mt < n_mt; mt += WT_WARPS) {
    const int row = n0 + 8 * mt + g;
    const bool valid = row < n1;
    const uint16_t* wrow = L.Bt + (size_t)(valid ? row : n0) * r + 8 * t;
    double c0[2] = {0.0, 0.0}, c1[2] = {0.0, 0.0}, pl[2] = {0.0, 0.0};
#pragma unroll 1
    for (int b0 = 0; b0 < nblk; b0 += 8) {
      uint4 w[8];
#pragma unroll
      for (int b = 0; b < 8; ++b)
        w[b] = (valid && (b0 + b) * 32 + 8 * t < r) ? ldg128(wrow + (b0 + b) * 32) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
      for (int b = 0; b < 8; ++b) {
        if (b0 + b < nblk) {
          double a[8], f[8];
          wt_cvt8<WD>(w[b], a);
          const double* zb = s_z + (b0 + b) * WT_XBLK + t * 10;
          if (ntile > 0) { wt_load8d(zb + g * RS, f); wt_mma_block(c0, a, f); }
          if (ntile > 1) { wt_load8d(zb + (8 + g) * RS, f); wt_mma_block(c1, a, f); }
#pragma unroll
          for (int q = 0; q < 2; ++q)
            if (q < nplain) {
              wt_load8d(zb + (8 * ntile + q) * RS, f);
#pragma unroll
              for (int k = 0; k < 8; ++k) pl[q] = fma(a[k], f[k], pl[q]);
            }
        }
      }
    }
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      pl[q] += __shfl_xor_sync(0xffffffffu, pl[q], 1);
      pl[q] += __shfl_xor_sync(0xffffffffu, pl[q], 2);
    }
    const double pcv = (valid && L.pc) ? (double)__ldg(L.pc + row) : 0.0;
    // this lane's evaluations: 2t, 2t+1 of every tile; lane t == q finishes plain evaluation q
    auto finish = [&](int e, double dot) {
      if (!valid || e >= E) return;
      const double s = canonical_score(dot * sh.inv[e] + pcv);
      __stcg(C.sc + (size_t)e * Fn + row, s);
      C.sb[(size_t)e * Fn + row] = (uint16_t)wt_bin_of(s, hi, scale);
      if (e == K) {
        if (last && C.out_scores) C.out_scores[row] = s;
        if (fabs(s) <= 1.7976931348623157e308) {
          const unsigned long long key = ordered_key(s);
          kmin = min(kmin, key);
          kmax = max(kmax, key);
        }
      }
    };
    if (ntile > 0) { finish(2 * t, c0[0]); finish(2 * t + 1, c0[1]); }
    if (ntile > 1) { finish(8 + 2 * t, c1[0]); finish(8 + 2 * t + 1, c1[1]); }
    if (t < nplain) finish(8 * ntile + t, t == 0 ? pl[0] : pl[1]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
    kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
  }
  if (lane == 0) { sh.redk[warp] = kmin; sh.redk[WT_WARPS + warp] = kmax; }
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < WT_WARPS; ++w) { kmin = min(kmin, sh.redk[w]); kmax = max(kmax, sh.redk[WT_WARPS + w]); }
    __stcg(C.kmm + 2 * blockIdx.x, kmin);
    __stcg(C.kmm + 2 * blockIdx.x + 1, kmax);
  }
}

// ---- P4: selection ---------------------------------------------------------------------------------------------------
// Bins of one evaluation to shared memory, histogram and exclusive prefix sum (pref[WT_NB] = Fn).
__device__ __forceinline__ void wt_hist_scan(const WtCall& C, WtShared& sh, unsigned char* smem, const uint16_t* sb, int Fn) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint16_t* s_bin = reinterpret_cast<uint16_t*>(smem + C.lay.u_off + C.lay.bin_off);
  unsigned* s_hist = reinterpret_cast<unsigned*>(smem + C.lay.u_off + C.lay.hist_off);
  unsigned* s_pref = reinterpret_cast<unsigned*>(smem + C.lay.u_off + C.lay.pref_off);
  for (int i = tid; i < WT_NB / 4; i += WT_THREADS) reinterpret_cast<uint4*>(s_hist)[i] = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  if ((reinterpret_cast<size_t>(sb) & 15) == 0) {
    const int n8 = Fn >> 3;
    for (int i = tid; i < n8; i += WT_THREADS) {
      const uint4 v = __ldcg(reinterpret_cast<const uint4*>(sb) + i);
      reinterpret_cast<uint4*>(s_bin)[i] = v;
      const unsigned ww[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        atomicAdd(&s_hist[ww[q] & 0xffffu], 1u);
        atomicAdd(&s_hist[ww[q] >> 16], 1u);
      }
    }
    for (int i = (n8 << 3) + tid; i < Fn; i += WT_THREADS) {
      const uint16_t b = __ldcg(sb + i);
      s_bin[i] = b;
      atomicAdd(&s_hist[b], 1u);
    }
  } else {
    for (int i = tid; i < Fn; i += WT_THREADS) {
      const uint16_t b = __ldcg(sb + i);
      s_bin[i] = b;
      atomicAdd(&s_hist[b], 1u);
    }
  }
  __syncthreads();
  constexpr int BPT = WT_NB / WT_THREADS;
  unsigned cnt[BPT], run = 0;
#pragma unroll
  for (int e = 0; e < BPT; ++e) { cnt[e] = s_hist[tid * BPT + e]; run += cnt[e]; }
  unsigned incl = run;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) sh.redu[warp] = incl;
  __syncthreads();
  unsigned base = incl - run;
  for (int w = 0; w < warp; ++w) base += sh.redu[w];
#pragma unroll
  for (int e = 0; e < BPT; ++e) { s_pref[tid * BPT + e] = base; base += cnt[e]; }
  if (tid == WT_THREADS - 1) s_pref[WT_NB] = base;
  __syncthreads();
}

// The refined set of an evaluation j < K (and, as the slow route, of the final one): exact top-k by ONE CTA.
// Fast: histogram, cut bin, exact comparison inside the cut bin.  Slow (cut bin too full): the general block top-k.
// Writes the key of the set's last member, the membership mask when a trace asks for it, and the ranked list when
// `ranked` is given (slow route of the final evaluation).
__device__ __noinline__ void wt_select_one(const WtCall& C, WtShared& sh, unsigned char* smem, int n, int j, int Fn, int keff,
                                           uint32_t* mask_out, int32_t* ranked, int* status) {
  const int tid = threadIdx.x;
  const int E = C.K + 1;
  uint16_t* s_bin = reinterpret_cast<uint16_t*>(smem + C.lay.u_off + C.lay.bin_off);
  unsigned* s_hist = reinterpret_cast<unsigned*>(smem + C.lay.u_off + C.lay.hist_off);
  unsigned* s_pref = reinterpret_cast<unsigned*>(smem + C.lay.u_off + C.lay.pref_off);
  unsigned long long* s_ckey = reinterpret_cast<unsigned long long*>(smem + C.lay.u_off + C.lay.ckey_off);
  int* s_cidx = reinterpret_cast<int*>(smem + C.lay.u_off + C.lay.cidx_off);
  unsigned* s_bits = reinterpret_cast<unsigned*>(smem + C.lay.bits_off);
  const double* sc = C.sc + (size_t)j * Fn;
  const int nwords = (Fn + 31) >> 5;
  if (mask_out)
    for (int w = tid; w < nwords; w += WT_THREADS) s_bits[w] = 0u;
  unsigned long long* cut_out = C.cuts + (size_t)n * E + j;
  if (keff <= 0) {
    if (tid == 0) *cut_out = 0xffffffffffffffffULL;
    if (mask_out) { __syncthreads(); for (int w = tid; w < nwords; w += WT_THREADS) mask_out[w] = 0u; }
    return;
  }
  bool slow = ranked != nullptr;
  int cb = 0;
  if (!slow) {
    wt_hist_scan(C, sh, smem, C.sb + (size_t)j * Fn, Fn);
    // cut bin: the bin that holds rank keff - 1
    if (tid == 0) sh.blo = 0;
    __syncthreads();
    constexpr int BPT = WT_NB / WT_THREADS;
#pragma unroll
    for (int e = 0; e < BPT; ++e) {
      const int b = tid * BPT + e;
      if ((int)s_pref[b] <= keff - 1 && (int)s_pref[b + 1] > keff - 1) sh.blo = b;
    }
    __syncthreads();
    cb = sh.blo;
    slow = (int)s_hist[cb] > WT_CANDCAP;
  }
  if (!slow) {
    if (tid == 0) sh.ncand = 0;
    __syncthreads();
    for (int i = tid; i < Fn; i += WT_THREADS) {
      const int b = s_bin[i];
      if (b == cb) {
        const int pos = atomicAdd(&sh.ncand, 1);
        if (pos < WT_CANDCAP) { s_cidx[pos] = i; s_ckey[pos] = ordered_key(__ldcg(sc + i)); }
      } else if (mask_out && b < cb) {
        atomicOr(&s_bits[i >> 5], 1u << (i & 31));
      }
    }
    __syncthreads();
    const int ncand = min(sh.ncand, WT_CANDCAP);
    const int want = keff - (int)s_pref[cb];  // members taken from the cut bin
    for (int q = tid; q < ncand; q += WT_THREADS) {
      const unsigned long long kq = s_ckey[q];
      const int iq = s_cidx[q];
      int before = 0;
      for (int u = 0; u < ncand; ++u) {
        const unsigned long long ku = s_ckey[u];
        before += (ku > kq) || (ku == kq && s_cidx[u] < iq);
      }
      if (before < want) {
        if (mask_out) atomicOr(&s_bits[iq >> 5], 1u << (iq & 31));
        if (before == want - 1) *cut_out = kq;
      }
    }
  } else {
    // general route: exact for any input (all scores equal, a range that does not fit), only slower
    __syncthreads();
    TopkSmem sm = topk_carve(smem + C.lay.u_off);
    block_topk_nt<WT_THREADS>(
        Fn, keff,
        [&](int v, double& s) {
          s = __ldcg(sc + v);
          return true;
        },
        [&](int rank, int v) {
          if (ranked) ranked[rank] = v;
          if (mask_out) atomicOr(&s_bits[v >> 5], 1u << (v & 31));
          if (rank == keff - 1) *cut_out = ordered_key(canonical_score(__ldcg(sc + v)));
        },
        sm, C.tk_key, C.tk_idx);
  }
  (void)status;
  if (mask_out) {
    __syncthreads();
    for (int w = tid; w < nwords; w += WT_THREADS) mask_out[w] = s_bits[w];
  }
  __syncthreads();
}

// Final evaluation: this CTA's slice [lo, hi) of the ranks, found from the histogram without any exchange.
// Returns false when the selection has to take the slow route (decided alike by every CTA).
__device__ __forceinline__ bool wt_select_mine(const WtCall& C, WtShared& sh, unsigned char* smem, const WtLayer& L, int keff, int lo, int hi,
                                               unsigned long long* cut_out) {
  const int tid = threadIdx.x;
  const int Fn = L.Fn, K = C.K;
  uint16_t* s_bin = reinterpret_cast<uint16_t*>(smem + C.lay.u_off + C.lay.bin_off);
  unsigned* s_hist = reinterpret_cast<unsigned*>(smem + C.lay.u_off + C.lay.hist_off);
  unsigned* s_pref = reinterpret_cast<unsigned*>(smem + C.lay.u_off + C.lay.pref_off);
  unsigned long long* s_ckey = reinterpret_cast<unsigned long long*>(smem + C.lay.u_off + C.lay.ckey_off);
  int* s_cidx = reinterpret_cast<int*>(smem + C.lay.u_off + C.lay.cidx_off);
  int* s_mine = reinterpret_cast<int*>(smem + C.lay.mine_off);
  const double* sc = C.sc + (size_t)K * Fn;
  if (tid == 0) { sh.blo = WT_NB; sh.bhi = -1; sh.ncand = 0; sh.slow = 0; sh.found = 0; }
  wt_hist_scan(C, sh, smem, C.sb + (size_t)K * Fn, Fn);
  constexpr int BPT = WT_NB / WT_THREADS;
  {
    int blo = WT_NB, bhi = -1, slow = 0;
#pragma unroll
    for (int e = 0; e < BPT; ++e) {
      const int b = tid * BPT + e;
      const int p0 = (int)s_pref[b], p1 = (int)s_pref[b + 1];
      if (p1 > p0) {
        if (p0 < keff && p1 - p0 > WT_BINCAP) slow = 1;
        if (p0 < hi && p1 > lo) { blo = min(blo, b); bhi = max(bhi, b); }
      }
    }
    if (slow) sh.slow = 1;
    if (bhi >= 0) { atomicMin(&sh.blo, blo); atomicMax(&sh.bhi, bhi); }
  }
  __syncthreads();
  if (sh.slow) return false;
  const int blo = sh.blo, bhi = sh.bhi;
  if (hi > lo) {
    for (int i = tid; i < Fn; i += WT_THREADS) {
      const int b = s_bin[i];
      if (b >= blo && b <= bhi) {
        const int pos = atomicAdd(&sh.ncand, 1);
        if (pos < WT_CANDCAP) { s_cidx[pos] = i; s_ckey[pos] = ordered_key(__ldcg(sc + i)); }
      }
    }
  }
  __syncthreads();
  const int ncand = min(sh.ncand, WT_CANDCAP);
  for (int q = tid; q < ncand; q += WT_THREADS) {
    const unsigned long long kq = s_ckey[q];
    const int iq = s_cidx[q];
    const int bq = s_bin[iq];
    int before = 0;
    for (int u = 0; u < ncand; ++u) {
      const int iu = s_cidx[u];
      if (s_bin[iu] != bq) continue;
      const unsigned long long ku = s_ckey[u];
      before += (ku > kq) || (ku == kq && iu < iq);
    }
    const int rank = (int)s_pref[bq] + before;
    if (rank >= lo && rank < hi) {
      s_mine[rank - lo] = iq;
      atomicAdd(&sh.found, 1);
    }
    if (rank == keff - 1) *cut_out = kq;
  }
  __syncthreads();
  if (tid == 0 && (sh.found != hi - lo || sh.ncand > WT_CANDCAP)) set_status(L.status, ST_INTERNAL);
  return true;
}

// New bin range of the layer's scores from what this launch observed (one CTA; used by the next launch).
__device__ __forceinline__ void wt_update_range(const WtCall& C, const WtLayer& L) {
  const int tid = threadIdx.x, G = gridDim.x;
  if (tid >= 32) return;
  unsigned long long kmin = 0xffffffffffffffffULL, kmax = 0ULL;
  for (int c = tid; c < G; c += 32) {
    kmin = min(kmin, __ldcg(C.kmm + 2 * c));
    kmax = max(kmax, __ldcg(C.kmm + 2 * c + 1));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
    kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
  }
  if (tid == 0 && kmax >= kmin) {
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
  const bool active = cta / C.gs < K;
  unsigned epoch = 0;
  auto stamp = [&](int n, int slot) {
    if (C.tr_ns && tid == 0) C.tr_ns[((size_t)n * G + cta) * WT_NSTAMP + slot] = wt_now_ns();
  };

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
    sh.inv_x = sh.L[0].norm == 0 ? (float)(1.0 / sqrt(t / (double)d + (double)sh.L[0].eps)) : 1.0f;
  }
  {
    const int count0 = max(0, min(__ldg(C.sel_count), C.sel_cap));
    int lo, hi;
    wt_share(count0, K, C.gs, cta, lo, hi);
    if (tid < hi - lo) s_mine[tid] = __ldg(C.sel_idx + lo + tid);
    if (tid == 0) { sh.nmine = hi - lo; sh.lo = lo; }
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
    stamp(n, 0);
    // next layer's arguments, this CTA's slices of the predictor matrix A (asynchronously), and its rows of B^T into L2
    if (!last && tid >= WT_THREADS - NW)
      reinterpret_cast<uint32_t*>(&sh.L[(n + 1) & 1])[tid - (WT_THREADS - NW)] =
          reinterpret_cast<const uint32_t*>(&g_layers[n + 1])[tid - (WT_THREADS - NW)];
    {
      const int nsl = (d + 31) >> 5;
      const int per_slice = L.r * 4;  // 16-byte pieces per slice
      unsigned char* s_a = smem + C.lay.u_off;
      for (int s = cta, si = 0; s < nsl; s += G, ++si)
        for (int i = tid; i < per_slice; i += WT_THREADS)
          wt_cp_async16(s_a + ((size_t)si * per_slice + i) * 16, reinterpret_cast<const unsigned char*>(L.At_sl) + ((size_t)s * per_slice + i) * 16);
      const int per = (L.Fn + G - 1) / G, n0 = min(L.Fn, cta * per), n1 = min(L.Fn, n0 + per);
      const unsigned char* b0 = reinterpret_cast<const unsigned char*>(L.Bt + (size_t)n0 * L.r);
      const size_t bytes = (size_t)(n1 - n0) * L.r * 2;
      for (size_t o = (size_t)tid * 128; o < bytes; o += (size_t)WT_THREADS * 128) wt_prefetch_l2(b0 + o);
    }
    // ---- S
    wt_stream<WD, CPT>(C, sh, L, smem, active);
    stamp(n, 1);
    wt_arrive(C, sh);
    ++epoch;
    wt_wait(C, sh, epoch * G);
    if (sh.dead) return;
    stamp(n, 2);
    // ---- P1
    float* x_out = last ? C.x_out : C.xbuf + (size_t)((n + 1) & 1) * d;
    wt_feature<WD>(C, sh, L, smem, n, x_out, E, rz);
    stamp(n, 3);
    wt_arrive(C, sh);
    ++epoch;
    wt_wait(C, sh, epoch * G);
    if (sh.dead) return;
    stamp(n, 4);
    // ---- P2
    wt_latent_sums(C, L.r, E, rz);
    if (!last)
      for (int c = tid * 4; c < d; c += WT_THREADS * 4) *reinterpret_cast<float4*>(s_x + c) = __ldcg(reinterpret_cast<const float4*>(x_out + c));
    stamp(n, 5);
    wt_arrive(C, sh);
    ++epoch;
    wt_wait(C, sh, epoch * G);
    if (sh.dead) return;
    stamp(n, 6);
    // ---- P3
    wt_scores<WD>(C, sh, L, smem, E, rz, last);
    stamp(n, 7);
    wt_arrive(C, sh);
    ++epoch;
    wt_wait(C, sh, epoch * G);
    if (sh.dead) return;
    stamp(n, 8);
    // ---- P4
    int lo, hi;
    wt_share(keff, K, C.gs, cta, lo, hi);
    if (tid == 0) sh.inv_x = (float)sh.inv[K];
    bool fast = wt_select_mine(C, sh, smem, L, keff, lo, hi, C.cuts + (size_t)n * E + K);
    if (!fast) {
      if (cta == 0) wt_select_one(C, sh, smem, n, K, L.Fn, keff, nullptr, C.sellist, L.status);
      wt_arrive(C, sh);
      ++epoch;
      wt_wait(C, sh, epoch * G);
      if (sh.dead) return;
      if (tid < hi - lo) s_mine[tid] = __ldcg(C.sellist + lo + tid);
      __syncthreads();
    }
    stamp(n, 9);
    if (tid == 0) { sh.nmine = hi - lo; sh.lo = lo; }
    // what leaves the layer: the ranked list (trace, and the caller's list after the last layer), the masks
    if (tid < hi - lo) {
      const int v = s_mine[tid], rank = lo + tid;
      if (C.tr_sel && rank < C.tr_cap) C.tr_sel[(size_t)(n + 1) * C.tr_cap + rank] = v;
      if (C.tr_masks) atomicOr(C.tr_masks + ((size_t)n * E + K) * C.tr_words + (v >> 5), 1u << (v & 31));
      if (last) {
        if (rank < C.out_cap) C.out_idx[rank] = v;
        if (C.out_mask) atomicOr(C.out_mask + (v >> 5), 1u << (v & 31));
      }
    }
    if (cta == 0 && tid == 0) {
      if (C.tr_cnt) C.tr_cnt[n + 1] = keff;
      if (last) *C.out_count = min(keff, C.out_cap);
    }
    if (cta == 0) wt_update_range(C, L);
    // refined sets of the evaluations j < K: by the CTAs without rows to stream when there are some
    {
      const int n_act = C.gs * K, n_idle = G - n_act;
#pragma unroll 1
      for (int j = 0; j < K; ++j) {
        const int owner = n_idle > 0 ? n_act + (j % n_idle) : G - 1 - (j % G);
        if (cta == owner) {
          // (the selection work area is shared with this CTA's own list: keep the list)
          wt_select_one(C, sh, smem, n, j, L.Fn, keff, C.tr_masks ? C.tr_masks + ((size_t)n * E + j) * C.tr_words : nullptr, nullptr, L.status);
        }
      }
    }
    __syncthreads();
    stamp(n, 10);
  }
}

}  // namespace ls
