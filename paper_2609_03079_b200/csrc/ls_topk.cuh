// Exact top-k with ranks inside one CTA (1024 threads), shared by the selection and the cache kernels.
//
// Elements v in [0, F) carry an fp64 score; the order is total: score descending, then v ascending.  Scores are binned
// by a monotone linear map, a histogram and its prefix sum give the rank range of every bin, and every element of the
// bins that reach into the first k ranks gets its exact rank by comparison inside its bin.  Cost is O(F) plus the
// (short) bins around the cut; a degenerate input (all scores equal) is still exact, only slower.
#pragma once
#include "ls_common.cuh"

namespace ls {

constexpr int TK_THREADS = 1024;
constexpr int TK_NB = 4096;
constexpr int TK_LCAP = 6144;

struct TopkSmem {
  unsigned long long* key;  // [TK_LCAP] candidate keys
  uint32_t* base;           // [TK_NB] histogram, then exclusive prefix
  uint32_t* cur;            // [TK_NB] scatter cursors (end up as the bin counts of candidate bins)
  int32_t* idx;             // [TK_LCAP] candidate elements
  double* redd;             // [64]
  int* redi;                // [64]
  uint16_t* bin;            // [F]
};

__host__ __device__ inline size_t topk_smem_bytes(int F) {
  return (size_t)TK_LCAP * 8 + (size_t)TK_NB * 8 + (size_t)TK_LCAP * 4 + 64 * 8 + 64 * 4 + (((size_t)F * 2 + 15) & ~(size_t)15);
}

__device__ inline TopkSmem topk_carve(unsigned char* raw) {
  TopkSmem s;
  s.key = reinterpret_cast<unsigned long long*>(raw);
  s.redd = reinterpret_cast<double*>(s.key + TK_LCAP);
  s.base = reinterpret_cast<uint32_t*>(s.redd + 64);
  s.cur = s.base + TK_NB;
  s.idx = reinterpret_cast<int32_t*>(s.cur + TK_NB);
  s.redi = reinterpret_cast<int*>(s.idx + TK_LCAP);
  s.bin = reinterpret_cast<uint16_t*>(s.redi + 64);
  return s;
}

// keyfn(v, s): returns whether element v takes part and, if so, its score in s.
// emit(rank, v): called by exactly one thread for every element with rank < min(k, participants).
// Every thread of the NT-thread block must call this (NT = 1024 or 512); returns min(k, participants) to all of them.
// g_key / g_idx: global fallback arrays of F entries, used when the candidates do not fit in shared memory.
template <int NT, class KeyFn, class EmitFn>
__device__ int block_topk_nt(int F, int k, KeyFn keyfn, EmitFn emit, const TopkSmem& sm, unsigned long long* g_key, int32_t* g_idx) {
  constexpr int BPT = TK_NB / NT;  // bins per thread in the prefix sum
  constexpr int TK_THREADS = NT;   // (shadows the namespace constant inside this function)
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  __syncthreads();
  for (int i = tid; i < TK_NB; i += TK_THREADS) { sm.base[i] = 0u; sm.cur[i] = 0u; }

  const double INF = __longlong_as_double(0x7ff0000000000000LL);
  const double DMAX = 1.7976931348623157e308;
  double lo = INF, hi = -INF;
  int npart = 0;
  for (int v = tid; v < F; v += TK_THREADS) {
    double s;
    if (!keyfn(v, s)) continue;
    s = fmin(fmax(canonical_score(s), -DMAX), DMAX);
    lo = fmin(lo, s);
    hi = fmax(hi, s);
    ++npart;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    lo = fmin(lo, __shfl_xor_sync(0xffffffffu, lo, o));
    hi = fmax(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    npart += __shfl_xor_sync(0xffffffffu, npart, o);
  }
  if (lane == 0) { sm.redd[warp] = lo; sm.redd[32 + warp] = hi; sm.redi[warp] = npart; }
  __syncthreads();
  if (warp == 0) {
    const bool have = lane < NT / 32;
    lo = have ? sm.redd[lane] : INF; hi = have ? sm.redd[32 + lane] : -INF; npart = have ? sm.redi[lane] : 0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      lo = fmin(lo, __shfl_xor_sync(0xffffffffu, lo, o));
      hi = fmax(hi, __shfl_xor_sync(0xffffffffu, hi, o));
      npart += __shfl_xor_sync(0xffffffffu, npart, o);
    }
    if (lane == 0) { sm.redd[0] = lo; sm.redd[32] = hi; sm.redi[0] = npart; }
  }
  __syncthreads();
  lo = sm.redd[0]; hi = sm.redd[32]; npart = sm.redi[0];
  const int keff = min(k, npart);
  const double range = hi - lo;
  const double scale = (range > 0.0 && range < INF) ? (double)TK_NB / range : 0.0;
  __syncthreads();

  // bins (bin 0 holds the highest scores) and histogram
  for (int v = tid; v < F; v += TK_THREADS) {
    double s;
    if (!keyfn(v, s)) { sm.bin[v] = 0xffffu; continue; }
    s = fmin(fmax(canonical_score(s), -DMAX), DMAX);
    int b = (int)((hi - s) * scale);
    b = max(0, min(TK_NB - 1, b));
    sm.bin[v] = (uint16_t)b;
    atomicAdd(&sm.base[b], 1u);
  }
  __syncthreads();

  // exclusive prefix sum over the bins, BPT consecutive bins per thread
  uint32_t cnt[BPT], run = 0;
#pragma unroll
  for (int e = 0; e < BPT; ++e) { cnt[e] = sm.base[tid * BPT + e]; run += cnt[e]; }
  uint32_t incl = run;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) sm.redi[32 + warp] = (int)incl;
  __syncthreads();
  if (warp == 0) {
    const uint32_t w = lane < NT / 32 ? (uint32_t)sm.redi[32 + lane] : 0u;
    uint32_t wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t t = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += t;
    }
    sm.redi[32 + lane] = (int)(wi - w);
  }
  if (tid == 0) sm.redi[1] = 0;
  __syncthreads();
  uint32_t base = (uint32_t)sm.redi[32 + warp] + incl - run;
#pragma unroll
  for (int e = 0; e < BPT; ++e) {
    sm.base[tid * BPT + e] = base;
    if (cnt[e] > 0 && (int)base < keff && (int)(base + cnt[e]) >= keff) sm.redi[1] = (int)(base + cnt[e]);
    base += cnt[e];
  }
  __syncthreads();
  const int ncand = sm.redi[1];
  unsigned long long* ck = ncand <= TK_LCAP ? sm.key : g_key;
  int32_t* ci = ncand <= TK_LCAP ? sm.idx : g_idx;

  // scatter the candidates (every element of a bin that starts before rank keff), grouped by bin
  for (int v = tid; v < F; v += TK_THREADS) {
    const uint32_t b = sm.bin[v];
    if (b == 0xffffu || (int)sm.base[b] >= keff) continue;
    double s;
    keyfn(v, s);
    const uint32_t pos = sm.base[b] + atomicAdd(&sm.cur[b], 1u);
    ck[pos] = ordered_key(canonical_score(s));
    ci[pos] = v;
  }
  __syncthreads();

  // exact rank inside the bin
  for (int p = tid; p < ncand; p += TK_THREADS) {
    const int v = ci[p];
    const unsigned long long kp = ck[p];
    const uint32_t b = sm.bin[v];
    const int s0 = (int)sm.base[b], s1 = s0 + (int)sm.cur[b];
    int before = 0;
    for (int q = s0; q < s1; ++q) {
      const unsigned long long kq = ck[q];
      before += (kq > kp) || (kq == kp && ci[q] < v);
    }
    const int rank = s0 + before;
    if (rank < keff) emit(rank, v);
  }
  __syncthreads();
  return keff;
}

template <class KeyFn, class EmitFn>
__device__ int block_topk(int F, int k, KeyFn keyfn, EmitFn emit, const TopkSmem& sm, unsigned long long* g_key, int32_t* g_idx) {
  return block_topk_nt<1024>(F, k, keyfn, emit, sm, g_key, g_idx);
}

// Block-wide exclusive scan of one int per thread (1024 threads); returns the exclusive prefix, total in `total`.
__device__ inline int block_scan_excl(int val, int* scratch /*[33]*/, int& total) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int incl = val;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  __syncthreads();
  if (lane == 31) scratch[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const int w = scratch[lane];
    int wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += t;
    }
    scratch[lane] = wi - w;
    if (lane == 31) scratch[32] = wi;
  }
  __syncthreads();
  total = scratch[32];
  return scratch[warp] + incl - val;
}

// Selection kernel: top-k of keys[0..F) (restricted to `filter` when given) -> idx in rank order, mask, count.
__global__ void __launch_bounds__(TK_THREADS, 1)
    ls_topk_kernel(const double* __restrict__ keys, int F, int k, const uint32_t* __restrict__ filter, int32_t* out_idx, int cap,
                   uint32_t* out_mask, int mask_or, int32_t* out_count, unsigned long long* g_key, int32_t* g_idx, int* status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const TopkSmem sm = topk_carve(smem_raw);
  uint32_t* s_mask = reinterpret_cast<uint32_t*>(smem_raw + topk_smem_bytes(F));
  const int nwords = (F + 31) >> 5;
  for (int i = threadIdx.x; i < nwords; i += TK_THREADS) s_mask[i] = 0u;
  const int keff = block_topk(
      F, k,
      [&](int v, double& s) {
        if (filter && !((filter[v >> 5] >> (v & 31)) & 1u)) return false;
        s = keys[v];
        return true;
      },
      [&](int rank, int v) {
        if (out_idx && rank < cap) out_idx[rank] = v;
        atomicOr(&s_mask[v >> 5], 1u << (v & 31));
      },
      sm, g_key, g_idx);
  if (out_idx && keff > cap && threadIdx.x == 0) set_status(status, ST_CAPACITY);  // list truncated to its capacity
  if (out_mask)
    for (int w = threadIdx.x; w < nwords; w += TK_THREADS) out_mask[w] = mask_or ? (out_mask[w] | s_mask[w]) : s_mask[w];
  if (threadIdx.x == 0 && out_count) *out_count = out_idx ? min(keff, cap) : keff;
}

inline size_t topk_kernel_smem(int F) { return topk_smem_bytes(F) + (size_t)((F + 31) / 32) * 4; }

}  // namespace ls
