// HBM neuron cache: residency tables on the device, backing store in pinned host memory, misses copied with
// cudaMemcpyAsync on a side stream.  Decisions (hit / miss / victim / slot) are taken by one-CTA kernels so that the
// logical state is a deterministic function of the request sequence; the host only reads the miss list and issues the
// copies.
#pragma once
#include <atomic>
#include <chrono>
#include <string>
#include <thread>

#include "ls_topk.cuh"

namespace ls {

struct CacheState {
  int F = 0, C = 0, max_sel = 0;
  size_t bundle_bytes = 0;
  void* h_bundles = nullptr;        // pinned [F][bundle_bytes]
  int32_t* d_slot_of = nullptr;     // [F]  slot of a resident neuron, -1 otherwise
  int32_t* d_neuron_of = nullptr;   // [C]  neuron held by a slot, -1 when free
  int* d_nres = nullptr;            // [1]  number of residents
  int32_t* d_exec_idx = nullptr;    // [max_sel] execution order of the last reserve: residents first, then misses
  int32_t* d_miss_neuron = nullptr; // [max_sel]
  int32_t* d_victim_slot = nullptr; // [max_sel]
  int32_t* d_free_list = nullptr;   // [max_sel]
  unsigned long long* d_key = nullptr;  // [F] top-k fallback scratch
  int32_t* d_idx = nullptr;             // [F]
  int32_t* h_out = nullptr;         // mapped pinned [8 + 2*max_sel]: nmiss, nhit, nvict, nres, then (neuron, slot) pairs
  int32_t* h_out_dev = nullptr;     // device view of h_out
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_list = nullptr, ev_copied = nullptr;
  bool copies_pending = false;
  int last_nhit = 0, last_nmiss = 0;
  int64_t hits = 0, misses = 0, evictions = 0, h2d_bytes = 0, h2d_copies = 0, resident = 0;
  double wait_limit_s = 30.0;
};

inline int32_t cache_fail(std::string& err, int32_t code, const char* what, cudaError_t e) {
  err = std::string(what) + ": " + cudaGetErrorString(e);
  return code;
}
#define LS_CACHE_CUDA(call)                                             \
  do {                                                                  \
    cudaError_t e_ = (call);                                            \
    if (e_ != cudaSuccess) return ls::cache_fail(err, -3, #call, e_);   \
  } while (0)

inline void cache_destroy(CacheState& c) {
  if (c.copy_stream) cudaStreamSynchronize(c.copy_stream);
  if (c.h_bundles) cudaFreeHost(c.h_bundles);
  if (c.h_out) cudaFreeHost(c.h_out);
  cudaFree(c.d_slot_of); cudaFree(c.d_neuron_of); cudaFree(c.d_nres); cudaFree(c.d_exec_idx); cudaFree(c.d_miss_neuron);
  cudaFree(c.d_victim_slot); cudaFree(c.d_free_list); cudaFree(c.d_key); cudaFree(c.d_idx);
  if (c.ev_list) cudaEventDestroy(c.ev_list);
  if (c.ev_copied) cudaEventDestroy(c.ev_copied);
  if (c.copy_stream) cudaStreamDestroy(c.copy_stream);
  c = CacheState();
}

inline int32_t cache_create(CacheState& c, int F, int C, size_t bundle_bytes, int max_sel, std::string& err) {
  c.F = F; c.C = C; c.bundle_bytes = bundle_bytes; c.max_sel = max_sel;
  cudaError_t e = cudaHostAlloc(&c.h_bundles, (size_t)F * bundle_bytes, cudaHostAllocDefault);
  if (e != cudaSuccess) return cache_fail(err, -2, "pinned backing store", e);
  e = cudaHostAlloc(reinterpret_cast<void**>(&c.h_out), (8 + 2 * (size_t)max_sel) * sizeof(int32_t), cudaHostAllocMapped);
  if (e != cudaSuccess) return cache_fail(err, -2, "pinned miss list", e);
  LS_CACHE_CUDA(cudaHostGetDevicePointer(reinterpret_cast<void**>(&c.h_out_dev), c.h_out, 0));
  LS_CACHE_CUDA(cudaMalloc(&c.d_slot_of, (size_t)F * 4));
  LS_CACHE_CUDA(cudaMalloc(&c.d_neuron_of, (size_t)C * 4));
  LS_CACHE_CUDA(cudaMalloc(&c.d_nres, 4));
  LS_CACHE_CUDA(cudaMalloc(&c.d_exec_idx, (size_t)max_sel * 4));
  LS_CACHE_CUDA(cudaMalloc(&c.d_miss_neuron, (size_t)max_sel * 4));
  LS_CACHE_CUDA(cudaMalloc(&c.d_victim_slot, (size_t)max_sel * 4));
  LS_CACHE_CUDA(cudaMalloc(&c.d_free_list, (size_t)max_sel * 4));
  LS_CACHE_CUDA(cudaMalloc(&c.d_key, (size_t)F * 8));
  LS_CACHE_CUDA(cudaMalloc(&c.d_idx, (size_t)F * 4));
  LS_CACHE_CUDA(cudaMemset(c.d_slot_of, 0xff, (size_t)F * 4));
  LS_CACHE_CUDA(cudaMemset(c.d_neuron_of, 0xff, (size_t)C * 4));
  LS_CACHE_CUDA(cudaMemset(c.d_nres, 0, 4));
  LS_CACHE_CUDA(cudaStreamCreateWithFlags(&c.copy_stream, cudaStreamNonBlocking));
  LS_CACHE_CUDA(cudaEventCreateWithFlags(&c.ev_list, cudaEventDisableTiming));
  LS_CACHE_CUDA(cudaEventCreateWithFlags(&c.ev_copied, cudaEventDisableTiming));
  return 0;
}

// ---------------------------------------------------------------------------------------------------------------------
__device__ inline bool bit_of(const uint32_t* m, int i) { return (m[i >> 5] >> (i & 31)) & 1u; }

// Picks the `need` lowest-priority residents that are neither wanted nor protected (the reverse of the keep order:
// priority ascending, index descending) and frees their slots.  Returns how many were evicted.
template <class OnVictim>
__device__ int evict_lowest(int F, int need, const double* prio, const uint32_t* s_want, const uint32_t* protect, int32_t* slot_of,
                            const TopkSmem& sm, unsigned long long* g_key, int32_t* g_idx, OnVictim on_victim) {
  return block_topk(
      F, need,
      [&](int v, double& s) {
        const int i = F - 1 - v;
        if (slot_of[i] < 0) return false;
        if (s_want && bit_of(s_want, i)) return false;
        if (protect && bit_of(protect, i)) return false;
        s = -canonical_score(prio[i]);
        return true;
      },
      [&](int rank, int v) {
        const int i = F - 1 - v;
        on_victim(rank, i, slot_of[i]);
        slot_of[i] = -1;
      },
      sm, g_key, g_idx);
}

__global__ void __launch_bounds__(TK_THREADS, 1)
    ls_cache_reserve_kernel(const double* __restrict__ prio, int F, int C, const int32_t* __restrict__ want,
                            const int32_t* __restrict__ count_ptr, int admit_ranks, int admit_num, int admit_den, int cap,
                            const uint32_t* __restrict__ protect, int32_t* slot_of, int32_t* neuron_of, int* nres_ptr,
                            int32_t* exec_idx, int32_t* miss_neuron, int32_t* victim_slot, int32_t* free_list, int32_t* h_out,
                            unsigned long long* g_key, int32_t* g_idx, int* status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const TopkSmem sm = topk_carve(smem_raw);
  const int nwords = (F + 31) >> 5;
  uint32_t* s_want = reinterpret_cast<uint32_t*>(smem_raw + topk_smem_bytes(F));
  uint32_t* s_valid = s_want + nwords;                 // [ceil(cap/32)] entry p is a first, in-range occurrence
  int* s_scan = reinterpret_cast<int*>(s_valid + ((cap + 31) >> 5) + 1);  // [40]
  const int tid = threadIdx.x;

  const int count = max(0, min(*count_ptr, cap));
  int n;
  if (admit_den > 0) n = (int)(((long long)count * admit_num + admit_den - 1) / admit_den);
  else n = admit_ranks < 0 ? count : min(admit_ranks, count);
  n = min(n, count);

  for (int w = tid; w < nwords; w += TK_THREADS) s_want[w] = 0u;
  for (int w = tid; w < ((cap + 31) >> 5) + 1; w += TK_THREADS) s_valid[w] = 0u;
  __syncthreads();
  for (int p = tid; p < n; p += TK_THREADS) {
    const int i = want[p];
    if ((unsigned)i >= (unsigned)F) { set_status(status, ST_BAD_INDEX); continue; }
    const uint32_t bit = 1u << (i & 31);
    const uint32_t old = atomicOr(&s_want[i >> 5], bit);
    if (old & bit) { set_status(status, ST_BAD_INDEX); continue; }  // duplicate entry: ignored
    atomicOr(&s_valid[p >> 5], 1u << (p & 31));
  }
  __syncthreads();

  // capacity: wanted + protected neurons must fit
  int pinned = 0;
  for (int w = tid; w < nwords; w += TK_THREADS) pinned += __popc(s_want[w] | (protect ? protect[w] : 0u));
  int total;
  block_scan_excl(pinned, s_scan, total);
  if (total > C) {
    if (tid == 0) { set_status(status, ST_CAPACITY); h_out[0] = -1; h_out[1] = 0; h_out[2] = 0; h_out[3] = *nres_ptr; }
    return;
  }

  // stable partition of the admitted ranks: residents, then misses
  int nhit = 0, nmiss = 0;
  for (int p0 = 0; p0 < n; p0 += TK_THREADS) {
    const int p = p0 + tid;
    int i = -1, hit = 0, miss = 0;
    if (p < n && ((s_valid[p >> 5] >> (p & 31)) & 1u)) {
      i = want[p];
      hit = slot_of[i] >= 0;
      miss = !hit;
    }
    int tot;
    const int ex = block_scan_excl(hit | (miss << 16), s_scan, tot);
    if (hit) exec_idx[nhit + (ex & 0xffff)] = i;
    if (miss) miss_neuron[nmiss + (ex >> 16)] = i;
    nhit += tot & 0xffff;
    nmiss += tot >> 16;
  }
  __syncthreads();
  for (int q = tid; q < nmiss; q += TK_THREADS) exec_idx[nhit + q] = miss_neuron[q];

  const int nres = *nres_ptr;
  const int nfree = C - nres;
  const int nvict = max(0, nmiss - nfree);
  if (nvict > 0)
    evict_lowest(F, nvict, prio, s_want, protect, slot_of, sm, g_key, g_idx,
                 [&](int rank, int /*neuron*/, int slot) { victim_slot[rank] = slot; });
  // free slots in ascending slot order for the misses that no victim serves
  const int nfs = nmiss - nvict;
  int found = 0;
  for (int s0 = 0; s0 < C && found < nfs; s0 += TK_THREADS) {
    const int s = s0 + tid;
    const int fr = (s < C && neuron_of[s] < 0) ? 1 : 0;
    int tot;
    const int ex = block_scan_excl(fr, s_scan, tot);
    if (fr && found + ex < nfs) free_list[found + ex] = s;
    found += tot;
  }
  __syncthreads();
  for (int q = tid; q < nmiss; q += TK_THREADS) {
    const int slot = q < nvict ? victim_slot[q] : free_list[q - nvict];
    const int i = miss_neuron[q];
    slot_of[i] = slot;
    neuron_of[slot] = i;
    h_out[8 + 2 * q] = i;
    h_out[9 + 2 * q] = slot;
  }
  if (tid == 0) {
    *nres_ptr = nres + nmiss - nvict;
    h_out[0] = nmiss; h_out[1] = nhit; h_out[2] = nvict; h_out[3] = nres + nmiss - nvict;
  }
}

__global__ void __launch_bounds__(TK_THREADS, 1)
    ls_cache_evict_kernel(const double* __restrict__ prio, int F, int C, int min_free, const uint32_t* __restrict__ protect,
                          int32_t* slot_of, int32_t* neuron_of, int* nres_ptr, int32_t* evicted, int32_t* nevicted, int32_t* h_out,
                          unsigned long long* g_key, int32_t* g_idx) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const TopkSmem sm = topk_carve(smem_raw);
  const int nres = *nres_ptr;
  const int need = min_free - (C - nres);
  int got = 0;
  if (need > 0)
    got = evict_lowest(F, need, prio, nullptr, protect, slot_of, sm, g_key, g_idx, [&](int rank, int neuron, int slot) {
      neuron_of[slot] = -1;
      if (evicted) evicted[rank] = neuron;
    });
  if (threadIdx.x == 0) {
    *nres_ptr = nres - got;
    if (nevicted) *nevicted = got;
    h_out[0] = 0; h_out[1] = 0; h_out[2] = got; h_out[3] = nres - got;
  }
}

__global__ void ls_cache_lookup_kernel(const int32_t* __restrict__ slot_of, int F, const int32_t* __restrict__ idx, int n,
                                       int32_t* slot, int32_t* nhit, int* status) {
  __shared__ int s_hits;
  if (threadIdx.x == 0) s_hits = 0;
  __syncthreads();
  int h = 0;
  for (int p = threadIdx.x; p < n; p += blockDim.x) {
    const int i = idx[p];
    int s = -1;
    if ((unsigned)i >= (unsigned)F) set_status(status, ST_BAD_INDEX);
    else s = slot_of[i];
    slot[p] = s;
    h += s >= 0;
  }
  atomicAdd(&s_hits, h);
  __syncthreads();
  if (threadIdx.x == 0 && nhit) *nhit = s_hits;
}

__global__ void ls_cache_snapshot_kernel(const int32_t* __restrict__ slot_of, int F, uint32_t* mask) {
  const int nwords = (F + 31) >> 5;
  for (int w = blockIdx.x * blockDim.x + threadIdx.x; w < nwords; w += gridDim.x * blockDim.x) {
    uint32_t m = 0u;
    for (int b = 0; b < 32; ++b) {
      const int i = w * 32 + b;
      if (i < F && slot_of[i] >= 0) m |= 1u << b;
    }
    mask[w] = m;
  }
}

// ---------------------------------------------------------------------------------------------------------------------
inline size_t cache_kernel_smem(int F, int cap) {
  return topk_smem_bytes(F) + (size_t)((F + 31) / 32) * 4 + (size_t)((cap + 31) / 32 + 1) * 4 + 48 * 4;
}

// Bounded host wait for an event (poll, then sleep); the limit guards against a stream that never drains.
inline int32_t wait_event_bounded(cudaEvent_t ev, double limit_s, std::string& err) {
  const auto t0 = std::chrono::steady_clock::now();
  for (long it = 0;; ++it) {
    const cudaError_t q = cudaEventQuery(ev);
    if (q == cudaSuccess) return 0;
    if (q != cudaErrorNotReady) return cache_fail(err, -3, "cudaEventQuery", q);
    if (it > 2000) std::this_thread::sleep_for(std::chrono::microseconds(50));
    if (std::chrono::duration<double>(std::chrono::steady_clock::now() - t0).count() > limit_s) {
      err = "timed out waiting for the cache decision kernel";
      return -6;
    }
  }
}

inline int32_t cache_reserve(CacheState& c, const double* prio, int F, const int32_t* want, const int32_t* count_ptr, int admit_ranks,
                             int admit_num, int admit_den, int cap, const uint32_t* protect, uint16_t* bundles, int* status,
                             cudaStream_t st, int32_t* h_nmiss, std::string& err, std::atomic<int64_t>& launches) {
  ls_cache_reserve_kernel<<<1, TK_THREADS, cache_kernel_smem(F, cap), st>>>(
      prio, F, c.C, want, count_ptr, admit_ranks, admit_num, admit_den, cap, protect, c.d_slot_of, c.d_neuron_of, c.d_nres,
      c.d_exec_idx, c.d_miss_neuron, c.d_victim_slot, c.d_free_list, c.h_out_dev, c.d_key, c.d_idx, status);
  launches.fetch_add(1, std::memory_order_relaxed);
  LS_CACHE_CUDA(cudaPeekAtLastError());
  LS_CACHE_CUDA(cudaEventRecord(c.ev_list, st));
  const int32_t rc = wait_event_bounded(c.ev_list, c.wait_limit_s, err);
  if (rc != 0) return rc;
  const int nmiss = c.h_out[0];
  if (nmiss < 0) {
    err = "wanted + protected neurons exceed the cache capacity";
    if (h_nmiss) *h_nmiss = 0;
    return -5;
  }
  c.last_nmiss = nmiss;
  c.last_nhit = c.h_out[1];
  c.hits += c.h_out[1];
  c.misses += nmiss;
  c.evictions += c.h_out[2];
  c.resident = c.h_out[3];
  // one copy per miss, merged when both the neuron and the slot are consecutive
  char* dev = reinterpret_cast<char*>(bundles);
  const char* host = static_cast<const char*>(c.h_bundles);
  int q = 0;
  while (q < nmiss) {
    const int i0 = c.h_out[8 + 2 * q], s0 = c.h_out[9 + 2 * q];
    int run = 1;
    while (q + run < nmiss && c.h_out[8 + 2 * (q + run)] == i0 + run && c.h_out[9 + 2 * (q + run)] == s0 + run) ++run;
    LS_CACHE_CUDA(cudaMemcpyAsync(dev + (size_t)s0 * c.bundle_bytes, host + (size_t)i0 * c.bundle_bytes, (size_t)run * c.bundle_bytes,
                                  cudaMemcpyHostToDevice, c.copy_stream));
    c.h2d_copies += 1;
    q += run;
  }
  c.h2d_bytes += (int64_t)nmiss * (int64_t)c.bundle_bytes;
  if (nmiss > 0) {
    LS_CACHE_CUDA(cudaEventRecord(c.ev_copied, c.copy_stream));
    c.copies_pending = true;
  }
  if (h_nmiss) *h_nmiss = nmiss;
  return 0;
}

inline int32_t cache_wait(CacheState& c, cudaStream_t st, std::string& err) {
  if (c.copies_pending) LS_CACHE_CUDA(cudaStreamWaitEvent(st, c.ev_copied, 0));
  return 0;
}

inline int32_t cache_evict(CacheState& c, const double* prio, int F, int min_free, const uint32_t* protect, int32_t* d_evicted,
                           int32_t* d_nevicted, int* /*status*/, cudaStream_t st, std::string& err, std::atomic<int64_t>& launches) {
  ls_cache_evict_kernel<<<1, TK_THREADS, cache_kernel_smem(F, 0), st>>>(prio, F, c.C, min_free, protect, c.d_slot_of, c.d_neuron_of,
                                                                         c.d_nres, d_evicted, d_nevicted, c.h_out_dev, c.d_key, c.d_idx);
  launches.fetch_add(1, std::memory_order_relaxed);
  LS_CACHE_CUDA(cudaPeekAtLastError());
  LS_CACHE_CUDA(cudaEventRecord(c.ev_list, st));
  const int32_t rc = wait_event_bounded(c.ev_list, c.wait_limit_s, err);
  if (rc != 0) return rc;
  c.evictions += c.h_out[2];
  c.resident = c.h_out[3];
  return 0;
}

inline int32_t cache_lookup(CacheState& c, int F, const int32_t* d_idx, int n, int32_t* d_slot, int32_t* d_nhit, int* status,
                            cudaStream_t st, std::string& err, std::atomic<int64_t>& launches) {
  ls_cache_lookup_kernel<<<1, 1024, 0, st>>>(c.d_slot_of, F, d_idx, n, d_slot, d_nhit, status);
  launches.fetch_add(1, std::memory_order_relaxed);
  LS_CACHE_CUDA(cudaPeekAtLastError());
  return 0;
}

inline int32_t cache_snapshot(CacheState& c, int F, uint32_t* mask, cudaStream_t st, std::string& err, std::atomic<int64_t>& launches) {
  ls_cache_snapshot_kernel<<<8, 256, 0, st>>>(c.d_slot_of, F, mask);
  launches.fetch_add(1, std::memory_order_relaxed);
  LS_CACHE_CUDA(cudaPeekAtLastError());
  return 0;
}

}  // namespace ls
