// HBM neuron cache: residency tables on the device, backing store in pinned host memory, misses served on a side stream.
// Decisions (hit / miss / victim / slot) are taken by one-CTA kernels so that the logical state is a deterministic
// function of the request sequence.  Nothing on the calling thread waits for a decision: the miss list is handed over by
// flags (Section 3.2.1 of the paper, Algorithm 1: per-block flags in memory both sides see, I/O lanes that never block the
// GPU), in one of two ways chosen per process:
//
//   I/O lane (MISS_PATH_LANE): the decision kernel writes the miss list and a sequence number to mapped pinned memory;
//     a host thread, the paper's I/O lane, polls that number, issues one cudaMemcpyAsync per run of adjacent slots on the
//     layer's copy stream and, behind them, a four-byte copy that raises the layer's "landed" word in device memory.
//     The kernel of request s waits (bounded) until the lane has taken over request s - 2: the list has two buffers.
//   gather (MISS_PATH_GATHER): the list stays on the device; the copy stream waits for the decision kernel's event and
//     runs one kernel that reads the missing bundles straight from the mapped pinned store over the host link, writes them
//     into their slots and raises the same "landed" word.  No host thread takes part.
//
// Either way the stage kernels that touch copied rows spin (bounded) on the landed word, so the stages made of residents
// only run while the copies are still in flight.
#pragma once
#include <atomic>
#include <chrono>
#include <mutex>
#include <string>
#include <thread>
#include <vector>

#include "ls_topk.cuh"

namespace ls {

constexpr int MISS_PATH_LANE = 0, MISS_PATH_GATHER = 1;
constexpr long long CACHE_SPIN_CLOCKS = 4000LL * 1000 * 1000;  // device-side waits give up after about two seconds
constexpr int CACHE_HDR = 8;  // ints in front of the (neuron, slot) pairs of a list: nmiss, nhit, nvict, nres, seq

struct CacheState {
  int device = 0, F = 0, C = 0, max_sel = 0;
  size_t bundle_bytes = 0;
  void* bundles_dev = nullptr;      // [C][bundle_bytes] the cache slots in HBM
  void* h_bundles = nullptr;        // mapped pinned [F][bundle_bytes]
  void* h_bundles_dev = nullptr;    // the device's view of it
  int32_t* d_slot_of = nullptr;     // [F]  slot of a resident neuron, -1 otherwise
  int32_t* d_neuron_of = nullptr;   // [C]  neuron held by a slot, -1 when free
  int* d_nres = nullptr;            // [1]  number of residents
  int32_t* d_exec_idx = nullptr;    // [max_sel] execution order of the last reserve: residents first, then misses
  int32_t* d_miss_neuron = nullptr; // [max_sel]
  int32_t* d_victim_slot = nullptr; // [max_sel]
  int32_t* d_free_list = nullptr;   // [max_sel]
  int32_t* d_list = nullptr;        // [2][CACHE_HDR + 2 max_sel] counters and (neuron, slot) pairs of the last two requests
  unsigned* d_landed = nullptr;     // [1] sequence number of the last request whose rows are in their slots
  unsigned* d_gdone = nullptr;      // [1] blocks of the gather kernel that have finished (reset by the last one)
  long long* d_stats = nullptr;     // [8] hits, misses, evictions, resident, bytes copied, gather launches with misses
  unsigned long long* d_key = nullptr;  // [F] top-k fallback scratch
  int32_t* d_idx = nullptr;             // [F]
  int32_t* h_list = nullptr;        // mapped pinned [2][CACHE_HDR + 2 max_sel]: the lists the I/O lane reads
  int32_t* h_list_dev = nullptr;
  unsigned* h_ack = nullptr;        // mapped pinned [1]: last request the I/O lane has taken over
  unsigned* h_ack_dev = nullptr;
  unsigned* h_seq = nullptr;        // pinned [64]: the values the copy stream writes to d_landed
  int32_t* h_res = nullptr;         // pinned [CACHE_HDR]: counters of a request, for the calls that report them
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_list = nullptr, ev_res = nullptr;
  cudaEvent_t ev_want = nullptr, ev_decided = nullptr;  // a decision kernel on the copy stream: its inputs are ready / it has run
  bool side_pending = false;        // a decision kernel was enqueued on the copy stream since the last join
  unsigned seq_issued = 0;          // requests enqueued by the calling thread
  unsigned seq_lane = 0;            // requests the I/O lane has taken over (lane thread only)
  std::atomic<long long> lane_copies{0};
  bool registered = false;
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

// ---- the I/O lane: one host thread per process that serves every cached layer registered with it ----------------------
class CopyLane {
 public:
  static CopyLane& get() {
    static CopyLane lane;
    return lane;
  }
  void add(CacheState* c) {
    std::lock_guard<std::mutex> lk(mu_);
    caches_.push_back(c);
    c->registered = true;
    if (!started_) {
      started_ = true;
      th_ = std::thread([this] { run(); });
    }
  }
  void remove(CacheState* c) {
    std::lock_guard<std::mutex> lk(mu_);
    for (size_t i = 0; i < caches_.size(); ++i)
      if (caches_[i] == c) { caches_.erase(caches_.begin() + i); break; }
    c->registered = false;
  }
  ~CopyLane() {
    stop_.store(true);
    if (th_.joinable()) th_.join();
  }

 private:
  // A new sequence number in a layer's list: its misses are copied (one cudaMemcpyAsync per run of adjacent neurons and
  // slots) and the landed word follows them on the same stream.  Returns whether there was anything to do.
  bool service(CacheState& c) {
    bool any = false;
    for (;;) {
      const unsigned want = c.seq_lane + 1;
      const volatile int32_t* L = c.h_list + (size_t)(want & 1u) * (CACHE_HDR + 2 * (size_t)c.max_sel);
      if ((unsigned)L[4] != want) return any;
      std::atomic_thread_fence(std::memory_order_acquire);
      any = true;
      cudaSetDevice(c.device);
      const int nmiss = L[0];
      char* dev = reinterpret_cast<char*>(c.bundles_dev);
      const char* host = static_cast<const char*>(c.h_bundles);
      long long ncopy = 0;
      for (int q = 0; q < nmiss;) {
        const int i0 = L[CACHE_HDR + 2 * q], s0 = L[CACHE_HDR + 2 * q + 1];
        int run = 1;
        while (q + run < nmiss && L[CACHE_HDR + 2 * (q + run)] == i0 + run && L[CACHE_HDR + 2 * (q + run) + 1] == s0 + run) ++run;
        cudaMemcpyAsync(dev + (size_t)s0 * c.bundle_bytes, host + (size_t)i0 * c.bundle_bytes, (size_t)run * c.bundle_bytes,
                        cudaMemcpyHostToDevice, c.copy_stream);
        ++ncopy;
        q += run;
      }
      c.h_seq[want & 63u] = want;
      cudaMemcpyAsync(c.d_landed, c.h_seq + (want & 63u), sizeof(unsigned), cudaMemcpyHostToDevice, c.copy_stream);
      c.lane_copies.fetch_add(ncopy, std::memory_order_relaxed);
      c.seq_lane = want;
      std::atomic_thread_fence(std::memory_order_release);
      *reinterpret_cast<volatile unsigned*>(c.h_ack) = want;  // the kernel of request want + 2 may reuse this buffer
    }
  }
  void run() {
    int idle = 0;
    while (!stop_.load(std::memory_order_relaxed)) {
      bool any = false;
      {
        std::lock_guard<std::mutex> lk(mu_);
        for (CacheState* c : caches_) any |= service(*c);
      }
      if (any) idle = 0;
      else if (++idle > 20000) std::this_thread::sleep_for(std::chrono::microseconds(50));
      else std::this_thread::yield();
    }
  }
  std::mutex mu_;
  std::vector<CacheState*> caches_;
  std::thread th_;
  std::atomic<bool> stop_{false};
  bool started_ = false;
};

inline void cache_destroy(CacheState& c) {
  if (c.registered) CopyLane::get().remove(&c);
  if (c.copy_stream) cudaStreamSynchronize(c.copy_stream);
  if (c.h_bundles) cudaFreeHost(c.h_bundles);
  if (c.h_list) cudaFreeHost(c.h_list);
  if (c.h_ack) cudaFreeHost(c.h_ack);
  if (c.h_seq) cudaFreeHost(c.h_seq);
  if (c.h_res) cudaFreeHost(c.h_res);
  cudaFree(c.d_slot_of); cudaFree(c.d_neuron_of); cudaFree(c.d_nres); cudaFree(c.d_exec_idx); cudaFree(c.d_miss_neuron);
  cudaFree(c.d_victim_slot); cudaFree(c.d_free_list); cudaFree(c.d_list); cudaFree(c.d_landed); cudaFree(c.d_gdone);
  cudaFree(c.d_stats); cudaFree(c.d_key); cudaFree(c.d_idx);
  if (c.ev_list) cudaEventDestroy(c.ev_list);
  if (c.ev_res) cudaEventDestroy(c.ev_res);
  if (c.ev_want) cudaEventDestroy(c.ev_want);
  if (c.ev_decided) cudaEventDestroy(c.ev_decided);
  if (c.copy_stream) cudaStreamDestroy(c.copy_stream);
  c.h_bundles = c.h_bundles_dev = nullptr; c.h_list = c.h_list_dev = nullptr; c.h_ack = c.h_ack_dev = nullptr; c.h_seq = nullptr; c.h_res = nullptr;
  c.d_slot_of = c.d_neuron_of = nullptr; c.d_nres = nullptr; c.d_exec_idx = c.d_miss_neuron = c.d_victim_slot = c.d_free_list = c.d_list = nullptr;
  c.d_landed = c.d_gdone = nullptr; c.d_stats = nullptr; c.d_key = nullptr; c.d_idx = nullptr;
  c.ev_list = c.ev_res = c.ev_want = c.ev_decided = nullptr; c.copy_stream = nullptr;
}

inline int32_t cache_create(CacheState& c, int device, int F, int C, size_t bundle_bytes, int max_sel, void* bundles_dev, std::string& err) {
  c.device = device; c.F = F; c.C = C; c.bundle_bytes = bundle_bytes; c.max_sel = max_sel; c.bundles_dev = bundles_dev;
  const size_t list_ints = CACHE_HDR + 2 * (size_t)max_sel;
  cudaError_t e = cudaHostAlloc(&c.h_bundles, (size_t)F * bundle_bytes, cudaHostAllocMapped);
  if (e != cudaSuccess) return cache_fail(err, -2, "pinned backing store", e);
  LS_CACHE_CUDA(cudaHostGetDevicePointer(&c.h_bundles_dev, c.h_bundles, 0));
  e = cudaHostAlloc(reinterpret_cast<void**>(&c.h_list), 2 * list_ints * sizeof(int32_t), cudaHostAllocMapped);
  if (e != cudaSuccess) return cache_fail(err, -2, "pinned miss lists", e);
  LS_CACHE_CUDA(cudaHostGetDevicePointer(reinterpret_cast<void**>(&c.h_list_dev), c.h_list, 0));
  memset(c.h_list, 0, 2 * list_ints * sizeof(int32_t));
  LS_CACHE_CUDA(cudaHostAlloc(reinterpret_cast<void**>(&c.h_ack), 64, cudaHostAllocMapped));
  LS_CACHE_CUDA(cudaHostGetDevicePointer(reinterpret_cast<void**>(&c.h_ack_dev), c.h_ack, 0));
  *c.h_ack = 0u;
  LS_CACHE_CUDA(cudaHostAlloc(reinterpret_cast<void**>(&c.h_seq), 64 * sizeof(unsigned), cudaHostAllocDefault));
  LS_CACHE_CUDA(cudaHostAlloc(reinterpret_cast<void**>(&c.h_res), CACHE_HDR * sizeof(int32_t), cudaHostAllocDefault));
  LS_CACHE_CUDA(cudaMalloc(&c.d_slot_of, (size_t)F * 4));
  LS_CACHE_CUDA(cudaMalloc(&c.d_neuron_of, (size_t)C * 4));
  LS_CACHE_CUDA(cudaMalloc(&c.d_nres, 4));
  LS_CACHE_CUDA(cudaMalloc(&c.d_exec_idx, (size_t)max_sel * 4));
  LS_CACHE_CUDA(cudaMalloc(&c.d_miss_neuron, (size_t)max_sel * 4));
  LS_CACHE_CUDA(cudaMalloc(&c.d_victim_slot, (size_t)max_sel * 4));
  LS_CACHE_CUDA(cudaMalloc(&c.d_free_list, (size_t)max_sel * 4));
  LS_CACHE_CUDA(cudaMalloc(&c.d_list, 2 * list_ints * 4));
  LS_CACHE_CUDA(cudaMalloc(&c.d_landed, 4));
  LS_CACHE_CUDA(cudaMalloc(&c.d_gdone, 4));
  LS_CACHE_CUDA(cudaMalloc(&c.d_stats, 8 * sizeof(long long)));
  LS_CACHE_CUDA(cudaMalloc(&c.d_key, (size_t)F * 8));
  LS_CACHE_CUDA(cudaMalloc(&c.d_idx, (size_t)F * 4));
  LS_CACHE_CUDA(cudaMemset(c.d_slot_of, 0xff, (size_t)F * 4));
  LS_CACHE_CUDA(cudaMemset(c.d_neuron_of, 0xff, (size_t)C * 4));
  LS_CACHE_CUDA(cudaMemset(c.d_nres, 0, 4));
  LS_CACHE_CUDA(cudaMemset(c.d_list, 0, 2 * list_ints * 4));
  LS_CACHE_CUDA(cudaMemset(c.d_landed, 0, 4));
  LS_CACHE_CUDA(cudaMemset(c.d_gdone, 0, 4));
  LS_CACHE_CUDA(cudaMemset(c.d_stats, 0, 8 * sizeof(long long)));
  LS_CACHE_CUDA(cudaStreamCreateWithFlags(&c.copy_stream, cudaStreamNonBlocking));
  LS_CACHE_CUDA(cudaEventCreateWithFlags(&c.ev_list, cudaEventDisableTiming));
  LS_CACHE_CUDA(cudaEventCreateWithFlags(&c.ev_res, cudaEventDisableTiming));
  LS_CACHE_CUDA(cudaEventCreateWithFlags(&c.ev_want, cudaEventDisableTiming));
  LS_CACHE_CUDA(cudaEventCreateWithFlags(&c.ev_decided, cudaEventDisableTiming));
  CopyLane::get().add(&c);
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
                            int32_t* exec_idx, int32_t* miss_neuron, int32_t* victim_slot, int32_t* free_list, int32_t* d_list,
                            long long* d_stats, unsigned seq, int32_t* h_list, const unsigned* h_ack, size_t bundle_bytes,
                            unsigned long long* g_key, int32_t* g_idx, int* status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const TopkSmem sm = topk_carve(smem_raw);
  const int nwords = (F + 31) >> 5;
  uint32_t* s_want = reinterpret_cast<uint32_t*>(smem_raw + topk_smem_bytes(F));
  uint32_t* s_valid = s_want + nwords;                 // [ceil(cap/32)] entry p is a first, in-range occurrence
  int* s_scan = reinterpret_cast<int*>(s_valid + ((cap + 31) >> 5) + 1);  // [40]
  const int tid = threadIdx.x;
  // This request's list goes to the buffer request seq - 2 used: wait until that one has been taken over (by the I/O
  // lane: its acknowledgement in mapped pinned memory; by the gather kernel: the landed word)
  if (tid == 0 && seq > 2u) {
    const long long t0 = clock64();
    while (*reinterpret_cast<const volatile unsigned*>(h_ack) + 2u < seq) {
      if (clock64() - t0 > CACHE_SPIN_CLOCKS) { set_status(status, ST_TIMEOUT); break; }
    }
  }
  __syncthreads();

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
  if (total > C) {  // nothing changes; the (empty) list still goes out so that nobody waits for this request
    if (tid == 0) {
      set_status(status, ST_CAPACITY);
      d_list[0] = -1; d_list[1] = 0; d_list[2] = 0; d_list[3] = *nres_ptr; d_list[4] = (int)seq;
      if (h_list) {
        h_list[0] = 0; h_list[1] = 0; h_list[2] = 0; h_list[3] = *nres_ptr;
        __threadfence_system();
        *reinterpret_cast<volatile int32_t*>(h_list + 4) = (int)seq;
      }
    }
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
    d_list[CACHE_HDR + 2 * q] = i;
    d_list[CACHE_HDR + 2 * q + 1] = slot;
    if (h_list) { h_list[CACHE_HDR + 2 * q] = i; h_list[CACHE_HDR + 2 * q + 1] = slot; }
  }
  if (h_list) __threadfence_system();
  __syncthreads();
  if (tid == 0) {
    *nres_ptr = nres + nmiss - nvict;
    d_list[0] = nmiss; d_list[1] = nhit; d_list[2] = nvict; d_list[3] = nres + nmiss - nvict; d_list[4] = (int)seq;
    d_stats[0] += nhit; d_stats[1] += nmiss; d_stats[2] += nvict; d_stats[3] = nres + nmiss - nvict;
    d_stats[4] += (long long)nmiss * (long long)bundle_bytes;
    if (h_list) {  // the sequence number goes last: the lane reads the list only after it has seen it
      h_list[0] = nmiss; h_list[1] = nhit; h_list[2] = nvict; h_list[3] = nres + nmiss - nvict;
      __threadfence_system();
      *reinterpret_cast<volatile int32_t*>(h_list + 4) = (int)seq;
    }
  }
}

// Gather (MISS_PATH_GATHER): the bundles of the last request's misses from the mapped pinned store into their slots,
// read over the host link by the kernel itself (16 bytes per thread and step); the last block to finish raises the
// landed word.
__global__ void __launch_bounds__(256) ls_cache_gather_kernel(const int32_t* __restrict__ d_list, const unsigned char* __restrict__ h_bundles,
                                                              unsigned char* bundles, size_t bundle_bytes, unsigned* landed, unsigned* gdone,
                                                              long long* d_stats, unsigned seq) {
  const int nmiss = d_list[0];
  for (int q = blockIdx.x; q < nmiss; q += gridDim.x) {
    const uint4* src = reinterpret_cast<const uint4*>(h_bundles + (size_t)d_list[CACHE_HDR + 2 * q] * bundle_bytes);
    uint4* dst = reinterpret_cast<uint4*>(bundles + (size_t)d_list[CACHE_HDR + 2 * q + 1] * bundle_bytes);
    const int n16 = (int)(bundle_bytes >> 4);
    for (int i = threadIdx.x; i < n16; i += 4 * 256) {
      uint4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (i + u * 256 < n16) v[u] = src[i + u * 256];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (i + u * 256 < n16) dst[i + u * 256] = v[u];
    }
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    if (atomicAdd(gdone, 1u) == gridDim.x - 1) {
      *gdone = 0u;
      if (nmiss > 0) d_stats[5] += 1;
      __threadfence();
      atomicMax(landed, seq);
    }
  }
}

// Makes the stream it runs on wait (bounded) until the rows of request `need` are in their slots.
__global__ void ls_cache_wait_kernel(const unsigned* landed, unsigned need, int* status) {
  if (threadIdx.x != 0) return;
  const long long t0 = clock64();
  while (*reinterpret_cast<const volatile unsigned*>(landed) < need) {
    if (clock64() - t0 > CACHE_SPIN_CLOCKS) { set_status(status, ST_TIMEOUT); break; }
  }
}

__global__ void __launch_bounds__(TK_THREADS, 1)
    ls_cache_evict_kernel(const double* __restrict__ prio, int F, int C, int min_free, const uint32_t* __restrict__ protect,
                          int32_t* slot_of, int32_t* neuron_of, int* nres_ptr, int32_t* evicted, int32_t* nevicted, long long* d_stats,
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
    d_stats[2] += got; d_stats[3] = nres - got;
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
    if (std::chrono::duration<double>(std::chrono::steady_clock::now() - t0).count() > limit_s) {
      err = "timed out waiting for the cache decision (the request stays enqueued and takes effect when the stream reaches it)";
      return -6;
    }
    if (it > 2000) std::this_thread::sleep_for(std::chrono::microseconds(50));
  }
}

// Enqueues a reserve: the decision kernel on `st`, then the hand-over of its miss list (see the top of this file).
// Nothing here waits; the request's sequence number is returned for the kernels that will need its rows.
// Host-side wait of the I/O-lane path (bounded): until the lane has taken over request `seq`.  A kernel must never spin on
// the device for something only the host can provide while that host work is not yet secured (the launching thread may be
// held up behind the spinning kernel), so in lane mode the calling thread (a) lets at most two requests of a layer be in
// flight and (b) enqueues the stages of a step only once the copies of the step's own request have been issued.
inline int32_t cache_lane_wait(CacheState& c, unsigned seq, double limit_s, std::string& err) {
  const auto t0 = std::chrono::steady_clock::now();
  for (long it = 0; *reinterpret_cast<const volatile unsigned*>(c.h_ack) < seq; ++it) {
    if (std::chrono::duration<double>(std::chrono::steady_clock::now() - t0).count() > limit_s) {
      err = "timed out waiting for the I/O lane to take over a cache request";
      return -6;
    }
    if (it > 4000) std::this_thread::sleep_for(std::chrono::microseconds(20));
  }
  return 0;
}

// Makes `st` wait for the decision kernels that were enqueued on the copy stream (`side` requests): everything that reads
// or changes the cache's tables, its priorities or a request's input list on `st` joins first.
inline int32_t cache_join(CacheState& c, cudaStream_t st, std::string& err) {
  if (c.side_pending) {
    LS_CACHE_CUDA(cudaStreamWaitEvent(st, c.ev_decided, 0));
    c.side_pending = false;
  }
  return 0;
}

// Enqueues one request: the decision kernel and the transport of its misses.  side = false: the decision kernel runs on
// `st` (whatever follows on `st` sees its tables).  side = true (gather transport only): `st` only marks the point at
// which the request's inputs (priorities, wanted list) are ready; the decision kernel runs on the copy stream, off the
// path of the kernels that follow on `st`, and the caller joins (cache_join) before `st` changes those inputs again or
// touches the tables.
inline int32_t cache_reserve_async(CacheState& c, int miss_path, const double* prio, int F, const int32_t* want, const int32_t* count_ptr,
                                   int admit_ranks, int admit_num, int admit_den, int cap, const uint32_t* protect, int* status,
                                   cudaStream_t st, unsigned* seq_out, double limit_s, std::string& err, std::atomic<int64_t>& launches,
                                   bool side = false) {
  const bool lane = miss_path == MISS_PATH_LANE;
  if (lane) side = false;
  if (lane && c.seq_issued >= 2) {
    const int32_t rc = cache_lane_wait(c, c.seq_issued - 1, limit_s, err);
    if (rc != 0) return rc;
  }
  if (!side) {
    const int32_t rc = cache_join(c, st, err);
    if (rc != 0) return rc;
  }
  const unsigned seq = ++c.seq_issued;
  const size_t list_ints = CACHE_HDR + 2 * (size_t)c.max_sel;
  int32_t* h_list = lane ? c.h_list_dev + (size_t)(seq & 1u) * list_ints : nullptr;
  int32_t* d_list = c.d_list + (size_t)(seq & 1u) * list_ints;
  cudaStream_t dst = st;
  if (side) {
    LS_CACHE_CUDA(cudaEventRecord(c.ev_want, st));
    LS_CACHE_CUDA(cudaStreamWaitEvent(c.copy_stream, c.ev_want, 0));
    dst = c.copy_stream;
  }
  ls_cache_reserve_kernel<<<1, TK_THREADS, cache_kernel_smem(F, cap), dst>>>(
      prio, F, c.C, want, count_ptr, admit_ranks, admit_num, admit_den, cap, protect, c.d_slot_of, c.d_neuron_of, c.d_nres, c.d_exec_idx,
      c.d_miss_neuron, c.d_victim_slot, c.d_free_list, d_list, c.d_stats, seq, h_list, lane ? c.h_ack_dev : c.d_landed, c.bundle_bytes,
      c.d_key, c.d_idx, status);
  launches.fetch_add(1, std::memory_order_relaxed);
  LS_CACHE_CUDA(cudaPeekAtLastError());
  if (side) {
    LS_CACHE_CUDA(cudaEventRecord(c.ev_decided, c.copy_stream));
    c.side_pending = true;
  }
  if (!lane) {
    if (!side) {
      LS_CACHE_CUDA(cudaEventRecord(c.ev_list, st));
      LS_CACHE_CUDA(cudaStreamWaitEvent(c.copy_stream, c.ev_list, 0));
    }
    ls_cache_gather_kernel<<<128, 256, 0, c.copy_stream>>>(d_list, static_cast<const unsigned char*>(c.h_bundles_dev),
                                                           static_cast<unsigned char*>(c.bundles_dev), c.bundle_bytes, c.d_landed, c.d_gdone,
                                                           c.d_stats, seq);
    launches.fetch_add(1, std::memory_order_relaxed);
    LS_CACHE_CUDA(cudaPeekAtLastError());
  }
  if (seq_out) *seq_out = seq;
  return 0;
}

// The counters of the request just enqueued on `st`, for the calls that report them: copied to pinned memory behind the
// decision kernel and awaited for at most limit_s seconds.
inline int32_t cache_request_result(CacheState& c, unsigned seq, cudaStream_t st, double limit_s, int32_t* h_nmiss, std::string& err) {
  const int32_t* d_list = c.d_list + (size_t)(seq & 1u) * (CACHE_HDR + 2 * (size_t)c.max_sel);
  LS_CACHE_CUDA(cudaMemcpyAsync(c.h_res, d_list, CACHE_HDR * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  LS_CACHE_CUDA(cudaEventRecord(c.ev_res, st));
  const int32_t rc = wait_event_bounded(c.ev_res, limit_s, err);
  if (rc != 0) return rc;
  if (c.h_res[0] < 0) {
    err = "wanted + protected neurons exceed the cache capacity";
    if (h_nmiss) *h_nmiss = 0;
    return -5;
  }
  if (h_nmiss) *h_nmiss = c.h_res[0];
  return 0;
}

inline const int32_t* cache_list_header(const CacheState& c, unsigned seq) {
  return c.d_list + (size_t)(seq & 1u) * (CACHE_HDR + 2 * (size_t)c.max_sel);
}

// Makes `st` wait (on the device, bounded) until the rows of every request enqueued so far are in their slots.
inline int32_t cache_wait(CacheState& c, int* status, cudaStream_t st, std::string& err, std::atomic<int64_t>& launches) {
  if (c.seq_issued == 0) return 0;
  { const int32_t rc = cache_join(c, st, err); if (rc != 0) return rc; }
  ls_cache_wait_kernel<<<1, 32, 0, st>>>(c.d_landed, c.seq_issued, status);
  launches.fetch_add(1, std::memory_order_relaxed);
  LS_CACHE_CUDA(cudaPeekAtLastError());
  return 0;
}

inline int32_t cache_evict(CacheState& c, const double* prio, int F, int min_free, const uint32_t* protect, int32_t* d_evicted,
                           int32_t* d_nevicted, int* /*status*/, cudaStream_t st, std::string& err, std::atomic<int64_t>& launches) {
  { const int32_t rc = cache_join(c, st, err); if (rc != 0) return rc; }
  ls_cache_evict_kernel<<<1, TK_THREADS, cache_kernel_smem(F, 0), st>>>(prio, F, c.C, min_free, protect, c.d_slot_of, c.d_neuron_of,
                                                                         c.d_nres, d_evicted, d_nevicted, c.d_stats, c.d_key, c.d_idx);
  launches.fetch_add(1, std::memory_order_relaxed);
  LS_CACHE_CUDA(cudaPeekAtLastError());
  return 0;
}

// Counters (device-resident, updated by the decision kernels): synchronises the device.
inline int32_t cache_stats(CacheState& c, long long out[8], std::string& err) {
  LS_CACHE_CUDA(cudaDeviceSynchronize());
  LS_CACHE_CUDA(cudaMemcpy(out, c.d_stats, 8 * sizeof(long long), cudaMemcpyDeviceToHost));
  out[5] += c.lane_copies.load(std::memory_order_relaxed);
  return 0;
}

inline int32_t cache_lookup(CacheState& c, int F, const int32_t* d_idx, int n, int32_t* d_slot, int32_t* d_nhit, int* status,
                            cudaStream_t st, std::string& err, std::atomic<int64_t>& launches) {
  { const int32_t rc = cache_join(c, st, err); if (rc != 0) return rc; }
  ls_cache_lookup_kernel<<<1, 1024, 0, st>>>(c.d_slot_of, F, d_idx, n, d_slot, d_nhit, status);
  launches.fetch_add(1, std::memory_order_relaxed);
  LS_CACHE_CUDA(cudaPeekAtLastError());
  return 0;
}

inline int32_t cache_snapshot(CacheState& c, int F, uint32_t* mask, cudaStream_t st, std::string& err, std::atomic<int64_t>& launches) {
  { const int32_t rc = cache_join(c, st, err); if (rc != 0) return rc; }
  ls_cache_snapshot_kernel<<<8, 256, 0, st>>>(c.d_slot_of, F, mask);
  launches.fetch_add(1, std::memory_order_relaxed);
  LS_CACHE_CUDA(cudaPeekAtLastError());
  return 0;
}

}  // namespace ls
