// Host side of the C ABI declared in include/leanstream.h: handles, argument checks, launches.
#include "../../include/leanstream.h"

#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cmath>
#include <cstring>
#include <limits>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "ls_cache.cuh"
#include "ls_hash.cuh"
#include "ls_kernels.cuh"
#include "ls_token.cuh"

namespace {

thread_local std::string g_err;
std::atomic<int64_t> g_launches{0};
std::atomic<int> g_opt_fused{1};
std::atomic<int> g_opt_miss_path{1};     // ls::MISS_PATH_GATHER
std::atomic<int> g_opt_host_wait_ms{30000};

int32_t fail(int32_t code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  g_err = buf;
  return code;
}

#define LS_CUDA(call)                                                                         \
  do {                                                                                        \
    cudaError_t e_ = (call);                                                                  \
    if (e_ != cudaSuccess) return fail(LS_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e_)); \
  } while (0)

#define LS_LAUNCHED()                                                                                   \
  do {                                                                                                  \
    g_launches.fetch_add(1, std::memory_order_relaxed);                                                 \
    cudaError_t e_ = cudaPeekAtLastError();                                                             \
    if (e_ != cudaSuccess) return fail(LS_ERR_CUDA, "kernel launch (%s:%d): %s", __FILE__, __LINE__,    \
                                       cudaGetErrorString(e_));                                        \
  } while (0)

// Optional per-kernel timing with CUDA events on the launching stream (roofline accounting; off by default).
struct TimedLaunch { int kind; cudaEvent_t a, b; };
std::atomic<int> g_timing{0};
std::mutex g_timing_mu;
std::vector<TimedLaunch> g_timed;

struct KernelTimer {
  cudaStream_t st;
  TimedLaunch t{};
  bool on;
  KernelTimer(int kind, cudaStream_t s) : st(s), on(g_timing.load(std::memory_order_relaxed) != 0) {
    if (!on) return;
    t.kind = kind;
    if (cudaEventCreate(&t.a) != cudaSuccess || cudaEventCreate(&t.b) != cudaSuccess) { on = false; return; }
    cudaEventRecord(t.a, st);
  }
  ~KernelTimer() {
    if (!on) return;
    cudaEventRecord(t.b, st);
    std::lock_guard<std::mutex> lk(g_timing_mu);
    g_timed.push_back(t);
  }
};

// Dynamic shared memory the whole-token kernel is launched with (it also has about 1 KB of static shared memory).
constexpr size_t kTokenSmemBudget = 222 * 1024;

struct DeviceGuard {
  int prev = -1;
  explicit DeviceGuard(int dev) {
    cudaGetDevice(&prev);
    if (prev != dev) cudaSetDevice(dev);
  }
  ~DeviceGuard() {
    int cur = -1;
    cudaGetDevice(&cur);
    if (prev >= 0 && cur != prev) cudaSetDevice(prev);
  }
};

}  // namespace

struct ls_layer {
  int device = 0;
  int d = 0, F = 0, gated = 1, act = 0, wd = 0, norm = 0, r = 0;
  float eps = 1e-5f;
  int n_mat = 3;
  int max_batch = 1, max_sel = 0;
  int nwords = 0;
  int sm_count = 148;
  int64_t cache_rows = 0;  // 0: resident
  int64_t nslots = 0;

  // weights (device)
  uint16_t* bundles = nullptr;  // [nslots][n_mat][d]
  float* b_gate = nullptr;
  float* b_down = nullptr;
  uint16_t* pred_at = nullptr;  // [r][d]
  uint16_t* pred_at_sl = nullptr;  // [ceil(d / 32)][r][32] (the fused kernel's column slices)
  uint16_t* pred_bt = nullptr;  // [F][r]
  uint16_t* pred_bt_pad = nullptr;  // resident layers: [F + 264][wt_brow_bytes(r) / 2], zero padded (whole-token kernel)
  float* pred_c = nullptr;

  // scratch (device)
  double* z = nullptr;       // [max_batch][r]
  double* sumsq = nullptr;   // [max_batch]
  double* scores = nullptr;  // [max_batch][F] (batch > 1 only)
  double* prio = nullptr;    // [F] latest priorities (retention priorities of the cache)
  unsigned long long* cand_key = nullptr;  // [F]
  int32_t* cand_idx = nullptr;             // [F]
  uint32_t* umask = nullptr;               // [nwords] union mask (batch > 1)
  int32_t* tmp_idx = nullptr;              // [max_sel] refined list of a stage j < K
  int32_t* tmp_count = nullptr;            // [1]
  uint32_t* tmp_mask = nullptr;            // [nwords]
  float* xin = nullptr;                    // [max_batch][d]
  float* xt = nullptr;                     // [max_batch][d] current partial residual feature
  float* actv = nullptr;                   // [max_batch][max_sel]
  float* ypart = nullptr;                  // [down_splits][max_batch][d]
  uint32_t* survive = nullptr;             // [nwords]
  int* status = nullptr;                   // [1]
  int down_splits = 0;

  // per-layer state of the fused kernel; its working scratch is shared per device (DeviceScratch below)
  double* wt_range = nullptr;  // [2] {hi, scale} of the score bins used when a fused step refines THIS layer (carried from call to call)

  ls::CacheState cache;  // residency tables, pinned backing store, copy stream
};

struct ls_hash_predictor {
  int device = 0, d = 0, r = 0, tau = 0, words = 0, n_layers = 0, F = 0, wd = 0, sm_count = 148;
  uint16_t* pca_t = nullptr;   // [r][d]
  float* w1 = nullptr;         // [r][tau]
  uint32_t* w = nullptr;       // [n_layers - 1][tau][words]
  uint32_t* tables = nullptr;  // [n_layers][2^tau][words]
  uint32_t* codes = nullptr;   // [F][words]
  double* z = nullptr;         // [r]
  double* sumsq = nullptr;     // [1]
  uint32_t* y = nullptr;       // [words]
  double* scores = nullptr;    // [F]
  unsigned long long* cand_key = nullptr;  // [F]
  int32_t* cand_idx = nullptr;             // [F]
  int* status = nullptr;
};

struct ls_stack {
  int device = 0, n = 0, d = 0, wd = 0, sm_count = 148, max_sel = 0;
  int r_max = 0, f_max = 0, ns_cta = 0, cpt = 1;
  std::vector<ls_layer*> layers;
  ls::WtLayer* d_layers = nullptr;       // [n] per-layer arguments (device)
  float* xbuf = nullptr;                 // [2][d] residual ping-pong between layers
  double* ranges = nullptr;              // [n][2] score-bin range of every layer's refinement, carried from launch to launch
  unsigned long long* cuts = nullptr;    // [n][WT_MAXE] key of the last member of every refined set
  int32_t* sellist = nullptr;            // [max_sel] ranked list of a selection that took the slow route
};

namespace {

template <typename T>
int32_t dalloc(T** p, size_t n) {
  *p = nullptr;
  if (n == 0) n = 1;
  cudaError_t e = cudaMalloc(reinterpret_cast<void**>(p), n * sizeof(T));
  if (e != cudaSuccess) return fail(e == cudaErrorMemoryAllocation ? LS_ERR_NOMEM : LS_ERR_CUDA, "cudaMalloc(%zu bytes): %s",
                                    n * sizeof(T), cudaGetErrorString(e));
  return LS_OK;
}

#define LS_TRY(expr)              \
  do {                            \
    int32_t rc_ = (expr);         \
    if (rc_ != LS_OK) return rc_; \
  } while (0)

void free_layer(ls_layer* L) {
  if (!L) return;
  ls::cache_destroy(L->cache);
  cudaFree(L->bundles); cudaFree(L->b_gate); cudaFree(L->b_down); cudaFree(L->pred_at); cudaFree(L->pred_at_sl); cudaFree(L->pred_bt); cudaFree(L->pred_bt_pad);
  cudaFree(L->pred_c); cudaFree(L->z); cudaFree(L->sumsq); cudaFree(L->scores); cudaFree(L->prio); cudaFree(L->cand_key);
  cudaFree(L->cand_idx); cudaFree(L->umask); cudaFree(L->tmp_idx); cudaFree(L->tmp_count); cudaFree(L->tmp_mask);
  cudaFree(L->wt_range);
  cudaFree(L->xin); cudaFree(L->xt); cudaFree(L->actv); cudaFree(L->ypart); cudaFree(L->survive); cudaFree(L->status);
  delete L;
}

int32_t upload_f32(float** dst, const float* src, size_t n) {
  LS_TRY(dalloc(dst, n));
  if (src) LS_CUDA(cudaMemcpy(*dst, src, n * sizeof(float), cudaMemcpyHostToDevice));
  else LS_CUDA(cudaMemset(*dst, 0, n * sizeof(float)));
  return LS_OK;
}

// [rows][cols] 16-bit host matrix -> transposed [cols][rows] on the device
int32_t upload_transposed16(uint16_t** dst, const void* src, int rows, int cols) {
  std::vector<uint16_t> t;
  try { t.resize((size_t)rows * cols); } catch (const std::bad_alloc&) { return fail(LS_ERR_NOMEM, "host staging buffer"); }
  const uint16_t* s = static_cast<const uint16_t*>(src);
  for (int i = 0; i < rows; ++i)
    for (int j = 0; j < cols; ++j) t[(size_t)j * rows + i] = s[(size_t)i * cols + j];
  LS_TRY(dalloc(dst, t.size()));
  LS_CUDA(cudaMemcpy(*dst, t.data(), t.size() * 2, cudaMemcpyHostToDevice));
  return LS_OK;
}

// [d][r] 16-bit host matrix A -> column slices [ceil(d / 32)][r][32] on the device, zero padded: slice s holds the rows
// 32 s .. 32 s + 31 of A, transposed, so that one contiguous copy brings a slice into shared memory.
int32_t upload_sliced16(uint16_t** dst, const void* src, int d, int r) {
  const int nsl = (d + ls::WT_SL - 1) / ls::WT_SL;
  std::vector<uint16_t> t;
  try { t.assign((size_t)nsl * r * ls::WT_SL, 0); } catch (const std::bad_alloc&) { return fail(LS_ERR_NOMEM, "host staging buffer"); }
  const uint16_t* s = static_cast<const uint16_t*>(src);
  for (int c = 0; c < d; ++c)
    for (int j = 0; j < r; ++j) t[((size_t)(c / ls::WT_SL) * r + j) * ls::WT_SL + (c % ls::WT_SL)] = s[(size_t)c * r + j];
  LS_TRY(dalloc(dst, t.size()));
  LS_CUDA(cudaMemcpy(*dst, t.data(), t.size() * 2, cudaMemcpyHostToDevice));
  return LS_OK;
}

// Working scratch of the fused kernel, one per device and shared by all layers on it: a decode loop runs its layers one
// after the other, and re-using the same few megabytes keeps them in L2 (per-layer copies would come back from HBM at
// every step).  Consequence: fused steps on one device must not overlap (issue them on one stream, or order the
// streams).  Sized for the largest shapes the fused path accepts; allocated at the first layer, kept until exit.
struct DeviceScratch {
  float* ypart = nullptr;             // [256 CTAs][16384] every CTA's partial output of its stage
  unsigned* ctr = nullptr;            // [64] word 32: the grid-barrier counter (zeroed before every launch)
  unsigned long long* cuts1 = nullptr;  // [WT_MAXE] cut keys of a single fused step
  double* z = nullptr;                // [FZ_MAXE][1024] latents, then [FZ_MAXE] sums of squares
  double* zpart = nullptr;            // [512 slices][FZ_MAXE][1025] per-slice partial latents
  double* sc = nullptr;               // [FZ_MAXE][32768] final scores of every evaluation
  uint16_t* sb = nullptr;             // [FZ_MAXE][32768] their fine bins
  uint4* bent = nullptr;              // [32768] members of the final evaluation, grouped by bin
  unsigned long long* kmm = nullptr;  // [2 x 1024] per-CTA smallest / largest key of the final evaluation
  bool ready = false;
};
constexpr int kScratchMaxD = 16384, kScratchMaxR = 1024, kScratchMaxF = 32768, kScratchMaxCtas = 256;
std::mutex g_scratch_mu;
DeviceScratch g_scratch[64];

int32_t device_scratch(int dev, DeviceScratch** out) {
  if (dev < 0 || dev >= 64) return fail(LS_ERR_INVALID, "device ordinal %d not supported", dev);
  std::lock_guard<std::mutex> lk(g_scratch_mu);
  DeviceScratch& S = g_scratch[dev];
  if (!S.ready) {
    const size_t NE = ls::WT_MAXE;
    LS_TRY(dalloc(&S.ypart, (size_t)kScratchMaxCtas * kScratchMaxD));
    LS_TRY(dalloc(&S.ctr, (size_t)64));
    LS_TRY(dalloc(&S.z, NE * (kScratchMaxR + 4) + NE));
    LS_TRY(dalloc(&S.zpart, (size_t)(kScratchMaxD / ls::WT_SL) * NE * (kScratchMaxR + 4)));
    LS_TRY(dalloc(&S.sc, NE * kScratchMaxF));
    LS_TRY(dalloc(&S.sb, NE * kScratchMaxF));
    LS_TRY(dalloc(&S.bent, (size_t)kScratchMaxF));
    LS_TRY(dalloc(&S.kmm, (size_t)2048));
    LS_TRY(dalloc(&S.cuts1, (size_t)ls::WT_MAXE));
    LS_CUDA(cudaMemset(S.cuts1, 0, ls::WT_MAXE * sizeof(unsigned long long)));
    LS_CUDA(cudaMemset(S.ctr, 0, 64 * sizeof(unsigned)));
    LS_CUDA(cudaMemset(S.z, 0, (NE * (kScratchMaxR + 4) + NE) * sizeof(double)));
    S.ready = true;
  }
  if (out) *out = &S;
  return LS_OK;
}

int32_t create_impl(const ls_layer_desc* D, ls_layer* L) {
  L->device = D->device; L->d = D->d_model; L->F = D->d_ff; L->gated = D->gated ? 1 : 0; L->act = D->act;
  L->wd = D->wdtype; L->norm = D->norm; L->eps = D->norm_eps; L->r = D->pred_rank; L->n_mat = L->gated ? 3 : 2;
  L->max_batch = D->max_batch > 0 ? D->max_batch : 1;
  L->max_sel = D->max_sel > 0 ? D->max_sel : D->d_ff;
  L->nwords = (L->F + 31) / 32;
  L->cache_rows = D->cache_rows;
  L->nslots = D->cache_rows > 0 ? D->cache_rows : L->F;
  cudaDeviceProp prop;
  LS_CUDA(cudaGetDeviceProperties(&prop, D->device));
  L->sm_count = prop.multiProcessorCount;
  const size_t d = L->d, F = L->F, row_bytes = d * 2, bundle_bytes = row_bytes * L->n_mat;

  LS_TRY(dalloc(&L->bundles, (size_t)L->nslots * L->n_mat * d));
  const void* mats[3] = {D->w_gate, L->gated ? D->w_up : D->w_down_t, D->w_down_t};
  if (L->cache_rows == 0) {
    for (int m = 0; m < L->n_mat; ++m)
      LS_CUDA(cudaMemcpy2D(reinterpret_cast<char*>(L->bundles) + m * row_bytes, bundle_bytes, mats[m], row_bytes, row_bytes, F,
                           cudaMemcpyHostToDevice));
  } else {
    LS_TRY(ls::cache_create(L->cache, D->device, (int)F, (int)L->cache_rows, bundle_bytes, L->max_sel, L->bundles, g_err));
    char* hb = static_cast<char*>(L->cache.h_bundles);
    for (int m = 0; m < L->n_mat; ++m) {
      const char* src = static_cast<const char*>(mats[m]);
      for (size_t i = 0; i < F; ++i) memcpy(hb + i * bundle_bytes + m * row_bytes, src + i * row_bytes, row_bytes);
    }
  }
  LS_TRY(upload_f32(&L->b_gate, D->b_gate, F));
  if (D->b_down) LS_TRY(upload_f32(&L->b_down, D->b_down, d));
  LS_TRY(upload_transposed16(&L->pred_at, D->pred_a, (int)d, L->r));
  LS_TRY(upload_sliced16(&L->pred_at_sl, D->pred_a, (int)d, L->r));
  LS_TRY(upload_transposed16(&L->pred_bt, D->pred_b, L->r, (int)F));
  if (L->cache_rows == 0) {
    // the same rows at the padded stride the whole-token kernel copies to shared memory, with zero rows behind the last
    const size_t rs = (size_t)ls::wt_brow_bytes(L->r) / 2, nrows = F + 264;
    LS_TRY(dalloc(&L->pred_bt_pad, nrows * rs));
    LS_CUDA(cudaMemset(L->pred_bt_pad, 0, nrows * rs * 2));
    LS_CUDA(cudaMemcpy2D(L->pred_bt_pad, rs * 2, L->pred_bt, (size_t)L->r * 2, (size_t)L->r * 2, F, cudaMemcpyDeviceToDevice));
  }
  LS_TRY(upload_f32(&L->pred_c, D->pred_c, F));

  const size_t MB = L->max_batch;
  LS_TRY(dalloc(&L->z, MB * L->r));
  LS_TRY(dalloc(&L->sumsq, MB));
  LS_TRY(dalloc(&L->scores, MB > 1 ? MB * F : 1));
  LS_TRY(dalloc(&L->prio, F));
  LS_TRY(dalloc(&L->cand_key, F));
  LS_TRY(dalloc(&L->cand_idx, F));
  LS_TRY(dalloc(&L->umask, (size_t)L->nwords));
  LS_TRY(dalloc(&L->tmp_idx, (size_t)L->max_sel));
  LS_TRY(dalloc(&L->tmp_count, 1));
  LS_TRY(dalloc(&L->tmp_mask, (size_t)L->nwords));
  LS_TRY(dalloc(&L->xin, MB * d));
  LS_TRY(dalloc(&L->xt, MB * d));
  LS_TRY(dalloc(&L->actv, MB * L->max_sel));
  L->down_splits = L->sm_count;
  LS_TRY(dalloc(&L->ypart, (size_t)L->down_splits * MB * d));
  LS_TRY(dalloc(&L->survive, (size_t)L->nwords));
  LS_TRY(dalloc(&L->status, 1));
  LS_CUDA(cudaMemset(L->status, 0, sizeof(int)));
  LS_CUDA(cudaMemset(L->prio, 0xff, F * sizeof(double)));  // NaN: ranks last until a prediction sets it

  if (L->cache_rows == 0) {
    LS_TRY(device_scratch(D->device, nullptr));
    LS_TRY(dalloc(&L->wt_range, 2));
    const double zr[2] = {1.0, (double)ls::WT_NB / 2.0};  // scores binned over [-1, 1] until a launch has observed their range
    LS_CUDA(cudaMemcpy(L->wt_range, zr, sizeof zr, cudaMemcpyHostToDevice));
  }
  // opt in to the large dynamic shared memory the kernels may ask for
  const int big = 200 * 1024;
  LS_CUDA(cudaFuncSetAttribute(ls::ls_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, big));
  LS_CUDA(cudaFuncSetAttribute(ls::ls_cache_reserve_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, big));
  LS_CUDA(cudaFuncSetAttribute(ls::ls_cache_evict_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, big));
  LS_CUDA(cudaFuncSetAttribute(ls::ls_scores_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024));
  LS_CUDA(cudaFuncSetAttribute(ls::ls_scores_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024));
#define LS_ATTR_GU(WD, BT) \
  LS_CUDA(cudaFuncSetAttribute(ls::ls_gateup_kernel<WD, BT>, cudaFuncAttributeMaxDynamicSharedMemorySize, big))
  LS_ATTR_GU(0, 1); LS_ATTR_GU(0, 4); LS_ATTR_GU(0, 8); LS_ATTR_GU(1, 1); LS_ATTR_GU(1, 4); LS_ATTR_GU(1, 8);
#undef LS_ATTR_GU
  LS_CUDA(cudaFuncSetAttribute(ls::ls_token_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTokenSmemBudget));
  LS_CUDA(cudaFuncSetAttribute(ls::ls_token_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTokenSmemBudget));
  LS_CUDA(cudaDeviceSynchronize());
  return LS_OK;
}

// Dynamic shared memory of the whole-token kernel for K stages (see ls_token.cuh): fixed regions, then one region whose
// users have disjoint lifetimes (the A slices, the latents of all evaluations, the selection's work area, the general
// top-k's work area).
struct TokenShape { int d, sm_count, r_max, f_max, ns_cta; };
bool token_layout_try(const TokenShape* S, int K, bool mma, ls::WtSmem* out);
// The shared-memory plan: with the tensor-core operand copy of x when d allows it and everything fits, else without
// (the dot products of the stream phase then run as FMA loops).
bool token_layout(const TokenShape* S, int K, ls::WtSmem* out, int* mma_out = nullptr) {
  if (S->d % 16 == 0 && token_layout_try(S, K, true, out)) {
    if (mma_out) *mma_out = 1;
    return true;
  }
  if (mma_out) *mma_out = 0;
  return token_layout_try(S, K, false, out);
}
bool token_layout_try(const TokenShape* S, int K, bool mma, ls::WtSmem* out) {
  const int E = K + 1, G = S->sm_count;
  ls::WtSmem L{};
  size_t o = 0;
  auto take = [&](size_t bytes) { const size_t at = o; o += (bytes + 127) & ~(size_t)127; return (unsigned)at; };
  L.x_off = take((size_t)S->d * 4);
  L.xs_off = take(mma ? (size_t)((S->d + 15) / 16) * 96 : 0);
  L.part_off = take(mma ? (size_t)ls::WT_WARPS * ls::WT_MMA_ROWS * 4 : 0);
  L.xt_off = take((size_t)(ls::WT_MAXE + 1) * ls::WT_XBLK * 8);
  L.dm_off = take((size_t)ls::WT_WARPS * 32 * 4);
  L.mine_off = take((size_t)ls::WT_MAXMINE * (4 + 16 + 4 + 4) + 32 * 4);
  L.bits_off = take((size_t)((S->f_max + 31) / 32) * 4);
  L.pc_off = take((size_t)((S->f_max + G - 1) / G) * 4);
  L.hist_off = take((size_t)(ls::WT_NB + 8) * 4);
  L.u_off = take(0);
  // A slices | B^T rows | max(a slice of the partial outputs, latents) | raw scores | work area (ring / selection lists)
  size_t q = 0;
  auto sub = [&](size_t bytes) { const size_t at = q; q += (bytes + 127) & ~(size_t)127; return (unsigned)at; };
  const int per8 = (((S->f_max + G - 1) / G) + 7) / 8 * 8;
  const int ne = E;  // evaluations scored at once
  sub((size_t)S->ns_cta * S->r_max * 32 * 2);
  L.b_off = sub((size_t)per8 * ls::wt_brow_bytes(S->r_max));
  L.yz_off = sub(std::max((size_t)G * 32 * 4, (size_t)ls::wt_rows(ne) * ls::wt_feat_stride(S->r_max) * 8));
  L.dot_off = sub((size_t)ls::wt_rows(ne) * per8 * 8);
  L.w_off = sub(0);
  L.bin_off = sub((size_t)((S->f_max + 7) / 8 * 8) * 2);
  L.pref_off = sub((size_t)(ls::WT_NB + 1) * 4);
  L.ckey_off = sub((size_t)ls::WT_CANDCAP * 8);
  L.cidx_off = sub((size_t)ls::WT_CANDCAP * 4);
  L.cbin_off = sub((size_t)ls::WT_CANDCAP * 2);
  const size_t bundle_rest = (size_t)2 * S->d * 2 + 16;  // up and down rows of one survivor (rows sit 16 bytes apart modulo 128)
  const size_t u_need = std::max(std::max(q, bundle_rest), ls::topk_smem_bytes(S->f_max));
  if (o + u_need > kTokenSmemBudget) return false;
  L.total = (unsigned)kTokenSmemBudget;  // the rest of the budget lets more rows travel at once
  if (out) *out = L;
  return true;
}

// Launch of the whole-token kernel (a table of layers, or the single layer in c.one): the part common to ls_stack_decode
// and to a fused ls_sparse_ffn_step.  The caller has filled the trace pointers, cuts, sellist, xbuf (and c.one).
int32_t launch_token(const TokenShape* shp, int device, int wd, const ls::WtLayer* d_layers, int n_layers, ls::WtCall& c, const float* d_x,
                     float* d_x_out, const ls_selection* sel_first, int K, int k_next, ls_selection* sel_out, int out_words, cudaStream_t st,
                     const char* who) {
  const int G = shp->sm_count, gs = std::max(1, G / K);
  auto per_cta = [&](int count) { const int m = (count + K - 1) / K; return (m + gs - 1) / gs; };
  if (per_cta(sel_first->cap) > ls::WT_MAXMINE || per_cta(k_next) > ls::WT_MAXMINE)
    return fail(LS_ERR_INVALID, "%s: selection too long for the whole-token kernel", who);
  DeviceScratch* D = nullptr;
  LS_TRY(device_scratch(device, &D));
  if (!token_layout(shp, K, &c.lay, &c.mma)) return fail(LS_ERR_STATE, "%s: %d stages do not fit the whole-token kernel's shared memory", who, K);
  c.n_layers = n_layers; c.d = shp->d; c.K = K; c.k_next = k_next; c.gs = gs;
  c.piece_len = ((shp->d + 3) / 4 + 255) / 256 * 256;
  c.ring_bytes = (int)(c.lay.total - c.lay.u_off);
  c.inv_d = 1.0 / (double)shp->d;
  c.x_in = d_x; c.x_out = d_x_out;
  c.sel_idx = sel_first->idx; c.sel_count = sel_first->count; c.sel_cap = sel_first->cap;
  c.out_idx = sel_out->idx; c.out_count = sel_out->count; c.out_mask = sel_out->mask; c.out_scores = sel_out->scores; c.out_cap = sel_out->cap;
  c.ypart = D->ypart; c.zpart = D->zpart; c.z = D->z; c.sc = D->sc; c.sb = D->sb; c.kmm = D->kmm;
  c.tk_key = reinterpret_cast<unsigned long long*>(D->bent);
  c.tk_idx = reinterpret_cast<int32_t*>(reinterpret_cast<unsigned char*>(D->bent) + (size_t)kScratchMaxF * 8);
  c.bar = D->ctr + 32;
  if (c.tr_masks) LS_CUDA(cudaMemsetAsync(c.tr_masks, 0, (size_t)n_layers * (K + 1) * c.tr_words * 4, st));
  if (sel_out->mask) LS_CUDA(cudaMemsetAsync(sel_out->mask, 0, (size_t)out_words * 4, st));
  LS_CUDA(cudaMemsetAsync(c.bar, 0, sizeof(unsigned), st));
  void* params[] = {&d_layers, &c};
  const void* fn = wd == 0 ? (const void*)ls::ls_token_kernel<0> : (const void*)ls::ls_token_kernel<1>;
  LS_CUDA(cudaLaunchCooperativeKernel(fn, dim3(G), dim3(ls::WT_THREADS), params, c.lay.total, st));
  LS_LAUNCHED();
  return LS_OK;
}

// ---- the fused per-layer step: the whole-token kernel on a single layer --------------------------------------------------
bool fused_shape(const ls_layer* L, const ls_layer* next, TokenShape* shp) {
  shp->d = L->d; shp->sm_count = L->sm_count; shp->r_max = next->r; shp->f_max = std::max(L->F, next->F);
  shp->ns_cta = (((L->d + 31) >> 5) + L->sm_count - 1) / L->sm_count;
  return true;
}
bool fused_eligible(const ls_layer* L, const ls_layer* next, int batch, int K, int sel_cap, int k_next) {
  if (!g_opt_fused.load(std::memory_order_relaxed)) return false;
  if (batch != 1 || !next || L->cache_rows != 0 || next->cache_rows != 0) return false;
  if (K > ls::WT_MAXK || L->d > 8 * ls::WT_THREADS * 2 || L->sm_count > kScratchMaxCtas || L->wd != next->wd) return false;
  const int G = L->sm_count, gs = std::max(1, G / K);
  auto per_cta = [&](int count) { const int m = (count + K - 1) / K; return (m + gs - 1) / gs; };
  if (per_cta(sel_cap) > ls::WT_MAXMINE || per_cta(k_next) > ls::WT_MAXMINE) return false;
  TokenShape shp{};
  fused_shape(L, next, &shp);
  return token_layout(&shp, K, nullptr);
}

int32_t fused_step(ls_layer* L, ls_layer* next, const float* d_x, float* d_x_out, const ls_selection* sel, int K, int k_next,
                   ls_selection* sel_next, const ls_step_trace& tr, cudaStream_t st) {
  ls::WtCall c{};
  TokenShape shp{};
  fused_shape(L, next, &shp);
  DeviceScratch* D = nullptr;
  LS_TRY(device_scratch(L->device, &D));
  ls::WtLayer& a = c.one;
  a.bundles = L->bundles; a.b_gate = L->b_gate; a.b_down = L->b_down;
  a.n_mat = L->n_mat; a.F = L->F; a.norm = L->norm; a.act = L->act; a.eps = L->eps;
  a.At_sl = next->pred_at_sl; a.Bt_pad = next->pred_bt_pad; a.pc = next->pred_c;
  a.r = next->r; a.Fn = next->F; a.norm_n = next->norm; a.eps_n = next->eps;
  a.per = (next->F + L->sm_count - 1) / L->sm_count;
  a.range = next->wt_range;
  a.status = L->status;
  c.cuts = D->cuts1; c.sellist = next->tmp_idx; c.xbuf = nullptr;
  c.tr_xtilde = tr.xtilde; c.tr_masks = tr.refine_masks; c.tr_words = next->nwords; c.tr_counts = tr.refine_counts;
  c.tr_survive = tr.survive_mask;
  if (c.tr_survive) LS_CUDA(cudaMemsetAsync(c.tr_survive, 0, (size_t)L->nwords * 4, st));
  if (tr.exec_idx) {
    ls::ls_copy_u32_kernel<<<8, 256, 0, st>>>(reinterpret_cast<const uint32_t*>(sel->idx), reinterpret_cast<uint32_t*>(tr.exec_idx),
                                              sel->cap);
    LS_LAUNCHED();
  }
  KernelTimer timer(LS_TIMED_FUSED, st);
  return launch_token(&shp, L->device, L->wd, nullptr, 1, c, d_x, d_x_out, sel, K, k_next, sel_next, next->nwords, st, "ls_sparse_ffn_step");
}

// ---- speculate / refine: latent -> scores -> top-k (-> union for batch > 1) ------------------------------------------
int32_t predict_impl(ls_layer* L, const float* d_feature, int B, int k, double* scores_user, uint32_t* mask_out,
                     int32_t* idx_out, int32_t* count_out, int cap, cudaStream_t st) {
  const int d = L->d, r = L->r, F = L->F;
  KernelTimer timer(LS_TIMED_PREDICT, st);
  {
    const int grid = (r + 1) / 2;  // two latent rows per block of eight warps
    if (L->wd == 0) ls::ls_latent_kernel<0><<<grid, 256, 0, st>>>(L->pred_at, d_feature, d, r, B, L->z, L->sumsq);
    else ls::ls_latent_kernel<1><<<grid, 256, 0, st>>>(L->pred_at, d_feature, d, r, B, L->z, L->sumsq);
    LS_LAUNCHED();
  }
  // (a cache decision enqueued on the copy stream may still be reading the priorities and the list of the evaluation
  //  before: the stream joins it here, behind the latents, so that the decision overlaps with whatever ran since)
  if (L->cache_rows > 0) LS_TRY(ls::cache_join(L->cache, st, g_err));
  {
    const int grid = std::min((F + 7) / 8, L->sm_count * 8);
    const size_t sm = (size_t)B * r * sizeof(double);
    if (L->wd == 0)
      ls::ls_scores_kernel<0><<<grid, 256, sm, st>>>(L->pred_bt, L->pred_c, L->z, L->sumsq, d, r, F, B, L->norm, L->eps, L->scores,
                                                     L->prio, scores_user);
    else
      ls::ls_scores_kernel<1><<<grid, 256, sm, st>>>(L->pred_bt, L->pred_c, L->z, L->sumsq, d, r, F, B, L->norm, L->eps, L->scores,
                                                     L->prio, scores_user);
    LS_LAUNCHED();
  }
  const size_t tsm = ls::topk_kernel_smem(F);
  if (B == 1) {
    ls::ls_topk_kernel<<<1, ls::TK_THREADS, tsm, st>>>(L->prio, F, k, nullptr, idx_out, cap, mask_out, 0, count_out, L->cand_key,
                                                       L->cand_idx, L->status);
    LS_LAUNCHED();
  } else {
    ls::ls_fill_u32_kernel<<<1, 256, 0, st>>>(L->umask, 0u, L->nwords);
    LS_LAUNCHED();
    for (int b = 0; b < B; ++b) {
      ls::ls_topk_kernel<<<1, ls::TK_THREADS, tsm, st>>>(L->scores + (size_t)b * F, F, k, nullptr, nullptr, 0, L->umask, 1, nullptr,
                                                         L->cand_key, L->cand_idx, L->status);
      LS_LAUNCHED();
    }
    ls::ls_topk_kernel<<<1, ls::TK_THREADS, tsm, st>>>(L->prio, F, F, L->umask, idx_out, cap, mask_out, 0, count_out, L->cand_key,
                                                       L->cand_idx, L->status);
    LS_LAUNCHED();
  }
  return LS_OK;
}

template <int WD, int BT>
int32_t launch_stage(ls_layer* L, int B, const int32_t* exec_idx, const int32_t* count_ptr, int sel_cap, int K, int c,
                     cudaStream_t st, unsigned need_seq) {
  const int d = L->d;
  const int32_t* slot_of = L->cache_rows > 0 ? L->cache.d_slot_of : nullptr;
  const int per_stage = (sel_cap + K - 1) / K;
  {
    KernelTimer timer(LS_TIMED_GATEUP, st);
    const int grid = std::max(1, std::min((per_stage + 1) / 2, L->sm_count * 4));  // two neurons per block
    const size_t sm = (size_t)B * d * sizeof(float);
    ls::ls_gateup_kernel<WD, BT><<<grid, 256, sm, st>>>(L->bundles, L->n_mat, L->gated, L->act, slot_of, L->b_gate, L->xin, B, d, L->norm,
                                                        L->eps, exec_idx, count_ptr, K, c, L->F, L->actv, L->max_sel, L->survive,
                                                        L->status, need_seq ? L->cache.d_landed : nullptr, need_seq,
                                                        need_seq ? ls::cache_list_header(L->cache, need_seq) : nullptr);
    LS_LAUNCHED();
  }
  {
    KernelTimer timer(LS_TIMED_DOWN, st);
    const int tiles = (d / 8 + 255) / 256;
    const int splits = std::max(1, std::min(L->down_splits, std::max(1, L->sm_count / tiles)));
    dim3 grid(tiles, splits);
    ls::ls_down_kernel<WD, BT><<<grid, 256, 0, st>>>(L->bundles, L->n_mat, slot_of, exec_idx, count_ptr, K, c, L->actv, L->max_sel, B,
                                                     d, L->F, L->ypart);
    LS_LAUNCHED();
    return splits;
  }
}

int32_t launch_stage_dispatch(ls_layer* L, int B, const int32_t* exec_idx, const int32_t* count_ptr, int sel_cap, int K, int c,
                              cudaStream_t st, unsigned need_seq) {
#define LS_STAGE(WD, BT) return launch_stage<WD, BT>(L, B, exec_idx, count_ptr, sel_cap, K, c, st, need_seq)
  if (L->wd == 0) {
    if (B == 1) LS_STAGE(0, 1);
    if (B <= 4) LS_STAGE(0, 4);
    LS_STAGE(0, 8);
  } else {
    if (B == 1) LS_STAGE(1, 1);
    if (B <= 4) LS_STAGE(1, 4);
    LS_STAGE(1, 8);
  }
#undef LS_STAGE
}

inline int32_t cache_rc(int32_t rc) { return rc; }  // (the cache layer returns the public codes and has set the error text)

int32_t check_layer_call(ls_layer* L, int batch, const char* what) {
  if (!L) return fail(LS_ERR_INVALID, "%s: layer is NULL", what);
  if (batch < 1 || batch > L->max_batch) return fail(LS_ERR_INVALID, "%s: batch %d outside [1, max_batch=%d]", what, batch, L->max_batch);
  return LS_OK;
}

}  // namespace

// ---- allocation-free top-k ------------------------------------------------------------------------------------------
// Scratch of ls_topk_select_static: candidate keys (8 bytes each) followed by candidate indices (4 bytes each) for up to
// LS_STATIC_TOPK_MAX_N scores.  It lives in the library image, so every GPU that loads the library holds these 384 KB
// until the process exits.  In host code this name is only a stand-in for the symbol, never a device address: the
// address is taken per device with cudaGetSymbolAddress (static_topk_setup) and handed to the kernel as an argument.
static __device__ __align__(256) unsigned char g_static_topk_scratch[(size_t)LS_STATIC_TOPK_MAX_N * 12];

namespace {

// Same selection as ls_topk_kernel, with the candidate lists kept in caller-independent static device memory instead of
// shared memory / per-layer scratch.  Every position of the lists that is read has been written earlier in the same
// launch, so nothing in the scratch has to start at zero and the previous call's contents do not matter.
__global__ void __launch_bounds__(ls::TK_THREADS, 1)
    ls_topk_static_kernel(const double* __restrict__ keys, int n, int k, int32_t* out_idx, uint32_t* out_mask, int32_t* out_count,
                          unsigned char* scratch) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  ls::TopkSmem sm = ls::topk_carve(smem_raw);
  unsigned long long* ckey = reinterpret_cast<unsigned long long*>(scratch);
  int32_t* cidx = reinterpret_cast<int32_t*>(scratch + (size_t)LS_STATIC_TOPK_MAX_N * 8);
  sm.key = ckey;  // the candidates go to the static scratch whatever their number
  sm.idx = cidx;
  uint32_t* s_mask = reinterpret_cast<uint32_t*>(smem_raw + ls::topk_smem_bytes(n));
  const int nwords = (n + 31) >> 5;
  for (int i = threadIdx.x; i < nwords; i += ls::TK_THREADS) s_mask[i] = 0u;
  const int keff = ls::block_topk(
      n, k,
      [&](int v, double& s) {
        s = keys[v];
        return true;
      },
      [&](int rank, int v) {
        out_idx[rank] = v;
        atomicOr(&s_mask[v >> 5], 1u << (v & 31));
      },
      sm, ckey, cidx);
  if (out_mask)
    for (int w = threadIdx.x; w < nwords; w += ls::TK_THREADS) out_mask[w] = s_mask[w];
  if (threadIdx.x == 0) *out_count = keff;
}

std::mutex g_static_mu;
unsigned char* g_static_ptr[64] = {nullptr};  // device address of the scratch, per device ordinal

// Once per device, with that device current: device address of the static scratch and the kernel's shared-memory opt-in.
int32_t static_topk_setup(int dev, unsigned char** out) {
  std::lock_guard<std::mutex> lk(g_static_mu);
  if (!g_static_ptr[dev]) {
    void* p = nullptr;
    LS_CUDA(cudaGetSymbolAddress(&p, g_static_topk_scratch));
    LS_CUDA(cudaFuncSetAttribute(ls_topk_static_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    g_static_ptr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_static_ptr[dev];
  return LS_OK;
}

}  // namespace

// =====================================================================================================================
extern "C" {

int32_t ls_version(void) { return 1000; }

size_t ls_last_error(char* buf, size_t n) {
  if (buf && n > 0) {
    const size_t m = std::min(n - 1, g_err.size());
    memcpy(buf, g_err.data(), m);
    buf[m] = 0;
  }
  return g_err.size();
}

int64_t ls_kernel_launches(void) { return g_launches.load(); }

int32_t ls_stack_create(ls_layer* const* layers, int32_t n_layers, ls_stack** out) {
  if (out) *out = nullptr;
  if (!layers || !out || n_layers < 1 || n_layers > 4096) return fail(LS_ERR_INVALID, "ls_stack_create: bad argument");
  for (int n = 0; n < n_layers; ++n) {
    const ls_layer* L = layers[n];
    if (!L) return fail(LS_ERR_INVALID, "ls_stack_create: layer %d is NULL", n);
    if (L->cache_rows != 0) return fail(LS_ERR_STATE, "ls_stack_create: layer %d has a cache; the whole-token kernel needs resident layers", n);
    if (L->device != layers[0]->device || L->d != layers[0]->d || L->wd != layers[0]->wd)
      return fail(LS_ERR_INVALID, "ls_stack_create: layer %d differs in device, d_model or weight type", n);
  }
  if (layers[0]->d > 8 * ls::WT_THREADS * 2) return fail(LS_ERR_STATE, "ls_stack_create: d_model %d is beyond the whole-token kernel (8192)", layers[0]->d);
  if (layers[0]->sm_count > kScratchMaxCtas) return fail(LS_ERR_STATE, "ls_stack_create: more SMs than the scratch is sized for");
  DeviceGuard guard(layers[0]->device);
  ls_stack* S = new (std::nothrow) ls_stack();
  if (!S) return fail(LS_ERR_NOMEM, "host allocation");
  S->device = layers[0]->device; S->n = n_layers; S->d = layers[0]->d; S->wd = layers[0]->wd; S->sm_count = layers[0]->sm_count;
  S->cpt = ((S->d >> 3) + ls::WT_THREADS - 1) / ls::WT_THREADS;
  S->ns_cta = (((S->d + 31) >> 5) + S->sm_count - 1) / S->sm_count;
  S->layers.assign(layers, layers + n_layers);
  for (int n = 0; n < n_layers; ++n) {
    S->max_sel = std::max(S->max_sel, layers[n]->max_sel);
    S->r_max = std::max(S->r_max, layers[n]->r);
    S->f_max = std::max(S->f_max, layers[n]->F);
  }
  auto cleanup = [&](int32_t rc) {
    const std::string keep = g_err;
    cudaFree(S->d_layers); cudaFree(S->xbuf); cudaFree(S->ranges); cudaFree(S->cuts); cudaFree(S->sellist);
    delete S;
    g_err = keep;
    return rc;
  };
  int32_t rc;
  if ((rc = device_scratch(S->device, nullptr)) != LS_OK) return cleanup(rc);
  if ((rc = dalloc(&S->d_layers, (size_t)n_layers)) != LS_OK) return cleanup(rc);
  if ((rc = dalloc(&S->xbuf, (size_t)2 * S->d)) != LS_OK) return cleanup(rc);
  if ((rc = dalloc(&S->ranges, (size_t)2 * n_layers)) != LS_OK) return cleanup(rc);
  if ((rc = dalloc(&S->cuts, (size_t)n_layers * ls::WT_MAXE)) != LS_OK) return cleanup(rc);
  if ((rc = dalloc(&S->sellist, (size_t)std::max(1, S->max_sel))) != LS_OK) return cleanup(rc);
  std::vector<ls::WtLayer> h(n_layers);
  std::vector<double> hr((size_t)2 * n_layers);
  for (int n = 0; n < n_layers; ++n) {
    ls_layer* L = layers[n];
    ls_layer* next = layers[n + 1 < n_layers ? n + 1 : n];  // the last layer refines a weight-tied copy of itself
    ls::WtLayer& a = h[n];
    a.bundles = L->bundles; a.b_gate = L->b_gate; a.b_down = L->b_down;
    a.n_mat = L->n_mat; a.F = L->F; a.norm = L->norm; a.act = L->act; a.eps = L->eps;
    a.At_sl = next->pred_at_sl; a.Bt_pad = next->pred_bt_pad; a.pc = next->pred_c;
    a.r = next->r; a.Fn = next->F; a.norm_n = next->norm; a.eps_n = next->eps;
    a.per = (next->F + L->sm_count - 1) / L->sm_count;
    a.range = S->ranges + 2 * n;
    a.status = L->status;
    hr[2 * n] = 1.0;                          // scores binned over [-1, 1] until a launch has observed their range
    hr[2 * n + 1] = (double)ls::WT_NB / 2.0;
  }
  if (cudaMemcpy(S->d_layers, h.data(), sizeof(ls::WtLayer) * n_layers, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(S->ranges, hr.data(), sizeof(double) * hr.size(), cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemset(S->cuts, 0, sizeof(unsigned long long) * n_layers * ls::WT_MAXE) != cudaSuccess)
    return cleanup(fail(LS_ERR_CUDA, "ls_stack_create: upload of the layer arguments failed"));
#define LS_ATTR_WT(WD)                                                                                                       \
  if (cudaFuncSetAttribute(ls::ls_token_kernel<WD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTokenSmemBudget) != \
      cudaSuccess)                                                                                                           \
    return cleanup(fail(LS_ERR_CUDA, "ls_stack_create: shared-memory opt-in failed"))
  LS_ATTR_WT(0); LS_ATTR_WT(1);
#undef LS_ATTR_WT
  {
    ls::WtSmem lay{};
    const TokenShape shp{S->d, S->sm_count, S->r_max, S->f_max, S->ns_cta};
    if (!token_layout(&shp, ls::WT_MAXK, &lay) && !token_layout(&shp, 1, &lay))
      return cleanup(fail(LS_ERR_STATE, "ls_stack_create: the stack does not fit the whole-token kernel's shared memory"));
  }
  *out = S;
  return LS_OK;
}

int32_t ls_stack_destroy(ls_stack* S) {
  if (!S) return LS_OK;
  DeviceGuard guard(S->device);
  cudaDeviceSynchronize();
  cudaFree(S->d_layers); cudaFree(S->xbuf); cudaFree(S->ranges); cudaFree(S->cuts); cudaFree(S->sellist);
  delete S;
  return LS_OK;
}

int32_t ls_stack_decode(ls_stack* S, const float* d_x, float* d_x_out, const ls_selection* sel_first, int32_t K, int32_t k_next,
                        ls_selection* sel_out, ls_stack_trace* trace, void* stream) {
  if (!S || !d_x || !d_x_out || !sel_first || !sel_first->idx || !sel_first->count || !sel_out || !sel_out->idx || !sel_out->count)
    return fail(LS_ERR_INVALID, "ls_stack_decode: x, x_out, sel_first and sel_out (idx, count) are required");
  if (K < 1 || K > ls::WT_MAXK) return fail(LS_ERR_INVALID, "ls_stack_decode: n_chunks %d outside [1, %d]", K, ls::WT_MAXK);
  if (sel_first->cap < 0 || sel_first->cap > S->layers[0]->max_sel) return fail(LS_ERR_INVALID, "ls_stack_decode: sel_first->cap outside [0, max_sel]");
  int fmin_ = 1 << 30;
  for (ls_layer* L : S->layers) fmin_ = std::min(fmin_, std::min(L->F, L->max_sel));
  if (k_next < 0 || k_next > fmin_) return fail(LS_ERR_INVALID, "ls_stack_decode: k_next %d outside [0, %d] (smallest d_ff / max_sel of the stack)", k_next, fmin_);
  if (sel_out->cap < k_next) return fail(LS_ERR_INVALID, "ls_stack_decode: sel_out->cap %d < k_next %d", sel_out->cap, k_next);
  DeviceGuard guard(S->device);
  cudaStream_t st = (cudaStream_t)stream;
  ls::WtCall c{};
  const int nwords_max = (S->f_max + 31) / 32;
  if (trace) {
    c.tr_x = trace->x; c.tr_sel = trace->sel_idx; c.tr_cnt = trace->sel_count; c.tr_cap = trace->sel_cap;
    c.tr_xtilde = trace->xtilde; c.tr_masks = trace->refine_masks; c.tr_words = trace->mask_words; c.tr_ns = trace->phase_ns;
    if (c.tr_sel && !c.tr_cnt) return fail(LS_ERR_INVALID, "ls_stack_decode: trace->sel_count is required with trace->sel_idx");
    if (c.tr_masks && c.tr_words < nwords_max)
      return fail(LS_ERR_INVALID, "ls_stack_decode: trace->mask_words %d < %d", c.tr_words, nwords_max);
  }
  c.cuts = S->cuts; c.sellist = S->sellist; c.xbuf = S->xbuf;
  const TokenShape shp{S->d, S->sm_count, S->r_max, S->f_max, S->ns_cta};
  KernelTimer timer(LS_TIMED_STACK, st);
  return launch_token(&shp, S->device, S->wd, S->d_layers, S->n, c, d_x, d_x_out, sel_first, K, k_next, sel_out, S->layers.back()->nwords, st,
                      "ls_stack_decode");
}

int32_t ls_topk_select_static(const double* d_scores, int32_t n, int32_t k, int32_t* d_idx, uint32_t* d_mask, int32_t* d_count,
                              void* stream) {
  if (!d_scores || !d_idx || !d_count) return fail(LS_ERR_INVALID, "ls_topk_select_static: scores, idx and count are required");
  if (n < 1 || n > LS_STATIC_TOPK_MAX_N)
    return fail(LS_ERR_INVALID, "ls_topk_select_static: n = %d is outside [1, %d] (the static scratch holds at most %d candidates)", n,
                LS_STATIC_TOPK_MAX_N, LS_STATIC_TOPK_MAX_N);
  if (k < 0 || k > n) return fail(LS_ERR_INVALID, "ls_topk_select_static: k = %d is outside [0, n = %d]", k, n);
  // the launch goes to the device that owns the scores (its copy of the static scratch), whatever device is current
  int dev = -1;
  cudaPointerAttributes at{};
  if (cudaPointerGetAttributes(&at, d_scores) == cudaSuccess && at.type == cudaMemoryTypeDevice) dev = at.device;
  else { cudaGetLastError(); LS_CUDA(cudaGetDevice(&dev)); }
  if (dev < 0 || dev >= 64) return fail(LS_ERR_INVALID, "ls_topk_select_static: device ordinal %d not supported", dev);
  DeviceGuard guard(dev);
  unsigned char* scratch = nullptr;
  LS_TRY(static_topk_setup(dev, &scratch));
  ls_topk_static_kernel<<<1, ls::TK_THREADS, ls::topk_kernel_smem(n), (cudaStream_t)stream>>>(d_scores, n, k, d_idx, d_mask, d_count,
                                                                                               scratch);
  LS_LAUNCHED();
  return LS_OK;
}


// ---- stacked hashing predictor ----------------------------------------------------------------------------------------
int32_t ls_hash_predictor_destroy(ls_hash_predictor* P) {
  if (!P) return LS_OK;
  DeviceGuard guard(P->device);
  cudaDeviceSynchronize();
  cudaFree(P->pca_t); cudaFree(P->w1); cudaFree(P->w); cudaFree(P->tables); cudaFree(P->codes); cudaFree(P->z); cudaFree(P->sumsq);
  cudaFree(P->y); cudaFree(P->scores); cudaFree(P->cand_key); cudaFree(P->cand_idx); cudaFree(P->status);
  delete P;
  return LS_OK;
}

int32_t ls_hash_predictor_create(const ls_hash_predictor_desc* D, ls_hash_predictor** out) {
  if (out) *out = nullptr;
  if (!D || !out) return fail(LS_ERR_INVALID, "ls_hash_predictor_create: NULL argument");
  if (D->struct_size != sizeof(ls_hash_predictor_desc))
    return fail(LS_ERR_INVALID, "ls_hash_predictor_create: struct_size %u, expected %zu", D->struct_size, sizeof(ls_hash_predictor_desc));
  if (D->d_model < 8 || D->d_model % 8 || D->d_model > 16384 || D->rank < 8 || D->rank % 8 || D->rank > 1024)
    return fail(LS_ERR_INVALID, "ls_hash_predictor_create: d_model, rank must be multiples of 8 within [8, 16384] / [8, 1024]");
  if (D->tau < 1 || D->tau > ls::HASH_MAX_TAU || D->d_code < 32 || D->d_code % 32 || D->d_code > 32 * ls::HASH_MAX_WORDS ||
      D->n_layers < 1 || D->n_layers > ls::HASH_MAX_LAYERS || D->d_ff < 1 || D->d_ff > 32768)
    return fail(LS_ERR_INVALID, "ls_hash_predictor_create: tau, d_code, n_layers or d_ff out of range");
  if (D->wdtype != LS_WDTYPE_BF16 && D->wdtype != LS_WDTYPE_FP16) return fail(LS_ERR_INVALID, "unknown wdtype");
  if (!D->pca || !D->w1 || !D->tables || !D->codes || (D->n_layers > 1 && !D->w)) return fail(LS_ERR_INVALID, "ls_hash_predictor_create: missing table");
  int ndev = 0;
  LS_CUDA(cudaGetDeviceCount(&ndev));
  if (D->device < 0 || D->device >= ndev) return fail(LS_ERR_INVALID, "device %d out of range", D->device);
  DeviceGuard guard(D->device);
  ls_hash_predictor* P = new (std::nothrow) ls_hash_predictor();
  if (!P) return fail(LS_ERR_NOMEM, "host allocation");
  P->device = D->device; P->d = D->d_model; P->r = D->rank; P->tau = D->tau; P->words = D->d_code / 32; P->n_layers = D->n_layers;
  P->F = D->d_ff; P->wd = D->wdtype;
  cudaDeviceProp prop;
  int32_t rc = LS_OK;
  auto up = [&](auto** dst, const void* src, size_t n) -> int32_t {
    LS_TRY(dalloc(dst, n));
    if (src && n) LS_CUDA(cudaMemcpy(*dst, src, n * sizeof(**dst), cudaMemcpyHostToDevice));
    return LS_OK;
  };
  const size_t W = P->words, nb = (size_t)1 << P->tau;
  if (cudaGetDeviceProperties(&prop, D->device) == cudaSuccess) P->sm_count = prop.multiProcessorCount;
  if ((rc = upload_transposed16(&P->pca_t, D->pca, P->d, P->r)) != LS_OK || (rc = up(&P->w1, D->w1, (size_t)P->r * P->tau)) != LS_OK ||
      (rc = up(&P->w, D->w, (size_t)(P->n_layers - 1) * P->tau * W)) != LS_OK || (rc = up(&P->tables, D->tables, (size_t)P->n_layers * nb * W)) != LS_OK ||
      (rc = up(&P->codes, D->codes, (size_t)P->F * W)) != LS_OK || (rc = dalloc(&P->z, (size_t)P->r)) != LS_OK ||
      (rc = dalloc(&P->sumsq, 1)) != LS_OK || (rc = dalloc(&P->y, W)) != LS_OK || (rc = dalloc(&P->scores, (size_t)P->F)) != LS_OK ||
      (rc = dalloc(&P->cand_key, (size_t)P->F)) != LS_OK || (rc = dalloc(&P->cand_idx, (size_t)P->F)) != LS_OK ||
      (rc = dalloc(&P->status, 1)) != LS_OK) {
    const std::string keep = g_err;
    ls_hash_predictor_destroy(P);
    g_err = keep;
    return rc;
  }
  cudaMemset(P->status, 0, sizeof(int));
  cudaFuncSetAttribute(ls::ls_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  LS_CUDA(cudaDeviceSynchronize());
  *out = P;
  return LS_OK;
}

int32_t ls_hash_predict(ls_hash_predictor* P, const float* d_feature, int32_t k, ls_selection* out, int32_t* d_layer_idx, void* stream) {
  if (!P || !d_feature || !out || !out->idx || !out->count) return fail(LS_ERR_INVALID, "ls_hash_predict: predictor, feature, out->idx and out->count are required");
  if (k < 0 || k > P->F) return fail(LS_ERR_INVALID, "ls_hash_predict: k %d outside [0, d_ff]", k);
  if (out->cap < k) return fail(LS_ERR_INVALID, "ls_hash_predict: out->cap %d < k %d", out->cap, k);
  DeviceGuard guard(P->device);
  cudaStream_t st = (cudaStream_t)stream;
  KernelTimer timer(LS_TIMED_PREDICT, st);
  {
    const int grid = (P->r + 1) / 2;  // two latent rows per block of eight warps
    if (P->wd == 0) ls::ls_latent_kernel<0><<<grid, 256, 0, st>>>(P->pca_t, d_feature, P->d, P->r, 1, P->z, P->sumsq);
    else ls::ls_latent_kernel<1><<<grid, 256, 0, st>>>(P->pca_t, d_feature, P->d, P->r, 1, P->z, P->sumsq);
    LS_LAUNCHED();
  }
  ls::ls_hash_layers_kernel<<<1, 256, 0, st>>>(P->z, P->w1, P->r, P->tau, P->words, P->n_layers, P->w, P->tables, P->y, d_layer_idx);
  LS_LAUNCHED();
  ls::ls_hash_scores_kernel<<<std::min((P->F + 255) / 256, P->sm_count * 4), 256, 0, st>>>(P->y, P->codes, P->words, P->F, P->scores, out->scores);
  LS_LAUNCHED();
  ls::ls_topk_kernel<<<1, ls::TK_THREADS, ls::topk_kernel_smem(P->F), st>>>(P->scores, P->F, k, nullptr, out->idx, out->cap, out->mask, 0, out->count,
                                                                          P->cand_key, P->cand_idx, P->status);
  LS_LAUNCHED();
  return LS_OK;
}

// ---- streaming controller (host side) -------------------------------------------------------------------------------
int32_t ls_controller_quantize(double remaining, double vmax, int32_t n_states) {
  if (n_states < 1 || !(vmax > 0.0)) return fail(LS_ERR_INVALID, "ls_controller_quantize: n_states >= 1 and vmax > 0 are required");
  if (!(remaining > 0.0)) return 0;
  const double b = floor(remaining / vmax * (double)n_states);
  return b >= (double)(n_states - 1) ? n_states - 1 : (int32_t)b;
}

int32_t ls_controller_build(int32_t N, int32_t Q, int32_t A, int32_t S, int32_t H, const double* t_bar, const int32_t* next_state,
                            int32_t* lut, double* value) {
  if (N < 1 || Q < 1 || A < 1 || S < 0 || H < 1 || !t_bar || !lut || (S > 0 && !next_state))
    return fail(LS_ERR_INVALID, "ls_controller_build: bad argument");
  for (size_t i = 0; S > 0 && i < (size_t)N * Q * A * S; ++i)
    if (next_state[i] >= Q) return fail(LS_ERR_INVALID, "ls_controller_build: state sample %d outside [0, %d)", next_state[i], Q);
  const double INF = std::numeric_limits<double>::infinity();
  std::vector<double> prev((size_t)(N + 1) * Q, 0.0), cur((size_t)(N + 1) * Q, 0.0);
  for (int h = 1; h <= H; ++h) {
    std::fill(cur.begin(), cur.end(), 0.0);
    for (int n = 0; n < N; ++n)
      for (int q = 0; q < Q; ++q) {
        double best = INF;
        int best_a = -1;
        for (int a = 0; a < A; ++a) {
          const double t = t_bar[((size_t)n * Q + q) * A + a];
          if (!(t >= 0.0) || t == INF) continue;
          double future = 0.0;
          if (n + 1 < N && S > 0) {
            const int32_t* smp = next_state + (((size_t)n * Q + q) * A + a) * S;
            double sum = 0.0;
            int cnt = 0;
            for (int s = 0; s < S; ++s)
              if (smp[s] >= 0) { sum += prev[(size_t)(n + 1) * Q + smp[s]]; ++cnt; }
            future = cnt > 0 ? sum / cnt : 0.0;
          }
          const double cost = t + future;
          if (cost < best) { best = cost; best_a = a; }
        }
        cur[(size_t)n * Q + q] = best_a >= 0 ? best : INF;
        if (h == H) lut[(size_t)n * Q + q] = best_a;
      }
    prev.swap(cur);
  }
  if (value)
    for (size_t i = 0; i < (size_t)N * Q; ++i) value[i] = prev[i];
  return LS_OK;
}

int32_t ls_set_option(int32_t option, int32_t value) {
  if (option == LS_OPT_FUSED) {
    g_opt_fused.store(value ? 1 : 0);
    return LS_OK;
  }
  if (option == LS_OPT_MISS_PATH) {
    if (value != LS_MISS_PATH_LANE && value != LS_MISS_PATH_GATHER) return fail(LS_ERR_INVALID, "ls_set_option: unknown miss path %d", value);
    g_opt_miss_path.store(value);
    return LS_OK;
  }
  if (option == LS_OPT_HOST_WAIT_MS) {
    if (value < 0) return fail(LS_ERR_INVALID, "ls_set_option: negative wait limit");
    g_opt_host_wait_ms.store(value);
    return LS_OK;
  }
  return fail(LS_ERR_INVALID, "ls_set_option: unknown option %d", option);
}

int32_t ls_timing_enable(int32_t on) {
  g_timing.store(on ? 1 : 0);
  return LS_OK;
}

int32_t ls_timing_read(int32_t kind, int64_t* launches, double* total_ms) {
  if (!launches || !total_ms) return fail(LS_ERR_INVALID, "ls_timing_read: NULL argument");
  std::lock_guard<std::mutex> lk(g_timing_mu);
  *launches = 0;
  *total_ms = 0.0;
  std::vector<TimedLaunch> keep;
  for (const TimedLaunch& t : g_timed) {
    if (t.kind != kind) { keep.push_back(t); continue; }
    float ms = 0.f;
    cudaError_t e = cudaEventSynchronize(t.b);
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, t.a, t.b);
    cudaEventDestroy(t.a);
    cudaEventDestroy(t.b);
    if (e != cudaSuccess) return fail(LS_ERR_CUDA, "ls_timing_read: %s", cudaGetErrorString(e));
    *launches += 1;
    *total_ms += ms;
  }
  g_timed.swap(keep);
  return LS_OK;
}

int32_t ls_layer_create(const ls_layer_desc* D, ls_layer** out) {
  if (out) *out = nullptr;
  if (!D || !out) return fail(LS_ERR_INVALID, "ls_layer_create: NULL argument");
  if (D->struct_size != sizeof(ls_layer_desc))
    return fail(LS_ERR_INVALID, "ls_layer_create: struct_size %u, expected %zu", D->struct_size, sizeof(ls_layer_desc));
  if (D->d_model < 8 || D->d_model % 8 || D->d_model > 16384) return fail(LS_ERR_INVALID, "d_model must be a multiple of 8 in [8, 16384]");
  if (D->d_ff < 1 || D->d_ff > 32768) return fail(LS_ERR_INVALID, "d_ff must be in [1, 32768]");
  if (D->pred_rank < 8 || D->pred_rank % 8 || D->pred_rank > 1024) return fail(LS_ERR_INVALID, "pred_rank must be a multiple of 8 in [8, 1024]");
  if (D->act != LS_ACT_RELU && D->act != LS_ACT_SILU) return fail(LS_ERR_INVALID, "act must be LS_ACT_RELU or LS_ACT_SILU");
  if (D->wdtype != LS_WDTYPE_BF16 && D->wdtype != LS_WDTYPE_FP16) return fail(LS_ERR_INVALID, "unknown wdtype");
  if (D->norm != LS_NORM_RMS && D->norm != LS_NORM_NONE) return fail(LS_ERR_INVALID, "unknown norm");
  if (!D->w_gate || !D->w_down_t || (D->gated && !D->w_up) || !D->pred_a || !D->pred_b)
    return fail(LS_ERR_INVALID, "ls_layer_create: missing weight pointer");
  if (D->cache_rows < 0 || D->cache_rows > D->d_ff) return fail(LS_ERR_INVALID, "cache_rows must be in [0, d_ff]");
  if (D->max_batch < 0 || D->max_batch > 8) return fail(LS_ERR_INVALID, "max_batch must be in [0, 8]");
  if (D->max_sel < 0 || D->max_sel > D->d_ff) return fail(LS_ERR_INVALID, "max_sel must be in [0, d_ff]");
  const int mb = D->max_batch > 0 ? D->max_batch : 1;
  if ((size_t)mb * D->d_model * 4 > 192 * 1024) return fail(LS_ERR_INVALID, "max_batch * d_model * 4 bytes must fit in 192 KB of shared memory");
  int ndev = 0;
  LS_CUDA(cudaGetDeviceCount(&ndev));
  if (D->device < 0 || D->device >= ndev) return fail(LS_ERR_INVALID, "device %d out of range", D->device);
  DeviceGuard guard(D->device);
  ls_layer* L = new (std::nothrow) ls_layer();
  if (!L) return fail(LS_ERR_NOMEM, "host allocation");
  const int32_t rc = create_impl(D, L);
  if (rc != LS_OK) {
    const std::string keep = g_err;
    free_layer(L);
    cudaGetLastError();
    g_err = keep;
    return rc;
  }
  *out = L;
  return LS_OK;
}

int32_t ls_layer_destroy(ls_layer* L) {
  if (!L) return LS_OK;
  DeviceGuard guard(L->device);
  cudaDeviceSynchronize();
  free_layer(L);
  return LS_OK;
}

int32_t ls_layer_status(ls_layer* L, int32_t* host_status) {
  if (!L || !host_status) return fail(LS_ERR_INVALID, "ls_layer_status: NULL argument");
  DeviceGuard guard(L->device);
  LS_CUDA(cudaDeviceSynchronize());
  LS_CUDA(cudaMemcpy(host_status, L->status, sizeof(int), cudaMemcpyDeviceToHost));
  LS_CUDA(cudaMemset(L->status, 0, sizeof(int)));
  return LS_OK;
}

int32_t ls_predict(ls_layer* L, const float* d_feature, int32_t batch, int32_t k, ls_selection* out, void* stream) {
  LS_TRY(check_layer_call(L, batch, "ls_predict"));
  if (!d_feature || !out || !out->idx || !out->count) return fail(LS_ERR_INVALID, "ls_predict: feature, out->idx and out->count are required");
  if (k < 0 || k > L->F) return fail(LS_ERR_INVALID, "ls_predict: k %d outside [0, d_ff]", k);
  const long need = std::min<long>((long)batch * k, L->F);
  if (out->cap < need) return fail(LS_ERR_INVALID, "ls_predict: out->cap %d < %ld", out->cap, need);
  DeviceGuard guard(L->device);
  return predict_impl(L, d_feature, batch, k, out->scores, out->mask, out->idx, out->count, out->cap, (cudaStream_t)stream);
}

int32_t ls_sparse_ffn_step(ls_layer* L, ls_layer* next, const float* d_x, float* d_x_out, int32_t batch, const ls_selection* sel,
                           int32_t K, int32_t k_next, ls_selection* sel_next, ls_step_trace* trace, void* stream) {
  LS_TRY(check_layer_call(L, batch, "ls_sparse_ffn_step"));
  if (!d_x || !d_x_out || !sel || !sel->idx || !sel->count) return fail(LS_ERR_INVALID, "ls_sparse_ffn_step: x, x_out, sel->idx, sel->count are required");
  if (K < 1 || K > 4096) return fail(LS_ERR_INVALID, "ls_sparse_ffn_step: n_chunks %d outside [1, 4096]", K);
  if (sel->cap < 0 || sel->cap > L->max_sel) return fail(LS_ERR_INVALID, "ls_sparse_ffn_step: sel->cap %d outside [0, max_sel=%d]", sel->cap, L->max_sel);
  if (next) {
    if (next->d != L->d) return fail(LS_ERR_INVALID, "ls_sparse_ffn_step: next layer has a different d_model");
    if (next->device != L->device) return fail(LS_ERR_INVALID, "ls_sparse_ffn_step: next layer is on another device");
    if (batch > next->max_batch) return fail(LS_ERR_INVALID, "ls_sparse_ffn_step: batch exceeds next->max_batch");
    if (!sel_next || !sel_next->idx || !sel_next->count) return fail(LS_ERR_INVALID, "ls_sparse_ffn_step: sel_next->idx and ->count are required with next");
    if (k_next < 0 || k_next > next->F) return fail(LS_ERR_INVALID, "ls_sparse_ffn_step: k_next outside [0, d_ff_next]");
    const long need = std::min<long>((long)batch * k_next, next->F);
    if (sel_next->cap < need || need > next->max_sel) return fail(LS_ERR_INVALID, "ls_sparse_ffn_step: sel_next->cap or next->max_sel below %ld", need);
  }
  DeviceGuard guard(L->device);
  cudaStream_t st = (cudaStream_t)stream;
  const int d = L->d, B = batch;
  const size_t bd = (size_t)B * d;
  ls_step_trace tr{};
  if (trace) tr = *trace;

  if (fused_eligible(L, next, B, K, sel->cap, k_next)) return fused_step(L, next, d_x, d_x_out, sel, K, k_next, sel_next, tr, st);

  ls::ls_step_init_kernel<<<std::min(64, (int)((bd + 255) / 256)), 256, 0, st>>>(d_x, L->b_down, L->xin, L->xt, tr.xtilde, B, d,
                                                                               L->survive, L->nwords, nullptr);
  LS_LAUNCHED();

  const int32_t* exec_idx = sel->idx;
  unsigned own_seq = 0;
  const int miss_path = g_opt_miss_path.load(std::memory_order_relaxed);
  if (L->cache_rows > 0) {
    // reserve the whole selection; residents run first, misses after (in the order their copies are issued).  Nothing
    // waits here: the stages that reach into the misses wait on the device for the request's rows.
    if (sel->cap > L->cache_rows) return fail(LS_ERR_CAPACITY, "ls_sparse_ffn_step: selection capacity %d exceeds the cache (%lld rows)", sel->cap, (long long)L->cache_rows);
    const double limit_s = g_opt_host_wait_ms.load(std::memory_order_relaxed) * 1e-3;
    LS_TRY(cache_rc(ls::cache_reserve_async(L->cache, miss_path, L->prio, L->F, sel->idx, sel->count, -1, 0, 0, sel->cap, nullptr, L->status, st,
                                            &own_seq, limit_s, g_err, g_launches)));
    // (I/O lane: the stages are enqueued once the copies of this request have been issued; see cache_lane_wait)
    if (miss_path == ls::MISS_PATH_LANE) LS_TRY(cache_rc(ls::cache_lane_wait(L->cache, own_seq, limit_s, g_err)));
    exec_idx = L->cache.d_exec_idx;
  }
  if (tr.exec_idx) {
    ls::ls_copy_u32_kernel<<<8, 256, 0, st>>>(reinterpret_cast<const uint32_t*>(exec_idx), reinterpret_cast<uint32_t*>(tr.exec_idx),
                                              sel->cap);
    LS_LAUNCHED();
  }

  auto refine = [&](int j) -> int32_t {
    if (!next) return LS_OK;
    const bool last = (j == K);
    uint32_t* mask_out = tr.refine_masks ? tr.refine_masks + (size_t)j * next->nwords : (last ? sel_next->mask : nullptr);
    int32_t* idx_out = last ? sel_next->idx : next->tmp_idx;
    int32_t* cnt_out = last ? sel_next->count : next->tmp_count;
    const int cap = last ? sel_next->cap : next->max_sel;
    LS_TRY(predict_impl(next, L->xt, B, k_next, last ? sel_next->scores : nullptr, mask_out, idx_out, cnt_out, cap, st));
    if (last && tr.refine_masks && sel_next->mask) {
      ls::ls_copy_u32_kernel<<<4, 256, 0, st>>>(mask_out, sel_next->mask, next->nwords);
      LS_LAUNCHED();
    }
    if (tr.refine_counts) {
      ls::ls_copy_u32_kernel<<<1, 32, 0, st>>>(reinterpret_cast<const uint32_t*>(cnt_out),
                                               reinterpret_cast<uint32_t*>(tr.refine_counts + j), 1);
      LS_LAUNCHED();
    }
    if (!last && next->cache_rows > 0 && next != L) {
      // fetch rule: the first ceil(count (j+1)/(K+1)) ranks of C^(j) are admitted
      LS_TRY(cache_rc(ls::cache_reserve_async(next->cache, miss_path, next->prio, next->F, idx_out, cnt_out, 0, j + 1, K + 1, next->max_sel,
                                              nullptr, next->status, st, nullptr, g_opt_host_wait_ms.load(std::memory_order_relaxed) * 1e-3,
                                              g_err, g_launches, /*side=*/true)));
    }
    return LS_OK;
  };

  LS_TRY(refine(0));
  for (int c = 0; c < K; ++c) {
    const int32_t splits = launch_stage_dispatch(L, B, exec_idx, sel->count, sel->cap, K, c, st, own_seq);
    if (splits < 0) return splits;
    const bool last = (c + 1 == K);
    ls::ls_stage_finalize_kernel<<<std::min(4 * L->sm_count, (int)((bd + 31) / 32)), 256, 0, st>>>(
        L->ypart, splits, B, d, L->xt, tr.xtilde ? tr.xtilde + (size_t)(c + 1) * bd : nullptr, last ? d_x_out : nullptr);
    LS_LAUNCHED();
    LS_TRY(refine(c + 1));
  }
  if (tr.survive_mask) {
    ls::ls_copy_u32_kernel<<<4, 256, 0, st>>>(L->survive, tr.survive_mask, L->nwords);
    LS_LAUNCHED();
  }
  return LS_OK;
}

// ---- cache entry points ---------------------------------------------------------------------------------------------
int32_t ls_cache_lookup(ls_layer* L, const int32_t* d_idx, int32_t n, int32_t* d_slot, int32_t* d_nhit, void* stream) {
  if (!L || !d_idx || !d_slot) return fail(LS_ERR_INVALID, "ls_cache_lookup: NULL argument");
  if (L->cache_rows == 0) return fail(LS_ERR_STATE, "ls_cache_lookup: layer has no cache");
  if (n < 0 || n > L->max_sel) return fail(LS_ERR_INVALID, "ls_cache_lookup: n outside [0, max_sel]");
  DeviceGuard guard(L->device);
  return ls::cache_lookup(L->cache, L->F, d_idx, n, d_slot, d_nhit, L->status, (cudaStream_t)stream, g_err, g_launches);
}

int32_t ls_cache_reserve(ls_layer* L, const ls_selection* want, int32_t admit_ranks, const uint32_t* d_protect_mask, int32_t* h_nmiss,
                         void* stream) {
  if (!L || !want || !want->idx || !want->count) return fail(LS_ERR_INVALID, "ls_cache_reserve: NULL argument");
  if (L->cache_rows == 0) return fail(LS_ERR_STATE, "ls_cache_reserve: layer has no cache");
  if (want->cap < 0 || want->cap > L->max_sel) return fail(LS_ERR_INVALID, "ls_cache_reserve: want->cap outside [0, max_sel]");
  DeviceGuard guard(L->device);
  cudaStream_t st = (cudaStream_t)stream;
  if (want->scores) LS_CUDA(cudaMemcpyAsync(L->prio, want->scores, (size_t)L->F * sizeof(double), cudaMemcpyDeviceToDevice, st));
  unsigned seq = 0;
  LS_TRY(cache_rc(ls::cache_reserve_async(L->cache, g_opt_miss_path.load(std::memory_order_relaxed), L->prio, L->F, want->idx, want->count,
                                          admit_ranks < 0 ? -1 : admit_ranks, 0, 0, want->cap, d_protect_mask, L->status, st, &seq,
                                          g_opt_host_wait_ms.load(std::memory_order_relaxed) * 1e-3, g_err, g_launches)));
  // this call reports the number of misses: it waits (bounded) for the decision, not for the copies
  return cache_rc(ls::cache_request_result(L->cache, seq, st, g_opt_host_wait_ms.load(std::memory_order_relaxed) * 1e-3, h_nmiss, g_err));
}

int32_t ls_cache_evict(ls_layer* L, int32_t min_free, const uint32_t* d_protect_mask, int32_t* d_evicted, int32_t* d_nevicted,
                       void* stream) {
  if (!L) return fail(LS_ERR_INVALID, "ls_cache_evict: NULL layer");
  if (L->cache_rows == 0) return fail(LS_ERR_STATE, "ls_cache_evict: layer has no cache");
  if (min_free < 0 || min_free > L->cache_rows) return fail(LS_ERR_INVALID, "ls_cache_evict: min_free outside [0, cache_rows]");
  DeviceGuard guard(L->device);
  return ls::cache_evict(L->cache, L->prio, L->F, min_free, d_protect_mask, d_evicted, d_nevicted, L->status, (cudaStream_t)stream,
                         g_err, g_launches);
}

int32_t ls_cache_snapshot(ls_layer* L, uint32_t* d_resident_mask, void* stream) {
  if (!L || !d_resident_mask) return fail(LS_ERR_INVALID, "ls_cache_snapshot: NULL argument");
  if (L->cache_rows == 0) return fail(LS_ERR_STATE, "ls_cache_snapshot: layer has no cache");
  DeviceGuard guard(L->device);
  return ls::cache_snapshot(L->cache, L->F, d_resident_mask, (cudaStream_t)stream, g_err, g_launches);
}

int32_t ls_cache_wait(ls_layer* L, void* stream) {
  if (!L) return fail(LS_ERR_INVALID, "ls_cache_wait: NULL layer");
  if (L->cache_rows == 0) return fail(LS_ERR_STATE, "ls_cache_wait: layer has no cache");
  DeviceGuard guard(L->device);
  return cache_rc(ls::cache_wait(L->cache, L->status, (cudaStream_t)stream, g_err, g_launches));
}

int32_t ls_cache_stats(ls_layer* L, ls_cache_stats_t* out) {
  if (!L || !out) return fail(LS_ERR_INVALID, "ls_cache_stats: NULL argument");
  if (L->cache_rows == 0) return fail(LS_ERR_STATE, "ls_cache_stats: layer has no cache");
  DeviceGuard guard(L->device);
  long long v[8];
  LS_TRY(cache_rc(ls::cache_stats(L->cache, v, g_err)));
  out->hits = v[0]; out->misses = v[1]; out->evictions = v[2]; out->resident = v[3]; out->h2d_bytes = v[4]; out->h2d_copies = v[5];
  return LS_OK;
}

}  // extern "C"
