// Host side and C ABI of the B200 (sm_100a) Deep Gradient Compression library.
// The kernels are in dgc_kernels.cuh; this file builds the launch plan (arena
// layout, parts, sampling ranks, candidate capacities), owns the device
// memory of a worker state and enqueues the kernels on the caller's stream.

#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "dgc.h"
#include "dgc_kernels.cuh"

using namespace dgc;

namespace {

std::atomic<uint64_t> g_launches{0};
constexpr int kClusterLaunchMinParts = 16;   // k_select_cluster when a tensor has this many parts

// ------------------------------------------------------------------ host side
int64_t topk_count(int64_t n, double sparsity) {
  const long long q = std::llround((1.0 - sparsity) * 1e9);
  long long k = ((long long)n * q + 999999999LL) / 1000000000LL;
  if (k < 1) k = 1;
  if (k > n) k = n;
  return k;
}

// Paper-literal mode (Sec. 5): elements drawn from a tensor of n, ceil(ratio * n) in integer
// arithmetic (parts per 1e9), at least 1, at most n.
int64_t sample_count(int64_t n, double ratio) {
  const long long q = std::llround(ratio * 1e9);
  long long S = ((long long)n * q + 999999999LL) / 1000000000LL;
  if (S < 1) S = 1;
  if (S > n) S = n;
  return S;
}

// Smallest r with P(Poisson(lambda) >= r) < eps.
int poisson_rank(double lambda, double eps) {
  if (lambda > 400.0) return (int)std::ceil(lambda + 6.2 * std::sqrt(lambda) + 5.0);
  double term = std::exp(-lambda), cdf = term;
  int r = 0;   // cdf = P(X <= r)
  while (1.0 - cdf >= eps && r < 100000) {
    ++r;
    term *= lambda / r;
    cdf += term;
  }
  return r + 1;
}

}  // namespace

struct dgc_state {
  dgc_config cfg{};
  std::vector<int64_t> numel;
  int device = 0;
  int sm_count = 0;
  int64_t arena_len = 0;
  double sparsity = 0.0;
  int64_t iterations = 0;
  // host plan
  std::vector<TensorMeta> tm;
  std::vector<PartMeta> pm;
  std::vector<int32_t> seg_part;
  std::vector<SampleBlock> sample_blocks;
  int64_t sample_keys_total = 0;
  std::vector<int32_t> big_parts, big_tensors;   // multi-block selection path
  int64_t max_nnz = 0;
  int64_t cand_total = 0;
  int64_t max_tensor_expect = 0;   // largest expected candidate count of one tensor
  int max_inblock_parts = 0;       // most parts of a tensor that k_select handles
  // device
  std::vector<void*> allocs;
  char* d_tables = nullptr;       // all plan tables in one allocation
  size_t d_tables_bytes = 0;
  int32_t* d_cand_idx = nullptr;
  float* d_cand_val = nullptr;
  int64_t cand_alloc = 0;
  uint32_t* d_sent_bits = nullptr;
  float* d_stage_g = nullptr;     // dgc_compress_host staging
  int32_t* d_stage_idx = nullptr;
  float* d_stage_val = nullptr;
  int64_t stage_nnz = 0;
  Plan plan{};
  // optional timing of the streaming kernel (dgc_profile_enable)
  std::vector<cudaEvent_t> prof_ev;   // 6 events per recorded call (stage boundaries)
  int prof_cap = 0, prof_n = 0;
  int norm_grid = 0;
  int select_smem_keys = 0;
  unsigned long long* d_timeline = nullptr;
  bool alive = false;
  bool broken = false;   // a sparsity change failed half-way: the plan on the device is not usable
};

namespace {

#define DGC_CUDA(call)                         \
  do {                                         \
    cudaError_t e__ = (call);                  \
    if (e__ != cudaSuccess) {                  \
      (void)cudaGetLastError();                \
      return e__ == cudaErrorMemoryAllocation ? DGC_ENOMEM : DGC_ECUDA; \
    }                                          \
  } while (0)

// Makes `dev` the current device and puts the caller's device back on scope exit.
struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { prev = -1; (void)cudaGetLastError(); }
    if (prev != dev) ok = cudaSetDevice(dev) == cudaSuccess;
    if (!ok) (void)cudaGetLastError();
  }
  ~DeviceGuard() { if (prev >= 0) (void)cudaSetDevice(prev); }
  DeviceGuard(const DeviceGuard&) = delete;
  DeviceGuard& operator=(const DeviceGuard&) = delete;
};

int32_t dev_alloc(dgc_state* st, void** out, size_t bytes) {
  void* ptr = nullptr;
  DGC_CUDA(cudaMalloc(&ptr, bytes ? bytes : 16));
  st->allocs.push_back(ptr);
  *out = ptr;
  return DGC_OK;
}

void dev_free(dgc_state* st, void* ptr) {
  if (!ptr) return;
  cudaFree(ptr);
  st->allocs.erase(std::remove(st->allocs.begin(), st->allocs.end(), ptr), st->allocs.end());
}

// Everything that depends on the sparsity: k, output offsets, sampling plan,
// candidate capacities.  Segments and parts depend only on the shapes.
// Scattered zeroing of u and v at the sent entries costs a sector read and write per touched
// 32-byte sector and array; recording one bit per element and zeroing in the next call's
// streaming pass costs 0.25 B/element flat.  The bitmap wins when more than about one entry
// in 512 is sent.
int defer_mask_for(double sparsity) { return (1.0 - sparsity) > 1.0 / 512.0 ? 1 : 0; }
// Emission from v' itself (k_emit_dense) instead of from the candidate lists: from this share
// of entries sent upwards, re-reading the part costs less than placing every candidate.
int dense_emit_for(double sparsity) { return (1.0 - sparsity) >= kDenseEmitFraction ? 1 : 0; }

// Keys one k_select block may hold in shared memory: two blocks per SM when there are more
// tensors than SMs, else one large block.
int select_key_cap(const dgc_state* st) {
  return st->cfg.num_tensors > st->sm_count ? 16384 : kSelectMaxSmemKeys;
}

void build_host_plan(dgc_state* st, double sparsity) {
  const int T = st->cfg.num_tensors;
  const double ratio = st->cfg.sample_ratio > 0.0 ? st->cfg.sample_ratio : 0.01;
  st->tm.assign(T, TensorMeta{});
  st->pm.clear();
  st->seg_part.clear();
  st->sample_blocks.clear();
  st->sample_keys_total = 0;
  st->big_parts.clear();
  st->big_tensors.clear();
  const int key_cap = select_key_cap(st);
  const bool literal = st->cfg.select_mode == 1;
  int64_t pos = 0, out = 0, cbase = 0;
  st->max_tensor_expect = 0;
  st->max_inblock_parts = 0;
  for (int j = 0; j < T; ++j) {
    const int64_t n = st->numel[j];
    const int64_t k = topk_count(n, sparsity);
    TensorMeta& t = st->tm[j];
    t.off = (int32_t)pos;
    t.end = (int32_t)(pos + n);
    t.k = (int32_t)k;
    t.out_off = (int32_t)out;
    out += literal ? std::min<int64_t>(n, 2 * k) : k;   // literal: capacity, the count varies
    const int64_t nseg = (n + kSeg - 1) / kSeg;
    const int64_t nparts = (nseg + kPartSegs - 1) / kPartSegs;
    // sampling plan
    bool sampled = literal || n > kSmallN;
    int groups = 0, rank = 0;
    int64_t samples = 0;
    double cap_total = (double)n;
    double expect_keys = (double)n;      // keys the select kernel should hold in shared memory
    if (literal) {
      // Sec. 5 as stated: ceil(ratio n) uniform draws from every tensor; thr = the sample's
      // k_s-th largest key, k_s = ceil(S (1 - s)); about k entries pass, at most 2k are sent,
      // anything beyond overflows into the exact path
      samples = sample_count(n, ratio);
      groups = (int)((samples + 3) / 4);
      rank = (int)topk_count(samples, sparsity);
      cap_total = std::min((double)n, 2.0 * (double)k + 1024.0);
      expect_keys = cap_total;
    } else if (sampled) {
      const int64_t Q = n / 4;
      int64_t G = (int64_t)std::ceil(ratio * (double)n / 4.0);
      // a sample that holds about 1024 of the entries to send pins the proposal to +-20 %;
      // at low sparsity that needs far fewer than ratio * n elements.  Where candidates are
      // cheap (few entries sent) a smaller sample with a wider margin is the better trade:
      // its rank stays within what the sampling kernel's pre-filter handles (one key per thread)
      const double sent = std::max(1.0 - sparsity, 1e-9);
      const double want = sent >= 1.0 / 32.0 ? 1024.0 : sent >= 1.0 / 128.0 ? 256.0 : 128.0;
      const int64_t enough = (int64_t)std::ceil(want / sent / 4.0);
      G = std::min<int64_t>(G, enough);
      G = std::max<int64_t>(G, 64);
      G = std::min<int64_t>(G, std::min<int64_t>(Q, kMaxSampleGroups));
      const double S = 4.0 * (double)G;
      const double lambda = S * (double)k / (double)n;
      rank = poisson_rank(lambda, 1e-9) + 2;
      if (st->cfg.debug_sample_rank > 0) rank = st->cfg.debug_sample_rank;
      if (rank >= S / 2) {
        sampled = false;
      } else {
        groups = (int)G;
        const double expect = (double)n * rank / S;
        cap_total = std::min((double)n, expect * (1.0 + 8.0 / std::sqrt((double)rank)) + 1024.0);
        expect_keys = std::min((double)n, expect * (1.0 + 4.0 / std::sqrt((double)rank)) + 256.0);
      }
    }
    t.rank = sampled ? rank : 0;
    t.groups = sampled ? groups : 0;
    t.samples = (int32_t)samples;
    if (sampled) {
      t.key_base = (int32_t)st->sample_keys_total;
      t.chunks = (groups + kSampleThreads - 1) / kSampleThreads;
      // keys a sampling block keeps for the merge: all `rank` where the sample's key must be
      // exact (paper-literal mode); otherwise a block's expected share of the tensor's `rank`
      // largest plus a wide margin (the proposal only has to be safe, see k_sample_threshold)
      t.rank_local = rank;
      if (!literal && t.chunks > 1) {
        const double mu = (double)rank / (double)t.chunks;
        t.rank_local = std::min(rank, (int)std::ceil(mu + 4.0 * std::sqrt(mu) + 4.0));
      }
      st->sample_keys_total += 4 * (int64_t)groups;
      for (int c = 0; c < t.chunks; ++c) {
        SampleBlock sb{};
        sb.tensor = j;
        sb.chunk = c;
        st->sample_blocks.push_back(sb);
      }
    }
    t.part_first = (int32_t)st->pm.size();
    t.part_num = (int32_t)nparts;
    // too many candidates (or parts) for one block: the multi-block selection path
    const bool big = expect_keys > (double)key_cap || nparts > kSelectMaxParts;
    t.big = big ? 1 : 0;
    t.big_slot = big ? (int32_t)st->big_tensors.size() : -1;
    if (big) st->big_tensors.push_back(j);
    for (int64_t q = 0; q < nparts; ++q) {
      const int64_t seg0 = pos / kSeg + q * kPartSegs;
      const int64_t ns = std::min<int64_t>(kPartSegs, nseg - q * kPartSegs);
      const int64_t pend = std::min<int64_t>(pos + n, (seg0 + ns) * kSeg);
      const int64_t elems = pend - seg0 * kSeg;
      int64_t cap = elems;
      if (sampled) {
        const int64_t share = (int64_t)std::ceil(cap_total / (double)nparts);
        cap = std::min<int64_t>(elems, std::max<int64_t>(4 * share, 8192));
        // paper-literal: a part may only overflow when more than 2k entries passed in all
        if (literal) cap = std::min<int64_t>(elems, std::max<int64_t>(cap, 2 * k + 1));
      }
      PartMeta m{};
      m.tensor = j;
      m.end = (int32_t)pend;
      m.seg0 = (int32_t)seg0;
      m.nseg = (int32_t)ns;
      m.cbase = (int32_t)cbase;
      m.cap = (int32_t)cap;
      m.first = q == 0 ? 1 : 0;
      m.big_slot = big ? (int32_t)st->big_parts.size() : -1;
      if (big) st->big_parts.push_back((int32_t)st->pm.size());
      st->pm.push_back(m);
      cbase += cap;
      for (int64_t s = 0; s < ns; ++s) st->seg_part.push_back((int32_t)(st->pm.size() - 1));
    }
    if (!big) st->max_tensor_expect = std::max<int64_t>(st->max_tensor_expect, (int64_t)expect_keys);
    if (!big) st->max_inblock_parts = std::max<int>(st->max_inblock_parts, (int)nparts);
    pos += nseg * kSeg;
  }
  // sampling blocks of the tensors with the most blocks first: their last block, which selects
  // among all of them, ends the kernel (a tensor's blocks stay together and in chunk order)
  std::stable_sort(st->sample_blocks.begin(), st->sample_blocks.end(),
                   [&](const SampleBlock& a, const SampleBlock& b) {
                     return st->tm[a.tensor].chunks > st->tm[b.tensor].chunks;
                   });
  for (SampleBlock& sb : st->sample_blocks) sb.t = st->tm[sb.tensor];   // (complete by now)
  st->arena_len = pos;
  st->max_nnz = out;
  st->cand_total = cbase;
  st->sparsity = sparsity;
}

int32_t upload_plan(dgc_state* st, bool first) {
  const size_t T = st->cfg.num_tensors, P = st->pm.size(), S = st->seg_part.size();
  const size_t NS = st->sample_blocks.size();
  // one block: [TensorMeta x T][PartMeta x P][PartSel x P][p_count P][p_thr P][t_kth T]
  //            [t_cand T][seg_part S][sampled NS], every array 16-byte aligned
  auto up16 = [](size_t x) { return (x + 15) & ~(size_t)15; };
  size_t o = 0;
  const size_t o_tm = o; o = up16(o + T * sizeof(TensorMeta));
  const size_t o_pm = o; o = up16(o + P * sizeof(PartMeta));
  const size_t o_psel = o; o = up16(o + P * sizeof(PartSel));
  const size_t o_pcount = o; o = up16(o + P * 4);
  const size_t o_pthr = o; o = up16(o + P * 4);
  const size_t o_peq = o; o = up16(o + P * 4);
  const size_t o_ptie = o; o = up16(o + P * 4);
  const size_t o_kth = o; o = up16(o + T * 4);
  const size_t o_cand = o; o = up16(o + T * 4);
  const size_t o_nnz = o; o = up16(o + T * 4);
  const size_t o_seg = o; o = up16(o + S * 4);
  const size_t o_samp = o; o = up16(o + NS * sizeof(SampleBlock));
  const size_t o_skeys = o; o = up16(o + (size_t)st->sample_keys_total * 4);
  const size_t o_sall = o; o = up16(o + (size_t)st->sample_keys_total * 4);
  const size_t o_stick = o; o = up16(o + T * 4);
  const size_t o_scnt = o; o = up16(o + NS * 4);
  const size_t NBP = st->big_parts.size(), NBT = st->big_tensors.size();
  const size_t o_bparts = o; o = up16(o + NBP * 4);
  const size_t o_btens = o; o = up16(o + NBT * 4);
  const size_t o_bhist = o; o = up16(o + NBT * 3 * kBigBins * 4);
  const size_t o_bstate = o; o = up16(o + NBT * kBigStateWords * 4);
  const size_t o_babove = o; o = up16(o + NBP * 4);
  const size_t o_blast = o; o = up16(o + NBP * kBigLastStride * 4);
  const bool per_tensor_clip = st->cfg.clip_scope == 1 && st->cfg.clip_threshold > 0.0f;
  const size_t o_segsq = o; o = up16(o + (per_tensor_clip ? S * 8 : 0));
  const size_t o_tnorm = o; o = up16(o + T * 8);
  const size_t o_tcoef = o; o = up16(o + T * 4);
  const size_t bytes = o + 16;
  if (first || bytes > st->d_tables_bytes) {
    if (st->d_tables) dev_free(st, st->d_tables);
    void* ptr = nullptr;
    int32_t rc = dev_alloc(st, &ptr, bytes);
    if (rc != DGC_OK) return rc;
    st->d_tables = (char*)ptr;
    st->d_tables_bytes = bytes;
  }
  std::vector<char> h(bytes, 0);     // p_count, p_thr (0 = every entry is a candidate), psel: zero
  std::memcpy(h.data() + o_tm, st->tm.data(), T * sizeof(TensorMeta));
  std::memcpy(h.data() + o_pm, st->pm.data(), P * sizeof(PartMeta));
  std::memcpy(h.data() + o_seg, st->seg_part.data(), S * 4);
  if (NS) std::memcpy(h.data() + o_samp, st->sample_blocks.data(), NS * sizeof(SampleBlock));
  if (NBP) std::memcpy(h.data() + o_bparts, st->big_parts.data(), NBP * 4);
  if (NBT) std::memcpy(h.data() + o_btens, st->big_tensors.data(), NBT * 4);
  DGC_CUDA(cudaMemcpy(st->d_tables, h.data(), bytes, cudaMemcpyHostToDevice));
  char* d = st->d_tables;
  Plan& p = st->plan;
  p.tm = (const TensorMeta*)(d + o_tm);
  p.pm = (const PartMeta*)(d + o_pm);
  p.psel = (PartSel*)(d + o_psel);
  p.p_count = (int32_t*)(d + o_pcount);
  p.p_thr = (uint32_t*)(d + o_pthr);
  p.p_eq = (int32_t*)(d + o_peq);
  p.p_tie = (uint32_t*)(d + o_ptie);
  p.t_kth = (uint32_t*)(d + o_kth);
  p.t_cand = (int32_t*)(d + o_cand);
  p.t_nnz = (int32_t*)(d + o_nnz);
  p.literal = st->cfg.select_mode == 1 ? 1 : 0;
  p.seg_part = (const int32_t*)(d + o_seg);
  p.sample_blocks = (const SampleBlock*)(d + o_samp);
  p.sample_keys = (uint32_t*)(d + o_skeys);
  p.sample_all = (uint32_t*)(d + o_sall);
  p.sample_ticket = (int32_t*)(d + o_stick);
  p.sample_cnt = (int32_t*)(d + o_scnt);
  p.big_parts = (const int32_t*)(d + o_bparts);
  p.big_tensors = (const int32_t*)(d + o_btens);
  p.big_hist = (int32_t*)(d + o_bhist);
  p.big_state = (int32_t*)(d + o_bstate);
  p.big_above = (int32_t*)(d + o_babove);
  p.big_last = (int32_t*)(d + o_blast);
  p.clip_scope = per_tensor_clip ? 1 : 0;
  p.seg_sumsq = (double*)(d + o_segsq);
  p.t_norm = (double*)(d + o_tnorm);
  p.t_coef = (float*)(d + o_tcoef);
  p.num_big_parts = (int32_t)NBP; p.num_big_tensors = (int32_t)NBT;
  p.num_tensors = (int32_t)T; p.num_parts = (int32_t)P; p.num_segs = (int32_t)S;
  // candidate lists
  if (st->cand_total > st->cand_alloc) {
    if (st->d_cand_idx) dev_free(st, st->d_cand_idx);
    if (st->d_cand_val) dev_free(st, st->d_cand_val);
    st->d_cand_idx = nullptr; st->d_cand_val = nullptr; st->cand_alloc = 0;
    void* a = nullptr; void* b = nullptr;
    int32_t rc = dev_alloc(st, &a, (size_t)st->cand_total * 4);
    if (rc != DGC_OK) return rc;
    rc = dev_alloc(st, &b, (size_t)st->cand_total * 4);
    if (rc != DGC_OK) return rc;
    st->d_cand_idx = (int32_t*)a; st->d_cand_val = (float*)b; st->cand_alloc = st->cand_total;
  }
  p.cand_idx = st->d_cand_idx; p.cand_val = st->d_cand_val;
  // shared memory of the select kernel
  int keys = (int)std::min<int64_t>(st->max_tensor_expect, select_key_cap(st));
  keys = std::max(keys, 1024);
  st->select_smem_keys = keys;
  // (the attribute is per function, not per state: always the largest any state may ask for)
  DGC_CUDA(cudaFuncSetAttribute(k_select<kSelectThreads>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (kSelectMaxSmemKeys + kHistWords(kSelectThreads)) * 4));
  DGC_CUDA(cudaFuncSetAttribute(k_select<kSelectBatchThreads>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (kSelectMaxSmemKeys + kHistWords(kSelectBatchThreads)) * 4));
  DGC_CUDA(cudaFuncSetAttribute(k_select_cluster<kClusterThreads>,
                                cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (kSelectMaxSmemKeys + kHistWords(kClusterThreads)) * 4));
  return DGC_OK;
}

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

// Launch with the programmatic-dependent-launch attribute (see pdl_enter in the kernels).
template <class... KArgs, class... Args>
inline void launch(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                   Args... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  (void)cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);   // error: check_launch()
}

// The same with a thread-block cluster of `cluster` blocks along x.
template <class... KArgs, class... Args>
inline void launch_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                           cudaStream_t s, unsigned cluster, Args... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = cluster;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  (void)cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);   // error: check_launch()
}

int32_t check_launch() {
  g_launches.fetch_add(1, std::memory_order_relaxed);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? DGC_OK : DGC_ECUDA;
}

int32_t flush_pending_mask(dgc_state* st, cudaStream_t s) {
  if (!st->plan.defer_mask) return DGC_OK;
  const long long words = st->arena_len / 32;
  launch(k_apply_pending_mask, 1184, 256, 0, s, st->plan, words);
  return check_launch();
}

}  // namespace

// ====================================================================== C ABI
extern "C" {

const char* dgc_error_string(int32_t code) {
  switch (code) {
    case DGC_OK: return "ok";
    case DGC_EINVAL: return "invalid argument";
    case DGC_ENOMEM: return "out of memory";
    case DGC_ECAPACITY: return "output capacity smaller than dgc_max_nnz";
    case DGC_ECUDA: return "CUDA runtime error";
    case DGC_ESTATE: return "invalid state handle";
    default: return "unknown error";
  }
}

uint64_t dgc_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int32_t dgc_warmup_sparsity(int32_t stage, double* sparsity_out) {
  static const double kStages[5] = {0.75, 0.9375, 0.984375, 0.996, 0.999};
  if (!sparsity_out || stage < 0 || stage > 4) return DGC_EINVAL;
  *sparsity_out = kStages[stage];
  return DGC_OK;
}

int32_t dgc_state_create(const dgc_config* cfg, dgc_state** out) {
  if (!cfg || !out) return DGC_EINVAL;
  *out = nullptr;
  if (cfg->num_tensors < 1 || !cfg->tensor_numel || cfg->num_workers < 1) return DGC_EINVAL;
  if (!(cfg->sparsity >= 0.0 && cfg->sparsity < 1.0)) return DGC_EINVAL;
  if (cfg->select_mode != 0 && cfg->select_mode != 1) return DGC_EINVAL;
  if (cfg->clip_scope != 0 && cfg->clip_scope != 1) return DGC_EINVAL;
  if (!(cfg->sample_ratio >= 0.0 && cfg->sample_ratio <= 0.5)) return DGC_EINVAL;
  if (!(cfg->momentum == cfg->momentum)) return DGC_EINVAL;
  int64_t padded = 0;
  for (int j = 0; j < cfg->num_tensors; ++j) {
    const int64_t n = cfg->tensor_numel[j];
    if (n < 1 || n >= (int64_t)1 << 31) return DGC_EINVAL;
    padded += (n + kSeg - 1) / kSeg * kSeg;
    if (padded >= (int64_t)1 << 31) return DGC_EINVAL;
  }
  int ndev = 0;
  DGC_CUDA(cudaGetDeviceCount(&ndev));
  if (cfg->device < 0 || cfg->device >= ndev) return DGC_EINVAL;
  DeviceGuard guard(cfg->device);       // the caller's current device is put back on return
  if (!guard.ok) return DGC_ECUDA;
  dgc_state* st = new (std::nothrow) dgc_state();
  if (!st) return DGC_ENOMEM;
  st->cfg = *cfg;
  st->numel.assign(cfg->tensor_numel, cfg->tensor_numel + cfg->num_tensors);
  st->cfg.tensor_numel = nullptr;
  st->device = cfg->device;
  st->alive = true;
  cudaDeviceProp prop{};
  if (cudaGetDeviceProperties(&prop, cfg->device) != cudaSuccess) { delete st; return DGC_ECUDA; }
  st->sm_count = prop.multiProcessorCount;
  build_host_plan(st, cfg->sparsity);
  int32_t rc = upload_plan(st, true);
  auto fail = [&](int32_t code) { dgc_state_destroy(st); return code; };
  if (rc != DGC_OK) return fail(rc);
  void* ptr = nullptr;
  if ((rc = dev_alloc(st, &ptr, (size_t)st->arena_len * 4)) != DGC_OK) return fail(rc);
  st->plan.u = (float*)ptr;
  if ((rc = dev_alloc(st, &ptr, (size_t)st->arena_len * 4)) != DGC_OK) return fail(rc);
  st->plan.v = (float*)ptr;
  if ((rc = dev_alloc(st, &ptr, (size_t)st->arena_len / 8)) != DGC_OK) return fail(rc);
  st->d_sent_bits = (uint32_t*)ptr;
  st->plan.sent_bits = st->d_sent_bits;
  if (cudaMemset(ptr, 0, (size_t)st->arena_len / 8) != cudaSuccess) return fail(DGC_ECUDA);
  st->plan.defer_mask = defer_mask_for(st->sparsity);
  st->plan.dense_emit = dense_emit_for(st->sparsity);
  // scalars: partials[kMaxNormGrid] doubles, norm, diag[8] long long, coef, ticket, iter
  const size_t scal_bytes = (kMaxNormGrid + 1) * 8 + 8 * 8 + 16 + 8;
  if ((rc = dev_alloc(st, &ptr, scal_bytes)) != DGC_OK) return fail(rc);
  char* sc = (char*)ptr;
  st->plan.partials = (double*)sc;
  st->plan.norm = (double*)(sc + kMaxNormGrid * 8);
  st->plan.diag = (long long*)(sc + (kMaxNormGrid + 1) * 8);
  st->plan.coef = (float*)(sc + (kMaxNormGrid + 1) * 8 + 64);
  st->plan.ticket = (unsigned int*)(sc + (kMaxNormGrid + 1) * 8 + 64 + 8);
  st->plan.iter = (long long*)(sc + (kMaxNormGrid + 1) * 8 + 64 + 16);
  if (cudaMemset(st->plan.u, 0, (size_t)st->arena_len * 4) != cudaSuccess) return fail(DGC_ECUDA);
  if (cudaMemset(st->plan.v, 0, (size_t)st->arena_len * 4) != cudaSuccess) return fail(DGC_ECUDA);
  if (cudaMemset(sc, 0, scal_bytes) != cudaSuccess) return fail(DGC_ECUDA);
  const float one = 1.0f;
  if (cudaMemcpy(st->plan.coef, &one, 4, cudaMemcpyHostToDevice) != cudaSuccess) return fail(DGC_ECUDA);
  // launch geometry
  st->norm_grid = std::min(kMaxNormGrid, st->sm_count * 8);
  if (cudaFuncSetAttribute(k_emit_mask, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kEmitSmemBytes) != cudaSuccess) return fail(DGC_ECUDA);
  if (cudaDeviceSynchronize() != cudaSuccess) return fail(DGC_ECUDA);
  *out = st;
  return DGC_OK;
}

int32_t dgc_state_destroy(dgc_state* st) {
  if (!st || !st->alive) return DGC_ESTATE;
  DeviceGuard guard(st->device);
  cudaDeviceSynchronize();
  for (void* ptr : st->allocs) cudaFree(ptr);
  st->allocs.clear();
  for (cudaEvent_t e : st->prof_ev) cudaEventDestroy(e);
  st->prof_ev.clear();
  st->alive = false;
  delete st;
  return DGC_OK;
}

int32_t dgc_set_sparsity(dgc_state* st, double sparsity) {
  if (!st || !st->alive) return DGC_ESTATE;
  if (!(sparsity >= 0.0 && sparsity < 1.0)) return DGC_EINVAL;
  if (st->broken) return DGC_ESTATE;
  DeviceGuard guard(st->device);
  if (!guard.ok) return DGC_ECUDA;
  // the device is idle before the state is touched: the flush below runs on the default
  // stream, which does not order itself against non-blocking streams
  DGC_CUDA(cudaDeviceSynchronize());
  int32_t rc = flush_pending_mask(st, nullptr);   // entries sent by the last call, if deferred
  if (rc != DGC_OK) return rc;
  DGC_CUDA(cudaDeviceSynchronize());
  build_host_plan(st, sparsity);
  rc = upload_plan(st, false);
  st->plan.sent_bits = st->d_sent_bits;
  st->plan.defer_mask = defer_mask_for(sparsity);
  st->plan.dense_emit = dense_emit_for(sparsity);
  if (rc != DGC_OK) st->broken = true;            // host plan and device tables no longer agree
  return rc;
}

int64_t dgc_max_nnz(const dgc_state* st) {
  if (!st || !st->alive) return DGC_ESTATE;
  return st->max_nnz;
}

int32_t dgc_layout(const dgc_state* st, int64_t* arena_offset, int64_t* k, int64_t* out_offset,
                   int64_t* arena_len) {
  if (!st || !st->alive) return DGC_ESTATE;
  const int T = st->cfg.num_tensors;
  for (int j = 0; j < T; ++j) {
    if (arena_offset) arena_offset[j] = st->tm[j].off;
    if (k) k[j] = st->tm[j].k;
    if (out_offset) out_offset[j] = st->tm[j].out_off;
  }
  if (out_offset) out_offset[T] = st->max_nnz;
  if (arena_len) *arena_len = st->arena_len;
  return DGC_OK;
}

// The three stages of one dgc_compress call, each enqueued on a stream of the caller's choice.
// Head: clipping norm and sampled threshold proposal.  Stream: the fused update + candidate
// emission pass.  Tail: exact selection, ordered emission, masking.
static int32_t enqueue_head(dgc_state* st, const float* grad_arena, cudaStream_t s,
                            cudaEvent_t after_norm) {
  const Plan& p = st->plan;
  const bool clip = st->cfg.clip_threshold > 0.0f;
  const bool nest = st->cfg.nesterov != 0;
  const float m = st->cfg.momentum;
  const uint64_t call_seed = st->cfg.seed * 0x9E3779B97F4A7C15ull;   // + the device's call count
  int32_t rc;
  if (clip) {
    const double thr_local =
        (double)st->cfg.clip_threshold / std::sqrt((double)st->cfg.num_workers);
    if (p.clip_scope) {
      const int grid = (p.num_segs + (kNormThreads / 32) - 1) / (kNormThreads / 32);
      launch(k_sumsq_segments, grid, kNormThreads, 0, s, p, grad_arena);
      if ((rc = check_launch()) != DGC_OK) return rc;
      launch(k_tensor_coef, p.num_tensors, kNormThreads, 0, s, p, thr_local);
    } else {
      launch(k_sumsq, st->norm_grid, kNormThreads, 0, s, p, grad_arena, thr_local, 1);
    }
    if ((rc = check_launch()) != DGC_OK) return rc;
  }
  if (after_norm) DGC_CUDA(cudaEventRecord(after_norm, s));
  if (!st->sample_blocks.empty()) {
    const int grid = (int)st->sample_blocks.size();
    const bool lit = st->cfg.select_mode == 1;
#define DGC_SAMPLE(C, N, L_) \
    launch(k_sample_threshold<C, N, L_>, grid, kSampleThreads, 0, s, p, grad_arena, m, call_seed)
    if (lit) {
      if (clip && nest) DGC_SAMPLE(true, true, true);
      else if (clip) DGC_SAMPLE(true, false, true);
      else if (nest) DGC_SAMPLE(false, true, true);
      else DGC_SAMPLE(false, false, true);
    } else {
      if (clip && nest) DGC_SAMPLE(true, true, false);
      else if (clip) DGC_SAMPLE(true, false, false);
      else if (nest) DGC_SAMPLE(false, true, false);
      else DGC_SAMPLE(false, false, false);
    }
#undef DGC_SAMPLE
    if ((rc = check_launch()) != DGC_OK) return rc;
  }
  return DGC_OK;
}

static int32_t enqueue_stream_pass(dgc_state* st, const float* grad_arena, cudaStream_t s) {
  const Plan& p = st->plan;
  const bool clip = st->cfg.clip_threshold > 0.0f;
  const bool nest = st->cfg.nesterov != 0;
  const float m = st->cfg.momentum;
  const int need = (p.num_segs + (kMainThreads / 32) - 1) / (kMainThreads / 32);
  if (clip && nest) launch(k_update_emit<true, true>, need, kMainThreads, 0, s, p, grad_arena, m);
  else if (clip) launch(k_update_emit<true, false>, need, kMainThreads, 0, s, p, grad_arena, m);
  else if (nest) launch(k_update_emit<false, true>, need, kMainThreads, 0, s, p, grad_arena, m);
  else launch(k_update_emit<false, false>, need, kMainThreads, 0, s, p, grad_arena, m);
  return check_launch();
}

static int32_t enqueue_tail(dgc_state* st, int32_t* out_idx, float* out_val, cudaStream_t s,
                            cudaEvent_t after_select = nullptr, bool batch = false) {
  const Plan& p = st->plan;
  int32_t rc;
  // 0: one block of 1024 threads per tensor; 1: one block of 512 (several workers' selections
  // run together); 2: a cluster of 8 x 512, which pays when some tensor has tens of parts (a
  // 15 M-element tensor: 34 -> 21 us) and costs where none has (its barriers and the smaller
  // blocks: the ResNet-50-shaped set 18.5 -> 25 us)
  int mode = st->max_inblock_parts >= kClusterLaunchMinParts ? 2 : batch ? 1 : 0;
  if (mode == 2)
    launch_cluster(k_select_cluster<kClusterThreads>, p.num_tensors * kClusterSize, kClusterThreads,
                   (size_t)(st->select_smem_keys + kHistWords(kClusterThreads)) * 4, s, kClusterSize,
                   p, st->select_smem_keys);
  else if (mode == 1)
    launch(k_select<kSelectBatchThreads>, p.num_tensors, kSelectBatchThreads,
           (size_t)(st->select_smem_keys + kHistWords(kSelectBatchThreads)) * 4, s, p,
           st->select_smem_keys);
  else
    launch(k_select<kSelectThreads>, p.num_tensors, kSelectThreads,
           (size_t)(st->select_smem_keys + kHistWords(kSelectThreads)) * 4, s, p,
           st->select_smem_keys);
  if ((rc = check_launch()) != DGC_OK) return rc;
  if (p.num_big_parts > 0) {
    launch(k_big_hist<0>, p.num_big_parts, kBigThreads, 0, s, p);
    if ((rc = check_launch()) != DGC_OK) return rc;
    launch(k_big_hist<1>, p.num_big_parts, kBigThreads, 0, s, p);
    if ((rc = check_launch()) != DGC_OK) return rc;
    launch(k_big_hist<2>, p.num_big_parts, kBigThreads, 0, s, p);
    if ((rc = check_launch()) != DGC_OK) return rc;
    launch(k_big_final, p.num_big_tensors, kSelectThreads, 0, s, p);
    if ((rc = check_launch()) != DGC_OK) return rc;
  }
  if (after_select) DGC_CUDA(cudaEventRecord(after_select, s));
  if (p.dense_emit) launch(k_emit_dense, p.num_parts, kEmitThreads, 0, s, p, out_idx, out_val);
  else launch(k_emit_mask, p.num_parts, kEmitThreads, kEmitSmemBytes, s, p, out_idx, out_val);
  return check_launch();
}

int32_t dgc_compress(dgc_state* st, const float* grad_arena, int32_t* out_idx, float* out_val,
                     int64_t capacity, void* stream) {
  if (!st || !st->alive || st->broken) return DGC_ESTATE;
  if (!grad_arena || !out_idx || !out_val) return DGC_EINVAL;
  if ((reinterpret_cast<uintptr_t>(grad_arena) & 15u) != 0) return DGC_EINVAL;
  if (capacity < st->max_nnz) return DGC_ECAPACITY;
  cudaStream_t s = as_stream(stream);
  int32_t rc;
  const bool prof = st->prof_n < st->prof_cap;
  cudaEvent_t* ev = prof ? &st->prof_ev[6 * st->prof_n] : nullptr;
  if (prof) DGC_CUDA(cudaEventRecord(ev[0], s));
  if ((rc = enqueue_head(st, grad_arena, s, prof ? ev[1] : nullptr)) != DGC_OK) return rc;
  if (prof) DGC_CUDA(cudaEventRecord(ev[2], s));
  if ((rc = enqueue_stream_pass(st, grad_arena, s)) != DGC_OK) return rc;
  if (prof) DGC_CUDA(cudaEventRecord(ev[3], s));
  if ((rc = enqueue_tail(st, out_idx, out_val, s, prof ? ev[4] : nullptr)) != DGC_OK) return rc;
  if (prof) {
    DGC_CUDA(cudaEventRecord(ev[5], s));
    st->prof_n += 1;
  }
  st->iterations += 1;
  return DGC_OK;
}

// Side streams and events of dgc_compress_batch, one set per device, created on first use.
namespace {
constexpr int kBatchStreams = 8;
struct BatchResources {
  cudaStream_t side[kBatchStreams] = {};
  cudaEvent_t fork = nullptr;
  cudaEvent_t join[kBatchStreams] = {};
  bool ready = false;
};
BatchResources g_batch[64];
std::mutex g_batch_mutex;
}  // namespace

// Shared by dgc_compress_batch (device buffers) and dgc_compress_host_batch (host buffers:
// `host` = true, every worker's gradient is copied into its state's staging first and its lists
// are copied out afterwards, on the worker's side stream, so that one worker's kernels run under
// the next worker's copy).
static int32_t batch_enqueue(int32_t num_states, dgc_state* const* states,
                             const float* const* grads, int32_t* const* out_idx,
                             float* const* out_val, cudaStream_t s, bool host) {
  const int dev = states[0]->device;
  if (dev < 0 || dev >= 64) return DGC_EINVAL;
  std::lock_guard<std::mutex> lock(g_batch_mutex);
  BatchResources& r = g_batch[dev];
  if (!r.ready) {
    for (int i = 0; i < kBatchStreams; ++i) {
      DGC_CUDA(cudaStreamCreateWithFlags(&r.side[i], cudaStreamNonBlocking));
      DGC_CUDA(cudaEventCreateWithFlags(&r.join[i], cudaEventDisableTiming));
    }
    DGC_CUDA(cudaEventCreateWithFlags(&r.fork, cudaEventDisableTiming));
    r.ready = true;
  }
  const int used = std::min<int>(num_states, kBatchStreams);
  int32_t rc;
  // Fork: the workers' calls go round robin over the side streams.  Measured on the
  // ResNet-50-shaped set with 8 workers: all streaming passes running side by side (0.78 ms
  // per step) beat running them one after the other with only the short kernels overlapped
  // (0.92 ms): a lone pass pays its launch gap and its ramp and drain, concurrent ones hide them.
  DGC_CUDA(cudaEventRecord(r.fork, s));
  for (int i = 0; i < used; ++i) DGC_CUDA(cudaStreamWaitEvent(r.side[i], r.fork, 0));
  rc = DGC_OK;
  for (int w = 0; w < num_states && rc == DGC_OK; ++w) {
    cudaStream_t q = r.side[w % kBatchStreams];
    dgc_state* st = states[w];
    const float* g = grads[w];
    int32_t* oi = out_idx[w];
    float* ov = out_val[w];
    if (host) {
      if (cudaMemcpyAsync(st->d_stage_g, grads[w], (size_t)st->arena_len * 4,
                          cudaMemcpyHostToDevice, q) != cudaSuccess) { rc = DGC_ECUDA; break; }
      g = st->d_stage_g;
      oi = st->d_stage_idx;
      ov = st->d_stage_val;
    }
    if ((rc = enqueue_head(st, g, q, nullptr)) != DGC_OK) break;
    if ((rc = enqueue_stream_pass(st, g, q)) != DGC_OK) break;
    if ((rc = enqueue_tail(st, oi, ov, q, nullptr, num_states >= 4)) != DGC_OK) break;
    st->iterations += 1;
    if (host) {
      if (cudaMemcpyAsync(out_idx[w], oi, (size_t)st->max_nnz * 4, cudaMemcpyDeviceToHost, q) !=
              cudaSuccess ||
          cudaMemcpyAsync(out_val[w], ov, (size_t)st->max_nnz * 4, cudaMemcpyDeviceToHost, q) !=
              cudaSuccess) { rc = DGC_ECUDA; break; }
    }
  }
  // Join, also after an enqueue error: the side streams were forked from the caller's stream
  // (inside a capture they belong to it) and what was enqueued on them must be ordered before
  // whatever the caller does next.
  for (int i = 0; i < used; ++i) {
    if (cudaEventRecord(r.join[i], r.side[i]) != cudaSuccess ||
        cudaStreamWaitEvent(s, r.join[i], 0) != cudaSuccess) {
      (void)cudaGetLastError();
      if (rc == DGC_OK) rc = DGC_ECUDA;
    }
  }
  if (rc != DGC_OK) (void)cudaGetLastError();
  return rc;
}

static int32_t batch_check(int32_t num_states, dgc_state* const* states, const void* const* a,
                           const void* const* b, const void* const* c, const int64_t* capacity,
                           bool aligned16) {
  if (num_states < 1 || !states || !a || !b || !c || !capacity) return DGC_EINVAL;
  for (int w = 0; w < num_states; ++w) {
    dgc_state* st = states[w];
    if (!st || !st->alive || st->broken) return DGC_ESTATE;
    if (st->device != states[0]->device) return DGC_EINVAL;
    if (!a[w] || !b[w] || !c[w]) return DGC_EINVAL;
    if (aligned16 && (reinterpret_cast<uintptr_t>(a[w]) & 15u) != 0) return DGC_EINVAL;
    if (capacity[w] < st->max_nnz) return DGC_ECAPACITY;
    for (int x = 0; x < w; ++x) if (states[x] == st) return DGC_EINVAL;
  }
  return DGC_OK;
}

int32_t dgc_compress_batch(int32_t num_states, dgc_state* const* states,
                           const float* const* grad_arenas, int32_t* const* out_idx,
                           float* const* out_val, const int64_t* capacity, void* stream) {
  const int32_t rc = batch_check(num_states, states, (const void* const*)grad_arenas,
                                 (const void* const*)out_idx, (const void* const*)out_val,
                                 capacity, true);
  if (rc != DGC_OK) return rc;
  return batch_enqueue(num_states, states, grad_arenas, out_idx, out_val, as_stream(stream), false);
}

// Device staging of the host-buffer entry points (gradient in, lists out), allocated on first use.
static int32_t ensure_staging(dgc_state* st) {
  int32_t rc;
  void* ptr = nullptr;
  if (!st->d_stage_g) {
    if ((rc = dev_alloc(st, &ptr, (size_t)st->arena_len * 4)) != DGC_OK) return rc;
    st->d_stage_g = (float*)ptr;
  }
  if (st->stage_nnz < st->max_nnz) {
    if (st->d_stage_idx) dev_free(st, st->d_stage_idx);
    if (st->d_stage_val) dev_free(st, st->d_stage_val);
    st->d_stage_idx = nullptr; st->d_stage_val = nullptr; st->stage_nnz = 0;
    if ((rc = dev_alloc(st, &ptr, (size_t)st->max_nnz * 4)) != DGC_OK) return rc;
    st->d_stage_idx = (int32_t*)ptr;
    if ((rc = dev_alloc(st, &ptr, (size_t)st->max_nnz * 4)) != DGC_OK) return rc;
    st->d_stage_val = (float*)ptr;
    st->stage_nnz = st->max_nnz;
  }
  return DGC_OK;
}

int32_t dgc_compress_host(dgc_state* st, const float* grad_host, int32_t* out_idx_host,
                          float* out_val_host, int64_t capacity, void* stream) {
  if (!st || !st->alive || st->broken) return DGC_ESTATE;
  if (!grad_host || !out_idx_host || !out_val_host) return DGC_EINVAL;
  if (capacity < st->max_nnz) return DGC_ECAPACITY;
  DeviceGuard guard(st->device);
  if (!guard.ok) return DGC_ECUDA;
  cudaStream_t s = as_stream(stream);
  int32_t rc;
  if ((rc = ensure_staging(st)) != DGC_OK) return rc;
  DGC_CUDA(cudaMemcpyAsync(st->d_stage_g, grad_host, (size_t)st->arena_len * 4,
                           cudaMemcpyHostToDevice, s));
  rc = dgc_compress(st, st->d_stage_g, st->d_stage_idx, st->d_stage_val, st->stage_nnz, stream);
  if (rc != DGC_OK) return rc;
  DGC_CUDA(cudaMemcpyAsync(out_idx_host, st->d_stage_idx, (size_t)st->max_nnz * 4,
                           cudaMemcpyDeviceToHost, s));
  DGC_CUDA(cudaMemcpyAsync(out_val_host, st->d_stage_val, (size_t)st->max_nnz * 4,
                           cudaMemcpyDeviceToHost, s));
  DGC_CUDA(cudaStreamSynchronize(s));
  return DGC_OK;
}

int32_t dgc_compress_host_batch(int32_t num_states, dgc_state* const* states,
                                const float* const* grads_host, int32_t* const* out_idx_host,
                                float* const* out_val_host, const int64_t* capacity,
                                void* stream) {
  int32_t rc = batch_check(num_states, states, (const void* const*)grads_host,
                           (const void* const*)out_idx_host, (const void* const*)out_val_host,
                           capacity, false);
  if (rc != DGC_OK) return rc;
  DeviceGuard guard(states[0]->device);
  if (!guard.ok) return DGC_ECUDA;
  for (int w = 0; w < num_states; ++w)
    if ((rc = ensure_staging(states[w])) != DGC_OK) return rc;
  cudaStream_t s = as_stream(stream);
  rc = batch_enqueue(num_states, states, grads_host, out_idx_host, out_val_host, s, true);
  const cudaError_t e = cudaStreamSynchronize(s);      // the lists are valid on return
  if (e != cudaSuccess) { (void)cudaGetLastError(); if (rc == DGC_OK) rc = DGC_ECUDA; }
  return rc;
}

}  // extern "C"

// Receive side.  The scratch of a decode call, caller-provided or built in, is
//   [num_workers x (tiles + 1) tile boundaries][num_workers x kDecodeBoundsBlocks reject counts]
static int64_t decode_scratch_words(int32_t num_workers, int64_t dense_len) {
  const int64_t tiles = (dense_len + kDecodeTile - 1) / kDecodeTile;
  return (int64_t)num_workers * (tiles + 1 + kDecodeBoundsBlocks);
}


// Argument checks and marshalling shared by the decode entry points, then the two launches.
// `out` is the dense gradient (MODE dense, dense + SGD) or the weights (MODE sparse SGD);
// `weights` only for dense + SGD.
template <int MODE>
static int32_t decode_enqueue(int32_t num_workers, const int32_t* const* idx_lists,
                              const float* const* val_lists, const int64_t* nnz, float* out,
                              float* weights, int64_t len, float lr, int32_t* scratch,
                              cudaStream_t s) {
  DecodeArgs a{};
  int64_t max_nnz = 0;
  for (int w = 0; w < num_workers; ++w) {
    if (nnz[w] < 0 || nnz[w] > len) return DGC_EINVAL;
    if (nnz[w] > 0 && (!idx_lists[w] || !val_lists[w])) return DGC_EINVAL;
    a.idx[w] = idx_lists[w];
    a.val[w] = val_lists[w];
    a.nnz[w] = (int32_t)nnz[w];
    max_nnz = std::max(max_nnz, nnz[w]);
  }
  a.num_workers = num_workers;
  a.num_tiles = (int32_t)((len + kDecodeTile - 1) / kDecodeTile);
  int32_t* rejected = scratch + (size_t)num_workers * (a.num_tiles + 1);
  int32_t rc;
  const int gx = (int)std::min<int64_t>((max_nnz + 1 + 255) / 256, kDecodeBoundsBlocks);
  launch(k_decode_bounds, dim3(gx, num_workers), 256, 0, s, a, scratch, rejected, (long long)len);
  if ((rc = check_launch()) != DGC_OK) return rc;
  launch(k_decode_tiles<MODE>, a.num_tiles, kDecodeThreads, 0, s, a, (const int32_t*)scratch, out,
         weights, (long long)len, lr);
  return check_launch();
}

static int32_t decode_check_common(int32_t num_workers, const int32_t* const* idx_lists,
                                   const float* const* val_lists, const int64_t* nnz,
                                   int64_t len) {
  if (num_workers < 1 || num_workers > DGC_MAX_DECODE_WORKERS) return DGC_EINVAL;
  if (!idx_lists || !val_lists || !nnz || len < 0 || len >= (int64_t)1 << 31) return DGC_EINVAL;
  return DGC_OK;
}

extern "C" {

int64_t dgc_decode_workspace_bytes(int32_t num_workers, int64_t dense_len) {
  if (num_workers < 1 || num_workers > DGC_MAX_DECODE_WORKERS || dense_len < 0) return DGC_EINVAL;
  return decode_scratch_words(num_workers, dense_len) * 4;
}

int32_t dgc_decode_accumulate(int32_t num_workers, const int32_t* const* idx_lists,
                              const float* const* val_lists, const int64_t* nnz, float* dense_out,
                              int64_t dense_len, void* workspace, int64_t workspace_bytes,
                              void* stream) {
  int32_t rc = decode_check_common(num_workers, idx_lists, val_lists, nnz, dense_len);
  if (rc != DGC_OK) return rc;
  if (dense_len == 0) return DGC_OK;
  if (!dense_out || !workspace) return DGC_EINVAL;
  if ((reinterpret_cast<uintptr_t>(dense_out) & 15u) != 0) return DGC_EINVAL;
  if (workspace_bytes < dgc_decode_workspace_bytes(num_workers, dense_len)) return DGC_ECAPACITY;
  return decode_enqueue<kDecodeDense>(num_workers, idx_lists, val_lists, nnz, dense_out, nullptr,
                                      dense_len, 0.0f, (int32_t*)workspace, as_stream(stream));
}

int32_t dgc_decode_apply_sgd(int32_t num_workers, const int32_t* const* idx_lists,
                             const float* const* val_lists, const int64_t* nnz, float* w,
                             int64_t len, float lr, void* workspace, int64_t workspace_bytes,
                             void* stream) {
  int32_t rc = decode_check_common(num_workers, idx_lists, val_lists, nnz, len);
  if (rc != DGC_OK) return rc;
  if (len == 0) return DGC_OK;
  if (!w || !workspace) return DGC_EINVAL;
  if (workspace_bytes < dgc_decode_workspace_bytes(num_workers, len)) return DGC_ECAPACITY;
  return decode_enqueue<kDecodeSparseSgd>(num_workers, idx_lists, val_lists, nnz, w, nullptr, len,
                                          lr, (int32_t*)workspace, as_stream(stream));
}

int32_t dgc_decode_accumulate_sgd(int32_t num_workers, const int32_t* const* idx_lists,
                                  const float* const* val_lists, const int64_t* nnz,
                                  float* dense_out, float* w, int64_t len, float lr,
                                  void* workspace, int64_t workspace_bytes, void* stream) {
  int32_t rc = decode_check_common(num_workers, idx_lists, val_lists, nnz, len);
  if (rc != DGC_OK) return rc;
  if (len == 0) return DGC_OK;
  if (!w || !dense_out || !workspace) return DGC_EINVAL;
  if (((reinterpret_cast<uintptr_t>(w) | reinterpret_cast<uintptr_t>(dense_out)) & 15u) != 0)
    return DGC_EINVAL;
  if (workspace_bytes < dgc_decode_workspace_bytes(num_workers, len)) return DGC_ECAPACITY;
  return decode_enqueue<kDecodeDenseSgd>(num_workers, idx_lists, val_lists, nnz, dense_out, w,
                                         len, lr, (int32_t*)workspace, as_stream(stream));
}

int64_t dgc_runlength_max_entries(int64_t nnz, int64_t dense_len) {
  if (nnz < 0 || dense_len < 0) return DGC_EINVAL;
  return nnz + dense_len / 65536 + 1;
}

int64_t dgc_runlength_workspace_bytes(int64_t entries) {
  if (entries < 0) return DGC_EINVAL;
  return ((entries + kRleBlock - 1) / kRleBlock + 1) * 8;
}

int32_t dgc_encode_runlength(const int32_t* idx, const float* val, int64_t nnz,
                             uint16_t* runs_out, float* values_out, int64_t capacity,
                             int64_t* count_out, void* workspace, int64_t workspace_bytes,
                             void* stream) {
  if (nnz < 0 || capacity < 0 || !count_out) return DGC_EINVAL;
  cudaStream_t s = as_stream(stream);
  int32_t rc;
  if (nnz == 0) {
    DGC_CUDA(cudaMemsetAsync(count_out, 0, 8, s));
    return DGC_OK;
  }
  if (!idx || !val || !runs_out || !values_out || !workspace) return DGC_EINVAL;
  if (workspace_bytes < dgc_runlength_workspace_bytes(nnz)) return DGC_ECAPACITY;
  if (capacity < nnz) return DGC_ECAPACITY;
  const int nblocks = (int)((nnz + kRleBlock - 1) / kRleBlock);
  unsigned long long* sums = (unsigned long long*)workspace;
  launch(k_rle_block_sums<true>, nblocks, kRleThreads, 0, s, idx, nullptr, nnz, sums);
  if ((rc = check_launch()) != DGC_OK) return rc;
  launch(k_rle_scan_sums, 1, 1024, 0, s, sums, nblocks, nnz, (long long*)count_out);
  if ((rc = check_launch()) != DGC_OK) return rc;
  launch(k_rle_write<true>, nblocks, kRleThreads, 0, s, idx, val, nullptr, nnz, sums, runs_out,
                                                    values_out, nullptr, capacity);
  return check_launch();
}

int32_t dgc_decode_runlength(const uint16_t* runs, const float* values, int64_t count,
                             int32_t* idx_out, float* val_out, int64_t* dense_len_out,
                             void* workspace, int64_t workspace_bytes, void* stream) {
  if (count < 0) return DGC_EINVAL;
  cudaStream_t s = as_stream(stream);
  int32_t rc;
  if (count == 0) {
    if (dense_len_out) DGC_CUDA(cudaMemsetAsync(dense_len_out, 0, 8, s));
    return DGC_OK;
  }
  if (!runs || !values || !idx_out || !val_out || !workspace || !dense_len_out) return DGC_EINVAL;
  if (workspace_bytes < dgc_runlength_workspace_bytes(count)) return DGC_ECAPACITY;
  const int nblocks = (int)((count + kRleBlock - 1) / kRleBlock);
  unsigned long long* sums = (unsigned long long*)workspace;
  launch(k_rle_block_sums<false>, nblocks, kRleThreads, 0, s, nullptr, runs, count, sums);
  if ((rc = check_launch()) != DGC_OK) return rc;
  launch(k_rle_scan_sums, 1, 1024, 0, s, sums, nblocks, 0, (long long*)dense_len_out);
  if ((rc = check_launch()) != DGC_OK) return rc;
  launch(k_rle_write<false>, nblocks, kRleThreads, 0, s, nullptr, values, runs, count, sums, nullptr,
                                                     val_out, idx_out, count);
  return check_launch();
}

int32_t dgc_apply_sgd(float* w, const float* dense_grad, int64_t len, float lr, void* stream) {
  if (len < 0) return DGC_EINVAL;
  if (len == 0) return DGC_OK;
  if (!w || !dense_grad) return DGC_EINVAL;
  if (((reinterpret_cast<uintptr_t>(w) | reinterpret_cast<uintptr_t>(dense_grad)) & 15u) != 0)
    return DGC_EINVAL;
  const int64_t n4 = std::max<int64_t>(len >> 2, 1);
  const int grid = (int)std::min<int64_t>((n4 + 255) / 256, 148 * 16);
  launch(k_sgd, grid, 256, 0, as_stream(stream), w, dense_grad, len, lr);
  return check_launch();
}

int32_t dgc_get_status(dgc_state* st, void* stream, dgc_status* out) {
  if (!st || !st->alive) return DGC_ESTATE;
  if (!out) return DGC_EINVAL;
  DGC_CUDA(cudaStreamSynchronize(as_stream(stream)));
  long long diag[8];
  double norm = 0.0;
  float coef = 1.0f;
  DGC_CUDA(cudaMemcpy(diag, st->plan.diag, sizeof diag, cudaMemcpyDeviceToHost));
  DGC_CUDA(cudaMemcpy(&norm, st->plan.norm, 8, cudaMemcpyDeviceToHost));
  DGC_CUDA(cudaMemcpy(&coef, st->plan.coef, 4, cudaMemcpyDeviceToHost));
  // the device's count is the truth: a captured call replayed n times counts n times
  long long done = 0;
  DGC_CUDA(cudaMemcpy(&done, st->plan.iter, 8, cudaMemcpyDeviceToHost));
  st->iterations = done;
  const int parity = (int)((st->iterations + 1) & 1);   // parity of the last call
  const bool clip = st->cfg.clip_threshold > 0.0f;
  if (clip && st->plan.clip_scope) {
    // per tensor: the norm of the whole set from the tensors' norms, the smallest coefficient
    const size_t T = st->cfg.num_tensors;
    std::vector<double> tn(T);
    std::vector<float> tc(T);
    DGC_CUDA(cudaMemcpy(tn.data(), st->plan.t_norm, T * 8, cudaMemcpyDeviceToHost));
    DGC_CUDA(cudaMemcpy(tc.data(), st->plan.t_coef, T * 4, cudaMemcpyDeviceToHost));
    double ss = 0.0;
    coef = 1.0f;
    for (size_t j = 0; j < T; ++j) {
      ss += tn[j] * tn[j];
      if (!(tc[j] >= coef)) coef = tc[j];              // (NaN propagates)
    }
    norm = done > 0 ? std::sqrt(ss) : 0.0;
    if (done == 0) coef = 1.0f;
  }
  out->grad_norm = clip ? norm : 0.0;
  out->clip_coef = clip ? coef : 1.0f;
  out->flags = (int32_t)(diag[parity * 4 + 0] & 0x1F);
  if (clip && !std::isfinite(norm)) out->flags |= DGC_FLAG_NONFINITE_NORM;
  out->iterations = st->iterations;
  out->full_select_last = diag[parity * 4 + 1];
  out->candidates_last = diag[parity * 4 + 2];
  return DGC_OK;
}

int32_t dgc_get_thresholds(dgc_state* st, void* stream, uint32_t* kth_key, int32_t* candidates) {
  if (!st || !st->alive) return DGC_ESTATE;
  DGC_CUDA(cudaStreamSynchronize(as_stream(stream)));
  const size_t T = st->cfg.num_tensors;
  if (kth_key) DGC_CUDA(cudaMemcpy(kth_key, st->plan.t_kth, T * 4, cudaMemcpyDeviceToHost));
  if (candidates) DGC_CUDA(cudaMemcpy(candidates, st->plan.t_cand, T * 4, cudaMemcpyDeviceToHost));
  return DGC_OK;
}

int32_t dgc_get_clip(dgc_state* st, void* stream, double* norms, float* coefs) {
  if (!st || !st->alive) return DGC_ESTATE;
  DGC_CUDA(cudaStreamSynchronize(as_stream(stream)));
  const size_t T = st->cfg.num_tensors;
  const bool clip = st->cfg.clip_threshold > 0.0f;
  if (clip && st->plan.clip_scope) {
    if (norms) DGC_CUDA(cudaMemcpy(norms, st->plan.t_norm, T * 8, cudaMemcpyDeviceToHost));
    if (coefs) DGC_CUDA(cudaMemcpy(coefs, st->plan.t_coef, T * 4, cudaMemcpyDeviceToHost));
    return DGC_OK;
  }
  double norm = 0.0;
  float coef = 1.0f;
  if (clip) {
    DGC_CUDA(cudaMemcpy(&norm, st->plan.norm, 8, cudaMemcpyDeviceToHost));
    DGC_CUDA(cudaMemcpy(&coef, st->plan.coef, 4, cudaMemcpyDeviceToHost));
  }
  for (size_t j = 0; j < T; ++j) {
    if (norms) norms[j] = norm;
    if (coefs) coefs[j] = coef;
  }
  return DGC_OK;
}

static int32_t timeline_reset(dgc_state* st) {
  unsigned long long init[8];
  for (int i = 0; i < 4; ++i) { init[2 * i] = ~0ull; init[2 * i + 1] = 0ull; }
  DGC_CUDA(cudaMemcpy(st->d_timeline, init, sizeof init, cudaMemcpyHostToDevice));
  return DGC_OK;
}

int32_t dgc_timeline_enable(dgc_state* st, int32_t on) {
  if (!st || !st->alive) return DGC_ESTATE;
  DeviceGuard guard(st->device);
  if (!guard.ok) return DGC_ECUDA;
  DGC_CUDA(cudaDeviceSynchronize());
  if (on && !st->d_timeline) {
    void* ptr = nullptr;
    const int32_t rc = dev_alloc(st, &ptr, 64);
    if (rc != DGC_OK) return rc;
    st->d_timeline = (unsigned long long*)ptr;
  }
  st->plan.timeline = on ? st->d_timeline : nullptr;
  return on ? timeline_reset(st) : DGC_OK;
}

int32_t dgc_timeline_read(dgc_state* st, void* stream, uint64_t* ns_out) {
  if (!st || !st->alive) return DGC_ESTATE;
  if (!ns_out) return DGC_EINVAL;
  if (!st->plan.timeline) return DGC_EINVAL;
  DGC_CUDA(cudaStreamSynchronize(as_stream(stream)));
  DGC_CUDA(cudaMemcpy(ns_out, st->d_timeline, 64, cudaMemcpyDeviceToHost));
  return timeline_reset(st);
}

int32_t dgc_profile_enable(dgc_state* st, int32_t max_calls) {
  if (!st || !st->alive) return DGC_ESTATE;
  if (max_calls < 0) return DGC_EINVAL;
  DeviceGuard guard(st->device);
  if (!guard.ok) return DGC_ECUDA;
  while ((int)st->prof_ev.size() < 6 * max_calls) {
    cudaEvent_t e;
    DGC_CUDA(cudaEventCreate(&e));
    st->prof_ev.push_back(e);
  }
  st->prof_cap = max_calls;
  st->prof_n = 0;
  return DGC_OK;
}

int32_t dgc_profile_read(dgc_state* st, float* ms_out, int32_t capacity, int32_t* count_out) {
  if (!st || !st->alive) return DGC_ESTATE;
  if (!count_out || (capacity > 0 && !ms_out)) return DGC_EINVAL;
  const int n = std::min<int>(st->prof_n, capacity);
  for (int i = 0; i < n; ++i) {
    DGC_CUDA(cudaEventSynchronize(st->prof_ev[6 * i + 5]));
    for (int k = 0; k < 5; ++k)
      DGC_CUDA(cudaEventElapsedTime(&ms_out[5 * i + k], st->prof_ev[6 * i + k],
                                    st->prof_ev[6 * i + k + 1]));
  }
  *count_out = n;
  return DGC_OK;
}

int32_t dgc_get_nnz(dgc_state* st, void* stream, int64_t* total_out, int64_t* per_tensor) {
  if (!st || !st->alive) return DGC_ESTATE;
  const size_t T = st->cfg.num_tensors;
  std::vector<int32_t> h(T);
  if (st->cfg.select_mode == 1) {
    DGC_CUDA(cudaStreamSynchronize(as_stream(stream)));
    // the device's count of completed calls decides (graph replays do not pass through the host)
    long long done = 0;
    DGC_CUDA(cudaMemcpy(&done, st->plan.iter, 8, cudaMemcpyDeviceToHost));
    st->iterations = done;
    if (done == 0) std::fill(h.begin(), h.end(), 0);
    else DGC_CUDA(cudaMemcpy(h.data(), st->plan.t_nnz, T * 4, cudaMemcpyDeviceToHost));
  } else {
    for (size_t j = 0; j < T; ++j) h[j] = st->tm[j].k;
  }
  int64_t total = 0;
  for (size_t j = 0; j < T; ++j) {
    if (per_tensor) per_tensor[j] = h[j];
    total += h[j];
  }
  if (total_out) *total_out = total;
  return DGC_OK;
}

int32_t dgc_state_read(dgc_state* st, float* u_host, float* v_host, void* stream) {
  if (!st || !st->alive) return DGC_ESTATE;
  cudaStream_t s = as_stream(stream);
  const int32_t frc = flush_pending_mask(st, s);
  if (frc != DGC_OK) return frc;
  const size_t bytes = (size_t)st->arena_len * 4;
  if (u_host) DGC_CUDA(cudaMemcpyAsync(u_host, st->plan.u, bytes, cudaMemcpyDeviceToHost, s));
  if (v_host) DGC_CUDA(cudaMemcpyAsync(v_host, st->plan.v, bytes, cudaMemcpyDeviceToHost, s));
  DGC_CUDA(cudaStreamSynchronize(s));
  return DGC_OK;
}

int32_t dgc_state_write(dgc_state* st, const float* u_host, const float* v_host, void* stream) {
  if (!st || !st->alive) return DGC_ESTATE;
  cudaStream_t s = as_stream(stream);
  const int32_t frc = flush_pending_mask(st, s);   // pending zeroing belongs to the old contents
  if (frc != DGC_OK) return frc;
  const size_t bytes = (size_t)st->arena_len * 4;
  if (u_host) DGC_CUDA(cudaMemcpyAsync(st->plan.u, u_host, bytes, cudaMemcpyHostToDevice, s));
  if (v_host) DGC_CUDA(cudaMemcpyAsync(st->plan.v, v_host, bytes, cudaMemcpyHostToDevice, s));
  DGC_CUDA(cudaStreamSynchronize(s));
  return DGC_OK;
}

int32_t dgc_state_set_iterations(dgc_state* st, int64_t iterations, void* stream) {
  if (!st || !st->alive) return DGC_ESTATE;
  if (iterations < 0) return DGC_EINVAL;
  cudaStream_t s = as_stream(stream);
  DGC_CUDA(cudaStreamSynchronize(s));
  const long long zeros[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  const long long it = iterations;
  DGC_CUDA(cudaMemcpy(st->plan.diag, zeros, sizeof zeros, cudaMemcpyHostToDevice));
  DGC_CUDA(cudaMemcpy(st->plan.iter, &it, 8, cudaMemcpyHostToDevice));
  st->iterations = iterations;
  return DGC_OK;
}

}  // extern "C"

// ====================================================================== allocation-free decode
// Scratch of dgc_decode_accumulate_static: the per-worker tile boundaries that the caller of
// dgc_decode_accumulate passes as `workspace`.  It lives in the library image, so every GPU
// that loads the library holds DGC_STATIC_DECODE_WORDS * 4 bytes of it until the process exits.
// In host code this name is only a stand-in for the symbol, not a device address: the address
// a kernel may use comes from cudaGetSymbolAddress, asked once per device (below).
static __device__ __align__(256) int32_t g_static_decode_bounds[DGC_STATIC_DECODE_WORDS];

namespace {
constexpr int kMaxDevices = 64;
std::atomic<int32_t*> g_static_bounds_ptr[kMaxDevices];   // device address per ordinal, 0 = not asked yet
}  // namespace

// Device address of the built-in scratch on the current device (looked up once per device).
static int32_t static_decode_scratch(int32_t** out) {
  int dev = -1;
  DGC_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return DGC_EINVAL;
  int32_t* ptr = g_static_bounds_ptr[dev].load(std::memory_order_acquire);
  if (!ptr) {
    void* sym = nullptr;
    DGC_CUDA(cudaGetSymbolAddress(&sym, g_static_decode_bounds));
    if (!sym) return DGC_ECUDA;
    ptr = static_cast<int32_t*>(sym);
    g_static_bounds_ptr[dev].store(ptr, std::memory_order_release);
  }
  *out = ptr;
  return DGC_OK;
}

extern "C" int32_t dgc_decode_accumulate_static(int32_t num_workers,
                                                 const int32_t* const* idx_lists,
                                                 const float* const* val_lists, const int64_t* nnz,
                                                 float* dense_out, int64_t dense_len, void* stream) {
  int32_t rc = decode_check_common(num_workers, idx_lists, val_lists, nnz, dense_len);
  if (rc != DGC_OK) return rc;
  if (dense_len == 0) return DGC_OK;
  if (!dense_out) return DGC_EINVAL;
  if ((reinterpret_cast<uintptr_t>(dense_out) & 15u) != 0) return DGC_EINVAL;
  // the fixed scratch bounds the problem: the boundary and reject words of all workers must fit
  if (decode_scratch_words(num_workers, dense_len) > (int64_t)DGC_STATIC_DECODE_WORDS)
    return DGC_ECAPACITY;
  // set-up, once per device, with that device current: the symbol's device address
  int32_t* scratch = nullptr;
  if ((rc = static_decode_scratch(&scratch)) != DGC_OK) return rc;
  // nothing needs clearing: k_decode_bounds writes every boundary word [0, tiles] and every
  // reject word of every worker before anything reads them, so the previous call's contents
  // are never seen
  return decode_enqueue<kDecodeDense>(num_workers, idx_lists, val_lists, nnz, dense_out, nullptr,
                                      dense_len, 0.0f, scratch, as_stream(stream));
}

extern "C" int32_t dgc_decode_rejected(int32_t num_workers, int64_t dense_len,
                                        const void* workspace, void* stream,
                                        int64_t* rejected_out) {
  if (num_workers < 1 || num_workers > DGC_MAX_DECODE_WORKERS || dense_len < 0 || !rejected_out)
    return DGC_EINVAL;
  *rejected_out = 0;
  if (dense_len == 0) return DGC_OK;
  const int32_t* scratch = static_cast<const int32_t*>(workspace);
  if (!scratch) {
    if (decode_scratch_words(num_workers, dense_len) > (int64_t)DGC_STATIC_DECODE_WORDS)
      return DGC_ECAPACITY;
    int32_t* ptr = nullptr;
    const int32_t rc = static_decode_scratch(&ptr);
    if (rc != DGC_OK) return rc;
    scratch = ptr;
  }
  const int64_t tiles = (dense_len + kDecodeTile - 1) / kDecodeTile;
  std::vector<int32_t> h((size_t)num_workers * kDecodeBoundsBlocks);
  DGC_CUDA(cudaStreamSynchronize(as_stream(stream)));
  DGC_CUDA(cudaMemcpy(h.data(), scratch + (size_t)num_workers * (tiles + 1), h.size() * 4,
                      cudaMemcpyDeviceToHost));
  int64_t total = 0;
  for (int32_t c : h) total += c;
  *rejected_out = total;
  return DGC_OK;
}
