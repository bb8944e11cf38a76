// B200 (sm_100a) kernels and C ABI of the Deep Gradient Compression hot path.
//
// One dgc_compress call = one iteration of Algorithm 4 (Appendix D) on one
// worker, as four stream-ordered launches over a padded fp32 arena:
//
//   k_sumsq            (only when clipping)  Sec. 3.2 / App. C: ||g||_2 in fp64, coef
//   k_sample_threshold Sec. 5: seeded sample of |v'| -> proposed threshold per tensor
//   k_update_emit      Eq. 5: u' = m u + g coef, v' = v + u', stored once; entries whose
//                      |v'| passes the proposal are compacted, in index order per
//                      512-element segment, into that part's candidate list
//   k_select           exact k-th largest |v'| among a tensor's candidates (radix
//                      select on the IEEE bit pattern), tie quota, per-part output bases
//   k_emit_mask        Alg. 4 "G~ <- V (.) Mask", Sec. 3.3 masking: ordered (index, value)
//                      pairs, then u = v = 0 at the sent entries
//
// The sample only proposes; if a proposal lets fewer than k_j or more than the
// list capacity through, that tensor is selected from the whole of v' instead
// (same result, slower).  All fp32 arithmetic uses explicit round-to-nearest
// intrinsics so that no FMA contraction can change a bit.
//
// Receive side: k_decode_bounds + k_decode_tiles (Alg. 4 aggregation line) and
// k_sgd (Alg. 4 update line).

#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <new>
#include <vector>

#include "dgc.h"

namespace {

// ------------------------------------------------------------------ constants
constexpr int kSeg = 512;              // elements per warp segment (4 x float4 per lane)
constexpr int kPartSegs = 512;         // segments per part (256 Ki elements)
constexpr int kSmallN = 8192;          // tensors up to this size are not sampled
constexpr int kMaxSampleGroups = 3072; // float4 groups sampled per tensor at most
constexpr int kSampleThreads = 512;
constexpr int kSelectThreads = 1024;
constexpr int kSelectMaxSmemKeys = 49152;
constexpr int kEmitThreads = kPartSegs;   // one thread per segment of the part
constexpr int kMaskStride = 17;           // words per segment in the winner bitmaps (16 + 1 pad)
constexpr int kEmitSmemBytes = 2 * kPartSegs * kMaskStride * 4;
constexpr int kMainThreads = 256;
constexpr int kNormThreads = 256;
constexpr int kMaxNormGrid = 2048;
constexpr int kDecodeTile = 4096;
constexpr int kDecodeThreads = 256;

std::atomic<uint64_t> g_launches{0};

// ------------------------------------------------------------------ plan (device views)
struct Plan {
  // per tensor
  const int32_t* t_off;
  const int32_t* t_end;
  const int32_t* t_k;
  const int32_t* t_out_off;
  const int32_t* t_part_first;
  const int32_t* t_part_num;
  const int32_t* t_rank;
  const int32_t* t_groups;
  uint32_t* t_kth;
  int32_t* t_cand;
  int32_t* t_dense;
  // per part
  const int32_t* p_tensor;
  const int32_t* p_end;     // arena index one past the part's last real element
  const int32_t* p_seg0;    // first segment of the part
  const int32_t* p_nseg;
  const int32_t* p_cbase;   // start of the part's candidate list
  const int32_t* p_cap;
  int32_t* p_count;
  uint32_t* p_thr;
  int32_t* p_out_base;
  int32_t* p_quota;
  int32_t* p_gt;
  int32_t* p_eq;
  // per segment
  const int32_t* seg_part;
  // sampled tensors
  const int32_t* sampled;
  // candidate lists
  int32_t* cand_idx;
  float* cand_val;
  // scalars
  float* coef;
  double* norm;
  double* partials;
  unsigned int* ticket;
  long long* diag;   // [2][4]: flags, full_select, candidates, unused
  // state
  float* u;
  float* v;
  int32_t num_tensors;
  int32_t num_parts;
  int32_t num_segs;
};

// ------------------------------------------------------------------ device helpers
__device__ __forceinline__ uint32_t mag_key(float x) { return __float_as_uint(x) & 0x7FFFFFFFu; }

// Eq. 5, one element: gc = g*coef ; u <- m*u + gc ; v <- v + u (each rounded once).
template <bool CLIP>
__device__ __forceinline__ void mc_step(float g, float coef, float m, float& u, float& v) {
  const float gc = CLIP ? __fmul_rn(g, coef) : g;
  const float t = __fmul_rn(m, u);
  u = __fadd_rn(t, gc);
  v = __fadd_rn(v, u);
}

__device__ __forceinline__ uint64_t mix64(uint64_t x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}

// Block-wide exclusive scan of one int per thread; returns the exclusive prefix
// and the block total.  `sh` needs 33 ints.  Contains two barriers.
__device__ __forceinline__ int block_excl_scan(int x, int* sh, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  int incl = x;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) sh[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = lane < nwarps ? sh[lane] : 0;
    int wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xFFFFFFFFu, wi, o);
      if (lane >= o) wi += t;
    }
    sh[lane] = wi - w;
    if (lane == 31) sh[32] = wi;
  }
  __syncthreads();
  const int res = sh[warp] + incl - x;
  total = sh[32];
  __syncthreads();
  return res;
}

// Radix select, descending: the `rank`-th largest key (rank >= 1) among the
// keys the iterator visits.  `for_each(f)` must call f(valid, key) the same
// number of times on every thread of the block (valid = false for padding
// calls).  hist: 256 words, sh: 2 words of shared memory.
// Returns the key; n_gt = number of keys strictly greater.
template <class ForEach>
__device__ uint32_t block_select_desc(ForEach for_each, int rank, uint32_t* hist, int* sh,
                                      int& n_gt) {
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31;
  uint32_t prefix = 0, mask = 0;
  int remaining = rank;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = tid; i < 256; i += nt) hist[i] = 0;
    __syncthreads();
    for_each([&](bool valid, uint32_t key) {
      uint32_t d = 0;
      if (valid && (key & mask) == prefix) d = (key >> shift) & 255u; else valid = false;
      // keys cluster on a few digits in the leading passes: lanes that share the digit of
      // the first valid lane are added with one atomic, the others one by one
      const unsigned vm = __ballot_sync(0xFFFFFFFFu, valid);
      if (vm != 0) {
        const uint32_t d0 = __shfl_sync(0xFFFFFFFFu, d, __ffs(vm) - 1);
        const unsigned m0 = __ballot_sync(0xFFFFFFFFu, valid && d == d0);
        if (valid) {
          if (d != d0) atomicAdd(&hist[d], 1u);
          else if (lane == __ffs(m0) - 1) atomicAdd(&hist[d], (uint32_t)__popc(m0));
        }
      }
    });
    __syncthreads();
    if (tid < 32) {
      const int hi = 255 - 8 * lane;          // this lane covers bins hi, hi-1, .., hi-7
      uint32_t loc[8];
      uint32_t s = 0;
#pragma unroll
      for (int q = 0; q < 8; ++q) { loc[q] = hist[hi - q]; s += loc[q]; }
      uint32_t incl = s;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += t;
      }
      const uint32_t excl = incl - s;
      if (excl < (uint32_t)remaining && (uint32_t)remaining <= incl) {
        uint32_t c = excl;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          if (c + loc[q] >= (uint32_t)remaining) { sh[0] = hi - q; sh[1] = (int)c; break; }
          c += loc[q];
        }
      }
    }
    __syncthreads();
    prefix |= (uint32_t)sh[0] << shift;
    mask |= 255u << shift;
    remaining -= sh[1];
    __syncthreads();
  }
  n_gt = rank - remaining;
  return prefix;
}

// ------------------------------------------------------------------ K1: clipping norm
// Sec. 3.2 / Appendix C.  Sum of squares of every real element of the gradient
// set: fp32 loads, exact fp64 products, fp64 accumulation; fixed reduction
// tree (grid size fixed per state), so the result does not depend on timing.
// The last block to finish folds the partials and writes norm and coef.
__global__ void __launch_bounds__(kNormThreads)
k_sumsq(Plan p, const float* __restrict__ g, double thr_local, int clip_on) {
  __shared__ double swarp[kNormThreads / 32];
  __shared__ bool is_last;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int warps_total = gridDim.x * (kNormThreads / 32);
  const float4* g4 = reinterpret_cast<const float4*>(g);
  double acc = 0.0;
  for (int seg = blockIdx.x * (kNormThreads / 32) + warp; seg < p.num_segs; seg += warps_total) {
    const int part = p.seg_part[seg];
    const int end = p.p_end[part];
    const int base = seg * kSeg;
    float4 x[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) x[i] = __ldg(g4 + (base >> 2) + i * 32 + lane);
    if (base + kSeg <= end) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        acc += (double)x[i].x * (double)x[i].x;
        acc += (double)x[i].y * (double)x[i].y;
        acc += (double)x[i].z * (double)x[i].z;
        acc += (double)x[i].w * (double)x[i].w;
      }
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int e = base + (i * 32 + lane) * 4;
        if (e + 0 < end) acc += (double)x[i].x * (double)x[i].x;
        if (e + 1 < end) acc += (double)x[i].y * (double)x[i].y;
        if (e + 2 < end) acc += (double)x[i].z * (double)x[i].z;
        if (e + 3 < end) acc += (double)x[i].w * (double)x[i].w;
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
  if (lane == 0) swarp[warp] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int w = 0; w < kNormThreads / 32; ++w) s += swarp[w];
    p.partials[blockIdx.x] = s;
    __threadfence();
    const unsigned int t = atomicAdd(p.ticket, 1u);
    is_last = (t == gridDim.x - 1);
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  // fold the per-block partials in a fixed order
  double s = 0.0;
  for (int i = threadIdx.x; i < (int)gridDim.x; i += kNormThreads) s += __ldcg(p.partials + i);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
  if (lane == 0) swarp[warp] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    double S = 0.0;
    for (int w = 0; w < kNormThreads / 32; ++w) S += swarp[w];
    const double norm = sqrt(S);
    float coef = 1.0f;
    if (clip_on && norm > thr_local) coef = (float)(thr_local / norm);
    *p.norm = norm;
    *p.coef = coef;
    *p.ticket = 0u;
  }
}

// ------------------------------------------------------------------ K2: sampled threshold proposal
// Sec. 5: sample |v'| (v' computed on the fly from g, u, v exactly as the main
// pass will), take the sample's rank-r key as the proposed threshold of the
// tensor.  One float4 group per stratum at a hashed position; one block per
// sampled tensor.
template <bool CLIP>
__global__ void __launch_bounds__(kSampleThreads)
k_sample_threshold(Plan p, const float* __restrict__ g, float m, uint64_t call_seed) {
  extern __shared__ uint32_t skeys[];
  __shared__ uint32_t hist[256];
  __shared__ int sh[2];
  const int j = p.sampled[blockIdx.x];
  const int off = p.t_off[j];
  const int n = p.t_end[j] - off;
  const int G = p.t_groups[j];
  const int rank = p.t_rank[j];
  const long long Q = n >> 2;
  const float coef = CLIP ? *p.coef : 1.0f;
  const float4* g4 = reinterpret_cast<const float4*>(g) + (off >> 2);
  const float4* u4 = reinterpret_cast<const float4*>(p.u) + (off >> 2);
  const float4* v4 = reinterpret_cast<const float4*>(p.v) + (off >> 2);
  constexpr int kBatch = kMaxSampleGroups / kSampleThreads;   // groups per thread at most
  float4 gg[kBatch], uu[kBatch], vv[kBatch];
#pragma unroll
  for (int b = 0; b < kBatch; ++b) {
    const int s = b * kSampleThreads + threadIdx.x;
    if (s < G) {
      const long long lo = (long long)s * Q / G;
      const long long hi = (long long)(s + 1) * Q / G;
      const uint64_t h = mix64(call_seed ^ ((uint64_t)(uint32_t)j << 32) ^ (uint64_t)(uint32_t)s);
      const long long pos = lo + (long long)(h % (uint64_t)(hi - lo));
      gg[b] = __ldg(g4 + pos);
      uu[b] = __ldcg(u4 + pos);
      vv[b] = __ldcg(v4 + pos);
    }
  }
#pragma unroll
  for (int b = 0; b < kBatch; ++b) {
    const int s = b * kSampleThreads + threadIdx.x;
    if (s < G) {
      float4 u = uu[b], v = vv[b];
      mc_step<CLIP>(gg[b].x, coef, m, u.x, v.x);
      mc_step<CLIP>(gg[b].y, coef, m, u.y, v.y);
      mc_step<CLIP>(gg[b].z, coef, m, u.z, v.z);
      mc_step<CLIP>(gg[b].w, coef, m, u.w, v.w);
      skeys[4 * s + 0] = mag_key(v.x);
      skeys[4 * s + 1] = mag_key(v.y);
      skeys[4 * s + 2] = mag_key(v.z);
      skeys[4 * s + 3] = mag_key(v.w);
    }
  }
  __syncthreads();
  const int count = 4 * G;
  const int iters = (count + kSampleThreads - 1) / kSampleThreads;
  int n_gt;
  const uint32_t kth = block_select_desc(
      [&](auto f) {
        for (int it = 0; it < iters; ++it) {
          const int i = it * kSampleThreads + threadIdx.x;
          const bool valid = i < count;
          f(valid, valid ? skeys[i] : 0u);
        }
      },
      rank, hist, sh, n_gt);
  // a proposal of 0 would let every entry through: insist on non-zero magnitude
  const uint32_t thr = kth > 1u ? kth : 1u;
  const int p0 = p.t_part_first[j], pn = p.t_part_num[j];
  for (int q = threadIdx.x; q < pn; q += kSampleThreads) p.p_thr[p0 + q] = thr;
}

// ------------------------------------------------------------------ K3: fused momentum correction + candidate emission
// The streaming pass: 12 B read + 8 B written per element.  Each warp owns one
// 512-element segment at a time (4 float4 per lane per array, 512 contiguous
// bytes per warp load), keeps everything in registers, and appends the
// segment's candidates -- in ascending index order -- to its part's list with
// one integer atomicAdd per segment that has any.
template <bool CLIP>
__global__ void __launch_bounds__(kMainThreads)
k_update_emit(Plan p, const float* __restrict__ g, float m) {
  const int lane = threadIdx.x & 31;
  const int warps_total = gridDim.x * (kMainThreads / 32);
  const float coef = CLIP ? *p.coef : 1.0f;
  const float4* g4 = reinterpret_cast<const float4*>(g);
  float4* u4 = reinterpret_cast<float4*>(p.u);
  float4* v4 = reinterpret_cast<float4*>(p.v);
  for (int seg = blockIdx.x * (kMainThreads / 32) + (threadIdx.x >> 5); seg < p.num_segs;
       seg += warps_total) {
    const int base = seg * kSeg;
    const int q0 = (base >> 2) + lane;
    float4 gg[4], uu[4], vv[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) gg[i] = __ldcs(g4 + q0 + i * 32);
#pragma unroll
    for (int i = 0; i < 4; ++i) uu[i] = __ldcs(u4 + q0 + i * 32);
#pragma unroll
    for (int i = 0; i < 4; ++i) vv[i] = __ldcs(v4 + q0 + i * 32);
    const int part = p.seg_part[seg];
    const int end = p.p_end[part];
    const uint32_t thr = p.p_thr[part];
    const bool full = base + kSeg <= end;
    uint32_t flags = 0;   // bit (4*i + c): element c of float4 i is a candidate
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      mc_step<CLIP>(gg[i].x, coef, m, uu[i].x, vv[i].x);
      mc_step<CLIP>(gg[i].y, coef, m, uu[i].y, vv[i].y);
      mc_step<CLIP>(gg[i].z, coef, m, uu[i].z, vv[i].z);
      mc_step<CLIP>(gg[i].w, coef, m, uu[i].w, vv[i].w);
      flags |= (uint32_t)(mag_key(vv[i].x) >= thr) << (4 * i + 0);
      flags |= (uint32_t)(mag_key(vv[i].y) >= thr) << (4 * i + 1);
      flags |= (uint32_t)(mag_key(vv[i].z) >= thr) << (4 * i + 2);
      flags |= (uint32_t)(mag_key(vv[i].w) >= thr) << (4 * i + 3);
    }
    if (full) {
#pragma unroll
      for (int i = 0; i < 4; ++i) __stcs(u4 + q0 + i * 32, uu[i]);
#pragma unroll
      for (int i = 0; i < 4; ++i) __stcs(v4 + q0 + i * 32, vv[i]);
    } else {
      // ragged end of a tensor: only real elements are stored or can be candidates
      uint32_t valid = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int e = base + (i * 32 + lane) * 4;
        const float uarr[4] = {uu[i].x, uu[i].y, uu[i].z, uu[i].w};
        const float varr[4] = {vv[i].x, vv[i].y, vv[i].z, vv[i].w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          if (e + c < end) {
            valid |= 1u << (4 * i + c);
            p.u[e + c] = uarr[c];
            p.v[e + c] = varr[c];
          }
        }
      }
      flags &= valid;
    }
    if (__any_sync(0xFFFFFFFFu, flags != 0)) {
      // per-lane counts of the four float4 rows packed one per byte (row totals <= 128)
      const uint32_t cnt = __popc(flags & 0xFu) | (__popc(flags & 0xF0u) << 8) |
                           (__popc(flags & 0xF00u) << 16) | (__popc(flags & 0xF000u) << 24);
      uint32_t incl = cnt;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += t;
      }
      const uint32_t tot = __shfl_sync(0xFFFFFFFFu, incl, 31);
      const uint32_t excl = incl - cnt;
      const int t0 = tot & 255, t1 = (tot >> 8) & 255, t2 = (tot >> 16) & 255, t3 = tot >> 24;
      const int seg_total = t0 + t1 + t2 + t3;
      int start = 0;
      if (lane == 0) start = atomicAdd(p.p_count + part, seg_total);
      start = __shfl_sync(0xFFFFFFFFu, start, 0);
      const int cap = p.p_cap[part];
      const int cbase = p.p_cbase[part];
      const int row_base[4] = {0, t0, t0 + t1, t0 + t1 + t2};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t nib = (flags >> (4 * i)) & 0xFu;
        if (nib) {
          int pos = start + row_base[i] + (int)((excl >> (8 * i)) & 255u);
          const int e = base + (i * 32 + lane) * 4;
          const float varr[4] = {vv[i].x, vv[i].y, vv[i].z, vv[i].w};
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            if (nib & (1u << c)) {
              if (pos < cap) {
                p.cand_idx[cbase + pos] = e + c;
                p.cand_val[cbase + pos] = varr[c];
              }
              ++pos;
            }
          }
        }
      }
    }
  }
}

// ------------------------------------------------------------------ K4: exact k-th key per tensor
// Algorithm 4 "thr <- s% of |V[j]|" made exact: the k_j-th largest |v'| among
// the tensor's candidates, the number of strictly larger ones and the tie
// quota; then each part's first output slot and its share of the ties (ties go
// to the lower index, so to the earlier part).  One block per tensor.
__global__ void __launch_bounds__(kSelectThreads)
k_select(Plan p, int smem_keys, int parity) {
  extern __shared__ uint32_t skeys[];
  __shared__ uint32_t hist[256];
  __shared__ int sh[40];
  __shared__ int s_flag;
  const int j = blockIdx.x;
  const int tid = threadIdx.x;
  const int p0 = p.t_part_first[j], pn = p.t_part_num[j];
  const int k = p.t_k[j];
  if (j == 0 && tid < 4) p.diag[(parity ^ 1) * 4 + tid] = 0;   // next call's counters
  if (tid == 0) s_flag = 0;
  __syncthreads();
  // total candidates, overflow check
  int my = 0;
  for (int q = tid; q < pn; q += kSelectThreads) {
    const int c = __ldcg(p.p_count + p0 + q);
    if (c > p.p_cap[p0 + q]) s_flag = 1;
    my += c;
  }
  int total;
  block_excl_scan(my, sh, total);
  const bool overflow = s_flag != 0;
  if (overflow || total < k) {
    if (tid == 0) {
      p.t_dense[j] = 1;
      p.t_cand[j] = -1;
      atomicOr((unsigned long long*)&p.diag[parity * 4 + 0],
               (unsigned long long)(DGC_FLAG_FULL_SELECT |
                                    (overflow ? DGC_FLAG_CAND_OVERFLOW : DGC_FLAG_CAND_SHORT)));
      atomicAdd((unsigned long long*)&p.diag[parity * 4 + 1], 1ull);
    }
    return;
  }
  const bool in_smem = total <= smem_keys;
  if (in_smem) {
    // gather the keys of all parts, compact, into shared memory
    int basek = 0;
    for (int q = 0; q < pn; ++q) {
      const int c = __ldcg(p.p_count + p0 + q);
      const float* src = p.cand_val + p.p_cbase[p0 + q];
      for (int i = tid; i < c; i += kSelectThreads) skeys[basek + i] = mag_key(__ldcg(src + i));
      basek += c;
    }
    __syncthreads();
  }
  int n_gt;
  uint32_t kth;
  if (in_smem) {
    const int iters = (total + kSelectThreads - 1) / kSelectThreads;
    kth = block_select_desc(
        [&](auto f) {
          for (int it = 0; it < iters; ++it) {
            const int i = it * kSelectThreads + tid;
            const bool valid = i < total;
            f(valid, valid ? skeys[i] : 0u);
          }
        },
        k, hist, sh, n_gt);
  } else {
    kth = block_select_desc(
        [&](auto f) {
          for (int q = 0; q < pn; ++q) {
            const int c = __ldcg(p.p_count + p0 + q);
            const float* src = p.cand_val + p.p_cbase[p0 + q];
            const int iters = (c + kSelectThreads - 1) / kSelectThreads;
            for (int it = 0; it < iters; ++it) {
              const int i = it * kSelectThreads + tid;
              const bool valid = i < c;
              f(valid, valid ? mag_key(__ldcg(src + i)) : 0u);
            }
          }
        },
        k, hist, sh, n_gt);
  }
  const int quota = k - n_gt;   // ties (|v'| == kth) to take, lowest indices first
  // per part: how many strictly-greater and how many tied candidates; one warp per part
  {
    const int lane = tid & 31, warp = tid >> 5;
    int basek = 0;
    // warps walk the parts round robin; basek must be tracked by every warp
    for (int q = 0; q < pn; ++q) {
      const int c = __ldcg(p.p_count + p0 + q);
      if ((q & 31) == warp) {
        const float* src = p.cand_val + p.p_cbase[p0 + q];
        int gt = 0, eq = 0;
        for (int i = lane; i < c; i += 32) {
          const uint32_t key = in_smem ? skeys[basek + i] : mag_key(__ldcg(src + i));
          gt += key > kth;
          eq += key == kth;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          gt += __shfl_xor_sync(0xFFFFFFFFu, gt, o);
          eq += __shfl_xor_sync(0xFFFFFFFFu, eq, o);
        }
        if (lane == 0) { p.p_gt[p0 + q] = gt; p.p_eq[p0 + q] = eq; }
      }
      basek += c;
    }
  }
  __syncthreads();
  // exclusive prefix over the tensor's parts (chunks of blockDim parts with a carry)
  int run_gt = 0, run_eq = 0;
  const int out_off = p.t_out_off[j];
  for (int q0 = 0; q0 < pn; q0 += kSelectThreads) {
    const int q = q0 + tid;
    const int gt = q < pn ? p.p_gt[p0 + q] : 0;
    const int eq = q < pn ? p.p_eq[p0 + q] : 0;
    int tg, te;
    const int bg = block_excl_scan(gt, sh, tg) + run_gt;
    const int be = block_excl_scan(eq, sh, te) + run_eq;
    if (q < pn) {
      p.p_out_base[p0 + q] = out_off + bg + min(be, quota);
      p.p_quota[p0 + q] = max(0, min(quota - be, eq));
    }
    run_gt += tg;
    run_eq += te;
  }
  if (tid == 0) {
    p.t_kth[j] = kth;
    p.t_cand[j] = total;
    p.t_dense[j] = 0;
    atomicAdd((unsigned long long*)&p.diag[parity * 4 + 2], (unsigned long long)total);
  }
}

// ------------------------------------------------------------------ K5: ordered emission + masking
// Algorithm 4: G~[j] <- V[j] (.) Mask ; V[j] <- V[j] (.) !Mask ; U[j] <- U[j] (.) !Mask.
// One block per part, one thread per segment.  The candidates that reach the
// threshold set one bit each in a shared-memory bitmap of the part (integer
// atomicOr; "greater" and "tied" bitmaps); per-segment popcounts and an
// exclusive scan give every segment its first output slot; each thread then
// walks its segment's bits in index order, reads v' at those entries, writes
// the pairs and zeroes u and v there.
//
// Full-selection path (dense flag set by k_select): the block of the tensor's
// first part selects from the whole of v' (radix select over global memory) and
// emits by walking the tensor in order.  Same result; slow; rare.
__device__ void dense_select_emit(const Plan& p, int j, int32_t* out_idx, float* out_val,
                                  uint32_t* hist, int* sh) {
  const int tid = threadIdx.x, nt = blockDim.x;
  const int off = p.t_off[j];
  const int n = p.t_end[j] - off;
  const int k = p.t_k[j];
  const float* v = p.v + off;
  const int iters = (n + nt - 1) / nt;
  int n_gt;
  const uint32_t kth = block_select_desc(
      [&](auto f) {
        for (int it = 0; it < iters; ++it) {
          const int i = it * nt + tid;
          const bool valid = i < n;
          f(valid, valid ? mag_key(__ldcg(v + i)) : 0u);
        }
      },
      k, hist, sh, n_gt);
  const int quota = k - n_gt;
  int run_w = 0, run_eq = 0;     // winners / ties seen so far
  const int out_off = p.t_out_off[j];
  for (int c0 = 0; c0 < n; c0 += nt * 4) {
    const int e0 = c0 + tid * 4;
    float x[4];
    int gt = 0, eq = 0;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      x[c] = (e0 + c < n) ? __ldcg(v + e0 + c) : 0.0f;
      const uint32_t key = mag_key(x[c]);
      if (e0 + c < n) { gt += key > kth; eq += key == kth; }
    }
    int tg, te;
    const int bg = block_excl_scan(gt, sh, tg);
    const int be = block_excl_scan(eq, sh, te) + run_eq;
    int pos = out_off + run_w + bg + (min(be, quota) - min(run_eq, quota));
    int eqr = be;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      if (e0 + c < n) {
        const uint32_t key = mag_key(x[c]);
        bool take = key > kth;
        if (key == kth) { take = eqr < quota; ++eqr; }
        if (take) {
          out_idx[pos] = off + e0 + c;
          out_val[pos] = x[c];
          p.u[off + e0 + c] = 0.0f;
          p.v[off + e0 + c] = 0.0f;
          ++pos;
        }
      }
    }
    run_w += tg + (min(run_eq + te, quota) - min(run_eq, quota));
    run_eq += te;
  }
  if (tid == 0) p.t_kth[j] = kth;
}

__global__ void __launch_bounds__(kEmitThreads)
k_emit_mask(Plan p, int32_t* __restrict__ out_idx, float* __restrict__ out_val) {
  extern __shared__ uint32_t smask[];          // winner bitmaps of the part: [gt | eq]
  __shared__ uint32_t hist[256];
  __shared__ int sh[40];
  uint32_t* mgt = smask;
  uint32_t* meq = smask + kPartSegs * kMaskStride;
  const int part = blockIdx.x;
  const int tid = threadIdx.x;
  const int j = p.p_tensor[part];
  const int count = __ldcg(p.p_count + part);
  const bool dense = __ldcg(p.t_dense + j) != 0;
  __syncthreads();
  if (tid == 0) p.p_count[part] = 0;          // ready for the next call
  if (dense) {
    if (part == p.t_part_first[j]) dense_select_emit(p, j, out_idx, out_val, hist, sh);
    return;
  }
  const uint32_t kth = __ldcg(p.t_kth + j);
  const int quota = __ldcg(p.p_quota + part);
  const int out_base = __ldcg(p.p_out_base + part);
  const int seg0 = p.p_seg0[part];
  const int nseg = p.p_nseg[part];
  const int32_t* cidx = p.cand_idx + p.p_cbase[part];
  const float* cval = p.cand_val + p.p_cbase[part];
  for (int i = tid; i < 2 * kPartSegs * kMaskStride; i += kEmitThreads) smask[i] = 0u;
  __syncthreads();
  // mark the candidates that reach the threshold: one bit per element of the part
  for (int i = tid; i < count; i += kEmitThreads) {
    const uint32_t key = mag_key(__ldcg(cval + i));
    if (key >= kth) {
      const int local = __ldcg(cidx + i) - seg0 * kSeg;
      const int word = (local >> 9) * kMaskStride + ((local >> 5) & 15);
      atomicOr((key > kth ? mgt : meq) + word, 1u << (local & 31));
    }
  }
  __syncthreads();
  // thread s owns segment s: count, scan, then walk its bits in index order
  int gt = 0, eq = 0;
  if (tid < nseg) {
#pragma unroll
    for (int w = 0; w < 16; ++w) {
      gt += __popc(mgt[tid * kMaskStride + w]);
      eq += __popc(meq[tid * kMaskStride + w]);
    }
  }
  int tg, te;
  const int bg = block_excl_scan(gt, sh, tg);
  int eqr = block_excl_scan(eq, sh, te);
  if (gt + eq == 0) return;
  int pos = out_base + bg + min(eqr, quota);
  const int ebase = (seg0 + tid) * kSeg;
  for (int w = 0; w < 16; ++w) {
    const uint32_t g = mgt[tid * kMaskStride + w];
    const uint32_t e = meq[tid * kMaskStride + w];
    uint32_t both = g | e;
    while (both) {
      const int b = __ffs(both) - 1;
      both &= both - 1;
      bool take = true;
      if ((e >> b) & 1u) { take = eqr < quota; ++eqr; }   // ties: lowest indices first
      if (take) {
        const int idx = ebase + w * 32 + b;
        out_idx[pos] = idx;
        out_val[pos] = __ldcg(p.v + idx);
        p.u[idx] = 0.0f;
        p.v[idx] = 0.0f;
        ++pos;
      }
    }
  }
}

// ------------------------------------------------------------------ receive side
// Alg. 4 "G_t <- sum_k encode(G~_k)".  k_decode_bounds finds, for every worker
// list (ascending indices), where each tile of the dense output starts;
// k_decode_tiles accumulates a tile in shared memory one worker after the other
// (indices within one worker are unique, so no two threads touch one slot
// between barriers) and writes it once.
struct DecodeArgs {
  const int32_t* idx[DGC_MAX_DECODE_WORKERS];
  const float* val[DGC_MAX_DECODE_WORKERS];
  int32_t nnz[DGC_MAX_DECODE_WORKERS];
  int32_t num_workers;
  int32_t num_tiles;
};

__global__ void __launch_bounds__(256)
k_decode_bounds(const __grid_constant__ DecodeArgs a, int32_t* __restrict__ bounds) {
  // bounds[w * (num_tiles + 1) + t] = first position in list w whose index >= t * tile
  const int w = blockIdx.y;
  const int n = a.nnz[w];
  const int32_t* idx = a.idx[w];
  int32_t* b = bounds + (size_t)w * (a.num_tiles + 1);
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i <= n; i += gridDim.x * blockDim.x) {
    const int t_prev = (i == 0) ? -1 : (__ldg(idx + i - 1) / kDecodeTile);
    const int t_cur = (i == n) ? a.num_tiles : (__ldg(idx + i) / kDecodeTile);
    for (int t = t_prev + 1; t <= t_cur; ++t) b[t] = i;
  }
}

__global__ void __launch_bounds__(kDecodeThreads)
k_decode_tiles(const __grid_constant__ DecodeArgs a, const int32_t* __restrict__ bounds,
               float* __restrict__ dense, long long dense_len) {
  __shared__ float tile[kDecodeTile];
  __shared__ int s_lo[DGC_MAX_DECODE_WORKERS], s_hi[DGC_MAX_DECODE_WORKERS];
  const int t = blockIdx.x;
  const long long base = (long long)t * kDecodeTile;
  if (threadIdx.x < a.num_workers) {
    const int32_t* b = bounds + (size_t)threadIdx.x * (a.num_tiles + 1);
    s_lo[threadIdx.x] = __ldg(b + t);
    s_hi[threadIdx.x] = __ldg(b + t + 1);
  }
#pragma unroll
  for (int i = threadIdx.x; i < kDecodeTile; i += kDecodeThreads) tile[i] = 0.0f;
  __syncthreads();
  for (int w = 0; w < a.num_workers; ++w) {
    const int lo = s_lo[w], hi = s_hi[w];
    if (hi > lo) {      // block-uniform
      const int32_t* idx = a.idx[w];
      const float* val = a.val[w];
      for (int i = lo + threadIdx.x; i < hi; i += kDecodeThreads) {
        const int l = __ldg(idx + i) - (int)base;
        tile[l] = __fadd_rn(tile[l], __ldg(val + i));
      }
      __syncthreads();
    }
  }
  const long long rem = dense_len - base;
  if (rem >= kDecodeTile) {
    float4* d4 = reinterpret_cast<float4*>(dense + base);
    const float4* t4 = reinterpret_cast<const float4*>(tile);
#pragma unroll
    for (int i = threadIdx.x; i < kDecodeTile / 4; i += kDecodeThreads) __stcs(d4 + i, t4[i]);
  } else {
    for (int i = threadIdx.x; i < (int)rem; i += kDecodeThreads) dense[base + i] = tile[i];
  }
}

// Alg. 4 "theta <- SGD(theta, G_t)": w <- w - lr*G, two roundings.
__global__ void __launch_bounds__(256)
k_sgd(float* __restrict__ w, const float* __restrict__ G, long long len, float lr) {
  const long long n4 = len >> 2;
  float4* w4 = reinterpret_cast<float4*>(w);
  const float4* g4 = reinterpret_cast<const float4*>(G);
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
    float4 a = __ldcs(w4 + i);
    const float4 b = __ldcs(g4 + i);
    a.x = __fsub_rn(a.x, __fmul_rn(lr, b.x));
    a.y = __fsub_rn(a.y, __fmul_rn(lr, b.y));
    a.z = __fsub_rn(a.z, __fmul_rn(lr, b.z));
    a.w = __fsub_rn(a.w, __fmul_rn(lr, b.w));
    __stcs(w4 + i, a);
  }
  if (blockIdx.x == 0 && threadIdx.x < (int)(len & 3)) {
    const long long i = (n4 << 2) + threadIdx.x;
    w[i] = __fsub_rn(w[i], __fmul_rn(lr, G[i]));
  }
}

// ------------------------------------------------------------------ host side
int64_t topk_count(int64_t n, double sparsity) {
  const long long q = std::llround((1.0 - sparsity) * 1e9);
  long long k = ((long long)n * q + 999999999LL) / 1000000000LL;
  if (k < 1) k = 1;
  if (k > n) k = n;
  return k;
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

struct DevBuf {
  void* ptr = nullptr;
  size_t bytes = 0;
};

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
  std::vector<int32_t> t_off, t_end, t_k, t_out_off, t_part_first, t_part_num, t_rank, t_groups;
  std::vector<int32_t> p_tensor, p_end, p_seg0, p_nseg, p_cbase, p_cap;
  std::vector<uint32_t> p_thr_init;
  std::vector<int32_t> seg_part, sampled;
  int64_t max_nnz = 0;
  int64_t cand_total = 0;
  int max_sample_keys = 0;
  int64_t max_tensor_expect = 0;   // largest expected candidate count of one tensor
  // device
  std::vector<void*> allocs;
  int32_t* d_ints = nullptr;      // all int32 plan tables in one allocation
  size_t d_ints_count = 0;
  int32_t* d_cand_idx = nullptr;
  float* d_cand_val = nullptr;
  int64_t cand_alloc = 0;
  float* d_stage_g = nullptr;     // dgc_compress_host staging
  int32_t* d_stage_idx = nullptr;
  float* d_stage_val = nullptr;
  int64_t stage_nnz = 0;
  Plan plan{};
  // optional timing of the streaming kernel (dgc_profile_enable)
  std::vector<cudaEvent_t> prof_ev;   // 2 events per recorded call
  int prof_cap = 0, prof_n = 0;
  int norm_grid = 0, main_grid = 0, main_grid_clip = 0;
  int select_smem_keys = 0;
  bool alive = false;
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
void build_host_plan(dgc_state* st, double sparsity) {
  const int T = st->cfg.num_tensors;
  const double ratio = st->cfg.sample_ratio > 0.0 ? st->cfg.sample_ratio : 0.01;
  st->t_off.assign(T, 0); st->t_end.assign(T, 0); st->t_k.assign(T, 0);
  st->t_out_off.assign(T, 0); st->t_part_first.assign(T, 0); st->t_part_num.assign(T, 0);
  st->t_rank.assign(T, 0); st->t_groups.assign(T, 0);
  st->p_tensor.clear(); st->p_end.clear(); st->p_seg0.clear(); st->p_nseg.clear();
  st->p_cbase.clear(); st->p_cap.clear(); st->p_thr_init.clear();
  st->seg_part.clear(); st->sampled.clear();
  int64_t pos = 0, out = 0, cbase = 0;
  st->max_sample_keys = 0;
  st->max_tensor_expect = 0;
  for (int j = 0; j < T; ++j) {
    const int64_t n = st->numel[j];
    const int64_t k = topk_count(n, sparsity);
    st->t_off[j] = (int32_t)pos;
    st->t_end[j] = (int32_t)(pos + n);
    st->t_k[j] = (int32_t)k;
    st->t_out_off[j] = (int32_t)out;
    out += k;
    const int64_t nseg = (n + kSeg - 1) / kSeg;
    const int64_t nparts = (nseg + kPartSegs - 1) / kPartSegs;
    // sampling plan
    bool sampled = n > kSmallN;
    int groups = 0, rank = 0;
    double cap_total = (double)n;
    if (sampled) {
      const int64_t Q = n / 4;
      int64_t G = (int64_t)std::ceil(ratio * (double)n / 4.0);
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
      }
    }
    if (sampled) {
      st->t_rank[j] = rank;
      st->t_groups[j] = groups;
      st->sampled.push_back(j);
      st->max_sample_keys = std::max(st->max_sample_keys, 4 * groups);
    }
    st->t_part_first[j] = (int32_t)st->p_tensor.size();
    st->t_part_num[j] = (int32_t)nparts;
    for (int64_t q = 0; q < nparts; ++q) {
      const int64_t seg0 = pos / kSeg + q * kPartSegs;
      const int64_t ns = std::min<int64_t>(kPartSegs, nseg - q * kPartSegs);
      const int64_t pend = std::min<int64_t>(pos + n, (seg0 + ns) * kSeg);
      const int64_t elems = pend - seg0 * kSeg;
      int64_t cap = elems;
      if (sampled) {
        const int64_t share = (int64_t)std::ceil(cap_total / (double)nparts);
        cap = std::min<int64_t>(elems, std::max<int64_t>(4 * share, 8192));
      }
      st->p_tensor.push_back(j);
      st->p_end.push_back((int32_t)pend);
      st->p_seg0.push_back((int32_t)seg0);
      st->p_nseg.push_back((int32_t)ns);
      st->p_cbase.push_back((int32_t)cbase);
      st->p_cap.push_back((int32_t)cap);
      st->p_thr_init.push_back(0u);      // not sampled: every entry is a candidate
      cbase += cap;
      for (int64_t s = 0; s < ns; ++s) st->seg_part.push_back((int32_t)(st->p_tensor.size() - 1));
    }
    st->max_tensor_expect = std::max<int64_t>(st->max_tensor_expect, (int64_t)cap_total);
    pos += nseg * kSeg;
  }
  st->arena_len = pos;
  st->max_nnz = out;
  st->cand_total = cbase;
  st->sparsity = sparsity;
}

int32_t upload_plan(dgc_state* st, bool first) {
  const size_t T = st->cfg.num_tensors, P = st->p_tensor.size(), S = st->seg_part.size();
  const size_t NS = st->sampled.size();
  // layout of the int32 table block
  const size_t count = 11 * T + 12 * P + S + NS + 16;
  if (first || count > st->d_ints_count) {
    if (st->d_ints) dev_free(st, st->d_ints);
    void* ptr = nullptr;
    int32_t rc = dev_alloc(st, &ptr, count * sizeof(int32_t));
    if (rc != DGC_OK) return rc;
    st->d_ints = (int32_t*)ptr;
    st->d_ints_count = count;
  }
  std::vector<int32_t> h(count, 0);
  size_t o = 0;
  auto put = [&](const std::vector<int32_t>& v) {
    const size_t at = o;
    if (!v.empty()) std::memcpy(h.data() + o, v.data(), v.size() * 4);
    o += v.size();
    return at;
  };
  auto skip = [&](size_t n) { size_t at = o; o += n; return at; };
  const size_t o_off = put(st->t_off), o_end = put(st->t_end), o_k = put(st->t_k),
               o_out = put(st->t_out_off), o_pf = put(st->t_part_first), o_pn = put(st->t_part_num),
               o_rank = put(st->t_rank), o_groups = put(st->t_groups);
  const size_t o_kth = skip(T), o_cand = skip(T), o_dense = skip(T);
  const size_t o_pt = put(st->p_tensor), o_pe = put(st->p_end), o_ps = put(st->p_seg0),
               o_pns = put(st->p_nseg), o_pcb = put(st->p_cbase), o_pcap = put(st->p_cap);
  const size_t o_pcount = skip(P);
  const size_t o_pthr = o;
  std::memcpy(h.data() + o, st->p_thr_init.data(), P * 4); o += P;
  const size_t o_pob = skip(P), o_pq = skip(P), o_pgt = skip(P), o_peq = skip(P);
  const size_t o_seg = put(st->seg_part), o_samp = put(st->sampled);
  DGC_CUDA(cudaMemcpy(st->d_ints, h.data(), count * 4, cudaMemcpyHostToDevice));
  int32_t* d = st->d_ints;
  Plan& p = st->plan;
  p.t_off = d + o_off; p.t_end = d + o_end; p.t_k = d + o_k; p.t_out_off = d + o_out;
  p.t_part_first = d + o_pf; p.t_part_num = d + o_pn; p.t_rank = d + o_rank; p.t_groups = d + o_groups;
  p.t_kth = (uint32_t*)(d + o_kth); p.t_cand = d + o_cand; p.t_dense = d + o_dense;
  p.p_tensor = d + o_pt; p.p_end = d + o_pe; p.p_seg0 = d + o_ps; p.p_nseg = d + o_pns;
  p.p_cbase = d + o_pcb; p.p_cap = d + o_pcap; p.p_count = d + o_pcount;
  p.p_thr = (uint32_t*)(d + o_pthr); p.p_out_base = d + o_pob; p.p_quota = d + o_pq;
  p.p_gt = d + o_pgt; p.p_eq = d + o_peq; p.seg_part = d + o_seg; p.sampled = d + o_samp;
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
  int keys = (int)std::min<int64_t>(st->max_tensor_expect, kSelectMaxSmemKeys);
  keys = std::max(keys, 1024);
  st->select_smem_keys = keys;
  DGC_CUDA(cudaFuncSetAttribute(k_select, cudaFuncAttributeMaxDynamicSharedMemorySize, keys * 4));
  return DGC_OK;
}

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

int32_t check_launch() {
  g_launches.fetch_add(1, std::memory_order_relaxed);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? DGC_OK : DGC_ECUDA;
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
  DGC_CUDA(cudaSetDevice(cfg->device));
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
  // scalars: partials[kMaxNormGrid] doubles, norm, diag[8] long long, coef, ticket
  const size_t scal_bytes = (kMaxNormGrid + 1) * 8 + 8 * 8 + 16;
  if ((rc = dev_alloc(st, &ptr, scal_bytes)) != DGC_OK) return fail(rc);
  char* sc = (char*)ptr;
  st->plan.partials = (double*)sc;
  st->plan.norm = (double*)(sc + kMaxNormGrid * 8);
  st->plan.diag = (long long*)(sc + (kMaxNormGrid + 1) * 8);
  st->plan.coef = (float*)(sc + (kMaxNormGrid + 1) * 8 + 64);
  st->plan.ticket = (unsigned int*)(sc + (kMaxNormGrid + 1) * 8 + 64 + 8);
  if (cudaMemset(st->plan.u, 0, (size_t)st->arena_len * 4) != cudaSuccess) return fail(DGC_ECUDA);
  if (cudaMemset(st->plan.v, 0, (size_t)st->arena_len * 4) != cudaSuccess) return fail(DGC_ECUDA);
  if (cudaMemset(sc, 0, scal_bytes) != cudaSuccess) return fail(DGC_ECUDA);
  const float one = 1.0f;
  if (cudaMemcpy(st->plan.coef, &one, 4, cudaMemcpyHostToDevice) != cudaSuccess) return fail(DGC_ECUDA);
  // launch geometry
  int occ = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_update_emit<false>, kMainThreads, 0) !=
      cudaSuccess) return fail(DGC_ECUDA);
  st->main_grid = st->sm_count * std::max(occ, 1);
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_update_emit<true>, kMainThreads, 0) !=
      cudaSuccess) return fail(DGC_ECUDA);
  st->main_grid_clip = st->sm_count * std::max(occ, 1);
  st->norm_grid = std::min(kMaxNormGrid, st->sm_count * 8);
  if (cudaFuncSetAttribute(k_sample_threshold<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kMaxSampleGroups * 16) != cudaSuccess) return fail(DGC_ECUDA);
  if (cudaFuncSetAttribute(k_sample_threshold<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kMaxSampleGroups * 16) != cudaSuccess) return fail(DGC_ECUDA);
  if (cudaFuncSetAttribute(k_emit_mask, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kEmitSmemBytes) != cudaSuccess) return fail(DGC_ECUDA);
  if (cudaDeviceSynchronize() != cudaSuccess) return fail(DGC_ECUDA);
  *out = st;
  return DGC_OK;
}

int32_t dgc_state_destroy(dgc_state* st) {
  if (!st || !st->alive) return DGC_ESTATE;
  cudaSetDevice(st->device);
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
  DGC_CUDA(cudaSetDevice(st->device));
  DGC_CUDA(cudaDeviceSynchronize());
  build_host_plan(st, sparsity);
  return upload_plan(st, false);
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
    if (arena_offset) arena_offset[j] = st->t_off[j];
    if (k) k[j] = st->t_k[j];
    if (out_offset) out_offset[j] = st->t_out_off[j];
  }
  if (out_offset) out_offset[T] = st->max_nnz;
  if (arena_len) *arena_len = st->arena_len;
  return DGC_OK;
}

int32_t dgc_compress(dgc_state* st, const float* grad_arena, int32_t* out_idx, float* out_val,
                     int64_t capacity, void* stream) {
  if (!st || !st->alive) return DGC_ESTATE;
  if (!grad_arena || !out_idx || !out_val) return DGC_EINVAL;
  if ((reinterpret_cast<uintptr_t>(grad_arena) & 15u) != 0) return DGC_EINVAL;
  if (capacity < st->max_nnz) return DGC_ECAPACITY;
  cudaStream_t s = as_stream(stream);
  const Plan& p = st->plan;
  const bool clip = st->cfg.clip_threshold > 0.0f;
  const float m = st->cfg.momentum;
  const int parity = (int)(st->iterations & 1);
  const uint64_t call_seed = st->cfg.seed * 0x9E3779B97F4A7C15ull + (uint64_t)st->iterations;
  int32_t rc;
  if (clip) {
    const double thr_local =
        (double)st->cfg.clip_threshold / std::sqrt((double)st->cfg.num_workers);
    k_sumsq<<<st->norm_grid, kNormThreads, 0, s>>>(p, grad_arena, thr_local, 1);
    if ((rc = check_launch()) != DGC_OK) return rc;
  }
  if (!st->sampled.empty()) {
    const int grid = (int)st->sampled.size();
    const size_t smem = (size_t)st->max_sample_keys * 4;
    if (clip) k_sample_threshold<true><<<grid, kSampleThreads, smem, s>>>(p, grad_arena, m, call_seed);
    else k_sample_threshold<false><<<grid, kSampleThreads, smem, s>>>(p, grad_arena, m, call_seed);
    if ((rc = check_launch()) != DGC_OK) return rc;
  }
  {
    const bool prof = st->prof_n < st->prof_cap;
    if (prof) DGC_CUDA(cudaEventRecord(st->prof_ev[2 * st->prof_n], s));
    const int need = (p.num_segs + (kMainThreads / 32) - 1) / (kMainThreads / 32);
    if (clip) k_update_emit<true><<<std::min(st->main_grid_clip, need), kMainThreads, 0, s>>>(p, grad_arena, m);
    else k_update_emit<false><<<std::min(st->main_grid, need), kMainThreads, 0, s>>>(p, grad_arena, m);
    if ((rc = check_launch()) != DGC_OK) return rc;
    if (prof) {
      DGC_CUDA(cudaEventRecord(st->prof_ev[2 * st->prof_n + 1], s));
      st->prof_n += 1;
    }
  }
  k_select<<<p.num_tensors, kSelectThreads, (size_t)st->select_smem_keys * 4, s>>>(
      p, st->select_smem_keys, parity);
  if ((rc = check_launch()) != DGC_OK) return rc;
  k_emit_mask<<<p.num_parts, kEmitThreads, kEmitSmemBytes, s>>>(p, out_idx, out_val);
  if ((rc = check_launch()) != DGC_OK) return rc;
  st->iterations += 1;
  return DGC_OK;
}

int32_t dgc_compress_host(dgc_state* st, const float* grad_host, int32_t* out_idx_host,
                          float* out_val_host, int64_t capacity, void* stream) {
  if (!st || !st->alive) return DGC_ESTATE;
  if (!grad_host || !out_idx_host || !out_val_host) return DGC_EINVAL;
  if (capacity < st->max_nnz) return DGC_ECAPACITY;
  DGC_CUDA(cudaSetDevice(st->device));
  cudaStream_t s = as_stream(stream);
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

int64_t dgc_decode_workspace_bytes(int32_t num_workers, int64_t dense_len) {
  if (num_workers < 1 || num_workers > DGC_MAX_DECODE_WORKERS || dense_len < 0) return DGC_EINVAL;
  const int64_t tiles = (dense_len + kDecodeTile - 1) / kDecodeTile;
  return (int64_t)num_workers * (tiles + 1) * 4;
}

int32_t dgc_decode_accumulate(int32_t num_workers, const int32_t* const* idx_lists,
                              const float* const* val_lists, const int64_t* nnz, float* dense_out,
                              int64_t dense_len, void* workspace, int64_t workspace_bytes,
                              void* stream) {
  if (num_workers < 1 || num_workers > DGC_MAX_DECODE_WORKERS) return DGC_EINVAL;
  if (!idx_lists || !val_lists || !nnz || dense_len < 0 || dense_len >= (int64_t)1 << 31)
    return DGC_EINVAL;
  if (dense_len == 0) return DGC_OK;
  if (!dense_out || !workspace) return DGC_EINVAL;
  if ((reinterpret_cast<uintptr_t>(dense_out) & 15u) != 0) return DGC_EINVAL;
  if (workspace_bytes < dgc_decode_workspace_bytes(num_workers, dense_len)) return DGC_ECAPACITY;
  DecodeArgs a{};
  int64_t max_nnz = 0;
  for (int w = 0; w < num_workers; ++w) {
    if (nnz[w] < 0 || nnz[w] > dense_len) return DGC_EINVAL;
    if (nnz[w] > 0 && (!idx_lists[w] || !val_lists[w])) return DGC_EINVAL;
    a.idx[w] = idx_lists[w];
    a.val[w] = val_lists[w];
    a.nnz[w] = (int32_t)nnz[w];
    max_nnz = std::max(max_nnz, nnz[w]);
  }
  a.num_workers = num_workers;
  a.num_tiles = (int32_t)((dense_len + kDecodeTile - 1) / kDecodeTile);
  cudaStream_t s = as_stream(stream);
  int32_t rc;
  const int gx = (int)std::min<int64_t>((max_nnz + 1 + 255) / 256, 1024);
  k_decode_bounds<<<dim3(gx, num_workers), 256, 0, s>>>(a, (int32_t*)workspace);
  if ((rc = check_launch()) != DGC_OK) return rc;
  k_decode_tiles<<<a.num_tiles, kDecodeThreads, 0, s>>>(a, (const int32_t*)workspace, dense_out,
                                                       dense_len);
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
  k_sgd<<<grid, 256, 0, as_stream(stream)>>>(w, dense_grad, len, lr);
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
  const int parity = (int)((st->iterations + 1) & 1);   // parity of the last call
  const bool clip = st->cfg.clip_threshold > 0.0f;
  out->grad_norm = clip ? norm : 0.0;
  out->clip_coef = clip ? coef : 1.0f;
  out->flags = (int32_t)(diag[parity * 4 + 0] & 0xF);
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

int32_t dgc_profile_enable(dgc_state* st, int32_t max_calls) {
  if (!st || !st->alive) return DGC_ESTATE;
  if (max_calls < 0) return DGC_EINVAL;
  DGC_CUDA(cudaSetDevice(st->device));
  while ((int)st->prof_ev.size() < 2 * max_calls) {
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
    DGC_CUDA(cudaEventSynchronize(st->prof_ev[2 * i + 1]));
    DGC_CUDA(cudaEventElapsedTime(&ms_out[i], st->prof_ev[2 * i], st->prof_ev[2 * i + 1]));
  }
  *count_out = n;
  return DGC_OK;
}

int32_t dgc_state_read(dgc_state* st, float* u_host, float* v_host, void* stream) {
  if (!st || !st->alive) return DGC_ESTATE;
  cudaStream_t s = as_stream(stream);
  const size_t bytes = (size_t)st->arena_len * 4;
  if (u_host) DGC_CUDA(cudaMemcpyAsync(u_host, st->plan.u, bytes, cudaMemcpyDeviceToHost, s));
  if (v_host) DGC_CUDA(cudaMemcpyAsync(v_host, st->plan.v, bytes, cudaMemcpyDeviceToHost, s));
  DGC_CUDA(cudaStreamSynchronize(s));
  return DGC_OK;
}

int32_t dgc_state_write(dgc_state* st, const float* u_host, const float* v_host, void* stream) {
  if (!st || !st->alive) return DGC_ESTATE;
  cudaStream_t s = as_stream(stream);
  const size_t bytes = (size_t)st->arena_len * 4;
  if (u_host) DGC_CUDA(cudaMemcpyAsync(st->plan.u, u_host, bytes, cudaMemcpyHostToDevice, s));
  if (v_host) DGC_CUDA(cudaMemcpyAsync(st->plan.v, v_host, bytes, cudaMemcpyHostToDevice, s));
  DGC_CUDA(cudaStreamSynchronize(s));
  return DGC_OK;
}

}  // extern "C"
