// sm_100a kernels of the Deep Gradient Compression hot path (device code only;
// the host side and the C ABI are in dgc.cu).
//
// One dgc_compress call = one iteration of Algorithm 4 (Appendix D) on one
// worker, as stream-ordered launches over a padded fp32 arena:
//
//   k_sumsq            (only when clipping)  Sec. 3.2 / App. C: ||g||_2 in fp64, coef
//   k_sample_threshold Sec. 5: seeded sample of |v'| -> proposed threshold per tensor
//   k_update_emit      Eq. 5: u' = m u + g coef, v' = v + u', stored once; entries whose
//                      |v'| reaches the proposal are compacted, in index order per
//                      512-element segment, into their part's candidate list
//   k_select           exact k-th largest |v'| among a tensor's candidates (radix
//                      select on the IEEE bit pattern), tie quota, per-part output bases
//   k_big_hist<0..2>,  the same selection for tensors whose candidates do not fit one block
//   k_big_final        (warm-up sparsities, very large tensors): three histogram rounds
//   k_emit_mask        Alg. 4 "G~ <- V (.) Mask", Sec. 3.3 masking: ordered (index, value)
//                      pairs; u = v = 0 at the sent entries, either at once or (low
//                      sparsity) recorded as bits that the next call's kernels apply
//
// The sample only proposes; if a proposal lets fewer than k_j entries or more
// than the list capacity through, that tensor is selected from the whole of v'
// instead (same result, slower).  All fp32 arithmetic uses explicit
// round-to-nearest intrinsics so that no FMA contraction can change a bit.
//
// The tail kernels (sample, select, emit) touch little data; their cost is the
// number of dependent global-memory round trips and block barriers on their
// critical path, so tables are packed into 16/32-byte records fetched with one
// load and the shared-memory phases are kept to two barriers per radix pass.
//
// Receive side: k_decode_bounds + k_decode_tiles (Alg. 4 aggregation line) and
// k_sgd (Alg. 4 update line).
#pragma once

#include <cooperative_groups.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "dgc.h"

namespace dgc {

// ------------------------------------------------------------------ constants
constexpr int kSeg = 512;              // elements per warp segment (4 x float4 per lane)
constexpr int kPartSegs = 512;         // segments per part (256 Ki elements)
constexpr int kSmallN = 8192;          // tensors up to this size are not sampled
constexpr int kMaxSampleGroups = 16384; // float4 groups sampled per tensor at most
constexpr int kSampleThreads = 512;    // one sampled float4 group per thread and block
static_assert(kMaxSampleGroups <= 32 * kSampleThreads,
              "exact mode: at most 32 sampling blocks per tensor, one warp scans their counts");
constexpr int kSampleSurvivors = 4096;
constexpr int kSelectThreads = 1024;
constexpr int kSelectBatchThreads = 512;   // k_select in a batch of several workers
constexpr int kSelectMaxSmemKeys = 51200;
constexpr int kSelectMaxParts = 256;   // parts of one tensor whose tables fit in shared memory
constexpr int kClusterSize = 8;        // k_select_cluster: blocks (SMs) that share one tensor
constexpr int kClusterThreads = 512;
constexpr int kClusterMinParts = 8;    // tensors of at least this many parts use the whole cluster
constexpr int kEmitThreads = kPartSegs;   // one thread per segment of the part
constexpr int kEmitRegs = 8;              // candidates per thread kept in registers
constexpr int kMaskStride = 17;           // words per segment in the winner bitmaps (16 + 1 pad)
constexpr int kEmitSmemBytes = 2 * kPartSegs * kMaskStride * 4;
constexpr int kDenseChunk = 64;            // segments per chunk of k_emit_dense (128 KiB of v')
constexpr double kDenseEmitFraction = 1.0 / 8.0;   // share of entries sent from which k_emit_dense runs
constexpr int kMainThreads = 256;
constexpr int kNormThreads = 256;
constexpr int kMaxNormGrid = 2048;
constexpr int kBigThreads = 512;
constexpr int kBigBins = 2048;         // 11-bit digits: key bits 30..20, 19..9, then 9 bits 8..0
constexpr int kBigLastBins = 512;
constexpr int kBigLastStride = 516;    // 513 suffix sums, padded to a multiple of 4 words
constexpr int kBigStateWords = 64;
constexpr int kBigNear = 64;           // round-0 digits this close above the proposal's get private bins
constexpr int kDecodeTile = 4096;
constexpr int kDecodeThreads = 256;

// ------------------------------------------------------------------ plan tables
struct __align__(16) TensorMeta {   // one per tensor, read-only for the kernels
  int32_t off, end;                 // arena range of the real elements
  int32_t k, out_off;               // entries to send, first output slot
  int32_t part_first, part_num;
  int32_t rank, groups;             // sampling: rank of the proposal, float4 groups sampled
  int32_t key_base, chunks;         // sampling: first key in the sample buffer, blocks that sample
  int32_t big, big_slot;            // big: selected by the multi-block path; slot in its tables
  int32_t samples;                  // paper-literal mode: elements drawn (4 per group, the last
                                    // group may be short); otherwise unused
  int32_t rank_local;               // keys each sampling block of the tensor keeps for the merge
  int32_t pad_[2];
};
struct __align__(16) SampleBlock {   // work item of one k_sample_threshold block: its tensor's
  TensorMeta t;                      // record travels with it (one round trip instead of two)
  int32_t tensor, chunk;
  int32_t pad_[2];
};
struct __align__(16) PartMeta {     // one per part (up to kPartSegs segments of one tensor)
  int32_t tensor, end;              // end: arena index one past the part's last real element
  int32_t seg0, nseg;
  int32_t cbase, cap;               // candidate list of the part
  int32_t first, big_slot;          // first: the tensor's first part; slot among the big parts or -1
};
struct __align__(16) PartSel {      // written by k_select, read by k_emit_mask
  uint32_t kth;                     // bit pattern of the k-th largest |v'| of the tensor
  int32_t quota;                    // entries tied with kth that this part sends
  int32_t out_base;                 // first output slot of this part
  int32_t dense;                    // 1: tensor takes the full-selection path
};

struct Plan {
  const TensorMeta* tm;
  const PartMeta* pm;
  PartSel* psel;
  int32_t* p_count;          // candidates appended per part (reset by k_emit_mask)
  uint32_t* p_thr;           // proposed threshold per part (0 for tensors that are not sampled)
  uint32_t* p_tie;           // per part, written with p_thr: 1 if the sample held its rank-th
                             // key more than once (masses of equal magnitudes are possible):
                             // only then does k_update_emit count the part's tied entries
  int32_t* p_eq;             // entries per part whose key is p_thr - 1, the sample's rank-th key
                             // (counted by k_update_emit, reset by k_emit_mask): what completes
                             // the list when fewer than k entries exceed that key
  int32_t* t_nnz;            // per tensor: entries sent by the last call (paper-literal mode)
  int32_t literal;           // 1: paper-literal sampled selection (Sec. 5), variable count
  uint32_t* t_kth;           // per tensor: threshold of the last call (reporting)
  int32_t* t_cand;           // per tensor: candidates of the last call, -1 = full selection
  const int32_t* seg_part;   // part of every segment
  const SampleBlock* sample_blocks;
  uint32_t* sample_keys;     // per sampling block: the keys it kept for its tensor's merge
  uint32_t* sample_all;      // |v'| keys of the current call's whole sample, all tensors
  int32_t* sample_ticket;    // per tensor: sampling blocks that have finished
  int32_t* sample_cnt;       // per sampling block: keys it kept in its slice of sample_keys
  // multi-block selection (tensors with too many candidates for one block)
  const int32_t* big_parts;  // parts of the big tensors
  const int32_t* big_tensors;
  int32_t* big_hist;         // [big tensor][3][2048] digit histograms of the three rounds
  int32_t* big_state;        // [big tensor][64]: prefix and remaining rank after round 0 (words
                             // 0,1) and after round 1 (words 32,33: a cache line of their own)
  int32_t* big_above;        // [big part]: candidates whose upper 22 key bits exceed the prefix
  int32_t* big_last;         // [big part][513]: suffix sums of the part's last-round digit
                             // counts: word d = candidates matching the prefix with digit >= d
  int32_t* cand_idx;
  float* cand_val;
  float* coef;
  double* norm;
  // clipping per tensor (clip_scope = 1): every tensor by its own norm
  int32_t clip_scope;
  double* seg_sumsq;         // [segment] sum of squares of the segment's real elements
  double* t_norm;            // [tensor] L2 norm of the tensor's gradient
  float* t_coef;             // [tensor] coefficient applied to it
  double* partials;
  unsigned int* ticket;
  long long* diag;           // [2][4]: flags, full_select, candidates, unused
  long long* iter;           // compress calls completed on this state: the kernels take the
                             // sampling seed and the counter bank from it, so that a captured
                             // call replays correctly; k_emit_mask advances it
  float* u;
  float* v;
  // deferred masking (low sparsity): k_emit_mask records the sent entries as one bit each and
  // the next call's kernels zero u and v at those entries in registers before using them
  uint32_t* sent_bits;       // arena_len / 32 words, 16 per segment
  int32_t defer_mask;        // 1: masking is deferred through sent_bits
  unsigned long long* timeline;   // measurement aid, NULL = off: per kernel of the call (sampling,
                             // streaming, selection, emission) the earliest and the latest
                             // block start on the GPU's nanosecond timer
  int32_t dense_emit;        // 1 (only with defer_mask): k_emit_dense emits from v' itself and
                             // the candidate indices are not written
  int32_t num_tensors, num_parts, num_segs;
  int32_t num_big_parts, num_big_tensors;
};

template <class T>
__device__ __forceinline__ T load_record(const T* ptr) {
  static_assert(sizeof(T) % 16 == 0, "records are whole int4s");
  T out;
  const int4* src = reinterpret_cast<const int4*>(ptr);
  int4* dst = reinterpret_cast<int4*>(&out);
#pragma unroll
  for (int i = 0; i < (int)(sizeof(T) / 16); ++i) dst[i] = __ldcg(src + i);
  return out;
}

// ------------------------------------------------------------------ device helpers
// Programmatic dependent launch: every kernel of the library is launched with the
// programmatic-serialization attribute and starts with pdl_enter().  The wait returns once
// the preceding kernel in the stream has completed and its writes are visible, so the order
// of the stream is kept; what is gained is that this kernel's launch was processed while the
// predecessor still ran, which hides the launch latency between the short kernels.  No kernel
// signals early (griddepcontrol.launch_dependents): blocks that sit on an SM waiting for a
// long predecessor would take the slots that another stream's streaming kernel needs (measured:
// 10 % slower steps with early signalling).  The wait is executed by every block, so that
// "grid N has completed" still implies "grid N-1 has completed".
__device__ __forceinline__ void pdl_enter() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Timeline aid: every block of the four kernels of a compress call notes when it started.
__device__ __forceinline__ void timeline_mark(unsigned long long* tl, int kernel) {
  if (tl != nullptr && threadIdx.x == 0) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    atomicMin(tl + 2 * kernel, t);
    atomicMax(tl + 2 * kernel + 1, t);
  }
}

__device__ __forceinline__ uint32_t mag_key(float x) { return __float_as_uint(x) & 0x7FFFFFFFu; }

// One 4-byte word from global to shared memory without passing through a register
// (cp.async); stage_wait() makes this thread's copies complete (a barrier then publishes them).
__device__ __forceinline__ void stage_word(void* smem_dst, const void* gmem_src) {
  const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void stage_wait() {
  asm volatile("cp.async.commit_group;" ::: "memory");
  asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// One element of the accumulation, every operation rounded once.
// Eq. 5 / Algorithm 4:           gc = g*coef ; u <- m*u + gc ; v <- v + u
// Algorithm 5 (NEST, Appendix B): gc = g*coef ; u <- m*(u + gc) ; v <- (v + u) + gc
template <bool CLIP, bool NEST>
__device__ __forceinline__ void mc_step(float g, float coef, float m, float& u, float& v) {
  const float gc = CLIP ? __fmul_rn(g, coef) : g;
  if (NEST) {
    u = __fmul_rn(m, __fadd_rn(u, gc));
    v = __fadd_rn(__fadd_rn(v, u), gc);
  } else {
    u = __fadd_rn(__fmul_rn(m, u), gc);
    v = __fadd_rn(v, u);
  }
}

__device__ __forceinline__ uint64_t mix64(uint64_t x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}

__device__ __forceinline__ int warp_incl_scan(int x) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xFFFFFFFFu, x, o);
    if (lane >= o) x += t;
  }
  return x;
}

// Block-wide exclusive scan of two ints per thread (a, b); returns the
// exclusive prefixes and the block totals.  `sh` needs 66 ints.  Two barriers;
// a third is needed before `sh` is reused.
__device__ __forceinline__ void block_excl_scan2(int a, int b, int* sh, int& ea, int& eb, int& ta,
                                                 int& tb) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const int ia = warp_incl_scan(a), ib = warp_incl_scan(b);
  if (lane == 31) { sh[warp] = ia; sh[33 + warp] = ib; }
  __syncthreads();
  if (warp == 0) {
    const int wa = lane < nwarps ? sh[lane] : 0, wb = lane < nwarps ? sh[33 + lane] : 0;
    const int sa = warp_incl_scan(wa), sb = warp_incl_scan(wb);
    sh[lane] = sa - wa;
    sh[33 + lane] = sb - wb;
    if (lane == 31) { sh[32] = sa; sh[65] = sb; }
  }
  __syncthreads();
  ea = sh[warp] + ia - a;
  eb = sh[33 + warp] + ib - b;
  ta = sh[32];
  tb = sh[65];
}

// Radix select, descending: the `rank`-th largest key (rank >= 1) among the
// keys the iterator visits.  `for_each(f)` must call f(valid, key) the same
// number of times on every thread of the block (valid = false for padding
// calls).  Every valid key lies in [base, maxkey]; only the bits in which
// maxkey - base can differ are scanned, 8 per pass from the top.
// Histograms: up to 16 private 256-bin copies (padded to 257 words so that the
// same bin of different copies falls in different banks), one per warp or pair
// of warps, so that the integer atomics of different warps do not collide;
// they are folded into one of two alternating 256-bin histograms, in which
// warp 0 finds the digit.  hist: kHistWords(blockDim.x) words of shared
// memory, sh: 3 words.  blockDim.x is a multiple of 256.
// Returns the key; n_gt = number of keys strictly greater.
// One warp: in a 256-bin histogram h of digit counts, the digit (from the largest) at which the
// cumulative count reaches `remaining` -> sh[0]; keys in larger digits -> sh[1]; keys in that
// digit -> sh[2].
__device__ __forceinline__ void warp_find_digit(const uint32_t* h, int remaining, int* sh) {
  const int lane = threadIdx.x & 31;
  const int hi = 255 - 8 * lane;          // this lane covers bins hi, hi-1, .., hi-7
  uint32_t loc[8];
  uint32_t s = 0;
#pragma unroll
  for (int q = 0; q < 8; ++q) { loc[q] = h[hi - q]; s += loc[q]; }
  const uint32_t incl = (uint32_t)warp_incl_scan((int)s);
  const uint32_t excl = incl - s;
  if (excl < (uint32_t)remaining && (uint32_t)remaining <= incl) {
    uint32_t c = excl;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      if (c + loc[q] >= (uint32_t)remaining) {
        sh[0] = hi - q;
        sh[1] = (int)c;
        sh[2] = (int)loc[q];     // after the last pass: keys equal to the result
        break;
      }
      c += loc[q];
    }
  }
}

__host__ __device__ constexpr int kHistCopies(int threads) { return threads / 32 < 16 ? threads / 32 : 16; }
__host__ __device__ constexpr int kHistWords(int threads) { return kHistCopies(threads) * 257 + 512; }

// PRIVATE = false skips the private copies (and the fold with its barrier): for a handful of
// keys per block the atomics hardly collide and the fixed cost per pass is what counts.
// max_passes < 4 stops after that many digits and returns the lower edge of the bin that holds
// the result (a lower bound that at least `rank` keys reach), for callers that only filter.
template <int THREADS, bool PRIVATE = true, class ForEach>
__device__ __forceinline__ uint32_t block_select_desc(ForEach for_each, int rank, uint32_t base,
                                                      uint32_t maxkey, uint32_t* hist, int* sh,
                                                      int& n_gt, int* n_eq = nullptr,
                                                      int max_passes = 4) {
  // THREADS = blockDim.x, a compile-time constant so that the slicing below costs no divisions
  constexpr int nt = THREADS;
  const int tid = threadIdx.x;
  constexpr int copies = kHistCopies(nt);
  uint32_t* mine = hist + ((tid >> 5) % copies) * 257;
  uint32_t* folded = hist + copies * 257;
  const uint32_t span = maxkey - base;
  const int passes = span == 0 ? 0 : (32 - __clz(span) + 7) / 8;
  uint32_t prefix = 0, mask = 0;
  int remaining = rank;
  if (PRIVATE) {
    for (int i = tid; i < copies * 257 + 512; i += nt) hist[i] = 0;
  } else {
    for (int i = tid; i < 512; i += nt) folded[i] = 0;
  }
  __syncthreads();
  int cur = 0;
  const int last_shift = 8 * max(passes - max_passes, 0);
  for (int shift = 8 * (passes - 1); shift >= last_shift; shift -= 8, cur ^= 1) {
    uint32_t* target = PRIVATE ? mine : folded + cur * 256;
    for_each([&](bool valid, uint32_t key) {
      key -= base;
      if (valid && (key & mask) == prefix) atomicAdd(&target[(key >> shift) & 255u], 1u);
    });
    __syncthreads();
    if (PRIVATE) {
      // fold (and clear) the private copies: thread t takes bin t & 255 of a slice of them
      constexpr int groups = nt >> 8;
      const int bin = tid & 255, grp = tid >> 8;
      const int c0 = grp * copies / groups, c1 = (grp + 1) * copies / groups;
      uint32_t t = 0;
      for (int c = c0; c < c1; ++c) {
        t += hist[c * 257 + bin];
        hist[c * 257 + bin] = 0;
      }
      if (t) atomicAdd(&folded[cur * 256 + bin], t);
      __syncthreads();
    }
    if (tid < 32) {
      warp_find_digit(folded + cur * 256, remaining, sh);
    } else {
      // the other warps clear the other histogram for the next pass
      for (int i = tid - 32; i < 256; i += nt - 32) folded[(cur ^ 1) * 256 + i] = 0;
    }
    __syncthreads();
    prefix |= (uint32_t)sh[0] << shift;
    mask |= 255u << shift;
    remaining -= sh[1];
  }
  n_gt = rank - remaining;
  // keys equal to the result: the chosen bin of the last pass (no pass: every key is maxkey)
  if (n_eq) *n_eq = passes == 0 ? 0x7FFFFFFF : sh[2];
  return base + prefix;
}

// ------------------------------------------------------------------ K1: clipping norm
// Sec. 3.2 / Appendix C.  Sum of squares of every real element of the gradient
// set: fp32 loads, exact fp64 products, fp64 accumulation; fixed reduction
// tree (grid size fixed per state), so the result does not depend on timing.
// The last block to finish folds the partials and writes norm and coef.
__global__ void __launch_bounds__(kNormThreads)
k_sumsq(Plan p, const float* __restrict__ g, double thr_local, int clip_on) {
  pdl_enter();
  __shared__ double swarp[kNormThreads / 32];
  __shared__ bool is_last;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int warps_total = gridDim.x * (kNormThreads / 32);
  const float4* g4 = reinterpret_cast<const float4*>(g);
  double acc = 0.0;
  for (int seg = blockIdx.x * (kNormThreads / 32) + warp; seg < p.num_segs; seg += warps_total) {
    const int base = seg * kSeg;
    float4 x[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) x[i] = __ldg(g4 + (base >> 2) + i * 32 + lane);
    const int part = __ldg(p.seg_part + seg);
    const int end = __ldg(&p.pm[part].end);
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

// Clipping per tensor (clip_scope = 1), two launches with a fixed summation order each:
// k_sumsq_segments: one warp per 512-element segment, fp64 sum of squares of its real elements;
// k_tensor_coef: one block per tensor folds its segments' sums, writes the tensor's norm and
// its coefficient thr_local / norm (1 unless the norm exceeds thr_local).
__global__ void __launch_bounds__(kNormThreads)
k_sumsq_segments(Plan p, const float* __restrict__ g) {
  pdl_enter();
  const int lane = threadIdx.x & 31;
  const int seg = blockIdx.x * (kNormThreads / 32) + (threadIdx.x >> 5);
  if (seg >= p.num_segs) return;
  const float4* g4 = reinterpret_cast<const float4*>(g);
  const int base = seg * kSeg;
  float4 x[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) x[i] = __ldg(g4 + (base >> 2) + i * 32 + lane);
  const int end = __ldg(&p.pm[__ldg(p.seg_part + seg)].end);
  double acc = 0.0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int e = base + (i * 32 + lane) * 4;
    if (e + 0 < end) acc += (double)x[i].x * (double)x[i].x;
    if (e + 1 < end) acc += (double)x[i].y * (double)x[i].y;
    if (e + 2 < end) acc += (double)x[i].z * (double)x[i].z;
    if (e + 3 < end) acc += (double)x[i].w * (double)x[i].w;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
  if (lane == 0) p.seg_sumsq[seg] = acc;
}

__global__ void __launch_bounds__(kNormThreads)
k_tensor_coef(Plan p, double thr_local) {
  pdl_enter();
  __shared__ double swarp[kNormThreads / 32];
  const int j = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const TensorMeta t = load_record(p.tm + j);
  const int s0 = t.off / kSeg, s1 = (t.end + kSeg - 1) / kSeg;
  double s = 0.0;
  for (int i = s0 + threadIdx.x; i < s1; i += kNormThreads) s += __ldcg(p.seg_sumsq + i);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
  if (lane == 0) swarp[warp] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    double S = 0.0;
    for (int w = 0; w < kNormThreads / 32; ++w) S += swarp[w];
    const double norm = sqrt(S);
    p.t_norm[j] = norm;
    p.t_coef[j] = norm > thr_local ? (float)(thr_local / norm) : 1.0f;
  }
}

// ------------------------------------------------------------------ K2: sampled threshold proposal
// Sec. 5: sample |v'| (v' computed on the fly from g, u, v exactly as the main
// pass will), take the sample's rank-r key as the proposed threshold of the
// tensor.  One float4 group per stratum at a hashed position.  The scattered
// 16-byte loads are what costs, so a tensor's strata are spread over several
// blocks (kSampleThreads groups each, one per thread); each block writes its
// keys to a buffer and the last block of the tensor to finish (integer ticket)
// selects.  r is small against the sample, so that block first bounds the
// answer from below by the rank-r of the per-thread maxima (at least r keys
// reach it), keeps the few keys that reach the bound and selects among them.
// LITERAL (Sec. 5 taken literally, select_mode 1): the sample is `samples` independent uniform
// draws of single elements, draw r of tensor j at floor(h n / 2^64), h = mix64(call seed xor
// (j << 32) xor r); a thread takes draws 4s .. 4s + 3.  Draws beyond `samples` count as key 0,
// which cannot move the rank-th largest key (rank <= samples).
// (Capping the registers at 32 for a fourth block per SM was measured: the spills cost more
// than the slot gains, 0.776 -> 0.785 ms per batched step.)
template <bool CLIP, bool NEST, bool LITERAL>
__global__ void __launch_bounds__(kSampleThreads)
k_sample_threshold(Plan p, const float* __restrict__ g, float m, uint64_t seed_base) {
  pdl_enter();
  timeline_mark(p.timeline, 0);
  // hashed, so that consecutive calls draw unrelated positions
  const uint64_t call_seed = mix64(seed_base + (uint64_t)__ldcg(p.iter));
  __shared__ uint32_t hist[kHistWords(kSampleThreads)];
  // the survivors share the private histogram copies' words: wherever survivors are kept the
  // selections run without private copies (only the last 512 words of hist are in use)
  uint32_t* surv = hist;
  static_assert(kSampleSurvivors <= kHistCopies(kSampleThreads) * 257, "survivors alias the copies");
  __shared__ int sh[66];
  __shared__ int s_cnt;
  __shared__ uint32_t s_max, s_min;
  __shared__ int s_last;
  const int tid = threadIdx.x, lane = tid & 31;
  const SampleBlock sb = load_record(p.sample_blocks + blockIdx.x);
  const int j = sb.tensor;
  const TensorMeta& t = sb.t;
  const int G = t.groups, rank = t.rank;
  uint4* gkeys = reinterpret_cast<uint4*>(p.sample_all + t.key_base);
  uint4 mykeys = make_uint4(0u, 0u, 0u, 0u);
  bool have = false;
  {
    const int s = sb.chunk * kSampleThreads + tid;
    if (LITERAL && s < G) {
      const float coef = CLIP ? __ldcg(p.clip_scope ? p.t_coef + j : p.coef) : 1.0f;
      const uint64_t n = (uint64_t)(uint32_t)(t.end - t.off);
      uint32_t karr[4] = {0u, 0u, 0u, 0u};
      uint32_t at[4];
      float gg[4], uu[4], vv[4];
      uint32_t sent[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const uint32_t r = 4u * (uint32_t)s + (uint32_t)c;
        const uint64_t h = mix64(call_seed ^ ((uint64_t)(uint32_t)j << 32) ^ (uint64_t)r);
        // (draws past the sample read position 0 of the tensor and are discarded)
        at[c] = (uint32_t)t.off + ((int)r < t.samples ? (uint32_t)__umul64hi(h, n) : 0u);
      }
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        gg[c] = __ldg(g + at[c]);
        uu[c] = __ldcg(p.u + at[c]);
        vv[c] = __ldcg(p.v + at[c]);
        sent[c] = p.defer_mask ? __ldcg(p.sent_bits + (at[c] >> 5)) : 0u;
      }
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        if ((sent[c] >> (at[c] & 31u)) & 1u) { uu[c] = 0.0f; vv[c] = 0.0f; }   // pending masking
        mc_step<CLIP, NEST>(gg[c], coef, m, uu[c], vv[c]);
        if ((int)(4u * (uint32_t)s + (uint32_t)c) < t.samples) karr[c] = mag_key(vv[c]);
      }
      mykeys = make_uint4(karr[0], karr[1], karr[2], karr[3]);
      have = true;
    } else if (!LITERAL && s < G) {
      const uint32_t W = (uint32_t)((t.end - t.off) >> 2) / (uint32_t)G;   // groups per stratum
      const float coef = CLIP ? __ldcg(p.clip_scope ? p.t_coef + j : p.coef) : 1.0f;
      // stratum s = groups [s*W, (s+1)*W); position inside it from a hash (multiply-high
      // instead of a modulo); the < G groups after the last stratum are never sampled
      const uint32_t h =
          (uint32_t)mix64(call_seed ^ ((uint64_t)(uint32_t)j << 32) ^ (uint64_t)(uint32_t)s);
      const uint32_t pos = (uint32_t)(t.off >> 2) + (uint32_t)s * W + __umulhi(h, W);
      const float4 gg = __ldg(reinterpret_cast<const float4*>(g) + pos);
      float4 u = __ldcg(reinterpret_cast<const float4*>(p.u) + pos);
      float4 v = __ldcg(reinterpret_cast<const float4*>(p.v) + pos);
      if (p.defer_mask) {
        // entries sent by the previous call are still to be zeroed
        const uint32_t nib = (__ldcg(p.sent_bits + (pos >> 3)) >> ((pos & 7u) * 4u)) & 0xFu;
        if (nib & 1u) { u.x = 0.0f; v.x = 0.0f; }
        if (nib & 2u) { u.y = 0.0f; v.y = 0.0f; }
        if (nib & 4u) { u.z = 0.0f; v.z = 0.0f; }
        if (nib & 8u) { u.w = 0.0f; v.w = 0.0f; }
      }
      mc_step<CLIP, NEST>(gg.x, coef, m, u.x, v.x);
      mc_step<CLIP, NEST>(gg.y, coef, m, u.y, v.y);
      mc_step<CLIP, NEST>(gg.z, coef, m, u.z, v.z);
      mc_step<CLIP, NEST>(gg.w, coef, m, u.w, v.w);
      mykeys = make_uint4(mag_key(v.x), mag_key(v.y), mag_key(v.z), mag_key(v.w));
      have = true;
    }
  }
  // Tensors sampled by several blocks: every block keeps only the keys that can be among the
  // tensor's `rank` largest -- its own `rank` largest (and their ties), zeros never -- and
  // writes them packed into its slice; the last block then selects among a few thousand keys
  // instead of re-reading the whole sample.  (If fewer than `rank` keys of the sample are
  // non-zero the union is short and the answer is 0.)
  // (larger ranks: tiny samples, or the large samples of the paper-literal mode, which can also
  // spread over more blocks than the one block scan of the blocks' counts covers)
  const bool local = t.chunks > 1 && t.chunks <= kSampleThreads && rank <= kSampleThreads;
  if (local) {
    uint32_t* slice = p.sample_keys + t.key_base + sb.chunk * (4 * kSampleThreads);
    const int nv = min(kSampleThreads, G - sb.chunk * kSampleThreads);   // threads with a group
    const uint32_t tmax = have ? max(max(mykeys.x, mykeys.y), max(mykeys.z, mykeys.w)) : 0u;
    if (tid == 0) { s_cnt = 0; s_max = 0u; }
    __syncthreads();
    uint32_t low = 1u;                             // zeros are never kept: see the union below
    // A block keeps its rank_local largest keys.  With rank_local = rank the union of the
    // blocks' lists surely holds the tensor's `rank` largest.  The exact mode keeps fewer -- the
    // share a block can expect of them plus a wide margin -- so that the merge handles a few
    // hundred keys instead of thousands; should a block have held more of them than that, the
    // merged key comes out a little low, which only lets a few more candidates through.
    const int rloc = t.rank_local;
    if (rloc < rank && have) gkeys[sb.chunk * kSampleThreads + tid] = mykeys;   // (see the merge)
    if (rloc <= 4 * nv) {
      const uint32_t wmax = __reduce_max_sync(0xFFFFFFFFu, tmax);
      if (lane == 0) atomicMax(&s_max, wmax);
      __syncthreads();
      int n_gt_local;
      low = max(1u, block_select_desc<kSampleThreads, false>(
                        [&](auto f) {
                          f(have, mykeys.x);
                          f(have, mykeys.y);
                          f(have, mykeys.z);
                          f(have, mykeys.w);
                        },
                        rloc, 0u, s_max, hist, sh, n_gt_local, nullptr, 2));
      // (two digits = 16 bits below the block's largest key: the bound is within 0.4 % of the
      // block's rloc-th key, the list a few keys longer, the block two radix passes shorter)
    }
    const uint32_t karr[4] = {mykeys.x, mykeys.y, mykeys.z, mykeys.w};
    if (__any_sync(0xFFFFFFFFu, have && tmax >= low)) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const bool keep = have && karr[c] >= low;
        const unsigned mk = __ballot_sync(0xFFFFFFFFu, keep);
        if (mk) {
          int basepos = 0;
          if (lane == __ffs(mk) - 1) basepos = atomicAdd(&s_cnt, __popc(mk));
          basepos = __shfl_sync(0xFFFFFFFFu, basepos, __ffs(mk) - 1);
          if (keep) slice[basepos + __popc(mk & ((1u << lane) - 1u))] = karr[c];
        }
      }
    }
    __syncthreads();
    if (tid == 0) p.sample_cnt[blockIdx.x] = s_cnt;
  } else if (have) {
    gkeys[sb.chunk * kSampleThreads + tid] = mykeys;
  }
  if (t.chunks > 1) {
    __threadfence();
    __syncthreads();
    if (tid == 0) {
      const int done = atomicAdd(p.sample_ticket + j, 1);
      s_last = done == t.chunks - 1;
      if (s_last) p.sample_ticket[j] = 0;       // ready for the next call
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
  }
  int n_gt, n_eq = 0;
  uint32_t kth = 0;
  bool done = false;
  if (local) {
    // the union of the blocks' slices: counts -> offsets (at most 32 blocks per tensor)
    __shared__ int s_off[kSampleThreads + 1];
    const int first = blockIdx.x - sb.chunk;
    if (tid == 0) { s_max = 0u; s_min = 0xFFFFFFFFu; }
    {
      // one thread per sampling block of the tensor (at most kSampleThreads of them)
      const int c = tid < t.chunks ? __ldcg(p.sample_cnt + first + tid) : 0;
      int ex, e2, tot, t2;
      block_excl_scan2(c, 0, sh, ex, e2, tot, t2);
      if (tid < t.chunks) s_off[tid] = ex;
      if (tid == 0) s_off[t.chunks] = tot;
    }
    __syncthreads();
    const int U = s_off[t.chunks];
    const uint32_t* keys0 = p.sample_keys + t.key_base;
    bool whole = false;
    if (U < rank && t.rank_local < rank) {
      whole = true;      // shortened lists that do not add up to `rank`: select from the whole sample
    } else if (U < rank) {
      kth = 0u;                                    // fewer than `rank` non-zero keys
      n_eq = 2;                                    // and the zeros beyond them are many
    } else if (U <= kSampleSurvivors) {
      // (the lists' keys lie within a factor of a few of each other: selecting between their
      // smallest and largest key saves the radix pass over the exponent bits they share)
      uint32_t tmax = 0u, tmin = 0xFFFFFFFFu;
      for (int q = tid >> 5; q < t.chunks; q += kSampleThreads / 32) {
        const int o = s_off[q], c = s_off[q + 1] - o;
        const uint32_t* src = keys0 + q * (4 * kSampleThreads);
        for (int i = lane; i < c; i += 32) {
          const uint32_t key = __ldcg(src + i);
          surv[o + i] = key;
          tmax = max(tmax, key);
          tmin = min(tmin, key);
        }
      }
      const uint32_t wmax = __reduce_max_sync(0xFFFFFFFFu, tmax);
      const uint32_t wmin = __reduce_min_sync(0xFFFFFFFFu, tmin);
      if (lane == 0) { atomicMax(&s_max, wmax); atomicMin(&s_min, wmin); }
      __syncthreads();
      const uint32_t smin = s_min;
      const int it2 = (U + kSampleThreads - 1) / kSampleThreads;
      kth = block_select_desc<kSampleThreads, false>(
          [&](auto f) {
            for (int it = 0; it < it2; ++it) {
              const int i = it * kSampleThreads + tid;
              f(i < U, i < U ? surv[i] : smin);
            }
          },
          rank, smin, s_max, hist, sh, n_gt, &n_eq);
    } else {
      kth = block_select_desc<kSampleThreads>(
          [&](auto f) {
            // one warp per slice: the warps' loads run side by side
            for (int q = tid >> 5; q < t.chunks; q += kSampleThreads / 32) {
              const int c = s_off[q + 1] - s_off[q];
              const uint32_t* src = keys0 + q * (4 * kSampleThreads);
              for (int i = lane; i < c; i += 32) f(true, __ldcg(src + i));
            }
          },
          rank, 0u, 0x7FFFFFFFu, hist, sh, n_gt, &n_eq);
    }
    done = !whole;
  }
  if (tid == 0 && !done) { s_cnt = 0; s_max = 0u; }
  __syncthreads();                                    // also orders this block's own key writes
  // (otherwise) this block now holds the whole sample of the tensor in gkeys[0 .. G)
  const int iters = done ? 0 : (G + kSampleThreads - 1) / kSampleThreads;
  uint32_t tmax = 0;
#pragma unroll 4
  for (int it = 0; it < iters; ++it) {
    const int i = it * kSampleThreads + tid;
    if (i < G) {
      const uint4 kk = __ldcg(gkeys + i);
      tmax = max(max(tmax, kk.x), max(kk.y, max(kk.z, kk.w)));
    }
  }
  {
    const uint32_t wmax = __reduce_max_sync(0xFFFFFFFFu, tmax);
    if (lane == 0) atomicMax(&s_max, wmax);
  }
  __syncthreads();
  const uint32_t kmax = s_max;
  const int owners = min(G, kSampleThreads);          // threads that hold at least one group
  if (!done && rank <= owners) {
    // lower bound: rank-th largest of the thread maxima
    const uint32_t low = block_select_desc<kSampleThreads, false>([&](auto f) { f(tid < owners, tmax); }, rank, 0u, kmax,
                                           hist, sh, n_gt);
    // keep the keys that reach it
#pragma unroll 4
    for (int it = 0; it < iters; ++it) {
      const int i = it * kSampleThreads + tid;
      uint4 kk = make_uint4(0u, 0u, 0u, 0u);
      if (i < G) kk = __ldcg(gkeys + i);
      const uint32_t karr[4] = {kk.x, kk.y, kk.z, kk.w};
      // survivors are rare: skip the four compactions when no lane of the warp has one
      if (!__any_sync(0xFFFFFFFFu, i < G && max(max(kk.x, kk.y), max(kk.z, kk.w)) >= low)) continue;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const bool keep = i < G && karr[c] >= low;
        const unsigned mk = __ballot_sync(0xFFFFFFFFu, keep);
        if (mk) {
          int basepos = 0;
          if (lane == __ffs(mk) - 1) basepos = atomicAdd(&s_cnt, __popc(mk));
          basepos = __shfl_sync(0xFFFFFFFFu, basepos, __ffs(mk) - 1);
          const int pos = basepos + __popc(mk & ((1u << lane) - 1u));
          if (keep && pos < kSampleSurvivors) surv[pos] = karr[c];
        }
      }
    }
    __syncthreads();
    const int ns = s_cnt;
    if (ns <= kSampleSurvivors) {
      const int it2 = (ns + kSampleThreads - 1) / kSampleThreads;
      kth = block_select_desc<kSampleThreads, false>(
          [&](auto f) {
            for (int it = 0; it < it2; ++it) {
              const int i = it * kSampleThreads + tid;
              f(i < ns, i < ns ? surv[i] : low);
            }
          },
          rank, low, kmax, hist, sh, n_gt, &n_eq);
      done = true;
    }
  }
  if (!done) {
    kth = block_select_desc<kSampleThreads>(
        [&](auto f) {
          for (int it = 0; it < iters; ++it) {
            const int i = it * kSampleThreads + tid;
            uint4 kk = make_uint4(0u, 0u, 0u, 0u);
            if (i < G) kk = __ldcg(gkeys + i);
            f(i < G, kk.x);
            f(i < G, kk.y);
            f(i < G, kk.z);
            f(i < G, kk.w);
          }
        },
        rank, 0u, kmax, hist, sh, n_gt, &n_eq);
  }
  // candidates are the entries that EXCEED the sample's rank-th key (p_thr = key + 1): entries
  // tied with it are only counted (p_eq), so that a tensor with masses of equal magnitudes (all
  // zeros, a few distinct values) neither floods the candidate lists nor needs a selection.
  // Paper-literal mode has the same mask: "|v| > thr", thr the sample's rank-k_s key.
  const uint32_t thr = kth + 1u;
  const uint32_t tie_on = n_eq > 1 ? 1u : 0u;     // the sample repeats its rank-th key
  for (int q = tid; q < t.part_num; q += kSampleThreads) {
    p.p_thr[t.part_first + q] = thr;
    p.p_tie[t.part_first + q] = tie_on;
  }
}

// ------------------------------------------------------------------ K3: fused momentum correction + candidate emission
// The streaming pass: 12 B read + 8 B written per element.  Each warp owns one
// 512-element segment at a time (4 float4 per lane per array, 512 contiguous
// bytes per warp load), keeps everything in registers, and appends the
// segment's candidates -- in ascending index order -- to its part's list with
// one integer atomicAdd per segment that has any.
template <bool CLIP, bool NEST>
__global__ void __launch_bounds__(kMainThreads)
k_update_emit(Plan p, const float* __restrict__ g, float m) {
  pdl_enter();
  timeline_mark(p.timeline, 1);
  const int lane = threadIdx.x & 31;
  const float4* g4 = reinterpret_cast<const float4*>(g);
  float4* u4 = reinterpret_cast<float4*>(p.u);
  float4* v4 = reinterpret_cast<float4*>(p.v);
  // one segment per warp, one launch-time block per 8 segments: short blocks let the
  // hardware interleave this kernel with the small kernels of other streams
  const int seg = blockIdx.x * (kMainThreads / 32) + (threadIdx.x >> 5);
  if (seg < p.num_segs) {
    const int base = seg * kSeg;
    const int q0 = (base >> 2) + lane;
    float4 gg[4], uu[4], vv[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) gg[i] = __ldcs(g4 + q0 + i * 32);
#pragma unroll
    for (int i = 0; i < 4; ++i) uu[i] = __ldcs(u4 + q0 + i * 32);
#pragma unroll
    for (int i = 0; i < 4; ++i) vv[i] = __ldcs(v4 + q0 + i * 32);
    const int part = __ldg(p.seg_part + seg);
    const PartMeta pm = load_record(p.pm + part);
    const uint32_t thr = __ldcg(p.p_thr + part);
    const bool tie_on = __ldcg(p.p_tie + part) != 0u;
    const float coef = CLIP ? __ldcg(p.clip_scope ? p.t_coef + pm.tensor : p.coef) : 1.0f;
    const int end = pm.end;
    const bool full = base + kSeg <= end;
    if (p.defer_mask) {
      // Sec. 3.3 masking of the previous call, applied here: the segment's 512 sent bits are 16
      // words; element c of float4 (i, lane) is bit (lane & 7) * 4 + c of word 4 * i + lane / 8
      const uint32_t myword = lane < 16 ? __ldcg(p.sent_bits + seg * 16 + lane) : 0u;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t w = __shfl_sync(0xFFFFFFFFu, myword, i * 4 + (lane >> 3));
        const uint32_t nib = (w >> ((lane & 7) * 4)) & 0xFu;
        if (nib & 1u) { uu[i].x = 0.0f; vv[i].x = 0.0f; }
        if (nib & 2u) { uu[i].y = 0.0f; vv[i].y = 0.0f; }
        if (nib & 4u) { uu[i].z = 0.0f; vv[i].z = 0.0f; }
        if (nib & 8u) { uu[i].w = 0.0f; vv[i].w = 0.0f; }
      }
    }
    uint32_t flags = 0;   // bit (4*i + c): element c of float4 i is a candidate
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      mc_step<CLIP, NEST>(gg[i].x, coef, m, uu[i].x, vv[i].x);
      mc_step<CLIP, NEST>(gg[i].y, coef, m, uu[i].y, vv[i].y);
      mc_step<CLIP, NEST>(gg[i].z, coef, m, uu[i].z, vv[i].z);
      mc_step<CLIP, NEST>(gg[i].w, coef, m, uu[i].w, vv[i].w);
      flags |= (uint32_t)(mag_key(vv[i].x) >= thr) << (4 * i + 0);
      flags |= (uint32_t)(mag_key(vv[i].y) >= thr) << (4 * i + 1);
      flags |= (uint32_t)(mag_key(vv[i].z) >= thr) << (4 * i + 2);
      flags |= (uint32_t)(mag_key(vv[i].w) >= thr) << (4 * i + 3);
    }
    uint32_t ties = 0;    // same layout: the element's key is thr - 1, the sample's rank-th key
    if (tie_on) {         // warp-uniform; off unless the sample showed repeated magnitudes
      const uint32_t tie_key = thr - 1u;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        ties |= (uint32_t)(mag_key(vv[i].x) == tie_key) << (4 * i + 0);
        ties |= (uint32_t)(mag_key(vv[i].y) == tie_key) << (4 * i + 1);
        ties |= (uint32_t)(mag_key(vv[i].z) == tie_key) << (4 * i + 2);
        ties |= (uint32_t)(mag_key(vv[i].w) == tie_key) << (4 * i + 3);
      }
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
      ties &= valid;
    }
    if (tie_on && __any_sync(0xFFFFFFFFu, ties != 0)) {
      const int c = __reduce_add_sync(0xFFFFFFFFu, __popc(ties));
      if (lane == 0) atomicAdd(p.p_eq + part, c);
    }
    if (__any_sync(0xFFFFFFFFu, flags != 0)) {
      // per-lane counts of the four float4 rows packed one per byte (row totals <= 128)
      const uint32_t cnt = __popc(flags & 0xFu) | (__popc(flags & 0xF0u) << 8) |
                           (__popc(flags & 0xF00u) << 16) | (__popc(flags & 0xF000u) << 24);
      const uint32_t incl = (uint32_t)warp_incl_scan((int)cnt);
      const uint32_t tot = __shfl_sync(0xFFFFFFFFu, incl, 31);
      const uint32_t excl = incl - cnt;
      const int t0 = tot & 255, t1 = (tot >> 8) & 255, t2 = (tot >> 16) & 255, t3 = tot >> 24;
      const int seg_total = t0 + t1 + t2 + t3;
      int start = 0;
      if (lane == 0) start = atomicAdd(p.p_count + part, seg_total);
      start = __shfl_sync(0xFFFFFFFFu, start, 0);
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
              if (pos < pm.cap) {
                if (!p.dense_emit) p.cand_idx[pm.cbase + pos] = e + c;
                p.cand_val[pm.cbase + pos] = varr[c];
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
// Tie-fill selection.  The candidates are the entries that exceed the sample's rank-th key
// (p_thr - 1).  If fewer than k exist but the entries tied with that key make up the rest, the
// exact top-k needs no selection: all candidates, then the k - total tied entries of lowest
// index; the threshold is that key.  Per part, its candidates are "greater" and its p_eq
// entries are ties; k_emit_mask finds the tied entries by reading the part (PartSel.dense == 2).
// This is the path of a tensor that is all or almost all zeros (a frozen layer, unused
// embedding rows: the key is 0) or holds a few distinct magnitudes (sign or low-bit
// gradients).  Returns false, having written nothing, if the ties do not suffice.
template <int THREADS>
__device__ __forceinline__ bool tie_fill_parts(const Plan& p, int p0, int pn, int k, int total,
                                               int out_off, uint32_t kth, int* sh) {
  const int tid = threadIdx.x;
  int mine = 0;
  for (int q = tid; q < pn; q += THREADS) mine += __ldcg(p.p_eq + p0 + q);
  int e1, e2, eq_total, t2;
  block_excl_scan2(mine, 0, sh, e1, e2, eq_total, t2);
  __syncthreads();
  if (total + eq_total < k) return false;
  const int quota = k - total;
  int run_gt = 0, run_eq = 0;
  for (int q0 = 0; q0 < pn; q0 += THREADS) {
    const int q = q0 + tid;
    int gt = 0, eq = 0;
    if (q < pn) {
      gt = __ldcg(p.p_count + p0 + q);
      eq = __ldcg(p.p_eq + p0 + q);
    }
    int bg, be, tg, te;
    block_excl_scan2(gt, eq, sh, bg, be, tg, te);
    bg += run_gt;
    be += run_eq;
    if (q < pn) {
      PartSel ps;
      ps.kth = kth;
      ps.quota = max(0, min(quota - be, eq));
      ps.out_base = out_off + bg + min(be, quota);
      ps.dense = 2;
      p.psel[p0 + q] = ps;
    }
    run_gt += tg;
    run_eq += te;
    __syncthreads();
  }
  return true;
}

// THREADS: 1024 for a call that runs alone (shortest chain for the largest tensor), 512 when
// several workers' selections run together (twice the blocks per SM: the batch's tail is
// bound by block slots, not by one block's chain).
// Shared memory of one selection block besides the dynamic [histograms | keys] area.
struct SelectShared {
  int sh[66];
  int flag;
  uint32_t max;
  int pbase[kSelectMaxParts + 1];   // first key of each part in the compact order
  int pcb[kSelectMaxParts];         // start of each part's candidate list
  int gt[kSelectMaxParts];
  int eq[kSelectMaxParts];
};

// The selection of tensor j by one block of THREADS threads (the whole of k_select, and what
// k_select_cluster does for tensors that one block handles).
template <int THREADS>
__device__ __forceinline__ void select_tensor(const Plan& p, int j, const TensorMeta& t,
                                              int smem_keys, int parity, uint32_t* dyn_smem,
                                              SelectShared& S) {
  uint32_t* hist = dyn_smem;
  uint32_t* skeys = dyn_smem + kHistWords(THREADS);
  int* sh = S.sh;
  int& s_flag = S.flag;
  uint32_t& s_max = S.max;
  int* s_pbase = S.pbase;
  int* s_pcb = S.pcb;
  int* s_gt = S.gt;
  int* s_eq = S.eq;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int p0 = t.part_first, pn = t.part_num, k = t.k;
  if (tid == 0) { s_flag = 0; s_max = 0u; }
  __syncthreads();
  // candidates per part (one load round for all parts), overflow check, compact bases
  int total = 0;
  if (pn <= 32) {
    if (warp == 0) {
      int c = 0;
      if (lane < pn) {
        const PartMeta pm = load_record(p.pm + p0 + lane);
        c = __ldcg(p.p_count + p0 + lane);
        if (c > pm.cap) s_flag = 1;
        s_pcb[lane] = pm.cbase;
      }
      const int incl = warp_incl_scan(c);
      if (lane < pn) s_pbase[lane] = incl - c;
      if (lane == 31) s_pbase[pn] = incl;
    }
    __syncthreads();
    total = s_pbase[pn];
  } else {
    for (int q0 = 0; q0 < pn; q0 += THREADS) {
      const int q = q0 + tid;
      int c = 0;
      if (q < pn) {
        const PartMeta pm = load_record(p.pm + p0 + q);
        c = __ldcg(p.p_count + p0 + q);
        if (c > pm.cap) s_flag = 1;
        s_pcb[q] = pm.cbase;
      }
      int ex, dummy_e, tot, dummy_t;
      block_excl_scan2(c, 0, sh, ex, dummy_e, tot, dummy_t);
      if (q < pn) s_pbase[q] = total + ex;
      total += tot;
      __syncthreads();
    }
    if (tid == 0) s_pbase[pn] = total;
    __syncthreads();
  }
  const bool overflow = s_flag != 0;
  // Paper-literal mode (Sec. 5): what passed the sampled threshold is sent as it is unless far
  // more than expected passed (more than 2k: then the precise top-k of the tensor, which all
  // lie among the candidates).  Every tensor is sampled in that mode.
  const bool literal = p.literal != 0;
  const bool lit_sampled_all = literal && !overflow && total <= 2 * k;
  const int rank = k;
  if (!overflow && !literal && total < k && t.groups > 0) {
    const uint32_t tie_key = __ldcg(p.p_thr + p0) - 1u;
    if (tie_fill_parts<THREADS>(p, p0, pn, k, total, t.out_off, tie_key, sh)) {
      if (tid == 0) {
        p.t_kth[j] = tie_key;
        p.t_cand[j] = total;
        p.t_nnz[j] = k;
        atomicOr((unsigned long long*)&p.diag[parity * 4 + 0], (unsigned long long)DGC_FLAG_TIE_FILL);
        atomicAdd((unsigned long long*)&p.diag[parity * 4 + 2], (unsigned long long)total);
      }
      return;
    }
  }
  if (overflow || (!literal && total < k)) {
    if (tid == 0) p.t_nnz[j] = k;
    // full-selection path: k_emit_mask's block of the tensor's first part does it
    for (int q = tid; q < pn; q += THREADS) {
      PartSel ps;
      ps.kth = 0u; ps.quota = 0; ps.out_base = 0; ps.dense = 1;
      p.psel[p0 + q] = ps;
    }
    if (tid == 0) {
      p.t_cand[j] = -1;
      atomicOr((unsigned long long*)&p.diag[parity * 4 + 0],
               (unsigned long long)(DGC_FLAG_FULL_SELECT |
                                    (overflow ? DGC_FLAG_CAND_OVERFLOW : DGC_FLAG_CAND_SHORT)));
      atomicAdd((unsigned long long*)&p.diag[parity * 4 + 1], 1ull);
    }
    return;
  }
  const bool in_smem = total <= smem_keys;
  const int slices = max(1, (THREADS / 32) / pn);
  uint32_t kmax = 0x7FFFFFFFu;
  uint32_t kbase = 0u;
  if (in_smem) {
    // gather the keys of all parts, compact, into shared memory: coalesced reads, a part is
    // shared by `slices` warps when the tensor has fewer parts than the block has warps
    uint32_t tmax = 0;
    // The candidate values are staged by asynchronous copies, so that all of a warp's loads
    // are in flight at once instead of four per round trip, and the keys are formed in shared
    // memory afterwards (measured on the ResNet-50-shaped set: selection 18.5 -> 17.3 us).
    for (int unit = warp; unit < pn * slices; unit += THREADS / 32) {
      const int q = unit / slices, sl = unit - q * slices;
      const int b0 = s_pbase[q], c = s_pbase[q + 1] - b0;
      const float* src = p.cand_val + s_pcb[q];
      for (int i = sl * 32 + lane; i < c; i += slices * 32) stage_word(skeys + b0 + i, src + i);
    }
    stage_wait();
    __syncthreads();
    for (int i = tid; i < total; i += THREADS) {
      const uint32_t key = skeys[i] & 0x7FFFFFFFu;
      skeys[i] = key;
      tmax = max(tmax, key);
    }
    const uint32_t wmax = __reduce_max_sync(0xFFFFFFFFu, tmax);
    if (lane == 0) atomicMax(&s_max, wmax);
    kbase = __ldcg(p.p_thr + p0);                // every candidate reached the proposal
    __syncthreads();
    kmax = s_max;
  }
  int n_gt;
  uint32_t kth;
  if (lit_sampled_all) {
    kth = __ldcg(p.p_thr + p0) - 1u;             // every candidate exceeds it (p_thr >= 1 here)
    n_gt = total;
  } else if (in_smem) {
    const int iters = (total + THREADS - 1) / THREADS;
    auto each = [&](auto f) {
      for (int it = 0; it < iters; ++it) {
        const int i = it * THREADS + tid;
        const bool valid = i < total;
        f(valid, valid ? skeys[i] : kbase);
      }
    };
    // up to two keys per thread: not worth private histograms
    if (total <= 8 * THREADS)
      kth = block_select_desc<THREADS, false>(each, rank, kbase, kmax, hist, sh, n_gt);
    else
      kth = block_select_desc<THREADS, true>(each, rank, kbase, kmax, hist, sh, n_gt);
  } else {
    kth = block_select_desc<THREADS>(
        [&](auto f) {
          for (int q = 0; q < pn; ++q) {
            const int c = __ldcg(p.p_count + p0 + q);
            const float* src = p.cand_val + __ldg(&p.pm[p0 + q].cbase);
            const int iters = (c + THREADS - 1) / THREADS;
            for (int it = 0; it < iters; ++it) {
              const int i = it * THREADS + tid;
              const bool valid = i < c;
              f(valid, valid ? mag_key(__ldcg(src + i)) : 0u);
            }
          }
        },
        rank, kbase, kmax, hist, sh, n_gt);
  }
  // ties (|v'| == kth) to take, lowest indices first
  const int quota = lit_sampled_all ? 0 : k - n_gt;
  const int nnz = lit_sampled_all ? total : k;
  const int out_off = literal ? 0 : t.out_off;   // paper-literal: k_emit_mask adds the tensor's base
  // per part: strictly-greater and tied candidates (a single part needs no count: it takes
  // the whole quota and k_emit_mask stops at the quota by itself)
  for (int q = tid; q < pn; q += THREADS) { s_gt[q] = 0; s_eq[q] = 0; }
  __syncthreads();
  if (pn > 1) {
    for (int unit = warp; unit < pn * slices; unit += THREADS / 32) {
      const int q = unit / slices, sl = unit - q * slices;
      const int b0 = s_pbase[q], c = s_pbase[q + 1] - b0;
      const float* src = p.cand_val + s_pcb[q];
      int gt = 0, eq = 0;
      for (int i = sl * 32 + lane; i < c; i += slices * 32) {
        const uint32_t key = in_smem ? skeys[b0 + i] : mag_key(__ldcg(src + i));
        gt += key > kth;
        eq += key == kth;
      }
      gt = __reduce_add_sync(0xFFFFFFFFu, gt);
      eq = __reduce_add_sync(0xFFFFFFFFu, eq);
      if (lane == 0) {
        if (gt) atomicAdd(&s_gt[q], gt);
        if (eq) atomicAdd(&s_eq[q], eq);
      }
    }
  } else if (tid == 0) {
    s_eq[0] = quota;     // upper bound is enough for one part
  }
  __syncthreads();
  if (pn <= 32) {
    if (warp == 0) {
      const int gt = lane < pn ? s_gt[lane] : 0, eq = lane < pn ? s_eq[lane] : 0;
      const int bg = warp_incl_scan(gt) - gt, be = warp_incl_scan(eq) - eq;
      if (lane < pn) {
        PartSel ps;
        ps.kth = kth;
        ps.quota = max(0, min(quota - be, eq));
        ps.out_base = out_off + bg + min(be, quota);
        ps.dense = 0;
        p.psel[p0 + lane] = ps;
      }
    }
  } else {
    int run_gt = 0, run_eq = 0;
    for (int q0 = 0; q0 < pn; q0 += THREADS) {
      const int q = q0 + tid;
      const int gt = q < pn ? s_gt[q] : 0, eq = q < pn ? s_eq[q] : 0;
      int bg, be, tg, te;
      block_excl_scan2(gt, eq, sh, bg, be, tg, te);
      bg += run_gt;
      be += run_eq;
      if (q < pn) {
        PartSel ps;
        ps.kth = kth;
        ps.quota = max(0, min(quota - be, eq));
        ps.out_base = out_off + bg + min(be, quota);
        ps.dense = 0;
        p.psel[p0 + q] = ps;
      }
      run_gt += tg;
      run_eq += te;
      __syncthreads();
    }
  }
  if (tid == 0) {
    p.t_kth[j] = kth;
    p.t_cand[j] = total;
    p.t_nnz[j] = nnz;
    atomicAdd((unsigned long long*)&p.diag[parity * 4 + 2], (unsigned long long)total);
  }
}

template <int THREADS>
__global__ void __launch_bounds__(THREADS)
k_select(Plan p, int smem_keys) {
  pdl_enter();
  timeline_mark(p.timeline, 2);
  const int parity = (int)(__ldcg(p.iter) & 1);
  extern __shared__ uint32_t dyn_smem[];          // [histograms | keys]
  __shared__ SelectShared S;
  const int j = blockIdx.x;
  const TensorMeta t = load_record(p.tm + j);
  if (j == 0 && threadIdx.x < 4) p.diag[(parity ^ 1) * 4 + threadIdx.x] = 0;   // next call's counters
  // k_big_* select the big tensors, which include every tensor of more than kSelectMaxParts
  // parts: the per-part tables always fit
  if (t.big || t.part_num > kSelectMaxParts) return;
  select_tensor<THREADS>(p, j, t, smem_keys, parity, dyn_smem, S);
}

// The same selection with a thread-block cluster per tensor: kClusterSize blocks on as many SMs
// share the candidates of one tensor (a contiguous range of its parts each) and exchange their
// digit histograms through distributed shared memory, so that the longest chain of the tail --
// the tensor with the most candidates -- is cut several times over: one block spends about
// 120 instructions per candidate, 41 us for the 30 K candidates of a 15 M-element tensor.
// Tensors of fewer than kClusterMinParts parts, and every case that needs no key (tie-fill,
// full selection, paper-literal pass-through), are handled by the cluster's first block alone;
// the other blocks leave at once.  Every decision that steers the cluster barriers is taken
// from values all blocks read alike (plan tables, the parts' counts), so that all blocks of a
// cluster pass the same barriers.
struct ClusterShared {
  uint32_t hist[2][256];   // this block's digit counts, current and next pass
  uint32_t folded[256];    // the cluster's digit counts
  uint32_t max;
};

template <int THREADS>
__global__ void __launch_bounds__(THREADS)
k_select_cluster(Plan p, int smem_keys) {
  namespace cg = cooperative_groups;
  pdl_enter();
  timeline_mark(p.timeline, 2);
  cg::cluster_group cluster = cg::this_cluster();
  const int r = (int)cluster.block_rank();
  const int parity = (int)(__ldcg(p.iter) & 1);
  extern __shared__ uint32_t dyn_smem[];          // [histograms | keys]
  __shared__ SelectShared S;
  __shared__ ClusterShared X;
  const int j = blockIdx.x / kClusterSize;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const TensorMeta t = load_record(p.tm + j);
  const int p0 = t.part_first, pn = t.part_num, k = t.k;
  if (blockIdx.x == 0 && tid < 4) p.diag[(parity ^ 1) * 4 + tid] = 0;   // next call's counters
  if (t.big || pn > kSelectMaxParts) return;                 // (same for the whole cluster)
  if (pn < kClusterMinParts) {
    if (r == 0) select_tensor<THREADS>(p, j, t, smem_keys, parity, dyn_smem, S);
    return;
  }
  static_assert(kSelectMaxParts <= THREADS, "one thread per part");
  // every block for itself: candidates per part, overflow, compact bases of all parts
  if (tid == 0) { S.flag = 0; X.max = 0u; }
  __syncthreads();
  {
    int c = 0;
    if (tid < pn) {
      const PartMeta pm = load_record(p.pm + p0 + tid);
      c = __ldcg(p.p_count + p0 + tid);
      if (c > pm.cap) S.flag = 1;
      S.pcb[tid] = pm.cbase;
    }
    int ex, e2, tot, t2;
    block_excl_scan2(c, 0, S.sh, ex, e2, tot, t2);
    if (tid < pn) S.pbase[tid] = ex;
    if (tid == 0) S.pbase[pn] = tot;
  }
  __syncthreads();
  const int total = S.pbase[pn];
  const bool overflow = S.flag != 0;
  const bool literal = p.literal != 0;
  if (overflow || (!literal && total < k) || (literal && total <= 2 * k)) {
    // no exact selection among the candidates: one block does what there is to do
    __syncthreads();
    if (r == 0) select_tensor<THREADS>(p, j, t, smem_keys, parity, dyn_smem, S);
    return;
  }
  // ---- the whole cluster: this block takes parts [q0, q1)
  uint32_t* skeys = dyn_smem;
  const int q0 = r * pn / kClusterSize, q1 = (r + 1) * pn / kClusterSize;
  const int m0 = S.pbase[q0], m = S.pbase[q1] - m0;
  const bool in_smem = m <= smem_keys;
  const int myparts = q1 - q0;
  const int slices = myparts > 0 ? max(1, (THREADS / 32) / myparts) : 1;
  if (in_smem) {
    uint32_t tmax = 0;
    for (int unit = warp; unit < myparts * slices; unit += THREADS / 32) {
      const int q = q0 + unit / slices, sl = unit % slices;
      const int b0 = S.pbase[q] - m0, c = S.pbase[q + 1] - S.pbase[q];
      const float* src = p.cand_val + S.pcb[q];
      for (int i = sl * 32 + lane; i < c; i += slices * 32) stage_word(skeys + b0 + i, src + i);
    }
    stage_wait();
    __syncthreads();
    for (int i = tid; i < m; i += THREADS) {
      const uint32_t key = skeys[i] & 0x7FFFFFFFu;
      skeys[i] = key;
      tmax = max(tmax, key);
    }
    const uint32_t wmax = __reduce_max_sync(0xFFFFFFFFu, tmax);
    if (lane == 0 && wmax) atomicMax(&X.max, wmax);
  } else if (tid == 0) {
    X.max = 0x7FFFFFFFu;                           // (keys stay in global memory: no maximum)
  }
  for (int i = tid; i < 512; i += THREADS) (&X.hist[0][0])[i] = 0u;
  __syncthreads();
  cluster.sync();
  uint32_t kmax = 0u;
#pragma unroll
  for (int rr = 0; rr < kClusterSize; ++rr) kmax = max(kmax, *cluster.map_shared_rank(&X.max, rr));
  const uint32_t kbase = __ldcg(p.p_thr + p0);     // every candidate reached the proposal
  // my keys, from shared or (a share that does not fit) from global memory
  auto each = [&](auto f) {
    if (in_smem) {
      for (int i = tid; i < m; i += THREADS) f(skeys[i]);
    } else {
      for (int q = q0; q < q1; ++q) {
        const int c = S.pbase[q + 1] - S.pbase[q];
        const float* src = p.cand_val + S.pcb[q];
        for (int i = tid; i < c; i += THREADS) f(mag_key(__ldcg(src + i)));
      }
    }
  };
  // radix select over the bits in which kmax - kbase can differ, 8 per pass: local counts,
  // cluster barrier, every block folds the eight histograms and finds the same digit
  const uint32_t span = kmax - kbase;
  const int passes = span == 0 ? 0 : (32 - __clz(span) + 7) / 8;
  uint32_t prefix = 0, mask = 0;
  int remaining = k;
  int cur = 0;
  for (int shift = 8 * (passes - 1); shift >= 0; shift -= 8, cur ^= 1) {
    each([&](uint32_t key) {
      key -= kbase;
      if ((key & mask) == prefix) atomicAdd(&X.hist[cur][(key >> shift) & 255u], 1u);
    });
    __syncthreads();
    cluster.sync();
    if (tid < 256) {
      uint32_t sum = 0;
#pragma unroll
      for (int rr = 0; rr < kClusterSize; ++rr) sum += *cluster.map_shared_rank(&X.hist[cur][tid], rr);
      X.folded[tid] = sum;
    } else if (tid < 512) {
      // next pass's counts start from zero (the others read this buffer a pass ago and have
      // passed the barrier above since)
      X.hist[cur ^ 1][tid - 256] = 0u;
    }
    __syncthreads();
    if (tid < 32) warp_find_digit(X.folded, remaining, S.sh);
    __syncthreads();
    prefix |= (uint32_t)S.sh[0] << shift;
    mask |= 255u << shift;
    remaining -= S.sh[1];
    __syncthreads();
  }
  static_assert(THREADS >= 512, "threads 256..511 clear the next pass's histogram");
  const uint32_t kth = kbase + prefix;
  const int n_gt = k - remaining;
  // per part of mine: candidates above and tied with the k-th key
  for (int q = q0 + tid; q < q1; q += THREADS) { S.gt[q] = 0; S.eq[q] = 0; }
  __syncthreads();
  for (int unit = warp; unit < myparts * slices; unit += THREADS / 32) {
    const int q = q0 + unit / slices, sl = unit % slices;
    const int b0 = S.pbase[q] - m0, c = S.pbase[q + 1] - S.pbase[q];
    const float* src = p.cand_val + S.pcb[q];
    int gt = 0, eq = 0;
    for (int i = sl * 32 + lane; i < c; i += slices * 32) {
      const uint32_t key = in_smem ? skeys[b0 + i] : mag_key(__ldcg(src + i));
      gt += key > kth;
      eq += key == kth;
    }
    gt = __reduce_add_sync(0xFFFFFFFFu, gt);
    eq = __reduce_add_sync(0xFFFFFFFFu, eq);
    if (lane == 0) {
      if (gt) atomicAdd(&S.gt[q], gt);
      if (eq) atomicAdd(&S.eq[q], eq);
    }
  }
  __syncthreads();
  cluster.sync();
  if (r == 0) {
    // the first block collects every part's counts from its owner and places the parts
    const int quota = k - n_gt;                    // ties with kth to send, lowest indices first
    const int out_off = literal ? 0 : t.out_off;   // paper-literal: k_emit_mask adds the tensor's base
    int gt = 0, eq = 0;
    if (tid < pn) {
      int owner = 0;
      while ((owner + 1) * pn / kClusterSize <= tid) ++owner;
      gt = *cluster.map_shared_rank(&S.gt[tid], owner);
      eq = *cluster.map_shared_rank(&S.eq[tid], owner);
    }
    int bg, be, tg, te;
    block_excl_scan2(gt, eq, S.sh, bg, be, tg, te);
    if (tid < pn) {
      PartSel ps;
      ps.kth = kth;
      ps.quota = max(0, min(quota - be, eq));
      ps.out_base = out_off + bg + min(be, quota);
      ps.dense = 0;
      p.psel[p0 + tid] = ps;
    }
    if (tid == 0) {
      p.t_kth[j] = kth;
      p.t_cand[j] = total;
      p.t_nnz[j] = k;
      atomicAdd((unsigned long long*)&p.diag[parity * 4 + 2], (unsigned long long)total);
    }
  }
  cluster.sync();      // the others' shared memory stays until the first block has read it
}

// ------------------------------------------------------------------ K4b: multi-block exact k-th key
// The same selection for tensors whose candidates do not fit one block's shared
// memory (warm-up sparsities, very large tensors): a radix select over the 31
// key bits in three rounds (11 + 11 + 9 bits), one block per part and round.
// Each round adds the part's digit counts to the tensor's histogram in global
// memory (integer atomics); the next round's blocks each read that histogram,
// find the digit that holds the k-th key (all blocks of a tensor compute the
// same value) and count the next digit among the keys that match the prefix.
// k_big_final then derives the threshold, every part's share and output base.
// No block waits for another: rounds are separate launches.

// The digit (counting from the largest) at which the cumulative count reaches
// `remaining`; returns the digit, `above` = keys in larger digits.  All threads
// of the block get the result.  bins <= 4 * blockDim.x.  sh: 66 + 2 ints.
__device__ __forceinline__ int block_find_digit(const int32_t* hist, int bins, int remaining,
                                                int* sh, int& above) {
  const int tid = threadIdx.x;
  const int per = (bins + blockDim.x - 1) / blockDim.x;      // bins per thread, descending order
  int loc[4];
  int sum = 0;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int bin = bins - 1 - (tid * per + q);
    loc[q] = (q < per && bin >= 0) ? __ldcg(hist + bin) : 0;
    sum += loc[q];
  }
  int ex, dummy, tot, dummy2;
  block_excl_scan2(sum, 0, sh, ex, dummy, tot, dummy2);
  if (ex < remaining && remaining <= ex + sum) {
    int c = ex;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if (c + loc[q] >= remaining) { sh[66] = bins - 1 - (tid * per + q); sh[67] = c; break; }
      c += loc[q];
    }
  }
  __syncthreads();
  const int digit = sh[66];
  above = sh[67];
  __syncthreads();
  return digit;
}

template <int ROUND>
__global__ void __launch_bounds__(kBigThreads)
k_big_hist(Plan p) {
  pdl_enter();
  __shared__ int hist[kBigBins];
  __shared__ int near[(kBigThreads / 32) * kBigNear];   // round 0: private bins near the proposal
  __shared__ int sh[68];
  __shared__ int s_above;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int part = __ldg(p.big_parts + blockIdx.x);
  const PartMeta pm = load_record(p.pm + part);
  const TensorMeta t = load_record(p.tm + pm.tensor);
  const int count = min(__ldcg(p.p_count + part), pm.cap);
  int32_t* thist = p.big_hist + (size_t)t.big_slot * 3 * kBigBins;
  int32_t* state = p.big_state + t.big_slot * kBigStateWords;
  // the prefix fixed by the earlier rounds
  uint32_t prefix = 0;        // upper key bits already decided (11 after round 0, 22 after round 1)
  if (ROUND == 1) {
    int above;
    const int d0 = block_find_digit(thist, kBigBins, t.k, sh, above);
    prefix = (uint32_t)d0;
    // every block of the tensor computes the same values; its first part's block records them
    if (tid == 0 && pm.first) { state[0] = d0; state[1] = t.k - above; }
  } else if (ROUND == 2) {
    const int d0 = __ldcg(state + 0), rem1 = __ldcg(state + 1);
    int above;
    const int d1 = block_find_digit(thist + kBigBins, kBigBins, rem1, sh, above);
    prefix = ((uint32_t)d0 << 11) | (uint32_t)d1;
    if (tid == 0 && pm.first) { state[32] = (int)prefix; state[33] = rem1 - above; }
  }
  for (int i = tid; i < kBigBins; i += kBigThreads) hist[i] = 0;
  if (ROUND == 0) for (int i = tid; i < (kBigThreads / 32) * kBigNear; i += kBigThreads) near[i] = 0;
  if (tid == 0) s_above = 0;
  __syncthreads();
  const float* cval = p.cand_val + pm.cbase;
  const int dthr = (int)(__ldcg(p.p_thr + part) >> 20);     // round-0 digit of the proposal
  int above_cnt = 0;
  for (int i0 = 0; i0 < count; i0 += kBigThreads * 4) {
    float vals[4];
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int i = i0 + b * kBigThreads + tid;
      vals[b] = i < count ? __ldcg(cval + i) : 0.0f;
    }
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int i = i0 + b * kBigThreads + tid;
      if (i < count) {
        const uint32_t key = mag_key(vals[b]);
        if (ROUND == 0) {
          // candidates crowd into the few digits just above the proposal: those go to a
          // per-warp private histogram, the rest to the shared one
          const int d = (int)(key >> 20), rel = d - dthr;
          if (rel >= 0 && rel < kBigNear) atomicAdd(&near[warp * kBigNear + rel], 1);
          else atomicAdd(&hist[d], 1);
        } else if (ROUND == 1) {
          if ((key >> 20) == prefix) atomicAdd(&hist[(key >> 9) & 2047u], 1);
        } else {
          const uint32_t up = key >> 9;
          if (up == prefix) atomicAdd(&hist[key & 511u], 1);
          else if (up > prefix) ++above_cnt;
        }
      }
    }
  }
  if (ROUND == 2) {
    above_cnt = __reduce_add_sync(0xFFFFFFFFu, above_cnt);
    if (lane == 0 && above_cnt) atomicAdd(&s_above, above_cnt);
  }
  __syncthreads();
  if (ROUND == 0) {
    for (int r = tid; r < kBigNear; r += kBigThreads) {
      int c = 0;
      for (int w = 0; w < kBigThreads / 32; ++w) c += near[w * kBigNear + r];
      if (c && dthr + r < kBigBins) atomicAdd(&hist[dthr + r], c);
    }
    __syncthreads();
  }
  int32_t* ghist = thist + ROUND * kBigBins;
  const int bins = ROUND == 2 ? kBigLastBins : kBigBins;
  for (int i = tid; i < bins; i += kBigThreads) {
    const int c = hist[i];
    if (c) atomicAdd(ghist + i, c);
  }
  if (ROUND == 2) {
    // what k_big_final needs of this part: for every digit d, the candidates that match the
    // prefix with last digit >= d (thread t holds digit 511 - t so that the scan runs downwards)
    static_assert(kBigThreads == kBigLastBins, "one last-round bin per thread");
    const int c = hist[kBigLastBins - 1 - tid];
    int ex, dummy, tot, dummy2;
    block_excl_scan2(c, 0, sh, ex, dummy, tot, dummy2);
    int32_t* L = p.big_last + (size_t)pm.big_slot * kBigLastStride;
    L[kBigLastBins - 1 - tid] = ex + c;
    if (tid == 0) { L[kBigLastBins] = 0; p.big_above[pm.big_slot] = s_above; }
  }
}

__global__ void __launch_bounds__(kSelectThreads)
k_big_final(Plan p) {
  pdl_enter();
  const int parity = (int)(__ldcg(p.iter) & 1);
  __shared__ int sh[68];
  __shared__ int s_gt[kSelectThreads];
  __shared__ int s_eq[kSelectThreads];
  const int tid = threadIdx.x;
  const int j = __ldg(p.big_tensors + blockIdx.x);
  const TensorMeta t = load_record(p.tm + j);
  const int p0 = t.part_first, pn = t.part_num, k = t.k;
  int32_t* thist = p.big_hist + (size_t)t.big_slot * 3 * kBigBins;
  const int32_t* state = p.big_state + t.big_slot * kBigStateWords;
  // total candidates and overflow
  int mine = 0, over = 0;
  for (int q = tid; q < pn; q += kSelectThreads) {
    const int c = __ldcg(p.p_count + p0 + q);
    const int cap = __ldg(&p.pm[p0 + q].cap);
    over |= c > cap;
    mine += min(c, cap);
  }
  int ex, exo, total, overflow;
  block_excl_scan2(mine, over, sh, ex, exo, total, overflow);
  __syncthreads();
  const bool literal = p.literal != 0;
  uint32_t kth = 0;
  bool tie_fill = false;
  if (overflow == 0 && !literal && total < k) {
    kth = __ldcg(p.p_thr + p0) - 1u;
    tie_fill = tie_fill_parts<kSelectThreads>(p, p0, pn, k, total, t.out_off, kth, sh);
  }
  const bool dense = !tie_fill && (overflow != 0 || (!literal && total < k));
  // paper-literal mode: at most 2k passed the sampled threshold -> all of them are sent
  const bool all_pass = literal && !dense && total <= 2 * k;
  const int out_off = literal ? 0 : t.out_off;
  int quota = 0;
  if (tie_fill) {
    // PartSel records already written
  } else if (all_pass) {
    kth = __ldcg(p.p_thr + p0) - 1u;            // every candidate exceeds it
    int run = 0;
    for (int q0 = 0; q0 < pn; q0 += kSelectThreads) {
      const int q = q0 + tid;
      const int c = q < pn ? __ldcg(p.p_count + p0 + q) : 0;
      int ex, e2, tot, t2;
      block_excl_scan2(c, 0, sh, ex, e2, tot, t2);
      if (q < pn) {
        PartSel ps;
        ps.kth = kth; ps.quota = 0; ps.out_base = out_off + run + ex; ps.dense = 0;
        p.psel[p0 + q] = ps;
      }
      run += tot;
      __syncthreads();
    }
  } else if (!dense) {
    const uint32_t prefix = (uint32_t)__ldcg(state + 32);
    const int rem2 = __ldcg(state + 33);
    int above;
    const int d2 = block_find_digit(thist + 2 * kBigBins, kBigLastBins, rem2, sh, above);
    kth = (prefix << 9) | (uint32_t)d2;
    quota = rem2 - above;                       // ties with kth to send, lowest indices first
    // parts in chunks of blockDim: one warp per part reads its last-round counts
    int run_gt = 0, run_eq = 0;
    for (int q0 = 0; q0 < pn; q0 += kSelectThreads) {
      s_gt[tid] = 0;
      s_eq[tid] = 0;
      const int qn = min(kSelectThreads, pn - q0);
      if (tid < qn) {
        const int slot = __ldg(&p.pm[p0 + q0 + tid].big_slot);
        const int32_t* L = p.big_last + (size_t)slot * kBigLastStride;
        const int ge = __ldcg(L + d2), gtl = __ldcg(L + d2 + 1);
        s_gt[tid] = gtl + __ldcg(p.big_above + slot);
        s_eq[tid] = ge - gtl;
      }
      __syncthreads();
      const int gt = s_gt[tid], eq = s_eq[tid];
      int bg, be, tg, te;
      block_excl_scan2(gt, eq, sh, bg, be, tg, te);
      bg += run_gt;
      be += run_eq;
      if (tid < qn) {
        PartSel ps;
        ps.kth = kth;
        ps.quota = max(0, min(quota - be, eq));
        ps.out_base = out_off + bg + min(be, quota);
        ps.dense = 0;
        p.psel[p0 + q0 + tid] = ps;
      }
      run_gt += tg;
      run_eq += te;
      __syncthreads();
    }
  } else {
    for (int q = tid; q < pn; q += kSelectThreads) {
      PartSel ps;
      ps.kth = 0u; ps.quota = 0; ps.out_base = 0; ps.dense = 1;
      p.psel[p0 + q] = ps;
    }
  }
  // histograms back to zero for the next call
  for (int i = tid; i < 3 * kBigBins; i += kSelectThreads) thist[i] = 0;
  if (tid == 0) {
    if (dense) {
      p.t_cand[j] = -1;
      atomicOr((unsigned long long*)&p.diag[parity * 4 + 0],
               (unsigned long long)(DGC_FLAG_FULL_SELECT |
                                    (overflow ? DGC_FLAG_CAND_OVERFLOW : DGC_FLAG_CAND_SHORT)));
      atomicAdd((unsigned long long*)&p.diag[parity * 4 + 1], 1ull);
    } else {
      p.t_kth[j] = kth;
      p.t_cand[j] = total;
      atomicAdd((unsigned long long*)&p.diag[parity * 4 + 2], (unsigned long long)total);
      if (tie_fill)
        atomicOr((unsigned long long*)&p.diag[parity * 4 + 0], (unsigned long long)DGC_FLAG_TIE_FILL);
    }
    p.t_nnz[j] = all_pass ? total : k;
  }
}

// ------------------------------------------------------------------ K5: ordered emission + masking
// Algorithm 4: G~[j] <- V[j] (.) Mask ; V[j] <- V[j] (.) !Mask ; U[j] <- U[j] (.) !Mask.
// One block per part.  The candidates that reach the threshold set one bit
// each in a shared-memory bitmap of the part (integer atomicOr; "greater" and
// "tied" bitmaps); per-segment popcounts and an exclusive scan give every
// segment its first output slot; every winner then finds its slot from the
// bits below its own, writes its (index, value) pair and zeroes u and v there.
//
// Full-selection path (dense flag set by k_select): the block of the tensor's
// first part selects from the whole of v' (radix select over global memory) and
// emits by walking the tensor in order.  Same result; slow; rare.
__device__ void dense_select_emit(const Plan& p, const TensorMeta& t, int j, int out_first,
                                  int32_t* out_idx, float* out_val, uint32_t* hist, int* sh) {
  const int tid = threadIdx.x, nt = blockDim.x;
  const int off = t.off;
  const int n = t.end - off;
  const int k = t.k;
  const float* v = p.v + off;
  int n_gt;
  const uint32_t kth = block_select_desc<kEmitThreads>(
      [&](auto f) {
        // batches of independent loads: one block streams the whole tensor in every pass
        for (int i0 = 0; i0 < n; i0 += nt * 8) {
          float x[8];
#pragma unroll
          for (int b = 0; b < 8; ++b) {
            const int i = i0 + b * nt + tid;
            x[b] = i < n ? __ldcg(v + i) : 0.0f;
          }
#pragma unroll
          for (int b = 0; b < 8; ++b) {
            const bool valid = i0 + b * nt + tid < n;
            f(valid, valid ? mag_key(x[b]) : 0u);
          }
        }
      },
      k, 0u, 0x7FFFFFFFu, hist, sh, n_gt);
  const int quota = k - n_gt;
  int run_w = 0, run_eq = 0;     // winners / ties seen so far
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
    int bg, be, tg, te;
    block_excl_scan2(gt, eq, sh, bg, be, tg, te);
    be += run_eq;
    int pos = out_first + run_w + bg + (min(be, quota) - min(run_eq, quota));
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
    __syncthreads();
  }
  if (tid == 0) p.t_kth[j] = kth;
}

// Pieces shared by the two emission kernels (block of kEmitThreads, one part per block).

// Paper-literal mode: the counts vary, so the tensors' lists are packed back to back; returns
// the first output slot of the part's tensor (what the earlier tensors send).
__device__ __forceinline__ int emit_literal_first(const Plan& p, const PartMeta& pm, int* s_first) {
  const int tid = threadIdx.x;
  if (tid == 0) *s_first = 0;
  __syncthreads();
  int mine = 0;
  for (int q = tid; q < pm.tensor; q += kEmitThreads) mine += __ldcg(p.t_nnz + q);
  mine = __reduce_add_sync(0xFFFFFFFFu, mine);
  if ((tid & 31) == 0 && mine) atomicAdd(s_first, mine);
  __syncthreads();
  return *s_first;
}

// Full-selection path of a tensor (PartSel.dense == 1): its first part's block does it all.
__device__ __forceinline__ void emit_full_selection(const Plan& p, const PartMeta& pm, int part,
                                                    int tensor_first, int32_t* out_idx,
                                                    float* out_val, uint32_t* smask, int* sh) {
  const int tid = threadIdx.x;
  __syncthreads();
  if (tid == 0) { p.p_count[part] = 0; p.p_eq[part] = 0; }
  if (p.defer_mask && tid < pm.nseg) {
    // the full-selection path zeroes u and v itself: nothing is pending for this part
    uint4* dst = reinterpret_cast<uint4*>(p.sent_bits + (size_t)(pm.seg0 + tid) * 16);
#pragma unroll
    for (int w = 0; w < 4; ++w) dst[w] = make_uint4(0u, 0u, 0u, 0u);
  }
  if (pm.first) {
    const TensorMeta t = load_record(p.tm + pm.tensor);
    dense_select_emit(p, t, pm.tensor, p.literal ? tensor_first : t.out_off, out_idx, out_val,
                      smask, sh);
  }
}

// Deferred masking: record what segment `tid` sent -- all "greater" bits and the tied bits
// within the quota (lowest indices first); the next call zeroes u and v there.
__device__ __forceinline__ void emit_record_sent(const Plan& p, const PartMeta& pm, int quota,
                                                 const uint32_t* mgt, const uint32_t* meq,
                                                 const int* s_eqb) {
  const int tid = threadIdx.x;
  if (tid >= pm.nseg) return;
  int left = max(0, quota - s_eqb[tid]);
  uint32_t words[16];
#pragma unroll
  for (int w = 0; w < 16; ++w) {
    uint32_t e = meq[tid * kMaskStride + w];
    uint32_t taken = 0;
    while (e != 0 && left > 0) {
      const uint32_t low = e & (0u - e);
      taken |= low;
      e ^= low;
      --left;
    }
    words[w] = mgt[tid * kMaskStride + w] | taken;
  }
  uint4* dst = reinterpret_cast<uint4*>(p.sent_bits + (size_t)(pm.seg0 + tid) * 16);
#pragma unroll
  for (int w = 0; w < 4; ++w)
    dst[w] = make_uint4(words[4 * w], words[4 * w + 1], words[4 * w + 2], words[4 * w + 3]);
}

// (three blocks per SM: the rare paths may spill, the usual one must not lose occupancy)
__global__ void __launch_bounds__(kEmitThreads, 3)
k_emit_mask(Plan p, int32_t* __restrict__ out_idx, float* __restrict__ out_val) {
  pdl_enter();
  timeline_mark(p.timeline, 3);
  extern __shared__ uint32_t smask[];          // winner bitmaps of the part: [gt | eq]
  __shared__ int sh[66];
  __shared__ int s_gtb[kPartSegs];             // winners before each segment
  __shared__ int s_eqb[kPartSegs];
  static_assert(kEmitSmemBytes >= kHistWords(kEmitThreads) * 4, "bitmaps double as histograms");
  uint32_t* mgt = smask;
  uint32_t* meq = smask + kPartSegs * kMaskStride;
  const int part = blockIdx.x;
  const int tid = threadIdx.x;
  // the call's last kernel counts the call: nothing in this grid reads the counter, and the
  // next call's kernels start after this grid has finished
  if (part == 0 && tid == 0) *p.iter += 1;
  // one round of independent loads: part record, selection result, candidate count
  const PartMeta pm = load_record(p.pm + part);
  PartSel ps = load_record(p.psel + part);
  const int count = __ldcg(p.p_count + part);
  int tensor_first = 0;      // first output slot of the tensor
  if (p.literal) {
    __shared__ int s_first;
    tensor_first = emit_literal_first(p, pm, &s_first);
    ps.out_base += tensor_first;
  }
  if (ps.dense == 1) {
    emit_full_selection(p, pm, part, tensor_first, out_idx, out_val, smask, sh);
    return;
  }
  const uint32_t kth = ps.kth;
  const int quota = ps.quota;
  const int32_t* cidx = p.cand_idx + pm.cbase;
  const float* cval = p.cand_val + pm.cbase;
  // first kEmitRegs candidates of every thread stay in registers
  // (values and indices in one round of loads: the index of a candidate that turns out not to
  // be sent is a wasted word, a dependent second round trip would cost the block's chain more)
  float vals[kEmitRegs];
  int locs[kEmitRegs];
#pragma unroll
  for (int b = 0; b < kEmitRegs; ++b) {
    const int i = b * kEmitThreads + tid;
    vals[b] = i < count ? __ldcg(cval + i) : 0.0f;
    locs[b] = i < count ? __ldcg(cidx + i) : 0;
  }
  // (only the part's own segments: most parts of a many-tensor set are a few segments long)
  for (int i = tid; i < pm.nseg * kMaskStride; i += kEmitThreads) {
    mgt[i] = 0u;
    meq[i] = 0u;
  }
  __syncthreads();
  if (tid == 0) { p.p_count[part] = 0; p.p_eq[part] = 0; }   // ready for the next call
  // mark the candidates that reach the threshold: one bit per element of the part
#pragma unroll
  for (int b = 0; b < kEmitRegs; ++b) {
    const int i = b * kEmitThreads + tid;
    const uint32_t key = mag_key(vals[b]);
    const int local = locs[b] - pm.seg0 * kSeg;
    locs[b] = -1;
    if (i < count && key >= kth) {
      locs[b] = local;
      const int word = (local >> 9) * kMaskStride + ((local >> 5) & 15);
      atomicOr((key > kth ? mgt : meq) + word, 1u << (local & 31));
    }
  }
  // longer lists (low sparsity): the rest in batches of four loads per array
  for (int i0 = kEmitRegs * kEmitThreads; i0 < count; i0 += 4 * kEmitThreads) {
    float v4[4];
    int x4[4];
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int i = i0 + b * kEmitThreads + tid;
      v4[b] = i < count ? __ldcg(cval + i) : 0.0f;
      x4[b] = i < count ? __ldcg(cidx + i) : 0;
    }
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int i = i0 + b * kEmitThreads + tid;
      const uint32_t key = mag_key(v4[b]);
      if (i < count && key >= kth) {
        const int local = x4[b] - pm.seg0 * kSeg;
        const int word = (local >> 9) * kMaskStride + ((local >> 5) & 15);
        atomicOr((key > kth ? mgt : meq) + word, 1u << (local & 31));
      }
    }
  }
  __syncthreads();
  const bool tie_fill = ps.dense == 2 && quota > 0;   // no quota: the part sends candidates only
  if (tie_fill) {
    // tie-fill selection: the ties are the part's entries whose key is the threshold; they are
    // in no candidate list, so the part is read (one warp per segment, one ballot per word)
    const int lane = tid & 31;
    for (int sgm = tid >> 5; sgm < pm.nseg; sgm += kEmitThreads / 32) {
      const int base = (pm.seg0 + sgm) * kSeg;
#pragma unroll 1
      for (int w0 = 0; w0 < 16; w0 += 4) {
        float x[4];
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          const int e = base + (w0 + w) * 32 + lane;
          x[w] = e < pm.end ? __ldcg(p.v + e) : 0.0f;
        }
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          const int e = base + (w0 + w) * 32 + lane;
          const uint32_t word = __ballot_sync(0xFFFFFFFFu, e < pm.end && mag_key(x[w]) == kth);
          if (lane == 0) meq[sgm * kMaskStride + w0 + w] = word;
        }
      }
    }
    __syncthreads();
  }
  // thread s owns segment s: popcounts (the count of the segment's first eight words goes to
  // its padding word), then winners before each segment
  bool has_eq;
  {
    int gt = 0, eq = 0;
    if (tid < pm.nseg) {
#pragma unroll
      for (int w = 0; w < 16; ++w) {
        if (w == 8) {
          mgt[tid * kMaskStride + 16] = (uint32_t)gt;
          meq[tid * kMaskStride + 16] = (uint32_t)eq;
        }
        gt += __popc(mgt[tid * kMaskStride + w]);
        eq += __popc(meq[tid * kMaskStride + w]);
      }
    }
    int bg, be, tg, te;
    block_excl_scan2(gt, eq, sh, bg, be, tg, te);
    s_gtb[tid] = bg;
    s_eqb[tid] = be;
    has_eq = te > 0;                             // hardly ever: then the tie counts are skipped
  }
  __syncthreads();
  auto emit = [&](int local, float val, uint32_t key) {
    const int s = local >> 9, w = (local >> 5) & 15;
    const uint32_t below = (1u << (local & 31)) - 1u;
    const uint32_t* mg = mgt + s * kMaskStride;
    const int x0 = w & 8;                        // words before x0 are in the padding word's count
    int lg = __popc(mg[w] & below) + (x0 ? (int)mg[16] : 0);
    for (int x = x0; x < w; ++x) lg += __popc(mg[x]);
    int le = 0;
    if (has_eq) {
      const uint32_t* me = meq + s * kMaskStride;
      le = __popc(me[w] & below) + (x0 ? (int)me[16] : 0);
      for (int x = x0; x < w; ++x) le += __popc(me[x]);
    }
    const int eq_before = s_eqb[s] + le;         // ties with a lower index, whole part
    int pos;
    if (key > kth) {
      pos = ps.out_base + s_gtb[s] + lg + min(eq_before, quota);
    } else {
      if (eq_before >= quota) return;            // ties: lowest indices first
      pos = ps.out_base + s_gtb[s] + lg + eq_before;
    }
    const int idx = pm.seg0 * kSeg + local;
    out_idx[pos] = idx;
    out_val[pos] = val;
    if (!p.defer_mask) {
      p.u[idx] = 0.0f;
      p.v[idx] = 0.0f;
    }
  };
#pragma unroll
  for (int b = 0; b < kEmitRegs; ++b)
    if (locs[b] >= 0) emit(locs[b], vals[b], mag_key(vals[b]));
  for (int i0 = kEmitRegs * kEmitThreads; i0 < count; i0 += 4 * kEmitThreads) {
    float v4[4];
    int x4[4];
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int i = i0 + b * kEmitThreads + tid;
      v4[b] = i < count ? __ldcg(cval + i) : 0.0f;
      x4[b] = i < count ? __ldcg(cidx + i) : 0;
    }
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int i = i0 + b * kEmitThreads + tid;
      const uint32_t key = mag_key(v4[b]);
      if (i < count && key >= kth) emit(x4[b] - pm.seg0 * kSeg, v4[b], key);
    }
  }
  if (tie_fill) {
    // the tied entries each segment sends (lowest indices first, up to the part's quota): one
    // warp per segment, one lane per entry of a 32-entry word
    const int lane = tid & 31;
    const uint32_t below = (1u << lane) - 1u;
    for (int sgm = tid >> 5; sgm < pm.nseg; sgm += kEmitThreads / 32) {
      int eq_before = s_eqb[sgm];
      if (eq_before >= quota) break;             // s_eqb does not decrease with the segment
      const int base = (pm.seg0 + sgm) * kSeg;
      int lg = s_gtb[sgm];
#pragma unroll 1
      for (int w0 = 0; w0 < 16 && eq_before < quota; w0 += 4) {
        uint32_t ew[4];
        float x[4];
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          ew[w] = meq[sgm * kMaskStride + w0 + w];
          x[w] = (ew[w] >> lane) & 1u ? __ldcg(p.v + base + (w0 + w) * 32 + lane) : 0.0f;
        }
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          const uint32_t gw = mgt[sgm * kMaskStride + w0 + w];
          const int eb = eq_before + __popc(ew[w] & below);
          if (((ew[w] >> lane) & 1u) && eb < quota) {
            const int idx = base + (w0 + w) * 32 + lane;
            const int pos = ps.out_base + lg + __popc(gw & below) + eb;
            out_idx[pos] = idx;
            out_val[pos] = x[w];
            if (!p.defer_mask) {
              p.u[idx] = 0.0f;
              p.v[idx] = 0.0f;
            }
          }
          eq_before += __popc(ew[w]);
          lg += __popc(gw);
        }
      }
    }
  }
  if (p.defer_mask) emit_record_sent(p, pm, quota, mgt, meq, s_eqb);
}

// ------------------------------------------------------------------ K5b: ordered emission from v' itself
// The same step at low sparsity (warm-up stages: a quarter of every tensor is sent).  There the
// candidate lists are long and marking and placing each candidate costs more than reading the
// part again, so the winners are found in v' itself -- which still holds the unmasked values,
// because masking is deferred at these sparsities.  One warp per 512-entry segment, float4 loads
// as in the streaming pass: a first pass counts each segment's winners, a block scan gives
// every segment its first slot, a second pass re-reads the segment, ranks its winners with one
// packed warp scan per 128 entries and stores the pairs in index order; the sent bits for the
// deferred masking are assembled from the lanes' 4-bit flags by shuffles.  No bitmaps, no
// atomics.  Candidate indices are not needed (k_update_emit does not write them in this
// mode); the candidate values only feed the selection kernels.  Tie-fill selections need
// nothing special here: the ties are found like every other entry.
__global__ void __launch_bounds__(kEmitThreads, 3)
k_emit_dense(Plan p, int32_t* __restrict__ out_idx, float* __restrict__ out_val) {
  pdl_enter();
  timeline_mark(p.timeline, 3);
  __shared__ uint32_t hist[kHistWords(kEmitThreads)];   // full-selection path only
  __shared__ int sh[66];
  __shared__ uint32_t s_cnt[kDenseChunk];      // per segment of the chunk: winners | ties << 16
  __shared__ uint32_t s_base[kDenseChunk + 1]; // the same before each segment; [64]: chunk total
  const int part = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (part == 0 && tid == 0) *p.iter += 1;     // the call's last kernel counts the call
  const PartMeta pm = load_record(p.pm + part);
  PartSel ps = load_record(p.psel + part);
  int tensor_first = 0;
  if (p.literal) {
    __shared__ int s_first;
    tensor_first = emit_literal_first(p, pm, &s_first);
    ps.out_base += tensor_first;
  }
  if (ps.dense == 1) {
    emit_full_selection(p, pm, part, tensor_first, out_idx, out_val, hist, sh);
    return;
  }
  const uint32_t kth = ps.kth;
  const int quota = ps.quota;
  if (tid == 0) { p.p_count[part] = 0; p.p_eq[part] = 0; }   // ready for the next call
  const float4* v4 = reinterpret_cast<const float4*>(p.v);
  // flags of the four entries of one float4: bits 0-3 "greater", bits 4-7 "tied"
  auto classify = [&](const float4& x, int e) -> uint32_t {
    const uint32_t k0 = mag_key(x.x), k1 = mag_key(x.y), k2 = mag_key(x.z), k3 = mag_key(x.w);
    uint32_t f = (uint32_t)(k0 > kth) | (uint32_t)(k1 > kth) << 1 | (uint32_t)(k2 > kth) << 2 |
                 (uint32_t)(k3 > kth) << 3 | (uint32_t)(k0 == kth) << 4 |
                 (uint32_t)(k1 == kth) << 5 | (uint32_t)(k2 == kth) << 6 |
                 (uint32_t)(k3 == kth) << 7;
    if (e + 4 > pm.end) {                        // ragged end of the tensor
      const int nv = max(0, pm.end - e);
      f &= ((1u << nv) - 1u) * 0x11u;
    }
    return f;
  };
  // The part goes through in chunks of kDenseChunk segments, so that the second pass of a chunk
  // finds in L2 what its first pass read (the chunks of all resident blocks fit there).
  constexpr int kWarps = kEmitThreads / 32, kPer = kDenseChunk / kWarps;
  static_assert(kDenseChunk == 64 && kDenseChunk % kWarps == 0, "two scan warps' worth per chunk");
  uint32_t run = 0;                                // winners | ties << 16 before the chunk ...
  int run_g = ps.out_base, run_e = 0;              // ... unpacked and accumulated over chunks
  for (int c0 = 0; c0 < pm.nseg; c0 += kDenseChunk) {
    // pass 1: winners and ties of each segment of the chunk
#pragma unroll 1
    for (int i = 0; i < kPer; ++i) {
      const int sgm = c0 + warp * kPer + i;
      uint32_t cnt = 0;
      if (sgm < pm.nseg) {
        const int base = (pm.seg0 + sgm) * kSeg;
        float4 x[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) x[r] = __ldcg(v4 + (base >> 2) + r * 32 + lane);
        if (base + kSeg <= pm.end) {
          // whole segment real: plain counting (the kernel is instruction-bound, not HBM-bound,
          // unless the per-entry work stays at a few instructions)
          int cg = 0, ce = 0;
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            const uint32_t k0 = mag_key(x[r].x), k1 = mag_key(x[r].y), k2 = mag_key(x[r].z),
                           k3 = mag_key(x[r].w);
            cg += (k0 > kth) + (k1 > kth) + (k2 > kth) + (k3 > kth);
            ce += (k0 == kth) + (k1 == kth) + (k2 == kth) + (k3 == kth);
          }
          cnt = (uint32_t)cg | ((uint32_t)ce << 16);
        } else {
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            const uint32_t f = classify(x[r], base + (r * 32 + lane) * 4);
            cnt += (uint32_t)__popc(f & 0xFu) | ((uint32_t)__popc(f & 0xF0u) << 16);
          }
        }
        cnt = __reduce_add_sync(0xFFFFFFFFu, cnt);
      }
      if (lane == 0) s_cnt[warp * kPer + i] = cnt;
    }
    __syncthreads();
    if (warp == 0) {
      // exclusive scan of the 64 packed counts (each half stays below 2^16: 64 x 512 entries)
      const uint32_t a = s_cnt[lane], b2 = s_cnt[32 + lane];
      const uint32_t ia = (uint32_t)warp_incl_scan((int)a), ib = (uint32_t)warp_incl_scan((int)b2);
      const uint32_t ta = __shfl_sync(0xFFFFFFFFu, ia, 31);
      s_base[lane] = ia - a;
      s_base[32 + lane] = ta + ib - b2;
      if (lane == 31) s_base[kDenseChunk] = ta + ib;
    }
    __syncthreads();
    // pass 2: the chunk's segments in index order
#pragma unroll 1
    for (int i = 0; i < kPer; ++i) {
      const int sgm = c0 + warp * kPer + i;
      if (sgm >= pm.nseg) break;
      const int base = (pm.seg0 + sgm) * kSeg;
      const uint32_t sb = s_base[warp * kPer + i];
      int lg = run_g + (int)(sb & 0xFFFFu), eqb = run_e + (int)(sb >> 16);
      if ((s_cnt[warp * kPer + i] >> 16) == 0u && base + kSeg <= pm.end) {
        // no ties in a whole segment (the usual case): winners only, one packed scan per two
        // rows (a row holds at most 128 winners)
        lg += min(eqb, quota);
#pragma unroll 1
        for (int r0 = 0; r0 < 4; r0 += 2) {
          float4 x[2];
#pragma unroll
          for (int r = 0; r < 2; ++r) x[r] = __ldcg(v4 + (base >> 2) + (r0 + r) * 32 + lane);
          uint32_t g[2];
#pragma unroll
          for (int r = 0; r < 2; ++r)
            g[r] = (uint32_t)(mag_key(x[r].x) > kth) | (uint32_t)(mag_key(x[r].y) > kth) << 1 |
                   (uint32_t)(mag_key(x[r].z) > kth) << 2 | (uint32_t)(mag_key(x[r].w) > kth) << 3;
          const uint32_t cnt = (uint32_t)__popc(g[0]) | (uint32_t)__popc(g[1]) << 16;
          const uint32_t incl = (uint32_t)warp_incl_scan((int)cnt);
          const uint32_t tot = __shfl_sync(0xFFFFFFFFu, incl, 31);
          const uint32_t excl = incl - cnt;
#pragma unroll
          for (int r = 0; r < 2; ++r) {
            const int e = base + ((r0 + r) * 32 + lane) * 4;
            int pos = lg + (int)((excl >> (16 * r)) & 0xFFFFu);
            if (g[r] & 1u) { out_idx[pos] = e; out_val[pos] = x[r].x; ++pos; }
            if (g[r] & 2u) { out_idx[pos] = e + 1; out_val[pos] = x[r].y; ++pos; }
            if (g[r] & 4u) { out_idx[pos] = e + 2; out_val[pos] = x[r].z; ++pos; }
            if (g[r] & 8u) { out_idx[pos] = e + 3; out_val[pos] = x[r].w; }
            uint32_t word = g[r] << (4 * (lane & 7));
            word |= __shfl_xor_sync(0xFFFFFFFFu, word, 1);
            word |= __shfl_xor_sync(0xFFFFFFFFu, word, 2);
            word |= __shfl_xor_sync(0xFFFFFFFFu, word, 4);
            if ((lane & 7) == 0)
              p.sent_bits[(size_t)(pm.seg0 + sgm) * 16 + 4 * (r0 + r) + (lane >> 3)] = word;
            lg += (int)((tot >> (16 * r)) & 0xFFFFu);
          }
        }
        continue;
      }
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int e = base + (r * 32 + lane) * 4;
        const float4 x = __ldcg(v4 + (e >> 2));
        const uint32_t f = classify(x, e);
        const uint32_t g = f & 0xFu, q = f >> 4;
        const int cnt = __popc(g) | (__popc(q) << 16);
        const int incl = warp_incl_scan(cnt);
        const int tot = __shfl_sync(0xFFFFFFFFu, incl, 31);
        const int excl = incl - cnt;
        int pos_g = lg + (excl & 0xFFFF);          // winners before this lane's entries
        int eb = eqb + (excl >> 16);               // ties before them, whole part
        const float xs[4] = {x.x, x.y, x.z, x.w};
        uint32_t took = g;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const bool gbit = (g >> c) & 1u;
          const bool ebit = ((q >> c) & 1u) && eb < quota;   // ties: lowest indices first
          if (gbit || ebit) {
            const int pos = pos_g + min(eb, quota);
            out_idx[pos] = e + c;
            out_val[pos] = xs[c];
          }
          if (ebit) took |= 1u << c;
          pos_g += gbit;
          eb += (q >> c) & 1u;
        }
        // the eight lanes that share a 32-entry word put their 4-bit flags together
        uint32_t word = took << (4 * (lane & 7));
        word |= __shfl_xor_sync(0xFFFFFFFFu, word, 1);
        word |= __shfl_xor_sync(0xFFFFFFFFu, word, 2);
        word |= __shfl_xor_sync(0xFFFFFFFFu, word, 4);
        // deferred masking: sent word 4r + lane/8 of the segment
        if ((lane & 7) == 0) p.sent_bits[(size_t)(pm.seg0 + sgm) * 16 + 4 * r + (lane >> 3)] = word;
        lg += tot & 0xFFFF;
        eqb += tot >> 16;
      }
    }
    run = s_base[kDenseChunk];
    run_g += (int)(run & 0xFFFFu);
    run_e += (int)(run >> 16);
    __syncthreads();                               // before the next chunk reuses the tables
  }
}

// Applies (and clears) whatever k_emit_mask left in sent_bits: u = v = 0 at the recorded
// entries.  Used when the state is read out or the masking mode changes.
__global__ void __launch_bounds__(256)
k_apply_pending_mask(Plan p, long long words) {
  pdl_enter();
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long w = (long long)blockIdx.x * blockDim.x + threadIdx.x; w < words; w += stride) {
    uint32_t bits = p.sent_bits[w];
    if (bits) {
      p.sent_bits[w] = 0u;
      while (bits) {
        const int b = __ffs(bits) - 1;
        bits &= bits - 1;
        p.u[w * 32 + b] = 0.0f;
        p.v[w * 32 + b] = 0.0f;
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

// The lists are the caller's: an index outside [0, dense_len) or out of order must neither
// write outside a bounds row or a tile nor read outside a list.  Tile numbers are clamped to
// [0, num_tiles] here, k_decode_tiles clamps the boundaries to the list and skips every pair
// that does not fall into its tile; what was wrong is counted per block (`rejected`:
// [worker][kDecodeBoundsBlocks], every word rewritten by every call, no atomics, no reset).
constexpr int kDecodeBoundsBlocks = 1024;   // blocks per worker at most = reject words per worker

__global__ void __launch_bounds__(256)
k_decode_bounds(const __grid_constant__ DecodeArgs a, int32_t* __restrict__ bounds,
                int32_t* __restrict__ rejected, long long dense_len) {
  pdl_enter();
  // bounds[w * (num_tiles + 1) + t] = first position in list w whose index >= t * tile
  __shared__ int s_bad[256 / 32];
  const int w = blockIdx.y;
  const long long n = a.nnz[w];
  const int32_t* idx = a.idx[w];
  int32_t* b = bounds + (size_t)w * (a.num_tiles + 1);
  auto tile_of = [&](int x) { return x < 0 ? 0 : min(x / kDecodeTile, a.num_tiles); };
  int bad = 0;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i <= n;
       i += (long long)gridDim.x * blockDim.x) {
    const int prev = i == 0 ? -1 : __ldg(idx + i - 1);
    const int cur = i == n ? 0x7FFFFFFF : __ldg(idx + i);
    // pair i breaks the precondition: outside the dense range, or not above its predecessor
    if (i < n && ((unsigned long long)(long long)cur >= (unsigned long long)dense_len ||
                  (i > 0 && cur <= prev)))
      ++bad;
    const int t_prev = i == 0 ? -1 : tile_of(prev);
    const int t_cur = i == n ? a.num_tiles : tile_of(cur);
    for (int t = t_prev + 1; t <= t_cur; ++t) b[t] = (int32_t)i;
  }
  bad = __reduce_add_sync(0xFFFFFFFFu, bad);
  if ((threadIdx.x & 31) == 0) s_bad[threadIdx.x >> 5] = bad;
  __syncthreads();
  if (threadIdx.x == 0) {
    int tot = 0;
    for (int q = 0; q < 256 / 32; ++q) tot += s_bad[q];
    rejected[w * kDecodeBoundsBlocks + blockIdx.x] = tot;
  }
  // the words of blocks that this launch does not have
  if (blockIdx.x == 0)
    for (int q = gridDim.x + threadIdx.x; q < kDecodeBoundsBlocks; q += blockDim.x)
      rejected[w * kDecodeBoundsBlocks + q] = 0;
}

// MODE 0: the tile of the dense gradient is written out (zero-fill fused).
// MODE 1 (Eq. 5, third term applied directly): `dense` is the weight array; only the entries
// some worker lists are updated, w <- w - lr * G with G summed as above -- bit for bit what
// the dense gradient followed by k_sgd gives, because w - lr * (+0) = w.
// MODE 2: MODE 0 plus the SGD step on `weights` in the same pass (the tile of G is still in
// shared memory when w is updated, so G is not read back): 12 B/element instead of 16.
constexpr int kDecodeDense = 0, kDecodeSparseSgd = 1, kDecodeDenseSgd = 2;

template <int MODE>
__global__ void __launch_bounds__(kDecodeThreads)
k_decode_tiles(const __grid_constant__ DecodeArgs a, const int32_t* __restrict__ bounds,
               float* __restrict__ dense, float* __restrict__ weights, long long dense_len,
               float lr) {
  constexpr bool SGD = MODE == kDecodeSparseSgd;
  pdl_enter();
  __shared__ float tile[kDecodeTile];
  __shared__ uint32_t touched[kDecodeTile / 32];
  __shared__ int s_lo[DGC_MAX_DECODE_WORKERS];
  __shared__ int s_cum[DGC_MAX_DECODE_WORKERS + 1];   // pairs of workers 0..w-1 inside this tile
  const int t = blockIdx.x;
  const int tid = threadIdx.x;
  const long long base = (long long)t * kDecodeTile;
  const int N = a.num_workers;
  if (tid < 32) {
    // the tile's slice of every worker list, and the running pair count in worker order
    int run = 0;
    for (int w0 = 0; w0 < N; w0 += 32) {
      const int w = w0 + tid;
      int lo = 0, len = 0;
      if (w < N) {
        // (clamped to the list: a list that is not ascending leaves boundaries unordered)
        const int32_t* b = bounds + (size_t)w * (a.num_tiles + 1);
        lo = min(max(__ldg(b + t), 0), a.nnz[w]);
        len = min(max(__ldg(b + t + 1), lo), a.nnz[w]) - lo;
        s_lo[w] = lo;
      }
      const int incl = warp_incl_scan(len);
      if (w < N) s_cum[w] = run + incl - len;
      run += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
    if (tid == 0) s_cum[N] = run;
  }
  if (SGD) {
    __syncthreads();
    if (s_cum[N] == 0) return;                    // nothing listed in this tile: w is unchanged
    if (tid < kDecodeTile / 32) touched[tid] = 0u;
  }
#pragma unroll
  for (int i = tid; i < kDecodeTile; i += kDecodeThreads) tile[i] = 0.0f;
  __syncthreads();
  const int total = s_cum[N];
  // pairs in (worker, position) order, a block's worth at a time: all loads of a chunk are
  // issued together, then the adds run one worker after the other (worker order, and no two
  // threads touch one slot between barriers because indices are unique within a worker)
  for (int q0 = 0; q0 < total; q0 += kDecodeThreads) {
    const int q = q0 + tid;
    int myw = -1, l = 0;
    float v = 0.0f;
    if (q < total) {
      int lo = 0, hi = N;                        // largest w with s_cum[w] <= q
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (s_cum[mid] <= q) lo = mid; else hi = mid;
      }
      myw = lo;
      const int pos = s_lo[lo] + (q - s_cum[lo]);
      l = (int)((unsigned)__ldg(a.idx[lo] + pos) - (unsigned)base);
      v = __ldg(a.val[lo] + pos);
      // a pair that is not of this tile (bad index; k_decode_bounds counted it) is skipped
      if ((unsigned)l >= (unsigned)kDecodeTile || base + l >= dense_len) myw = -1;
    }
    // workers present in this chunk (block-uniform bounds)
    int wfirst = 0, wlast = N - 1;
    {
      const int qa = q0, qb = min(q0 + kDecodeThreads, total) - 1;
      int lo = 0, hi = N;
      while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (s_cum[mid] <= qa) lo = mid; else hi = mid; }
      wfirst = lo;
      lo = 0; hi = N;
      while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (s_cum[mid] <= qb) lo = mid; else hi = mid; }
      wlast = lo;
    }
    for (int w = wfirst; w <= wlast; ++w) {
      if (myw == w) tile[l] = __fadd_rn(tile[l], v);
      __syncthreads();
    }
    if (SGD && myw >= 0) atomicOr(&touched[l >> 5], 1u << (l & 31));
  }
  if (SGD) {
    __syncthreads();
    for (int i = tid; i < kDecodeTile; i += kDecodeThreads) {
      if ((touched[i >> 5] >> (i & 31)) & 1u) {
        float* wp = dense + base + i;
        *wp = __fsub_rn(*wp, __fmul_rn(lr, tile[i]));
      }
    }
    return;
  }
  const long long rem = dense_len - base;
  if (rem >= kDecodeTile) {
    float4* d4 = reinterpret_cast<float4*>(dense + base);
    const float4* t4 = reinterpret_cast<const float4*>(tile);
    if (MODE == kDecodeDenseSgd) {
      float4* w4 = reinterpret_cast<float4*>(weights + base);
      float4 wv[kDecodeTile / 4 / kDecodeThreads];
#pragma unroll
      for (int q = 0; q < kDecodeTile / 4 / kDecodeThreads; ++q)
        wv[q] = __ldcs(w4 + q * kDecodeThreads + tid);
#pragma unroll
      for (int q = 0; q < kDecodeTile / 4 / kDecodeThreads; ++q) {
        const int i = q * kDecodeThreads + tid;
        const float4 gq = t4[i];
        wv[q].x = __fsub_rn(wv[q].x, __fmul_rn(lr, gq.x));
        wv[q].y = __fsub_rn(wv[q].y, __fmul_rn(lr, gq.y));
        wv[q].z = __fsub_rn(wv[q].z, __fmul_rn(lr, gq.z));
        wv[q].w = __fsub_rn(wv[q].w, __fmul_rn(lr, gq.w));
        __stcs(d4 + i, gq);
        __stcs(w4 + i, wv[q]);
      }
    } else {
#pragma unroll
      for (int i = tid; i < kDecodeTile / 4; i += kDecodeThreads) __stcs(d4 + i, t4[i]);
    }
  } else {
    for (int i = tid; i < (int)rem; i += kDecodeThreads) {
      dense[base + i] = tile[i];
      if (MODE == kDecodeDenseSgd)
        weights[base + i] = __fsub_rn(weights[base + i], __fmul_rn(lr, tile[i]));
    }
  }
}

// Alg. 4 "theta <- SGD(theta, G_t)": w <- w - lr*G, two roundings.
__global__ void __launch_bounds__(256)
k_sgd(float* __restrict__ w, const float* __restrict__ G, long long len, float lr) {
  pdl_enter();
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

// ------------------------------------------------------------------ wire format: values + 16-bit zero run lengths
// Sec. 3.1, encode(): 32-bit values of the sent entries + 16-bit lengths of the zero runs.
// Entry t = (run_t, value_t): run_t zeros are skipped, then value_t is stored.  A gap of
// more than 65535 zeros is bridged by filler entries (65535, +0.0f), each standing for 65535
// zeros and one slot holding an explicit zero (the paper gives no rule; this is the reading).
// Both directions are an exclusive prefix sum over the list -- fillers per entry when
// encoding, run + 1 when decoding -- done as block sums, one block scanning the block sums,
// and a write pass (three launches, no block waits for another).
constexpr int kRleThreads = 256;
constexpr int kRlePer = 4;                         // entries per thread
constexpr int kRleBlock = kRleThreads * kRlePer;   // entries per block

// ENCODE: x_i = fillers before entry i = (zeros before it) >> 16.   DECODE: x_t = run_t + 1.
template <bool ENCODE>
__device__ __forceinline__ uint32_t rle_term(const int32_t* idx, const uint16_t* runs, long long i) {
  if (ENCODE) {
    const long long prev = i == 0 ? -1 : (long long)__ldg(idx + i - 1);
    return (uint32_t)(((long long)__ldg(idx + i) - prev - 1) >> 16);
  }
  return (uint32_t)__ldg(runs + i) + 1u;
}

template <bool ENCODE>
__global__ void __launch_bounds__(kRleThreads)
k_rle_block_sums(const int32_t* __restrict__ idx, const uint16_t* __restrict__ runs, long long n,
                 unsigned long long* __restrict__ block_sums) {
  pdl_enter();
  __shared__ unsigned long long swarp[kRleThreads / 32];
  const long long base = (long long)blockIdx.x * kRleBlock + threadIdx.x * kRlePer;
  unsigned long long s = 0;
#pragma unroll
  for (int q = 0; q < kRlePer; ++q)
    if (base + q < n) s += rle_term<ENCODE>(idx, runs, base + q);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
  if ((threadIdx.x & 31) == 0) swarp[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long t = 0;
    for (int w = 0; w < kRleThreads / 32; ++w) t += swarp[w];
    block_sums[blockIdx.x] = t;
  }
}

// One block: exclusive scan of the block sums in place; total (plus `add`) to *total_out.
__global__ void __launch_bounds__(1024)
k_rle_scan_sums(unsigned long long* __restrict__ block_sums, int nblocks, long long add,
                long long* __restrict__ total_out) {
  pdl_enter();
  __shared__ unsigned long long swarp[32];
  __shared__ unsigned long long s_run;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) s_run = 0;
  __syncthreads();
  for (int b0 = 0; b0 < nblocks; b0 += 1024) {
    const int b = b0 + tid;
    const unsigned long long x = b < nblocks ? block_sums[b] : 0ull;
    unsigned long long incl = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) swarp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      const unsigned long long w = swarp[lane];
      unsigned long long wi = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, wi, o);
        if (lane >= o) wi += t;
      }
      swarp[lane] = wi - w;
    }
    __syncthreads();
    const unsigned long long run = s_run;
    const unsigned long long ex = run + swarp[warp] + incl - x;
    if (b < nblocks) block_sums[b] = ex;
    __syncthreads();
    if (tid == 1023) s_run = ex + x;
    __syncthreads();
  }
  if (tid == 0) *total_out = (long long)s_run + add;
}

template <bool ENCODE>
__global__ void __launch_bounds__(kRleThreads)
k_rle_write(const int32_t* __restrict__ idx, const float* __restrict__ val,
            const uint16_t* __restrict__ runs, long long n,
            const unsigned long long* __restrict__ block_sums, uint16_t* __restrict__ runs_out,
            float* __restrict__ values_out, int32_t* __restrict__ idx_out, long long capacity) {
  pdl_enter();
  __shared__ unsigned long long swarp[kRleThreads / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long base = (long long)blockIdx.x * kRleBlock + tid * kRlePer;
  uint32_t x[kRlePer];
  unsigned long long s = 0;
#pragma unroll
  for (int q = 0; q < kRlePer; ++q) {
    x[q] = base + q < n ? rle_term<ENCODE>(idx, runs, base + q) : 0u;
    s += x[q];
  }
  unsigned long long incl = s;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) swarp[warp] = incl;
  __syncthreads();
  unsigned long long before = block_sums[blockIdx.x] + incl - s;
  for (int w = 0; w < warp; ++w) before += swarp[w];
#pragma unroll
  for (int q = 0; q < kRlePer; ++q) {
    const long long i = base + q;
    if (i < n) {
      if (ENCODE) {
        // entry i goes after the `before` fillers of earlier entries and its own x fillers
        long long o = i + (long long)before;
        for (uint32_t f = 0; f < x[q]; ++f, ++o) {
          if (o < capacity) { runs_out[o] = 65535; values_out[o] = 0.0f; }
        }
        const long long prev = i == 0 ? -1 : (long long)__ldg(idx + i - 1);
        const long long gap = (long long)__ldg(idx + i) - prev - 1;
        if (o < capacity) {
          runs_out[o] = (uint16_t)(gap - ((long long)x[q] << 16));
          values_out[o] = __ldg(val + i);
        }
      } else {
        // entry i sits run_i positions after everything before it
        idx_out[i] = (int32_t)((long long)before + (long long)x[q] - 1);
        values_out[i] = __ldg(val + i);
      }
    }
    before += x[q];
  }
}

}  // namespace dgc
