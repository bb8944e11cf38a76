// Oracle for the per-worker hot path of Deep Gradient Compression.
//
// TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, single-threaded CPU
// statement of what the path computes, written from the paper.  It shares no
// code with the CUDA library and nothing in the product path may call it.
// Build: g++ -O2 -std=c++17 -ffp-contract=off -fPIC -shared (no fast-math, so
// every fp32 operation below is rounded once, in the order written).
//
// Steps and the passages they follow (Algorithm 4 = "Deep Gradient Compression
// for vanilla momentum SGD on node k", Appendix D):
//   clip coefficient        Sec. 3.2 "Local Gradient Clipping", Appendix C (thr * N^-1/2)
//   momentum correction     Eq. 5 (u <- m u + g ; v <- v + u), Algorithm 4 lines "U <- ...", "V <- ...";
//                           Nesterov form: Algorithm 5 / Appendix B Eq. 8
//   per-tensor selection    Algorithm 4 inner loop over j (thr <- s% of |V[j]|, Mask)
//   emission                Algorithm 4  G~[j] <- V[j] (.) Mask
//   momentum factor masking Sec. 3.3 (V <- V (.) !Mask ; U <- U (.) !Mask)
//   aggregate               Algorithm 4  G_t <- sum_k encode(G~_k)
//   SGD step                Algorithm 4  theta <- SGD(theta, G_t); Eq. 5 third term
//   warm-up sparsities      Sec. 4.1 (75%, 93.75%, 98.4375%, 99.6%, 99.9%)
//
// Readings where the paper leaves a choice (each one is also listed in the
// design notes of the repository):
//   * "s% of |V[j]|" with a strict ">" does not define a count.  Here the mask
//     of tensor j is the exact top-k_j set, k_j = ceil(n_j * (1 - s)), under
//     the total order (|v| as its IEEE bit pattern, descending; index,
//     ascending).  k_j is computed in integers: q = llround((1 - s) * 1e9),
//     k_j = max(1, ceil(n_j * q / 1e9)).
//   * Clipping uses one L2 norm over the worker's whole gradient set and no
//     epsilon: g <- g * thr_local / ||g|| iff ||g|| > thr_local.
//   * The new u enters v (v_t = v_{t-1} + u_t).
//   * Masked entries become +0.0f; the dense sum starts from +0.0f.
//
// Pins (tests/test_oracle_*.py): hand-worked dyadic traces, brute-force full
// sort for n <= 4096, closed forms of Eq. 4/5, conservation, s = 0 reducing to
// plain synchronous SGD, numpy's float64 norm, numpy's stable argsort; for the
// Sec. 5 selection: numpy partition on hand-chosen sample positions (rank
// k_s against k_s +- 1, ties at the threshold, 2k against 2k + 1 passing) and
// the published SplitMix64 outputs for the position generator.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <functional>
#include <utility>
#include <vector>

namespace {

inline uint32_t magnitude_key(float x) {
  uint32_t b;
  std::memcpy(&b, &x, sizeof b);
  return b & 0x7FFFFFFFu;  // monotone in |x|; NaN sorts above Inf
}

struct KeyIdx {
  uint32_t key;
  int64_t idx;
};

// "comes first" in the selection order: larger magnitude, then lower index.
inline bool before(const KeyIdx& a, const KeyIdx& b) {
  if (a.key != b.key) return a.key > b.key;
  return a.idx < b.idx;
}

}  // namespace

extern "C" {

// k_j = ceil(n_j (1 - s)) in integer arithmetic (parts per 1e9), at least 1.
int64_t dgc_oracle_topk_count(int64_t n, double sparsity) {
  const long long q = std::llround((1.0 - sparsity) * 1e9);
  long long k = (static_cast<long long>(n) * q + 999999999LL) / 1000000000LL;
  if (k < 1) k = 1;
  if (k > n) k = n;
  return k;
}

// Sec. 4.1: the sparsity of warm-up stage 0..4.  Returns -1 for other stages.
double dgc_oracle_warmup_sparsity(int32_t stage) {
  switch (stage) {
    case 0: return 0.75;
    case 1: return 0.9375;
    case 2: return 0.984375;
    case 3: return 0.996;
    case 4: return 0.999;
    default: return -1.0;
  }
}

// Sec. 3.2 / Appendix C.  S = sum g^2 over every tensor of the set, left to
// right, in fp64 (each product of two fp32 values is exact in fp64).
// thr_local = thr_G * N^-1/2 ; coef = thr_local / ||g|| when ||g|| > thr_local.
// clip_threshold <= 0 means clipping is off: coef = 1, norm still reported.
void dgc_oracle_clip_coef(int32_t num_tensors, const int64_t* offset, const int64_t* numel,
                          const float* g, double clip_threshold, int32_t num_workers,
                          double* norm_out, float* coef_out) {
  double S = 0.0;
  for (int32_t j = 0; j < num_tensors; ++j) {
    const float* gj = g + offset[j];
    for (int64_t i = 0; i < numel[j]; ++i) {
      const double x = static_cast<double>(gj[i]);
      S += x * x;
    }
  }
  const double norm = std::sqrt(S);
  float coef = 1.0f;
  if (clip_threshold > 0.0) {
    const double thr_local = clip_threshold / std::sqrt(static_cast<double>(num_workers));
    if (norm > thr_local) coef = static_cast<float>(thr_local / norm);
  }
  *norm_out = norm;
  *coef_out = coef;
}

// Eq. 5 / Algorithm 4: u <- m*u + gc ; v <- v + u, with gc = g*coef.
// Three (four with clipping) separately rounded fp32 operations per element.
// nesterov != 0: Algorithm 5 (Appendix B, Eq. 8 with U = m*u): U <- m*(U + gc) ;
// V <- (V + U) + gc, the sum taken left to right as the algorithm prints it.
void dgc_oracle_momentum_correction(int32_t num_tensors, const int64_t* offset,
                                    const int64_t* numel, float* u, float* v, const float* g,
                                    float momentum, float coef, int32_t nesterov) {
  for (int32_t j = 0; j < num_tensors; ++j) {
    const int64_t o = offset[j];
    for (int64_t i = 0; i < numel[j]; ++i) {
      const float gc = g[o + i] * coef;
      if (nesterov) {
        const float t = u[o + i] + gc;
        const float un = momentum * t;
        u[o + i] = un;
        const float w = v[o + i] + un;
        v[o + i] = w + gc;
      } else {
        const float t = momentum * u[o + i];
        const float un = t + gc;
        u[o + i] = un;
        v[o + i] = v[o + i] + un;
      }
    }
  }
}

// The exact top-k set of one tensor under (|v| bits descending, index
// ascending); the k chosen local indices come back ascending.
// brute_force != 0 sorts everything (used by the tests for small n);
// otherwise a selection (nth_element) finds the same set.
void dgc_oracle_select_topk(int64_t n, const float* v, int64_t k, int64_t* sel_idx,
                            int32_t brute_force) {
  std::vector<KeyIdx> a(static_cast<size_t>(n));
  for (int64_t i = 0; i < n; ++i) a[static_cast<size_t>(i)] = KeyIdx{magnitude_key(v[i]), i};
  if (brute_force) {
    std::sort(a.begin(), a.end(), before);
  } else if (k < n) {
    std::nth_element(a.begin(), a.begin() + k, a.end(), before);
  }
  std::vector<int64_t> chosen(static_cast<size_t>(k));
  for (int64_t r = 0; r < k; ++r) chosen[static_cast<size_t>(r)] = a[static_cast<size_t>(r)].idx;
  std::sort(chosen.begin(), chosen.end());
  for (int64_t r = 0; r < k; ++r) sel_idx[r] = chosen[static_cast<size_t>(r)];
}

// One iteration of Algorithm 4 on one worker, from the clipping line to the
// end of the loop over tensors.  All arrays are host memory.
//   offset[j], numel[j] : where tensor j lies in g/u/v (any non-overlapping placement)
//   k[j]                : number of entries to send from tensor j
//   out_offset[j]       : where tensor j's pairs start in out_idx/out_val
//   out_idx             : index into g/u/v (offset[j] + local index), ascending per tensor
//   nesterov            : non-zero selects Algorithm 5's update instead of Algorithm 4's
//   coef_override_flag  : when non-zero, coef_override replaces the computed clip
//                         coefficient (so that state can be compared after two
//                         implementations rounded the norm differently)
// norm_out / coef_out receive the computed norm and the coefficient used.
void dgc_oracle_compress(int32_t num_tensors, const int64_t* offset, const int64_t* numel,
                         const int64_t* k, const int64_t* out_offset, float* u, float* v,
                         const float* g, float momentum, double clip_threshold,
                         int32_t num_workers, int32_t coef_override_flag, float coef_override,
                         int32_t brute_force, int32_t nesterov, int32_t* out_idx, float* out_val,
                         double* norm_out, float* coef_out) {
  // Local gradient clipping, before the accumulation.
  double norm = 0.0;
  float coef = 1.0f;
  dgc_oracle_clip_coef(num_tensors, offset, numel, g, clip_threshold, num_workers, &norm, &coef);
  if (coef_override_flag) coef = coef_override;
  *norm_out = norm;
  *coef_out = coef;

  // Momentum correction.
  dgc_oracle_momentum_correction(num_tensors, offset, numel, u, v, g, momentum, coef, nesterov);

  // Per tensor: select, emit, mask.
  std::vector<int64_t> sel;
  for (int32_t j = 0; j < num_tensors; ++j) {
    const int64_t o = offset[j];
    sel.assign(static_cast<size_t>(k[j]), 0);
    dgc_oracle_select_topk(numel[j], v + o, k[j], sel.data(), brute_force);
    for (int64_t r = 0; r < k[j]; ++r) {
      const int64_t i = o + sel[static_cast<size_t>(r)];
      out_idx[out_offset[j] + r] = static_cast<int32_t>(i);
      out_val[out_offset[j] + r] = v[i];
      v[i] = 0.0f;
      u[i] = 0.0f;
    }
  }
}

// The same iteration with clipping per tensor (an option beside the paper's reading, which
// clips by one norm over the whole set: Sec. 3.2 speaks of "their L2-norms", Appendix C of one
// ||G^k||_2).  Tensor j is rescaled by coef_j = thr_local / ||g[j]||_2 iff ||g[j]||_2 >
// thr_local, thr_local = thr_G N^-1/2 as before; everything after the clipping is unchanged.
//   coef_override : NULL, or one coefficient per tensor that replaces the computed ones
//   norms_out, coefs_out : per tensor, the computed norm and the coefficient used
void dgc_oracle_compress_clip_per_tensor(int32_t num_tensors, const int64_t* offset,
                                         const int64_t* numel, const int64_t* k,
                                         const int64_t* out_offset, float* u, float* v,
                                         const float* g, float momentum, double clip_threshold,
                                         int32_t num_workers, const float* coef_override,
                                         int32_t brute_force, int32_t nesterov, int32_t* out_idx,
                                         float* out_val, double* norms_out, float* coefs_out) {
  std::vector<int64_t> sel;
  for (int32_t j = 0; j < num_tensors; ++j) {
    // clip this tensor by its own norm, then Eq. 5 on it
    double norm = 0.0;
    float coef = 1.0f;
    dgc_oracle_clip_coef(1, offset + j, numel + j, g, clip_threshold, num_workers, &norm, &coef);
    if (coef_override) coef = coef_override[j];
    norms_out[j] = norm;
    coefs_out[j] = coef;
    dgc_oracle_momentum_correction(1, offset + j, numel + j, u, v, g, momentum, coef, nesterov);
    // select, emit, mask: as in dgc_oracle_compress
    const int64_t o = offset[j];
    sel.assign(static_cast<size_t>(k[j]), 0);
    dgc_oracle_select_topk(numel[j], v + o, k[j], sel.data(), brute_force);
    for (int64_t r = 0; r < k[j]; ++r) {
      const int64_t i = o + sel[static_cast<size_t>(r)];
      out_idx[out_offset[j] + r] = static_cast<int32_t>(i);
      out_val[out_offset[j] + r] = v[i];
      v[i] = 0.0f;
      u[i] = 0.0f;
    }
  }
}

// Algorithm 4, aggregation line: G = sum over workers of their sparse
// gradients, added in worker order starting from +0.0f.
void dgc_oracle_decode_accumulate(int32_t num_workers, const int32_t* const* idx_lists,
                                  const float* const* val_lists, const int64_t* nnz,
                                  float* dense, int64_t dense_len) {
  for (int64_t i = 0; i < dense_len; ++i) dense[i] = 0.0f;
  for (int32_t w = 0; w < num_workers; ++w) {
    for (int64_t p = 0; p < nnz[w]; ++p) {
      const int64_t i = idx_lists[w][p];
      dense[i] = dense[i] + val_lists[w][p];
    }
  }
}

// Algorithm 4, last line, with plain SGD (the momentum already lives in u):
// w <- w - lr * G, two roundings.
void dgc_oracle_apply_sgd(float* w, const float* dense_grad, int64_t len, float lr) {
  for (int64_t i = 0; i < len; ++i) {
    const float p = lr * dense_grad[i];
    w[i] = w[i] - p;
  }
}

// Sec. 3.1, encode(): the wire format is 32-bit values plus 16-bit zero run lengths.
// Entry t = (run_t, value_t): run_t zeros are skipped, then value_t
// is stored.  The paper gives no rule for more than 65535 zeros in a row; the reading used
// here bridges the gap with filler entries (65535, +0.0f), each standing for 65535 zeros
// followed by one slot that holds an explicit zero.  Zeros after the last entry are not
// encoded (the receiver knows the dense length).
// idx ascending, no duplicates.  Returns the number of entries written, or -1 if
// `capacity` is too small.  Encoded size = 6 bytes per entry.
int64_t dgc_oracle_encode_runlength(const int32_t* idx, const float* val, int64_t nnz,
                                    uint16_t* runs, float* values, int64_t capacity) {
  int64_t out = 0;
  int64_t pos = 0;                       // next dense position not yet accounted for
  for (int64_t i = 0; i < nnz; ++i) {
    int64_t gap = static_cast<int64_t>(idx[i]) - pos;     // zeros before this entry
    while (gap > 65535) {
      if (out >= capacity) return -1;
      runs[out] = 65535;
      values[out] = 0.0f;
      ++out;
      gap -= 65536;                      // 65535 zeros and the filler's own slot
    }
    if (out >= capacity) return -1;
    runs[out] = static_cast<uint16_t>(gap);
    values[out] = val[i];
    ++out;
    pos = static_cast<int64_t>(idx[i]) + 1;
  }
  return out;
}

// The inverse: entry t lands at position sum_{j<t} (run_j + 1) + run_t.  Fillers come back
// as explicit (index, +0.0f) pairs (they cannot be told from a sent zero), which a sum
// ignores.  Returns the number of pairs (= count).
int64_t dgc_oracle_decode_runlength(const uint16_t* runs, const float* values, int64_t count,
                                    int32_t* idx, float* val) {
  int64_t pos = 0;
  for (int64_t t = 0; t < count; ++t) {
    pos += runs[t];
    idx[t] = static_cast<int32_t>(pos);
    val[t] = values[t];
    pos += 1;
  }
  return count;
}

// ---------------------------------------------------------------------------------------
// The sampled selection as Sec. 5 states it ("paper-literal" mode).  Sec. 5 in short: draw a
// sample of 0.1 % to 1 % of the tensor, take the top-k threshold of the sample as the threshold
// of the whole tensor, and only when far more entries than expected pass it, select precisely
// among those that passed.  The number of entries sent then varies from call to call.
//
// Readings (Sec. 5 gives no numbers beyond the 0.1 % .. 1 % range):
//   * sample size   S = ceil(rho n_j), rho the configured sample ratio (integer arithmetic in
//                   parts per 1e9, like k_j; at least 1, at most n_j); every tensor is sampled
//   * positions     S independent uniform draws from [0, n_j), with replacement; they are an
//                   INPUT of the selection below (the draws come from the counter-based
//                   generator further down, which holds no arithmetic of the method)
//   * threshold     thr = the k_s-th largest sampled |v|, k_s = ceil(S (1 - s)) (the top-k
//                   selection of Alg. 4 applied to the sample, same integer k formula)
//   * mask          |v| > thr over the whole tensor (Alg. 4's strict compare)
//   * "far more than expected" = more than 2 k_j entries pass; then exactly the top k_j of the
//                   tensor are sent (all of them passed, so this is the precise selection
//                   among the already-selected entries; ties go to the lower index)
//   * fewer than k_j pass (also none): what passed is sent as it is

// S = ceil(rho n), at least 1, at most n (rho <= 0 selects the default 1 %).
int64_t dgc_oracle_sample_count(int64_t n, double sample_ratio) {
  const double ratio = sample_ratio > 0.0 ? sample_ratio : 0.01;
  const long long q = std::llround(ratio * 1e9);
  long long S = (static_cast<long long>(n) * q + 999999999LL) / 1000000000LL;
  if (S < 1) S = 1;
  if (S > n) S = n;
  return S;
}

// Selection of one tensor from an explicit sample.  v: the n accumulated values (already
// updated); positions[0..S): the sampled indices, each in [0, n), repeats allowed and counted
// as separate draws.  Returns the number of entries chosen, their indices ascending in sel_idx
// (room for min(n, 2k)).  thr_key_out (may be NULL) receives the threshold's bit pattern.
int64_t dgc_oracle_select_from_sample(int64_t n, const float* v, const int64_t* positions,
                                      int64_t S, int64_t k, double sparsity, int64_t* sel_idx,
                                      uint32_t* thr_key_out) {
  // top-k_s of the sample -> threshold
  std::vector<uint32_t> sample(static_cast<size_t>(S));
  for (int64_t r = 0; r < S; ++r) sample[static_cast<size_t>(r)] = magnitude_key(v[positions[r]]);
  const int64_t ks = dgc_oracle_topk_count(S, sparsity);
  std::sort(sample.begin(), sample.end(), std::greater<uint32_t>());
  const uint32_t thr = sample[static_cast<size_t>(ks - 1)];
  if (thr_key_out) *thr_key_out = thr;
  // mask of the whole tensor
  int64_t passed = 0;
  for (int64_t i = 0; i < n; ++i) passed += magnitude_key(v[i]) > thr;
  if (passed > 2 * k) {
    // far more than expected: the precise top-k_j
    dgc_oracle_select_topk(n, v, k, sel_idx, 0);
    return k;
  }
  int64_t c = 0;
  for (int64_t i = 0; i < n; ++i)
    if (magnitude_key(v[i]) > thr) sel_idx[c++] = i;
  return c;
}

// Counter-based generator of the sample positions (no arithmetic of the method): draw r of
// tensor j in a call is floor(h n / 2^64) with h = mix(call_seed xor (j << 32) xor r), mix =
// the SplitMix64 step (add the golden-ratio increment, then its two multiply-xorshift rounds).
// The CUDA library implements the same generator on its side.
static inline uint64_t oracle_mix64(uint64_t x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}

uint64_t dgc_oracle_mix64(uint64_t x) { return oracle_mix64(x); }

void dgc_oracle_sample_positions(int64_t n, int64_t S, uint64_t call_seed, int32_t tensor_index,
                                 int64_t* positions) {
  for (int64_t r = 0; r < S; ++r) {
    const uint64_t h = oracle_mix64(call_seed ^
                                    (static_cast<uint64_t>(static_cast<uint32_t>(tensor_index)) << 32) ^
                                    static_cast<uint64_t>(r));
    positions[r] = static_cast<int64_t>(
        (static_cast<unsigned __int128>(h) * static_cast<unsigned __int128>(n)) >> 64);
  }
}

// One iteration in paper-literal mode: clip, momentum correction, then per tensor the sample
// positions of this call, the selection from that sample, emission and masking.  The pairs of all tensors are packed back to
// back (tensor order, ascending index); nnz_out[j] = entries sent from tensor j.
// seed/iteration give call_seed = mix(seed * 0x9E3779B97F4A7C15 + iteration) (mod 2^64), so
// that consecutive calls draw unrelated positions.
int64_t dgc_oracle_compress_sampled(int32_t num_tensors, const int64_t* offset,
                                    const int64_t* numel, const int64_t* k, float* u, float* v,
                                    const float* g, float momentum, double clip_threshold,
                                    int32_t num_workers, int32_t coef_override_flag,
                                    float coef_override, int32_t nesterov, double sparsity,
                                    double sample_ratio, uint64_t seed, int64_t iteration,
                                    int32_t* out_idx, float* out_val, int64_t* nnz_out,
                                    double* norm_out, float* coef_out) {
  double norm = 0.0;
  float coef = 1.0f;
  dgc_oracle_clip_coef(num_tensors, offset, numel, g, clip_threshold, num_workers, &norm, &coef);
  if (coef_override_flag) coef = coef_override;
  *norm_out = norm;
  *coef_out = coef;
  dgc_oracle_momentum_correction(num_tensors, offset, numel, u, v, g, momentum, coef, nesterov);
  const uint64_t call_seed =
      oracle_mix64(seed * 0x9E3779B97F4A7C15ull + static_cast<uint64_t>(iteration));
  std::vector<int64_t> sel, pos;
  int64_t out = 0;
  for (int32_t j = 0; j < num_tensors; ++j) {
    const int64_t o = offset[j];
    sel.assign(static_cast<size_t>(std::min(numel[j], 2 * k[j])), 0);
    const int64_t S = dgc_oracle_sample_count(numel[j], sample_ratio);
    pos.assign(static_cast<size_t>(S), 0);
    dgc_oracle_sample_positions(numel[j], S, call_seed, j, pos.data());
    const int64_t c = dgc_oracle_select_from_sample(numel[j], v + o, pos.data(), S, k[j], sparsity,
                                                    sel.data(), nullptr);
    nnz_out[j] = c;
    for (int64_t r = 0; r < c; ++r) {
      const int64_t i = o + sel[static_cast<size_t>(r)];
      out_idx[out] = static_cast<int32_t>(i);
      out_val[out] = v[i];
      ++out;
      v[i] = 0.0f;
      u[i] = 0.0f;
    }
  }
  return out;
}

}  // extern "C"
