// CPU oracle for the entropy-aware verify step of Hierarchical Speculative Decoding (HSD).
//
// THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, scalar fp64 restatement of what the
// verify step computes, written to be checked against the paper by eye.  It shares no code, header, table or
// helper with the CUDA library; only the test-suite, the smoke check and the benchmark's CPU-baseline leg may
// build, load or call it.
//
// What it follows:
//   * HSD section, entropy definition  H = -sum_i p_i log p_i  (natural log), p = softmax of the verifier's
//     LM-head logits at one verify position.
//   * HSD section, gate  g(t) = 1[H < tau]  (strict), and Eq. (1): a gated position takes the draft token,
//     any other position falls back to the verifier (Algorithm 1, the HSD loop).
//   * The paper does not say how the verifier decides.  The reading taken here is the speculative-sampling
//     rule: accept the draft token x with probability min(1, p(x)/q(x)); at the first rejection draw the
//     replacement from the normalised residual max(0, p - q); when all k drafts pass, draw one more token from
//     the verifier's distribution at position k.  All randomness is supplied by the caller as uniforms.
//
// Steps, per sequence b, in order (no blocking, no fusion, ascending index order in every sum):
//   1. l[j][v] = sum_h hidden[b,j,h] * W[v,h]                         (fp64, ascending h)
//   2. m_j = max_v l ; s_j = sum_v exp(l - m_j) ; logZ_j = m_j + log s_j ; p_j(v) = exp(l[j][v] - logZ_j)
//   3. H_j = -sum_v p_j(v) * (l[j][v] - logZ_j)   (the definition, term by term; clamped at >= 0)
//   4. for j = 0..k-1: H_j < tau -> accept; else accept iff u_j < min(1, p_j(x_j)/q_j(x_j)); stop at the first
//      position that is not accepted; accept_len = number accepted.
//   5. n = accept_len.  r(v) = max(0, p_n(v) - q_n(v)) if n < k, else r(v) = p_k(v).  R = sum_v r(v).
//      If R <= 0 then r = p_n.  next_tok = smallest v whose running sum c(v) = sum_{w<=v} r(w) exceeds u_k * R.
//   6. decision margins, so that a comparison can tell a near-tie from an error.
//
// Two variants of steps 4-5, selected by arguments (defaults reproduce the steps above):
//   gate_source = 1: the gate looks at the entropy of the DRAFT distribution, H^q_j = -sum_v q_j(v) ln q_j(v), which
//      is how the HSD section's prose describes H (a measure of how unsure the draft model is); q is used as given, terms
//      with q = 0 contribute 0, the result is clamped at >= 0.  The target entropy is still computed and returned.
//   fallback = 1: the verifier decides greedily (Eq. 1 read as "take the verifier's own token"): at a position
//      where the gate is off the draft token is kept iff it equals argmax_v p_j(v) (lowest token id on ties);
//      the token that follows the accepted run is argmax p_n.  No uniform is consumed.
//
// Parity pins live in tests/test_oracle_pins.py (closed forms, invariants, exact-integer products, brute-force
// marginals on 8- and 16-token vocabularies).  The choice of verifier rule itself (step 4/5) has no counterpart
// in the authors' code to compare with: "parity unpinned" for that choice, pinned for its arithmetic.
//
// Build: g++ -O2 -fopenmp -shared -fPIC (no -ffast-math: summation order is part of the definition).

#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

enum RefDtype { REF_BF16 = 0, REF_F32 = 1, REF_F64 = 2 };

// bf16 is the upper 16 bits of an IEEE-754 binary32; widening is exact.
inline double widen_bf16(uint16_t bits) {
  uint32_t w = static_cast<uint32_t>(bits) << 16;
  float f;
  std::memcpy(&f, &w, sizeof f);
  return static_cast<double>(f);
}

inline double load_as_double(const void* base, int dtype, size_t idx) {
  switch (dtype) {
    case REF_BF16: return widen_bf16(static_cast<const uint16_t*>(base)[idx]);
    case REF_F32:  return static_cast<double>(static_cast<const float*>(base)[idx]);
    default:       return static_cast<const double*>(base)[idx];
  }
}

const double kInf = std::numeric_limits<double>::infinity();

// Step 2 and 3 for one row of logits.
void softmax_entropy_row(const double* l, int V, double* logZ_out, double* H_out) {
  double m = l[0];
  for (int v = 1; v < V; ++v) if (l[v] > m) m = l[v];
  double s = 0.0;
  for (int v = 0; v < V; ++v) s += std::exp(l[v] - m);
  const double logZ = m + std::log(s);
  double H = 0.0;
  for (int v = 0; v < V; ++v) {
    const double logp = l[v] - logZ;
    const double p = std::exp(logp);
    if (p > 0.0) H -= p * logp;
  }
  if (H < 0.0) H = 0.0;
  *logZ_out = logZ;
  *H_out = H;
}

// Steps 2-6 for one sequence, given its (k+1) rows of fp64 logits.
void verify_one_sequence(int k, int V, const double* logits /*[k+1][V]*/, const int32_t* tok /*[k]*/,
                         const void* q /*[k][V]*/, int q_dtype, const float* u /*[k+1]*/, double tau,
                         int gate_source, int fallback,
                         int32_t* accept_len, int32_t* next_tok, double* entropy /*[k+1]*/,
                         double* logZ /*[k+1]*/, double* margin_accept /*[k] or null*/,
                         double* margin_gate /*[k] or null*/, double* margin_cdf /*[1] or null*/,
                         double* draft_entropy /*[k] or null*/, double* margin_argmax /*[k+1] or null*/,
                         uint32_t* flags) {
  for (int j = 0; j <= k; ++j)
    softmax_entropy_row(logits + static_cast<size_t>(j) * V, V, &logZ[j], &entropy[j]);
  for (int j = 0; j < k; ++j) {
    if (margin_accept) margin_accept[j] = kInf;
    if (margin_gate) margin_gate[j] = kInf;
  }

  // Entropy of each draft row (gate_source = 1), by the definition, term by term.
  std::vector<double> Hq(static_cast<size_t>(k), 0.0);
  if (gate_source == 1 || draft_entropy) {
    for (int j = 0; j < k; ++j) {
      double h = 0.0;
      for (int v = 0; v < V; ++v) {
        const double qv = load_as_double(q, q_dtype, static_cast<size_t>(j) * V + v);
        if (qv > 0.0) h -= qv * std::log(qv);
      }
      if (h < 0.0) h = 0.0;
      Hq[j] = h;
      if (draft_entropy) draft_entropy[j] = h;
    }
  }

  // Greedy verifier (fallback = 1): the verifier's own token at every position, lowest id on ties, and the gap
  // to the runner-up as the decision margin.
  std::vector<int32_t> amax(static_cast<size_t>(k) + 1, 0);
  std::vector<double> gap(static_cast<size_t>(k) + 1, kInf);
  if (fallback == 1) {
    for (int j = 0; j <= k; ++j) {
      const double* lj = logits + static_cast<size_t>(j) * V;
      int best = 0;
      for (int v = 1; v < V; ++v) if (lj[v] > lj[best]) best = v;
      double second = -kInf;
      for (int v = 0; v < V; ++v) if (v != best && lj[v] > second) second = lj[v];
      amax[j] = best;
      gap[j] = lj[best] - second;
      if (margin_argmax) margin_argmax[j] = gap[j];
    }
  }

  // Step 4: gate, then the verifier's test, in draft order.
  int n = k;
  for (int j = 0; j < k; ++j) {
    const int32_t x = tok[j];
    if (x < 0 || x >= V) {          // a token outside the vocabulary can never be emitted
      *flags |= 1u;
      n = j;
      break;
    }
    const double gate_value = gate_source == 1 ? Hq[j] : entropy[j];
    if (margin_gate) margin_gate[j] = std::fabs(gate_value - tau);
    if (gate_value < tau) continue;                       // fast path: gate fired
    if (fallback == 1) {
      if (margin_accept) margin_accept[j] = gap[j];
      if (x != amax[j]) { n = j; break; }
      continue;
    }
    double uj = static_cast<double>(u[j]);
    if (!(uj >= 0.0)) { uj = 0.0; *flags |= 2u; }
    if (uj >= 1.0) { uj = static_cast<double>(std::nextafter(1.0f, 0.0f)); *flags |= 2u; }
    const double px = std::exp(logits[static_cast<size_t>(j) * V + x] - logZ[j]);
    const double qx = load_as_double(q, q_dtype, static_cast<size_t>(j) * V + x);
    double ratio;
    if (qx > 0.0) { ratio = px / qx; if (ratio > 1.0) ratio = 1.0; }
    else          { ratio = (px > 0.0) ? 1.0 : 0.0; }
    if (margin_accept) margin_accept[j] = std::fabs(uj - ratio);
    if (!(uj < ratio)) { n = j; break; }
  }
  *accept_len = n;
  if (fallback == 1) {              // greedy: the verifier's own token follows the accepted run
    *next_tok = amax[n];
    if (margin_cdf) *margin_cdf = kInf;
    return;
  }

  // Step 5: residual (or the verifier's own distribution at the bonus position) and inverse-CDF draw.
  const double* ln = logits + static_cast<size_t>(n) * V;
  std::vector<double> r(static_cast<size_t>(V));
  double R = 0.0;
  for (int v = 0; v < V; ++v) {
    const double p = std::exp(ln[v] - logZ[n]);
    double rv = p;
    if (n < k) {
      rv = p - load_as_double(q, q_dtype, static_cast<size_t>(n) * V + v);
      if (!(rv > 0.0)) rv = 0.0;
    }
    r[v] = rv;
    R += rv;
  }
  if (!(R > 0.0)) {                 // p <= q everywhere (possible only when sum q > 1): fall back to p
    *flags |= 8u;
    R = 0.0;
    for (int v = 0; v < V; ++v) { r[v] = std::exp(ln[v] - logZ[n]); R += r[v]; }
  }
  double uk = static_cast<double>(u[k]);
  if (!(uk >= 0.0)) { uk = 0.0; *flags |= 2u; }
  if (uk >= 1.0) { uk = static_cast<double>(std::nextafter(1.0f, 0.0f)); *flags |= 2u; }
  const double target = uk * R;
  double c = 0.0, c_before = 0.0;
  int pick = -1, last_positive = -1;
  for (int v = 0; v < V; ++v) {
    if (r[v] > 0.0) last_positive = v;
    const double c_new = c + r[v];
    if (c_new > target) { pick = v; c_before = c; c = c_new; break; }
    c = c_new;
  }
  if (pick < 0) {                   // rounding left the running sum a hair below u*R: take the last token with mass
    pick = last_positive;
    c_before = c - r[pick];
  }
  *next_tok = pick;
  if (margin_cdf) {
    const double lo = target - c_before, hi = c - target;
    *margin_cdf = (lo < hi ? lo : hi) / R;
  }
}

}  // namespace

extern "C" {

// Step 1 alone: logits64[r][v] for r in [0, M).  hidden is [M][H], W is [V][H], dtype codes as RefDtype.
int hola_ref_logits(int M, int H, int V, const void* hidden, const void* W, int in_dtype, double* logits64,
                    int nthreads) {
  if (M < 0 || H <= 0 || V <= 0 || !hidden || !W || !logits64) return 1;
#ifdef _OPENMP
  if (nthreads > 0) omp_set_num_threads(nthreads);
#endif
  // Widen the (small) hidden block once; the dot products below still run in ascending h.
  std::vector<double> hd(static_cast<size_t>(M) * H);
  for (size_t i = 0; i < hd.size(); ++i) hd[i] = load_as_double(hidden, in_dtype, i);
#pragma omp parallel for schedule(static)
  for (int v = 0; v < V; ++v) {
    std::vector<double> w(static_cast<size_t>(H));
    for (int h = 0; h < H; ++h) w[h] = load_as_double(W, in_dtype, static_cast<size_t>(v) * H + h);
    for (int r = 0; r < M; ++r) {
      const double* hr = hd.data() + static_cast<size_t>(r) * H;
      double acc = 0.0;
      for (int h = 0; h < H; ++h) acc += hr[h] * w[h];
      logits64[static_cast<size_t>(r) * V + v] = acc;
    }
  }
  return 0;
}

// Steps 2-3 alone for M rows of given fp64 logits.
int hola_ref_softmax_entropy(int M, int V, const double* logits64, double* logZ, double* entropy) {
  if (M < 0 || V <= 0 || !logits64 || !logZ || !entropy) return 1;
  for (int r = 0; r < M; ++r)
    softmax_entropy_row(logits64 + static_cast<size_t>(r) * V, V, &logZ[r], &entropy[r]);
  return 0;
}

// Steps 2-6 from given fp64 logits [B][k+1][V].  q is [B][k][V] in q_dtype.  Margin pointers may be null.
// flags_out (optional, [B]): bit0 bad token, bit1 uniform outside [0,1), bit3 residual mass was zero.
// gate_source / fallback select the variants described at the top; draft_entropy ([B][k]) and margin_argmax
// ([B][k+1]) are optional outputs.
int hola_verify_from_logits_ref_ex(int B, int k, int V, const double* logits64, const int32_t* draft_tok,
                                   const void* draft_q, int q_dtype, const float* uniforms, double tau,
                                   int gate_source, int fallback,
                                   int32_t* accept_len, int32_t* next_tok, double* entropy, double* logZ,
                                   double* margin_accept, double* margin_gate, double* margin_cdf,
                                   double* draft_entropy, double* margin_argmax, uint32_t* flags_out) {
  if (B < 0 || k < 0 || V <= 0 || !logits64 || !uniforms || !accept_len || !next_tok || !entropy || !logZ)
    return 1;
  if (k > 0 && (!draft_tok || !draft_q)) return 1;
  if (gate_source < 0 || gate_source > 1 || fallback < 0 || fallback > 1) return 1;
  const size_t qElem = (q_dtype == REF_BF16) ? 2 : (q_dtype == REF_F32 ? 4 : 8);
  for (int b = 0; b < B; ++b) {
    uint32_t flags = 0;
    const char* qb = static_cast<const char*>(draft_q) + static_cast<size_t>(b) * k * V * qElem;
    verify_one_sequence(k, V, logits64 + static_cast<size_t>(b) * (k + 1) * V,
                        draft_tok ? draft_tok + static_cast<size_t>(b) * k : nullptr, qb, q_dtype,
                        uniforms + static_cast<size_t>(b) * (k + 1), tau, gate_source, fallback, &accept_len[b],
                        &next_tok[b], entropy + static_cast<size_t>(b) * (k + 1),
                        logZ + static_cast<size_t>(b) * (k + 1),
                        margin_accept ? margin_accept + static_cast<size_t>(b) * k : nullptr,
                        margin_gate ? margin_gate + static_cast<size_t>(b) * k : nullptr,
                        margin_cdf ? margin_cdf + b : nullptr,
                        draft_entropy ? draft_entropy + static_cast<size_t>(b) * k : nullptr,
                        margin_argmax ? margin_argmax + static_cast<size_t>(b) * (k + 1) : nullptr, &flags);
    if (flags_out) flags_out[b] = flags;
  }
  return 0;
}

int hola_verify_from_logits_ref(int B, int k, int V, const double* logits64, const int32_t* draft_tok,
                                const void* draft_q, int q_dtype, const float* uniforms, double tau,
                                int32_t* accept_len, int32_t* next_tok, double* entropy, double* logZ,
                                double* margin_accept, double* margin_gate, double* margin_cdf,
                                uint32_t* flags_out) {
  return hola_verify_from_logits_ref_ex(B, k, V, logits64, draft_tok, draft_q, q_dtype, uniforms, tau, 0, 0,
                                        accept_len, next_tok, entropy, logZ, margin_accept, margin_gate,
                                        margin_cdf, nullptr, nullptr, flags_out);
}

// The whole verify step.  hidden [B][k+1][H] and W [V][H] in in_dtype; logits64 is optional output/scratch
// ([B][k+1][V]; allocated internally when null).
int hola_verify_ref_ex(int B, int k, int H, int V, const void* hidden, const void* W, int in_dtype,
                       const int32_t* draft_tok, const void* draft_q, int q_dtype, const float* uniforms,
                       double tau, int gate_source, int fallback, int32_t* accept_len, int32_t* next_tok,
                       double* entropy, double* logZ, double* margin_accept, double* margin_gate,
                       double* margin_cdf, double* draft_entropy, double* margin_argmax, double* logits64,
                       uint32_t* flags_out, int nthreads) {
  if (B < 0 || k < 0 || H <= 0 || V <= 0) return 1;
  const size_t M = static_cast<size_t>(B) * (k + 1);
  std::vector<double> own;
  if (!logits64) { own.resize(M * V); logits64 = own.data(); }
  int rc = hola_ref_logits(static_cast<int>(M), H, V, hidden, W, in_dtype, logits64, nthreads);
  if (rc) return rc;
  return hola_verify_from_logits_ref_ex(B, k, V, logits64, draft_tok, draft_q, q_dtype, uniforms, tau, gate_source,
                                        fallback, accept_len, next_tok, entropy, logZ, margin_accept, margin_gate,
                                        margin_cdf, draft_entropy, margin_argmax, flags_out);
}

int hola_verify_ref(int B, int k, int H, int V, const void* hidden, const void* W, int in_dtype,
                    const int32_t* draft_tok, const void* draft_q, int q_dtype, const float* uniforms,
                    double tau, int32_t* accept_len, int32_t* next_tok, double* entropy, double* logZ,
                    double* margin_accept, double* margin_gate, double* margin_cdf, double* logits64,
                    uint32_t* flags_out, int nthreads) {
  return hola_verify_ref_ex(B, k, H, V, hidden, W, in_dtype, draft_tok, draft_q, q_dtype, uniforms, tau, 0, 0,
                            accept_len, next_tok, entropy, logZ, margin_accept, margin_gate, margin_cdf, nullptr,
                            nullptr, logits64, flags_out, nthreads);
}

int hola_ref_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

}  // extern "C"
