// TEST INFRASTRUCTURE — not part of the product path.
//
// Plain fp64 CPU oracle for hybrid-batch attention over a paged bf16 KV cache.
// It is the definition written out: per request, per q head, per new-token row,
// gather the keys through the block table, materialise the mask row explicitly,
// compute scores, softmax and the weighted sum of values in double precision.
// No tiling, no online softmax, no page-run logic, nothing shared with the
// CUDA library (no common header, helper, table or constant).
//
// Only tests, the smoke check and the bench's cpu_baseline / reference arm may
// load this library.
//
// What each function follows (paper = XY-Serve, arXiv 2412.18106):
//   * attention = QK -> Softmax -> SV per tile unit, Section 4.2.1;
//   * K/V read block by block through the block table, valid-token count of the
//     last block tracked, Section 4.1.1; padded positions excluded, Section 5.2;
//   * history columns fully visible and only the specLen x specLen corner
//     masked for verify, Section 4.1.2; causal corner for prefill, Section 4.2.2;
//   * merge of partial results over a split of the K/V dimension = the Update
//     stage, Section 4.2.1.
// Readings taken where the paper is silent: kv_len counts cached tokens BEFORE
// the new ones; tree mask = ancestor-or-self of a parent array in topological
// order; q head a reads kv head floor(a / (Hq/Hkv)); LSE is the natural log of
// the sum of exp(sm_scale * q.k) over allowed keys.
//
// Pins (tests/test_oracle_*.py): softmax rows sum to 1; chunked == unchunked
// prefill; prefix reuse == full recompute; chain tree == causal; decode == last
// prefill row; closed forms (Q = 0, equal keys, constant V, single key, one-hot
// V); star tree; an independently written brute force; torch fp64 softmax /
// logsumexp on gathered K/V; page-permutation invariance; key-shift identity;
// merge identity over arbitrary partitions; GQA special cases; append-then-gather round trip.
//
// fp8 KV-cache variant (an extension beside the paper's method: the paper
// itself defines no fp8 cache, so format, scale granularity and rounding are this build's
// reading - parity unpinned by the paper): K and V are stored as e4m3 bytes (1 sign, 4 exponent
// bits of bias 7, 3 mantissa bits, no infinities, 0x7F / 0xFF = NaN) with one fp32 scale per
// (page, kv head) for K and one for V; the attended value is decode(byte) * scale, exactly, in
// fp64, and everything after that is the same definition as above.  Pins: the 256-entry decode
// against a library conversion; scale = 1 on values representable in e4m3 equals the bf16 path.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// bf16 -> fp64, exact: bf16 is the top 16 bits of an IEEE fp32.
inline double widen(uint16_t b) {
  uint32_t u = static_cast<uint32_t>(b) << 16;
  float f;
  std::memcpy(&f, &u, sizeof f);
  return static_cast<double>(f);
}

// e4m3 ("fn" flavour) byte -> fp64, exact.  exponent field 0: subnormal m/8 * 2^-6; else
// (1 + m/8) * 2^(e-7); exponent 15 with mantissa 7 is NaN (there are no infinities).
inline double decode_e4m3(uint8_t b) {
  const int sign = b >> 7, e = (b >> 3) & 15, m = b & 7;
  double v;
  if (e == 15 && m == 7) v = std::numeric_limits<double>::quiet_NaN();
  else if (e == 0) v = std::ldexp(static_cast<double>(m) / 8.0, -6);
  else v = std::ldexp(1.0 + static_cast<double>(m) / 8.0, e - 7);
  return sign ? -v : v;
}

struct Problem {
  int R, Hq, Hkv, D, B;
  // fp8 variant: byte pools (same strides, in elements) and per-(page, kv head) scales; null = bf16
  const uint8_t* k8 = nullptr;
  const uint8_t* v8 = nullptr;
  const float* k_scale = nullptr;
  const float* v_scale = nullptr;
  const int32_t* q_len;
  const int32_t* kv_len;
  const int32_t* mask_kind;   // 0 causal, 1 tree
  const int32_t* parent_off;  // into parents, tree requests only
  const int32_t* parents;
  const uint16_t* q;
  int64_t q_token_stride;
  const uint16_t* k_pool;
  const uint16_t* v_pool;
  int64_t page_stride, head_stride, token_stride;
  const int32_t* block_table;
  int32_t bt_stride;
  double sm_scale;
};

// Step 2: one explicit mask row, M[i][0..L).  History is always visible; the
// corner is causal (j' <= i) or ancestor-or-self of the parent array.
void mask_row(const Problem& p, int r, int i, std::vector<uint8_t>& m) {
  const int n = p.q_len[r], h = p.kv_len[r], L = n + h;
  m.assign(L, 0);
  for (int j = 0; j < h; ++j) m[j] = 1;
  if (p.mask_kind[r] == 0) {
    for (int jp = 0; jp <= i; ++jp) m[h + jp] = 1;
  } else {
    const int32_t* par = p.parents + p.parent_off[r];
    int node = i;
    while (node >= 0) {
      m[h + node] = 1;
      node = par[node];
    }
  }
}

// Step 1: address of cached token j of request r, kv head g (elements).
inline int64_t kv_offset(const Problem& p, int r, int g, int j) {
  const int64_t page = p.block_table[static_cast<int64_t>(r) * p.bt_stride + j / p.B];
  const int slot = j % p.B;
  return page * p.page_stride + static_cast<int64_t>(g) * p.head_stride +
         static_cast<int64_t>(slot) * p.token_stride;
}

// Element d of the K (which = 0) or V (which = 1) row of cached token j of request r, kv head g.
inline double kv_elem(const Problem& p, int which, int r, int g, int j, int d) {
  const int64_t off = kv_offset(p, r, g, j) + d;
  if (p.k8 == nullptr) return widen((which ? p.v_pool : p.k_pool)[off]);
  const int64_t page = p.block_table[static_cast<int64_t>(r) * p.bt_stride + j / p.B];
  const float sc = (which ? p.v_scale : p.k_scale)[page * p.Hkv + g];
  return decode_e4m3((which ? p.v8 : p.k8)[off]) * static_cast<double>(sc);
}

// Steps 1-3 for one (request, q head, row).  Outputs: o[D], lse, sum of p,
// and optionally the probabilities p[0..L).
// `keep` (nullable, u8[L]) restricts the allowed set further (used to form the
// partial results the merge identity is tested on); with no allowed key the
// row's LSE is -inf and its O is 0.
void attend_row(const Problem& p, int r, int64_t q_start, int a, int i, double* o, double* lse,
                double* psum, double* probs, const uint8_t* keep = nullptr) {
  const int n = p.q_len[r], h = p.kv_len[r], L = n + h, D = p.D;
  const int g = a / (p.Hq / p.Hkv);
  std::vector<uint8_t> m;
  mask_row(p, r, i, m);
  if (keep) {
    bool any = false;
    for (int j = 0; j < L; ++j) {
      m[j] = m[j] && keep[j];
      any = any || m[j];
    }
    if (!any) {
      for (int d = 0; d < D; ++d) o[d] = 0.0;
      *lse = -std::numeric_limits<double>::infinity();
      if (psum) *psum = 0.0;
      if (probs) for (int j = 0; j < L; ++j) probs[j] = 0.0;
      return;
    }
  }
  const uint16_t* qrow = p.q + (q_start + i) * p.q_token_stride + static_cast<int64_t>(a) * D;
  std::vector<double> s(L, 0.0);
  double mx = -std::numeric_limits<double>::infinity();
  for (int j = 0; j < L; ++j) {
    if (!m[j]) continue;
    double acc = 0.0;
    for (int d = 0; d < D; ++d) acc += widen(qrow[d]) * kv_elem(p, 0, r, g, j, d);
    s[j] = p.sm_scale * acc;
    if (s[j] > mx) mx = s[j];
  }
  double Z = 0.0;
  for (int j = 0; j < L; ++j)
    if (m[j]) Z += std::exp(s[j] - mx);
  const double l = mx + std::log(Z);
  for (int d = 0; d < D; ++d) o[d] = 0.0;
  double ps = 0.0;
  for (int j = 0; j < L; ++j) {
    double pj = 0.0;
    if (m[j]) {
      pj = std::exp(s[j] - l);
      for (int d = 0; d < D; ++d) o[d] += pj * kv_elem(p, 1, r, g, j, d);
      ps += pj;
    }
    if (probs) probs[j] = pj;
  }
  *lse = l;
  if (psum) *psum = ps;
}

Problem make_problem(int R, int Hq, int Hkv, int D, int B, const int32_t* q_len,
                     const int32_t* kv_len, const int32_t* mask_kind, const int32_t* parent_off,
                     const int32_t* parents, const uint16_t* q, int64_t q_token_stride,
                     const uint16_t* k_pool, const uint16_t* v_pool, int64_t page_stride,
                     int64_t head_stride, int64_t token_stride, const int32_t* block_table,
                     int32_t bt_stride, double sm_scale) {
  Problem p;
  p.R = R; p.Hq = Hq; p.Hkv = Hkv; p.D = D; p.B = B;
  p.q_len = q_len; p.kv_len = kv_len; p.mask_kind = mask_kind;
  p.parent_off = parent_off; p.parents = parents;
  p.q = q; p.q_token_stride = q_token_stride;
  p.k_pool = k_pool; p.v_pool = v_pool;
  p.page_stride = page_stride; p.head_stride = head_stride; p.token_stride = token_stride;
  p.block_table = block_table; p.bt_stride = bt_stride; p.sm_scale = sm_scale;
  return p;
}

}  // namespace

#define PROBLEM_ARGS                                                                             \
  int R, int Hq, int Hkv, int D, int B, const int32_t *q_len, const int32_t *kv_len,             \
      const int32_t *mask_kind, const int32_t *parent_off, const int32_t *parents,               \
      const uint16_t *q, int64_t q_token_stride, const uint16_t *k_pool, const uint16_t *v_pool, \
      int64_t page_stride, int64_t head_stride, int64_t token_stride,                            \
      const int32_t *block_table, int32_t bt_stride, double sm_scale
#define PROBLEM_PASS                                                                          \
  R, Hq, Hkv, D, B, q_len, kv_len, mask_kind, parent_off, parents, q, q_token_stride, k_pool, \
      v_pool, page_stride, head_stride, token_stride, block_table, bt_stride, sm_scale

extern "C" {

int oracle_num_threads() {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

// Whole batch (or the requests flagged in `only`, nullable): O fp64 [T, Hq, D],
// LSE fp64 [T, Hq], psum fp64 [T, Hq] (nullable) = sum of each row's probabilities.
int oracle_attention(PROBLEM_ARGS, const uint8_t* only, double* O, double* LSE, double* psum) {
  Problem p = make_problem(PROBLEM_PASS);
  if (Hkv <= 0 || Hq % Hkv != 0) return -1;
  std::vector<int64_t> q_start(R + 1, 0);
  for (int r = 0; r < R; ++r) q_start[r + 1] = q_start[r] + q_len[r];
  for (int r = 0; r < R; ++r) {
    if (only && !only[r]) continue;
    const int n = q_len[r];
    const int64_t units = static_cast<int64_t>(n) * Hq;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t u = 0; u < units; ++u) {
      const int i = static_cast<int>(u / Hq), a = static_cast<int>(u % Hq);
      const int64_t row = (q_start[r] + i) * Hq + a;
      attend_row(p, r, q_start[r], a, i, O + row * D, LSE + row, psum ? psum + row : nullptr,
                 nullptr);
    }
  }
  return 0;
}

// Sampled outputs: for s in [0, S): (req[s], head[s], row[s]) -> O fp64 [S, D], LSE fp64 [S].
int oracle_attention_rows(PROBLEM_ARGS, int S, const int32_t* req, const int32_t* head,
                          const int32_t* row, double* O, double* LSE) {
  Problem p = make_problem(PROBLEM_PASS);
  if (Hkv <= 0 || Hq % Hkv != 0) return -1;
  std::vector<int64_t> q_start(R + 1, 0);
  for (int r = 0; r < R; ++r) q_start[r + 1] = q_start[r] + q_len[r];
#pragma omp parallel for schedule(dynamic, 1)
  for (int s = 0; s < S; ++s)
    attend_row(p, req[s], q_start[req[s]], head[s], row[s], O + static_cast<int64_t>(s) * D,
               LSE + s, nullptr, nullptr);
  return 0;
}

// fp8 KV-cache variant of the two calls above: k_pool / v_pool of PROBLEM_ARGS are ignored (pass
// null); k8 / v8 are the byte pools with the same element strides, k_scale / v_scale fp32
// [pages, Hkv].  rows-mode when S >= 0 (req / head / row select the outputs), whole batch when S < 0.
int oracle_attention_fp8(PROBLEM_ARGS, const uint8_t* k8, const uint8_t* v8, const float* k_scale,
                         const float* v_scale, int S, const int32_t* req, const int32_t* head, const int32_t* row,
                         double* O, double* LSE) {
  Problem p = make_problem(PROBLEM_PASS);
  if (Hkv <= 0 || Hq % Hkv != 0 || !k8 || !v8 || !k_scale || !v_scale) return -1;
  p.k8 = k8; p.v8 = v8; p.k_scale = k_scale; p.v_scale = v_scale;
  std::vector<int64_t> q_start(R + 1, 0);
  for (int r = 0; r < R; ++r) q_start[r + 1] = q_start[r] + q_len[r];
  if (S >= 0) {
#pragma omp parallel for schedule(dynamic, 1)
    for (int s = 0; s < S; ++s)
      attend_row(p, req[s], q_start[req[s]], head[s], row[s], O + static_cast<int64_t>(s) * D, LSE + s, nullptr,
                 nullptr);
    return 0;
  }
  for (int r = 0; r < R; ++r) {
    const int64_t units = static_cast<int64_t>(q_len[r]) * Hq;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t u = 0; u < units; ++u) {
      const int i = static_cast<int>(u / Hq), a = static_cast<int>(u % Hq);
      const int64_t orow = (q_start[r] + i) * Hq + a;
      attend_row(p, r, q_start[r], a, i, O + orow * D, LSE + orow, nullptr, nullptr);
    }
  }
  return 0;
}

// The 256 decoded e4m3 values (for the table pin).
int oracle_e4m3_table(double* out) {
  for (int b = 0; b < 256; ++b) out[b] = decode_e4m3(static_cast<uint8_t>(b));
  return 0;
}

// Probabilities of one (request, q head): P fp64 [n, L]; also the mask M u8 [n, L].
int oracle_probs(PROBLEM_ARGS, int r, int a, double* P, uint8_t* M) {
  Problem p = make_problem(PROBLEM_PASS);
  std::vector<int64_t> q_start(R + 1, 0);
  for (int x = 0; x < R; ++x) q_start[x + 1] = q_start[x] + q_len[x];
  const int n = q_len[r], L = n + kv_len[r];
  std::vector<double> o(D);
  for (int i = 0; i < n; ++i) {
    double lse, ps;
    attend_row(p, r, q_start[r], a, i, o.data(), &lse, &ps, P + static_cast<int64_t>(i) * L);
    std::vector<uint8_t> m;
    mask_row(p, r, i, m);
    std::memcpy(M + static_cast<int64_t>(i) * L, m.data(), L);
  }
  return 0;
}

// One row restricted to the keys flagged in keep[0..L): partial (O_c, LSE_c).
int oracle_attention_keys(PROBLEM_ARGS, int r, int a, int i, const uint8_t* keep, double* O,
                          double* LSE) {
  Problem p = make_problem(PROBLEM_PASS);
  std::vector<int64_t> q_start(R + 1, 0);
  for (int x = 0; x < R; ++x) q_start[x + 1] = q_start[x] + q_len[x];
  attend_row(p, r, q_start[r], a, i, O, LSE, nullptr, nullptr, keep);
  return 0;
}

// Step 5: the gathered K and V rows of (request r, kv head g), bf16 bits, [L, D] each.
int oracle_gather(PROBLEM_ARGS, int r, int g, uint16_t* K_out, uint16_t* V_out) {
  Problem p = make_problem(PROBLEM_PASS);
  const int L = q_len[r] + kv_len[r];
  for (int j = 0; j < L; ++j) {
    const int64_t off = kv_offset(p, r, g, j);
    std::memcpy(K_out + static_cast<int64_t>(j) * D, k_pool + off, sizeof(uint16_t) * D);
    std::memcpy(V_out + static_cast<int64_t>(j) * D, v_pool + off, sizeof(uint16_t) * D);
  }
  return 0;
}

// KV-cache append (the step before attention; Sections 4.1.1 and 5.4): for every request r and
// new token i, the K and V head rows of the fused QKV tensor [T, Hq + 2 Hkv, D] are written to
// the cache slot of logical position kv_len[r] + i, found through the block table.  Plain copy
// of bf16 bits; K heads follow the Hq query heads, V heads follow the K heads.
int oracle_append_kv(int R, int Hq, int Hkv, int D, int B, const int32_t* q_len, const int32_t* kv_len,
                     const uint16_t* qkv, int64_t qkv_token_stride, uint16_t* k_pool, uint16_t* v_pool,
                     int64_t page_stride, int64_t head_stride, int64_t token_stride,
                     const int32_t* block_table, int32_t bt_stride) {
  int64_t t = 0;
  for (int r = 0; r < R; ++r) {
    for (int i = 0; i < q_len[r]; ++i, ++t) {
      const int j = kv_len[r] + i;
      const int64_t page = block_table[static_cast<int64_t>(r) * bt_stride + j / B];
      const int slot = j % B;
      for (int g = 0; g < Hkv; ++g) {
        const int64_t dst = page * page_stride + g * head_stride + static_cast<int64_t>(slot) * token_stride;
        const uint16_t* ksrc = qkv + t * qkv_token_stride + static_cast<int64_t>(Hq + g) * D;
        const uint16_t* vsrc = qkv + t * qkv_token_stride + static_cast<int64_t>(Hq + Hkv + g) * D;
        std::memcpy(k_pool + dst, ksrc, sizeof(uint16_t) * D);
        std::memcpy(v_pool + dst, vsrc, sizeof(uint16_t) * D);
      }
    }
  }
  return 0;
}

// Step 4 (Update stage): merge C partial results of `rows` rows each.
//   LSE = ln sum_c exp(LSE_c);  O = sum_c exp(LSE_c - LSE) O_c.
// A chunk with LSE_c = -inf (no allowed key) contributes nothing.
// O_c fp64 [C, rows, D], LSE_c fp64 [C, rows] -> O [rows, D], LSE [rows].
int oracle_merge(int C, int64_t rows, int D, const double* O_c, const double* LSE_c, double* O,
                 double* LSE) {
  for (int64_t x = 0; x < rows; ++x) {
    double mx = -std::numeric_limits<double>::infinity();
    for (int c = 0; c < C; ++c) mx = std::fmax(mx, LSE_c[c * rows + x]);
    double Z = 0.0;
    for (int c = 0; c < C; ++c) {
      const double l = LSE_c[c * rows + x];
      if (std::isinf(l) && l < 0) continue;
      Z += std::exp(l - mx);
    }
    const double lse = mx + std::log(Z);
    for (int d = 0; d < D; ++d) O[x * D + d] = 0.0;
    for (int c = 0; c < C; ++c) {
      const double l = LSE_c[c * rows + x];
      if (std::isinf(l) && l < 0) continue;
      const double w = std::exp(l - lse);
      for (int d = 0; d < D; ++d) O[x * D + d] += w * O_c[(c * rows + x) * D + d];
    }
    LSE[x] = lse;
  }
  return 0;
}

}  // extern "C"
