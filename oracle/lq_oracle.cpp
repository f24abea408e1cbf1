// LogQuant CPU oracle  --  TEST INFRASTRUCTURE, NOT PRODUCT CODE.
//
// A plain, slow, single-pass C++17 restatement of what the decode-time hot path of
// LogQuant computes.  It exists so that the CUDA library can be checked element by
// element; only the test-suite, the smoke check and the benchmark's CPU-baseline leg
// may call it.  It shares no code, header, table or helper with the CUDA library.
//
// What each part follows (paper = "LogQuant: Log-Distributed 2-Bit Quantization of
// KV Cache", arXiv 2503.19950):
//   * filter        : Algorithm 1 (AppendToken) with Python slice semantics, Sec. 2.5.
//   * quantiser     : the paper only names "INT2", group size G and the "Key-per-channel
//                     strategy" (Sec. 2.5 Implementation, Sec. 3.1 Settings).  The reading
//                     taken here is asymmetric min/max quantisation:
//                         zero  = min(group)                         (a bf16 value, exact; -0 -> +0)
//                         scale = bf16_rne((max - min) / 3)          (fp32 IEEE ops)
//                         code  = clamp(rint((x - zero) / scale), 0, 3), all 0 if scale == 0
//                         x^    = zero + code * scale
//                     keys: one group = G consecutive evicted tokens of one channel;
//                     values: one group = G consecutive channels of one token.
//                     When W is not a multiple of G (the paper's own settings, Sec. 3.1: G = 64
//                     with a reserved length of 128 or 256 tokens, i.e. W = 42 or 85) an overflow
//                     step does not yield whole key groups.  The paper does not say what happens
//                     then; the reading taken here: tokens the filter removes wait, still at
//                     original precision, in removal order, and every time G of them are waiting
//                     the oldest G form one key group and are quantised.
//                     The paper's second precision (the 4-bit rows of its accuracy tables,
//                     Sec. 3.2) is the same quantiser with 16 levels: scale = bf16_rne((max -
//                     min) / 15), codes 0..15.
//   * packer        : 2-bit: 4 codes per byte, channel 4j+i in bits [2i+1:2i] of byte j;
//                     4-bit: 2 codes per byte, channel 2j+i in bits [4i+3:4i] of byte j.
//   * attention     : Eq. 2 with the 1/sqrt(d) scale of the appendix (passed in as
//                     sm_scale), float64, one pass with max subtraction, over the union
//                     of the full-precision list and the dequantised store.  Eq. 3
//                     (position-agnostic attention) is what allows the union to be
//                     visited in any order.
//   * attention over a subset: the same sum over fewer tokens.  (i) Full-precision tokens only:
//                     what the eviction variants of Sec. 2.3 compute (tokens the filter removes are
//                     dropped, not quantised).  (ii) Left padding: the first pad[b] positions of
//                     sequence b are padding of a ragged batch; they pass through filter and
//                     quantiser like any token (both are position-based) and attention leaves
//                     them out.
//
// Parity status: filter, quantiser, packer and attention are pinned by tests that do
// not go through this file's own formulas (hand simulation of Algorithm 1, closed
// forms, a hand-worked quantiser example, library softmax attention, brute force).
// Parity with the paper's own numbers is UNPINNED: the paper prints no worked numeric
// example and delegates its quantiser to a library it does not describe.
//
// Build:  g++ -O2 -std=c++17 -ffp-contract=off -fPIC -shared -pthread

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>

namespace {

// ---- bf16 <-> fp32 (bit manipulation; finite inputs) -------------------------------
float bf16_to_f32(uint16_t h) {
  uint32_t u = static_cast<uint32_t>(h) << 16;
  float f;
  std::memcpy(&f, &u, sizeof f);
  return f;
}

uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  std::memcpy(&u, &f, sizeof u);
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb;  // round to nearest, ties to even
  return static_cast<uint16_t>(u >> 16);
}

// ---- quantiser: one group of n values, read with a stride --------------------------
// All arithmetic is IEEE binary32 with one rounding per operation (the file is built
// with -ffp-contract=off so no multiply-add is ever contracted).
// top = highest code: 3 for 2 bits, 15 for 4 bits.
void quantize_group(const uint16_t* x, int n, int64_t stride, uint16_t* scale_out,
                    uint16_t* zero_out, uint8_t* codes, int64_t code_stride, int top = 3) {
  float mn = bf16_to_f32(x[0]);
  float mx = mn;
  for (int i = 1; i < n; ++i) {
    float v = bf16_to_f32(x[i * stride]);
    if (v < mn) mn = v;
    if (v > mx) mx = v;
  }
  mn = mn + 0.0f;  // a zero-valued min or max is taken as +0 (the sign of zero is not information)
  mx = mx + 0.0f;
  volatile float range = mx - mn;
  volatile float third = range / static_cast<float>(top);  // one step of the code grid
  uint16_t sb = f32_to_bf16_rne(third);
  float scale = bf16_to_f32(sb);
  *scale_out = sb;
  *zero_out = f32_to_bf16_rne(mn);  // mn is a bf16 value already: conversion is exact
  for (int i = 0; i < n; ++i) {
    uint8_t c = 0;
    if (scale != 0.0f) {
      volatile float d = bf16_to_f32(x[i * stride]) - mn;
      volatile float q = d / scale;
      float r = std::nearbyintf(q);  // default rounding mode: ties to even
      if (r < 0.0f) r = 0.0f;
      if (r > static_cast<float>(top)) r = static_cast<float>(top);
      c = static_cast<uint8_t>(r);
    }
    codes[i * code_stride] = c;
  }
}

double dequant(uint16_t scale, uint16_t zero, uint8_t code) {
  return static_cast<double>(bf16_to_f32(zero)) +
         static_cast<double>(code) * static_cast<double>(bf16_to_f32(scale));
}

// ---- the cache ---------------------------------------------------------------------
struct Head {  // one (batch row, kv head)
  std::vector<uint16_t> fp_k, fp_v;      // [len(A)][D], rows in the order of list A
  std::vector<uint16_t> pend_k, pend_v;  // [len(P)][D], rows in the order of list P
  std::vector<uint8_t> k_codes, v_codes;  // [nq][D], one code per byte (unpacked)
  std::vector<uint16_t> k_scale, k_zero;  // [nq/G][D]
  std::vector<uint16_t> v_scale, v_zero;  // [nq][D/G]
};

struct Cache {
  int B, Hq, Hkv, D, W, G;
  int bits = 2;
  int recent_only = 0;  // comparator: the W oldest tokens leave instead of Algorithm 1's odd positions
  int64_t n_seen = 0, n_events = 0;
  std::vector<int64_t> A;  // ids of the tokens kept at original precision, age order
  std::vector<int64_t> P;  // ids of the tokens the filter removed that still wait for a full key group
  std::vector<int64_t> Q;  // ids of the quantised tokens, store order
  std::vector<Head> heads;  // [B*Hkv]
};

// One window-overflow event (Algorithm 1, the else-branch): the entries at odd positions
// of A[0:2W] leave the list, in age order; A becomes A[0:2W:2] ++ A[2W:3W].
void overflow_event(Cache& c) {
  const int W = c.W, D = c.D, G = c.G;
  std::vector<int64_t> evict_pos, keep_pos;
  if (c.recent_only) {
    // Comparator (not the paper's method): only a recent window stays at full precision, as in the
    // sliding-window quantisers the paper compares with (Sec. 2.2-2.3): A becomes A[W:3W].
    for (int i = 0; i < 3 * W; ++i) (i < W ? evict_pos : keep_pos).push_back(i);
  } else {
    for (int i = 0; i < 2 * W; ++i) (i % 2 ? evict_pos : keep_pos).push_back(i);
    for (int i = 2 * W; i < 3 * W; ++i) keep_pos.push_back(i);
  }
  for (auto& h : c.heads) {
    // the W leaving rows join the waiting rows, in removal order
    for (int e = 0; e < W; ++e) {
      h.pend_k.insert(h.pend_k.end(), &h.fp_k[evict_pos[e] * D], &h.fp_k[evict_pos[e] * D] + D);
      h.pend_v.insert(h.pend_v.end(), &h.fp_v[evict_pos[e] * D], &h.fp_v[evict_pos[e] * D] + D);
    }
    // shrink the full-precision rows to the kept positions
    std::vector<uint16_t> nk(keep_pos.size() * D), nv(keep_pos.size() * D);
    for (size_t i = 0; i < keep_pos.size(); ++i) {
      std::memcpy(&nk[i * D], &h.fp_k[keep_pos[i] * D], D * 2);
      std::memcpy(&nv[i * D], &h.fp_v[keep_pos[i] * D], D * 2);
    }
    h.fp_k.swap(nk);
    h.fp_v.swap(nv);
  }
  std::vector<int64_t> nA;
  for (auto p : evict_pos) c.P.push_back(c.A[p]);
  for (auto p : keep_pos) nA.push_back(c.A[p]);
  c.A.swap(nA);
  c.n_events++;
  // every G waiting tokens form one key group (W a multiple of G: exactly W / G groups, nothing waits)
  while (static_cast<int>(c.P.size()) >= G) {
    for (auto& h : c.heads) {
      const size_t nq0 = h.k_codes.size() / D;
      h.k_codes.resize((nq0 + G) * D);
      h.v_codes.resize((nq0 + G) * D);
      h.k_scale.resize((nq0 + G) / G * D);
      h.k_zero.resize((nq0 + G) / G * D);
      h.v_scale.resize((nq0 + G) * (D / G));
      h.v_zero.resize((nq0 + G) * (D / G));
      // keys: group = the G oldest waiting tokens of one channel
      for (int d = 0; d < D; ++d) {
        size_t grp = (nq0 / G) * D + d;
        quantize_group(&h.pend_k[d], G, D, &h.k_scale[grp], &h.k_zero[grp], &h.k_codes[nq0 * D + d], D,
                       (1 << c.bits) - 1);
      }
      // values: group = G consecutive channels of one token
      for (int e = 0; e < G; ++e)
        for (int g = 0; g < D / G; ++g) {
          size_t grp = (nq0 + e) * (D / G) + g;
          quantize_group(&h.pend_v[static_cast<size_t>(e) * D + g * G], G, 1, &h.v_scale[grp], &h.v_zero[grp],
                         &h.v_codes[(nq0 + e) * D + g * G], 1, (1 << c.bits) - 1);
        }
      h.pend_k.erase(h.pend_k.begin(), h.pend_k.begin() + static_cast<size_t>(G) * D);
      h.pend_v.erase(h.pend_v.begin(), h.pend_v.begin() + static_cast<size_t>(G) * D);
    }
    c.Q.insert(c.Q.end(), c.P.begin(), c.P.begin() + G);
    c.P.erase(c.P.begin(), c.P.begin() + G);
  }
}

// Dense softmax attention of one query over n tokens, float64 (Eq. 2 with sm_scale).
void attention_dense(const double* q, const double* K, const double* V, int64_t n, int D,
                     double sm_scale, double* out) {
  std::vector<double> s(n);
  double m = -INFINITY;
  for (int64_t t = 0; t < n; ++t) {
    double acc = 0.0;
    for (int d = 0; d < D; ++d) acc += q[d] * K[t * D + d];
    s[t] = acc * sm_scale;
    if (s[t] > m) m = s[t];
  }
  double l = 0.0;
  for (int64_t t = 0; t < n; ++t) {
    s[t] = std::exp(s[t] - m);
    l += s[t];
  }
  for (int d = 0; d < D; ++d) out[d] = 0.0;
  for (int64_t t = 0; t < n; ++t) {
    double p = s[t] / l;
    for (int d = 0; d < D; ++d) out[d] += p * V[t * D + d];
  }
}

// All tokens of one head as float64 rows: first the full-precision list (order of A), the
// waiting rows (order of P), then the quantised store (order of Q), dequantised.
void dense_rows(const Cache& c, const Head& h, std::vector<double>& K, std::vector<double>& V) {
  const int D = c.D, G = c.G;
  const size_t na = c.A.size(), nf = c.A.size() + c.P.size(), nq = c.Q.size();
  K.resize((nf + nq) * D);
  V.resize((nf + nq) * D);
  for (size_t i = 0; i < na * D; ++i) {
    K[i] = bf16_to_f32(h.fp_k[i]);
    V[i] = bf16_to_f32(h.fp_v[i]);
  }
  for (size_t i = 0; i < c.P.size() * D; ++i) {
    K[na * D + i] = bf16_to_f32(h.pend_k[i]);
    V[na * D + i] = bf16_to_f32(h.pend_v[i]);
  }
  for (size_t t = 0; t < nq; ++t)
    for (int d = 0; d < D; ++d) {
      size_t kg = (t / G) * D + d;
      size_t vg = t * (D / G) + d / G;
      K[(nf + t) * D + d] = dequant(h.k_scale[kg], h.k_zero[kg], h.k_codes[t * D + d]);
      V[(nf + t) * D + d] = dequant(h.v_scale[vg], h.v_zero[vg], h.v_codes[t * D + d]);
    }
}

}  // namespace

extern "C" {

// ---- stand-alone pieces --------------------------------------------------------------
// Algorithm 1 on token ids 0..N-1.  kept/quant must hold 3W and N entries; returns the
// number of events and writes the two lengths.
int64_t lqo_filter(int W, int64_t N, int64_t* kept, int64_t* n_kept, int64_t* quant, int64_t* n_quant) {
  std::vector<int64_t> A, Q;
  int64_t events = 0;
  for (int64_t t = 0; t < N; ++t) {
    if (static_cast<int64_t>(A.size()) < 3 * static_cast<int64_t>(W)) {
      A.push_back(t);
    } else {
      std::vector<int64_t> nA;
      for (int i = 0; i < 2 * W; i += 2) nA.push_back(A[i]);
      for (int i = 1; i < 2 * W; i += 2) Q.push_back(A[i]);
      for (int i = 2 * W; i < 3 * W; ++i) nA.push_back(A[i]);
      nA.push_back(t);
      A.swap(nA);
      events++;
    }
  }
  std::copy(A.begin(), A.end(), kept);
  std::copy(Q.begin(), Q.end(), quant);
  *n_kept = static_cast<int64_t>(A.size());
  *n_quant = static_cast<int64_t>(Q.size());
  return events;
}

void lqo_quantize_group(const uint16_t* x, int n, uint16_t* scale, uint16_t* zero, uint8_t* codes) {
  quantize_group(x, n, 1, scale, zero, codes, 1);
}

// the same with 2 or 4 bits per code
void lqo_quantize_group_bits(const uint16_t* x, int n, int bits, uint16_t* scale, uint16_t* zero, uint8_t* codes) {
  quantize_group(x, n, 1, scale, zero, codes, 1, (1 << bits) - 1);
}

double lqo_dequant(uint16_t scale, uint16_t zero, uint8_t code) { return dequant(scale, zero, code); }

// 4 codes per byte: code of element 4j+i in bits [2i+1:2i] of byte j.  n % 4 == 0.
void lqo_pack2(const uint8_t* codes, int64_t n, uint8_t* bytes) {
  for (int64_t j = 0; j < n / 4; ++j) {
    uint8_t b = 0;
    for (int i = 0; i < 4; ++i) b |= static_cast<uint8_t>((codes[4 * j + i] & 3u) << (2 * i));
    bytes[j] = b;
  }
}

void lqo_unpack2(const uint8_t* bytes, int64_t n, uint8_t* codes) {
  for (int64_t j = 0; j < n / 4; ++j)
    for (int i = 0; i < 4; ++i) codes[4 * j + i] = (bytes[j] >> (2 * i)) & 3u;
}

// 2 codes per byte: code of element 2j+i in bits [4i+3:4i] of byte j.  n % 2 == 0.
void lqo_pack4(const uint8_t* codes, int64_t n, uint8_t* bytes) {
  for (int64_t j = 0; j < n / 2; ++j)
    bytes[j] = static_cast<uint8_t>((codes[2 * j] & 15u) | ((codes[2 * j + 1] & 15u) << 4));
}

void lqo_unpack4(const uint8_t* bytes, int64_t n, uint8_t* codes) {
  for (int64_t j = 0; j < n / 2; ++j) {
    codes[2 * j] = bytes[j] & 15u;
    codes[2 * j + 1] = bytes[j] >> 4;
  }
}

uint16_t lqo_f32_to_bf16(float f) { return f32_to_bf16_rne(f); }
float lqo_bf16_to_f32(uint16_t h) { return bf16_to_f32(h); }

void lqo_attention_dense(const double* q, const double* K, const double* V, int64_t n, int D,
                         double sm_scale, double* out) {
  attention_dense(q, K, V, n, D, sm_scale, out);
}

// Partial softmax state of one segment: m = max score, l = sum exp(s - m),
// o = sum exp(s - m) * v (not normalised).  n may be 0 (m = -inf, l = 0, o = 0).
void lqo_attention_partial(const double* q, const double* K, const double* V, int64_t n, int D,
                           double sm_scale, double* m_out, double* l_out, double* o) {
  double m = -INFINITY;
  std::vector<double> s(n);
  for (int64_t t = 0; t < n; ++t) {
    double acc = 0.0;
    for (int d = 0; d < D; ++d) acc += q[d] * K[t * D + d];
    s[t] = acc * sm_scale;
    if (s[t] > m) m = s[t];
  }
  double l = 0.0;
  for (int d = 0; d < D; ++d) o[d] = 0.0;
  for (int64_t t = 0; t < n; ++t) {
    double p = std::exp(s[t] - m);
    l += p;
    for (int d = 0; d < D; ++d) o[d] += p * V[t * D + d];
  }
  *m_out = m;
  *l_out = l;
}

// Merge of S partial states: m = max m_s, l = sum l_s e^{m_s-m}, out = sum o_s e^{m_s-m} / l.
void lqo_attention_merge(const double* m, const double* l, const double* o, int S, int D, double* out) {
  double mm = -INFINITY;
  for (int s = 0; s < S; ++s) mm = std::max(mm, m[s]);
  double ll = 0.0;
  for (int d = 0; d < D; ++d) out[d] = 0.0;
  for (int s = 0; s < S; ++s) {
    if (l[s] == 0.0) continue;
    double w = std::exp(m[s] - mm);
    ll += l[s] * w;
    for (int d = 0; d < D; ++d) out[d] += o[s * D + d] * w;
  }
  for (int d = 0; d < D; ++d) out[d] /= ll;
}

// ---- the cache object ------------------------------------------------------------------
void* lqo_create(int B, int Hq, int Hkv, int D, int W, int G) {
  if (B < 1 || Hkv < 1 || Hq % Hkv || D < 1 || W < 1 || G < 1 || D % G || D % 4) return nullptr;
  Cache* c = new Cache;
  c->B = B; c->Hq = Hq; c->Hkv = Hkv; c->D = D; c->W = W; c->G = G;
  c->heads.resize(static_cast<size_t>(B) * Hkv);
  return c;
}

// the same cache with 2 or 4 bits per code
void* lqo_create_bits(int B, int Hq, int Hkv, int D, int W, int G, int bits) {
  if (bits != 2 && bits != 4) return nullptr;
  Cache* c = static_cast<Cache*>(lqo_create(B, Hq, Hkv, D, W, G));
  if (c) c->bits = bits;
  return c;
}

// ... and with the recent-window comparator in place of Algorithm 1's filter
void* lqo_create_policy(int B, int Hq, int Hkv, int D, int W, int G, int bits, int recent_only) {
  Cache* c = static_cast<Cache*>(lqo_create_bits(B, Hq, Hkv, D, W, G, bits));
  if (c) c->recent_only = recent_only ? 1 : 0;
  return c;
}

void lqo_destroy(void* p) { delete static_cast<Cache*>(p); }

// k, v: [B][Hkv][n][D] bf16 bit patterns.  A prompt of n tokens is n single appends.
void lqo_append(void* p, const uint16_t* k, const uint16_t* v, int n) {
  Cache& c = *static_cast<Cache*>(p);
  for (int t = 0; t < n; ++t) {
    if (static_cast<int64_t>(c.A.size()) >= 3 * static_cast<int64_t>(c.W)) overflow_event(c);
    for (int b = 0; b < c.B; ++b)
      for (int h = 0; h < c.Hkv; ++h) {
        Head& hd = c.heads[static_cast<size_t>(b) * c.Hkv + h];
        const size_t off = ((static_cast<size_t>(b) * c.Hkv + h) * n + t) * c.D;
        hd.fp_k.insert(hd.fp_k.end(), k + off, k + off + c.D);
        hd.fp_v.insert(hd.fp_v.end(), v + off, v + off + c.D);
      }
    c.A.push_back(c.n_seen++);
  }
}

int64_t lqo_n_seen(void* p) { return static_cast<Cache*>(p)->n_seen; }
// tokens at original precision: the filter's list plus those waiting for a full key group
int64_t lqo_n_fp(void* p) {
  return static_cast<int64_t>(static_cast<Cache*>(p)->A.size() + static_cast<Cache*>(p)->P.size());
}
int64_t lqo_n_quant(void* p) { return static_cast<int64_t>(static_cast<Cache*>(p)->Q.size()); }
int64_t lqo_n_events(void* p) { return static_cast<Cache*>(p)->n_events; }

// Canonical image.  kept_ids ascending (list A is in age order, hence ascending);
// quant_ids in store order; codes packed 4 per byte (2 per byte at 4 bits); scale/zero as bf16 bit patterns;
// fp rows in kept_ids order.  Any pointer may be null to skip that array.
void lqo_export(void* p, int32_t* kept_ids, int32_t* quant_ids, uint8_t* k_codes, uint8_t* v_codes,
                uint16_t* k_scale, uint16_t* k_zero, uint16_t* v_scale, uint16_t* v_zero,
                uint16_t* fp_k, uint16_t* fp_v) {
  Cache& c = *static_cast<Cache*>(p);
  const size_t nq = c.Q.size(), D = c.D, G = c.G;
  // tokens at original precision in ascending id order: (id, list, position in that list)
  struct Row { int64_t id; int from_p; size_t pos; };
  std::vector<Row> rows;
  for (size_t i = 0; i < c.A.size(); ++i) rows.push_back({c.A[i], 0, i});
  for (size_t i = 0; i < c.P.size(); ++i) rows.push_back({c.P[i], 1, i});
  std::sort(rows.begin(), rows.end(), [](const Row& x, const Row& y) { return x.id < y.id; });
  const size_t nf = rows.size();
  if (kept_ids) for (size_t i = 0; i < nf; ++i) kept_ids[i] = static_cast<int32_t>(rows[i].id);
  if (quant_ids) for (size_t i = 0; i < nq; ++i) quant_ids[i] = static_cast<int32_t>(c.Q[i]);
  for (size_t hh = 0; hh < c.heads.size(); ++hh) {
    const Head& h = c.heads[hh];
    if (c.bits == 2) {
      if (k_codes) lqo_pack2(h.k_codes.data(), nq * D, k_codes + hh * nq * D / 4);
      if (v_codes) lqo_pack2(h.v_codes.data(), nq * D, v_codes + hh * nq * D / 4);
    } else {
      if (k_codes) lqo_pack4(h.k_codes.data(), nq * D, k_codes + hh * nq * D / 2);
      if (v_codes) lqo_pack4(h.v_codes.data(), nq * D, v_codes + hh * nq * D / 2);
    }
    if (k_scale) std::copy(h.k_scale.begin(), h.k_scale.end(), k_scale + hh * (nq / G) * D);
    if (k_zero) std::copy(h.k_zero.begin(), h.k_zero.end(), k_zero + hh * (nq / G) * D);
    if (v_scale) std::copy(h.v_scale.begin(), h.v_scale.end(), v_scale + hh * nq * (D / G));
    if (v_zero) std::copy(h.v_zero.begin(), h.v_zero.end(), v_zero + hh * nq * (D / G));
    for (size_t i = 0; i < nf; ++i) {
      const uint16_t* sk = (rows[i].from_p ? h.pend_k.data() : h.fp_k.data()) + rows[i].pos * D;
      const uint16_t* sv = (rows[i].from_p ? h.pend_v.data() : h.fp_v.data()) + rows[i].pos * D;
      if (fp_k) std::copy(sk, sk + D, fp_k + (hh * nf + i) * D);
      if (fp_v) std::copy(sv, sv + D, fp_v + (hh * nf + i) * D);
    }
  }
}

// Every token of head (b, kv) as float64 rows: the full-precision list then the
// dequantised store.  K, V: [(n_fp + n_quant)][D].
void lqo_dense_rows(void* p, int b, int kv, double* K, double* V) {
  Cache& c = *static_cast<Cache*>(p);
  std::vector<double> k, v;
  dense_rows(c, c.heads[static_cast<size_t>(b) * c.Hkv + kv], k, v);
  std::copy(k.begin(), k.end(), K);
  std::copy(v.begin(), v.end(), V);
}

// Decode attention of one query token per (b, query head) over the whole mixed cache.
// q: [B][Hq][D] bf16 bits; out: [B][Hq][D] float64.  Query head h reads KV head
// h / (Hq/Hkv).  n_threads > 1 spreads (b, kv head) pairs over std::threads.
void lqo_attention(void* p, const uint16_t* q, double sm_scale, double* out, int n_threads) {
  Cache& c = *static_cast<Cache*>(p);
  const int r = c.Hq / c.Hkv, D = c.D;
  const int n_pairs = c.B * c.Hkv;
  auto work = [&](int first, int step) {
    std::vector<double> K, V, qd(D);
    for (int pair = first; pair < n_pairs; pair += step) {
      const int b = pair / c.Hkv, kv = pair % c.Hkv;
      dense_rows(c, c.heads[pair], K, V);
      const int64_t n = static_cast<int64_t>(K.size()) / D;
      for (int j = 0; j < r; ++j) {
        const size_t qo = (static_cast<size_t>(b) * c.Hq + kv * r + j) * D;
        for (int d = 0; d < D; ++d) qd[d] = bf16_to_f32(q[qo + d]);
        attention_dense(qd.data(), K.data(), V.data(), n, D, sm_scale, out + qo);
      }
    }
  };
  if (n_threads <= 1) {
    work(0, 1);
  } else {
    std::vector<std::thread> th;
    for (int i = 0; i < n_threads; ++i) th.emplace_back(work, i, n_threads);
    for (auto& t : th) t.join();
  }
}

// Decode attention over a subset of the cache.  fp_only != 0: the tokens at original precision only.
// pad (may be null): [B], tokens of sequence b with id < pad[b] are left out.  A query whose subset is
// empty gets zeros.
void lqo_attention_subset(void* p, const uint16_t* q, double sm_scale, double* out, int fp_only, const int32_t* pad) {
  Cache& c = *static_cast<Cache*>(p);
  const int r = c.Hq / c.Hkv, D = c.D;
  std::vector<int64_t> ids;  // token id of every row dense_rows returns, in its order
  ids.insert(ids.end(), c.A.begin(), c.A.end());
  ids.insert(ids.end(), c.P.begin(), c.P.end());
  const size_t nf = ids.size();
  ids.insert(ids.end(), c.Q.begin(), c.Q.end());
  std::vector<double> K, V, Ks, Vs, qd(D);
  for (int pair = 0; pair < c.B * c.Hkv; ++pair) {
    const int b = pair / c.Hkv, kv = pair % c.Hkv;
    dense_rows(c, c.heads[pair], K, V);
    Ks.clear();
    Vs.clear();
    for (size_t i = 0; i < ids.size(); ++i) {
      if (fp_only && i >= nf) continue;
      if (pad && ids[i] < pad[b]) continue;
      Ks.insert(Ks.end(), K.begin() + i * D, K.begin() + (i + 1) * D);
      Vs.insert(Vs.end(), V.begin() + i * D, V.begin() + (i + 1) * D);
    }
    const int64_t n = static_cast<int64_t>(Ks.size()) / D;
    for (int j = 0; j < r; ++j) {
      const size_t qo = (static_cast<size_t>(b) * c.Hq + kv * r + j) * D;
      for (int d = 0; d < D; ++d) qd[d] = bf16_to_f32(q[qo + d]);
      if (n == 0) std::fill(out + qo, out + qo + D, 0.0);
      else attention_dense(qd.data(), Ks.data(), Vs.data(), n, D, sm_scale, out + qo);
    }
  }
}

unsigned lqo_hardware_threads() { return std::thread::hardware_concurrency(); }

}  // extern "C"
