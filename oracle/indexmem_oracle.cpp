// IndexMem CPU oracle — TEST INFRASTRUCTURE, NOT PRODUCT CODE.
//
// A plain, slow, step-by-step CPU statement of the IndexMem per-layer hot path
// (indexer score -> budgeted top-B selection -> latent-memory write -> attention
// over the retained KV + gated memory readout), written from the paper's
// equations in the paper's order and notation.  It shares no code with the CUDA
// library and must only be used by the tests, the smoke check and the CPU
// baseline leg of the benchmark.
//
// Arithmetic: every input/weight is a bf16 value widened exactly to float;
// every sum is accumulated in double; rounding happens only at the three
// storage points of the method as built here:
//   * the cached indexer key  -> bf16          (Sec. 3.1: "k are continuously cached")
//   * the pooled importance   -> float32       (Sec. 3.1: imp_t = max_s A_{s,t})
//   * the layer output        -> bf16 (an unrounded double copy is also returned)
//
// Pins (see tests/test_oracle_pins.py): infinite budget == textbook softmax
// attention; memory disabled == attention over exactly the retained set;
// brute-force top-B on tiny inputs; order invariance of (M,b) at lambda = 1;
// identity activation closed form; alpha == 0 tie case; single-pair rank-one
// closed form; lambda^j decay; the 19.92M indexer parameter count of the
// efficiency paragraph; score reuse by a following layer (App. B): the leader's
// positions, a numpy attention over the follower's own cache, the clone
// identity; per-KV-head retained sets (Sec. 2.2): brute-force Knorm selection
// per head, the assembled memory write against numpy, and the reduction to
// the shared-row path when every head is handed the same scores.
// Parity unpinned (no value in the paper fixes them): the memory widths under
// GQA (the printed 0.52M parameter count matches no stated width), act = ReLU,
// RMSNorm epsilon, the scalar sigmoid form of the gate g(q), softmax scale
// 1/sqrt(d_head), sinks counted inside the budget, and - with a retained set per
// KV head - how the slices a token loses in one evict step enter the memory
// (assembled into one model-space pair, zeros at the heads that keep the token).
//
// One handle = one layer.  Sequences inside a handle are independent.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>

namespace {

struct Cfg {
  int32_t H, Hkv, d;          // query heads, KV heads, head dim          (App. Notation)
  int32_t HI, dI, dM;         // H_index, d_index, d_mem                  (Sec. 4 hyperparameters)
  int32_t B;                  // KV budget B_max, sinks included          (Sec. 4 schedule)
  int32_t tau;                // compression interval                     (Sec. 4 schedule)
  int32_t n_sink;             // always-kept first tokens                 (Sec. 4 setup)
  int32_t act;                // 0 ReLU, 1 identity
  int32_t enable_memory;      // 0: no write, readout contributes nothing
  int32_t scorer;             // 0: the learnable indexer (one score row per sequence, Sec. 3.1); per-KV-head retained sets
                              // (Sec. 2.2 framework, S in R^{B x H_kv x L}): 1 Knorm S_t = ||K_t||_2, 2 scores given by the caller
  double scale;               // softmax scale
  double lambda, eta, eps, norm_eps;
};

inline double bf16_round(double x) {
  // round-to-nearest-even of x to a bfloat16 value, returned as double
  if (x == 0.0 || !std::isfinite(x)) return x;
  int e;
  double m = std::frexp(x, &e);            // x = m * 2^e, 0.5 <= |m| < 1
  // bf16 has 8 significant bits: scale so the integer part keeps 8 bits
  int min_e = -125;                        // normal range lower bound (2^-126 = 0.5 * 2^-125)
  int keep = 8;
  if (e < min_e) keep -= (min_e - e);      // subnormal: fewer bits
  if (keep <= 0) {
    // below half of the smallest subnormal rounds to zero, otherwise to it
    double tiny = std::ldexp(1.0, -133);   // smallest bf16 subnormal 2^-133
    if (std::fabs(x) > tiny * 0.5) return std::copysign(tiny, x);
    return std::copysign(0.0, x);
  }
  double scaled = std::ldexp(m, keep);     // |scaled| in [2^(keep-1), 2^keep)
  double r = std::nearbyint(scaled);       // default rounding mode: nearest-even
  return std::ldexp(r, e - keep);
}

struct Entry {
  int32_t pos;
  std::vector<float> k, v;     // [Hkv*d] each (bf16 values)
  std::vector<float> kidx;     // [dI]      (bf16 values)
  float acc;                   // pooled importance since the last compression
};

struct HEntry {                // one KV head's slice of a cached token (per-KV-head retained sets)
  int32_t pos;
  std::vector<float> k, v;     // [d] each (bf16 values)
  float score;                 // importance of the token for this head
};

struct Seq {
  std::vector<Entry> R;
  std::vector<std::vector<HEntry>> RH;           // per-KV-head mode: [Hkv] lists, ascending position
  std::vector<std::vector<int32_t>> h_evicted;   // [Hkv] positions evicted by the latest COMPRESS, ascending
  std::vector<std::vector<int32_t>> h_sel_pos;   // [Hkv] what the latest COMPRESS chose among ...
  std::vector<std::vector<float>> h_sel_score;   // ... and the scores it saw
  std::vector<double> M;       // [dM x D]  model space, Eq. 6
  std::vector<double> b;       // [dM]      Eq. 7
  int64_t T = 0;               // tokens appended so far (next position)
  int32_t since = 0;           // decode tokens since the last compression
  std::vector<int32_t> last_evicted;   // positions evicted by the latest COMPRESS, ascending
  std::vector<int32_t> sel_pos;        // what the latest COMPRESS chose among: positions ...
  std::vector<float> sel_acc;          // ... and pooled importance (cache order)
  int64_t n_evict_steps = 0;
};

struct Layer {
  Cfg c;
  int D, Dkv, Gq;
  std::vector<float> Uq, Uk, G, Wt, wg;   // [HI*dI x D], [dI x D], [HI x D], [dM x D], [D]
  float bg = 0.f;
  std::vector<Seq> seqs;
};

// ---------------------------------------------------------------- stage functions

// Sec. 3.1 "Architecture": k_t = Norm(U_k X_t), rounded to the bf16 cache format.
void index_key(const Layer& L, const float* x, float* kidx_out) {
  const int dI = L.c.dI, D = L.D;
  std::vector<double> u(dI);
  double ms = 0.0;
  for (int r = 0; r < dI; ++r) {
    double s = 0.0;
    for (int i = 0; i < D; ++i) s += (double)L.Uk[(size_t)r * D + i] * (double)x[i];
    u[r] = s;
    ms += s * s;
  }
  double inv = 1.0 / std::sqrt(ms / dI + L.c.norm_eps);
  for (int r = 0; r < dI; ++r) kidx_out[r] = (float)bf16_round(u[r] * inv);
}

// Sec. 3.1: q_s = U_q flatten(Q_s), viewed [H_index, d_index], RMSNorm over d_index;
// alpha_s = G X_s / sqrt(H_index d_index).
void index_query(const Layer& L, const float* x, const float* q_pre, double* qf, double* alpha) {
  const int HI = L.c.HI, dI = L.c.dI, D = L.D;
  for (int h = 0; h < HI; ++h) {
    double ms = 0.0;
    for (int r = 0; r < dI; ++r) {
      double s = 0.0;
      const float* w = &L.Uq[(size_t)(h * dI + r) * D];
      for (int i = 0; i < D; ++i) s += (double)w[i] * (double)q_pre[i];
      qf[h * dI + r] = s;
      ms += s * s;
    }
    double inv = 1.0 / std::sqrt(ms / dI + L.c.norm_eps);
    for (int r = 0; r < dI; ++r) qf[h * dI + r] *= inv;
  }
  const double gs = 1.0 / std::sqrt((double)HI * (double)dI);
  for (int h = 0; h < HI; ++h) {
    double s = 0.0;
    const float* w = &L.G[(size_t)h * D];
    for (int i = 0; i < D; ++i) s += (double)w[i] * (double)x[i];
    alpha[h] = s * gs;
  }
}

// Sec. 3.1: z = act(q_s . k_t) per indexer head, A_{s,t} = alpha_s^T z_{s,t}.
double index_score(const Cfg& c, const double* qf, const double* alpha, const float* kidx) {
  double A = 0.0;
  for (int h = 0; h < c.HI; ++h) {
    double z = 0.0;
    for (int r = 0; r < c.dI; ++r) z += qf[h * c.dI + r] * (double)kidx[r];
    if (c.act == 0 && z < 0.0) z = 0.0;
    A += alpha[h] * z;
  }
  return A;
}

// Sec. 2.2 scoring-and-selection: keep the B entries with the largest key, key = +inf for the
// sink positions, order (key descending, original position ascending); -0.0 == +0.0 numerically.
// keep[i] = 1 for retained entries.  Returns the number evicted.
int select_top_b(const float* score, const int32_t* pos, int n, int B, int n_sink, uint8_t* keep) {
  std::vector<int> order(n);
  for (int i = 0; i < n; ++i) order[i] = i;
  auto key = [&](int i) -> double {
    return pos[i] < n_sink ? std::numeric_limits<double>::infinity() : (double)score[i];
  };
  std::stable_sort(order.begin(), order.end(), [&](int a, int b2) {
    double ka = key(a), kb = key(b2);
    if (ka != kb) return ka > kb;
    return pos[a] < pos[b2];
  });
  int kept = std::min(n, B);
  for (int i = 0; i < n; ++i) keep[i] = 0;
  for (int i = 0; i < kept; ++i) keep[order[i]] = 1;
  return n - kept;
}

// phi(.) = Linear_theta(.) on a model-space vector (App. Notation).
void phi_of(const Layer& L, const double* u /*[D]*/, double* phi /*[dM]*/) {
  for (int m = 0; m < L.c.dM; ++m) {
    double s = 0.0;
    const float* w = &L.Wt[(size_t)m * L.D];
    for (int i = 0; i < L.D; ++i) s += (double)w[i] * u[i];
    phi[m] = s;
  }
}

// lift a cached [Hkv, d] key/value to model space the way the backbone's grouped-query
// attention does: query head j reads KV head j / G_q.
void repeat_kv(const Layer& L, const float* kv, double* out /*[D]*/) {
  for (int j = 0; j < L.c.H; ++j)
    for (int c = 0; c < L.c.d; ++c) out[j * L.c.d + c] = (double)kv[(j / L.Gq) * L.c.d + c];
}

// Eq. 6-7: one evict step over the evicted set E.
void mem_write(const Layer& L, Seq& S, const std::vector<const Entry*>& E) {
  const int dM = L.c.dM, D = L.D;
  std::vector<double> sumM((size_t)dM * D, 0.0), sumb(dM, 0.0), ku(D), vu(D), phi(dM);
  for (const Entry* e : E) {
    repeat_kv(L, e->k.data(), ku.data());
    repeat_kv(L, e->v.data(), vu.data());
    phi_of(L, ku.data(), phi.data());
    for (int m = 0; m < dM; ++m) {
      double p = phi[m];
      double* row = &sumM[(size_t)m * D];
      for (int i = 0; i < D; ++i) row[i] += p * vu[i];
      sumb[m] += p * p;
    }
  }
  for (size_t i = 0; i < S.M.size(); ++i) S.M[i] = L.c.lambda * S.M[i] + L.c.eta * sumM[i];
  for (int m = 0; m < dM; ++m) S.b[m] = L.c.lambda * S.b[m] + L.c.eta * sumb[m];
}

// Eq. 5: m(q) = phi(q)^T M / (phi(q)^{.2 T} b + eps)   -> [D]
void mem_read(const Layer& L, const Seq& S, const float* q /*[D]*/, double* m_out) {
  const int dM = L.c.dM, D = L.D;
  std::vector<double> qd(D), phi(dM);
  for (int i = 0; i < D; ++i) qd[i] = (double)q[i];
  phi_of(L, qd.data(), phi.data());
  double den = L.c.eps;
  for (int m = 0; m < dM; ++m) den += phi[m] * phi[m] * S.b[m];
  for (int i = 0; i < D; ++i) m_out[i] = 0.0;
  for (int m = 0; m < dM; ++m) {
    const double* row = &S.M[(size_t)m * D];
    for (int i = 0; i < D; ++i) m_out[i] += phi[m] * row[i];
  }
  for (int i = 0; i < D; ++i) m_out[i] /= den;
}

// g(q) in [0,1] (Eq. 4): scalar sigmoid gate on the head-concatenated query.
double gate_of(const Layer& L, const float* q) {
  double s = (double)L.bg;
  for (int i = 0; i < L.D; ++i) s += (double)L.wg[i] * (double)q[i];
  return 1.0 / (1.0 + std::exp(-s));
}

// Sec. 2.1 KV caching: o_j = sum_t softmax_t(scale q_j . k_t) v_t over the retained set.
// `max_pos`: only entries at positions <= max_pos take part (the causal mask of a chunk's own queries);
// entries are kept in ascending position, so these are a prefix of the list.
void attention(const Layer& L, const Seq& S, const float* q /*[H,d]*/, double* o /*[H,d]*/,
               int64_t max_pos = std::numeric_limits<int64_t>::max()) {
  const int d = L.c.d;
  size_t n = 0;
  while (n < S.R.size() && (int64_t)S.R[n].pos <= max_pos) ++n;
  std::vector<double> logit(n);
  for (int j = 0; j < L.c.H; ++j) {
    const int g = j / L.Gq;
    double mx = -std::numeric_limits<double>::infinity();
    for (size_t t = 0; t < n; ++t) {
      double s = 0.0;
      const float* kk = &S.R[t].k[(size_t)g * d];
      for (int c = 0; c < d; ++c) s += (double)q[j * d + c] * (double)kk[c];
      logit[t] = s * L.c.scale;
      mx = std::max(mx, logit[t]);
    }
    double den = 0.0;
    for (size_t t = 0; t < n; ++t) { logit[t] = std::exp(logit[t] - mx); den += logit[t]; }
    for (int c = 0; c < d; ++c) o[j * d + c] = 0.0;
    for (size_t t = 0; t < n; ++t) {
      double p = logit[t] / den;
      const float* vv = &S.R[t].v[(size_t)g * d];
      for (int c = 0; c < d; ++c) o[j * d + c] += p * (double)vv[c];
    }
  }
}

// Sec. 4 schedule: compress to the budget, write the evicted set to memory, restart pooling.
void compress(const Layer& L, Seq& S) {
  S.since = 0;
  S.last_evicted.clear();
  const int n = (int)S.R.size();
  S.sel_pos.resize(n);
  S.sel_acc.resize(n);
  for (int i = 0; i < n; ++i) { S.sel_pos[i] = S.R[i].pos; S.sel_acc[i] = S.R[i].acc; }
  if (n > L.c.B) {
    std::vector<float> sc(n);
    std::vector<int32_t> ps(n);
    std::vector<uint8_t> keep(n);
    for (int i = 0; i < n; ++i) { sc[i] = S.R[i].acc; ps[i] = S.R[i].pos; }
    select_top_b(sc.data(), ps.data(), n, L.c.B, L.c.n_sink, keep.data());
    std::vector<const Entry*> E;
    for (int i = 0; i < n; ++i) if (!keep[i]) E.push_back(&S.R[i]);
    if (L.c.enable_memory) mem_write(L, S, E);
    for (const Entry* e : E) S.last_evicted.push_back(e->pos);
    std::sort(S.last_evicted.begin(), S.last_evicted.end());
    std::vector<Entry> kept;
    kept.reserve(L.c.B);
    for (int i = 0; i < n; ++i) if (keep[i]) kept.push_back(std::move(S.R[i]));
    S.R.swap(kept);
    S.n_evict_steps++;
  }
  for (Entry& e : S.R) e.acc = -std::numeric_limits<float>::infinity();
}

void append(const Layer& L, Seq& S, const float* x, const float* k, const float* v) {
  Entry e;
  e.pos = (int32_t)S.T;
  e.k.assign(k, k + L.Dkv);
  e.v.assign(v, v + L.Dkv);
  e.kidx.resize(L.c.dI);
  index_key(L, x, e.kidx.data());
  e.acc = -std::numeric_limits<float>::infinity();
  S.R.push_back(std::move(e));
  S.T += 1;
}

// App. B "From Running Mean to IndexCache": a layer that reuses the indexer scores of a neighbouring layer computes
// no indexer features of its own; its cached entries carry no indexer key.
void append_without_index(const Layer& L, Seq& S, const float* k, const float* v) {
  Entry e;
  e.pos = (int32_t)S.T;
  e.k.assign(k, k + L.Dkv);
  e.v.assign(v, v + L.Dkv);
  e.kidx.assign(L.c.dI, 0.f);
  e.acc = -std::numeric_limits<float>::infinity();
  S.R.push_back(std::move(e));
  S.T += 1;
}

// App. B: "compute the indexer scores once within a short group of neighbouring layers and reuse the resulting
// scores ... for the remaining layers in the group".  The scores reused are the pooled importances the leading
// layer's latest compression chose among, matched by token position.  Returns false if the leading layer has no
// score for one of this layer's entries (the two layers must have seen the same tokens and made the same calls).
bool adopt_scores(Seq& S, const Seq& lead) {
  for (Entry& e : S.R) {
    bool found = false;
    for (size_t i = 0; i < lead.sel_pos.size(); ++i)
      if (lead.sel_pos[i] == e.pos) {
        e.acc = lead.sel_acc[i];
        found = true;
        break;
      }
    if (!found) return false;
  }
  return true;
}

// ---------------------------------------------------------------- per-KV-head retained sets (Sec. 2.2)
// Sec. 2.2 states eviction as S = f(.) in R^{B x H_kv x L}, I = TopK(S, L'), [K', V'] = Gather(K, V, I): every KV head keeps
// its own set of token positions.  Two scorers with a head axis: Knorm (S_t = ||K_t||_2, Sec. 2.2) and scores handed in
// by the caller (the memory module on top of another eviction policy, Sec. 5 ablation "SnapKV+Memory").

// Knorm, Sec. 2.2: the key's magnitude for this head, kept as float32
float knorm_score(const float* k, int d) {
  double s = 0.0;
  for (int c = 0; c < d; ++c) s += (double)k[c] * (double)k[c];
  return (float)std::sqrt(s);
}

void ph_init(const Layer& L, Seq& S) {
  if ((int)S.RH.size() != L.c.Hkv) {
    S.RH.assign(L.c.Hkv, {});
    S.h_evicted.assign(L.c.Hkv, {});
    S.h_sel_pos.assign(L.c.Hkv, {});
    S.h_sel_score.assign(L.c.Hkv, {});
  }
}

void ph_append(const Layer& L, Seq& S, const float* k /*[Hkv,d]*/, const float* v) {
  ph_init(L, S);
  const int d = L.c.d;
  for (int h = 0; h < L.c.Hkv; ++h) {
    HEntry e;
    e.pos = (int32_t)S.T;
    e.k.assign(k + (size_t)h * d, k + (size_t)(h + 1) * d);
    e.v.assign(v + (size_t)h * d, v + (size_t)(h + 1) * d);
    e.score = L.c.scorer == 1 ? knorm_score(e.k.data(), d) : -std::numeric_limits<float>::infinity();
    S.RH[h].push_back(std::move(e));
  }
  S.T += 1;
}

// Eq. 6-7 over model-space pairs (k~_i, v~_i)
void mem_write_model(const Layer& L, Seq& S, const std::vector<std::vector<double>>& ku, const std::vector<std::vector<double>>& vu) {
  const int dM = L.c.dM, D = L.D;
  std::vector<double> sumM((size_t)dM * D, 0.0), sumb(dM, 0.0), phi(dM);
  for (size_t i = 0; i < ku.size(); ++i) {
    phi_of(L, ku[i].data(), phi.data());
    for (int m = 0; m < dM; ++m) {
      const double p = phi[m];
      double* row = &sumM[(size_t)m * D];
      for (int c = 0; c < D; ++c) row[c] += p * vu[i][c];
      sumb[m] += p * p;
    }
  }
  for (size_t i = 0; i < S.M.size(); ++i) S.M[i] = L.c.lambda * S.M[i] + L.c.eta * sumM[i];
  for (int m = 0; m < dM; ++m) S.b[m] = L.c.lambda * S.b[m] + L.c.eta * sumb[m];
}

// Compression with a set of retained positions per KV head.  ext: scores handed in by the caller, [Hkv][n_pos] indexed
// by token position (scorer 2), else null.  The memory write of this evict step (Alg. 1: "evicted_v is summed across
// heads per token"): for every token that loses at least one head slice in this step, the evicted slices are assembled
// into ONE model-space key and value - the slice of KV head g at the places of its query heads, zeros at the heads
// that keep the token - and written as one pair of Eq. 6-7.
bool ph_compress(const Layer& L, Seq& S, const float* ext, int64_t n_pos) {
  const int Hkv = L.c.Hkv, d = L.c.d;
  S.since = 0;
  std::vector<std::vector<uint8_t>> keep(Hkv);
  bool any = false;
  for (int h = 0; h < Hkv; ++h) {
    std::vector<HEntry>& R = S.RH[h];
    const int n = (int)R.size();
    if (L.c.scorer == 2) {
      if (!ext) return false;
      for (HEntry& e : R) {
        if (e.pos >= n_pos) return false;
        e.score = ext[(size_t)h * n_pos + e.pos];
      }
    }
    S.h_evicted[h].clear();
    S.h_sel_pos[h].resize(n);
    S.h_sel_score[h].resize(n);
    std::vector<float> sc(n);
    std::vector<int32_t> ps(n);
    for (int i = 0; i < n; ++i) { S.h_sel_pos[h][i] = ps[i] = R[i].pos; S.h_sel_score[h][i] = sc[i] = R[i].score; }
    keep[h].assign(n, 1);
    if (n > L.c.B) {
      select_top_b(sc.data(), ps.data(), n, L.c.B, L.c.n_sink, keep[h].data());
      any = true;
    }
  }
  if (any) {
    // tokens that lose a slice, ascending position, with the heads that evict them
    std::vector<int32_t> toks;
    for (int h = 0; h < Hkv; ++h)
      for (size_t i = 0; i < S.RH[h].size(); ++i)
        if (!keep[h][i]) { toks.push_back(S.RH[h][i].pos); S.h_evicted[h].push_back(S.RH[h][i].pos); }
    std::sort(toks.begin(), toks.end());
    toks.erase(std::unique(toks.begin(), toks.end()), toks.end());
    if (L.c.enable_memory) {
      std::vector<std::vector<double>> ku(toks.size(), std::vector<double>(L.D, 0.0)), vu(toks.size(), std::vector<double>(L.D, 0.0));
      for (int h = 0; h < Hkv; ++h)
        for (size_t i = 0; i < S.RH[h].size(); ++i) {
          if (keep[h][i]) continue;
          const HEntry& e = S.RH[h][i];
          const size_t r = std::lower_bound(toks.begin(), toks.end(), e.pos) - toks.begin();
          for (int j = h * L.Gq; j < (h + 1) * L.Gq; ++j)       // the query heads that read KV head h
            for (int c = 0; c < d; ++c) { ku[r][(size_t)j * d + c] = (double)e.k[c]; vu[r][(size_t)j * d + c] = (double)e.v[c]; }
        }
      mem_write_model(L, S, ku, vu);
    }
    for (int h = 0; h < Hkv; ++h) {
      std::vector<HEntry> kept;
      for (size_t i = 0; i < S.RH[h].size(); ++i) if (keep[h][i]) kept.push_back(std::move(S.RH[h][i]));
      S.RH[h].swap(kept);
    }
    S.n_evict_steps++;
  }
  return true;
}

// Sec. 2.1 attention with every KV head's own retained set
void ph_attention(const Layer& L, const Seq& S, const float* q /*[H,d]*/, double* o /*[H,d]*/, int64_t max_pos) {
  const int d = L.c.d;
  for (int j = 0; j < L.c.H; ++j) {
    const std::vector<HEntry>& R = S.RH[j / L.Gq];
    size_t n = 0;
    while (n < R.size() && (int64_t)R[n].pos <= max_pos) ++n;
    std::vector<double> logit(n);
    double mx = -std::numeric_limits<double>::infinity();
    for (size_t t = 0; t < n; ++t) {
      double s = 0.0;
      for (int c = 0; c < d; ++c) s += (double)q[j * d + c] * (double)R[t].k[c];
      logit[t] = s * L.c.scale;
      mx = std::max(mx, logit[t]);
    }
    double den = 0.0;
    for (size_t t = 0; t < n; ++t) { logit[t] = std::exp(logit[t] - mx); den += logit[t]; }
    for (int c = 0; c < d; ++c) o[j * d + c] = 0.0;
    for (size_t t = 0; t < n; ++t) {
      const double p = logit[t] / den;
      for (int c = 0; c < d; ++c) o[j * d + c] += p * (double)R[t].v[c];
    }
  }
}

void ph_layer_output(const Layer& L, const Seq& S, const float* q, int64_t max_pos, float* out_bf16, double* out_f64) {
  const int D = L.D;
  std::vector<double> o(D), m(D, 0.0);
  ph_attention(L, S, q, o.data(), max_pos);
  double gate = 0.0;
  if (L.c.enable_memory) {
    mem_read(L, S, q, m.data());
    gate = gate_of(L, q);
  }
  for (int j = 0; j < D; ++j) {
    const double val = o[j] + gate * m[j];
    if (out_f64) out_f64[j] = val;
    if (out_bf16) out_bf16[j] = (float)bf16_round(val);
  }
}

// Eq. 4-5 for one query: attention over the retained set plus the gated memory readout
void layer_output(const Layer& L, const Seq& S, const float* q, int64_t max_pos, float* out_bf16, double* out_f64) {
  const int D = L.D;
  std::vector<double> o(D), m(D, 0.0);
  attention(L, S, q, o.data(), max_pos);
  double gate = 0.0;
  if (L.c.enable_memory) {
    mem_read(L, S, q, m.data());
    gate = gate_of(L, q);
  }
  for (int j = 0; j < D; ++j) {
    const double val = o[j] + gate * m[j];
    if (out_f64) out_f64[j] = val;
    if (out_bf16) out_bf16[j] = (float)bf16_round(val);
  }
}

}  // namespace

// ------------------------------------------------------------------------ C API
extern "C" {

struct orc_config {          // mirrors Cfg; kept separate so the ABI is explicit
  int32_t H, Hkv, d, HI, dI, dM, B, tau, n_sink, act, enable_memory, scorer;
  double scale, lambda, eta, eps, norm_eps;
};

void* orc_create(const orc_config* cfg, int n_seq) {
  Layer* L = new Layer();
  std::memcpy(&L->c, cfg, sizeof(Cfg));
  L->D = cfg->H * cfg->d;
  L->Dkv = cfg->Hkv * cfg->d;
  L->Gq = cfg->H / cfg->Hkv;
  L->Uq.assign((size_t)cfg->HI * cfg->dI * L->D, 0.f);
  L->Uk.assign((size_t)cfg->dI * L->D, 0.f);
  L->G.assign((size_t)cfg->HI * L->D, 0.f);
  L->Wt.assign((size_t)cfg->dM * L->D, 0.f);
  L->wg.assign((size_t)L->D, 0.f);
  L->seqs.resize(n_seq);
  for (Seq& s : L->seqs) {
    s.M.assign((size_t)cfg->dM * L->D, 0.0);
    s.b.assign((size_t)cfg->dM, 0.0);
  }
  return L;
}

void orc_destroy(void* h) { delete static_cast<Layer*>(h); }

// which: 0 U_q, 1 U_k, 2 G, 3 Linear_theta, 4 w_g, 5 b_g (1 float)
int orc_set_weights(void* h, int which, const float* data, int64_t n) {
  Layer* L = static_cast<Layer*>(h);
  std::vector<float>* dst = nullptr;
  switch (which) {
    case 0: dst = &L->Uq; break;
    case 1: dst = &L->Uk; break;
    case 2: dst = &L->G; break;
    case 3: dst = &L->Wt; break;
    case 4: dst = &L->wg; break;
    case 5: if (n != 1) return -1; L->bg = data[0]; return 0;
    default: return -1;
  }
  if ((int64_t)dst->size() != n) return -1;
  std::copy(data, data + n, dst->begin());
  return 0;
}

// Sec. 4 schedule, prefill side: append the chunk, pool the chunk's query scores over every cached
// entry under the causal mask, then compress to the budget.
// Optional layer outputs of the chunk's own queries (Q != null; Eq. 4-5): query s attends to what is cached
// when the chunk arrives plus the chunk's tokens up to itself (Sec. 2.1 causal attention; the chunk is
// compressed only after it has been processed, Sec. 4), and reads the memory as the previous evict steps
// left it.  out_bf16 / out_f64: [C,H,d], either may be null.
int orc_prefill_chunk_out(void* h, int seq, int C, const float* X /*[C,D]*/, const float* Qpre /*[C,H,d]*/,
                          const float* Q /*[C,H,d] or null*/, const float* K /*[C,Hkv,d]*/,
                          const float* V /*[C,Hkv,d]*/, float* out_bf16, double* out_f64) {
  Layer* L = static_cast<Layer*>(h);
  Seq& S = L->seqs[seq];
  const int D = L->D, Dkv = L->Dkv, HI = L->c.HI, dI = L->c.dI;
  const int64_t T0 = S.T;
  for (int c = 0; c < C; ++c)
    append(*L, S, X + (size_t)c * D, K + (size_t)c * Dkv, V + (size_t)c * Dkv);
  if (Q && (out_bf16 || out_f64)) {
    std::vector<double> o(D), m(D);
    for (int c = 0; c < C; ++c) {
      const float* q = Q + (size_t)c * D;
      attention(*L, S, q, o.data(), T0 + c);
      double gate = 0.0;
      std::fill(m.begin(), m.end(), 0.0);
      if (L->c.enable_memory) {
        mem_read(*L, S, q, m.data());
        gate = gate_of(*L, q);
      }
      for (int j = 0; j < D; ++j) {
        const double val = o[j] + gate * m[j];
        if (out_f64) out_f64[(size_t)c * D + j] = val;
        if (out_bf16) out_bf16[(size_t)c * D + j] = (float)bf16_round(val);
      }
    }
  }
  std::vector<double> qf((size_t)C * HI * dI), alpha((size_t)C * HI);
  for (int c = 0; c < C; ++c)
    index_query(*L, X + (size_t)c * D, Qpre + (size_t)c * D, &qf[(size_t)c * HI * dI], &alpha[(size_t)c * HI]);
  for (Entry& e : S.R) {
    for (int c = 0; c < C; ++c) {
      if (T0 + c < e.pos) continue;                       // causal mask: query sees keys at or before it
      double A = index_score(L->c, &qf[(size_t)c * HI * dI], &alpha[(size_t)c * HI], e.kidx.data());
      float Af = (float)A;
      if (Af > e.acc) e.acc = Af;
    }
  }
  compress(*L, S);
  return 0;
}
int orc_prefill_chunk(void* h, int seq, int C, const float* X, const float* Qpre, const float* K, const float* V) {
  return orc_prefill_chunk_out(h, seq, C, X, Qpre, nullptr, K, V, nullptr, nullptr);
}

// One decode token for one sequence (Sec. 4 schedule, decode side; Eq. 4-7).
// out_bf16: [H,d] rounded to bf16 values; out_f64: [H,d] unrounded (may be null).
int orc_decode_step(void* h, int seq, const float* x, const float* q_pre, const float* q,
                    const float* k_new, const float* v_new, float* out_bf16, double* out_f64) {
  Layer* L = static_cast<Layer*>(h);
  Seq& S = L->seqs[seq];
  const int D = L->D, d = L->c.d;
  append(*L, S, x, k_new, v_new);
  std::vector<double> qf((size_t)L->c.HI * L->c.dI), alpha(L->c.HI);
  index_query(*L, x, q_pre, qf.data(), alpha.data());
  for (Entry& e : S.R) {
    float Af = (float)index_score(L->c, qf.data(), alpha.data(), e.kidx.data());
    if (Af > e.acc) e.acc = Af;
  }
  S.since += 1;
  if (S.since == L->c.tau) compress(*L, S);
  std::vector<double> o(D), m(D, 0.0);
  attention(*L, S, q, o.data());
  double gate = 0.0;
  if (L->c.enable_memory) {
    mem_read(*L, S, q, m.data());
    gate = gate_of(*L, q);
  }
  for (int j = 0; j < L->c.H; ++j)
    for (int c = 0; c < d; ++c) {
      double val = o[j * d + c] + gate * m[j * d + c];
      if (out_f64) out_f64[j * d + c] = val;
      if (out_bf16) out_bf16[j * d + c] = (float)bf16_round(val);
    }
  return 0;
}

// The two calls for a layer that reuses the indexer scores of the leading layer of its group (App. B, IndexCache-style
// reuse; the paper reuses scores "across every four consecutive layers").  `lead` / `lead_seq`: the leading layer's
// handle and sequence, which must already have made the same call for the same tokens.  The layer appends its own
// K / V, adopts the leading layer's pooled importances when a compression is due, and does everything else - selection
// under its own budget and sinks, memory write from its own evicted pairs (Eq. 6-7), attention over its own retained
// entries and readout of its own memory (Eq. 4-5) - as any layer does.  Returns -1 if the leading layer's scores do
// not cover this layer's entries.
int orc_decode_step_follow(void* h, int seq, void* lead, int lead_seq, const float* q, const float* k_new,
                           const float* v_new, float* out_bf16, double* out_f64) {
  Layer* L = static_cast<Layer*>(h);
  Seq& S = L->seqs[seq];
  const Seq& LS = static_cast<Layer*>(lead)->seqs[lead_seq];
  append_without_index(*L, S, k_new, v_new);
  S.since += 1;
  if (S.since == L->c.tau) {
    if (!adopt_scores(S, LS)) return -1;
    compress(*L, S);
  }
  layer_output(*L, S, q, std::numeric_limits<int64_t>::max(), out_bf16, out_f64);
  return 0;
}
int orc_prefill_chunk_follow(void* h, int seq, void* lead, int lead_seq, int C, const float* Q /*[C,H,d] or null*/,
                             const float* K, const float* V, float* out_bf16, double* out_f64) {
  Layer* L = static_cast<Layer*>(h);
  Seq& S = L->seqs[seq];
  const Seq& LS = static_cast<Layer*>(lead)->seqs[lead_seq];
  const int D = L->D, Dkv = L->Dkv;
  const int64_t T0 = S.T;
  for (int c = 0; c < C; ++c) append_without_index(*L, S, K + (size_t)c * Dkv, V + (size_t)c * Dkv);
  if (Q && (out_bf16 || out_f64))
    for (int c = 0; c < C; ++c)
      layer_output(*L, S, Q + (size_t)c * D, T0 + c, out_bf16 ? out_bf16 + (size_t)c * D : nullptr,
                   out_f64 ? out_f64 + (size_t)c * D : nullptr);
  if (!adopt_scores(S, LS)) return -1;
  compress(*L, S);
  return 0;
}

// The two calls with a retained set per KV head (configuration scorer = 1 Knorm, 2 scores from the caller).  ext: float32
// [Hkv][n_pos], the importance of token position p for KV head h at ext[h * n_pos + p]; it must cover every position
// cached after the call's append (scorer 2; ignored by Knorm).  Returns -1 if scores are missing.
int orc_ph_decode_step(void* h, int seq, const float* q, const float* k_new, const float* v_new, const float* ext,
                       int64_t n_pos, float* out_bf16, double* out_f64) {
  Layer* L = static_cast<Layer*>(h);
  Seq& S = L->seqs[seq];
  ph_append(*L, S, k_new, v_new);
  S.since += 1;
  if (S.since == L->c.tau && !ph_compress(*L, S, ext, n_pos)) return -1;
  ph_layer_output(*L, S, q, std::numeric_limits<int64_t>::max(), out_bf16, out_f64);
  return 0;
}
int orc_ph_prefill_chunk(void* h, int seq, int C, const float* Q /*[C,H,d] or null*/, const float* K, const float* V,
                         const float* ext, int64_t n_pos, float* out_bf16, double* out_f64) {
  Layer* L = static_cast<Layer*>(h);
  Seq& S = L->seqs[seq];
  const int D = L->D, Dkv = L->Dkv;
  const int64_t T0 = S.T;
  for (int c = 0; c < C; ++c) ph_append(*L, S, K + (size_t)c * Dkv, V + (size_t)c * Dkv);
  if (Q && (out_bf16 || out_f64))
    for (int c = 0; c < C; ++c)
      ph_layer_output(*L, S, Q + (size_t)c * D, T0 + c, out_bf16 ? out_bf16 + (size_t)c * D : nullptr,
                      out_f64 ? out_f64 + (size_t)c * D : nullptr);
  return ph_compress(*L, S, ext, n_pos) ? 0 : -1;
}
int orc_ph_count(void* h, int seq, int head) {
  Seq& S = static_cast<Layer*>(h)->seqs[seq];
  return head < (int)S.RH.size() ? (int)S.RH[head].size() : 0;
}
void orc_ph_export(void* h, int seq, int head, int32_t* pos, float* score, float* K, float* V) {
  Layer* L = static_cast<Layer*>(h);
  const std::vector<HEntry>& R = L->seqs[seq].RH[head];
  const int d = L->c.d;
  for (size_t i = 0; i < R.size(); ++i) {
    if (pos) pos[i] = R[i].pos;
    if (score) score[i] = R[i].score;
    if (K) std::memcpy(K + i * d, R[i].k.data(), sizeof(float) * d);
    if (V) std::memcpy(V + i * d, R[i].v.data(), sizeof(float) * d);
  }
}
int orc_ph_last_evicted(void* h, int seq, int head, int32_t* pos, int cap) {
  const std::vector<int32_t>& e = static_cast<Layer*>(h)->seqs[seq].h_evicted[head];
  if (pos) for (size_t i = 0; i < e.size() && (int)i < cap; ++i) pos[i] = e[i];
  return (int)e.size();
}
int orc_ph_last_selection(void* h, int seq, int head, int32_t* pos, float* score, int cap) {
  const Seq& S = static_cast<Layer*>(h)->seqs[seq];
  const int n = (int)S.h_sel_pos[head].size();
  for (int i = 0; i < n && i < cap; ++i) {
    if (pos) pos[i] = S.h_sel_pos[head][i];
    if (score) score[i] = S.h_sel_score[head][i];
  }
  return n;
}

// The same two calls over several independent sequences (one OpenMP thread per sequence).
int orc_decode_batch(void* h, int n_seq, const int32_t* seq_ids, const float* x, const float* q_pre,
                     const float* q, const float* k_new, const float* v_new, float* out_bf16, double* out_f64) {
  Layer* L = static_cast<Layer*>(h);
  const size_t D = L->D, Dkv = L->Dkv;
#pragma omp parallel for schedule(dynamic, 1)
  for (int i = 0; i < n_seq; ++i)
    orc_decode_step(h, seq_ids[i], x + i * D, q_pre + i * D, q + i * D, k_new + i * Dkv, v_new + i * Dkv,
                    out_bf16 ? out_bf16 + i * D : nullptr, out_f64 ? out_f64 + i * D : nullptr);
  return 0;
}
int orc_prefill_batch_out(void* h, int n_seq, const int32_t* seq_ids, int C, const float* X, const float* Qpre,
                          const float* Q, const float* K, const float* V, float* out_bf16, double* out_f64) {
  Layer* L = static_cast<Layer*>(h);
  const size_t D = L->D, Dkv = L->Dkv;
#pragma omp parallel for schedule(dynamic, 1)
  for (int i = 0; i < n_seq; ++i)
    orc_prefill_chunk_out(h, seq_ids[i], C, X + (size_t)i * C * D, Qpre + (size_t)i * C * D,
                          Q ? Q + (size_t)i * C * D : nullptr, K + (size_t)i * C * Dkv, V + (size_t)i * C * Dkv,
                          out_bf16 ? out_bf16 + (size_t)i * C * D : nullptr, out_f64 ? out_f64 + (size_t)i * C * D : nullptr);
  return 0;
}
int orc_prefill_batch(void* h, int n_seq, const int32_t* seq_ids, int C, const float* X, const float* Qpre,
                      const float* K, const float* V) {
  return orc_prefill_batch_out(h, n_seq, seq_ids, C, X, Qpre, nullptr, K, V, nullptr, nullptr);
}

// ---- state export (entries in cache order = ascending position)
int orc_count(void* h, int seq) { return (int)static_cast<Layer*>(h)->seqs[seq].R.size(); }
int64_t orc_tokens_seen(void* h, int seq) { return static_cast<Layer*>(h)->seqs[seq].T; }
int orc_since(void* h, int seq) { return static_cast<Layer*>(h)->seqs[seq].since; }
int64_t orc_evict_steps(void* h, int seq) { return static_cast<Layer*>(h)->seqs[seq].n_evict_steps; }

void orc_export_entries(void* h, int seq, int32_t* pos, float* acc, float* kidx, float* K, float* V) {
  Layer* L = static_cast<Layer*>(h);
  Seq& S = L->seqs[seq];
  for (size_t i = 0; i < S.R.size(); ++i) {
    const Entry& e = S.R[i];
    if (pos) pos[i] = e.pos;
    if (acc) acc[i] = e.acc;
    if (kidx) std::copy(e.kidx.begin(), e.kidx.end(), kidx + i * L->c.dI);
    if (K) std::copy(e.k.begin(), e.k.end(), K + i * L->Dkv);
    if (V) std::copy(e.v.begin(), e.v.end(), V + i * L->Dkv);
  }
}
void orc_export_memory(void* h, int seq, double* M /*[dM,D]*/, double* b /*[dM]*/) {
  Layer* L = static_cast<Layer*>(h);
  Seq& S = L->seqs[seq];
  if (M) std::copy(S.M.begin(), S.M.end(), M);
  if (b) std::copy(S.b.begin(), S.b.end(), b);
}
int orc_last_evicted(void* h, int seq, int32_t* pos, int cap) {
  Seq& S = static_cast<Layer*>(h)->seqs[seq];
  int n = (int)S.last_evicted.size();
  for (int i = 0; i < n && i < cap; ++i) pos[i] = S.last_evicted[i];
  return n;
}

int orc_last_selection(void* h, int seq, int32_t* pos, float* acc, int cap) {
  Seq& S = static_cast<Layer*>(h)->seqs[seq];
  int n = (int)S.sel_pos.size();
  for (int i = 0; i < n && i < cap; ++i) { pos[i] = S.sel_pos[i]; acc[i] = S.sel_acc[i]; }
  return n;
}

// ---- stage functions exposed for pins and stage-wise parity
void orc_index_key(void* h, const float* x, float* kidx) { index_key(*static_cast<Layer*>(h), x, kidx); }
void orc_index_query(void* h, const float* x, const float* q_pre, double* qf, double* alpha) {
  index_query(*static_cast<Layer*>(h), x, q_pre, qf, alpha);
}
void orc_index_scores(void* h, const double* qf, const double* alpha, const float* kidx, int n, double* A) {
  Layer* L = static_cast<Layer*>(h);
  for (int t = 0; t < n; ++t) A[t] = index_score(L->c, qf, alpha, kidx + (size_t)t * L->c.dI);
}
int orc_select_top_b(const float* score, const int32_t* pos, int n, int B, int n_sink, uint8_t* keep) {
  return select_top_b(score, pos, n, B, n_sink, keep);
}
void orc_phi(void* h, const float* u_model /*[D]*/, double* phi) {
  Layer* L = static_cast<Layer*>(h);
  std::vector<double> u(L->D);
  for (int i = 0; i < L->D; ++i) u[i] = (double)u_model[i];
  phi_of(*L, u.data(), phi);
}
void orc_phi_kv(void* h, const float* kv /*[Hkv,d]*/, double* phi) {
  Layer* L = static_cast<Layer*>(h);
  std::vector<double> u(L->D);
  repeat_kv(*L, kv, u.data());
  phi_of(*L, u.data(), phi);
}
void orc_mem_read(void* h, int seq, const float* q, double* m_out, double* gate_out) {
  Layer* L = static_cast<Layer*>(h);
  mem_read(*L, L->seqs[seq], q, m_out);
  if (gate_out) *gate_out = gate_of(*L, q);
}
void orc_attention(void* h, int seq, const float* q, double* o) {
  Layer* L = static_cast<Layer*>(h);
  attention(*L, L->seqs[seq], q, o);
}
double orc_bf16_round(double x) { return bf16_round(x); }

}  // extern "C"
