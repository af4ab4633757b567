// Greedy search and coordinate descent over per-layer bit-widths (Section 2.2), as host loops
// over the scheme evaluator and the analytic arithmetic intensity.
//
//   L(q; lambda) = -lambda * AI(q) + (1 - lambda) * AccLoss(q)                  (Section 2.1)
//
// The paper states neither the units of AccLoss nor a normalisation of AI.  Used here:
// AccLoss(q) = 100 * (acc(q_FP32) - acc(q)) in percentage points, with acc measured on the
// caller's image set (aiq_eval_schemes), and AI in FLOP per byte (aiq_scheme_ai, batch 1).
// Every candidate move of an iteration is scored by ONE aiq_eval_schemes call, so the
// candidates share the activations of their common prefix.  All arithmetic on the loss is
// host double precision on integer counts; the kernels are those of the evaluator.
#include "common.cuh"

#include <vector>

namespace aiq {
namespace {

double loss_of(double ai, double acc, double acc_fp, double lambda) {
  return -lambda * ai + (1.0 - lambda) * 100.0 * (acc_fp - acc);
}

struct SearchCtx {
  const aiq_model_t* model;
  const float* x;
  const int32_t* labels;
  int n_images;
  void* ws;
  size_t ws_bytes;
  void* stream;
  int L;
  std::vector<float> acc;
  std::vector<int32_t> counts;

  // accuracies (as doubles from the integer counts) of `n` schemes stored row-major in `schemes`
  aiq_status_t eval(const std::vector<uint8_t>& schemes, int n, std::vector<double>& out) {
    acc.resize(n);
    counts.resize(n);
    aiq_status_t st = aiq_eval_schemes(model, schemes.data(), n, x, labels, n_images, acc.data(), counts.data(),
                                       nullptr, ws, ws_bytes, stream);
    if (st != AIQ_OK) return st;
    out.resize(n);
    for (int i = 0; i < n; ++i) out[i] = (double)counts[i] / (double)n_images;
    return AIQ_OK;
  }
  aiq_status_t ai(const uint8_t* scheme, double& out) { return aiq_scheme_ai(model, scheme, 1, &out, nullptr, nullptr); }
};

aiq_status_t check_args(const aiq_model_t* model, const int32_t* layers, int n_layers, const uint8_t* options,
                        int n_options, double lambda, const float* x, const int32_t* labels, int n_images,
                        uint8_t* scheme_out, void* ws, const char* who) {
  if (!model || !options || !x || !labels || !scheme_out || !ws)
    return set_error(AIQ_ERR_INVALID_ARG, "%s: null pointer", who);
  const int L = aiq_model_num_layers(model);
  if (n_images <= 0 || n_options <= 0 || n_options > 4 || n_layers < 0 || n_layers > L)
    return set_error(AIQ_ERR_INVALID_ARG, "%s: n_images=%d n_options=%d n_layers=%d", who, n_images, n_options, n_layers);
  if (!(lambda >= 0.0 && lambda <= 1.0)) return set_error(AIQ_ERR_INVALID_ARG, "%s: lambda must lie in [0, 1]", who);
  for (int i = 0; i < n_options; ++i)
    if (!bits_ok(options[i])) return set_error(AIQ_ERR_UNSUPPORTED_BITS, "%s: option %d", who, (int)options[i]);
  if (layers)
    for (int i = 0; i < n_layers; ++i)
      if (layers[i] < 0 || layers[i] >= L) return set_error(AIQ_ERR_INVALID_ARG, "%s: layer index %d", who, layers[i]);
  return AIQ_OK;
}

}  // namespace
}  // namespace aiq

extern "C" aiq_status_t aiq_search_greedy(const aiq_model_t* model, const int32_t* layers, int n_layers,
                                          const uint8_t* options, int n_options, double lambda, const float* x,
                                          const int32_t* labels, int n_images, uint8_t* scheme_out,
                                          aiq_search_step_t* trace, int trace_capacity, int* n_trace,
                                          void* workspace, size_t workspace_bytes, void* stream) {
  using namespace aiq;
  aiq_status_t st = check_args(model, layers, n_layers, options, n_options, lambda, x, labels, n_images, scheme_out,
                               workspace, "aiq_search_greedy");
  if (st != AIQ_OK) return st;
  SearchCtx cx{model, x, labels, n_images, workspace, workspace_bytes, stream, aiq_model_num_layers(model)};
  const int L = cx.L;
  std::vector<int> sel;
  if (layers) sel.assign(layers, layers + n_layers);
  else for (int i = 0; i < L; ++i) sel.push_back(i);
  std::vector<uint8_t> q(L, 32), cands;
  std::vector<double> accs;
  cands = q;
  if ((st = cx.eval(cands, 1, accs)) != AIQ_OK) return st;
  const double acc_fp = accs[0];
  double ai = 0.0;
  if ((st = cx.ai(q.data(), ai)) != AIQ_OK) return st;
  double cur = loss_of(ai, acc_fp, acc_fp, lambda), cur_acc = acc_fp;
  int nt = 0;
  for (size_t it = 0; it < sel.size(); ++it) {
    // candidate moves: every still unquantized selectable layer to every lower option
    std::vector<std::pair<int, int>> moves;
    for (int i : sel)
      if (q[i] == 32)
        for (int o = 0; o < n_options; ++o)
          if (options[o] < 32) moves.push_back({i, (int)options[o]});
    if (moves.empty()) break;
    const int n = (int)moves.size();
    cands.resize((size_t)n * L);
    for (int r = 0; r < n; ++r) {
      std::copy(q.begin(), q.end(), cands.begin() + (size_t)r * L);
      cands[(size_t)r * L + moves[r].first] = (uint8_t)moves[r].second;
    }
    if ((st = cx.eval(cands, n, accs)) != AIQ_OK) return st;
    int best = -1;
    double best_delta = 0.0, best_ai = 0.0;
    for (int r = 0; r < n; ++r) {
      if ((st = cx.ai(&cands[(size_t)r * L], ai)) != AIQ_OK) return st;
      const double delta = loss_of(ai, accs[r], acc_fp, lambda) - cur;
      if (best < 0 || delta < best_delta) { best = r; best_delta = delta; best_ai = ai; }
    }
    const bool accepted = best_delta < 0.0;
    if (accepted) {
      std::copy(cands.begin() + (size_t)best * L, cands.begin() + (size_t)(best + 1) * L, q.begin());
      cur += best_delta;
      cur_acc = accs[best];
    }
    if (trace && nt < trace_capacity) {
      aiq_search_step_t& t = trace[nt];
      t.layer = moves[best].first; t.bits = moves[best].second; t.accepted = accepted ? 1 : 0;
      t.candidates = n; t.loss = cur; t.acc = accepted ? cur_acc : accs[best]; t.ai = best_ai;
    }
    ++nt;
    if (!accepted) break;                      // the scheme, hence the candidate set, can no longer change
  }
  std::copy(q.begin(), q.end(), scheme_out);
  if (n_trace) *n_trace = nt;
  return AIQ_OK;
}

extern "C" aiq_status_t aiq_search_coordinate_descent(const aiq_model_t* model, const int32_t* layers, int n_layers,
                                                      const uint8_t* options, int n_options, double lambda,
                                                      int max_passes, const float* x, const int32_t* labels,
                                                      int n_images, uint8_t* scheme_out, aiq_search_step_t* trace,
                                                      int trace_capacity, int* n_trace, void* workspace,
                                                      size_t workspace_bytes, void* stream) {
  using namespace aiq;
  aiq_status_t st = check_args(model, layers, n_layers, options, n_options, lambda, x, labels, n_images, scheme_out,
                               workspace, "aiq_search_coordinate_descent");
  if (st != AIQ_OK) return st;
  if (max_passes <= 0) return set_error(AIQ_ERR_INVALID_ARG, "aiq_search_coordinate_descent: max_passes=%d", max_passes);
  SearchCtx cx{model, x, labels, n_images, workspace, workspace_bytes, stream, aiq_model_num_layers(model)};
  const int L = cx.L;
  std::vector<int> sel;
  if (layers) sel.assign(layers, layers + n_layers);
  else for (int i = 0; i < L; ++i) sel.push_back(i);
  std::vector<uint8_t> q(L, 32), cands;
  std::vector<double> accs;
  cands = q;
  if ((st = cx.eval(cands, 1, accs)) != AIQ_OK) return st;
  const double acc_fp = accs[0];
  double ai = 0.0;
  if ((st = cx.ai(q.data(), ai)) != AIQ_OK) return st;
  double cur = loss_of(ai, acc_fp, acc_fp, lambda), cur_acc = acc_fp, cur_ai = ai;
  int nt = 0;
  for (int pass = 0; pass < max_passes; ++pass) {
    bool changed_any = false;
    for (int i : sel) {
      std::vector<int> alts;
      for (int o = 0; o < n_options; ++o)
        if (options[o] != q[i]) alts.push_back(options[o]);
      const int n = (int)alts.size();
      if (n == 0) continue;
      cands.resize((size_t)n * L);
      for (int r = 0; r < n; ++r) {
        std::copy(q.begin(), q.end(), cands.begin() + (size_t)r * L);
        cands[(size_t)r * L + i] = (uint8_t)alts[r];
      }
      if ((st = cx.eval(cands, n, accs)) != AIQ_OK) return st;
      int best = -1;
      double best_loss = cur, best_ai = cur_ai;
      for (int r = 0; r < n; ++r) {
        if ((st = cx.ai(&cands[(size_t)r * L], ai)) != AIQ_OK) return st;
        const double loss = loss_of(ai, accs[r], acc_fp, lambda);
        if (loss < best_loss) { best = r; best_loss = loss; best_ai = ai; }
      }
      if (best >= 0) {
        q[i] = (uint8_t)alts[best];
        cur = best_loss; cur_acc = accs[best]; cur_ai = best_ai;
        changed_any = true;
      }
      if (trace && nt < trace_capacity) {
        aiq_search_step_t& t = trace[nt];
        t.layer = i; t.bits = q[i]; t.accepted = best >= 0 ? 1 : 0; t.candidates = n;
        t.loss = cur; t.acc = cur_acc; t.ai = cur_ai;
      }
      ++nt;
    }
    if (!changed_any) break;
  }
  std::copy(q.begin(), q.end(), scheme_out);
  if (n_trace) *n_trace = nt;
  return AIQ_OK;
}
