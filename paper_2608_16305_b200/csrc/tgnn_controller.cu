// Adaptive runtime controller (Eq. 6-9, Algorithm 2): host-side state machine behind the C ABI.
// It holds two exponential moving averages and answers, before each batch, whether a candidate
// cache-refresh boundary should refresh (S_r) and whether the batch runs in heavy-load mode (H_r).
#include <cmath>
#include <new>

#include "../../include/tgnn.h"

struct tgnn_controller {
  double alpha, beta, tau_g, tau_c;
  int K;
  double g_bar, g_last, c_bar, c_prev;
};

namespace {
// Eq. 6 / Eq. 8.  Two roundings (no fused multiply-add) so that the averages are reproducible.
inline double ema(double prev, double x, double f) {
  if (prev == 0.0) return x;
  const double a = f * x;
  const double b = (1.0 - f) * prev;
  return a + b;
}
inline bool bad(double v) { return !(v == v) || std::isinf(v); }
}  // namespace

extern "C" {

int tgnn_controller_create(double alpha, double beta, double tau_g, double tau_c, int K, tgnn_controller** out) {
  if (!out) return TGNN_EINVAL;
  *out = nullptr;
  if (bad(alpha) || bad(beta) || bad(tau_g) || bad(tau_c)) return TGNN_EINVAL;
  if (!(alpha > 0.0 && alpha <= 1.0) || !(beta > 0.0 && beta <= 1.0) || !(tau_g > 0.0) || !(tau_c > 0.0) || K < 1)
    return TGNN_EINVAL;
  tgnn_controller* c = new (std::nothrow) tgnn_controller{alpha, beta, tau_g, tau_c, K, 0.0, 0.0, 0.0, 0.0};
  if (!c) return TGNN_ECAPACITY;  // host allocation failed
  *out = c;
  return TGNN_OK;
}

int tgnn_controller_destroy(tgnn_controller* ctl) {
  delete ctl;
  return TGNN_OK;
}

int tgnn_controller_begin_batch(tgnn_controller* ctl, int64_t r, int* boundary_out, int* sync_out, int* heavy_out) {
  if (!ctl || r < 0 || !boundary_out || !sync_out || !heavy_out) return TGNN_EINVAL;
  const int boundary = (r % ctl->K) == 0 ? 1 : 0;
  *boundary_out = boundary;
  // Eq. 7: skip only when the last norm sits below tau_g times its average
  *sync_out = !boundary ? -1 : ((r > 0 && ctl->g_bar > 0.0 && ctl->g_last < ctl->tau_g * ctl->g_bar) ? 0 : 1);
  // Eq. 9: heavy when the last batch time exceeds tau_c times its average
  *heavy_out = (r > 0 && ctl->c_bar > 0.0 && ctl->c_prev > ctl->tau_c * ctl->c_bar) ? 1 : 0;
  return TGNN_OK;
}

int tgnn_controller_end_batch(tgnn_controller* ctl, double g_r, double c_r) {
  if (!ctl || bad(g_r) || bad(c_r) || g_r < 0.0 || c_r < 0.0) return TGNN_EINVAL;
  ctl->g_bar = ema(ctl->g_bar, g_r, ctl->alpha);
  ctl->g_last = g_r;
  ctl->c_bar = ema(ctl->c_bar, c_r, ctl->beta);
  ctl->c_prev = c_r;
  return TGNN_OK;
}

int tgnn_controller_state(const tgnn_controller* ctl, double* out_host) {
  if (!ctl || !out_host) return TGNN_EINVAL;
  out_host[0] = ctl->g_bar; out_host[1] = ctl->g_last; out_host[2] = ctl->c_bar; out_host[3] = ctl->c_prev;
  return TGNN_OK;
}

}  // extern "C"
