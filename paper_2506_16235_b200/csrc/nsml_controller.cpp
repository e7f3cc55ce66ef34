// Host-side network-sensing controller (Alg. 1, Eq. 1-3).  Pure host code.
// See include/nsml.h for the contract and for the readings taken where the
// paper is silent (start-up increment and exit, estimator windows, which
// data size enters Eq. 3).
#include <cmath>
#include <cstring>
#include <limits>
#include <new>
#include <vector>

#include "nsml.h"

namespace {

constexpr int kMaxWindow = 4096;
constexpr uint32_t kBlobTag = 0x314C5443u;  // "CTL1"

// Running extreme over the last `window` samples (window 0: over all samples).
struct Extreme {
  bool want_max = true;
  int window = 0;
  std::vector<double> ring;  // the last `window` samples, oldest overwritten
  int filled = 0, next = 0;
  double all_time = 0.0;

  void init(bool is_max, int w) {
    want_max = is_max;
    window = w;
    ring.assign(w > 0 ? w : 0, 0.0);
    filled = next = 0;
    all_time = is_max ? 0.0 : std::numeric_limits<double>::infinity();
  }
  double better(double a, double b) const { return want_max ? (a > b ? a : b) : (a < b ? a : b); }
  double push(double x) {
    if (window == 0) {
      all_time = better(all_time, x);
      return all_time;
    }
    ring[next] = x;
    next = (next + 1) % window;
    if (filled < window) ++filled;
    double best = ring[0];
    for (int i = 1; i < filled; ++i) best = better(best, ring[i]);
    return best;
  }
};

}  // namespace

struct nsml_ctrl {
  nsml_ctrl_params p;
  double ratio;
  double ebb, btlbw, rtprop, bdp;
  int phase;  // 0 start-up, 1 NetSense
  int startup_steps;
  int64_t calls;
  Extreme bw, rt;
};

static void fill_defaults(nsml_ctrl_params* p) {
  p->ratio_init = 0.01;
  p->ratio_min = 0.005;
  p->ratio_max = 1.0;
  p->alpha = 0.5;
  p->beta1 = 0.1;
  p->beta2 = 0.01;
  p->bdp_frac = 0.9;
  p->rtt_excess = 1.25;
  p->startup_max_steps = 10;
  p->btlbw_window = 10;
  p->rtprop_window = 100;
  p->reserved = 0;
}

static bool params_ok(const nsml_ctrl_params& p) {
  auto fin = [](double x) { return std::isfinite(x); };
  if (!fin(p.ratio_init) || !fin(p.ratio_min) || !fin(p.ratio_max) || !fin(p.alpha) || !fin(p.beta1) ||
      !fin(p.beta2) || !fin(p.bdp_frac) || !fin(p.rtt_excess))
    return false;
  if (!(p.ratio_min > 0.0 && p.ratio_min <= p.ratio_init && p.ratio_init <= p.ratio_max && p.ratio_max <= 1.0))
    return false;
  if (!(p.alpha > 0.0 && p.alpha < 1.0) || !(p.beta1 > 0.0) || !(p.beta2 > 0.0)) return false;
  if (!(p.bdp_frac > 0.0) || !(p.rtt_excess >= 1.0)) return false;
  if (p.startup_max_steps < 0 || p.btlbw_window < 0 || p.rtprop_window < 0) return false;
  if (p.btlbw_window > kMaxWindow || p.rtprop_window > kMaxWindow) return false;
  return true;
}

static void reset_state(nsml_ctrl* c) {
  c->ratio = c->p.ratio_init;
  c->ebb = 0.0;
  c->btlbw = 0.0;
  c->rtprop = std::numeric_limits<double>::infinity();
  c->bdp = 0.0;
  c->phase = c->p.startup_max_steps > 0 ? 0 : 1;
  c->startup_steps = 0;
  c->calls = 0;
  c->bw.init(true, c->p.btlbw_window);
  c->rt.init(false, c->p.rtprop_window);
}

extern "C" {

int nsml_ctrl_default_params(nsml_ctrl_params* p) {
  if (p == nullptr) return NSML_ERR_ARG;
  fill_defaults(p);
  return NSML_OK;
}

int nsml_ctrl_create(const nsml_ctrl_params* p, nsml_ctrl** out) {
  if (out == nullptr) return NSML_ERR_ARG;
  nsml_ctrl_params q;
  if (p != nullptr) q = *p; else fill_defaults(&q);
  if (!params_ok(q)) return NSML_ERR_ARG;
  nsml_ctrl* c = new (std::nothrow) nsml_ctrl();
  if (c == nullptr) return NSML_ERR_ARG;
  c->p = q;
  reset_state(c);
  *out = c;
  return NSML_OK;
}

void nsml_ctrl_destroy(nsml_ctrl* c) { delete c; }

int nsml_select_ratio(nsml_ctrl* c, double last_bytes, double last_seconds, double next_dense_bytes,
                      double* ratio_out) {
  if (c == nullptr || ratio_out == nullptr) return NSML_ERR_ARG;
  if (!(std::isfinite(next_dense_bytes) && next_dense_bytes >= 0.0)) return NSML_ERR_ARG;
  if (c->calls == 0) {  // nothing was sent yet
    c->calls = 1;
    *ratio_out = c->ratio;
    return NSML_OK;
  }
  if (!(std::isfinite(last_bytes) && last_bytes >= 0.0)) return NSML_ERR_ARG;
  if (!(std::isfinite(last_seconds) && last_seconds > 0.0)) return NSML_ERR_ARG;
  c->calls += 1;

  // Eq. 1, then the BtlBw / RTprop filters, then Eq. 2
  c->ebb = last_bytes / last_seconds;
  c->btlbw = c->bw.push(c->ebb);
  c->rtprop = c->rt.push(last_seconds);
  c->bdp = c->btlbw * c->rtprop;

  if (c->phase == 0) {
    const bool leave = last_seconds > c->p.rtt_excess * c->rtprop || c->startup_steps >= c->p.startup_max_steps ||
                       c->ratio >= c->p.ratio_max;
    if (!leave) {
      c->ratio = std::fmin(c->p.ratio_max, c->ratio + c->p.beta1);
      c->startup_steps += 1;
      *ratio_out = c->ratio;
      return NSML_OK;
    }
    c->phase = 1;
  }
  // Eq. 3
  const double data_size = c->ratio * next_dense_bytes;
  if (data_size > c->p.bdp_frac * c->bdp) c->ratio = std::fmax(c->p.ratio_min, c->ratio * c->p.alpha);
  else c->ratio = std::fmin(c->p.ratio_max, c->ratio + c->p.beta2);
  *ratio_out = c->ratio;
  return NSML_OK;
}

int nsml_ctrl_get_state(const nsml_ctrl* c, nsml_ctrl_state* out) {
  if (c == nullptr || out == nullptr) return NSML_ERR_ARG;
  out->ratio = c->ratio;
  out->ebb = c->ebb;
  out->btlbw = c->btlbw;
  out->rtprop = c->rtprop;
  out->bdp = c->bdp;
  out->phase = c->phase;
  out->startup_steps = c->startup_steps;
  out->calls = c->calls;
  return NSML_OK;
}

// Blob: tag, params, scalar state, then both filters (window counters and ring).
struct BlobHead {
  uint32_t tag, bytes;
  nsml_ctrl_params p;
  double ratio, ebb, btlbw, rtprop, bdp;
  int32_t phase, startup_steps;
  int64_t calls;
  int32_t bw_filled, bw_next, rt_filled, rt_next;
  double bw_all, rt_all;
};

size_t nsml_ctrl_save_bytes(const nsml_ctrl* c) {
  if (c == nullptr) return 0;
  return sizeof(BlobHead) + (c->bw.ring.size() + c->rt.ring.size()) * sizeof(double);
}

int nsml_ctrl_save(const nsml_ctrl* c, void* buf, size_t cap) {
  if (c == nullptr || buf == nullptr) return NSML_ERR_ARG;
  const size_t need = nsml_ctrl_save_bytes(c);
  if (cap < need) return NSML_ERR_CAPACITY;
  BlobHead h;
  std::memset(&h, 0, sizeof(h));
  h.tag = kBlobTag;
  h.bytes = (uint32_t)need;
  h.p = c->p;
  h.ratio = c->ratio; h.ebb = c->ebb; h.btlbw = c->btlbw; h.rtprop = c->rtprop; h.bdp = c->bdp;
  h.phase = c->phase; h.startup_steps = c->startup_steps; h.calls = c->calls;
  h.bw_filled = c->bw.filled; h.bw_next = c->bw.next; h.rt_filled = c->rt.filled; h.rt_next = c->rt.next;
  h.bw_all = c->bw.all_time; h.rt_all = c->rt.all_time;
  unsigned char* out = static_cast<unsigned char*>(buf);
  std::memcpy(out, &h, sizeof(h));
  out += sizeof(h);
  if (!c->bw.ring.empty()) std::memcpy(out, c->bw.ring.data(), c->bw.ring.size() * sizeof(double));
  out += c->bw.ring.size() * sizeof(double);
  if (!c->rt.ring.empty()) std::memcpy(out, c->rt.ring.data(), c->rt.ring.size() * sizeof(double));
  return NSML_OK;
}

int nsml_ctrl_load(nsml_ctrl* c, const void* buf, size_t bytes) {
  if (c == nullptr || buf == nullptr || bytes < sizeof(BlobHead)) return NSML_ERR_ARG;
  BlobHead h;
  std::memcpy(&h, buf, sizeof(h));
  if (h.tag != kBlobTag || h.bytes != bytes || !params_ok(h.p)) return NSML_ERR_ARG;
  const size_t rings = (size_t)h.p.btlbw_window + (size_t)h.p.rtprop_window;
  if (bytes != sizeof(BlobHead) + rings * sizeof(double)) return NSML_ERR_ARG;
  if (h.bw_filled < 0 || h.bw_filled > h.p.btlbw_window || h.rt_filled < 0 || h.rt_filled > h.p.rtprop_window)
    return NSML_ERR_ARG;
  if (h.bw_next < 0 || (h.p.btlbw_window > 0 && h.bw_next >= h.p.btlbw_window) || h.rt_next < 0 ||
      (h.p.rtprop_window > 0 && h.rt_next >= h.p.rtprop_window))
    return NSML_ERR_ARG;
  if (h.phase != 0 && h.phase != 1) return NSML_ERR_ARG;
  c->p = h.p;
  reset_state(c);
  c->ratio = h.ratio; c->ebb = h.ebb; c->btlbw = h.btlbw; c->rtprop = h.rtprop; c->bdp = h.bdp;
  c->phase = h.phase; c->startup_steps = h.startup_steps; c->calls = h.calls;
  c->bw.filled = h.bw_filled; c->bw.next = h.bw_next; c->bw.all_time = h.bw_all;
  c->rt.filled = h.rt_filled; c->rt.next = h.rt_next; c->rt.all_time = h.rt_all;
  const unsigned char* in = static_cast<const unsigned char*>(buf) + sizeof(BlobHead);
  if (!c->bw.ring.empty()) std::memcpy(c->bw.ring.data(), in, c->bw.ring.size() * sizeof(double));
  in += c->bw.ring.size() * sizeof(double);
  if (!c->rt.ring.empty()) std::memcpy(c->rt.ring.data(), in, c->rt.ring.size() * sizeof(double));
  return NSML_OK;
}

}  // extern "C"
