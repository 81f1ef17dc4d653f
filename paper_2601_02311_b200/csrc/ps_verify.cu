// Batched brute-force verifier: the paper's verification protocol (Section 7.1)
// as a data-parallel workload.  One thread runs one case: a tiny layered network
// trained with Adam in fp64 on D logical devices that hold every state exactly
// as its placement mode says (Definition 1), with explicit ring collectives that
// count the bytes each device sends (Section 2.3), next to the single-device run
// on the global batch (Definition 4's yardstick).  Whatever a placement leaves
// unavailable when it is needed reads as zeros, so a placement that breaks
// gradient integrity (Theorem 3) or state consistency (Theorem 4) really leaves
// the single-device trajectory (Theorem 5).  Per case the kernel reports whether
// every step's reassembled Theta and Omega equal the single-device run, and the
// bytes held, sent and moved over the host link in the last step.
//
// The kernel knows none of the closed-form rules; it executes the mechanism:
//   (1) make Theta available, forward      (2) keep, shard, offload or drop A
//   (3) make Theta available, backward     (4) synchronise and deliver G
//   (5) update on the range this device commits (all of it if Omega is
//       replicated, its shard if Omega's home is a shard)
//   (6) put Theta back into its home.
//
// Layout.  A case's arrays live in a workspace that is interleaved over the
// cases (element k of case c at ws[k * n_cases + c]): threads of a warp that
// execute the same statement touch consecutive addresses.
#include "ps_device.cuh"
#include "ps_internal.h"

namespace {

constexpr int MAX_D = 4;
enum { ST_THETA = 0, ST_OMEGA = 1, ST_GRAD = 2, ST_ACT = 3 };

struct Dims {
  int units, h, b, D, P, EA, accum, steps, nbuf;
  int wT, wO, wG;
  double lr, beta1, beta2, eps, rtol, atol;
};

// the interleaved workspace of one case
struct Work {
  double* base;
  size_t stride;
  __device__ __forceinline__ double& operator()(size_t k) const { return base[k * stride]; }
};

// offsets (in doubles) of a case's arrays
struct Layout {
  size_t th_home, om_home, th_use, local, grad, newth, acts, kept, ring, ref_th, ref_om, ref_g, ref_act, total;
};
__host__ __device__ inline Layout make_layout(int D, int P, int EA, int units, int h) {
  Layout l;
  size_t o = 0;
  l.th_home = o; o += (size_t)D * P;        // Theta at home (device or host arena), at global positions
  l.om_home = o; o += (size_t)D * 3 * P;    // Omega at home: master, first and second moment
  l.th_use = o; o += (size_t)D * P;         // Theta as forward / backward see it
  l.local = o; o += (size_t)D * P;          // un-reduced local gradients (not a placed state)
  l.grad = o; o += (size_t)D * P;           // gradients as the update reads them
  l.newth = o; o += (size_t)D * P;          // updated parameters on the committed range
  l.acts = o; o += (size_t)D * EA;          // activations written by forward
  l.kept = o; o += (size_t)D * EA;          // activations as backward reads them
  l.ring = o; o += (size_t)D * P;           // travelling partial sums of a reduce-scatter
  l.ref_th = o; o += (size_t)P;             // the single-device run
  l.ref_om = o; o += (size_t)3 * P;
  l.ref_g = o; o += (size_t)P;
  l.ref_act = o; o += (size_t)units * h;    // one sample's activations
  l.total = o;
  return l;
}

struct Books {
  long long persist[4][MAX_D];   // per state and device: high-water bytes held
  long long transient[4];        // per state: the unit buffer
  long long comm;                // sum over collectives of the busiest device's bytes
  long long host[MAX_D];         // bytes over each device's host link
  __device__ void clear() {
    for (int s = 0; s < 4; ++s) { transient[s] = 0; for (int i = 0; i < MAX_D; ++i) persist[s][i] = 0; }
    comm = 0;
    for (int i = 0; i < MAX_D; ++i) host[i] = 0;
  }
  __device__ void hold(int st, int dev, long long n) { if (n > persist[st][dev]) persist[st][dev] = n; }
  __device__ void unit_buffer(int st, long long n) { if (n > transient[st]) transient[st] = n; }
  __device__ void phase(const long long* sent, int D) {
    long long m = 0;
    for (int i = 0; i < D; ++i) if (sent[i] > m) m = sent[i];
    comm += m;
  }
  __device__ long long memory(int D) const {
    long long total = 0;
    for (int s = 0; s < 4; ++s) {
      long long m = 0;
      for (int i = 0; i < D; ++i) if (persist[s][i] > m) m = persist[s][i];
      total += m + transient[s];
    }
    return total;
  }
  __device__ long long host_bytes(int D) const {
    long long m = 0;
    for (int i = 0; i < D; ++i) if (host[i] > m) m = host[i];
    return m;
  }
};

// eq. (2): shard i of E elements over D devices is [floor(i E / D), floor((i+1) E / D))
__device__ __forceinline__ int cut_of(int E, int D, int i) { return (int)(((long long)i * E) / D); }

// A ring all-gather of pieces of the given lengths (Section 2.3): in step s device i
// passes on the piece that started at device (i - s) mod D.  Counts what each device sends.
__device__ void ring_gather_count(const int* len, int D, int width, long long* sent) {
  for (int s = 0; s + 1 < D; ++s)
    for (int i = 0; i < D; ++i) sent[i] += (long long)len[((i - s) % D + D) % D] * width;
}

// A ring reduce-scatter of each device's vector v_i[lo, hi) cut at c[0..D]: in step s
// device i adds its part to the travelling partial sum of chunk (i - 1 - s) mod D and
// passes it on; device i ends with the sum of chunk i in ring(i)[c[i], c[i+1]).
// ring(i) starts as a copy of v_i.  Sums in ring order, as a real ring does.
template <typename RingAt>
__device__ void ring_reduce_scatter(RingAt ring, const int* c, int D, int width, long long* sent) {
  for (int s = 0; s + 1 < D; ++s) {
    for (int i = 0; i < D; ++i) {
      const int ch = ((i - 1 - s) % D + D) % D;
      const int to = (i + 1) % D;
      sent[i] += (long long)(c[ch + 1] - c[ch]) * width;
      for (int e = c[ch]; e < c[ch + 1]; ++e) ring(to, e) = ring(to, e) + ring(i, e);
    }
  }
}

__global__ void __launch_bounds__(128) k_verify(Dims dm, const ps_verify_case* __restrict__ cases, u64 n_cases,
                                                 const double* __restrict__ data, u64 data_len, double* ws,
                                                 double* theta_out, ps_verify_result* __restrict__ out, u32* status) {
  const u64 idx = (u64)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n_cases) return;
  const ps_verify_case cs = cases[idx];
  const int P = dm.P, h = dm.h, b = dm.b, units = dm.units, EA = dm.EA;
  {
    // a case that names more devices than supported, no placement, or data outside the
    // given array is reported, not run
    const u64 need = (u64)P + 2ull * dm.accum * cs.D * b * h;
    if (cs.D < 1 || cs.D > MAX_D || cs.code > 624 || cs.data_offset > data_len || need > data_len - cs.data_offset) {
      ps_verify_result r;
      r.mem = 0; r.comm = 0; r.host = 0; r.match = 0; r.pad = 0; r.max_rel_err = 0.0;
      out[idx] = r;
      if (theta_out) for (int e = 0; e < P; ++e) theta_out[idx * (u64)P + e] = 0.0;
      atomicOr(status, ST_BAD_CASE);
      return;
    }
  }
  const int D = (int)cs.D;
  const int pT = cs.code % 5, pO = (cs.code / 5) % 5, pG = (cs.code / 25) % 5, pA = (cs.code / 125) % 5;
  const Layout L = make_layout(MAX_D, P, EA, units, h);
  const Work W{ws + idx, (size_t)n_cases};
  const double* prob = data + cs.data_offset;
  // problem data: theta0[P], xs[accum][D][b][h], ys[accum][D][b][h]
  const double* theta0 = prob;
  const double* xs = prob + P;
  const double* ys = xs + (size_t)dm.accum * D * b * h;
  auto sample = [&](const double* base, int j, int i, int s) { return base + (((size_t)j * D + i) * b + s) * h; };

  int cut[MAX_D + 1], cutA[MAX_D + 1];
  for (int i = 0; i <= D; ++i) { cut[i] = cut_of(P, D, i); cutA[i] = cut_of(EA, D, i); }
  const bool on_shard = (pO == PS_MODE_S || pO == PS_MODE_SG || pO == PS_MODE_O);
  const int nbuf = dm.nbuf < units ? dm.nbuf : units;     // a second unit buffer needs a second unit

  auto th_home = [&](int i, int e) -> double& { return W(L.th_home + (size_t)i * P + e); };
  auto om_home = [&](int i, int row, int e) -> double& { return W(L.om_home + ((size_t)i * 3 + row) * P + e); };
  auto th_use = [&](int i, int e) -> double& { return W(L.th_use + (size_t)i * P + e); };
  auto local = [&](int i, int e) -> double& { return W(L.local + (size_t)i * P + e); };
  auto grad = [&](int i, int e) -> double& { return W(L.grad + (size_t)i * P + e); };
  auto newth = [&](int i, int e) -> double& { return W(L.newth + (size_t)i * P + e); };
  auto acts = [&](int i, int e) -> double& { return W(L.acts + (size_t)i * EA + e); };      // e = (l * b + s) * h + j
  auto kept = [&](int i, int e) -> double& { return W(L.kept + (size_t)i * EA + e); };
  auto ring = [&](int i, int e) -> double& { return W(L.ring + (size_t)i * P + e); };

  // ---- homes (Definition 1): what each device holds of Theta and Omega
  for (int i = 0; i < D; ++i)
    for (int e = 0; e < P; ++e) {
      const bool mine = e >= cut[i] && e < cut[i + 1];
      const bool th_here = pT == PS_MODE_R || ((pT == PS_MODE_S || pT == PS_MODE_SG || pT == PS_MODE_O) && mine);
      th_home(i, e) = th_here ? theta0[e] : 0.0;
      const bool om_here = pO == PS_MODE_R || ((pO == PS_MODE_S || pO == PS_MODE_SG || pO == PS_MODE_O) && mine);
      om_home(i, 0, e) = om_here ? theta0[e] : 0.0;     // the master copy lives inside Omega
      om_home(i, 1, e) = 0.0;
      om_home(i, 2, e) = 0.0;
    }
  // ---- the single-device run starts from the same point
  for (int e = 0; e < P; ++e) {
    W(L.ref_th + e) = theta0[e];
    W(L.ref_om + e) = theta0[e];
    W(L.ref_om + P + e) = 0.0;
    W(L.ref_om + 2 * P + e) = 0.0;
  }

  auto adam_elem = [&](double& master, double& m, double& v, double g, int t) {
    m = dm.beta1 * m + (1.0 - dm.beta1) * g;
    v = dm.beta2 * v + (1.0 - dm.beta2) * g * g;
    const double mh = m / (1.0 - pow(dm.beta1, (double)t));
    const double vh = v / (1.0 - pow(dm.beta2, (double)t));
    master = master - dm.lr * mh / (sqrt(vh) + dm.eps);
  };

  Books books;
  books.clear();
  bool match = true;
  double worst = 0.0;

  // Theta as forward / backward see it on every device (steps (1) and (3))
  auto theta_for_compute = [&]() {
    if (pT == PS_MODE_R) {
      for (int i = 0; i < D; ++i) {
        books.hold(ST_THETA, i, (long long)P * dm.wT);
        for (int e = 0; e < P; ++e) th_use(i, e) = th_home(i, e);
      }
    } else if (pT == PS_MODE_S) {
      for (int i = 0; i < D; ++i) {
        books.hold(ST_THETA, i, (long long)(cut[i + 1] - cut[i]) * dm.wT);
        for (int e = 0; e < P; ++e) th_use(i, e) = (e >= cut[i] && e < cut[i + 1]) ? th_home(i, e) : 0.0;
      }
    } else if (pT == PS_MODE_SG || pT == PS_MODE_O) {
      for (int i = 0; i < D; ++i) {
        const long long shard = (long long)(cut[i + 1] - cut[i]) * dm.wT;
        if (pT == PS_MODE_SG) books.hold(ST_THETA, i, shard);
        else books.host[i] += shard;                              // host -> device
      }
      // gathered one reconstruction unit (layer) at a time into a unit buffer
      long long sent[MAX_D] = {0, 0, 0, 0};
      for (int l = 0; l < units; ++l) {
        const int a = l * h, z = (l + 1) * h;
        int len[MAX_D];
        for (int i = 0; i < D; ++i) {
          const int s0 = max(a, cut[i]), s1 = min(z, cut[i + 1]);
          len[i] = s1 > s0 ? s1 - s0 : 0;
        }
        ring_gather_count(len, D, dm.wT, sent);
        if (pT == PS_MODE_SG) books.unit_buffer(ST_THETA, (long long)nbuf * h * dm.wT);
        for (int e = a; e < z; ++e) {
          int owner = 0;
          while (!(e >= cut[owner] && e < cut[owner + 1])) ++owner;
          const double v = th_home(owner, e);
          for (int i = 0; i < D; ++i) th_use(i, e) = v;
        }
      }
      books.phase(sent, D);
    } else {  // M: cast from the master copy, where Omega is resident on the device
      for (int i = 0; i < D; ++i) {
        for (int e = 0; e < P; ++e) {
          double v = 0.0;
          if (pO == PS_MODE_R) v = om_home(i, 0, e);
          else if ((pO == PS_MODE_S || pO == PS_MODE_SG) && e >= cut[i] && e < cut[i + 1]) v = om_home(i, 0, e);
          th_use(i, e) = v;
        }
        books.unit_buffer(ST_THETA, (long long)h * dm.wT);
      }
    }
  };

  // forward of device i on micro-batch j with the parameters it sees; stores every layer's input
  auto forward = [&](int i, int j, bool into_kept) {
    for (int s = 0; s < b; ++s) {
      const double* x = sample(xs, j, i, s);
      for (int jj = 0; jj < h; ++jj) {
        double cur = x[jj];
        for (int l = 0; l < units; ++l) {
          const int e = (l * b + s) * h + jj;
          if (into_kept) kept(i, e) = cur; else acts(i, e) = cur;
          cur = tanh(th_use(i, l * h + jj) * cur);
        }
      }
    }
  };
  // mean-over-samples gradient of 0.5 ||out - y||^2 from the given parameters and kept activations,
  // added to the local sum with weight 1 / accum
  auto backward = [&](int i, int j) {
    for (int jj = 0; jj < h; ++jj) {
      double g[8];
      for (int l = 0; l < units; ++l) g[l] = 0.0;
      for (int s = 0; s < b; ++s) {
        const double* y = sample(ys, j, i, s);
        const int top = ((units - 1) * b + s) * h + jj;
        const double last = tanh(th_use(i, (units - 1) * h + jj) * kept(i, top));
        double dh = (last - y[jj]) / b;
        for (int l = units - 1; l >= 0; --l) {
          const double th = th_use(i, l * h + jj);
          const double a = kept(i, (l * b + s) * h + jj);
          const double o = tanh(th * a);
          const double dz = dh * (1.0 - o * o);
          g[l] += dz * a;
          dh = dz * th;
        }
      }
      for (int l = 0; l < units; ++l) local(i, l * h + jj) += g[l] / dm.accum;
    }
  };

  for (int t = 1; t <= dm.steps; ++t) {
    books.clear();
    for (int i = 0; i < D; ++i)
      for (int e = 0; e < P; ++e) local(i, e) = 0.0;
    for (int j = 0; j < dm.accum; ++j) {
      // (1) forward
      theta_for_compute();
      for (int i = 0; i < D; ++i) forward(i, j, false);
      // (2) activations between forward and backward
      if (pA == PS_MODE_R || pA == PS_MODE_O) {
        for (int i = 0; i < D; ++i) {
          if (pA == PS_MODE_R) books.hold(ST_ACT, i, EA);
          else books.host[i] += 2LL * EA;                          // device -> host, host -> device
          for (int e = 0; e < EA; ++e) kept(i, e) = acts(i, e);
        }
      } else if (pA == PS_MODE_S || pA == PS_MODE_SG) {
        for (int i = 0; i < D; ++i) books.hold(ST_ACT, i, cutA[i + 1] - cutA[i]);
        if (pA == PS_MODE_S) {
          for (int i = 0; i < D; ++i)
            for (int e = 0; e < EA; ++e) kept(i, e) = (e >= cutA[i] && e < cutA[i + 1]) ? acts(i, e) : 0.0;
        } else {
          // gathered from the peers, whose slices belong to other samples
          books.unit_buffer(ST_ACT, (long long)nbuf * b * h);
          for (int e = 0; e < EA; ++e) {
            int owner = 0;
            while (!(e >= cutA[owner] && e < cutA[owner + 1])) ++owner;
            const double v = acts(owner, e);
            for (int i = 0; i < D; ++i) kept(i, e) = v;
          }
        }
      }
      // (3) Theta again for backward
      theta_for_compute();
      if (pA == PS_MODE_M) {
        books.unit_buffer(ST_ACT, (long long)b * h);
        for (int i = 0; i < D; ++i) forward(i, j, true);           // recomputed
      }
      for (int i = 0; i < D; ++i) backward(i, j);
    }

    // (4) synchronise / deliver gradients (mean over the D replicas)
    for (int i = 0; i < D; ++i)
      for (int e = 0; e < P; ++e) { grad(i, e) = 0.0; ring(i, e) = local(i, e); }
    if (pG == PS_MODE_R || pG == PS_MODE_S || pG == PS_MODE_O || pG == PS_MODE_SG) {
      long long sent[MAX_D] = {0, 0, 0, 0};
      ring_reduce_scatter(ring, cut, D, dm.wG, sent);
      books.phase(sent, D);
      if (pG == PS_MODE_R) {
        int len[MAX_D];
        for (int i = 0; i < D; ++i) len[i] = cut[i + 1] - cut[i];
        long long sent2[MAX_D] = {0, 0, 0, 0};
        ring_gather_count(len, D, dm.wG, sent2);
        books.phase(sent2, D);
        for (int i = 0; i < D; ++i) {
          books.hold(ST_GRAD, i, (long long)P * dm.wG);
          for (int c = 0; c < D; ++c)
            for (int e = cut[c]; e < cut[c + 1]; ++e) grad(i, e) = ring(c, e) / D;
        }
      } else if (pG == PS_MODE_S || pG == PS_MODE_O) {
        for (int i = 0; i < D; ++i) {
          const long long n = cut[i + 1] - cut[i];
          if (pG == PS_MODE_S) books.hold(ST_GRAD, i, n * dm.wG);
          else books.host[i] += 2 * n * dm.wG;                     // offload, reload at the update
          for (int e = cut[i]; e < cut[i + 1]; ++e) grad(i, e) = ring(i, e) / D;
        }
      } else {  // S*: reduce-scatter, then gathered unit by unit before use
        for (int i = 0; i < D; ++i) books.hold(ST_GRAD, i, (long long)(cut[i + 1] - cut[i]) * dm.wG);
        long long sent2[MAX_D] = {0, 0, 0, 0};
        for (int l = 0; l < units; ++l) {
          const int a = l * h, z = (l + 1) * h;
          int len[MAX_D];
          for (int i = 0; i < D; ++i) {
            const int s0 = max(a, cut[i]), s1 = min(z, cut[i + 1]);
            len[i] = s1 > s0 ? s1 - s0 : 0;
          }
          ring_gather_count(len, D, dm.wG, sent2);
          books.unit_buffer(ST_GRAD, (long long)nbuf * h * dm.wG);
        }
        books.phase(sent2, D);
        for (int i = 0; i < D; ++i)
          for (int c = 0; c < D; ++c)
            for (int e = cut[c]; e < cut[c + 1]; ++e) grad(i, e) = ring(c, e) / D;
      }
    } else {  // M: reduced unit by unit as produced, consumed at once
      long long sent_rs[MAX_D] = {0, 0, 0, 0}, sent_ag[MAX_D] = {0, 0, 0, 0};
      for (int l = 0; l < units; ++l) {
        const int a = l * h, z = (l + 1) * h;
        int ucut[MAX_D + 1];
        for (int i = 0; i <= D; ++i) ucut[i] = min(max(cut[i], a), z);
        ring_reduce_scatter(ring, ucut, D, dm.wG, sent_rs);
        books.unit_buffer(ST_GRAD, (long long)h * dm.wG);
        if (on_shard) {
          for (int i = 0; i < D; ++i)
            for (int e = ucut[i]; e < ucut[i + 1]; ++e) grad(i, e) = ring(i, e) / D;
        } else {
          int len[MAX_D];
          for (int i = 0; i < D; ++i) len[i] = ucut[i + 1] - ucut[i];
          ring_gather_count(len, D, dm.wG, sent_ag);
          for (int i = 0; i < D; ++i)
            for (int c = 0; c < D; ++c)
              for (int e = ucut[c]; e < ucut[c + 1]; ++e) grad(i, e) = ring(c, e) / D;
        }
      }
      books.phase(sent_rs, D);
      if (!on_shard) books.phase(sent_ag, D);
    }

    // (5) update on the range whose update this device commits
    for (int i = 0; i < D; ++i)
      for (int e = 0; e < P; ++e) newth(i, e) = 0.0;
    if (pO == PS_MODE_SG) {
      // gather all of Omega unit by unit (three rows of w_O / 3 bytes), use it, keep the own shard's update
      long long sent[MAX_D] = {0, 0, 0, 0};
      for (int l = 0; l < units; ++l) {
        const int a = l * h, z = (l + 1) * h;
        int len[MAX_D];
        for (int i = 0; i < D; ++i) {
          const int s0 = max(a, cut[i]), s1 = min(z, cut[i + 1]);
          len[i] = s1 > s0 ? s1 - s0 : 0;
        }
        for (int row = 0; row < 3; ++row) ring_gather_count(len, D, dm.wO / 3, sent);
        books.unit_buffer(ST_OMEGA, (long long)nbuf * h * dm.wO);
      }
      books.phase(sent, D);
    }
    for (int i = 0; i < D; ++i) {
      const int lo = cut[i], hi = cut[i + 1];
      if (pO == PS_MODE_R) {
        books.hold(ST_OMEGA, i, (long long)P * dm.wO);
        for (int e = 0; e < P; ++e) {
          adam_elem(om_home(i, 0, e), om_home(i, 1, e), om_home(i, 2, e), grad(i, e), t);
          newth(i, e) = om_home(i, 0, e);
        }
      } else if (pO == PS_MODE_S || pO == PS_MODE_SG || pO == PS_MODE_O) {
        if (pO == PS_MODE_O) books.host[i] += 2LL * (hi - lo) * dm.wO;        // load, store
        else books.hold(ST_OMEGA, i, (long long)(hi - lo) * dm.wO);
        for (int e = lo; e < hi; ++e) {
          adam_elem(om_home(i, 0, e), om_home(i, 1, e), om_home(i, 2, e), grad(i, e), t);
          newth(i, e) = om_home(i, 0, e);
        }
      } else {  // M: nothing was kept, the update starts from nothing
        for (int e = 0; e < P; ++e) {
          double master = 0.0, m = 0.0, v = 0.0;
          adam_elem(master, m, v, grad(i, e), t);
          newth(i, e) = master;
        }
      }
    }

    // (6) Theta back to its home
    if (pT == PS_MODE_R) {
      if (on_shard) {
        int len[MAX_D];
        for (int i = 0; i < D; ++i) len[i] = cut[i + 1] - cut[i];
        long long sent[MAX_D] = {0, 0, 0, 0};
        ring_gather_count(len, D, dm.wT, sent);                    // re-replicate the updated shards
        books.phase(sent, D);
        for (int i = 0; i < D; ++i)
          for (int c = 0; c < D; ++c)
            for (int e = cut[c]; e < cut[c + 1]; ++e) th_home(i, e) = newth(c, e);
      } else {
        for (int i = 0; i < D; ++i)
          for (int e = 0; e < P; ++e) th_home(i, e) = newth(i, e);
      }
    } else if (pT == PS_MODE_S || pT == PS_MODE_SG || pT == PS_MODE_O) {
      for (int i = 0; i < D; ++i) {
        if (pT == PS_MODE_O) books.host[i] += (long long)(cut[i + 1] - cut[i]) * dm.wT;   // device -> host
        for (int e = cut[i]; e < cut[i + 1]; ++e) th_home(i, e) = newth(i, e);
      }
    }

    // ---- the single-device step on the global batch
    {
      const int n_all = dm.accum * D * b;
      for (int e = 0; e < P; ++e) W(L.ref_g + e) = 0.0;
      for (int j = 0; j < dm.accum; ++j)
        for (int i = 0; i < D; ++i)
          for (int s = 0; s < b; ++s) {
            const double* x = sample(xs, j, i, s);
            const double* y = sample(ys, j, i, s);
            for (int jj = 0; jj < h; ++jj) {
              double cur = x[jj];
              for (int l = 0; l < units; ++l) {
                W(L.ref_act + l * h + jj) = cur;
                cur = tanh(W(L.ref_th + l * h + jj) * cur);
              }
              double dh = (cur - y[jj]) / n_all;
              for (int l = units - 1; l >= 0; --l) {
                const double th = W(L.ref_th + l * h + jj);
                const double a = W(L.ref_act + l * h + jj);
                const double o = tanh(th * a);
                const double dz = dh * (1.0 - o * o);
                W(L.ref_g + l * h + jj) += dz * a;
                dh = dz * th;
              }
            }
          }
      for (int e = 0; e < P; ++e) {
        adam_elem(W(L.ref_om + e), W(L.ref_om + P + e), W(L.ref_om + 2 * P + e), W(L.ref_g + e), t);
        W(L.ref_th + e) = W(L.ref_om + e);
      }
    }

    // ---- Definition 4: every holder's view of Theta and Omega against the single-device state
    auto differs = [&](double got, double want) {
      const double d = fabs(got - want);
      const double rel = d / (fabs(want) > 1e-300 ? fabs(want) : 1e-300);
      if (d > dm.atol && rel > worst) worst = rel;
      return !(d <= dm.atol + dm.rtol * fabs(want));
    };
    if (pO == PS_MODE_M) {
      match = false;                                   // Omega is held nowhere
    } else {
      const int views = pO == PS_MODE_R ? D : 1;
      for (int v = 0; v < views; ++v)
        for (int row = 0; row < 3; ++row)
          for (int e = 0; e < P; ++e) {
            int holder = v;
            if (pO != PS_MODE_R) { holder = 0; while (!(e >= cut[holder] && e < cut[holder + 1])) ++holder; }
            if (differs(om_home(holder, row, e), W(L.ref_om + (size_t)row * P + e))) match = false;
          }
    }
    if (pT == PS_MODE_M) {
      // Theta exists only as the master copy, compared above
    } else {
      const int views = pT == PS_MODE_R ? D : 1;
      for (int v = 0; v < views; ++v)
        for (int e = 0; e < P; ++e) {
          int holder = v;
          if (pT != PS_MODE_R) { holder = 0; while (!(e >= cut[holder] && e < cut[holder + 1])) ++holder; }
          if (differs(th_home(holder, e), W(L.ref_th + e))) match = false;
        }
    }
  }

  ps_verify_result r;
  r.mem = (u64)books.memory(D);
  r.comm = (u64)books.comm;
  r.host = (u64)books.host_bytes(D);
  r.match = match ? 1u : 0u;
  r.pad = 0;
  r.max_rel_err = worst;
  out[idx] = r;
  if (theta_out) {
    // the parameters the job holds after the last step (first holder's view)
    for (int e = 0; e < P; ++e) {
      double v;
      if (pT == PS_MODE_R) v = th_home(0, e);
      else if (pT == PS_MODE_M) {
        int holder = 0;
        if (pO != PS_MODE_R) while (!(e >= cut[holder] && e < cut[holder + 1])) ++holder;
        v = pO == PS_MODE_M ? 0.0 : om_home(holder, 0, e);
      } else {
        int holder = 0;
        while (!(e >= cut[holder] && e < cut[holder + 1])) ++holder;
        v = th_home(holder, e);
      }
      theta_out[idx * (u64)P + e] = v;
    }
  }
}

}  // namespace

size_t verify_workspace_doubles(const ps_verify_shape& s) {
  const int P = (int)(s.units * s.h), EA = (int)(s.units * s.b * s.h);
  return make_layout(MAX_D, P, EA, (int)s.units, (int)s.h).total;
}

cudaError_t launch_verify(const ps_verify_shape& s, const ps_verify_case* d_cases, u64 n, const double* d_data,
                          u64 data_len, double* d_ws, double* d_theta_out, ps_verify_result* d_out, u32* status,
                          cudaStream_t stream) {
  Dims dm;
  dm.units = (int)s.units; dm.h = (int)s.h; dm.b = (int)s.b; dm.D = 0;
  dm.P = dm.units * dm.h; dm.EA = dm.units * dm.b * dm.h;
  dm.accum = (int)s.accum; dm.steps = (int)s.steps; dm.nbuf = (int)s.gather_buffers;
  dm.wT = (int)s.w_theta; dm.wO = (int)s.w_omega; dm.wG = (int)s.w_grad;
  dm.lr = s.lr; dm.beta1 = s.beta1; dm.beta2 = s.beta2; dm.eps = s.eps; dm.rtol = s.rtol; dm.atol = s.atol;
  const unsigned blocks = (unsigned)((n + 127) / 128);
  k_verify<<<blocks, 128, 0, stream>>>(dm, d_cases, n, d_data, data_len, d_ws, d_theta_out, d_out, status);
  return cudaGetLastError();
}
