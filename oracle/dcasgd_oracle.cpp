// CPU checker for the DC-ASGD parameter-server update.  TEST INFRASTRUCTURE ONLY.
//
// This is the slow, plain, single-threaded statement of what the server computes, written
// from the paper (Zheng et al., "Asynchronous Stochastic Gradient Descent with Delay
// Compensation", arXiv 1609.08326).  Only the test-suite, the smoke check and the CPU-baseline
// leg of the benchmark may load it.  It shares no code, header, table or helper with the CUDA
// library; the library never calls it and has no CPU fallback.
//
// What it follows, step by step and in the paper's order:
//   Algorithm 2, "Initialize"     : t = 0,  w_bak(m) = w_0 for every worker m
//   Algorithm 2, pull branch      : w_bak(m) <- w_t
//   Algorithm 2, gradient branch  : w_{t+1} <- w_t - eta*( g_m + lambda_t * g_m.g_m.(w_t - w_bak(m)) ),  t <- t+1
//                                   (the update rule of Section 4, Eq. 10, with w_bak(m) as the snapshot)
//   Section 6, "MeanSquare" equation (DC-ASGD-a):
//                                   MeanSquare(t) = m*MeanSquare(t-1) + (1-m)*g^2
//                                   lambda_t = lambda_0 / sqrt(MeanSquare(t) + eps)
//   Section 2, ASGD update rule   : the lambda = 0 special case (Section 5's closing discussion)
//
// Readings where the paper is silent (each is also listed in the design notes):
//   * MeanSquare is updated with the incoming gradient first and lambda_t uses the new value;
//     eps sits inside the root; MeanSquare(0) = 0; one MeanSquare vector on the server, fed by
//     every worker's raw (uncompensated) gradient in server order.
//   * The paper's moving-average constant "m" is called mu here (m is the worker index).
//   * Arithmetic is IEEE binary32 (binary64 in the *_f64 twins), every operation rounded on its
//     own, never fused, in this order:
//         gg = g*g ; [ms = mu*ms + (1-mu)*gg ; lam = lambda0 / sqrt(ms + eps)] ;
//         d = w - w_bak ; c = (lam*gg)*d ; u = g + c ; w = w - eta*u
//     with (1-mu) rounded once.  Build with -ffp-contract=off and without fast-math.
//   * A push with no earlier pull uses whatever w_bak(m) holds (w_0 after Initialize).
//   * bfloat16 gradients widen exactly (16 zero bits appended) before any arithmetic.
//
//   * Momentum (optional).  Section 6 says in a footnote that momentum variants were implemented
//     and gives no formula.  Reading taken: classical (heavy-ball) momentum on the
//     delay-compensated gradient u, as in the solvers the paper's ResNet code uses:
//         v = beta*v + eta*u ;  w = w - v          (v starts at 0; beta = 0 is Eq. 10 itself)
//     with beta*v and eta*u rounded separately, then their sum, then the difference.
//
// Pins (tests/test_oracle_pins.py): hand-worked dyadic examples checked against exact rational
// arithmetic, the closed form of repeated pushes on one snapshot, lambda = 0 against an
// independent ASGD loop, tau = 0 against plain SGD, MeanSquare against its unrolled sum,
// mu = 0 against g^2, and a brute-force element-outer replay on tiny inputs.
// Also pinned for momentum: beta = 0 equals the plain update bit for bit; with lambda = 0 and no
// delay it is textbook momentum SGD; exact rational replay with dyadic beta.
// Parity unpinned: the CHOICE of the momentum formula (the paper prints none); everything else
// in this file is pinned.  (The paper's accuracy tables need CIFAR-10/ImageNet and are outside
// what this checker computes.)

#include <cmath>
#include <cstdint>
#include <cstring>

extern "C" {
struct oracle_event { uint8_t kind; uint8_t pad[3]; uint32_t worker; uint32_t grad_id; float eta; };
enum { ORACLE_PULL = 0, ORACLE_PUSH = 1 };
enum { ORACLE_OK = 0, ORACLE_BAD_KIND = 1, ORACLE_BAD_WORKER = 2, ORACLE_BAD_GRAD = 3 };
}

namespace {

inline float widen_bf16(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return f;
}

template <class T> inline T root(T x);
template <> inline float root<float>(float x) { return sqrtf(x); }
template <> inline double root<double>(double x) { return sqrt(x); }

// Algorithm 2, "Initialize".
template <class T>
void init(uint64_t n, uint32_t M, const T* w, T* wb, T* ms) {
    for (uint32_t m = 0; m < M; ++m)
        for (uint64_t i = 0; i < n; ++i) wb[(uint64_t)m * n + i] = w[i];
    if (ms)
        for (uint64_t i = 0; i < n; ++i) ms[i] = (T)0;
}

// Algorithm 2, pull branch.
template <class T>
void pull(uint64_t n, uint32_t m, const T* w, T* wb) {
    for (uint64_t i = 0; i < n; ++i) wb[(uint64_t)m * n + i] = w[i];
}

// Algorithm 2, gradient branch (Eq. 10), with the MeanSquare rule of Section 6 when adaptive.
// G is the stored gradient type (T, or uint16_t holding bfloat16 when T is float).
template <class T, class G>
void push(uint64_t n, uint32_t m, int adaptive, T eta, T lambda, T mu, T eps,
          T* w, const T* wb, T* ms, const G* g, T beta, T* vel) {
    const T omm = (T)1 - mu;
    const T* snap = wb + (uint64_t)m * n;
    for (uint64_t i = 0; i < n; ++i) {
        T gi;
        if constexpr (sizeof(G) == 2) gi = (T)widen_bf16((uint16_t)g[i]); else gi = (T)g[i];
        T gg = gi * gi;
        T lam = lambda;
        if (adaptive) {
            T a = mu * ms[i];
            T b = omm * gg;
            T v = a + b;
            ms[i] = v;
            T s = v + eps;
            T r = root<T>(s);
            lam = lambda / r;
        }
        T d = w[i] - snap[i];
        T c = lam * gg;
        c = c * d;
        T u = gi + c;
        T p = eta * u;
        if (vel) {                                // momentum reading: v = beta*v + eta*u ; w = w - v
            T bv = beta * vel[i];
            T nv = bv + p;
            vel[i] = nv;
            p = nv;
        }
        w[i] = w[i] - p;
    }
}

template <class T, class G>
int replay(uint64_t n, uint32_t M, int adaptive, T default_eta, T lambda, T mu, T eps,
           T* w, T* wb, T* ms, const oracle_event* ev, uint64_t count,
           const G* grads, uint64_t grad_stride, uint32_t num_grads, uint64_t* t, T beta, T* vel) {
    for (uint64_t e = 0; e < count; ++e) {
        const oracle_event& r = ev[e];
        if (r.worker >= M) return ORACLE_BAD_WORKER;
        if (r.kind == ORACLE_PULL) {
            pull<T>(n, r.worker, w, wb);
        } else if (r.kind == ORACLE_PUSH) {
            if (r.grad_id >= num_grads) return ORACLE_BAD_GRAD;
            T eta = r.eta < 0.0f ? default_eta : (T)r.eta;
            push<T, G>(n, r.worker, adaptive, eta, lambda, mu, eps, w, wb, ms,
                       grads + (uint64_t)r.grad_id * grad_stride, beta, vel);
            if (t) *t += 1;                       // Algorithm 2: t advances on a gradient only
        } else {
            return ORACLE_BAD_KIND;
        }
    }
    return ORACLE_OK;
}

}  // namespace

extern "C" {

void oracle_init_f32(uint64_t n, uint32_t M, const float* w, float* wb, float* ms) { init<float>(n, M, w, wb, ms); }
void oracle_init_f64(uint64_t n, uint32_t M, const double* w, double* wb, double* ms) { init<double>(n, M, w, wb, ms); }

void oracle_pull_f32(uint64_t n, uint32_t m, const float* w, float* wb) { pull<float>(n, m, w, wb); }
void oracle_pull_f64(uint64_t n, uint32_t m, const double* w, double* wb) { pull<double>(n, m, w, wb); }

// beta, vel: momentum coefficient and velocity vector (n elements, starts at 0); vel == NULL
// means no momentum.
void oracle_push_f32(uint64_t n, uint32_t m, int adaptive, float eta, float lambda, float mu, float eps,
                     float* w, const float* wb, float* ms, const void* g, int g_is_bf16, float beta, float* vel) {
    if (g_is_bf16) push<float, uint16_t>(n, m, adaptive, eta, lambda, mu, eps, w, wb, ms, (const uint16_t*)g, beta, vel);
    else           push<float, float>(n, m, adaptive, eta, lambda, mu, eps, w, wb, ms, (const float*)g, beta, vel);
}
void oracle_push_f64(uint64_t n, uint32_t m, int adaptive, double eta, double lambda, double mu, double eps,
                     double* w, const double* wb, double* ms, const double* g, double beta, double* vel) {
    push<double, double>(n, m, adaptive, eta, lambda, mu, eps, w, wb, ms, g, beta, vel);
}

// Serial replay of a log (the repeat-loop of Algorithm 2).  grads: num_grads buffers,
// grad_stride ELEMENTS apart; record.eta < 0 selects default_eta.  *t counts pushes.
int oracle_replay_f32(uint64_t n, uint32_t M, int adaptive, float default_eta, float lambda, float mu,
                      float eps, float* w, float* wb, float* ms, const oracle_event* ev, uint64_t count,
                      const void* grads, uint64_t grad_stride, uint32_t num_grads, int g_is_bf16,
                      uint64_t* t, float beta, float* vel) {
    if (g_is_bf16)
        return replay<float, uint16_t>(n, M, adaptive, default_eta, lambda, mu, eps, w, wb, ms, ev, count,
                                       (const uint16_t*)grads, grad_stride, num_grads, t, beta, vel);
    return replay<float, float>(n, M, adaptive, default_eta, lambda, mu, eps, w, wb, ms, ev, count,
                                (const float*)grads, grad_stride, num_grads, t, beta, vel);
}
int oracle_replay_f64(uint64_t n, uint32_t M, int adaptive, double default_eta, double lambda, double mu,
                      double eps, double* w, double* wb, double* ms, const oracle_event* ev, uint64_t count,
                      const double* grads, uint64_t grad_stride, uint32_t num_grads, uint64_t* t,
                      double beta, double* vel) {
    return replay<double, double>(n, M, adaptive, default_eta, lambda, mu, eps, w, wb, ms, ev, count,
                                  grads, grad_stride, num_grads, t, beta, vel);
}

}  // extern "C"
