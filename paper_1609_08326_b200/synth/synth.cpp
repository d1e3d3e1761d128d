// Seeded synthetic inputs for the DC-ASGD parameter-server replay: parameter vectors,
// gradient pools and worker event logs.
//
// This file holds NO arithmetic of the method (no update rule, no mean-square recurrence).
// It only turns (seed, stream, index) into numbers, so that the GPU library and the CPU
// checker can both be fed the very same bytes.  Every value is a pure function of
// (seed, stream, element index): any sub-range or any scattered subset of a vector can be
// regenerated on its own, by any number of threads, with identical results.
//
// Random bits: Philox4x32-10, written from its published definition (Salmon, Moraes, Dror,
// Shaw, "Parallel random numbers: as easy as 1, 2, 3", SC'11): ten rounds of
//   (c0,c1,c2,c3) <- (hi(M1*c2)^c1^k0, lo(M1*c2), hi(M0*c0)^c3^k1, lo(M0*c0))
// with the key bumped by the Weyl constants after every round.
// Normals: Box-Muller on two 24-bit uniforms in (0,1).

#include <cmath>
#include <cstdint>
#include <cstring>
#include <algorithm>
#include <thread>
#include <vector>

namespace {

struct U4 { uint32_t v[4]; };

inline U4 philox4x32_10(uint64_t counter_lo, uint64_t counter_hi, uint64_t key) {
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = (uint32_t)counter_lo, c1 = (uint32_t)(counter_lo >> 32);
    uint32_t c2 = (uint32_t)counter_hi, c3 = (uint32_t)(counter_hi >> 32);
    uint32_t k0 = (uint32_t)key, k1 = (uint32_t)(key >> 32);
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)M0 * c0;
        uint64_t p1 = (uint64_t)M1 * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0; k1 += W1;
    }
    return U4{{c0, c1, c2, c3}};
}

inline float u01(uint32_t x) {               // 24 random bits -> (0,1), never 0 or 1
    return ((float)(x >> 8) + 0.5f) * (1.0f / 16777216.0f);
}

// Four standard normals for block `blk` of stream `stream`.
inline void normal4(uint64_t seed, uint64_t stream, uint64_t blk, float out[4]) {
    U4 r = philox4x32_10(blk, stream, seed);
    const float two_pi = 6.28318530717958647692f;
    for (int p = 0; p < 2; ++p) {
        float u1 = u01(r.v[2 * p]), u2 = u01(r.v[2 * p + 1]);
        float rad = std::sqrt(-2.0f * std::log(u1));
        float a = two_pi * u2;
        out[2 * p]     = rad * std::cos(a);
        out[2 * p + 1] = rad * std::sin(a);
    }
}

inline float sigma_of(uint64_t i, const float* sigma, uint32_t nseg, uint64_t seg_len) {
    if (nseg <= 1 || seg_len == 0) return sigma[0];
    uint64_t s = i / seg_len;
    if (s >= nseg) s = nseg - 1;             // the remainder belongs to the last segment
    return sigma[s];
}

inline uint16_t f32_to_bf16_rne(float f) {   // round to nearest, ties to even
    uint32_t u; std::memcpy(&u, &f, 4);
    if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu)) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

template <class Store>
void fill_range(uint64_t first, uint64_t count, uint64_t seed, uint64_t stream,
                const float* sigma, uint32_t nseg, uint64_t seg_len, Store store) {
    uint64_t i = first, end = first + count;
    while (i < end) {
        uint64_t blk = i >> 2;
        float z[4];
        normal4(seed, stream, blk, z);
        uint64_t lane0 = i & 3u;
        for (uint64_t l = lane0; l < 4 && i < end; ++l, ++i)
            store(i - first, z[l] * sigma_of(i, sigma, nseg, seg_len));
    }
}

template <class Fn>
void run_threads(uint64_t count, int threads, Fn fn) {
    if (threads < 1) threads = 1;
    uint64_t chunk = (count + (uint64_t)threads - 1) / (uint64_t)threads;
    chunk = (chunk + 3u) & ~(uint64_t)3u;    // keep Philox blocks whole per thread
    if (threads == 1 || count < (1u << 16)) { fn((uint64_t)0, count); return; }
    std::vector<std::thread> pool;
    for (uint64_t b = 0; b < count; b += chunk)
        pool.emplace_back(fn, b, std::min(chunk, count - b));
    for (auto& t : pool) t.join();
}

}  // namespace

extern "C" {

// 16-byte log record; the same layout the server library and the checker read.
struct synth_event { uint8_t kind; uint8_t pad[3]; uint32_t worker; uint32_t grad_id; float eta; };

enum { SYNTH_PULL = 0, SYNTH_PUSH = 1 };
enum { SYNTH_ORDER_ROUND_ROBIN_JITTER = 0, SYNTH_ORDER_UNIFORM = 1, SYNTH_ORDER_ZIPF = 2 };
enum { SYNTH_PROTO_ASYNC = 0, SYNTH_PROTO_TAU0 = 1, SYNTH_PROTO_SYNC = 2 };

int synth_hardware_threads(void) {
    unsigned t = std::thread::hardware_concurrency();
    return t ? (int)t : 1;
}

// out[k] = sigma(first+k) * z(first+k), k in [0,count); z standard normal of (seed, stream).
// sigma: nseg values; element i uses sigma[min(i / seg_len, nseg-1)] (nseg==1: sigma[0]).
void synth_normal_f32(float* out, uint64_t first, uint64_t count, uint64_t seed, uint64_t stream,
                      const float* sigma, uint32_t nseg, uint64_t seg_len, int threads) {
    uint64_t mis = (4 - (first & 3u)) & 3u;   // align thread chunks to Philox blocks
    if (mis > count) mis = count;
    fill_range(first, mis, seed, stream, sigma, nseg, seg_len,
               [&](uint64_t k, float v) { out[k] = v; });
    run_threads(count - mis, threads, [=](uint64_t b, uint64_t c) {
        float* o = out + mis + b;
        fill_range(first + mis + b, c, seed, stream, sigma, nseg, seg_len,
                   [=](uint64_t k, float v) { o[k] = v; });
    });
}

// Same values, rounded to bfloat16 (nearest even) and stored as raw 16-bit patterns.
void synth_normal_bf16(uint16_t* out, uint64_t first, uint64_t count, uint64_t seed, uint64_t stream,
                       const float* sigma, uint32_t nseg, uint64_t seg_len, int threads) {
    uint64_t mis = (4 - (first & 3u)) & 3u;
    if (mis > count) mis = count;
    fill_range(first, mis, seed, stream, sigma, nseg, seg_len,
               [&](uint64_t k, float v) { out[k] = f32_to_bf16_rne(v); });
    run_threads(count - mis, threads, [=](uint64_t b, uint64_t c) {
        uint16_t* o = out + mis + b;
        fill_range(first + mis + b, c, seed, stream, sigma, nseg, seg_len,
                   [=](uint64_t k, float v) { o[k] = f32_to_bf16_rne(v); });
    });
}

// Scattered subset: out[k] = value of element idx[k] (fp32; bf16 flag rounds through bfloat16
// and widens back, so the subset holds exactly what the full bf16 vector would hold).
void synth_normal_gather(float* out, const uint64_t* idx, uint64_t count, uint64_t seed,
                         uint64_t stream, const float* sigma, uint32_t nseg, uint64_t seg_len,
                         int through_bf16) {
    for (uint64_t k = 0; k < count; ++k) {
        uint64_t i = idx[k];
        float z[4];
        normal4(seed, stream, i >> 2, z);
        float v = z[i & 3u] * sigma_of(i, sigma, nseg, seg_len);
        if (through_bf16) {
            uint32_t u = (uint32_t)f32_to_bf16_rne(v) << 16;
            std::memcpy(&v, &u, 4);
        }
        out[k] = v;
    }
}

// sigma[s] = 10^U, U uniform in [lo_exp, hi_exp]: per-segment gradient scales.
void synth_log_uniform_sigma(float* sigma, uint32_t nseg, double lo_exp, double hi_exp,
                             uint64_t seed, uint64_t stream) {
    for (uint32_t s = 0; s < nseg; ++s) {
        U4 r = philox4x32_10(s, stream, seed);
        double u = ((double)r.v[0] + 0.5) / 4294967296.0;
        sigma[s] = (float)std::pow(10.0, lo_exp + (hi_exp - lo_exp) * u);
    }
}

// Raw 32-bit words of a stream, for callers that shape their own integers (batch picks etc.).
void synth_u32(uint32_t* out, uint64_t first, uint64_t count, uint64_t seed, uint64_t stream) {
    for (uint64_t k = 0; k < count; ++k) {
        uint64_t i = first + k;
        U4 r = philox4x32_10(i >> 2, stream, seed);
        out[k] = r.v[i & 3u];
    }
}

// Number of records synth_event_log writes for these settings.
uint64_t synth_event_log_size(uint32_t M, uint64_t pushes, uint32_t proto) {
    if (proto == SYNTH_PROTO_ASYNC) return (uint64_t)M + 2 * pushes;
    if (proto == SYNTH_PROTO_TAU0) return 2 * pushes;
    /* SYNC: rounds of (M pulls, M pushes); pushes is rounded down to whole rounds */
    return 2 * (pushes / M) * (uint64_t)M;
}

// Worker event log standing in for M asynchronous workers that loop pull -> compute -> push.
//   order : who pushes next (round-robin with +-1 jitter, uniform, or Zipf(order_param) speeds)
//   proto : ASYNC = M leading pulls, then every PUSH(m) is followed at once by PULL(m)
//           TAU0  = every PUSH(m) is preceded at once by PULL(m)        (no delay at all)
//           SYNC  = rounds: all M workers pull, then all M push in the drawn order
//   grad_id of the e-th push is e mod num_grads; every record carries `eta`.
// Returns the number of records written, or 0 if `capacity` is too small / arguments invalid.
uint64_t synth_event_log(synth_event* out, uint64_t capacity, uint32_t M, uint64_t pushes,
                         uint32_t order, double order_param, uint32_t proto, uint32_t num_grads,
                         float eta, uint64_t seed, uint64_t stream) {
    if (M == 0 || num_grads == 0 || order > 2 || proto > 2) return 0;
    if (proto == SYNTH_PROTO_SYNC) pushes = (pushes / M) * M;
    uint64_t need = synth_event_log_size(M, pushes, proto);
    if (capacity < need) return 0;

    std::vector<uint32_t> who(pushes);
    if (order == SYNTH_ORDER_ROUND_ROBIN_JITTER) {
        // key_e = e + j_e, j_e in {-1,0,+1}; stable sort by key; e-th slot keeps worker e mod M
        std::vector<std::pair<int64_t, uint64_t>> key(pushes);
        for (uint64_t e = 0; e < pushes; ++e) {
            U4 r = philox4x32_10(e, stream, seed);
            int64_t j = (int64_t)(((uint64_t)r.v[0] * 3u) >> 32) - 1;
            key[e] = {(int64_t)e + j, e};
        }
        std::stable_sort(key.begin(), key.end(),
                         [](const std::pair<int64_t, uint64_t>& a,
                            const std::pair<int64_t, uint64_t>& b) { return a.first < b.first; });
        for (uint64_t p = 0; p < pushes; ++p) who[p] = (uint32_t)(key[p].second % M);
    } else if (order == SYNTH_ORDER_UNIFORM) {
        for (uint64_t e = 0; e < pushes; ++e) {
            U4 r = philox4x32_10(e, stream, seed);
            who[e] = (uint32_t)(((uint64_t)r.v[0] * M) >> 32);
        }
    } else {
        // worker of rank k (1-based) pushes with probability proportional to k^-s
        std::vector<double> cdf(M);
        double tot = 0.0;
        for (uint32_t k = 0; k < M; ++k) { tot += std::pow((double)(k + 1), -order_param); cdf[k] = tot; }
        for (uint64_t e = 0; e < pushes; ++e) {
            U4 r = philox4x32_10(e, stream, seed);
            double u = (((double)r.v[0] + 0.5) / 4294967296.0) * tot;
            uint32_t k = (uint32_t)(std::lower_bound(cdf.begin(), cdf.end(), u) - cdf.begin());
            who[e] = k < M ? k : M - 1;
        }
    }

    uint64_t n = 0;
    auto put = [&](uint8_t kind, uint32_t m, uint32_t gid) {
        synth_event ev; std::memset(&ev, 0, sizeof ev);
        ev.kind = kind; ev.worker = m; ev.grad_id = gid; ev.eta = eta;
        out[n++] = ev;
    };
    if (proto == SYNTH_PROTO_ASYNC) {
        for (uint32_t m = 0; m < M; ++m) put(SYNTH_PULL, m, 0);
        for (uint64_t e = 0; e < pushes; ++e) {
            put(SYNTH_PUSH, who[e], (uint32_t)(e % num_grads));
            put(SYNTH_PULL, who[e], 0);
        }
    } else if (proto == SYNTH_PROTO_TAU0) {
        for (uint64_t e = 0; e < pushes; ++e) {
            put(SYNTH_PULL, who[e], 0);
            put(SYNTH_PUSH, who[e], (uint32_t)(e % num_grads));
        }
    } else {
        for (uint64_t r0 = 0; r0 < pushes; r0 += M) {
            for (uint32_t m = 0; m < M; ++m) put(SYNTH_PULL, m, 0);
            // push order inside the round: workers sorted by their drawn value (a permutation)
            std::vector<std::pair<uint32_t, uint32_t>> perm(M);
            for (uint32_t m = 0; m < M; ++m) {
                U4 r = philox4x32_10(r0 + m, stream ^ 0x5343u, seed);
                perm[m] = {r.v[1], m};
            }
            std::sort(perm.begin(), perm.end());
            for (uint32_t j = 0; j < M; ++j)
                put(SYNTH_PUSH, perm[j].second, (uint32_t)((r0 + j) % num_grads));
        }
    }
    return n;
}

}  // extern "C"
