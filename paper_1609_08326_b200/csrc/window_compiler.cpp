// Window compiler for the fused replay of Algorithm 2's message loop.
//
// Algorithm 2 handles one message at a time.  Its update (Section 4, Eq. 10) and the MeanSquare
// rule (Section 6) are elementwise, so for ONE element the whole window can be replayed with w
// in a register.  What has to survive the window is decided here, per window, by a liveness
// pass over the records:
//   * a PUSH(m) whose worker pulled earlier in the window uses that in-window value of w
//     (kept in a slot); otherwise it reads w_bak[m] as it was before the window;
//   * only the LAST pull of a worker in the window writes w_bak[m];
//   * a pull that is superseded before being used does nothing.
#include "window_compiler.h"

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <vector>

namespace dcasgd {

static thread_local char g_err[512] = "";

void set_error(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
}
const char* get_error() { return g_err; }

namespace {

// One attempt at compiling records [0,K).  Returns 0 on success, otherwise the smaller K (>= 1)
// at which the window has to end.
uint64_t attempt(WindowCompiler& c, const dcasgd_event* ev, uint64_t K, float default_eta,
                 int32_t max_slots, dcasgd_window_program* out) {
    auto &uses = c.uses, &pending = c.pending, &remaining = c.remaining;
    auto &is_last = c.is_last, &seen = c.seen, &pulled = c.pulled;
    auto &first_consumer = c.first_consumer, &first_push = c.first_push;
    auto &cur_slot = c.cur_slot;
    // backward: how often each pull is used, and whether it is its worker's last one
    for (uint64_t r = K; r-- > 0;) {
        const uint32_t m = ev[r].worker;
        if (ev[r].kind == DCASGD_PUSH) {
            pending[m] += 1;
            first_push[m] = r;
        } else {
            uses[r] = pending[m];
            first_consumer[r] = first_push[m];
            is_last[r] = !seen[m];
            pending[m] = 0;
            seen[m] = 1;
        }
    }
    for (uint64_t r = 0; r < K; ++r) {           // leave the per-worker scratch clean
        const uint32_t m = ev[r].worker;
        pending[m] = 0; seen[m] = 0; cur_slot[m] = -1; remaining[m] = 0; pulled[m] = 0;
    }

    std::memset(out, 0, sizeof *out);
    uint32_t slot_ref[DCASGD_MAX_WINDOW_SLOTS] = {0};
    uint32_t j = 0, n_stores = 0, n_slots = 0;
    out->save_slot[0] = -1;
    out->store_begin[0] = 0;
    uint64_t cut = 0;
    uint64_t r = 0;
    for (; r < K; ++r) {
        const uint32_t m = ev[r].worker;
        if (ev[r].kind == DCASGD_PUSH) {
            if (j == DCASGD_MAX_WINDOW_PUSHES) { cut = r; break; }
            out->grad_id[j] = ev[r].grad_id;
            out->eta[j] = ev[r].eta < 0.0f ? default_eta : ev[r].eta;
            if (pulled[m]) {
                const int32_t s = cur_slot[m];
                out->src[j] = -(s + 1);
                if (--remaining[m] == 0) { slot_ref[s] -= 1; cur_slot[m] = -1; }
            } else {
                out->src[j] = (int32_t)m;
                out->n_snapshot_reads += 1;
            }
            ++j;
            out->save_slot[j] = -1;
            out->store_begin[j] = n_stores;
        } else {
            pulled[m] = 1;
            if (uses[r] == 0 && !is_last[r]) { out->n_dead_pulls += 1; continue; }
            if (is_last[r]) {
                if (n_stores == DCASGD_MAX_WINDOW_STORES) { cut = r; break; }
                out->store_worker[n_stores++] = m;
            }
            if (uses[r] > 0) {
                int32_t s = out->save_slot[j];
                if (s < 0) {
                    for (int32_t k = 0; k < max_slots; ++k)
                        if (slot_ref[k] == 0) { s = k; break; }
                    if (s < 0) { cut = first_consumer[r]; break; }   // no slot: end before its first use
                    out->save_slot[j] = s;
                    if ((uint32_t)s + 1 > n_slots) n_slots = (uint32_t)s + 1;
                }
                slot_ref[s] += 1;
                cur_slot[m] = s;
                remaining[m] = uses[r];
            }
        }
    }
    for (uint64_t q = 0; q < K; ++q) {
        const uint32_t m = ev[q].worker;
        cur_slot[m] = -1; remaining[m] = 0; pulled[m] = 0;
    }
    if (cut) return cut;
    out->store_begin[j + 1] = n_stores;
    out->n_records = (uint32_t)K;
    out->n_pushes = j;
    out->n_slots = n_slots;
    out->n_stores = n_stores;
    return 0;
}

}  // namespace

WindowCompiler::WindowCompiler(uint32_t num_workers)
    : M(num_workers), pending(num_workers, 0), remaining(num_workers, 0), seen(num_workers, 0),
      pulled(num_workers, 0), first_push(num_workers, 0), cur_slot(num_workers, -1) {}

int WindowCompiler::compile(const dcasgd_event* ev, uint64_t count, uint32_t window_k, float default_eta,
                            uint32_t max_slots, dcasgd_window_program* out) {
    if (max_slots == 0 || max_slots > DCASGD_MAX_WINDOW_SLOTS) max_slots = DCASGD_MAX_WINDOW_SLOTS;
    uint64_t K = count < window_k ? count : window_k;
    // A window holds a few hundred pushes and stores at most, and every attempt below walks all K
    // records: bound K so that compiling a long log with a huge window_k stays linear in the log.
    // (A shorter window is always legal and the results are the same bit for bit.)
    if (K > kMaxWindowScan) K = kMaxWindowScan;
    for (uint64_t r = 0; r < K; ++r) {
        if (ev[r].kind > DCASGD_PUSH) { set_error("log record %llu: unknown kind %u", (unsigned long long)r, ev[r].kind); return DCASGD_ELOG; }
        if (ev[r].worker >= M) { set_error("log record %llu: worker %u >= %u", (unsigned long long)r, ev[r].worker, M); return DCASGD_ELOG; }
        if (ev[r].kind == DCASGD_PUSH && !std::isfinite(ev[r].eta)) { set_error("log record %llu: eta is not finite", (unsigned long long)r); return DCASGD_ELOG; }
    }
    if (uses.size() < K) { uses.resize(K); is_last.resize(K); first_consumer.resize(K); }
    for (;;) {
        uint64_t cut = attempt(*this, ev, K, default_eta, (int32_t)max_slots, out);
        if (cut == 0) return DCASGD_OK;
        K = cut;
    }
}

}  // namespace dcasgd

extern "C" int dcasgd_compile_window(const dcasgd_event* ev, uint64_t count, uint32_t num_workers,
                                     uint32_t window_k, float default_eta, uint32_t max_slots,
                                     dcasgd_window_program* out) {
    using namespace dcasgd;
    if (!ev || !out) { set_error("dcasgd_compile_window: NULL argument"); return DCASGD_EINVAL; }
    if (count == 0 || window_k == 0 || num_workers == 0) {
        set_error("dcasgd_compile_window: count, window_k and num_workers must be positive");
        return DCASGD_EINVAL;
    }
    if (max_slots > DCASGD_MAX_WINDOW_SLOTS) {
        set_error("dcasgd_compile_window: max_slots %u > %u", max_slots, (unsigned)DCASGD_MAX_WINDOW_SLOTS);
        return DCASGD_EINVAL;
    }
    try {
        WindowCompiler c(num_workers);
        return c.compile(ev, count, window_k, default_eta, max_slots, out);
    } catch (...) {
        set_error("dcasgd_compile_window: out of host memory");
        return DCASGD_ENOMEM;
    }
}
