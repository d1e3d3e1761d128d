// Host-side window compiler: turns a run of log records into the step program that the fused
// replay kernel walks.  No CUDA in this translation unit.
#pragma once
#include <cstdint>
#include <vector>

#include "dcasgd.h"

namespace dcasgd {

// Thread-local error text shared by the host API (defined in window_compiler.cpp).
void set_error(const char* fmt, ...);
const char* get_error();

// Records one window may span at most, whatever window_k says (see WindowCompiler::compile).
constexpr uint64_t kMaxWindowScan = 2048;

// Reusable scratch for compiling many windows of one log (per-worker arrays are allocated once).
struct WindowCompiler {
    explicit WindowCompiler(uint32_t num_workers);
    // Same contract as dcasgd_compile_window; arguments must be non-NULL and positive
    // (max_slots 0 or out of range means DCASGD_MAX_WINDOW_SLOTS).
    int compile(const dcasgd_event* ev, uint64_t count, uint32_t window_k, float default_eta,
                uint32_t max_slots, dcasgd_window_program* out);

    uint32_t M;
    std::vector<uint32_t> uses, pending, remaining;
    std::vector<uint8_t> is_last, seen, pulled;
    std::vector<uint64_t> first_consumer, first_push;
    std::vector<int32_t> cur_slot;
};

}  // namespace dcasgd
