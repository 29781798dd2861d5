// Shared between the dedup kernels and the code that sets a workspace up.
#pragma once
#include <cstdint>

namespace mfet {

// The dedup's digit totals sit at the start of WsLayout::hist and must be zero between calls: the
// library clears them when a workspace is set, and every call leaves them at zero.
constexpr uint64_t kDedupTotalsBytes = 8 * 256 * 4;

}  // namespace mfet
