// Sizes shared by the permutation kernels and the no-allocation histogram entry point.
#pragma once

namespace moe {

constexpr int P_TOKENS_PER_BLOCK = 256;  // tokens handled by one block of the count/place kernels
constexpr int P_MAX_LOCAL = 256;         // most local experts supported

}  // namespace moe
