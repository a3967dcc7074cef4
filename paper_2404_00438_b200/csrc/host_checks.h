// Argument checks shared by the host-side entry points (no device code here).
#pragma once

#include <cmath>
#include <cstddef>
#include <cstdint>

namespace dlion {

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline bool aligned16(const void* p) { return aligned(p, 16); }
inline bool unit_interval(float v) { return v >= 0.0f && v <= 1.0f; }        // false for NaN
inline bool nonneg_finite(float v) { return v >= 0.0f && std::isfinite(v); }  // false for NaN, Inf

}  // namespace dlion
