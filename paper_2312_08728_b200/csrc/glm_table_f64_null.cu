#include "glm_table.cuh"

namespace bmgdk {
const GlmVariant* glm_variants_f64_null(bool aligned16, int* count) { return glm_variants<double, false, true>(aligned16, count); }
}  // namespace bmgdk
