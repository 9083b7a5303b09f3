#include "glm_table.cuh"

namespace bmgdk {
const GlmVariant* glm_variants_f64_logistic(bool aligned16, int* count) { return glm_variants<double, true, false>(aligned16, count); }
}  // namespace bmgdk
