#include "glm_table.cuh"

namespace bmgdk {
const GlmVariant* glm_variants_f32_null(bool aligned16, int* count) { return glm_variants<float, false, true>(aligned16, count); }
}  // namespace bmgdk
