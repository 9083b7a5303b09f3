// The table of compiled step kernels: for each element type and loss, the variants (lanes per row, values per lane)
// ordered by predictor capacity, each in every flavour and for both CTA sizes.  The six tables are built in
// translation units of their own (glm_table_*.cu), so that they compile side by side; the host code reaches them
// through the functions declared at the end.
#pragma once

#include "glm_kernel.cuh"

namespace bmgdk {

typedef void (*GlmKernel)(const GlmParams, const CUtensorMap);

struct GlmVariant {
    // [flavour][0: CTAs of up to kGlmSmallCta threads (more registers per thread), 1: the variant's second size (glm_max_threads), or null]
    GlmKernel k[kGlmFlavours][2];
    GlmKernel fn(int cta_threads, int flavour) const {
        const int large = (cta_threads > kGlmSmallCta && k[flavour][1]) ? 1 : 0;
        return k[flavour][large];
    }
    int vec, lpr, kch, maxc, maxt;
    int cap() const { return vec * lpr * kch; }
    int max_consumer_threads() const { return maxc; }  // warps that compute
    int max_threads() const { return maxt; }           // consumers plus producers
};

// The flavour of the step kernel a launch takes: a plain one wherever the step is Eq. (2.1) with a constant rate.
inline int glm_flavour(int opt_kind, int sched, int cpc) {
    if (opt_kind != kOptSgd || sched != kLrConstant) return kGlmAny;
    return cpc == 1 ? kGlmPlainOne : kGlmPlainTeam;
}

template <typename T, int VEC, int LPR, int KCH, bool LG, bool NULLSTEP>
constexpr GlmVariant make_variant() {
    constexpr int MT = glm_max_threads<T, VEC, KCH>();
    GlmVariant v{};
    v.k[kGlmAny][0] = glm_kernel<T, VEC, LPR, KCH, LG, kGlmSmallCta, kGlmAny, NULLSTEP>;
    v.k[kGlmPlainOne][0] = glm_kernel<T, VEC, LPR, KCH, LG, kGlmSmallCta, kGlmPlainOne, NULLSTEP>;
    v.k[kGlmPlainTeam][0] = glm_kernel<T, VEC, LPR, KCH, LG, kGlmSmallCta, kGlmPlainTeam, NULLSTEP>;
    if constexpr (MT != kGlmSmallCta) {
        v.k[kGlmAny][1] = glm_kernel<T, VEC, LPR, KCH, LG, MT, kGlmAny, NULLSTEP>;
        v.k[kGlmPlainOne][1] = glm_kernel<T, VEC, LPR, KCH, LG, MT, kGlmPlainOne, NULLSTEP>;
        v.k[kGlmPlainTeam][1] = glm_kernel<T, VEC, LPR, KCH, LG, MT, kGlmPlainTeam, NULLSTEP>;
    }
    v.vec = VEC; v.lpr = LPR; v.kch = KCH;
    v.maxc = glm_max_consumer_threads<T, VEC, KCH>();
    v.maxt = MT;
    return v;
}

// aligned16: rows are multiples of 16 bytes on a 16-byte boundary (vector loads, bulk copies); else one element per lane.
template <typename T, bool LG, bool NULLSTEP>
const GlmVariant* glm_variants(bool aligned16, int* count) {
    constexpr int V = 16 / (int)sizeof(T);
#define BMGD_VAR(VEC, LPR, KCH) make_variant<T, VEC, LPR, KCH, LG, NULLSTEP>()
    // ordered by capacity; among equal capacities the one listed first is the default, the others are reached
    // through cfg.lanes_per_row
    static const GlmVariant wide[] = {BMGD_VAR(V, 8, 1), BMGD_VAR(V, 8, 2), BMGD_VAR(V, 4, 4), BMGD_VAR(V, 4, 7),
                                      BMGD_VAR(V, 8, 4), BMGD_VAR(V, 8, 8), BMGD_VAR(V, 16, 8), BMGD_VAR(V, 32, 8)};
    static const GlmVariant narrow[] = {BMGD_VAR(1, 32, 1), BMGD_VAR(1, 32, 2), BMGD_VAR(1, 32, 4), BMGD_VAR(1, 32, 8)};
#undef BMGD_VAR
    if (aligned16) { *count = 8; return wide; }
    *count = 4;
    return narrow;
}

// One per translation unit.  The latency probe does not depend on the loss: it is built beside the least-squares
// kernels only ("null": the same launch without rows).
const GlmVariant* glm_variants_f32_linear(bool aligned16, int* count);
const GlmVariant* glm_variants_f32_logistic(bool aligned16, int* count);
const GlmVariant* glm_variants_f32_null(bool aligned16, int* count);
const GlmVariant* glm_variants_f64_linear(bool aligned16, int* count);
const GlmVariant* glm_variants_f64_logistic(bool aligned16, int* count);
const GlmVariant* glm_variants_f64_null(bool aligned16, int* count);

}  // namespace bmgdk
