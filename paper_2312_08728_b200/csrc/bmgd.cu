// Host side of the BMGD library: the C ABI of include/bmgd.h, the handle, the two buffer slots
// with their copy/compute event ordering (the buffering step of Section 2.1 overlapped with the
// computation step), launch-shape selection and kernel dispatch.
#include "../../include/bmgd.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <thread>
#include <vector>

#include "aux_kernels.cuh"
#include "glm_table.cuh"
#include "softmax_kernel.cuh"

namespace {

using bmgdk::GlmKernel;
using bmgdk::GlmParams;
using bmgdk::GlmVariant;

constexpr int64_t kAlign = 256;
constexpr int kMaxClustersForExchange = 160;  // upper bound on clusters in one grid (148 SMs)
constexpr int kVersion = 1000;

inline int64_t align_up(int64_t v, int64_t a = kAlign) { return (v + a - 1) / a * a; }

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

struct EventPair {
    cudaEvent_t a, b;
};

struct Layout {
    int64_t slot_x[2], slot_y[2];
    int64_t theta, opt1, opt2, ll, status, softmax_scratch;
    int64_t total;
};

}  // namespace

struct bmgd {
    bmgd_config cfg;
    int device = 0;
    int sm_count = 0;
    int smem_optin = 0;
    int64_t N0cap = 0;
    int xb = 4, yb = 4, tb = 4;  // bytes per stored x, y, theta element
    int num_slots = 2;
    unsigned char* base = nullptr;
    bool owns_base = false;
    Layout lay{};
    cudaStream_t compute = nullptr;
    bool owns_stream = false;
    cudaEvent_t loaded[2] = {nullptr, nullptr};
    cudaEvent_t freed[2] = {nullptr, nullptr};
    int64_t slot_rows[2] = {0, 0};
    bool slot_has_data[2] = {false, false};
    int next_slot = 0;
    uint64_t tag_base = 0;
    int last_cuda = 0;
    bmgd_stats stats{};
    std::vector<EventPair> kernel_events, copy_events, event_pool;
    uint64_t timeout_ns = 2000000000ull;
    // update rule and learning-rate schedule (bmgd_set_optimizer, bmgd_set_lr_schedule)
    int opt_kind = BMGD_OPT_SGD;
    double opt_a = 0.0, opt_b = 0.0, opt_eps = 0.0;
    int64_t opt_steps = 0;     // updates taken since the rule was set: Adam's t
    int sched = BMGD_LR_CONSTANT;
    int64_t sched_period = 0;  // updates per pass
    int64_t sched_pos = 0;     // updates of the current pass already taken
};

namespace {

int cuda_fail(bmgd* h, cudaError_t e) {
    if (h) h->last_cuda = (int)e;
    cudaGetLastError();  // clear the sticky-less error state
    return BMGD_ERR_CUDA;
}

#define BMGD_CUDA(h, call)                                   \
    do {                                                     \
        cudaError_t e__ = (call);                            \
        if (e__ != cudaSuccess) return cuda_fail((h), e__);  \
    } while (0)

int elem_bytes_x(int dtype) { return dtype == BMGD_F64 ? 8 : dtype == BMGD_F32 ? 4 : 2; }
int elem_bytes_theta(int dtype) { return dtype == BMGD_F64 ? 8 : 4; }

int validate(const bmgd_config* c) {
    if (!c) return BMGD_ERR_ARG;
    if (c->N <= 0 || c->p <= 0 || c->K <= 0 || c->K > c->N) return BMGD_ERR_ARG;
    if (c->loss < BMGD_LOSS_LINEAR || c->loss > BMGD_LOSS_SOFTMAX) return BMGD_ERR_ARG;
    if (c->dtype < BMGD_F64 || c->dtype > BMGD_BF16X_F32W) return BMGD_ERR_ARG;
    if (c->Rc < 1 || c->Rc > 65536) return BMGD_ERR_ARG;
    if (c->loss == BMGD_LOSS_SOFTMAX) {
        if (c->C < 2 || c->C > 16) return c->C < 2 ? BMGD_ERR_ARG : BMGD_ERR_UNIMPLEMENTED;
        if (c->dtype != BMGD_BF16X_F32W) return BMGD_ERR_UNIMPLEMENTED;
    } else {
        if (c->C != 1) return BMGD_ERR_ARG;
        if (c->dtype == BMGD_BF16X_F32W) return BMGD_ERR_UNIMPLEMENTED;
    }
    const int64_t N0 = (c->N + c->K - 1) / c->K;
    if (N0 > 0x7FFFFFFFll) return BMGD_ERR_ARG;
    for (int i = 0; i < 4; ++i)
        if (c->reserved[i] != 0) return BMGD_ERR_ARG;
    if (c->first_chain < 0 || (int64_t)c->first_chain + c->Rc > 0x7FFFFFFFll) return BMGD_ERR_ARG;

    if (c->lanes_per_row != 0 && c->lanes_per_row != 4 && c->lanes_per_row != 8 && c->lanes_per_row != 16 &&
        c->lanes_per_row != 32)
        return BMGD_ERR_ARG;
    if (c->producer_warps < 0 || c->producer_warps > 8) return BMGD_ERR_ARG;
    if (c->cluster_size != 0 && c->cluster_size != 1 && c->cluster_size != 2 && c->cluster_size != 4 &&
        c->cluster_size != 8 && c->cluster_size != 16)
        return BMGD_ERR_ARG;
    if (c->threads_per_cta != 0 && (c->threads_per_cta % 32 != 0 || c->threads_per_cta < 256 || c->threads_per_cta > 1024))
        return BMGD_ERR_ARG;
    if (c->pipeline_depth != 0 && (c->pipeline_depth < 2 || c->pipeline_depth > 8)) return BMGD_ERR_ARG;
    if (c->subpasses_per_stage != 0 && c->subpasses_per_stage != 1 && c->subpasses_per_stage != 2 &&
        c->subpasses_per_stage != 4 && c->subpasses_per_stage != 8 && c->subpasses_per_stage != 16 &&
        c->subpasses_per_stage != 32)
        return BMGD_ERR_ARG;
    if (c->ctas_per_chain < 0) return BMGD_ERR_ARG;
    if (c->workspace && ((uintptr_t)c->workspace % kAlign) != 0) return BMGD_ERR_ARG;
    return BMGD_OK;
}

Layout make_layout(const bmgd_config* c) {
    Layout L{};
    const int64_t N0 = (c->N + c->K - 1) / c->K;
    const int xb = elem_bytes_x(c->dtype), tb = elem_bytes_theta(c->dtype);
    const int yb = c->loss == BMGD_LOSS_SOFTMAX ? 4 : tb;
    int64_t off = 0;
    const int slots = (c->flags & BMGD_FLAG_NO_SLOTS) ? 0 : 2;
    for (int s = 0; s < 2; ++s) {
        L.slot_x[s] = off; if (s < slots) off += align_up(N0 * c->p * xb);
        L.slot_y[s] = off; if (s < slots) off += align_up(N0 * yb);
    }
    L.theta = off; off += align_up((int64_t)c->Rc * c->p * c->C * tb);
    // state of the update rule, beside theta: Nesterov's velocity or Adam's first moment, and Adam's second moment
    L.opt1 = off; if (c->loss != BMGD_LOSS_SOFTMAX) off += align_up((int64_t)c->Rc * c->p * tb);
    L.opt2 = off; if (c->loss != BMGD_LOSS_SOFTMAX) off += align_up((int64_t)c->Rc * c->p * tb);
    L.ll = off;
    if (c->loss != BMGD_LOSS_SOFTMAX) off += align_up((int64_t)2 * kMaxClustersForExchange * c->p * 2 * 8);
    L.status = off; off += kAlign;
    L.softmax_scratch = off;
    if (c->loss == BMGD_LOSS_SOFTMAX) off += align_up(bmgdk::softmax_scratch_bytes(c->p, c->C));
    L.total = off;
    return L;
}

// ------------------------------------------------------------------ tensor map of a buffer

// cuTensorMapEncodeTiled, looked up through the runtime so that the library links against cudart only.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static std::once_flag once;
    static EncodeTiledFn fn = nullptr;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            cudaGetLastError();
    });
    return fn;
}

// X [rows][p] as a 2-D tensor whose box is one row of `box` values (the kernel's predictor capacity): the step kernel
// gathers four rows per copy; columns from p on, and rows from `rows` on, read as zeros.  dev_x and the row size are
// 16-byte multiples.  Host-only work: nothing is allocated.
int make_row_map(const void* dev_x, int64_t rows, int p, int elem_bytes, int box, CUtensorMap* out) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return BMGD_ERR_CUDA;
    const cuuint64_t dims[2] = {(cuuint64_t)p, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)p * (cuuint64_t)elem_bytes};
    const cuuint32_t boxdim[2] = {(cuuint32_t)box, 1u};
    const cuuint32_t estr[2] = {1u, 1u};
    const CUresult r = enc(out, elem_bytes == 8 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT64 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                           const_cast<void*>(dev_x), dims, strides, boxdim, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? BMGD_OK : BMGD_ERR_CUDA;
}

// ------------------------------------------------------------------ GLM kernel table

// null_step: the latency probe of that shape instead of the step kernel (it does not depend on the loss)
const GlmVariant* pick_variant(int dtype, int loss, int p, bool aligned16, int lanes_per_row = 0, bool null_step = false) {
    int cnt = 0;
    const bool lg = loss == BMGD_LOSS_LOGISTIC;
    const GlmVariant* v = null_step
        ? (dtype == BMGD_F64 ? bmgdk::glm_variants_f64_null(aligned16, &cnt) : bmgdk::glm_variants_f32_null(aligned16, &cnt))
        : dtype == BMGD_F64
        ? (lg ? bmgdk::glm_variants_f64_logistic(aligned16, &cnt) : bmgdk::glm_variants_f64_linear(aligned16, &cnt))
        : (lg ? bmgdk::glm_variants_f32_logistic(aligned16, &cnt) : bmgdk::glm_variants_f32_linear(aligned16, &cnt));
    if (lanes_per_row)  // the smallest variant with that many lanes per row, if there is one
        for (int i = 0; i < cnt; ++i)
            if (v[i].cap() >= p && v[i].lpr == lanes_per_row) return &v[i];
    for (int i = 0; i < cnt; ++i)
        if (v[i].cap() >= p) return &v[i];
    return nullptr;
}

// How often a waiting thread looks at the clock and the abort flag.  A budget below a microsecond cannot be measured:
// it counts as no budget at all, and every failed poll looks, so that a wait that does not succeed at its first look
// gives up.
void set_poll_cadence(GlmParams* P) {
    const bool tiny = P->timeout_ns < 1000ull;
    if (tiny) P->timeout_ns = 0;
    P->poll_mask = tiny ? 0u : 0x3FFu;
    P->mbar_mask = tiny ? 0u : 0x3Fu;
}

int floor_pow2(int v) {
    int r = 1;
    while (r * 2 <= v) r *= 2;
    return r;
}

struct LaunchShape {
    int S, cpc, nteams, threads, pwarps, depth, passes, rb, smem;  // threads: of the consumer warps
};

int max_active_clusters(bmgd* h, GlmKernel fn, int S, int threads, int smem, int* out) {
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3((unsigned)(S * h->sm_count), 1, 1);
    lc.blockDim = dim3((unsigned)threads, 1, 1);
    lc.dynamicSmemBytes = (size_t)smem;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)S; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    lc.attrs = at; lc.numAttrs = 1;
    int n = 0;
    BMGD_CUDA(h, cudaOccupancyMaxActiveClusters(&n, (const void*)fn, &lc));
    *out = n;
    return BMGD_OK;
}

int plan_glm(bmgd* h, const GlmVariant* var, int64_t rows, int n, LaunchShape* out) {
    const bmgd_config& c = h->cfg;
    const int eb = h->tb;
    const int gpw = 32 / var->lpr;
    const int pcap = var->cap();
    LaunchShape L{};
    // Replicate chains keep every SM busy with several chains' rows in flight: throughput, not the per-step latency,
    // sets the pace there, so variants with little per-lane state run as large a CTA as the register file allows
    // (measured on B200: 16 consumer warps and 4 producer warps beat 12 + 8 and 14 + 6 once rows arrive four per
    // gather).  Variants with wide per-lane state always run 8 consumer warps at 168 registers.
    const bool throughput = c.Rc > 1 && var->max_consumer_threads() >= 512;
    L.threads = c.threads_per_cta ? std::min(c.threads_per_cta, var->max_consumer_threads()) : (throughput ? 512 : 256);
    // Producer warps only evaluate the shuffle and issue copies; this is how many the CTA has room for.  Their number is
    // settled below, once the ring is known: rows fetched by gathers are dealt to all producers stage by stage (4 by
    // default), other layouts give every ring slot its own producer warp (or several that share its rows).
    const int max_pwarps = std::min(8, (var->max_threads() - L.threads) / 32);
    if (max_pwarps < 2) return BMGD_ERR_ARG;
    const int warps = L.threads / 32;
    const int spp = warps * gpw;  // rows a CTA works on at once (one sub-pass)
    const bool pre = bmgdk::glm_prereduce(var->kch * var->vec, var->lpr);
    const bool gathered = bmgdk::glm_gathered(var->vec * eb, pcap);

    // Cluster size.  Measured on B200: a step costs one exchange through distributed shared memory (about 0.8 us among
    // 16 CTAs) inside one cluster, and about 2.5 us more once partial sums have to cross clusters through L2, while a
    // sub-pass of spp rows costs about 0.15-0.3 us.  So a chain gets the largest cluster the device admits and stays inside it unless a CTA would have to
    // sweep many sub-passes per step.
    int S = c.cluster_size;
    if (S == 0) {
        if (c.Rc > 1) S = std::min(8, floor_pow2(std::max(1, h->sm_count / c.Rc)));
        else S = 16;
        // do not spread a mini-batch thinner than two sweeps of a CTA over its rows: below that a larger cluster only
        // adds exchange latency (measured on B200, n = 100 in fp64: 1.46 us per step on one CTA, 1.58-1.71 on two, 1.65 on
        // four, 1.9 on eight)
        while (S > 1 && n / S < 2 * spp) S /= 2;
    }

    // How many clusters can be resident depends on shared memory, which depends on the ring; ask with
    // the largest ring we would use (a smaller one can only admit more).
    int max_clusters = 0, fixed_smem = 0, ring_budget = 0;
    for (;;) {
        fixed_smem = bmgdk::glm_smem_plan(warps, gpw, pre, 1, 0, pcap, eb, S, false, gathered).total_bytes;
        ring_budget = h->smem_optin - fixed_smem - 1024;  // all of the CTA's shared memory but a small reserve
        if (ring_budget < 2 * bmgdk::glm_smem_plan(warps, gpw, pre, 1, 1, pcap, eb, S, false, gathered).stage_bytes) {  // the per-peer exchange buffers of a large cluster leave no room for rows
            if (c.cluster_size == 0 && S > 1) { S /= 2; continue; }
            return BMGD_ERR_UNIMPLEMENTED;
        }
        const int probe_smem = fixed_smem + ring_budget;
        // whichever flavour and CTA size the launch takes in the end (they depend on the clusters per chain and the ring
        // depth chosen below), it runs with these limits; a CTA takes nearly all of an SM's shared memory, so one
        // instance answers for all on residency
        for (int fl = 0; fl < bmgdk::kGlmFlavours; ++fl) {
            for (int size = 0; size < 2; ++size) {
                const void* fn = (const void*)var->k[fl][size];
                if (!fn) continue;
                BMGD_CUDA(h, cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, probe_smem));
                BMGD_CUDA(h, cudaFuncSetAttribute(fn, cudaFuncAttributeNonPortableClusterSizeAllowed, S > 8 ? 1 : 0));
            }
        }
        max_clusters = h->sm_count;
        if (S > 1) {
            const int probe_threads = L.threads + 32 * max_pwarps;
            int rc = max_active_clusters(h, var->fn(probe_threads, bmgdk::kGlmAny), S, probe_threads, probe_smem, &max_clusters);
            if (rc != BMGD_OK) {
                if (c.cluster_size == 0 && S > 8) { S = 8; continue; }  // clusters of 16 are optional in hardware
                return rc;
            }
        }
        if (max_clusters < 1 && c.cluster_size == 0 && S > 8) { S = 8; continue; }
        break;
    }
    if (max_clusters < 1) return BMGD_ERR_LAUNCH;
    max_clusters = std::min(max_clusters, kMaxClustersForExchange);
    L.S = S;

    if (c.Rc > 1 && c.ctas_per_chain == 0) {
        L.cpc = 1;
        L.nteams = std::min(c.Rc, max_clusters);
    } else {
        int cpc;
        if (c.ctas_per_chain) {
            if (c.ctas_per_chain % S != 0) return BMGD_ERR_ARG;
            cpc = c.ctas_per_chain / S;
        } else {
            const int sp1 = (n + S * spp - 1) / (S * spp);  // sub-passes per step with a single cluster
            cpc = sp1 <= 6 ? 1 : std::min(max_clusters, (sp1 + 1) / 2);
        }
        cpc = std::max(1, std::min(cpc, bmgdk::kMaxCpc));
        if (cpc > max_clusters) return BMGD_ERR_LAUNCH;
        L.cpc = cpc;
        L.nteams = std::max(1, std::min(c.Rc, max_clusters / cpc));
    }
    // a chain that spans clusters keeps only its slice of the peers' packets in shared memory: more room for rows
    const bool multi = L.cpc > 1;
    fixed_smem = bmgdk::glm_smem_plan(warps, gpw, pre, 1, 0, pcap, eb, S, multi, gathered).total_bytes;
    ring_budget = h->smem_optin - fixed_smem - 1024;  // all of the CTA's shared memory but a small reserve
    const int G = L.cpc * S;
    const int rows_per_cta = (n + G - 1) / G;
    const int subpasses = std::max(1, (rows_per_cta + spp - 1) / spp);

    // sub-passes per ring stage: two or more let a group keep two rows in flight and amortise the per-stage
    // bookkeeping; measured on B200, two stages of two sub-passes beat four stages of one when rows come from L2
    auto stage_bytes_of = [&](int r) { return bmgdk::glm_smem_plan(warps, gpw, pre, r, 1, pcap, eb, S, multi, gathered).stage_bytes; };
    // narrow rows (at most 32 bytes per lane) are swept four sub-passes at a time by the kernel, others two
    int rb = c.subpasses_per_stage ? c.subpasses_per_stage : ((var->kch * 16 <= 32) ? 4 : 2);
    rb = floor_pow2(std::max(1, std::min(rb, subpasses)));
    int shared_pwarps = 0;  // gathered rows: producer warps, all of which work on every stage
    if (gathered) {
        shared_pwarps = std::min(c.producer_warps ? c.producer_warps : 4, max_pwarps);
        // a producer warp takes at most kMaxBatchesPerProducer batches of 32 row slots per stage
        while (rb > 1 && rb * spp > 32 * bmgdk::kMaxBatchesPerProducer * shared_pwarps) rb /= 2;
        if (spp > 32 * bmgdk::kMaxBatchesPerProducer * shared_pwarps) return BMGD_ERR_ARG;
    }
    while (rb > 1 && 2 * stage_bytes_of(rb) > ring_budget) rb /= 2;
    L.rb = rb;
    L.passes = (subpasses + rb - 1) / rb;
    const int stage_bytes = stage_bytes_of(rb);
    // ring stages: 2 to 8.  Where partial sums cross clusters through global memory, copies in flight for later steps
    // delay the packets on the same path (measured on B200: cfg3 4.8 us per step with two stages, 5.7 with three).
    int depth = c.pipeline_depth ? c.pipeline_depth : (L.cpc > 1 ? 2 : 4);
    if (!gathered) depth = std::min(depth, max_pwarps);  // one producer warp per ring slot at least
    while (depth > 2 && depth * stage_bytes > ring_budget) --depth;
    if (depth * stage_bytes > ring_budget) return BMGD_ERR_UNIMPLEMENTED;
    L.depth = depth;
    if (gathered) {
        L.pwarps = shared_pwarps;
    } else {  // a multiple of the ring depth (cfg.producer_warps is rounded down to one; default: one per slot)
        const int per_slot = std::max(1, std::min(c.producer_warps ? c.producer_warps : depth, max_pwarps) / depth);
        L.pwarps = per_slot * depth;
    }
    L.smem = bmgdk::glm_smem_plan(warps, gpw, pre, rb, depth, pcap, eb, S, multi, gathered).total_bytes;
    (void)rows;
    *out = L;
    return BMGD_OK;
}

int take_events(bmgd* h, EventPair* ep) {
    if (!h->event_pool.empty()) {
        *ep = h->event_pool.back();
        h->event_pool.pop_back();
        return BMGD_OK;
    }
    BMGD_CUDA(h, cudaEventCreate(&ep->a));
    BMGD_CUDA(h, cudaEventCreate(&ep->b));
    return BMGD_OK;
}

int drain_events(bmgd* h, std::vector<EventPair>& v, double* acc) {
    for (EventPair& ep : v) {
        float ms = 0.f;
        BMGD_CUDA(h, cudaEventSynchronize(ep.b));
        BMGD_CUDA(h, cudaEventElapsedTime(&ms, ep.a, ep.b));
        *acc += ms;
        h->event_pool.push_back(ep);
    }
    v.clear();
    return BMGD_OK;
}

int check_status_word(bmgd* h) {
    int st[2] = {0, 0};
    BMGD_CUDA(h, cudaMemcpy(st, h->base + h->lay.status, sizeof st, cudaMemcpyDeviceToHost));
    if (st[0] != 0 || st[1] != 0) {
        // report once, then clear so that the handle stays usable
        cudaMemset(h->base + h->lay.status, 0, kAlign);
        return st[0] != 0 ? st[0] : BMGD_ERR_TIMEOUT;
    }
    return BMGD_OK;
}

// null_step: launch the latency probe of the same shape instead (dx and dy are not read; theta and the update rule's
// state stay as they are).
int run_glm(bmgd* h, const void* dx, const void* dy, int64_t rows, int rounds, int n, double lr, uint64_t seed,
            bool null_step = false) {
    const bmgd_config& c = h->cfg;
    const bool aligned16 = ((int64_t)c.p * h->tb) % 16 == 0 && ((uintptr_t)dx % 16) == 0;
    const GlmVariant* var = pick_variant(c.dtype, c.loss, c.p, aligned16, c.lanes_per_row, null_step);
    if (!var) return BMGD_ERR_UNIMPLEMENTED;
    if (((uintptr_t)dx % h->tb) != 0 || ((uintptr_t)dy % h->tb) != 0) return BMGD_ERR_ARG;
    LaunchShape L{};
    int rc = plan_glm(h, var, rows, n, &L);
    if (rc != BMGD_OK) return rc;

    const uint32_t M = (uint32_t)((rows + n - 1) / n);
    const int chains_per_team = (c.Rc + L.nteams - 1) / L.nteams;
    const uint64_t steps_per_team = (uint64_t)chains_per_team * (uint64_t)rounds * M;
    if (steps_per_team * (uint64_t)L.passes >= 0xFFFFFFF0ull) return BMGD_ERR_ARG;
    if (h->tag_base + steps_per_team >= 0xFFFFFFF0ull) {
        // tags would wrap: wipe the packet area (on-stream, after earlier launches) and start over
        BMGD_CUDA(h, cudaMemsetAsync(h->base + h->lay.ll, 0, (size_t)(h->lay.status - h->lay.ll), h->compute));
        h->tag_base = 0;
    }

    GlmParams P{};
    P.X = dx; P.y = dy;
    P.theta = h->base + h->lay.theta;
    P.ll = reinterpret_cast<unsigned long long*>(h->base + h->lay.ll);
    P.status = reinterpret_cast<int*>(h->base + h->lay.status);
    P.seed = seed;
    P.timeout_ns = h->timeout_ns;
    P.scale_full = lr / (double)n;
    P.scale_last = lr / (double)(rows - (int64_t)(M - 1) * n);
    P.lr = lr;
    P.inv_full = 1.0 / (double)n;
    P.inv_last = 1.0 / (double)(rows - (int64_t)(M - 1) * n);
    P.opt1 = h->base + h->lay.opt1; P.opt2 = h->base + h->lay.opt2;
    P.opt_kind = h->opt_kind; P.opt_a = h->opt_a; P.opt_b = h->opt_b; P.opt_eps = h->opt_eps;
    P.adam_b1pow0 = std::pow(h->opt_a, (double)h->opt_steps);
    P.adam_b2pow0 = std::pow(h->opt_b, (double)h->opt_steps);
    P.sched = h->sched; P.sched_period = h->sched_period; P.sched_pos0 = h->sched_pos;
    if (null_step) { P.opt_kind = bmgdk::kOptSgd; P.sched = bmgdk::kLrConstant; }  // a zero gradient under Eq. (2.1): nothing changes
    P.N0 = (uint32_t)rows; P.n = (uint32_t)n; P.M = M; P.T = rounds; P.p = c.p;
    P.Rc = c.Rc; P.S = L.S; P.cpc = L.cpc; P.nteams = L.nteams;
    P.passes = L.passes; P.rb = L.rb; P.depth = L.depth;
    P.consumer_warps = L.threads / 32; P.producer_warps = L.pwarps;
    P.q_full = (uint32_t)n / (uint32_t)(L.cpc * L.S); P.r_full = (uint32_t)n % (uint32_t)(L.cpc * L.S);
    P.ll_stride = c.p * 2;
    P.tag_base = (uint32_t)h->tag_base;
    P.chain0 = (uint32_t)c.first_chain;
    P.fixed_partition = (c.flags & BMGD_FLAG_FIXED_PARTITION) ? 1 : 0;
    set_poll_cadence(&P);
#ifdef BMGD_TRACE
    P.trace = bmgdk::trace_buffer(0); P.ptrace = bmgdk::trace_buffer(1);
#endif
    if ((int64_t)L.nteams * L.cpc > kMaxClustersForExchange) return BMGD_ERR_LAUNCH;

    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3((unsigned)(L.nteams * L.cpc * L.S), 1, 1);
    lc.blockDim = dim3((unsigned)(L.threads + 32 * L.pwarps), 1, 1);
    lc.dynamicSmemBytes = (size_t)L.smem;
    lc.stream = h->compute;
    cudaLaunchAttribute at[2];
    int na = 0;
    if (L.S > 1) {
        at[na].id = cudaLaunchAttributeClusterDimension;
        at[na].val.clusterDim.x = (unsigned)L.S; at[na].val.clusterDim.y = 1; at[na].val.clusterDim.z = 1;
        ++na;
    }
    if (L.cpc > 1) {  // CTAs of different clusters wait on one another: they must all be resident
        at[na].id = cudaLaunchAttributeCooperative;
        at[na].val.cooperative = 1;
        ++na;
    }
    lc.attrs = at; lc.numAttrs = (unsigned)na;

    EventPair ep{};
    const bool timing = (c.flags & BMGD_FLAG_TIMING) != 0;
    if (timing) {
        rc = take_events(h, &ep);
        if (rc != BMGD_OK) return rc;
        BMGD_CUDA(h, cudaEventRecord(ep.a, h->compute));
    }
    CUtensorMap xmap;
    std::memset(&xmap, 0, sizeof xmap);
    if (!null_step && bmgdk::glm_gathered(var->vec * h->tb, var->cap())) {
        rc = make_row_map(dx, rows, c.p, h->tb, var->cap(), &xmap);
        if (rc != BMGD_OK) {
            if (timing) h->event_pool.push_back(ep);
            return rc;
        }
    }
    cudaError_t e = cudaLaunchKernelEx(&lc, var->fn(L.threads + 32 * L.pwarps, bmgdk::glm_flavour(P.opt_kind, P.sched, L.cpc)), P, xmap);
    if (e != cudaSuccess) {
        h->last_cuda = (int)e;
        cudaGetLastError();
        if (timing) h->event_pool.push_back(ep);
        return (e == cudaErrorCooperativeLaunchTooLarge || e == cudaErrorLaunchOutOfResources) ? BMGD_ERR_LAUNCH
                                                                                                : BMGD_ERR_CUDA;
    }
    if (timing) {
        BMGD_CUDA(h, cudaEventRecord(ep.b, h->compute));
        h->kernel_events.push_back(ep);
    }
    h->tag_base += steps_per_team;
    h->stats.launches += 1;
    if (!null_step) {
        h->opt_steps += (int64_t)rounds * M;
        if (h->sched == BMGD_LR_COSINE) h->sched_pos = (h->sched_pos + (int64_t)rounds * M) % h->sched_period;
        h->stats.steps += (int64_t)c.Rc * rounds * M;
        h->stats.sample_grads += (int64_t)c.Rc * rounds * rows;
    }
    h->stats.grid_ctas = L.nteams * L.cpc * L.S;
    h->stats.cluster_size = L.S;
    h->stats.ctas_per_chain = L.cpc * L.S;
    h->stats.threads_per_cta = L.threads + 32 * L.pwarps;
    h->stats.pipeline_depth = L.depth;
    h->stats.subpasses_per_stage = L.rb;
    h->stats.smem_bytes = L.smem;
    h->stats.chains_in_flight = L.nteams;
    return BMGD_OK;
}

int run_softmax(bmgd* h, const void* dx, const void* dy, int64_t rows, int rounds, int n, double lr, uint64_t seed, bool null_step) {
    bmgdk::SoftmaxLaunchInfo info{};
    EventPair ep{};
    const bool timing = (h->cfg.flags & BMGD_FLAG_TIMING) != 0;
    if (timing) {
        int rc = take_events(h, &ep);
        if (rc != BMGD_OK) return rc;
        BMGD_CUDA(h, cudaEventRecord(ep.a, h->compute));
    }
    int rc = bmgdk::softmax_run(dx, dy, rows, h->cfg.p, h->cfg.C, h->cfg.Rc, (uint32_t)h->cfg.first_chain, h->base + h->lay.theta,
                               reinterpret_cast<int*>(h->base + h->lay.status), rounds, n, lr, seed,
                               (h->cfg.flags & BMGD_FLAG_FIXED_PARTITION) ? 1 : 0, h->timeout_ns, h->cfg.cluster_size,
                               (h->cfg.flags & BMGD_FLAG_SOFTMAX_CUDA_CORES) ? 1 : 0, null_step ? 1 : 0, h->smem_optin,
                               h->compute, &info);
    if (rc != BMGD_OK) {
        if (info.cuda_error) h->last_cuda = info.cuda_error;
        if (timing) h->event_pool.push_back(ep);
        return rc;
    }
    if (timing) {
        BMGD_CUDA(h, cudaEventRecord(ep.b, h->compute));
        h->kernel_events.push_back(ep);
    }
    const int64_t M = (rows + n - 1) / n;
    h->stats.launches += info.launches;
    if (!null_step) {
        h->stats.steps += (int64_t)h->cfg.Rc * rounds * M;
        h->stats.sample_grads += (int64_t)h->cfg.Rc * rounds * rows;
    }
    h->stats.grid_ctas = info.grid_ctas;
    h->stats.cluster_size = info.cluster_size;
    h->stats.ctas_per_chain = info.cluster_size;
    h->stats.threads_per_cta = info.threads;
    h->stats.pipeline_depth = info.depth;
    h->stats.subpasses_per_stage = 0;
    h->stats.smem_bytes = info.smem;
    h->stats.chains_in_flight = info.chains_in_flight;
    return BMGD_OK;
}

int run_any(bmgd* h, const void* dx, const void* dy, int64_t rows, int rounds, int n, double lr, uint64_t seed) {
    if (rows <= 0 || rows > 0x7FFFFFFFll || rounds < 0 || n <= 0 || !std::isfinite(lr)) return BMGD_ERR_ARG;
    if (rounds == 0) return BMGD_OK;
    if (n > rows) n = (int)rows;
    if (h->cfg.loss == BMGD_LOSS_SOFTMAX) return run_softmax(h, dx, dy, rows, rounds, n, lr, seed, false);
    return run_glm(h, dx, dy, rows, rounds, n, lr, seed);
}

}  // namespace

// ====================================================================== C ABI

extern "C" {

void bmgd_config_init(bmgd_config* cfg) {
    if (!cfg) return;
    std::memset(cfg, 0, sizeof *cfg);
    cfg->loss = BMGD_LOSS_LINEAR;
    cfg->dtype = BMGD_F32;
    cfg->C = 1;
    cfg->Rc = 1;
    cfg->K = 1;
    cfg->device = -1;
}

int bmgd_workspace_bytes(const bmgd_config* cfg, int64_t* bytes) {
    if (!bytes) return BMGD_ERR_ARG;
    int rc = validate(cfg);
    if (rc != BMGD_OK) return rc;
    *bytes = make_layout(cfg).total;
    return BMGD_OK;
}

int bmgd_create(int64_t N, int32_t p, int32_t K, int32_t loss, bmgd_t** out) {
    bmgd_config cfg;
    bmgd_config_init(&cfg);
    cfg.N = N; cfg.p = p; cfg.K = K; cfg.loss = loss;
    return bmgd_create_ex(&cfg, out);
}

int bmgd_create_ex(const bmgd_config* cfg, bmgd_t** out) {
    if (!out) return BMGD_ERR_ARG;
    int rc = validate(cfg);
    if (rc != BMGD_OK) return rc;
    int dev = cfg->device;
    if (dev < 0 && cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return BMGD_ERR_CUDA; }
    DeviceGuard guard(dev);
    if (!guard.ok) { cudaGetLastError(); return BMGD_ERR_CUDA; }

    bmgd* h = new (std::nothrow) bmgd();
    if (!h) return BMGD_ERR_ALLOC;
    h->cfg = *cfg;
    h->device = dev;
    h->xb = elem_bytes_x(cfg->dtype);
    h->tb = elem_bytes_theta(cfg->dtype);
    h->yb = cfg->loss == BMGD_LOSS_SOFTMAX ? 4 : h->tb;
    h->N0cap = (cfg->N + cfg->K - 1) / cfg->K;
    h->num_slots = (cfg->flags & BMGD_FLAG_NO_SLOTS) ? 0 : 2;
    h->timeout_ns = (uint64_t)((cfg->timeout_ms > 0 ? cfg->timeout_ms : 2000.0) * 1e6);
    h->lay = make_layout(cfg);

    auto fail = [&](int code) { bmgd_destroy(h); return code; };
    if (cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&h->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) {
        cudaGetLastError();
        return fail(BMGD_ERR_CUDA);
    }
    if (cfg->workspace) {
        if (cfg->workspace_bytes < h->lay.total) return fail(BMGD_ERR_CAPACITY);
        h->base = static_cast<unsigned char*>(cfg->workspace);
    } else {
        void* p = nullptr;
        if (cudaMalloc(&p, (size_t)h->lay.total) != cudaSuccess) { cudaGetLastError(); return fail(BMGD_ERR_ALLOC); }
        h->base = static_cast<unsigned char*>(p);
        h->owns_base = true;
    }
    if (cfg->compute_stream) {
        h->compute = static_cast<cudaStream_t>(cfg->compute_stream);
    } else {
        if (cudaStreamCreateWithFlags(&h->compute, cudaStreamNonBlocking) != cudaSuccess) { cudaGetLastError(); return fail(BMGD_ERR_CUDA); }
        h->owns_stream = true;
    }
    for (int s = 0; s < h->num_slots; ++s) {
        if (cudaEventCreateWithFlags(&h->loaded[s], cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&h->freed[s], cudaEventDisableTiming) != cudaSuccess) {
            cudaGetLastError();
            return fail(BMGD_ERR_CUDA);
        }
    }
    // theta = 0, packet area and status words = 0
    if (cudaMemsetAsync(h->base + h->lay.theta, 0, (size_t)(h->lay.total - h->lay.theta), h->compute) != cudaSuccess ||
        cudaStreamSynchronize(h->compute) != cudaSuccess) {
        cudaGetLastError();
        return fail(BMGD_ERR_CUDA);
    }
    *out = h;
    return BMGD_OK;
}

int bmgd_destroy(bmgd_t* h) {
    if (!h) return BMGD_OK;
    DeviceGuard guard(h->device);
    if (h->compute) cudaStreamSynchronize(h->compute);
    for (int s = 0; s < 2; ++s) {
        if (h->loaded[s]) { cudaEventSynchronize(h->loaded[s]); cudaEventDestroy(h->loaded[s]); }
        if (h->freed[s]) cudaEventDestroy(h->freed[s]);
    }
    auto kill = [](std::vector<EventPair>& v) {
        for (EventPair& ep : v) { cudaEventDestroy(ep.a); cudaEventDestroy(ep.b); }
        v.clear();
    };
    kill(h->kernel_events); kill(h->copy_events); kill(h->event_pool);
    if (h->owns_stream && h->compute) cudaStreamDestroy(h->compute);
    if (h->owns_base && h->base) cudaFree(h->base);
    cudaGetLastError();
    delete h;
    return BMGD_OK;
}

int bmgd_load_buffer(bmgd_t* h, const void* host_x, const void* host_y, int64_t rows, void* stream, int32_t* slot) {
    if (!h || !host_x || !host_y || !slot || rows <= 0) return BMGD_ERR_ARG;
    if (h->num_slots == 0) return BMGD_ERR_STATE;
    if (rows > h->N0cap) return BMGD_ERR_CAPACITY;
    DeviceGuard guard(h->device);
    if (!guard.ok) return cuda_fail(h, cudaErrorInvalidDevice);
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const int s = h->next_slot;
    // the kernel that last read this slot must be done before the slot is overwritten
    if (h->slot_has_data[s]) BMGD_CUDA(h, cudaStreamWaitEvent(cs, h->freed[s], 0));
    EventPair ep{};
    const bool timing = (h->cfg.flags & BMGD_FLAG_TIMING) != 0;
    if (timing) {
        int rc = take_events(h, &ep);
        if (rc != BMGD_OK) return rc;
        BMGD_CUDA(h, cudaEventRecord(ep.a, cs));
    }
    const size_t xbytes = (size_t)rows * h->cfg.p * h->xb, ybytes = (size_t)rows * h->yb;
    BMGD_CUDA(h, cudaMemcpyAsync(h->base + h->lay.slot_x[s], host_x, xbytes, cudaMemcpyHostToDevice, cs));
    BMGD_CUDA(h, cudaMemcpyAsync(h->base + h->lay.slot_y[s], host_y, ybytes, cudaMemcpyHostToDevice, cs));
    if (timing) {
        BMGD_CUDA(h, cudaEventRecord(ep.b, cs));
        h->copy_events.push_back(ep);
    }
    BMGD_CUDA(h, cudaEventRecord(h->loaded[s], cs));
    h->slot_rows[s] = rows;
    h->slot_has_data[s] = true;
    h->stats.h2d_bytes += (int64_t)(xbytes + ybytes);
    h->next_slot = (s + 1) % h->num_slots;
    *slot = s;
    return BMGD_OK;
}

int bmgd_run_rounds(bmgd_t* h, int32_t slot, int32_t rounds, int32_t batch_size, double lr, uint64_t seed) {
    if (!h) return BMGD_ERR_ARG;
    if (slot < 0 || slot >= h->num_slots) return BMGD_ERR_ARG;
    if (!h->slot_has_data[slot]) return BMGD_ERR_STATE;
    DeviceGuard guard(h->device);
    if (!guard.ok) return cuda_fail(h, cudaErrorInvalidDevice);
    BMGD_CUDA(h, cudaStreamWaitEvent(h->compute, h->loaded[slot], 0));
    int rc = run_any(h, h->base + h->lay.slot_x[slot], h->base + h->lay.slot_y[slot], h->slot_rows[slot], rounds,
                     batch_size, lr, seed);
    if (rc != BMGD_OK) return rc;
    BMGD_CUDA(h, cudaEventRecord(h->freed[slot], h->compute));
    return BMGD_OK;
}

int bmgd_run_rounds_resident(bmgd_t* h, const void* dev_x, const void* dev_y, int64_t rows, int32_t rounds,
                             int32_t batch_size, double lr, uint64_t seed) {
    if (!h || !dev_x || !dev_y) return BMGD_ERR_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return cuda_fail(h, cudaErrorInvalidDevice);
    return run_any(h, dev_x, dev_y, rows, rounds, batch_size, lr, seed);
}

int bmgd_sync(bmgd_t* h) {
    if (!h) return BMGD_ERR_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return cuda_fail(h, cudaErrorInvalidDevice);
    BMGD_CUDA(h, cudaStreamSynchronize(h->compute));
    for (int s = 0; s < h->num_slots; ++s)
        if (h->slot_has_data[s]) BMGD_CUDA(h, cudaEventSynchronize(h->loaded[s]));
    return check_status_word(h);
}

int bmgd_get_theta(bmgd_t* h, void* out_host, int64_t bytes) {
    if (!h || !out_host) return BMGD_ERR_ARG;
    const int64_t want = (int64_t)h->cfg.Rc * h->cfg.p * h->cfg.C * h->tb;
    if (bytes != want) return BMGD_ERR_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return cuda_fail(h, cudaErrorInvalidDevice);
    BMGD_CUDA(h, cudaStreamSynchronize(h->compute));
    int rc = check_status_word(h);
    BMGD_CUDA(h, cudaMemcpy(out_host, h->base + h->lay.theta, (size_t)want, cudaMemcpyDeviceToHost));
    if (rc != BMGD_OK) return rc;
    const int64_t cnt = want / h->tb;
    bool finite = true;
    if (h->tb == 8) { const double* v = static_cast<const double*>(out_host); for (int64_t i = 0; i < cnt; ++i) finite &= std::isfinite(v[i]); }
    else { const float* v = static_cast<const float*>(out_host); for (int64_t i = 0; i < cnt; ++i) finite &= std::isfinite(v[i]); }
    return finite ? BMGD_OK : BMGD_ERR_NONFINITE;
}

int bmgd_set_theta(bmgd_t* h, const void* host, int64_t bytes) {
    if (!h || !host) return BMGD_ERR_ARG;
    const int64_t want = (int64_t)h->cfg.Rc * h->cfg.p * h->cfg.C * h->tb;
    if (bytes != want) return BMGD_ERR_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return cuda_fail(h, cudaErrorInvalidDevice);
    BMGD_CUDA(h, cudaStreamSynchronize(h->compute));
    BMGD_CUDA(h, cudaMemcpy(h->base + h->lay.theta, host, (size_t)want, cudaMemcpyHostToDevice));
    return BMGD_OK;
}

int bmgd_set_optimizer(bmgd_t* h, int32_t kind, double a, double b, double eps) {
    if (!h) return BMGD_ERR_ARG;
    if (kind < BMGD_OPT_SGD || kind > BMGD_OPT_ADAM) return BMGD_ERR_ARG;
    if (kind == BMGD_OPT_NESTEROV && !(a >= 0.0 && a < 1.0)) return BMGD_ERR_ARG;
    if (kind == BMGD_OPT_ADAM && !(a >= 0.0 && a < 1.0 && b >= 0.0 && b < 1.0 && eps > 0.0)) return BMGD_ERR_ARG;
    if (h->cfg.loss == BMGD_LOSS_SOFTMAX) return kind == BMGD_OPT_SGD ? BMGD_OK : BMGD_ERR_UNIMPLEMENTED;
    DeviceGuard guard(h->device);
    if (!guard.ok) return cuda_fail(h, cudaErrorInvalidDevice);
    // the state starts from zero, ordered after the launches already issued
    BMGD_CUDA(h, cudaMemsetAsync(h->base + h->lay.opt1, 0, (size_t)(h->lay.ll - h->lay.opt1), h->compute));
    h->opt_kind = kind; h->opt_a = a; h->opt_b = b; h->opt_eps = eps;
    h->opt_steps = 0;
    return BMGD_OK;
}

int bmgd_set_timeout(bmgd_t* h, double timeout_ms) {
    if (!h || !std::isfinite(timeout_ms)) return BMGD_ERR_ARG;
    h->timeout_ns = (uint64_t)((timeout_ms > 0 ? timeout_ms : 2000.0) * 1e6);
    return BMGD_OK;
}

int bmgd_set_lr_schedule(bmgd_t* h, int32_t kind, int64_t updates_per_pass) {
    if (!h) return BMGD_ERR_ARG;
    if (kind != BMGD_LR_CONSTANT && kind != BMGD_LR_COSINE) return BMGD_ERR_ARG;
    if (kind == BMGD_LR_COSINE && updates_per_pass <= 0) return BMGD_ERR_ARG;
    if (h->cfg.loss == BMGD_LOSS_SOFTMAX) return kind == BMGD_LR_CONSTANT ? BMGD_OK : BMGD_ERR_UNIMPLEMENTED;
    h->sched = kind;
    h->sched_period = kind == BMGD_LR_COSINE ? updates_per_pass : 0;
    h->sched_pos = 0;
    return BMGD_OK;
}

int bmgd_get_stats(bmgd_t* h, bmgd_stats* out) {
    if (!h || !out) return BMGD_ERR_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return cuda_fail(h, cudaErrorInvalidDevice);
    BMGD_CUDA(h, cudaStreamSynchronize(h->compute));
    int rc = drain_events(h, h->kernel_events, &h->stats.kernel_ms);
    if (rc != BMGD_OK) return rc;
    rc = drain_events(h, h->copy_events, &h->stats.h2d_ms);
    if (rc != BMGD_OK) return rc;
    *out = h->stats;
    return check_status_word(h);
}

int bmgd_debug_perm(bmgd_t* h, uint64_t seed, uint32_t chain, uint32_t round, uint32_t N0, uint32_t* out_host) {
    if (!h || !out_host || N0 == 0 || N0 > 0x7FFFFFFFu) return BMGD_ERR_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return cuda_fail(h, cudaErrorInvalidDevice);
    uint32_t* d = nullptr;
    if (cudaMalloc(&d, (size_t)N0 * 4) != cudaSuccess) { cudaGetLastError(); return BMGD_ERR_ALLOC; }
    const int threads = 256;
    const int blocks = (int)std::min<int64_t>(((int64_t)N0 + threads - 1) / threads, (int64_t)h->sm_count * 8);
    bmgdk::perm_kernel<<<blocks, threads, 0, h->compute>>>(seed, chain, round, N0, d);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaMemcpyAsync(out_host, d, (size_t)N0 * 4, cudaMemcpyDeviceToHost, h->compute);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->compute);
    cudaFree(d);
    if (e != cudaSuccess) return cuda_fail(h, e);
    return BMGD_OK;
}

// ---------------------------------------------------------------------------------------------
// Allocation-free variant of the computation step.
//
// The step kernel needs scratch in global memory besides its inputs and outputs: the tagged
// packets through which clusters exchange partial gradients, and two status words.  A handle
// gets that scratch from cudaMalloc or from the caller's workspace.  Here it lives in a fixed
// array that is part of the loaded library image instead.
static __device__ __align__(256) unsigned char g_noalloc_scratch[BMGD_NOALLOC_SCRATCH_BYTES];

namespace {
constexpr int kNoallocMaxDevices = 64;
void* g_noalloc_ptr[kNoallocMaxDevices];  // device address of g_noalloc_scratch, per device ordinal
std::mutex g_noalloc_mutex;

// In host code `g_noalloc_scratch` is only a handle for the symbol; the address a kernel can use
// comes from cudaGetSymbolAddress, asked once per device with that device current.
int noalloc_scratch_for_current_device(int dev, unsigned char** out) {
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess || !p) { cudaGetLastError(); return BMGD_ERR_CUDA; }
        g_noalloc_ptr[dev] = p;
    }
    *out = static_cast<unsigned char*>(g_noalloc_ptr[dev]);
    return BMGD_OK;
}
}  // namespace

int bmgd_run_rounds_noalloc(const void* dev_x, const void* dev_y, int64_t rows, int32_t p, int32_t loss,
                            int32_t dtype, int32_t Rc, void* dev_theta, int32_t rounds, int32_t batch_size,
                            double lr, uint64_t seed, void* stream) {
    if (!dev_x || !dev_y || !dev_theta) return BMGD_ERR_ARG;
    if (loss != BMGD_LOSS_LINEAR && loss != BMGD_LOSS_LOGISTIC) return BMGD_ERR_UNIMPLEMENTED;
    if (dtype != BMGD_F64 && dtype != BMGD_F32) return BMGD_ERR_UNIMPLEMENTED;
    if (p <= 0 || Rc < 1 || Rc > 65536) return BMGD_ERR_ARG;
    if (p > BMGD_NOALLOC_MAX_P) return BMGD_ERR_CAPACITY;  // the fixed scratch holds packets for at most this many predictors
    if (rows <= 0 || rows > 0x7FFFFFFFll || rounds < 0 || batch_size <= 0 || !std::isfinite(lr)) return BMGD_ERR_ARG;
    if (rounds == 0) return BMGD_OK;
    int n = batch_size > rows ? (int)rows : batch_size;

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return BMGD_ERR_CUDA; }
    if (dev < 0 || dev >= kNoallocMaxDevices) return BMGD_ERR_ARG;
    unsigned char* scratch = nullptr;
    int rc = noalloc_scratch_for_current_device(dev, &scratch);
    if (rc != BMGD_OK) return rc;

    // A handle on the stack, never registered anywhere: it only carries what the launch planner reads.
    bmgd tmp;
    bmgd_config_init(&tmp.cfg);
    tmp.cfg.N = rows; tmp.cfg.p = p; tmp.cfg.K = 1; tmp.cfg.loss = loss; tmp.cfg.dtype = dtype; tmp.cfg.Rc = Rc;
    tmp.device = dev;
    tmp.tb = elem_bytes_theta(dtype);
    if (cudaDeviceGetAttribute(&tmp.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&tmp.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) {
        cudaGetLastError();
        return BMGD_ERR_CUDA;
    }
    const int tb = tmp.tb;
    if (((uintptr_t)dev_x % tb) != 0 || ((uintptr_t)dev_y % tb) != 0 || ((uintptr_t)dev_theta % tb) != 0) return BMGD_ERR_ARG;
    const bool aligned16 = ((int64_t)p * tb) % 16 == 0 && ((uintptr_t)dev_x % 16) == 0;
    const GlmVariant* var = pick_variant(dtype, loss, p, aligned16);
    if (!var) return BMGD_ERR_UNIMPLEMENTED;
    LaunchShape L{};
    rc = plan_glm(&tmp, var, rows, n, &L);
    if (rc != BMGD_OK) return rc;

    const uint32_t M = (uint32_t)((rows + n - 1) / n);
    const int chains_per_team = (Rc + L.nteams - 1) / L.nteams;
    if ((uint64_t)chains_per_team * (uint64_t)rounds * M * (uint64_t)L.passes >= 0xFFFFFFF0ull) return BMGD_ERR_ARG;
    if ((int64_t)L.nteams * L.cpc > kMaxClustersForExchange) return BMGD_ERR_LAUNCH;
    const size_t packet_bytes = (size_t)2 * kMaxClustersForExchange * p * 2 * 8;
    if (256 + packet_bytes > (size_t)BMGD_NOALLOC_SCRATCH_BYTES) return BMGD_ERR_CAPACITY;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The array still holds the packets and status of whoever called last: start from zero, so that
    // tag 0 again means "nothing written yet".
    if (cudaMemsetAsync(scratch, 0, 256 + packet_bytes, st) != cudaSuccess) { cudaGetLastError(); return BMGD_ERR_CUDA; }

    GlmParams P{};
    P.X = dev_x; P.y = dev_y;
    P.theta = dev_theta;
    P.status = reinterpret_cast<int*>(scratch);
    P.ll = reinterpret_cast<unsigned long long*>(scratch + 256);
    P.seed = seed;
    P.timeout_ns = 2000000000ull;
    P.scale_full = lr / (double)n;
    P.scale_last = lr / (double)(rows - (int64_t)(M - 1) * n);
    P.lr = lr;
    P.inv_full = 1.0 / (double)n;
    P.inv_last = 1.0 / (double)(rows - (int64_t)(M - 1) * n);
    P.opt_kind = bmgdk::kOptSgd; P.sched = bmgdk::kLrConstant;  // Eq. (2.1) with a constant rate: no state beside theta
    P.N0 = (uint32_t)rows; P.n = (uint32_t)n; P.M = M; P.T = rounds; P.p = p;
    P.Rc = Rc; P.S = L.S; P.cpc = L.cpc; P.nteams = L.nteams;
    P.passes = L.passes; P.rb = L.rb; P.depth = L.depth;
    P.consumer_warps = L.threads / 32; P.producer_warps = L.pwarps;
    P.q_full = (uint32_t)n / (uint32_t)(L.cpc * L.S); P.r_full = (uint32_t)n % (uint32_t)(L.cpc * L.S);
    P.ll_stride = p * 2;
    P.tag_base = 0;
    P.fixed_partition = 0;
    set_poll_cadence(&P);

    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3((unsigned)(L.nteams * L.cpc * L.S), 1, 1);
    lc.blockDim = dim3((unsigned)(L.threads + 32 * L.pwarps), 1, 1);
    lc.dynamicSmemBytes = (size_t)L.smem;
    lc.stream = st;
    cudaLaunchAttribute at[2];
    int na = 0;
    if (L.S > 1) {
        at[na].id = cudaLaunchAttributeClusterDimension;
        at[na].val.clusterDim.x = (unsigned)L.S; at[na].val.clusterDim.y = 1; at[na].val.clusterDim.z = 1;
        ++na;
    }
    if (L.cpc > 1) {
        at[na].id = cudaLaunchAttributeCooperative;
        at[na].val.cooperative = 1;
        ++na;
    }
    lc.attrs = at; lc.numAttrs = (unsigned)na;
    CUtensorMap xmap;  // encoded on the host, passed by value: no allocation
    std::memset(&xmap, 0, sizeof xmap);
    if (bmgdk::glm_gathered(var->vec * tb, var->cap())) {
        rc = make_row_map(dev_x, rows, p, tb, var->cap(), &xmap);
        if (rc != BMGD_OK) return rc;
    }
    cudaError_t e = cudaLaunchKernelEx(&lc, var->fn(L.threads + 32 * L.pwarps, bmgdk::glm_flavour(P.opt_kind, P.sched, L.cpc)), P, xmap);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return (e == cudaErrorCooperativeLaunchTooLarge || e == cudaErrorLaunchOutOfResources) ? BMGD_ERR_LAUNCH : BMGD_ERR_CUDA;
    }
    // Wait for the kernel and read its status words back into a local: no other call could report them.
    int status[2] = {0, 0};
    if (cudaMemcpyAsync(status, scratch, sizeof status, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return BMGD_ERR_CUDA;
    }
    if (status[0] != 0) return status[0];
    if (status[1] != 0) return BMGD_ERR_TIMEOUT;
    return BMGD_OK;
}

// ---------------------------------------------------------------------------------------------
// Partition of the whole sample into buffers (Algorithm 1, line 2) and the CPU side of the buffering step
// (line 3): gather the rows of one buffer of one pass into a staging buffer, with host threads.

int bmgd_partition_index(uint64_t seed, uint32_t pass, int64_t N, int64_t j, int64_t* row) {
    if (!row || N <= 0 || N > 0x7FFFFFFFll || j < 0 || j >= N) return BMGD_ERR_ARG;
    const bmgdk::FeistelDomain dom = bmgdk::make_domain((uint32_t)N);
    const bmgdk::RoundKeys rk = bmgdk::round_keys(seed, 0xFFFFFFFFu, pass);
    *row = (int64_t)bmgdk::perm_index((uint32_t)j, dom, rk);
    return BMGD_OK;
}

int bmgd_gather_buffer(const void* host_x, const void* host_y, int64_t N, int64_t row_bytes, int64_t y_bytes,
                       int32_t K, uint64_t seed, uint32_t pass, int32_t k, void* stage_x, void* stage_y,
                       int32_t threads, int64_t* rows_out) {
    if (!host_x || !host_y || !stage_x || !stage_y || !rows_out) return BMGD_ERR_ARG;
    if (N <= 0 || N > 0x7FFFFFFFll || row_bytes <= 0 || y_bytes <= 0 || K <= 0 || K > N || k < 0 || k >= K) return BMGD_ERR_ARG;
    const int64_t N0 = (N + K - 1) / K;
    const int64_t first = (int64_t)k * N0;
    const int64_t rows = std::max<int64_t>(0, std::min(N0, N - first));
    *rows_out = rows;
    if (rows == 0) return BMGD_OK;
    const bmgdk::FeistelDomain dom = bmgdk::make_domain((uint32_t)N);
    const bmgdk::RoundKeys rk = bmgdk::round_keys(seed, 0xFFFFFFFFu, pass);
    const unsigned char* sx = static_cast<const unsigned char*>(host_x);
    const unsigned char* sy = static_cast<const unsigned char*>(host_y);
    unsigned char* dx = static_cast<unsigned char*>(stage_x);
    unsigned char* dy = static_cast<unsigned char*>(stage_y);
    auto work = [&](int64_t lo, int64_t hi) {
        for (int64_t i = lo; i < hi; ++i) {
            const size_t src = (size_t)bmgdk::perm_index((uint32_t)(first + i), dom, rk);
            std::memcpy(dx + (size_t)i * row_bytes, sx + src * (size_t)row_bytes, (size_t)row_bytes);
            std::memcpy(dy + (size_t)i * y_bytes, sy + src * (size_t)y_bytes, (size_t)y_bytes);
        }
    };
    int nt = threads > 0 ? threads : (int)std::thread::hardware_concurrency();
    nt = (int)std::max<int64_t>(1, std::min<int64_t>(nt, rows / 1024 + 1));
    if (nt == 1) { work(0, rows); return BMGD_OK; }
    std::vector<std::thread> pool;
    try {
        for (int t = 0; t < nt; ++t) pool.emplace_back(work, rows * t / nt, rows * (t + 1) / nt);
    } catch (...) {
        for (auto& th : pool) th.join();
        return BMGD_ERR_ALLOC;
    }
    for (auto& th : pool) th.join();
    return BMGD_OK;
}

int bmgd_debug_null_rounds(bmgd_t* h, int64_t rows, int32_t rounds, int32_t batch_size) {
    if (!h) return BMGD_ERR_ARG;
    if (rows <= 0 || rows > 0x7FFFFFFFll || rounds < 0 || batch_size <= 0) return BMGD_ERR_ARG;
    if (rounds == 0) return BMGD_OK;
    DeviceGuard guard(h->device);
    if (!guard.ok) return cuda_fail(h, cudaErrorInvalidDevice);
    const int n = batch_size > rows ? (int)rows : batch_size;
    if (h->cfg.loss == BMGD_LOSS_SOFTMAX) return run_softmax(h, h->base, h->base, rows, rounds, n, 0.0, 0, true);
    // the probe reads no rows; the workspace base stands in for an aligned buffer address
    return run_glm(h, h->base, h->base, rows, rounds, n, 0.0, 0, true);
}

int bmgd_debug_wait_timeout(bmgd_t* h, double budget_ms) {
    if (!h || !(budget_ms > 0) || budget_ms > 1000.0) return BMGD_ERR_ARG;
    if (h->cfg.loss == BMGD_LOSS_SOFTMAX) return BMGD_ERR_UNIMPLEMENTED;
    DeviceGuard guard(h->device);
    if (!guard.ok) return cuda_fail(h, cudaErrorInvalidDevice);
    // tag 0xFFFFFFFF is never written: the host keeps step tags below 0xFFFFFFF0
    bmgdk::wait_probe_kernel<<<1, 1, 0, h->compute>>>(reinterpret_cast<const unsigned long long*>(h->base + h->lay.ll),
                                                    0xFFFFFFFFu, (unsigned long long)(budget_ms * 1e6),
                                                    reinterpret_cast<int*>(h->base + h->lay.status));
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(h, e);
    return BMGD_OK;
}

const char* bmgd_strerror(int status) {
    switch (status) {
        case BMGD_OK: return "ok";
        case BMGD_ERR_ARG: return "invalid argument";
        case BMGD_ERR_ALLOC: return "out of memory";
        case BMGD_ERR_CUDA: return "CUDA runtime error";
        case BMGD_ERR_CAPACITY: return "more rows than the slot or workspace holds";
        case BMGD_ERR_TIMEOUT: return "a device-side wait ran out of time";
        case BMGD_ERR_NONFINITE: return "theta is not finite";
        case BMGD_ERR_LAUNCH: return "the grid cannot be made co-resident";
        case BMGD_ERR_UNIMPLEMENTED: return "no kernel for this loss, type or shape";
        case BMGD_ERR_STATE: return "call out of order";
        default: return "unknown status";
    }
}

int bmgd_last_cuda_error(const bmgd_t* h) { return h ? h->last_cuda : 0; }

#ifdef BMGD_TRACE
}  // extern "C"
namespace bmgdk {
// Debug build only: the two stamp arrays, allocated and zeroed on the device that is current at the first call (the
// trace reader works on one device).  Null if that fails: the kernels then take no stamps.
long long* trace_buffer(int which) {
    static long long* buf[2] = {nullptr, nullptr};
    static std::once_flag once;
    std::call_once(once, [] {
        const size_t bytes = sizeof(long long) * (size_t)kTraceBlocks * kTraceSteps * kTracePhases;
        for (int i = 0; i < 2; ++i) {
            void* ptr = nullptr;
            if (cudaMalloc(&ptr, bytes) != cudaSuccess || cudaMemset(ptr, 0, bytes) != cudaSuccess) { cudaGetLastError(); ptr = nullptr; }
            buf[i] = static_cast<long long*>(ptr);
        }
    });
    return (which == 0 || which == 1) ? buf[which] : nullptr;
}
}  // namespace bmgdk
extern "C" {
// Debug build only: copy out the clock stamps [block][step][phase] that thread 0 of every CTA took at the phase
// boundaries of its first steps (which = 0), or those of every CTA's first producer warp (which = 1).
int bmgd_debug_trace(int which, long long* out_host, int count) {
    const int total = bmgdk::kTraceBlocks * bmgdk::kTraceSteps * bmgdk::kTracePhases;
    if (!out_host || count <= 0 || count > total || which < 0 || which > 1) return BMGD_ERR_ARG;
    const long long* src = bmgdk::trace_buffer(which);
    if (!src) return BMGD_ERR_CUDA;
    cudaError_t e = cudaMemcpy(out_host, src, sizeof(long long) * (size_t)count, cudaMemcpyDeviceToHost);
    return e == cudaSuccess ? BMGD_OK : BMGD_ERR_CUDA;
}
int bmgd_debug_trace_dims(int* blocks, int* steps, int* phases) {
    if (!blocks || !steps || !phases) return BMGD_ERR_ARG;
    *blocks = bmgdk::kTraceBlocks; *steps = bmgdk::kTraceSteps; *phases = bmgdk::kTracePhases;
    return BMGD_OK;
}
#endif

int bmgd_version(void) { return kVersion; }

}  // extern "C"
