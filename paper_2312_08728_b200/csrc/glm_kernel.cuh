// Fused persistent step kernel for least-squares and logistic BMGD (Algorithm 1, inner loops;
// Eq. (2.1)).  One launch runs every round and every mini-batch step of one call.
//
// Work split.  A chain (one theta) is worked on by a team of `cpc` thread-block clusters of `S`
// CTAs, G = cpc*S CTAs in all; the rows of a mini-batch are dealt out evenly among them.  With
// replicate chains there are several teams, each taking chains team, team+nteams, ...
//
// Per step, in every CTA:
//   1. rows pi(j) of this CTA's share were prefetched into a shared-memory ring by cp.async,
//      several stages ahead (rows do not depend on theta, the shuffle is stateless); each lane
//      evaluates pi for one row and the warp shares the 32 results by shuffle; the copies for a
//      later stage are issued while the CTA would otherwise wait at a barrier;
//   2. a group of LPR lanes owns one row: x.theta by an LPR-lane butterfly, the residual
//      (x.theta - y, or sigmoid(x.theta) - y), then g += r * x with x still in registers, so a
//      row is read from HBM once and from shared memory once;
//   3. the group partials are summed in fixed order (shuffles, then shared memory).  With one
//      cluster per chain every CTA pushes its partial to every peer through distributed shared
//      memory and one cluster barrier follows.  With several clusters the partials are
//      reduce-scattered inside the cluster (CTA r owns a slice of the predictors), the slice sums
//      cross clusters as tagged 8-byte packets in global memory (value and step tag travel in one
//      64-bit store, so a reader needs no separate flag or fence; only the slice owner polls), and
//      the totals are pushed back to every peer before a second cluster barrier;
//   4. every CTA applies theta <- theta - (alpha/n_m) g to its own register copy of theta.
// All sums have a fixed order, so all CTAs hold bit-identical theta and runs are reproducible.
//
// Every wait on another CTA is bounded: when the budget runs out the kernel records
// BMGD_ERR_TIMEOUT in the status word, stops waiting for the rest of the launch (barriers stay
// matched) and returns.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "shuffle.cuh"

namespace bmgdk {

constexpr int kMaxCpc = 20;        // clusters per chain the packet exchange is unrolled for
constexpr int kStatusTimeout = -5; // == BMGD_ERR_TIMEOUT

struct GlmParams {
    const void* X;        // [N0][p] rows
    const void* y;        // [N0]
    void* theta;          // [Rc][p]
    unsigned long long* ll;  // packets: [team][2][cpc][ll_stride]
    int* status;          // [0] first error code, [1] abort flag
    unsigned long long seed;
    unsigned long long timeout_ns;
    double scale_full;    // alpha / n: step size over a full mini-batch
    double scale_last;    // alpha / (size of the ragged last mini-batch of a round)
    uint32_t N0;
    uint32_t n;           // mini-batch size
    uint32_t M;           // mini-batches per round
    int T;                // rounds
    int p;
    int Rc;
    int S;                // cluster size
    int cpc;              // clusters per chain
    int nteams;
    int passes;           // ring stages per step
    int rb;               // sub-passes per ring stage (a power of two, at most LPR)
    int depth;            // ring stages in flight: 2, 3 or 4
    uint32_t q_full, r_full;  // n / G and n % G: how a full mini-batch is dealt to the G CTAs
    int ll_stride;        // packets per cluster slot
    uint32_t tag_base;
    int fixed_partition;
    int bulk_rows;        // rows travel as one bulk copy each (cp.async.bulk) instead of 16-byte cp.async chunks
};

// ---------------------------------------------------------------- small PTX wrappers

template <int BYTES>
__device__ __forceinline__ void cp_async(uint32_t dst_smem, const void* src) {
    if constexpr (BYTES == 16)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_smem), "l"(src) : "memory");
    else if constexpr (BYTES == 8)
        asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst_smem), "l"(src) : "memory");
    else
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst_smem), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// cp.async.wait_group takes an immediate: the ring is 2, 3 or 4 stages deep.
__device__ __forceinline__ void cp_async_wait_ring(int depth) {
    if (depth == 4) asm volatile("cp.async.wait_group 3;" ::: "memory");
    else if (depth == 3) asm volatile("cp.async.wait_group 2;" ::: "memory");
    else asm volatile("cp.async.wait_group 1;" ::: "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

// One predicated copy chunk at a constant byte offset from both addresses.
template <int BYTES, int OFF>
__device__ __forceinline__ void cp_async_at(uint32_t dst_smem, const void* src, uint32_t pred) {
    if constexpr (BYTES == 16)
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %2, 0;\n\t@p cp.async.cg.shared.global [%0+%3], [%1+%3], 16;\n\t}"
                     ::"r"(dst_smem), "l"(src), "r"(pred), "n"(OFF) : "memory");
    else if constexpr (BYTES == 8)
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %2, 0;\n\t@p cp.async.ca.shared.global [%0+%3], [%1+%3], 8;\n\t}"
                     ::"r"(dst_smem), "l"(src), "r"(pred), "n"(OFF) : "memory");
    else
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %2, 0;\n\t@p cp.async.ca.shared.global [%0+%3], [%1+%3], 4;\n\t}"
                     ::"r"(dst_smem), "l"(src), "r"(pred), "n"(OFF) : "memory");
}
template <int BYTES, int STRIDE, int K, int KCH>
__device__ __forceinline__ void cp_async_chunks(uint32_t dst_smem, const void* src, uint32_t kmask) {
    if constexpr (K < KCH) {
        cp_async_at<BYTES, K * STRIDE>(dst_smem, src, kmask & (1u << K));
        cp_async_chunks<BYTES, STRIDE, K + 1, KCH>(dst_smem, src, kmask);
    }
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t cta) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(cta));
    return r;
}
__device__ __forceinline__ void st_cluster(uint32_t addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void st_shared_zero16(uint32_t addr) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0) : "memory");
}
__device__ __forceinline__ void st_cluster(uint32_t addr, double v) {
    asm volatile("st.shared::cluster.f64 [%0], %1;" ::"r"(addr), "d"(v) : "memory");
}
__device__ __forceinline__ void cluster_arrive_release() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait_acquire() {
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// ---- mbarriers (8 bytes of shared memory each) and bulk copies
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// the arrival happens once every cp.async this thread has issued so far has landed
__device__ __forceinline__ void mbar_arrive_after_copies(uint32_t bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
// generic-proxy writes to shared memory become ordered with the bulk copies' writes and the tensor core's reads
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// one row, global -> shared, completion counted in bytes on `bar`; addresses and size are 16-byte multiples
__device__ __forceinline__ void bulk_copy_row(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

__device__ __forceinline__ void st_packet(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long ld_packet(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ float sigmoid_of(float u) { return __fdividef(1.0f, 1.0f + __expf(-u)); }
__device__ __forceinline__ double sigmoid_of(double u) { return 1.0 / (1.0 + exp(-u)); }

// 32-bit words of a value, for the tagged packets
template <typename T> struct Words;
template <> struct Words<float> {
    static constexpr int N = 1;
    __device__ static uint32_t get(float v, int) { return __float_as_uint(v); }
    __device__ static float make(const uint32_t* w) { return __uint_as_float(w[0]); }
};
template <> struct Words<double> {
    static constexpr int N = 2;
    __device__ static uint32_t get(double v, int i) {
        const unsigned long long b = (unsigned long long)__double_as_longlong(v);
        return i == 0 ? (uint32_t)b : (uint32_t)(b >> 32);
    }
    __device__ static double make(const uint32_t* w) {
        return __longlong_as_double((long long)(((unsigned long long)w[1] << 32) | w[0]));
    }
};

// ---------------------------------------------------------------- shared-memory plan (host and device agree on it)

struct GlmSmemPlan {
    int pitch;             // bytes from one ring row to the next: the full predictor capacity, then 16 bytes for y
    int warp_stage_bytes;  // one warp's share of one ring stage
    int ring_off, ring_bytes;
    int gpart_rows;        // partial-gradient rows summed per CTA
    int gpart_off, cpart_off, gfin_off;
    int total_bytes;
};

__host__ __device__ inline GlmSmemPlan glm_smem_plan(int warps, int gpw, bool prereduce, int rb, int depth, int pcap,
                                                     int elem_bytes, int S) {
    GlmSmemPlan s;
    s.pitch = pcap * elem_bytes + 16;
    s.warp_stage_bytes = rb * gpw * s.pitch;
    s.ring_off = 1024;  // room for one mbarrier per (warp, stage) in front of the ring
    s.ring_bytes = warps * depth * s.warp_stage_bytes;
    s.gpart_rows = prereduce ? warps : warps * gpw;
    s.gpart_off = s.ring_off + s.ring_bytes;
    s.cpart_off = s.gpart_off + s.gpart_rows * pcap * elem_bytes;
    s.gfin_off = s.cpart_off + 2 * S * pcap * elem_bytes;
    s.total_bytes = s.gfin_off + pcap * elem_bytes;
    return s;
}

#ifdef BMGD_TRACE
// Debug build only: clock stamps of one CTA at the phase boundaries of its first steps.
#ifndef BMGD_TRACE_BLOCK
#define BMGD_TRACE_BLOCK 0
#endif
constexpr int kTraceSteps = 64, kTracePhases = 16;
__device__ long long g_trace[kTraceSteps * kTracePhases];
#define BMGD_STAMP(ph)                                                                              \
    do {                                                                                            \
        if (blockIdx.x == BMGD_TRACE_BLOCK && threadIdx.x == 0 && step_count < (uint32_t)kTraceSteps) \
            g_trace[step_count * kTracePhases + (ph)] = clock64();                                  \
    } while (0)
#else
#define BMGD_STAMP(ph) do { } while (0)
#endif

// ---------------------------------------------------------------- the kernel

// Largest CTA a variant is compiled for: wide per-lane state (or fp64) needs the 255-register budget.
template <typename T, int VEC, int KCH>
__host__ __device__ constexpr int glm_max_threads() {
    return (sizeof(T) == 8 || KCH * VEC >= 32) ? 256 : 512;
}
// Few values per lane: fold the row groups of a warp together by shuffles before shared memory.
template <int VEC, int KCH>
__host__ __device__ constexpr bool glm_prereduce() {
    return KCH * VEC <= 16;
}

// How mini-batch rows [lo, lo+nm) are dealt to CTA g of G: a contiguous run of `cnt` rows from lo+a.
// nsp is the number of sub-passes of the step in which the calling warp has at least one row.
struct RowShare {
    uint32_t lo, a, cnt, nsp;
};
__device__ __forceinline__ RowShare row_share(uint32_t m, uint32_t n, uint32_t N0, uint32_t g, uint32_t G,
                                              uint32_t q_full, uint32_t r_full, uint32_t warp_first, int spp_log2) {
    RowShare s;
    s.lo = m * n;
    const uint32_t nm = min(n, N0 - s.lo);
    uint32_t q = q_full, r = r_full;
    if (nm != n) { q = nm / G; r = nm % G; }
    s.a = g * q + min(g, r);
    s.cnt = q + (g < r ? 1u : 0u);
    s.nsp = (s.cnt > warp_first) ? ((s.cnt - warp_first - 1u) >> spp_log2) + 1u : 0u;
    return s;
}

// Sum `rows` values spaced `stride` elements apart, eight loads in flight at a time, fixed order.
template <typename T>
__device__ __forceinline__ T strided_sum(const T* col, int rows, int stride) {
    T s0 = T(0), s1 = T(0);
    for (int r0 = 0; r0 < rows; r0 += 8) {
        T v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = (r0 + j < rows) ? col[(r0 + j) * stride] : T(0);
        s0 += (v[0] + v[1]) + (v[2] + v[3]);
        s1 += (v[4] + v[5]) + (v[6] + v[7]);
    }
    return s0 + s1;
}

// One row per LPR-lane group: residual from the dot product with theta, then g += r * x.
// `rowp` is this lane's first chunk of the row in shared memory; y sits y_rel bytes from it.
template <typename T, int VEC, int LPR, int KCH, bool LOGISTIC>
__device__ __forceinline__ void row_step(const unsigned char* rowp, int y_rel, const T (&th)[KCH * VEC],
                                         T (&gacc)[KCH * VEC]) {
    constexpr int NV = KCH * VEC;
    constexpr int CB = VEC * (int)sizeof(T);
    T x[NV];
#pragma unroll
    for (int k = 0; k < KCH; ++k) {
        if constexpr (CB == 16 && sizeof(T) == 4) {
            const float4 v = *reinterpret_cast<const float4*>(rowp + k * LPR * CB);
            x[k * VEC + 0] = v.x; x[k * VEC + 1] = v.y; x[k * VEC + 2] = v.z; x[k * VEC + 3] = v.w;
        } else if constexpr (CB == 16) {
            const double2 d = *reinterpret_cast<const double2*>(rowp + k * LPR * CB);
            x[k * VEC + 0] = d.x; x[k * VEC + 1] = d.y;
        } else {
            x[k] = *reinterpret_cast<const T*>(rowp + k * LPR * CB);
        }
    }
    const T yv = *reinterpret_cast<const T*>(rowp + y_rel);
    T part[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) part[e] = T(0);
#pragma unroll
    for (int k = 0; k < KCH; ++k)
#pragma unroll
        for (int e = 0; e < VEC; ++e) part[e] = fma(x[k * VEC + e], th[k * VEC + e], part[e]);
    T dot = part[0];
#pragma unroll
    for (int e = 1; e < VEC; ++e) dot += part[e];
#pragma unroll
    for (int off = LPR / 2; off > 0; off >>= 1) dot += __shfl_xor_sync(0xFFFFFFFFu, dot, off);
    // an empty slot has x = 0 and y = 0: whatever the residual is, it multiplies zeros
    T res;
    if constexpr (LOGISTIC) res = sigmoid_of(dot) - yv;
    else res = dot - yv;
#pragma unroll
    for (int i = 0; i < NV; ++i) gacc[i] = fma(res, x[i], gacc[i]);
}

// T: float or double.  VEC: elements per copy chunk (16 bytes worth, or 1 when rows are not
// 16-byte multiples).  LPR: lanes per row.  KCH: chunks per lane.  A row has at most
// PCAP = LPR*KCH*VEC predictors.  LOGISTIC: sigmoid residual instead of the linear one.
//
// Row slots of a CTA within one step are numbered u = (sp*W + warp)*GPW + grp, sp = sub-pass:
// in sub-pass sp every warp works on GPW rows at once.  A ring stage holds `rb` sub-passes.
// A ring row is PCAP values wide whatever p is; the part beyond p is zeroed once and never written,
// and a slot without a row is zero-filled, so the inner loop carries no predicates.
// blockDim.x is 256, 512 or 1024.
template <typename T, int VEC, int LPR, int KCH, bool LOGISTIC>
__global__ void __launch_bounds__(glm_max_threads<T, VEC, KCH>(), 1) glm_kernel(const GlmParams P) {
    constexpr int GPW = 32 / LPR;            // row groups per warp
    constexpr int NV = KCH * VEC;            // values per lane
    constexpr int PCAP = LPR * KCH * VEC;    // predictor capacity
    constexpr int FPT = (PCAP + 255) / 256;  // features per thread in the reductions (blockDim >= 256)
    constexpr int CB = VEC * (int)sizeof(T); // copy chunk bytes
    constexpr int NW = Words<T>::N;
    constexpr bool PRE = glm_prereduce<VEC, KCH>();
    constexpr int YOFF = PCAP * (int)sizeof(T);  // y sits behind the predictors of its row
    constexpr uint32_t kNoRow = 0xFFFFFFFFu;

    extern __shared__ __align__(16) unsigned char smem[];

    const int tid = threadIdx.x, nthreads = blockDim.x;
    const int W = nthreads >> 5, warp = tid >> 5, lane = tid & 31;
    const int grp = lane / LPR, sub = lane % LPR;
    const int S = P.S, cpc = P.cpc, G = cpc * S;
    const int rank = (S > 1) ? (int)cluster_ctarank() : 0;
    const int cluster_id = blockIdx.x / S;
    const int team = cluster_id / cpc, kc = cluster_id % cpc;
    const int g = kc * S + rank;
    const int p = P.p, nchunks = p / VEC;
    const uint32_t N0 = P.N0, n = P.n, M = P.M;
    const int T_rounds = P.T, passes = P.passes, RB = P.rb, D = P.depth;
    const int spp_log2 = 31 - __clz(W * GPW);          // rows per sub-pass is a power of two
    const uint32_t warp_first = (uint32_t)(warp * GPW); // first row slot of this warp in sub-pass 0

    const GlmSmemPlan plan = glm_smem_plan(W, GPW, PRE, RB, D, PCAP, (int)sizeof(T), S);
    const int pitch = plan.pitch;
    unsigned char* my_ring = smem + plan.ring_off + warp * D * plan.warp_stage_bytes;
    const uint32_t my_bars = smem_u32(smem) + (uint32_t)(warp * D * 8);  // one mbarrier per stage of this warp's ring
    const bool bulk = P.bulk_rows != 0;
    T* gpart = reinterpret_cast<T*>(smem + plan.gpart_off);
    T* cpart = reinterpret_cast<T*>(smem + plan.cpart_off);
    T* gfin = reinterpret_cast<T*>(smem + plan.gfin_off);
    const int lane_off = grp * pitch + sub * CB;  // this lane's first chunk inside a sub-pass of its warp
    const int subpass_bytes = GPW * pitch;
    const int y_rel = YOFF - sub * CB;

    const unsigned char* Xb = static_cast<const unsigned char*>(P.X) + sub * CB;
    const T* yb = static_cast<const T*>(P.y);
    const uint32_t row_bytes = (uint32_t)p * (uint32_t)sizeof(T);
    const FeistelDomain dom = make_domain(N0);
    const int slice = (p + S - 1) / S;  // predictors owned by one CTA of a cluster in the sliced exchange
    uint32_t kmask = 0;                 // chunk k of this lane lies inside the row
#pragma unroll
    for (int k = 0; k < KCH; ++k) kmask |= (sub + k * LPR < nchunks) ? (1u << k) : 0u;
    const T scale_full = (T)P.scale_full, scale_last = (T)P.scale_last;

    const int nch = (team < P.Rc) ? (P.Rc - team + P.nteams - 1) / P.nteams : 0;
    uint32_t to_issue = (uint32_t)nch * (uint32_t)T_rounds * M * (uint32_t)passes;  // the host keeps this below 2^32

    // zero all of shared memory once: row tails beyond p and never-written slots must read as zero
    for (int i = plan.ring_off + tid * 16; i < plan.total_bytes; i += nthreads * 16) st_shared_zero16(smem_u32(smem + i));
    if (tid < W * D) mbar_init(smem_u32(smem) + (uint32_t)(tid * 8), 33u);  // 32 lanes after their copies + the byte count
    fence_barrier_init();
    fence_async_proxy();  // bulk copies will overwrite bytes zeroed here
    __syncthreads();
    if (S > 1) {  // peers must be running (and zeroed) before anyone writes into their shared memory
        cluster_arrive_release();
        cluster_wait_acquire();
    }

    // ---- prefetch cursor: runs D stages ahead of the compute cursor
    int pf_ci = 0, pf_t = 0, pf_sidx = 0, pf_slot = 0;
    uint32_t pf_m = 0;
    uint32_t pf_rows = kNoRow;  // this lane's row of the current batch of 32 row slots
    RoundKeys pfk = round_keys(P.seed, (uint32_t)team, 0u);
    RowShare pfs = row_share(0u, n, N0, (uint32_t)g, (uint32_t)G, P.q_full, P.r_full, warp_first, spp_log2);

    auto issue_one = [&]() {
        if (to_issue != 0u) {
            --to_issue;
            uint32_t dst = smem_u32(my_ring + pf_slot * plan.warp_stage_bytes) + lane_off;
            const uint32_t pf_bar = my_bars + (uint32_t)(pf_slot * 8);
            int pf_rows_in_stage = 0;
            int sp = pf_sidx * RB;
            for (int r = 0; r < RB; ++r, ++sp, dst += subpass_bytes) {
                const int bi = sp & (LPR - 1);
                if (bi == 0) {  // a new batch: lane l takes sub-pass sp + l/GPW, group l%GPW
                    const uint32_t u = (((uint32_t)(sp + lane / GPW)) << spp_log2) + warp_first + (lane % GPW);
                    pf_rows = (u < pfs.cnt) ? perm_index(pfs.lo + pfs.a + u, dom, pfk) : kNoRow;
                }
                if ((uint32_t)sp < pfs.nsp) {  // otherwise the whole warp skips this sub-pass, here and in the compute loop
                    const uint32_t row = __shfl_sync(0xFFFFFFFFu, pf_rows, bi * GPW + grp);
                    if (row != kNoRow) {
                        if (bulk) {
                            if (sub == 0) {  // one bulk copy per row; its bytes are counted on the stage's mbarrier
                                bulk_copy_row(dst, Xb + (size_t)row * row_bytes, row_bytes, pf_bar);
                                cp_async<(int)sizeof(T)>(dst + YOFF, yb + row);
                            }
                        } else {
                            cp_async_chunks<CB, LPR * CB, 0, KCH>(dst, Xb + (size_t)row * row_bytes, kmask);
                            cp_async_at<(int)sizeof(T), 0>(dst + y_rel, yb + row, sub == 0 ? 1u : 0u);
                        }
                    } else {  // no row for this slot: it must contribute nothing
#pragma unroll
                        for (int k = 0; k < KCH; ++k) {
                            if constexpr (CB == 16) st_shared_zero16(dst + k * LPR * CB);
                            else if constexpr (CB == 8) asm volatile("st.shared.b64 [%0], %1;" ::"r"(dst + k * LPR * CB), "l"(0ull) : "memory");
                            else asm volatile("st.shared.b32 [%0], %1;" ::"r"(dst + k * LPR * CB), "r"(0) : "memory");
                        }
                        if (sub == 0) st_shared_zero16(dst + y_rel);
                        if (bulk) fence_async_proxy();  // a later bulk copy will overwrite these bytes
                    }
                    if (bulk) pf_rows_in_stage += __popc(__ballot_sync(0xFFFFFFFFu, row != kNoRow && sub == 0));
                }
            }
            if (++pf_sidx == passes) {
                pf_sidx = 0;
                if (++pf_m == M) {
                    pf_m = 0;
                    if (++pf_t == T_rounds) { pf_t = 0; ++pf_ci; }
                    if (pf_ci < nch)
                        pfk = round_keys(P.seed, (uint32_t)(team + pf_ci * P.nteams),
                                         P.fixed_partition ? 0u : (uint32_t)pf_t);
                }
                pfs = row_share(pf_m, n, N0, (uint32_t)g, (uint32_t)G, P.q_full, P.r_full, warp_first, spp_log2);
            }
            if (bulk) {
                if (lane == 0) mbar_arrive_expect_tx(pf_bar, (uint32_t)pf_rows_in_stage * row_bytes);
                mbar_arrive_after_copies(pf_bar);
            }
            if (++pf_slot == D) pf_slot = 0;
        }
        if (!bulk) cp_async_commit();
        __syncwarp();  // lanes walked the cycle for different lengths: meet again before any aligned barrier
    };

    for (int s = 0; s < D; ++s) issue_one();

    int cs_slot = 0;         // ring slot the compute cursor reads next
    uint32_t cs_phase = 0;   // parity of that slot's mbarrier phase (bulk-copy mode)
    uint32_t step_count = 0; // steps this team has finished in this launch
    bool aborted = false;

    for (int ci = 0; ci < nch; ++ci) {
        const int chain = team + ci * P.nteams;
        T* theta_g = static_cast<T*>(P.theta) + (size_t)chain * p;

        T th[NV];
#pragma unroll
        for (int k = 0; k < KCH; ++k) {
            const int c = sub + k * LPR;
#pragma unroll
            for (int e = 0; e < VEC; ++e) th[k * VEC + e] = (c < nchunks) ? theta_g[c * VEC + e] : T(0);
        }

        for (int t = 0; t < T_rounds; ++t) {
            for (uint32_t m = 0; m < M; ++m) {
                const RowShare sh = row_share(m, n, N0, (uint32_t)g, (uint32_t)G, P.q_full, P.r_full, warp_first, spp_log2);
                BMGD_STAMP(0);

                T gacc[NV];
#pragma unroll
                for (int i = 0; i < NV; ++i) gacc[i] = T(0);

                int sp_left = (int)sh.nsp;  // sub-passes of this step in which the warp still has rows
                for (int sidx = 0; sidx < passes; ++sidx) {
                    if (bulk) {  // bounded wait on this warp's stage barrier
                        const uint32_t bar = my_bars + (uint32_t)(cs_slot * 8);
                        unsigned long long t0 = 0;
                        uint32_t spins = 0;
                        while (!aborted && !mbar_try_wait(bar, cs_phase)) {
                            if ((++spins & 0x3Fu) == 0u) {
                                const unsigned long long now = global_ns();
                                if (t0 == 0) t0 = now;
                                if (now - t0 > P.timeout_ns || ((volatile int*)P.status)[1] != 0) {
                                    atomicCAS(P.status, 0, kStatusTimeout);
                                    atomicExch(P.status + 1, 1);
                                    aborted = true;
                                }
                            }
                        }
                    } else {
                        cp_async_wait_ring(D);
                    }
                    __syncwarp();
                    const unsigned char* rowp = my_ring + cs_slot * plan.warp_stage_bytes + lane_off;
                    if (++cs_slot == D) { cs_slot = 0; cs_phase ^= 1u; }
                    int nsub = min(sp_left, RB);
                    sp_left -= nsub;
                    if constexpr (NV * (int)sizeof(T) <= 32) {  // narrow rows: four independent rows in flight per group
                        for (; nsub >= 4; nsub -= 4, rowp += 4 * subpass_bytes) {
                            row_step<T, VEC, LPR, KCH, LOGISTIC>(rowp, y_rel, th, gacc);
                            row_step<T, VEC, LPR, KCH, LOGISTIC>(rowp + subpass_bytes, y_rel, th, gacc);
                            row_step<T, VEC, LPR, KCH, LOGISTIC>(rowp + 2 * subpass_bytes, y_rel, th, gacc);
                            row_step<T, VEC, LPR, KCH, LOGISTIC>(rowp + 3 * subpass_bytes, y_rel, th, gacc);
                        }
                    }
                    for (; nsub >= 2; nsub -= 2, rowp += 2 * subpass_bytes) {  // two independent rows in flight per group
                        row_step<T, VEC, LPR, KCH, LOGISTIC>(rowp, y_rel, th, gacc);
                        row_step<T, VEC, LPR, KCH, LOGISTIC>(rowp + subpass_bytes, y_rel, th, gacc);
                    }
                    if (nsub) row_step<T, VEC, LPR, KCH, LOGISTIC>(rowp, y_rel, th, gacc);
                    if (sidx + 1 < passes) {  // refill the slot just read; the last one of a step waits for a barrier
                        __syncwarp();
                        issue_one();
                    }
                }
                BMGD_STAMP(1);

                // ---- sum the partial gradients of this CTA in fixed order
                if constexpr (PRE) {
#pragma unroll
                    for (int off = LPR; off < 32; off <<= 1)
#pragma unroll
                        for (int i = 0; i < NV; ++i) gacc[i] += __shfl_xor_sync(0xFFFFFFFFu, gacc[i], off);
                }
                if (!PRE || grp == 0) {
                    T* gp = gpart + (PRE ? warp : warp * GPW + grp) * PCAP + sub * VEC;
#pragma unroll
                    for (int k = 0; k < KCH; ++k) {
                        if constexpr (CB == 16 && sizeof(T) == 4)
                            *reinterpret_cast<float4*>(gp + k * LPR * VEC) =
                                make_float4(gacc[k * VEC], gacc[k * VEC + 1], gacc[k * VEC + 2], gacc[k * VEC + 3]);
                        else if constexpr (CB == 16)
                            *reinterpret_cast<double2*>(gp + k * LPR * VEC) = make_double2(gacc[k * VEC], gacc[k * VEC + 1]);
                        else
                            gp[k * LPR] = gacc[k];
                    }
                }
                if (S == 1 && cpc == 1) {
                    __syncwarp();
                    issue_one();
                }
                __syncthreads();
                BMGD_STAMP(2);
                T tot[FPT];
#pragma unroll
                for (int i = 0; i < FPT; ++i) {
                    const int f = tid + i * nthreads;
                    tot[i] = (f < p) ? strided_sum(gpart + f, plan.gpart_rows, PCAP) : T(0);
                }
                BMGD_STAMP(3);

                const int parity = (int)(step_count & 1u);
                T* cp = cpart + parity * S * PCAP;

                if (cpc == 1) {
                    // ---- one cluster per chain: push to every peer, one barrier, sum locally
                    if (S > 1) {
                        const uint32_t mine = smem_u32(cp + rank * PCAP);
#pragma unroll
                        for (int i = 0; i < FPT; ++i) {
                            const int f = tid + i * nthreads;
                            if (f < p)
                                for (int peer = 0; peer < S; ++peer)
                                    st_cluster(map_to_cta(mine + f * (uint32_t)sizeof(T), (uint32_t)peer), tot[i]);
                        }
                        __syncwarp();
                        cluster_arrive_release();
                        issue_one();  // the copies for a later stage go out while the barrier completes
                        cluster_wait_acquire();
#pragma unroll
                        for (int i = 0; i < FPT; ++i) {
                            const int f = tid + i * nthreads;
                            tot[i] = (f < p) ? strided_sum(cp + f, S, PCAP) : T(0);
                        }
                    }
                    BMGD_STAMP(4);
                    BMGD_STAMP(5);
#pragma unroll
                    for (int i = 0; i < FPT; ++i) {
                        const int f = tid + i * nthreads;
                        if (f < p) gfin[f] = tot[i];
                    }
                    __syncthreads();
                } else {
                    // ---- several clusters per chain: reduce-scatter in the cluster, packets between the slice
                    //      owners of different clusters, all-gather of the totals in the cluster
                    if (S > 1) {
                        const uint32_t mine = smem_u32(cp + rank * PCAP);
#pragma unroll
                        for (int i = 0; i < FPT; ++i) {
                            const int f = tid + i * nthreads;
                            if (f < p) st_cluster(map_to_cta(mine + f * (uint32_t)sizeof(T), (uint32_t)(f / slice)), tot[i]);
                        }
                        __syncwarp();
                        cluster_arrive_release();
                        cluster_wait_acquire();
                    }
                    BMGD_STAMP(4);
                    const uint32_t tag = P.tag_base + step_count + 1u;
                    unsigned long long* slot = P.ll + ((size_t)(team * 2 + parity) * cpc) * (size_t)P.ll_stride;
                    // thread j of the CTA owns predictor f = rank*slice + j of the slice (all of them if S == 1)
#pragma unroll
                    for (int i = 0; i < FPT; ++i) {
                        const int j = tid + i * nthreads;
                        const int f = rank * slice + j;
                        if (j < slice && f < p) {
                            const T mine_sum = (S > 1) ? strided_sum(cp + f, S, PCAP) : tot[i];
#pragma unroll
                            for (int w = 0; w < NW; ++w)
                                st_packet(slot + (size_t)kc * P.ll_stride + f * NW + w,
                                          ((unsigned long long)tag << 32) | Words<T>::get(mine_sum, w));
                        }
                    }
                    BMGD_STAMP(12);
#pragma unroll
                    for (int i = 0; i < FPT; ++i) {
                        const int j = tid + i * nthreads;
                        const int f = rank * slice + j;
                        if (j >= slice || f >= p) continue;
                        unsigned long long v[kMaxCpc][NW];
                        unsigned long long t0 = 0;
                        uint32_t spins = 0;
                        while (!aborted) {
                            // all loads first, all tag checks after: a check between two loads would make the
                            // second load wait for the first one's round trip to L2
#pragma unroll
                            for (int k = 0; k < kMaxCpc; ++k) {
                                if (k < cpc) {
#pragma unroll
                                    for (int w = 0; w < NW; ++w) v[k][w] = ld_packet(slot + (size_t)k * P.ll_stride + f * NW + w);
                                }
                            }
                            bool ok = true;
#pragma unroll
                            for (int k = 0; k < kMaxCpc; ++k) {
                                if (k < cpc) {
#pragma unroll
                                    for (int w = 0; w < NW; ++w) ok &= ((uint32_t)(v[k][w] >> 32) == tag);
                                }
                            }
                            if (ok) break;
                            if ((++spins & 0x3FFu) == 0u) {
                                const unsigned long long now = global_ns();
                                if (t0 == 0) t0 = now;
                                if (now - t0 > P.timeout_ns || ((volatile int*)P.status)[1] != 0) {
                                    atomicCAS(P.status, 0, kStatusTimeout);
                                    atomicExch(P.status + 1, 1);
                                    aborted = true;
                                }
                            }
                        }
#ifdef BMGD_TRACE
                        if (blockIdx.x == BMGD_TRACE_BLOCK && tid == 0 && step_count < (uint32_t)kTraceSteps) {
                            g_trace[step_count * kTracePhases + 13] = clock64();
                            g_trace[step_count * kTracePhases + 14] = spins;
                        }
#endif
                        T s = T(0);
                        if (!aborted) {
#pragma unroll
                            for (int k = 0; k < kMaxCpc; ++k) {
                                if (k < cpc) {
                                    uint32_t w32[NW];
#pragma unroll
                                    for (int w = 0; w < NW; ++w) w32[w] = (uint32_t)v[k][w];
                                    s += Words<T>::make(w32);
                                }
                            }
                        }
                        if (S > 1) {
                            const uint32_t dst = smem_u32(gfin + f);
                            for (int peer = 0; peer < S; ++peer) st_cluster(map_to_cta(dst, (uint32_t)peer), s);
                        } else {
                            gfin[f] = s;
                        }
                    }
                    BMGD_STAMP(5);
                    // The copies for a later stage go out only now: issued earlier they would sit in front of the
                    // packet stores and polls on the same load/store path and delay the exchange by their drain time.
                    __syncwarp();
                    if (S > 1) {
                        cluster_arrive_release();
                        issue_one();
                        cluster_wait_acquire();
                    } else {
                        issue_one();
                        __syncthreads();
                    }
                }
                BMGD_STAMP(6);

                // ---- everyone updates its own copy of theta
                const T scale = (min(n, N0 - sh.lo) == n) ? scale_full : scale_last;
                {
                    const T* gf = gfin + sub * VEC;
#pragma unroll
                    for (int k = 0; k < KCH; ++k) {
                        if constexpr (CB == 16 && sizeof(T) == 4) {
                            const float4 v = *reinterpret_cast<const float4*>(gf + k * LPR * VEC);
                            th[k * VEC + 0] = fma(-scale, v.x, th[k * VEC + 0]);
                            th[k * VEC + 1] = fma(-scale, v.y, th[k * VEC + 1]);
                            th[k * VEC + 2] = fma(-scale, v.z, th[k * VEC + 2]);
                            th[k * VEC + 3] = fma(-scale, v.w, th[k * VEC + 3]);
                        } else {
#pragma unroll
                            for (int e = 0; e < VEC; ++e)
                                th[k * VEC + e] = fma(-scale, gf[k * LPR * VEC + e], th[k * VEC + e]);
                        }
                    }
                }
                BMGD_STAMP(7);
                ++step_count;
            }
        }

        if (g == 0 && warp == 0 && grp == 0) {
#pragma unroll
            for (int k = 0; k < KCH; ++k) {
                const int c = sub + k * LPR;
                if (c < nchunks)
#pragma unroll
                    for (int e = 0; e < VEC; ++e) theta_g[c * VEC + e] = th[k * VEC + e];
            }
        }
    }
    cp_async_wait_all();
}

// Waits, with the step kernel's protocol, for a packet tag that nobody writes: the wait must run out of its
// budget, record BMGD_ERR_TIMEOUT in the status word, raise the abort flag and return.  For testing the error path.
__global__ void wait_probe_kernel(const unsigned long long* packet, uint32_t tag, unsigned long long timeout_ns, int* status) {
    unsigned long long t0 = 0;
    uint32_t spins = 0;
    bool aborted = false;
    while (!aborted) {
        if ((uint32_t)(ld_packet(packet) >> 32) == tag) break;
        if ((++spins & 0x3FFu) == 0u) {
            const unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            if (now - t0 > timeout_ns || ((volatile int*)status)[1] != 0) {
                atomicCAS(status, 0, kStatusTimeout);
                atomicExch(status + 1, 1);
                aborted = true;
            }
        }
    }
}

// Writes out[j] = pi(j) for one (seed, chain, round): the shuffle exactly as the step kernel uses it.
__global__ void perm_kernel(unsigned long long seed, uint32_t chain, uint32_t round, uint32_t N0, uint32_t* out) {
    const FeistelDomain dom = make_domain(N0);
    const RoundKeys rk = round_keys(seed, chain, round);
    for (unsigned long long j = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x; j < N0;
         j += (unsigned long long)gridDim.x * blockDim.x)
        out[j] = perm_index((uint32_t)j, dom, rk);
}

}  // namespace bmgdk
