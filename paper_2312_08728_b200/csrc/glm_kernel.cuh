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
//   3. the group partials are summed in fixed order in shared memory, then across the cluster
//      through distributed shared memory (every CTA pushes its partial to every peer), then
//      across clusters through tagged 8-byte packets in global memory (value and step tag
//      travel in one 64-bit store, so a reader needs no separate flag or fence);
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
    double alpha;
    uint32_t N0;
    uint32_t n;           // mini-batch size
    uint32_t M;           // mini-batches per round
    int T;                // rounds
    int p;
    int loss;             // 0 linear, 1 logistic
    int Rc;
    int S;                // cluster size
    int cpc;              // clusters per chain
    int nteams;
    int passes;           // ring stages per step
    int rb;               // sub-passes per ring stage (a power of two, at most LPR)
    int depth;            // ring stages in flight
    uint32_t q_full, r_full;  // n / G and n % G: how a full mini-batch is dealt to the G CTAs
    int pitch;            // bytes between rows in the ring (multiple of 16)
    int ll_stride;        // packets per cluster slot
    uint32_t tag_base;
    int fixed_partition;
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
__device__ __forceinline__ void cp_async_wait_pending(int n) {
    switch (n) {  // the operand must be an immediate
        case 0: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
        case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
        case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
        case 3: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
        case 4: asm volatile("cp.async.wait_group 4;" ::: "memory"); break;
        case 5: asm volatile("cp.async.wait_group 5;" ::: "memory"); break;
        case 6: asm volatile("cp.async.wait_group 6;" ::: "memory"); break;
        case 7: asm volatile("cp.async.wait_group 7;" ::: "memory"); break;
        case 8: asm volatile("cp.async.wait_group 8;" ::: "memory"); break;
        case 9: asm volatile("cp.async.wait_group 9;" ::: "memory"); break;
        case 10: asm volatile("cp.async.wait_group 10;" ::: "memory"); break;
        case 11: asm volatile("cp.async.wait_group 11;" ::: "memory"); break;
        case 12: asm volatile("cp.async.wait_group 12;" ::: "memory"); break;
        case 13: asm volatile("cp.async.wait_group 13;" ::: "memory"); break;
        case 14: asm volatile("cp.async.wait_group 14;" ::: "memory"); break;
        default: asm volatile("cp.async.wait_group 15;" ::: "memory"); break;
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
__device__ __forceinline__ void st_cluster(uint32_t addr, double v) {
    asm volatile("st.shared::cluster.f64 [%0], %1;" ::"r"(addr), "d"(v) : "memory");
}
__device__ __forceinline__ void cluster_arrive_release() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait_acquire() {
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void st_packet(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long ld_packet(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ float sigmoid_of(float u) { return 1.0f / (1.0f + expf(-u)); }
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
    int warp_stage_bytes;  // one warp's share of one ring stage: its rows, then its y values
    int ring_bytes;
    int gpart_off, cpart_off, gfin_off;
    int total_bytes;
};

__host__ __device__ inline GlmSmemPlan glm_smem_plan(int warps, int gpw, int rb, int depth, int pitch, int pcap,
                                                     int elem_bytes, int S) {
    GlmSmemPlan s;
    s.warp_stage_bytes = rb * gpw * (pitch + 16);
    s.ring_bytes = warps * depth * s.warp_stage_bytes;
    s.gpart_off = s.ring_bytes;
    s.cpart_off = s.gpart_off + warps * gpw * pcap * elem_bytes;
    s.gfin_off = s.cpart_off + 2 * S * pcap * elem_bytes;
    s.total_bytes = s.gfin_off + pcap * elem_bytes;
    return s;
}

#ifdef BMGD_TRACE
// Debug build only: clock stamps of CTA 0 at the phase boundaries of its first steps.
constexpr int kTraceSteps = 64, kTracePhases = 8;
__device__ long long g_trace[kTraceSteps * kTracePhases];
#define BMGD_STAMP(ph)                                                                              \
    do {                                                                                            \
        if (blockIdx.x == 0 && threadIdx.x == 0 && step_count < (uint32_t)kTraceSteps)              \
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

// How mini-batch rows [lo, lo+nm) are dealt to CTA g of G: a contiguous run of `cnt` rows from lo+a.
struct RowShare {
    uint32_t lo, a, cnt;
};
__device__ __forceinline__ RowShare row_share(uint32_t m, uint32_t n, uint32_t N0, uint32_t g, uint32_t G,
                                              uint32_t q_full, uint32_t r_full) {
    RowShare s;
    s.lo = m * n;
    const uint32_t nm = min(n, N0 - s.lo);
    uint32_t q = q_full, r = r_full;
    if (nm != n) { q = nm / G; r = nm % G; }
    s.a = g * q + min(g, r);
    s.cnt = q + (g < r ? 1u : 0u);
    return s;
}

// T: float or double.  VEC: elements per copy chunk (16 bytes worth, or 1 when rows are not
// 16-byte multiples).  LPR: lanes per row.  KCH: chunks per lane.  A row has at most
// LPR*KCH*VEC predictors.
//
// Row slots of a CTA within one step are numbered u = (sp*W + warp)*GPW + grp, sp = sub-pass:
// in sub-pass sp every warp works on GPW rows at once.  A ring stage holds `rb` sub-passes.
template <typename T, int VEC, int LPR, int KCH>
__global__ void __launch_bounds__(glm_max_threads<T, VEC, KCH>(), 1) glm_kernel(const GlmParams P) {
    constexpr int GPW = 32 / LPR;            // row groups per warp
    constexpr int NV = KCH * VEC;            // values per lane
    constexpr int PCAP = LPR * KCH * VEC;    // predictor capacity
    constexpr int FPT = (PCAP + 255) / 256;  // features per thread in the reductions (blockDim >= 256)
    constexpr int CB = VEC * (int)sizeof(T); // copy chunk bytes
    constexpr int NW = Words<T>::N;
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
    const int T_rounds = P.T, passes = P.passes, RB = P.rb, D = P.depth, pitch = P.pitch;

    const GlmSmemPlan plan = glm_smem_plan(W, GPW, RB, D, pitch, PCAP, (int)sizeof(T), S);
    unsigned char* my_ring = smem + (size_t)warp * D * plan.warp_stage_bytes;
    const int y_off = RB * GPW * pitch;  // y values follow the rows of a warp's stage
    T* gpart = reinterpret_cast<T*>(smem + plan.gpart_off);
    T* cpart = reinterpret_cast<T*>(smem + plan.cpart_off);
    T* gfin = reinterpret_cast<T*>(smem + plan.gfin_off);

    const unsigned char* Xb = static_cast<const unsigned char*>(P.X);
    const T* yb = static_cast<const T*>(P.y);
    const size_t row_bytes = (size_t)p * sizeof(T);
    const FeistelDomain dom = make_domain(N0);

    const int nch = (team < P.Rc) ? (P.Rc - team + P.nteams - 1) / P.nteams : 0;
    const long long nstages = (long long)nch * T_rounds * M * passes;

    if (S > 1) {  // peers must be running before anyone writes into their shared memory
        cluster_arrive_release();
        cluster_wait_acquire();
    }

    // ---- prefetch cursor: runs D stages ahead of the compute cursor
    int pf_ci = 0, pf_t = 0, pf_sidx = 0, pf_slot = 0;
    uint32_t pf_m = 0;
    uint32_t pf_rows = kNoRow;  // this lane's row of the current batch of 32 row slots
    long long issued = 0;
    RoundKeys pfk = round_keys(P.seed, (uint32_t)team, 0u);
    RowShare pfs = row_share(0u, n, N0, (uint32_t)g, (uint32_t)G, P.q_full, P.r_full);

    auto issue_one = [&]() {
        if (issued < nstages) {
            unsigned char* stage = my_ring + (size_t)pf_slot * plan.warp_stage_bytes;
            for (int r = 0; r < RB; ++r) {
                const int sp = pf_sidx * RB + r;
                const int bi = sp & (LPR - 1);
                if (bi == 0) {  // a new batch: lane l takes sub-pass sp + l/GPW, group l%GPW
                    const uint32_t u = ((uint32_t)(sp + lane / GPW) * (uint32_t)W + (uint32_t)warp) * GPW + (lane % GPW);
                    pf_rows = (u < pfs.cnt) ? perm_index(pfs.lo + pfs.a + u, dom, pfk) : kNoRow;
                }
                const uint32_t row = __shfl_sync(0xFFFFFFFFu, pf_rows, bi * GPW + grp);
                if (row != kNoRow) {
                    const unsigned char* src = Xb + (size_t)row * row_bytes;
                    const int slot_row = r * GPW + grp;
                    const uint32_t dst = smem_u32(stage + slot_row * pitch);
#pragma unroll
                    for (int k = 0; k < KCH; ++k) {
                        const int c = sub + k * LPR;
                        if (c < nchunks) cp_async<CB>(dst + c * CB, src + (size_t)c * CB);
                    }
                    if (sub == 0) cp_async<(int)sizeof(T)>(smem_u32(stage + y_off + slot_row * 16), yb + row);
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
                pfs = row_share(pf_m, n, N0, (uint32_t)g, (uint32_t)G, P.q_full, P.r_full);
            }
            if (++pf_slot == D) pf_slot = 0;
        }
        cp_async_commit();
        ++issued;
        __syncwarp();  // lanes walked the cycle for different lengths: meet again before any aligned barrier
    };

    for (int s = 0; s < D; ++s) issue_one();

    int cs_slot = 0;         // ring slot the compute cursor reads next
    uint32_t step_count = 0; // steps this team has finished in this launch
    bool aborted = false;
    const bool logistic = (P.loss == 1);

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
                const RowShare sh = row_share(m, n, N0, (uint32_t)g, (uint32_t)G, P.q_full, P.r_full);
                const uint32_t nm = min(n, N0 - sh.lo);
                BMGD_STAMP(0);

                T gacc[NV];
#pragma unroll
                for (int i = 0; i < NV; ++i) gacc[i] = T(0);

                for (int sidx = 0; sidx < passes; ++sidx) {
                    cp_async_wait_pending(D - 1);
                    __syncwarp();
                    const unsigned char* stage = my_ring + (size_t)cs_slot * plan.warp_stage_bytes;
                    if (++cs_slot == D) cs_slot = 0;

                    for (int r = 0; r < RB; ++r) {
                        const uint32_t u = ((uint32_t)(sidx * RB + r) * (uint32_t)W + (uint32_t)warp) * GPW + grp;
                        const bool valid = u < sh.cnt;
                        const int slot_row = r * GPW + grp;

                        T x[NV];
                        const unsigned char* rowp = stage + slot_row * pitch;
#pragma unroll
                        for (int k = 0; k < KCH; ++k) {
                            const int c = sub + k * LPR;
                            if (valid && c < nchunks) {
                                if constexpr (CB == 16 && sizeof(T) == 4) {
                                    const float4 v = *reinterpret_cast<const float4*>(rowp + c * 16);
                                    x[k * VEC + 0] = v.x; x[k * VEC + 1] = v.y; x[k * VEC + 2] = v.z; x[k * VEC + 3] = v.w;
                                } else if constexpr (CB == 16) {
                                    const double2 d = *reinterpret_cast<const double2*>(rowp + c * 16);
                                    x[k * VEC + 0] = d.x; x[k * VEC + 1] = d.y;
                                } else {
                                    x[k] = *reinterpret_cast<const T*>(rowp + c * CB);
                                }
                            } else {
#pragma unroll
                                for (int e = 0; e < VEC; ++e) x[k * VEC + e] = T(0);
                            }
                        }
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

                        T res = T(0);
                        if (valid) {
                            const T yv = *reinterpret_cast<const T*>(stage + y_off + slot_row * 16);
                            res = (logistic ? sigmoid_of(dot) : dot) - yv;
                        }
#pragma unroll
                        for (int i = 0; i < NV; ++i) gacc[i] = fma(res, x[i], gacc[i]);
                    }
                    if (sidx + 1 < passes) {  // refill the slot just read; the last one of a step waits for a barrier
                        __syncwarp();
                        issue_one();
                    }
                }
                BMGD_STAMP(1);

                // ---- sum the group partials of this CTA in fixed order
                {
                    T* gp = gpart + (size_t)(warp * GPW + grp) * PCAP;
#pragma unroll
                    for (int k = 0; k < KCH; ++k) {
                        const int c = sub + k * LPR;
#pragma unroll
                        for (int e = 0; e < VEC; ++e) gp[c * VEC + e] = gacc[k * VEC + e];
                    }
                }
                if (S == 1 && cpc == 1) {
                    __syncwarp();
                    issue_one();
                }
                __syncthreads();
                BMGD_STAMP(2);
                const int spp = W * GPW;
                T tot[FPT];
#pragma unroll
                for (int i = 0; i < FPT; ++i) {
                    const int f = tid + i * nthreads;
                    T s0 = T(0), s1 = T(0), s2 = T(0), s3 = T(0);
                    if (f < p) {
                        const T* col = gpart + f;
                        int r4 = 0;
                        for (; r4 + 3 < spp; r4 += 4) {
                            s0 += col[(size_t)(r4 + 0) * PCAP];
                            s1 += col[(size_t)(r4 + 1) * PCAP];
                            s2 += col[(size_t)(r4 + 2) * PCAP];
                            s3 += col[(size_t)(r4 + 3) * PCAP];
                        }
                        for (; r4 < spp; ++r4) s0 += col[(size_t)r4 * PCAP];
                    }
                    tot[i] = (s0 + s1) + (s2 + s3);
                }
                BMGD_STAMP(3);

                const int parity = (int)(step_count & 1u);

                // ---- across the cluster: push to every peer, one barrier, sum locally
                if (S > 1) {
                    T* cp = cpart + (size_t)parity * S * PCAP;
                    const uint32_t mine = smem_u32(cp + (size_t)rank * PCAP);
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
                        T s = T(0);
                        if (f < p)
                            for (int r2 = 0; r2 < S; ++r2) s += cp[(size_t)r2 * PCAP + f];
                        tot[i] = s;
                    }
                }
                BMGD_STAMP(4);

                // ---- across clusters: tagged packets through global memory
                if (cpc > 1) {
                    const uint32_t tag = P.tag_base + step_count + 1u;
                    unsigned long long* slot =
                        P.ll + ((size_t)(team * 2 + parity) * cpc) * (size_t)P.ll_stride;
#pragma unroll
                    for (int i = 0; i < FPT; ++i) {
                        const int f = tid + i * nthreads;
                        if (f < p && (f % S) == rank) {
#pragma unroll
                            for (int w = 0; w < NW; ++w)
                                st_packet(slot + (size_t)kc * P.ll_stride + f * NW + w,
                                          ((unsigned long long)tag << 32) | Words<T>::get(tot[i], w));
                        }
                    }
                    if (S == 1) issue_one();
#pragma unroll
                    for (int i = 0; i < FPT; ++i) {
                        const int f = tid + i * nthreads;
                        T s = T(0);
                        if (f < p) {
                            unsigned long long v[kMaxCpc][NW];
                            unsigned long long t0 = 0;
                            uint32_t spins = 0;
                            while (!aborted) {
                                bool ok = true;
#pragma unroll
                                for (int k = 0; k < kMaxCpc; ++k) {
                                    if (k < cpc) {
#pragma unroll
                                        for (int w = 0; w < NW; ++w) {
                                            v[k][w] = ld_packet(slot + (size_t)k * P.ll_stride + f * NW + w);
                                            ok &= ((uint32_t)(v[k][w] >> 32) == tag);
                                        }
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
                        }
                        tot[i] = s;
                    }
                }
                BMGD_STAMP(5);

                // ---- everyone updates its own copy of theta
#pragma unroll
                for (int i = 0; i < FPT; ++i) {
                    const int f = tid + i * nthreads;
                    if (f < PCAP) gfin[f] = (f < p) ? tot[i] : T(0);
                }
                // a thread that gave up tells the rest of its CTA, so that no one else waits out its own budget
                aborted = __syncthreads_or(aborted ? 1 : 0) != 0;
                BMGD_STAMP(6);
                const T scale = (T)(P.alpha / (double)nm);
#pragma unroll
                for (int k = 0; k < KCH; ++k) {
                    const int c = sub + k * LPR;
#pragma unroll
                    for (int e = 0; e < VEC; ++e) th[k * VEC + e] -= scale * gfin[c * VEC + e];
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
    cp_async_wait_pending(0);
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
