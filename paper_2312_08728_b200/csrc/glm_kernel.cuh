// Fused persistent step kernel for least-squares and logistic BMGD (Algorithm 1, inner loops;
// Eq. (2.1)).  One launch runs every round and every mini-batch step of one call.
//
// Work split.  A chain (one theta) is worked on by a team of `cpc` thread-block clusters of `S`
// CTAs, G = cpc*S CTAs in all; the rows of a mini-batch are dealt out evenly among them.  With
// replicate chains there are several teams, each taking chains team, team+nteams, ...
//
// Per step, in every CTA:
//   1. rows pi(j) of this CTA's share were fetched into a shared-memory ring by dedicated producer warps, several
//      stages ahead: four rows per tensor-map gather (cp.async.bulk.tensor tile::gather4) where rows are 16-byte
//      multiples of at most 256 values, one bulk copy per row where they are wider, element-wise cp.async otherwise;
//      completion is counted on one mbarrier per ring stage.  Rows do not depend on theta and the shuffle is
//      stateless, so the producers run through step, round and chain boundaries and the evaluation of pi never sits
//      on the path from one theta to the next;
//   2. in the consumer warps a group of LPR lanes owns one row: x.theta by an LPR-lane butterfly, the residual
//      (x.theta - y, or sigmoid(x.theta) - y), then g += r * x with x still in registers, so a
//      row is read from HBM once and from shared memory once;
//   3. the group partials are summed in fixed order (shuffles, then shared memory).  With one cluster per chain
//      every CTA pushes its partial sums into the shared memory of every peer as tagged 8-byte packets (value and
//      step tag travel in one 64-bit store, so a reader needs no separate flag, fence or barrier) and sums the
//      packets that arrive in its own.  With several clusters the partials are reduce-scattered inside the
//      cluster the same way (CTA r owns a slice of the predictors), the slice sums cross clusters as tagged
//      packets in global memory (only the slice owner polls), and the totals are pushed to every peer;
//   4. in every CTA the thread that holds predictor f's total applies the update rule (Eq. (2.1); or Nesterov's or
//      Adam's, Section 4.3; with a constant or a per-update cosine rate, Section 4.4) to its master copy of theta_f
//      and the lanes reload the coefficients they multiply rows with.
// All sums have a fixed order and every CTA does the same arithmetic, so all CTAs hold bit-identical theta and runs
// are reproducible.
//
// Every wait on another warp or CTA is bounded: when the budget runs out the kernel records
// BMGD_ERR_TIMEOUT in the status word, stops waiting for the rest of the launch and returns.
#pragma once
#include <cstdint>
#include <cuda.h>
#include <cuda_runtime.h>

#include "shuffle.cuh"

namespace bmgdk {

constexpr int kMaxCpc = 20;        // clusters per chain the packet exchange is unrolled for
constexpr int kMaxClusterSize = 16; // CTAs per cluster
constexpr int kMaxBatchesPerProducer = 2;  // gathered rows: batches of 32 row slots one producer warp takes in one ring stage
constexpr int kStatusTimeout = -5; // == BMGD_ERR_TIMEOUT
constexpr unsigned long long kDrainNs = 1000000ull;  // at the end of a launch: how long a warp waits for its own copies in flight
constexpr int kCtaAbortOff = 512;  // shared-memory word (in front of the ring) through which a CTA's consumers agree to stop
constexpr int kOptSgd = 0, kOptNesterov = 1, kOptAdam = 2;  // == BMGD_OPT_*
constexpr int kLrConstant = 0, kLrCosine = 1;               // == BMGD_LR_*
constexpr int kGlmAny = 0, kGlmPlainOne = 1, kGlmPlainTeam = 2, kGlmFlavours = 3;  // see glm_kernel

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
    double lr;            // alpha
    double inv_full, inv_last;  // 1 / n and 1 / (size of the last mini-batch)
    void* opt1;           // update-rule state [Rc][p]: Nesterov's velocity, Adam's first moment
    void* opt2;           // Adam's second moment [Rc][p]
    double opt_a, opt_b, opt_eps;        // momentum; or beta1, beta2, epsilon
    double adam_b1pow0, adam_b2pow0;     // beta1^t, beta2^t after the steps taken by earlier calls
    long long sched_period, sched_pos0;  // cosine rate: updates per pass, and how many of this pass are done
    int opt_kind;         // kOptSgd / kOptNesterov / kOptAdam
    int sched;            // kLrConstant / kLrCosine
    uint32_t N0;
    uint32_t n;           // mini-batch size
    uint32_t M;           // mini-batches per round
    int T;                // rounds
    int p;
    int Rc;
    int S;                // cluster size
    int cpc;              // clusters per chain
    int nteams;
    int consumer_warps;   // warps that compute (at least 8)
    int producer_warps;   // warps that fetch rows
    int passes;           // ring stages per step
    int rb;               // sub-passes per ring stage
    int depth;            // ring stages: 2 to 8
    uint32_t q_full, r_full;  // n / G and n % G: how a full mini-batch is dealt to the G CTAs
    int ll_stride;        // packets per cluster slot
    uint32_t tag_base;
    int fixed_partition;
    uint32_t chain0;      // shuffle id of this launch's first chain (chains of one job may be spread over several handles)
    uint32_t poll_mask;   // a packet poll looks at the clock and the abort flag every poll_mask+1 failed sweeps
    uint32_t mbar_mask;   // the same for the waits on the ring's mbarriers
#ifdef BMGD_TRACE
    long long* trace;     // debug build: clock stamps of thread 0 of every CTA, [block][step][phase] (null: none taken)
    long long* ptrace;    // and of the first producer warp, per pair of stages or per stage of its slot
#endif
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
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
// One chunk of BYTES bytes: copied from `src` if `have`, otherwise written as zeros (nothing is read from `src`).
template <int BYTES>
__device__ __forceinline__ void cp_async_fill(uint32_t dst_smem, const void* src, bool have) {
    const uint32_t n = have ? (uint32_t)BYTES : 0u;
    if constexpr (BYTES == 16)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst_smem), "l"(src), "r"(n) : "memory");
    else if constexpr (BYTES == 8)
        asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(dst_smem), "l"(src), "r"(n) : "memory");
    else
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst_smem), "l"(src), "r"(n) : "memory");
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
__device__ __forceinline__ void st_shared_zero16(uint32_t addr) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0) : "memory");
}
// A 64-bit store into a peer's shared memory and a re-read of one's own: value and tag travel together.
__device__ __forceinline__ void st_cluster_u64(uint32_t addr, unsigned long long v) {
    asm volatile("st.shared::cluster.u64 [%0], %1;" ::"r"(addr), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long ld_shared_volatile_u64(uint32_t addr) {
    unsigned long long v;
    asm volatile("ld.volatile.shared.u64 %0, [%1];" : "=l"(v) : "r"(addr) : "memory");
    return v;
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
// one row, global -> shared, completion counted in bytes on `bar`; addresses and size are 16-byte multiples
__device__ __forceinline__ void bulk_copy_row(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// four rows of a 2-D tensor map (box: one row of `box` values), rows y0..y3 from column x on, land back to back at
// dst (128-byte aligned); rows or columns outside the tensor read as zero; 4 * box bytes are counted on `bar`
__device__ __forceinline__ void tma_gather4_rows(uint32_t dst_smem, const void* tmap, int x, int y0, int y1, int y2, int y3,
                                                 uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes"
                 " [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
                 ::"r"(dst_smem), "l"(tmap), "r"(x), "r"(y0), "r"(y1), "r"(y2), "r"(y3), "r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
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
// the same without suspending the thread: false at once if the phase has not completed
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
// generic-proxy writes to shared memory become ordered with bulk copies into, and tensor-core reads of, the same bytes
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// a barrier among the consumer warps only (the producer warps never join it)
__device__ __forceinline__ void consumer_sync(int consumer_threads) {
    asm volatile("bar.sync 1, %0;" ::"r"(consumer_threads) : "memory");
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
    int pitch;             // bytes from one ring row to the next
    int stage_bytes;       // one ring stage: rb sub-passes of warps*gpw rows (and, in the gathered layout, their y values)
    int stage_y_off;       // gathered layout: where the y values of a stage start inside it
    int ring_off, ring_bytes;
    int gpart_rows;        // partial-gradient rows summed per CTA
    int gpart_off, gfin_off;
    int cpk_off, cpk_stride;  // tagged packets from the cluster's CTAs: [2][S][cpk_stride] 64-bit words
    int gpk_off;              // tagged packets carrying the totals (several clusters per chain): [2][pcap * words]
    int total_bytes;
};

// Rows of at most 256 values that are 16-byte multiples are fetched four at a time by the tensor-map gather; its
// four rows land back to back, so a ring row is exactly the predictor capacity wide and y lives in a per-stage array.
// Otherwise a ring row is the predictor capacity plus 16 bytes that hold y.
__host__ __device__ constexpr bool glm_gathered(int chunk_bytes, int pcap) { return chunk_bytes == 16 && pcap <= 256; }

// `multi`: a chain spans several clusters, so a CTA receives only its slice of the predictors from its peers.
__host__ __device__ inline GlmSmemPlan glm_smem_plan(int warps, int gpw, bool prereduce, int rb, int depth, int pcap,
                                                     int elem_bytes, int S, bool multi, bool gathered) {
    GlmSmemPlan s;
    const int words = elem_bytes / 4;
    const int R = rb * warps * gpw;
    s.pitch = gathered ? pcap * elem_bytes : pcap * elem_bytes + 16;
    s.stage_y_off = R * s.pitch;
    s.stage_bytes = gathered ? s.stage_y_off + (R * elem_bytes + 127) / 128 * 128 : s.stage_y_off;
    s.ring_off = 1024;  // the stages' mbarriers sit in front of the ring
    s.ring_bytes = depth * s.stage_bytes;
    // rounded up to a multiple of eight: the rows beyond the real ones stay zero, so the column sums need no guards
    s.gpart_rows = ((prereduce ? warps : warps * gpw) + 7) & ~7;
    s.gpart_off = s.ring_off + s.ring_bytes;
    s.gfin_off = s.gpart_off + s.gpart_rows * pcap * elem_bytes;
    s.cpk_off = s.gfin_off + pcap * elem_bytes;
    s.cpk_stride = (multi ? (pcap + S - 1) / S : pcap) * words;
    s.gpk_off = s.cpk_off + (S > 1 ? 2 * S * s.cpk_stride * 8 : 0);
    s.total_bytes = s.gpk_off + ((multi && S > 1) ? 2 * pcap * words * 8 : 0);
    return s;
}

#ifdef BMGD_TRACE
// Debug build only (build.py, trace=True): clock stamps of thread 0 of every CTA at the phase boundaries of its first
// steps, and of the first producer warp per pair of stages (gathered rows) or per stage of its slot: the SM's cycle counter.
constexpr int kTraceBlocks = 64, kTraceSteps = 48, kTracePhases = 16;
long long* trace_buffer(int which);  // host: the device array of the consumers' (0) or producers' (1) stamps, zeroed when first asked for
// The stamps go to two arrays of kTraceBlocks * kTraceSteps * kTracePhases words that the host hands over in the
// kernel's parameters (P.trace, P.ptrace; null: no stamps).
#define BMGD_STAMP(ph)                                                                                        \
    do {                                                                                                      \
        if (threadIdx.x == 0 && P.trace && blockIdx.x < (unsigned)kTraceBlocks && step_count < (uint32_t)kTraceSteps) \
            P.trace[((int)blockIdx.x * kTraceSteps + (int)step_count) * kTracePhases + (ph)] = clock64();     \
    } while (0)
#define BMGD_PSTAMP(ph)                                                                                       \
    do {                                                                                                      \
        if (pw == 0 && lane == 0 && P.ptrace && blockIdx.x < (unsigned)kTraceBlocks && pstep < (uint32_t)kTraceSteps) \
            P.ptrace[((int)blockIdx.x * kTraceSteps + (int)pstep) * kTracePhases + (ph)] = clock64();         \
    } while (0)
#else
#define BMGD_STAMP(ph) do { } while (0)
#define BMGD_PSTAMP(ph) do { } while (0)
#endif

// ---------------------------------------------------------------- the kernel

// Consumer warps a variant can run with, and the largest CTA it is compiled for (consumers plus producers): wide
// per-lane state (or fp64) needs a large register budget per thread.
template <typename T, int VEC, int KCH>
__host__ __device__ constexpr int glm_max_consumer_threads() {
    return (sizeof(T) == 8 || KCH * VEC >= 24) ? 256 : 512;
}
// CTA sizes a kernel is compiled for (consumers plus producers; registers come in units of four warps): kGlmSmallCta
// leaves 168 registers per thread, kGlmMidCta 128, kGlmLargeCta 96.  Every variant is built for the small size; fp32
// variants also for a second one: with little per-lane state the large size (16 consumer warps), with wide per-lane
// state the middle size, whose 8 consumer warps still fit 128 registers (a few bytes of spills) and which makes room
// for 8 producer warps: replicate chains over wide rows are paced by their producers.
constexpr int kGlmSmallCta = 256 + 128, kGlmMidCta = 256 + 256, kGlmLargeCta = 512 + 128;
template <typename T, int VEC, int KCH>
__host__ __device__ constexpr int glm_max_threads() {
    return sizeof(T) == 8 ? kGlmSmallCta : (KCH * VEC >= 24 ? kGlmMidCta : kGlmLargeCta);
}
// Fold the row groups of a warp together by shuffles before shared memory where that is cheap: few values per lane,
// or only two groups per warp (one shuffle level).  Fewer partial rows also leave more shared memory for the ring.
__host__ __device__ constexpr bool glm_prereduce(int values_per_lane, int lanes_per_row) {
    return values_per_lane <= 16 || (lanes_per_row >= 16 && values_per_lane <= 32);
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

// Two indices through the shuffle at once, each under its own round keys: the two Feistel chains are independent,
// so their latencies overlap.  Nearly every index leaves the network below N0 after one pass.
__device__ __forceinline__ void perm_index2(uint32_t& x0, const RoundKeys& k0, uint32_t& x1, const RoundKeys& k1,
                                            const FeistelDomain& d) {
    bool w0 = true, w1 = true;  // still walking the cycle
    do {
        uint32_t L0, R0, L1, R1;
        feistel_split(x0, d, L0, R0);
        feistel_split(x1, d, L1, R1);
#pragma unroll
        for (int r = 0; r < 8; r += 2) {
            feistel_round_pair(L0, R0, k0.k[r], k0.k[r + 1], d);
            feistel_round_pair(L1, R1, k1.k[r], k1.k[r + 1], d);
        }
        x0 = w0 ? L0 * d.c + R0 : x0;  // selects, not branches: the chains stay side by side
        x1 = w1 ? L1 * d.c + R1 : x1;
        w0 = w0 && x0 >= d.N0;
        w1 = w1 && x1 >= d.N0;
    } while (w0 || w1);
}

// N indices of one round through the shuffle at once (the same round keys): the N Feistel chains are independent, so
// their latencies overlap.
template <int N>
__device__ __forceinline__ void perm_index_n(uint32_t (&x)[N], const RoundKeys& rk, const FeistelDomain& d) {
    bool walking[N];
#pragma unroll
    for (int i = 0; i < N; ++i) walking[i] = true;
    bool any;
    do {
        uint32_t L[N], R[N];
#pragma unroll
        for (int i = 0; i < N; ++i) feistel_split(x[i], d, L[i], R[i]);
#pragma unroll
        for (int r = 0; r < 8; r += 2) {
#pragma unroll
            for (int i = 0; i < N; ++i) feistel_round_pair(L[i], R[i], rk.k[r], rk.k[r + 1], d);
        }
        any = false;
#pragma unroll
        for (int i = 0; i < N; ++i) {
            x[i] = walking[i] ? L[i] * d.c + R[i] : x[i];  // selects, not branches: the chains stay side by side
            walking[i] = walking[i] && x[i] >= d.N0;
            any |= walking[i];
        }
    } while (any);
}

// The rare part of every bounded wait: look at the clock and at the launch's abort flag.  When the budget has run
// out, or another thread has given up, record the error (first one wins), raise the flag and stop waiting.
__device__ __forceinline__ void wait_slow_path(unsigned long long& t0, bool& aborted, const GlmParams& P) {
    const unsigned long long now = global_ns();
    if (t0 == 0) t0 = now;
    if (now - t0 >= P.timeout_ns || ((volatile int*)P.status)[1] != 0) {
        atomicCAS(P.status, 0, kStatusTimeout);
        atomicExch(P.status + 1, 1);
        aborted = true;
    }
}

// Reads `count` tagged packets (NW 64-bit words each: value word in the low half, step tag in the high half) through
// `load(k, w)` until every tag equals `tag`, then returns the sum of the values in the order k = 0, 1, ....  Packets
// are taken CH at a time: all loads of a sweep over a chunk are issued before the first tag is checked.  The wait is
// bounded: when the budget runs out, or another thread has given up, the error is recorded, `aborted` is set and the
// result is void.
template <typename T, int MAXK, int CH, typename Load>
__device__ __forceinline__ T gather_packets(int count, uint32_t tag, bool& aborted, const GlmParams& P, Load load) {
    constexpr int NW = Words<T>::N;
    T s = T(0);
#pragma unroll
    for (int k0 = 0; k0 < MAXK; k0 += CH) {
        if (k0 >= count) break;
        unsigned long long v[CH][NW];
        unsigned long long t0 = 0;
        uint32_t spins = 0;
        while (!aborted) {
            // no guards on the loads (a guarded load waits for the one before it): a packet index past the last one
            // re-reads the last packet, whose tag has to match anyway
#pragma unroll
            for (int k = 0; k < CH; ++k) {
                const int kk = min(k0 + k, count - 1);
#pragma unroll
                for (int w = 0; w < NW; ++w) v[k][w] = load(kk, w);
            }
            bool ok = true;
#pragma unroll
            for (int k = 0; k < CH; ++k) {
#pragma unroll
                for (int w = 0; w < NW; ++w) ok &= ((uint32_t)(v[k][w] >> 32) == tag);
            }
            if (ok) break;
            if ((++spins & P.poll_mask) == 0u) wait_slow_path(t0, aborted, P);
        }
        if (!aborted) {
#pragma unroll
            for (int k = 0; k < CH; ++k) {
                uint32_t w32[NW];
#pragma unroll
                for (int w = 0; w < NW; ++w) w32[w] = (uint32_t)v[k][w];
                const T val = Words<T>::make(w32);
                s += (k0 + k < count) ? val : T(0);
            }
        }
    }
    return s;
}

// Sum `rows` (a multiple of eight) values spaced `stride` elements apart, fixed order.  The loads carry no guards, so
// that all eight of a sweep are in flight together (a guarded load waits for the one before it).
template <typename T>
__device__ __forceinline__ T strided_sum(const T* col, int rows, int stride) {
    T s0 = T(0), s1 = T(0);
    for (int r0 = 0; r0 < rows; r0 += 8) {
        T v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = col[(r0 + j) * stride];
        s0 += (v[0] + v[1]) + (v[2] + v[3]);
        s1 += (v[4] + v[5]) + (v[6] + v[7]);
    }
    return s0 + s1;
}

// One row per LPR-lane group: residual from the dot product with theta, then g += r * x.
// `rowp` is this lane's first chunk of the row in shared memory, `yp` the row's y.
template <typename T, int VEC, int LPR, int KCH, bool LOGISTIC>
__device__ __forceinline__ void row_step(const unsigned char* rowp, const unsigned char* yp, const T (&th)[KCH * VEC],
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
    const T yv = *reinterpret_cast<const T*>(yp);
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

// NR rows of one group at once (rows `row_stride` bytes apart, their y values `y_stride` apart): all loads first, then
// the NR dot products side by side, so that the latencies of the rows overlap by construction.  The gradient takes the
// rows in ascending order, exactly as NR calls of row_step would.
template <typename T, int VEC, int LPR, int KCH, bool LOGISTIC, int NR>
__device__ __forceinline__ void rows_step(const unsigned char* rowp, int row_stride, const unsigned char* yp, int y_stride,
                                          const T (&th)[KCH * VEC], T (&gacc)[KCH * VEC]) {
    constexpr int NV = KCH * VEC;
    constexpr int CB = VEC * (int)sizeof(T);
    T x[NR][NV], yv[NR], dot[NR];
#pragma unroll
    for (int r = 0; r < NR; ++r) {
#pragma unroll
        for (int k = 0; k < KCH; ++k) {
            const unsigned char* src = rowp + r * row_stride + k * LPR * CB;
            if constexpr (CB == 16 && sizeof(T) == 4) {
                const float4 v = *reinterpret_cast<const float4*>(src);
                x[r][k * VEC + 0] = v.x; x[r][k * VEC + 1] = v.y; x[r][k * VEC + 2] = v.z; x[r][k * VEC + 3] = v.w;
            } else if constexpr (CB == 16) {
                const double2 d = *reinterpret_cast<const double2*>(src);
                x[r][k * VEC + 0] = d.x; x[r][k * VEC + 1] = d.y;
            } else {
                x[r][k] = *reinterpret_cast<const T*>(src);
            }
        }
        yv[r] = *reinterpret_cast<const T*>(yp + r * y_stride);
    }
#pragma unroll
    for (int r = 0; r < NR; ++r) {
        T part[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) part[e] = T(0);
#pragma unroll
        for (int k = 0; k < KCH; ++k)
#pragma unroll
            for (int e = 0; e < VEC; ++e) part[e] = fma(x[r][k * VEC + e], th[k * VEC + e], part[e]);
        dot[r] = part[0];
#pragma unroll
        for (int e = 1; e < VEC; ++e) dot[r] += part[e];
    }
#pragma unroll
    for (int off = LPR / 2; off > 0; off >>= 1)
#pragma unroll
        for (int r = 0; r < NR; ++r) dot[r] += __shfl_xor_sync(0xFFFFFFFFu, dot[r], off);
    T res[NR];
#pragma unroll
    for (int r = 0; r < NR; ++r) {
        if constexpr (LOGISTIC) res[r] = sigmoid_of(dot[r]) - yv[r];
        else res[r] = dot[r] - yv[r];
    }
#pragma unroll
    for (int i = 0; i < NV; ++i)
#pragma unroll
        for (int r = 0; r < NR; ++r) gacc[i] = fma(res[r], x[r][i], gacc[i]);
}

// Waits for a phase of an mbarrier in this CTA's shared memory with the kernel's bounded-wait protocol.
__device__ __forceinline__ void bounded_mbar_wait(uint32_t bar, uint32_t parity, bool& aborted, const GlmParams& P) {
    if (mbar_test_wait(bar, parity)) return;  // the usual case where the ring runs ahead: the phase is long complete
    unsigned long long t0 = 0;
    uint32_t spins = 0;
    // try_wait suspends the thread in hardware for a while before it answers false; with no budget at all (mask 0) the
    // wait has to give up at its first look, so it asks without suspending
    while (!aborted && !(P.mbar_mask ? mbar_try_wait(bar, parity) : mbar_test_wait(bar, parity))) {
        if ((++spins & P.mbar_mask) == 0u) wait_slow_path(t0, aborted, P);
    }
}

// T: float or double.  VEC: elements per copy chunk (16 bytes worth, or 1 when rows are not
// 16-byte multiples).  LPR: lanes per row.  KCH: chunks per lane.  A row has at most
// PCAP = LPR*KCH*VEC predictors.  LOGISTIC: sigmoid residual instead of the linear one.
//
// A CTA has P.consumer_warps warps that compute and P.producer_warps warps that only fetch rows.
// Row slots of a CTA within one step are numbered u = (sp*W + warp)*GPW + grp, sp = sub-pass: in sub-pass sp
// consumer warp `warp` works on GPW rows at once.  A ring stage holds `rb` sub-passes, i.e. R = rb*W*GPW
// consecutive slots, laid out in this order with a pitch of PCAP values plus 16 bytes for y; the part of a ring
// row beyond p is zeroed once and never written, and a slot without a row is zero-filled by its copy, so the
// inner loop carries no predicates.  Each stage has a "full" mbarrier (the producers' copies have landed) and an
// "empty" one (every consumer warp has read it).
//
// NULLSTEP = true is the latency probe of the same kernel: every wait, barrier, packet exchange and update of a step
// runs with the same launch shape, but no row is fetched and none is multiplied (the gradient is zero and theta
// stays as it is).  Its time per step is what the step's synchronisation structure alone costs.
//
// FLAVOUR says which of the step's options a compiled kernel carries.  The step from one theta to the next is a chain
// of dependent phases a few thousand cycles long, so the code of options that a launch does not use (the exchange
// between clusters, the update rules with state, the rate schedule) costs time on that chain even when it is only
// branched around: measured on B200, 10 to 14 % of the step of a chain that runs inside one cluster.  kGlmAny decides
// everything at run time; the two plain flavours are Eq. (2.1) with a constant rate, compiled for a chain inside one
// cluster (kGlmPlainOne) or spread over several (kGlmPlainTeam).  All flavours do the same arithmetic in the same order.
template <typename T, int VEC, int LPR, int KCH, bool LOGISTIC, int MAXT, int FLAVOUR = kGlmAny, bool NULLSTEP = false>
__global__ void __launch_bounds__(MAXT, 1)
glm_kernel(const GlmParams P, const __grid_constant__ CUtensorMap xmap) {
    constexpr int GPW = 32 / LPR;            // row groups per warp
    constexpr int NV = KCH * VEC;            // values per lane
    constexpr int PCAP = LPR * KCH * VEC;    // predictor capacity
    constexpr int FPT = (PCAP + 255) / 256;  // features per thread in the reductions (at least 256 consumer threads)
    constexpr int CB = VEC * (int)sizeof(T); // copy chunk bytes
    constexpr int NW = Words<T>::N;
    constexpr bool PRE = glm_prereduce(KCH * VEC, LPR);
    constexpr bool G4 = glm_gathered(CB, PCAP);  // rows arrive four at a time through the tensor map `xmap` of X
    constexpr int YOFF = PCAP * (int)sizeof(T);  // other layouts: y sits behind the predictors of its row
    constexpr uint32_t kNoRow = 0xFFFFFFFFu;
    constexpr int kClusterChunk = (sizeof(T) == 4 && MAXT <= kGlmSmallCta) ? 8 : 4;  // packets of the cluster's CTAs read per sweep of a poll

    extern __shared__ __align__(1024) unsigned char smem[];  // gathers want 128-byte aligned destinations

    const int tid = threadIdx.x;
    const int W = P.consumer_warps, NPW = P.producer_warps;  // blockDim.x == 32 * (W + NPW)
    const int nthreads = W * 32;                             // consumer threads: the ones that reduce and exchange
    const int warp = tid >> 5, lane = tid & 31;
    constexpr bool PLAIN = FLAVOUR != kGlmAny;
    const int S = P.S, cpc = (FLAVOUR == kGlmPlainOne) ? 1 : P.cpc, G = cpc * S;
    const bool one_cluster = (FLAVOUR == kGlmPlainOne) ? true : (FLAVOUR == kGlmPlainTeam) ? false : cpc == 1;
    const int opt_kind = PLAIN ? kOptSgd : P.opt_kind;
    const bool cosine = !PLAIN && P.sched == kLrCosine;
    const int rank = (S > 1) ? (int)cluster_ctarank() : 0;
    const int cluster_id = blockIdx.x / S;
    const int team = cluster_id / cpc, kc = cluster_id % cpc;
    const int g = kc * S + rank;
    const int p = P.p;
    const uint32_t N0 = P.N0, n = P.n, M = P.M;
    const int T_rounds = P.T, passes = P.passes, RB = P.rb, D = P.depth;
    const int spp = W * GPW;  // rows the CTA works on at once (one sub-pass)

    const GlmSmemPlan plan = glm_smem_plan(W, GPW, PRE, RB, D, PCAP, (int)sizeof(T), S, !one_cluster, G4);
    const int pitch = plan.pitch;
    const int stage_bytes = plan.stage_bytes;
    const uint32_t full_bars = smem_u32(smem), empty_bars = smem_u32(smem) + 128u;  // one 8-byte mbarrier per stage each
    const int nch = (team < P.Rc) ? (P.Rc - team + P.nteams - 1) / P.nteams : 0;
    const uint32_t total_stages = (uint32_t)nch * (uint32_t)T_rounds * M * (uint32_t)passes;  // the host keeps this below 2^32

    // zero all of shared memory once: row tails beyond p and packet tags must read as zero
    for (int i = plan.ring_off + tid * 16; i < plan.total_bytes; i += (int)blockDim.x * 16) st_shared_zero16(smem_u32(smem + i));
    volatile int* const cta_abort = reinterpret_cast<volatile int*>(smem + kCtaAbortOff);
    if (tid == 0) *cta_abort = 0;
    if (tid < D) {
        // every producer lane, once its element copies have landed; with bulk row copies, also one lane per producer
        // warp announcing that warp's byte count
        // gathered rows: every producer warp; other layouts: the producer warps of this slot
        mbar_init(full_bars + (uint32_t)(tid * 8), (uint32_t)((G4 ? NPW : NPW / D) * (CB == 16 ? 33 : 32)));
        mbar_init(empty_bars + (uint32_t)(tid * 8), (uint32_t)W);           // one lane of every consumer warp
    }
    fence_barrier_init();
    fence_async_proxy();  // bulk copies will overwrite bytes zeroed here
    __syncthreads();
    if (S > 1) {  // peers must be running (and zeroed) before anyone writes into their shared memory
        cluster_arrive_release();
        cluster_wait_acquire();
    }

    bool aborted = false;

    if (warp >= W) {
        // ================================================================ producer warps
        // Rows do not depend on theta and the shuffle is stateless, so the producers run up to D stages ahead of
        // the consumers, through mini-batch, round and chain boundaries.  Two schemes, by row layout (measured on B200):
        //  * gathered rows (four rows per tensor-map gather): all producer warps work on the same stage, each on its
        //    share of the stage's batches of 32 row slots, two consecutive stages together so that their shuffle
        //    evaluations overlap.  The gathers of a stage are issued by several warps side by side, which is what the
        //    copy engine wants (one warp issuing all 32 gathers of a stage: cfg2 4.06 instead of 3.69 us per step);
        //  * other layouts (one bulk copy per row, or element-wise copies): producer warp pw serves ring slot pw % D
        //    and nobody else's: it fills every stage that lands in that slot (stages slot, slot + D, ... of the launch)
        //    independently of the other warps, so the shuffle evaluation for one slot overlaps the copies into the
        //    others (p = 500, 100 chains: 24.0 instead of 27.2 us per step).  With NPW = nsub * D warps, the nsub
        //    warps of a slot share a stage's batches.
        const int pw = warp - W;
        const int R = RB * spp;  // row slots of a stage: a multiple of four
        const int nchunks = p / VEC;
        int lpr_c = 1;  // lanes that copy one row: the power of two at or above nchunks, at most 32
        while (lpr_c < nchunks && lpr_c < 32) lpr_c <<= 1;
        const int rpi = 32 / lpr_c;                        // rows per copy iteration
        const int cpl = (nchunks + lpr_c - 1) / lpr_c;     // chunks per lane and row
        const int rsub = lane / lpr_c, cl = lane % lpr_c;
        const unsigned char* Xrows = static_cast<const unsigned char*>(P.X);
        const unsigned char* Xb = Xrows + (size_t)cl * CB;
        const T* yb = static_cast<const T*>(P.y);
        const uint32_t row_bytes = (uint32_t)p * (uint32_t)sizeof(T);
        const FeistelDomain dom = make_domain(N0);
        const uint32_t ring_base = smem_u32(smem + plan.ring_off);
        uint32_t issued_mask = 0, issued_par = 0;  // ring slots this warp has sent copies into, and the parity of the last such phase
        if constexpr (G4) {
        const int nbatch = (R + 31) >> 5;
        struct Cursor {  // which stage comes next, and what it needs
            int ci, t, sidx;
            uint32_t m;
            RoundKeys rk;
            RowShare sh;
        };
        Cursor cur;
        cur.ci = 0; cur.t = 0; cur.sidx = 0; cur.m = 0u;
        cur.rk = round_keys(P.seed, P.chain0 + (uint32_t)team, 0u);
        cur.sh = row_share(0u, n, N0, (uint32_t)g, (uint32_t)G, P.q_full, P.r_full);
        auto advance = [&](Cursor& c) {
            if (++c.sidx == passes) {
                c.sidx = 0;
                if (++c.m == M) {
                    c.m = 0;
                    if (++c.t == T_rounds) { c.t = 0; ++c.ci; }
                    if (c.ci < nch)
                        c.rk = round_keys(P.seed, P.chain0 + (uint32_t)(team + c.ci * P.nteams), P.fixed_partition ? 0u : (uint32_t)c.t);
                }
                c.sh = row_share(c.m, n, N0, (uint32_t)g, (uint32_t)G, P.q_full, P.r_full);
            }
        };
        int slot = 0;
        uint32_t empty_parity = 1u;  // a fresh mbarrier lets a wait on parity 1 through

        // Copies the batch whose first slot is s0; lane l holds the row of slot s0 + l (kNoRow: the slot stays empty).
        // Returns the number of gathers issued, whose bytes are counted on the stage's barrier.
        auto copy_batch = [&](uint32_t stage_base, uint32_t full_bar, int s0, uint32_t rows) -> uint32_t {
            const int left = R - s0;  // slots of this batch that exist
            {
                // lane l < 8 fetches slots 4l..4l+3 with one gather; a slot without a row asks for the row behind the
                // last one, which reads as zeros
                const int q = (lane & 7) * 4;
                const uint32_t r0 = __shfl_sync(0xFFFFFFFFu, rows, q), r1 = __shfl_sync(0xFFFFFFFFu, rows, q + 1);
                const uint32_t r2 = __shfl_sync(0xFFFFFFFFu, rows, q + 2), r3 = __shfl_sync(0xFFFFFFFFu, rows, q + 3);
                const bool mine = lane < 8 && q < left;  // R is a multiple of 4
                if (mine)
                    tma_gather4_rows(stage_base + (uint32_t)((s0 + q) * pitch), &xmap, 0, (int)min(r0, N0), (int)min(r1, N0),
                                     (int)min(r2, N0), (int)min(r3, N0), full_bar);
                if (lane < left) {
                    const bool have = rows != kNoRow;
                    cp_async_fill<(int)sizeof(T)>(stage_base + (uint32_t)(plan.stage_y_off + (s0 + lane) * (int)sizeof(T)),
                                                  yb + (have ? rows : 0u), have);
                }
                // gathers issued for this batch: one per four slots that exist (the same in every lane: no vote needed)
                return (uint32_t)min(8, (left + 3) >> 2);
            }
        };
        // closes this warp's part of a stage: every lane arrives once its element copies have landed, one lane
        // announces the bytes of the warp's bulk copies
        auto finish_stage = [&](uint32_t full_bar, uint32_t bulk_rows) {  // bulk_rows: row copies, or gathers of four rows
            mbar_arrive_after_copies(full_bar);
            {
                __syncwarp();
                if (lane == 0) mbar_arrive_expect_tx(full_bar, bulk_rows * (uint32_t)(4 * PCAP * (int)sizeof(T)));
            }
        };

        uint32_t rot = (uint32_t)pw;  // (pw - pair * nbatch) mod NPW, kept incrementally: ownership of batches rotates
        const uint32_t rot_step = (uint32_t)(nbatch % NPW);
        for (uint32_t it = 0; it < total_stages; it += 2) {
            [[maybe_unused]] const uint32_t pstep = it >> 1;  // trace build: stamps per pair of stages
            BMGD_PSTAMP(0);
            const Cursor A = cur;
            advance(cur);
            const bool two = it + 1 < total_stages;
            const Cursor B = cur;
            if (two) advance(cur);
            const int slotA = slot;
            const uint32_t parA = empty_parity;
            if (++slot == D) { slot = 0; empty_parity ^= 1u; }
            const int slotB = slot;
            const uint32_t parB = empty_parity;
            if (two && ++slot == D) { slot = 0; empty_parity ^= 1u; }
            const uint32_t baseA = ring_base + (uint32_t)(slotA * stage_bytes), baseB = ring_base + (uint32_t)(slotB * stage_bytes);
            const int b0 = (int)rot;  // this producer's first batch in this pair of stages
            rot += (uint32_t)NPW - rot_step;  // below 2 * NPW
            if (rot >= (uint32_t)NPW) rot -= (uint32_t)NPW;

            // the shuffle of both stages first (it needs no ring slot), then the copies of A, then those of B
            uint32_t rowsA[kMaxBatchesPerProducer], rowsB[kMaxBatchesPerProducer];
#pragma unroll
            for (int kk = 0; kk < kMaxBatchesPerProducer; ++kk) {
                const int bb = b0 + kk * NPW;
                rowsA[kk] = kNoRow; rowsB[kk] = kNoRow;
                if (!NULLSTEP && bb < nbatch) {
                    const int s = 32 * bb + lane;
                    const uint32_t ua = (uint32_t)(A.sidx * R + s), ub = (uint32_t)(B.sidx * R + s);
                    const bool va = s < R && ua < A.sh.cnt;
                    const bool vb = two && s < R && ub < B.sh.cnt;
                    uint32_t ra = va ? A.sh.lo + A.sh.a + ua : 0u, rb_ = vb ? B.sh.lo + B.sh.a + ub : 0u;
                    if (__any_sync(0xFFFFFFFFu, va || vb)) perm_index2(ra, A.rk, rb_, B.rk, dom);
                    __syncwarp();  // lanes walked the cycle for different lengths
                    if (va) rowsA[kk] = ra;
                    if (vb) rowsB[kk] = rb_;
                }
            }
            const uint32_t fullA = full_bars + (uint32_t)(slotA * 8), fullB = full_bars + (uint32_t)(slotB * 8);
            BMGD_PSTAMP(1);
            bounded_mbar_wait(empty_bars + (uint32_t)(slotA * 8), parA, aborted, P);
            aborted = __any_sync(0xFFFFFFFFu, aborted);
            if (aborted) break;  // the launch has been given up: no further copies are issued
            uint32_t sent = 0;
#pragma unroll
            for (int kk = 0; kk < kMaxBatchesPerProducer; ++kk) {
                const int bb = b0 + kk * NPW;
                if (!NULLSTEP && bb < nbatch) sent += copy_batch(baseA, fullA, 32 * bb, rowsA[kk]);
            }
            BMGD_PSTAMP(3);
            finish_stage(fullA, sent);  // a producer without a batch in this stage still counts on its barrier
            issued_mask |= 1u << slotA;
            issued_par = (issued_par & ~(1u << slotA)) | ((parA ^ 1u) << slotA);
            BMGD_PSTAMP(4);
            if (two) {
                bounded_mbar_wait(empty_bars + (uint32_t)(slotB * 8), parB, aborted, P);
                aborted = __any_sync(0xFFFFFFFFu, aborted);
                if (aborted) break;
                sent = 0;
#pragma unroll
                for (int kk = 0; kk < kMaxBatchesPerProducer; ++kk) {
                    const int bb = b0 + kk * NPW;
                    if (!NULLSTEP && bb < nbatch) sent += copy_batch(baseB, fullB, 32 * bb, rowsB[kk]);
                }
                finish_stage(fullB, sent);
                issued_mask |= 1u << slotB;
                issued_par = (issued_par & ~(1u << slotB)) | ((parB ^ 1u) << slotB);
                BMGD_PSTAMP(6);
            }
        }
        } else {
        const int slot = pw % D, sub = pw / D, nsub = NPW / D;  // the host launches a multiple of D producer warps
        const uint32_t stage_base = ring_base + (uint32_t)(slot * stage_bytes);
        const uint32_t full_bar = full_bars + (uint32_t)(slot * 8), empty_bar = empty_bars + (uint32_t)(slot * 8);

        // Copies 32 consecutive row slots from s0 on; lane l holds the row of slot s0 + l (kNoRow: the slot stays empty).
        // Layouts other than the gathered one: rows that are 16-byte multiples travel as one bulk copy each, counted in
        // bytes on the stage's barrier (the return value is the number of rows sent that way); others go element by element.
        auto copy_batch = [&](int s0, uint32_t rows) -> uint32_t {
            const int left = R - s0;  // slots of this batch that exist
            if constexpr (CB == 16) {
                const bool have = lane < left && rows != kNoRow;
                const uint32_t dst = stage_base + (uint32_t)((s0 + lane) * pitch);
                if (have) {
                    bulk_copy_row(dst, Xrows + (size_t)rows * row_bytes, row_bytes, full_bar);
                    cp_async_fill<(int)sizeof(T)>(dst + YOFF, yb + rows, true);
                } else if (lane < left) {  // no row for this slot: it must contribute nothing
                    for (int k = 0; k < nchunks; ++k) st_shared_zero16(dst + (uint32_t)(k * 16));
                    st_shared_zero16(dst + YOFF);
                    fence_async_proxy();  // a later bulk copy will overwrite these bytes
                }
                return (uint32_t)__popc(__ballot_sync(0xFFFFFFFFu, have));
            } else {
                const int iters = min(32, left + rpi - 1) / rpi;
                for (int i = 0; i < iters; ++i) {
                    const int sl = i * rpi + rsub;
                    const uint32_t row = __shfl_sync(0xFFFFFFFFu, rows, sl);
                    const bool have = row != kNoRow;
                    const unsigned char* src = Xb + (have ? (size_t)row * row_bytes : 0);
                    const uint32_t dst = stage_base + (uint32_t)((s0 + sl) * pitch + cl * CB);
                    if (sl < left) {
                        for (int k = 0; k < cpl; ++k) {
                            const int ch = cl + k * lpr_c;
                            if (ch < nchunks) cp_async_fill<CB>(dst + (uint32_t)(k * lpr_c * CB), src + (have ? (size_t)k * lpr_c * CB : 0), have);
                        }
                    }
                }
                if (lane < left) {
                    const bool have = rows != kNoRow;
                    cp_async_fill<(int)sizeof(T)>(stage_base + (uint32_t)((s0 + lane) * pitch + YOFF), yb + (have ? rows : 0u), have);
                }
                return 0u;
            }
        };

        // where the stage that this warp fills next sits in the job: chain of the team, round, mini-batch, ring stage of
        // the step; kept by counting (D stages forward per stage filled)
        int c_ci = 0, c_t = 0, c_sidx = 0;
        uint32_t c_m = 0;
        auto forward = [&](int stages) {
            for (int i = 0; i < stages; ++i) {
                if (++c_sidx == passes) {
                    c_sidx = 0;
                    if (++c_m == M) {
                        c_m = 0;
                        if (++c_t == T_rounds) { c_t = 0; ++c_ci; }
                    }
                }
            }
        };
        forward(slot);
        int k_ci = -1, k_t = -1;  // chain and round the keys below belong to
        RoundKeys rk;
        uint32_t empty_parity = 1u;  // a fresh mbarrier lets a wait on parity 1 through
        constexpr int kPair = 2;     // batches of 32 row slots whose shuffle indices are evaluated side by side

        for (uint32_t it = (uint32_t)slot; it < total_stages; it += (uint32_t)D) {
            [[maybe_unused]] const uint32_t pstep = it / (uint32_t)D;  // trace build: stamps per stage of this warp's slot
            BMGD_PSTAMP(0);
            if (c_ci != k_ci || c_t != k_t) {
                k_ci = c_ci; k_t = c_t;
                rk = round_keys(P.seed, P.chain0 + (uint32_t)(team + c_ci * P.nteams), P.fixed_partition ? 0u : (uint32_t)c_t);
            }
            const RowShare sh = row_share(c_m, n, N0, (uint32_t)g, (uint32_t)G, P.q_full, P.r_full);
            const uint32_t u0 = (uint32_t)(c_sidx * R);  // the stage's first row slot within this CTA's share of the mini-batch
            uint32_t sent = 0;   // bulk row copies that this warp sends into the stage
            bool waited = false;  // the slot is known to be empty
            {
                const int nbatch = (R + 31) >> 5;
                for (int b0 = sub * kPair; b0 < nbatch; b0 += nsub * kPair) {
                    uint32_t row[kPair];
                    bool valid[kPair];
#pragma unroll
                    for (int j = 0; j < kPair; ++j) {
                        const int s = 32 * (b0 + j) + lane;
                        const uint32_t u = u0 + (uint32_t)s;
                        valid[j] = !NULLSTEP && s < R && u < sh.cnt;
                        row[j] = valid[j] ? sh.lo + sh.a + u : 0u;
                    }
                    if constexpr (!NULLSTEP) {
                        if (__any_sync(0xFFFFFFFFu, valid[0] || valid[1])) perm_index_n<kPair>(row, rk, dom);
                        __syncwarp();
                    }
                    if (!waited) {
                        BMGD_PSTAMP(1);
                        bounded_mbar_wait(empty_bar, empty_parity, aborted, P);
                        aborted = __any_sync(0xFFFFFFFFu, aborted);
                        if (aborted) break;  // the launch has been given up: no further copies are issued
                        waited = true;
                    }
                    if constexpr (!NULLSTEP) {
#pragma unroll
                        for (int j = 0; j < kPair; ++j)
                            if (b0 + j < nbatch) sent += copy_batch(32 * (b0 + j), valid[j] ? row[j] : kNoRow);
                    }
                }
            }
            if (aborted) break;
            if (!waited) {  // a warp without a chunk in this stage still counts on its barrier
                BMGD_PSTAMP(1);
                bounded_mbar_wait(empty_bar, empty_parity, aborted, P);
                aborted = __any_sync(0xFFFFFFFFu, aborted);
                if (aborted) break;
            }
            BMGD_PSTAMP(3);
            // closes this warp's part of the stage: every lane arrives once its element copies have landed, one lane
            // announces the bytes of the warp's bulk copies
            mbar_arrive_after_copies(full_bar);
            if constexpr (CB == 16) {
                __syncwarp();  // the zero fills of all lanes come before the announcing lane's arrival
                if (lane == 0) mbar_arrive_expect_tx(full_bar, sent * row_bytes);
            }
            issued_mask = 1u << slot;
            issued_par = (empty_parity ^ 1u) << slot;
            empty_parity ^= 1u;
            forward(D);
            BMGD_PSTAMP(4);
        }
        }
        cp_async_wait_all();
        // No CTA may exit while bulk copies into its shared memory are in flight.  After a normal run the consumers
        // have waited for every stage; after a launch that was given up they have not, so every producer warp waits
        // here, for a bounded time, until the last phase it sent copies into has completed on each ring slot (a phase
        // completes once all producers of the slot have arrived and all bytes have landed; if one of them gave up before
        // arriving, the time limit ends the wait, long after the copies themselves have landed).
        {
            const unsigned long long t0 = global_ns();
            for (int s = 0; s < D; ++s) {
                if (!((issued_mask >> s) & 1u)) continue;
                while (!mbar_try_wait(full_bars + (uint32_t)(s * 8), (issued_par >> s) & 1u))
                    if (global_ns() - t0 > kDrainNs) break;
            }
        }
    } else {
        // ================================================================ consumer warps
        const int grp = lane / LPR, sub = lane % LPR;
        const int nchunks = p / VEC;
        T* gpart = reinterpret_cast<T*>(smem + plan.gpart_off);
        T* gfin = reinterpret_cast<T*>(smem + plan.gfin_off);
        const uint32_t cpk_base = smem_u32(smem + plan.cpk_off), gpk_base = smem_u32(smem + plan.gpk_off);
        const int lane_off = (warp * GPW + grp) * pitch + sub * CB;  // this lane's first chunk inside a sub-pass
        const int subpass_bytes = spp * pitch;
        // this group's y in sub-pass 0 of a stage, and how far it moves per sub-pass
        const int y_off = G4 ? plan.stage_y_off + (warp * GPW + grp) * (int)sizeof(T) : (warp * GPW + grp) * pitch + YOFF;
        const int y_step = G4 ? spp * (int)sizeof(T) : subpass_bytes;
        const uint32_t warp_first = (uint32_t)(warp * GPW);  // first row slot of this warp in sub-pass 0
        const int slice = (p + S - 1) / S;  // predictors owned by one CTA of a cluster in the sliced exchange
        // Pushing one predictor's sum to all S peers is a run of S dependent remote stores in one thread.  Where the
        // consumer threads outnumber the predictors, xg_n threads share the pushes of a predictor: thread (xf, xg) sends
        // predictor xf to peers xg, xg + xg_n, ...  (each of them sums the CTA's partial rows for xf itself).
        int fw_log2 = 5;  // predictors rounded up to a power of two of at least a warp
        while ((1 << fw_log2) < p) ++fw_log2;
        // threads that share a predictor's pushes: a power of two, at most S (cluster sizes are powers of two)
        const int xg_n = (FPT == 1 && one_cluster && S > 1) ? max(1, min(S, nthreads >> fw_log2)) : 1;
        const int xf = (xg_n > 1) ? (tid & ((1 << fw_log2) - 1)) : tid, xg = (xg_n > 1) ? (tid >> fw_log2) : 0;
        // Where this thread's packets go in its peers' shared memory (parity 0; the other parity lies a fixed distance
        // behind), worked out once when a thread has at most four peers to serve: the address arithmetic and the mapping
        // into the peer's window would otherwise be redone in every step, on the path from one theta to the next.
        constexpr int kFastPeers = 4;
        const int my_peers = (S + xg_n - 1 - xg) / xg_n;  // peers xg, xg + xg_n, ... below S
        const bool fast_push = FPT == 1 && one_cluster && S > 1 && S / xg_n <= kFastPeers;
        uint32_t push_addr[kFastPeers];
#pragma unroll
        for (int i = 0; i < kFastPeers; ++i)
            push_addr[i] = (fast_push && i < my_peers)
                ? map_to_cta(cpk_base + (uint32_t)((rank * plan.cpk_stride + xf * NW) * 8), (uint32_t)(xg + i * xg_n)) : 0u;
        const uint32_t parity_bytes = (uint32_t)(S * plan.cpk_stride * 8);
        const T scale_full = (T)P.scale_full, scale_last = (T)P.scale_last;
        const T inv_full = (T)P.inv_full, inv_last = (T)P.inv_last, lr_const = (T)P.lr;

        // A full mini-batch is dealt to the CTAs the same way in every step: its share, and the sub-passes in which this
        // warp has rows, are worked out once (the divisions would otherwise sit at the head of every step).
        const RowShare share_full = row_share(0u, n, n, (uint32_t)g, (uint32_t)G, P.q_full, P.r_full);
        const int sp_full = (share_full.cnt > warp_first) ? (int)((share_full.cnt - warp_first - 1u) / (uint32_t)spp) + 1 : 0;
        int cs_slot = 0;         // ring slot the compute cursor reads next
        uint32_t cs_phase = 0;   // parity of that slot's "full" phase
        uint32_t step_count = 0; // steps this team has finished in this launch
        // Where a step has an exchange to wait for, the wait for the next step's first ring stage is taken while this
        // step's packets are under way (the stage has usually long been filled, but asking costs about 120 cycles, which
        // would otherwise sit at the head of the next step, on the path from one theta to the next).
        bool prewaited = false;
        auto wait_next_stage_early = [&]() {
            prewaited = (step_count + 1u) * (uint32_t)passes < total_stages;  // there is a next stage in this launch
            if (prewaited) bounded_mbar_wait(full_bars + (uint32_t)(cs_slot * 8), cs_phase, aborted, P);
        };

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
            // thread f's master copy of theta_f and the update rule's state for it (velocity; or first and second moment)
            T thm[FPT], st1[FPT], st2[FPT];
            T* st1_g = static_cast<T*>(P.opt1) + (size_t)chain * p;
            T* st2_g = static_cast<T*>(P.opt2) + (size_t)chain * p;
#pragma unroll
            for (int i = 0; i < FPT; ++i) {
                const int f = tid + i * nthreads;
                thm[i] = (f < p) ? theta_g[f] : T(0);
                st1[i] = (f < p && opt_kind != kOptSgd) ? st1_g[f] : T(0);
                st2[i] = (f < p && opt_kind == kOptAdam) ? st2_g[f] : T(0);
            }
            double b1pow = P.adam_b1pow0, b2pow = P.adam_b2pow0;  // beta^t after the steps of earlier calls
            long long sched_pos = P.sched_pos0;                   // updates already taken in this pass

            for (int t = 0; t < T_rounds; ++t) {
                for (uint32_t m = 0; m < M; ++m) {
                    const bool full_batch = m * n + n <= N0;
                    RowShare sh = share_full;
                    sh.lo = m * n;
                    if (!full_batch) sh = row_share(m, n, N0, (uint32_t)g, (uint32_t)G, P.q_full, P.r_full);
                    BMGD_STAMP(0);

                    T gacc[NV];
#pragma unroll
                    for (int i = 0; i < NV; ++i) gacc[i] = T(0);

                    // sub-passes of this step in which the warp has at least one row
                    int sp_left = sp_full;
                    if (!full_batch) sp_left = (sh.cnt > warp_first) ? (int)((sh.cnt - warp_first - 1u) / (uint32_t)spp) + 1 : 0;
                    for (int sidx = 0; sidx < passes; ++sidx) {
                        if (sidx == 0) BMGD_STAMP(11);
                        if (!(sidx == 0 && prewaited)) bounded_mbar_wait(full_bars + (uint32_t)(cs_slot * 8), cs_phase, aborted, P);
                        __syncwarp();
                        if (sidx == 0) BMGD_STAMP(10);
                        const unsigned char* rowp = smem + plan.ring_off + cs_slot * stage_bytes + lane_off;
                        const unsigned char* yp = smem + plan.ring_off + cs_slot * stage_bytes + y_off;
                        int nsub = NULLSTEP ? 0 : min(sp_left, RB);
                        sp_left -= nsub;
                        if constexpr (NV * (int)sizeof(T) <= 32) {  // narrow rows: four independent rows in flight per group
                            for (; nsub >= 4; nsub -= 4, rowp += 4 * subpass_bytes, yp += 4 * y_step)
                                rows_step<T, VEC, LPR, KCH, LOGISTIC, 4>(rowp, subpass_bytes, yp, y_step, th, gacc);
                        }
                        for (; nsub >= 2; nsub -= 2, rowp += 2 * subpass_bytes, yp += 2 * y_step) {  // two independent rows in flight per group
                            if constexpr (NV <= 16) {
                                rows_step<T, VEC, LPR, KCH, LOGISTIC, 2>(rowp, subpass_bytes, yp, y_step, th, gacc);
                            } else {  // wide per-lane state: two rows' values at once would not fit the registers
                                row_step<T, VEC, LPR, KCH, LOGISTIC>(rowp, yp, th, gacc);
                                row_step<T, VEC, LPR, KCH, LOGISTIC>(rowp + subpass_bytes, yp + y_step, th, gacc);
                            }
                        }
                        if (nsub) row_step<T, VEC, LPR, KCH, LOGISTIC>(rowp, yp, th, gacc);
                        if (sidx == 0) BMGD_STAMP(13);
                        __syncwarp();  // every lane has its values in registers: the slot may be refilled
                        // A lane that has given up did not wait for the stage and must not hand its slot back: a producer
                        // would refill it while copies of the phase before are in flight, the phases of the slot's barrier
                        // would run into one another, and the wait for the last copies at the end of the launch would
                        // no longer mean that they have landed.
                        if (lane == 0 && !aborted) mbar_arrive(empty_bars + (uint32_t)(cs_slot * 8));
                        if (++cs_slot == D) { cs_slot = 0; cs_phase ^= 1u; }
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
                    consumer_sync(nthreads);
                    BMGD_STAMP(2);
                    T tot[FPT];
#pragma unroll
                    for (int i = 0; i < FPT; ++i) {
                        const int f = xf + i * nthreads;  // xf == tid unless this thread helps with another thread's pushes
                        tot[i] = (f < p && xg < xg_n) ? strided_sum(gpart + f, plan.gpart_rows, PCAP) : T(0);
                    }
                    BMGD_STAMP(3);

                    const int parity = (int)(step_count & 1u);
                    // Tag of this step's packets, in shared memory (zeroed at launch) and in global memory (tags of
                    // earlier launches are smaller): never 0, never repeated while a packet of the same slot can be read.
                    const uint32_t tag = P.tag_base + step_count + 1u;
                    const uint32_t cpk = cpk_base + (uint32_t)(parity * S * plan.cpk_stride * 8);

                    if (one_cluster) {
                        // ---- one cluster per chain: every CTA pushes its partial sums, as tagged packets, into the
                        //      shared memory of every CTA of the cluster and then sums, in rank order, the S packets per
                        //      predictor that arrive in its own.  No cluster barrier: a packet is its own flag.
                        if (S > 1) {
                            if (fast_push) {
                                if (xf < p && xg < xg_n) {
                                    const uint32_t poff = parity ? parity_bytes : 0u;
    #pragma unroll
                                    for (int w = 0; w < NW; ++w) {
                                        const unsigned long long pk = ((unsigned long long)tag << 32) | Words<T>::get(tot[0], w);
    #pragma unroll
                                        for (int i = 0; i < kFastPeers; ++i)
                                            if (i < my_peers) st_cluster_u64(push_addr[i] + poff + (uint32_t)(w * 8), pk);
                                    }
                                }
                            } else {
    #pragma unroll
                                for (int i = 0; i < FPT; ++i) {
                                    const int f = xf + i * nthreads;
                                    if (f < p && xg < xg_n) {
    #pragma unroll
                                        for (int w = 0; w < NW; ++w) {
                                            const unsigned long long pk = ((unsigned long long)tag << 32) | Words<T>::get(tot[i], w);
                                            const uint32_t mine = cpk + (uint32_t)((rank * plan.cpk_stride + f * NW + w) * 8);
                                            for (int peer = xg; peer < S; peer += xg_n) st_cluster_u64(map_to_cta(mine, (uint32_t)peer), pk);
                                        }
                                    }
                                }
                            }
                            BMGD_STAMP(8);
                            wait_next_stage_early();
    #pragma unroll
                            for (int i = 0; i < FPT; ++i) {
                                const int f = tid + i * nthreads;
                                if (f < p)
                                    tot[i] = gather_packets<T, kMaxClusterSize, kClusterChunk>(
                                        S, tag, aborted, P,
                                        [&](int k, int w) { return ld_shared_volatile_u64(cpk + (uint32_t)((k * plan.cpk_stride + f * NW + w) * 8)); });
                            }
                        }
                        BMGD_STAMP(4);
                        BMGD_STAMP(5);
                    } else {
                        // ---- several clusters per chain: reduce-scatter in the cluster (CTA r owns a slice of the
                        //      predictors and receives its peers' partial sums as tagged packets), packets through global
                        //      memory between the slice owners of different clusters, totals pushed to every peer
                        if (S > 1) {
    #pragma unroll
                            for (int i = 0; i < FPT; ++i) {
                                const int f = tid + i * nthreads;
                                if (f < p) {
                                    const int owner = f / slice;
    #pragma unroll
                                    for (int w = 0; w < NW; ++w)
                                        st_cluster_u64(map_to_cta(cpk + (uint32_t)((rank * plan.cpk_stride + (f - owner * slice) * NW + w) * 8),
                                                                  (uint32_t)owner),
                                                       ((unsigned long long)tag << 32) | Words<T>::get(tot[i], w));
                                }
                            }
                        }
                        BMGD_STAMP(4);
                        wait_next_stage_early();
                        unsigned long long* slot = P.ll + ((size_t)(team * 2 + parity) * cpc) * (size_t)P.ll_stride;
                        const uint32_t gpk = gpk_base + (uint32_t)(parity * PCAP * NW * 8);
                        // thread j of the CTA owns predictor f = rank*slice + j of the slice (all of them if S == 1)
    #pragma unroll
                        for (int i = 0; i < FPT; ++i) {
                            const int j = tid + i * nthreads;
                            const int f = rank * slice + j;
                            if (j < slice && f < p) {
                                const T mine_sum = (S > 1)
                                    ? gather_packets<T, kMaxClusterSize, kClusterChunk>(
                                          S, tag, aborted, P,
                                          [&](int k, int w) { return ld_shared_volatile_u64(cpk + (uint32_t)((k * plan.cpk_stride + j * NW + w) * 8)); })
                                    : tot[i];
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
                            const unsigned long long* src = slot + f * NW;
                            const int stride = P.ll_stride;
                            const T s = gather_packets<T, kMaxCpc, 4>(
                                cpc, tag, aborted, P, [&](int k, int w) { return ld_packet(src + (size_t)k * stride + w); });
                            if (S > 1) {
    #pragma unroll
                                for (int w = 0; w < NW; ++w) {
                                    const unsigned long long pk = ((unsigned long long)tag << 32) | Words<T>::get(s, w);
                                    const uint32_t dst = gpk + (uint32_t)((f * NW + w) * 8);
                                    for (int peer = 0; peer < S; ++peer) st_cluster_u64(map_to_cta(dst, (uint32_t)peer), pk);
                                }
                            } else {
                                tot[i] = s;  // one CTA per cluster: j == f
                            }
                        }
                        BMGD_STAMP(5);
                        if (S > 1) {
    #pragma unroll
                            for (int i = 0; i < FPT; ++i) {
                                const int f = tid + i * nthreads;
                                if (f < p)
                                    tot[i] = gather_packets<T, 1, 1>(
                                        1, tag, aborted, P,
                                        [&](int, int w) { return ld_shared_volatile_u64(gpk + (uint32_t)((f * NW + w) * 8)); });
                            }
                        }
                    }
                    BMGD_STAMP(6);

                    // ---- the thread that holds predictor f's gradient sum applies the update rule to its master copy of
                    //      theta_f (the same arithmetic in every CTA, so all copies stay bit-identical) and publishes it;
                    //      then every lane refreshes the coefficients it multiplies rows with
                    const bool full = full_batch;
                    T lr = lr_const;
                    if (cosine) {  // Section 4.4: rate of the j-th update of a pass of J updates
                        const long long j = sched_pos + 1;
                        lr = (T)(P.lr * (0.5 + 0.5 * cospi((double)j / (double)P.sched_period)));
                        sched_pos = (j == P.sched_period) ? 0 : j;
                    }
                    if (opt_kind == kOptSgd) {
                        const T scale = cosine ? lr * (full ? inv_full : inv_last) : (full ? scale_full : scale_last);
#pragma unroll
                        for (int i = 0; i < FPT; ++i) {
                            const int f = tid + i * nthreads;
                            if (f < p) { thm[i] = fma(-scale, tot[i], thm[i]); gfin[f] = thm[i]; }
                        }
                    } else if (opt_kind == kOptNesterov) {
                        const T inv = full ? inv_full : inv_last, mu = (T)P.opt_a;
#pragma unroll
                        for (int i = 0; i < FPT; ++i) {
                            const int f = tid + i * nthreads;
                            if (f < p) {
                                const T gm = tot[i] * inv;
                                st1[i] = mu * st1[i] - lr * gm;
                                thm[i] = thm[i] + mu * st1[i] - lr * gm;
                                gfin[f] = thm[i];
                            }
                        }
                    } else {  // Adam
                        const T inv = full ? inv_full : inv_last, b1 = (T)P.opt_a, b2 = (T)P.opt_b, eps = (T)P.opt_eps;
                        b1pow *= P.opt_a; b2pow *= P.opt_b;  // beta^t, in double
                        const T c1 = (T)(1.0 - b1pow), c2 = (T)(1.0 - b2pow);
#pragma unroll
                        for (int i = 0; i < FPT; ++i) {
                            const int f = tid + i * nthreads;
                            if (f < p) {
                                const T gm = tot[i] * inv;
                                st1[i] = b1 * st1[i] + (T(1) - b1) * gm;
                                st2[i] = b2 * st2[i] + (T(1) - b2) * gm * gm;
                                thm[i] = thm[i] - lr * (st1[i] / c1) / (sqrt(st2[i] / c2) + eps);
                                gfin[f] = thm[i];
                            }
                        }
                    }
                    BMGD_STAMP(9);
                    if (aborted) *cta_abort = 1;  // a thread of this CTA has given up a wait: after the barrier all consumers know
                    consumer_sync(nthreads);
                    const int stop = *cta_abort;
                    {
                        const T* gf = gfin + sub * VEC;
#pragma unroll
                        for (int k = 0; k < KCH; ++k) {
                            if constexpr (CB == 16 && sizeof(T) == 4) {
                                const float4 v = *reinterpret_cast<const float4*>(gf + k * LPR * VEC);
                                th[k * VEC + 0] = v.x; th[k * VEC + 1] = v.y; th[k * VEC + 2] = v.z; th[k * VEC + 3] = v.w;
                            } else {
#pragma unroll
                                for (int e = 0; e < VEC; ++e) th[k * VEC + e] = gf[k * LPR * VEC + e];
                            }
                        }
                    }
                    BMGD_STAMP(7);
                    ++step_count;
                    if (stop) goto consumers_done;  // the same decision in every consumer thread; theta is not written back
                }
            }

            if (g == 0) {
#pragma unroll
                for (int i = 0; i < FPT; ++i) {
                    const int f = tid + i * nthreads;
                    if (f < p) {
                        theta_g[f] = thm[i];
                        if (opt_kind != kOptSgd) st1_g[f] = st1[i];
                        if (opt_kind == kOptAdam) st2_g[f] = st2[i];
                    }
                }
            }
        }
    consumers_done:;
    }
    if (S > 1) {  // no CTA leaves while a peer's packets for it may still be on their way
        __syncwarp();
        cluster_arrive_release();
        cluster_wait_acquire();
    }
}

}  // namespace bmgdk
