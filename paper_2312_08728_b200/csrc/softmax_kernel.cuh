// Softmax (multinomial logistic) BMGD step kernel: bf16 rows, fp32 parameters W [p][C].
// The C-class extension of the logistic step of Eq. (2.1); the paper itself stops at generalised
// linear models.  Per step, on the mini-batch rows X_b [n_m x p]:
//     Z = X_b W,  P = softmax over classes,  R = P - onehot(y),  W <- W - (alpha/n_m) X_b^T R.
//
// One thread-block cluster of S CTAs works on a chain, split by predictors: CTA r owns a slice of ps = NP*64
// predictors (NP panels of 64; predictors from p on are zero columns), i.e. ps rows of W.  With several chains
// (replicates with their own W and their own partitions) every cluster takes chains cluster, cluster + clusters, ...
// Per step:
//   1. the CTA's slice of the mini-batch rows (256 row slots x ps bf16) was gathered by cp.async into shared
//      memory one step ahead by sixteen producer warps, as NP panels of [256 rows][128 bytes] with the 128-byte
//      swizzle the tensor core reads (16-byte chunk index XOR row%8); their arrival is counted on an mbarrier;
//   2. forward: partial logits Zp = X_slice W_slice, bf16 x bf16 -> fp32, on the 5th-generation tensor cores
//      (tcgen05.mma, M=128 N=16 K=16, accumulators in tensor memory).  The two halves of the 256 rows are issued by
//      two threads and committed to two mbarriers, so that reading the first half out of tensor memory overlaps
//      the second half's arithmetic;
//   3. the partial logits are reduce-scattered through distributed shared memory: the thread that holds row
//      slot i sends its classes in 16-byte pieces (st.async) straight into the shared memory of the CTA that owns
//      that row; the bytes are counted on the owner's mbarrier, so there is no cluster barrier and no flag.  The
//      owner sums the S partials in fixed order, takes the softmax and the residual R;
//   4. R (bf16) is sent to every peer the same way (16-byte pieces, counted on the peer's mbarrier);
//   5. backward: G_slice = X_slice^T R with the same panels read MN-major (no second copy of X); its one or two
//      tiles of 128 predictors are again issued by two threads and committed separately;
//   6. the owner threads of W_slice (fp32 master copy in registers) apply the update and refresh the bf16 copy.
// All sums have a fixed order: runs are bitwise reproducible.  Every wait is bounded (see glm_kernel.cuh).
//
// USE_TC = false runs the two contractions on the CUDA cores from the same shared-memory layout (same bf16
// inputs, fp32 accumulation): the cross-check of the tensor-core path.  NULLSTEP = true is the latency probe: the
// waits, exchanges and updates of every step without gathering or multiplying rows (the gradient is zero).
#pragma once
#include <cstdint>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "glm_kernel.cuh"
#include "shuffle.cuh"

namespace bmgdk {

constexpr int kSmxThreads = 768;     // 8 compute warps (one thread per row slot) + 16 producer warps
constexpr int kSmxCompute = 256;     // compute threads
constexpr int kSmxRows = 256;        // row slots per step (mini-batch size limit)
constexpr int kSmxMaxPanels = 3;     // 64-predictor panels per CTA slice
constexpr int kSmxClasses = 16;      // padded class count
// Accumulators per contraction in tensor memory (K-step ks goes to accumulator ks % kSmxAcc, the partial sums are added
// in registers after the read-out).  Measured on B200: a 128 x 16 x 16 multiply-accumulate takes about 70 cycles of the
// tensor core whether or not it accumulates into the tile of the one before it, so more than one accumulator only adds
// read-outs (four of them: forward 2,590 -> 2,730 cycles, backward 1,940 -> 2,250).
constexpr unsigned long long kSmxLingerNs = 20000ull;  // how long a CTA of a launch that was given up stays before it exits
constexpr int kSmxAcc = 1;
constexpr int kSmxTmemCols = 4 * kSmxAcc * kSmxClasses;  // forward halves 0 and 1, backward tiles 0 and 1

struct SoftmaxParams {
    const void* X;      // [N0][p] bf16
    const int* y;       // [N0] labels
    float* W;           // [Rc][p][C] fp32
    int* status;
    unsigned long long seed;
    unsigned long long timeout_ns;
    double scale_full, scale_last;
    uint32_t N0, n, M;
    int T, p, C, S, NP, Rc, nclusters;
    int ntile;          // tiles of 256 row slots per mini-batch
    uint32_t chain0;
    int fixed_partition;
    uint32_t mbar_mask;
#ifdef BMGD_TRACE
    long long* trace;   // debug build: clock stamps of thread 0 of every CTA (null: none taken)
#endif
};

struct SoftmaxLaunchInfo {
    int launches, grid_ctas, cluster_size, threads, depth, smem, chains_in_flight, cuda_error;
};

inline int64_t softmax_scratch_bytes(int /*p*/, int /*C*/) { return 256; }

// ---------------------------------------------------------------- shared-memory plan
struct SmxPlan {
    int panels;       // panels a buffer is laid out for: at least two, so that a 128-predictor tile never leaves it
    int xbuf_bytes;   // one X buffer: `panels` panels of 256 rows x 128 bytes
    int x_off[2], wt_off, zpart_off, r_off, lab_off, bar_off, total;
};
__host__ __device__ inline SmxPlan smx_plan(int NP) {
    SmxPlan s;
    s.panels = NP < 2 ? 2 : NP;
    s.xbuf_bytes = s.panels * kSmxRows * 128;
    s.x_off[0] = 0;
    s.x_off[1] = s.xbuf_bytes;
    s.wt_off = 2 * s.xbuf_bytes;                               // [panels][16 classes][128 B], swizzled like X
    s.zpart_off = s.wt_off + s.panels * kSmxClasses * 128;     // [S][256/S rows][16] fp32 = 16 KB
    s.r_off = s.zpart_off + kSmxRows * kSmxClasses * 4;        // residuals, 8 KB (layout depends on the path)
    s.lab_off = s.r_off + kSmxRows * kSmxClasses * 2;          // [2][256] labels of the rows this CTA owns
    s.bar_off = s.lab_off + 2 * kSmxRows * 4;                  // mbarriers, tensor-memory base address, stop flag
    s.total = s.bar_off + 128;
    return s;
}

// byte offset of predictor-chunk `chunk` (8 bf16) of row `row` inside a buffer of panels [panel][rows][128 B]
__device__ __forceinline__ int smx_chunk_off(int row, int chunk, int rows_per_panel) {
    return ((chunk >> 3) * rows_per_panel + row) * 128 + (((chunk & 7) ^ (row & 7)) << 4);
}

// 16 bytes into a peer's shared memory; the bytes are counted on the mbarrier `bar` of that same peer.  Only for
// CTAs other than the executing one (the instruction is not defined for one's own shared memory).
__device__ __forceinline__ void st_async_16(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint32_t bar) {
    asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
                 ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d), "r"(bar) : "memory");
}

// named CTA barrier: `count` threads take part
__device__ __forceinline__ void named_sync(int id, int count) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

// ---------------------------------------------------------------- bounded waits
struct WaitCtx {
    int* status;
    unsigned long long timeout_ns;
    uint32_t mask;
    bool aborted;
};
// `likely_done`: the phase has usually completed long before (a buffer filled a step ahead): ask once without suspending
// the thread first, which answers faster than try_wait does even on a completed phase.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, WaitCtx& w, bool likely_done = false) {
    if (likely_done && mbar_test_wait(bar, parity)) return;
    unsigned long long t0 = 0;
    uint32_t spins = 0;
    // (with no budget at all, mask 0, the wait asks without suspending the thread: it gives up at its first look)
    while (!w.aborted && !(w.mask ? mbar_try_wait(bar, parity) : mbar_test_wait(bar, parity))) {
        if ((++spins & w.mask) == 0u) {
            const unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            if (now - t0 >= w.timeout_ns || ((volatile int*)w.status)[1] != 0) {
                atomicCAS(w.status, 0, kStatusTimeout);
                atomicExch(w.status + 1, 1);
                w.aborted = true;
            }
        }
    }
}

// ---------------------------------------------------------------- tensor-core plumbing (tcgen05, cta_group::1)
__device__ __forceinline__ void tc_alloc(uint32_t dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// D[tmem] (+)= A[smem] * B[smem], bf16 inputs, fp32 accumulate; issued by one thread
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// the mbarrier gets one arrival when every MMA issued so far by this thread has finished
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 16 consecutive fp32 columns of this thread's tensor-memory lane
__device__ __forceinline__ void tc_load16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
// sum of the kSmxAcc partial accumulators (16 columns each, side by side from column `col` on) of this thread's lane
__device__ __forceinline__ void tc_load_sum(uint32_t tmem_lane_base, uint32_t col, float (&v)[16]) {
    tc_load16(tmem_lane_base + col, v);
#pragma unroll
    for (int a = 1; a < kSmxAcc; ++a) {
        float t[16];
        tc_load16(tmem_lane_base + col + (uint32_t)(a * kSmxClasses), t);
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] += t[i];
    }
}
// shared-memory matrix descriptor, 128-byte swizzle: start address, leading and stride byte offsets in 16-byte units
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFFu);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;   // descriptor version of this architecture
    d |= (uint64_t)2 << 61;   // 128-byte swizzle
    return d;
}
// instruction descriptor: fp32 accumulator, bf16 A and B, M x N tile, A read K-major or MN-major, B K-major
__device__ __forceinline__ uint32_t tc_idesc(int M, int N, bool a_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}

// ---------------------------------------------------------------- the kernel

template <bool USE_TC, bool NULLSTEP>
__global__ void __launch_bounds__(kSmxThreads, 1) softmax_kernel(const SoftmaxParams P) {
    extern __shared__ __align__(1024) unsigned char smx_smem[];
    unsigned char* const smem = smx_smem;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int S = P.S, NP = P.NP, C = P.C, p = P.p;
    const int rank = (S > 1) ? (int)cluster_ctarank() : 0;
    const int cluster = (int)blockIdx.x / S;
    const int ps = NP * 64;                 // predictor capacity of this CTA's slice
    const int f_first = rank * ps;
    const int RO = kSmxRows / S;            // row slots whose logits this CTA sums
    const uint32_t N0 = P.N0, n = P.n, M = P.M;
    const SmxPlan plan = smx_plan(NP);
    unsigned char* xbuf[2] = {smem + plan.x_off[0], smem + plan.x_off[1]};
    unsigned char* wt = smem + plan.wt_off;
    float* zpart = reinterpret_cast<float*>(smem + plan.zpart_off);
    unsigned char* rbuf = smem + plan.r_off;
    int* lab = reinterpret_cast<int*>(smem + plan.lab_off);
    // mbarriers: rows of buffer b have landed / buffer b may be refilled; forward half h / backward tile t has finished;
    // the partial logits of the rows this CTA owns / everybody's residuals have arrived
    const uint32_t bars = smem_u32(smem + plan.bar_off);
    const uint32_t xfull = bars, xempty = bars + 16, fbar = bars + 32, gbar = bars + 48, zbar = bars + 64, rbar = bars + 72;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + plan.bar_off + 80);
    volatile int* const cta_abort = reinterpret_cast<volatile int*>(smem + plan.bar_off + 96);

    const __nv_bfloat16* Xg = static_cast<const __nv_bfloat16*>(P.X);
    const FeistelDomain dom = make_domain(N0);
    WaitCtx wc{P.status, P.timeout_ns, P.mbar_mask, false};
    const int nch = (cluster < P.Rc) ? (P.Rc - cluster + P.nclusters - 1) / P.nclusters : 0;
    // A mini-batch of more than 256 rows is taken in `ntile` tiles of 256 row slots: each tile goes through the gather,
    // the forward contraction, the two exchanges and the backward contraction on its own (the backward one adds into
    // the same accumulators); W is updated after the last tile.  "step" below counts tiles.
    const uint32_t ntile = (uint32_t)P.ntile;
    const uint32_t steps_per_chain = (uint32_t)P.T * M * ntile;
    const uint32_t total_steps = (uint32_t)nch * steps_per_chain;
    const int zchunks = (C + 3) >> 2;       // 16-byte pieces of a row's logits that carry real classes
    const int ntiles = NP > 2 ? 2 : 1;      // backward tiles of 128 predictors (tile 1: predictors 64..191)

    // ---- set-up
    for (int i = tid * 16; i < plan.total; i += kSmxThreads * 16) st_shared_zero16(smem_u32(smem + i));
    __syncthreads();
    if (tid == 0) {
        constexpr uint32_t kProducerLanes = (kSmxThreads - kSmxCompute);
        for (int b = 0; b < 2; ++b) {
            mbar_init(xfull + (uint32_t)(b * 8), kProducerLanes);
            mbar_init(xempty + (uint32_t)(b * 8), 1u);
            mbar_init(fbar + (uint32_t)(b * 8), 1u);
            mbar_init(gbar + (uint32_t)(b * 8), 1u);
        }
        mbar_init(zbar, 1u);
        mbar_init(rbar, 1u);
        *cta_abort = 0;
        fence_barrier_init();
    }
    uint32_t tmem_base = 0;
    if constexpr (USE_TC) {
        if (warp == 0) tc_alloc(smem_u32(tmem_slot), (uint32_t)kSmxTmemCols);
        tc_fence_before();
    }
    fence_async_proxy();
    __syncthreads();
    if constexpr (USE_TC) {
        tc_fence_after();
        tmem_base = *tmem_slot;
    }
    if (S > 1) {  // peers must be running, with their barriers initialised, before anyone writes into their shared memory
        cluster_arrive_release();
        cluster_wait_acquire();
    }

    auto step_rows = [&](uint32_t step, uint32_t& lo, uint32_t& nm) {  // rows [lo, lo + nm) of the round's order: this tile's
        const uint32_t in_chain = step % steps_per_chain;
        const uint32_t m = (in_chain / ntile) % M, tau = in_chain % ntile;
        const uint32_t batch = min(n, N0 - m * n);
        lo = m * n + tau * (uint32_t)kSmxRows;
        nm = batch > tau * (uint32_t)kSmxRows ? min((uint32_t)kSmxRows, batch - tau * (uint32_t)kSmxRows) : 0u;
    };

    if (warp >= kSmxCompute / 32) {
        // ================================================================ producer warps
        // Sixteen warps take 16 row slots each: lanes 0..15 evaluate the shuffle for one slot each, then the warp copies
        // the 16 rows one after the other, lanes taking consecutive 16-byte chunks of the CTA's slice.  They run one step
        // ahead of the compute warps, through mini-batch, round and chain boundaries.
        constexpr int kProducers = kSmxThreads / 32 - kSmxCompute / 32;
        constexpr int kSlots = kSmxRows / kProducers;
        const int pw = warp - kSmxCompute / 32;
        const int slot0 = pw * kSlots;
        const int chunk_first = f_first + lane * 8;            // first predictor of this lane's chunk
        const bool active = lane < NP * 8 && chunk_first < p;  // chunks from p on stay zero (zeroed once, never written)
        const __nv_bfloat16* src_lane = Xg + chunk_first;
        RoundKeys rk = round_keys(P.seed, P.chain0 + (uint32_t)cluster, 0u);
        uint32_t rk_chain = 0, rk_round = 0;
        for (uint32_t step = 0; step < total_steps; ++step) {
            const int b = (int)(step & 1u);
            const uint32_t ci = step / steps_per_chain;
            const uint32_t t = P.fixed_partition ? 0u : (step % steps_per_chain) / (M * ntile);
            if (ci != rk_chain || t != rk_round) {
                rk = round_keys(P.seed, P.chain0 + (uint32_t)(cluster + (int)ci * P.nclusters), t);
                rk_chain = ci; rk_round = t;
            }
            uint32_t lo, nm;
            step_rows(step, lo, nm);
            const int slot = slot0 + lane;
            uint32_t r = 0xFFFFFFFFu;
            if (!NULLSTEP && lane < kSlots && (uint32_t)slot < nm) r = perm_index(lo + (uint32_t)slot, dom, rk);
            // the buffer's last reader (the backward contraction two steps ago) must have finished
            mbar_wait(xempty + (uint32_t)(b * 8), ((step >> 1) & 1u) ^ 1u, wc, true);
            wc.aborted = __any_sync(0xFFFFFFFFu, wc.aborted);
            if (wc.aborted) break;
            if constexpr (!NULLSTEP) {
                const uint32_t dst_lane = smem_u32(xbuf[b]) + (uint32_t)((lane >> 3) * kSmxRows * 128);
#pragma unroll 4
                for (int i = 0; i < kSlots; ++i) {
                    const uint32_t ri = __shfl_sync(0xFFFFFFFFu, r, i);
                    const int row = slot0 + i;
                    const uint32_t dst = dst_lane + (uint32_t)(row * 128 + (((lane & 7) ^ (row & 7)) << 4));
                    if (active) {
                        const bool have = ri != 0xFFFFFFFFu;  // an empty slot is filled with zeros: it contributes nothing
                        cp_async_fill<16>(dst, src_lane + (have ? (size_t)ri * p : 0), have);
                    }
                }
                // labels of the slots this CTA owns, for the step that will read buffer b
                if (lane < kSlots && slot / RO == rank) {
                    const bool have = r != 0xFFFFFFFFu;
                    cp_async_fill<4>(smem_u32(lab + b * kSmxRows + slot % RO), P.y + (have ? r : 0u), have);
                }
            }
            // the lane waits for its own copies, makes them visible to the tensor core's reads (they went through the
            // generic proxy) and only then counts itself in; the producers are a step ahead, so this wait is off the
            // path from one W to the next
            asm volatile("cp.async.commit_group;" ::: "memory");
            cp_async_wait_all();
            if constexpr (USE_TC) fence_async_proxy();
            mbar_arrive(xfull + (uint32_t)(b * 8));
        }
        cp_async_wait_all();
    } else {
        // ================================================================ compute warps (thread = row slot)
        // W master: thread f (< 128) owns predictor f of the slice, thread f + 64 owns predictor f >= 128: the threads
        // that read that predictor's row of the backward accumulator from tensor memory
        const int my_f = (tid < 128) ? tid : (tid >= 192 ? tid - 64 : -1);
        const bool owns_w = my_f >= 0 && my_f < ps && f_first + my_f < p;
        float w[kSmxClasses];
        auto write_wt = [&]() {  // bf16 copy of W_slice^T in the panel layout [panel][class][128 B]
            if (owns_w) {
#pragma unroll
                for (int c = 0; c < kSmxClasses; ++c)
                    *reinterpret_cast<__nv_bfloat16*>(wt + smx_chunk_off(c, my_f >> 3, kSmxClasses) + (my_f & 7) * 2) =
                        __float2bfloat16_rn(w[c]);
            }
            if constexpr (USE_TC) fence_async_proxy();  // the tensor core reads these bytes
        };
        // where this thread's pieces go: the partial logits of its row slot to the CTA that owns the row, the residual
        // chunks it forwards (two per thread when S > 1) to one peer each
        const int z_owner = tid / RO, z_rloc = tid % RO;
        const uint32_t z_local = smem_u32(zpart + ((size_t)rank * RO + z_rloc) * kSmxClasses);
        const bool z_remote = z_owner != rank;
        const uint32_t z_dst = z_remote ? map_to_cta(z_local, (uint32_t)z_owner) : z_local;
        const uint32_t z_bar = z_remote ? map_to_cta(zbar, (uint32_t)z_owner) : zbar;
        const uint32_t z_expect = (uint32_t)((S - 1) * RO * zchunks * 16);    // bytes of partial logits from the peers per step
        const uint32_t r_expect = (uint32_t)((S - 1) * 2 * RO * 16);          // bytes of residuals from the peers per step
        const int per_class = RO / 8;  // 16-byte chunks (8 row slots) of one class among the rows this CTA owns
        // The owned part of R is 2*RO chunks of 16 bytes and every one of them goes to every peer: 2*RO*S pairs, two per
        // thread in a cluster of 16.  Where each pair's chunk sits and where it lands is worked out once.
        constexpr int kPushSlots = 2;
        const int push_pairs = (S > 1) ? 2 * RO * S : 0;
        uint32_t push_src[kPushSlots], push_dst[kPushSlots], push_bar[kPushSlots];
#pragma unroll
        for (int i = 0; i < kPushSlots; ++i) {
            const int q = tid + i * kSmxCompute;
            push_src[i] = 0u; push_dst[i] = 0u; push_bar[i] = 0u;
            if (q < push_pairs && push_pairs <= kPushSlots * kSmxCompute) {
                const int chunk = q / S, peer = q % S;
                const int off = USE_TC ? smx_chunk_off(chunk / per_class, rank * per_class + chunk % per_class, kSmxClasses)
                                       : (rank * RO * kSmxClasses * 2 + chunk * 16);
                if (peer != rank) {
                    push_src[i] = smem_u32(rbuf + off);
                    push_dst[i] = map_to_cta(push_src[i], (uint32_t)peer);
                    push_bar[i] = map_to_cta(rbar, (uint32_t)peer);
                }
            }
        }

        uint32_t step = 0;
        for (int ci = 0; ci < nch; ++ci) {
            const int chain = cluster + ci * P.nclusters;
            float* Wg = P.W + (size_t)chain * p * C;
#pragma unroll
            for (int c = 0; c < kSmxClasses; ++c) w[c] = 0.f;
            if (owns_w) {
#pragma unroll
                for (int c = 0; c < kSmxClasses; ++c)
                    if (c < C) w[c] = Wg[(size_t)(f_first + my_f) * C + c];
            }
            write_wt();
            named_sync(1, kSmxCompute);

            uint32_t m = 0, tau = 0;  // mini-batch of the round and tile of the mini-batch (kept by counting: no division here)
            float gr_cc[kSmxClasses];  // CUDA-core path: the gradient row of this thread's predictor, summed over the tiles
#pragma unroll
            for (int c = 0; c < kSmxClasses; ++c) gr_cc[c] = 0.f;
            for (uint32_t s_in = 0; s_in < steps_per_chain; ++s_in, ++step) {
                const int b = (int)(step & 1u);
                const uint32_t par = step & 1u;           // phase parity of the once-per-tile barriers
                const uint32_t xpar = (step >> 1) & 1u;   // and of the per-buffer ones
                const uint32_t batch = min(n, N0 - m * n);  // rows of the mini-batch
                const uint32_t nm = batch > tau * (uint32_t)kSmxRows ? min((uint32_t)kSmxRows, batch - tau * (uint32_t)kSmxRows) : 0u;
                const bool first_tile = tau == 0, last_tile = tau + 1 == ntile;
                if (++tau == ntile) { tau = 0; if (++m == M) m = 0; }
#ifdef BMGD_TRACE
                const uint32_t step_count = step;
#endif
                BMGD_STAMP(0);
                if (tid == 64) {  // this step's incoming bytes (they may start to arrive before this line runs); a thread of a warp that issues no contraction
                    if (S > 1) { mbar_arrive_expect_tx(zbar, z_expect); mbar_arrive_expect_tx(rbar, r_expect); }
                    else { mbar_arrive(zbar); mbar_arrive(rbar); }
                }
                mbar_wait(xfull + (uint32_t)(b * 8), xpar, wc, true);  // this step's rows (gathered during the previous step)
                BMGD_STAMP(1);

                // ---- forward: partial logits of row slot `tid` over this CTA's predictors
                float z[kSmxClasses];
#pragma unroll
                for (int c = 0; c < kSmxClasses; ++c) z[c] = 0.f;
                if constexpr (USE_TC) {
                    const int half = warp >> 2;
                    if ((tid & 127) == 0) {  // threads 0 and 128 issue one half each
                        if constexpr (!NULLSTEP) {
                            // (the rows and the bf16 copy of W were made visible to the tensor core by their writers)
                            tc_fence_after();
                            const uint32_t idesc = tc_idesc(128, kSmxClasses, false);
                            const uint32_t xa = smem_u32(xbuf[b]), wb = smem_u32(wt);
                            for (int ks = 0; ks < NP * 4; ++ks) {  // K = 16 predictors per instruction
                                const uint32_t a_addr = xa + (uint32_t)((ks >> 2) * kSmxRows * 128 + half * 128 * 128 + (ks & 3) * 32);
                                const uint32_t b_addr = wb + (uint32_t)((ks >> 2) * kSmxClasses * 128 + (ks & 3) * 32);
                                tc_mma_bf16(tmem_base + (uint32_t)((half * kSmxAcc + (ks % kSmxAcc)) * kSmxClasses),
                                            tc_smem_desc(a_addr, 16, 1024), tc_smem_desc(b_addr, 16, 1024), idesc,
                                            ks >= kSmxAcc ? 1u : 0u);
                            }
                            tc_commit(fbar + (uint32_t)(half * 8));
                        } else {
                            mbar_arrive(fbar + (uint32_t)(half * 8));
                        }
                    }
                    mbar_wait(fbar + (uint32_t)(half * 8), par, wc);
                    if constexpr (!NULLSTEP) {
                        tc_fence_after();
                        // warp w reads lanes 32*(w%4).. of accumulator w/4: lane = row slot within the half
                        tc_load_sum(tmem_base + ((uint32_t)((warp & 3) * 32) << 16), (uint32_t)(half * kSmxAcc * kSmxClasses), z);
                        tc_fence_before();
                    }
                } else if constexpr (!NULLSTEP) {
                    for (int ch = 0; ch < NP * 8; ++ch) {
                        const uint4 xv = *reinterpret_cast<const uint4*>(xbuf[b] + smx_chunk_off(tid, ch, kSmxRows));
                        const __nv_bfloat16* xe = reinterpret_cast<const __nv_bfloat16*>(&xv);
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const float xf = __bfloat162float(xe[e]);
                            const int f = ch * 8 + e;
#pragma unroll
                            for (int c = 0; c < kSmxClasses; ++c) {
                                const __nv_bfloat16 wv =
                                    *reinterpret_cast<const __nv_bfloat16*>(wt + smx_chunk_off(c, f >> 3, kSmxClasses) + (f & 7) * 2);
                                z[c] = fmaf(xf, __bfloat162float(wv), z[c]);
                            }
                        }
                    }
                }
                BMGD_STAMP(2);

                // ---- reduce-scatter of the partial logits: row slot -> the CTA that owns it, counted on its barrier
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4) {
                    if (c4 >= zchunks) continue;
                    if (z_remote)
                        st_async_16(z_dst + (uint32_t)(c4 * 16), __float_as_uint(z[c4 * 4]), __float_as_uint(z[c4 * 4 + 1]),
                                    __float_as_uint(z[c4 * 4 + 2]), __float_as_uint(z[c4 * 4 + 3]), z_bar);
                    else  // rows this CTA owns itself: a plain store, seen by the other threads after the barrier below
                        *reinterpret_cast<float4*>(zpart + ((size_t)rank * RO + z_rloc) * kSmxClasses + c4 * 4) =
                            make_float4(z[c4 * 4], z[c4 * 4 + 1], z[c4 * 4 + 2], z[c4 * 4 + 3]);
                }
                named_sync(3, kSmxCompute);
                mbar_wait(zbar, par, wc);
                BMGD_STAMP(3);

                // ---- softmax and residual for the rows this CTA owns
                for (int r0 = 0; r0 < RO; r0 += 16) {
                    const int rloc = r0 + (tid >> 4), c = tid & 15;
                    const int slot = rank * RO + rloc;
                    float zz = 0.f;
                    for (int src = 0; src < S; ++src) zz += zpart[((size_t)src * RO + rloc) * kSmxClasses + c];
                    const bool live = c < C;
                    float mx = live ? zz : -INFINITY;
#pragma unroll
                    for (int off = 8; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, off));
                    float e = live ? __expf(zz - mx) : 0.f;
                    float den = e;
#pragma unroll
                    for (int off = 8; off > 0; off >>= 1) den += __shfl_xor_sync(0xFFFFFFFFu, den, off);
                    float res = 0.f;
                    if (!NULLSTEP && live && (uint32_t)slot < nm) res = __fdividef(e, den) - (c == lab[b * kSmxRows + rloc] ? 1.f : 0.f);
                    // tensor-core path: R^T as B operand, [row panel of 64][class][128 B] swizzled; otherwise [row][class]
                    const int off = USE_TC ? (smx_chunk_off(c, slot >> 3, kSmxClasses) + (slot & 7) * 2) : (slot * kSmxClasses + c) * 2;
                    *reinterpret_cast<__nv_bfloat16*>(rbuf + off) = __float2bfloat16_rn(res);
                }
                if constexpr (USE_TC) fence_async_proxy();  // the backward contraction reads these bytes
                if (wc.aborted) *cta_abort = 1;
                named_sync(2, kSmxCompute);  // the owned part of R is complete in this CTA's shared memory
                const int stop = *cta_abort;
                // ---- the owned part of R is 2*RO chunks of 16 bytes: each goes to every peer, counted on the peer's barrier
                if (push_pairs > 0 && push_pairs <= kPushSlots * kSmxCompute) {
#pragma unroll
                    for (int i = 0; i < kPushSlots; ++i) {
                        if (push_bar[i] == 0u) continue;
                        uint4 v;
                        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(push_src[i]) : "memory");
                        st_async_16(push_dst[i], v.x, v.y, v.z, v.w, push_bar[i]);
                    }
                } else if (S > 1) {
                    for (int q = tid; q < 2 * RO * S; q += kSmxCompute) {
                        const int chunk = q / S, peer = q % S;
                        if (peer == rank) continue;
                        const int off = USE_TC ? smx_chunk_off(chunk / per_class, rank * per_class + chunk % per_class, kSmxClasses)
                                               : (rank * RO * kSmxClasses * 2 + chunk * 16);
                        const uint4 v = *reinterpret_cast<const uint4*>(rbuf + off);
                        st_async_16(map_to_cta(smem_u32(rbuf + off), (uint32_t)peer), v.x, v.y, v.z, v.w, map_to_cta(rbar, (uint32_t)peer));
                    }
                }
                BMGD_STAMP(4);
                mbar_wait(rbar, par, wc);
                BMGD_STAMP(5);

                // ---- backward: gradient rows of this CTA's predictors
                float gr[kSmxClasses];
#pragma unroll
                for (int c = 0; c < kSmxClasses; ++c) gr[c] = 0.f;
                if constexpr (USE_TC) {
                    const int tile = tid >= 128 ? 1 : 0;   // threads 0..127 read tile 0, threads 192..255 the upper half of tile 1
                    if ((tid & 127) == 0 && tile < ntiles) {
                        if constexpr (!NULLSTEP) {
                            fence_async_proxy();  // own and peers' residuals were written through the generic proxy
                            tc_fence_after();
                            const uint32_t idesc = tc_idesc(128, kSmxClasses, true);
                            const uint32_t xa = smem_u32(xbuf[b]), rb = smem_u32(rbuf);
                            for (int ks = 0; ks < kSmxRows / 16; ++ks) {  // K = 16 row slots per instruction
                                const uint32_t a_addr = xa + (uint32_t)(tile * kSmxRows * 128 + ks * 16 * 128);
                                const uint32_t b_addr = rb + (uint32_t)((ks >> 2) * kSmxClasses * 128 + (ks & 3) * 32);
                                tc_mma_bf16(tmem_base + (uint32_t)(((2 + tile) * kSmxAcc + (ks % kSmxAcc)) * kSmxClasses),
                                            tc_smem_desc(a_addr, kSmxRows * 128, 1024), tc_smem_desc(b_addr, 16, 1024), idesc,
                                            (ks >= kSmxAcc || !first_tile) ? 1u : 0u);
                            }
                            tc_commit(gbar + (uint32_t)(tile * 8));
                        } else {
                            mbar_arrive(gbar + (uint32_t)(tile * 8));
                        }
                    }
                    if (tile < ntiles) {
                        mbar_wait(gbar + (uint32_t)(tile * 8), par, wc);
                        if (!NULLSTEP && last_tile) {
                            tc_fence_after();
                            if (tid < 128) tc_load_sum(tmem_base + ((uint32_t)((warp & 3) * 32) << 16), (uint32_t)(2 * kSmxAcc * kSmxClasses), gr);
                            else if (tid >= 192) tc_load_sum(tmem_base + ((uint32_t)((warp & 3) * 32) << 16), (uint32_t)(3 * kSmxAcc * kSmxClasses), gr);
                            tc_fence_before();
                        }
                    }
                    // both tiles have finished reading the rows: the buffer may be refilled
                    if (tid == 0 && ntiles > 1) mbar_wait(gbar + 8u, par, wc);
                    if (tid == 0) mbar_arrive(xempty + (uint32_t)(b * 8));
                } else {
                    if (!NULLSTEP && owns_w) {
                        for (int row = 0; row < kSmxRows; ++row) {
                            const float xf = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(
                                xbuf[b] + smx_chunk_off(row, my_f >> 3, kSmxRows) + (my_f & 7) * 2));
                            const __nv_bfloat16* rr = reinterpret_cast<const __nv_bfloat16*>(rbuf + row * kSmxClasses * 2);
#pragma unroll
                            for (int c = 0; c < kSmxClasses; ++c) gr_cc[c] = fmaf(xf, __bfloat162float(rr[c]), gr_cc[c]);
                        }
                    }
                    if (last_tile) {
#pragma unroll
                        for (int c = 0; c < kSmxClasses; ++c) { gr[c] = gr_cc[c]; gr_cc[c] = 0.f; }
                    }
                    named_sync(3, kSmxCompute);  // every thread has read the rows and the residuals
                    if (tid == 0) mbar_arrive(xempty + (uint32_t)(b * 8));
                }
                BMGD_STAMP(6);

                // ---- update of W_slice and of its bf16 copy
                if (last_tile) {
                    const float scale = (float)((batch == n) ? P.scale_full : P.scale_last);
                    if (owns_w) {
#pragma unroll
                        for (int c = 0; c < kSmxClasses; ++c) w[c] = fmaf(-scale, gr[c], w[c]);
                    }
                    write_wt();
                }
                // every thread is past this tile's contractions (the residual buffer and the tensor-memory tiles may be
                // reused) and, after the last tile, the bf16 copy is complete before the next forward contraction reads it
                named_sync(1, kSmxCompute);
                BMGD_STAMP(7);
                if (stop) goto compute_done;  // the same decision in every compute thread; W is not written back
            }
            if (owns_w) {
#pragma unroll
                for (int c = 0; c < kSmxClasses; ++c)
                    if (c < C) Wg[(size_t)(f_first + my_f) * C + c] = w[c];
            }
        }
    compute_done:;
    }

    __syncthreads();
    if constexpr (USE_TC) {
        tc_fence_after();
        if (warp == 0) tc_dealloc(tmem_base, (uint32_t)kSmxTmemCols);
    }
    if (S > 1) {  // no CTA leaves while a peer's pieces for it may still be on their way
        __syncwarp();
        cluster_arrive_release();
        cluster_wait_acquire();
        // In a launch that was given up, pieces sent with st.async may count on barriers that nobody waits for any more,
        // and nothing else says when they have landed.  Every peer has stopped sending by now (the barrier above), and a
        // piece is under way for well below a microsecond: the CTA stays for twenty before it gives up its shared memory.
        if (reinterpret_cast<volatile int*>(P.status)[1] != 0) {
            const unsigned long long t0 = global_ns();
            while (global_ns() - t0 < kSmxLingerNs) { }
        }
    }
}

// ---------------------------------------------------------------- host side

// Runs `rounds` rounds over the buffer on `stream` for Rc chains.  Shapes this kernel covers: C <= 16, any batch size
// (taken in tiles of 256 rows), p a multiple of 8 (rows are 16-byte multiples) up to 16 * 192; the predictors are spread over the smallest cluster of
// S in {1, 2, 4, 8, 16} CTAs whose slices of 64, 128 or 192 predictors hold them.  Returns a bmgd_status value.
inline int softmax_run(const void* dx, const void* dy, int64_t rows, int p, int C, int Rc, uint32_t chain0, void* W, int* status,
                       int rounds, int n, double lr, unsigned long long seed, int fixed, unsigned long long timeout_ns,
                       int cluster_size, int use_cuda_cores, int null_step, int smem_optin, cudaStream_t stream,
                       SoftmaxLaunchInfo* info) {
    *info = SoftmaxLaunchInfo{};
    if (C > kSmxClasses || p % 8 != 0) return -8;
    int S = 0, NP = 0;
    for (int s = 1; s <= 16 && !S; s <<= 1) {
        if (cluster_size && s != cluster_size) continue;
        const int np = (p + s * 64 - 1) / (s * 64);
        if (np <= kSmxMaxPanels) { S = s; NP = np; }
    }
    if (!S) return -8;
    if (((uintptr_t)dx % 16) != 0 || ((uintptr_t)dy % 4) != 0) return -1;
    const SmxPlan plan = smx_plan(NP);
    if (plan.total > smem_optin) return -8;
    const uint32_t M = (uint32_t)((rows + n - 1) / n);

    void (*fn)(const SoftmaxParams) = null_step ? softmax_kernel<true, true>
                                      : (use_cuda_cores ? softmax_kernel<false, false> : softmax_kernel<true, false>);
    cudaError_t e = cudaFuncSetAttribute((const void*)fn, cudaFuncAttributeMaxDynamicSharedMemorySize, plan.total);
    if (e == cudaSuccess && S > 8) e = cudaFuncSetAttribute((const void*)fn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) { info->cuda_error = (int)e; cudaGetLastError(); return -3; }
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3((unsigned)S, 1, 1);
    lc.blockDim = dim3(kSmxThreads, 1, 1);
    lc.dynamicSmemBytes = (size_t)plan.total;
    lc.stream = stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)S; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    lc.attrs = at; lc.numAttrs = S > 1 ? 1u : 0u;
    int nclusters = 0;
    if (S > 1) {
        e = cudaOccupancyMaxActiveClusters(&nclusters, (const void*)fn, &lc);
        if (e != cudaSuccess) { info->cuda_error = (int)e; cudaGetLastError(); return -3; }
    } else {
        int per_sm = 0, sms = 0, dev = 0;
        e = cudaGetDevice(&dev);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, (const void*)fn, kSmxThreads, (size_t)plan.total);
        if (e != cudaSuccess) { info->cuda_error = (int)e; cudaGetLastError(); return -3; }
        nclusters = per_sm * sms;
    }
    if (nclusters < 1) return -7;
    nclusters = nclusters < Rc ? nclusters : Rc;  // clusters are independent: no need for all of them to be resident at once
    const int chains_per_cluster = (Rc + nclusters - 1) / nclusters;
    const int ntile = (n + kSmxRows - 1) / kSmxRows;
    if ((uint64_t)chains_per_cluster * (uint64_t)rounds * M * (uint64_t)ntile >= 0xFFFFFFF0ull) return -1;
    lc.gridDim = dim3((unsigned)(S * nclusters), 1, 1);

    SoftmaxParams P{};
    P.X = dx; P.y = static_cast<const int*>(dy); P.W = static_cast<float*>(W); P.status = status;
    P.seed = seed; P.timeout_ns = timeout_ns;
    P.scale_full = lr / (double)n;
    P.scale_last = lr / (double)(rows - (int64_t)(M - 1) * n);
    P.N0 = (uint32_t)rows; P.n = (uint32_t)n; P.M = M; P.T = rounds; P.p = p; P.C = C; P.S = S; P.NP = NP;
    P.Rc = Rc; P.nclusters = nclusters; P.chain0 = chain0; P.ntile = ntile;
    P.fixed_partition = fixed;
    const bool tiny = timeout_ns < 1000ull;  // below a microsecond: no budget at all, every failed look gives up
    if (tiny) P.timeout_ns = 0;
    P.mbar_mask = tiny ? 0u : 0x3Fu;
#ifdef BMGD_TRACE
    P.trace = trace_buffer(0);
#endif

    e = cudaLaunchKernelEx(&lc, fn, P);
    if (e != cudaSuccess) { info->cuda_error = (int)e; cudaGetLastError(); return e == cudaErrorLaunchOutOfResources ? -7 : -3; }
    info->launches = 1; info->grid_ctas = S * nclusters; info->cluster_size = S; info->threads = kSmxThreads;
    info->depth = 2; info->smem = plan.total; info->chains_in_flight = nclusters;
    return 0;
}

}  // namespace bmgdk
