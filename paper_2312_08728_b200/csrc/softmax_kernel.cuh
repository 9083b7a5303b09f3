// Softmax (multinomial logistic) BMGD step kernel: bf16 rows, fp32 parameters W [p][C].
// The C-class extension of the logistic step of Eq. (2.1); the paper itself stops at generalised
// linear models.  Per step, on the mini-batch rows X_b [n_m x p]:
//     Z = X_b W,  P = softmax over classes,  R = P - onehot(y),  W <- W - (alpha/n_m) X_b^T R.
//
// One thread-block cluster of S CTAs works on the chain, split by predictors: CTA r owns the slice
// [r*ps, (r+1)*ps) of the p predictors (ps = NP panels of 64), i.e. ps rows of W.  Per step:
//   1. the CTA's slice of the mini-batch rows (256 row slots x ps bf16) was gathered by cp.async into
//      shared memory one step ahead by sixteen producer warps, as NP panels of [256 rows][128 bytes] with the 128-byte swizzle
//      the tensor core reads (16-byte chunk index XOR row%8);
//   2. forward: partial logits Zp = X_slice W_slice, bf16 x bf16 -> fp32, on the 5th-generation
//      tensor cores (tcgen05.mma, M=128 N=16 K=16, accumulator in tensor memory), A = the panels
//      read K-major, B = the bf16 copy of W_slice^T;
//   3. the partial logits are reduce-scattered through distributed shared memory: CTA r receives the
//      256/S rows it owns from every peer, sums them in fixed order, takes the softmax and the
//      residual R, and pushes R (bf16) to every peer;
//   4. backward: G_slice = X_slice^T R with the same panels read MN-major (no second copy of X);
//   5. the owner threads of W_slice (fp32 master copy in registers) apply the update and refresh the
//      bf16 copy.
// Two cluster barriers per step.  All sums have a fixed order: runs are bitwise reproducible.
//
// With USE_TC = false the two contractions run on the CUDA cores from the same shared-memory
// layout (same bf16 inputs, fp32 accumulation): the fallback for checking the tensor-core path.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "glm_kernel.cuh"
#include "shuffle.cuh"

namespace bmgdk {

constexpr int kSmxThreads = 768;     // 8 compute warps (one thread per row slot) + 16 producer warps
constexpr int kSmxRows = 256;       // row slots per step (mini-batch size limit)
constexpr int kSmxMaxPanels = 3;    // 64-predictor panels per CTA slice
constexpr int kSmxClasses = 16;     // padded class count

struct SoftmaxParams {
    const void* X;      // [N0][p] bf16
    const int* y;       // [N0] labels
    float* W;           // [p][C] fp32
    int* status;
    unsigned long long seed;
    unsigned long long timeout_ns;
    double scale_full, scale_last;
    uint32_t N0, n, M;
    int T, p, C, S, NP;
    int fixed_partition;
    int use_tc;
};

struct SoftmaxLaunchInfo {
    int launches, grid_ctas, cluster_size, threads, depth, smem, cuda_error;
};

inline int64_t softmax_scratch_bytes(int /*p*/, int /*C*/) { return 256; }

// ---------------------------------------------------------------- shared-memory plan
struct SmxPlan {
    int xbuf_bytes;   // one X buffer: NP panels of 256 rows x 128 bytes
    int x_off[2], wt_off, zpart_off, r_off, idx_off, lab_off, bar_off, total;
};
__host__ __device__ inline SmxPlan smx_plan(int NP) {
    SmxPlan s;
    s.xbuf_bytes = NP * kSmxRows * 128;
    s.x_off[0] = 0;
    s.x_off[1] = s.xbuf_bytes;
    s.wt_off = 2 * s.xbuf_bytes;                       // [NP][16 classes][128 B], swizzled like X
    s.zpart_off = s.wt_off + NP * kSmxClasses * 128;   // [S][256/S rows][16] fp32 = 16 KB
    s.r_off = s.zpart_off + kSmxRows * kSmxClasses * 4;  // residuals, 8 KB (layout depends on the path)
    s.idx_off = s.r_off + kSmxRows * kSmxClasses * 2;  // [2][256] row indices
    s.lab_off = s.idx_off + 2 * kSmxRows * 4;          // [2][256] labels of the rows this CTA owns
    s.bar_off = s.lab_off + 2 * kSmxRows * 4;          // mbarrier + tensor-memory base address
    s.total = s.bar_off + 64;
    return s;
}

// byte offset of predictor-chunk `chunk` (8 bf16) of row `row` inside a buffer of panels [panel][rows][128 B]
__device__ __forceinline__ int smx_chunk_off(int row, int chunk, int rows_per_panel) {
    return ((chunk >> 3) * rows_per_panel + row) * 128 + (((chunk & 7) ^ (row & 7)) << 4);
}

__device__ __forceinline__ void st_cluster_v4(uint32_t addr, float a, float b, float c, float d) {
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ void st_cluster_u16(uint32_t addr, unsigned short v) {
    asm volatile("st.shared::cluster.u16 [%0], %1;" ::"r"(addr), "h"(v) : "memory");
}

// named CTA barriers: `count` threads take part, by arriving (no wait) or by arriving and waiting
__device__ __forceinline__ void named_arrive(int id, int count) {
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ void named_sync(int id, int count) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

// ---------------------------------------------------------------- mbarrier and proxy helpers
// (mbar_init, mbar_try_wait, fence_barrier_init and fence_async_proxy come from glm_kernel.cuh)

// Bounded wait: when the budget runs out the thread records BMGD_ERR_TIMEOUT, raises the abort flag and
// stops waiting for the rest of the launch.
struct WaitCtx {
    int* status;
    unsigned long long timeout_ns;
    bool aborted;
};
__device__ __noinline__ void wait_slow_path(WaitCtx& w, unsigned long long& t0) {
    const unsigned long long now = global_ns();
    if (t0 == 0) t0 = now;
    if (now - t0 > w.timeout_ns) {
        atomicCAS(w.status, 0, kStatusTimeout);
        atomicExch(w.status + 1, 1);
        w.aborted = true;
    } else if (((volatile int*)w.status)[1] != 0) {
        w.aborted = true;
    }
}
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, WaitCtx& w) {
    if (w.aborted) return;
    unsigned long long t0 = 0;
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0x3Fu) == 0u) {
            wait_slow_path(w, t0);
            if (w.aborted) return;
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

template <bool USE_TC>
__global__ void __launch_bounds__(kSmxThreads, 1) softmax_kernel(const SoftmaxParams P) {
    extern __shared__ __align__(1024) unsigned char smx_smem[];
    unsigned char* const smem = smx_smem;
    const int tid = threadIdx.x, warp = tid >> 5;
    const int S = P.S, NP = P.NP, C = P.C, p = P.p;
    const int rank = (S > 1) ? (int)cluster_ctarank() : 0;
    const int ps = NP * 64;                 // predictors of this CTA
    const int f_first = rank * ps;
    const int RO = kSmxRows / S;            // row slots whose logits this CTA sums
    const uint32_t N0 = P.N0, n = P.n, M = P.M;
    const SmxPlan plan = smx_plan(NP);
    unsigned char* xbuf[2] = {smem + plan.x_off[0], smem + plan.x_off[1]};
    unsigned char* wt = smem + plan.wt_off;
    float* zpart = reinterpret_cast<float*>(smem + plan.zpart_off);
    unsigned char* rbuf = smem + plan.r_off;
    int* lab = reinterpret_cast<int*>(smem + plan.lab_off);
    const uint32_t mma_bar = smem_u32(smem + plan.bar_off);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + plan.bar_off + 16);

    const __nv_bfloat16* Xg = static_cast<const __nv_bfloat16*>(P.X);
    const FeistelDomain dom = make_domain(N0);
    WaitCtx wc{P.status, P.timeout_ns, false};
    const uint32_t total_steps = (uint32_t)P.T * M;

    // W master: thread f (< 128) owns predictor f of the slice, thread f+64 owns predictor f >= 128:
    // the threads that read that predictor's row of the backward accumulator from tensor memory
    const int my_f = (tid < 128) ? tid : ((tid >= 192 && tid < 256) ? tid - 64 : -1);
    const bool owns_w = my_f >= 0 && my_f < ps;
    float w[kSmxClasses];
#pragma unroll
    for (int c = 0; c < kSmxClasses; ++c) w[c] = 0.f;
    if (owns_w)
        for (int c = 0; c < C; ++c) w[c] = P.W[(size_t)(f_first + my_f) * C + c];

    // ---- set-up
    for (int i = tid * 16; i < plan.total; i += kSmxThreads * 16) st_shared_zero16(smem_u32(smem + i));
    __syncthreads();
    if (tid == 0) {
        mbar_init(mma_bar, 1u);
        fence_barrier_init();
    }
    uint32_t tmem_base = 0;
    if constexpr (USE_TC) {
        if (warp == 0) tc_alloc(smem_u32(tmem_slot), 64u);
        tc_fence_before();
    }
    auto write_wt = [&]() {  // bf16 copy of W_slice^T in the panel layout [panel][class][128 B]
        if (owns_w) {
#pragma unroll
            for (int c = 0; c < kSmxClasses; ++c)
                *reinterpret_cast<__nv_bfloat16*>(wt + smx_chunk_off(c, my_f >> 3, kSmxClasses) + (my_f & 7) * 2) =
                    __float2bfloat16_rn(w[c]);
        }
    };
    write_wt();
    __syncthreads();
    if constexpr (USE_TC) {
        tc_fence_after();
        tmem_base = *tmem_slot;
    }
    if (S > 1) {
        cluster_arrive_release();
        cluster_wait_acquire();
    }

    // ---- gather of one step's rows into buffer b (issued one step ahead)
    RoundKeys rk = round_keys(P.seed, 0u, 0u);
    int rk_round = 0;
    auto step_rows = [&](uint32_t step, uint32_t& lo, uint32_t& nm) {
        const uint32_t m = step % M;
        lo = m * n;
        nm = min(n, N0 - lo);
    };
    auto keys_for = [&](uint32_t step) {
        const int t = P.fixed_partition ? 0 : (int)(step / M);
        if (t != rk_round) { rk = round_keys(P.seed, 0u, (uint32_t)t); rk_round = t; }
    };
    auto gather = [&](uint32_t step, int b) {
        // copies the step's 256 row slots (this CTA's NP*8 chunks of 16 bytes each) into the swizzled panels of
        // buffer b and the owned labels into lab[b].  No barrier inside; ends with a commit by every thread.
        uint32_t lo, nm;
        step_rows(step, lo, nm);
        keys_for(step);
        if (warp >= kSmxRows / 32) {
            // Producer warps take 256/16 = 16 row slots each: one warp can keep only a few copy instructions in
            // flight, so many warps share the gather.  Lanes 0..15 evaluate the shuffle for one slot each; then the
            // warp copies the 16 rows one after the other, lanes taking consecutive 16-byte chunks.
            constexpr int kProducers = kSmxThreads / 32 - kSmxRows / 32;
            constexpr int kSlots = kSmxRows / kProducers;
            const int lane = tid & 31;
            const bool active = lane < NP * 8;
            const uint32_t dst_lane = smem_u32(xbuf[b]) + (uint32_t)((lane >> 3) * kSmxRows * 128);
            const __nv_bfloat16* src_lane = Xg + f_first + lane * 8;
            {
                const int slot0 = (warp - kSmxRows / 32) * kSlots;
                const int slot = slot0 + lane;
                uint32_t r = 0xFFFFFFFFu;
                int label = -1;
                if (lane < kSlots && (uint32_t)slot < nm) {
                    r = perm_index(lo + (uint32_t)slot, dom, rk);
                    if (slot / RO == rank) label = P.y[r];
                }
#pragma unroll 4
                for (int i = 0; i < kSlots; ++i) {
                    const uint32_t ri = __shfl_sync(0xFFFFFFFFu, r, i);
                    const int row = slot0 + i;
                    const uint32_t dst = dst_lane + (uint32_t)(row * 128 + (((lane & 7) ^ (row & 7)) << 4));
                    if (active) {
                        if (ri != 0xFFFFFFFFu) cp_async<16>(dst, src_lane + (size_t)ri * p);
                        else st_shared_zero16(dst);  // an empty slot must contribute nothing
                    }
                }
                // labels of the slots this CTA owns, for the step that will read buffer b
                if (lane < kSlots && slot / RO == rank) lab[b * kSmxRows + slot % RO] = label;
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    if (total_steps > 0) {
        gather(0, 0);
    }
    uint32_t mma_phase = 0;

    for (uint32_t step = 0; step < total_steps; ++step) {
        const int b = (int)(step & 1u);
        uint32_t lo, nm;
        step_rows(step, lo, nm);
#ifdef BMGD_TRACE
        const uint32_t step_count = step;
#endif
        BMGD_STAMP(0);
        asm volatile("cp.async.wait_group 0;" ::: "memory");  // this step's rows (issued during the previous step)
        if constexpr (USE_TC) fence_async_proxy();  // cp.async and st.shared wrote what the tensor core will read
        __syncthreads();
        BMGD_STAMP(1);

        if (warp >= kSmxRows / 32) {
            // ---- producer warps: arrive at the first barrier at once, fetch the next step's rows into the other
            //      buffer (its last reader, the previous step's backward contraction, has finished), then join
            //      the second barrier
            if (S > 1) cluster_arrive_release(); else named_arrive(1, kSmxThreads);
            if (step + 1 < total_steps) gather(step + 1, b ^ 1);
            __syncwarp();
            if (S > 1) { cluster_wait_acquire(); cluster_arrive_release(); cluster_wait_acquire(); }
            else named_sync(2, kSmxThreads);
            continue;
        }

        // ---- forward: partial logits of row slot `tid` (threads 0..255) over this CTA's predictors
        float z[kSmxClasses];
#pragma unroll
        for (int c = 0; c < kSmxClasses; ++c) z[c] = 0.f;
        if constexpr (USE_TC) {
            if (tid == 0) {
                tc_fence_after();
                const uint32_t idesc = tc_idesc(128, kSmxClasses, false);
                const uint32_t xa = smem_u32(xbuf[b]), wb = smem_u32(wt);
                for (int half = 0; half < 2; ++half)
                    for (int ks = 0; ks < NP * 4; ++ks) {  // K = 16 predictors per instruction
                        const uint32_t a_addr = xa + (uint32_t)((ks >> 2) * kSmxRows * 128 + half * 128 * 128 + (ks & 3) * 32);
                        const uint32_t b_addr = wb + (uint32_t)((ks >> 2) * kSmxClasses * 128 + (ks & 3) * 32);
                        tc_mma_bf16(tmem_base + (uint32_t)(half * 16), tc_smem_desc(a_addr, 16, 1024),
                                    tc_smem_desc(b_addr, 16, 1024), idesc, ks > 0 ? 1u : 0u);
                    }
                tc_commit(mma_bar);
            }
            mbar_wait(mma_bar, mma_phase, wc);
            mma_phase ^= 1u;
            tc_fence_after();
            if (tid < kSmxRows)  // warp w reads lanes 32*(w%4).. of accumulator w/4: lane = row slot within the half
                tc_load16(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * 16), z);
            tc_fence_before();
        } else {
            if (tid < kSmxRows) {
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
        }

        BMGD_STAMP(2);
        // ---- reduce-scatter of the partial logits: row slot -> the CTA that owns it
        if (tid < kSmxRows) {
            const int owner = tid / RO, rloc = tid % RO;
            const uint32_t dst_local = smem_u32(zpart + ((size_t)rank * RO + rloc) * kSmxClasses);
            const uint32_t dst = (S > 1) ? map_to_cta(dst_local, (uint32_t)owner) : dst_local;
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) st_cluster_v4(dst + c4 * 16, z[c4 * 4], z[c4 * 4 + 1], z[c4 * 4 + 2], z[c4 * 4 + 3]);
        }
        if (S > 1) { __syncwarp(); cluster_arrive_release(); cluster_wait_acquire(); } else named_sync(1, kSmxThreads);

        BMGD_STAMP(3);
        // ---- softmax and residual for the rows this CTA owns; push R to every peer
        for (int r0 = 0; r0 < RO; r0 += 16) {
            if (tid < 256) {
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
                if (live && (uint32_t)slot < nm) res = __fdividef(e, den) - (c == lab[b * kSmxRows + rloc] ? 1.f : 0.f);
                // tensor-core path: R^T as B operand, [row panel of 64][class][128 B] swizzled; otherwise [row][class]
                const int off = USE_TC ? (smx_chunk_off(c, slot >> 3, kSmxClasses) + (slot & 7) * 2) : (slot * kSmxClasses + c) * 2;
                *reinterpret_cast<__nv_bfloat16*>(rbuf + off) = __float2bfloat16_rn(res);
            }
        }
        if (S > 1) {
            // the owned part of R is 2*RO chunks of 16 bytes: copy each to every peer
            named_sync(3, kSmxRows);
            if (tid < 2 * RO) {
                const int per_class = RO / 8;
                const int off = USE_TC ? smx_chunk_off(tid / per_class, rank * per_class + tid % per_class, kSmxClasses)
                                       : (rank * RO * kSmxClasses * 2 + tid * 16);
                const float4 v = *reinterpret_cast<const float4*>(rbuf + off);
                const uint32_t dst_local = smem_u32(rbuf + off);
                for (int peer = 0; peer < S; ++peer)
                    if (peer != rank) st_cluster_v4(map_to_cta(dst_local, (uint32_t)peer), v.x, v.y, v.z, v.w);
            }
        }
        BMGD_STAMP(4);
        if constexpr (USE_TC) fence_async_proxy();
        if (S > 1) { __syncwarp(); cluster_arrive_release(); cluster_wait_acquire(); } else named_sync(2, kSmxThreads);
        if constexpr (USE_TC) fence_async_proxy();  // the peers' residuals arrived through the generic proxy

        BMGD_STAMP(5);
        // ---- backward: gradient rows of this CTA's predictors
        float gr[kSmxClasses];
#pragma unroll
        for (int c = 0; c < kSmxClasses; ++c) gr[c] = 0.f;
        if constexpr (USE_TC) {
            const int ntiles = NP - 1;  // tile 0: predictors 0..127; tile 1 (three panels): predictors 64..191
            if (tid == 0) {
                tc_fence_after();
                const uint32_t idesc = tc_idesc(128, kSmxClasses, true);
                const uint32_t xa = smem_u32(xbuf[b]), rb = smem_u32(rbuf);
                for (int tile = 0; tile < ntiles; ++tile)
                    for (int ks = 0; ks < kSmxRows / 16; ++ks) {  // K = 16 row slots per instruction
                        const uint32_t a_addr = xa + (uint32_t)(tile * kSmxRows * 128 + ks * 16 * 128);
                        const uint32_t b_addr = rb + (uint32_t)((ks >> 2) * kSmxClasses * 128 + (ks & 3) * 32);
                        tc_mma_bf16(tmem_base + 32u + (uint32_t)(tile * 16), tc_smem_desc(a_addr, kSmxRows * 128, 1024),
                                    tc_smem_desc(b_addr, 16, 1024), idesc, ks > 0 ? 1u : 0u);
                    }
                tc_commit(mma_bar);
            }
            mbar_wait(mma_bar, mma_phase, wc);
            mma_phase ^= 1u;
            tc_fence_after();
            if (tid < 128) tc_load16(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + 32u, gr);
            else if (tid >= 192 && tid < 256 && ntiles > 1) tc_load16(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + 48u, gr);
            tc_fence_before();
        } else {
            if (owns_w) {
                for (int row = 0; row < kSmxRows; ++row) {
                    const float xf = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(
                        xbuf[b] + smx_chunk_off(row, my_f >> 3, kSmxRows) + (my_f & 7) * 2));
                    const __nv_bfloat16* rr = reinterpret_cast<const __nv_bfloat16*>(rbuf + row * kSmxClasses * 2);
#pragma unroll
                    for (int c = 0; c < kSmxClasses; ++c) gr[c] = fmaf(xf, __bfloat162float(rr[c]), gr[c]);
                }
            }
        }

        BMGD_STAMP(6);
        // ---- update of W_slice and of its bf16 copy
        const float scale = (float)((nm == n) ? P.scale_full : P.scale_last);
        if (owns_w) {
#pragma unroll
            for (int c = 0; c < kSmxClasses; ++c) w[c] = fmaf(-scale, gr[c], w[c]);
        }
        write_wt();
        BMGD_STAMP(7);
        // the next iteration's barrier orders these writes, and the end of the reads of xbuf[b], before their next use
    }

    if (owns_w)
        for (int c = 0; c < C; ++c) P.W[(size_t)(f_first + my_f) * C + c] = w[c];
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    if constexpr (USE_TC) {
        tc_fence_after();
        if (warp == 0) tc_dealloc(tmem_base, 64u);
    }
    if (S > 1) { __syncwarp(); cluster_arrive_release(); cluster_wait_acquire(); }
}

// ---------------------------------------------------------------- host side

// Runs `rounds` rounds over the buffer on `stream`.  Shapes this kernel covers: C <= 16, batch_size <= 256,
// p = S * NP * 64 with S in {1,2,4,8,16} and NP in {2,3}.  Returns a bmgd_status value.
inline int softmax_run(const void* dx, const void* dy, int64_t rows, int p, int C, void* W, void* /*scratch*/, int* status,
                       int rounds, int n, double lr, unsigned long long seed, int fixed, unsigned long long timeout_ns,
                       int cluster_size, int /*threads*/, int use_cuda_cores, int /*sm_count*/, int smem_optin,
                       cudaStream_t stream, SoftmaxLaunchInfo* info) {
    *info = SoftmaxLaunchInfo{};
    if (C > kSmxClasses || n > kSmxRows) return -8;
    int S = 0, NP = 0;
    for (int s = 16; s >= 1 && !S; s >>= 1) {
        if (cluster_size && s != cluster_size) continue;
        for (int np = kSmxMaxPanels; np >= 2; --np)
            if (p == s * np * 64) { S = s; NP = np; break; }
    }
    if (!S) return -8;
    if (((uintptr_t)dx % 16) != 0 || ((uintptr_t)dy % 4) != 0) return -1;
    const SmxPlan plan = smx_plan(NP);
    if (plan.total > smem_optin) return -8;
    const uint32_t M = (uint32_t)((rows + n - 1) / n);
    if ((uint64_t)rounds * M >= 0xFFFFFFF0ull) return -1;

    SoftmaxParams P{};
    P.X = dx; P.y = static_cast<const int*>(dy); P.W = static_cast<float*>(W); P.status = status;
    P.seed = seed; P.timeout_ns = timeout_ns;
    P.scale_full = lr / (double)n;
    P.scale_last = lr / (double)(rows - (int64_t)(M - 1) * n);
    P.N0 = (uint32_t)rows; P.n = (uint32_t)n; P.M = M; P.T = rounds; P.p = p; P.C = C; P.S = S; P.NP = NP;
    P.fixed_partition = fixed;
    P.use_tc = use_cuda_cores ? 0 : 1;

    void (*fn)(const SoftmaxParams) = use_cuda_cores ? softmax_kernel<false> : softmax_kernel<true>;
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
    if (S > 1) {
        int nclusters = 0;
        e = cudaOccupancyMaxActiveClusters(&nclusters, (const void*)fn, &lc);
        if (e != cudaSuccess) { info->cuda_error = (int)e; cudaGetLastError(); return -3; }
        if (nclusters < 1) return -7;
    }
    e = cudaLaunchKernelEx(&lc, fn, P);
    if (e != cudaSuccess) { info->cuda_error = (int)e; cudaGetLastError(); return e == cudaErrorLaunchOutOfResources ? -7 : -3; }
    info->launches = 1; info->grid_ctas = S; info->cluster_size = S; info->threads = kSmxThreads;
    info->depth = 2; info->smem = plan.total;
    return 0;
}

}  // namespace bmgdk
