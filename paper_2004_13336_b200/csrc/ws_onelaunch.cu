// LAMB and LARS for all shards as ONE persistent kernel.
//
// Both optimizers need a per-tensor norm ratio before any element of the tensor can take its
// step (paper Section 4.1, "Non-elementwise operators": the shards' partial reduce results are
// combined, Section 5.2: as one batched scalar exchange).  Run as separate launches, phase 2
// reads the weight and the new moments again from DRAM.  Here the two phases of every tensor are
// work items of one kernel, ordered (by the plan's one-launch schedule) so that a tensor's phase-2
// items run shortly after its phase-1 items, while other tensors' phase-1 items stream from DRAM:
// phase 2 then finds its operands in L2 and every operand crosses HBM once.
//
// A CTA is kBlock worker threads plus one scheduling warp.  The scheduling warp takes tickets
// from a global counter (items are handed out in schedule order), fetches the item descriptor and,
// for a phase-2 item, waits until the tensor's ratio is published; it hands items to the workers
// through a two-slot ring in shared memory, so the workers never wait for a descriptor, a ticket
// or a ratio.  The worker CTA that completes a tensor's last phase-1 item sums the tensor's partial
// norms in a fixed order in double (run-to-run bit-stable) and publishes the ratio.
//
// Progress: a phase-2 item waits only for phase-1 items that come earlier in the schedule.  Tickets
// are taken in order by CTAs that are running, so the earliest unfinished item is always held by a
// running CTA that waits for nothing unfinished; no co-residency of the grid is assumed.  Every
// wait has an iteration limit; when it runs out the kernel sets the status word in the workspace
// and all CTAs stop taking work.
#include "ws_kernels.cuh"

namespace wsk {
namespace {

constexpr int kThreads = kBlock + 32;        // workers + the scheduling warp
constexpr int kSpinLimit = 1 << 22;          // polls of a ready flag (about 100 ns apart) before giving up
enum { BAR_FULL0 = 2, BAR_EMPTY0 = 4 };      // named barriers (1 is the workers' own barrier)

struct Slot {
    ItemCtx it;
    char* wt;        // fused formatting: the item's weight tensor
    float lr_rho;    // phase 2: lr * ratio of the item's tensor
    int kind;        // 0: phase 1, 1: phase 2, -1: no more work
};

__device__ __forceinline__ void bar_sync(int id) { asm volatile("bar.sync %0, %1;" :: "r"(id), "n"(kThreads) : "memory"); }
__device__ __forceinline__ void bar_arrive(int id) { asm volatile("bar.arrive %0, %1;" :: "r"(id), "n"(kThreads) : "memory"); }
__device__ __forceinline__ int ld_acquire(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release(int* p, int v) {
    asm volatile("st.release.gpu.global.s32 [%0], %1;" :: "l"(p), "r"(v) : "memory");
}

// PAIR 0: LAMB, 1: LARS.  VEC1, U1, RB, NP: phase 1's vector width, accesses per pass, tree block and
// pointer capacity; VEC2: phase 2's vector width.  Other parameters as for process_item.
template <int PAIR, bool GBF, int OUT, int VEC1, int U1, int RB, int NP, int VEC2, bool FUSED>
__global__ void __launch_bounds__(kThreads, RB > 8 ? kMinBlocksWide : kMinBlocks)
two_phase_kernel(const UpdParams P, const __grid_constant__ GradPtrs<NP> gp, const OneLaunch Q) {
    constexpr int OPT1 = PAIR == 0 ? K_LAMB1 : K_LARS1;
    constexpr int OPT2 = PAIR == 0 ? K_LAMB2 : K_LARS2;
    constexpr int OUT1 = (FUSED && OUT == O_F32M) ? O_F32M : O_NONE;
    __shared__ Slot slot[2];
    __shared__ const void* sgp[2][FUSED ? NP : 1];
    __shared__ float2 red[kBlock / 32];
    __shared__ double fin_a[kBlock], fin_b[kBlock];
    __shared__ int s_last;
    const int tid = threadIdx.x;

    if (tid >= kBlock) {
        // ------------------------------------------------------------ scheduling warp
        const int lane = tid - kBlock;
        for (unsigned n = 0;; ++n) {
            const int s = n & 1;
            if (n >= 2) bar_sync(BAR_EMPTY0 + s);        // the workers are done with this slot
            unsigned long long tk = 0;
            if (lane == 0) tk = atomicAdd(Q.ticket, 1ULL);
            tk = __shfl_sync(0xffffffffu, tk, 0);
            int kind = -1;
            WsItem wi = {};
            unsigned pidx = 0;
            float lr_rho = 0.f;
            if (tk < Q.nsched && *reinterpret_cast<volatile int*>(Q.status) == 0) {
                const unsigned e = __ldg(Q.sched + tk);
                kind = (int)(e & 1u);
                pidx = e >> 1;
                const uint4* src = reinterpret_cast<const uint4*>(Q.items + pidx);
                uint4 a = __ldg(src), b = __ldg(src + 1);
                wi.pos = (long long)(((unsigned long long)a.y << 32) | a.x);
                wi.toff = (long long)(((unsigned long long)a.w << 32) | a.z);
                wi.seg = (int)b.x;
                wi.nvalid = (int)b.y;
                wi.len = (unsigned short)(b.z & 0xffffu);
                wi.shard = (unsigned short)(b.z >> 16);
                wi.flags = b.w;
                if (kind == 1) {
                    // the tensor's ratio: published by the CTA that finished the tensor's last phase-1 item
                    int ready = 0;
                    if (lane == 0) {
                        for (int tries = 0; tries < kSpinLimit; ++tries) {
                            if (ld_acquire(Q.flag + wi.seg) != 0) { ready = 1; break; }
                            if ((tries & 255) == 255 && *reinterpret_cast<volatile int*>(Q.status) != 0) break;
                            __nanosleep(100);
                        }
                        if (!ready) atomicExch(Q.status, 1);   // gave up: every CTA stops taking work
                    }
                    ready = __shfl_sync(0xffffffffu, ready, 0);
                    if (ready) lr_rho = P.c.lr * __ldcg(Q.rho + wi.seg);
                    else kind = -1;
                }
            }
            if (kind >= 0) {
                if constexpr (FUSED) {
                    if (kind == 0)
                        for (int k = lane; k < P.R; k += 32) sgp[s][k] = P.gtab[(long long)wi.seg * P.R + k];
                }
                if (lane == 0) {
                    Slot& sl = slot[s];
                    const long long base = (long long)wi.shard * P.S + wi.pos;
                    sl.it.len = wi.len;
                    sl.it.nvalid = wi.nvalid;
                    sl.it.seg = wi.seg;
                    sl.it.gbase = base;
                    sl.it.sbase = base;
                    sl.it.obase = base;
                    sl.it.toff = wi.toff;
                    sl.it.partial = Q.ipart + pidx;
                    sl.it.keep = kind == 0 && (wi.flags & 1u) != 0;
                    sl.wt = nullptr;
                    if constexpr (FUSED) {
                        if (kind == 1 || OUT == O_F32M) sl.wt = reinterpret_cast<char*>(P.wtab[(long long)wi.seg * P.nw]);
                    }
                    sl.lr_rho = lr_rho;
                    sl.kind = kind;
                }
            } else if (lane == 0) {
                slot[s].kind = -1;
            }
            __syncwarp();
            __threadfence_block();
            bar_arrive(BAR_FULL0 + s);
            if (kind < 0) return;
        }
    }

    // --------------------------------------------------------------------- workers
    if (blockIdx.x == 0) {
        // tensors without any element take part in no item: ratio 1, norms 0
        for (int t = tid; t < Q.T; t += kBlock)
            if (Q.segs[t].count == 0) {
                Q.rho[t] = 1.0f;
                Q.norms[2 * t] = 0.0;
                Q.norms[2 * t + 1] = 0.0;
            }
    }
    const GradPtrs<1> none = {};
    for (unsigned n = 0;; ++n) {
        const int s = n & 1;
        bar_sync(BAR_FULL0 + s);
        const int kind = slot[s].kind;
        if (kind < 0) return;
        const ItemCtx it = slot[s].it;
        char* wt = slot[s].wt;
        if (kind == 0) {
            process_item<OPT1, GBF, OUT1, VEC1, U1, RB, NP, FUSED, true, true>(P, gp, it, sgp[s], nullptr, wt, 0.f, red);
            // thread 0 has stored the item's partial sums; count the item, and the CTA that counts a
            // tensor's last one forms the ratio
            if (tid == 0) {
                __threadfence();
                const WsItemSeg sg = Q.segs[it.seg];
                s_last = (atomicAdd(Q.count + it.seg, 1) + 1 == sg.count) ? 1 : 0;
            }
            worker_sync<true>();
            if (s_last) {
                __threadfence();
                const WsItemSeg sg = Q.segs[it.seg];
                double a = 0.0, b = 0.0;
                for (int i = tid; i < sg.count; i += kBlock) {        // fixed order: bit-stable
                    const float2 p = __ldcg(Q.ipart + sg.first + i);
                    a += (double)p.x;
                    b += (double)p.y;
                }
                fin_a[tid] = a;
                fin_b[tid] = b;
                worker_sync<true>();
                for (int h = kBlock / 2; h > 0; h >>= 1) {
                    if (tid < h) {
                        fin_a[tid] += fin_a[tid + h];
                        fin_b[tid] += fin_b[tid + h];
                    }
                    worker_sync<true>();
                }
                if (tid == 0) {
                    a = fin_a[0];
                    b = fin_b[0];
                    Q.norms[2 * it.seg] = a;
                    Q.norms[2 * it.seg + 1] = b;
                    float ratio = 1.0f;
                    if (a > 0.0 && b > 0.0)
                        ratio = PAIR == 1 ? (float)(Q.eta * sqrt(a) / (sqrt(b) + Q.beta * sqrt(a))) : (float)(sqrt(a) / sqrt(b));
                    Q.rho[it.seg] = ratio;
                    __threadfence();
                    st_release(Q.flag + it.seg, 1);
                }
            }
        } else {
            process_item<OPT2, false, OUT, VEC2, 1, 1, 1, FUSED, true, true>(P, none, it, nullptr, nullptr, wt, slot[s].lr_rho, red);
        }
        bar_arrive(BAR_EMPTY0 + s);
    }
}

template <int PAIR, bool GBF, int OUT, int VEC1, int U1, int RB, int NP, int VEC2, bool FUSED>
ws_status launch(const UpdParams& P, const void* const* gptrs, const OneLaunch& Q, cudaStream_t st) {
    GradPtrs<NP> gp;
    for (int k = 0; k < NP; ++k) gp.p[k] = (!FUSED && gptrs && k < P.R) ? gptrs[k] : nullptr;
    auto kern = two_phase_kernel<PAIR, GBF, OUT, VEC1, U1, RB, NP, VEC2, FUSED>;
    int dev = 0, sms = 0, per_sm = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kThreads, 0);
    if (e != cudaSuccess) return ws_cuda_fail(e, "one-launch update (occupancy)");
    if (per_sm < 1) per_sm = 1;
    long long grid = (long long)sms * per_sm;
    if (grid > (long long)Q.nsched) grid = Q.nsched;
    if (grid < 1) return WS_OK;
    kern<<<(unsigned)grid, kThreads, 0, st>>>(P, gp, Q);
    return ws_check_launch("one-launch update");
}

// Phase 1's flavour follows the separate-launch kernels: 256-bit accesses when the fp32 streams
// dominate (R <= 2) or the gradients are bf16, tree blocks of 8, a loop with compensation beyond.
template <int PAIR, bool GBF, int OUT, bool FUSED>
ws_status launch_r(const UpdParams& P, const void* const* gptrs, const OneLaunch& Q, bool wide, cudaStream_t st) {
    if (P.R <= 2) {
        if (wide) return launch<PAIR, GBF, OUT, 8, 1, 2, 2, 8, FUSED>(P, gptrs, Q, st);
        return launch<PAIR, GBF, OUT, 4, 1, 2, 2, 4, FUSED>(P, gptrs, Q, st);
    }
    if (P.R <= 8) {
        if (wide) return launch<PAIR, GBF, OUT, GBF ? 8 : 4, 1, 8, 8, 8, FUSED>(P, gptrs, Q, st);
        return launch<PAIR, GBF, OUT, 4, 1, 8, 8, 4, FUSED>(P, gptrs, Q, st);
    }
    if (P.R <= 32) {
        if (wide) return launch<PAIR, GBF, OUT, GBF ? 8 : 4, 1, 8, 32, 8, FUSED>(P, gptrs, Q, st);
        return launch<PAIR, GBF, OUT, 4, 1, 8, 32, 4, FUSED>(P, gptrs, Q, st);
    }
    return WS_ERR_TOO_LARGE;      // (more copies: the caller runs the separate launches)
}

template <int PAIR, bool GBF>
ws_status launch_o(const UpdParams& P, const void* const* gptrs, const OneLaunch& Q, int out, bool fused, bool wide,
                   cudaStream_t st) {
    if (fused) {
        switch (out) {
            case O_F32: return launch_r<PAIR, GBF, O_F32, true>(P, gptrs, Q, wide, st);
            case O_BF16: return launch_r<PAIR, GBF, O_BF16, true>(P, gptrs, Q, wide, st);
            case O_F32M: return launch_r<PAIR, GBF, O_F32M, true>(P, gptrs, Q, wide, st);
            default: return WS_ERR_INVALID_ARG;
        }
    }
    switch (out) {
        case O_NONE: return launch_r<PAIR, GBF, O_NONE, false>(P, gptrs, Q, wide, st);
        case O_F32: return launch_r<PAIR, GBF, O_F32, false>(P, gptrs, Q, wide, st);
        case O_BF16: return launch_r<PAIR, GBF, O_BF16, false>(P, gptrs, Q, wide, st);
        default: return WS_ERR_INVALID_ARG;
    }
}

}  // namespace

bool one_launch_supports(int R) { return R >= 1 && R <= 32; }

ws_status launch_one_launch(int pair, bool gbf, int out, bool fused, bool wide, const UpdParams& P,
                            const void* const* gptrs, const OneLaunch& Q, cudaStream_t st) {
    if (pair == 0) return gbf ? launch_o<0, true>(P, gptrs, Q, out, fused, wide, st) : launch_o<0, false>(P, gptrs, Q, out, fused, wide, st);
    return gbf ? launch_o<1, true>(P, gptrs, Q, out, fused, wide, st) : launch_o<1, false>(P, gptrs, Q, out, fused, wide, st);
}

}  // namespace wsk
