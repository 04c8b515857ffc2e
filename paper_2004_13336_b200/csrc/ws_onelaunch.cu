// LAMB (and, by the same scheme, LARS) for all shards as ONE kernel.
//
// Both optimizers need a per-tensor norm ratio before any element of the tensor can take its
// step (paper Section 4.1, "Non-elementwise operators": the shards' partial reduce results are
// combined, Section 5.2: as one batched scalar exchange).  Run as separate launches, phase 2
// reads the weight and the new moments again from DRAM.  Here the two phases of every tensor are
// work items of one kernel, ordered (by the plan's one-launch schedule) so that a tensor's phase-2
// items run shortly after its phase-1 items, while other tensors' phase-1 items stream from DRAM:
// phase 2 then finds its operands in L2 and every operand crosses HBM once.
//
// One CTA per schedule entry.  A CTA draws a ticket from a global counter when it starts running and
// takes the schedule entry of that number, so entries are started in schedule order whatever order the
// hardware launches CTAs in.  The CTA that completes a tensor's last phase-1 item sums the tensor's
// partial norms in a fixed order in double (run-to-run bit-stable) and publishes the ratio.
//
// Progress: a phase-2 entry waits only for phase-1 entries that come earlier in the schedule.  Tickets
// are drawn by running CTAs, so every earlier entry belongs to a CTA that is running or has finished,
// and the earliest unfinished entry never waits for anything unfinished; no co-residency of the grid is
// assumed.  Every wait has an iteration limit; when it runs out the CTA sets the status word in the
// workspace and returns (the update is then incomplete and the caller can tell).
#include "ws_kernels.cuh"

namespace wsk {
namespace {

constexpr int kSpinLimit = 1 << 22;          // polls of a ready flag (about 100 ns apart) before giving up
constexpr int kU2 = 2;                       // phase 2: vector accesses per stream in flight per thread (1: 0.8 % slower)

// A tensor's ready word: 0 until its ratio is known, then (ratio bits << 32) | 1 - flag and ratio in
// one 64-bit word, so that a reader can never pair a set flag with a ratio from before it.
__device__ __forceinline__ unsigned long long ld_acquire(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release(unsigned long long* p, unsigned long long v) {
    asm volatile("st.release.gpu.global.u64 [%0], %1;" :: "l"(p), "l"(v) : "memory");
}
// Loads of the schedule tables (never written while the kernel runs).
__device__ __forceinline__ unsigned ld_u32(const unsigned* p) {
    unsigned v;
    asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ uint4 ld_u128(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ int ld_volatile_s32(const int* p) {
    int v;
    asm volatile("ld.volatile.global.s32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ const void* ld_ptr(const void* const* p) {
    unsigned long long v;
    asm volatile("ld.global.nc.u64 %0, [%1];" : "=l"(v) : "l"(p));
    return reinterpret_cast<const void*>(v);
}

// PAIR 0: LAMB, 1: LARS.  VEC1, U1, RB, NP: phase 1's vector width, accesses per pass, tree block and
// pointer capacity; VEC2: phase 2's vector width.  Other parameters as for process_item.
// One CTA per schedule entry; the CTA's entry is the ticket it draws when it starts running.
template <int PAIR, bool GBF, int OUT, int VEC1, int U1, int RB, int NP, int VEC2, bool FUSED>
__global__ void __launch_bounds__(kBlock, RB > 8 ? kMinBlocksWide : kMinBlocks)
two_phase_kernel(const UpdParams P, const __grid_constant__ GradPtrs<NP> gp, const OneLaunch Q) {
    constexpr int OPT1 = PAIR == 0 ? K_LAMB1 : K_LARS1;
    constexpr int OPT2 = PAIR == 0 ? K_LAMB2 : K_LARS2;
    constexpr int OUT1 = (FUSED && OUT == O_F32M) ? O_F32M : O_NONE;
    __shared__ unsigned long long s_word;      // the ticket, later the tensor's ready word
    __shared__ const void* sgp[FUSED ? NP : 1];
    __shared__ float2 red[kBlock / 32];
    __shared__ double fin_a[kBlock / 32], fin_b[kBlock / 32];   // (small on purpose: shared memory comes out of the L1)
    __shared__ int s_last;
    const int tid = threadIdx.x;

    if (tid == 0) s_word = atomicAdd(Q.ticket, 1ULL);
    __syncthreads();
    const unsigned long long tk = s_word;
    if (tk == 0) {
        // tensors without any element take part in no item: ratio 1, norms 0
        for (int t = tid; t < Q.T; t += kBlock)
            if (Q.segs[t].count == 0) {
                Q.rho[t] = 1.0f;
                Q.norms[2 * t] = 0.0;
                Q.norms[2 * t + 1] = 0.0;
            }
    }
    if (tk >= Q.nsched) return;
    const unsigned e = ld_u32(Q.sched + tk);
    const unsigned pidx = e >> 1;
    const int kind = (int)(e & 1u);
    const char* src = reinterpret_cast<const char*>(Q.items + pidx);
    const uint4 da = ld_u128(src), db = ld_u128(src + 16);
    ItemCtx it;
    const long long pos = (long long)(((unsigned long long)da.y << 32) | da.x);
    const int shard = (int)(db.z >> 16);
    const long long base = (long long)shard * P.S + pos;
    it.len = (int)(db.z & 0xffffu);
    it.nvalid = (int)db.y;
    it.seg = (int)db.x;
    it.gbase = base;
    it.sbase = base;
    it.obase = base;
    it.toff = (long long)(((unsigned long long)da.w << 32) | da.z);
    it.partial = Q.ipart + pidx;
    it.keep = kind == 0 && (db.w & 1u) != 0;
    char* wt = nullptr;
    if constexpr (FUSED) {
        if (kind == 1 || OUT == O_F32M)
            wt = reinterpret_cast<char*>(const_cast<void*>(ld_ptr(reinterpret_cast<const void* const*>(P.wtab) + (long long)it.seg * P.nw)));
    }

    if (kind == 0) {
        if constexpr (FUSED) {
            for (int k = tid; k < P.R; k += kBlock) sgp[k] = ld_ptr(P.gtab + (long long)it.seg * P.R + k);
            __syncthreads();
        }
        process_item<OPT1, GBF, OUT1, VEC1, U1, RB, NP, FUSED, true>(P, gp, it, sgp, nullptr, wt, 0.f, red);
        // thread 0 has stored the item's partial sums; count the item, and the CTA that counts a tensor's
        // last one forms the ratio
        if (tid == 0) {
            __threadfence();
            const WsItemSeg sg = Q.segs[it.seg];
            s_last = (atomicAdd(Q.count + it.seg, 1) + 1 == sg.count) ? 1 : 0;
        }
        __syncthreads();
        if (!s_last) return;
        __threadfence();
        const WsItemSeg sg = Q.segs[it.seg];
        double a = 0.0, b = 0.0;
        for (int i = tid; i < sg.count; i += kBlock) {        // fixed order: bit-stable
            const float2 p = __ldcg(Q.ipart + sg.first + i);
            a += (double)p.x;
            b += (double)p.y;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {                    // fixed tree inside the warp ...
            a += __shfl_xor_sync(0xffffffffu, a, o);
            b += __shfl_xor_sync(0xffffffffu, b, o);
        }
        if ((tid & 31) == 0) {
            fin_a[tid >> 5] = a;
            fin_b[tid >> 5] = b;
        }
        __syncthreads();
        if (tid == 0) {
            a = 0.0;
            b = 0.0;
            for (int i = 0; i < kBlock / 32; ++i) {           // ... and the warps in order
                a += fin_a[i];
                b += fin_b[i];
            }
            Q.norms[2 * it.seg] = a;
            Q.norms[2 * it.seg + 1] = b;
            float ratio = 1.0f;
            if (a > 0.0 && b > 0.0)
                ratio = PAIR == 1 ? (float)(Q.eta * sqrt(a) / (sqrt(b) + Q.beta * sqrt(a))) : (float)(sqrt(a) / sqrt(b));
            Q.rho[it.seg] = ratio;
            __threadfence();
            st_release(Q.flag + it.seg, ((unsigned long long)__float_as_uint(ratio) << 32) | 1ULL);
        }
        return;
    }

    // phase 2: the tensor's ratio.  The schedule puts this entry well behind the tensor's last phase-1
    // entry, so the word is normally there at the first look.
    __syncthreads();                                   // (every thread has read the ticket out of s_word)
    if (tid == 0) {
        unsigned long long word = 0;
        for (int tries = 0; tries < kSpinLimit; ++tries) {
            word = ld_acquire(Q.flag + it.seg);
            if (word & 1ULL) break;
            if ((tries & 255) == 255 && ld_volatile_s32(Q.status) != 0) break;
            __nanosleep(100);
        }
        if (!(word & 1ULL)) atomicExch(Q.status, 1);    // gave up: the update stays incomplete, the caller can tell
        s_word = word;
    }
    __syncthreads();
    const unsigned long long word = s_word;
    if (!(word & 1ULL)) return;
    const float rho = __uint_as_float((unsigned)(word >> 32));
    const GradPtrs<1> none = {};
    process_item<OPT2, false, OUT, VEC2, kU2, 1, 1, FUSED, true>(P, none, it, nullptr, nullptr, wt, P.c.lr * rho, red);
}

template <int PAIR, bool GBF, int OUT, int VEC1, int U1, int RB, int NP, int VEC2, bool FUSED>
ws_status launch(const UpdParams& P, const void* const* gptrs, const OneLaunch& Q, cudaStream_t st) {
    GradPtrs<NP> gp;
    for (int k = 0; k < NP; ++k) gp.p[k] = (!FUSED && gptrs && k < P.R) ? gptrs[k] : nullptr;
    auto kern = two_phase_kernel<PAIR, GBF, OUT, VEC1, U1, RB, NP, VEC2, FUSED>;
    const long long grid = Q.nsched;            // one CTA per schedule entry
    if (grid < 1) return WS_OK;
    kern<<<(unsigned)grid, kBlock, 0, st>>>(P, gp, Q);
    return ws_check_launch("one-launch update");
}

// Phase 1's flavour follows the separate-launch kernels: 256-bit accesses when the gradients are
// bf16, tree blocks of 8, a loop with compensation beyond one block.
template <int PAIR, bool GBF, int OUT, bool FUSED>
ws_status launch_r(const UpdParams& P, const void* const* gptrs, const OneLaunch& Q, bool wide, cudaStream_t st) {
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

// Where the one-kernel route measured faster than the three launches on a B200: LAMB with 8 to 32
// gradient copies (BERT-large set, R = 16: 4.87 ms against 5.13 ms, R = 8: 3.27 against 3.46 ms;
// Transformer set under LAMB: 5 % faster at R = 8, 3.6 % at R = 32).  With few copies phase 1 is as
// short as phase 2 and the three launches win (Transformer set, R = 4: 1.64 ms against 1.67 ms, R = 2:
// 1.38 against 1.49 ms), and so they do for LARS on the ResNet-50 set, whose 161 mostly tiny tensors
// make a step of 0.24 ms.
bool one_launch_supports(int pair, int R) { return pair == 0 && R >= 8 && R <= 32; }

ws_status launch_one_launch(int pair, bool gbf, int out, bool fused, bool wide, const UpdParams& P,
                            const void* const* gptrs, const OneLaunch& Q, cudaStream_t st) {
    if (pair != 0) return WS_ERR_INVALID_ARG;
    return gbf ? launch_o<0, true>(P, gptrs, Q, out, fused, wide, st) : launch_o<0, false>(P, gptrs, Q, out, fused, wide, st);
}

}  // namespace wsk
