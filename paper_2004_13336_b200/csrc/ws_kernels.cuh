// Device code shared by the update kernels: memory access helpers, the optimizer arithmetic and
// the body that processes one work item (a run of consecutive shard positions inside one tensor's
// piece).  Included by the translation units that define kernels; nothing here is part of the
// public ABI.
#pragma once
#include <cuda_bf16.h>
#include <math.h>

#include "ws_internal.h"

namespace wsk {

constexpr int kBlock = 256;
// Resident CTAs per SM the compiler must allow for (register budget): 3 measured best (4 forces
// spills, 2 leaves bandwidth unused); the bf16-gradient wide kernel on packed buffers and the
// many-replica kernel are faster with the registers of 2.
constexpr int kMinBlocks = 3;
constexpr int kMinBlocksWide = 2;
constexpr int kTreeBlockLarge = 16;   // gradients per tree block when R > 32
constexpr int kAf2Unroll = 2;         // Adafactor's pass 2: vectors in flight per thread
constexpr int kAf2Ctas = 4;           // ... and its resident CTAs per SM (a persistent grid)
// 128-bit accesses per thread per pass in Adafactor's pass 1 with up to 2 / up to 4 / more copies
constexpr int kUAf2 = 2, kUAf4 = 2, kUAf8 = 1;
// Kernel flavours.  The norm-based optimizers run as two phases around a finalize step:
// phase 1 (K_LAMB1, K_LARS1) reduces the gradients and leaves per-tile partial sums of the
// two norms; phase 2 (K_LAMB2, K_LARS2) applies the step with the per-tensor ratio.
// Adafactor runs as three passes around two finalize steps: K_AF1 reduces the gradients, keeps
// the sum and accumulates row / column sums of g^2 + eps1; K_AF2 sums U^2 per tensor (a kernel of its
// own, af_sumsq_kernel; the id only names the pass to the argument checks); K_AF3 applies.
enum { K_SGDM = 0, K_ADAM = 1, K_LAMB1 = 2, K_LAMB2 = 3, K_LARS1 = 4, K_LARS2 = 5, K_AF1 = 6, K_AF2 = 7, K_AF3 = 8 };
__host__ __device__ constexpr bool is_af(int o) { return o == K_AF1 || o == K_AF2 || o == K_AF3; }
// phase 1: reduces the gradient lists and leaves partial sums, no weight step
__host__ __device__ constexpr bool is_phase1(int o) { return o == K_LAMB1 || o == K_LARS1 || o == K_AF1; }
// phase 2: does not read the gradient lists (works from state and the stored gradient sum)
__host__ __device__ constexpr bool is_phase2(int o) { return o == K_LAMB2 || o == K_LARS2 || o == K_AF2 || o == K_AF3; }
__host__ __device__ constexpr bool writes_weights(int o) { return !is_phase1(o) && o != K_AF2; }
__host__ __device__ constexpr bool leaves_partials(int o) { return is_phase1(o) || o == K_AF2; }
// O_F32M: fused formatting with the fp32 weight tensors as the master copy (no sharded w exists)
enum { O_NONE = 0, O_F32 = 1, O_BF16 = 2, O_F32M = 3 };

template <int N>
struct GradPtrs {
    const void* p[N];
};

struct UpdParams {
    const WsTile* tiles;
    long long ntiles;
    long long nitems;       // shards in this launch * ntiles
    long long S;
    long long g_stride;     // per-shard element stride inside a gradient buffer (S, or 0 in slice mode)
    long long st_stride;    // per-shard element stride inside w/m/v (S for [R][S] state, 0 for one shard)
    int R;
    int r0;                 // first shard of this launch
    int concat;             // concatenated layout: tiles [tile_lo, tile_lo + nitems), each names its shard
    long long tile_lo;
    float* w;
    float* m;
    float* v;
    void* gathered;         // base of the G-element gathered buffer, or null
    const void* const* gtab; // fused formatting: device table [T][R] of gradient tensor pointers
    void* const* wtab;       // fused formatting: device table [T][nw] of weight tensor pointers (outputs)
    int nw;                  // number of weight lists written (1, or one per replica)
    int keep;                // norm pairs, phase 1: leave w and what phase 2 reads again in L2 (small models)
    int reverse;             // norm pairs, phase 2: walk the items back to front (phase 1's last items are still in L2)
    float2* partials;       // phase 1: [R][ntiles] partial sums of the two norms
    const float* rho;       // phase 2: [T] trust ratio (LAMB) / local rate (LARS)
    float* ghat;            // LARS, Adafactor: [R][S] summed gradients, written by phase 1, read afterwards
    const WsSegAf* segaf;   // Adafactor: [T] matrix view of every tensor
    float* af_acc;          // Adafactor pass 1: [F] row / column sums of g^2 + eps1 (atomic adds)
    const float* af_fac;    // Adafactor passes 2, 3: [F] 1/sqrt factors of V
    WsConsts c;
#ifdef WS_DEBUG_BOUNDS
    unsigned* bounds;       // status word of the bounds checks
    long long state_elems;  // elements of w / m / v as this launch addresses them
    long long grad_elems;   // ... of every packed gradient buffer
    long long out_elems;    // ... of the gathered buffer and of the stored gradient sum
#endif
};

// ---------------------------------------------------------------- memory ---
// A thread moves VEC consecutive elements at a time: VEC = 4 as one 128-bit access,
// VEC = 8 as one 256-bit access (ld/st.global.v8.b32, new with sm_100) for fp32 data
// and one 128-bit access for bf16 data.
template <int VEC>
struct Fv {
    float f[VEC];
};

template <int VEC>
__device__ __forceinline__ Fv<VEC> load_f32(const float* p) {
    Fv<VEC> o;
    if (VEC == 4) {
        const float4 v = __ldcs(reinterpret_cast<const float4*>(p));
        o.f[0] = v.x; o.f[1] = v.y; o.f[2] = v.z; o.f[3] = v.w;
    } else {
        unsigned r[8];
        asm volatile("ld.global.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                     : "l"(p));
#pragma unroll
        for (int i = 0; i < 8; ++i) o.f[i % VEC] = __uint_as_float(r[i]);
    }
    return o;
}

template <int VEC>
__device__ __forceinline__ void store_f32(float* p, const Fv<VEC>& x) {
    if (VEC == 4) {
        __stcs(reinterpret_cast<float4*>(p), make_float4(x.f[0], x.f[1], x.f[2], x.f[3]));
    } else {
        asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                     :: "l"(p), "r"(__float_as_uint(x.f[0])), "r"(__float_as_uint(x.f[1])), "r"(__float_as_uint(x.f[2])),
                        "r"(__float_as_uint(x.f[3])), "r"(__float_as_uint(x.f[4 % VEC])), "r"(__float_as_uint(x.f[5 % VEC])),
                        "r"(__float_as_uint(x.f[6 % VEC])), "r"(__float_as_uint(x.f[7 % VEC]))
                     : "memory");
    }
}

// Gradients as they come from memory (bf16 stays packed until it is summed).
template <bool GBF, int VEC>
struct GradRaw {
    float f[VEC];
};
template <>
struct GradRaw<true, 4> {
    uint2 u;
};
template <>
struct GradRaw<true, 8> {
    uint4 u;
};

template <bool GBF, int VEC>
__device__ __forceinline__ GradRaw<GBF, VEC> load_grad(const void* base, long long idx) {
    GradRaw<GBF, VEC> g;
    if constexpr (GBF) {
        const unsigned short* p = reinterpret_cast<const unsigned short*>(base) + idx;
        if constexpr (VEC == 4) g.u = __ldcs(reinterpret_cast<const uint2*>(p));
        else g.u = __ldcs(reinterpret_cast<const uint4*>(p));
    } else {
        const Fv<VEC> v = load_f32<VEC>(reinterpret_cast<const float*>(base) + idx);
#pragma unroll
        for (int i = 0; i < VEC; ++i) g.f[i] = v.f[i];
    }
    return g;
}

// The one vector of a tensor that holds its last element: only the first n elements exist.
template <bool GBF, int VEC>
__device__ __forceinline__ GradRaw<GBF, VEC> load_grad_partial(const void* base, long long idx, int n) {
    GradRaw<GBF, VEC> g;
    if constexpr (GBF) {
        const unsigned short* p = reinterpret_cast<const unsigned short*>(base) + idx;
        unsigned w[VEC / 2];
#pragma unroll
        for (int i = 0; i < VEC / 2; ++i) {
            const unsigned lo = (2 * i < n) ? p[2 * i] : 0u;
            const unsigned hi = (2 * i + 1 < n) ? p[2 * i + 1] : 0u;
            w[i] = lo | (hi << 16);
        }
        if constexpr (VEC == 4) g.u = make_uint2(w[0], w[1]);
        else g.u = make_uint4(w[0], w[1], w[2], w[3]);
    } else {
        const float* p = reinterpret_cast<const float*>(base) + idx;
#pragma unroll
        for (int i = 0; i < VEC; ++i) g.f[i] = (i < n) ? p[i] : 0.f;
    }
    return g;
}

template <int VEC>
__device__ __forceinline__ void store_f32_partial(float* p, const Fv<VEC>& x, int n) {
#pragma unroll
    for (int i = 0; i < VEC; ++i)
        if (i < n) p[i] = x.f[i];
}

template <int VEC>
__device__ __forceinline__ void store_bf16_partial(unsigned short* p, const Fv<VEC>& x, int n) {
#pragma unroll
    for (int i = 0; i < VEC; ++i)
        if (i < n) {
            const __nv_bfloat16 b = __float2bfloat16_rn(x.f[i]);
            p[i] = *reinterpret_cast<const unsigned short*>(&b);
        }
}

// bf16 -> fp32 widening is a 16-bit shift, exact
template <bool GBF, int VEC>
__device__ __forceinline__ Fv<VEC> widen(const GradRaw<GBF, VEC>& g) {
    Fv<VEC> o;
    if constexpr (GBF) {
        o.f[0] = __uint_as_float(g.u.x << 16);
        o.f[1] = __uint_as_float(g.u.x & 0xffff0000u);
        o.f[2] = __uint_as_float(g.u.y << 16);
        o.f[3] = __uint_as_float(g.u.y & 0xffff0000u);
        if constexpr (VEC == 8) {
            o.f[4] = __uint_as_float(g.u.z << 16);
            o.f[5] = __uint_as_float(g.u.z & 0xffff0000u);
            o.f[6] = __uint_as_float(g.u.w << 16);
            o.f[7] = __uint_as_float(g.u.w & 0xffff0000u);
        }
    } else {
#pragma unroll
        for (int i = 0; i < VEC; ++i) o.f[i] = g.f[i];
    }
    return o;
}

template <int VEC>
__device__ __forceinline__ void store_bf16(unsigned short* p, const Fv<VEC>& x) {
    unsigned pk[VEC / 2];
#pragma unroll
    for (int i = 0; i < VEC / 2; ++i) {
        const __nv_bfloat162 b = __floats2bfloat162_rn(x.f[2 * i], x.f[2 * i + 1]);
        pk[i] = *reinterpret_cast<const unsigned int*>(&b);
    }
    if constexpr (VEC == 4) __stcs(reinterpret_cast<uint2*>(p), make_uint2(pk[0], pk[1]));
    else __stcs(reinterpret_cast<uint4*>(p), make_uint4(pk[0], pk[1], pk[2], pk[3]));
}

// Kahan step: (sum, comp) += x
__device__ __forceinline__ void kahan1(float& s, float& c, float x) {
    const float y = x - c;
    const float t = s + y;
    c = (t - s) - y;
    s = t;
}

// ------------------------------------------------------------------ math ---
template <int OPT>
__device__ __forceinline__ void update_elem(const WsConsts& c, float g, float& w, float& m, float& v, float lr_rho,
                                            float& sw, float& su) {
    if (OPT == K_SGDM) {
        const float gp = fmaf(c.wd, w, g);
        m = fmaf(c.mu, m, gp);
        w = fmaf(-c.lr, m, w);
    } else if (OPT == K_LARS1) {          // norms of the weight and of the summed gradient
        sw = fmaf(w, w, sw);
        su = fmaf(g, g, su);
    } else if (OPT == K_LARS2) {          // lr_rho = lr * local rate of this tensor
        const float gp = fmaf(c.wd, w, g);
        m = fmaf(c.mu, m, lr_rho * gp);
        w = w - m;
    } else {
        if (OPT != K_LAMB2) {
            m = fmaf(c.beta1, m, c.omb1 * g);
            v = fmaf(c.beta2, v, c.omb2 * (g * g));
        }
        const float mhat = m * c.inv_bc1;
        const float vhat = v * c.inv_bc2;
        const float dir = mhat / (sqrtf(vhat) + c.eps);
        if (OPT == K_ADAM) {
            w = fmaf(-c.lr, dir, w);
        } else {
            const float u = fmaf(c.wd, w, dir);
            if (OPT == K_LAMB1) {
                sw = fmaf(w, w, sw);
                su = fmaf(u, u, su);
            } else {
                w = fmaf(-lr_rho, u, w);
            }
        }
    }
}

// Adds VEC consecutive floats to global memory with vector reductions (one or two
// red.global.add.v4.f32; p is 16-byte aligned).  Floating-point reductions on global memory are
// native at the L2; on shared memory they would be compare-and-swap loops.
template <int VEC>
__device__ __forceinline__ void red_add_vec(float* p, const float* x) {
#pragma unroll
    for (int j = 0; j < VEC; j += 4)
        asm volatile("red.global.add.v4.f32 [%0], {%1,%2,%3,%4};"
                     :: "l"(p + j), "f"(x[j]), "f"(x[j + 1]), "f"(x[j + 2]), "f"(x[j + 3]) : "memory");
}

// ---------------------------------------------------------------- kernel ---
// One work item: a run of `len` consecutive shard positions inside one tensor's piece.
struct ItemCtx {
    int len;             // elements, multiple of 8
    int nvalid;          // how many of them exist in the tensor (the rest is padding)
    int seg;             // tensor index
    long long gbase;     // first element inside each packed gradient buffer
    long long sbase;     // ... inside w / m / v
    long long obase;     // ... inside the gathered buffer and the stored gradient sum
    long long toff;      // ... inside tensor `seg` (fused formatting, Adafactor's rows and columns)
    float2* partial;     // where a phase-1 item leaves its two partial sums
    bool keep;           // HINT only: the state this item touches is read again soon (keep it in L2)
};

// Sums two values over the CTA at once (one pair of barriers for both); the totals are valid in
// thread 0.  The order of the additions is fixed, so the result is run-to-run bit-stable.
__device__ __forceinline__ float2 block_sum2(float x, float y, float2* smem /* kBlock/32 entries */) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        x += __shfl_xor_sync(0xffffffffu, x, o);
        y += __shfl_xor_sync(0xffffffffu, y, o);
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) smem[warp] = make_float2(x, y);
    __syncthreads();
    float2 t = make_float2(0.f, 0.f);
    if (threadIdx.x < 32) {
        if (lane < kBlock / 32) t = smem[lane];
#pragma unroll
        for (int o = 4; o > 0; o >>= 1) {
            t.x += __shfl_xor_sync(0xffffffffu, t.x, o);
            t.y += __shfl_xor_sync(0xffffffffu, t.y, o);
        }
    }
    return t;
}

// State loads and stores of an item.  Normally streaming (every operand crosses the chip once); with
// HINT and it.keep they leave the lines in L2 at normal priority, for a phase 2 that follows closely.
template <int VEC, bool HINT>
__device__ __forceinline__ Fv<VEC> load_state(const float* p, bool keep) {
    if constexpr (HINT) {
        if (keep) {
            Fv<VEC> o;
#pragma unroll
            for (int j = 0; j < VEC; j += 4) {
                const float4 v = __ldcg(reinterpret_cast<const float4*>(p + j));
                o.f[j] = v.x; o.f[j + 1] = v.y; o.f[j + 2] = v.z; o.f[j + 3] = v.w;
            }
            return o;
        }
    }
    return load_f32<VEC>(p);
}
template <int VEC, bool HINT>
__device__ __forceinline__ void store_state(float* p, const Fv<VEC>& x, bool keep) {
    if constexpr (HINT) {
        if (keep) {
#pragma unroll
            for (int j = 0; j < VEC; j += 4)
                __stcg(reinterpret_cast<float4*>(p + j), make_float4(x.f[j], x.f[j + 1], x.f[j + 2], x.f[j + 3]));
            return;
        }
    }
    store_f32<VEC>(p, x);
}
// The first n of VEC consecutive floats (the vector that holds a tensor's last element).
template <int VEC>
__device__ __forceinline__ Fv<VEC> load_f32_partial(const float* p, int n) {
    Fv<VEC> o;
#pragma unroll
    for (int i = 0; i < VEC; ++i) o.f[i] = (i < n) ? p[i] : 0.f;
    return o;
}

// OPT: optimizer / phase.  GBF: gradients are bf16.  OUT: where the updated weights go.
// VEC: elements per thread access.  U: accesses per thread per pass.
// RB: gradients summed per tree block.  NP: capacity of the by-value pointer table.
// FUSED: the formatting steps are fused in (Section 5.1) - gradients are read straight
// from the replicas' tensor lists and the updated weights are written straight to the
// weight tensors, so no packed gradient buffer and no gathered buffer exist.  With
// OUT == O_F32M the fp32 weight tensors are the master copy themselves: the weight is read
// from its tensor and written back there, and no sharded copy of w exists.
// HINT: see ItemCtx::keep.
// sgp: this item's R gradient tensor pointers (FUSED), swp: its weight tensor pointers when the
// result goes to several weight lists, wt: its first weight tensor; red: kBlock/32 float2 of
// shared memory.
template <int OPT, bool GBF, int OUT, int VEC, int U, int RB, int NP, bool FUSED, bool HINT>
__device__ __forceinline__ void process_item(const UpdParams& P, const GradPtrs<NP>& gp, const ItemCtx& it,
                                             const void* const* sgp, void* const* swp, char* wt, float lr_rho,
                                             float2* red) {
    constexpr bool HAS_V = (OPT == K_ADAM || OPT == K_LAMB1 || OPT == K_LAMB2);
    constexpr bool READS_G = !is_phase2(OPT);     // phase 2 works from state (and the stored gradient sum)
    constexpr bool READS_W = true;
    constexpr bool READS_M = (OPT != K_LARS1 && !is_af(OPT));
    constexpr bool READS_GHAT = (OPT == K_LARS2 || OPT == K_AF3);
    constexpr bool WRITES_W = writes_weights(OPT);   // phase 1 only zeroes the pads of w
    constexpr bool WRITES_M = (OPT != K_LAMB2 && OPT != K_LARS1 && !is_af(OPT));
    constexpr bool WRITES_GHAT = (OPT == K_LARS1 || OPT == K_AF1);
    constexpr bool LOOPK = (NP > RB);   // R may exceed one tree block: loop and compensate
    constexpr bool WMASTER = FUSED && OUT == O_F32M;   // w lives in the weight tensors only
    const int nvalid = it.nvalid;
    const long long gbase = it.gbase, sbase = it.sbase, obase = it.obase, toff = it.toff;
    const int nvec = it.len / VEC;
#ifdef WS_DEBUG_BOUNDS
    {
        // every access of the item lies in [base, base + len) of its buffer: check the three ranges once
        unsigned bits = 0;
        if (sbase < 0 || sbase + it.len > P.state_elems) bits |= WS_BOUNDS_STATE;
        if (READS_G && !FUSED && (gbase < 0 || gbase + it.len > P.grad_elems)) bits |= WS_BOUNDS_GRAD;
        const bool uses_out = (WRITES_W && !FUSED && OUT != O_NONE) || READS_GHAT || WRITES_GHAT;
        if (uses_out && (obase < 0 || obase + it.len > P.out_elems)) bits |= WS_BOUNDS_OUT;
        if (bits) {                                    // uniform over the CTA: the item is skipped
            if (threadIdx.x == 0 && P.bounds) atomicOr(P.bounds, bits);
            return;
        }
    }
#endif
    float sw = 0.f, su = 0.f;
    // Adafactor: where the tile starts inside its tensor's rows x cols matrix
    WsSegAf af = {};
    long long row0 = 0, c0 = 0;
    bool rowsum = false, bigcol = false;
    if constexpr (is_af(OPT)) {
        af = P.segaf[it.seg];
        rowsum = af.nrow > 0;                          // unfactored tensors are one row
        if (af.ncol > 0) {
            if ((((unsigned long long)toff | (unsigned long long)af.ncol) >> 32) == 0) {
                const unsigned q32 = (unsigned)toff / (unsigned)af.ncol;   // the usual case: no 64-bit division
                row0 = q32;
                c0 = (unsigned)toff - q32 * (unsigned)af.ncol;
            } else {
                row0 = toff / af.ncol;
                c0 = toff - row0 * af.ncol;
            }
        }
        bigcol = af.ncol >= it.len;                    // the tile touches at most two rows
    }
    // When the row length is a multiple of VEC a vector never straddles rows and starts on a
    // multiple of VEC (colrun).  Pass 1 then adds a vector's g^2 + eps1 to the column sums with
    // one vector reduction; when the row length also divides the distance between a thread's
    // consecutive vectors, the thread meets the same VEC columns in every vector, keeps their sums
    // in registers and adds them once per tile (stationary).
    const bool colrun = is_af(OPT) && af.ncol % VEC == 0;
    const bool stationary = colrun && (kBlock * VEC) % af.ncol == 0;   // (the stride between ANY two of its vectors)
    // the thread's first vector starts at column run_col of row run_rl (relative to the tile's first
    // row); consecutive vectors of a thread lie kBlock * VEC elements apart = sub_rl rows and
    // sub_col columns, so rows and columns advance without a division per vector
    long long run_col = 0, sub_col = 0;
    unsigned run_rl = 0, sub_rl = 0;
    if constexpr (is_af(OPT)) {
        run_col = c0 + (long long)threadIdx.x * VEC;
        sub_col = kBlock * VEC;
        if (bigcol) {
            if (run_col >= af.ncol) { run_rl = 1; run_col -= af.ncol; }
        } else {
            run_rl = (unsigned)run_col / (unsigned)af.ncol;
            run_col = (unsigned)run_col - run_rl * (unsigned)af.ncol;
        }
        if (af.ncol <= kBlock * VEC) {
            sub_rl = (unsigned)(kBlock * VEC) / (unsigned)af.ncol;
            sub_col = (unsigned)(kBlock * VEC) - sub_rl * (unsigned)af.ncol;
        }
    }
    float cacc[OPT == K_AF1 ? VEC : 1];
    long long cbase = -1;
#pragma unroll
    for (int j = 0; j < (OPT == K_AF1 ? VEC : 1); ++j) cacc[j] = 0.f;

    for (int q0 = 0; q0 < nvec; q0 += U * kBlock) {
        int e0[U];
        int nv[U];
        Fv<VEC> wv[U], mv[U], vv[U], gv[U], gc[U];
        unsigned rl0[is_af(OPT) ? U : 1];      // Adafactor: row (relative to the tile's first) and
        long long col0[is_af(OPT) ? U : 1];    // column of each vector's first element
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int q = q0 + u * kBlock + threadIdx.x;
            e0[u] = q * VEC;
            if constexpr (is_af(OPT)) {
                // this vector's row and column, then on to the thread's next vector
                rl0[u] = run_rl;
                col0[u] = run_col;
                run_col += sub_col;
                run_rl += sub_rl;
                if (run_col >= af.ncol) { run_col -= af.ncol; ++run_rl; }
            }
            const int left = nvalid - e0[u];
            nv[u] = q < nvec ? (left < 0 ? 0 : (left > VEC ? VEC : left)) : -1;  // -1: nothing here
#pragma unroll
            for (int j = 0; j < VEC; ++j) wv[u].f[j] = mv[u].f[j] = vv[u].f[j] = gv[u].f[j] = gc[u].f[j] = 0.f;
        }
        // issue every load of the pass before any arithmetic
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (nv[u] > 0) {
                if constexpr (WMASTER) {
                    const float* src = reinterpret_cast<const float*>(wt) + toff + e0[u];
                    wv[u] = nv[u] == VEC ? load_state<VEC, HINT>(src, it.keep) : load_f32_partial<VEC>(src, nv[u]);
                } else if (READS_W) {
                    wv[u] = load_state<VEC, HINT>(P.w + sbase + e0[u], it.keep);
                }
                if (READS_M) mv[u] = load_state<VEC, HINT>(P.m + sbase + e0[u], it.keep);
                if (HAS_V) vv[u] = load_state<VEC, HINT>(P.v + sbase + e0[u], it.keep);
                if (READS_GHAT) gv[u] = load_state<VEC, HINT>(P.ghat + obase + e0[u], it.keep);   // summed gradient from phase 1
            }
        }
        if (READS_G) {
            for (int k0 = 0; k0 < (LOOPK ? P.R : 1); k0 += RB) {
                GradRaw<GBF, VEC> raw[U][RB];
                bool have[RB];
#pragma unroll
                for (int j = 0; j < RB; ++j) {
                    have[j] = (RB == 1) || (k0 + j < P.R);
#pragma unroll
                    for (int u = 0; u < U; ++u)
                        if (have[j] && nv[u] > 0) {
                            if constexpr (FUSED) {
                                const void* gk = sgp[k0 + j];
                                if (nv[u] == VEC) raw[u][j] = load_grad<GBF, VEC>(gk, toff + e0[u]);
                                else raw[u][j] = load_grad_partial<GBF, VEC>(gk, toff + e0[u], nv[u]);
                            } else {
                                raw[u][j] = load_grad<GBF, VEC>(gp.p[k0 + j], gbase + e0[u]);
                            }
                        }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    Fv<VEC> gb[RB];
#pragma unroll
                    for (int j = 0; j < RB; ++j) {
                        if (have[j] && nv[u] > 0) {
                            gb[j] = widen<GBF, VEC>(raw[u][j]);
                        } else {
#pragma unroll
                            for (int i = 0; i < VEC; ++i) gb[j].f[i] = 0.f;
                        }
                    }
#pragma unroll
                    for (int s = 1; s < RB; s <<= 1)
#pragma unroll
                        for (int j = 0; j + s < RB; j += 2 * s)
#pragma unroll
                            for (int i = 0; i < VEC; ++i) gb[j].f[i] += gb[j + s].f[i];
                    if (!LOOPK || k0 == 0) {
                        gv[u] = gb[0];
                    } else {
#pragma unroll
                        for (int i = 0; i < VEC; ++i) kahan1(gv[u].f[i], gc[u].f[i], gb[0].f[i]);
                    }
                }
            }
        }
        if constexpr (OPT == K_AF1) {
            // g^2 + eps1 of every valid element goes to its row and to its column.  A thread's
            // elements are consecutive, so they form one run per row; when a whole warp sits in
            // one row (the usual case) the runs are combined by shuffles before the one add.
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const bool has = nv[u] > 0;
                long long col = col0[u];
                unsigned rl = rl0[u];
                unsigned cur = rl;
                bool simple = true;
                float racc = 0.f;
                if (has) {
                    float* gcol = P.af_acc + af.icol;
                    float xs[VEC];
#pragma unroll
                    for (int j = 0; j < VEC; ++j) {
                        xs[j] = 0.f;
                        if (j < nv[u]) {
                            const float g = gv[u].f[j] * P.c.gscale;
                            gv[u].f[j] = g;
                            sw = fmaf(wv[u].f[j], wv[u].f[j], sw);
                            xs[j] = fmaf(g, g, P.c.eps);
                        }
                    }
                    if (colrun) {
                        // the whole vector lies in one row, on VEC aligned columns
                        if (!rowsum) {
                            // unfactored: every element has its own slot
#pragma unroll
                            for (int j = 0; j < VEC; j += 4)
                                *reinterpret_cast<float4*>(gcol + col + j) = make_float4(xs[j], xs[j + 1], xs[j + 2], xs[j + 3]);
                        } else {
#pragma unroll
                            for (int j = 0; j < VEC; ++j) racc += xs[j];
                            if (stationary) {
                                cbase = col;
#pragma unroll
                                for (int j = 0; j < VEC; ++j) cacc[j] += xs[j];
                            } else {
                                red_add_vec<VEC>(gcol + col, xs);
                            }
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < VEC; ++j) {
                            if (j < nv[u]) {
                                if (!rowsum) {
                                    gcol[col] = xs[j];
                                } else {
                                    atomicAdd(&gcol[col], xs[j]);
                                    if (rl != cur) {
                                        atomicAdd(&P.af_acc[af.irow + row0 + cur], racc);
                                        racc = 0.f;
                                        cur = rl;
                                        simple = false;
                                    }
                                    racc += xs[j];
                                }
                                if (++col == af.ncol) { col = 0; ++rl; }
                            }
                        }
                    }
                }
                if (rowsum) {   // uniform over the CTA
                    const unsigned act = __ballot_sync(0xffffffffu, has);
                    if (act) {
                        const int lead = __ffs(act) - 1;
                        const unsigned lead_row = __shfl_sync(0xffffffffu, cur, lead);
                        const bool uni = __all_sync(0xffffffffu, !has || (simple && cur == lead_row));
                        if (uni) {
                            float tsum = has ? racc : 0.f;
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1) tsum += __shfl_xor_sync(0xffffffffu, tsum, o);
                            if ((int)(threadIdx.x & 31) == lead) atomicAdd(&P.af_acc[af.irow + row0 + lead_row], tsum);
                        } else if (has) {
                            atomicAdd(&P.af_acc[af.irow + row0 + cur], racc);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (nv[u] < 0) continue;
            if constexpr (OPT == K_AF3) {
                // U = g / sqrt(V) with V = Rv' Cv'^T / sum(Rv'): the finalize step left
                // sqrt(sum(Rv') / Rv'_i) and 1 / sqrt(Cv'_j), so U = g * fr_i * fc_j
                long long col = col0[u];
                unsigned rl = rl0[u];
                const float* frp = P.af_fac + af.irow + row0;
                const float* fcp = P.af_fac + af.icol;
                float fr = 1.f;
                if (rowsum && nv[u] > 0) fr = __ldg(frp + rl);
                if (colrun && nv[u] > 0) {
                    // the vector lies in one row and its column factors are one aligned vector
                    float fc[VEC];
#pragma unroll
                    for (int j4 = 0; j4 < VEC; j4 += 4) {
                        const float4 t4 = __ldg(reinterpret_cast<const float4*>(fcp + col + j4));
                        fc[j4] = t4.x; fc[j4 + 1] = t4.y; fc[j4 + 2] = t4.z; fc[j4 + 3] = t4.w;
                    }
#pragma unroll
                    for (int j = 0; j < VEC; ++j) {
                        if (j < nv[u]) {
                            const float uu = (gv[u].f[j] * fr) * fc[j];
                            wv[u].f[j] = fmaf(-lr_rho, uu, wv[u].f[j]);
                        } else {
                            wv[u].f[j] = 0.f;
                        }
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < VEC; ++j) {
                        if (j < nv[u]) {
                            const float uu = (gv[u].f[j] * fr) * __ldg(fcp + col);
                            wv[u].f[j] = fmaf(-lr_rho, uu, wv[u].f[j]);
                            if (++col == af.ncol) {
                                col = 0;
                                ++rl;
                                if (rowsum && j + 1 < nv[u]) fr = __ldg(frp + rl);
                            }
                        } else {
                            wv[u].f[j] = 0.f;
                        }
                    }
                }
            } else {
#pragma unroll
                for (int j = 0; j < VEC; ++j) {
                    if (j < nv[u]) {
                        if (READS_G && OPT != K_AF1) gv[u].f[j] *= P.c.gscale;     // (phase 1 stored it already scaled)
                        if (OPT != K_AF1) update_elem<OPT>(P.c, gv[u].f[j], wv[u].f[j], mv[u].f[j], vv[u].f[j], lr_rho, sw, su);
                    } else {  // pad: identity for the sums, +0 for every output
                        wv[u].f[j] = 0.f; mv[u].f[j] = 0.f; vv[u].f[j] = 0.f; gv[u].f[j] = 0.f;
                    }
                }
            }
            const long long so = sbase + e0[u];
            if constexpr (!WMASTER)
                if (WRITES_W || (READS_W && nv[u] < VEC)) store_state<VEC, HINT>(P.w + so, wv[u], it.keep && !WRITES_W);
            if (WRITES_M) store_state<VEC, HINT>(P.m + so, mv[u], it.keep);
            if (HAS_V && OPT != K_LAMB2) store_state<VEC, HINT>(P.v + so, vv[u], it.keep);
            if (WRITES_GHAT) store_state<VEC, HINT>(P.ghat + obase + e0[u], gv[u], it.keep);   // keep the sum for the later passes
            if constexpr (!WRITES_W) {
                // no weight output in this pass
            } else if constexpr (FUSED) {
                if (OUT == O_F32 || OUT == O_F32M) {
                    float* dst = reinterpret_cast<float*>(wt) + toff + e0[u];
                    if (nv[u] == VEC) store_f32<VEC>(dst, wv[u]);
                    else store_f32_partial<VEC>(dst, wv[u], nv[u]);
                } else if (OUT == O_BF16) {
                    unsigned short* dst = reinterpret_cast<unsigned short*>(wt) + toff + e0[u];
                    if (nv[u] == VEC) store_bf16<VEC>(dst, wv[u]);
                    else store_bf16_partial<VEC>(dst, wv[u], nv[u]);
                }
                if constexpr (READS_G) {
                    for (int k = 1; k < P.nw; ++k) {      // the other replicas' weight tensors
                        if (OUT == O_F32) {
                            float* dst = reinterpret_cast<float*>(swp[k]) + toff + e0[u];
                            if (nv[u] == VEC) store_f32<VEC>(dst, wv[u]);
                            else store_f32_partial<VEC>(dst, wv[u], nv[u]);
                        } else if (OUT == O_BF16) {
                            unsigned short* dst = reinterpret_cast<unsigned short*>(swp[k]) + toff + e0[u];
                            if (nv[u] == VEC) store_bf16<VEC>(dst, wv[u]);
                            else store_bf16_partial<VEC>(dst, wv[u], nv[u]);
                        }
                    }
                }
            } else if (OUT == O_F32) {
                store_f32<VEC>(reinterpret_cast<float*>(P.gathered) + obase + e0[u], wv[u]);
            } else if (OUT == O_BF16) {
                store_bf16<VEC>(reinterpret_cast<unsigned short*>(P.gathered) + obase + e0[u], wv[u]);
            }
        }
    }
    if constexpr (OPT == K_AF1) {
        // (these adds of partial reduce results across tiles and shards stand where the paper
        // combines them with an all-reduce, Section 4.1)
        if (cbase >= 0) red_add_vec<VEC>(P.af_acc + af.icol + cbase, cacc);
    }
    if (leaves_partials(OPT)) {
        // (Adafactor's passes leave one sum each)
        const float2 ab = block_sum2(sw, su, red);
        if (threadIdx.x == 0) *it.partial = make_float2(ab.x, ab.y);   // (Adafactor's pass 1: y = 0, pass 2 adds its sum there)
    }
}


// ---------------------------------------------------------- one-launch update ---
// What the one-kernel LAMB / LARS update (ws_onelaunch.cu) needs beyond UpdParams: the plan's
// schedule and the synchronisation scratch inside the workspace.
struct OneLaunch {
    const unsigned* sched;       // [nsched] item index * 2 + phase, in execution order
    unsigned nsched;
    const WsItem* items;
    const WsItemSeg* segs;       // [T] item range of every tensor
    int T;
    float2* ipart;               // [items] partial norm sums of every item's phase 1
    int* count;                  // [T] finished phase-1 items per tensor        (cleared before the launch)
    unsigned long long* flag;    // [T] (ratio bits << 32) | 1 once the ratio is known (cleared before the launch)
    unsigned long long* ticket;  // next schedule entry to hand out              (cleared before the launch)
    int* status;                 // 0, or 1 after a wait ran out                  (cleared before the launch)
    float* rho;                  // [T] ratios
    double* norms;               // [T][2]
    double eta, beta;            // LARS: trust coefficient and weight decay
};
bool one_launch_supports(int pair, int R);
// pair 0: LAMB, 1: LARS.  P carries the arguments of both phases (gradient sources, state, outputs).
ws_status launch_one_launch(int pair, bool gbf, int out, bool fused, bool wide, const UpdParams& P,
                            const void* const* gptrs, const OneLaunch& Q, cudaStream_t st);

}  // namespace wsk
