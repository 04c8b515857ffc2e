// Fused reduce + optimizer update + gathered-layout write.
//
// One kernel does, for every element of a shard (paper Section 2.2): sum the R
// replicas' gradients for that position (the reduce-scatter arithmetic), apply
// the optimizer to the weight and its slots, store them, and store the updated
// weight into slot r of the all-gather layout (fp32, or bf16 rounded from the
// fp32 result, Section 4.2).  Intermediates live in registers only (the
// "fusion" of Section 2.1); every operand crosses HBM exactly once.
//
// Work item = (shard r, tile); a thread owns quads of 4 consecutive elements
// and moves them as 16-byte vectors.  Pads are recognised by location
// (element index within the tile vs. the tile's valid length for shard r), so
// gradient pads are never read into a result and output pads are +0
// (Section 4.1, "Non-elementwise operators": mask with the identity).
//
// The R-way sum is formed as tree sums over blocks of RB gradients combined by
// a compensated (Kahan) accumulation, never as one sequential fp32 chain: the
// loads of a block are independent (memory-level parallelism) and the rounding
// error stays near one ulp for R up to 1024.
#include <cuda_bf16.h>
#include <math.h>

#include "ws_internal.h"

namespace {

constexpr int kBlock = 256;
enum { K_SGDM = 0, K_ADAM = 1, K_LAMB1 = 2, K_LAMB2 = 3 };
enum { O_NONE = 0, O_F32 = 1, O_BF16 = 2 };

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
    float* w;
    float* m;
    float* v;
    void* gathered;         // base of the G-element gathered buffer, or null
    float2* partials;       // LAMB: [R][ntiles]
    const float* rho;       // LAMB phase 2: [T]
    WsConsts c;
};

// ---------------------------------------------------------------- memory ---
__device__ __forceinline__ float4 ldg_f4(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ void stg_f4(float* p, float4 v) { __stcs(reinterpret_cast<float4*>(p), v); }

template <bool BF16>
__device__ __forceinline__ float4 load_grad4(const void* base, long long idx) {
    if (BF16) {
        const uint2 u = __ldcs(reinterpret_cast<const uint2*>(reinterpret_cast<const unsigned short*>(base) + idx));
        float4 g;  // bf16 -> fp32 widening is a 16-bit shift, exact
        g.x = __uint_as_float(u.x << 16);
        g.y = __uint_as_float(u.x & 0xffff0000u);
        g.z = __uint_as_float(u.y << 16);
        g.w = __uint_as_float(u.y & 0xffff0000u);
        return g;
    } else {
        return ldg_f4(reinterpret_cast<const float*>(base) + idx);
    }
}

__device__ __forceinline__ float4 add4(float4 a, float4 b) { return make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w); }

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

__device__ __forceinline__ float block_sum(float x, float* smem /* kBlock/32 floats */) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) smem[warp] = x;
    __syncthreads();
    float t = 0.f;
    if (threadIdx.x < 32) {
        t = lane < kBlock / 32 ? smem[lane] : 0.f;
#pragma unroll
        for (int o = 4; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    }
    return t;  // valid in thread 0
}

// ---------------------------------------------------------------- kernel ---
// OPT: optimizer / phase.  GBF: gradients are bf16.  OUT: gathered dtype.
// U: quads per thread per pass.  RB: gradients summed per tree block.
// NP: capacity of the by-value gradient pointer table.
template <int OPT, bool GBF, int OUT, int U, int RB, int NP>
__global__ void __launch_bounds__(kBlock) update_kernel(const UpdParams P, const __grid_constant__ GradPtrs<NP> gp) {
    constexpr bool HAS_V = (OPT != K_SGDM);
    constexpr bool READS_G = (OPT != K_LAMB2);
    __shared__ float red[2][kBlock / 32];

    for (long long item = blockIdx.x; item < P.nitems; item += gridDim.x) {
        const long long rs = item / P.ntiles;              // shard index inside this launch
        const long long ti = item - rs * P.ntiles;
        const long long r = P.r0 + rs;
        const WsTile tl = P.tiles[ti];
        long long nvl = tl.vt - r * tl.piece;              // valid elements in this tile for shard r
        const int nvalid = nvl < 0 ? 0 : (nvl > tl.len ? tl.len : (int)nvl);
        const long long gbase = rs * P.g_stride + tl.pos;  // into each gradient buffer
        const long long sbase = rs * P.st_stride + tl.pos; // into w/m/v
        const long long obase = r * P.S + tl.pos;          // into the gathered buffer
        const int nquad = tl.len >> 2;
        float lr_rho = 0.f;
        if (OPT == K_LAMB2) lr_rho = P.c.lr * P.rho[tl.seg];
        float sw = 0.f, su = 0.f;

        for (int q0 = 0; q0 < nquad; q0 += U * kBlock) {
            int e0[U];
            int nv[U];
            float4 w4[U], m4[U], v4[U], g4[U], gc[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int q = q0 + u * kBlock + threadIdx.x;
                e0[u] = q << 2;
                const int left = nvalid - e0[u];
                nv[u] = q < nquad ? (left < 0 ? 0 : (left > 4 ? 4 : left)) : -1;  // -1: no quad here
                w4[u] = m4[u] = v4[u] = g4[u] = gc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            // issue every load of the pass before any arithmetic
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (nv[u] > 0) {
                    w4[u] = ldg_f4(P.w + sbase + e0[u]);
                    m4[u] = ldg_f4(P.m + sbase + e0[u]);
                    if (HAS_V) v4[u] = ldg_f4(P.v + sbase + e0[u]);
                }
            }
            if (READS_G) {
                for (int k0 = 0; k0 < P.R; k0 += RB) {
                    float4 gb[U][RB];
#pragma unroll
                    for (int j = 0; j < RB; ++j) {
#pragma unroll
                        for (int u = 0; u < U; ++u) {
                            gb[u][j] = make_float4(0.f, 0.f, 0.f, 0.f);
                            if (k0 + j < P.R && nv[u] > 0) gb[u][j] = load_grad4<GBF>(gp.p[k0 + j], gbase + e0[u]);
                        }
                    }
#pragma unroll
                    for (int u = 0; u < U; ++u) {
#pragma unroll
                        for (int s = 1; s < RB; s <<= 1)
#pragma unroll
                            for (int j = 0; j + s < RB; j += 2 * s) gb[u][j] = add4(gb[u][j], gb[u][j + s]);
                        if (k0 == 0) {
                            g4[u] = gb[u][0];
                        } else {
                            kahan1(g4[u].x, gc[u].x, gb[u][0].x);
                            kahan1(g4[u].y, gc[u].y, gb[u][0].y);
                            kahan1(g4[u].z, gc[u].z, gb[u][0].z);
                            kahan1(g4[u].w, gc[u].w, gb[u][0].w);
                        }
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (nv[u] < 0) continue;
                float wv[4] = {w4[u].x, w4[u].y, w4[u].z, w4[u].w};
                float mv[4] = {m4[u].x, m4[u].y, m4[u].z, m4[u].w};
                float vv[4] = {v4[u].x, v4[u].y, v4[u].z, v4[u].w};
                const float gv[4] = {g4[u].x, g4[u].y, g4[u].z, g4[u].w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (j < nv[u]) {
                        update_elem<OPT>(P.c, gv[j] * P.c.gscale, wv[j], mv[j], vv[j], lr_rho, sw, su);
                    } else {  // pad: identity for the sums, +0 for every output
                        wv[j] = 0.f; mv[j] = 0.f; vv[j] = 0.f;
                    }
                }
                const long long so = sbase + e0[u];
                if (OPT != K_LAMB1) stg_f4(P.w + so, make_float4(wv[0], wv[1], wv[2], wv[3]));
                if (OPT == K_LAMB1 && nv[u] < 4) stg_f4(P.w + so, make_float4(wv[0], wv[1], wv[2], wv[3]));
                if (OPT != K_LAMB2) {
                    stg_f4(P.m + so, make_float4(mv[0], mv[1], mv[2], mv[3]));
                    if (HAS_V) stg_f4(P.v + so, make_float4(vv[0], vv[1], vv[2], vv[3]));
                }
                if (OUT == O_F32) {
                    stg_f4(reinterpret_cast<float*>(P.gathered) + obase + e0[u], make_float4(wv[0], wv[1], wv[2], wv[3]));
                } else if (OUT == O_BF16) {
                    const __nv_bfloat162 lo = __floats2bfloat162_rn(wv[0], wv[1]);
                    const __nv_bfloat162 hi = __floats2bfloat162_rn(wv[2], wv[3]);
                    uint2 pk;
                    pk.x = *reinterpret_cast<const unsigned int*>(&lo);
                    pk.y = *reinterpret_cast<const unsigned int*>(&hi);
                    __stcs(reinterpret_cast<uint2*>(reinterpret_cast<unsigned short*>(P.gathered) + obase + e0[u]), pk);
                }
            }
        }
        if (OPT == K_LAMB1) {
            const float a = block_sum(sw, red[0]);
            const float b = block_sum(su, red[1]);
            if (threadIdx.x == 0) P.partials[r * P.ntiles + ti] = make_float2(a, b);
        }
    }
}

// Sum every shard's per-tile partials of tensor t in a fixed order, in double
// (stands where the paper combines per-replica reduce results with one batched
// scalar all-reduce, Section 4.1 / 5.2), then rho_t = sqrt(a)/sqrt(b).
__global__ void __launch_bounds__(kBlock) lamb_finalize_kernel(const WsSegTiles* segtiles, const float2* partials,
                                                               long long ntiles, int R, float* rho, double* norms) {
    __shared__ double sa[kBlock], sb[kBlock];
    const int t = blockIdx.x;
    const WsSegTiles st = segtiles[t];
    const long long n = (long long)R * st.tile_count;
    double a = 0.0, b = 0.0;
    for (long long i = threadIdx.x; i < n; i += kBlock) {
        const long long r = i / st.tile_count, k = i - r * st.tile_count;
        const float2 p = partials[r * ntiles + st.tile_begin + k];
        a += (double)p.x;
        b += (double)p.y;
    }
    sa[threadIdx.x] = a;
    sb[threadIdx.x] = b;
    __syncthreads();
    for (int s = kBlock / 2; s > 0; s >>= 1) {
        if (threadIdx.x < s) {
            sa[threadIdx.x] += sa[threadIdx.x + s];
            sb[threadIdx.x] += sb[threadIdx.x + s];
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        a = sa[0];
        b = sb[0];
        norms[2 * t] = a;
        norms[2 * t + 1] = b;
        rho[t] = (a > 0.0 && b > 0.0) ? (float)(sqrt(a) / sqrt(b)) : 1.0f;
    }
}

// -------------------------------------------------------------- dispatch ---
int sm_count() {
    static thread_local int dev_cached = -1, sms = 148;
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev != dev_cached) {
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        dev_cached = dev;
    }
    return sms;
}

template <int OPT, bool GBF, int OUT, int U, int RB, int NP>
ws_status launch(const UpdParams& P, const void* const* gptrs, cudaStream_t st) {
    GradPtrs<NP> gp;
    for (int k = 0; k < NP; ++k) gp.p[k] = (gptrs && k < P.R) ? gptrs[k] : nullptr;
    long long grid = P.nitems;
    const long long cap = (long long)sm_count() * 32;
    if (grid > cap) grid = cap;
    if (grid < 1) return WS_OK;
    update_kernel<OPT, GBF, OUT, U, RB, NP><<<(unsigned)grid, kBlock, 0, st>>>(P, gp);
    return ws_check_launch("ws_shard_update");
}

template <int OPT, bool GBF, int OUT>
ws_status launch_r(const UpdParams& P, const void* const* gptrs, cudaStream_t st) {
    if (OPT == K_LAMB2) return launch<OPT, GBF, OUT, 2, 1, 1>(P, gptrs, st);
    if (P.R <= 2) return launch<OPT, GBF, OUT, 2, 2, 8>(P, gptrs, st);
    if (P.R <= 4) return launch<OPT, GBF, OUT, 2, 4, 8>(P, gptrs, st);
    if (P.R <= 32) return launch<OPT, GBF, OUT, 1, 8, 32>(P, gptrs, st);
    if (P.R <= 1024) return launch<OPT, GBF, OUT, 1, 8, 1024>(P, gptrs, st);
    return WS_ERR_TOO_LARGE;
}

template <int OPT, bool GBF>
ws_status launch_o(const UpdParams& P, const void* const* gptrs, int out, cudaStream_t st) {
    if (OPT == K_LAMB1) return launch_r<OPT, GBF, O_NONE>(P, gptrs, st);
    switch (out) {
        case O_NONE: return launch_r<OPT, GBF, O_NONE>(P, gptrs, st);
        case O_F32: return launch_r<OPT, GBF, O_F32>(P, gptrs, st);
        default: return launch_r<OPT, GBF, O_BF16>(P, gptrs, st);
    }
}

ws_status launch_any(int opt, bool gbf, int out, const UpdParams& P, const void* const* gptrs, cudaStream_t st) {
    switch (opt) {
        case K_SGDM: return gbf ? launch_o<K_SGDM, true>(P, gptrs, out, st) : launch_o<K_SGDM, false>(P, gptrs, out, st);
        case K_ADAM: return gbf ? launch_o<K_ADAM, true>(P, gptrs, out, st) : launch_o<K_ADAM, false>(P, gptrs, out, st);
        case K_LAMB1: return gbf ? launch_o<K_LAMB1, true>(P, gptrs, out, st) : launch_o<K_LAMB1, false>(P, gptrs, out, st);
        default: return launch_o<K_LAMB2, false>(P, gptrs, out, st);
    }
}

WsConsts make_consts(const ws_hyper* h) {
    WsConsts c;
    const double bc1 = 1.0 - pow(h->beta1, (double)h->step);
    const double bc2 = 1.0 - pow(h->beta2, (double)h->step);
    c.lr = (float)h->lr;
    c.beta1 = (float)h->beta1;
    c.omb1 = (float)(1.0 - h->beta1);
    c.beta2 = (float)h->beta2;
    c.omb2 = (float)(1.0 - h->beta2);
    c.eps = (float)h->eps;
    c.wd = (float)h->weight_decay;
    c.mu = (float)h->momentum;
    c.gscale = (float)h->grad_scale;
    c.inv_bc1 = (float)(1.0 / bc1);
    c.inv_bc2 = (float)(1.0 / bc2);
    return c;
}

// Argument checks shared by the entry points; fills P.  phase: K_* kernel id.
ws_status prepare(const ws_plan* p, int32_t r, const ws_grads* g, const ws_state* s, const ws_hyper* h,
                  const ws_out* out, int phase, UpdParams& P, int& out_kind, bool& gbf) {
    if (!p || !s || !h) return WS_ERR_INVALID_ARG;
    if (!p->d_tiles) return WS_ERR_NOT_UPLOADED;
    if (r < -1 || r >= p->R) return WS_ERR_INVALID_ARG;
    if (h->step < 1) return WS_ERR_INVALID_ARG;
    const bool needs_v = (phase != K_SGDM);
    if (!s->w || !s->m || (needs_v && !s->v)) return WS_ERR_INVALID_ARG;
    if (!ws_aligned16(s->w) || !ws_aligned16(s->m) || (needs_v && !ws_aligned16(s->v))) return WS_ERR_ALIGNMENT;
    gbf = false;
    if (phase != K_LAMB2) {
        if (!g || !g->ptrs || g->R < 1) return WS_ERR_INVALID_ARG;
        if (g->dtype != WS_F32 && g->dtype != WS_BF16) return WS_ERR_DTYPE;
        if (g->slice_mode != 0 && g->slice_mode != 1) return WS_ERR_INVALID_ARG;
        if (g->slice_mode == 0 && g->R != p->R) return WS_ERR_INVALID_ARG;
        if (g->slice_mode == 1 && r < 0) return WS_ERR_INVALID_ARG;
        if (g->R > 1024) return WS_ERR_TOO_LARGE;
        for (int k = 0; k < g->R; ++k) {
            if (!g->ptrs[k]) return WS_ERR_INVALID_ARG;
            if (!ws_aligned16(g->ptrs[k])) return WS_ERR_ALIGNMENT;
        }
        gbf = (g->dtype == WS_BF16);
        // shard r of a packed buffer starts r*S elements in; S is a multiple of 8,
        // so the start keeps 16-byte alignment for both dtypes
    }
    out_kind = O_NONE;
    if (out && out->gathered) {
        if (out->dtype != WS_F32 && out->dtype != WS_BF16) return WS_ERR_DTYPE;
        if (!ws_aligned16(out->gathered)) return WS_ERR_ALIGNMENT;
        out_kind = out->dtype == WS_F32 ? O_F32 : O_BF16;
    }
    P.tiles = p->d_tiles;
    P.ntiles = p->ntiles;
    P.S = p->S;
    P.R = g ? g->R : p->R;
    const int nshards = (r < 0) ? p->R : 1;
    P.r0 = (r < 0) ? 0 : r;
    P.nitems = (long long)nshards * p->ntiles;
    P.st_stride = (r < 0) ? p->S : 0;
    if (g && phase != K_LAMB2) {
        // slice mode 0: pointer is the packed buffer; the launch starts at shard r0
        P.g_stride = (g->slice_mode == 0) ? p->S : 0;
    } else {
        P.g_stride = 0;
    }
    P.w = (float*)s->w;
    P.m = (float*)s->m;
    P.v = (float*)s->v;
    P.gathered = (out_kind != O_NONE) ? out->gathered : nullptr;
    P.partials = nullptr;
    P.rho = nullptr;
    P.c = make_consts(h);
    return WS_OK;
}

// In slice mode 0 with a single shard r the kernel indexes gradient buffers by
// the launch-local shard index (0), so the pointers are advanced to shard r.
void offset_grad_ptrs(const ws_plan* p, int32_t r, const ws_grads* g, std::vector<const void*>& v) {
    v.resize(g->R);
    const size_t eb = g->dtype == WS_BF16 ? 2 : 4;
    for (int k = 0; k < g->R; ++k) {
        const char* b = (const char*)g->ptrs[k];
        if (g->slice_mode == 0 && r > 0) b += (size_t)r * (size_t)p->S * eb;
        v[k] = b;
    }
}

ws_status check_ws(const ws_plan* p, void* workspace, size_t bytes) {
    if (!workspace || bytes < ws_workspace_bytes(p, WS_LAMB)) return WS_ERR_WORKSPACE;
    if (!ws_aligned16(workspace)) return WS_ERR_ALIGNMENT;
    return WS_OK;
}

}  // namespace

extern "C" ws_status ws_lamb_partial(const ws_plan* plan, int32_t r, const ws_grads* grads, const ws_state* state,
                                     const ws_hyper* hyper, void* workspace, size_t workspace_bytes, void* stream) {
    UpdParams P;
    int ok;
    bool gbf;
    ws_status s = prepare(plan, r, grads, state, hyper, nullptr, K_LAMB1, P, ok, gbf);
    if (s != WS_OK) return s;
    if ((s = check_ws(plan, workspace, workspace_bytes)) != WS_OK) return s;
    P.partials = ws_lamb_layout(plan, workspace).partials;
    std::vector<const void*> gp;
    offset_grad_ptrs(plan, r, grads, gp);
    return launch_any(K_LAMB1, gbf, O_NONE, P, gp.data(), (cudaStream_t)stream);
}

extern "C" ws_status ws_lamb_finalize(const ws_plan* plan, void* workspace, size_t workspace_bytes, void* stream) {
    if (!plan) return WS_ERR_INVALID_ARG;
    if (!plan->d_tiles) return WS_ERR_NOT_UPLOADED;
    ws_status s = check_ws(plan, workspace, workspace_bytes);
    if (s != WS_OK) return s;
    WsLambWs L = ws_lamb_layout(plan, workspace);
    lamb_finalize_kernel<<<plan->T, kBlock, 0, (cudaStream_t)stream>>>(plan->d_segtiles, L.partials, plan->ntiles,
                                                                      plan->R, L.rho, L.norms);
    return ws_check_launch("ws_lamb_finalize");
}

extern "C" ws_status ws_lamb_apply(const ws_plan* plan, int32_t r, const ws_state* state, const ws_hyper* hyper,
                                   const ws_out* out, void* workspace, size_t workspace_bytes, void* stream) {
    UpdParams P;
    int ok;
    bool gbf;
    ws_status s = prepare(plan, r, nullptr, state, hyper, out, K_LAMB2, P, ok, gbf);
    if (s != WS_OK) return s;
    if ((s = check_ws(plan, workspace, workspace_bytes)) != WS_OK) return s;
    P.rho = ws_lamb_layout(plan, workspace).rho;
    return launch_any(K_LAMB2, false, ok, P, nullptr, (cudaStream_t)stream);
}

extern "C" ws_status ws_shard_update(const ws_plan* plan, int32_t r, const ws_grads* grads, const ws_state* state,
                                     const ws_hyper* hyper, const ws_out* out, void* workspace,
                                     size_t workspace_bytes, void* stream) {
    if (!hyper) return WS_ERR_INVALID_ARG;
    if (hyper->opt == WS_LAMB) {
        if (r != -1) return WS_ERR_INVALID_ARG;
        ws_status s = ws_lamb_partial(plan, -1, grads, state, hyper, workspace, workspace_bytes, stream);
        if (s != WS_OK) return s;
        if ((s = ws_lamb_finalize(plan, workspace, workspace_bytes, stream)) != WS_OK) return s;
        return ws_lamb_apply(plan, -1, state, hyper, out, workspace, workspace_bytes, stream);
    }
    if (hyper->opt != WS_SGDM && hyper->opt != WS_ADAM) return WS_ERR_INVALID_ARG;
    const int phase = hyper->opt == WS_SGDM ? K_SGDM : K_ADAM;
    UpdParams P;
    int ok;
    bool gbf;
    ws_status s = prepare(plan, r, grads, state, hyper, out, phase, P, ok, gbf);
    if (s != WS_OK) return s;
    std::vector<const void*> gp;
    offset_grad_ptrs(plan, r, grads, gp);
    return launch_any(phase, gbf, ok, P, gp.data(), (cudaStream_t)stream);
}
