// Fused reduce + optimizer update + gathered-layout write.
//
// One kernel does, for every element of a shard (paper Section 2.2): sum the R
// replicas' gradients for that position (the reduce-scatter arithmetic), apply
// the optimizer to the weight and its slots, store them, and store the updated
// weight into slot r of the all-gather layout (fp32, or bf16 rounded from the
// fp32 result, Section 4.2).  Intermediates live in registers only (the
// "fusion" of Section 2.1); every operand crosses HBM exactly once.
//
// Work item = (shard r, tile), one CTA each; a thread owns runs of 4 or 8
// consecutive elements and moves them as 128- or 256-bit vectors.  Pads are
// recognised by location (element index within the tile vs. the tile's valid
// length for shard r), so gradient pads are never read into a result and
// output pads are +0 (Section 4.1, "Non-elementwise operators": mask with the
// identity).
//
// The R-way sum is formed as tree sums over blocks of RB gradients; when R
// exceeds one block the blocks are combined by a compensated (Kahan)
// accumulation, never as one sequential fp32 chain: the loads of a block are
// independent (memory-level parallelism) and the rounding error stays near one
// ulp for R up to 1024.
//
// With FUSED the formatting steps are part of the same kernel (Section 5.1):
// gradients come straight from the replicas' tensor lists and the updated
// weights go straight to the weight tensors.
//
// The k* constants below are the values measured best on a B200.
#include "ws_kernels.cuh"

namespace {
constexpr long long kKeepReverseBytes = 256ll << 20;   // twice the L2: at least half of phase 2's re-reads can hit
using namespace wsk;

// One CTA handles one (shard, tile) work item; the grid is the item count, so the
// hardware CTA scheduler walks the buffers front to back.
template <int OPT, bool GBF, int OUT, int VEC, int U, int RB, int NP, bool FUSED>
__global__ void __launch_bounds__(kBlock, ((VEC == 8 && GBF && !FUSED) || RB > 8) ? kMinBlocksWide : kMinBlocks) update_kernel(const UpdParams P, const __grid_constant__ GradPtrs<NP> gp) {
    constexpr bool READS_G = !is_phase2(OPT);
    constexpr bool NEEDS_WT = FUSED && (OUT != O_NONE);
    __shared__ float2 red[kBlock / 32];
    // fused formatting: this tile's R gradient tensor pointers, fetched once per work item (the
    // streaming data would push the table's lines out of L1 between passes)
    __shared__ const void* sgp[(FUSED && READS_G) ? NP : 1];
    // ... and, when the updated weights go to several weight lists (one per replica: the all-gather
    // of Section 2.2 written straight into every replica's tensors), the tile's further output pointers
    __shared__ void* swp[(FUSED && READS_G && writes_weights(OPT)) ? NP : 1];

    // the next kernel of the stream may start its prologue while this grid's last CTAs run
    asm volatile("griddepcontrol.launch_dependents;");
    constexpr bool HINT = (OPT == K_LAMB1 || OPT == K_LARS1);
    for (long long item0 = blockIdx.x; item0 < P.nitems; item0 += gridDim.x) {
        const long long item = ((OPT == K_LAMB2 || OPT == K_LARS2) && P.reverse) ? P.nitems - 1 - item0 : item0;
        long long rs = P.concat ? 0 : item / P.ntiles;     // shard index inside this launch
        const long long ti = P.concat ? P.tile_lo + item : item - rs * P.ntiles;
        const WsTile tl = P.tiles[ti];
        if (P.concat) rs = tl.shard - P.r0;
        const long long r = P.r0 + rs;
        long long nvl = tl.vt - r * tl.piece;              // valid elements in this tile for shard r
        ItemCtx it;
        it.len = tl.len;
        it.nvalid = nvl < 0 ? 0 : (nvl > tl.len ? tl.len : (int)nvl);
        it.seg = tl.seg;
        it.gbase = rs * P.g_stride + tl.pos;               // into each gradient buffer
        it.sbase = rs * P.st_stride + tl.pos;              // into w/m/v
        it.obase = r * P.S + tl.pos;                       // into the gathered buffer
        it.toff = r * tl.piece + tl.poff;                  // element index inside tensor tl.seg (fused formatting)
        it.partial = P.partials + (P.concat ? ti : r * P.ntiles + ti);
        it.keep = HINT && P.keep;
        char* wt = nullptr;
        if constexpr (FUSED) {
            if (NEEDS_WT) wt = reinterpret_cast<char*>(P.wtab[(long long)tl.seg * P.nw]);
            if constexpr (READS_G) {
                const void* const* gt = P.gtab + (long long)tl.seg * P.R;
                __syncthreads();   // the previous item's readers are done with sgp
                for (int k = threadIdx.x; k < P.R; k += kBlock) sgp[k] = gt[k];
                if constexpr (writes_weights(OPT)) {
                    if (OUT != O_NONE)
                        for (int k = threadIdx.x; k < P.nw; k += kBlock) swp[k] = P.wtab[(long long)tl.seg * P.nw + k];
                }
                __syncthreads();
            }
        }
        // the plan's tables and the tensor-pointer tables do not depend on the previous kernel of the
        // stream; everything read from here on may
        asm volatile("griddepcontrol.wait;" ::: "memory");
        float lr_rho = 0.f;
        if (OPT == K_LAMB2 || OPT == K_LARS2) lr_rho = P.c.lr * P.rho[tl.seg];
        if (OPT == K_AF3) lr_rho = P.rho[tl.seg];         // alpha_t / max(1, RMS(U_t)/d)
        process_item<OPT, GBF, OUT, VEC, U, RB, NP, FUSED, HINT>(P, gp, it, sgp, swp, wt, lr_rho, red);
    }
}

// Sum every shard's per-tile partials of tensor t in a fixed order, in double
// (stands where the paper combines per-replica reduce results with one batched
// scalar all-reduce, Section 4.1 / 5.2), then rho_t = sqrt(a)/sqrt(b).
// With lars != 0 the ratio is the LARS local rate eta sqrt(a) / (sqrt(b) + beta sqrt(a)).
// Sums tensor t's per-tile partials over all shards in a fixed order, in double; the totals
// are valid in thread 0.
__device__ __forceinline__ void sum_partials(const WsSegTiles st, const float2* partials, long long ntiles, int R,
                                             double& a, double& b) {
    __shared__ double sa[kBlock], sb[kBlock];
    const long long n = (long long)R * st.tile_count;
    a = 0.0;
    b = 0.0;
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
    a = sa[0];
    b = sb[0];
}

__global__ void __launch_bounds__(kBlock) lamb_finalize_kernel(const WsSegTiles* segtiles, const float2* partials,
                                                               long long ntiles, int R, float* rho, double* norms,
                                                               int lars, double eta, double beta) {
    // R == 1 with the concatenated layout: a tensor's tiles of all shards are one contiguous run
    const int t = blockIdx.x;
    double a, b;
    const WsSegTiles mine = segtiles[t];
    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    sum_partials(mine, partials, ntiles, R, a, b);
    if (threadIdx.x == 0) {
        norms[2 * t] = a;
        norms[2 * t + 1] = b;
        if (!(a > 0.0 && b > 0.0)) rho[t] = 1.0f;
        else if (lars) rho[t] = (float)(eta * sqrt(a) / (sqrt(b) + beta * sqrt(a)));
        else rho[t] = (float)(sqrt(a) / sqrt(b));
    }
}

// Adafactor, after pass 1, one CTA per chunk of at most 1024 state entries: the moving averages
// Rv' = beta Rv + (1-beta) acc (rows, then columns; the full v' for an unfactored tensor), and the
// sum of the tensor's new row accumulators (double atomic adds into rsum[t], cleared with acc).
__global__ void __launch_bounds__(kBlock) af_moments_kernel(const WsAfChunk* chunks, const WsSegAf* segaf, float* state,
                                                            const float* acc, double* rsum, double beta) {
    __shared__ double srs[kBlock];
    const WsAfChunk ch = chunks[blockIdx.x];
    const WsSegAf a = segaf[ch.seg];
    double rs = 0.0;
    for (int i = threadIdx.x; i < ch.count; i += kBlock) {
        const long long e = ch.begin + i;
        const bool isrow = e < a.nrow;
        const long long k = isrow ? a.irow + e : a.icol + (e - a.nrow);
        const double v = beta * (double)state[a.foff + e] + (1.0 - beta) * (double)acc[k];
        state[a.foff + e] = (float)v;
        if (isrow) rs += v;
    }
    if (ch.begin >= a.nrow) return;     // a chunk of columns only (uniform over the CTA)
    srs[threadIdx.x] = rs;
    __syncthreads();
    for (int s = kBlock / 2; s > 0; s >>= 1) {
        if (threadIdx.x < s) srs[threadIdx.x] += srs[threadIdx.x + s];
        __syncthreads();
    }
    if (threadIdx.x == 0) atomicAdd(&rsum[ch.seg], srs[0]);
}

// ... then the factors the elementwise passes multiply by: sqrt(sum(Rv') / Rv'_i) per row,
// 1/sqrt(Cv'_j) per column (1/sqrt(v'_i) for an unfactored tensor), so that U = g * fr_i * fc_j.
__global__ void __launch_bounds__(kBlock) af_factors_kernel(const WsAfChunk* chunks, const WsSegAf* segaf,
                                                            const float* state, const double* rsum, float* fac) {
    const WsAfChunk ch = chunks[blockIdx.x];
    const WsSegAf a = segaf[ch.seg];
    const double rs = rsum[ch.seg];
    for (int i = threadIdx.x; i < ch.count; i += kBlock) {
        const long long e = ch.begin + i;
        const double v = (double)state[a.foff + e];
        if (e < a.nrow) fac[a.irow + e] = (float)sqrt(rs / v);
        else fac[a.icol + (e - a.nrow)] = (float)(1.0 / sqrt(v));
    }
}

// Adafactor, after pass 2 (one CTA per tensor): the step size alpha_t = max(eps2, RMS(w_t)) *
// rho_step from pass 1's partial sums of w^2, RMS(U_t) from pass 2's partial sums of U^2, and
// the applied step size rho[t] = alpha_t / max(1, RMS(U_t) / d).
__global__ void __launch_bounds__(kBlock) af_finalize_clip_kernel(const WsSegTiles* segtiles, const WsSegAf* segaf,
                                                                  const float2* partials, long long ntiles, int R,
                                                                  float* alpha, float* rho, double* norms, double eps2,
                                                                  double rho_step, double d) {
    const int t = blockIdx.x;
    double sw, su;
    sum_partials(segtiles[t], partials, ntiles, R, sw, su);
    if (threadIdx.x == 0) {
        const long long n = segaf[t].numel;
        const double rms_w = n > 0 ? sqrt(sw / (double)n) : 0.0;
        const double rms_u = n > 0 ? sqrt(su / (double)n) : 0.0;
        const double al = (eps2 > rms_w ? eps2 : rms_w) * rho_step;
        const double clip = rms_u / d > 1.0 ? rms_u / d : 1.0;
        norms[2 * t] = sw;
        norms[2 * t + 1] = su;
        alpha[t] = (float)al;
        rho[t] = (float)(al / clip);
    }
}

// Adafactor pass 2 on its own: sum of U^2 per tile, U = g * fr_i * fc_j, from the stored gradient
// sum and the factors.  It reads 4 bytes per parameter and nothing else, so a CTA that handled
// one tile would spend most of its life waiting for the tile descriptor, then the matrix view,
// then the row factor; here a CTA walks many tiles and fetches the next tile's descriptor and
// matrix view while it works on the current one.
__global__ void __launch_bounds__(kBlock, kAf2Ctas) af_sumsq_kernel(const UpdParams P) {
    long long item = blockIdx.x;
    if (item >= P.nitems) return;
    auto tile_of = [&](long long it, long long& rs) {
        rs = P.concat ? 0 : it / P.ntiles;
        return P.concat ? P.tile_lo + it : it - rs * P.ntiles;
    };
    long long rs, ti = tile_of(item, rs);
    WsTile tl = P.tiles[ti];
    WsSegAf af = P.segaf[tl.seg];
    while (true) {
        const long long nxt = item + gridDim.x;
        const bool more = nxt < P.nitems;
        long long rs_n = 0, ti_n = 0;
        WsTile tn = tl;
        if (more) {
            ti_n = tile_of(nxt, rs_n);
            tn = P.tiles[ti_n];                        // in flight during this tile's work
        }
        if (P.concat) rs = tl.shard - P.r0;
        const long long r = P.r0 + rs;
        const long long nvl = tl.vt - r * tl.piece;
        const int nvalid = nvl < 0 ? 0 : (nvl > tl.len ? tl.len : (int)nvl);
        const float* g = P.ghat + r * P.S + tl.pos;
        const long long toff = r * tl.piece + tl.poff;
        long long row0 = 0, c0 = 0;
        if (af.ncol > 0) {
            if ((((unsigned long long)toff | (unsigned long long)af.ncol) >> 32) == 0) {
                const unsigned q32 = (unsigned)toff / (unsigned)af.ncol;
                row0 = q32;
                c0 = (unsigned)toff - q32 * (unsigned)af.ncol;
            } else {
                row0 = toff / af.ncol;
                c0 = toff - row0 * af.ncol;
            }
        }
        const bool rowsum = af.nrow > 0;
        const float* frp = P.af_fac + af.irow + row0;
        const float* fcp = P.af_fac + af.icol;
        float su = 0.f;
        if (af.ncol % 8 == 0 && af.ncol < (1LL << 30)) {
            // a vector of 8 never straddles rows; rows and columns advance by a fixed step per vector
            const unsigned ncol = (unsigned)af.ncol;
            unsigned col = (unsigned)c0 + 8u * threadIdx.x, rl = 0;
            if (col >= ncol) { rl = col / ncol; col -= rl * ncol; }
            unsigned sub_col = 8 * kBlock, sub_rl = 0;
            if (ncol <= 8 * kBlock) { sub_rl = (8 * kBlock) / ncol; sub_col = 8 * kBlock - sub_rl * ncol; }
            const int nfull = nvalid / 8;
            int q = threadIdx.x;
            // a row length that divides the CTA's stride: the thread's 8 column factors never change
            const bool stationary = sub_col == 0;
            float4 fa = make_float4(0.f, 0.f, 0.f, 0.f), fb = fa;
            if (stationary && q < nfull) {
                fa = __ldg(reinterpret_cast<const float4*>(fcp + col));
                fb = __ldg(reinterpret_cast<const float4*>(fcp + col + 4));
            }
#pragma unroll kAf2Unroll
            for (; q < nfull; q += kBlock) {
                const Fv<8> gv = load_f32<8>(g + 8 * q);
                if (!stationary) {
                    fa = __ldg(reinterpret_cast<const float4*>(fcp + col));
                    fb = __ldg(reinterpret_cast<const float4*>(fcp + col + 4));
                }
                const float fr = rowsum ? __ldg(frp + rl) : 1.f;
                float t = 0.f, x;
                x = gv.f[0] * fa.x; t = fmaf(x, x, t);
                x = gv.f[1] * fa.y; t = fmaf(x, x, t);
                x = gv.f[2] * fa.z; t = fmaf(x, x, t);
                x = gv.f[3] * fa.w; t = fmaf(x, x, t);
                x = gv.f[4] * fb.x; t = fmaf(x, x, t);
                x = gv.f[5] * fb.y; t = fmaf(x, x, t);
                x = gv.f[6] * fb.z; t = fmaf(x, x, t);
                x = gv.f[7] * fb.w; t = fmaf(x, x, t);
                su = fmaf(t, fr * fr, su);
                col += sub_col;
                rl += sub_rl;
                if (col >= ncol) { col -= ncol; ++rl; }
            }
            if (q == nfull && (nvalid & 7)) {          // the one ragged vector of the tile
                const float fr = rowsum ? __ldg(frp + rl) : 1.f;
                for (int j = 0; j < (nvalid & 7); ++j) {
                    const float u = g[8 * q + j] * fr * __ldg(fcp + col + j);
                    su = fmaf(u, u, su);
                }
            }
        } else {
            for (int e = threadIdx.x; e < nvalid; e += kBlock) {
                const long long c = c0 + e;
                const long long rl = c / af.ncol;
                const float fr = rowsum ? __ldg(frp + rl) : 1.f;
                const float u = __ldcs(g + e) * fr * __ldg(fcp + (c - rl * af.ncol));
                su = fmaf(u, u, su);
            }
        }
        WsSegAf an = af;
        if (more) an = P.segaf[tn.seg];                // the next descriptor arrived long ago
        // no CTA-wide barrier at the end of a tile (it would drain the CTA's loads once per tile): every
        // warp adds its own sum to the tile's slot, which pass 1 left at zero
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) su += __shfl_xor_sync(0xffffffffu, su, o);
        if ((threadIdx.x & 31) == 0) atomicAdd(&P.partials[P.concat ? ti : r * P.ntiles + ti].y, su);
        if (!more) break;
        item = nxt; rs = rs_n; ti = ti_n; tl = tn; af = an;
    }
}

// -------------------------------------------------------------- dispatch ---
void launch_lamb_finalize(int T, cudaStream_t st, const WsSegTiles* segtiles, const float2* partials, long long ntiles,
                          int R, float* rho, double* norms, int lars, double eta, double beta) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)T);
    cfg.blockDim = dim3(kBlock);
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, lamb_finalize_kernel, segtiles, partials, ntiles, R, rho, norms, lars, eta, beta);
}

template <int OPT, bool GBF, int OUT, int VEC, int U, int RB, int NP, bool FUSED>
ws_status launch(const UpdParams& P, const void* const* gptrs, cudaStream_t st) {
    GradPtrs<NP> gp;
    for (int k = 0; k < NP; ++k) gp.p[k] = (!FUSED && gptrs && k < P.R) ? gptrs[k] : nullptr;
    long long grid = P.nitems;
    if (grid < 1) return WS_OK;
    if (grid > 0x7fffffffLL) grid = 0x7fffffffLL;
    // programmatic dependent launch: the kernel may start while the previous kernel of the stream drains
    // (it reads only the plan and pointer tables before it waits for that kernel)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kBlock);
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, update_kernel<OPT, GBF, OUT, VEC, U, RB, NP, FUSED>, P, gp);
    return ws_check_launch(FUSED ? "ws_fused_update" : "ws_shard_update");
}

// Wide (256-bit) accesses need 32-byte aligned buffers; they pay off when the
// gradients are bf16 (a 128-bit gradient load then covers 8 elements) and for
// small R, where the fp32 streams dominate.
template <int OPT, bool GBF, int OUT, bool FUSED>
ws_status launch_r(const UpdParams& P, const void* const* gptrs, bool wide_ok, cudaStream_t st) {
    if constexpr (is_phase2(OPT)) {
        if (wide_ok) return launch<OPT, GBF, OUT, 8, 1, 1, 1, FUSED>(P, gptrs, st);
        return launch<OPT, GBF, OUT, 4, 1, 1, 1, FUSED>(P, gptrs, st);
    } else {
        if (P.R <= 2) {
            if constexpr (OPT != K_AF1) if (wide_ok) return launch<OPT, GBF, OUT, 8, 1, 2, 2, FUSED>(P, gptrs, st);
            return launch<OPT, GBF, OUT, 4, OPT == K_AF1 ? kUAf2 : 1, 2, 2, FUSED>(P, gptrs, st);
        }
        if (P.R <= 4) {
            if constexpr (GBF && OPT != K_AF1) if (wide_ok) return launch<OPT, GBF, OUT, 8, 1, 4, 4, FUSED>(P, gptrs, st);
            return launch<OPT, GBF, OUT, 4, OPT == K_AF1 ? kUAf4 : 1, 4, 4, FUSED>(P, gptrs, st);
        }
        if (P.R <= 8) {
            if constexpr (GBF && OPT != K_AF1) if (wide_ok) return launch<OPT, GBF, OUT, 8, 1, 8, 8, FUSED>(P, gptrs, st);
            return launch<OPT, GBF, OUT, 4, OPT == K_AF1 ? kUAf8 : 1, 8, 8, FUSED>(P, gptrs, st);
        }
        if (P.R <= 32) {
            if constexpr (GBF && OPT != K_AF1) if (wide_ok) return launch<OPT, GBF, OUT, 8, 1, 8, 32, FUSED>(P, gptrs, st);
            return launch<OPT, GBF, OUT, 4, 1, 8, 32, FUSED>(P, gptrs, st);
        }
        // many replicas make small shards and few CTAs: more loads in flight per thread
        if (P.R <= 1024) return launch<OPT, GBF, OUT, 4, 1, kTreeBlockLarge, 1024, FUSED>(P, gptrs, st);
        return WS_ERR_TOO_LARGE;
    }
}

bool aligned32(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 31u) == 0; }

// `wide` on entry: whether the caller-side tensors (fused formatting) allow 256-bit accesses.
template <int OPT, bool GBF, bool FUSED>
ws_status launch_o(const UpdParams& P, const void* const* gptrs, int out, bool wide, cudaStream_t st) {
    wide = wide && aligned32(P.w) && aligned32(P.m) && aligned32(P.v) && aligned32(P.gathered);
    if (!FUSED && !is_phase2(OPT))
        for (int k = 0; k < P.R && wide; ++k) wide = aligned32(gptrs[k]);
    if (OPT == K_LARS1 || OPT == K_LARS2 || is_af(OPT)) wide = wide && aligned32(P.ghat);
    if (OPT == K_AF1) wide = false;   // pass 1 is instruction-heavy: 128-bit vectors measured faster at every R
    if constexpr (is_phase1(OPT)) {
        if constexpr (FUSED) if (out == O_F32M) return launch_r<OPT, GBF, O_F32M, FUSED>(P, gptrs, wide, st);
        return launch_r<OPT, GBF, O_NONE, FUSED>(P, gptrs, wide, st);
    } else {
        switch (out) {
            case O_NONE:
                if constexpr (FUSED) return WS_ERR_INVALID_ARG;
                else return launch_r<OPT, GBF, O_NONE, FUSED>(P, gptrs, wide, st);
            case O_F32: return launch_r<OPT, GBF, O_F32, FUSED>(P, gptrs, wide, st);
            case O_F32M:
                if constexpr (FUSED) return launch_r<OPT, GBF, O_F32M, FUSED>(P, gptrs, wide, st);
                else return WS_ERR_INVALID_ARG;
            default: return launch_r<OPT, GBF, O_BF16, FUSED>(P, gptrs, wide, st);
        }
    }
}

template <bool FUSED>
ws_status launch_f(int opt, bool gbf, int out, const UpdParams& P, const void* const* gptrs, bool wide, cudaStream_t st) {
    switch (opt) {
        case K_SGDM: return gbf ? launch_o<K_SGDM, true, FUSED>(P, gptrs, out, wide, st) : launch_o<K_SGDM, false, FUSED>(P, gptrs, out, wide, st);
        case K_ADAM: return gbf ? launch_o<K_ADAM, true, FUSED>(P, gptrs, out, wide, st) : launch_o<K_ADAM, false, FUSED>(P, gptrs, out, wide, st);
        case K_LAMB1: return gbf ? launch_o<K_LAMB1, true, FUSED>(P, gptrs, out, wide, st) : launch_o<K_LAMB1, false, FUSED>(P, gptrs, out, wide, st);
        case K_LARS1: return gbf ? launch_o<K_LARS1, true, FUSED>(P, gptrs, out, wide, st) : launch_o<K_LARS1, false, FUSED>(P, gptrs, out, wide, st);
        case K_LARS2: return launch_o<K_LARS2, false, FUSED>(P, gptrs, out, wide, st);
        case K_AF1: return gbf ? launch_o<K_AF1, true, FUSED>(P, gptrs, out, wide, st) : launch_o<K_AF1, false, FUSED>(P, gptrs, out, wide, st);
        case K_AF3: return launch_o<K_AF3, false, FUSED>(P, gptrs, out, wide, st);
        default: return launch_o<K_LAMB2, false, FUSED>(P, gptrs, out, wide, st);
    }
}

ws_status launch_any(int opt, bool gbf, int out, const UpdParams& P, const void* const* gptrs, cudaStream_t st) {
    return launch_f<false>(opt, gbf, out, P, gptrs, true, st);
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
                  const ws_out* out, int phase, UpdParams& P, int& out_kind, bool& gbf, bool fused = false) {
    if (!p || !s || !h) return WS_ERR_INVALID_ARG;
    if (!p->d_tiles) return WS_ERR_NOT_UPLOADED;
    if (r < -1 || r >= p->R) return WS_ERR_INVALID_ARG;
    if (h->step < 1) return WS_ERR_INVALID_ARG;
    const bool needs_v = (phase == K_ADAM || phase == K_LAMB1 || phase == K_LAMB2);
    const bool needs_m = !is_af(phase);
    // (fused formatting with fp32 weight tensors: the tensors may be the master copy, then w is null)
    if ((!s->w && !fused) || (needs_m && !s->m) || (needs_v && !s->v)) return WS_ERR_INVALID_ARG;
    if (!ws_aligned16(s->w) || (needs_m && !ws_aligned16(s->m)) || (needs_v && !ws_aligned16(s->v))) return WS_ERR_ALIGNMENT;
    gbf = false;
    P.gtab = nullptr;
    P.wtab = nullptr;
    P.nw = 1;
    // Norm pairs on all shards of a model small enough that a good part of what phase 2 reads again fits
    // the L2: phase 1 leaves those lines in L2 (its gradient loads are evict-first) and phase 2 walks the
    // items back to front, starting where phase 1 ended.  ResNet-50 set under LARS, 8 copies: 0.249 ms ->
    // 0.241 ms; on models many times the L2 it costs 1 - 2 %, hence the limit.
    {
        const bool pair = phase == K_LAMB1 || phase == K_LAMB2 || phase == K_LARS1 || phase == K_LARS2;
        const long long again = (phase == K_LAMB1 || phase == K_LAMB2) ? 12 : 8;     // bytes per parameter read twice
        const int on = (pair && r == -1 && p->N * again <= kKeepReverseBytes) ? 1 : 0;
        P.keep = on;
        P.reverse = on;
    }
    if (!is_phase2(phase) && !fused) {
        if (!g || !g->ptrs || g->R < 1) return WS_ERR_INVALID_ARG;
        if (g->dtype != WS_F32 && g->dtype != WS_BF16) return WS_ERR_DTYPE;
        if (g->slice_mode != 0 && g->slice_mode != 1) return WS_ERR_INVALID_ARG;
        // g->R need not equal the plan's shard count: with partial sharding (Section 5.2) the
        // replicas form groups that each shard M ways, and shard j sums all groups' copies
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
    P.concat = (p->layout == WS_LAYOUT_CONCAT);
    P.tile_lo = 0;
    if (P.concat) {
        P.tile_lo = (r < 0) ? 0 : p->shard_tile_begin[r];
        P.nitems = (r < 0) ? p->ntiles : p->shard_tile_begin[r + 1] - p->shard_tile_begin[r];
    }
    P.st_stride = (r < 0) ? p->S : 0;
    if (g && !is_phase2(phase) && !fused) {
        // slice mode 0: pointer is the packed buffer; the launch starts at shard r0
        P.g_stride = (g->slice_mode == 0) ? p->S : 0;
    } else {
        P.g_stride = 0;
    }
    P.w = (float*)s->w;
    P.m = needs_m ? (float*)s->m : nullptr;
    P.v = needs_v ? (float*)s->v : nullptr;
    P.segaf = p->d_segaf;
    P.af_acc = nullptr;
    P.af_fac = nullptr;
    P.gathered = (out_kind != O_NONE) ? out->gathered : nullptr;
    P.partials = nullptr;
    P.rho = nullptr;
    P.ghat = nullptr;
    P.c = make_consts(h);
#ifdef WS_DEBUG_BOUNDS
    P.bounds = ws_bounds_word();
    P.state_elems = (long long)nshards * p->S;
    // (one shard of a packed buffer: the pointers are advanced to the shard, S elements remain in view)
    P.grad_elems = (g && g->slice_mode == 0 && r < 0) ? (long long)p->R * p->S : p->S;
    P.out_elems = (long long)p->R * p->S;
#endif
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

// How many strided repetitions of a tensor's tile run the finalize step sums: R (one run per
// shard, ntiles apart) for the per-tensor layout, 1 for the concatenated layout.
int finalize_reps(const ws_plan* p) { return p->layout == WS_LAYOUT_CONCAT ? 1 : p->R; }

ws_status check_ws(const ws_plan* p, void* workspace, size_t bytes, ws_opt opt = WS_LAMB) {
    if (!workspace || bytes < ws_workspace_bytes(p, opt)) return WS_ERR_WORKSPACE;
    if (!ws_aligned16(workspace)) return WS_ERR_ALIGNMENT;
    return WS_OK;
}

}  // namespace

extern "C" ws_status ws_lamb_partial(const ws_plan* plan, int32_t r, const ws_grads* grads, const ws_state* state,
                                     const ws_hyper* hyper, void* workspace, size_t workspace_bytes, void* stream) {
    WsRange range_("ws_lamb_partial");
    if (!hyper || hyper->opt != WS_LAMB) return WS_ERR_INVALID_ARG;
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
    WsRange range_("ws_lamb_finalize");
    if (!plan) return WS_ERR_INVALID_ARG;
    if (!plan->d_tiles) return WS_ERR_NOT_UPLOADED;
    ws_status s = check_ws(plan, workspace, workspace_bytes);
    if (s != WS_OK) return s;
    WsLambWs L = ws_lamb_layout(plan, workspace);
    launch_lamb_finalize(plan->T, (cudaStream_t)stream, plan->d_segtiles, L.partials, plan->ntiles,
                                                                      finalize_reps(plan), L.rho, L.norms, 0, 0.0, 0.0);
    return ws_check_launch("ws_lamb_finalize");
}

extern "C" ws_status ws_lamb_apply(const ws_plan* plan, int32_t r, const ws_state* state, const ws_hyper* hyper,
                                   const ws_out* out, void* workspace, size_t workspace_bytes, void* stream) {
    WsRange range_("ws_lamb_apply");
    if (!hyper || hyper->opt != WS_LAMB) return WS_ERR_INVALID_ARG;
    UpdParams P;
    int ok;
    bool gbf;
    ws_status s = prepare(plan, r, nullptr, state, hyper, out, K_LAMB2, P, ok, gbf);
    if (s != WS_OK) return s;
    if ((s = check_ws(plan, workspace, workspace_bytes)) != WS_OK) return s;
    P.rho = ws_lamb_layout(plan, workspace).rho;
    return launch_any(K_LAMB2, false, ok, P, nullptr, (cudaStream_t)stream);
}

extern "C" ws_status ws_lars_partial(const ws_plan* plan, int32_t r, const ws_grads* grads, const ws_state* state,
                                     const ws_hyper* hyper, void* workspace, size_t workspace_bytes, void* stream) {
    WsRange range_("ws_lars_partial");
    if (!hyper || hyper->opt != WS_LARS) return WS_ERR_INVALID_ARG;
    UpdParams P;
    int ok;
    bool gbf;
    ws_status s = prepare(plan, r, grads, state, hyper, nullptr, K_LARS1, P, ok, gbf);
    if (s != WS_OK) return s;
    if ((s = check_ws(plan, workspace, workspace_bytes, WS_LARS)) != WS_OK) return s;
    const WsLambWs L = ws_lamb_layout(plan, workspace);
    P.partials = L.partials;
    P.ghat = L.ghat;
    std::vector<const void*> gp;
    offset_grad_ptrs(plan, r, grads, gp);
    return launch_any(K_LARS1, gbf, O_NONE, P, gp.data(), (cudaStream_t)stream);
}

extern "C" ws_status ws_lars_finalize(const ws_plan* plan, const ws_hyper* hyper, void* workspace,
                                      size_t workspace_bytes, void* stream) {
    WsRange range_("ws_lars_finalize");
    if (!plan || !hyper || hyper->opt != WS_LARS) return WS_ERR_INVALID_ARG;
    if (!plan->d_tiles) return WS_ERR_NOT_UPLOADED;
    ws_status s = check_ws(plan, workspace, workspace_bytes, WS_LARS);
    if (s != WS_OK) return s;
    const WsLambWs L = ws_lamb_layout(plan, workspace);
    launch_lamb_finalize(plan->T, (cudaStream_t)stream, plan->d_segtiles, L.partials, plan->ntiles,
                                                                      finalize_reps(plan), L.rho, L.norms, 1,
                                                                      hyper->trust_coeff, hyper->weight_decay);
    return ws_check_launch("ws_lars_finalize");
}

extern "C" ws_status ws_lars_apply(const ws_plan* plan, int32_t r, const ws_state* state, const ws_hyper* hyper,
                                   const ws_out* out, void* workspace, size_t workspace_bytes, void* stream) {
    WsRange range_("ws_lars_apply");
    if (!hyper || hyper->opt != WS_LARS) return WS_ERR_INVALID_ARG;
    UpdParams P;
    int ok;
    bool gbf;
    ws_status s = prepare(plan, r, nullptr, state, hyper, out, K_LARS2, P, ok, gbf);
    if (s != WS_OK) return s;
    if ((s = check_ws(plan, workspace, workspace_bytes, WS_LARS)) != WS_OK) return s;
    const WsLambWs L = ws_lamb_layout(plan, workspace);
    P.rho = L.rho;
    P.ghat = L.ghat;
    return launch_any(K_LARS2, false, ok, P, nullptr, (cudaStream_t)stream);
}

namespace {
ws_status af_update(const ws_plan* plan, int32_t r, const ws_grads* grads, const ws_tensor_table* gtab,
                    const ws_state* state, const ws_hyper* hyper, const ws_out* out, const ws_tensor_table* wtab,
                    void* workspace, size_t workspace_bytes, cudaStream_t st);

// LAMB (pair 0) or LARS (pair 1) for all shards as one kernel, when the plan's one-launch
// schedule is on the device and the number of gradient copies is supported; `done` says whether the
// update was enqueued here (false: the caller runs the separate launches).  Either the packed-buffer
// arguments (grads, out) or the tensor tables (gtab, wtab) are given.
ws_status try_one_launch(const ws_plan* plan, int pair, const ws_grads* grads, const ws_tensor_table* gtab,
                         const ws_state* state, const ws_hyper* hyper, const ws_out* out, const ws_tensor_table* wtab,
                         void* workspace, size_t workspace_bytes, cudaStream_t st, bool& done) {
    done = false;
    if (!plan || !plan->d_sched) return WS_OK;
    const bool fused = gtab != nullptr;
    const int copies = fused ? gtab->nsets : (grads ? grads->R : 0);
    if (!one_launch_supports(pair, copies)) return WS_OK;
    UpdParams P;
    int out_kind;
    bool gbf;
    ws_status s = prepare(plan, -1, grads, state, hyper, fused ? nullptr : out, pair == 0 ? K_LAMB1 : K_LARS1, P, out_kind,
                          gbf, fused);
    if (s != WS_OK) return s;
    if (pair == 0 && (!state->v || !ws_aligned16(state->v))) return state->v ? WS_ERR_ALIGNMENT : WS_ERR_INVALID_ARG;
    if ((s = check_ws(plan, workspace, workspace_bytes, pair == 0 ? WS_LAMB : WS_LARS)) != WS_OK) return s;
    const WsLambWs L = ws_lamb_layout(plan, workspace);
    bool wide = aligned32(P.w) && aligned32(P.m) && aligned32(P.v) && aligned32(P.gathered);
    std::vector<const void*> gp;
    if (fused) {
        const bool master = state->w == nullptr;
        if (master && (wtab->dtype != WS_F32 || wtab->nsets != 1)) return WS_ERR_INVALID_ARG;
        if (wtab->nsets != 1) return WS_ERR_INVALID_ARG;
        P.gtab = (const void* const*)gtab->dev;
        P.R = gtab->nsets;
        gbf = gtab->dtype == WS_BF16;
        P.wtab = (void* const*)wtab->dev;
        P.nw = 1;
        out_kind = master ? O_F32M : (wtab->dtype == WS_F32 ? O_F32 : O_BF16);
        wide = wide && (gbf || gtab->min_align >= 32) && (wtab->dtype == WS_BF16 || wtab->min_align >= 32);
    } else {
        offset_grad_ptrs(plan, -1, grads, gp);
        for (int k = 0; k < grads->R && wide; ++k) wide = aligned32(gp[k]);
    }
    if (pair == 1) {
        P.ghat = L.ghat;
        wide = wide && aligned32(P.ghat);
    }
    OneLaunch Q;
    Q.sched = plan->d_sched;
    Q.nsched = (unsigned)(2 * plan->n_items);
    Q.items = plan->d_items;
    Q.segs = plan->d_itemsegs;
    Q.T = plan->T;
    Q.ipart = L.ipart;
    Q.count = L.count;
    Q.flag = L.flag;
    Q.ticket = L.ticket;
    Q.status = L.status;
    Q.rho = L.rho;
    Q.norms = L.norms;
    Q.eta = hyper->trust_coeff;
    Q.beta = hyper->weight_decay;
    cudaError_t e = cudaMemsetAsync(L.count, 0, L.sync_bytes, st);     // counters, ready words, ticket, status
    if (e != cudaSuccess) return ws_cuda_fail(e, "one-launch update (clear counters)");
    s = launch_one_launch(pair, gbf, out_kind, fused, wide, P, fused ? nullptr : gp.data(), Q, st);
    if (s == WS_OK) done = true;
    return s;
}

// The argument checks of the apply phase (state pointers, `out` dtype and alignment), with no launch.
ws_status check_phase2_args(const ws_plan* plan, const ws_state* state, const ws_hyper* hyper, const ws_out* out,
                            int phase) {
    UpdParams P;
    int ok;
    bool gbf;
    return prepare(plan, -1, nullptr, state, hyper, out, phase, P, ok, gbf);
}
}

ws_status ws_lamb_check_apply_args(const ws_plan* plan, const ws_state* state, const ws_hyper* hyper, const ws_out* out) {
    return check_phase2_args(plan, state, hyper, out, K_LAMB2);
}

extern "C" ws_status ws_shard_update(const ws_plan* plan, int32_t r, const ws_grads* grads, const ws_state* state,
                                     const ws_hyper* hyper, const ws_out* out, void* workspace,
                                     size_t workspace_bytes, void* stream) {
    WsRange range_("ws_shard_update");
    if (!hyper) return WS_ERR_INVALID_ARG;
    if (hyper->opt == WS_ADAFACTOR)
        return af_update(plan, r, grads, nullptr, state, hyper, out, nullptr, workspace, workspace_bytes, (cudaStream_t)stream);
    if (hyper->opt == WS_LAMB) {
        if (r != -1) return WS_ERR_INVALID_ARG;
        // every phase's arguments are checked before the first launch: an error must not leave the
        // moments advanced and the weights not
        ws_status s = check_phase2_args(plan, state, hyper, out, K_LAMB2);
        if (s != WS_OK) return s;
        bool done = false;
        s = try_one_launch(plan, 0, grads, nullptr, state, hyper, out, nullptr, workspace, workspace_bytes, (cudaStream_t)stream, done);
        if (s != WS_OK || done) return s;
        if ((s = ws_lamb_partial(plan, -1, grads, state, hyper, workspace, workspace_bytes, stream)) != WS_OK) return s;
        if ((s = ws_lamb_finalize(plan, workspace, workspace_bytes, stream)) != WS_OK) return s;
        return ws_lamb_apply(plan, -1, state, hyper, out, workspace, workspace_bytes, stream);
    }
    if (hyper->opt == WS_LARS) {
        // LARS (the optimizer of the paper's ResNet-50 runs, Table 1): phase 1 reduces the gradients,
        // keeps the sum in the workspace and leaves partial sums of ||w||^2 and ||g||^2; the finalize
        // step forms each tensor's local rate; phase 2 applies the momentum step.
        if (r != -1) return WS_ERR_INVALID_ARG;
        ws_status s = check_phase2_args(plan, state, hyper, out, K_LARS2);
        if (s != WS_OK) return s;
        bool done = false;
        s = try_one_launch(plan, 1, grads, nullptr, state, hyper, out, nullptr, workspace, workspace_bytes, (cudaStream_t)stream, done);
        if (s != WS_OK || done) return s;
        if ((s = ws_lars_partial(plan, -1, grads, state, hyper, workspace, workspace_bytes, stream)) != WS_OK) return s;
        if ((s = ws_lars_finalize(plan, hyper, workspace, workspace_bytes, stream)) != WS_OK) return s;
        return ws_lars_apply(plan, -1, state, hyper, out, workspace, workspace_bytes, stream);
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

// ------------------------------------------------ fused formatting path ---

extern "C" size_t ws_tensor_table_bytes(const ws_plan* plan, int32_t nsets) {
    if (!plan || nsets < 1) return 0;
    return ((size_t)plan->T * (size_t)nsets * sizeof(void*) + 15) & ~(size_t)15;
}

extern "C" ws_status ws_tensor_table_upload(const ws_plan* plan, const void* const* ptrs, int32_t nsets, ws_dtype dtype,
                                            void* dev_buf, size_t bytes, void* stream, ws_tensor_table* out) {
    if (!plan || !ptrs || !dev_buf || !out || nsets < 1 || nsets > 1024) return WS_ERR_INVALID_ARG;
    if (dtype != WS_F32 && dtype != WS_BF16) return WS_ERR_DTYPE;
    if (!ws_aligned16(dev_buf)) return WS_ERR_ALIGNMENT;
    if (bytes < ws_tensor_table_bytes(plan, nsets)) return WS_ERR_WORKSPACE;
    const int T = plan->T;
    std::vector<const void*> host((size_t)T * nsets);
    int min_align = 256;
    for (int k = 0; k < nsets; ++k)
        for (int t = 0; t < T; ++t) {
            const void* q = ptrs[(size_t)k * T + t];
            host[(size_t)t * nsets + k] = q;   // device layout [T][nsets]: a tile finds its pointers side by side
            if (plan->segs[t].numel == 0) continue;   // empty tensor: never dereferenced, may be null
            if (!q) return WS_ERR_INVALID_ARG;
            if (!ws_aligned16(q)) return WS_ERR_ALIGNMENT;
            while (min_align > 16 && (reinterpret_cast<uintptr_t>(q) & (uintptr_t)(min_align - 1)) != 0) min_align >>= 1;
        }
    cudaError_t e = cudaMemcpyAsync(dev_buf, host.data(), host.size() * sizeof(void*), cudaMemcpyHostToDevice,
                                    (cudaStream_t)stream);
    if (e != cudaSuccess) return ws_cuda_fail(e, "ws_tensor_table_upload");
    // the host vector is pageable: the runtime has staged it before cudaMemcpyAsync returns
    out->dev = dev_buf;
    out->nsets = nsets;
    out->T = T;
    out->dtype = dtype;
    out->min_align = min_align;
    return WS_OK;
}

namespace {

ws_status fused_phase(const ws_plan* plan, int32_t r, const ws_tensor_table* grads, const ws_state* state,
                      const ws_hyper* hyper, const ws_tensor_table* weights, int phase, void* workspace,
                      cudaStream_t st) {
    UpdParams P;
    int ok;
    bool gbf;
    ws_status s = prepare(plan, r, nullptr, state, hyper, nullptr, phase, P, ok, gbf, true);
    if (s != WS_OK) return s;
    bool wide = true;
    int out_kind = O_NONE;
    // no sharded copy of w: the fp32 weight tensors are the master, read and written in place
    const bool master = state->w == nullptr;
    if (master && (weights->dtype != WS_F32 || weights->nsets != 1)) return WS_ERR_INVALID_ARG;
    if (!is_phase2(phase)) {
        P.gtab = (const void* const*)grads->dev;
        P.R = grads->nsets;
        gbf = grads->dtype == WS_BF16;
        wide = wide && (gbf || grads->min_align >= 32);
    }
    if (!is_phase1(phase) || master) {
        P.wtab = (void* const*)weights->dev;
        P.nw = weights->nsets;
        out_kind = master ? O_F32M : (weights->dtype == WS_F32 ? O_F32 : O_BF16);
        wide = wide && (weights->dtype == WS_BF16 || weights->min_align >= 32);
    }
    if (is_phase1(phase) || is_phase2(phase)) {
        WsLambWs L = ws_lamb_layout(plan, workspace);
        P.partials = L.partials;
        P.rho = L.rho;
        P.ghat = L.ghat;
        if (is_af(phase)) {
            P.af_acc = L.acc;
            P.af_fac = L.fac;
        }
    }
    return launch_f<true>(phase, gbf, out_kind, P, nullptr, wide, st);
}

// Adafactor, all shards: zero the row / column sums, pass 1 (reduce, keep the sum, partial row and
// column sums), moments + step size, pass 2 (sum U^2), clipping, pass 3 (apply).  Either the
// packed-buffer arguments (grads, out) or the tensor tables (gtab, wtab) are given.
// One stage of Adafactor for shard r (or all shards with r == -1); see ws_adafactor_stage in ws.h.
// Either the packed-buffer arguments (grads, out) or the tensor tables (gtab, wtab) are given.
ws_status af_stage(const ws_plan* plan, int stage, int32_t r, const ws_grads* grads, const ws_tensor_table* gtab,
                   const ws_state* state, const ws_hyper* hyper, const ws_out* out, const ws_tensor_table* wtab,
                   void* workspace, size_t workspace_bytes, cudaStream_t st) {
    if (!plan || !hyper) return WS_ERR_INVALID_ARG;
    if (!plan->d_tiles) return WS_ERR_NOT_UPLOADED;
    if (r < -1 || r >= plan->R) return WS_ERR_INVALID_ARG;
    if (hyper->opt != WS_ADAFACTOR || hyper->weight_decay != 0.0 || !(hyper->clip_threshold > 0.0) ||
        !(hyper->decay_exponent > 0.0) || !(hyper->eps >= 0.0) || !(hyper->eps2 >= 0.0) || hyper->step < 1)
        return WS_ERR_INVALID_ARG;
    ws_status s = check_ws(plan, workspace, workspace_bytes, WS_ADAFACTOR);
    if (s != WS_OK) return s;
    // pass 2 reads the stored gradient sum (256 bytes into the workspace and onwards) with 256-bit loads
    if (!aligned32(workspace)) return WS_ERR_ALIGNMENT;
    const WsLambWs L = ws_lamb_layout(plan, workspace);
    const bool fused = gtab != nullptr;
    UpdParams P;
    int ok;
    bool gbf;
    switch (stage) {
        case WS_AF_BEGIN: {
            cudaError_t e = cudaMemsetAsync(L.acc, 0, L.acc_bytes, st);
            return e == cudaSuccess ? WS_OK : ws_cuda_fail(e, "adafactor(clear sums)");
        }
        case WS_AF_SUMS: {
            if (fused) return fused_phase(plan, r, gtab, state, hyper, wtab, K_AF1, workspace, st);
            if ((s = prepare(plan, r, grads, state, hyper, nullptr, K_AF1, P, ok, gbf)) != WS_OK) return s;
            P.partials = L.partials;
            P.ghat = L.ghat;
            P.af_acc = L.acc;
            std::vector<const void*> gp;
            offset_grad_ptrs(plan, r, grads, gp);
            return launch_any(K_AF1, gbf, O_NONE, P, gp.data(), st);
        }
        case WS_AF_MOMENTS: {
            if (!state || !state->v) return WS_ERR_INVALID_ARG;
            if (!ws_aligned16(state->v)) return WS_ERR_ALIGNMENT;
            const double beta = 1.0 - pow((double)hyper->step, -hyper->decay_exponent);
            const unsigned nchunks = (unsigned)plan->afchunks.size();
            if (nchunks == 0) return WS_OK;
            af_moments_kernel<<<nchunks, kBlock, 0, st>>>(plan->d_afchunks, plan->d_segaf, (float*)state->v, L.acc, L.rsum, beta);
            if ((s = ws_check_launch("adafactor(moments)")) != WS_OK) return s;
            af_factors_kernel<<<nchunks, kBlock, 0, st>>>(plan->d_afchunks, plan->d_segaf, (const float*)state->v, L.rsum, L.fac);
            return ws_check_launch("adafactor(factors)");
        }
        case WS_AF_SUMSQ: {
            // (the pass reads only the workspace; `state` is not touched, w stands in for the argument checks)
            ws_state dummy = {workspace, nullptr, nullptr};
            if ((s = prepare(plan, r, nullptr, &dummy, hyper, nullptr, K_AF2, P, ok, gbf)) != WS_OK) return s;
            P.partials = L.partials;
            P.ghat = L.ghat;
            P.af_fac = L.fac;
            if (P.nitems < 1) return WS_OK;
            int dev = 0, sms = 148;
            cudaGetDevice(&dev);
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
            const long long cap = (long long)sms * kAf2Ctas;
            af_sumsq_kernel<<<(unsigned)(P.nitems < cap ? P.nitems : cap), kBlock, 0, st>>>(P);
            return ws_check_launch("adafactor(pass 2)");
        }
        case WS_AF_CLIP: {
            const double inv_sqrt_t = 1.0 / sqrt((double)hyper->step);
            const double rho_step = hyper->lr < inv_sqrt_t ? hyper->lr : inv_sqrt_t;
            af_finalize_clip_kernel<<<plan->T, kBlock, 0, st>>>(plan->d_segtiles, plan->d_segaf, L.partials, plan->ntiles,
                                                               finalize_reps(plan), L.alpha, L.rho, L.norms, hyper->eps2,
                                                               rho_step, hyper->clip_threshold);
            return ws_check_launch("adafactor(clipping)");
        }
        case WS_AF_APPLY: {
            if (fused) return fused_phase(plan, r, gtab, state, hyper, wtab, K_AF3, workspace, st);
            if ((s = prepare(plan, r, nullptr, state, hyper, out, K_AF3, P, ok, gbf)) != WS_OK) return s;
            P.rho = L.rho;
            P.ghat = L.ghat;
            P.af_fac = L.fac;
            return launch_any(K_AF3, false, ok, P, nullptr, st);
        }
        default: return WS_ERR_INVALID_ARG;
    }
}

// Adafactor, all shards: the six stages in order.
ws_status af_update(const ws_plan* plan, int32_t r, const ws_grads* grads, const ws_tensor_table* gtab,
                    const ws_state* state, const ws_hyper* hyper, const ws_out* out, const ws_tensor_table* wtab,
                    void* workspace, size_t workspace_bytes, cudaStream_t st) {
    if (r != -1 || !state) return WS_ERR_INVALID_ARG;
    for (int stage = WS_AF_BEGIN; stage <= WS_AF_APPLY; ++stage) {
        const ws_status s = af_stage(plan, stage, -1, grads, gtab, state, hyper, out, wtab, workspace, workspace_bytes, st);
        if (s != WS_OK) return s;
    }
    return WS_OK;
}

}  // namespace

extern "C" ws_status ws_adafactor_stage(const ws_plan* plan, ws_af_stage stage, int32_t r, const ws_grads* grads,
                                        const ws_state* state, const ws_hyper* hyper, const ws_out* out,
                                        void* workspace, size_t workspace_bytes, void* stream) {
    WsRange range_("ws_adafactor_stage");
    return af_stage(plan, (int)stage, r, grads, nullptr, state, hyper, out, nullptr, workspace, workspace_bytes,
                    (cudaStream_t)stream);
}

extern "C" ws_status ws_fused_update(const ws_plan* plan, int32_t r, const ws_tensor_table* grads, const ws_state* state,
                                     const ws_hyper* hyper, const ws_tensor_table* weights, void* workspace,
                                     size_t workspace_bytes, void* stream) {
    WsRange range_("ws_fused_update");
    if (!plan || !grads || !weights || !hyper || !state) return WS_ERR_INVALID_ARG;
    if (!grads->dev || !weights->dev) return WS_ERR_INVALID_ARG;
    if (grads->T != plan->T || weights->T != plan->T || grads->nsets < 1 || weights->nsets < 1) return WS_ERR_INVALID_ARG;
    // several weight lists (every replica's tensors written by the one kernel) only where one kernel both
    // reads the gradient lists and writes the weights, and never more lists than gradient sets
    if (weights->nsets > 1 && ((hyper->opt != WS_SGDM && hyper->opt != WS_ADAM) || weights->nsets > grads->nsets))
        return WS_ERR_INVALID_ARG;
    if ((grads->dtype != WS_F32 && grads->dtype != WS_BF16) || (weights->dtype != WS_F32 && weights->dtype != WS_BF16))
        return WS_ERR_DTYPE;
    cudaStream_t st = (cudaStream_t)stream;
    if (hyper->opt == WS_ADAFACTOR)
        return af_update(plan, r, nullptr, grads, state, hyper, nullptr, weights, workspace, workspace_bytes, st);
    if (hyper->opt == WS_LAMB) {
        if (r != -1) return WS_ERR_INVALID_ARG;
        ws_status s = check_ws(plan, workspace, workspace_bytes);
        if (s != WS_OK) return s;
        bool done = false;
        s = try_one_launch(plan, 0, nullptr, grads, state, hyper, nullptr, weights, workspace, workspace_bytes, st, done);
        if (s != WS_OK || done) return s;
        if ((s = fused_phase(plan, -1, grads, state, hyper, weights, K_LAMB1, workspace, st)) != WS_OK) return s;
        if ((s = ws_lamb_finalize(plan, workspace, workspace_bytes, stream)) != WS_OK) return s;
        return fused_phase(plan, -1, grads, state, hyper, weights, K_LAMB2, workspace, st);
    }
    if (hyper->opt == WS_LARS) {
        if (r != -1) return WS_ERR_INVALID_ARG;
        ws_status s = check_ws(plan, workspace, workspace_bytes, WS_LARS);
        if (s != WS_OK) return s;
        bool done = false;
        s = try_one_launch(plan, 1, nullptr, grads, state, hyper, nullptr, weights, workspace, workspace_bytes, st, done);
        if (s != WS_OK || done) return s;
        if ((s = fused_phase(plan, -1, grads, state, hyper, weights, K_LARS1, workspace, st)) != WS_OK) return s;
        const WsLambWs L = ws_lamb_layout(plan, workspace);
        launch_lamb_finalize(plan->T, st, plan->d_segtiles, L.partials, plan->ntiles, finalize_reps(plan), L.rho,
                                                        L.norms, 1, hyper->trust_coeff, hyper->weight_decay);
        if ((s = ws_check_launch("ws_fused_update(LARS finalize)")) != WS_OK) return s;
        return fused_phase(plan, -1, grads, state, hyper, weights, K_LARS2, workspace, st);
    }
    if (hyper->opt != WS_SGDM && hyper->opt != WS_ADAM) return WS_ERR_INVALID_ARG;
    return fused_phase(plan, r, grads, state, hyper, weights, hyper->opt == WS_SGDM ? K_SGDM : K_ADAM, nullptr, st);
}
