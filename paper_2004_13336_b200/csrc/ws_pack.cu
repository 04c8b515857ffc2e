// Pack / unpack kernels: bit copies between a model's tensor list and the
// shard-major [R][S] layout (paper Section 4.1: pad + dynamic-slice by replica
// id; Section 4.2: reverse formatting after the all-gather).  Padding is
// produced in place: a tensor is never read past n_t and pads are written as
// all-zero bits (Section 4.1: the pad is fused into the slice).
//
// Work item = (shard r, tile).  A tile is moved as 32-byte vectors (ld/st.global.v8.b32) when every
// pointer and the alignment A allow it, else as 16-byte vectors; the one vector that straddles n_t
// is moved element by element.  In the concatenated
// layout every shard has its own tiles and a tile names its shard.
#include "ws_internal.h"

namespace {

constexpr int kBlock = 256;     // largest CTA; the launch picks 64 ... 256 threads by tile size
constexpr int kPtrChunk = 1024;  // tensor pointers passed by value per launch (8 KB)

struct PtrChunk {
    void* p[kPtrChunk];
};

struct PackParams {
    const WsTile* tiles;
    long long tile_lo;    // first tile handled by this launch
    long long ntl;        // tiles handled by this launch
    long long nitems;     // R * ntl
    long long S;
    int seg_lo;           // tensor index of PtrChunk::p[0]
    int concat;           // concatenated layout: every tile names its own shard
#ifdef WS_DEBUG_BOUNDS
    unsigned* bounds;     // status word of the bounds checks
    long long flat_elems; // elements of the flat buffer
#endif
};

// VB-byte vector (16 or 32) moved with streaming accesses
template <int VB>
struct Vec {
    unsigned w[VB / 4];
};
template <int VB>
__device__ __forceinline__ Vec<VB> ld_stream(const char* p) {
    Vec<VB> v;
    if constexpr (VB == 16) {
        const uint4 t = __ldcs(reinterpret_cast<const uint4*>(p));
        v.w[0] = t.x; v.w[1] = t.y; v.w[2] = t.z; v.w[3] = t.w;
    } else {
        asm volatile("ld.global.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]), "=r"(v.w[4]), "=r"(v.w[5]), "=r"(v.w[6]), "=r"(v.w[7])
                     : "l"(p));
    }
    return v;
}
template <int VB>
__device__ __forceinline__ void st_stream(char* p, const Vec<VB>& v) {
    if constexpr (VB == 16) {
        __stcs(reinterpret_cast<uint4*>(p), make_uint4(v.w[0], v.w[1], v.w[2], v.w[3]));
    } else {
        asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                     :: "l"(p), "r"(v.w[0]), "r"(v.w[1]), "r"(v.w[2]), "r"(v.w[3]), "r"(v.w[4]), "r"(v.w[5]), "r"(v.w[6]), "r"(v.w[7])
                     : "memory");
    }
}
template <int VB>
__device__ __forceinline__ Vec<VB> zero_vec() {
    Vec<VB> v;
#pragma unroll
    for (int i = 0; i < VB / 4; ++i) v.w[i] = 0u;
    return v;
}

// Programmatic dependent launch: the grid may become resident while the previous kernel of the stream
// drains; the kernels read only tables that were uploaded once before their griddepcontrol.wait.
template <typename... KArgs, typename... Args>
static void launch_pdl(void (*kernel)(KArgs...), long long grid, int block, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// EB = element bytes (4 or 2); PACK = true: tensors -> flat, false: flat -> tensors; VB = vector bytes
template <int EB, bool PACK, int VB>
__global__ void __launch_bounds__(kBlock) pack_kernel(PackParams P, const __grid_constant__ PtrChunk tab,
                                                      char* __restrict__ flat) {
    constexpr int EPV = VB / EB;  // elements per vector
    // the next kernel of the stream may start its prologue while this grid's last CTAs run
    asm volatile("griddepcontrol.launch_dependents;");
    for (long long item = blockIdx.x; item < P.nitems; item += gridDim.x) {
        long long r = P.concat ? 0 : item / P.ntl;
        const WsTile tl = P.tiles[P.tile_lo + (item - r * P.ntl)];
        if (P.concat) r = tl.shard;
        char* tensor = (char*)tab.p[tl.seg - P.seg_lo];
        // the plan's tile table does not depend on the previous kernel of the stream; the data does
        asm volatile("griddepcontrol.wait;" ::: "memory");
        const long long src0 = r * tl.piece + tl.poff;      // element index in the tensor
        long long nv = tl.vt - r * tl.piece;                // valid elements in this tile
        nv = nv < 0 ? 0 : (nv > tl.len ? (long long)tl.len : nv);
#ifdef WS_DEBUG_BOUNDS
        if (r * P.S + tl.pos < 0 || r * P.S + tl.pos + tl.len > P.flat_elems) {
            if (threadIdx.x == 0 && P.bounds) atomicOr(P.bounds, (unsigned)WS_BOUNDS_FLAT);
            continue;
        }
#endif
        char* fl = flat + (r * P.S + tl.pos) * EB;
        char* tn = tensor + src0 * EB;
        const int nvec = tl.len / EPV;
#pragma unroll 4
        for (int i = threadIdx.x; i < nvec; i += blockDim.x) {
            const long long e0 = (long long)i * EPV;
            if (e0 + EPV <= nv) {
                if (PACK) st_stream<VB>(fl + (long long)i * VB, ld_stream<VB>(tn + (long long)i * VB));
                else      st_stream<VB>(tn + (long long)i * VB, ld_stream<VB>(fl + (long long)i * VB));
            } else if (e0 >= nv) {
                if (PACK) st_stream<VB>(fl + (long long)i * VB, zero_vec<VB>());
            } else {
                // the vector holding the last valid element
                const int k = (int)(nv - e0);
                if (EB == 4) {
                    unsigned int* f = (unsigned int*)fl + e0;
                    unsigned int* t = (unsigned int*)tn + e0;
                    for (int j = 0; j < EPV; ++j) {
                        if (PACK) f[j] = j < k ? t[j] : 0u;
                        else if (j < k) t[j] = f[j];
                    }
                } else {
                    unsigned short* f = (unsigned short*)fl + e0;
                    unsigned short* t = (unsigned short*)tn + e0;
                    for (int j = 0; j < EPV; ++j) {
                        if (PACK) f[j] = j < k ? t[j] : (unsigned short)0;
                        else if (j < k) t[j] = f[j];
                    }
                }
            }
        }
    }
}

// All gradient lists of a step in one launch: set k's tensors (found through the device table
// [T][nsets]) go to flats.p[k].  Work items are set-major, so each set is walked front to back.
struct FlatPtrs {
    void* p[kPtrChunk];
};

template <int EB, int VB>
__global__ void __launch_bounds__(kBlock) pack_sets_kernel(PackParams P, const void* const* __restrict__ table, int nsets,
                                                           const __grid_constant__ FlatPtrs flats) {
    constexpr int EPV = VB / EB;
    const long long total = P.nitems * nsets;
    asm volatile("griddepcontrol.launch_dependents;");
    for (long long gi = blockIdx.x; gi < total; gi += gridDim.x) {
        const int k = (int)(gi / P.nitems);
        const long long item = gi - (long long)k * P.nitems;
        long long r = P.concat ? 0 : item / P.ntl;
        const WsTile tl = P.tiles[item - r * P.ntl];
        if (P.concat) r = tl.shard;
        const char* tn = (const char*)table[(long long)tl.seg * nsets + k] + (r * tl.piece + tl.poff) * EB;
        // tile and pointer tables were uploaded once; the previous kernel of the stream may own the data
        asm volatile("griddepcontrol.wait;" ::: "memory");
        long long nv = tl.vt - r * tl.piece;
        nv = nv < 0 ? 0 : (nv > tl.len ? (long long)tl.len : nv);
#ifdef WS_DEBUG_BOUNDS
        if (r * P.S + tl.pos < 0 || r * P.S + tl.pos + tl.len > P.flat_elems) {
            if (threadIdx.x == 0 && P.bounds) atomicOr(P.bounds, (unsigned)WS_BOUNDS_FLAT);
            continue;
        }
#endif
        char* fl = (char*)flats.p[k] + (r * P.S + tl.pos) * EB;
        const int nvec = tl.len / EPV;
#pragma unroll 4
        for (int i = threadIdx.x; i < nvec; i += blockDim.x) {
            const long long e0 = (long long)i * EPV;
            if (e0 + EPV <= nv) {
                st_stream<VB>(fl + (long long)i * VB, ld_stream<VB>(tn + (long long)i * VB));
            } else if (e0 >= nv) {
                st_stream<VB>(fl + (long long)i * VB, zero_vec<VB>());
            } else {
                const int kk = (int)(nv - e0);
                if (EB == 4) {
                    unsigned int* f = (unsigned int*)fl + e0;
                    const unsigned int* t = (const unsigned int*)tn + e0;
                    for (int j = 0; j < EPV; ++j) f[j] = j < kk ? t[j] : 0u;
                } else {
                    unsigned short* f = (unsigned short*)fl + e0;
                    const unsigned short* t = (const unsigned short*)tn + e0;
                    for (int j = 0; j < EPV; ++j) f[j] = j < kk ? t[j] : (unsigned short)0;
                }
            }
        }
    }
}

// A tile of the default 2048 elements is 256 32-byte vectors: with 256 threads every thread would move
// one vector behind ~100 instructions of tile bookkeeping.  Two or more vectors per thread measured
// best (ResNet-50 set: pack of the 8 lists 0.90 -> 0.99 of the copy bandwidth with 128 threads), while
// 8192-element tiles keep 256 threads.
int pack_block(const ws_plan* p, int eb, int vb) {
    const long long vecs = (long long)p->K * eb / vb;     // vectors per full tile
    int b = 256;
    while (b > 64 && vecs < 2LL * b) b >>= 1;
    return b;
}

template <bool PACK>
ws_status run(const ws_plan* p, void* const* tensor_ptrs, ws_dtype dtype, void* flat, void* stream) {
    if (!p || !tensor_ptrs || !flat) return WS_ERR_INVALID_ARG;
    if (dtype != WS_F32 && dtype != WS_BF16) return WS_ERR_DTYPE;
    if (!p->d_tiles) return WS_ERR_NOT_UPLOADED;
    if (!ws_aligned16(flat)) return WS_ERR_ALIGNMENT;
    // 32-byte vectors when the flat buffer, every tensor and every piece start on a 32-byte boundary
    const int eb = dtype == WS_BF16 ? 2 : 4;
    bool wide = (reinterpret_cast<uintptr_t>(flat) & 31u) == 0 && (p->A * eb) % 32 == 0;
    for (int t = 0; t < p->T; ++t) {
        if (p->segs[t].numel == 0) continue;   // empty tensor: never dereferenced, may be null
        if (!tensor_ptrs[t]) return WS_ERR_INVALID_ARG;
        if (!ws_aligned16(tensor_ptrs[t])) return WS_ERR_ALIGNMENT;
        wide = wide && (reinterpret_cast<uintptr_t>(tensor_ptrs[t]) & 31u) == 0;
    }
    cudaStream_t st = (cudaStream_t)stream;
    for (int seg_lo = 0; seg_lo < p->T; seg_lo += kPtrChunk) {
        const int seg_hi = seg_lo + kPtrChunk < p->T ? seg_lo + kPtrChunk : p->T;
        PtrChunk tab = {};
        for (int t = seg_lo; t < seg_hi; ++t) tab.p[t - seg_lo] = tensor_ptrs[t];
        PackParams P;
        P.tiles = p->d_tiles;
        P.tile_lo = p->segtiles[seg_lo].tile_begin;
        const long long tile_hi = (long long)p->segtiles[seg_hi - 1].tile_begin + p->segtiles[seg_hi - 1].tile_count;
        P.ntl = tile_hi - P.tile_lo;
        P.concat = (p->layout == WS_LAYOUT_CONCAT);
        P.nitems = P.concat ? P.ntl : P.ntl * p->R;
        P.S = p->S;
        P.seg_lo = seg_lo;
#ifdef WS_DEBUG_BOUNDS
        P.bounds = ws_bounds_word();
        P.flat_elems = (long long)p->R * p->S;
#endif
        long long grid = P.nitems;   // one CTA per (shard, tile): the CTA scheduler walks the buffers in order
        if (grid > 0x7fffffffLL) grid = 0x7fffffffLL;
        if (grid < 1) continue;
        const int nb = pack_block(p, eb, wide ? 32 : 16);
        if (wide) {
            if (dtype == WS_F32) launch_pdl(pack_kernel<4, PACK, 32>, grid, nb, st, P, tab, (char*)flat);
            else                 launch_pdl(pack_kernel<2, PACK, 32>, grid, nb, st, P, tab, (char*)flat);
        } else {
            if (dtype == WS_F32) launch_pdl(pack_kernel<4, PACK, 16>, grid, nb, st, P, tab, (char*)flat);
            else                 launch_pdl(pack_kernel<2, PACK, 16>, grid, nb, st, P, tab, (char*)flat);
        }
        ws_status s = ws_check_launch(PACK ? "ws_pack" : "ws_unpack");
        if (s != WS_OK) return s;
    }
    return WS_OK;
}

}  // namespace

extern "C" ws_status ws_pack(const ws_plan* plan, const void* const* tensor_ptrs, ws_dtype dtype, void* flat,
                             void* stream) {
    WsRange range_("ws_pack");
    return run<true>(plan, (void* const*)tensor_ptrs, dtype, flat, stream);
}

extern "C" ws_status ws_unpack(const ws_plan* plan, const void* flat, ws_dtype dtype, void* const* tensor_ptrs,
                               void* stream) {
    WsRange range_("ws_unpack");
    return run<false>(plan, tensor_ptrs, dtype, (void*)flat, stream);
}

extern "C" ws_status ws_pack_sets(const ws_plan* p, const ws_tensor_table* table, void* const* flats, void* stream) {
    WsRange range_("ws_pack_sets");
    if (!p || !table || !table->dev || !flats) return WS_ERR_INVALID_ARG;
    if (!p->d_tiles) return WS_ERR_NOT_UPLOADED;
    if (table->T != p->T || table->nsets < 1 || table->nsets > kPtrChunk) return WS_ERR_INVALID_ARG;
    if (table->dtype != WS_F32 && table->dtype != WS_BF16) return WS_ERR_DTYPE;
    FlatPtrs fp = {};
    for (int k = 0; k < table->nsets; ++k) {
        if (!flats[k]) return WS_ERR_INVALID_ARG;
        if (!ws_aligned16(flats[k])) return WS_ERR_ALIGNMENT;
        fp.p[k] = flats[k];
    }
    PackParams P;
    P.tiles = p->d_tiles;
    P.tile_lo = 0;
    P.ntl = p->ntiles;
    P.concat = (p->layout == WS_LAYOUT_CONCAT);
    P.nitems = P.concat ? P.ntl : P.ntl * p->R;
    P.S = p->S;
    P.seg_lo = 0;
#ifdef WS_DEBUG_BOUNDS
    P.bounds = ws_bounds_word();
    P.flat_elems = (long long)p->R * p->S;
#endif
    long long grid = P.nitems * table->nsets;
    if (grid < 1) return WS_OK;
    if (grid > 0x7fffffffLL) grid = 0x7fffffffLL;
    cudaStream_t st = (cudaStream_t)stream;
    const int eb = table->dtype == WS_BF16 ? 2 : 4;
    bool wide = table->min_align >= 32 && (p->A * eb) % 32 == 0;
    for (int k = 0; k < table->nsets; ++k) wide = wide && (reinterpret_cast<uintptr_t>(flats[k]) & 31u) == 0;
    const void* const* tb = (const void* const*)table->dev;
    const int nb = pack_block(p, eb, wide ? 32 : 16);
    const int ns = table->nsets;
    if (wide) {
        if (table->dtype == WS_F32) launch_pdl(pack_sets_kernel<4, 32>, grid, nb, st, P, tb, ns, fp);
        else                        launch_pdl(pack_sets_kernel<2, 32>, grid, nb, st, P, tb, ns, fp);
    } else {
        if (table->dtype == WS_F32) launch_pdl(pack_sets_kernel<4, 16>, grid, nb, st, P, tb, ns, fp);
        else                        launch_pdl(pack_sets_kernel<2, 16>, grid, nb, st, P, tb, ns, fp);
    }
    return ws_check_launch("ws_pack_sets");
}
