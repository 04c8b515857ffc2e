// Pack / unpack kernels: bit copies between a model's tensor list and the
// shard-major [R][S] layout (paper Section 4.1: pad + dynamic-slice by replica
// id; Section 4.2: reverse formatting after the all-gather).  Padding is
// produced in place: a tensor is never read past n_t and pads are written as
// all-zero bits (Section 4.1: the pad is fused into the slice).
//
// Work item = (shard r, tile).  A tile is moved as 16-byte vectors; the one
// vector that straddles n_t is moved element by element.  In the concatenated
// layout every shard has its own tiles and a tile names its shard.
#include "ws_internal.h"

namespace {

constexpr int kBlock = 256;
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
};

__device__ __forceinline__ uint4 ld_stream(const uint4* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(uint4* p, uint4 v) { __stcs(p, v); }

// EB = element bytes (4 or 2); PACK = true: tensors -> flat, false: flat -> tensors
template <int EB, bool PACK>
__global__ void __launch_bounds__(kBlock) pack_kernel(PackParams P, const __grid_constant__ PtrChunk tab,
                                                      char* __restrict__ flat) {
    constexpr int EPV = 16 / EB;  // elements per 16-byte vector
    for (long long item = blockIdx.x; item < P.nitems; item += gridDim.x) {
        long long r = P.concat ? 0 : item / P.ntl;
        const WsTile tl = P.tiles[P.tile_lo + (item - r * P.ntl)];
        if (P.concat) r = tl.shard;
        char* tensor = (char*)tab.p[tl.seg - P.seg_lo];
        const long long src0 = r * tl.piece + tl.poff;      // element index in the tensor
        long long nv = tl.vt - r * tl.piece;                // valid elements in this tile
        nv = nv < 0 ? 0 : (nv > tl.len ? (long long)tl.len : nv);
        char* fl = flat + (r * P.S + tl.pos) * EB;
        char* tn = tensor + src0 * EB;
        const int nvec = tl.len / EPV;
        for (int i = threadIdx.x; i < nvec; i += kBlock) {
            const long long e0 = (long long)i * EPV;
            if (e0 + EPV <= nv) {
                if (PACK) st_stream((uint4*)(fl) + i, ld_stream((const uint4*)(tn) + i));
                else      st_stream((uint4*)(tn) + i, ld_stream((const uint4*)(fl) + i));
            } else if (e0 >= nv) {
                if (PACK) st_stream((uint4*)(fl) + i, make_uint4(0, 0, 0, 0));
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

template <int EB>
__global__ void __launch_bounds__(kBlock) pack_sets_kernel(PackParams P, const void* const* __restrict__ table, int nsets,
                                                           const __grid_constant__ FlatPtrs flats) {
    constexpr int EPV = 16 / EB;
    const long long total = P.nitems * nsets;
    for (long long gi = blockIdx.x; gi < total; gi += gridDim.x) {
        const int k = (int)(gi / P.nitems);
        const long long item = gi - (long long)k * P.nitems;
        long long r = P.concat ? 0 : item / P.ntl;
        const WsTile tl = P.tiles[item - r * P.ntl];
        if (P.concat) r = tl.shard;
        const char* tn = (const char*)table[(long long)tl.seg * nsets + k] + (r * tl.piece + tl.poff) * EB;
        long long nv = tl.vt - r * tl.piece;
        nv = nv < 0 ? 0 : (nv > tl.len ? (long long)tl.len : nv);
        char* fl = (char*)flats.p[k] + (r * P.S + tl.pos) * EB;
        const int nvec = tl.len / EPV;
        for (int i = threadIdx.x; i < nvec; i += kBlock) {
            const long long e0 = (long long)i * EPV;
            if (e0 + EPV <= nv) {
                st_stream((uint4*)(fl) + i, ld_stream((const uint4*)(tn) + i));
            } else if (e0 >= nv) {
                st_stream((uint4*)(fl) + i, make_uint4(0, 0, 0, 0));
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

template <bool PACK>
ws_status run(const ws_plan* p, void* const* tensor_ptrs, ws_dtype dtype, void* flat, void* stream) {
    if (!p || !tensor_ptrs || !flat) return WS_ERR_INVALID_ARG;
    if (dtype != WS_F32 && dtype != WS_BF16) return WS_ERR_DTYPE;
    if (!p->d_tiles) return WS_ERR_NOT_UPLOADED;
    if (!ws_aligned16(flat)) return WS_ERR_ALIGNMENT;
    for (int t = 0; t < p->T; ++t) {
        if (p->segs[t].numel == 0) continue;   // empty tensor: never dereferenced, may be null
        if (!tensor_ptrs[t]) return WS_ERR_INVALID_ARG;
        if (!ws_aligned16(tensor_ptrs[t])) return WS_ERR_ALIGNMENT;
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
        long long grid = P.nitems;   // one CTA per (shard, tile): the CTA scheduler walks the buffers in order
        if (grid > 0x7fffffffLL) grid = 0x7fffffffLL;
        if (grid < 1) continue;
        if (dtype == WS_F32) pack_kernel<4, PACK><<<(unsigned)grid, kBlock, 0, st>>>(P, tab, (char*)flat);
        else                 pack_kernel<2, PACK><<<(unsigned)grid, kBlock, 0, st>>>(P, tab, (char*)flat);
        ws_status s = ws_check_launch(PACK ? "ws_pack" : "ws_unpack");
        if (s != WS_OK) return s;
    }
    return WS_OK;
}

}  // namespace

extern "C" ws_status ws_pack(const ws_plan* plan, const void* const* tensor_ptrs, ws_dtype dtype, void* flat,
                             void* stream) {
    return run<true>(plan, (void* const*)tensor_ptrs, dtype, flat, stream);
}

extern "C" ws_status ws_unpack(const ws_plan* plan, const void* flat, ws_dtype dtype, void* const* tensor_ptrs,
                               void* stream) {
    return run<false>(plan, tensor_ptrs, dtype, (void*)flat, stream);
}

extern "C" ws_status ws_pack_sets(const ws_plan* p, const ws_tensor_table* table, void* const* flats, void* stream) {
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
    long long grid = P.nitems * table->nsets;
    if (grid < 1) return WS_OK;
    if (grid > 0x7fffffffLL) grid = 0x7fffffffLL;
    cudaStream_t st = (cudaStream_t)stream;
    if (table->dtype == WS_F32)
        pack_sets_kernel<4><<<(unsigned)grid, kBlock, 0, st>>>(P, (const void* const*)table->dev, table->nsets, fp);
    else
        pack_sets_kernel<2><<<(unsigned)grid, kBlock, 0, st>>>(P, (const void* const*)table->dev, table->nsets, fp);
    return ws_check_launch("ws_pack_sets");
}
