// Shard planner and plan upload (host code).
//
// Sharding format (paper Section 4.1): a tensor's dimensions are combined,
// the result is padded so that the shard count divides it, and shard r is the
// r-th equal slice.  On linear GPU memory combining ALL dimensions is free, so
// the format is "flatten, pad, slice"; each slice (piece) is also rounded up
// to A elements so that 16-byte vectors never straddle two tensors.
// One combined shard is piece r of every tensor, in order (Section 5.2).
#include <stdio.h>
#include <string.h>

#include <new>

#include "ws_internal.h"

static thread_local char g_cuda_err[256] = "";

ws_status ws_cuda_fail(cudaError_t e, const char* what) {
    snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s", what, cudaGetErrorString(e));
    return WS_ERR_CUDA;
}

ws_status ws_check_launch(const char* what) {
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? WS_OK : ws_cuda_fail(e, what);
}

extern "C" const char* ws_last_cuda_error(void) { return g_cuda_err; }

extern "C" const char* ws_status_string(ws_status s) {
    switch (s) {
        case WS_OK: return "ok";
        case WS_ERR_INVALID_ARG: return "invalid argument";
        case WS_ERR_ALIGNMENT: return "device pointer not 16-byte aligned";
        case WS_ERR_DTYPE: return "unsupported dtype combination";
        case WS_ERR_WORKSPACE: return "workspace missing or too small";
        case WS_ERR_NOT_UPLOADED: return "plan not uploaded to the device";
        case WS_ERR_CUDA: return "CUDA error";
        case WS_ERR_TOO_LARGE: return "size beyond a fixed limit";
    }
    return "unknown status";
}

// Adafactor's matrix view of every tensor: columns = last dimension, rows = all leading
// dimensions together; fewer than two dimensions: one row, no row accumulator.
static void ws_matrix_views(ws_plan* p, const ws_tensor_desc* descs) {
    p->segaf.resize(p->T);
    p->afchunks.clear();
    long long foff = 0, ioff = 0;
    for (int t = 0; t < p->T; ++t) {
        const ws_tensor_desc& d = descs[t];
        const long long n = p->segs[t].numel;
        WsSegAf a;
        a.foff = foff;
        a.numel = n;
        if (d.ndim >= 2 && n > 0) {
            a.ncol = d.dims[d.ndim - 1];
            a.nrow = n / a.ncol;
        } else {
            a.nrow = 0;
            a.ncol = n;
        }
        foff += a.nrow + a.ncol;
        a.irow = ioff;
        ioff += (a.nrow + 7) / 8 * 8;
        a.icol = ioff;
        ioff += (a.ncol + 7) / 8 * 8;
        p->segaf[t] = a;
        for (long long b = 0; b < a.nrow + a.ncol; b += 1024) {
            WsAfChunk c;
            c.begin = b;
            c.count = (int)((a.nrow + a.ncol - b) < 1024 ? (a.nrow + a.ncol - b) : 1024);
            c.seg = t;
            p->afchunks.push_back(c);
        }
    }
    p->F = foff;
    p->Fi = ioff;
}

// Work items of the one-launch schedule: every tile cut into runs of kWsItemElems elements, for every
// shard it serves.  Plans beyond the item fields' ranges get no schedule (n_items stays 0).
static void ws_count_items(ws_plan* p) {
    p->n_items = 0;
    if (p->R > 65535) return;
    long long per_shard = 0;
    for (const WsTile& tl : p->tiles) per_shard += (tl.len + kWsItemElems - 1) / kWsItemElems;
    const long long n = p->layout == WS_LAYOUT_CONCAT ? per_shard : per_shard * p->R;
    if (n > 0x3fffffffLL) return;
    p->n_items = n;
}

extern "C" ws_status ws_plan_create(const ws_tensor_desc* descs, int32_t T, int32_t R,
                                    int32_t align_elems, int32_t tile_elems, ws_plan** out) {
    return ws_plan_create_layout(descs, T, R, align_elems, tile_elems, WS_LAYOUT_PER_TENSOR, out);
}

extern "C" int32_t ws_plan_layout(const ws_plan* p) { return p ? p->layout : 0; }

extern "C" ws_status ws_plan_create_layout(const ws_tensor_desc* descs, int32_t T, int32_t R, int32_t align_elems,
                                           int32_t tile_elems, ws_layout layout, ws_plan** out) {
    if (!out) return WS_ERR_INVALID_ARG;
    *out = nullptr;
    if (!descs || T < 1 || R < 1) return WS_ERR_INVALID_ARG;
    if (layout != WS_LAYOUT_PER_TENSOR && layout != WS_LAYOUT_CONCAT) return WS_ERR_INVALID_ARG;
    if (align_elems < 8 || (align_elems & (align_elems - 1)) != 0) return WS_ERR_INVALID_ARG;
    if (tile_elems == 0) {
        // Default: the largest tile that still leaves >= 20000 work items for an all-shard
        // launch.  A CTA reads its tile descriptor before it can issue any data load, so a
        // large tile amortises that latency; small models keep small tiles so that the
        // grid still spreads evenly over the SMs.
        long long total = 0;
        for (int t = 0; t < T; ++t) {
            long long n = 1;
            for (int i = 0; i < descs[t].ndim && i < WS_MAX_DIMS; ++i) n *= (descs[t].dims[i] > 0 ? descs[t].dims[i] : 0);
            total += n;
        }
        // ... and >= 600 items for a single-shard launch (many replicas make tiny shards; a CTA
        // then walks all R gradient slices for its tile, so the grid needs the parallelism).
        tile_elems = 1024;
        if (total / R / 2048 >= 600) tile_elems = 2048;
        while (tile_elems >= 2048 && tile_elems < 8192 && total / (2 * tile_elems) >= 20000 &&
               total / R / (2 * tile_elems) >= 600)
            tile_elems *= 2;
    }
    if (tile_elems < 1024 || tile_elems % 1024 != 0 || tile_elems > (1 << 20)) return WS_ERR_INVALID_ARG;

    ws_plan* p = new (std::nothrow) ws_plan;
    if (!p) return WS_ERR_INVALID_ARG;
    p->T = T;
    p->R = R;
    p->A = align_elems;
    p->K = tile_elems;
    p->layout = layout;
    try {
        p->segs.resize(T);
        p->segtiles.resize(T);
        long long off = 0;
        for (int t = 0; layout == WS_LAYOUT_CONCAT && t < T; ++t) {
            // Concatenated layout (Section 5.2): tensors back to back, each start rounded up to A.
            const ws_tensor_desc& d = descs[t];
            if (d.ndim < 0 || d.ndim > WS_MAX_DIMS) { delete p; return WS_ERR_INVALID_ARG; }
            long long n = 1;
            for (int i = 0; i < d.ndim; ++i) {
                if (d.dims[i] < 0 || (d.dims[i] > 0 && n > (1LL << 46) / d.dims[i])) { delete p; return WS_ERR_INVALID_ARG; }
                n *= d.dims[i];
            }
            p->segs[t].numel = n;
            p->segs[t].piece = 0;
            p->segs[t].shard_off = off;          // start inside the concatenation
            p->N += n;
            p->arena_off.push_back(p->arena_elems);
            p->arena_elems += (n + 7) / 8 * 8;
            off = (off + n + align_elems - 1) / align_elems * align_elems;
        }
        if (layout == WS_LAYOUT_CONCAT) {
            const long long C = off;
            const long long per = (C + R - 1) / R;
            p->S = (per + align_elems - 1) / align_elems * align_elems;
            const long long G = p->S * R;
            // region of tensor t: from its start to the next tensor's start (the alignment gap
            // belongs to it as padding); the last region runs to the end of the last shard
            int t = 0;
            p->shard_tile_begin.assign(R + 1, 0);
            for (int k = 0; k < T; ++k) { p->segtiles[k].tile_begin = 0; p->segtiles[k].tile_count = 0; }
            std::vector<char> seen(T, 0);
            for (int r = 0; r < R; ++r) {
                p->shard_tile_begin[r] = (long long)p->tiles.size();
                long long pos = (long long)r * p->S;            // global position
                const long long end = pos + p->S;
                while (pos < end) {
                    // tensor whose region holds `pos`
                    while (t < T - 1 && p->segs[t + 1].shard_off <= pos) ++t;
                    const long long reg_end = (t < T - 1) ? p->segs[t + 1].shard_off : G;
                    long long stop = reg_end < end ? reg_end : end;
                    long long len = stop - pos;
                    if (len > tile_elems) len = tile_elems;
                    WsTile tl;
                    memset(&tl, 0, sizeof(tl));
                    tl.pos = pos - (long long)r * p->S;
                    tl.poff = pos - p->segs[t].shard_off;
                    tl.vt = p->segs[t].numel - tl.poff;
                    tl.piece = 0;
                    tl.len = (int)len;
                    tl.seg = t;
                    tl.shard = r;
                    if ((long long)p->tiles.size() >= 0x7fffffffLL) { delete p; return WS_ERR_TOO_LARGE; }
                    if (!seen[t]) { seen[t] = 1; p->segtiles[t].tile_begin = (int)p->tiles.size(); }
                    p->segtiles[t].tile_count += 1;
                    p->tiles.push_back(tl);
                    pos += len;
                }
            }
            p->shard_tile_begin[R] = (long long)p->tiles.size();
            p->ntiles = (long long)p->tiles.size();
            // a tensor without tiles (empty, and no padding region of its own) still names the place
            // in the tile list where its tiles would be, so that a range of tensors maps to a range of tiles
            for (int k = 0; k < T; ++k)
                if (!seen[k])
                    p->segtiles[k].tile_begin = k > 0 ? p->segtiles[k - 1].tile_begin + p->segtiles[k - 1].tile_count : 0;
            ws_matrix_views(p, descs);
            ws_count_items(p);
            *out = p;
            return WS_OK;
        }
        for (int t = 0; t < T; ++t) {
            const ws_tensor_desc& d = descs[t];
            if (d.ndim < 0 || d.ndim > WS_MAX_DIMS) { delete p; return WS_ERR_INVALID_ARG; }
            long long n = 1;
            for (int i = 0; i < d.ndim; ++i) {
                if (d.dims[i] < 0 || (d.dims[i] > 0 && n > (1LL << 46) / d.dims[i])) { delete p; return WS_ERR_INVALID_ARG; }
                n *= d.dims[i];   // a zero dimension makes an empty tensor: no piece, no tiles
            }
            long long per = (n + R - 1) / R;
            long long piece = (per + align_elems - 1) / align_elems * align_elems;
            p->segs[t].numel = n;
            p->segs[t].piece = piece;
            p->segs[t].shard_off = off;
            p->N += n;
            p->arena_off.push_back(p->arena_elems);
            p->arena_elems += (n + 7) / 8 * 8;
            // cut the piece into tiles that stay inside it
            long long ntile = (piece + tile_elems - 1) / tile_elems;
            if ((long long)p->tiles.size() + ntile > 0x7fffffffLL) { delete p; return WS_ERR_TOO_LARGE; }
            p->segtiles[t].tile_begin = (int)p->tiles.size();
            p->segtiles[t].tile_count = (int)ntile;
            for (long long i = 0; i < ntile; ++i) {
                WsTile tl;
                memset(&tl, 0, sizeof(tl));
                tl.poff = i * tile_elems;
                tl.pos = off + tl.poff;
                tl.vt = n - tl.poff;
                tl.piece = piece;
                long long len = piece - tl.poff;
                tl.len = (int)(len < tile_elems ? len : tile_elems);
                tl.seg = t;
                p->tiles.push_back(tl);
            }
            off += piece;
        }
        p->S = off;
        p->ntiles = (long long)p->tiles.size();
        ws_matrix_views(p, descs);
        ws_count_items(p);
    } catch (...) {
        delete p;
        return WS_ERR_INVALID_ARG;
    }
    *out = p;
    return WS_OK;
}

extern "C" void ws_plan_destroy(ws_plan* plan) { delete plan; }
extern "C" int32_t ws_plan_num_tensors(const ws_plan* p) { return p ? p->T : 0; }
extern "C" int32_t ws_plan_num_shards(const ws_plan* p) { return p ? p->R : 0; }
extern "C" int32_t ws_plan_align(const ws_plan* p) { return p ? p->A : 0; }
extern "C" int64_t ws_plan_shard_elems(const ws_plan* p) { return p ? p->S : 0; }
extern "C" int64_t ws_plan_valid_elems(const ws_plan* p) { return p ? p->N : 0; }
extern "C" int64_t ws_plan_num_tiles(const ws_plan* p) { return p ? p->ntiles : 0; }

extern "C" ws_status ws_plan_segments(const ws_plan* p, const ws_segment** segs, int32_t* T) {
    if (!p || !segs || !T) return WS_ERR_INVALID_ARG;
    *segs = p->segs.data();
    *T = p->T;
    return WS_OK;
}

static size_t round16(size_t x) { return (x + 15) & ~(size_t)15; }

extern "C" size_t ws_plan_device_bytes(const ws_plan* p) {
    if (!p) return 0;
    return round16(p->tiles.size() * sizeof(WsTile)) + round16(p->segtiles.size() * sizeof(WsSegTiles)) +
           round16(p->segaf.size() * sizeof(WsSegAf)) + round16(p->afchunks.size() * sizeof(WsAfChunk));
}

extern "C" int64_t ws_plan_factored_elems(const ws_plan* p) { return p ? p->F : 0; }

extern "C" ws_status ws_plan_factored_layout(const ws_plan* p, int64_t* layout) {
    if (!p || !layout) return WS_ERR_INVALID_ARG;
    for (int t = 0; t < p->T; ++t) {
        const WsSegAf& a = p->segaf[t];
        layout[3 * t] = a.foff;
        layout[3 * t + 1] = a.nrow > 0 ? a.nrow : a.ncol;
        layout[3 * t + 2] = a.nrow > 0 ? a.ncol : 0;
    }
    return WS_OK;
}

extern "C" ws_status ws_plan_upload(ws_plan* p, void* dev_buf, size_t bytes, void* stream) {
    if (!p || !dev_buf) return WS_ERR_INVALID_ARG;
    if (!ws_aligned16(dev_buf)) return WS_ERR_ALIGNMENT;
    if (bytes < ws_plan_device_bytes(p)) return WS_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    size_t tb = p->tiles.size() * sizeof(WsTile);
    char* base = (char*)dev_buf;
    cudaError_t e = cudaMemcpyAsync(base, p->tiles.data(), tb, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return ws_cuda_fail(e, "ws_plan_upload(tiles)");
    e = cudaMemcpyAsync(base + round16(tb), p->segtiles.data(), p->segtiles.size() * sizeof(WsSegTiles),
                        cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return ws_cuda_fail(e, "ws_plan_upload(segments)");
    const size_t ab = round16(tb) + round16(p->segtiles.size() * sizeof(WsSegTiles));
    e = cudaMemcpyAsync(base + ab, p->segaf.data(), p->segaf.size() * sizeof(WsSegAf), cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return ws_cuda_fail(e, "ws_plan_upload(matrix views)");
    p->d_tiles = (const WsTile*)base;
    p->d_segtiles = (const WsSegTiles*)(base + round16(tb));
    p->d_segaf = (const WsSegAf*)(base + ab);
    const size_t cb = ab + round16(p->segaf.size() * sizeof(WsSegAf));
    if (!p->afchunks.empty()) {
        e = cudaMemcpyAsync(base + cb, p->afchunks.data(), p->afchunks.size() * sizeof(WsAfChunk), cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) return ws_cuda_fail(e, "ws_plan_upload(state chunks)");
    }
    p->d_afchunks = (const WsAfChunk*)(base + cb);
    return WS_OK;
}

WsLambWs ws_lamb_layout(const ws_plan* p, void* workspace) {
    WsLambWs L;
    char* b = (char*)workspace;
    size_t o = 0;
    L.rho = (float*)(b + o);
    o = round16(o + sizeof(float) * (size_t)p->T);
    L.norms = (double*)(b + o);
    o = round16(o + sizeof(double) * 2 * (size_t)p->T);
    L.partials = (float2*)(b + o);
    o = round16(o + sizeof(float2) * (size_t)(p->layout == WS_LAYOUT_CONCAT ? 1 : p->R) * (size_t)p->ntiles);
    L.ipart = (float2*)(b + o);
    o = round16(o + sizeof(float2) * (size_t)p->n_items);
    const size_t sync0 = o;
    L.count = (int*)(b + o);
    o = (o + sizeof(int) * (size_t)p->T + 7) & ~(size_t)7;
    L.flag = (unsigned long long*)(b + o);
    o += sizeof(unsigned long long) * (size_t)p->T;
    L.ticket = (unsigned long long*)(b + o);
    o += sizeof(unsigned long long);
    L.status = (int*)(b + o);
    o = round16(o + sizeof(int));
    L.sync_bytes = o - sync0;
    L.bytes = o;
    o = (o + 255) & ~(size_t)255;
    L.ghat = (float*)(b + o);
    L.bytes_lars = o + sizeof(float) * (size_t)p->R * (size_t)p->S;
    o = (L.bytes_lars + 255) & ~(size_t)255;
    L.acc = (float*)(b + o);
    const size_t acc0 = o;
    o = (o + sizeof(float) * (size_t)p->Fi + 15) & ~(size_t)15;
    L.rsum = (double*)(b + o);
    o += sizeof(double) * (size_t)p->T;
    L.acc_bytes = o - acc0;
    o = (o + 255) & ~(size_t)255;
    L.fac = (float*)(b + o);
    o = (o + sizeof(float) * (size_t)p->Fi + 255) & ~(size_t)255;
    L.alpha = (float*)(b + o);
    L.bytes_af = o + sizeof(float) * (size_t)p->T;
    return L;
}

extern "C" ws_status ws_workspace_partials(const ws_plan* p, size_t* offset_bytes, size_t* row_bytes) {
    if (!p || !offset_bytes || !row_bytes || p->layout != WS_LAYOUT_PER_TENSOR) return WS_ERR_INVALID_ARG;
    const WsLambWs L = ws_lamb_layout(p, nullptr);
    *offset_bytes = (size_t)((char*)L.partials - (char*)nullptr);
    *row_bytes = sizeof(float2) * (size_t)p->ntiles;
    return WS_OK;
}

extern "C" ws_status ws_workspace_adafactor_sums(const ws_plan* p, size_t* offset_bytes, size_t* bytes) {
    if (!p || !offset_bytes || !bytes) return WS_ERR_INVALID_ARG;
    const WsLambWs L = ws_lamb_layout(p, nullptr);
    *offset_bytes = (size_t)((char*)L.acc - (char*)nullptr);
    *bytes = sizeof(float) * (size_t)p->Fi;
    return WS_OK;
}

extern "C" size_t ws_workspace_bytes(const ws_plan* p, ws_opt opt) {
    if (!p) return 0;
    if (opt == WS_LAMB) return ws_lamb_layout(p, nullptr).bytes;
    if (opt == WS_LARS) return ws_lamb_layout(p, nullptr).bytes_lars;
    if (opt == WS_ADAFACTOR) return ws_lamb_layout(p, nullptr).bytes_af;
    return 0;
}

// ------------------------------------------------------ one-launch schedule ---
// Order of execution for the one-kernel LAMB / LARS update.  Tensors are taken in groups of a few
// megabytes of state; a group's phase-2 items follow its phase-1 items at a distance of at least
// kLag schedule entries (by then every CTA that worked on the group's phase 1 has finished and the
// tensors' ratios are known, so no CTA waits), interleaved one to one with the phase-1 items of the
// following groups: phase 2 then reads w, m', v' out of L2 while phase 1 of the next tensors streams
// from DRAM, and each operand crosses HBM once (Section 2.2).  When more than kLag eligible phase-2
// items are waiting (a tensor larger than L2 has just finished) they run first.
namespace {
constexpr long long kGroupBytes = 6LL << 20;    // state bytes (12 per element) that close a group
constexpr int kLag = 512;

void ws_build_schedule(ws_plan* p) {
    const int T = p->T, R = p->R;
    const bool concat = p->layout == WS_LAYOUT_CONCAT;
    p->items.clear();
    p->items.reserve((size_t)p->n_items);
    p->itemsegs.assign(T, WsItemSeg{0, 0});
    std::vector<long long> seg_bytes(T, 0);
    for (int t = 0; t < T; ++t) {
        p->itemsegs[t].first = (int)p->items.size();
        const WsSegTiles st = p->segtiles[t];
        for (int r = 0; r < (concat ? 1 : R); ++r)
            for (int k = 0; k < st.tile_count; ++k) {
                const WsTile& tl = p->tiles[st.tile_begin + k];
                const long long toff0 = concat ? tl.poff : (long long)r * tl.piece + tl.poff;
                const long long valid0 = concat ? tl.vt : tl.vt - (long long)r * tl.piece;
                for (int so = 0; so < tl.len; so += kWsItemElems) {
                    WsItem it;
                    memset(&it, 0, sizeof(it));
                    const int len = tl.len - so < kWsItemElems ? tl.len - so : kWsItemElems;
                    long long nv = valid0 - so;
                    it.pos = tl.pos + so;
                    it.toff = toff0 + so;
                    it.seg = t;
                    it.nvalid = (int)(nv < 0 ? 0 : (nv > len ? len : nv));
                    it.len = (unsigned short)len;
                    it.shard = (unsigned short)(concat ? tl.shard : r);
                    p->items.push_back(it);
                    seg_bytes[t] += 12LL * len;
                }
            }
        p->itemsegs[t].count = (int)p->items.size() - p->itemsegs[t].first;
    }
    // groups of consecutive tensors
    struct Group { int first, end; };     // item range
    std::vector<Group> groups;
    {
        long long acc = 0;
        int gfirst = 0, t0 = 0;
        for (int t = 0; t < T; ++t) {
            acc += seg_bytes[t];
            const bool last = t == T - 1;
            if (acc >= kGroupBytes || last) {
                const int gend = p->itemsegs[t].first + p->itemsegs[t].count;
                if (gend > gfirst) {
                    groups.push_back(Group{gfirst, gend});
                    // (every group leaves its state in L2 at normal priority: phase 2 reads a group back to
                    // front, so even a tensor many times the L2 finds its last-written part there)
                    const unsigned keep = 1u;
                    for (int i = gfirst; i < gend; ++i) p->items[i].flags = keep;
                }
                gfirst = gend;
                acc = 0;
                t0 = t + 1;
            }
        }
        (void)t0;
    }
    // merge the phase-1 stream and the phase-2 stream
    const long long n = (long long)p->items.size();
    p->sched.clear();
    p->sched.reserve((size_t)(2 * n));
    const int G = (int)groups.size();
    std::vector<long long> p1_done_at(G, -1);     // schedule position of each group's last phase-1 item
    int ag = 0, eg = 0;                           // group of the next phase-1 item; first group not yet eligible
    long long ai = 0, bi = 0;                     // next phase-1 / phase-2 item
    long long eligible = 0;                       // phase-2 items of groups whose phase 1 ended >= kLag entries ago
    int last_kind = 1;
    // phase 2 walks every group back to front: the items phase 1 wrote last are the ones most likely to be
    // in L2 still, and a group larger than the L2 then keeps its tail instead of nothing (reading it front
    // to back would evict each line just before its turn)
    std::vector<unsigned> p2item((size_t)n);
    for (const Group& g : groups)
        for (int i = g.first; i < g.end; ++i) p2item[(size_t)i] = (unsigned)(g.end - 1 - (i - g.first));
    while (bi < n) {
        const long long pos = (long long)p->sched.size();
        while (eg < ag && pos - p1_done_at[eg] >= kLag) {
            eligible += groups[eg].end - groups[eg].first;
            ++eg;
        }
        const long long backlog = eligible - bi;
        const bool may2 = backlog > 0;
        if (ai < n && !(may2 && (last_kind == 0 || backlog > kLag))) {
            p->sched.push_back((unsigned)(ai << 1));
            last_kind = 0;
            if (++ai == groups[ag].end) {
                p1_done_at[ag] = pos;
                ++ag;
            }
        } else {
            // (at the very end the last groups' phase 2 follows their phase 1 directly: the scheduling
            // warps then wait for the ratios, a few microseconds once per launch)
            p->sched.push_back((p2item[(size_t)bi] << 1) | 1u);
            last_kind = 1;
            ++bi;
            if (!may2) eligible = bi;             // keep the backlog arithmetic consistent in the tail
        }
    }
}

size_t schedule_bytes(const ws_plan* p) {
    return round16((size_t)p->n_items * sizeof(WsItem)) + round16((size_t)p->T * sizeof(WsItemSeg)) +
           round16((size_t)p->n_items * 2 * sizeof(unsigned));
}
}  // namespace

extern "C" size_t ws_plan_schedule_bytes(const ws_plan* p) {
    if (!p || p->n_items <= 0) return 0;
    return schedule_bytes(p);
}

extern "C" ws_status ws_plan_upload_schedule(ws_plan* p, void* dev_buf, size_t bytes, void* stream) {
    if (!p || !dev_buf) return WS_ERR_INVALID_ARG;
    if (p->n_items <= 0) return WS_ERR_TOO_LARGE;
    if (!ws_aligned16(dev_buf)) return WS_ERR_ALIGNMENT;
    if (bytes < schedule_bytes(p)) return WS_ERR_WORKSPACE;
    try {
        if (p->sched.empty()) ws_build_schedule(p);
    } catch (...) {
        return WS_ERR_INVALID_ARG;
    }
    if ((long long)p->items.size() != p->n_items) return WS_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    char* base = (char*)dev_buf;
    const size_t ib = (size_t)p->n_items * sizeof(WsItem), sb = (size_t)p->T * sizeof(WsItemSeg);
    cudaError_t e = cudaMemcpyAsync(base, p->items.data(), ib, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return ws_cuda_fail(e, "ws_plan_upload_schedule(items)");
    e = cudaMemcpyAsync(base + round16(ib), p->itemsegs.data(), sb, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return ws_cuda_fail(e, "ws_plan_upload_schedule(tensor ranges)");
    e = cudaMemcpyAsync(base + round16(ib) + round16(sb), p->sched.data(), p->sched.size() * sizeof(unsigned),
                        cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return ws_cuda_fail(e, "ws_plan_upload_schedule(order)");
    p->d_items = (const WsItem*)base;
    p->d_itemsegs = (const WsItemSeg*)(base + round16(ib));
    p->d_sched = (const unsigned*)(base + round16(ib) + round16(sb));
    return WS_OK;
}

extern "C" ws_status ws_plan_schedule_view(ws_plan* p, const uint32_t** order, int64_t* n_entries) {
    if (!p || !order || !n_entries) return WS_ERR_INVALID_ARG;
    if (p->n_items <= 0) return WS_ERR_TOO_LARGE;
    try {
        if (p->sched.empty()) ws_build_schedule(p);
    } catch (...) {
        return WS_ERR_INVALID_ARG;
    }
    *order = p->sched.data();
    *n_entries = (int64_t)p->sched.size();
    return WS_OK;
}

extern "C" ws_status ws_plan_schedule_item(ws_plan* p, int64_t item, ws_sched_item* out) {
    if (!p || !out) return WS_ERR_INVALID_ARG;
    if (p->n_items <= 0) return WS_ERR_TOO_LARGE;
    try {
        if (p->sched.empty()) ws_build_schedule(p);
    } catch (...) {
        return WS_ERR_INVALID_ARG;
    }
    if (item < 0 || item >= p->n_items) return WS_ERR_INVALID_ARG;
    const WsItem& it = p->items[(size_t)item];
    out->tensor = it.seg;
    out->shard = it.shard;
    out->pos = it.pos;
    out->tensor_off = it.toff;
    out->len = it.len;
    out->nvalid = it.nvalid;
    return WS_OK;
}

extern "C" ws_status ws_workspace_sync_status(const ws_plan* p, size_t* offset_bytes) {
    if (!p || !offset_bytes) return WS_ERR_INVALID_ARG;
    const WsLambWs L = ws_lamb_layout(p, nullptr);
    *offset_bytes = (size_t)((char*)L.status - (char*)nullptr);
    return WS_OK;
}
