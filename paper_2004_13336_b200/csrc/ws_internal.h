// Internal declarations shared by the translation units of libws.so.
// Nothing here is part of the public ABI (see include/ws.h).
#pragma once
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>
#include <stdint.h>

#include <vector>

#include "ws.h"

// A named range around an entry point for timeline tools (NVTX; costs a few nanoseconds when no tool
// is attached).  Covers the host side of the call: argument checks and launches.
struct WsRange {
    explicit WsRange(const char* name) { nvtxRangePushA(name); }
    ~WsRange() { nvtxRangePop(); }
    WsRange(const WsRange&) = delete;
    WsRange& operator=(const WsRange&) = delete;
};

// One work tile: a run of at most `tile_elems` consecutive shard positions that
// lies inside one tensor's piece.  A tile carries everything a kernel needs to
// address and mask its elements, so the kernels never search the segment table.
//   shard position of element e of the tile : pos + e
//   index of that element in tensor `seg`    : r*piece + poff + e      (shard r)
//   it exists in the tensor iff              : e < vt - r*piece
// Per-tensor layout: one tile list serves every shard r.  Concatenated layout: every shard
// has its own tiles (`shard` says which), piece is 0 and poff / vt are absolute.
struct __align__(16) WsTile {
    long long pos;    // start inside a shard, multiple of 8
    long long vt;     // numel - poff: valid elements from the tile start in shard 0
    long long piece;  // p_t
    long long poff;   // pos - off_t: start inside the piece
    int len;          // elements in the tile, multiple of 8, <= tile_elems
    int seg;          // tensor index t
    int shard;        // concatenated layout only: the shard this tile lies in
    int pad1;
};
static_assert(sizeof(WsTile) == 48, "WsTile is read as three 16-byte words");

// Per tensor: which tiles of a shard belong to it (contiguous range).
struct WsSegTiles {
    int tile_begin;
    int tile_count;
};

// Adafactor's view of a tensor: foff = start of its factored state (floats); nrow row
// accumulators (0 for an unfactored tensor) followed by ncol column accumulators (the full
// second moment for an unfactored tensor, which is handled as a single row).
struct WsSegAf {
    long long foff;
    long long nrow;
    long long ncol;
    long long numel;
    // the workspace arrays (this step's sums, the 1/sqrt factors) use a padded layout so that a
    // thread's run of columns can be moved as one vector: row part and column part each start on
    // a multiple of 8 floats
    long long irow;
    long long icol;
};

// The finalize steps walk the factored state in chunks of at most 1024 entries (one CTA each).
struct WsAfChunk {
    long long begin;   // first entry inside tensor seg's state (0 .. nrow + ncol)
    int count;
    int seg;
};

// One-launch schedule of the norm-based optimizers (LAMB, LARS): the update of all shards as ONE
// kernel.  A work item is a run of at most kWsItemElems consecutive shard positions inside
// one tile; every item appears twice in the schedule, once for phase 1 (reduce, moments, partial
// norm sums) and once for phase 2 (apply the step with the tensor's ratio).
constexpr int kWsItemElems = 8192;
struct __align__(16) WsItem {
    long long pos;        // start inside the shard, multiple of 8
    long long toff;       // element index of the first element inside tensor `seg`
    int seg;              // tensor index
    int nvalid;           // elements of the item that exist in the tensor (the rest is padding)
    unsigned short len;   // elements, multiple of 8
    unsigned short shard;
    unsigned flags;       // bit 0: the tensor group is small enough to stay in L2 between its phases
};
static_assert(sizeof(WsItem) == 32, "WsItem is read as two 16-byte words");
// Items are numbered tensor by tensor (then shard by shard), so a tensor's items - and with them its
// partial norm sums - are one contiguous range.
struct WsItemSeg {
    int first;
    int count;
};

struct ws_plan {
    int T = 0, R = 0, A = 0, K = 0;
    int layout = 0;                           // ws_layout
    long long S = 0, N = 0;
    long long ntiles = 0;                     // per-tensor layout: tiles per shard; concatenated: all tiles
    std::vector<long long> shard_tile_begin;  // concatenated layout: [R+1] first tile of every shard
    std::vector<ws_segment> segs;
    std::vector<WsTile> tiles;
    std::vector<WsSegTiles> segtiles;
    // tensor arena: tensors back to back, each start rounded up to 8 elements
    std::vector<long long> arena_off;
    long long arena_elems = 0;
    // device copies (caller-owned memory, set by ws_plan_upload)
    const WsTile* d_tiles = nullptr;
    const WsSegTiles* d_segtiles = nullptr;
    std::vector<WsSegAf> segaf;
    std::vector<WsAfChunk> afchunks;
    long long F = 0;                          // total factored-state floats
    long long Fi = 0;                         // floats of the padded workspace layout
    const WsSegAf* d_segaf = nullptr;
    const WsAfChunk* d_afchunks = nullptr;
    // one-launch schedule: counted at creation, built and uploaded by ws_plan_upload_schedule
    long long n_items = 0;                    // work items (0: the plan has no one-launch schedule)
    std::vector<WsItem> items;
    std::vector<WsItemSeg> itemsegs;          // [T]
    std::vector<unsigned> sched;              // [2 n_items]: item index * 2 + phase, in execution order
    const WsItem* d_items = nullptr;
    const WsItemSeg* d_itemsegs = nullptr;
    const unsigned* d_sched = nullptr;
};

// Optimizer constants narrowed to fp32 for the kernels.
struct WsConsts {
    float lr, beta1, omb1, beta2, omb2, eps, wd, mu, gscale, inv_bc1, inv_bc2;
};

// LAMB workspace layout (see ws_workspace_bytes in ws.h).
struct WsLambWs {
    float* rho;        // [T]
    double* norms;     // [T][2]
    float2* partials;  // [R][ntiles]
    // one-launch update: per-item partial sums, per-tensor arrival counters and ready flags, the
    // ticket counter and the status word (sync_bytes from `count` on are cleared before every launch)
    float2* ipart;     // [n_items]
    int* count;        // [T]
    unsigned long long* flag;   // [T] ready words
    unsigned long long* ticket;
    int* status;
    size_t sync_bytes; // from count on
    size_t bytes;      // through the one-launch scratch: what LAMB needs
    float* ghat;       // LARS only: [R][S] summed gradients, 256-byte aligned after the partials
    size_t bytes_lars; // through ghat: what LARS needs
    float* acc;        // Adafactor: [Fi] this step's row / column sums (padded layout)
    double* rsum;      // Adafactor: [T] sum of the new row accumulators, directly after acc
    size_t acc_bytes;  // acc and rsum together: cleared at the start of every step
    float* fac;        // Adafactor: [Fi] 1/sqrt factors of V (padded layout)
    float* alpha;      // Adafactor: [T] step sizes
    size_t bytes_af;   // through alpha: what Adafactor needs
};
WsLambWs ws_lamb_layout(const ws_plan* plan, void* workspace);

// Argument checks of LAMB's apply phase for an all-shard call, with no launch (so that a sequence of
// launches can refuse bad arguments before its first one).
ws_status ws_lamb_check_apply_args(const ws_plan* plan, const ws_state* state, const ws_hyper* hyper, const ws_out* out);

// Debug build (-DWS_DEBUG_BOUNDS): before a kernel touches a work item it compares the item's range
// with the extents of the buffers it was given; a range outside them sets a bit in a status word that
// the caller can read (ws_debug_bounds_read) and the item is skipped - no trap, no assert, no access.
enum {
    WS_BOUNDS_STATE = 1,      // w / m / v
    WS_BOUNDS_GRAD = 2,       // a packed gradient buffer
    WS_BOUNDS_OUT = 4,        // the gathered buffer or the stored gradient sum
    WS_BOUNDS_FLAT = 8,       // the flat buffer of ws_pack / ws_unpack
    WS_BOUNDS_SELFTEST = 0x40000000
};
#ifdef WS_DEBUG_BOUNDS
unsigned* ws_bounds_word();   // device address of the status word on the current device, or null
#endif

// error bookkeeping
ws_status ws_cuda_fail(cudaError_t e, const char* what);
ws_status ws_check_launch(const char* what);

static inline bool ws_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
