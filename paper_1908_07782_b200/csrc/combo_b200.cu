// libcombo_b200.so: C ABI over the sm_100a kernels (argument checks, tile
// planning, launches).  See include/combo_b200.h for the contract.
#include "../../include/combo_b200.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include "segment_aggregate.cuh"
#include "divergence.cuh"
#include "select_peers.cuh"
#include "pull_aggregate.cuh"

namespace {

using combo::AggParams;

thread_local char t_cuda_err[256] = "";
thread_local int t_last_path = 0;
thread_local int t_force_path = 0;
thread_local int t_tile = 0;
thread_local int t_stages = 0;
thread_local int t_overlap = 1;
#ifndef COMBO_DENSE_MAX
#define COMBO_DENSE_MAX 32
#endif
constexpr int kDenseMaxWorkers = COMBO_DENSE_MAX;   // most workers the dense evaluation of many replicas is chosen for
constexpr long long kTileMaxCtas = 1LL << 18;   // largest grid the one-tile-per-CTA kernel is chosen for

struct DeviceInfo {
    int known;       // 0 unknown, 1 supported, -1 unsupported
    int sms;
    int smem_optin;
    int smem_per_sm;
};
DeviceInfo g_dev[64];

combo_status cuda_fail(cudaError_t e, const char* what) {
    snprintf(t_cuda_err, sizeof(t_cuda_err), "%s: %s", what, cudaGetErrorString(e));
    return COMBO_ERR_CUDA;
}

combo_status device_info(DeviceInfo** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= 64) return COMBO_ERR_UNSUPPORTED;
    DeviceInfo& d = g_dev[dev];
    if (d.known == 0) {
        int major = 0, sms = 0, smem = 0, smem_sm = 0;
        if ((e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev)) != cudaSuccess ||
            (e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess ||
            (e = cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) != cudaSuccess ||
            (e = cudaDeviceGetAttribute(&smem_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev)) != cudaSuccess)
            return cuda_fail(e, "cudaDeviceGetAttribute");
        d.sms = sms;
        d.smem_optin = smem;
        d.smem_per_sm = smem_sm;
        d.known = (major == 10) ? 1 : -1;
    }
    if (d.known < 0) return COMBO_ERR_UNSUPPORTED;
    *out = &d;
    return COMBO_OK;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline bool overlaps(const void* a, const void* b, size_t bytes) {
    uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
    return x < y + bytes && y < x + bytes;
}

inline unsigned round_up(unsigned v, unsigned q) { return (v + q - 1) / q * q; }

// ---------------------------------------------------------------- tile dispensers
// Launches of the staged kernel take the slots of combo::g_tile_slots in turn.  A slot is
// zero when idle (the kernel's last CTA resets it), so launches that overlap on the device
// only need different slots: 256 of them cover any number of kernels that can be resident.
combo::TileSlot* g_slot_base[64];
unsigned g_slot_seq[2] = {0, 0};      // [0] ordinary launches, [1] launches being captured into a graph

combo_status next_tile_slot(combo::TileSlot** out, cudaStream_t st) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= 64) return COMBO_ERR_UNSUPPORTED;
    if (!g_slot_base[dev]) {
        combo::TileSlot* ptr = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), combo::g_tile_slots);
        if (e != cudaSuccess || !ptr) return cuda_fail(e, "cudaGetSymbolAddress(tile slots)");
        g_slot_base[dev] = ptr;
    }
    // A graph keeps the slots its kernels were captured with for as long as it is replayed,
    // while ordinary launches move on through the ring: the two kinds draw from separate
    // halves, so that a replay running beside ordinary launches never meets them on a slot.
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) { cudaGetLastError(); cap = cudaStreamCaptureStatusNone; }
    const int kind = cap == cudaStreamCaptureStatusActive ? 1 : 0;
    const unsigned half = combo::kTileSlots / 2;
    const unsigned seq = __atomic_fetch_add(&g_slot_seq[kind], 1u, __ATOMIC_RELAXED);
    *out = g_slot_base[dev] + kind * half + (seq % half);
    return COMBO_OK;
}

// ---------------------------------------------------------------- staged plan
struct StagedPlan {
    bool ok;
    int gb;          // shared-memory read granule in bytes
    int rt;          // R the kernel is specialised on, or -1
    size_t smem;
    int grid;
    bool unw;        // bfloat16 rows with unit weights: the mixed-precision sum (see RowCtxU)
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

int gcd_int(long long a, long long b) { while (b) { long long t = a % b; a = b; b = t; } return (int)a; }

// Tensor map of row class j of one [N][pitch] array: origin = start of row j rounded down
// to 16 bytes, x extent up to the last local column, rows m*pitch apart.
bool encode_class_map(CUtensorMap* map, const unsigned char* base, int EB, int j, int m, int N, long long pitch,
                      long long width, int box_w) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    const long long pitch_bytes = pitch * EB;
    const long long row0 = (long long)j * pitch_bytes;
    const long long phase = row0 & 15;
    const int rows = (N - j + m - 1) / m;
    cuuint64_t dims[2] = {(cuuint64_t)(phase / EB + width), (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)((long long)m * pitch_bytes)};
    cuuint32_t box[2] = {(cuuint32_t)box_w, (cuuint32_t)rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(map, EB == 4 ? CU_TENSOR_MAP_DATA_TYPE_UINT32 : CU_TENSOR_MAP_DATA_TYPE_UINT16, 2,
                     const_cast<unsigned char*>(base) + row0 - phase, dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(t_cuda_err, sizeof(t_cuda_err), "cuTensorMapEncodeTiled failed with %d", (int)r);
        return false;
    }
    return true;
}

StagedPlan plan_staged(AggParams& p, combo::TileMaps& maps, int EB, bool sgd, const DeviceInfo& dev) {
    StagedPlan plan = {false, 16, -1, 0, 0, false};
    const int V = 16 / EB;
    const int narr = sgd ? 2 : 1;
    if (p.R > combo::kStagedMaxR) return plan;
    const long long pitch_bytes = p.pitch * EB;
    const int m = 16 / gcd_int(16, pitch_bytes % 16 == 0 ? 16 : pitch_bytes % 16);
    const bool unaligned = m > 1;
    if ((p.N + m - 1) / m > 256) return plan;                       // box rows
    if ((unsigned long long)m * (unsigned long long)pitch_bytes >= (1ull << 40)) return plan;
    if ((unsigned long long)p.width + 256 >= (1ull << 31)) return plan;   // TMA coordinates are signed 32-bit
    plan.gb = !unaligned ? 16 : (EB == 4 ? 4 : ((p.pitch % 2 == 0) ? 4 : 2));
    // the kernel is specialised on R for 1..4 and 8 (the values Section 5.2 sweeps, with 16)
    // except on the rarely used granules
    plan.rt = (((p.R >= 1 && p.R <= 4) || p.R == 8) && (plan.gb == 16 || (EB == 2 && plan.gb == 4))) ? p.R : -1;
    if (p.R > combo::kGenericR) plan.rt = -2;                       // the wide unspecialised kernel
    // Many replicas among few workers (Section 5.2 sweeps R to 16 with 30 workers): whole tiles
    // are evaluated densely, a block of output rows against all N staged rows, which reads
    // each staged piece once per block instead of once per provider.  Measured with 30 workers
    // of 11.7 M floats, S = 10: 0.66 of the peak for every R from 9 to 16, against 0.64 / 0.59 /
    // 0.53 at R = 9 / 12 / 16 in the warp-per-row form (bfloat16: 0.39 against 0.35 / 0.30 /
    // 0.24); with 40 and 48 workers at R = 12 the warp-per-row form wins (0.50 / 0.55 against
    // 0.46 / 0.45), hence the limit of 32.  Needs rows of one 16-byte phase and every row
    // readable (no newcomer).
    bool any_newcomer = false;
    for (int i = 0; i < 256; ++i) any_newcomer |= p.newcomer.w[i] != 0;
    const bool dense = plan.rt == -2 && plan.gb == 16 && !any_newcomer && p.N <= kDenseMaxWorkers;
    if (dense) plan.rt = -3;
    const int rmax = combo::rmax_of(plan.rt);
    plan.unw = EB == 2 && !p.weights && !sgd && !dense && plan.gb != 2;
    const unsigned header = round_up((unsigned)sizeof(combo::StagedHeader), 128);
    // the coefficient table holds every segment when that is small (no rebuilds on the way,
    // which matters for short kernels), else two segments at a time
    const int dense_br = EB == 4 ? 8 : 4;
    const unsigned dslot = dense ? round_up((unsigned)((p.N + dense_br - 1) / dense_br * (p.N + 2) * dense_br * 4), 128) : 0;
    const unsigned entry = (unsigned)(plan.unw ? combo::entry_unw_bytes(rmax) : combo::table_entry_bytes(rmax));
    const unsigned long long slot_bytes = (unsigned long long)p.N * entry + dslot;
    int tab_slots = ((unsigned long long)p.S * slot_bytes <= 24u * 1024u && p.S >= 2) ? p.S : 2;
    unsigned table = round_up((unsigned)tab_slots * p.N * entry, 128) + (unsigned)tab_slots * dslot;
    const long long budget = (long long)dev.smem_optin - header - table - 256;

    // candidate tiles: (T, box_w, nbx)
    struct Cand { int T, box_w, nbx; };
    Cand cands[combo::kMaxBoxes + 3];
    int nc = 0;
    if (unaligned) {
        // every box carries 256 - V columns of the tile plus room for the row phase
        for (int n = 1; n <= combo::kMaxBoxes; ++n) cands[nc++] = {(256 - V) * n, 256, n};
    } else {
        // with very many rows two stages of 256 columns do not fit: narrower boxes (512 or 256
        // bytes per row) keep such inputs on the staged path
        if (EB == 4) cands[nc++] = {64, 64, 1};
        cands[nc++] = {128, 128, 1};
        for (int n = 1; n <= combo::kMaxBoxes; ++n) cands[nc++] = {256 * n, 256, n};
    }
    auto stage_bytes = [&](const Cand& c) { return (long long)narr * c.nbx * p.N * c.box_w * EB; };
    auto tiles = [&](const Cand& c) { return (p.width + c.T - 1) / c.T; };
    auto feasible = [&](const Cand& c) {
        return (long long)c.T <= p.L && 2 * stage_bytes(c) <= budget && narr * c.nbx * m <= 32;
    };
    int pick = -1;
    if (t_tile > 0) {
        for (int i = 0; i < nc; ++i)
            if ((unaligned ? cands[i].nbx * 256 == t_tile : cands[i].T == t_tile) && feasible(cands[i])) pick = i;
        if (pick < 0) return plan;
    } else {
        // Long kernels: the widest tile whose stage stays within 64 KB.  Short kernels (fewer
        // than 32 such tiles per CTA, i.e. up to some hundred microseconds): the widest tile
        // whose stage stays within 32 KB -- they spend a good part of their time filling and
        // draining the ring, which narrower stages do faster, and tiles are handed out
        // dynamically, which balances better with more of them.  (Measured on shapes from
        // 8 x 256 K to 16 x 1 M floats: the 32 KB choice was the best or within 1 % of it;
        // 8 x 1 M: 14.4 us with 64 KB stages, 13.5 us with 32 KB.)  Boxes narrower than 256
        // columns are the last resort: the widest of them that fits.
        int wide = -1, mid = -1, narrowest = -1, narrow_box = -1;
        for (int i = 0; i < nc; ++i) {
            if (!feasible(cands[i])) continue;
            if (cands[i].box_w < 256) { narrow_box = i; continue; }
            if (narrowest < 0) narrowest = i;
            if (stage_bytes(cands[i]) <= 64 * 1024) wide = i;
            if (stage_bytes(cands[i]) <= 32 * 1024) mid = i;
        }
        pick = wide >= 0 ? wide : narrowest;
        if (wide >= 0 && tiles(cands[wide]) < 32LL * dev.sms && mid >= 0) pick = mid;
        if (pick < 0) pick = narrow_box;
        if (pick < 0) return plan;
    }
    const Cand c = cands[pick];
    if (plan.rt == -3 && c.box_w != 256) plan.rt = -2;   // the dense form walks whole 512-byte chunks of 256-column boxes
    // Measured on B200: throughput peaks with about 128-160 KB of staged data per SM (the stage
    // being consumed included) and drops by up to 5-10 % beyond that on some GPUs, so the ring is
    // kept that short: two stages of 64 KB, else as many as stay within 160 KB (48 rows of
    // binary32, 48 KB stages: 0.93 with two, 0.97 with three; 40 rows: 0.89 / 0.97; a third
    // stage of 64 KB gave +2 % to -1.6 % depending on shape and GPU).
    const int fit = (int)(budget / stage_bytes(c));
    int stages = (int)(((stage_bytes(c) < 64 * 1024 ? 160 : 128) * 1024) / stage_bytes(c));
    if (stages < 2) stages = 2;
    if (t_stages > 0) stages = t_stages;
    if (stages > combo::kMaxStages) stages = combo::kMaxStages;
    if (stages > fit) stages = fit;
    if (stages < 2) return plan;
    // a larger table that still fits beside the stages chosen is taken whole as well (a rebuild
    // costs two consumer barriers and a round trip to the peer table: it shows in kernels of
    // a hundred microseconds with many segments)
    if (tab_slots < p.S) {
        const unsigned long long whole = round_up((unsigned)((unsigned long long)p.S * p.N * entry), 128) +
                                         (unsigned long long)p.S * dslot;
        if ((unsigned long long)p.S * slot_bytes < (1u << 20) &&
            (long long)(whole - table) <= budget - (long long)stages * stage_bytes(c)) {
            tab_slots = p.S;
            table = (unsigned)whole;
        }
    }
    p.T = c.T;
    p.m = m;
    p.nbx = c.nbx;
    p.box_w = c.box_w;
    p.stages = stages;
    p.row_bytes = c.box_w * EB;
    p.stage_bytes = (unsigned)stage_bytes(c);
    p.tab_off = header;
    p.tab_slots = tab_slots;
    p.dtab_off = header + round_up((unsigned)tab_slots * p.N * entry, 128);
    p.dslot_bytes = (int)dslot;
    p.stage_off = header + table;
    p.n_tiles = tiles(c);
    for (int a = 0; a < narr; ++a)
        for (int j = 0; j < m && j < p.N; ++j)
            if (!encode_class_map(&maps.map[a][j], a == 0 ? p.in : p.grads, EB, j, m, p.N, p.pitch, p.width,
                                  c.box_w))
                return plan;
    // 16 bytes of slack: unmasked reads of a ragged item may run a row phase past the last row
    plan.smem = (size_t)p.stage_off + (size_t)stages * p.stage_bytes + 16;
    plan.grid = (int)(p.n_tiles < dev.sms ? p.n_tiles : dev.sms);
    plan.ok = plan.grid > 0;
    return plan;
}

template <int EB, int GB, bool SGD, int RT, bool UNW = false>
cudaError_t launch_staged_inst(const AggParams& p, const combo::TileMaps& maps, const StagedPlan& plan,
                               cudaStream_t st) {
    auto kern = combo::k_staged<EB, GB, SGD, RT, UNW>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem);
    if (e != cudaSuccess) return e;
    // Programmatic stream serialization: the kernel may be scheduled while the preceding
    // kernel of the stream drains (it waits for that kernel's completion itself, before its
    // first global access), which hides launch latency and set-up between back-to-back rounds.
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)plan.grid);
    cfg.blockDim = dim3((unsigned)combo::kStagedThreads);
    cfg.dynamicSmemBytes = plan.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = t_overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, p, maps);
}

template <int EB, int GB, bool SGD>
cudaError_t launch_staged_r(const AggParams& p, const combo::TileMaps& maps, const StagedPlan& plan,
                            cudaStream_t st) {
    switch (plan.rt) {
        case 1: return launch_staged_inst<EB, GB, SGD, 1>(p, maps, plan, st);
        case 2: return launch_staged_inst<EB, GB, SGD, 2>(p, maps, plan, st);
        case 3: return launch_staged_inst<EB, GB, SGD, 3>(p, maps, plan, st);
        case 4: return launch_staged_inst<EB, GB, SGD, 4>(p, maps, plan, st);
        case 8: return launch_staged_inst<EB, GB, SGD, 8>(p, maps, plan, st);
        case -2: return launch_staged_inst<EB, GB, SGD, -2>(p, maps, plan, st);
        case -3: return launch_staged_inst<EB, GB, SGD, -3>(p, maps, plan, st);
        default: return launch_staged_inst<EB, GB, SGD, -1>(p, maps, plan, st);
    }
}

template <int EB, int GB, bool SGD>
cudaError_t launch_staged_generic(const AggParams& p, const combo::TileMaps& maps, const StagedPlan& plan,
                                  cudaStream_t st) {
    if (plan.rt == -2) return launch_staged_inst<EB, GB, SGD, -2>(p, maps, plan, st);
    return launch_staged_inst<EB, GB, SGD, -1>(p, maps, plan, st);
}

// bfloat16 rows with unit weights
template <int GB>
cudaError_t launch_staged_unw(const AggParams& p, const combo::TileMaps& maps, const StagedPlan& plan,
                              cudaStream_t st) {
    switch (plan.rt) {
        case 1: return launch_staged_inst<2, GB, false, 1, true>(p, maps, plan, st);
        case 2: return launch_staged_inst<2, GB, false, 2, true>(p, maps, plan, st);
        case 3: return launch_staged_inst<2, GB, false, 3, true>(p, maps, plan, st);
        case 4: return launch_staged_inst<2, GB, false, 4, true>(p, maps, plan, st);
        case 8: return launch_staged_inst<2, GB, false, 8, true>(p, maps, plan, st);
        case -2: return launch_staged_inst<2, GB, false, -2, true>(p, maps, plan, st);
        default: return launch_staged_inst<2, GB, false, -1, true>(p, maps, plan, st);
    }
}

cudaError_t launch_staged(const AggParams& p, const combo::TileMaps& maps, const StagedPlan& plan, int EB, bool sgd,
                          cudaStream_t st) {
    if (EB == 4) {
        if (plan.gb == 16) return sgd ? launch_staged_r<4, 16, true>(p, maps, plan, st)
                                      : launch_staged_r<4, 16, false>(p, maps, plan, st);
        return sgd ? launch_staged_generic<4, 4, true>(p, maps, plan, st)
                   : launch_staged_generic<4, 4, false>(p, maps, plan, st);
    }
    if (plan.unw) return plan.gb == 16 ? launch_staged_unw<16>(p, maps, plan, st) : launch_staged_unw<4>(p, maps, plan, st);
    if (plan.gb == 16) return launch_staged_r<2, 16, false>(p, maps, plan, st);
    if (plan.gb == 4) return launch_staged_r<2, 4, false>(p, maps, plan, st);
    return launch_staged_generic<2, 2, false>(p, maps, plan, st);
}

// Plan of the one-tile-per-CTA kernel (k_tile): rows that share one 16-byte phase only, one
// stage, a table of two segments.  `short_enough` tells whether the automatic choice should
// take it (few rows: small tiles, many CTAs per SM).
StagedPlan plan_tile(AggParams& p, combo::TileMaps& maps, int EB, bool sgd, const DeviceInfo& dev,
                     bool* short_enough) {
    StagedPlan plan = {false, 16, -1, 0, 0, false};
    *short_enough = false;
    const int V = 16 / EB;
    const int narr = sgd ? 2 : 1;
    if (p.R > combo::kStagedMaxR) return plan;
    if ((p.pitch * EB) % 16 != 0) return plan;                      // one row class only
    if (p.N > 256) return plan;                                     // box rows
    if ((unsigned long long)p.pitch * EB >= (1ull << 40)) return plan;
    if ((unsigned long long)p.width + 256 >= (1ull << 31)) return plan;   // TMA coordinates are signed 32-bit
    plan.rt = ((p.R >= 1 && p.R <= 4) || p.R == 8) ? p.R : -1;
    if (p.R > combo::kGenericR) plan.rt = -2;
    const int rmax = combo::rmax_of(plan.rt);
    const unsigned header = round_up((unsigned)sizeof(combo::StagedHeader), 128);
    const unsigned table = round_up(2u * p.N * (unsigned)combo::table_entry_bytes(rmax), 128);
    // Tile: at least 1 KB of every row (256 binary32 or 512 bfloat16 columns; shorter row
    // pieces cost HBM efficiency) and as close to 16 KB in all as it gets from below: the
    // smaller the tile, the more CTAs share an SM and the finer the hand-over between
    // consecutive launches, but every tile pays its set-up once (measured: 8 rows of 1 M
    // floats take 13.1 us with 8 KB tiles, 12.5 with 16 KB, 13.5 with 24 KB; 4 rows of 4 M
    // 36.8 / 25.1 / 24.6 us with 4 / 8 / 12 KB; 2 rows of 4 M 29.4 / 17.4 / 14.1 us with
    // 2 / 4 / 6 KB; 16 rows of 1 M 23.6 / 24.6 us with 16 / 32 KB).  t_tile overrides.
    int nbx = 0;
    for (int n = 1; n <= combo::kMaxBoxes; ++n) {
        if (256LL * n > p.L || narr * n > 32) break;
        if (t_tile > 0) {
            if (256 * n == t_tile) nbx = n;
            continue;
        }
        // the widest tile of at most 16 KB, but never less than 1 KB of a row
        if (nbx > 0 && 256 * nbx * EB >= 1024 && (long long)narr * n * p.N * 256 * EB > 16 * 1024) break;
        nbx = n;
    }
    if (nbx == 0) return plan;
    const long long stage = (long long)narr * nbx * p.N * 256 * EB;
    const size_t smem = (size_t)header + table + (size_t)stage + 16;
    if ((long long)smem > dev.smem_optin) return plan;
    p.T = 256 * nbx;
    p.m = 1;
    p.nbx = nbx;
    p.box_w = 256;
    p.stages = 1;
    p.row_bytes = 256 * EB;
    p.stage_bytes = (unsigned)stage;
    p.tab_off = header;
    p.tab_slots = 2;
    p.stage_off = header + table;
    p.n_tiles = (p.width + p.T - 1) / p.T;
    if (p.n_tiles > 0x7fffffffLL) return plan;
    for (int a = 0; a < narr; ++a)
        if (!encode_class_map(&maps.map[a][0], a == 0 ? p.in : p.grads, EB, 0, 1, p.N, p.pitch, p.width, 256))
            return plan;
    plan.smem = smem;
    plan.grid = (int)p.n_tiles;
    plan.ok = plan.grid > 0;
    (void)V;
    // Taken automatically where it measured faster than the persistent kernel's ring: tiles of
    // 8 to 24 KB (up to 24 rows), which let nine or more CTAs share an SM, and at most two
    // replicas.  (8 x 1 M floats, R = 2: 12.5 us against 13.6; 16 x 1 M: 23.5 against 24.4;
    // 24 x 1 M: 34.1 against 35.3; 2 x 64 M, R = 1: 163 against 260; 8 x 64 M: 635 against 638.
    // With R = 3 or 4 the ring wins by 2 to 10 %, with 32 and more rows it is as good or
    // better, bfloat16 tiles of 8 KB lose 5 %.)
    *short_enough = stage >= 8 * 1024 && stage <= 24 * 1024 && p.R <= 2 && (EB == 4 || stage >= 16 * 1024) &&
                    p.n_tiles <= kTileMaxCtas;
    return plan;
}

template <int EB, bool SGD, int RT>
cudaError_t launch_tile_inst(const AggParams& p, const combo::TileMaps& maps, const StagedPlan& plan,
                             cudaStream_t st) {
    auto kern = combo::k_tile<EB, 16, SGD, RT>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)plan.grid);
    cfg.blockDim = dim3((unsigned)combo::kTileThreads);
    cfg.dynamicSmemBytes = plan.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = t_overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, p, maps);
}

template <int EB, bool SGD>
cudaError_t launch_tile_r(const AggParams& p, const combo::TileMaps& maps, const StagedPlan& plan,
                          cudaStream_t st) {
    switch (plan.rt) {
        case 1: return launch_tile_inst<EB, SGD, 1>(p, maps, plan, st);
        case 2: return launch_tile_inst<EB, SGD, 2>(p, maps, plan, st);
        case 3: return launch_tile_inst<EB, SGD, 3>(p, maps, plan, st);
        case 4: return launch_tile_inst<EB, SGD, 4>(p, maps, plan, st);
        case 8: return launch_tile_inst<EB, SGD, 8>(p, maps, plan, st);
        case -2: return launch_tile_inst<EB, SGD, -2>(p, maps, plan, st);
        default: return launch_tile_inst<EB, SGD, -1>(p, maps, plan, st);
    }
}

cudaError_t launch_tile(const AggParams& p, const combo::TileMaps& maps, const StagedPlan& plan, int EB, bool sgd,
                        cudaStream_t st) {
    if (EB == 4) return sgd ? launch_tile_r<4, true>(p, maps, plan, st) : launch_tile_r<4, false>(p, maps, plan, st);
    return launch_tile_r<2, false>(p, maps, plan, st);
}

cudaError_t launch_direct(const AggParams& p, int EB, bool sgd, const DeviceInfo& dev, cudaStream_t st,
                          bool worker_major) {
    const int V = 16 / EB;
    const long long groups = (p.width + V - 1) / V + 1;
    const long long blocks_per_row = (groups + 255) / 256;
    const long long total = blocks_per_row * p.N;
    // persistent CTAs, eight per SM, that take the blocks in their numbered order
    const long long cap = (long long)dev.sms * 8;
    const unsigned grid = (unsigned)(total < cap ? total : cap);
    const int wm = worker_major ? 1 : 0;
    const size_t smem = (size_t)(p.R + 1) * 16;          // providers and coefficients of two segments
    cudaError_t e = cudaSuccess;
    if (EB == 4) {
        if (sgd) {
            if (smem > 48 * 1024) e = cudaFuncSetAttribute(combo::k_direct<4, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e == cudaSuccess) combo::k_direct<4, true><<<grid, 256, smem, st>>>(p, blocks_per_row, wm);
        } else {
            if (smem > 48 * 1024) e = cudaFuncSetAttribute(combo::k_direct<4, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e == cudaSuccess) combo::k_direct<4, false><<<grid, 256, smem, st>>>(p, blocks_per_row, wm);
        }
    } else {
        if (smem > 48 * 1024) e = cudaFuncSetAttribute(combo::k_direct<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess) combo::k_direct<2, false><<<grid, 256, smem, st>>>(p, blocks_per_row, wm);
    }
    return e != cudaSuccess ? e : cudaGetLastError();
}

// widest column range one launch takes: a multiple of 64 elements (shards start on 16-byte
// boundaries) that keeps every TMA coordinate, box width included, below 2^31
constexpr long long kMaxShardColumns = 1LL << 30;
thread_local long long t_shard_columns = kMaxShardColumns;

combo_status aggregate_cols(const void* in, const void* grads, float lr, void* out, int EB,
                            const float* weights, const int32_t* idx, int N, long long P_total, int S, int R,
                            long long p_begin, long long width, long long pitch, void* stream,
                            const uint8_t* h_newcomer = nullptr) {
    if (EB != 4 && EB != 2) return COMBO_ERR_INVALID_ARG;
    if (N < 1 || N > COMBO_MAX_WORKERS || S < 1 || S > COMBO_MAX_SEGMENTS || R < 0 || R > N - 1)
        return COMBO_ERR_INVALID_ARG;
    if (P_total < 1 || p_begin < 0 || width < 1 || p_begin + width > P_total || pitch < width)
        return COMBO_ERR_INVALID_ARG;
    if (!in || !out || (R > 0 && !idx)) return COMBO_ERR_INVALID_ARG;
    if (grads && EB != 4) return COMBO_ERR_INVALID_ARG;
    if (!aligned16(in) || !aligned16(out) || (grads && !aligned16(grads))) return COMBO_ERR_INVALID_ARG;
    if ((unsigned long long)pitch > (1ull << 40) / (unsigned)N) return COMBO_ERR_INVALID_ARG;
    const size_t extent = (size_t)(((long long)(N - 1) * pitch + width) * EB);
    if (overlaps(in, out, extent) || (grads && overlaps(grads, out, extent))) return COMBO_ERR_ALIAS;

    // The staged kernels address columns with signed 32-bit TMA coordinates.  Wider inputs are
    // cut into column shards, which Eq. 3 allows (workers are coupled only at equal column).
    if (width > t_shard_columns) {
        for (long long c0 = 0; c0 < width; c0 += t_shard_columns) {
            const long long w = width - c0 < t_shard_columns ? width - c0 : t_shard_columns;
            combo_status rcs = aggregate_cols(static_cast<const char*>(in) + c0 * EB,
                                              grads ? static_cast<const char*>(grads) + c0 * EB : nullptr, lr,
                                              static_cast<char*>(out) + c0 * EB, EB, weights, idx, N, P_total, S, R,
                                              p_begin + c0, w, pitch, stream, h_newcomer);
            if (rcs != COMBO_OK) return rcs;
        }
        return COMBO_OK;
    }

    DeviceInfo* dev = nullptr;
    combo_status rc = device_info(&dev);
    if (rc != COMBO_OK) return rc;

    AggParams p;
    memset(&p, 0, sizeof(p));
    p.in = static_cast<const unsigned char*>(in);
    p.grads = static_cast<const unsigned char*>(grads);
    p.out = static_cast<unsigned char*>(out);
    p.weights = weights;
    p.idx = idx;
    p.pitch = pitch;
    p.p_begin = p_begin;
    p.width = width;
    p.L = (P_total + S - 1) / S;
    p.N = N; p.S = S; p.R = R;
    p.lr = lr;
    if (h_newcomer)
        for (int v = 0; v < N; ++v)
            if (h_newcomer[v]) p.newcomer.w[v >> 5] |= 1u << (v & 31);
    const bool sgd = grads != nullptr;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    bool want_staged = t_force_path != 1 && t_force_path != 6;
    if (t_force_path == 0 && (long long)N * width < (1 << 16)) want_staged = false;   // too small to pipeline
    if (want_staged && t_force_path != 2) {
        // short inputs: one tile per CTA, several CTAs per SM
        combo::TileMaps maps;
        AggParams q = p;
        bool short_enough = false;
        StagedPlan plan = plan_tile(q, maps, EB, sgd, *dev, &short_enough);
        if (plan.ok && (short_enough || t_force_path == 5)) {
            cudaError_t e = launch_tile(q, maps, plan, EB, sgd, st);
            if (e != cudaSuccess) return cuda_fail(e, "tile aggregation launch");
            t_last_path = 5;
            return COMBO_OK;
        }
    }
    if (want_staged) {
        combo::TileMaps maps;
        StagedPlan plan = plan_staged(p, maps, EB, sgd, *dev);
        if (plan.ok) {
            rc = next_tile_slot(&p.sched, st);
            if (rc != COMBO_OK) return rc;
            cudaError_t e = launch_staged(p, maps, plan, EB, sgd, st);
            if (e != cudaSuccess) return cuda_fail(e, "staged aggregation launch");
            t_last_path = 2;
            return COMBO_OK;
        }
    }
    cudaError_t e = launch_direct(p, EB, sgd, *dev, st, t_force_path == 6);
    if (e != cudaSuccess) return cuda_fail(e, "direct aggregation launch");
    t_last_path = 1;
    return COMBO_OK;
}

// ---------------------------------------------------------------- aggregation divergence
// Blocks whose partial sums the scratch must hold: the staged kernel launches at most one
// CTA per SM, the fallback at most four.
inline long long divergence_max_blocks(const DeviceInfo& dev) { return (long long)dev.sms * 4; }

combo_status divergence_impl(const void* models, const void* mean_of, int EB, const float* weights, int N,
                             long long P, double* rho_out, double* scratch, size_t scratch_bytes, void* stream) {
    if (EB != 4 && EB != 2) return COMBO_ERR_INVALID_ARG;
    if (N < 1 || N > COMBO_MAX_WORKERS || P < 1 || !models || !rho_out || !scratch) return COMBO_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(models) & (EB - 1)) || (mean_of && (reinterpret_cast<uintptr_t>(mean_of) & (EB - 1))))
        return COMBO_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(scratch) & 7) || (reinterpret_cast<uintptr_t>(rho_out) & 7)) return COMBO_ERR_INVALID_ARG;
    if ((unsigned long long)P > (1ull << 40) / (unsigned)N) return COMBO_ERR_INVALID_ARG;
    DeviceInfo* dev = nullptr;
    combo_status rc = device_info(&dev);
    if (rc != COMBO_OK) return rc;
    if (scratch_bytes < (size_t)divergence_max_blocks(*dev) * (size_t)N * sizeof(double)) return COMBO_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool two = mean_of != nullptr && mean_of != models;

    combo::DivParams p;
    memset(&p, 0, sizeof(p));
    p.models = static_cast<const unsigned char*>(models);
    p.src = static_cast<const unsigned char*>(two ? mean_of : models);
    p.weights = weights;
    p.partial = scratch;
    p.pitch = P;
    p.width = P;
    p.N = N;
    p.narr = two ? 2 : 1;

    int nblocks = 0;
    // staged path: rows at least 4-byte aligned, at most 256 workers, two stages must fit
    const long long pitch_bytes = P * EB;
    const int m = 16 / gcd_int(16, pitch_bytes % 16 == 0 ? 16 : pitch_bytes % 16);   // row classes
    const bool word = m > 1;
    if (t_force_path != 1 && (pitch_bytes % 4) == 0 && aligned16(models) && aligned16(p.src) &&
        N <= combo::kDivMaxStagedN && (long long)N * P >= (1 << 16) && (unsigned long long)P + 256 < (1ull << 31) &&
        (unsigned long long)m * (unsigned long long)pitch_bytes < (1ull << 40) && 2 * m <= 32) {
        const int V = 16 / EB;
        const unsigned header = round_up((unsigned)sizeof(combo::StagedHeader), 128);
        p.coef_off = header;
        p.rowoff_off = p.coef_off + round_up((unsigned)N * 4u, 128);
        p.part_off = p.rowoff_off + round_up((unsigned)N * 4u, 128);
        p.m = m;
        // shared memory in front of the stages for a box of c columns.  Vector mode: two copies
        // of G * PSTR floats of partial sums and two of the widest tile's means.  Word mode: two
        // copies of [consumer warps][words per row rounded up to a power of two] sums and two
        // of 256 means.
        auto front = [&](int c) {
            unsigned part, mean;
            if (word) {
                const int nu = (c - V) * EB / 4;
                int nup = 16;
                while (nup < nu) nup <<= 1;
                part = 2u * combo::kConsumerWarps * (unsigned)(nup * (4 / EB)) * 4u;
                mean = 2u * combo::kDivWordMeans * 4u;
            } else {
                part = 2u * combo::kConsumerThreads * V * 4u;
                mean = 2u * combo::kDivTile * 4u;
            }
            p.mean_off = p.part_off + part;
            p.stage_off = p.mean_off + mean;
            return (long long)dev->smem_optin - p.stage_off - 256;
        };
        // tile: the widest whose stage stays within 64 KB (at least 64 columns if two stages
        // fit at all); tiles beyond 256 columns are made of 256-column boxes.  With row phases
        // one box of at most 256 columns: the widest of which three stages fit (the consumers
        // then hold two tiles at a time and need one barrier per tile), else the widest of
        // which two fit.
        int TC = 0, box = 0;
        bool pipe = !word;
        if (word) {
            for (int need = 3; need >= 2 && TC == 0; --need)
                for (int c = combo::kDivBox; c >= 64; c >>= 1) {
                    if (t_tile > 0 && c != t_tile) continue;
                    if ((long long)need * p.narr * N * c * EB <= front(c)) { TC = c - V; box = c; pipe = need == 3; break; }
                }
        } else {
            for (int c = combo::kDivTile; c >= 64; c >>= 1) {
                const long long stage = (long long)p.narr * N * c * EB;
                if (2 * stage > front(c) || p.narr * (c > combo::kDivBox ? c / combo::kDivBox : 1) > 32) continue;
                if (stage <= 64 * 1024 || c == 64 || c <= combo::kDivBox) { TC = c; break; }
            }
            box = TC > combo::kDivBox ? combo::kDivBox : TC;
        }
        const long long budget = TC > 0 ? front(box) : 0;
        combo::TileMaps maps;
        bool ok = TC > 0;
        for (int a = 0; ok && a < p.narr; ++a)
            for (int j = 0; ok && j < m && j < N; ++j)
                ok = encode_class_map(&maps.map[a][j], a == 0 ? p.models : p.src, EB, j, m, N, P, P, box);
        if (ok) {
            p.row_bytes = box * EB;
            p.stage_bytes = (unsigned)(p.narr * N * p.row_bytes) * (unsigned)(word ? 1 : TC / box);
            const int fit = (int)(budget / p.stage_bytes);
            // two tiles are in the consumers' hands at a time: three stages keep a load in flight
            int stages = (int)((112 * 1024) / p.stage_bytes);
            if (stages < 3) stages = 3;
            if (t_stages >= 2) stages = t_stages;
            if (stages > combo::kMaxStages) stages = combo::kMaxStages;
            if (stages > fit) stages = fit;
            p.stages = stages;
            p.n_tiles = (P + TC - 1) / TC;
            nblocks = (int)(p.n_tiles < dev->sms ? p.n_tiles : dev->sms);
            const size_t smem = (size_t)p.stage_off + (size_t)stages * p.stage_bytes + 16;
            cudaError_t e = cudaErrorInvalidValue;
#define COMBO_DIV_LAUNCH_P(EBV, TCV, WV, PV)                                                                    \
    if (EB == EBV && TC == TCV && word == WV && pipe == PV) {                                                   \
        e = cudaFuncSetAttribute(combo::k_divergence_staged<EBV, TCV, WV, PV>,                                  \
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);                       \
        if (e == cudaSuccess)                                                                                   \
            combo::k_divergence_staged<EBV, TCV, WV, PV><<<nblocks, combo::kStagedThreads, smem, st>>>(p, maps); \
    }
#define COMBO_DIV_LAUNCH(EBV, TCV, WV) COMBO_DIV_LAUNCH_P(EBV, TCV, WV, true)
#define COMBO_DIV_LAUNCH_W(EBV, TCV) COMBO_DIV_LAUNCH_P(EBV, TCV, true, true) COMBO_DIV_LAUNCH_P(EBV, TCV, true, false)
            COMBO_DIV_LAUNCH(4, 1024, false) COMBO_DIV_LAUNCH(4, 512, false)
            COMBO_DIV_LAUNCH(2, 1024, false) COMBO_DIV_LAUNCH(2, 512, false)
            COMBO_DIV_LAUNCH(4, 256, false) COMBO_DIV_LAUNCH(4, 128, false) COMBO_DIV_LAUNCH(4, 64, false)
            COMBO_DIV_LAUNCH(2, 256, false) COMBO_DIV_LAUNCH(2, 128, false) COMBO_DIV_LAUNCH(2, 64, false)
            COMBO_DIV_LAUNCH_W(4, 252) COMBO_DIV_LAUNCH_W(4, 124) COMBO_DIV_LAUNCH_W(4, 60)
            COMBO_DIV_LAUNCH_W(2, 248) COMBO_DIV_LAUNCH_W(2, 120) COMBO_DIV_LAUNCH_W(2, 56)
#undef COMBO_DIV_LAUNCH
#undef COMBO_DIV_LAUNCH_P
#undef COMBO_DIV_LAUNCH_W
            if (e == cudaSuccess) e = cudaGetLastError();
            if (e != cudaSuccess) return cuda_fail(e, "divergence launch");
            t_last_path = 2;
        }
    }
    if (nblocks == 0) {
        const long long n_blk = (P + 255) / 256;
        const long long cap = divergence_max_blocks(*dev);
        nblocks = (int)(n_blk < cap ? n_blk : cap);
        const size_t smem = (size_t)N * 12 + 16;
        cudaError_t e = cudaSuccess;
        if (EB == 4) {
            if (smem > 48 * 1024) e = cudaFuncSetAttribute(combo::k_divergence_direct<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e == cudaSuccess) combo::k_divergence_direct<4><<<nblocks, 256, smem, st>>>(p);
        } else {
            if (smem > 48 * 1024) e = cudaFuncSetAttribute(combo::k_divergence_direct<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e == cudaSuccess) combo::k_divergence_direct<2><<<nblocks, 256, smem, st>>>(p);
        }
        if (e == cudaSuccess) e = cudaGetLastError();
        if (e != cudaSuccess) return cuda_fail(e, "divergence launch");
        t_last_path = 1;
    }
    combo::k_divergence_finish<<<(N + 127) / 128, 128, 0, st>>>(scratch, nblocks, N, rho_out);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "divergence finish launch");
    return COMBO_OK;
}

// ---------------------------------------------------------------- divergence without allocation
// Fixed scratch for callers that cannot allocate device memory.  Every GPU that loads the
// library holds this array (1 MiB) until the process exits.  In host code the array's name
// is only a handle: the device address the kernels need comes from cudaGetSymbolAddress,
// asked once per device with that device current.
constexpr int kNoAllocMaxBlocks = 1024;
static __device__ __align__(256) double g_noalloc_scratch[(size_t)kNoAllocMaxBlocks * COMBO_NOALLOC_MAX_WORKERS];
double* g_noalloc_ptr[64];

combo_status noalloc_scratch(double** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= 64) return COMBO_ERR_UNSUPPORTED;
    if (!g_noalloc_ptr[dev]) {
        double* ptr = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_noalloc_scratch);
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(fixed scratch)");
        if (!ptr) return COMBO_ERR_CUDA;
        g_noalloc_ptr[dev] = ptr;
    }
    *out = g_noalloc_ptr[dev];
    return COMBO_OK;
}

// Streams and events of the host-memory entry point, created on its first call on a device.
constexpr int kPipeChunks = 32;
struct HostPipe {
    bool ready;
    cudaStream_t s_in, s_out;
    cudaEvent_t ev_start, ev_end, ev_in[kPipeChunks], ev_done[kPipeChunks];
};
HostPipe g_pipe[64];

combo_status host_pipe(HostPipe** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= 64) return COMBO_ERR_UNSUPPORTED;
    HostPipe& h = g_pipe[dev];
    if (!h.ready) {
        if ((e = cudaStreamCreateWithFlags(&h.s_in, cudaStreamNonBlocking)) != cudaSuccess ||
            (e = cudaStreamCreateWithFlags(&h.s_out, cudaStreamNonBlocking)) != cudaSuccess ||
            (e = cudaEventCreateWithFlags(&h.ev_start, cudaEventDisableTiming)) != cudaSuccess ||
            (e = cudaEventCreateWithFlags(&h.ev_end, cudaEventDisableTiming)) != cudaSuccess)
            return cuda_fail(e, "creating the copy streams");
        for (int i = 0; i < kPipeChunks; ++i)
            if ((e = cudaEventCreateWithFlags(&h.ev_in[i], cudaEventDisableTiming)) != cudaSuccess ||
                (e = cudaEventCreateWithFlags(&h.ev_done[i], cudaEventDisableTiming)) != cudaSuccess)
                return cuda_fail(e, "creating the chunk events");
        h.ready = true;
    }
    *out = &h;
    return COMBO_OK;
}

combo_status select_peers_impl(uint64_t seed, uint32_t round, int N, int S, int R, int32_t* idx_out,
                               cudaStream_t st, const uint8_t* h_online = nullptr) {
    if (N < 1 || N > COMBO_MAX_WORKERS || S < 1 || S > COMBO_MAX_SEGMENTS || R < 0 || R > N - 1)
        return COMBO_ERR_INVALID_ARG;
    combo::WorkerBits bits;
    memset(&bits, 0, sizeof(bits));
    if (h_online) {
        int n_on = 0;
        for (int v = 0; v < N; ++v)
            if (h_online[v]) { bits.w[v >> 5] |= 1u << (v & 31); ++n_on; }
        if (R > 0 && R > n_on - 1) return COMBO_ERR_INVALID_ARG;
    }
    if (R == 0) return COMBO_OK;
    if (!idx_out) return COMBO_ERR_INVALID_ARG;
    DeviceInfo* dev = nullptr;
    combo_status rc = device_info(&dev);
    if (rc != COMBO_OK) return rc;
    // one warp per worker, up to four workers per CTA while their arrays fit
    const size_t per_worker = (combo::select_peers_smem_bytes(N) + 15) / 16 * 16;
    int wpb = (int)((96 * 1024) / per_worker);
    if (wpb > combo::kSelectThreads / 32) wpb = combo::kSelectThreads / 32;
    if (wpb < 1) wpb = 1;
    const size_t smem = per_worker * (size_t)wpb;
    const int blocks = (N + wpb - 1) / wpb;
    cudaError_t e = cudaSuccess;
    auto kern = h_online ? combo::k_select_peers<true> : combo::k_select_peers<false>;
    if (smem > 48 * 1024) e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) {
        // may start under the preceding kernel of the stream (it waits before its first write)
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof(cfg));
        cfg.gridDim = dim3((unsigned)blocks);
        cfg.blockDim = dim3(32u * (unsigned)wpb);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = t_overlap ? 1 : 0;
        e = cudaLaunchKernelEx(&cfg, kern, seed, round, N, S, R, idx_out, bits, (int)per_worker);
    }
    if (e != cudaSuccess) return cuda_fail(e, "select_peers launch");
    return COMBO_OK;
}

}  // namespace

extern "C" {

combo_status combo_select_peers(uint64_t seed, uint32_t round, int N, int S, int R, int32_t* idx_out) {
    return select_peers_impl(seed, round, N, S, R, idx_out, (cudaStream_t)0);
}

combo_status combo_select_peers_async(uint64_t seed, uint32_t round, int N, int S, int R, int32_t* idx_out,
                                      void* stream) {
    return select_peers_impl(seed, round, N, S, R, idx_out, static_cast<cudaStream_t>(stream));
}

combo_status combo_segment_aggregate(const float* params_in, float* params_out, const float* weights,
                                     const int32_t* idx, int N, int64_t P, int S, int R, void* stream) {
    return aggregate_cols(params_in, nullptr, 0.0f, params_out, 4, weights, idx, N, P, S, R, 0, P, P, stream);
}

combo_status combo_segment_aggregate_bf16(const uint16_t* params_in, uint16_t* params_out, const float* weights,
                                          const int32_t* idx, int N, int64_t P, int S, int R, void* stream) {
    return aggregate_cols(params_in, nullptr, 0.0f, params_out, 2, weights, idx, N, P, S, R, 0, P, P, stream);
}

combo_status combo_segment_aggregate_sgd(const float* params_in, const float* grads, float lr, float* params_out,
                                         const float* weights, const int32_t* idx, int N, int64_t P, int S, int R,
                                         void* stream) {
    if (!grads) return COMBO_ERR_INVALID_ARG;
    return aggregate_cols(params_in, grads, lr, params_out, 4, weights, idx, N, P, S, R, 0, P, P, stream);
}

combo_status combo_segment_aggregate_cols(const void* params_in, const void* grads, float lr, void* params_out,
                                          int elem_bytes, const float* weights, const int32_t* idx, int N,
                                          int64_t P_total, int S, int R, int64_t p_begin, int64_t width,
                                          int64_t pitch, void* stream) {
    return aggregate_cols(params_in, grads, lr, params_out, elem_bytes, weights, idx, N, P_total, S, R, p_begin,
                          width, pitch, stream);
}

combo_status combo_select_peers_online(uint64_t seed, uint32_t round, int N, int S, int R, const uint8_t* h_online,
                                       int32_t* idx_out, void* stream) {
    return select_peers_impl(seed, round, N, S, R, idx_out, static_cast<cudaStream_t>(stream), h_online);
}

combo_status combo_segment_aggregate_members(const void* params_in, void* params_out, int elem_bytes,
                                             const float* weights, const int32_t* idx, const uint8_t* h_newcomer,
                                             int N, int64_t P, int S, int R, void* stream) {
    return aggregate_cols(params_in, nullptr, 0.0f, params_out, elem_bytes, weights, idx, N, P, S, R, 0, P, P, stream,
                          h_newcomer);
}

combo_status combo_segment_aggregate_rows(const void* const* d_rows, void* out, int64_t out_pitch, int elem_bytes,
                                          const float* weights, const int32_t* idx, int N, int64_t P, int S, int R,
                                          int w_begin, int n_local, void* stream) {
    if (elem_bytes != 4 && elem_bytes != 2) return COMBO_ERR_INVALID_ARG;
    if (N < 1 || N > COMBO_MAX_WORKERS || S < 1 || S > COMBO_MAX_SEGMENTS || R < 0 || R > N - 1 || P < 1)
        return COMBO_ERR_INVALID_ARG;
    if (w_begin < 0 || n_local < 1 || w_begin + n_local > N) return COMBO_ERR_INVALID_ARG;
    if (!d_rows || !out || (R > 0 && !idx) || !aligned16(out)) return COMBO_ERR_INVALID_ARG;
    if (out_pitch < P || (out_pitch * elem_bytes) % 16 != 0) return COMBO_ERR_INVALID_ARG;
    DeviceInfo* dev = nullptr;
    combo_status rc = device_info(&dev);
    if (rc != COMBO_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const long long L = (P + S - 1) / S;

    // Staged form: the distinct rows a column tile needs are brought into shared memory once.
    // A stage must hold the hosted rows and everything they can pull for up to two segments.
    if (t_force_path != 3 && N <= combo::kPullMaxN && R <= combo::kStagedMaxR && (long long)n_local * P >= (1 << 16)) {
        long long d_max = (long long)n_local * (1 + 2 * R);
        if (d_max > N) d_max = N;
        const int rt = ((R >= 1 && R <= 4) || R == 8) ? R : (R > combo::kGenericR ? -2 : -1);
        const int rmax = combo::rmax_of(rt);
        combo::PullStagedParams q;
        memset(&q, 0, sizeof(q));
        q.ptr_off = 0;
        q.slot_off = round_up((unsigned)N * 8u, 128);
        q.list_off = q.slot_off + round_up((unsigned)N * 2u, 128);
        q.tab_off = q.list_off + round_up((unsigned)d_max * 8u, 128);
        q.stage_off = q.tab_off + round_up(2u * (unsigned)n_local * (unsigned)combo::table_entry_bytes(rmax), 128);
        int T = 0;
        // Tile: boxes of 256 columns (128 of binary32 when three stages of 256 do not fit), as
        // many of them -- a power of two -- as keep a stage within 32 KB (bfloat16: 64 KB up to
        // 2 KB of a row); the tuning knob overrides with any 256 * 2^k.  Measured on one GPU, 11.7 M
        // columns: 16 rows of binary32 0.63 / 0.86 / 0.83 with 256 / 512 / 1024 columns, 8 rows
        // 0.40 / 0.61 / 0.81 / 0.78 with 256 / 512 / 1024 / 2048, 32 rows 0.88 / 0.86 with 256 /
        // 512; 32 rows of bfloat16 0.58 / 0.81 / 0.90 with 256 / 512 / 1024.
        int nbx = 1;
        for (int t = 256; t >= (elem_bytes == 4 ? 128 : 256); t >>= 1) {
            const long long need = (long long)q.stage_off + 3LL * d_max * t * elem_bytes + 16;
            if (need <= dev->smem_optin && t <= L) { T = t; break; }
        }
        if (T == 256) {
            for (int n = 2; n <= combo::kMaxBoxes; n <<= 1) {
                const long long stage = d_max * 256LL * n * elem_bytes;
                const long long need = (long long)q.stage_off + 3LL * stage + 16;
                if (256LL * n > L || 256LL * n * elem_bytes / 16 > combo::kPullThreads || need > dev->smem_optin) break;
                if (t_tile > 0 ? 256 * n > t_tile : stage > (elem_bytes == 2 && n <= 4 ? 64 : 32) * 1024) break;
                nbx = n;
            }
            T = 256 * nbx;
        }
        if (T > 0) {
            q.rows = d_rows;
            q.out = static_cast<unsigned char*>(out);
            q.weights = weights;
            q.idx = idx;
            q.P = P;
            q.L = L;
            q.out_pitch = out_pitch;
            q.N = N; q.S = S; q.R = R;
            q.w_begin = w_begin;
            q.n_local = n_local;
            q.T = T;
            q.nbx = nbx;
            q.row_bytes = (T / nbx) * elem_bytes;
            for (q.gpb_log2 = 0; (16 << q.gpb_log2) < q.row_bytes; ++q.gpb_log2) {}
            for (q.gpr_log2 = 0; (16 << q.gpr_log2) < nbx * q.row_bytes; ++q.gpr_log2) {}
            q.d_max = (int)d_max;
            q.stage_bytes = (unsigned)(d_max * T * elem_bytes);
            q.n_tiles = (P + T - 1) / T;
            // about 64 KB of loads in flight beside the tile being consumed (measured: 3 stages of 32 KB beat 5), at least three stages
            int stages = 1 + (int)((64 * 1024 + q.stage_bytes - 1) / q.stage_bytes);
            const int fit = (int)(((long long)dev->smem_optin - q.stage_off - 16) / q.stage_bytes);
            if (t_stages >= 3) stages = t_stages;
            if (stages > 8) stages = 8;
            if (stages > fit) stages = fit;
            if (stages < 3) stages = 3;
            q.stages = stages;
            const size_t smem = (size_t)q.stage_off + (size_t)stages * (size_t)q.stage_bytes + 16;
            const int grid = (int)(q.n_tiles < dev->sms ? q.n_tiles : dev->sms);
            cudaError_t e = cudaErrorInvalidValue;
            // bfloat16 rows with unit weights are summed by the mixed-precision add
            const bool unw = elem_bytes == 2 && !weights;
#define COMBO_PULL_LAUNCH(EBV, RTV, UNWV)                                                                        \
    if (elem_bytes == EBV && rt == RTV && unw == UNWV) {                                                         \
        e = cudaFuncSetAttribute(combo::k_pull_staged<EBV, RTV, UNWV>,                                           \
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);                        \
        if (e == cudaSuccess) combo::k_pull_staged<EBV, RTV, UNWV><<<grid, combo::kPullThreads, smem, st>>>(q);  \
    }
#define COMBO_PULL_LAUNCH_R(EBV, UNWV)                                                                           \
    COMBO_PULL_LAUNCH(EBV, 1, UNWV) COMBO_PULL_LAUNCH(EBV, 2, UNWV) COMBO_PULL_LAUNCH(EBV, 3, UNWV)              \
    COMBO_PULL_LAUNCH(EBV, 4, UNWV) COMBO_PULL_LAUNCH(EBV, 8, UNWV) COMBO_PULL_LAUNCH(EBV, -1, UNWV)             \
    COMBO_PULL_LAUNCH(EBV, -2, UNWV)
            COMBO_PULL_LAUNCH_R(4, false) COMBO_PULL_LAUNCH_R(2, false) COMBO_PULL_LAUNCH_R(2, true)
#undef COMBO_PULL_LAUNCH_R
#undef COMBO_PULL_LAUNCH
            if (e == cudaSuccess) e = cudaGetLastError();
            if (e != cudaSuccess) return cuda_fail(e, "staged pull aggregation launch");
            t_last_path = 4;
            return COMBO_OK;
        }
    }

    combo::PullParams p;
    memset(&p, 0, sizeof(p));
    p.rows = d_rows;
    p.out = static_cast<unsigned char*>(out);
    p.weights = weights;
    p.idx = idx;
    p.P = P;
    p.L = L;
    p.out_pitch = out_pitch;
    p.N = N; p.S = S; p.R = R;
    p.w_begin = w_begin;
    p.n_local = n_local;
    const int V = 16 / elem_bytes;
    const long long groups = (P + V - 1) / V;
    // about eight resident CTAs per SM over all hosted workers together
    long long bx = (groups + 255) / 256;
    long long cap = ((long long)dev->sms * 8 + n_local - 1) / n_local;
    if (cap < 1) cap = 1;
    if (bx > cap) bx = cap;
    const dim3 grid((unsigned)bx, (unsigned)n_local);
    const size_t smem = (size_t)N * sizeof(void*);
    cudaError_t e = cudaSuccess;
    if (elem_bytes == 4) {
        if (smem > 48 * 1024) e = cudaFuncSetAttribute(combo::k_pull_aggregate<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess) combo::k_pull_aggregate<4><<<grid, 256, smem, st>>>(p);
    } else {
        if (smem > 48 * 1024) e = cudaFuncSetAttribute(combo::k_pull_aggregate<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess) combo::k_pull_aggregate<2><<<grid, 256, smem, st>>>(p);
    }
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "pull aggregation launch");
    t_last_path = 3;
    return COMBO_OK;
}

combo_status combo_check_rows(const void* const* d_rows, int N, void* stream, int32_t* dev_flag) {
    if (!d_rows || N < 1 || !dev_flag) return COMBO_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(dev_flag, 0, sizeof(int32_t), st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync");
    combo::k_check_rows<<<(N + 255) / 256, 256, 0, st>>>(d_rows, N, dev_flag);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "check_rows launch");
    return COMBO_OK;
}

combo_status combo_validate_idx(const int32_t* idx, int N, int S, int R, void* stream, int32_t* dev_flag) {
    if (N < 1 || S < 1 || R < 0 || !dev_flag || (R > 0 && !idx)) return COMBO_ERR_INVALID_ARG;
    DeviceInfo* dev = nullptr;
    combo_status rc = device_info(&dev);
    if (rc != COMBO_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(dev_flag, 0, sizeof(int32_t), st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync");
    if (R == 0) return COMBO_OK;
    const long long total = (long long)N * S * R;
    long long blocks = (total + 255) / 256;
    if (blocks > dev->sms * 8) blocks = dev->sms * 8;
    combo::k_validate_idx<<<(int)blocks, 256, 0, st>>>(idx, N, S, R, dev_flag);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "validate_idx launch");
    return COMBO_OK;
}

combo_status combo_round_host(const void* h_params_in, const void* h_grads, float lr, void* h_params_out,
                              int elem_bytes, const float* h_weights, uint64_t seed, uint32_t round, int rounds,
                              int N, int64_t P, int S, int R, void* d_in, void* d_grads, void* d_out,
                              float* d_weights, int32_t* d_idx, int32_t* h_idx_out, void* stream) {
    if (!h_params_in || !h_params_out || !d_in || !d_out) return COMBO_ERR_INVALID_ARG;
    if ((h_grads != nullptr) != (d_grads != nullptr)) return COMBO_ERR_INVALID_ARG;
    if (h_weights && !d_weights) return COMBO_ERR_INVALID_ARG;
    if (elem_bytes != 4 && elem_bytes != 2) return COMBO_ERR_INVALID_ARG;
    if (N < 1 || P < 1 || R < 0 || rounds < 1 || (R > 0 && !d_idx)) return COMBO_ERR_INVALID_ARG;
    DeviceInfo* dev = nullptr;
    combo_status rc = device_info(&dev);
    if (rc != COMBO_OK) return rc;
    HostPipe* hp = nullptr;
    rc = host_pipe(&hp);
    if (rc != COMBO_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t EB = (size_t)elem_bytes;
    const size_t pitch_bytes = (size_t)P * EB;
    cudaError_t e;
    if (h_weights &&
        (e = cudaMemcpyAsync(d_weights, h_weights, sizeof(float) * (size_t)N, cudaMemcpyHostToDevice, st)) !=
            cudaSuccess)
        return cuda_fail(e, "copy weights to device");

    // Eq. 3 couples workers only at equal column, in every round: a column chunk can run
    // through ALL rounds on its own.  Chunks are therefore pipelined over three streams:
    // chunk c+1 is copied in and chunk c-1 copied out while chunk c is aggregated.
    const size_t total = (size_t)N * pitch_bytes;
    int K = (int)((total + (8u << 20) - 1) / (8u << 20));     // chunks of at least 8 MB, at most kPipeChunks
    if (K > kPipeChunks) K = kPipeChunks;
    if (K < 1) K = 1;
    int64_t cw = ((P + K - 1) / K + 63) / 64 * 64;        // chunk width, 16-byte aligned starts
    if ((e = cudaEventRecord(hp->ev_start, st)) != cudaSuccess) return cuda_fail(e, "cudaEventRecord");
    if ((e = cudaStreamWaitEvent(hp->s_in, hp->ev_start, 0)) != cudaSuccess ||
        (e = cudaStreamWaitEvent(hp->s_out, hp->ev_start, 0)) != cudaSuccess)
        return cuda_fail(e, "cudaStreamWaitEvent");
    for (int c = 0; c < K; ++c) {
        const int64_t p0 = (int64_t)c * cw;
        if (p0 >= P) break;
        const int64_t w = (p0 + cw <= P) ? cw : P - p0;
        const size_t off = (size_t)p0 * EB;
        if ((e = cudaMemcpy2DAsync(static_cast<char*>(d_in) + off, pitch_bytes,
                                   static_cast<const char*>(h_params_in) + off, pitch_bytes, (size_t)w * EB,
                                   (size_t)N, cudaMemcpyHostToDevice, hp->s_in)) != cudaSuccess)
            return cuda_fail(e, "copy params to device");
        if (h_grads && (e = cudaMemcpy2DAsync(static_cast<char*>(d_grads) + off, pitch_bytes,
                                              static_cast<const char*>(h_grads) + off, pitch_bytes, (size_t)w * EB,
                                              (size_t)N, cudaMemcpyHostToDevice, hp->s_in)) != cudaSuccess)
            return cuda_fail(e, "copy grads to device");
        if ((e = cudaEventRecord(hp->ev_in[c], hp->s_in)) != cudaSuccess ||
            (e = cudaStreamWaitEvent(st, hp->ev_in[c], 0)) != cudaSuccess)
            return cuda_fail(e, "chunk hand-over to the compute stream");
        char* cur = static_cast<char*>(d_in) + off;
        char* nxt = static_cast<char*>(d_out) + off;
        for (int t = 0; t < rounds; ++t) {
            rc = select_peers_impl(seed, round + (uint32_t)t, N, S, R, d_idx, st);
            if (rc != COMBO_OK) return rc;
            rc = aggregate_cols(cur, d_grads ? static_cast<char*>(d_grads) + off : nullptr, lr, nxt, elem_bytes,
                                h_weights ? d_weights : nullptr, d_idx, N, P, S, R, p0, w, P, stream);
            if (rc != COMBO_OK) return rc;
            char* sw = cur; cur = nxt; nxt = sw;
        }
        if ((e = cudaEventRecord(hp->ev_done[c], st)) != cudaSuccess ||
            (e = cudaStreamWaitEvent(hp->s_out, hp->ev_done[c], 0)) != cudaSuccess)
            return cuda_fail(e, "chunk hand-over to the copy-out stream");
        if ((e = cudaMemcpy2DAsync(static_cast<char*>(h_params_out) + off, pitch_bytes, cur, pitch_bytes,
                                   (size_t)w * EB, (size_t)N, cudaMemcpyDeviceToHost, hp->s_out)) != cudaSuccess)
            return cuda_fail(e, "copy result to host");
    }
    if (h_idx_out && R > 0 &&
        (e = cudaMemcpyAsync(h_idx_out, d_idx, sizeof(int32_t) * (size_t)N * S * R, cudaMemcpyDeviceToHost, st)) !=
            cudaSuccess)
        return cuda_fail(e, "copy idx to host");
    if ((e = cudaEventRecord(hp->ev_end, hp->s_out)) != cudaSuccess ||
        (e = cudaStreamWaitEvent(st, hp->ev_end, 0)) != cudaSuccess)
        return cuda_fail(e, "join of the copy-out stream");
    if ((e = cudaStreamSynchronize(st)) != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
    return COMBO_OK;
}

size_t combo_divergence_scratch_bytes(int N) {
    DeviceInfo* dev = nullptr;
    if (N < 1 || N > COMBO_MAX_WORKERS || device_info(&dev) != COMBO_OK) return 0;
    return (size_t)divergence_max_blocks(*dev) * (size_t)N * sizeof(double);
}

combo_status combo_aggregation_divergence(const void* models, const void* mean_of, int elem_bytes,
                                          const float* weights, int N, int64_t P, double* rho_out, void* scratch,
                                          size_t scratch_bytes, void* stream) {
    return divergence_impl(models, mean_of, elem_bytes, weights, N, P, rho_out, static_cast<double*>(scratch),
                           scratch_bytes, stream);
}

combo_status combo_aggregation_divergence_noalloc(const void* models, const void* mean_of, int elem_bytes,
                                                  const float* weights, int N, int64_t P, double* rho_out,
                                                  void* stream) {
    if (N > COMBO_NOALLOC_MAX_WORKERS) {
        snprintf(t_cuda_err, sizeof(t_cuda_err), "N = %d exceeds the fixed scratch (at most %d workers)", N,
                 COMBO_NOALLOC_MAX_WORKERS);
        return COMBO_ERR_TOO_LARGE;
    }
    double* scratch = nullptr;
    combo_status rc = noalloc_scratch(&scratch);
    if (rc != COMBO_OK) return rc;
    return divergence_impl(models, mean_of, elem_bytes, weights, N, P, rho_out, scratch,
                           sizeof(double) * (size_t)kNoAllocMaxBlocks * COMBO_NOALLOC_MAX_WORKERS, stream);
}

combo_status combo_device_status(void) {
    int v = 0;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceSynchronize");
    if ((e = cudaMemcpyFromSymbol(&v, combo::g_dev_status, sizeof(int))) != cudaSuccess)
        return cuda_fail(e, "cudaMemcpyFromSymbol");
    if (v != 0) {
        int zero = 0;
        cudaMemcpyToSymbol(combo::g_dev_status, &zero, sizeof(int));
        // a kernel that gave up may have left its tile dispenser half used: clear the ring
        // (the device is idle here), so that the launch that next takes that slot starts clean
        static const combo::TileSlot clean[combo::kTileSlots] = {};
        cudaMemcpyToSymbol(combo::g_tile_slots, clean, sizeof(clean));
        snprintf(t_cuda_err, sizeof(t_cuda_err), "bounded wait gave up at site %d", v);
        return COMBO_ERR_DEVICE_TIMEOUT;
    }
    return COMBO_OK;
}

int combo_last_kernel_path(void) { return t_last_path; }

void combo_set_kernel_path(int path) { t_force_path = (path == 1 || path == 2 || path == 3 || path == 5 || path == 6) ? path : 0; }

void combo_set_tuning(int tile_elems, int stages) {
    t_tile = tile_elems > 0 ? tile_elems : 0;
    t_stages = stages > 0 ? stages : 0;
}

void combo_set_launch_overlap(int on) { t_overlap = on ? 1 : 0; }

int64_t combo_max_launch_columns(void) { return kMaxShardColumns; }

void combo_set_launch_columns(int64_t columns) {
    long long c = columns / 64 * 64;
    t_shard_columns = (c < 64 || c > kMaxShardColumns) ? kMaxShardColumns : c;
}

combo_status combo_debug_dead_wait(void* stream) {
    DeviceInfo* dev = nullptr;
    combo_status rc = device_info(&dev);
    if (rc != COMBO_OK) return rc;
    combo::k_debug_dead_wait<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "debug wait launch");
    return COMBO_OK;
}

const char* combo_status_string(combo_status status) {
    switch (status) {
        case COMBO_OK: return "ok";
        case COMBO_ERR_INVALID_ARG: return "invalid argument";
        case COMBO_ERR_ALIAS: return "input and output overlap";
        case COMBO_ERR_UNSUPPORTED: return "device is not compute capability 10.x";
        case COMBO_ERR_CUDA: return "CUDA error";
        case COMBO_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
        case COMBO_ERR_TOO_LARGE: return "size exceeds the fixed scratch of the no-allocation entry point";
        default: return "unknown status";
    }
}

const char* combo_last_cuda_error(void) { return t_cuda_err; }

int combo_version(void) { return 100; }

}  // extern "C"
