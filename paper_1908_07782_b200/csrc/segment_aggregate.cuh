// Segment-wise aggregation kernels (Eq. 3 and Eq. 4), all workers at once.
//
// Eq. 3 couples workers only at equal column p, and the peer table depends on
// (worker, segment) alone.  The unit of work is therefore a column tile taken
// through ALL N rows: the N x T block is brought from HBM into shared memory
// once by tiled TMA copies (completion counted on an mbarrier), every worker's
// output for those columns is formed from it (R+1 shared-memory reads per
// output element instead of R+1 HBM/L2 reads), and the N x T result goes out
// with streaming stores.  HBM traffic is then the compulsory one: each
// worker-parameter read once and written once.
//
//   k_staged  persistent CTAs, 1 producer warp + 16 consumer warps, a ring of
//             stages; warp-per-row accumulation in binary32
//   k_direct  plain gather from global memory (any R, any N, tiny segments);
//             also the "naive (R+1)-reads" contrast case for profiling
//
// Row alignment.  The ABI fixes dense [N][pitch] arrays, so row k starts at
// byte phase (k*pitch*e) mod 16.  A tensor map needs a 16-byte aligned base
// and row stride, so the rows are split into m = 16/gcd(16, pitch*e) classes
// (k mod m): within a class all rows share one phase and are m*pitch apart, a
// legal stride.  Each class gets its own tensor map whose origin is the row
// start rounded DOWN to 16 bytes; its box is V = 16/e columns wider than the
// tile, so a staged row holds the tile's columns at byte offset phase.
// When all phases are 0 (m = 1) consumers read and write 128-bit vectors; when
// they differ, lanes take interleaved 4-byte (or 2-byte) words of the row, so
// that shared-memory reads stay conflict-free and global stores stay
// contiguous per warp whatever the phases are.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace combo {

// device status word: 0, or the code of the first bounded wait that gave up
__device__ int g_dev_status;

#ifndef COMBO_CONSUMER_WARPS
#define COMBO_CONSUMER_WARPS 16
#endif
constexpr int kConsumerWarps = COMBO_CONSUMER_WARPS;
constexpr int kConsumerThreads = 32 * kConsumerWarps;
constexpr int kStagedThreads = 32 + kConsumerThreads;
constexpr int kMaxStages = 8;
constexpr int kStagedMaxR = 16;            // most replicas the staged kernel takes (Section 5.2 sweeps R up to 16)
constexpr int kGenericR = 8;               // replicas of the unspecialised kernel; beyond: the wide one
// Replicas a kernel instance is built for: RT >= 0 exactly RT; -1 any up to kGenericR; -2 any up
// to kStagedMaxR; -3 the same with the dense evaluation of whole tiles (see aggregate_dense).
__host__ __device__ constexpr int rmax_of(int rt) { return rt >= 0 ? rt : (rt == -1 ? 8 : 16); }
constexpr int kMaxClasses = 8;
constexpr int kMaxBoxes = 8;              // x-boxes per tile
constexpr uint32_t kWaitCap = 1u << 23;   // polls before a wait is declared dead
constexpr uint32_t kWaitHintNs = 1000;    // time a single poll may stay suspended
#ifndef COMBO_FAST_POLLS
#define COMBO_FAST_POLLS 32
#endif
constexpr uint32_t kFastPolls = COMBO_FAST_POLLS;   // polls without a suspend hint before the hinted ones

// Tile dispenser of one launch (global memory owned by the library, one of a ring of
// slots).  `next` hands out tiles beyond the first one of each CTA; the last CTA to leave
// puts the slot back to zero, so a slot is clean whenever a launch picks it up.
struct TileSlot {
    unsigned long long next;
    unsigned int done;
    unsigned int pad;
};
constexpr int kTileSlots = 256;
__device__ TileSlot g_tile_slots[kTileSlots];

// One flag per worker (up to COMBO_MAX_WORKERS), passed by value (Section 4.2: online /
// offline workers, newcomers).
struct WorkerBits {
    uint32_t w[256];
    __host__ __device__ bool get(int i) const { return (w[i >> 5] >> (i & 31)) & 1u; }
};

struct AggParams {
    const unsigned char* in;
    const unsigned char* grads;
    unsigned char* out;
    const float* weights;
    const int32_t* idx;
    long long pitch;     // elements between rows
    long long p_begin;   // global column of local column 0
    long long width;     // local columns
    long long L;         // segment length of the whole vector
    long long n_tiles;
    int N, S, R;
    float lr;
    int T;               // tile width in elements
    int m;               // row classes (tensor maps per array)
    int nbx;             // x-boxes per tile
    int box_w;           // box width in elements (tile part + phase room)
    int stages;
    int row_bytes;       // shared-memory bytes per staged row of one box = box_w * e
    unsigned tab_off;    // byte offset of the coefficient table in shared memory
    int tab_slots;       // segments the table holds: all S of them, or 2 (rebuilt on the way)
    unsigned dtab_off;   // byte offset of the dense coefficient blocks (dense mode only)
    int dslot_bytes;     // bytes of one segment's dense blocks
    int stage_rows;      // rows between the x-boxes of a staged tile; 0 = N (a stage may have room for more rows than it holds)
    unsigned stage_off;  // byte offset of stage 0
    unsigned stage_bytes;
    TileSlot* sched;     // tile dispenser of this launch
    WorkerBits newcomer; // workers that aggregate without their own model (Section 4.2)
};

// Tensor maps of one launch: [array][class], array 0 = parameters, 1 = gradients.
struct alignas(64) TileMaps {
    CUtensorMap map[2][kMaxClasses];
};

// ---------------------------------------------------------------- small helpers
__device__ __forceinline__ float bf16_widen(uint32_t bits16) { return __uint_as_float(bits16 << 16); }

__device__ __forceinline__ uint32_t pack_bf16x2_rn(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);   // round to nearest even
    return *reinterpret_cast<uint32_t*>(&v);
}

template <int EB> struct ElemOps;
template <> struct ElemOps<4> {
    static constexpr int V = 4;
    __device__ static __forceinline__ float load(const void* p) { return *reinterpret_cast<const float*>(p); }
    __device__ static __forceinline__ void store(void* p, float v) { __stcs(reinterpret_cast<float*>(p), v); }
    __device__ static __forceinline__ void store_vec(void* p, const float (&a)[4]) {
        __stcs(reinterpret_cast<float4*>(p), make_float4(a[0], a[1], a[2], a[3]));
    }
};
template <> struct ElemOps<2> {
    static constexpr int V = 8;
    __device__ static __forceinline__ float load(const void* p) {
        return bf16_widen(*reinterpret_cast<const uint16_t*>(p));
    }
    __device__ static __forceinline__ void store(void* p, float v) {
        __stcs(reinterpret_cast<unsigned short*>(p), (unsigned short)(pack_bf16x2_rn(v, 0.0f) & 0xffffu));
    }
    __device__ static __forceinline__ void store_vec(void* p, const float (&a)[8]) {
        __stcs(reinterpret_cast<uint4*>(p),
               make_uint4(pack_bf16x2_rn(a[0], a[1]), pack_bf16x2_rn(a[2], a[3]),
                          pack_bf16x2_rn(a[4], a[5]), pack_bf16x2_rn(a[6], a[7])));
    }
};

// Reads one output-aligned group (16 bytes of elements) at granule GB.
template <int EB, int GB> struct GroupLoad;
template <> struct GroupLoad<4, 16> {
    __device__ static __forceinline__ void run(const unsigned char* p, float (&x)[4]) {
        float4 v = *reinterpret_cast<const float4*>(p);
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    }
};
template <> struct GroupLoad<2, 16> {
    __device__ static __forceinline__ void run(const unsigned char* p, float (&x)[8]) {
        uint4 v = *reinterpret_cast<const uint4*>(p);
        x[0] = bf16_widen(v.x & 0xffffu); x[1] = __uint_as_float(v.x & 0xffff0000u);
        x[2] = bf16_widen(v.y & 0xffffu); x[3] = __uint_as_float(v.y & 0xffff0000u);
        x[4] = bf16_widen(v.z & 0xffffu); x[5] = __uint_as_float(v.z & 0xffff0000u);
        x[6] = bf16_widen(v.w & 0xffffu); x[7] = __uint_as_float(v.w & 0xffff0000u);
    }
};
// ---- packed binary32 pairs -----------------------------------------------------
// Two binary32 values travel in one 64-bit register (low half = first element), the
// operand form of the f32x2 instructions: one instruction, two IEEE operations.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pair_bits(uint32_t lo, uint32_t hi) { return ((f32x2)hi << 32) | (f32x2)lo; }
__device__ __forceinline__ f32x2 pair_dup(float c) { return pair_bits(__float_as_uint(c), __float_as_uint(c)); }
__device__ __forceinline__ float pair_lo(f32x2 v) { return __uint_as_float((uint32_t)v); }
__device__ __forceinline__ float pair_hi(f32x2 v) { return __uint_as_float((uint32_t)(v >> 32)); }
__device__ __forceinline__ f32x2 mul2(f32x2 c, f32x2 x) {
    f32x2 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(c), "l"(x));
    return d;
}
__device__ __forceinline__ f32x2 fma2(f32x2 c, f32x2 x, f32x2 acc) {
#ifdef COMBO_SCALAR_FMA
    return pair_bits(__float_as_uint(fmaf(pair_lo(c), pair_lo(x), pair_lo(acc))),
                     __float_as_uint(fmaf(pair_hi(c), pair_hi(x), pair_hi(acc))));
#else
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(c), "l"(x));
    return acc;
#endif
}
// a 32-bit word holding two bf16 -> the pair of their binary32 values
__device__ __forceinline__ f32x2 bf16x2_widen(uint32_t w) { return pair_bits(w << 16, w & 0xffff0000u); }

// One lane's share of a 512-byte item as V/2 pairs.  GB = 16: one 128-bit vector at the
// lane's 16 bytes.  Narrower granules: the lane owns 16/GB pieces of GB bytes, 32*GB
// bytes apart, so that consecutive lanes touch consecutive pieces whatever the row phase.
// Shared-memory loads by 32-bit shared-window address (volatile: they must stay behind
// the mbarrier wait that publishes the stage).
template <int OFF> __device__ __forceinline__ uint32_t lds32(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.b32 %0, [%1+%2];" : "=r"(v) : "r"(a), "n"(OFF));
    return v;
}
template <int OFF> __device__ __forceinline__ uint32_t lds16(uint32_t a) {
    unsigned short v;
    asm volatile("ld.shared.u16 %0, [%1+%2];" : "=h"(v) : "r"(a), "n"(OFF));
    return (uint32_t)v;
}
__device__ __forceinline__ void lds128_pairs(uint32_t a, f32x2& x0, f32x2& x1) {
    asm volatile("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(x0), "=l"(x1) : "r"(a));
}
__device__ __forceinline__ uint4 lds128(uint32_t a) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}

template <int EB, int GB> struct PairLoad;
template <> struct PairLoad<4, 16> {
    __device__ static __forceinline__ void run(uint32_t a, f32x2 (&x)[2]) { lds128_pairs(a, x[0], x[1]); }
};
template <> struct PairLoad<2, 16> {
    __device__ static __forceinline__ void run(uint32_t a, f32x2 (&x)[4]) {
        const uint4 v = lds128(a);
        x[0] = bf16x2_widen(v.x); x[1] = bf16x2_widen(v.y); x[2] = bf16x2_widen(v.z); x[3] = bf16x2_widen(v.w);
    }
};
template <> struct PairLoad<4, 4> {
    __device__ static __forceinline__ void run(uint32_t a, f32x2 (&x)[2]) {
        x[0] = pair_bits(lds32<0>(a), lds32<128>(a));
        x[1] = pair_bits(lds32<256>(a), lds32<384>(a));
    }
};
template <> struct PairLoad<2, 4> {
    __device__ static __forceinline__ void run(uint32_t a, f32x2 (&x)[4]) {
        x[0] = bf16x2_widen(lds32<0>(a)); x[1] = bf16x2_widen(lds32<128>(a));
        x[2] = bf16x2_widen(lds32<256>(a)); x[3] = bf16x2_widen(lds32<384>(a));
    }
};
template <> struct PairLoad<2, 2> {
    __device__ static __forceinline__ void run(uint32_t a, f32x2 (&x)[4]) {
        x[0] = pair_bits(lds16<0>(a) << 16, lds16<64>(a) << 16);
        x[1] = pair_bits(lds16<128>(a) << 16, lds16<192>(a) << 16);
        x[2] = pair_bits(lds16<256>(a) << 16, lds16<320>(a) << 16);
        x[3] = pair_bits(lds16<384>(a) << 16, lds16<448>(a) << 16);
    }
};

// Stores of the same pieces; bit i of `mask` = piece i lies inside the row.
template <int EB, int GB> struct PairStore;
template <> struct PairStore<4, 16> {
    __device__ static __forceinline__ void run(unsigned char* p, const f32x2 (&a)[2], unsigned) {
        __stcs(reinterpret_cast<ulonglong2*>(p), make_ulonglong2(a[0], a[1]));
    }
};
template <> struct PairStore<2, 16> {
    __device__ static __forceinline__ void run(unsigned char* p, const f32x2 (&a)[4], unsigned) {
        __stcs(reinterpret_cast<uint4*>(p),
               make_uint4(pack_bf16x2_rn(pair_lo(a[0]), pair_hi(a[0])), pack_bf16x2_rn(pair_lo(a[1]), pair_hi(a[1])),
                          pack_bf16x2_rn(pair_lo(a[2]), pair_hi(a[2])), pack_bf16x2_rn(pair_lo(a[3]), pair_hi(a[3]))));
    }
};
// 32-bit streaming store executed only where `on` is non-zero (predicated, no branch)
__device__ __forceinline__ void stcs_b32_if(unsigned char* p, uint32_t v, unsigned on) {
    asm volatile("{ .reg .pred q; setp.ne.u32 q, %2, 0; @q st.global.cs.b32 [%0], %1; }" ::"l"(p), "r"(v), "r"(on));
}
template <> struct PairStore<4, 4> {
    __device__ static __forceinline__ void run(unsigned char* p, const f32x2 (&a)[2], unsigned mask) {
        stcs_b32_if(p, (uint32_t)a[0], mask & 1u);
        stcs_b32_if(p + 128, (uint32_t)(a[0] >> 32), mask & 2u);
        stcs_b32_if(p + 256, (uint32_t)a[1], mask & 4u);
        stcs_b32_if(p + 384, (uint32_t)(a[1] >> 32), mask & 8u);
    }
};
template <> struct PairStore<2, 4> {
    __device__ static __forceinline__ void run(unsigned char* p, const f32x2 (&a)[4], unsigned mask) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
            stcs_b32_if(p + i * 128, pack_bf16x2_rn(pair_lo(a[i]), pair_hi(a[i])), mask & (1u << i));
    }
};
template <> struct PairStore<2, 2> {
    __device__ static __forceinline__ void run(unsigned char* p, const f32x2 (&a)[4], unsigned mask) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t w = pack_bf16x2_rn(pair_lo(a[i]), pair_hi(a[i]));
            if (mask >> (2 * i) & 1u) __stcs(reinterpret_cast<unsigned short*>(p + (2 * i) * 64), (unsigned short)(w & 0xffffu));
            if (mask >> (2 * i + 1) & 1u) __stcs(reinterpret_cast<unsigned short*>(p + (2 * i + 1) * 64), (unsigned short)(w >> 16));
        }
    }
};

// Word-mode stores of a whole box: every piece lies inside the row except, for the lanes
// with `last_on` false, the last piece of the box's last 512-byte item (the box holds
// 16 bytes less than a whole number of items).
template <int EB, int GB> struct PairStoreBox;
template <> struct PairStoreBox<4, 4> {
    template <bool LAST>
    __device__ static __forceinline__ void run(unsigned char* p, const f32x2 (&a)[2], bool last_on) {
        __stcs(reinterpret_cast<uint32_t*>(p), (uint32_t)a[0]);
        __stcs(reinterpret_cast<uint32_t*>(p + 128), (uint32_t)(a[0] >> 32));
        __stcs(reinterpret_cast<uint32_t*>(p + 256), (uint32_t)a[1]);
        if (LAST) stcs_b32_if(p + 384, (uint32_t)(a[1] >> 32), last_on);
        else __stcs(reinterpret_cast<uint32_t*>(p + 384), (uint32_t)(a[1] >> 32));
    }
};
template <> struct PairStoreBox<2, 4> {
    template <bool LAST>
    __device__ static __forceinline__ void run(unsigned char* p, const f32x2 (&a)[4], bool last_on) {
#pragma unroll
        for (int i = 0; i < 3; ++i)
            __stcs(reinterpret_cast<uint32_t*>(p + i * 128), pack_bf16x2_rn(pair_lo(a[i]), pair_hi(a[i])));
        const uint32_t w3 = pack_bf16x2_rn(pair_lo(a[3]), pair_hi(a[3]));
        if (LAST) stcs_b32_if(p + 384, w3, last_on);             // predicated, no branch
        else __stcs(reinterpret_cast<uint32_t*>(p + 384), w3);
    }
};
template <> struct PairStoreBox<2, 2> {
    template <bool LAST>
    __device__ static __forceinline__ void run(unsigned char* p, const f32x2 (&a)[4], bool last_on) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t w = pack_bf16x2_rn(pair_lo(a[i]), pair_hi(a[i]));
            __stcs(reinterpret_cast<unsigned short*>(p + (2 * i) * 64), (unsigned short)(w & 0xffffu));
            if (i < 3 || !LAST || last_on)
                __stcs(reinterpret_cast<unsigned short*>(p + (2 * i + 1) * 64), (unsigned short)(w >> 16));
        }
    }
};

// ---------------------------------------------------------------- direct gather
template <int EB, bool SGD>
__device__ __forceinline__ float direct_x(const AggParams& p, int k, long long c) {
    const size_t off = ((size_t)k * (size_t)p.pitch + (size_t)c) * EB;
    float x = ElemOps<EB>::load(p.in + off);
    if (SGD) x = fmaf(-p.lr, ElemOps<EB>::load(p.grads + off), x);
    return x;
}

// Providers of (worker w, segment l) in the fixed order: the worker itself unless it is a
// newcomer, then its peers ascending (negative entries are absent); the worker alone if that
// leaves nobody.  Returns the count; prov needs room for R+1 entries only when R is small,
// so callers iterate with this helper instead of storing the list.
struct ProviderIter {
    const int32_t* peers;
    int w, R, pos;      // pos: -1 = self pending, 0..R-1 = next peer slot
    bool self_in;
    __device__ ProviderIter(const AggParams& p, int w_, long long l)
        : peers(p.R > 0 ? p.idx + ((size_t)w_ * p.S + (size_t)l) * (size_t)p.R : nullptr), w(w_), R(p.R), pos(-1) {
        self_in = !p.newcomer.get(w_);
        if (!self_in) {
            bool any = false;
            for (int r = 0; r < R; ++r) any |= peers[r] >= 0;
            if (!any) self_in = true;
        }
    }
    __device__ void rewind() { pos = -1; }
    // next provider or -1
    __device__ int next() {
        if (pos < 0) {
            pos = 0;
            if (self_in) return w;
        }
        while (pos < R) {
            const int k = peers[pos++];
            if (k >= 0) return k;
        }
        return -1;
    }
};

// One output element straight from the definition (providers, weight sum and coefficients
// worked out on the spot): for blocks that span more than two segments (segments shorter
// than a block), where the per-block tables below do not reach.
template <int EB, bool SGD>
__device__ __noinline__ void direct_element(const AggParams& p, int w, long long c) {
    ProviderIter pi(p, w, (p.p_begin + c) / p.L);
    float den = 0.0f;
    bool first = true;
    for (int k = pi.next(); k >= 0; k = pi.next()) {
        const float D = p.weights ? p.weights[k] : 1.0f;
        den = first ? D : __fadd_rn(den, D);
        first = false;
    }
    pi.rewind();
    int np = 0;
    for (int k = pi.next(); k >= 0; k = pi.next()) ++np;
    pi.rewind();
    float acc = 0.0f;
    first = true;
    for (int k = pi.next(); k >= 0; k = pi.next()) {
        const float cf = (np == 1 || !p.weights) ? 1.0f : p.weights[k];      // a single provider is taken as it is
        const float x = direct_x<EB, SGD>(p, k, c);
        acc = first ? __fmul_rn(cf, x) : fmaf(cf, x, acc);
        first = false;
    }
    if (np > 1) acc = __fmul_rn(acc, __fdiv_rn(1.0f, den));
    ElemOps<EB>::store(p.out + ((size_t)w * (size_t)p.pitch + (size_t)c) * EB, acc);
}

// Work is cut into blocks of 256 column groups of one worker's row.  The blocks are numbered
// with the WORKER running fastest, and CTAs take them in that order: at any moment the
// resident CTAs work on all workers' rows over the same narrow band of columns, so a provider
// row's piece that one worker has brought into L2 is still there when the R other workers
// that selected it ask for it -- the gather's re-reads are served by L2 and DRAM sees each
// input element about once.  (worker_major = 1 numbers the blocks row after row instead: the
// naive order, in which the re-reads of a row are spread over the whole run and mostly come
// from DRAM; kept as the contrast case for profiling.)
//
// Per block the providers and weights of the (at most two) segments it touches are worked
// out once, into shared memory: slot s of [2][R+1] holds the provider list and the weights
// |D_j| of segment la + s, la = the segment of the block's first column, and s_den[s] the
// scale 1 / sum |D_j| (Eq. 3 as written: numerator in the fixed order, times the reciprocal
// of the denominator; a single provider is taken as it is).
template <int EB, bool SGD>
__global__ void __launch_bounds__(256) k_direct(const AggParams p, long long blocks_per_row, int worker_major) {
    constexpr int V = ElemOps<EB>::V;
    extern __shared__ __align__(16) unsigned char dsm[];
    const int cap = p.R + 1;
    int* s_prov = reinterpret_cast<int*>(dsm);                       // [2][cap]
    float* s_coef = reinterpret_cast<float*>(s_prov + 2 * cap);      // [2][cap]
    __shared__ int s_np[2];
    __shared__ float s_den[2];
    const long long G = (p.width + V - 1) / V + 1;      // groups per row, phase spill included
    const bool rows_aligned = (p.pitch % V) == 0;
    const long long total = blocks_per_row * p.N;
    for (long long q = blockIdx.x; q < total; q += gridDim.x) {
        const long long blk = worker_major ? q % blocks_per_row : q / p.N;
        const int w = (int)(worker_major ? q / blocks_per_row : q % p.N);
        const int a_w = (int)(((long long)w * p.pitch) & (V - 1));
        // first column the block can touch and its segment
        long long cfirst = blk * 256LL * V - a_w;
        if (cfirst < 0) cfirst = 0;
        if (cfirst >= p.width) continue;                                 // uniform: nothing in this block
        const long long la = (p.p_begin + cfirst) / p.L;
        __syncthreads();                                                 // the previous block's readers are done
        if (threadIdx.x < 2) {
            // the provider list in the fixed order and the sum of the weights in that order
            const int sl = threadIdx.x;
            int np = 0;
            float den = 0.0f;
            if (la + sl < p.S) {
                ProviderIter pi(p, w, la + sl);
                for (int k = pi.next(); k >= 0; k = pi.next()) {
                    const float D = p.weights ? p.weights[k] : 1.0f;
                    den = np == 0 ? D : __fadd_rn(den, D);
                    s_prov[sl * cap + np++] = k;
                }
            }
            s_np[sl] = np;
            s_den[sl] = np > 1 ? __fdiv_rn(1.0f, den) : 1.0f;
        }
        __syncthreads();
        for (int t = threadIdx.x; t < 2 * cap; t += 256) {
            const int sl = t / cap, r = t - sl * cap;
            if (r < s_np[sl]) s_coef[t] = (s_np[sl] == 1 || !p.weights) ? 1.0f : p.weights[s_prov[t]];
        }
        __syncthreads();
        const long long g = blk * 256LL + threadIdx.x;
        if (g >= G) continue;
        const long long c0 = g * V - a_w;
        const long long lo = c0 < 0 ? 0 : c0;
        const long long hi = (c0 + V > p.width) ? p.width : c0 + V;
        if (lo >= hi) continue;
        const long long l_lo = (p.p_begin + lo) / p.L, l_hi = (p.p_begin + hi - 1) / p.L;
        if (hi - lo == V && l_lo == l_hi && rows_aligned && l_lo - la < 2) {
            const int sl = (int)(l_lo - la);
            const int np = s_np[sl];
            const int* prov = s_prov + sl * cap;
            const float* coef = s_coef + sl * cap;
            float acc[V], x[V];
            for (int r = 0; r < np; ++r) {
                const size_t off = ((size_t)prov[r] * (size_t)p.pitch + (size_t)c0) * EB;
                GroupLoad<EB, 16>::run(p.in + off, x);
                if (SGD) {
                    float gx[V];
                    GroupLoad<EB, 16>::run(p.grads + off, gx);
#pragma unroll
                    for (int i = 0; i < V; ++i) x[i] = fmaf(-p.lr, gx[i], x[i]);
                }
                const float c = coef[r];
                if (r == 0) {
#pragma unroll
                    for (int i = 0; i < V; ++i) acc[i] = __fmul_rn(c, x[i]);
                } else {
#pragma unroll
                    for (int i = 0; i < V; ++i) acc[i] = fmaf(c, x[i], acc[i]);
                }
            }
            const float scale = s_den[sl];
#pragma unroll
            for (int i = 0; i < V; ++i) acc[i] = __fmul_rn(scale, acc[i]);
            ElemOps<EB>::store_vec(p.out + ((size_t)w * (size_t)p.pitch + (size_t)c0) * EB, acc);
        } else {
            for (long long c = lo; c < hi; ++c) {
                const long long sl64 = (p.p_begin + c) / p.L - la;
                if (sl64 >= 2) { direct_element<EB, SGD>(p, w, c); continue; }
                const int sl = (int)sl64;
                const int np = s_np[sl];
                const int* prov = s_prov + sl * cap;
                const float* coef = s_coef + sl * cap;
                float acc = 0.0f;
                for (int r = 0; r < np; ++r) {
                    const float x = direct_x<EB, SGD>(p, prov[r], c);
                    acc = r == 0 ? __fmul_rn(coef[r], x) : fmaf(coef[r], x, acc);
                }
                acc = __fmul_rn(s_den[sl], acc);
                ElemOps<EB>::store(p.out + ((size_t)w * (size_t)p.pitch + (size_t)c) * EB, acc);
            }
        }
    }
}

// ---------------------------------------------------------------- mbarrier / TMA (PTX)
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("{ .reg .b64 st; mbarrier.arrive.shared::cta.b64 st, [%0]; }" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("{ .reg .b64 st; mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1; }" ::"r"(bar),
                 "r"(bytes)
                 : "memory");
}
// Bounded wait: false when the phase did not complete within kWaitCap polls.  The first
// polls return as soon as the hardware allows (hand-offs between producer and consumers
// are latency critical); later ones let the warp stay suspended for up to kWaitHintNs.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
#pragma unroll 1
    for (uint32_t it = 0; it < kFastPolls; ++it) {
        asm volatile(
            "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
    }
#pragma unroll 1
    for (uint32_t it = 0; it < kWaitCap; ++it) {
        asm volatile(
            "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3; selp.u32 %0, 1, 0, p; }"
            : "=r"(ok)
            : "r"(bar), "r"(parity), "r"(kWaitHintNs)
            : "memory");
        if (ok) return true;
    }
    return false;
}
// The producer warp is always ahead of the consumers, so it spends the kernel waiting for a
// free stage.  Spinning there would compete for issue slots with the consumer warps of the
// same scheduler; it sleeps between polls instead (a stage is re-armed a tile ahead of its
// use, so a fraction of a microsecond of wake-up latency costs nothing).
__device__ __forceinline__ bool mbar_wait_patient(uint32_t bar, uint32_t parity) {
    uint32_t ok;
#pragma unroll 1
    for (uint32_t it = 0; it < kWaitCap; ++it) {
        asm volatile(
            "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
        __nanosleep(256);
    }
    return false;
}
// Tiled 2-D TMA load of one box (x = element column, y = row of the class) into this CTA's
// shared memory; completion bytes are counted on `bar`.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}

// The same box brought into L2 only (no shared-memory destination, nothing to wait for).
__device__ __forceinline__ void tma_prefetch_2d(const CUtensorMap* map, int x, int y) {
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(map), "r"(x), "r"(y)
                 : "memory");
}

// 16 bytes, written and read as one vector (the producer's shared-memory operations queue
// behind the consumers' stores, so each one saved shortens its per-tile path)
struct alignas(16) TileMeta {
    long long bnd;   // local column where segment l0+1 starts
    int tile;        // tile held by the stage, or -1: no more work
    int l0;          // segment of the tile's first column
};


// shared-memory header: barriers and per-stage metadata
struct StagedHeader {
    unsigned long long full[kMaxStages];
    unsigned long long empty[kMaxStages];
    unsigned long long csync;            // consumer-wide barrier (16 arrivals)
    unsigned long long pad;
    TileMeta meta[kMaxStages];
};

__device__ __forceinline__ void staged_fail(int code) { atomicCAS(&g_dev_status, 0, code); }

// Bounded wait that never lets the warp be suspended for long: for barriers between
// consumer warps, which complete within a fraction of a microsecond.
__device__ __forceinline__ bool mbar_wait_brisk(uint32_t bar, uint32_t parity) {
    uint32_t ok;
#pragma unroll 1
    for (uint32_t it = 0; it < (kWaitCap << 3); ++it) {
        asm volatile(
            "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
    }
    return false;
}

// Self-check of the give-up path every bounded wait shares: one warp waits, with a cap of a
// thousand polls, on a barrier of its own that nothing ever arrives at, then reports through
// the status word exactly as the aggregation kernels do and returns.  Nothing is left armed:
// the barrier lives in this CTA's shared memory and no copy was started.
constexpr int kDebugWaitSite = 99;
__global__ void k_debug_dead_wait() {
    __shared__ unsigned long long bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const uint32_t b = smem_u32(&bar);
    uint32_t ok = 0;
#pragma unroll 1
    for (uint32_t it = 0; it < 1000u && !ok; ++it)
        asm volatile(
            "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
            : "=r"(ok)
            : "r"(b), "r"(0u)
            : "memory");
    if (!ok && threadIdx.x == 0) staged_fail(kDebugWaitSite);
}

// Consumer-wide barrier with a bounded wait (all 16 consumer warps).
__device__ __forceinline__ bool consumers_sync(uint32_t bar, uint32_t& phase, int lane) {
    __syncwarp();
    if (lane == 0) mbar_arrive(bar);
    bool ok = mbar_wait_brisk(bar, phase & 1u);
    phase ^= 1u;
    return ok;
}

// Eq. 3 is evaluated as it is written: the numerator sum |D_j| x_j is accumulated over the
// providers in the fixed order (the first term a product, the others fused multiply-adds),
// and the result is the numerator times the binary32 reciprocal of the denominator, which
// is summed in the same order.  A single provider is taken as it is (weight and scale 1).
//
// Coefficient table entry of one (slot, row): c2[RMAX+1] weights |D_j| of the providers,
// each already duplicated into a binary32 pair, then poff[RMAX+1] ints (shared-memory byte
// offset of each provider's staged row inside a box block, its phase included), then the
// scale 1 / sum |D_j| as one float; padded to 16.
__host__ __device__ constexpr int table_entry_bytes(int rmax) { return ((rmax + 1) * 12 + 4 + 15) / 16 * 16; }
__host__ __device__ constexpr int entry_scale_word(int rmax) { return 3 * (rmax + 1); }

template <int RMAX>
struct RowCtx {
    f32x2 c2[RMAX + 1];    // weight of each provider, duplicated into a pair
    int poff[RMAX + 1];
    f32x2 s2;              // the scale, duplicated
};

// `entry` is the entry's shared-window address; it is read as whole 128-bit vectors exactly
// once (through the generic pointer the compiler fetched some coefficient pairs a second time).
template <int RMAX>
__device__ __forceinline__ void load_entry(uint32_t entry, RowCtx<RMAX>& c) {
    constexpr int ENT = table_entry_bytes(RMAX);
    uint32_t raw[ENT / 4];
#pragma unroll
    for (int i = 0; i < ENT / 16; ++i) {
        const uint4 v = lds128(entry + 16 * i);
        raw[4 * i] = v.x; raw[4 * i + 1] = v.y; raw[4 * i + 2] = v.z; raw[4 * i + 3] = v.w;
    }
#pragma unroll
    for (int r = 0; r <= RMAX; ++r) {
        c.c2[r] = pair_bits(raw[2 * r], raw[2 * r + 1]);
        c.poff[r] = (int)raw[2 * (RMAX + 1) + r];
    }
    c.s2 = pair_bits(raw[entry_scale_word(RMAX)], raw[entry_scale_word(RMAX)]);
}

// One lane's share of an item (512 bytes of an output row): self first, then the
// peers ascending (Eq. 3, fixed order).  Loads are never masked: a piece beyond the
// row's payload reads bytes that still lie inside the stage (or its 16-byte slack)
// and its result is dropped by the store mask.
template <int EB, int GB, int RMAX, bool FIXED_R>
__device__ __forceinline__ void item_fast(uint32_t base, const RowCtx<RMAX>& c, int R, unsigned char* outp,
                                          unsigned mask) {
    constexpr int NP = ElemOps<EB>::V / 2;
    f32x2 acc[NP], x[NP];
    PairLoad<EB, GB>::run(base + c.poff[0], x);
#pragma unroll
    for (int i = 0; i < NP; ++i) acc[i] = mul2(c.c2[0], x[i]);
#pragma unroll
    for (int r = 1; r <= RMAX; ++r) {
        if (FIXED_R || r <= R) {
            PairLoad<EB, GB>::run(base + c.poff[r], x);
#pragma unroll
            for (int i = 0; i < NP; ++i) acc[i] = fma2(c.c2[r], x[i], acc[i]);
        }
    }
#pragma unroll
    for (int i = 0; i < NP; ++i) acc[i] = mul2(c.s2, acc[i]);
    PairStore<EB, GB>::run(outp, acc, mask);
}

// The same for a lane's share of an item of a whole word-mode box (see PairStoreBox).
template <int EB, int GB, int RMAX, bool FIXED_R, bool LAST>
__device__ __forceinline__ void item_box(uint32_t base, const RowCtx<RMAX>& c, int R, unsigned char* outp,
                                         bool last_on) {
    constexpr int NP = ElemOps<EB>::V / 2;
    f32x2 acc[NP], x[NP];
    PairLoad<EB, GB>::run(base + c.poff[0], x);
#pragma unroll
    for (int i = 0; i < NP; ++i) acc[i] = mul2(c.c2[0], x[i]);
#pragma unroll
    for (int r = 1; r <= RMAX; ++r) {
        if (FIXED_R || r <= R) {
            PairLoad<EB, GB>::run(base + c.poff[r], x);
#pragma unroll
            for (int i = 0; i < NP; ++i) acc[i] = fma2(c.c2[r], x[i], acc[i]);
        }
    }
#pragma unroll
    for (int i = 0; i < NP; ++i) acc[i] = mul2(c.s2, acc[i]);
    PairStoreBox<EB, GB>::template run<LAST>(outp, acc, last_on);
}

// ---- bfloat16 rows with unit weights (weights == NULL) --------------------------------
// The numerator of Eq. 3 is then the plain sum of the providers' values in the fixed order,
// and sm_100 adds a bfloat16 operand to a binary32 one in a single instruction
// (add.rn.f32.bf16: the bfloat16 value is widened exactly, one rounding, either half of a
// 32-bit register) -- the same result as widening first and adding, without the two integer
// instructions per packed word that the widening costs.  Entries need no weights:
// poff[RMAX+1], the scale 1 / np as one float, np = number of providers; padded to 16.
// Providers are packed into the first np slots; the others are never read.
__host__ __device__ constexpr int entry_unw_bytes(int rmax) { return ((rmax + 1) * 4 + 8 + 15) / 16 * 16; }

template <int RMAX>
struct RowCtxU {
    int poff[RMAX + 1];
    f32x2 s2;
    int np;
};
template <int RMAX, bool UNW> struct CtxSel { typedef RowCtx<RMAX> type; };
template <int RMAX> struct CtxSel<RMAX, true> { typedef RowCtxU<RMAX> type; };
template <int RMAX, bool UNW> __host__ __device__ constexpr int entry_bytes_of() {
    return UNW ? entry_unw_bytes(RMAX) : table_entry_bytes(RMAX);
}

template <int RMAX>
__device__ __forceinline__ void load_entry(uint32_t entry, RowCtxU<RMAX>& c) {
    constexpr int ENT = entry_unw_bytes(RMAX);
    uint32_t raw[ENT / 4];
#pragma unroll
    for (int i = 0; i < ENT / 16; ++i) {
        const uint4 v = lds128(entry + 16 * i);
        raw[4 * i] = v.x; raw[4 * i + 1] = v.y; raw[4 * i + 2] = v.z; raw[4 * i + 3] = v.w;
    }
#pragma unroll
    for (int r = 0; r <= RMAX; ++r) c.poff[r] = (int)raw[r];
    c.s2 = pair_bits(raw[RMAX + 1], raw[RMAX + 1]);
    c.np = (int)raw[RMAX + 2];
}

// binary32 + bfloat16 from the low / the high half of a packed word
__device__ __forceinline__ float add_bf16_lo(uint32_t w, float c) {
    const unsigned short h = (unsigned short)(w & 0xffffu);
    asm("add.rn.f32.bf16 %0, %1, %0;" : "+f"(c) : "h"(h));
    return c;
}
__device__ __forceinline__ float add_bf16_hi(uint32_t w, float c) {
    const unsigned short h = (unsigned short)(w >> 16);
    asm("add.rn.f32.bf16 %0, %1, %0;" : "+f"(c) : "h"(h));
    return c;
}

// the four packed words of a lane's share of an item
template <int GB> struct WordLoad;
template <> struct WordLoad<16> {
    __device__ static __forceinline__ void run(uint32_t a, uint32_t (&w)[4]) {
        const uint4 v = lds128(a);
        w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
    }
};
template <> struct WordLoad<4> {
    __device__ static __forceinline__ void run(uint32_t a, uint32_t (&w)[4]) {
        w[0] = lds32<0>(a); w[1] = lds32<128>(a); w[2] = lds32<256>(a); w[3] = lds32<384>(a);
    }
};

// Sum of the providers' values in the fixed order, times the scale: a lane's share of an item.
template <int GB, int RMAX, bool FIXED_R>
__device__ __forceinline__ void sum_unw(uint32_t base, const RowCtxU<RMAX>& c, f32x2 (&acc)[4]) {
    uint32_t w[4];
    float a[8];
    WordLoad<GB>::run(base + c.poff[0], w);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        a[2 * i] = __uint_as_float(w[i] << 16);
        a[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
    if (FIXED_R && c.np == RMAX + 1) {
        // all replicas present (the usual case): straight-line code
#pragma unroll
        for (int r = 1; r <= RMAX; ++r) {
            WordLoad<GB>::run(base + c.poff[r], w);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                a[2 * i] = add_bf16_lo(w[i], a[2 * i]);
                a[2 * i + 1] = add_bf16_hi(w[i], a[2 * i + 1]);
            }
        }
    } else {
#pragma unroll
        for (int r = 1; r <= RMAX; ++r) {
            if (r < c.np) {
                WordLoad<GB>::run(base + c.poff[r], w);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    a[2 * i] = add_bf16_lo(w[i], a[2 * i]);
                    a[2 * i + 1] = add_bf16_hi(w[i], a[2 * i + 1]);
                }
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
        acc[i] = mul2(c.s2, pair_bits(__float_as_uint(a[2 * i]), __float_as_uint(a[2 * i + 1])));
}
template <int EB, int GB, int RMAX, bool FIXED_R>
__device__ __forceinline__ void item_fast(uint32_t base, const RowCtxU<RMAX>& c, int, unsigned char* outp,
                                          unsigned mask) {
    static_assert(EB == 2 && (GB == 16 || GB == 4), "bfloat16 only");
    f32x2 acc[4];
    sum_unw<GB, RMAX, FIXED_R>(base, c, acc);
    PairStore<EB, GB>::run(outp, acc, mask);
}
template <int EB, int GB, int RMAX, bool FIXED_R, bool LAST>
__device__ __forceinline__ void item_box(uint32_t base, const RowCtxU<RMAX>& c, int, unsigned char* outp,
                                         bool last_on) {
    static_assert(EB == 2 && GB == 4, "bfloat16 word mode only");
    f32x2 acc[4];
    sum_unw<GB, RMAX, FIXED_R>(base, c, acc);
    PairStoreBox<EB, GB>::template run<LAST>(outp, acc, last_on);
}

// Fused local step on a staged tile, in place: x <- fma(-lr, g, x) for every staged row; the
// gradients of the tile lie `bytes` behind the parameters.  Thread t of nthreads.
__device__ __forceinline__ void sgd_step_in_place(unsigned char* stage, int bytes, float lr, int t, int nthreads) {
    const int nvec = bytes / 16;
    float4* xs = reinterpret_cast<float4*>(stage);
    const float4* gs = reinterpret_cast<const float4*>(stage + (size_t)bytes);
    const float nlr = -lr;
    for (int v = t; v < nvec; v += nthreads) {
        float4 x = xs[v];
        const float4 g = gs[v];
        x.x = fmaf(nlr, g.x, x.x); x.y = fmaf(nlr, g.y, x.y);
        x.z = fmaf(nlr, g.z, x.z); x.w = fmaf(nlr, g.w, x.w);
        xs[v] = x;
    }
}

// Coefficient / offset table of `nslots` consecutive segments starting at l0_build, built by
// `nthreads` threads of which the caller is number t: entry [slot][w] of ENT bytes.
template <int EB, int RMAX, bool UNW = false>
__device__ __forceinline__ void build_coef_table(const AggParams& p, unsigned char* tab, int R, int l0_build,
                                                 int nslots, int t, int nthreads) {
    constexpr int ENT = entry_bytes_of<RMAX, UNW>();
    const int N = p.N;
    for (int q = t; q < nslots * N; q += nthreads) {
        const int slot = q / N, w = q - slot * N;
        const int l = l0_build + slot;
        if (l < p.S) {
            const int32_t* peers = p.idx + ((size_t)w * p.S + (size_t)l) * (size_t)R;
            float* cf = reinterpret_cast<float*>(tab + ((size_t)slot * N + w) * ENT);   // pairs
            int* po = UNW ? reinterpret_cast<int*>(cf) : reinterpret_cast<int*>(cf + 2 * (RMAX + 1));
            // providers in the fixed order: the worker itself (unless it is a newcomer), then
            // the peers ascending; a negative entry is a pull that found no online peer
            int prov[RMAX + 1];
            int np = 0;
            if (!p.newcomer.get(w)) prov[np++] = w;
            for (int r = 0; r < R; ++r) {
                const int k = peers[r];
                if (k >= 0) prov[np++] = k;
            }
            if (np == 0) prov[np++] = w;                 // nothing to aggregate: keep the own values
            float den = p.weights ? p.weights[prov[0]] : 1.0f;
            for (int i = 1; i < np; ++i) den = __fadd_rn(den, p.weights ? p.weights[prov[i]] : 1.0f);
            // a single provider is taken as it is
            const float scale = np == 1 ? 1.0f : __fdiv_rn(1.0f, den);
            if (UNW) {
                cf[RMAX + 1] = scale;
                po[RMAX + 2] = np;
            } else {
                cf[entry_scale_word(RMAX)] = scale;
            }
            for (int r = 0; r < np; ++r) {
                const int k = prov[r];
                if (!UNW) cf[2 * r] = cf[2 * r + 1] = (np == 1 || !p.weights) ? 1.0f : p.weights[k];
                // staged row of worker k: classes are stored one after another
                const int jk = k % p.m;
                int base = 0;
                for (int q2 = 0; q2 < jk; ++q2) base += (N - q2 + p.m - 1) / p.m;
                const int phase = (int)(((long long)k * p.pitch * EB) & 15);
                po[r] = (base + k / p.m) * p.row_bytes + phase;
            }
            // unused slots: weight zero on a row that is known to hold finite values
            for (int r = np; r <= RMAX; ++r) {
                if (!UNW) cf[2 * r] = cf[2 * r + 1] = 0.0f;
                po[r] = po[0];
            }
        }
    }
}

// The share of a tile that one of `nwarps` warps works on.  A unit of work is one row of one
// x-box: CPB chunks of 512 bytes; a warp takes a contiguous range of units.
template <int EB, int GB>
struct WarpShare {
    static constexpr int CPB = (EB == 4) ? 2 : 1;         // boxes are at most 256 elements wide
    static constexpr int PIECES = 16 / GB;                // pieces a lane owns per item
    static constexpr int PSTRIDE = 32 * GB;               // bytes between a lane's pieces
    int u_begin, u_end, row_begin, xb_begin;
    int cw, nwarps;                                       // this warp's number among those sharing the tile
    int box_payload;                                      // tile bytes per row held by one x-box
    size_t pitch_bytes;
    unsigned pmask[CPB];    // store masks of the unit's chunks: bit i = piece i of this lane lies inside the payload
    __device__ __forceinline__ WarpShare(const AggParams& p, int cw_, int nwarps_, int lane) : cw(cw_), nwarps(nwarps_) {
        box_payload = (p.T / p.nbx) * EB;
        const int n_units = p.N * p.nbx;
        const int upw = (n_units + nwarps - 1) / nwarps;
        u_begin = cw * upw;
        u_end = (cw + 1) * upw < n_units ? (cw + 1) * upw : n_units;
        row_begin = u_begin / p.nbx;
        xb_begin = u_begin - row_begin * p.nbx;
        pitch_bytes = (size_t)p.pitch * EB;
#pragma unroll
        for (int ch = 0; ch < CPB; ++ch) {
            pmask[ch] = 0;
#pragma unroll
            for (int i = 0; i < PIECES; ++i)
                if (ch * 512 + lane * GB + i * PSTRIDE < box_payload) pmask[ch] |= 1u << i;
        }
    }
};

// ---------------------------------------------------------------- dense evaluation (many replicas)
// With R + 1 providers per output the warp-per-row loop reads R + 1 staged rows per output
// row; beyond R of about 8 those shared-memory reads, not HBM, set the pace.  When R + 1 is a
// good part of N (the paper sweeps R up to 16 with 30 workers, Section 5.2) it is cheaper to
// take a BLOCK of BR output rows at once and walk over ALL N staged rows: each staged piece
// is read once per block and multiplied into the BR accumulators with that row's
// coefficients, which are zero where the row is not a provider.  fma(0, x, acc) leaves acc
// as it is for finite x, so every output still sees exactly the fixed order of Eq. 3 (own
// term first, then providers ascending).  Rows must hold finite values, all of them, since
// every row meets every accumulator; not used when a newcomer flag is set (a newcomer's own
// row must never be read).
// A block is as many output rows as keep the accumulators within 32 registers of pairs: 8 of
// binary32 (a lane's 16 bytes are 4 elements), 4 of bfloat16 (8 elements).  Per staged row a
// unit then reads 512 bytes of data and 32 or 16 bytes of coefficients.  (Twice the columns
// per lane would halve the coefficient reads per output but spills registers, which measured
// no faster than the warp-per-row form.)
template <int EB> struct DenseRows {
    static constexpr int BR = (EB == 4) ? 8 : 4;
    static constexpr int CH = 1;                     // 512-byte chunks a unit spans
};

// Dense coefficient blocks of `nslots` segments: [slot][block][k = 0..N+1][BR] floats; k < N:
// weight |D_k| of staged row k for output row BR*block + b, zero if it is not a provider or is
// the output row itself; k = N: the output row's own weight; k = N + 1: its scale 1 / sum.
template <int EB>
__device__ __forceinline__ void build_dense_table(const AggParams& p, unsigned char* dtab, int R, int l0_build,
                                                  int nslots, int t, int nthreads) {
    constexpr int BR = DenseRows<EB>::BR;
    const int N = p.N;
    const int nblk = (N + BR - 1) / BR;
    for (int q = t; q < nslots * nblk * BR; q += nthreads) {
        const int slot = q / (nblk * BR), w = q - slot * nblk * BR;     // w may be a padding row >= N
        const int l = l0_build + slot;
        if (l >= p.S) continue;
        float* col = reinterpret_cast<float*>(dtab + (size_t)slot * p.dslot_bytes) +
                     (size_t)(w / BR) * (N + 2) * BR + (w % BR);
        for (int k = 0; k <= N + 1; ++k) col[(size_t)k * BR] = 0.0f;
        if (w >= N) continue;
        const int32_t* peers = p.idx + ((size_t)w * p.S + (size_t)l) * (size_t)R;
        float den = p.weights ? p.weights[w] : 1.0f;
        int np = 1;
        for (int r = 0; r < R; ++r)
            if (peers[r] >= 0) { den = __fadd_rn(den, p.weights ? p.weights[peers[r]] : 1.0f); ++np; }
        // a single provider is taken as it is
        col[(size_t)N * BR] = (np == 1 || !p.weights) ? 1.0f : p.weights[w];
        col[(size_t)(N + 1) * BR] = np == 1 ? 1.0f : __fdiv_rn(1.0f, den);
        for (int r = 0; r < R; ++r) {
            const int k = peers[r];
            if (k >= 0) col[(size_t)k * BR] = p.weights ? p.weights[k] : 1.0f;
        }
    }
}

// the BR coefficients of one staged row, each duplicated into a pair
template <int BR>
__device__ __forceinline__ void dense_coefs(uint32_t a, f32x2 (&c)[BR]) {
#pragma unroll
    for (int b = 0; b < BR; b += 4) {
        const uint4 v = lds128(a + b * 4);
        c[b] = pair_bits(v.x, v.x); c[b + 1] = pair_bits(v.y, v.y);
        c[b + 2] = pair_bits(v.z, v.z); c[b + 3] = pair_bits(v.w, v.w);
    }
}

// A whole tile lying in one segment, dense: warp number cw of nwarps takes the units
// (row block, group of CH chunks) cw, cw + nwarps, ...
template <int EB>
__device__ __forceinline__ void aggregate_dense(const AggParams& p, uint32_t stage_s, const unsigned char* dtab0,
                                                long long t0, int cw, int nwarps, int lane) {
    constexpr int BR = DenseRows<EB>::BR;
    constexpr int CH = DenseRows<EB>::CH;
    constexpr int NP = ElemOps<EB>::V / 2;          // pairs per 16-byte piece
    const int N = p.N;
    const int nblk = (N + BR - 1) / BR;
    const int box_payload = (p.T / p.nbx) * EB;     // a multiple of CH * 512 (checked by the planner)
    const int groups_per_box = box_payload / (CH * 512);
    const int groups = p.nbx * groups_per_box;
    const int block_bytes = N * p.row_bytes;
    const size_t pitch_bytes = (size_t)p.pitch * EB;
    const uint32_t dt_s = smem_u32(dtab0);
    for (int u = cw; u < nblk * groups; u += nwarps) {
        const int blk = u / groups, gq = u - blk * groups;
        const int xb = gq / groups_per_box, gi = gq - xb * groups_per_box;
        const int w0 = blk * BR;
        const int col_off = gi * CH * 512 + lane * 16;                 // byte offset inside the box payload
        const uint32_t base = stage_s + xb * block_bytes + col_off;
        uint32_t ct = dt_s + (uint32_t)(blk * (N + 2) * BR * 4);
        f32x2 acc[BR][CH * NP], x[CH * NP], c[BR];
        // own terms first
        dense_coefs<BR>(ct + (uint32_t)(N * BR * 4), c);
#pragma unroll
        for (int b = 0; b < BR; ++b) {
            const int w = w0 + b < N ? w0 + b : N - 1;                  // padding rows: any staged row, coefficient 0
#pragma unroll
            for (int h = 0; h < CH; ++h) {
                f32x2 xx[NP];
                PairLoad<EB, 16>::run(base + w * p.row_bytes + h * 512, xx);
#pragma unroll
                for (int i = 0; i < NP; ++i) acc[b][h * NP + i] = mul2(c[b], xx[i]);
            }
        }
        // then every staged row in ascending order
        uint32_t xa = base;
#pragma unroll 1
        for (int k = 0; k < N; ++k) {
#pragma unroll
            for (int h = 0; h < CH; ++h) {
                f32x2 xx[NP];
                PairLoad<EB, 16>::run(xa + h * 512, xx);
#pragma unroll
                for (int i = 0; i < NP; ++i) x[h * NP + i] = xx[i];
            }
            dense_coefs<BR>(ct, c);
#pragma unroll
            for (int b = 0; b < BR; ++b)
#pragma unroll
                for (int i = 0; i < CH * NP; ++i) acc[b][i] = fma2(c[b], x[i], acc[b][i]);
            xa += p.row_bytes;
            ct += BR * 4;
        }
        // ct now points at row N (the own weights); the scales follow
        dense_coefs<BR>(ct + (uint32_t)(BR * 4), c);
        unsigned char* o = p.out + (size_t)w0 * pitch_bytes + (size_t)t0 * EB + (size_t)xb * box_payload + col_off;
#pragma unroll
        for (int b = 0; b < BR; ++b) {
#pragma unroll
            for (int i = 0; i < CH * NP; ++i) acc[b][i] = mul2(c[b], acc[b][i]);
            if (w0 + b < N) {
#pragma unroll
                for (int h = 0; h < CH; ++h) {
                    f32x2 r[NP];
#pragma unroll
                    for (int i = 0; i < NP; ++i) r[i] = acc[b][h * NP + i];
                    PairStore<EB, 16>::run(o + (size_t)b * pitch_bytes + h * 512, r, 0xffu);
                }
            }
        }
    }
}

// One warp's share of a staged tile: Eq. 3 in the fixed order for every unit of `ws`, results
// stored to the output rows.  `stage` holds the tile (its shared-window address is stage_s),
// tab0 the table entries of segment l0 (those of l0 + 1 follow them), m_bnd is the local
// column where segment l0 + 1 starts.
template <int EB, int GB, int RT, bool UNW = false>
__device__ __forceinline__ void aggregate_tile(const AggParams& p, const WarpShare<EB, GB>& ws,
                                               const unsigned char* stage, uint32_t stage_s,
                                               const unsigned char* tab0, long long tile, long long m_bnd,
                                               int lane, const unsigned char* dtab0 = nullptr) {
    constexpr int V = ElemOps<EB>::V;
    constexpr int RMAX = rmax_of(RT);
    constexpr int ENT = entry_bytes_of<RMAX, UNW>();
    typedef typename CtxSel<RMAX, UNW>::type Ctx;
    constexpr int CPB = WarpShare<EB, GB>::CPB;
    constexpr int PIECES = WarpShare<EB, GB>::PIECES;
    constexpr int PSTRIDE = WarpShare<EB, GB>::PSTRIDE;
    constexpr int EPP = GB / EB;               // elements per piece
    const int N = p.N, R = (RT >= 0) ? RT : p.R;
    const int block_bytes = (p.stage_rows ? p.stage_rows : N) * p.row_bytes;   // one x-box of all rows
    const int box_payload = ws.box_payload;
    const size_t pitch_bytes = ws.pitch_bytes;
    const int u_begin = ws.u_begin, u_end = ws.u_end;
    const long long t0 = tile * (long long)p.T;
    const long long t1 = (t0 + p.T < p.width) ? t0 + p.T : p.width;
    const bool interior = (m_bnd >= t1) && (t0 + p.T <= p.width);   // one segment, whole tile
    const uint32_t tab_s = smem_u32(tab0);
    if constexpr (RT == -3 && GB == 16) {
        if (interior) {
            aggregate_dense<EB>(p, stage_s, dtab0, t0, ws.cw, ws.nwarps, lane);
            return;
        }
    }

    int row = ws.row_begin, xb = ws.xb_begin;
    if (GB < 16 && interior) {
        // word mode: a unit is a whole row of a box, and only the last piece of it can lie
        // outside the box's payload (a loop-invariant lane predicate)
        if constexpr (GB < 16) {
            Ctx c;
            const uint32_t lane_base = stage_s + lane * GB;
            const bool last_on = (CPB - 1) * 512 + lane * GB + (PIECES - 1) * PSTRIDE < box_payload;
            if (p.nbx == 1) {
                // the tile is one box (many rows): a unit is a row
                uint32_t ent = tab_s + (uint32_t)(u_begin * ENT);
                unsigned char* orow = p.out + (size_t)u_begin * pitch_bytes + (size_t)t0 * EB + lane * GB;
                // The entry of the next row is fetched while this row is worked on (the last
                // fetch reads the entry behind the warp's rows: inside the table or the stage
                // ring, never used).
                // (Not with the wide entries of the many-replica kernels: they would spill.)
                constexpr bool AHEAD = RMAX <= 8;
                typename CtxSel<AHEAD ? RMAX : 0, UNW>::type c_next;
                if constexpr (AHEAD) load_entry<RMAX>(ent, c_next);
#pragma unroll 4   // measured: 2 -> 4 gains 1.7 % with 128 bf16 rows, 8 gains nothing
                for (int u = u_begin; u < u_end; ++u) {
                    if constexpr (AHEAD) {
                        c = c_next;
                        load_entry<RMAX>(ent + ENT, c_next);
                    } else {
                        load_entry<RMAX>(ent, c);
                    }
#pragma unroll
                    for (int ch = 0; ch < CPB - 1; ++ch)
                        item_box<EB, GB, RMAX, (RT >= 0), false>(lane_base + ch * 512, c, R, orow + ch * 512, true);
                    item_box<EB, GB, RMAX, (RT >= 0), true>(lane_base + (CPB - 1) * 512, c, R,
                                                            orow + (CPB - 1) * 512, last_on);
                    ent += ENT;
                    orow += pitch_bytes;
                }
            } else {
                // several boxes per tile (few rows): rows outside, boxes inside
                const int nbx = p.nbx;
                uint32_t ent = tab_s + (uint32_t)(row * ENT);
                unsigned char* orow = p.out + (size_t)row * pitch_bytes + (size_t)t0 * EB + lane * GB;
                int u = u_begin;
                while (u < u_end) {
                    load_entry<RMAX>(ent, c);
                    for (; xb < nbx && u < u_end; ++xb, ++u) {
                        const uint32_t ubase = lane_base + xb * block_bytes;
                        unsigned char* uout = orow + xb * box_payload;
#pragma unroll
                        for (int ch = 0; ch < CPB - 1; ++ch)
                            item_box<EB, GB, RMAX, (RT >= 0), false>(ubase + ch * 512, c, R, uout + ch * 512, true);
                        item_box<EB, GB, RMAX, (RT >= 0), true>(ubase + (CPB - 1) * 512, c, R,
                                                                uout + (CPB - 1) * 512, last_on);
                    }
                    xb = 0;
                    ent += ENT;
                    orow += pitch_bytes;
                }
            }
        }
    } else if (GB == 16 && interior && box_payload <= 256) {
        // quarter-kilobyte row pieces (so many rows that wider ones do not fit): a warp takes
        // two rows at a time, one per half-warp, each lane its 16 bytes
        const int half = lane >> 4, hl = lane & 15;
        Ctx c;
        const uint32_t lane_base = stage_s + hl * 16;
        unsigned char* ocol = p.out + (size_t)t0 * EB + hl * 16;
        for (int u = u_begin; u < u_end; u += 2) {
            const int myrow = u + half;
            if (myrow < u_end && hl * 16 < box_payload) {
                load_entry<RMAX>(tab_s + (uint32_t)(myrow * ENT), c);
                item_fast<EB, GB, RMAX, (RT >= 0)>(lane_base, c, R, ocol + (size_t)myrow * pitch_bytes, 0xffu);
            }
        }
    } else if (interior) {
        // every unit is whole and lies in segment l0: the lean loop, rows outside, boxes inside
        Ctx c;
        const int nbx = p.nbx;
        uint32_t ent = tab_s + (uint32_t)(row * ENT);
        unsigned char* orow = p.out + (size_t)row * pitch_bytes + (size_t)t0 * EB + lane * GB;
        const uint32_t lane_base = stage_s + lane * GB;
        int u = u_begin;
        while (u < u_end) {
            load_entry<RMAX>(ent, c);
            for (; xb < nbx && u < u_end; ++xb, ++u) {
                const uint32_t ubase = lane_base + xb * block_bytes;
                unsigned char* uout = orow + xb * box_payload;
#pragma unroll
                for (int ch = 0; ch < CPB; ++ch)
                    if (ch * 512 < box_payload)
                        item_fast<EB, GB, RMAX, (RT >= 0)>(ubase + ch * 512, c, R, uout + ch * 512, ws.pmask[ch]);
            }
            xb = 0;
            ent += ENT;
            orow += pitch_bytes;
        }
    } else {
        // last tile of the rows, or a tile holding a segment boundary: element by element,
        // except whole 128-bit groups that lie in one segment
        for (int u = u_begin; u < u_end; ++u) {
#pragma unroll 1
            for (int ch = 0; ch < CPB; ++ch) {
                if (ch * 512 >= box_payload) continue;               // half-width boxes hold one item per row
                const int ib = xb * box_payload + ch * 512;          // byte offset of the item in the row
                const uint32_t ubase = stage_s + xb * block_bytes + ch * 512 + lane * GB;
                bool done = false;
                if (GB == 16 && ch * 512 + lane * 16 < box_payload) {
                    const long long c0 = t0 + (ib + lane * 16) / EB;
                    const bool whole = c0 + V <= p.width;
                    const bool one_seg = (c0 + V <= m_bnd) || (c0 >= m_bnd);
                    if (whole && one_seg) {
                        Ctx cc;
                        load_entry<RMAX>(tab_s + (uint32_t)(((c0 >= m_bnd ? 1 : 0) * N + row) * ENT), cc);
                        item_fast<EB, GB, RMAX, (RT >= 0)>(
                            ubase, cc, R, p.out + (size_t)row * pitch_bytes + (size_t)c0 * EB, 0xffu);
                        done = true;
                    }
                }
                if (!done) {
#pragma unroll 1
                    for (int i = 0; i < PIECES; ++i) {
                        const int pin = ch * 512 + lane * GB + i * PSTRIDE;  // byte offset inside the box payload
                        if (pin >= box_payload) continue;
#pragma unroll 1
                        for (int e = 0; e < EPP; ++e) {
                            const long long col = t0 + (xb * box_payload + pin) / EB + e;
                            if (col >= p.width) continue;
                            const unsigned char* ent = tab0 + ((size_t)(col >= m_bnd ? 1 : 0) * N + row) * ENT;
                            const float* cf = reinterpret_cast<const float*>(ent);       // pairs
                            const unsigned char* eb = stage + xb * block_bytes + pin + e * EB;
                            float acc;
                            if constexpr (UNW) {
                                const int* po = reinterpret_cast<const int*>(ent);
                                const int np = po[RMAX + 2];
                                acc = ElemOps<EB>::load(eb + po[0]);
                                for (int r = 1; r < np; ++r) acc = __fadd_rn(ElemOps<EB>::load(eb + po[r]), acc);
                                acc = __fmul_rn(cf[RMAX + 1], acc);
                            } else {
                                const int* po = reinterpret_cast<const int*>(cf + 2 * (RMAX + 1));
                                acc = __fmul_rn(cf[0], ElemOps<EB>::load(eb + po[0]));
                                for (int r = 1; r <= R; ++r)
                                    acc = fmaf(cf[2 * r], ElemOps<EB>::load(eb + po[r]), acc);
                                acc = __fmul_rn(cf[entry_scale_word(RMAX)], acc);
                            }
                            ElemOps<EB>::store(p.out + (size_t)row * pitch_bytes + (size_t)col * EB, acc);
                        }
                    }
                }
            }
            if (++xb == p.nbx) { xb = 0; ++row; }
        }
    }
}

template <int EB, int GB, bool SGD, int RT, bool UNW = false>
__global__ void __launch_bounds__(kStagedThreads, 1)
k_staged(const AggParams p, const __grid_constant__ TileMaps maps) {
    // RT: the number of replicas the kernel is specialised on, -1 = any up to kGenericR,
    // -2 = any up to kStagedMaxR.  UNW: bfloat16 rows with unit weights (see RowCtxU).
    constexpr int RMAX = rmax_of(RT);
    constexpr int ENT = entry_bytes_of<RMAX, UNW>();
    extern __shared__ __align__(128) unsigned char smem[];
    StagedHeader* hdr = reinterpret_cast<StagedHeader*>(smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int N = p.N, R = (RT >= 0) ? RT : p.R;
    const int stages = p.stages;
    const int narr = SGD ? 2 : 1;
    unsigned char* tab = smem + p.tab_off;                 // [tab_slots][N] entries of ENT bytes
    const bool whole_table = p.tab_slots >= p.S;           // every segment has its slot: never rebuilt
    const int block_bytes = N * p.row_bytes;               // one x-box of all rows

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(&hdr->full[s]), 1);
            mbar_init(smem_u32(&hdr->empty[s]), kConsumerWarps);
        }
        mbar_init(smem_u32(&hdr->csync), kConsumerWarps);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // When launched with programmatic stream serialization this CTA may have started while
    // the preceding kernel of the stream was still draining: everything above touched only
    // this CTA's shared memory.  From here on global memory is read and written, so wait for
    // that kernel to have completed, then let the next launch of the stream start its own
    // set-up as SMs become free.  (Both are no-ops in an ordinary launch.)
    auto wait_for_preceding_kernel = [] {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    };

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        // lane -> one TMA box per tile: (array a, x-box b, class j)
        const int per_arr = p.nbx * p.m;
        const int a = lane / per_arr, rem = lane - a * per_arr;
        const int b = rem / p.m, j = rem - b * p.m;
        const bool issuer = lane < narr * per_arr && j < N;
        int class_base = 0;                                 // staged row index of the class's first row
        for (int q = 0; q < j; ++q) class_base += (N - q + p.m - 1) / p.m;
        const CUtensorMap* my_map = &maps.map[issuer ? a : 0][issuer ? j : 0];
        if (issuer) asm volatile("prefetch.tensormap [%0];" ::"l"(my_map) : "memory");   // a kernel parameter
        // What the first tile needs is worked out, and the launch parameters it reads are
        // brought into the constant cache, before the wait: after it only the copy is left.
        const int l0_first = (int)((p.p_begin + (long long)blockIdx.x * p.T) / p.L);
        const uint32_t my_dst_off = (uint32_t)((a * p.nbx + b) * block_bytes + class_base * p.row_bytes);
        const int tile_cols_per_box = p.T / p.nbx;
        // In a short kernel (fewer than 32 tiles per CTA) three quarters of the tiles are dealt
        // out in fixed rounds (see below); the first ring always is.
        long long static_rounds = stages;
        if (p.n_tiles < 32LL * gridDim.x) static_rounds = (p.n_tiles * 3 / 4) / gridDim.x;
        if (static_rounds < stages) static_rounds = stages;
        const long long n_static = static_rounds * gridDim.x;
        asm volatile("" ::"l"(p.n_tiles), "l"(p.sched), "l"(n_static), "r"(p.stage_bytes), "r"(p.stage_off),
                     "r"(l0_first), "r"(my_dst_off), "r"(tile_cols_per_box));
        // The wait for the preceding kernel comes as late as it can: the first step arms its
        // barrier and writes its metadata (shared memory only) before it, so that after the
        // wait nothing but the copy instruction itself is left to issue.
        bool waited = false;
        // Tiles are handed out dynamically: SMs differ by some 10 % in the HBM bandwidth they
        // get, and with a fixed share of tiles the slowest CTA would set the kernel time.  The
        // first ring of tiles is fixed (tile blockIdx.x + i * gridDim.x fills stage i), so that
        // the pipeline fills without waiting for anything; every further tile comes from the
        // launch's counter.  The round trip of that atomic takes about a microsecond, more than
        // a narrow tile takes to load, so the counter is asked two tiles ahead: the claim made
        // at the top of step n is the tile of step n + 2 and is first read at the end of step
        // n + 1.  Two registers take the claims in turn (a read of one must not have to wait
        // for the atomic just sent into the other), hence the loop is unrolled by two.
        long long n = 0;
        long long tile = blockIdx.x;
        // In a short kernel three quarters of the tiles are dealt out in fixed rounds as well: a
        // claim is one more global operation in the producer's path, which is the critical one
        // there.  (Measured: 1 % faster with 7 tiles per CTA, 1.3 % slower with hundreds, where
        // the claims cost nothing and balance more.)
        bool open = true;                // false once a claim came back beyond the last tile
        // segment of the current tile's first column: a CTA's tiles come in ascending order,
        // so it is stepped forward instead of divided out per tile
        int l0 = l0_first;
        long long l0_end = (long long)(l0_first + 1) * p.L - p.p_begin;   // local column where l0 ends
        // one step; `mine` holds the claim for step n + 1 (made a step ago), `next2` takes
        // the claim for step n + 2.  Returns false when the producer is done.
        auto step = [&](unsigned long long& mine, unsigned long long& next2) -> bool {
            const int s = (int)(n % stages);
            const uint32_t ph = (uint32_t)((n / stages) & 1);
            const bool last = tile >= p.n_tiles;
            const bool claim = n + 2 >= static_rounds && open && !last;
            if (claim && !waited) { wait_for_preceding_kernel(); waited = true; }   // global access ahead
            if (claim && lane == 0) next2 = atomicAdd(&p.sched->next, 1ULL);
            if (!mbar_wait_patient(smem_u32(&hdr->empty[s]), ph ^ 1u)) { staged_fail(1); return false; }
            const long long t0 = tile * (long long)p.T;
            const uint32_t bar = smem_u32(&hdr->full[s]);
            if (lane == 0) {
                if (!last)
                    while (t0 >= l0_end) { ++l0; l0_end += p.L; }
                TileMeta mt;
                mt.bnd = l0_end;
                mt.tile = last ? -1 : (int)tile;                   // -1 tells the consumers to leave
                mt.l0 = l0;
                *reinterpret_cast<int4*>(&hdr->meta[s]) = *reinterpret_cast<const int4*>(&mt);
                if (last) mbar_arrive(bar);
                else mbar_arrive_expect_tx(bar, p.stage_bytes);
            }
            __syncwarp();
            ++n;
            if (last) return false;
            if (!waited) { wait_for_preceding_kernel(); waited = true; }
            if (issuer)
                tma_load_2d(smem_u32(smem + p.stage_off + (size_t)s * p.stage_bytes) + my_dst_off, my_map,
                            (int)(t0 + (long long)b * tile_cols_per_box), 0, bar);
            // tile of the next step
            if (n < static_rounds) {
                tile = (long long)blockIdx.x + n * (long long)gridDim.x;
            } else if (open) {
                tile = n_static + (long long)__shfl_sync(0xffffffffu, mine, 0);
                if (tile >= p.n_tiles) open = false;
            } else {
                tile = p.n_tiles;
            }
            return true;
        };
        {
            unsigned long long claim_a = 0, claim_b = 0;
            // step n reads the claim made at the top of step n - 1, which went into the
            // register that step n - 1 was given as `next2`
            while (step(claim_a, claim_b) && step(claim_b, claim_a)) {}
        }
        if (!waited) wait_for_preceding_kernel();
        // Leave last: every stage this warp armed must have landed before the CTA's
        // shared memory can be released, even if the consumers gave up.
        if (lane == 0) {
            const long long first = n > stages ? n - stages : 0;
            for (long long q = first; q < n; ++q) {
                const int s = (int)(q % stages);
                if (!mbar_wait(smem_u32(&hdr->full[s]), (uint32_t)((q / stages) & 1))) staged_fail(2);
            }
            // the last CTA to get here leaves the dispenser clean for the next launch that uses it
            __threadfence();
            if (atomicAdd(&p.sched->done, 1u) == gridDim.x - 1) {
                p.sched->next = 0;
                p.sched->done = 0;
                __threadfence();
            }
        }
        return;
    }

    // ---------------------------------------------------------------- consumers
    wait_for_preceding_kernel();
    const int cw = warp - 1;
    const int ctid = tid - 32;
    uint32_t csync_phase = 0;
    int cached_l0 = -1;
    const WarpShare<EB, GB> ws(p, cw, kConsumerWarps, lane);
    const uint32_t csync = smem_u32(&hdr->csync);

    // The first tile's table does not depend on the staged data: build it while the
    // first TMA loads are in flight.
    constexpr bool DENSE = (RT == -3 && GB == 16);
    unsigned char* dtab = smem + p.dtab_off;               // dense coefficient blocks, one set per table slot
    if ((long long)blockIdx.x < p.n_tiles) {
        if (whole_table) {
            build_coef_table<EB, RMAX, UNW>(p, tab, R, 0, p.S, ctid, kConsumerThreads);
            if (DENSE) build_dense_table<EB>(p, dtab, R, 0, p.S, ctid, kConsumerThreads);
        } else {
            cached_l0 = (int)((p.p_begin + (long long)blockIdx.x * p.T) / p.L);
            build_coef_table<EB, RMAX, UNW>(p, tab, R, cached_l0, 2, ctid, kConsumerThreads);
            if (DENSE) build_dense_table<EB>(p, dtab, R, cached_l0, 2, ctid, kConsumerThreads);
        }
        if (!consumers_sync(csync, csync_phase, lane)) { staged_fail(7); return; }
    }

    for (long long n = 0;; ++n) {
        const int s = (int)(n % stages);
        const uint32_t ph = (uint32_t)((n / stages) & 1);
        if (!mbar_wait(smem_u32(&hdr->full[s]), ph)) { staged_fail(3); return; }
        const uint4 mt = lds128(smem_u32(&hdr->meta[s]));          // {bnd lo, bnd hi, tile, l0}
        const long long tile = (int)mt.z;
        if (tile < 0) break;
        const long long m_bnd = (long long)(((unsigned long long)mt.y << 32) | mt.x);
        const int m_l0 = (int)mt.w;
        unsigned char* stage = smem + p.stage_off + (size_t)s * p.stage_bytes;
        const uint32_t stage_s = smem_u32(stage);
        // entries of segment l0 (those of l0 + 1 follow them)
        const unsigned char* tab0 = whole_table ? tab + (size_t)m_l0 * N * ENT : tab;

        if (!whole_table && m_l0 != cached_l0) {
            // table for segments l0 and l0+1 (rebuilt at most S times per CTA)
            if (!consumers_sync(csync, csync_phase, lane)) { staged_fail(4); return; }
            build_coef_table<EB, RMAX, UNW>(p, tab, R, m_l0, 2, ctid, kConsumerThreads);
            if (DENSE) build_dense_table<EB>(p, dtab, R, m_l0, 2, ctid, kConsumerThreads);
            if (!consumers_sync(csync, csync_phase, lane)) { staged_fail(5); return; }
            cached_l0 = m_l0;
        }

        if (SGD) {
            // local step on the staged tile, in place: x <- fma(-lr, g, x), every row
            sgd_step_in_place(stage, p.nbx * block_bytes, p.lr, ctid, kConsumerThreads);
            if (!consumers_sync(csync, csync_phase, lane)) { staged_fail(6); return; }
        }

        aggregate_tile<EB, GB, RT, UNW>(p, ws, stage, stage_s, tab0, tile, m_bnd, lane,
                                   DENSE ? dtab + (size_t)(whole_table ? m_l0 : 0) * p.dslot_bytes : nullptr);

        // The fused step rewrote the stage with ordinary stores; the copy that refills it goes
        // through the asynchronous proxy, so the two are ordered by a proxy fence.
        if (SGD) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&hdr->empty[s]));
    }
}

// ---------------------------------------------------------------- one tile per CTA
// Short kernels (a few tiles per SM in all) spend much of their time filling and draining a
// ring; here every tile is a CTA of its own and several CTAs share an SM.  All loads of the
// first wave are in flight at once, a CTA leaves as soon as its tile is written, and the
// hardware's block scheduler does what the tile dispenser does in k_staged.  One TMA load
// (issued by warp 0), the coefficient table of the tile's two possible segments built
// meanwhile, then the same per-warp aggregation as above.
constexpr int kTileWarps = 4;
constexpr int kTileThreads = 32 * kTileWarps;

template <int EB, int GB, bool SGD, int RT>
__global__ void __launch_bounds__(kTileThreads)
k_tile(const AggParams p, const __grid_constant__ TileMaps maps) {
    constexpr int RMAX = rmax_of(RT);
    extern __shared__ __align__(128) unsigned char smem[];
    StagedHeader* hdr = reinterpret_cast<StagedHeader*>(smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int N = p.N, R = (RT >= 0) ? RT : p.R;
    const int narr = SGD ? 2 : 1;
    unsigned char* tab = smem + p.tab_off;                 // two slots: segments l0 and l0 + 1
    unsigned char* stage = smem + p.stage_off;
    const int block_bytes = N * p.row_bytes;
    const uint32_t bar = smem_u32(&hdr->full[0]);
    const long long tile = blockIdx.x;
    const long long t0 = tile * (long long)p.T;
    const int l0 = (int)((p.p_begin + t0) / p.L);
    const long long bnd = (long long)(l0 + 1) * p.L - p.p_begin;   // local column where l0 + 1 starts

    // lane of warp 0 -> one TMA box: (array a, x-box b, class j), as in k_staged
    const int per_arr = p.nbx * p.m;
    const int a = lane / per_arr, rem = lane - a * per_arr;
    const int b = rem / p.m, j = rem - b * p.m;
    const bool issuer = warp == 0 && lane < narr * per_arr && j < N;
    int class_base = 0;
    for (int q = 0; q < j; ++q) class_base += (N - q + p.m - 1) / p.m;
    const CUtensorMap* my_map = &maps.map[issuer ? a : 0][issuer ? j : 0];
    if (issuer) asm volatile("prefetch.tensormap [%0];" ::"l"(my_map) : "memory");
    if (tid == 0) {
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_arrive_expect_tx(bar, p.stage_bytes);
    }
    // A CTA of this kernel is small, so under programmatic stream serialization it becomes
    // resident while the preceding kernel still runs.  Its tile is asked into L2 right away:
    // a prefetch has no architectural effect (if the preceding kernel is still writing these
    // lines, L2 keeps them coherent and the load below sees the final values), but the read
    // from HBM then overlaps the preceding kernel's tail instead of following it.
    const int box_x = (int)(t0 + (long long)b * (p.T / p.nbx));
    if (issuer) tma_prefetch_2d(my_map, box_x, 0);
    __syncthreads();
    // everything above touched only this CTA's shared memory and the launch parameters (see
    // k_staged on programmatic stream serialization)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (issuer)
        tma_load_2d(smem_u32(stage) + (uint32_t)((a * p.nbx + b) * block_bytes + class_base * p.row_bytes), my_map,
                    box_x, 0, bar);
    // the second slot only where the tile reaches into segment l0 + 1
    build_coef_table<EB, RMAX>(p, tab, R, l0, bnd < t0 + p.T ? 2 : 1, tid, kTileThreads);
    __syncthreads();
    if (!mbar_wait(bar, 0)) {
        // give the copy one more bounded chance to land before the shared memory is released
        staged_fail(8);
        mbar_wait(bar, 0);
        return;
    }
    if (SGD) {
        sgd_step_in_place(stage, p.nbx * block_bytes, p.lr, tid, kTileThreads);
        __syncthreads();
    }
    const WarpShare<EB, GB> ws(p, warp, kTileWarps, lane);
    aggregate_tile<EB, GB, RT>(p, ws, stage, smem_u32(stage), tab, tile, bnd, lane);
}

}  // namespace combo
