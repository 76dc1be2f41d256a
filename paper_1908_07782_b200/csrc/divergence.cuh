// Aggregation divergence (Section 4.3, Definition 2, Eq. 7):
//   rho_i = || W_{t,i} - W_t ||_2,   W_t = sum_j |D_j| W_j / sum_j |D_j|  (the FedAvg result)
// for all N workers in one pass over HBM.
//
//   k_divergence_staged  column tiles through all rows, staged by tiled TMA like the
//                        aggregation kernel; per tile: (A) column means from the staged
//                        block, (B) warp-per-row sums of squared deviations, carried in
//                        binary64 registers across the CTA's tiles
//   k_divergence_direct  fallback for rows that are not even 4-byte aligned or N > 256:
//                        thread per column, two passes through L1/L2
//   k_divergence_finish  sums the per-CTA partial sums in block order and takes the root
//
// The per-CTA partial sums [grid][N] (binary64) live in scratch memory supplied by the
// caller; every entry is written before it is read, so the scratch needs no clearing.
#pragma once
#include "segment_aggregate.cuh"

namespace combo {

constexpr int kDivSlots = 16;                          // rows a consumer warp can own
constexpr int kDivMaxStagedN = kDivSlots * kConsumerWarps;
constexpr int kDivBox = 256;                           // widest TMA box in columns
constexpr int kDivTile = 1024;                         // widest tile in columns (four boxes)
constexpr int kDivWordMeans = 256;                     // floats per copy of the column means in word mode

struct DivParams {
    const unsigned char* models;
    const unsigned char* src;      // rows the mean is taken over (== models when narr == 1)
    const float* weights;
    double* partial;               // scratch [grid][N]
    long long pitch, width, n_tiles;
    int N, narr, m, stages, row_bytes;
    unsigned coef_off, rowoff_off, part_off, mean_off, stage_off, stage_bytes;
};

// N consecutive floats of shared memory as one access (N = 1 or 2)
template <int N_> __device__ __forceinline__ void store_floats_w(float* q, const float (&v)[N_]) {
    if constexpr (N_ == 2) *reinterpret_cast<float2*>(q) = make_float2(v[0], v[1]);
    else q[0] = v[0];
}
template <int N_> __device__ __forceinline__ void load_floats_w(const float* q, float (&v)[N_]) {
    if constexpr (N_ == 2) { const float2 t = *reinterpret_cast<const float2*>(q); v[0] = t.x; v[1] = t.y; }
    else v[0] = q[0];
}

// TC = columns per tile.  Rows that are 16-byte aligned: 64 to 1024 (the widest whose stage
// stays within 64 KB; tiles wider than 256 columns are staged as several boxes, which keeps
// the per-tile costs -- a consumer-wide barrier, the producer's bookkeeping -- small against
// the data when there are few rows), threads work on 128-bit vectors.  WORD: rows whose pitch is only a
// multiple of 4 bytes are staged per row class with their phase (see the aggregation
// kernel), TC = 256 - 16/e, and threads work on 4-byte words at the row's phase.
template <int EB, int TC, bool WORD, bool PIPE = !WORD>
__global__ void __launch_bounds__(kStagedThreads, 1)
k_divergence_staged(const DivParams p, const __grid_constant__ TileMaps maps) {
    constexpr int UB = WORD ? 4 : 16;                  // bytes a thread takes at a time
    constexpr int EPU = UB / EB;                       // elements in them
    constexpr int NU = TC * EB / UB;                   // such units per row per tile
    constexpr int NBX = TC > kDivBox ? TC / kDivBox : 1;  // boxes per tile
    constexpr int UPB = NU / NBX;                      // units per row held by one box
    constexpr int NUP = NU <= 16 ? 16 : NU <= 32 ? 32 : NU <= 64 ? 64 : NU <= 128 ? 128 : NU <= 256 ? 256 : 512;
    static_assert(NU <= kConsumerThreads, "a tile has more units than there are consumer threads");
    constexpr int G = kConsumerThreads / NUP;          // row groups of phase A
    constexpr int PSTR = NUP * EPU;                    // floats per row group in `part`
    extern __shared__ __align__(128) unsigned char smem[];
    StagedHeader* hdr = reinterpret_cast<StagedHeader*>(smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int N = p.N, stages = p.stages;
    float* coef = reinterpret_cast<float*>(smem + p.coef_off);     // c_j = |D_j| / sum |D|
    int* rowoff = reinterpret_cast<int*>(smem + p.rowoff_off);     // staged byte offset of worker j's tile part
    float* part = reinterpret_cast<float*>(smem + p.part_off);     // [2][G][PSTR]
    float* mean = reinterpret_cast<float*>(smem + p.mean_off);     // [2][kDivTile]
    const int block_bytes = N * p.row_bytes;

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(&hdr->full[s]), 1);
            mbar_init(smem_u32(&hdr->empty[s]), kConsumerWarps);
        }
        mbar_init(smem_u32(&hdr->csync), kConsumerWarps);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // coefficients (the denominator is summed in worker order by every thread alike) and
    // where each worker's row sits in a stage: classes one after another, phase included
    {
        float den = 0.0f;
        for (int j = 0; j < N; ++j) den = __fadd_rn(den, p.weights ? p.weights[j] : 1.0f);
        for (int j = tid; j < N; j += kStagedThreads) {
            coef[j] = __fdiv_rn(p.weights ? p.weights[j] : 1.0f, den);
            const int jc = j % p.m;
            int base = 0;
            for (int q = 0; q < jc; ++q) base += (N - q + p.m - 1) / p.m;
            rowoff[j] = (base + j / p.m) * p.row_bytes + (int)(((long long)j * p.pitch * EB) & 15);
        }
    }
    __syncthreads();

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        // lane -> one TMA box per tile: (array a, x-box b, class j)
        const int per_arr = NBX * p.m;
        const int a = lane / per_arr, rem = lane - a * per_arr;
        const int b = rem / p.m, j = rem - b * p.m;
        const bool issuer = lane < p.narr * per_arr && j < N;
        int class_base = 0;
        for (int q = 0; q < j; ++q) class_base += (N - q + p.m - 1) / p.m;
        const CUtensorMap* my_map = &maps.map[issuer ? a : 0][issuer ? j : 0];
        if (issuer) asm volatile("prefetch.tensormap [%0];" ::"l"(my_map) : "memory");
        const uint32_t my_dst_off = (uint32_t)((a * NBX + b) * block_bytes + class_base * p.row_bytes);
        long long n = 0;
        for (long long tile = blockIdx.x; tile < p.n_tiles; tile += gridDim.x, ++n) {
            const int s = (int)(n % stages);
            const uint32_t ph = (uint32_t)((n / stages) & 1);
            if (!mbar_wait_patient(smem_u32(&hdr->empty[s]), ph ^ 1u)) { staged_fail(11); break; }
            const uint32_t bar = smem_u32(&hdr->full[s]);
            if (lane == 0) mbar_arrive_expect_tx(bar, p.stage_bytes);
            __syncwarp();
            if (issuer)
                tma_load_2d(smem_u32(smem + p.stage_off + (size_t)s * p.stage_bytes) + my_dst_off, my_map,
                            (int)(tile * TC) + b * (TC / NBX), 0, bar);
        }
        if (lane == 0) {
            const long long first = n > stages ? n - stages : 0;
            for (long long q = first; q < n; ++q) {
                const int s = (int)(q % stages);
                if (!mbar_wait(smem_u32(&hdr->full[s]), (uint32_t)((q / stages) & 1))) staged_fail(12);
            }
        }
        return;
    }

    // ---------------------------------------------------------------- consumers
    const int cw = warp - 1;
    const int ctid = tid - 32;
    uint32_t csync_phase = 0;
    const uint32_t csync = smem_u32(&hdr->csync);
    const int au = ctid % NUP, ag = ctid / NUP;         // phase A: unit and row group
    double acc[kDivSlots];
#pragma unroll
    for (int s = 0; s < kDivSlots; ++s) acc[s] = 0.0;

    if constexpr (WORD) {
        // Rows with differing 16-byte phases: warp per row in both phases.  Warp cw owns rows
        // cw, cw + 16, ...; lane l takes the 4-byte words l, l + 32, ... of a row (conflict-free
        // whatever the row's phase), i.e. the same columns in every row, so that its column
        // sums and, later, its column means stay in registers while it walks over its rows.
        // Where a row lies in a stage does not depend on the tile: those offsets are registers
        // too.  What goes through shared memory per row and phase is the row itself.
        // bfloat16 operands enter binary32 adds directly (add.rn.f32.bf16: exact widening, one
        // rounding); with unit weights the column sum needs no multiplication at all.
        // The warp's rows are walked from the last to the first by a switch that falls through
        // (straight-line code with fixed registers and no test per row).  A lane's last word
        // may lie beyond the row's payload: it is read all the same (the bytes are inside the
        // stage or its 16 bytes of slack); its column sums land in entries nobody reads, and
        // for the deviations the word and its means are replaced by zero.
        constexpr int WPL = (NU + 31) / 32;             // words per lane per row
        constexpr int FPL = WPL * EPU;                  // binary32 values per lane per row
        static_assert(NBX == 1, "word mode uses one box per tile");
        int ro[kDivSlots];
#pragma unroll
        for (int sl = 0; sl < kDivSlots; ++sl) {
            const int r = cw + sl * kConsumerWarps;
            ro[sl] = r < N ? rowoff[r] : 0;
        }
        const int nrows = cw < N ? (N - cw + kConsumerWarps - 1) / kConsumerWarps : 0;
        const bool weighted = p.weights != nullptr;
        const float mscale = weighted ? 1.0f : coef[0];                 // unit weights: 1 / N
        const bool tail_on = lane + 32 * (WPL - 1) < NU;               // the lane's last word exists
        float* part_w = part + cw * (NUP * EPU);                       // this warp's column sums
        const uint32_t lane_off = (uint32_t)lane * 4u;
        const long long n_mine = (p.n_tiles > (long long)blockIdx.x)
                                     ? (p.n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
#define COMBO_DIV_CASES(ROW)                                                                             \
    case 16: ROW(15) case 15: ROW(14) case 14: ROW(13) case 13: ROW(12) case 12: ROW(11) case 11: ROW(10) \
    case 10: ROW(9) case 9: ROW(8) case 8: ROW(7) case 7: ROW(6) case 6: ROW(5) case 5: ROW(4)           \
    case 4: ROW(3) case 3: ROW(2) case 2: ROW(1) case 1: ROW(0) default: break;
        // One consumer-wide barrier per tile, as in vector mode (PIPE; needs three stages):
        // step i sums tile i, and after the barrier forms its means and takes the deviations
        // of tile i - 1 (two copies of the sums and of the means keep neighbouring steps apart).
        for (long long i = 0; i <= n_mine; ++i) {
            if (i < n_mine) {
                const int s = (int)(i % stages);
                if (!mbar_wait(smem_u32(&hdr->full[s]), (uint32_t)((i / stages) & 1))) { staged_fail(13); return; }
                const uint32_t src_s = smem_u32(smem + p.stage_off + (size_t)s * p.stage_bytes) +
                                       (uint32_t)((p.narr - 1) * block_bytes) + lane_off;
                // (A) column sums over this warp's rows
                float a[FPL];
#pragma unroll
                for (int e = 0; e < FPL; ++e) a[e] = 0.0f;
#define COMBO_DIV_ROW_A(SL)                                                                              \
    {                                                                                                    \
        const uint32_t row = src_s + (uint32_t)ro[SL];                                                   \
        const float c = weighted ? coef[cw + SL * kConsumerWarps] : 1.0f;                                \
        _Pragma("unroll") for (int q = 0; q < WPL; ++q) {                                                \
            const uint32_t w = lds32<0>(row + 128u * q);                                                 \
            if constexpr (EB == 4) {                                                                     \
                a[q] = weighted ? fmaf(c, __uint_as_float(w), a[q]) : __fadd_rn(__uint_as_float(w), a[q]); \
            } else if (weighted) {                                                                       \
                a[2 * q] = fmaf(c, __uint_as_float(w << 16), a[2 * q]);                                  \
                a[2 * q + 1] = fmaf(c, __uint_as_float(w & 0xffff0000u), a[2 * q + 1]);                  \
            } else {                                                                                     \
                a[2 * q] = add_bf16_lo(w, a[2 * q]);                                                     \
                a[2 * q + 1] = add_bf16_hi(w, a[2 * q + 1]);                                             \
            }                                                                                            \
        }                                                                                                \
    }
                switch (nrows) { COMBO_DIV_CASES(COMBO_DIV_ROW_A) }
#undef COMBO_DIV_ROW_A
                float* pw = part_w + (i & 1) * (kConsumerWarps * NUP * EPU);
#pragma unroll
                for (int q = 0; q < WPL; ++q) {
                    float v[EPU];
#pragma unroll
                    for (int e = 0; e < EPU; ++e) v[e] = a[q * EPU + e];
                    store_floats_w<EPU>(pw + (lane + 32 * q) * EPU, v);
                }
            }
            if (!consumers_sync(csync, csync_phase, lane)) { staged_fail(14); return; }
            if (i < n_mine) {
                // (A2) column means: the warps' sums added in warp order
                const float* pt = part + (i & 1) * (kConsumerWarps * NUP * EPU);
                for (int c = ctid; c < TC; c += kConsumerThreads) {
                    float m = 0.0f;
#pragma unroll
                    for (int g = 0; g < kConsumerWarps; ++g) m = __fadd_rn(m, pt[g * (NUP * EPU) + c]);
                    mean[(i & 1) * kDivWordMeans + c] = __fmul_rn(m, mscale);
                }
            }
            if (!PIPE) {
                // too few stages to hold two tiles at a time: the deviations of tile i follow
                // its means in the same step, behind a second barrier
                if (!consumers_sync(csync, csync_phase, lane)) { staged_fail(15); return; }
            }
            if (PIPE ? (i >= 1) : (i < n_mine)) {
                // (B) squared deviations of this warp's rows of tile t from the means of the
                // lane's columns (pipelined: written in step i - 1, before this step's barrier)
                const long long t = PIPE ? i - 1 : i;
                const int s = (int)(t % stages);
                const float* mn = mean + (t & 1) * kDivWordMeans;
                float nmu[FPL];
#pragma unroll
                for (int q = 0; q < WPL; ++q) {
                    float v[EPU];
                    load_floats_w<EPU>(mn + (lane + 32 * q) * EPU, v);
#pragma unroll
                    for (int e = 0; e < EPU; ++e) nmu[q * EPU + e] = (q < WPL - 1 || tail_on) ? -v[e] : 0.0f;
                }
                const uint32_t own_s = smem_u32(smem + p.stage_off + (size_t)s * p.stage_bytes) + lane_off;
#define COMBO_DIV_ROW_B(SL)                                                                              \
    {                                                                                                    \
        const uint32_t row = own_s + (uint32_t)ro[SL];                                                   \
        float ssum = 0.0f;                                                                               \
        _Pragma("unroll") for (int q = 0; q < WPL; ++q) {                                                \
            uint32_t w = lds32<0>(row + 128u * q);                                                       \
            if (q == WPL - 1) w = tail_on ? w : 0u;                                                      \
            if constexpr (EB == 4) {                                                                     \
                const float d = __fadd_rn(__uint_as_float(w), nmu[q]);                                   \
                ssum = fmaf(d, d, ssum);                                                                 \
            } else {                                                                                     \
                const float d0 = add_bf16_lo(w, nmu[2 * q]), d1 = add_bf16_hi(w, nmu[2 * q + 1]);        \
                ssum = fmaf(d0, d0, ssum);                                                               \
                ssum = fmaf(d1, d1, ssum);                                                               \
            }                                                                                            \
        }                                                                                                \
        acc[SL] += (double)ssum;                                                                         \
    }
                switch (nrows) { COMBO_DIV_CASES(COMBO_DIV_ROW_B) }
#undef COMBO_DIV_ROW_B
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&hdr->empty[s]));
            }
        }
#undef COMBO_DIV_CASES
    } else {
    // byte offset of unit u of a row inside an array's part of a stage (its box, then its place)
    auto unit_off = [&](int u) { return NBX == 1 ? u * UB : (u / UPB) * block_bytes + (u % UPB) * UB; };
    // one unit of a staged row as EPU binary32 values
    auto load_unit = [](const unsigned char* q, float (&x)[EPU]) {
        if constexpr (!WORD) {
            GroupLoad<EB, 16>::run(q, x);
        } else if constexpr (EB == 4) {
            x[0] = *reinterpret_cast<const float*>(q);
        } else {
            const uint32_t w = *reinterpret_cast<const uint32_t*>(q);
            x[0] = bf16_widen(w & 0xffffu);
            x[1] = __uint_as_float(w & 0xffff0000u);
        }
    };

    // EPU consecutive floats of shared memory as one vector access (16-byte aligned groups)
    auto store_floats = [](float* q, const float (&v)[EPU]) {
        if constexpr (EPU % 4 == 0) {
#pragma unroll
            for (int e = 0; e < EPU; e += 4) *reinterpret_cast<float4*>(q + e) = make_float4(v[e], v[e + 1], v[e + 2], v[e + 3]);
        } else if constexpr (EPU == 2) {
            *reinterpret_cast<float2*>(q) = make_float2(v[0], v[1]);
        } else {
            q[0] = v[0];
        }
    };
    auto load_floats = [](const float* q, float (&v)[EPU]) {
        if constexpr (EPU % 4 == 0) {
#pragma unroll
            for (int e = 0; e < EPU; e += 4) {
                const float4 t = *reinterpret_cast<const float4*>(q + e);
                v[e] = t.x; v[e + 1] = t.y; v[e + 2] = t.z; v[e + 3] = t.w;
            }
        } else if constexpr (EPU == 2) {
            const float2 t = *reinterpret_cast<const float2*>(q);
            v[0] = t.x; v[1] = t.y;
        } else {
            v[0] = q[0];
        }
    };

    // Software pipeline over this CTA's tiles, one consumer-wide barrier per tile:
    //   step i:  (A) partial column sums of tile i      -> part[i & 1]
    //            barrier
    //            (A2) column means of tile i            -> mean[i & 1]
    //            (B) squared deviations of tile i-1 against mean[(i-1) & 1], stage released
    // The barrier of step i orders A2(i-1) before B(i-1) and B(i-2) before A2(i); the two
    // copies of `part` and `mean` keep neighbouring steps off each other's data.
    const long long n_my = (p.n_tiles > (long long)blockIdx.x)
                               ? (p.n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    for (long long i = 0; i <= n_my; ++i) {
        if (i < n_my) {
            const int s = (int)(i % stages);
            if (!mbar_wait(smem_u32(&hdr->full[s]), (uint32_t)((i / stages) & 1))) { staged_fail(13); return; }
            const unsigned char* xsrc = smem + p.stage_off + (size_t)s * p.stage_bytes + (p.narr - 1) * NBX * block_bytes;
            float* pt = part + (i & 1) * (G * PSTR);
            // (A) weighted column sums of this thread's row group; columns past the end of the
            // rows were zero-filled by the TMA unit and contribute nothing anywhere below
            if (au < NU) {
                float a[EPU];
#pragma unroll
                for (int e = 0; e < EPU; ++e) a[e] = 0.0f;
                for (int j = ag; j < N; j += G) {
                    float x[EPU];
                    load_unit(xsrc + rowoff[j] + unit_off(au), x);
                    const float c = coef[j];
#pragma unroll
                    for (int e = 0; e < EPU; ++e) a[e] = fmaf(c, x[e], a[e]);
                }
                store_floats(pt + ag * PSTR + au * EPU, a);
            }
        }
        if (!consumers_sync(csync, csync_phase, lane)) { staged_fail(14); return; }
        if (i < n_my) {
            const float* pt = part + (i & 1) * (G * PSTR);
            for (int c = ctid; c < TC; c += kConsumerThreads) {
                float m = 0.0f;
#pragma unroll
                for (int g = 0; g < G; ++g) m = __fadd_rn(m, pt[g * PSTR + c]);
                mean[(i & 1) * kDivTile + c] = m;
            }
        }
        if (!PIPE) {
            // unpipelined form: the means of tile i must be complete before its deviations
            if (!consumers_sync(csync, csync_phase, lane)) { staged_fail(15); return; }
        }
        if (PIPE ? (i >= 1) : (i < n_my)) {
            // (B) warp per row: squared deviations of the workers' own models, tile i-1 (i when unpipelined)
            const long long t = PIPE ? i - 1 : i;
            const int s = (int)(t % stages);
            const unsigned char* stage = smem + p.stage_off + (size_t)s * p.stage_bytes;
            const float* mn = mean + (t & 1) * kDivTile;
#pragma unroll
            for (int sl = 0; sl < kDivSlots; ++sl) {
                const int r = cw + sl * kConsumerWarps;
                if (r < N) {
                    float ssum = 0.0f;
                    const unsigned char* row = stage + rowoff[r];
#pragma unroll
                    for (int u = lane; u < NU; u += 32) {
                        float x[EPU], mu[EPU];
                        load_unit(row + unit_off(u), x);
                        load_floats(mn + u * EPU, mu);
#pragma unroll
                        for (int e = 0; e < EPU; ++e) {
                            const float d = __fsub_rn(x[e], mu[e]);
                            ssum = fmaf(d, d, ssum);
                        }
                    }
                    acc[sl] += (double)ssum;
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&hdr->empty[s]));
        }
    }
    }   // vector mode
    // per-CTA partial sums: one entry per row, written by the warp that owns the row
#pragma unroll
    for (int sl = 0; sl < kDivSlots; ++sl) {
        const int i = cw + sl * kConsumerWarps;
        if (i < N) {
            double v = acc[sl];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (lane == 0) p.partial[(size_t)blockIdx.x * N + i] = v;
        }
    }
}

// Fallback: any alignment, any N.  256 columns per step, thread per column.
template <int EB>
__global__ void __launch_bounds__(256)
k_divergence_direct(const DivParams p) {
    extern __shared__ __align__(16) unsigned char dsm[];
    double* acc = reinterpret_cast<double*>(dsm);                       // [N]
    float* coef = reinterpret_cast<float*>(acc + p.N);                  // [N]
    const int tid = threadIdx.x, lane = tid & 31;
    const int N = p.N;
    {
        float den = 0.0f;
        for (int j = 0; j < N; ++j) den = __fadd_rn(den, p.weights ? p.weights[j] : 1.0f);
        for (int j = tid; j < N; j += 256) {
            coef[j] = __fdiv_rn(p.weights ? p.weights[j] : 1.0f, den);
            acc[j] = 0.0;
        }
    }
    __syncthreads();
    const long long n_blk = (p.width + 255) / 256;
    for (long long blk = blockIdx.x; blk < n_blk; blk += gridDim.x) {
        const long long col = blk * 256 + tid;
        const bool valid = col < p.width;
        float mean = 0.0f;
        if (valid)
            for (int j = 0; j < N; ++j)
                mean = fmaf(coef[j], ElemOps<EB>::load(p.src + ((size_t)j * p.pitch + (size_t)col) * EB), mean);
        for (int i = 0; i < N; ++i) {
            float d = 0.0f;
            if (valid) d = __fsub_rn(ElemOps<EB>::load(p.models + ((size_t)i * p.pitch + (size_t)col) * EB), mean);
            float sq = d * d;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
            if (lane == 0) atomicAdd(&acc[i], (double)sq);
        }
    }
    __syncthreads();
    for (int i = tid; i < N; i += 256) p.partial[(size_t)blockIdx.x * N + i] = acc[i];
}

__global__ void k_divergence_finish(const double* __restrict__ partial, int nblocks, int N,
                                    double* __restrict__ rho) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    double s = 0.0;
    for (int b = 0; b < nblocks; ++b) s += partial[(size_t)b * N + i];
    rho[i] = sqrt(s);
}

}  // namespace combo
