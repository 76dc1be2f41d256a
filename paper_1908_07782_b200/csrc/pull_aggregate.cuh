// Worker-sharded aggregation (Section 3 "Segmented Pulling", Eq. 2 and Eq. 3): the workers'
// rows live in separate allocations -- on this GPU or, through peer mappings, on other GPUs
// of the node -- and this GPU forms the new models of the workers it hosts.
//
// A pull is a load: for worker w and segment l the kernel reads W_w[l] and the R segments
// W_k[l] of its peers straight from where they live (plain 128-bit global loads, which work
// on peer memory over NVLink; no bulk-tensor copy, no multicast), combines them in the fixed
// order of Eq. 3 (self, then peers ascending) and writes the result to local memory.  What
// crosses NVLink is what the paper's workers send each other: R segments per (hosted worker,
// segment).
//
//   k_pull_staged     the rows a column tile needs -- the hosted workers' own rows and every
//                     DISTINCT row some hosted worker pulls for the tile's segment -- are
//                     brought into shared memory once (per-thread 16-byte asynchronous loads,
//                     which are ordinary global loads and work on peer mappings), and all
//                     hosted workers' outputs for the tile are formed from there.  Two hosted
//                     workers that pull the same (peer, segment) share the copy, so such a
//                     segment crosses NVLink once per GPU, and the hosted rows are read from
//                     HBM once instead of R+1 times.
//   k_pull_aggregate  nothing staged (every provider element loaded where it is used); the
//                     fallback when the needed rows of a tile do not fit in shared memory.
#pragma once
#include "segment_aggregate.cuh"

namespace combo {

struct PullParams {
    const void* const* rows;   // device array of N row pointers (row j = model of worker j)
    unsigned char* out;        // [n_local][out_pitch] rows of workers w_begin .. w_begin+n_local-1
    const float* weights;
    const int32_t* idx;
    long long P, L, out_pitch;
    int N, S, R, w_begin, n_local;
};

// grid: x over 16-byte column groups (grid stride), y = hosted worker.  Shared memory:
// the N row pointers.
template <int EB>
__global__ void __launch_bounds__(256) k_pull_aggregate(const PullParams p) {
    constexpr int V = ElemOps<EB>::V;
    extern __shared__ __align__(16) unsigned char pull_smem[];
    const unsigned char** rows = reinterpret_cast<const unsigned char**>(pull_smem);
    for (int j = threadIdx.x; j < p.N; j += 256) rows[j] = static_cast<const unsigned char*>(p.rows[j]);
    __syncthreads();
    const int w = p.w_begin + blockIdx.y;
    const int R = p.R;
    const int32_t* my_idx = R > 0 ? p.idx + (size_t)w * p.S * (size_t)R : nullptr;
    unsigned char* orow = p.out + (size_t)blockIdx.y * (size_t)p.out_pitch * EB;
    const long long groups = (p.P + V - 1) / V;
    for (long long g = blockIdx.x * 256LL + threadIdx.x; g < groups; g += (long long)gridDim.x * 256LL) {
        const long long c0 = g * V;
        const long long hi = (c0 + V > p.P) ? p.P : c0 + V;
        const long long l_lo = c0 / p.L, l_hi = (hi - 1) / p.L;
        if (hi - c0 == V && l_lo == l_hi) {
            // providers: the worker itself, then its peers ascending; a negative entry is a pull
            // that found no online peer (Section 4.2) and is skipped
            const int32_t* peers = my_idx + (size_t)l_lo * R;
            // Eq. 3 as written: numerator in the fixed order, times the reciprocal of the
            // denominator; a single provider is taken as it is
            float den = p.weights ? p.weights[w] : 1.0f;
            int np = 1;
            for (int r = 0; r < R; ++r)
                if (peers[r] >= 0) { den = __fadd_rn(den, p.weights ? p.weights[peers[r]] : 1.0f); ++np; }
            float acc[V], x[V];
            GroupLoad<EB, 16>::run(rows[w] + (size_t)c0 * EB, x);
            float c = (np == 1 || !p.weights) ? 1.0f : p.weights[w];
#pragma unroll
            for (int i = 0; i < V; ++i) acc[i] = __fmul_rn(c, x[i]);
            for (int r = 0; r < R; ++r) {
                const int k = peers[r];
                if (k < 0) continue;
                GroupLoad<EB, 16>::run(rows[k] + (size_t)c0 * EB, x);
                c = p.weights ? p.weights[k] : 1.0f;
#pragma unroll
                for (int i = 0; i < V; ++i) acc[i] = fmaf(c, x[i], acc[i]);
            }
            if (np > 1) {
                const float scale = __fdiv_rn(1.0f, den);
#pragma unroll
                for (int i = 0; i < V; ++i) acc[i] = __fmul_rn(scale, acc[i]);
            }
            ElemOps<EB>::store_vec(orow + (size_t)c0 * EB, acc);
        } else {
            // a group that holds a segment boundary or the end of the row: element by element
            for (long long col = c0; col < hi; ++col) {
                const int32_t* peers = my_idx + (size_t)(col / p.L) * R;
                float den = p.weights ? p.weights[w] : 1.0f;
                int np = 1;
                for (int r = 0; r < R; ++r)
                    if (peers[r] >= 0) { den = __fadd_rn(den, p.weights ? p.weights[peers[r]] : 1.0f); ++np; }
                float acc = __fmul_rn((np == 1 || !p.weights) ? 1.0f : p.weights[w],
                                      ElemOps<EB>::load(rows[w] + (size_t)col * EB));
                for (int r = 0; r < R; ++r) {
                    const int k = peers[r];
                    if (k < 0) continue;
                    acc = fmaf(p.weights ? p.weights[k] : 1.0f, ElemOps<EB>::load(rows[k] + (size_t)col * EB), acc);
                }
                if (np > 1) acc = __fmul_rn(__fdiv_rn(1.0f, den), acc);
                ElemOps<EB>::store(orow + (size_t)col * EB, acc);
            }
        }
    }
}

// ---------------------------------------------------------------- staged form
constexpr int kPullThreads = 512;
constexpr int kPullWarps = kPullThreads / 32;
constexpr int kPullMaxN = 2048;          // workers whose row pointers and slots fit the header

struct PullStagedParams {
    const void* const* rows;
    unsigned char* out;
    const float* weights;
    const int32_t* idx;
    long long P, L, out_pitch, n_tiles;
    int N, S, R, w_begin, n_local;
    int T;                 // tile width in elements: nbx boxes of row_bytes / elem_bytes columns
    int nbx;               // x-boxes per tile, a power of two; a stage is [nbx][d_max][row_bytes]
    int row_bytes;         // bytes of a staged row of one box, a power of two
    int gpr_log2;          // log2 of the 16-byte groups of a row's tile piece (nbx * row_bytes / 16 <= kPullThreads)
    int gpb_log2;          // log2 of the 16-byte groups per box row (row_bytes / 16)
    int d_max;             // rows a stage has room for
    int stages;            // 3..8 stages of stage_bytes each
    unsigned ptr_off, slot_off, list_off, tab_off, stage_off, stage_bytes;
};

// 16-byte asynchronous copy global -> shared by the calling thread; only the first
// src_bytes (0..16) are read, the rest of the 16 bytes is filled with zeros.
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N_> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N_) : "memory");
}
// waits until at most n (0..7) of the calling thread's copy groups are still in flight
__device__ __forceinline__ void cp_async_wait_n(int n) {
    switch (n) {
        case 0: cp_async_wait<0>(); break;
        case 1: cp_async_wait<1>(); break;
        case 2: cp_async_wait<2>(); break;
        case 3: cp_async_wait<3>(); break;
        case 4: cp_async_wait<4>(); break;
        case 5: cp_async_wait<5>(); break;
        case 6: cp_async_wait<6>(); break;
        default: cp_async_wait<7>(); break;
    }
}

// One CTA works through a contiguous range of column tiles.  A "context" is what a run of
// tiles shares: the segment l0 of their first column and whether the tile reaches into
// l0 + 1 (then it is a run of one tile and needs the rows of both segments).  Per context
// the CTA marks the rows it needs, numbers them (hosted workers first, then the pulled rows
// in ascending worker order) and builds the coefficient table, whose provider offsets point
// at those numbered slots of a stage.  Inside a run the tiles go through a ring of stages: the
// loads of tile j + stages - 1 are issued before tile j is consumed, one copy group per tile.
// UNW: bfloat16 rows with unit weights, summed by the mixed-precision add (see RowCtxU).
template <int EB, int RT, bool UNW = false>
__global__ void __launch_bounds__(kPullThreads, 1) k_pull_staged(const PullStagedParams p) {
    constexpr int RMAX = (RT >= 0) ? RT : (RT == -2 ? kStagedMaxR : kGenericR);
    constexpr int ENT = entry_bytes_of<RMAX, UNW>();
    extern __shared__ __align__(128) unsigned char smem[];
    const unsigned char** rowp = reinterpret_cast<const unsigned char**>(smem + p.ptr_off);
    short* slot_of = reinterpret_cast<short*>(smem + p.slot_off);     // [N]: stage slot of a worker's row or -1
    const unsigned char** srcp = reinterpret_cast<const unsigned char**>(smem + p.list_off);   // [d_max]: row held by each slot
    unsigned char* tab = smem + p.tab_off;                            // [2][n_local] entries
    __shared__ int s_nd;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int N = p.N, R = (RT >= 0) ? RT : p.R, nl = p.n_local;

    for (int j = tid; j < N; j += kPullThreads) rowp[j] = static_cast<const unsigned char*>(p.rows[j]);

    // the aggregation below sees the stage as an [nl + pulled][T] block and the output as
    // [nl][out_pitch]
    AggParams ap;
    ap.out = p.out;
    ap.pitch = p.out_pitch;
    ap.p_begin = 0;
    ap.width = p.P;
    ap.L = p.L;
    ap.N = nl;
    ap.S = p.S;
    ap.R = p.R;
    ap.T = p.T;
    ap.m = 1;
    ap.nbx = p.nbx;
    ap.box_w = p.T / p.nbx;
    ap.row_bytes = p.row_bytes;
    ap.stage_rows = p.d_max;
    ap.dslot_bytes = 0;
    const WarpShare<EB, 16> ws(ap, warp, kPullWarps, lane);

    // contiguous share of the tiles
    const long long per = (p.n_tiles + gridDim.x - 1) / gridDim.x;
    long long i = (long long)blockIdx.x * per;
    const long long i_end = i + per < p.n_tiles ? i + per : p.n_tiles;

    // A thread copies the same 16-byte group of every sstep-th staged row (the groups per row
    // are a power of two that divides the block size), so nothing is divided per copy.
    const int my_g = tid & ((1 << p.gpr_log2) - 1), my_s0 = tid >> p.gpr_log2;
    const int sstep = kPullThreads >> p.gpr_log2;
    auto issue = [&](long long tile, int st, int nd) {
        const long long t0 = tile * (long long)p.T;
        const long long left = (p.P - t0) * EB - 16LL * my_g;        // bytes of a row from this group to its end
        const int nb = left >= 16 ? 16 : (left > 0 ? (int)left : 0);
        // a group wholly past the row's end reads nothing (its address is not formed)
        const size_t off = nb > 0 ? (size_t)t0 * EB + 16u * my_g : 0;
        // group my_g of the tile piece lies in box my_g >> gpb_log2
        uint32_t dst = smem_u32(smem + p.stage_off + (size_t)st * p.stage_bytes) +
                       (uint32_t)((my_g >> p.gpb_log2) * p.d_max * p.row_bytes + my_s0 * p.row_bytes +
                                  16 * (my_g & ((1 << p.gpb_log2) - 1)));
        const uint32_t dstep = (uint32_t)(sstep * p.row_bytes);
        for (int s_ = my_s0; s_ < nd; s_ += sstep, dst += dstep) cp_async_16(dst, srcp[s_] + off, nb);
        cp_async_commit();
    };

    while (i < i_end) {
        const long long t0 = i * (long long)p.T;
        const int l0 = (int)(t0 / p.L);
        const long long bnd = (long long)(l0 + 1) * p.L;             // column where l0 + 1 starts
        const long long t1 = t0 + p.T < p.P ? t0 + p.T : p.P;
        const bool straddle = bnd < t1 && l0 + 1 < p.S;
        // run of tiles sharing this context
        long long run_end = i + 1;
        if (!straddle) {
            // tiles that end at or before bnd (or the end of the rows)
            const long long last = ((bnd < p.P ? bnd : p.P) ) / p.T;       // first tile not wholly inside
            run_end = last > i ? last : i + 1;
            if (run_end > i_end) run_end = i_end;
        }
        const int nseg = straddle ? 2 : 1;

        // ---- context: rows needed, their slots, the coefficient table
        __syncthreads();                                             // previous run fully consumed
        for (int j = tid; j < N; j += kPullThreads) slot_of[j] = -1;
        __syncthreads();
        for (int q = tid; q < nl * nseg * (R > 0 ? R : 1); q += kPullThreads) {
            if (R == 0) break;
            const int r = q % R, rest = q / R;
            const int sg = rest % nseg, wi = rest / nseg;
            const int k = p.idx[((size_t)(p.w_begin + wi) * p.S + (size_t)(l0 + sg)) * (size_t)R + r];
            if (k >= 0) slot_of[k] = -2;                             // needed (benign races: same value)
        }
        __syncthreads();
        if (warp == 0) {
            // hosted workers take slots 0 .. nl-1, the other needed rows follow in ascending order
            int nd = nl;
            for (int v0 = 0; v0 < N; v0 += 32) {
                const int v = v0 + lane;
                const bool hosted = v >= p.w_begin && v < p.w_begin + nl;
                const bool bit = v < N && !hosted && slot_of[v] == -2;
                const unsigned b = __ballot_sync(0xffffffffu, bit);
                if (bit) {
                    const int sl = nd + __popc(b & ((1u << lane) - 1u));
                    if (sl < p.d_max) { slot_of[v] = (short)sl; srcp[sl] = rowp[v]; }
                }
                nd += __popc(b);
            }
            for (int wi = lane; wi < nl; wi += 32) { slot_of[p.w_begin + wi] = (short)wi; srcp[wi] = rowp[p.w_begin + wi]; }
            if (lane == 0) s_nd = nd;
        }
        __syncthreads();
        const int nd = s_nd;
        if (nd > p.d_max) { staged_fail(20); return; }               // host bound violated: report, do not touch memory
        for (int q = tid; q < nseg * nl; q += kPullThreads) {
            const int sg = q / nl, wi = q - sg * nl;
            const int w = p.w_begin + wi;
            const int32_t* peers = p.idx + ((size_t)w * p.S + (size_t)(l0 + sg)) * (size_t)R;
            float* cf = reinterpret_cast<float*>(tab + ((size_t)sg * nl + wi) * ENT);
            int* po = UNW ? reinterpret_cast<int*>(cf) : reinterpret_cast<int*>(cf + 2 * (RMAX + 1));
            int prov[RMAX + 1];
            int np = 0;
            prov[np++] = w;
            for (int r = 0; r < R; ++r) {
                const int k = peers[r];
                if (k >= 0) prov[np++] = k;
            }
            float den = p.weights ? p.weights[prov[0]] : 1.0f;
            for (int t = 1; t < np; ++t) den = __fadd_rn(den, p.weights ? p.weights[prov[t]] : 1.0f);
            const float scale = np == 1 ? 1.0f : __fdiv_rn(1.0f, den);
            if (UNW) {
                cf[RMAX + 1] = scale;
                po[RMAX + 2] = np;
            } else {
                cf[entry_scale_word(RMAX)] = scale;
            }
            for (int r = 0; r < np; ++r) {
                if (!UNW) cf[2 * r] = cf[2 * r + 1] = (np == 1 || !p.weights) ? 1.0f : p.weights[prov[r]];
                po[r] = (int)slot_of[prov[r]] * p.row_bytes;
            }
            for (int r = np; r <= RMAX; ++r) {
                if (!UNW) cf[2 * r] = cf[2 * r + 1] = 0.0f;
                po[r] = po[0];
            }
        }
        __syncthreads();

        // ---- the run, through the ring.  One CTA-wide barrier per tile: a thread passes the
        // barrier of step j only after it has consumed tile j - 1, so behind that barrier the
        // stage of tile j - 1 is free and takes the loads of tile j + NS - 1.  A group is
        // committed per step even when the run has no tile left for it, so that "all but the
        // newest NS - 2 groups" always means tile j.
        const int NS = p.stages;                                     // >= 3
        for (int a = 0; a < NS - 1; ++a) {
            if (i + a < run_end) issue(i + a, a, nd);
            else cp_async_commit();
        }
        for (long long j = i; j < run_end; ++j) {
            const int st = (int)((j - i) % NS);
            cp_async_wait_n(NS - 2);
            __syncthreads();
            if (j + NS - 1 < run_end) issue(j + NS - 1, (int)((j - i + NS - 1) % NS), nd);
            else cp_async_commit();
            unsigned char* stage = smem + p.stage_off + (size_t)st * p.stage_bytes;
            aggregate_tile<EB, 16, RT, UNW>(ap, ws, stage, smem_u32(stage), tab, j, straddle ? bnd : (long long)1 << 62, lane);
        }
        cp_async_wait<0>();
        i = run_end;
    }
}

// Checks a table of row pointers on the device: non-null and 16-byte aligned.
__global__ void k_check_rows(const void* const* rows, int N, int32_t* flag) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j < N) {
        const uintptr_t a = reinterpret_cast<uintptr_t>(rows[j]);
        if (a == 0 || (a & 15u)) atomicCAS(flag, 0, j + 1);
    }
}

}  // namespace combo
