// Aggregation divergence (Section 4.3, Definition 2, Eq. 7):
//   rho_i = || W_{t,i} - W_t ||_2,   W_t = sum_j |D_j| W_j / sum_j |D_j|  (the FedAvg result)
// for all N workers in one pass over HBM.
//
//   k_divergence_staged  column tiles through all rows, staged by tiled TMA like the
//                        aggregation kernel; per tile: (A) column means from the staged
//                        block, (B) warp-per-row sums of squared deviations, carried in
//                        binary64 registers across the CTA's tiles
//   k_divergence_direct  fallback for rows that are not 16-byte aligned or N > 256:
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
constexpr int kDivTile = 256;                          // columns per tile = one TMA box

struct DivParams {
    const unsigned char* models;
    const unsigned char* src;      // rows the mean is taken over (== models when narr == 1)
    const float* weights;
    double* partial;               // scratch [grid][N]
    long long pitch, width, n_tiles;
    int N, narr, stages, row_bytes;
    unsigned coef_off, part_off, mean_off, stage_off, stage_bytes;
};

template <int EB>
__global__ void __launch_bounds__(kStagedThreads, 1)
k_divergence_staged(const DivParams p, const __grid_constant__ TileMaps maps) {
    constexpr int V = ElemOps<EB>::V;
    constexpr int NV = kDivTile / V;                   // vectors per row per tile
    constexpr int G = kConsumerThreads / NV;           // row groups of phase A
    extern __shared__ __align__(128) unsigned char smem[];
    StagedHeader* hdr = reinterpret_cast<StagedHeader*>(smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int N = p.N, stages = p.stages;
    float* coef = reinterpret_cast<float*>(smem + p.coef_off);     // c_j = |D_j| / sum |D|
    float* part = reinterpret_cast<float*>(smem + p.part_off);     // [G][kDivTile]
    float* mean = reinterpret_cast<float*>(smem + p.mean_off);     // [kDivTile]
    const int block_bytes = N * p.row_bytes;

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(&hdr->full[s]), 1);
            mbar_init(smem_u32(&hdr->empty[s]), kConsumerWarps);
        }
        mbar_init(smem_u32(&hdr->csync), kConsumerWarps);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // coefficients: the denominator is summed in worker order by every thread alike
    {
        float den = 0.0f;
        for (int j = 0; j < N; ++j) den = __fadd_rn(den, p.weights ? p.weights[j] : 1.0f);
        for (int j = tid; j < N; j += kStagedThreads) coef[j] = __fdiv_rn(p.weights ? p.weights[j] : 1.0f, den);
    }
    __syncthreads();

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        const bool issuer = lane < p.narr;
        const CUtensorMap* my_map = &maps.map[issuer ? lane : 0][0];
        if (issuer) asm volatile("prefetch.tensormap [%0];" ::"l"(my_map) : "memory");
        long long n = 0;
        for (long long tile = blockIdx.x; tile < p.n_tiles; tile += gridDim.x, ++n) {
            const int s = (int)(n % stages);
            const uint32_t ph = (uint32_t)((n / stages) & 1);
            if (!mbar_wait(smem_u32(&hdr->empty[s]), ph ^ 1u)) { staged_fail(11); break; }
            const uint32_t bar = smem_u32(&hdr->full[s]);
            if (lane == 0) mbar_arrive_expect_tx(bar, p.stage_bytes);
            __syncwarp();
            if (issuer)
                tma_load_2d(smem_u32(smem + p.stage_off + (size_t)s * p.stage_bytes) + lane * block_bytes, my_map,
                            (int)(tile * kDivTile), 0, bar);
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
    const int av = ctid % NV, ag = ctid / NV;           // phase A: vector and row group
    double acc[kDivSlots];
#pragma unroll
    for (int s = 0; s < kDivSlots; ++s) acc[s] = 0.0;

    long long n = 0;
    for (long long tile = blockIdx.x; tile < p.n_tiles; tile += gridDim.x, ++n) {
        const int s = (int)(n % stages);
        const uint32_t ph = (uint32_t)((n / stages) & 1);
        if (!mbar_wait(smem_u32(&hdr->full[s]), ph)) { staged_fail(13); return; }
        const unsigned char* stage = smem + p.stage_off + (size_t)s * p.stage_bytes;
        const unsigned char* xsrc = stage + (p.narr - 1) * block_bytes;     // rows the mean is taken over

        // (A) weighted column sums of this thread's row group; columns past the end of the
        // rows were zero-filled by the TMA unit and contribute nothing anywhere below
        {
            float a[V];
#pragma unroll
            for (int i = 0; i < V; ++i) a[i] = 0.0f;
            for (int j = ag; j < N; j += G) {
                float x[V];
                GroupLoad<EB, 16>::run(xsrc + (size_t)j * p.row_bytes + av * 16, x);
                const float c = coef[j];
#pragma unroll
                for (int i = 0; i < V; ++i) a[i] = fmaf(c, x[i], a[i]);
            }
#pragma unroll
            for (int i = 0; i < V; ++i) part[ag * kDivTile + av * V + i] = a[i];
        }
        if (!consumers_sync(csync, csync_phase, lane)) { staged_fail(14); return; }
        if (ctid < kDivTile) {
            float m = 0.0f;
#pragma unroll
            for (int g = 0; g < G; ++g) m = __fadd_rn(m, part[g * kDivTile + ctid]);
            mean[ctid] = m;
        }
        if (!consumers_sync(csync, csync_phase, lane)) { staged_fail(15); return; }

        // (B) warp per row: squared deviations of the workers' own models
#pragma unroll
        for (int sl = 0; sl < kDivSlots; ++sl) {
            const int i = cw + sl * kConsumerWarps;
            if (i < N) {
                float ssum = 0.0f;
#pragma unroll
                for (int q = 0; q < NV / 32; ++q) {
                    const int v = lane + 32 * q;
                    float x[V];
                    GroupLoad<EB, 16>::run(stage + (size_t)i * p.row_bytes + v * 16, x);
#pragma unroll
                    for (int e = 0; e < V; ++e) {
                        const float d = __fsub_rn(x[e], mean[v * V + e]);
                        ssum = fmaf(d, d, ssum);
                    }
                }
                acc[sl] += (double)ssum;
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&hdr->empty[s]));
    }
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
