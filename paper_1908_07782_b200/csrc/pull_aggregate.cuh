// Worker-sharded aggregation (Section 3 "Segmented Pulling", Eq. 2 and Eq. 3): the workers'
// rows live in separate allocations -- on this GPU or, through peer mappings, on other GPUs
// of the node -- and this GPU forms the new models of the workers it hosts.
//
// A pull is a load: for worker w and segment l the kernel reads W_w[l] and the R segments
// W_k[l] of its peers straight from where they live (plain 128-bit global loads, which work
// on peer memory over NVLink; no bulk-tensor copy, no multicast), combines them in the fixed
// order of Eq. 3 (self, then peers ascending) and writes the result to local memory.  What
// crosses NVLink is exactly what the paper's workers send each other: R segments per
// (hosted worker, segment), each once.  Nothing is staged: a remote element is used by one
// hosted worker only, so there is no reuse to stage for.
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
            float den = p.weights ? p.weights[w] : 1.0f;
            for (int r = 0; r < R; ++r)
                if (peers[r] >= 0) den = __fadd_rn(den, p.weights ? p.weights[peers[r]] : 1.0f);
            float acc[V], x[V];
            GroupLoad<EB, 16>::run(rows[w] + (size_t)c0 * EB, x);
            float c = __fdiv_rn(p.weights ? p.weights[w] : 1.0f, den);
#pragma unroll
            for (int i = 0; i < V; ++i) acc[i] = __fmul_rn(c, x[i]);
            for (int r = 0; r < R; ++r) {
                const int k = peers[r];
                if (k < 0) continue;
                GroupLoad<EB, 16>::run(rows[k] + (size_t)c0 * EB, x);
                c = __fdiv_rn(p.weights ? p.weights[k] : 1.0f, den);
#pragma unroll
                for (int i = 0; i < V; ++i) acc[i] = fmaf(c, x[i], acc[i]);
            }
            ElemOps<EB>::store_vec(orow + (size_t)c0 * EB, acc);
        } else {
            // a group that holds a segment boundary or the end of the row: element by element
            for (long long col = c0; col < hi; ++col) {
                const int32_t* peers = my_idx + (size_t)(col / p.L) * R;
                float den = p.weights ? p.weights[w] : 1.0f;
                for (int r = 0; r < R; ++r)
                    if (peers[r] >= 0) den = __fadd_rn(den, p.weights ? p.weights[peers[r]] : 1.0f);
                float acc = __fmul_rn(__fdiv_rn(p.weights ? p.weights[w] : 1.0f, den),
                                      ElemOps<EB>::load(rows[w] + (size_t)col * EB));
                for (int r = 0; r < R; ++r) {
                    const int k = peers[r];
                    if (k < 0) continue;
                    acc = fmaf(__fdiv_rn(p.weights ? p.weights[k] : 1.0f, den),
                               ElemOps<EB>::load(rows[k] + (size_t)col * EB), acc);
                }
                ElemOps<EB>::store(orow + (size_t)col * EB, acc);
            }
        }
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
