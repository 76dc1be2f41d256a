// Peer selection kernel (Section 4.1 step 2, "Segments Pulling").
//
// One warp per worker.  The random draw positions of a shuffle are a pure
// function of (seed, round, worker, epoch, position), so the lanes compute
// them in parallel; the swaps themselves are inherently sequential and are
// applied by one lane.  The peers of the segment being filled are kept as a
// byte map over worker ids, which serves both the "skip what this segment
// already holds" rule after a refill and the ascending output order.
//
// Section 4.1 notes that the pull requests can be sent before the local update has
// finished, since they do not depend on it.  The kernel follows that: when launched with
// programmatic stream serialization it draws the first shuffle while the preceding kernel
// of the stream (the previous round's aggregation, which still reads the old table) runs,
// and waits for it only before the first write to the table.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "segment_aggregate.cuh"

namespace combo {

// splitmix64 output function (Steele, Lea, Flood 2014) and its increment.
__device__ __forceinline__ uint64_t splitmix_out(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
__device__ __forceinline__ uint64_t splitmix_step(uint64_t state) {
    return splitmix_out(state + 0x9E3779B97F4A7C15ull);
}

constexpr int kSelectThreads = 128;

__host__ __device__ inline size_t select_peers_smem_bytes(int N) {
    // perm[N] + aux[N] + pool[N] as int32, mark[N] as bytes, rounded up
    return (size_t)N * 12 + (size_t)N + 16;
}

// One WARP per worker (several workers per CTA): everything is ordered by __syncwarp, no
// CTA-wide barrier.  MASKED: the pool of worker w is the ONLINE others (ascending); an
// offline worker issues no requests and its rows are filled with -1.
template <bool MASKED>
__global__ void __launch_bounds__(kSelectThreads)
k_select_peers(uint64_t seed, uint32_t round, int N, int S, int R, int32_t* __restrict__ idx,
               const WorkerBits online, int per_worker_bytes) {
    extern __shared__ __align__(16) unsigned char sp_smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int w = blockIdx.x * (blockDim.x >> 5) + warp;
    // the next kernel of the stream may be scheduled as soon as SMs have room for it
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (w >= N) return;
    unsigned char* mine = sp_smem + (size_t)warp * per_worker_bytes;
    int32_t* perm = reinterpret_cast<int32_t*>(mine);
    int32_t* aux = perm + N;
    int32_t* pool = aux + N;
    uint8_t* mark = reinterpret_cast<uint8_t*>(pool + N);

    int M = N - 1;
    if (MASKED) {
        if (!online.get(w)) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            for (long long i = lane; i < (long long)S * R; i += 32) idx[(size_t)w * S * R + i] = -1;
            return;
        }
        int k = 0;
        for (int v0 = 0; v0 < N; v0 += 32) {
            const int v = v0 + lane;
            const bool bit = (v < N) && (v != w) && online.get(v);
            const unsigned b = __ballot_sync(0xffffffffu, bit);
            if (bit) pool[k + __popc(b & ((1u << lane) - 1u))] = v;
            k += __popc(b);
        }
        M = k;
    }
    for (int v = lane; v < N; v += 32) mark[v] = 0;

    // chain: seed -> (round | worker) -> (epoch | position)
    uint64_t hw = splitmix_step(seed);
    hw = splitmix_step(hw ^ (((uint64_t)round << 32) | (uint64_t)(uint32_t)w));

    const long long total = (long long)S * (long long)R;
    const uint32_t epochs = (uint32_t)((total + M - 1) / M);
    long long done = 0, row = 0;   // warp-uniform
    int nc = 0;                    // peers the current segment holds so far

    for (uint32_t e = 0; e < epochs; ++e) {
        for (int t = 1 + lane; t < M; t += 32) {
            uint64_t h = splitmix_step(hw ^ (((uint64_t)e << 32) | (uint64_t)(uint32_t)t));
            aux[t] = (int32_t)(((h >> 32) * (uint64_t)(t + 1)) >> 32);   // in [0, t]
        }
        for (int i = lane; i < M; i += 32) perm[i] = MASKED ? pool[i] : i + (i >= w ? 1 : 0);
        __syncwarp();
        if (lane == 0) {
            for (int t = M - 1; t >= 1; --t) {          // Fisher-Yates
                int j = aux[t];
                int32_t a = perm[t]; perm[t] = perm[j]; perm[j] = a;
            }
            if (nc > 0) {                                // held peers go last, order kept
                int a = 0;
                for (int i = 0; i < M; ++i) if (!mark[perm[i]]) aux[a++] = perm[i];
                for (int i = 0; i < M; ++i) if (mark[perm[i]]) aux[a++] = perm[i];
                for (int i = 0; i < M; ++i) perm[i] = aux[i];
            }
        }
        __syncwarp();
        // first write to the table ahead: the preceding kernel must be done with the old one
        if (e == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
        int pos = 0;
        while (pos < M && done < total) {
            int take = R - nc;
            if (take > M - pos) take = M - pos;
            for (int i = lane; i < take; i += 32) mark[perm[pos + i]] = 1;
            pos += take; nc += take; done += take;
            __syncwarp();
            if (nc == R) {                               // emit the row ascending
                int32_t* out = idx + (size_t)((long long)w * S + row) * (size_t)R;
                int k = 0;
                for (int v0 = 0; v0 < N; v0 += 32) {
                    int v = v0 + lane;
                    bool bit = (v < N) && mark[v];
                    unsigned b = __ballot_sync(0xffffffffu, bit);
                    if (bit) {
                        out[k + __popc(b & ((1u << lane) - 1u))] = v;
                        mark[v] = 0;
                    }
                    k += __popc(b);
                }
                __syncwarp();
                nc = 0;
                ++row;
            }
        }
        __syncwarp();
    }
}

// Checks an idx table: range, never self, strictly ascending rows.
__global__ void k_validate_idx(const int32_t* __restrict__ idx, int N, int S, int R,
                               int32_t* __restrict__ flag) {
    long long total = (long long)N * S * R;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        int r = (int)(i % R);
        int w = (int)(i / ((long long)S * R));
        int v = idx[i];
        bool bad = v < 0 || v >= N || v == w || (r > 0 && idx[i - 1] >= v);
        if (bad) atomicCAS(flag, 0, (int32_t)(i < 0x7ffffffeLL ? i + 1 : 0x7fffffff));
    }
}

}  // namespace combo
