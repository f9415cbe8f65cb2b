// Generic kernels of the transposable N:M mask search: one thread per M x M block, plain vector
// loads and stores.  They accept every supported (N, M, method, dtype, ld) and every shape; the
// bandwidth-tuned kernels take over the cases they cover.
//
// Work item = 32 consecutive blocks of one block row: the lanes of a warp load M rows of 32*M
// contiguous elements (fully coalesced), solve their blocks in registers, exchange mask bits with
// shuffles into whole 32-bit words, and write masked weights with the same vector width.  Every warp
// owns a contiguous range of items, so objective partials are produced in a fixed order.
#include "tm_launch.h"
#include "tm_solvers.cuh"

namespace tmask {

namespace {

constexpr int kWarpsPerCta = 8;
// The flow solver keeps three warps per scheduler busy where its 168 registers allow it (a CTA of 12 warps holds all of an
// SM's registers and, at 512 bytes of edge costs per thread, nearly all of its shared memory).
constexpr int kFlowWarpsPerCta = 12;
constexpr bool takes_flow(int N, int M, int method) { return method == kMethodExact && !(M == 4 && N == 2); }
constexpr int warps_for(int N, int M, int method) { return takes_flow(N, M, method) ? kFlowWarpsPerCta : kWarpsPerCta; }

template <int M>
__device__ __forceinline__ void load_block(const DevProblem& P, long long row0, long long col0, bool active, uint32_t (&w)[M * M]) {
    // raw element bits, one row of the block per vector load
    if (!active) {
#pragma unroll
        for (int p = 0; p < M * M; ++p) w[p] = 0;
        return;
    }
    if (P.dtype == kF32) {
        const float* base = reinterpret_cast<const float*>(P.W) + row0 * P.ld + col0;
#pragma unroll
        for (int i = 0; i < M; ++i) {
#pragma unroll
            for (int v = 0; v < M / 4; ++v) {
                const uint4 t = __ldg(reinterpret_cast<const uint4*>(base + i * P.ld) + v);
                w[i * M + 4 * v + 0] = t.x; w[i * M + 4 * v + 1] = t.y; w[i * M + 4 * v + 2] = t.z; w[i * M + 4 * v + 3] = t.w;
            }
        }
    } else {
        const uint16_t* base = reinterpret_cast<const uint16_t*>(P.W) + row0 * P.ld + col0;
#pragma unroll
        for (int i = 0; i < M; ++i) {
            if constexpr (M == 4) {
                const uint2 t = __ldg(reinterpret_cast<const uint2*>(base + i * P.ld));
                w[i * 4 + 0] = t.x << 16; w[i * 4 + 1] = t.x & 0xFFFF0000u; w[i * 4 + 2] = t.y << 16; w[i * 4 + 3] = t.y & 0xFFFF0000u;
            } else {
                const uint4 t = __ldg(reinterpret_cast<const uint4*>(base + i * P.ld));
                const uint32_t r[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
                for (int v = 0; v < 4; ++v) { w[i * 8 + 2 * v] = r[v] << 16; w[i * 8 + 2 * v + 1] = r[v] & 0xFFFF0000u; }
            }
        }
    }
}

// w holds fp32 patterns (bf16 widened); pruned entries are already zeroed
template <int M>
__device__ __forceinline__ void store_block(const DevProblem& P, long long row0, long long col0, const uint32_t (&w)[M * M]) {
    if (P.dtype == kF32) {
        float* base = reinterpret_cast<float*>(P.masked) + row0 * P.ld + col0;
#pragma unroll
        for (int i = 0; i < M; ++i) {
#pragma unroll
            for (int v = 0; v < M / 4; ++v)
                reinterpret_cast<uint4*>(base + i * P.ld)[v] = make_uint4(w[i * M + 4 * v], w[i * M + 4 * v + 1], w[i * M + 4 * v + 2], w[i * M + 4 * v + 3]);
        }
    } else {
        uint16_t* base = reinterpret_cast<uint16_t*>(P.masked) + row0 * P.ld + col0;
#pragma unroll
        for (int i = 0; i < M; ++i) {
            if constexpr (M == 4) {
                *reinterpret_cast<uint2*>(base + i * P.ld) =
                    make_uint2((w[i * 4] >> 16) | (w[i * 4 + 1] & 0xFFFF0000u), (w[i * 4 + 2] >> 16) | (w[i * 4 + 3] & 0xFFFF0000u));
            } else {
                uint32_t r[4];
#pragma unroll
                for (int v = 0; v < 4; ++v) r[v] = (w[i * 8 + 2 * v] >> 16) | (w[i * 8 + 2 * v + 1] & 0xFFFF0000u);
                *reinterpret_cast<uint4*>(base + i * P.ld) = make_uint4(r[0], r[1], r[2], r[3]);
            }
        }
    }
}

__device__ __forceinline__ const DevProblem& find_problem(const DevProblem* table, int count, long long item, int& k) {
    // items are numbered problem after problem; k is the caller's last position
    while (k + 1 < count && table[k + 1].item_begin <= item) ++k;
    return table[k];
}

// The flow solver runs a warp's 32 blocks in lockstep: every lane waits for the block that needs the most augmenting
// paths.  How many a block needs is known beforehand -- the units by which its columns exceed M - N once every row has
// pruned its M - N lightest entries -- so the blocks of kSortItems consecutive work items are dealt to the solver's
// rounds in the order of that number, and the 32 blocks of a round need about the same.
// The same block can be solved as it stands or turned (rows for columns): the optimum is the same set of entries, and the
// turned start often needs fewer paths, so every block takes the cheaper of the two.
constexpr int kSortItems = 8;
constexpr int kSortBytesPerWarp = kSortItems * 32 * (8 + 2);          // a kept mask and an order entry per block

// TURNED: the count for the block with rows and columns exchanged
template <int N, int M, bool TURNED>
__device__ __forceinline__ int repair_units(const uint32_t (&u)[M * M]) {
    int load[M];
#pragma unroll
    for (int j = 0; j < M; ++j) load[j] = 0;
#pragma unroll
    for (int i = 0; i < M; ++i) {
#pragma unroll
        for (int j = 0; j < M; ++j) {
            int heavier = 0;
            const uint32_t me = TURNED ? u[j * M + i] : u[i * M + j];
#pragma unroll
            for (int k = 0; k < M; ++k) {
                const uint32_t other = TURNED ? u[k * M + i] : u[i * M + k];
                heavier += (k != j) && (other > me || (other == me && k > j));
            }
            load[j] += heavier >= N ? 1 : 0;
        }
    }
    int d = 0;
#pragma unroll
    for (int j = 0; j < M; ++j) d += max(0, load[j] - (M - N));
    return d;
}

template <int M>
__device__ __forceinline__ void magnitudes(const uint32_t (&w)[M * M], uint32_t (&u)[M * M], int& status) {
    bool bad = false;
#pragma unroll
    for (int p = 0; p < M * M; ++p) { u[p] = w[p] & 0x7FFFFFFFu; bad |= (u[p] >> 23) == 0xFFu; }
    if (bad) status |= kDevNonFinite;
}

// mask words of one work item: row i of the item spans M words; a lane's M bits sit at M * (lane % (32 / M))
template <int M>
__device__ __forceinline__ void store_mask_words(const DevProblem& P, long long row0, int chunk, int lane, uint64_t kept) {
    constexpr int kLanesPerWord = 32 / M;          // lanes whose blocks share one mask word
#pragma unroll
    for (int i = 0; i < M; ++i) {
        uint32_t bits = (uint32_t)((kept >> (i * M)) & ((1u << M) - 1)) << (M * (lane % kLanesPerWord));
#pragma unroll
        for (int o = 1; o < kLanesPerWord; o <<= 1) bits |= __shfl_xor_sync(0xFFFFFFFFu, bits, o);
        const int word = chunk * M + lane / kLanesPerWord;
        if (lane % kLanesPerWord == 0 && word < P.wpr) P.mask[(row0 + i) * P.wpr + word] = bits;
    }
}

// Items [item, item + n) of problem P (n <= kSortItems) through the flow solver; returns the lane's share of the objective.
template <int N, int M, int W>
__device__ __forceinline__ double flow_group(const DevProblem& P, long long item, int n, unsigned char* flow_smem, unsigned char* sort_smem, int& status) {
    const int lane = threadIdx.x & 31;
    const unsigned lt = (1u << lane) - 1u;
    uint64_t* keptbuf = reinterpret_cast<uint64_t*>(sort_smem);
    unsigned short* order = reinterpret_cast<unsigned short*>(sort_smem + kSortItems * 32 * 8);   // block | turned << 15
    const long long local0 = item - P.item_begin;
    // ---- how many units each block needs ----
    int need[kSortItems], dmax = -1;
    unsigned turned = 0;                                                // bit r: block r of this lane is solved turned
#pragma unroll
    for (int r = 0; r < kSortItems; ++r) {
        need[r] = -1;
        if (r < n) {
            const long long local = local0 + r, bi = local / P.chunks;
            const int chunk = (int)(local - bi * P.chunks), bj = chunk * 32 + lane;
            if (bj < P.bcols) {
                uint32_t w[M * M], u[M * M];
                int ignored = 0;
                load_block<M>(P, bi * M, (long long)bj * M, true, w);
                magnitudes<M>(w, u, ignored);
                const int as_is = repair_units<N, M, false>(u), other_way = repair_units<N, M, true>(u);
                need[r] = min(as_is, other_way);
                turned |= (other_way < as_is ? 1u : 0u) << r;
            }
        }
        dmax = max(dmax, need[r]);
    }
    for (int o = 16; o; o >>= 1) dmax = max(dmax, __shfl_xor_sync(0xFFFFFFFFu, dmax, o));
    // ---- the blocks in descending order of that number (a counting sort by warp votes) ----
    int sorted = 0;
    for (int v = dmax; v >= 0; --v) {
#pragma unroll
        for (int r = 0; r < kSortItems; ++r) {
            const bool mine = need[r] == v;
            const unsigned m = __ballot_sync(0xFFFFFFFFu, mine);
            if (mine) order[sorted + __popc(m & lt)] = (unsigned short)((r * 32 + lane) | (((turned >> r) & 1u) << 15));
            sorted += __popc(m);
        }
    }
    __syncwarp();
    // ---- the solver, 32 blocks of about equal need at a time ----
    double acc = 0.0;
    for (int base = 0; base < sorted; base += 32) {
        const bool live = base + lane < sorted;
        const int entry = live ? order[base + lane] : 0, id = entry & 0x7FFF, r = id >> 5, l = id & 31;
        const bool turn = (entry >> 15) != 0;
        const long long local = local0 + r, bi = local / P.chunks;
        const int chunk = (int)(local - bi * P.chunks);
        const long long row0 = bi * M, col0 = ((long long)chunk * 32 + l) * M;
        uint32_t w[M * M], u[M * M];
        load_block<M>(P, row0, col0, live, w);
        magnitudes<M>(w, u, status);
        uint64_t kept = exact_ssp<N, M, W * 32>(u, status, flow_smem, (int)threadIdx.x, live, turn);
        if (!live) kept = 0;
        float sum = 0.f;
#pragma unroll
        for (int p = 0; p < M * M; ++p) sum += ((kept >> p) & 1) ? pattern_as_float(u[p]) : 0.f;
        acc += (double)sum;
        if (P.masked && live) {
#pragma unroll
            for (int p = 0; p < M * M; ++p) w[p] = ((kept >> p) & 1) ? w[p] : 0u;
            store_block<M>(P, row0, col0, w);
        }
        if (live) keptbuf[id] = kept;
    }
    __syncwarp();
    // ---- the items' mask words ----
    for (int r = 0; r < n; ++r) {
        const long long local = local0 + r, bi = local / P.chunks;
        const int chunk = (int)(local - bi * P.chunks);
        const uint64_t kept = chunk * 32 + lane < P.bcols ? keptbuf[r * 32 + lane] : 0ull;
        store_mask_words<M>(P, bi * M, chunk, lane, kept);
    }
    __syncwarp();
    return acc;
}

template <int N, int M, int METHOD>
// the exact 2:4 scorer is register-hungry: two CTAs per SM cap it at 128 registers (its rare wide-integer path spills)
__global__ void __launch_bounds__(warps_for(N, M, METHOD) * 32, (METHOD == kMethodExact && M == 4 && N == 2) ? 2 : 1)
generic_kernel(const DevProblem single, const DevProblem* __restrict__ table, int count, long long total_items,
               double* __restrict__ partials, int* __restrict__ status_out) {
    constexpr int kW = warps_for(N, M, METHOD);
    const int lane = threadIdx.x & 31;
    const long long gw = (long long)blockIdx.x * kW + (threadIdx.x >> 5);
    const long long nwarps = (long long)gridDim.x * kW;
    // even split: total / nwarps items each, the first warps one more
    const long long order = gw;
    const long long share = total_items / nwarps, surplus = total_items - share * nwarps;
    const long long begin = order * share + (order < surplus ? order : surplus);
    const long long end = begin + share + (order < surplus ? 1 : 0);
    const DevProblem* tab = table ? table : &single;

    // per-thread columns of the flow solver's state (only the exact instantiations that use it get dynamic shared memory)
    extern __shared__ __align__(16) unsigned char flow_smem[];

    int k = 0, status = 0;
    double acc = 0.0;
    int acc_k = -1;
    constexpr int kLanesPerWord = 32 / M;          // lanes whose blocks share one mask word
    constexpr int kWordsPerItem = M;               // 32 blocks * M columns / 32 bits

    if (begin < end) {          // the warp's first problem: every lane tests its own table entries (independent loads)
        int n = 0;
        for (int base = 1; base < count; base += 32) {
            const int q = base + lane;
            n += __popc(__ballot_sync(0xFFFFFFFFu, q < count && tab[q].item_begin <= begin));
        }
        k = n;
    }
    constexpr bool kFlow = METHOD == kMethodExact && !(M == 4 && N == 2);
    for (long long item = begin; item < end; ++item) {
        const DevProblem& P = find_problem(tab, count, item, k);
        if (k != acc_k) {
            if (acc_k >= 0) {
                for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
                if (lane == 0) partials[(long long)acc_k * nwarps + gw] = acc;
            }
            acc = 0.0; acc_k = k;
        }
        if constexpr (kFlow) {
            // a group of consecutive items of this problem at a time
            const long long stop = k + 1 < count ? min(end, tab[k + 1].item_begin) : end;
            const int n = (int)min((long long)kSortItems, stop - item);
            unsigned char* sort_smem = flow_smem + (size_t)flow_shared_bytes_per_thread(M) * kW * 32 + (threadIdx.x >> 5) * kSortBytesPerWarp;
            acc += flow_group<N, M, kW>(P, item, n, flow_smem, sort_smem, status);
            item += n - 1;
            continue;
        }
        const long long local = item - P.item_begin;
        const long long bi = local / P.chunks;
        const int chunk = (int)(local - bi * P.chunks);
        const int bj = chunk * 32 + lane;
        const bool active = bj < P.bcols;
        const long long row0 = bi * M, col0 = (long long)bj * M;

        uint32_t w[M * M], u[M * M];
        load_block<M>(P, row0, col0, active, w);
        bool bad = false;
#pragma unroll
        for (int p = 0; p < M * M; ++p) { u[p] = w[p] & 0x7FFFFFFFu; bad |= (u[p] >> 23) == 0xFFu; }
        if (bad) status |= kDevNonFinite;

        uint64_t kept;
        if constexpr (METHOD == kMethodExact) {
            if constexpr (M == 4 && N == 2) kept = exact_2_4(u, P.dtype == kBF16 ? 16 : 0);
            else kept = exact_ssp<N, M, kW * 32>(u, status, flow_smem, (int)threadIdx.x, active, false);
        } else {
            kept = cover_mask<N, M>(u);
            if constexpr (METHOD == kMethodApprox) {
                int rk[M], ck[M]; bool full = true;
                line_counts<M>(kept, rk, ck);
#pragma unroll
                for (int i = 0; i < M; ++i) full &= rk[i] == N;
                if (!full) kept = complete_mask<N, M>(u, kept, status);
            }
        }
        if (!active) kept = 0;

        // objective: fp32 adds inside the block, fp64 across blocks
        float s = 0.f;
#pragma unroll
        for (int p = 0; p < M * M; ++p) s += ((kept >> p) & 1) ? pattern_as_float(u[p]) : 0.f;
        acc += (double)s;

        // masked weights
        if (P.masked && active) {
#pragma unroll
            for (int p = 0; p < M * M; ++p) w[p] = ((kept >> p) & 1) ? w[p] : 0u;
            store_block<M>(P, row0, col0, w);
        }

        // mask words: row i of the item spans kWordsPerItem words; a lane's M bits sit at M*(lane % kLanesPerWord)
#pragma unroll
        for (int i = 0; i < M; ++i) {
            uint32_t bits = (uint32_t)((kept >> (i * M)) & ((1u << M) - 1)) << (M * (lane % kLanesPerWord));
#pragma unroll
            for (int o = 1; o < kLanesPerWord; o <<= 1) bits |= __shfl_xor_sync(0xFFFFFFFFu, bits, o);
            const int word = chunk * kWordsPerItem + lane / kLanesPerWord;
            if (lane % kLanesPerWord == 0 && word < P.wpr) P.mask[(row0 + i) * P.wpr + word] = bits;
        }
    }
    if (acc_k >= 0) {
        for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        if (lane == 0) partials[(long long)acc_k * nwarps + gw] = acc;
    }
    status |= __shfl_xor_sync(0xFFFFFFFFu, status, 16);
    status |= __shfl_xor_sync(0xFFFFFFFFu, status, 8);
    status |= __shfl_xor_sync(0xFFFFFFFFu, status, 4);
    status |= __shfl_xor_sync(0xFFFFFFFFu, status, 2);
    status |= __shfl_xor_sync(0xFFFFFFFFu, status, 1);
    if (lane == 0 && status && status_out) atomicOr(status_out, status);
}

// objective[k] = sum of the problem's partials in a fixed order (one CTA per problem)
__global__ void __launch_bounds__(256)
reduce_kernel(const DevProblem single, const DevProblem* __restrict__ table, const double* __restrict__ partials, long long stride) {
    const DevProblem& P = table ? table[blockIdx.x] : single;
    __shared__ double sm[256];
    double s = 0.0;
    for (long long i = threadIdx.x; i < stride; i += 256) s += partials[(long long)blockIdx.x * stride + i];
    sm[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o; o >>= 1) {
        if ((int)threadIdx.x < o) sm[threadIdx.x] += sm[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0 && P.objective) *P.objective = sm[0];
}

template <int N, int M>
cudaError_t launch_nm(const LaunchArgs& a) {
    const dim3 grid((unsigned)a.ctas), block(warps_for(N, M, a.method) * 32);
    switch (a.method) {
    case kMethodExact: {
        // the flow solver (everything but 2:4) keeps its edge costs in shared memory, and the sorted rounds their bookkeeping
        constexpr int kW = warps_for(N, M, kMethodExact);
        constexpr size_t smem = (N == 2 && M == 4) ? 0 : (size_t)flow_shared_bytes_per_thread(M) * kW * 32 + (size_t)kSortBytesPerWarp * kW;
        static_assert(smem <= 232448, "at most 227 KB of shared memory per CTA");
        static PerDeviceOnce configured;   // per instantiation
        if (smem > 48 * 1024) {
            const cudaError_t e = configured.run([&] { return cudaFuncSetAttribute(generic_kernel<N, M, kMethodExact>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); });
            if (e != cudaSuccess) return e;
        }
        generic_kernel<N, M, kMethodExact><<<grid, block, smem, a.stream>>>(a.single, a.table, a.count, a.total_items, a.partials, a.status);
        break;
    }
    case kMethodApprox: generic_kernel<N, M, kMethodApprox><<<grid, block, 0, a.stream>>>(a.single, a.table, a.count, a.total_items, a.partials, a.status); break;
    default: generic_kernel<N, M, kMethodCover><<<grid, block, 0, a.stream>>>(a.single, a.table, a.count, a.total_items, a.partials, a.status); break;
    }
    return cudaGetLastError();
}

}  // namespace

int generic_warps_per_cta(int N, int M, int method) { return warps_for(N, M, method); }
// CTAs per SM worth launching.  A flow CTA fills its SM, but its blocks take very different times: four CTAs per SM queued
// one behind the other even out what a single fat share per warp does not (8192^2, 4:8: 4.05 ms against 5.12 ms), although
// shorter shares leave the warps fewer items to sort at a time.
int generic_ctas_per_sm(int, int, int) { return 4; }

cudaError_t launch_generic(const LaunchArgs& a) {
    const int wpc = warps_for(a.N, a.M, a.method);
    cudaError_t e = cudaMemsetAsync(a.partials, 0, sizeof(double) * (size_t)a.count * (size_t)a.ctas * wpc, a.stream);
    if (e != cudaSuccess) return e;
    if (a.total_items > 0) {
        if (a.M == 4) e = a.N == 2 ? launch_nm<2, 4>(a) : (a.N == 1 ? launch_nm<1, 4>(a) : launch_nm<3, 4>(a));
        else e = a.N == 4 ? launch_nm<4, 8>(a) : (a.N == 2 ? launch_nm<2, 8>(a) : launch_nm<6, 8>(a));
        if (e != cudaSuccess) return e;
    }
    reduce_kernel<<<a.count, 256, 0, a.stream>>>(a.single, a.table, a.partials, (long long)a.ctas * wpc);
    return cudaGetLastError();
}

}  // namespace tmask
