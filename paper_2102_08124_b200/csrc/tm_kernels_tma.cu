// Bandwidth kernels of the approximate 2:4 search (TM_APPROX / TM_APPROX_COVER, M = 4).
//
// Every warp runs its own software pipeline over a contiguous range of work items (4 rows x 256
// columns of one matrix).  Items are processed two at a time:
//   1. lane 0 keeps bulk-tensor (TMA) loads of the next batch in flight into a private ring of
//      shared-memory stages (two stage sets, used alternately);
//   2. each lane reads its two 4x4 blocks of a landed item with 128-bit shared loads and runs steps
//      A and B of the search bit-parallel in registers (tm_core24.cuh); the rounds of step B are
//      warp-uniform (a vote decides whether any lane still has candidates);
//   3. the blocks that need step C (about one in six) are queued in shared memory and fixed by as
//      many lanes at once as there are queued blocks, each reading the few magnitudes it must compare
//      straight from the stage;
//   4. the lanes write the masked weights back into the stage, lane 0 sends it out with a TMA store,
//      mask bytes meet in shared memory and leave as whole 32-bit words.
// No CTA-wide synchronisation exists; every wait is bounded.
#include "tm_core24.cuh"
#include "tm_launch.h"
#include "tm_pair_bf16.cuh"
#include "tm_tma.cuh"
#include "tm_tma_items.cuh"

#include <cstring>

namespace tmask {

namespace {

constexpr int kItemRows = 4;
constexpr int kItemCols = 256;
constexpr int kBatch = 2;                  // items per pipeline step
constexpr int kStages = 2 * kBatch;

template <int DT> struct Geometry {
    static constexpr int kElem = DT == kF32 ? 4 : 2;
    static constexpr int kWarps = DT == kF32 ? 12 : 16;       // warps per CTA, one CTA per SM
    static constexpr int kRowPitch = kItemCols * kElem;        // bytes between rows inside a stage
    static constexpr int kStageBytes = kItemRows * kRowPitch;
    // stages | mask bytes [batch][4][32] | kept [batch][32] | swap candidates [batch][32] | queue | barriers
    static constexpr int kWarpBytes = kStages * kStageBytes + kBatch * 128 + 2 * kBatch * 128 + 128 + 64 + 64;
};

// ------------------------------------------------------------------------------------------
// per-dtype front end: relation masks of the lane's two blocks; largest magnitude seen
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t max_u16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.u16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

template <int DT>
__device__ __forceinline__ void front_end(const unsigned char* stage, int lane, Rel24& rel, uint32_t& worst) {
    if constexpr (DT == kBF16) {
        uint4 v[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] = *reinterpret_cast<const uint4*>(stage + i * 512 + lane * 16);
        PairKeys pk;
        interleave_keys(v, pk);
        uint32_t m[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) m[i] = max_u16x2(max_u16x2(pk.x[i][0], pk.x[i][1]), max_u16x2(pk.x[i][2], pk.x[i][3]));
        worst = max_u16x2(worst, max_u16x2(max_u16x2(m[0], m[1]), max_u16x2(m[2], m[3])));
        relations_bf16(pk, rel);
    } else {
        uint32_t ka[16], kb[16];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint4 a = *reinterpret_cast<const uint4*>(stage + i * 1024 + lane * 32);
            const uint4 b = *reinterpret_cast<const uint4*>(stage + i * 1024 + lane * 32 + 16);
            ka[4 * i] = a.x & 0x7FFFFFFFu; ka[4 * i + 1] = a.y & 0x7FFFFFFFu; ka[4 * i + 2] = a.z & 0x7FFFFFFFu; ka[4 * i + 3] = a.w & 0x7FFFFFFFu;
            kb[4 * i] = b.x & 0x7FFFFFFFu; kb[4 * i + 1] = b.y & 0x7FFFFFFFu; kb[4 * i + 2] = b.z & 0x7FFFFFFFu; kb[4 * i + 3] = b.w & 0x7FFFFFFFu;
        }
        rel = Rel24{0, 0, 0, 0, 0, 0};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t (&k)[16] = h ? kb : ka;
            const int shift = 16 * h;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t a = k[4 * i], b = k[4 * i + 1], c = k[4 * i + 2], d = k[4 * i + 3];
                rel.hr1 |= ((b >= a ? 1u : 0u) | (c >= b ? 2u : 0u) | (d >= c ? 4u : 0u) | (a > d ? 8u : 0u)) << (4 * i + shift);
                rel.hr2 |= ((c >= a ? 1u : 0u) | (d >= b ? 2u : 0u)) << (4 * i + shift);
                const uint32_t e = k[i], f = k[4 + i], g = k[8 + i], hh = k[12 + i];
                rel.hc1 |= ((f >= e ? 0x1u : 0u) | (g >= f ? 0x10u : 0u) | (hh >= g ? 0x100u : 0u) | (e > hh ? 0x1000u : 0u)) << (i + shift);
                rel.hc2 |= ((g >= e ? 0x1u : 0u) | (hh >= f ? 0x10u : 0u)) << (i + shift);
                worst = max(worst, max(max(a, b), max(c, d)));
            }
        }
        complete_relations(rel);
    }
}

// Step C, second half, on a block whose magnitudes sit in shared memory (natural layout).
template <int DT>
__device__ __forceinline__ bool swap_apply_smem(const unsigned char* blk, uint32_t& kept16, uint32_t cands16) {
    const uint32_t a = kept16, t = a | (a >> 1) | (a >> 2);
    const uint32_t rshort = ((maj3(a, a >> 1, a >> 2) | ((a >> 3) & t)) & 0x1111u) ^ 0x1111u;
    const uint32_t u = a | (a >> 4) | (a >> 8);
    const uint32_t cshort = ((maj3(a, a >> 4, a >> 8) | ((a >> 12) & u)) & 0xFu) ^ 0xFu;
    if (__popc(rshort) != 1 || __popc(cshort) != 1 || cands16 == 0 || __popc(cands16) > 3) return false;
    int x = -1; uint32_t best = 0;
#pragma unroll
    for (int n = 0; n < 3; ++n) {                                   // ascending positions: the earliest of equals wins
        if (cands16) {
            const int p = __ffs(cands16) - 1;
            cands16 &= cands16 - 1;
            uint32_t kp;
            if constexpr (DT == kBF16) kp = *reinterpret_cast<const unsigned short*>(blk + (p >> 2) * 512 + (p & 3) * 2) & 0x7FFFu;
            else kp = *reinterpret_cast<const uint32_t*>(blk + (p >> 2) * 1024 + (p & 3) * 4) & 0x7FFFFFFFu;
            if (x < 0 || kp < best) { x = p; best = kp; }
        }
    }
    const int r4 = __ffs(rshort) - 1, c = __ffs(cshort) - 1;        // r4 = 4 * short row
    if (!((kept16 >> (r4 + c)) & 1)) return false;
    kept16 = (kept16 & ~(1u << x)) | (1u << (r4 + (x & 3))) | (1u << ((x & ~3) + c));
    return true;
}

// Masked weights back into the stage, mask bytes, objective contribution of the lane's two blocks.
template <int DT, bool HAS_OUT>
__device__ __forceinline__ float back_end(unsigned char* stage, unsigned char* mrow /* [4][32] */, int lane, uint32_t kept) {
    float s4 = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if constexpr (DT == kBF16) {
            const uint4 r = *reinterpret_cast<const uint4*>(stage + i * 512 + lane * 16);
            const uint32_t raw[4] = {r.x, r.y, r.z, r.w};
            uint32_t o[4], m[4];
            lane_masks(kept, i, m);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                o[q] = raw[q] & m[q];
                const uint32_t ab = raw[q] & m[q] & 0x7FFF7FFFu;
                unsigned short lo, hi;
                asm("mov.b32 {%0,%1}, %2;" : "=h"(lo), "=h"(hi) : "r"(ab));
                asm("add.rn.f32.bf16 %0, %1, %0;" : "+f"(s4) : "h"(lo));        // fp32 accumulator + bf16 addend
                asm("add.rn.f32.bf16 %0, %1, %0;" : "+f"(s4) : "h"(hi));
            }
            if constexpr (HAS_OUT) *reinterpret_cast<uint4*>(stage + i * 512 + lane * 16) = make_uint4(o[0], o[1], o[2], o[3]);
        } else {
            const uint4 ra = *reinterpret_cast<const uint4*>(stage + i * 1024 + lane * 32);
            const uint4 rb = *reinterpret_cast<const uint4*>(stage + i * 1024 + lane * 32 + 16);
            const uint32_t raw[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w};
            uint32_t o[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const uint32_t bit = (kept >> (4 * i + (q & 3) + (q >> 2) * 16)) & 1u;
                o[q] = bit ? raw[q] : 0u;
                s4 += fabsf(__uint_as_float(o[q]));
            }
            if constexpr (HAS_OUT) {
                *reinterpret_cast<uint4*>(stage + i * 1024 + lane * 32) = make_uint4(o[0], o[1], o[2], o[3]);
                *reinterpret_cast<uint4*>(stage + i * 1024 + lane * 32 + 16) = make_uint4(o[4], o[5], o[6], o[7]);
            }
        }
        mrow[i * 32 + lane] = (unsigned char)(((kept >> (4 * i)) & 0xFu) | ((kept >> (12 + 4 * i)) & 0xF0u));
    }
    return s4;
}

template <int DT, int METHOD, bool HAS_OUT>
__global__ void __launch_bounds__(Geometry<DT>::kWarps * 32, 1)
tma24_kernel(const __grid_constant__ TmaEntry single, const TmaEntry* __restrict__ table, int count, long long total_items,
             double* __restrict__ partials, int* __restrict__ status_out) {
    using G = Geometry<DT>;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned char* stages = smem_raw + (size_t)warp * G::kWarpBytes;
    unsigned char* mbytes = stages + kStages * G::kStageBytes;
    uint32_t* kbuf = reinterpret_cast<uint32_t*>(mbytes + kBatch * 128);
    uint32_t* cbuf = kbuf + kBatch * 32;
    unsigned char* queue = reinterpret_cast<unsigned char*>(cbuf + kBatch * 32);
    uint64_t* bars = reinterpret_cast<uint64_t*>(queue + 128);

    const long long gw = (long long)blockIdx.x * G::kWarps + warp, nwarps = (long long)gridDim.x * G::kWarps;
    const long long per = (total_items + nwarps - 1) / nwarps;
    const long long begin = gw * per, end = min(total_items, begin + per);
    const int n_items = (int)max(0ll, end - begin);
    const TmaEntry* tab = table ? table : &single;

    if (lane == 0) {
        for (int s = 0; s < kStages; ++s) mbar_init(&bars[s], 1);
        fence_mbar_init();
    }
    __syncwarp();

    Cursor ld, cur;                        // next item to request / first item of the batch in process
    ld.seek(tab, count, begin);
    cur = ld;
    int loaded = 0;
    auto issue_next = [&](int s) {         // all lanes track the cursor, lane 0 issues the copy
        if (lane == 0) {
            mbar_expect_tx(&bars[s], G::kStageBytes);
            tma_load_2d(stages + s * G::kStageBytes, &tab[ld.k].in, ld.cj * kItemCols, ld.bi * kItemRows, &bars[s]);
        }
        ld.advance(tab, count);
        ++loaded;
    };
    for (int g = 0; g < kBatch && loaded < n_items; ++g) issue_next(g);

    int status = 0, acc_k = -1;
    float facc = 0.f; double acc = 0.0;
    uint32_t worst = 0;                                                  // largest magnitude pattern seen (per 16-bit lane for bf16)
    const uint32_t lt = (1u << lane) - 1u;
    bool alive = true;

    for (int done = 0, batch = 0; done < n_items && alive; done += kBatch, ++batch) {
        const int nb = min(kBatch, n_items - done), set = batch & 1;
        const uint32_t parity = (uint32_t)((batch >> 1) & 1);
        int qn = 0;
        // ---- steps A and B on every item of the batch -------------------------------------------
#pragma unroll
        for (int g = 0; g < kBatch; ++g) {
            if (g < nb) {
                const int s = set * kBatch + g;
                if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(&bars[s], parity))) { status |= kDevInternal; alive = false; }
                Rel24 rel;
                front_end<DT>(stages + s * G::kStageBytes, lane, rel, worst);
                uint32_t k = cover_2_4(rel);
                if constexpr (METHOD == kMethodApprox) {
                    LineFill f = line_fill(k);
                    uint32_t cand = open_candidates(k, f);
                    int rounds = 0;
                    while (__any_sync(0xFFFFFFFFu, cand != 0)) {
                        if (++rounds > 4) { status |= kDevInternal; break; }    // a block lacks at most four entries
                        k |= fill_accept(rel, k, cand);
                        f = line_fill(k);
                        cand = open_candidates(k, f);
                    }
                    const uint32_t sb = short_blocks(f);
                    if (__any_sync(0xFFFFFFFFu, sb != 0)) {
                        cbuf[g * 32 + lane] = swap_candidates(rel, f, k);
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const bool need = (sb >> h) & 1;
                            const uint32_t m = __ballot_sync(0xFFFFFFFFu, need);
                            if (need) queue[qn + __popc(m & lt)] = (unsigned char)((g << 6) | (h << 5) | lane);
                            qn += __popc(m);
                        }
                    }
                }
                kbuf[g * 32 + lane] = k;
            }
            if (g == 0) {      // refill the other stage set: its stores were issued one batch ago
                if constexpr (HAS_OUT) { if (lane == 0 && batch > 0) tma_wait_read<0>(); }
                for (int gg = 0; gg < kBatch; ++gg) if (loaded < n_items) issue_next((set ^ 1) * kBatch + gg);
            }
        }
        __syncwarp();
        // ---- step C on the queued blocks ---------------------------------------------------------
        if constexpr (METHOD == kMethodApprox) {
            for (int q0 = 0; q0 < qn; q0 += 32) {
                if (q0 + lane < qn) {
                    const uint32_t e = queue[q0 + lane];
                    const int g = e >> 6, h = (e >> 5) & 1, ln = e & 31;
                    unsigned short* kh = reinterpret_cast<unsigned short*>(kbuf + g * 32 + ln) + h;
                    uint32_t k16 = *kh;
                    const uint32_t c16 = reinterpret_cast<const unsigned short*>(cbuf + g * 32 + ln)[h];
                    const unsigned char* blk = stages + (set * kBatch + g) * G::kStageBytes + ln * (8 * G::kElem) + h * (4 * G::kElem);
                    if (!swap_apply_smem<DT>(blk, k16, c16)) status |= kDevInternal;
                    *kh = (unsigned short)k16;
                }
            }
            __syncwarp();
        }
        // ---- outputs ---------------------------------------------------------------------------
        Cursor out = cur;
#pragma unroll
        for (int g = 0; g < kBatch; ++g) {
            if (g < nb) {
                if (out.k != acc_k) {                                   // a new matrix starts: flush the objective partial
                    if (acc_k >= 0) {
                        acc += (double)facc;
                        for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
                        if (lane == 0) partials[(long long)acc_k * nwarps + gw] = acc;
                    }
                    acc = 0.0; facc = 0.f; acc_k = out.k;
                }
                uint32_t k = kbuf[g * 32 + lane];
                // blocks past the last column (zero-filled by the copy) contribute nothing
                const int col0 = out.cj * kItemCols + lane * 8;
                const int cols = (int)tab[out.k].p.cols;
                if (col0 >= cols) k = 0;
                else if (col0 + 4 >= cols) k &= 0xFFFFu;
                facc += back_end<DT, HAS_OUT>(stages + (set * kBatch + g) * G::kStageBytes, mbytes + g * 128, lane, k);
                out.advance(tab, count);
            }
        }
        if constexpr (HAS_OUT) fence_proxy_async_smem();
        __syncwarp();
        out = cur;
#pragma unroll
        for (int g = 0; g < kBatch; ++g) {
            if (g < nb) {
                const TmaEntry& e = tab[out.k];
                if constexpr (HAS_OUT) {
                    if (lane == 0) tma_store_2d(&e.out, out.cj * kItemCols, out.bi * kItemRows, stages + (set * kBatch + g) * G::kStageBytes);
                }
                const int row = lane >> 3, word = out.cj * 8 + (lane & 7);
                const uint32_t w = *reinterpret_cast<const uint32_t*>(mbytes + g * 128 + row * 32 + (lane & 7) * 4);
                if (word < e.p.wpr) e.p.mask[((long long)out.bi * kItemRows + row) * e.p.wpr + word] = w;
                out.advance(tab, count);
            }
        }
        if constexpr (HAS_OUT) { if (lane == 0) tma_commit(); }
        cur = out;
        if ((batch & 31) == 31) { acc += (double)facc; facc = 0.f; }       // keep the fp32 partial short
        __syncwarp();
    }
    if (!alive && lane == 0) {
        // a copy never landed: give the copies still in flight a bounded chance to finish before the stages die
        for (int s = 0; s < kStages; ++s) { mbar_wait_bounded(&bars[s], 0, 1u << 14); mbar_wait_bounded(&bars[s], 1, 1u << 14); }
    }
    if (lane == 0) tma_wait_all<0>();
    if (acc_k >= 0) {
        acc += (double)facc;
        for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        if (lane == 0) partials[(long long)acc_k * nwarps + gw] = acc;
    }
    if constexpr (DT == kF32) { if (worst >= 0x7F800000u) status |= kDevNonFinite; }
    else { if ((worst & 0xFFFFu) >= 0x7F80u || (worst >> 16) >= 0x7F80u) status |= kDevNonFinite; }
    for (int o = 16; o; o >>= 1) status |= __shfl_xor_sync(0xFFFFFFFFu, status, o);
    if (lane == 0 && status && status_out) atomicOr(status_out, status);
}

// objective[k] = sum of the problem's partials in a fixed order (one CTA per problem)
__global__ void __launch_bounds__(256)
reduce_tma_kernel(const __grid_constant__ TmaEntry single, const TmaEntry* __restrict__ table, const double* __restrict__ partials, long long stride) {
    const DevProblem& P = table ? table[blockIdx.x].p : single.p;
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

template <int DT, int METHOD, bool HAS_OUT>
cudaError_t launch_one(const TmaLaunch& a, const TmaEntry& single, const TmaEntry* table) {
    using G = Geometry<DT>;
    const size_t smem = (size_t)G::kWarps * G::kWarpBytes;
    auto kern = tma24_kernel<DT, METHOD, HAS_OUT>;
    static bool configured = false;        // per instantiation
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    kern<<<a.ctas, G::kWarps * 32, smem, a.stream>>>(single, table, a.count, a.total_items, a.partials, a.status);
    return cudaGetLastError();
}

}  // namespace

size_t tma_entry_bytes() { return sizeof(TmaEntry); }
int tma_warps_per_cta(int dtype, int M) { return M == 8 ? tma48_warps_per_cta(dtype) : (dtype == kF32 ? Geometry<kF32>::kWarps : Geometry<kBF16>::kWarps); }

bool tma_eligible(const DevProblem& p, int N, int M, int method) {
    if (!((N == 2 && M == 4) || (N == 4 && M == 8)) || (method != kMethodApprox && method != kMethodCover)) return false;
    const size_t elem = p.dtype == kF32 ? 4 : 2;
    if ((uintptr_t)p.W % 16 || ((size_t)p.ld * elem) % 16) return false;
    if (p.masked && (uintptr_t)p.masked % 16) return false;
    if (p.rows >= (1ll << 31) || p.cols >= (1ll << 31) - kItemCols || (size_t)p.ld * elem >= (1ull << 40)) return false;
    if ((p.rows / M) * ((p.cols + kItemCols - 1) / kItemCols) >= (1ll << 30)) return false;
    return encode_fn() != nullptr;
}

// Fills `entries_host` (count TmaEntry records) for problems that all passed tma_eligible(); an item is M rows x 256 columns.
bool tma_build_entries(const DevProblem* probs, int count, void* entries_host, long long* total_items, int M) {
    return build_entries(probs, count, static_cast<TmaEntry*>(entries_host), total_items, M, kItemCols);
}

cudaError_t tma_reduce(const void* entries_host, const void* entries_dev, int count, const double* partials, long long stride, cudaStream_t stream) {
    const TmaEntry* host = static_cast<const TmaEntry*>(entries_host);
    reduce_tma_kernel<<<count, 256, 0, stream>>>(host[0], static_cast<const TmaEntry*>(entries_dev), partials, stride);
    return cudaGetLastError();
}

// All problems of one launch share dtype and the presence of masked_w_out (the caller groups them).
cudaError_t launch_tma(const TmaLaunch& a) {
    if (a.M == 8) return launch_tma48(a);
    const int wpc = tma_warps_per_cta(a.dtype, 4);
    cudaError_t err = cudaMemsetAsync(a.partials, 0, sizeof(double) * (size_t)a.count * (size_t)a.ctas * wpc, a.stream);
    if (err != cudaSuccess) return err;
    const TmaEntry* host = static_cast<const TmaEntry*>(a.entries_host);
    const TmaEntry* table = static_cast<const TmaEntry*>(a.entries_dev);   // nullptr when count == 1
    if (a.total_items > 0) {
#define TM_DISPATCH(DT, METHOD)                                                                                   \
    err = a.has_out ? launch_one<DT, METHOD, true>(a, host[0], table) : launch_one<DT, METHOD, false>(a, host[0], table)
        if (a.dtype == kF32) { if (a.method == kMethodApprox) TM_DISPATCH(kF32, kMethodApprox); else TM_DISPATCH(kF32, kMethodCover); }
        else { if (a.method == kMethodApprox) TM_DISPATCH(kBF16, kMethodApprox); else TM_DISPATCH(kBF16, kMethodCover); }
#undef TM_DISPATCH
        if (err != cudaSuccess) return err;
    }
    reduce_tma_kernel<<<a.count, 256, 0, a.stream>>>(host[0], table, a.partials, (long long)a.ctas * wpc);
    return cudaGetLastError();
}

}  // namespace tmask
