// Neighbouring operations of the mask search (Section 5 of the paper and the operand preparation the
// transposable mask exists for):
//   nm1d_kernel        1-D N:M magnitude pruning along rows, with the pattern-violation count and the
//                      optional mean absorption, fused with the packed mask / masked weights / objective;
//   violations_kernel  pattern-violations of an arbitrary packed mask;
//   compress24_kernel  2:4 compressed values + 2-bit indices for W and for W^T from one transposable mask,
//                      one read of W (the transposed half goes through a shared-memory tile).
// All three stream the matrix once with vector loads; they are bound by HBM bandwidth.
#include <type_traits>

#include "tm_launch.h"
#include "tm_tma.cuh"
#include "tm_tma_items.cuh"

namespace tmask {

namespace {

constexpr int kAuxWarps = 8;
constexpr int kUnit = 8;                      // elements per thread and step: one mask byte


// raw element bits of one unit (8 elements from column c0 of row r); elements past `cols` read as 0
template <int DT>
__device__ __forceinline__ void load_unit(const AuxProblem& P, long long r, long long c0, uint32_t (&raw)[kUnit]) {
    const int valid = (int)min((long long)kUnit, P.cols - c0);
    if constexpr (DT == kF32) {
        const uint32_t* p = reinterpret_cast<const uint32_t*>(P.W) + r * P.ld + c0;
        if (valid == kUnit && ((uintptr_t)p & 15) == 0) {
            const uint4 a = __ldg(reinterpret_cast<const uint4*>(p)), b = __ldg(reinterpret_cast<const uint4*>(p) + 1);
            raw[0] = a.x; raw[1] = a.y; raw[2] = a.z; raw[3] = a.w; raw[4] = b.x; raw[5] = b.y; raw[6] = b.z; raw[7] = b.w;
        } else {
#pragma unroll
            for (int j = 0; j < kUnit; ++j) raw[j] = j < valid ? __ldg(p + j) : 0u;
        }
    } else {
        const uint16_t* p = reinterpret_cast<const uint16_t*>(P.W) + r * P.ld + c0;
        if (valid == kUnit && ((uintptr_t)p & 15) == 0) {
            const uint4 a = __ldg(reinterpret_cast<const uint4*>(p));
            const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) { raw[2 * j] = w[j] & 0xFFFFu; raw[2 * j + 1] = w[j] >> 16; }
        } else {
#pragma unroll
            for (int j = 0; j < kUnit; ++j) raw[j] = j < valid ? (uint32_t)__ldg(p + j) : 0u;
        }
    }
}
template <int DT>
__device__ __forceinline__ void store_unit(const AuxProblem& P, long long r, long long c0, const uint32_t (&out)[kUnit]) {
    const int valid = (int)min((long long)kUnit, P.cols - c0);
    if constexpr (DT == kF32) {
        uint32_t* p = reinterpret_cast<uint32_t*>(P.masked) + r * P.ld + c0;
        if (valid == kUnit && ((uintptr_t)p & 15) == 0) {
            reinterpret_cast<uint4*>(p)[0] = make_uint4(out[0], out[1], out[2], out[3]);
            reinterpret_cast<uint4*>(p)[1] = make_uint4(out[4], out[5], out[6], out[7]);
        } else {
#pragma unroll
            for (int j = 0; j < kUnit; ++j) if (j < valid) p[j] = out[j];
        }
    } else {
        uint16_t* p = reinterpret_cast<uint16_t*>(P.masked) + r * P.ld + c0;
        if (valid == kUnit && ((uintptr_t)p & 15) == 0) {
            *reinterpret_cast<uint4*>(p) = make_uint4(out[0] | (out[1] << 16), out[2] | (out[3] << 16), out[4] | (out[5] << 16), out[6] | (out[7] << 16));
        } else {
#pragma unroll
            for (int j = 0; j < kUnit; ++j) if (j < valid) p[j] = (uint16_t)out[j];
        }
    }
}

template <int DT> __device__ __forceinline__ uint32_t magnitude(uint32_t raw) { return DT == kF32 ? (raw & 0x7FFFFFFFu) : (raw & 0x7FFFu); }
template <int DT> __device__ __forceinline__ float value_of(uint32_t raw) { return DT == kF32 ? __uint_as_float(raw) : bf16_to_float(raw); }

constexpr int kSub = 4;                       // units per thread and item: keeps 64-128 bytes per thread in flight

// MODE 0: 1-D N:M pruning (N kept per group of M).  MODE 1: violations of a given mask.
// Work item = 128 consecutive units (1024 elements) of one row: lane l handles units l, l+32, l+64, l+96.
template <int DT, int M, int MODE>
__global__ void __launch_bounds__(kAuxWarps * 32)
nm1d_kernel(const AuxProblem P, int N, int flags, double* __restrict__ obj_partials, unsigned long long* __restrict__ viol_partials,
            int* __restrict__ status_out) {
    const int lane = threadIdx.x & 31;
    const long long gw = (long long)blockIdx.x * kAuxWarps + (threadIdx.x >> 5), nwarps = (long long)gridDim.x * kAuxWarps;
    const long long units = (P.cols + kUnit - 1) / kUnit, chunks = (units + 32 * kSub - 1) / (32 * kSub), total = P.rows * chunks;
    const long long per = (total + nwarps - 1) / nwarps, begin = gw * per, end = min(total, begin + per);
    double acc = 0.0; unsigned long long viol = 0; bool bad = false;
    long long r = begin < end ? begin / chunks : 0, chunk = begin < end ? begin - r * chunks : 0;
    for (long long item = begin; item < end; ++item) {
        uint32_t raw[kSub][kUnit];
        uint32_t given[kSub];
#pragma unroll
        for (int s = 0; s < kSub; ++s) {                 // all loads of the item first
            const long long unit = (chunk * kSub + s) * 32 + lane, c0 = unit * kUnit;
            if (c0 < P.cols) load_unit<DT>(P, r, c0, raw[s]);
            else {
#pragma unroll
                for (int j = 0; j < kUnit; ++j) raw[s][j] = 0;
            }
            if constexpr (MODE == 1) {
                const long long word = unit >> 2;
                given[s] = (c0 < P.cols && word < P.wpr) ? (__ldg(P.mask + r * P.wpr + word) >> (8 * (unit & 3))) & 0xFFu : 0xFFu;
            }
        }
#pragma unroll
        for (int s = 0; s < kSub; ++s) {
            const long long unit = (chunk * kSub + s) * 32 + lane, c0 = unit * kUnit;
            const bool active = c0 < P.cols;
            uint32_t mag[kUnit];
#pragma unroll
            for (int j = 0; j < kUnit; ++j) { mag[j] = magnitude<DT>(raw[s][j]); bad |= mag[j] >= (DT == kF32 ? 0x7F800000u : 0x7F80u); }
            if constexpr (MODE == 0) {
                uint32_t keep = 0;
#pragma unroll
                for (int j = 0; j < kUnit; ++j) {      // kept iff fewer than N entries of the group are heavier
                    int heavier = 0;
#pragma unroll
                    for (int k = (j / M) * M; k < (j / M) * M + M; ++k)
                        if (k != j) heavier += (k > j) ? (mag[k] >= mag[j]) : (mag[k] > mag[j]);
                    keep |= (heavier < N ? 1u : 0u) << j;
                }
                const int valid = active ? (int)min((long long)kUnit, P.cols - c0) : 0;
                keep &= (1u << valid) - 1u;
                float sum = 0.f;
                uint32_t out[kUnit];
#pragma unroll
                for (int j = 0; j < kUnit; ++j) {
                    const bool k = (keep >> j) & 1u;
                    out[j] = k ? raw[s][j] : 0u;
                    sum += k ? __uint_as_float(DT == kF32 ? mag[j] : (mag[j] << 16)) : 0.f;
                    viol += (!k && j < valid && mag[j] != 0) ? 1ull : 0ull;
                }
                acc += (double)sum;
                if (flags & 1) {                         // mean absorption, fp64, one rounding to fp32 (then to bf16)
#pragma unroll
                    for (int g = 0; g < kUnit / M; ++g) {
                        double psum = 0.0; int pcnt = 0;
#pragma unroll
                        for (int j = g * M; j < g * M + M; ++j) if (!((keep >> j) & 1u)) { psum += (double)value_of<DT>(raw[s][j]); ++pcnt; }
                        const double mu = pcnt ? psum / (double)pcnt : 0.0;
#pragma unroll
                        for (int j = g * M; j < g * M + M; ++j)
                            if ((keep >> j) & 1u) {
                                const float v = (float)((double)value_of<DT>(raw[s][j]) + mu);
                                out[j] = DT == kF32 ? __float_as_uint(v) : float_to_bf16_bits(v);
                            }
                    }
                }
                if (P.masked && active) store_unit<DT>(P, r, c0, out);
                // four lanes share a mask word
                uint32_t bits = keep << (8 * (lane & 3));
                bits |= __shfl_xor_sync(0xFFFFFFFFu, bits, 1);
                bits |= __shfl_xor_sync(0xFFFFFFFFu, bits, 2);
                const long long word = (chunk * kSub + s) * 8 + (lane >> 2);
                if ((lane & 3) == 0 && word < P.wpr) P.mask[r * P.wpr + word] = bits;
            } else {
#pragma unroll
                for (int j = 0; j < kUnit; ++j) viol += (!((given[s] >> j) & 1u) && mag[j] != 0) ? 1ull : 0ull;
            }
        }
        if (++chunk == chunks) { chunk = 0; ++r; }
    }
    for (int o = 16; o; o >>= 1) { acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o); viol += __shfl_xor_sync(0xFFFFFFFFu, viol, o); }
    if (lane == 0) { obj_partials[gw] = acc; viol_partials[gw] = viol; }
    if (__any_sync(0xFFFFFFFFu, bad) && lane == 0 && status_out) atomicOr(status_out, kDevNonFinite);
}

__global__ void __launch_bounds__(256)
aux_reduce_kernel(const double* __restrict__ obj_partials, const unsigned long long* __restrict__ viol_partials, int n,
                  double* objective_out, unsigned long long* violations_out) {
    __shared__ double so[256]; __shared__ unsigned long long sv[256];
    double a = 0.0; unsigned long long v = 0;
    for (int i = threadIdx.x; i < n; i += 256) { a += obj_partials[i]; v += viol_partials[i]; }
    so[threadIdx.x] = a; sv[threadIdx.x] = v;
    __syncthreads();
    for (int o = 128; o; o >>= 1) {
        if ((int)threadIdx.x < o) { so[threadIdx.x] += so[threadIdx.x + o]; sv[threadIdx.x] += sv[threadIdx.x + o]; }
        __syncthreads();
    }
    if (threadIdx.x == 0) { if (objective_out) *objective_out = so[0]; if (violations_out) *violations_out = sv[0]; }
}

// Pattern violations of a given mask, streaming form for aligned matrices (16-byte aligned rows, cols % 8 == 0):
// a lane takes eight consecutive weights (one mask byte) at a time, four such units in flight; the non-zero
// test is two weights per operation for bf16.  Work item = 1024 consecutive weights of one row.
template <int DT>
__global__ void __launch_bounds__(kAuxWarps * 32)
violations_stream_kernel(const AuxProblem P, unsigned long long* __restrict__ viol_partials) {
    const int lane = threadIdx.x & 31;
    const long long gw = (long long)blockIdx.x * kAuxWarps + (threadIdx.x >> 5), nwarps = (long long)gridDim.x * kAuxWarps;
    const long long units = P.cols / kUnit, chunks = (units + 127) / 128, total = P.rows * chunks;
    const unsigned char* mbytes = reinterpret_cast<const unsigned char*>(P.mask);
    unsigned long long viol = 0;
    // items dealt round-robin: the grid reads one dense window of the matrix at a time
    const long long dr = nwarps / chunks, dc = nwarps - dr * chunks;
    long long r = gw / chunks, chunk = gw - r * chunks;
    for (long long item = gw; item < total; item += nwarps) {
        constexpr int kWords = DT == kF32 ? 8 : 4;
        uint32_t w[4][kWords], given[4];
#pragma unroll
        for (int s = 0; s < 4; ++s) {                         // all loads of the item first
            const long long unit = (chunk * 4 + s) * 32 + lane;
            const bool in = unit < units;
            given[s] = in ? (uint32_t)__ldg(mbytes + r * P.wpr * 4 + unit) : 0xFFu;
            if constexpr (DT == kF32) {
                const uint4* p = reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(P.W) + r * P.ld + unit * kUnit);
                const uint4 a = in ? __ldg(p) : make_uint4(0, 0, 0, 0), b = in ? __ldg(p + 1) : make_uint4(0, 0, 0, 0);
                w[s][0] = a.x; w[s][1] = a.y; w[s][2] = a.z; w[s][3] = a.w; w[s][4] = b.x; w[s][5] = b.y; w[s][6] = b.z; w[s][7] = b.w;
            } else {
                const uint4* p = reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(P.W) + r * P.ld + unit * kUnit);
                const uint4 a = in ? __ldg(p) : make_uint4(0, 0, 0, 0);
                w[s][0] = a.x; w[s][1] = a.y; w[s][2] = a.z; w[s][3] = a.w;
            }
        }
#pragma unroll
        for (int s = 0; s < 4; ++s) {
            uint32_t nz = 0;
            if constexpr (DT == kF32) {
#pragma unroll
                for (int j = 0; j < 8; ++j) nz |= ((w[s][j] & 0x7FFFFFFFu) ? 1u : 0u) << j;
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {                 // 15-bit magnitude + 0x7FFF has its top bit set iff the magnitude is not zero
                    const uint32_t t = ((w[s][j] & 0x7FFF7FFFu) + 0x7FFF7FFFu) >> 15;
                    nz |= ((t & 1u) | ((t >> 15) & 2u)) << (2 * j);
                }
            }
            viol += (unsigned)__popc(nz & ~given[s]);
        }
        r += dr; chunk += dc;
        if (chunk >= chunks) { chunk -= chunks; ++r; }
    }
    for (int o = 16; o; o >>= 1) viol += __shfl_xor_sync(0xFFFFFFFFu, viol, o);
    if (lane == 0) viol_partials[gw] = viol;
}

// number of differing bits of two packed masks (how much a refresh changed the mask)
__global__ void __launch_bounds__(kAuxWarps * 32)
hamming_kernel(const uint32_t* __restrict__ a, const uint32_t* __restrict__ b, long long words, unsigned long long* __restrict__ partials) {
    const int lane = threadIdx.x & 31;
    const long long gw = (long long)blockIdx.x * kAuxWarps + (threadIdx.x >> 5), nwarps = (long long)gridDim.x * kAuxWarps;
    unsigned long long n = 0;
    if ((((uintptr_t)a | (uintptr_t)b) & 15) == 0) {
        // 16 bytes per lane and load, the warps of the grid side by side (one dense window of both masks at a time)
        const long long quads = words / 4;
        const uint4* a4 = reinterpret_cast<const uint4*>(a);
        const uint4* b4 = reinterpret_cast<const uint4*>(b);
#pragma unroll 2
        for (long long i = gw * 32 + lane; i < quads; i += nwarps * 32) {
            const uint4 x = __ldg(a4 + i), y = __ldg(b4 + i);
            n += __popc(x.x ^ y.x) + __popc(x.y ^ y.y) + __popc(x.z ^ y.z) + __popc(x.w ^ y.w);
        }
        if (gw == 0 && quads * 4 + lane < words) n += __popc(__ldg(a + quads * 4 + lane) ^ __ldg(b + quads * 4 + lane));
    } else {
        const long long per = ((words + nwarps - 1) / nwarps + 31) / 32 * 32, begin = gw * per, end = min(words, begin + per);
        for (long long i = begin + lane; i < end; i += 32) n += __popc(__ldg(a + i) ^ __ldg(b + i));
    }
    for (int o = 16; o; o >>= 1) n += __shfl_xor_sync(0xFFFFFFFFu, n, o);
    if (lane == 0) partials[gw] = n;
}
__global__ void __launch_bounds__(256)
hamming_reduce_kernel(const unsigned long long* __restrict__ partials, int n, unsigned long long* out) {
    __shared__ unsigned long long sv[256];
    unsigned long long v = 0;
    for (int i = threadIdx.x; i < n; i += 256) v += partials[i];
    sv[threadIdx.x] = v;
    __syncthreads();
    for (int o = 128; o; o >>= 1) { if ((int)threadIdx.x < o) sv[threadIdx.x] += sv[threadIdx.x + o]; __syncthreads(); }
    if (threadIdx.x == 0) *out = sv[0];
}

// ---- 2:4 compression ---------------------------------------------------------------------------
// CTA tile: 128 rows x 128 columns = 32 x 32 blocks of 4x4; a warp takes block rows 4w .. 4w+3 of the
// tile, lane = block column.  The row form (values, meta) is written straight from registers, 128 bytes per
// row and warp.  The column form is collected in shared memory so that every column of the tile leaves as one
// run of 64 values (128 bytes of bf16) written with 16-byte stores, and its four metadata words in one go.
// Shared tile: the kept pair of (column c, block row br) at word ((c & 3) * 32 + (c >> 2)) * pitch + br * kVW:
// lanes of a warp (columns four apart) fall into different banks.
// Metadata nibble idx0 | idx1 << 2 of a keep nibble with exactly two bits set (never zero), 0 for any other nibble:
// sixteen 4-bit entries in one 64-bit word.
__device__ __forceinline__ uint32_t pair_nibble(uint32_t m) {
    constexpr unsigned long long kTable = (4ull << 12) | (8ull << 20) | (9ull << 24) | (12ull << 36) | (13ull << 40) | (14ull << 48);
    return (uint32_t)(kTable >> (4 * m)) & 0xFu;
}

template <int DT>
__global__ void __launch_bounds__(256)
compress24_kernel(const AuxProblem P, void* __restrict__ values, uint32_t* __restrict__ meta, void* __restrict__ values_t,
                  uint32_t* __restrict__ meta_t, int* __restrict__ status_out) {
    constexpr int kVW = DT == kF32 ? 2 : 1;             // words per kept pair
    constexpr int kPitch = 32 * kVW + 1;
    __shared__ uint32_t tile_t[128 * kPitch];
    // transposed metadata: word k (block rows 8k .. 8k+7) of column 4*lane + j at [k][j][lane]; a warp owns one 16-bit
    // half of its words (its four block rows), so no two warps ever write the same bytes
    __shared__ uint32_t tile_mt[4][4][32];
    // bf16: the kept pair of four 16-bit values held in two words leaves with one byte permute; entry m of the table is
    // that permute's selector for keep nibble m (halfwords idx0, idx1) with the metadata nibble above it, 0 for a nibble
    // that does not keep exactly two
    __shared__ uint32_t pair_tab[16];
    if (threadIdx.x < 16) {
        const uint32_t nib = pair_nibble(threadIdx.x), i0 = nib & 3u, i1 = nib >> 2;
        pair_tab[threadIdx.x] = nib ? ((2 * i0) | ((2 * i0 + 1) << 4) | ((2 * i1) << 8) | ((2 * i1 + 1) << 12) | (nib << 16)) : 0u;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long tiles_c = (P.cols + 127) / 128, tiles_r = (P.rows + 127) / 128;
    const long long wpr_t = (P.rows + 31) / 32, half_c = P.cols / 2, half_r = P.rows / 2;
    const size_t ebytes = DT == kF32 ? 4 : 2;
    const bool vec_t = (uintptr_t)values_t % 16 == 0 && ((size_t)half_r * ebytes) % 16 == 0;
    bool bad = false;
    for (long long t = blockIdx.x; t < tiles_r * tiles_c; t += gridDim.x) {
        const long long tr = t / tiles_c, tc = t - tr * tiles_c;
        const long long c0 = tc * 128 + lane * 4;
        uint32_t col_nibbles[4] = {0, 0, 0, 0};      // nibble `it` = metadata of column j in block row 4 * warp + it
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int br = warp * 4 + it;                // block row inside the tile
            const long long r0 = tr * 128 + br * 4;
            const bool active = r0 < P.rows && c0 < P.cols;
            uint32_t v[4][4] = {}, mbits = 0;            // mbits bit 4i+j = mask of (row i, column j)
            uint2 raw[4] = {};                           // bf16: the row's four values as loaded
            if (active) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if constexpr (DT == kF32) {
                        const uint4 a = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const uint32_t*>(P.W) + (r0 + i) * P.ld + c0));
                        v[i][0] = a.x; v[i][1] = a.y; v[i][2] = a.z; v[i][3] = a.w;
                    } else {
                        raw[i] = __ldg(reinterpret_cast<const uint2*>(reinterpret_cast<const uint16_t*>(P.W) + (r0 + i) * P.ld + c0));
                    }
                    mbits |= ((__ldg(P.mask + (r0 + i) * P.wpr + (c0 >> 5)) >> (c0 & 31)) & 0xFu) << (4 * i);
                }
            }
            // row form: two kept values per row, in column order, and their indices
            uint32_t row_nibbles = 0;                    // nibble i = metadata of row i
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t m = (mbits >> (4 * i)) & 0xFu;
                uint32_t nib;
                if constexpr (DT == kF32) {
                    uint32_t a = 0, b = 0;
                    nib = pair_nibble(m);
                    if (nib) {
                        const int i0 = nib & 3, i1 = nib >> 2;
                        a = i0 == 0 ? v[i][0] : (i0 == 1 ? v[i][1] : v[i][2]);
                        b = i1 == 1 ? v[i][1] : (i1 == 2 ? v[i][2] : v[i][3]);
                    }
                    if (active) *reinterpret_cast<uint2*>(reinterpret_cast<uint32_t*>(values) + (r0 + i) * half_c + (c0 >> 1)) = make_uint2(a, b);
                } else {
                    const uint32_t e = pair_tab[m];
                    nib = e >> 16;
                    const uint32_t pair = nib ? __byte_perm(raw[i].x, raw[i].y, e) : 0u;
                    if (active) *reinterpret_cast<uint32_t*>(reinterpret_cast<uint16_t*>(values) + (r0 + i) * half_c + (c0 >> 1)) = pair;
                }
                if (!nib && active) bad = true;
                row_nibbles |= nib << (4 * i);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {                // eight lanes share a metadata word of a row
                uint32_t w = ((row_nibbles >> (4 * i)) & 0xFu) << (4 * (lane & 7));
                w |= __shfl_xor_sync(0xFFFFFFFFu, w, 1); w |= __shfl_xor_sync(0xFFFFFFFFu, w, 2); w |= __shfl_xor_sync(0xFFFFFFFFu, w, 4);
                if ((lane & 7) == 0 && active) meta[(r0 + i) * P.wpr + (c0 >> 5)] = w;
            }
            // column form into the shared tile
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                // bit j of the four row nibbles, gathered by a multiplication (bits 0, 4, 8, 12 land on 9, 10, 11, 12)
                const uint32_t m = ((((mbits >> j) & 0x1111u) * 0x249u) >> 9) & 0xFu;
                uint32_t* slot = tile_t + (j * 32 + lane) * kPitch + br * kVW;
                uint32_t nib;
                if constexpr (DT == kF32) {
                    uint32_t a = 0, b = 0;
                    nib = pair_nibble(m);
                    if (nib) {
                        const int i0 = nib & 3, i1 = nib >> 2;
                        a = i0 == 0 ? v[0][j] : (i0 == 1 ? v[1][j] : v[2][j]);
                        b = i1 == 1 ? v[1][j] : (i1 == 2 ? v[2][j] : v[3][j]);
                    }
                    slot[0] = a; slot[1] = b;
                } else {
                    // the column's four values as two words (rows 0,1 and rows 2,3), then the same table
                    const uint32_t sel = (j & 1) ? 0x7632u : 0x5410u;
                    const uint32_t c01 = j < 2 ? __byte_perm(raw[0].x, raw[1].x, sel) : __byte_perm(raw[0].y, raw[1].y, sel);
                    const uint32_t c23 = j < 2 ? __byte_perm(raw[2].x, raw[3].x, sel) : __byte_perm(raw[2].y, raw[3].y, sel);
                    const uint32_t e = pair_tab[m];
                    nib = e >> 16;
                    slot[0] = nib ? __byte_perm(c01, c23, e) : 0u;
                }
                if (!nib && active) bad = true;
                col_nibbles[j] |= nib << (4 * it);
            }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j)
            reinterpret_cast<unsigned short*>(&tile_mt[warp >> 1][j][lane])[warp & 1] = (unsigned short)col_nibbles[j];
        __syncthreads();
        {   // 128 columns: two threads per column, each half of its 64 values and two of its four metadata words
            const int c = threadIdx.x >> 1, h = threadIdx.x & 1;
            const long long col = tc * 128 + c;
            if (col < P.cols) {
                const uint32_t* src = tile_t + ((c & 3) * 32 + (c >> 2)) * kPitch + h * 16 * kVW;
                const long long v0 = tr * 64 + h * 32;                      // first value index along the transposed row
                unsigned char* dst = reinterpret_cast<unsigned char*>(values_t) + ((size_t)col * half_r + v0) * ebytes;
                if (vec_t && v0 + 32 <= half_r) {
#pragma unroll
                    for (int q = 0; q < 4 * kVW; ++q)
                        reinterpret_cast<uint4*>(dst)[q] = make_uint4(src[4 * q], src[4 * q + 1], src[4 * q + 2], src[4 * q + 3]);
                } else {
                    for (int k = 0; k < 16 * kVW; ++k)                      // pairs of values (bf16) or single values (fp32), 4 bytes each
                        if (v0 + (DT == kF32 ? k : 2 * k) < half_r) reinterpret_cast<uint32_t*>(dst)[k] = src[k];
                }
#pragma unroll
                for (int k = 0; k < 2; ++k)
                    if (tr * 4 + h * 2 + k < wpr_t) meta_t[col * wpr_t + tr * 4 + h * 2 + k] = tile_mt[h * 2 + k][c & 3][c >> 2];
            }
        }
        __syncthreads();
    }
    if (bad && status_out) atomicOr(status_out, kDevBadMask);
}

}  // namespace

int aux_partial_slots() { return 8192; }

cudaError_t launch_aux_reduce(const double* obj_partials, const unsigned long long* viol_partials, int n, double* objective_out,
                              unsigned long long* violations_out, cudaStream_t stream) {
    aux_reduce_kernel<<<1, 256, 0, stream>>>(obj_partials, viol_partials, n, objective_out, violations_out);
    return cudaGetLastError();
}

static int aux_grid(long long items, int sms) {
    const long long want = (items + kAuxWarps - 1) / kAuxWarps;
    const long long cap = (long long)sms * 8 < 1024 ? (long long)sms * 8 : 1024;
    return (int)(want < 1 ? 1 : (want > cap ? cap : want));
}

cudaError_t launch_nm1d(const AuxProblem& P, int N, int M, int flags, bool violations_only, double* obj_partials,
                        unsigned long long* viol_partials, double* objective_out, unsigned long long* violations_out,
                        int* status, int sms, cudaStream_t stream) {
    const long long units = (P.cols + kUnit - 1) / kUnit, items = P.rows * ((units + 32 * kSub - 1) / (32 * kSub));
    const int grid = aux_grid(items, sms);
#define TM_NM1D(DT, MM, MODE) nm1d_kernel<DT, MM, MODE><<<grid, kAuxWarps * 32, 0, stream>>>(P, N, flags, obj_partials, viol_partials, status)
    const size_t elem = P.dtype == kF32 ? 4 : 2;
    const bool streamable = violations_only && P.cols % kUnit == 0 && (uintptr_t)P.W % 16 == 0 && ((size_t)P.ld * elem) % 16 == 0;
    if (streamable) {
        if (P.dtype == kF32) violations_stream_kernel<kF32><<<grid, kAuxWarps * 32, 0, stream>>>(P, viol_partials);
        else violations_stream_kernel<kBF16><<<grid, kAuxWarps * 32, 0, stream>>>(P, viol_partials);
        cudaError_t es = cudaGetLastError();
        if (es != cudaSuccess) return es;
        hamming_reduce_kernel<<<1, 256, 0, stream>>>(viol_partials, grid * kAuxWarps, violations_out);
        return cudaGetLastError();
    }
    if (violations_only) { if (P.dtype == kF32) TM_NM1D(kF32, 8, 1); else TM_NM1D(kBF16, 8, 1); }
    else if (P.dtype == kF32) { if (M == 2) TM_NM1D(kF32, 2, 0); else if (M == 4) TM_NM1D(kF32, 4, 0); else TM_NM1D(kF32, 8, 0); }
    else { if (M == 2) TM_NM1D(kBF16, 2, 0); else if (M == 4) TM_NM1D(kBF16, 4, 0); else TM_NM1D(kBF16, 8, 0); }
#undef TM_NM1D
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    aux_reduce_kernel<<<1, 256, 0, stream>>>(obj_partials, viol_partials, grid * kAuxWarps, objective_out, violations_out);
    return cudaGetLastError();
}

cudaError_t launch_hamming(const uint32_t* a, const uint32_t* b, long long words, unsigned long long* partials, unsigned long long* out,
                           int sms, cudaStream_t stream) {
    const int grid = aux_grid((words + 31) / 32, sms);
    hamming_kernel<<<grid, kAuxWarps * 32, 0, stream>>>(a, b, words, partials);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    hamming_reduce_kernel<<<1, 256, 0, stream>>>(partials, grid * kAuxWarps, out);
    return cudaGetLastError();
}

cudaError_t launch_compress24(const AuxProblem& P, void* values, uint32_t* meta, void* values_t, uint32_t* meta_t, int* status,
                              int sms, cudaStream_t stream) {
    const long long tiles = ((P.rows + 127) / 128) * ((P.cols + 127) / 128);
    if (tiles == 0) return cudaSuccess;
    // bf16 matrices with 16-byte aligned rows and mask rows stream through per-warp pipelines (tm_kernels_compress.cu)
    if (compress24_stream_eligible(P, values, meta, meta_t)) return launch_compress24_stream(P, values, meta, values_t, meta_t, status, sms, stream);
    const int grid = (int)(tiles < (long long)sms * 8 ? tiles : (long long)sms * 8);
    if (P.dtype == kF32) compress24_kernel<kF32><<<grid, 256, 0, stream>>>(P, values, meta, values_t, meta_t, status);
    else compress24_kernel<kBF16><<<grid, 256, 0, stream>>>(P, values, meta, values_t, meta_t, status);
    return cudaGetLastError();
}

}  // namespace tmask
