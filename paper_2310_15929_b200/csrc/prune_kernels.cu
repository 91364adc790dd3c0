// Producer side of the E-Sparse hot path: channel statistics (Eq. 1, Eq. 2), score (Eq. 3), global
// naive shuffle, local block shuffle (Algorithm 1, Eq. 5), 2-of-4 selection and compression.
//
// All of these stream fp16 matrices once or twice; they are HBM-bound or (block shuffle) bound by plain
// fp64 compares.  Every quantity that feeds a discrete decision is fp64 with explicit round-to-nearest
// multiplies/adds (no FMA contraction), and every sum over rows of |W| is taken exactly in 64-bit
// integers of 2^-24, so results do not depend on the order in which threads visit rows.
#include "esp_common.cuh"

#include <math.h>

namespace esp {

namespace {

constexpr int kLbsMax = 256;       // widest local-shuffle block
constexpr int kLbsGroups = kLbsMax / 4;

__device__ __forceinline__ double half_bits_abs_to_double(uint16_t h) {
    return (double)__half2float(__ushort_as_half((unsigned short)(h & 0x7FFFu)));
}

// |h| as an integer multiple of 2^-24 (exact for every finite fp16).
__device__ __forceinline__ long long half_bits_abs_fixed(uint16_t h) {
    int e = (h >> 10) & 31;
    long long m = h & 1023;
    return e == 0 ? m : ((1024 + m) << (e - 1));
}

// --------------------------------------------------------------------------------------------------
// K1: per-channel sum of squares (fp64), min and max over a slice of tokens.   Eq. 2 / range of Eq. 1.
// grid (ceil(C/256), splits), block 256 = 32 channel-vectors of 8 x 8 token lanes.
// --------------------------------------------------------------------------------------------------
constexpr int kColAhead = 8;                                              // rows each thread keeps in flight
constexpr int kColSmem = (kColAhead + 1) * 256 * 16;                      // the threads' load rings; >= the partial results after
static_assert(kColSmem >= (int)(sizeof(double) * 8 * 257 + 2 * sizeof(float) * 8 * 257), "the reduction reuses the ring");
__global__ void __launch_bounds__(256) colstats_kernel(const __half *__restrict__ X, int T, int C, long ldx,
                                                       int rows_per_split, double *__restrict__ part_sumsq,
                                                       float *__restrict__ part_min, float *__restrict__ part_max) {
    extern __shared__ __align__(16) unsigned char s_dyn[];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int c0 = (blockIdx.x * 32 + tx) * 8;
    const int r_begin = blockIdx.y * rows_per_split;
    const int r_end = min(T, r_begin + rows_per_split);
    double acc[8];
    float mn[8], mx[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) { acc[k] = 0.0; mn[k] = INFINITY; mx[k] = -INFINITY; }
    if (c0 < C) {
        auto add_row = [&](const uint4 &v) {
            const __half *h = reinterpret_cast<const __half *>(&v);
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                float f = __half2float(h[k]);
                acc[k] = __dadd_rn(acc[k], (double)(f * f));   // f*f is exact in fp32 (22-bit product)
                mn[k] = fminf(mn[k], f);
                mx[k] = fmaxf(mx[k], f);
            }
        };
        // Rows in the same order as a plain loop (the order of the fp64 additions is part of the result).  This thread's rows
        // are r_begin + ty + 8 i, i < n; kColAhead of its 16-byte pieces are kept in flight through a private slot ring in
        // shared memory (asynchronous copies, one group per row; one slot more than rows in flight, so the slot being
        // refilled is the one read an iteration ago) -- the registers leave no room for that many rows.
        const int n = (r_end - r_begin - ty + 7) / 8;
        const __half *xcol = X + (long)(r_begin + ty) * ldx + c0;
        uint4 *ring = reinterpret_cast<uint4 *>(s_dyn) + threadIdx.x;      // slot j of this thread: ring[256 * j]
        const uint32_t ring_s = (uint32_t)__cvta_generic_to_shared(ring);
        int wr = 0;
        auto fetch = [&](int i) {
            if (i < n)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ring_s + (uint32_t)(wr * 4096)), "l"(xcol + (long)i * 8 * ldx)
                             : "memory");
            asm volatile("cp.async.commit_group;" ::: "memory");          // (an empty group past the end keeps the count in step)
            wr = wr == kColAhead ? 0 : wr + 1;
        };
#pragma unroll
        for (int i = 0; i < kColAhead; ++i) fetch(i);
        int rd = 0;
        for (int i = 0; i < n; ++i) {
            asm volatile("cp.async.wait_group %0;" ::"n"(kColAhead - 1) : "memory");
            const uint4 v = ring[256 * rd];
            rd = rd == kColAhead ? 0 : rd + 1;
            fetch(i + kColAhead);
            add_row(v);
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();                         // every thread is done with its ring: the buffer now holds the partial results
    double (*s_acc)[256 + 1] = reinterpret_cast<double (*)[256 + 1]>(s_dyn);
    float (*s_mn)[256 + 1] = reinterpret_cast<float (*)[256 + 1]>(s_dyn + sizeof(double) * 8 * 257);
    float (*s_mx)[256 + 1] = reinterpret_cast<float (*)[256 + 1]>(s_dyn + sizeof(double) * 8 * 257 + sizeof(float) * 8 * 257);
#pragma unroll
    for (int k = 0; k < 8; ++k) { s_acc[ty][tx * 8 + k] = acc[k]; s_mn[ty][tx * 8 + k] = mn[k]; s_mx[ty][tx * 8 + k] = mx[k]; }
    __syncthreads();
    const int c = blockIdx.x * 256 + threadIdx.x;
    if (c < C) {
        double a = 0.0;
        float lo = INFINITY, hi = -INFINITY;
#pragma unroll
        for (int y = 0; y < 8; ++y) {      // fixed order: deterministic
            a = __dadd_rn(a, s_acc[y][threadIdx.x]);
            lo = fminf(lo, s_mn[y][threadIdx.x]);
            hi = fmaxf(hi, s_mx[y][threadIdx.x]);
        }
        part_sumsq[(long)blockIdx.y * C + c] = a;
        part_min[(long)blockIdx.y * C + c] = lo;
        part_max[(long)blockIdx.y * C + c] = hi;
    }
}

__global__ void colstats_finish_kernel(int C, int splits, const double *__restrict__ part_sumsq,
                                       const float *__restrict__ part_min, const float *__restrict__ part_max,
                                       double *__restrict__ norm, double *__restrict__ lo, double *__restrict__ hi) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    double a = 0.0;
    float mn = INFINITY, mx = -INFINITY;
    for (int s = 0; s < splits; ++s) {
        a = __dadd_rn(a, part_sumsq[(long)s * C + c]);
        mn = fminf(mn, part_min[(long)s * C + c]);
        mx = fmaxf(mx, part_max[(long)s * C + c]);
    }
    norm[c] = sqrt(a);
    lo[c] = (double)mn;
    hi[c] = (double)mx;
}

// The layer-wide bin range: every channel's [lo, hi] replaced by the minimum and maximum over all channels (one CTA).
__global__ void __launch_bounds__(1024) global_range_kernel(int C, double *__restrict__ lo, double *__restrict__ hi) {
    __shared__ double s_lo[32], s_hi[32];
    double mn = INFINITY, mx = -INFINITY;
    for (int c = threadIdx.x; c < C; c += 1024) { mn = fmin(mn, lo[c]); mx = fmax(mx, hi[c]); }
    for (int o = 16; o > 0; o >>= 1) {
        mn = fmin(mn, __shfl_xor_sync(0xFFFFFFFFu, mn, o));
        mx = fmax(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
    }
    if ((threadIdx.x & 31) == 0) { s_lo[threadIdx.x >> 5] = mn; s_hi[threadIdx.x >> 5] = mx; }
    __syncthreads();
    mn = s_lo[0]; mx = s_hi[0];
    for (int w = 1; w < 32; ++w) { mn = fmin(mn, s_lo[w]); mx = fmax(mx, s_hi[w]); }
    __syncthreads();
    for (int c = threadIdx.x; c < C; c += 1024) { lo[c] = mn; hi[c] = mx; }
}

// Streaming calibration: fold one chunk's partial statistics into the running state (chunk order = call order).
__global__ void calib_merge_kernel(int C, int splits, const double *__restrict__ part_sumsq, const float *__restrict__ part_min,
                                   const float *__restrict__ part_max, double *__restrict__ sumsq, double *__restrict__ lo,
                                   double *__restrict__ hi) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    double a = 0.0;
    float mn = INFINITY, mx = -INFINITY;
    for (int s = 0; s < splits; ++s) {
        a = __dadd_rn(a, part_sumsq[(long)s * C + c]);
        mn = fminf(mn, part_min[(long)s * C + c]);
        mx = fmaxf(mx, part_max[(long)s * C + c]);
    }
    sumsq[c] = __dadd_rn(sumsq[c], a);
    lo[c] = fmin(lo[c], (double)mn);
    hi[c] = fmax(hi[c], (double)mx);
}
__global__ void calib_reset_kernel(int C, int bins, double *sumsq, double *lo, double *hi, unsigned int *counts) {
    const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < C) { sumsq[i] = 0.0; lo[i] = INFINITY; hi[i] = -INFINITY; }
    if (i < (long)C * bins) counts[i] = 0u;
}
__global__ void calib_norm_kernel(int C, const double *__restrict__ sumsq, double *__restrict__ norm) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c < C) norm[c] = sqrt(sumsq[c]);
}

// --------------------------------------------------------------------------------------------------
// K2: per-channel histogram with K equal-width bins on [lo_c, hi_c] (Eq. 1's bins), exact integer counts.
// bin = min(K-1, floor((x - lo) * K / (hi - lo))) in fp64: the numerator is exact and the quotient is
// correctly rounded, which yields the exact bin for fp16 data.
// grid (ceil(C/64), splits), block 256 = 8 channel-vectors of 8 x 32 token lanes; counters in shared memory.
// --------------------------------------------------------------------------------------------------
// The exact bin of one element (fp64), for the few elements the fp32 estimate cannot decide.  Kept out of line so that the
// streaming loop carries none of its operands in registers: the channel's range is re-read (from L1) when needed.
__device__ __noinline__ int histogram_exact_bin(float xf, int c, int bins, const double *__restrict__ lo,
                                                const double *__restrict__ hi) {
    const double l = lo[c];
    const double rng = __dsub_rn(hi[c], l);
    if (!(rng > 0.0)) return 0;                                          // a constant channel: everything in bin 0
    const double q = __ddiv_rn(__dmul_rn(__dsub_rn((double)xf, l), (double)bins), rng);
    return max(0, min(bins - 1, (int)floor(q)));                         // (the clamp at 0 only keeps a NaN in bounds)
}

// Counters in shared memory: [k = channel within the thread's eight][bin][tx = the thread's channel group][replica].
// The 32 lanes of a warp are 8 channel groups x 4 token rows, and one instruction counts the same k in all of them, so a
// lane's bank is (bin * 8 + tx) * R + replica: lanes of different channel groups never meet in a bank, and the four lanes
// of a group meet only through the low bits of their bins.  R = 4 gives each of them a counter row of its own (no conflict
// at all), R = 2 one per two, R = 1 none (expected 1.0 / 1.5 / 2.1 passes per counting instruction; the plain
// [channel][bin] layout needed 3.3).  R is chosen so that three CTAs still fit an SM.
constexpr int kHistAhead = 8;                 // rows each thread keeps in flight
template <int R>
__global__ void __launch_bounds__(256, 3) histogram_kernel(const __half *__restrict__ X, int T, int C, long ldx,
                                                           int rows_per_split, int bins, const double *__restrict__ lo,
                                                           const double *__restrict__ hi, unsigned int *__restrict__ counts) {
    extern __shared__ __align__(16) unsigned int s_cnt[];   // [8][bins][8][R] | the threads' load rings: [kHistAhead + 1][256] x 16 bytes
    for (int i = threadIdx.x; i < 64 * R * bins; i += 256) s_cnt[i] = 0;
    __syncthreads();
    const int tx = threadIdx.x & 7, ty = threadIdx.x >> 3;
    const int cl = tx * 8;
    const int c0 = blockIdx.x * 64 + cl;
    const int r_begin = blockIdx.y * rows_per_split;
    const int r_end = min(T, r_begin + rows_per_split);
    if (c0 < C) {
        // Exact bin: floor of the fp64 quotient q = (x - lo) * K / (hi - lo).  Almost every element gets there with one fp32
        // subtraction and one fused multiply-add, and no float <-> integer conversion (those run at a quarter of the fp32
        // rate): with 2^S the largest power of two such that K * 2^S <= 2^22 and r = K * 2^S / (hi - lo) rounded once,
        //     t = fma(x - lo, r, 2^23)
        // lies in [2^23, 2^24), where floats are the integers, so the low 23 bits of t ARE n = round((x - lo) * r), and
        // |n - q * 2^S| <= 1: the subtraction (lo is exact in fp32) and r are each within 2^-24 relative, together at most
        // q * 2^S * 2^-23 <= 1/2, and the fma rounds once to an integer, at most 1/2.  So wherever n mod 2^S is neither
        // 0, 1, 2^S - 2 nor 2^S - 1, n >> S is the exact bin.  The other elements (4 in 2^S: about one in ten thousand for
        // a hundred bins, and always the channel's minimum and maximum) take the fp64 division.  r = 0 gives n = 0 and sends
        // every element of a channel there (a constant channel, or a range whose lower end is not an fp16 value).
        const int S = 22 - (32 - __clz(bins - 1));                            // bins >= 2
        const unsigned int frac_mask = (1u << S) - 1u;
        float lf[8], rf[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const double l = lo[c0 + k];
            const double rng = __dsub_rn(hi[c0 + k], l);
            lf[k] = (float)l;
            rf[k] = (rng > 0.0 && (double)lf[k] == l) ? (float)(((double)bins / rng) * (double)(1 << S)) : 0.f;
            if (!(rf[k] <= 0x1p60f)) rf[k] = 0.f;                            // (a range so small that r overflows: exact path)
        }
        uint32_t cnt_k[8];                                                 // this thread's counter of bin 0 for each of its channels
#pragma unroll
        for (int k = 0; k < 8; ++k)
            cnt_k[k] = (uint32_t)__cvta_generic_to_shared(s_cnt + ((k * bins) * 8 + tx) * R + (ty & (R - 1)));
        const unsigned int last_bin = (unsigned int)(bins - 1);
        // One branch per row of eight elements, not one per element: the eight estimates are formed first, together with the
        // smallest distance-to-a-boundary code among them; only a row that holds an undecided element (about one row in a
        // thousand) goes back over its elements.
        auto count_row = [&](const uint4 &v) {
            const __half2 *h2 = reinterpret_cast<const __half2 *>(&v);
            unsigned int b[8], closest = 0xFFFFFFFFu;
#pragma unroll
            for (int k2 = 0; k2 < 4; ++k2) {
                const float2 xf2 = __half22float2(h2[k2]);
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int k = 2 * k2 + e;
                    const float xf = e ? xf2.y : xf2.x;
                    const unsigned int n = __float_as_uint(fmaf(xf - lf[k], rf[k], 8388608.f)) - 0x4B000000u;
                    // (the clamp keeps the index inside the counter row whatever the input, e.g. a NaN)
                    b[k] = min(n >> S, last_bin);
                    closest = min(closest, (n + 2u) & frac_mask);
                }
            }
            if (closest < 4u) {
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float xf = __half2float(reinterpret_cast<const __half *>(&v)[k]);
                    const unsigned int n = __float_as_uint(fmaf(xf - lf[k], rf[k], 8388608.f)) - 0x4B000000u;
                    if (((n + 2u) & frac_mask) < 4u) b[k] = (unsigned int)histogram_exact_bin(xf, c0 + k, bins, lo, hi);
                }
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) asm volatile("red.shared.add.u32 [%0], 1;" ::"r"(cnt_k[k] + (uint32_t)(32 * R) * b[k]) : "memory");
        };
        // This thread's rows are r_begin + ty + 32 * i, i < n.  Loads and counting must overlap, and with 80 registers per thread
        // (three CTAs per SM) there is no room for a second set of rows in registers: every thread keeps kHistAhead of its own
        // 16-byte pieces in flight into a private slot ring in shared memory (asynchronous copies, one group per row; no
        // other thread touches the slots, so no barrier is needed).
        const int n = (r_end - r_begin - ty + 31) / 32;
        const __half *xcol = X + (long)(r_begin + ty) * ldx + c0;
        uint4 *ring = reinterpret_cast<uint4 *>(s_cnt + 64 * R * bins) + threadIdx.x;      // slot j of this thread: ring[256 * j]
        const uint32_t ring_s = (uint32_t)__cvta_generic_to_shared(ring);
        // (one slot more than rows in flight: the slot being refilled is the one read an iteration ago, whose values are used up)
        int wr = 0;
        auto fetch = [&](int i) {
            if (i < n)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ring_s + (uint32_t)(wr * 4096)),
                             "l"(xcol + (long)i * 32 * ldx)
                             : "memory");
            asm volatile("cp.async.commit_group;" ::: "memory");          // (an empty group past the end keeps the count in step)
            wr = wr == kHistAhead ? 0 : wr + 1;
        };
#pragma unroll
        for (int i = 0; i < kHistAhead; ++i) fetch(i);
        int rd = 0;
        for (int i = 0; i < n; ++i) {
            asm volatile("cp.async.wait_group %0;" ::"n"(kHistAhead - 1) : "memory");
            const uint4 v = ring[256 * rd];
            rd = rd == kHistAhead ? 0 : rd + 1;
            fetch(i + kHistAhead);
            count_row(v);
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 64 * bins; i += 256) {
        const int cc = i / bins, b = i - cc * bins;                        // channel of this CTA, bin
        const int c = blockIdx.x * 64 + cc;
        const unsigned int *src = s_cnt + (((cc & 7) * bins + b) * 8 + (cc >> 3)) * R;
        unsigned int n = 0;
#pragma unroll
        for (int rep = 0; rep < R; ++rep) n += src[rep];
        if (c < C && n) atomicAdd(&counts[(long)c * bins + b], n);
    }
}

// Counter replicas for a bin count: as many as keep three CTAs on an SM (about 75 KB each), none beyond.
inline esp_status_t launch_histogram(const __half *X, int T, int C, long ldx, int splits, int bins, const double *lo,
                                     const double *hi, unsigned int *counts, cudaStream_t stream) {
    const size_t per_replica = sizeof(unsigned int) * 64 * (size_t)bins;
    const size_t ring = (size_t)(kHistAhead + 1) * 256 * 16;
    const int R = per_replica * 4 + ring <= 75 * 1024 ? 4 : per_replica * 2 + ring <= 75 * 1024 ? 2 : 1;
    const size_t smem = per_replica * R + ring;
    const dim3 grid(ceil_div(C, 64), splits);
    const int rows = ceil_div(T, splits);
    if (R == 4) {
        ESP_CUDA_OK(cudaFuncSetAttribute(histogram_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        histogram_kernel<4><<<grid, 256, smem, stream>>>(X, T, C, ldx, rows, bins, lo, hi, counts);
    } else if (R == 2) {
        ESP_CUDA_OK(cudaFuncSetAttribute(histogram_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        histogram_kernel<2><<<grid, 256, smem, stream>>>(X, T, C, ldx, rows, bins, lo, hi, counts);
    } else {
        ESP_CUDA_OK(cudaFuncSetAttribute(histogram_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        histogram_kernel<1><<<grid, 256, smem, stream>>>(X, T, C, ldx, rows, bins, lo, hi, counts);
    }
    return ESP_OK;
}

// IR_c = -sum_k p_k ln p_k (Eq. 1, bins in index order, empty bins skipped) and s_c = IR_c + alpha*AM_c (Eq. 3).
__global__ void entropy_score_kernel(int C, int T, int bins, const unsigned int *__restrict__ counts,
                                     const double *__restrict__ norm, double alpha, int use_entropy, int use_norm,
                                     const double *__restrict__ score_override, double *__restrict__ entropy,
                                     double *__restrict__ score) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    double ir = 0.0;
    if (counts) {
        for (int k = 0; k < bins; ++k) {
            unsigned int n = counts[(long)c * bins + k];
            if (n) {
                double p = __ddiv_rn((double)n, (double)T);
                ir = __dsub_rn(ir, __dmul_rn(p, log(p)));
            }
        }
        entropy[c] = ir;
    }
    double s = 0.0;
    if (score_override) {
        s = score_override[c];
    } else {
        if (use_entropy) s = __dadd_rn(s, ir);
        if (use_norm) s = __dadd_rn(s, __dmul_rn(alpha, norm[c]));
    }
    score[c] = s;
}

// --------------------------------------------------------------------------------------------------
// K3: exact column sums of |W| (units of 2^-24) -> mean of the metric per channel (for the global shuffle).
// --------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) colabs_kernel(const __half *__restrict__ W, int No, int C, long ldw,
                                                     int rows_per_split, unsigned long long *__restrict__ colsum) {
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int c0 = (blockIdx.x * 32 + tx) * 8;
    const int r_begin = blockIdx.y * rows_per_split;
    const int r_end = min(No, r_begin + rows_per_split);
    long long acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (c0 < C) {
        for (int r = r_begin + ty; r < r_end; r += 8) {
            uint4 v = __ldg(reinterpret_cast<const uint4 *>(W + (long)r * ldw + c0));
            const uint16_t *h = reinterpret_cast<const uint16_t *>(&v);
#pragma unroll
            for (int k = 0; k < 8; ++k) acc[k] += half_bits_abs_fixed(h[k]);
        }
    }
    __shared__ long long s_acc[8][256 + 1];
#pragma unroll
    for (int k = 0; k < 8; ++k) s_acc[ty][tx * 8 + k] = acc[k];
    __syncthreads();
    const int c = blockIdx.x * 256 + threadIdx.x;
    if (c < C) {
        long long a = 0;
#pragma unroll
        for (int y = 0; y < 8; ++y) a += s_acc[y][threadIdx.x];
        atomicAdd(&colsum[c], (unsigned long long)a);      // integer: order-independent
    }
}

__global__ void mean_metric_kernel(int C, int No, const unsigned long long *__restrict__ colsum,
                                   const double *__restrict__ score, double *__restrict__ mean) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    double a = __dmul_rn(__ll2double_rn((long long)colsum[c]), 0x1p-24);
    mean[c] = __ddiv_rn(__dmul_rn(score[c], a), (double)No);
}

// --------------------------------------------------------------------------------------------------
// K4: global naive shuffle.  rank(c) = number of channels ahead of c in a stable descending sort of the
// mean metric; the channel of rank r goes to group r mod G, slot r div G (neighbours in rank never share
// a group).
// --------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) gns_rank_kernel(int C, const double *__restrict__ mean, int use_gns, int m_group,
                                                       int32_t *__restrict__ theta0, double *__restrict__ sorted_mean) {
    __shared__ double tile[256];
    const int c = blockIdx.x * 256 + threadIdx.x;
    if (!use_gns) {
        if (c < C) theta0[c] = c;
        return;
    }
    const double mine = (c < C) ? mean[c] : 0.0;
    int rank = 0;
    for (int base = 0; base < C; base += 256) {
        __syncthreads();
        if (base + threadIdx.x < C) tile[threadIdx.x] = mean[base + threadIdx.x];
        __syncthreads();
        const int n = min(256, C - base);
        for (int i = 0; i < n; ++i) {
            double other = tile[i];
            rank += (other > mine || (other == mine && base + i < c)) ? 1 : 0;
        }
    }
    if (c < C) {
        const int G = C / m_group;
        theta0[(rank % G) * m_group + rank / G] = c;
        sorted_mean[rank] = mine;
    }
}

// Near-ties of the sort: neighbours in rank whose means differ by less than 1e-6 relative (the order of such a pair
// hangs on the last bits of the score).  counters[2] receives the count.
__global__ void __launch_bounds__(256) gns_near_tie_kernel(int C, const double *__restrict__ sorted_mean,
                                                           unsigned long long *__restrict__ counters) {
    const int r = blockIdx.x * 256 + threadIdx.x;
    unsigned int near = 0;
    if (r + 1 < C) {
        const double a = sorted_mean[r], b = sorted_mean[r + 1];
        near = __dsub_rn(a, b) < __dmul_rn(1e-6, fabs(a)) ? 1u : 0u;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) near += __shfl_xor_sync(0xFFFFFFFFu, near, off);
    if ((threadIdx.x & 31) == 0 && near) atomicAdd(&counters[2], (unsigned long long)near);
}

// --------------------------------------------------------------------------------------------------
// K5: local block shuffle (Algorithm 1 lines 3-14).
// Wt[c][j] = |W[j,c]| bits, channel-major and zero-padded to ldt rows, so a channel's column is contiguous.
// --------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) abs_transpose_kernel(const __half *__restrict__ W, int No, int C, long ldw,
                                                            uint16_t *__restrict__ Wt, long ldt) {
    __shared__ uint16_t tile[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int c_base = blockIdx.x * 32, r_base = blockIdx.y * 32;
    const uint16_t *Wb = reinterpret_cast<const uint16_t *>(W);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int r = r_base + ty + i * 8, c = c_base + tx;
        tile[ty + i * 8][tx] = (r < No && c < C) ? (uint16_t)(Wb[(long)r * ldw + c] & 0x7FFFu) : (uint16_t)0;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int c = c_base + ty + i * 8, r = r_base + tx;
        if (c < C && r < ldt) Wt[(long)c * ldt + r] = tile[tx][ty + i * 8];
    }
}

// Retained metric sum of one group of 4 channels over all rows (Eq. 5 restricted to the group), computed
// by one warp.  Every lane returns the value.
//   kept(j,k): slot k is among the 2 largest xi[j,.] = |w| * s (ties: lower slot)
//   A_k = sum_j kept(j,k) |w_jk| exactly;  V = ((s0*a0 + s1*a1) + s2*a2) + s3*a3
__device__ double group_value_warp(const uint16_t *__restrict__ Wt, long ldt, const double *__restrict__ score,
                                   int c0, int c1, int c2, int c3) {
    const int lane = threadIdx.x & 31;
    const int ch[4] = {c0, c1, c2, c3};
    double sc[4];
    long long A[4] = {0, 0, 0, 0};
#pragma unroll
    for (int k = 0; k < 4; ++k) sc[k] = score[ch[k]];
    for (long j = lane * 8; j < ldt; j += 256) {
        uint4 v[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) v[k] = *reinterpret_cast<const uint4 *>(Wt + (long)ch[k] * ldt + j);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            uint16_t h[4];
            double xi[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                h[k] = reinterpret_cast<const uint16_t *>(&v[k])[e];
                xi[k] = __dmul_rn(half_bits_abs_to_double(h[k]), sc[k]);
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                int ahead = 0;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    if (q == k) continue;
                    ahead += (xi[q] > xi[k] || (xi[q] == xi[k] && q < k)) ? 1 : 0;
                }
                if (ahead < 2) A[k] += half_bits_abs_fixed(h[k]);
            }
        }
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) A[k] += __shfl_xor_sync(0xFFFFFFFFu, A[k], off);
    }
    double t0 = __dmul_rn(sc[0], __dmul_rn(__ll2double_rn(A[0]), 0x1p-24));
    double t1 = __dmul_rn(sc[1], __dmul_rn(__ll2double_rn(A[1]), 0x1p-24));
    double t2 = __dmul_rn(sc[2], __dmul_rn(__ll2double_rn(A[2]), 0x1p-24));
    double t3 = __dmul_rn(sc[3], __dmul_rn(__ll2double_rn(A[3]), 0x1p-24));
    return __dadd_rn(__dadd_rn(__dadd_rn(t0, t1), t2), t3);
}

// --------------------------------------------------------------------------------------------------
// V(group with slot k replaced by candidate x) for all candidates x of a block, without re-ranking four columns
// per row and candidate.  With the three fixed slots ordered f1, f2, f3 by the metric (ties: lower slot), the
// candidate is kept exactly when it is ahead of f2; f1 is always kept, f2 is kept exactly when the candidate is not,
// f3 never.  So per row only f2's slot and |w| matter: phase 1 stores them (4 bytes per row, shared memory) and the
// exact sums B_q of |w_q| over rows where q is f1 or f2; phase 2 (one warp per candidate) needs one multiply and one
// compare per row and candidate:  A_x = sum kept |w_x|,  A_q = B_q - sum [q is f2 and x kept] |w_q|.
// The kept sets, the exact integer sums and the order of the four multiplies and three adds are those of
// group_value_warp, so the values are bit-identical to it.
// --------------------------------------------------------------------------------------------------
__device__ __forceinline__ bool metric_ahead(double xa, int sa, double xb, int sb) { return xa > xb || (xa == xb && sa < sb); }

// Phase 1, whole CTA.  ch[4]: the group's channels; k: the slot to be replaced.  pk[j] = f2 slot << 16 | |w_f2| bits.
// s_B[4] (shared, zeroed by the caller before the preceding barrier) receives B_q.
__device__ void lbs_slot_prepare(const uint16_t *__restrict__ Wt, long ldt, const double *__restrict__ score,
                                 const int (&ch)[4], int k, uint32_t *__restrict__ pk, unsigned long long *s_B) {
    double sc[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) sc[q] = score[ch[q]];
    long long B[4] = {0, 0, 0, 0};
    for (long j = (long)threadIdx.x * 8; j < ldt; j += (long)blockDim.x * 8) {
        uint4 v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q)
            if (q != k) v[q] = *reinterpret_cast<const uint4 *>(Wt + (long)ch[q] * ldt + j);
        uint32_t out[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            uint16_t h[4];
            double xi[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                h[q] = (q != k) ? reinterpret_cast<const uint16_t *>(&v[q])[e] : (uint16_t)0;
                xi[q] = __dmul_rn(half_bits_abs_to_double(h[q]), sc[q]);
            }
            // rank of each fixed slot among the three fixed ones
            int f1 = -1, f2 = -1;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (q == k) continue;
                int ahead = 0;
#pragma unroll
                for (int r = 0; r < 4; ++r)
                    if (r != k && r != q) ahead += metric_ahead(xi[r], r, xi[q], q) ? 1 : 0;
                if (ahead == 0) f1 = q;
                if (ahead == 1) f2 = q;
            }
#pragma unroll
            for (int q = 0; q < 4; ++q)
                if (q == f1 || q == f2) B[q] += half_bits_abs_fixed(h[q]);
            uint16_t hf2 = 0;
#pragma unroll
            for (int q = 0; q < 4; ++q)
                if (q == f2) hf2 = h[q];
            out[e] = ((uint32_t)f2 << 16) | hf2;
        }
        *reinterpret_cast<uint4 *>(pk + j) = make_uint4(out[0], out[1], out[2], out[3]);
        *reinterpret_cast<uint4 *>(pk + j + 4) = make_uint4(out[4], out[5], out[6], out[7]);
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) B[q] += __shfl_xor_sync(0xFFFFFFFFu, B[q], off);
        if ((threadIdx.x & 31) == 0 && B[q]) atomicAdd(&s_B[q], (unsigned long long)B[q]);   // integers: order-free
    }
}

// Phase 2, one warp: the value for candidate channel cx in slot k.  Every lane returns it.
__device__ double lbs_slot_candidate(const uint16_t *__restrict__ Wt, long ldt, const double (&sc_fixed)[4], int k, int cx,
                                     double sx, const uint32_t *__restrict__ pk, const unsigned long long *s_B) {
    const int lane = threadIdx.x & 31;
    // Per-lane sums of |w| are kept as doubles: every term is a multiple of 2^-24 below 2^16 and a lane adds fewer than
    // 2^11 of them, so every partial sum is a multiple of 2^-24 below 2^27 -- 51 bits, exact in fp64 -- and equals the
    // integer sum of group_value_warp once scaled by 2^24.  (One conversion and one predicated add per term instead of the
    // shifts, selects and 64-bit adds of the integer form: this loop is bound by instruction issue.)
    double Ax = 0.0, D0 = 0.0, D1 = 0.0, D2 = 0.0, D3 = 0.0;
    const uint16_t *col = Wt + (long)cx * ldt;
    // The decision "is the candidate ahead of f2" is the fp64 comparison of |w_x| * s_x with |w_f2| * s_f2.  Its fp32 image
    // (exact |w|, scores rounded once, one rounded multiply: each product within 2^-23 relative of its fp64 counterpart)
    // decides it whenever the two products differ by more than 2^-21 of the larger: then the fp64 products differ the same
    // way.  Only the rows that are closer (ties, zero padding) take the fp64 multiplies.
    const float sx32 = (float)sx;
    const float s32[4] = {(float)sc_fixed[0], (float)sc_fixed[1], (float)sc_fixed[2], (float)sc_fixed[3]};
    auto rows8 = [&](const uint4 &vx, long j) {
        const uint4 p0 = *reinterpret_cast<const uint4 *>(pk + j);
        const uint4 p1 = *reinterpret_cast<const uint4 *>(pk + j + 4);
        const uint32_t pkv[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const uint16_t hx = reinterpret_cast<const uint16_t *>(&vx)[e];
            const uint32_t rec = pkv[e];
            const uint16_t hf = (uint16_t)(rec & 0xFFFFu);
            const bool f2_odd = (rec & 0x10000u) != 0, f2_high = (rec & 0x20000u) != 0;
            const float wx = __half2float(__ushort_as_half(hx));           // (hx, hf hold magnitudes: the sign bit is clear)
            const float wf = __half2float(__ushort_as_half(hf));
            const float sf32 = f2_high ? (f2_odd ? s32[3] : s32[2]) : (f2_odd ? s32[1] : s32[0]);
            const float px = wx * sx32, pf = wf * sf32;
            const float big = fmaxf(fabsf(px), fabsf(pf));                 // (scores may be negative when the caller supplies them)
            const float diff = px - pf;
            bool kept = diff > 0.f;
            // undecided in fp32: closer than the margin, or so small that fp32 products lose relative accuracy
            if (!(fabsf(diff) > big * 0x1p-21f && big >= 0x1p-100f)) {
                const int f2 = (int)(rec >> 16);
                const double sf = f2 == 0 ? sc_fixed[0] : f2 == 1 ? sc_fixed[1] : f2 == 2 ? sc_fixed[2] : sc_fixed[3];
                const double xx = __dmul_rn(half_bits_abs_to_double(hx), sx);
                const double xf = __dmul_rn(half_bits_abs_to_double(hf), sf);
                kept = metric_ahead(xx, k, xf, f2);
            }
            if (kept) {
                const double wfd = (double)wf;
                Ax = __dadd_rn(Ax, (double)wx);
                if (f2_high) { if (f2_odd) D3 = __dadd_rn(D3, wfd); else D2 = __dadd_rn(D2, wfd); }
                else { if (f2_odd) D1 = __dadd_rn(D1, wfd); else D0 = __dadd_rn(D0, wfd); }
            }
        }
    };
    // the column comes from L2: four 16-byte loads per lane are in flight before the first is used
    long j = lane * 8;
    for (; j + 3 * 256 < ldt; j += 4 * 256) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = __ldg(reinterpret_cast<const uint4 *>(col + j + u * 256));
#pragma unroll
        for (int u = 0; u < 4; ++u) rows8(v[u], j + u * 256);
    }
    for (; j < ldt; j += 256) rows8(__ldg(reinterpret_cast<const uint4 *>(col + j)), j);
    long long Axi = __double2ll_rn(__dmul_rn(Ax, 0x1p24));                  // exact: see above
    long long D[4] = {__double2ll_rn(__dmul_rn(D0, 0x1p24)), __double2ll_rn(__dmul_rn(D1, 0x1p24)),
                      __double2ll_rn(__dmul_rn(D2, 0x1p24)), __double2ll_rn(__dmul_rn(D3, 0x1p24))};
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        Axi += __shfl_xor_sync(0xFFFFFFFFu, Axi, off);
#pragma unroll
        for (int q = 0; q < 4; ++q) D[q] += __shfl_xor_sync(0xFFFFFFFFu, D[q], off);
    }
    double t[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const long long A = (q == k) ? Axi : (long long)s_B[q] - D[q];
        const double sq = (q == k) ? sx : sc_fixed[q];
        t[q] = __dmul_rn(sq, __dmul_rn(__ll2double_rn(A), 0x1p-24));
    }
    return __dadd_rn(__dadd_rn(__dadd_rn(t[0], t[1]), t[2]), t[3]);
}

// table[b][g][slot][x] = V(group g of block b with its slot replaced by block channel x); base[G] = V(g).
// grid (nblocks * 64 * 4): one CTA per (block, group, slot); block 256 (8 warps); dynamic shared memory ldt * 4 bytes.
__global__ void __launch_bounds__(256, 4) lbs_table_kernel(const uint16_t *__restrict__ Wt, long ldt,
                                                        const double *__restrict__ score,
                                                        const int32_t *__restrict__ theta0, int C, int lbs_block,
                                                        double *__restrict__ table, double *__restrict__ base) {
    extern __shared__ uint32_t s_pk[];
    __shared__ unsigned long long s_B[4];
    const int slot = blockIdx.x & 3;
    const int g = (blockIdx.x >> 2) % kLbsGroups, b = (blockIdx.x >> 2) / kLbsGroups;
    const int p0 = b * lbs_block;
    const int m = min(lbs_block, C - p0);
    if (g * 4 >= m) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int grp[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) grp[k] = theta0[p0 + g * 4 + k];
    if (threadIdx.x < 4) s_B[threadIdx.x] = 0;
    __syncthreads();
    lbs_slot_prepare(Wt, ldt, score, grp, slot, s_pk, s_B);
    __syncthreads();
    double sc[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) sc[k] = score[grp[k]];
    double *tb = table + (((long)b * kLbsGroups + g) * 4 + slot) * kLbsMax;
    for (int x = warp; x < m; x += 8) {
        const int cx = theta0[p0 + x];
        const double v = lbs_slot_candidate(Wt, ldt, sc, slot, cx, score[cx], s_pk, s_B);
        if (lane == 0) tb[x] = v;
    }
    if (slot == 0 && warp == 0) {
        double v = group_value_warp(Wt, ldt, score, grp[0], grp[1], grp[2], grp[3]);
        if (lane == 0) base[p0 / 4 + g] = v;
    }
}

// (Two CTAs per SM, at 64 registers per thread with a few spills: one cluster of eight occupies eight SMs whatever its
// CTAs need, only 15 such clusters fit 148 SMs, and a weight has 32 to 86 blocks -- the second CTA per SM halves the number
// of waves, and the LLaMA-65B-shaped layer's producer went from 3.4 to 2.1 s.)
// One cluster of 8 CTAs per block of positions: repeat { best cross-group swap by table lookup; apply if gain > 0;
// refresh the two touched groups }.  Every CTA takes the same decision from the same table (no exchange needed), then
// refreshes one of the 2 groups x 4 slots of table rows; a cluster barrier publishes the rows before the next
// decision.  grid (nblocks * 8), cluster (8), block 512, dynamic shared memory ldt * 4 bytes.
constexpr int kLbsCluster = 8;
__global__ void __launch_bounds__(512, 2) lbs_greedy_kernel(const uint16_t *__restrict__ Wt, long ldt,
                                                          const double *__restrict__ score,
                                                          const int32_t *__restrict__ theta0, int C, int lbs_block,
                                                          int max_swaps, double *__restrict__ table,
                                                          double *__restrict__ base, int32_t *__restrict__ theta,
                                                          unsigned long long *__restrict__ counters) {
    extern __shared__ uint32_t s_pk[];
    const int b = blockIdx.x / kLbsCluster;
    const int unit = blockIdx.x % kLbsCluster;                  // rank in the cluster: which (group, slot) this CTA refreshes
    const int p0 = b * lbs_block;
    const int m = min(lbs_block, C - p0);
    const int G = m / 4;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    __shared__ int pos2x[kLbsMax];
    __shared__ int chan[kLbsMax];
    __shared__ double s_base[kLbsGroups];
    __shared__ double red_gain[16], red_second[16];
    __shared__ int red_idx[16];
    __shared__ int decision;      // linear pair index i*256+j, or -1 to stop
    __shared__ unsigned long long s_B[4];
    double *tb = table + (long)b * kLbsGroups * 4 * kLbsMax;
    if (tid < m) { pos2x[tid] = tid; chan[tid] = theta0[p0 + tid]; }
    if (tid < G) s_base[tid] = base[p0 / 4 + tid];
    __syncthreads();
    int swaps = 0;
    int near_swaps = 0;                                        // kept by thread 0 only
    for (;;) {
        double best = -INFINITY, second = -INFINITY;           // second: largest gain once one instance of the best is set aside
        int best_e = 0x7FFFFFFF;
        if (max_swaps <= 0 || swaps < max_swaps) {
            for (int e = tid; e < kLbsMax * kLbsMax; e += 512) {
                const int i = e >> 8, j = e & 255;
                if (j <= i || j >= m || (i >> 2) == (j >> 2)) continue;
                const int gi = i >> 2, si = i & 3, gj = j >> 2, sj = j & 3;
                // rows of the table are rewritten by other CTAs of the cluster: read them from L2, never from this SM's L1
                double after = __dadd_rn(__ldcg(&tb[(gi * 4 + si) * kLbsMax + pos2x[j]]), __ldcg(&tb[(gj * 4 + sj) * kLbsMax + pos2x[i]]));
                double gain = __dsub_rn(after, __dadd_rn(s_base[gi], s_base[gj]));
                if (gain > best || (gain == best && e < best_e)) { second = fmax(second, best); best = gain; best_e = e; }
                else second = fmax(second, gain);
            }
        }
        // merging two (best, second) pairs: the larger best wins (ties: smaller pair index), the loser's best competes
        // with both seconds -- the result is the second-largest of the union whatever the order of merging
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            double og = __shfl_xor_sync(0xFFFFFFFFu, best, off);
            double os = __shfl_xor_sync(0xFFFFFFFFu, second, off);
            int oe = __shfl_xor_sync(0xFFFFFFFFu, best_e, off);
            second = fmax(fmax(second, os), fmin(best, og));
            if (og > best || (og == best && oe < best_e)) { best = og; best_e = oe; }
        }
        if (lane == 0) { red_gain[warp] = best; red_second[warp] = second; red_idx[warp] = best_e; }
        __syncthreads();
        if (warp == 0) {
            best = lane < 16 ? red_gain[lane] : -INFINITY;
            second = lane < 16 ? red_second[lane] : -INFINITY;
            best_e = lane < 16 ? red_idx[lane] : 0x7FFFFFFF;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                double og = __shfl_xor_sync(0xFFFFFFFFu, best, off);
                double os = __shfl_xor_sync(0xFFFFFFFFu, second, off);
                int oe = __shfl_xor_sync(0xFFFFFFFFu, best_e, off);
                second = fmax(fmax(second, os), fmin(best, og));
                if (og > best || (og == best && oe < best_e)) { best = og; best_e = oe; }
            }
            if (lane == 0) {
                decision = (best > 0.0) ? best_e : -1;
                // an applied swap whose runner-up is within 1e-6 relative: counted, not acted on
                if (best > 0.0 && second > -INFINITY && __dsub_rn(best, second) < __dmul_rn(1e-6, fabs(best))) ++near_swaps;
            }
        }
        __syncthreads();
        const int d = decision;
        if (d < 0) break;
        const int bi = d >> 8, bj = d & 255;
        if (tid == 0) { int t = pos2x[bi]; pos2x[bi] = pos2x[bj]; pos2x[bj] = t; }
        ++swaps;
        __syncthreads();
        // Refresh.  Row (g, slot) of the table holds the values of group g with that slot replaced by each candidate, so it
        // depends on g's OTHER three channels only: of the eight rows of the two touched groups, the two rows of the swapped
        // slots themselves stay as they are, six need new values.  Their candidates are dealt in quarters, three of the 24
        // quarters to each of the cluster's eight CTAs (a CTA prepares the per-row records of each row it has a share of);
        // units 0 and 4 also recompute the base value of one group each.
        {
            if ((unit == 0 || unit == 4) && warp == 0) {
                const int g = unit == 0 ? (bi >> 2) : (bj >> 2);
                double v = group_value_warp(Wt, ldt, score, chan[pos2x[g * 4]], chan[pos2x[g * 4 + 1]], chan[pos2x[g * 4 + 2]],
                                            chan[pos2x[g * 4 + 3]]);
                if (lane == 0) base[p0 / 4 + g] = v;
            }
            const int quarter_size = (m + 3) >> 2;
            int prepared = -1;
            for (int qq = 3 * unit; qq < 3 * unit + 3; ++qq) {
                const int row = qq >> 2, quarter = qq & 3, which = row / 3;
                int slot = row - 3 * which;                      // the (row mod 3)-th slot other than the swapped one
                if (slot >= ((which ? bj : bi) & 3)) ++slot;
                const int g = (which ? bj : bi) >> 2;
                int ch[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) ch[k] = chan[pos2x[g * 4 + k]];
                double sc[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) sc[k] = score[ch[k]];
                if (row != prepared) {
                    __syncthreads();                             // the previous row's records are no longer being read
                    if (tid < 4) s_B[tid] = 0;
                    __syncthreads();
                    lbs_slot_prepare(Wt, ldt, score, ch, slot, s_pk, s_B);
                    __syncthreads();
                    prepared = row;
                }
                const int x_end = min(m, (quarter + 1) * quarter_size);
                for (int x = quarter * quarter_size + warp; x < x_end; x += 16) {
                    const int cx = chan[x];
                    const double v = lbs_slot_candidate(Wt, ldt, sc, slot, cx, score[cx], s_pk, s_B);
                    if (lane == 0) tb[(g * 4 + slot) * kLbsMax + x] = v;
                }
            }
        }
        __threadfence();
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
        if (tid < 2) {                                          // the two refreshed base values, written by units 0 and 4
            const int g = tid == 0 ? (bi >> 2) : (bj >> 2);
            s_base[g] = *reinterpret_cast<volatile double *>(base + p0 / 4 + g);
        }
        __syncthreads();
    }
    if (unit != 0) return;
    if (tid < m) theta[p0 + tid] = chan[pos2x[tid]];
    if (tid < G) base[p0 / 4 + tid] = s_base[tid];
    if (tid == 0 && swaps) atomicAdd(&counters[1], (unsigned long long)swaps);
    if (tid == 0 && near_swaps) atomicAdd(&counters[3], (unsigned long long)near_swaps);
}

// Sum of the group values in group order (Eq. 5 objective), one thread: deterministic.
__global__ void objective_kernel(int G, const double *__restrict__ base, double *__restrict__ out) {
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        double t = 0.0;
        for (int g = 0; g < G; ++g) t = __dadd_rn(t, base[g]);
        *out = t;
    }
}

// base[g] = V(g) under theta for every group (the objective of an order that the block shuffle does not produce itself).
__global__ void __launch_bounds__(256) group_values_kernel(const uint16_t *__restrict__ Wt, long ldt,
                                                           const double *__restrict__ score,
                                                           const int32_t *__restrict__ theta, int G,
                                                           double *__restrict__ base) {
    const int g = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (g >= G) return;
    int c[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) c[k] = theta ? theta[4 * g + k] : 4 * g + k;      // NULL: the identity order
    double v = group_value_warp(Wt, ldt, score, c[0], c[1], c[2], c[3]);
    if ((threadIdx.x & 31) == 0) base[g] = v;
}

// --------------------------------------------------------------------------------------------------
// K6: 2-of-4 selection + compression.  One CTA per output row: the row is staged in shared memory, then
// each thread handles 8 permuted positions (2 groups): 4 kept values + 1 metadata byte.
// --------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) select_compress_kernel(const __half *__restrict__ W, int No, int C, long ldw,
                                                              const double *__restrict__ score,
                                                              const int32_t *__restrict__ theta,
                                                              __half *__restrict__ vals, uint8_t *__restrict__ meta,
                                                              unsigned long long *__restrict__ counters, int rows_per_cta) {
    // A CTA takes rows_per_cta consecutive output rows into shared memory; a thread then reads the permutation and the
    // scores of its eight positions ONCE and applies them to every one of those rows (with one row per CTA the two gathers
    // were six times the bytes of the row itself).
    extern __shared__ __align__(16) uint16_t s_rows[];                  // [rows_per_cta][C]
    const int j0 = blockIdx.x * rows_per_cta;
    const int nrows = min(rows_per_cta, No - j0);
    const int chunks_per_row = C / 8;
    for (int idx = threadIdx.x; idx < nrows * chunks_per_row; idx += 256) {
        const int r = idx / chunks_per_row, c = (idx - r * chunks_per_row) * 8;
        *reinterpret_cast<uint4 *>(s_rows + (size_t)r * C + c) =
            __ldg(reinterpret_cast<const uint4 *>(reinterpret_cast<const uint16_t *>(W) + (long)(j0 + r) * ldw + c));
    }
    __syncthreads();
    unsigned int near = 0;
    for (int u = threadIdx.x; u < C / 8; u += 256) {
        int ch[8];
        double sc[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) { ch[k] = theta[u * 8 + k]; sc[k] = score[ch[k]]; }
        for (int r = 0; r < nrows; ++r) {
            const uint16_t *s_row = s_rows + (size_t)r * C;
            const long j = j0 + r;
            uint16_t out[4];
            unsigned int byte = 0;
#pragma unroll
            for (int gg = 0; gg < 2; ++gg) {
                uint16_t h[4];
                double xi[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    h[k] = s_row[ch[gg * 4 + k]];
                    xi[k] = __dmul_rn(half_bits_abs_to_double(h[k]), sc[gg * 4 + k]);
                }
                int kept[2], nk = 0;
                double second = 0.0, third = 0.0;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    int ahead = 0;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        if (q == k) continue;
                        ahead += (xi[q] > xi[k] || (xi[q] == xi[k] && q < k)) ? 1 : 0;
                    }
                    if (ahead < 2) { if (nk < 2) kept[nk] = k; ++nk; }
                    if (ahead == 1) second = xi[k];
                    if (ahead == 2) third = xi[k];
                }
                if (__dsub_rn(second, third) < __dmul_rn(1e-6, second)) ++near;
                out[gg * 2 + 0] = h[kept[0]];
                out[gg * 2 + 1] = h[kept[1]];
                byte |= (unsigned int)(kept[0] | (kept[1] << 2)) << (4 * gg);
            }
            uint2 packed;
            packed.x = (unsigned int)out[0] | ((unsigned int)out[1] << 16);
            packed.y = (unsigned int)out[2] | ((unsigned int)out[3] << 16);
            *reinterpret_cast<uint2 *>(reinterpret_cast<uint16_t *>(vals) + j * (C / 2) + u * 4) = packed;
            meta[j * (C / 8) + u] = (uint8_t)byte;
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) near += __shfl_xor_sync(0xFFFFFFFFu, near, off);
    if ((threadIdx.x & 31) == 0 && near) atomicAdd(&counters[0], (unsigned long long)near);
}

// 4-of-8 selection + compression (the 4:8 pattern of the paper's Table 1; no tensor-core form exists for it, so the
// output is plain: 4 kept values per group in position order and one mask byte per group, bit p = position p kept).
// One CTA per output row, one thread per group of 8 permuted positions.
__global__ void __launch_bounds__(256) select_compress_48_kernel(const __half *__restrict__ W, int No, int C, long ldw,
                                                                 const double *__restrict__ score,
                                                                 const int32_t *__restrict__ theta,
                                                                 __half *__restrict__ vals, uint8_t *__restrict__ mask,
                                                                 unsigned long long *__restrict__ counters) {
    extern __shared__ uint16_t s_row[];
    const int j = blockIdx.x;
    const uint16_t *Wr = reinterpret_cast<const uint16_t *>(W) + (long)j * ldw;
    for (int c = threadIdx.x * 8; c < C; c += 256 * 8)
        *reinterpret_cast<uint4 *>(s_row + c) = __ldg(reinterpret_cast<const uint4 *>(Wr + c));
    __syncthreads();
    unsigned int near = 0;
    for (int u = threadIdx.x; u < C / 8; u += 256) {
        uint16_t h[8];
        double xi[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int c = theta[u * 8 + k];
            h[k] = s_row[c];
            xi[k] = __dmul_rn(half_bits_abs_to_double(h[k]), score[c]);
        }
        uint16_t out[4] = {0, 0, 0, 0};
        unsigned int byte = 0;
        int nk = 0;
        double fourth = 0.0, fifth = 0.0;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            int ahead = 0;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                if (q == k) continue;
                ahead += (xi[q] > xi[k] || (xi[q] == xi[k] && q < k)) ? 1 : 0;
            }
            if (ahead < 4) {
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (e == nk) out[e] = h[k];
                ++nk;
                byte |= 1u << k;
            }
            if (ahead == 3) fourth = xi[k];
            if (ahead == 4) fifth = xi[k];
        }
        if (__dsub_rn(fourth, fifth) < __dmul_rn(1e-6, fourth)) ++near;
        uint2 packed;
        packed.x = (unsigned int)out[0] | ((unsigned int)out[1] << 16);
        packed.y = (unsigned int)out[2] | ((unsigned int)out[3] << 16);
        *reinterpret_cast<uint2 *>(reinterpret_cast<uint16_t *>(vals) + (long)j * (C / 2) + u * 4) = packed;
        mask[(long)j * (C / 8) + u] = (uint8_t)byte;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) near += __shfl_xor_sync(0xFFFFFFFFu, near, off);
    if ((threadIdx.x & 31) == 0 && near) atomicAdd(&counters[0], (unsigned long long)near);
}

// --------------------------------------------------------------------------------------------------
// K7: re-tile (vals, meta) into the layout the sparse MMA reads.
// Per (feature tile ft, channel tile kt) 18432 contiguous bytes:
//   [0, 16384)      128 rows x 128 bytes of kept values, 16-byte chunk q of row r stored at chunk q ^ (r & 7)
//                   (the 128-byte swizzle of a K-major shared-memory operand)
//   [16384, 18432)  128 lanes x 4 words; lane l, word c: low half = metadata of row (l&7) + 16*(l>>4), high half =
//                   that row + 8, for channels 32c + 16*((l>>3)&1) .. +16 of the tile (the order in which the
//                   tensor-memory copy lays 16 bytes per lane next to the accumulator lanes)
// --------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) pack_kernel(const __half *__restrict__ vals, const uint8_t *__restrict__ meta,
                                                   int No, int C, uint8_t *__restrict__ packed, int k_tiles) {
    const int kt = blockIdx.x, ft = blockIdx.y;
    uint8_t *tile = packed + ((long)ft * k_tiles + kt) * kTileBytes;
    const uint16_t *v16 = reinterpret_cast<const uint16_t *>(vals);
    const long half_c = C / 2, meta_c = C / 8;
    // values: 128 rows x 8 chunks
    for (int i = threadIdx.x; i < 128 * 8; i += 256) {
        const int r = i >> 3, q = i & 7;
        const long row = (long)ft * 128 + r;
        const long col = (long)kt * 64 + q * 8;      // in kept-value units
        uint4 v = make_uint4(0, 0, 0, 0);
        if (row < No && col + 8 <= half_c && (half_c & 7) == 0) {      // rows of vals are 16-byte aligned
            v = *reinterpret_cast<const uint4 *>(v16 + row * half_c + col);
        } else if (row < No && col < half_c) {
            uint16_t *p = reinterpret_cast<uint16_t *>(&v);
            for (int e = 0; e < 8; ++e) if (col + e < half_c) p[e] = v16[row * half_c + col + e];
        }
        *reinterpret_cast<uint4 *>(tile + r * 128 + ((q ^ (r & 7)) << 4)) = v;
    }
    // metadata: 128 lanes x 4 words
    for (int i = threadIdx.x; i < 128 * 4; i += 256) {
        const int l = i >> 2, c = i & 3;
        const int r_lo = (l & 7) + 16 * (l >> 4);
        const int khalf = (l >> 3) & 1;
        unsigned int word = 0;
#pragma unroll
        for (int hi = 0; hi < 2; ++hi) {
            const long row = (long)ft * 128 + r_lo + 8 * hi;
            const long mb = (long)kt * 16 + c * 4 + khalf * 2;   // metadata byte column
            unsigned int m16 = 0x4444u;                          // padding: legal nibbles, values are zero
            if (row < No) {
                unsigned int b0 = (mb < meta_c) ? meta[row * meta_c + mb] : 0x44u;
                unsigned int b1 = (mb + 1 < meta_c) ? meta[row * meta_c + mb + 1] : 0x44u;
                m16 = b0 | (b1 << 8);
            }
            word |= m16 << (16 * hi);
        }
        reinterpret_cast<unsigned int *>(tile + kTileValBytes)[l * 4 + c] = word;
    }
}

// K11: dense [No, C] in original channel order, zeros where pruned.
__global__ void __launch_bounds__(256) decompress_kernel(const __half *__restrict__ vals, const uint8_t *__restrict__ meta,
                                                         const int32_t *__restrict__ perm, int No, int C,
                                                         __half *__restrict__ out, long ldw) {
    const int j = blockIdx.x;
    const uint16_t *v16 = reinterpret_cast<const uint16_t *>(vals) + (long)j * (C / 2);
    uint16_t *o = reinterpret_cast<uint16_t *>(out) + (long)j * ldw;
    for (int g = threadIdx.x; g < C / 4; g += 256) {
        unsigned int byte = meta[(long)j * (C / 8) + (g >> 1)];
        unsigned int nib = (g & 1) ? (byte >> 4) : (byte & 0xF);
        int i0 = nib & 3, i1 = (nib >> 2) & 3;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            int c = perm ? perm[4 * g + k] : 4 * g + k;
            uint16_t v = 0;
            if (k == i0) v = v16[2 * g];
            if (k == i1) v = v16[2 * g + 1];
            o[c] = v;
        }
    }
}

}  // namespace

// ----------------------------------------------------------------------------------------------------
// Host side
// ----------------------------------------------------------------------------------------------------
static int pick_splits(int rows, int col_blocks, int sm_count) {
    // enough CTAs to fill the machine a few times over, each with a worthwhile slice of rows
    int want = ceil_div(4L * sm_count, col_blocks);
    int max_by_rows = ceil_div(rows, 64);
    int s = want < 1 ? 1 : want;
    if (s > max_by_rows) s = max_by_rows;
    if (s > 1024) s = 1024;
    return s < 1 ? 1 : s;
}

PruneWorkspace carve_prune_workspace(void *ws, int No, int C, int T, const esp_prune_opts &o) {
    PruneWorkspace w{};
    size_t off = 0;
    auto take = [&](size_t bytes) { void *p = ws ? (char *)ws + off : nullptr; off += align_up(bytes, 256); return p; };
    // the split count must not depend on the device so the size query and the call agree
    w.splits = ceil_div(T > 0 ? T : 1, 256);
    if (w.splits > 64) w.splits = 64;
    w.part_sumsq = (double *)take(sizeof(double) * (size_t)w.splits * C);
    w.part_min = (float *)take(sizeof(float) * (size_t)w.splits * C);
    w.part_max = (float *)take(sizeof(float) * (size_t)w.splits * C);
    w.lo = (double *)take(sizeof(double) * C);
    w.hi = (double *)take(sizeof(double) * C);
    w.norm = (double *)take(sizeof(double) * C);
    w.entropy = (double *)take(sizeof(double) * C);
    w.score = (double *)take(sizeof(double) * C);
    w.mean = (double *)take(sizeof(double) * C);
    w.counts = (unsigned int *)take(sizeof(unsigned int) * (size_t)C * o.bins);
    w.colsum = (unsigned long long *)take(sizeof(unsigned long long) * C);
    w.theta0 = (int32_t *)take(sizeof(int32_t) * C);
    w.counters = (unsigned long long *)take(sizeof(unsigned long long) * 8);
    w.objective = (double *)take(sizeof(double) * 4);
    w.sorted_mean = (double *)take(sizeof(double) * C);
    w.ldt = (long)align_up((size_t)No, 256);
    w.wt = (uint16_t *)take(sizeof(uint16_t) * (size_t)C * w.ldt);
    int nblocks = ceil_div(C, o.lbs_block > 0 ? o.lbs_block : kLbsMax);
    w.table = (double *)take(sizeof(double) * (size_t)nblocks * kLbsGroups * 4 * kLbsMax);
    w.base = (double *)take(sizeof(double) * (size_t)(C / 4 + 1));
    w.total_bytes = off;
    return w;
}

esp_status_t launch_pack(const __half *vals, const uint8_t *meta, int No, int C, void *packed, cudaStream_t stream) {
    const int k_tiles = ceil_div(C, kTileK), f_tiles = ceil_div(No, kTileFeat);
    pack_kernel<<<dim3(k_tiles, f_tiles), 256, 0, stream>>>(vals, meta, No, C, (uint8_t *)packed, k_tiles);
    ESP_CUDA_OK(cudaGetLastError());
    return ESP_OK;
}

// ---- streaming calibration: state = sumsq | lo | hi | norm (f64[C] each) | counts u32[C][bins] | chunk partials [64][C]
CalibState carve_calib_state(void *state, int C, int bins) {
    CalibState c{};
    size_t off = 0;
    auto take = [&](size_t bytes) { void *p = state ? (char *)state + off : nullptr; off += align_up(bytes, 256); return p; };
    c.sumsq = (double *)take(sizeof(double) * C);
    c.lo = (double *)take(sizeof(double) * C);
    c.hi = (double *)take(sizeof(double) * C);
    c.norm = (double *)take(sizeof(double) * C);
    c.counts = (unsigned int *)take(sizeof(unsigned int) * (size_t)C * bins);
    c.part_sumsq = (double *)take(sizeof(double) * 64 * (size_t)C);
    c.part_min = (float *)take(sizeof(float) * 64 * (size_t)C);
    c.part_max = (float *)take(sizeof(float) * 64 * (size_t)C);
    c.total_bytes = off;
    return c;
}

esp_status_t launch_calib_reset(const CalibState &c, int C, int bins, cudaStream_t stream) {
    const long n = (long)C * bins;
    calib_reset_kernel<<<ceil_div(n, 256), 256, 0, stream>>>(C, bins, c.sumsq, c.lo, c.hi, c.counts);
    ESP_CUDA_OK(cudaGetLastError());
    return ESP_OK;
}

esp_status_t launch_calib_range(const CalibState &c, const __half *X, int T, int C, long ldx, cudaStream_t stream) {
    int splits = ceil_div(T, 256);
    if (splits > 64) splits = 64;
    colstats_kernel<<<dim3(ceil_div(C, 256), splits), 256, kColSmem, stream>>>(X, T, C, ldx, ceil_div(T, splits), c.part_sumsq, c.part_min,
                                                                       c.part_max);
    calib_merge_kernel<<<ceil_div(C, 256), 256, 0, stream>>>(C, splits, c.part_sumsq, c.part_min, c.part_max, c.sumsq, c.lo, c.hi);
    ESP_CUDA_OK(cudaGetLastError());
    return ESP_OK;
}

esp_status_t launch_calib_histogram(const CalibState &c, const __half *X, int T, int C, long ldx, int bins, cudaStream_t stream) {
    DeviceInfo di;
    esp_status_t st = device_info(&di);
    if (st != ESP_OK) return st;
    const int hsplits = pick_splits(T, ceil_div(C, 64), di.sm_count);
    if (launch_histogram(X, T, C, ldx, hsplits, bins, c.lo, c.hi, c.counts, stream) != ESP_OK) return ESP_ERR_CUDA;
    ESP_CUDA_OK(cudaGetLastError());
    return ESP_OK;
}

esp_status_t launch_calib_finish(const CalibState &c, int C, int bins, long long T_total, const esp_prune_opts &o, double *chan_norm,
                                 double *chan_entropy, double *chan_score, cudaStream_t stream) {
    calib_norm_kernel<<<ceil_div(C, 256), 256, 0, stream>>>(C, c.sumsq, c.norm);
    // entropy needs a scratch output even when the caller does not want it: the chunk partials are free by now
    double *entropy = chan_entropy ? chan_entropy : c.part_sumsq;
    entropy_score_kernel<<<ceil_div(C, 256), 256, 0, stream>>>(C, (int)T_total, bins, c.counts, c.norm, o.alpha, o.use_entropy,
                                                               o.use_norm, nullptr, entropy, chan_score);
    ESP_CUDA_OK(cudaGetLastError());
    if (chan_norm) ESP_CUDA_OK(cudaMemcpyAsync(chan_norm, c.norm, sizeof(double) * C, cudaMemcpyDeviceToDevice, stream));
    return ESP_OK;
}

esp_status_t launch_decompress(const __half *vals, const uint8_t *meta, const int32_t *perm, int No, int C,
                               __half *out, long ldw, cudaStream_t stream) {
    decompress_kernel<<<No, 256, 0, stream>>>(vals, meta, perm, No, C, out, ldw);
    ESP_CUDA_OK(cudaGetLastError());
    return ESP_OK;
}

esp_status_t launch_prune(const __half *W, int No, int C, long ldw, const __half *Xcal, int T, long ldx,
                          const esp_prune_opts &o, __half *vals, uint8_t *meta, int32_t *perm, void *packed,
                          double *chan_norm, double *chan_entropy, double *chan_score, esp_prune_stats *stats,
                          PruneWorkspace &w, cudaStream_t stream) {
    DeviceInfo di;
    esp_status_t st = device_info(&di);
    if (st != ESP_OK) return st;
    const int cthreads = 256;
    const int cblocks = ceil_div(C, cthreads);
    ESP_CUDA_OK(cudaMemsetAsync(w.counters, 0, sizeof(unsigned long long) * 8, stream));
    ESP_CUDA_OK(cudaMemsetAsync(w.objective, 0, sizeof(double) * 4, stream));

    const bool need_stats_pass = (o.score_override == nullptr) || chan_norm || chan_entropy;
    if (need_stats_pass && Xcal) {
        // K1
        const int rows1 = ceil_div(T, w.splits);
        colstats_kernel<<<dim3(ceil_div(C, 256), w.splits), 256, kColSmem, stream>>>(Xcal, T, C, ldx, rows1, w.part_sumsq,
                                                                             w.part_min, w.part_max);
        colstats_finish_kernel<<<cblocks, cthreads, 0, stream>>>(C, w.splits, w.part_sumsq, w.part_min, w.part_max,
                                                                 w.norm, w.lo, w.hi);
        if (o.global_bin_range) global_range_kernel<<<1, 1024, 0, stream>>>(C, w.lo, w.hi);
        // K2
        ESP_CUDA_OK(cudaMemsetAsync(w.counts, 0, sizeof(unsigned int) * (size_t)C * o.bins, stream));
        const int hsplits = pick_splits(T, ceil_div(C, 64), di.sm_count);
        if (launch_histogram(Xcal, T, C, ldx, hsplits, o.bins, w.lo, w.hi, w.counts, stream) != ESP_OK) return ESP_ERR_CUDA;
        entropy_score_kernel<<<cblocks, cthreads, 0, stream>>>(C, T, o.bins, w.counts, w.norm, o.alpha, o.use_entropy,
                                                               o.use_norm, o.score_override, w.entropy, w.score);
    } else {
        entropy_score_kernel<<<cblocks, cthreads, 0, stream>>>(C, T, o.bins, nullptr, w.norm, o.alpha, o.use_entropy,
                                                               o.use_norm, o.score_override, w.entropy, w.score);
    }
    ESP_CUDA_OK(cudaGetLastError());
    if (chan_norm) ESP_CUDA_OK(cudaMemcpyAsync(chan_norm, w.norm, sizeof(double) * C, cudaMemcpyDeviceToDevice, stream));
    if (chan_entropy) ESP_CUDA_OK(cudaMemcpyAsync(chan_entropy, w.entropy, sizeof(double) * C, cudaMemcpyDeviceToDevice, stream));
    if (chan_score) ESP_CUDA_OK(cudaMemcpyAsync(chan_score, w.score, sizeof(double) * C, cudaMemcpyDeviceToDevice, stream));

    // K3 + K4
    if (o.use_gns && !o.perm_override) {
        ESP_CUDA_OK(cudaMemsetAsync(w.colsum, 0, sizeof(unsigned long long) * C, stream));
        const int wsplits = pick_splits(No, ceil_div(C, 256), di.sm_count);
        colabs_kernel<<<dim3(ceil_div(C, 256), wsplits), 256, 0, stream>>>(W, No, C, ldw, ceil_div(No, wsplits), w.colsum);
        mean_metric_kernel<<<cblocks, cthreads, 0, stream>>>(C, No, w.colsum, w.score, w.mean);
    }
    int32_t *theta0 = (o.use_lbs || stats) ? w.theta0 : perm;
    if (o.perm_override)
        ESP_CUDA_OK(cudaMemcpyAsync(theta0, o.perm_override, sizeof(int32_t) * C, cudaMemcpyDeviceToDevice, stream));
    else {
        gns_rank_kernel<<<ceil_div(C, 256), 256, 0, stream>>>(C, w.mean, o.use_gns, o.m_group, theta0, w.sorted_mean);
        if (o.use_gns && stats) gns_near_tie_kernel<<<ceil_div(C, 256), 256, 0, stream>>>(C, w.sorted_mean, w.counters);
    }
    ESP_CUDA_OK(cudaGetLastError());

    // K5
    const int G = C / 4;
    if (o.use_lbs || stats) {
        abs_transpose_kernel<<<dim3(ceil_div(C, 32), ceil_div(w.ldt, 32)), 256, 0, stream>>>(W, No, C, ldw, w.wt, w.ldt);
    }
    if (stats) {                             // Eq. 5 under the identity order (w.base is rewritten below)
        group_values_kernel<<<ceil_div(G, 8), 256, 0, stream>>>(w.wt, w.ldt, w.score, nullptr, G, w.base);
        objective_kernel<<<1, 32, 0, stream>>>(G, w.base, w.objective + 2);
    }
    if (o.use_lbs) {
        const int nblocks = ceil_div(C, o.lbs_block);
        const size_t pk_smem = (size_t)w.ldt * sizeof(uint32_t);          // per-row f2 record of one (group, slot)
        if (pk_smem > (size_t)di.max_smem_optin - 8192) return ESP_ERR_UNSUPPORTED;   // No beyond ~56000 rows
        ESP_CUDA_OK(cudaFuncSetAttribute(lbs_table_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pk_smem));
        ESP_CUDA_OK(cudaFuncSetAttribute(lbs_greedy_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pk_smem));
        lbs_table_kernel<<<nblocks * kLbsGroups * 4, 256, pk_smem, stream>>>(w.wt, w.ldt, w.score, w.theta0, C, o.lbs_block,
                                                                            w.table, w.base);
        if (stats) objective_kernel<<<1, 32, 0, stream>>>(G, w.base, w.objective);
        {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(nblocks * kLbsCluster);
            cfg.blockDim = dim3(512);
            cfg.dynamicSmemBytes = pk_smem;
            cfg.stream = stream;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = kLbsCluster;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            ESP_CUDA_OK(cudaLaunchKernelEx(&cfg, lbs_greedy_kernel, (const uint16_t *)w.wt, w.ldt, (const double *)w.score,
                                           (const int32_t *)w.theta0, C, o.lbs_block, o.lbs_max_swaps, w.table, w.base, perm,
                                           w.counters));
        }
        if (stats) objective_kernel<<<1, 32, 0, stream>>>(G, w.base, w.objective + 1);
    } else if (stats) {
        group_values_kernel<<<ceil_div(G, 8), 256, 0, stream>>>(w.wt, w.ldt, w.score, w.theta0, G, w.base);
        objective_kernel<<<1, 32, 0, stream>>>(G, w.base, w.objective);
        ESP_CUDA_OK(cudaMemcpyAsync(w.objective + 1, w.objective, sizeof(double), cudaMemcpyDeviceToDevice, stream));
        ESP_CUDA_OK(cudaMemcpyAsync(perm, w.theta0, sizeof(int32_t) * C, cudaMemcpyDeviceToDevice, stream));
    }
    ESP_CUDA_OK(cudaGetLastError());

    // K6 + K7
    const size_t row_smem = sizeof(uint16_t) * (size_t)C;
    // rows per CTA of the 2:4 kernel: as many as fit about 96 KB of shared memory (two CTAs per SM), eight at most
    // (and no more than leave the grid two CTAs per SM)
    int sel_rows = (int)std::max<size_t>(1, std::min<size_t>(8, (96 * 1024) / row_smem));
    sel_rows = std::max(1, std::min(sel_rows, No / (2 * std::max(1, di.sm_count))));
    ESP_CUDA_OK(cudaFuncSetAttribute(select_compress_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(row_smem * sel_rows)));
    if (o.m_group == 8) {
        ESP_CUDA_OK(cudaFuncSetAttribute(select_compress_48_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)row_smem));
        select_compress_48_kernel<<<No, 256, row_smem, stream>>>(W, No, C, ldw, w.score, perm, vals, meta, w.counters);
    } else
        select_compress_kernel<<<ceil_div(No, sel_rows), 256, row_smem * sel_rows, stream>>>(W, No, C, ldw, w.score, perm, vals, meta,
                                                                                             w.counters, sel_rows);
    ESP_CUDA_OK(cudaGetLastError());
    if (packed) {
        st = launch_pack(vals, meta, No, C, packed, stream);
        if (st != ESP_OK) return st;
    }
    if (stats) {
        unsigned long long h_counters[8];
        double h_obj[4];
        ESP_CUDA_OK(cudaMemcpyAsync(h_counters, w.counters, sizeof(h_counters), cudaMemcpyDeviceToHost, stream));
        ESP_CUDA_OK(cudaMemcpyAsync(h_obj, w.objective, sizeof(h_obj), cudaMemcpyDeviceToHost, stream));
        ESP_CUDA_OK(cudaStreamSynchronize(stream));
        stats->near_tie_groups = (long long)h_counters[0];
        stats->near_tie_sort = (long long)h_counters[2];
        stats->near_tie_swaps = (long long)h_counters[3];
        stats->lbs_swaps_total = (long long)h_counters[1];
        stats->obj_identity = h_obj[2];
        stats->obj_after_gns = h_obj[0];
        stats->obj_after_lbs = h_obj[1];
    }
    return ESP_OK;
}

}  // namespace esp
