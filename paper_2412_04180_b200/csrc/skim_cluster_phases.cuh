// Device code shared by the row-clustering kernels (SKIM Algorithm 3; objective of Section 3.2,
// diagonal form): order-preserving keys, the phases the sort kernels run once a row is sorted
// (distinct-value count, group index, binary64 block prefix sums, the row record), and the one-warp
// Lloyd iteration with the error table entry and the optional labels that the Lloyd kernel runs on
// a row record.  Used by skim_cluster.cu, skim_cluster16.cu and skim_lloyd.cu.
#pragma once

#include "skim_internal.cuh"

namespace skimk {

template <typename KeyT> struct KeyOps;

// Order-preserving image of a binary32 value (the scaled path).
template <> struct KeyOps<uint32_t> {
    static constexpr uint32_t PAD = 0xffffffffu;
    __device__ static __forceinline__ uint32_t from_float(float x)
    {
        uint32_t u = __float_as_uint(x);
        return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    }
    __device__ static __forceinline__ float to_float(uint32_t k)
    {
        return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
    }
    // key of the largest representable value <= t
    __device__ static __forceinline__ uint32_t floor_key(float t) { return from_float(t); }
    // eight consecutive keys from a 16-byte aligned address
    __device__ static __forceinline__ void load8(const uint32_t *p, uint32_t *k)
    {
        const uint4 a = *reinterpret_cast<const uint4 *>(p), b = *reinterpret_cast<const uint4 *>(p + 4);
        k[0] = a.x; k[1] = a.y; k[2] = a.z; k[3] = a.w;
        k[4] = b.x; k[5] = b.y; k[6] = b.z; k[7] = b.w;
    }
};

// Order-preserving image of a binary16 bit pattern (no scale installed).
template <> struct KeyOps<uint16_t> {
    static constexpr uint16_t PAD = 0xffffu;
    __device__ static __forceinline__ uint16_t from_half_bits(uint16_t h)
    {
        return (h & 0x8000u) ? (uint16_t)~h : (uint16_t)(h | 0x8000u);
    }
    __device__ static __forceinline__ float to_float(uint16_t k)
    {
        uint16_t h = (k & 0x8000u) ? (uint16_t)(k & 0x7fffu) : (uint16_t)~k;
        return __half2float(__ushort_as_half(h));
    }
    __device__ static __forceinline__ uint16_t floor_key(float t)
    {
        uint16_t h = __half_as_ushort(__float2half_rd(t));
        if (h == 0x8000u) h = 0;
        return from_half_bits(h);
    }
    __device__ static __forceinline__ void load8(const uint16_t *p, uint16_t *k)
    {
        const uint4 a = *reinterpret_cast<const uint4 *>(p);
        const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            k[2 * u] = (uint16_t)(w[u] & 0xffffu);
            k[2 * u + 1] = (uint16_t)(w[u] >> 16);
        }
    }
};

struct ClusterArgs {
    const uint16_t *W;
    const float *G;
    const float *rscale;      // nullptr: no scale installed
    const uint8_t *row_bits;  // nullptr: every width
    int64_t rows;
    int64_t ld;
    int m;                    // cols
    int nb, bmin, sumk;
    int iters;
    float *centroids;
    uint8_t *codes;
    float *err;
    unsigned long long *status;
    unsigned char *scratch;   // row records of the current chunk (written by the sort kernel, read by the Lloyd kernel)
    long long rec_stride;     // bytes between row records
    int64_t row0;             // first row of the current chunk
    int rec_half;             // the records are in the compact format of the fp16-key sort kernel
    int early_exit;           // stop a row once no boundary moved
    unsigned long long *iter_stats;   // nullptr, or two counters: iterations run, rows counted
};

// Row record: what the sort kernel leaves in global memory for the Lloyd kernel.  All offsets are
// multiples of 16 bytes; values are binary32 whatever key type sorted the row.
//   hdr     int nd (number of distinct values) at byte 0; float dvals[16] at byte 64
//   seg     one 32-byte entry per segment of 32 groups (256 elements): the binary64 sums of g,
//           g*x and g*x^2 over all earlier segments; entry nseg holds the row totals
//   groups  one 96-byte record per group of 8 sorted elements, three whole 32-byte sectors: the 8
//           values | the 8 importances | the binary64 sums of g, g*x and g*x^2 from the start of
//           the group's segment to the group's first element (and 8 bytes of padding).  With the
//           segment entry that is everything a boundary needs in one Lloyd iteration.  The last
//           group is padded with the largest finite value and zero importance.  Every sector is
//           written by one 32-byte store and never touched again.
//   gi      group index: first value of every group, sk_entries(m) floats (padded likewise)
struct RowRecord {
    size_t seg, groups, gi, total;
    size_t gi_bytes;
    int ngrp, nseg;
};
constexpr int SKIM_GROUP_BYTES = 96;                // three 32-byte sectors
// Compact record of the fp16-key sort kernel (no scale installed, so a value IS a binary16 number): a group is
// two sectors, 8 binary16 values | the binary64 sums of g and g*x from the segment start | the 8 importances.
// The g*x^2 sums are not kept per group: the error of a width is  sum g x^2 (row total, last segment entry)
// minus  sum_j c_j (2 S1_j - c_j S0_j),  which needs the interval sums of g and g*x only.
constexpr int SKIM_GROUP_BYTES_HALF = 64;
constexpr unsigned short SKIM_PAD_HALF = 0x7bffu;   // largest finite binary16
constexpr int SKIM_SEG_SHIFT = 5;                   // a segment is 32 groups (256 elements): one group per lane of a warp
constexpr float SKIM_PAD_VALUE = 3.402823466e38f;   // largest finite binary32: 0 * padding stays 0

__host__ __device__ inline int sk_entries(int m) { return ((((m + 7) >> 3) + 7) & ~7) + 16; }

__host__ __device__ inline RowRecord row_record(int m, bool half_groups = false)
{
    RowRecord R;
    R.ngrp = (m + 7) >> 3;
    R.nseg = (R.ngrp + (1 << SKIM_SEG_SHIFT) - 1) >> SKIM_SEG_SHIFT;
    R.gi_bytes = (size_t)sk_entries(m) * 4;
    size_t off = 128;
    R.seg = off; off += (size_t)(R.nseg + 1) * 32;
    R.groups = off; off += (size_t)R.ngrp * (half_groups ? SKIM_GROUP_BYTES_HALF : SKIM_GROUP_BYTES);
    R.gi = off; off += R.gi_bytes;
    R.total = (off + 127) & ~(size_t)127;
    return R;
}

// Copies `bytes` (a multiple of 16, both pointers 16-byte aligned) with all threads of the block.
template <int THREADS>
__device__ __forceinline__ void copy16(void *dst, const void *src, size_t bytes)
{
    uint4 *d = reinterpret_cast<uint4 *>(dst);
    const uint4 *s = reinterpret_cast<const uint4 *>(src);
    for (size_t i = threadIdx.x; i < bytes / 16; i += THREADS) d[i] = s[i];
}

// One 32-byte store to a 32-byte aligned global address (a whole sector in one instruction).
__device__ __forceinline__ void st_sector(void *p, const float *v)
{
    asm volatile("st.global.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "f"(v[0]), "f"(v[1]), "f"(v[2]),
                 "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7])
                 : "memory");
}
__device__ __forceinline__ void st_sector(void *p, double a, double b, double c)
{
    asm volatile("st.global.v4.f64 [%0], {%1, %2, %3, %4};" ::"l"(p), "d"(a), "d"(b), "d"(c), "d"(0.0) : "memory");
}

// The sorted row as the record pass sees it.  A source gives the keys and importances of one group
// of 8 sorted elements (positions e .. e+7; the caller masks positions >= m), returns the OR of the
// bit patterns of those importances if it has not validated them (else 0), and gives single keys.
// This one: keys and importance in two shared-memory arrays, padded to whole groups.
template <typename KeyT> struct SortedArrays {
    const KeyT *skeys;
    const float *sg;
    __device__ __forceinline__ unsigned group(int e, int, KeyT *ks, float *gs) const
    {
        KeyOps<KeyT>::load8(skeys + e, ks);
        const float4 ga = *reinterpret_cast<const float4 *>(sg + e), gb = *reinterpret_cast<const float4 *>(sg + e + 4);
        gs[0] = ga.x; gs[1] = ga.y; gs[2] = ga.z; gs[3] = ga.w;
        gs[4] = gb.x; gs[5] = gb.y; gs[6] = gb.z; gs[7] = gb.w;
        return 0u;
    }
    __device__ __forceinline__ KeyT key_at(int p) const { return skeys[p]; }
};

// Small per-block scratch of the phases below.
struct PhaseSmem {
    double segtot[96][3];   // sums of every segment (rows of up to 24 576 elements have 96 segments of 32 groups)
    double wsum2[32];       // compact record: every warp's sum of g*x^2
    float tfs[32];     // scratch of collect_distinct
    float dvals[32];   // the row's distinct values when there are at most 16
    int misc[4];       // [0] distinct count, [1] slot counter
};

// Rare path: the row has nd <= 16 distinct values; stores them ascending in ps.dvals.
template <typename KeyT, int THREADS, typename Src>
__device__ __forceinline__ void collect_distinct(const Src &src, int m, int nd, PhaseSmem &ps)
{
    for (int p = threadIdx.x; p < m; p += THREADS) {
        if (p == 0 || src.key_at(p) != src.key_at(p - 1)) {
            const int slot = atomicAdd(&ps.misc[1], 1);
            if (slot >= 0 && slot < 16) ps.tfs[slot] = __int_as_float(p);
        }
    }
    __syncthreads();
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        const int p = lane < nd ? __float_as_int(ps.tfs[lane]) : 0x7fffffff;
        int rank = 0;
        for (int u = 0; u < nd; ++u) rank += (__shfl_sync(0xffffffffu, p, u) < p) ? 1 : 0;
        __syncwarp();
        if (lane < nd && SKIM_IDX(rank, 32, nullptr) && SKIM_IDX(p, m, nullptr)) ps.dvals[rank] = KeyOps<KeyT>::to_float(src.key_at(p));
    }
    __syncthreads();
}

// Writes the row record from the sorted row (a source, see above; padded to whole groups: largest
// key / zero importance).  One pass: a lane takes 2^(SKIM_SEG_SHIFT - 5) adjacent groups of 8 elements (one, as measured best), decodes them,
// stores their values and importances, sums g, g*x, g*x^2 in binary64 (pairwise); one warp scan over
// the lanes' totals turns the group sums of a segment into prefix sums, which complete the
// group records in global memory.  Segments are independent, so no warp waits for another.
// Afterwards one warp turns the segment sums into the segment table.  Call with all threads.
// COUNT: the pass also counts the row's distinct values (ps.misc[0..1] zeroed before, and synced)
// and returns the count; otherwise the caller passes the count (any number above 16 stands for
// "more than 16") in nd_known.
template <typename KeyT, int THREADS, bool COUNT, typename Src>
__device__ __forceinline__ int write_row_record(const ClusterArgs &a, const Src &src, PhaseSmem &ps, int nd_known,
                                                int local_row)
{
    constexpr int NW = THREADS / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int m = a.m;
    const RowRecord R = row_record(m);
    unsigned char *rec = a.scratch + (size_t)local_row * (size_t)a.rec_stride;     // local_row: the row's index inside the chunk
    float *gi = reinterpret_cast<float *>(rec + R.gi);
    int distinct = 0;
    unsigned bad = 0u;
    for (int sgm = warp; sgm < R.nseg; sgm += NW) {
        constexpr int GPL = 1 << (SKIM_SEG_SHIFT - 5);        // groups per lane
        const int q0 = (sgm << SKIM_SEG_SHIFT) + GPL * lane;
        double a0 = 0.0, a1 = 0.0, a2 = 0.0;       // sums of the lane's first group
        double w0 = 0.0, w1 = 0.0, w2 = 0.0;       // sums of both
        float first[2] = {0.0f, 0.0f};
#pragma unroll
        for (int h = 0; h < GPL; ++h) {
            const int q = q0 + h;
            if (q < R.ngrp) {
                const int e = q << 3;
                KeyT ks[8];
                float gs[8], x[8];
                const unsigned gbits = src.group(e, m, ks, gs);
                KeyT prev = (COUNT && e > 0) ? src.key_at(e - 1) : (KeyT)0;
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const bool real = e + u < m;
                    x[u] = real ? KeyOps<KeyT>::to_float(ks[u]) : SKIM_PAD_VALUE;
                    if (COUNT) {
                        distinct += (real && (e + u == 0 || ks[u] != prev)) ? 1 : 0;
                        prev = ks[u];
                    }
                }
                unsigned char *gr = rec + R.groups + (size_t)q * SKIM_GROUP_BYTES;
                st_sector(gr, x);
                st_sector(gr + 32, gs);
                first[h] = x[0];
                double t0[8], t1[8], t2[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const double g = (double)gs[u], xd = (double)x[u];      // padding: g = 0, x finite
                    t0[u] = g;
                    t1[u] = g * xd;
                    t2[u] = t1[u] * xd;
                }
                const double v0 = ((t0[0] + t0[1]) + (t0[2] + t0[3])) + ((t0[4] + t0[5]) + (t0[6] + t0[7]));
                const double v1 = ((t1[0] + t1[1]) + (t1[2] + t1[3])) + ((t1[4] + t1[5]) + (t1[6] + t1[7]));
                const double v2 = ((t2[0] + t2[1]) + (t2[2] + t2[3])) + ((t2[4] + t2[5]) + (t2[6] + t2[7]));
                // importance the source has not validated: a sign bit or a non-finite sum asks for a closer look
                if ((gbits >> 31) || !(v0 < 1.0e300)) {
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        if (!(gs[u] >= 0.0f) || gs[u] > 3.0e38f) bad |= 2u;
                }
                if (h == 0) { a0 = v0; a1 = v1; a2 = v2; }
                w0 += v0; w1 += v1; w2 += v2;
            }
        }
        double i0 = w0, i1 = w1, i2 = w2;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const double u0 = __shfl_up_sync(0xffffffffu, i0, off);
            const double u1 = __shfl_up_sync(0xffffffffu, i1, off);
            const double u2 = __shfl_up_sync(0xffffffffu, i2, off);
            if (lane >= off) { i0 += u0; i1 += u1; i2 += u2; }
        }
        if (lane == 31 && SKIM_IDX(sgm, 96, a.status)) { ps.segtot[sgm][0] = i0; ps.segtot[sgm][1] = i1; ps.segtot[sgm][2] = i2; }
        // sums from the segment start to the lane's first group: the neighbour's inclusive value itself,
        // not inclusive minus own (which would add a rounding error of its own to every prefix)
        double e0 = __shfl_up_sync(0xffffffffu, i0, 1), e1 = __shfl_up_sync(0xffffffffu, i1, 1),
               e2 = __shfl_up_sync(0xffffffffu, i2, 1);
        if (lane == 0) { e0 = 0.0; e1 = 0.0; e2 = 0.0; }
#pragma unroll
        for (int h = 0; h < GPL; ++h) {
            const int q = q0 + h;
            if (q < R.ngrp) {
                st_sector(rec + R.groups + (size_t)q * SKIM_GROUP_BYTES + 64, e0, e1, e2);
            }
            e0 += a0; e1 += a1; e2 += a2;
        }
        // the two groups' entries of the group index, as one store (q0 is even)
        if (GPL == 2 && q0 + 1 < R.ngrp) *reinterpret_cast<float2 *>(gi + q0) = make_float2(first[0], first[1]);
        else if (q0 < R.ngrp) gi[q0] = first[0];
    }
    if (bad) atomicOr(a.status, (unsigned long long)bad);
    for (int q = R.ngrp + threadIdx.x; q < sk_entries(m); q += THREADS) gi[q] = SKIM_PAD_VALUE;
    int nd = nd_known;
    if (COUNT) {
#pragma unroll
        for (int off = 16; off; off >>= 1) distinct += __shfl_xor_sync(0xffffffffu, distinct, off);
        if (lane == 0 && distinct) atomicAdd(&ps.misc[0], distinct);
    }
    __syncthreads();
    if (COUNT) nd = ps.misc[0];
    if (warp == 0) {
        // segment table: sums over all earlier segments (4 entries per lane cover the 49 possible)
        double run0 = 0.0, run1 = 0.0, run2 = 0.0, loc[4][3];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int sgm = lane * 4 + u;
#pragma unroll
            for (int c = 0; c < 3; ++c) loc[u][c] = sgm < R.nseg ? ps.segtot[sgm][c] : 0.0;
            run0 += loc[u][0]; run1 += loc[u][1]; run2 += loc[u][2];
        }
        double i0 = run0, i1 = run1, i2 = run2;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const double u0 = __shfl_up_sync(0xffffffffu, i0, off);
            const double u1 = __shfl_up_sync(0xffffffffu, i1, off);
            const double u2 = __shfl_up_sync(0xffffffffu, i2, off);
            if (lane >= off) { i0 += u0; i1 += u1; i2 += u2; }
        }
        double b0 = __shfl_up_sync(0xffffffffu, i0, 1), b1 = __shfl_up_sync(0xffffffffu, i1, 1),
               b2 = __shfl_up_sync(0xffffffffu, i2, 1);
        if (lane == 0) { b0 = 0.0; b1 = 0.0; b2 = 0.0; }
        double4 *seg = reinterpret_cast<double4 *>(rec + R.seg);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int sgm = lane * 4 + u;
            if (sgm <= R.nseg) seg[sgm] = make_double4(b0, b1, b2, 0.0);   // entry nseg: the row totals
            b0 += loc[u][0]; b1 += loc[u][1]; b2 += loc[u][2];
        }
        if (lane == 0) *reinterpret_cast<int *>(rec) = nd;
    }
    return nd;
}

// One 32-byte store of four 64-bit words.
__device__ __forceinline__ void st_sector(void *p, unsigned long long a, unsigned long long b, unsigned long long c, unsigned long long d)
{
    asm volatile("st.global.v4.b64 [%0], {%1, %2, %3, %4};" ::"l"(p), "l"(a), "l"(b), "l"(c), "l"(d) : "memory");
}

// The compact row record (see SKIM_GROUP_BYTES_HALF) from a row sorted by 16-bit keys; the counterpart of
// write_row_record for the fp16-key sort kernel.  One pass, one group per lane; only the sums of g and g*x are
// scanned, the g*x^2 terms are added up per warp and meet in the row total.  nd: the distinct-value count
// (any number above 16 stands for "more than 16").  Call with all threads.
template <int THREADS, typename Src>
__device__ __forceinline__ void write_row_record_half(const ClusterArgs &a, const Src &src, PhaseSmem &ps, int nd, int local_row)
{
    constexpr int NW = THREADS / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int m = a.m;
    const RowRecord R = row_record(m, true);
    unsigned char *rec = a.scratch + (size_t)local_row * (size_t)a.rec_stride;
    float *gi = reinterpret_cast<float *>(rec + R.gi);
    unsigned bad = 0u;
    double w2acc = 0.0;
    for (int sgm = warp; sgm < R.nseg; sgm += NW) {
        const int q = (sgm << SKIM_SEG_SHIFT) + lane;
        double v0 = 0.0, v1 = 0.0;
        unsigned long long xq0 = 0ull, xq1 = 0ull;
        float first = 0.0f;
        if (q < R.ngrp) {
            const int e = q << 3;
            uint16_t ks[8];
            float gs[8];
            const unsigned gbits = src.group(e, m, ks, gs);
            uint32_t hb[8];
            double xd[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const uint16_t k = ks[u];
                const uint16_t h = (e + u < m) ? ((k & 0x8000u) ? (uint16_t)(k & 0x7fffu) : (uint16_t)~k) : (uint16_t)SKIM_PAD_HALF;
                hb[u] = h;
                xd[u] = (double)__half2float(__ushort_as_half(h));
            }
            xq0 = (unsigned long long)(hb[0] | (hb[1] << 16)) | ((unsigned long long)(hb[2] | (hb[3] << 16)) << 32);
            xq1 = (unsigned long long)(hb[4] | (hb[5] << 16)) | ((unsigned long long)(hb[6] | (hb[7] << 16)) << 32);
            first = (float)xd[0];
            st_sector(rec + R.groups + (size_t)q * SKIM_GROUP_BYTES_HALF + 32, gs);
            double t0[8], t1[8], t2[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const double g = (double)gs[u];                       // padding: g = 0, x finite
                t0[u] = g;
                t1[u] = g * xd[u];
                t2[u] = t1[u] * xd[u];
            }
            v0 = ((t0[0] + t0[1]) + (t0[2] + t0[3])) + ((t0[4] + t0[5]) + (t0[6] + t0[7]));
            v1 = ((t1[0] + t1[1]) + (t1[2] + t1[3])) + ((t1[4] + t1[5]) + (t1[6] + t1[7]));
            w2acc += ((t2[0] + t2[1]) + (t2[2] + t2[3])) + ((t2[4] + t2[5]) + (t2[6] + t2[7]));
            if ((gbits >> 31) || !(v0 < 1.0e300)) {
#pragma unroll
                for (int u = 0; u < 8; ++u)
                    if (!(gs[u] >= 0.0f) || gs[u] > 3.0e38f) bad |= 2u;
            }
        }
        double i0 = v0, i1 = v1;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const double u0 = __shfl_up_sync(0xffffffffu, i0, off);
            const double u1 = __shfl_up_sync(0xffffffffu, i1, off);
            if (lane >= off) { i0 += u0; i1 += u1; }
        }
        if (lane == 31 && SKIM_IDX(sgm, 96, a.status)) { ps.segtot[sgm][0] = i0; ps.segtot[sgm][1] = i1; }
        double e0 = __shfl_up_sync(0xffffffffu, i0, 1), e1 = __shfl_up_sync(0xffffffffu, i1, 1);
        if (lane == 0) { e0 = 0.0; e1 = 0.0; }
        if (q < R.ngrp) {
            st_sector(rec + R.groups + (size_t)q * SKIM_GROUP_BYTES_HALF, xq0, xq1,
                      (unsigned long long)__double_as_longlong(e0), (unsigned long long)__double_as_longlong(e1));
            gi[q] = first;
        }
    }
    if (bad) atomicOr(a.status, (unsigned long long)bad);
    for (int q = R.ngrp + threadIdx.x; q < sk_entries(m); q += THREADS) gi[q] = SKIM_PAD_VALUE;
    // every warp's sum of g*x^2, lanes added in a fixed order
#pragma unroll
    for (int off = 16; off; off >>= 1) w2acc += __shfl_xor_sync(0xffffffffu, w2acc, off);
    if (lane == 0) ps.wsum2[warp] = w2acc;
    __syncthreads();
    if (warp == 0) {
        double run0 = 0.0, run1 = 0.0, loc[4][2];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int sgm = lane * 4 + u;
#pragma unroll
            for (int c = 0; c < 2; ++c) loc[u][c] = sgm < R.nseg ? ps.segtot[sgm][c] : 0.0;
            run0 += loc[u][0]; run1 += loc[u][1];
        }
        double i0 = run0, i1 = run1;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const double u0 = __shfl_up_sync(0xffffffffu, i0, off);
            const double u1 = __shfl_up_sync(0xffffffffu, i1, off);
            if (lane >= off) { i0 += u0; i1 += u1; }
        }
        double b0 = __shfl_up_sync(0xffffffffu, i0, 1), b1 = __shfl_up_sync(0xffffffffu, i1, 1);
        if (lane == 0) { b0 = 0.0; b1 = 0.0; }
        double s2 = 0.0;
        for (int w = 0; w < NW; ++w) s2 += ps.wsum2[w];
        double4 *seg = reinterpret_cast<double4 *>(rec + R.seg);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int sgm = lane * 4 + u;
            if (sgm <= R.nseg) seg[sgm] = make_double4(b0, b1, sgm == R.nseg ? s2 : 0.0, 0.0);   // entry nseg: the row totals
            b0 += loc[u][0]; b1 += loc[u][1];
        }
        if (lane == 0) *reinterpret_cast<int *>(rec) = nd;
    }
}

// Stores the row's distinct values (nd <= 16 of them, from collect_distinct) in the record header.
__device__ __forceinline__ void write_distinct_values(const ClusterArgs &a, int nd, const float *dvals, int local_row)
{
    unsigned char *rec = a.scratch + (size_t)local_row * (size_t)a.rec_stride;
    if (threadIdx.x < 16) reinterpret_cast<float *>(rec + 64)[threadIdx.x] = threadIdx.x < nd ? dvals[threadIdx.x] : 0.0f;
}

}  // namespace skimk

// fp16-key sort kernel (skim_cluster16.cu).  Fills args.rec_stride when `launch`
// is false (planning) and launches over `rows` rows otherwise.  Returns SKIM_OK, or 1 when the
// call does not meet the kernel's requirements (then the generic sort kernel must be used).
int skim_launch_sort16(skim_ctx *ctx, skimk::ClusterArgs &args, int64_t rows, bool launch);
// Exact clustering kernel (skim_exact.cu): one block per row record; `scratch` holds `slots` slots of
// skim_exact_slot_bytes(cols) bytes.
int skim_launch_exact(skim_ctx *ctx, const skimk::ClusterArgs &args, int64_t rows, void *scratch, int slots);
// Lloyd kernel (skim_lloyd.cu): one warp per row record.
int skim_launch_lloyd(skim_ctx *ctx, const skimk::ClusterArgs &args, int64_t rows);
