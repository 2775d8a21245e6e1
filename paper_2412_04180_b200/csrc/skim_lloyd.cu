// Lloyd kernel, the second half of the row clustering (SKIM Algorithm 3, error pre-recording loop;
// objective of Section 3.2, diagonal form): one warp per row iterates on the row record the sort
// kernel left in global memory (sorted values and importance by groups of 8 with their binary64
// prefix sums, a group index) and writes the row's centroids and error table entries.
//
// An iteration is a chain of dependent small steps (midpoint, search, a few loads, a quotient), so a
// single row cannot go fast; the kernel gets its throughput from the number of rows in flight: up to 32
// warps per SM, each on its own row.  A warp first copies its row's group index (4 bytes per 8
// elements) into shared memory, so that the boundary search never waits on global memory; per
// iteration a lane then reads one 96-byte group record through the read-only path, the one global
// round trip of the iteration.
#include "skim_cluster_phases.cuh"

namespace {

using namespace skimk;

constexpr int LLOYD_WARPS = 4;   // rows per block
constexpr int WIN = 16;          // group-index entries held in registers

// dynamic shared memory of one warp: the group index (binary32, or binary16 with compact records), then 16 bytes
// per segment and for the row totals
__host__ __device__ inline size_t lloyd_warp_bytes(int m, bool half_index)
{
    const int nseg = ((((m + 7) >> 3) + (1 << SKIM_SEG_SHIFT) - 1) >> SKIM_SEG_SHIFT);
    const size_t idx = ((size_t)sk_entries(m) * (half_index ? 2 : 4) + 15) & ~(size_t)15;
    return idx + (size_t)(nseg + 1) * 16;
}

struct LloydSmem {
    double errs[32];
    float tfs[32];
    float dvals[16];
};

// One 32-byte read-only load from a 32-byte aligned global address.
__device__ __forceinline__ void ld_sector(const unsigned char *p, float4 &a, float4 &b)
{
    asm volatile("ld.global.nc.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=f"(a.x), "=f"(a.y), "=f"(a.z), "=f"(a.w), "=f"(b.x), "=f"(b.y), "=f"(b.z), "=f"(b.w)
                 : "l"(p));
}

// One group record in registers.  HALF = false: the full record (three sectors: binary32 values | importances |
// sums incl. g*x^2); HALF = true: the compact record of the fp16-key sort kernel (two sectors: binary16 values
// and the sums of g and g*x | importances).
template <bool HALF> struct Group;

template <> struct Group<false> {
    static constexpr int BYTES = SKIM_GROUP_BYTES;
    float4 xa, xb, ga, gb;
    double2 p;   // prefix sums of g and g*x at the group's first element
    __device__ __forceinline__ void load(const unsigned char *gr)
    {
        // the record is three 32-byte sectors: values, importances, sums; one read-only load each
        ld_sector(gr, xa, xb);
        ld_sector(gr + 32, ga, gb);
        p = __ldg(reinterpret_cast<const double2 *>(gr + 64));   // the g*x^2 sum at +80 is read once, for the error
    }
    // number of values <= t (values ascend; the padding is the largest finite value)
    __device__ __forceinline__ int count_le(float t) const
    {
        return (xa.x <= t) + (xa.y <= t) + (xa.z <= t) + (xa.w <= t) + (xb.x <= t) + (xb.y <= t) + (xb.z <= t) + (xb.w <= t);
    }
    __device__ __forceinline__ void values(double *x) const
    {
        x[0] = (double)xa.x; x[1] = (double)xa.y; x[2] = (double)xa.z; x[3] = (double)xa.w;
        x[4] = (double)xb.x; x[5] = (double)xb.y; x[6] = (double)xb.z; x[7] = (double)xb.w;
    }
    static __device__ __forceinline__ float value_at(const unsigned char *groups, int idx)
    {
        return __ldg(reinterpret_cast<const float *>(groups + (size_t)(idx >> 3) * BYTES) + (idx & 7));
    }
};

template <> struct Group<true> {
    static constexpr int BYTES = SKIM_GROUP_BYTES_HALF;
    uint32_t xh[4];      // 8 binary16 values
    float4 ga, gb;
    double2 p;
    __device__ __forceinline__ void load(const unsigned char *gr)
    {
        unsigned long long q0, q1, q2, q3;
        asm volatile("ld.global.nc.v4.b64 {%0, %1, %2, %3}, [%4];" : "=l"(q0), "=l"(q1), "=l"(q2), "=l"(q3) : "l"(gr));
        xh[0] = (uint32_t)q0; xh[1] = (uint32_t)(q0 >> 32); xh[2] = (uint32_t)q1; xh[3] = (uint32_t)(q1 >> 32);
        p = make_double2(__longlong_as_double((long long)q2), __longlong_as_double((long long)q3));
        ld_sector(gr + 32, ga, gb);
    }
    // a binary16 value is <= t exactly when it is <= t rounded down to binary16: four packed compares
    __device__ __forceinline__ int count_le(float t) const
    {
        const __half2 th = __half2half2(__float2half_rd(t));
        __half2 c = __hle2(*reinterpret_cast<const __half2 *>(&xh[0]), th);
        c = __hadd2(c, __hle2(*reinterpret_cast<const __half2 *>(&xh[1]), th));
        c = __hadd2(c, __hle2(*reinterpret_cast<const __half2 *>(&xh[2]), th));
        c = __hadd2(c, __hle2(*reinterpret_cast<const __half2 *>(&xh[3]), th));
        return (int)(__low2float(c) + __high2float(c));
    }
    __device__ __forceinline__ void values(double *x) const
    {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&xh[u]));
            x[2 * u] = (double)f.x;
            x[2 * u + 1] = (double)f.y;
        }
    }
    static __device__ __forceinline__ float value_at(const unsigned char *groups, int idx)
    {
        return __half2float(__ushort_as_half(__ldg(reinterpret_cast<const unsigned short *>(groups + (size_t)(idx >> 3) * BYTES) + (idx & 7))));
    }
};

// Adds the first n (0..8) elements of a group to (s0, s1[, s2]): the eight terms are summed pairwise,
// a fixed order with a short dependency chain.  Elements past n are masked before any arithmetic.
template <bool WANT_C, typename G>
__device__ __forceinline__ void add_group(const G &grp, int n, double &s0, double &s1, double &s2)
{
    double xs[8];
    grp.values(xs);
    const float gs[8] = {grp.ga.x, grp.ga.y, grp.ga.z, grp.ga.w, grp.gb.x, grp.gb.y, grp.gb.z, grp.gb.w};
    double t0[8], t1[8], t2[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        const bool in = u < n;
        const double g = (double)(in ? gs[u] : 0.0f), x = xs[u];   // padding values are finite, so 0 * x = 0
        t0[u] = g;
        t1[u] = g * x;
        if (WANT_C) t2[u] = t1[u] * x;
    }
    s0 += ((t0[0] + t0[1]) + (t0[2] + t0[3])) + ((t0[4] + t0[5]) + (t0[6] + t0[7]));
    s1 += ((t1[0] + t1[1]) + (t1[2] + t1[3])) + ((t1[4] + t1[5]) + (t1[6] + t1[7]));
    if (WANT_C) s2 += ((t2[0] + t2[1]) + (t2[2] + t2[3])) + ((t2[4] + t2[5]) + (t2[6] + t2[7]));
}

// A window of 16 ascending group-index entries around the previous boundary position (at least 4
// entries, i.e. 32 elements, on either side), read from shared memory with four independent loads;
// only when the boundary left it does the search fall back to a binary search of the whole index.
template <bool HALF> struct Window;

template <> struct Window<false> {
    typedef float Entry;
    static __device__ __forceinline__ bool le(float e, float t) { return e <= t; }
    float4 v[4];
    int ws;
    __device__ __forceinline__ void load(const float *gi, int ngi, int guess)   // gi: shared memory
    {
        ws = max(0, min((((guess + 4) >> 3) << 3) - 8, ngi - WIN));     // may reach into the 16 padding entries behind the index
        const float4 *p = reinterpret_cast<const float4 *>(gi + ws);
#pragma unroll
        for (int q = 0; q < 4; ++q) v[q] = p[q];
    }
    // number of window entries <= t: a 4-step binary search over the 16 ascending registers
    __device__ __forceinline__ int count_le(float t) const
    {
        const bool b3 = v[1].w <= t;                                   // entry 7
        const float4 h = b3 ? v[3] : v[1], l = b3 ? v[2] : v[0];      // entries 8..15 or 0..7: h = upper four, l = lower four
        const bool b2 = l.w <= t;                                      // entry 3 of the half
        const float4 q = b2 ? h : l;
        const bool b1 = q.y <= t;
        const float e = b1 ? q.z : q.x;
        const float e2 = b1 ? q.w : q.y;
        const bool b0 = e <= t;
        // position inside the quad: entries <= t among (x, y, z, w)
        const int inq = b1 ? (b0 ? ((e2 <= t) ? 4 : 3) : 2) : (b0 ? 1 : 0);
        return (b3 ? 8 : 0) + (b2 ? 4 : 0) + inq;
    }
};

// The same window over a binary16 copy of the index (compact records: every value is a binary16 number, and a
// binary16 value is <= t exactly when it is <= t rounded down to binary16): two loads, eight packed compares.
template <> struct Window<true> {
    typedef __half Entry;
    static __device__ __forceinline__ bool le(__half e, float t) { return __half2float(e) <= t; }
    uint4 v[2];
    int ws;
    __device__ __forceinline__ void load(const __half *gi, int ngi, int guess)   // gi: shared memory
    {
        ws = max(0, min((((guess + 4) >> 3) << 3) - 8, ngi - WIN));
        const uint4 *p = reinterpret_cast<const uint4 *>(gi + ws);
        v[0] = p[0];
        v[1] = p[1];
    }
    __device__ __forceinline__ int count_le(float t) const
    {
        const __half2 th = __half2half2(__float2half_rd(t));
        const uint32_t w[8] = {v[0].x, v[0].y, v[0].z, v[0].w, v[1].x, v[1].y, v[1].z, v[1].w};
        __half2 c = __hle2(*reinterpret_cast<const __half2 *>(&w[0]), th);
#pragma unroll
        for (int u = 1; u < 8; ++u) c = __hadd2(c, __hle2(*reinterpret_cast<const __half2 *>(&w[u]), th));
        return (int)(__low2float(c) + __high2float(c));
    }
};

// s1 / s0 for s0 > 0: binary32 reciprocal seed and two binary64 Newton corrections (relative
// error about 2^-60, i.e. the correctly rounded quotient up to the last bit or so); operands far
// outside the binary32 range take the plain division.
__device__ __forceinline__ double quotient(double s1, double s0)
{
    const float s0f = (float)s0;
    if (!(s0f > 1e-30f && s0f < 1e30f) || !(fabs(s1) < 1e30)) return s1 / s0;
    const float rf = __frcp_rn(s0f);
    const double rd = (double)rf;
    double q = (double)((float)s1 * rf);
    q = fma(fma(-q, s0, s1), rd, q);
    q = fma(fma(-q, s0, s1), rd, q);
    return q;
}

// Lloyd iterations and the error table entry of one row, run by ONE warp (all 32 lanes call).
// Lane L owns centroid L of the row's concatenated centroid record and the boundary above it.
// Per iteration a lane: forms the exact midpoint; counts the group-index entries below it in the
// register window (falling back to a binary search of the group index when the boundary left the
// window); loads that one group record, which gives the exact boundary position (values), the
// prefix sums at the group start and the few elements in between.
// On return sm.tfs[L] holds the boundary (largest binary32 value still assigned to centroid L).
template <bool HALF>
__device__ __forceinline__ void lloyd_warp(const unsigned char *rec, const typename Window<HALF>::Entry *gi, const double2 *segs,
                                           int nd, const ClusterArgs &a, int64_t row, LloydSmem &sm)
{
    const int lane = threadIdx.x & 31;
    const int m = a.m;
    const RowRecord R = row_record(m, HALF);
    const unsigned char *groups = rec + R.groups;
    const double4 *seg = reinterpret_cast<const double4 *>(rec + R.seg);   // 32-byte entries; a few hot lines, served by L1
    const int ngi = sk_entries(m) - 16;                 // group-index entries up to the padding margin
    const float INF = __int_as_float(0x7f800000);
    int bi = 0, off = 0;
    while (bi < a.nb && lane >= off + (1 << (a.bmin + bi))) { off += 1 << (a.bmin + bi); ++bi; }
    const bool in_set = lane < a.sumk;
    const int width = a.bmin + bi;
    const int k = 1 << width;
    const int j = lane - off;
    const bool wanted = in_set && (!a.row_bits || a.row_bits[row] == width);
    const bool degenerate = wanted && (nd <= k);      // every value gets its own centroid
    const bool normal = wanted && !degenerate;
    const bool has_boundary = wanted && j < k - 1;
    const bool searches = normal && j < k - 1;
    float c = 0.0f;
    if (degenerate) c = sm.dvals[min(j, nd - 1)];
    if (normal) {
        const int idx = (int)(((long long)(2 * j + 1) * m) / (2 * k));
        if (SKIM_IDX(idx, m, a.status)) c = Group<HALF>::value_at(groups, idx);
    }

    int Bprev = -1;
    float tf = INF;                                   // no boundary above the last centroid
    double err_j = 0.0;
    int gprev = -1;                                   // group of the previous boundary position
    int gstep = 0;                                    // its last move: boundaries keep drifting the same way
    for (int it = 0;; ++it) {
        const float c_up = __shfl_down_sync(0xffffffffu, c, 1);
        int B = m, grp_i = 0, cntk = 0;
        Group<HALF> grp;
        if (has_boundary) {
            // exact midpoint of two binary32 centroids, rounded down to binary32: x <= midpoint
            // holds for a binary32 x exactly when x <= tf
            tf = __double2float_rd(0.5 * ((double)c + (double)c_up));
            if (tf == 0.0f) tf = 0.0f;
        }
        if (searches) {
            int nle = -1;                              // group-index entries <= tf
            if (gprev >= 0) {
                Window<HALF> win;
                win.load(gi, ngi, gprev + 1 + gstep);     // centred where the boundary is heading
                const int cnt = win.count_le(tf);
                // valid unless the boundary may lie outside the window: below its first entry (unless the window
                // starts the index) or above its last (unless only padding follows)
                if ((cnt > 0 || win.ws == 0) && (cnt < WIN || win.ws + WIN >= ngi)) nle = win.ws + cnt;
            }
            if (nle < 0) {
                int lo = 0, hi = ngi;
                while (lo < hi) {
                    const int mid = (lo + hi) >> 1;
                    if (Window<HALF>::le(gi[mid], tf)) lo = mid + 1; else hi = mid;
                }
                nle = lo;
            }
            grp_i = max(nle - 1, 0);
            if (!SKIM_IDX(grp_i, R.ngrp, a.status)) grp_i = 0;
            gstep = gprev >= 0 ? grp_i - gprev : 0;
            gprev = grp_i;
            const unsigned char *gr = groups + (size_t)grp_i * Group<HALF>::BYTES;
            grp.load(gr);
            cntk = grp.count_le(tf);
            B = min((grp_i << 3) + cntk, m);
        }
        const bool same = __all_sync(0xffffffffu, B == Bprev);
        const bool final = (it >= a.iters) || (same && a.early_exit);
        Bprev = B;
        double P0 = 0.0, P1 = 0.0, Pc = 0.0;
        if (normal) {
            if (searches) {
                const double2 sb = segs[grp_i >> SKIM_SEG_SHIFT];   // sums of the earlier segments (shared memory)
                P0 = sb.x + grp.p.x;
                P1 = sb.y + grp.p.y;
                if (final && !HALF) {
                    Pc = __ldg(&seg[grp_i >> SKIM_SEG_SHIFT].z) + __ldg(reinterpret_cast<const double *>(groups + (size_t)grp_i * SKIM_GROUP_BYTES + 80));
                    add_group<true>(grp, cntk, P0, P1, Pc);
                } else {
                    add_group<false>(grp, cntk, P0, P1, Pc);
                }
            } else {
                // the last centroid of a width has no boundary above it: its prefix is the row total
                const double2 tot = segs[R.nseg];
                P0 = tot.x;
                P1 = tot.y;
                if (final && !HALF) Pc = __ldg(&seg[R.nseg].z);
            }
        }
        double Q0 = __shfl_up_sync(0xffffffffu, P0, 1);
        double Q1 = __shfl_up_sync(0xffffffffu, P1, 1);
        double Qc = (final && !HALF) ? __shfl_up_sync(0xffffffffu, Pc, 1) : 0.0;
        if (j == 0) { Q0 = 0.0; Q1 = 0.0; Qc = 0.0; }
        const double S0 = P0 - Q0, S1 = P1 - Q1;
        if (final) {
            if (normal) {
                const double cd = (double)c, S2 = Pc - Qc;
                // full record: the cluster's own error; compact record: the part the row total of g*x^2 is
                // reduced by, c (2 S1 - c S0)
                err_j = HALF ? cd * fma(-cd, S0, 2.0 * S1) : fmax(fma(cd, fma(cd, S0, -2.0 * S1), S2), 0.0);
            }
            if (a.iter_stats && lane == 0) {
                atomicAdd(a.iter_stats, (unsigned long long)it);       // assign/update pairs this row ran
                atomicAdd(a.iter_stats + 1, 1ull);
            }
            break;
        }
        // a cluster without weight keeps its centroid.  S0 is a difference of rounded prefix sums: over a
        // run of zero importances that crosses a group or segment border it is rounding noise of either
        // sign, not 0, so "has weight" means: above 2^-40 of the prefix it was taken from
        if (normal && S0 > P0 * 0x1p-40) c = (float)quotient(S1, S0);
    }
    sm.errs[lane] = err_j;
    sm.tfs[lane] = has_boundary ? tf : INF;
    __syncwarp();
    if (wanted) {
        if (a.centroids) a.centroids[row * a.sumk + lane] = c;
        if (j == 0 && a.err) {
            double e = 0.0;
            for (int u = 0; u < k; ++u) e += sm.errs[lane + u];
            if (HALF) e = normal ? fmax(__ldg(&reinterpret_cast<const double4 *>(rec + R.seg)[R.nseg].z) - e, 0.0) : 0.0;
            if (a.row_bits) a.err[row] = (float)e; else a.err[row * a.nb + bi] = (float)e;
        }
    }
}

// Optional labels of the final assignment, in column order (test/diagnostic output).
__device__ __forceinline__ void write_codes(const ClusterArgs &a, int64_t row, const LloydSmem &sm)
{
    const int m = a.m, lane = threadIdx.x & 31;
    const uint16_t *Wr = a.W + row * a.ld;
    int only = -1;
    if (a.row_bits) only = (int)a.row_bits[row] - a.bmin;
    for (int e = lane; e < m; e += 32) {
        float x = __half2float(__ushort_as_half(Wr[e]));
        if (a.rscale) x = __fmul_rn(x, a.rscale[e]);
        int off = 0;
        for (int bi = 0; bi < a.nb; ++bi) {
            const int k = 1 << (a.bmin + bi);
            if (only < 0 || only == bi) {
                // number of boundaries below x: the boundaries of a width ascend, so log2(k) probes find it
                int code = 0;
                for (int step = k >> 1; step >= 1; step >>= 1)
                    if (sm.tfs[off + code + step - 1] < x) code += step;
                if (only < 0) a.codes[((int64_t)bi * a.rows + row) * m + e] = (uint8_t)code;
                else a.codes[row * (int64_t)m + e] = (uint8_t)code;
            }
            off += k;
        }
    }
}

// Seven blocks of four rows per SM: an eighth would hold the kernel to 64 registers, which measured slower on every
// shape (the full-record form spills there).
template <bool HALF>
__global__ void __launch_bounds__(LLOYD_WARPS * 32, 7) skim_lloyd_kernel(ClusterArgs a, int rows_in_chunk)
{
    __shared__ LloydSmem sm_all[LLOYD_WARPS];
    extern __shared__ __align__(16) unsigned char gi_all[];      // [LLOYD_WARPS][sk_entries(m)] index entries (binary32, or binary16 with compact records)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int local = blockIdx.x * LLOYD_WARPS + warp;
    if (local >= rows_in_chunk) return;
    LloydSmem &sm = sm_all[warp];
    const int64_t row = a.row0 + local;
    const unsigned char *rec = a.scratch + (size_t)local * (size_t)a.rec_stride;
    const int nd_rec = *reinterpret_cast<const int *>(rec);
    if (nd_rec < 0) return;                 // the sort kernel gave this row up (status word says why): no output
    const int nd = max(nd_rec, 1);          // indexes sm.dvals below
    if (lane < 16) sm.dvals[lane] = reinterpret_cast<const float *>(rec + 64)[lane];
    // the row's group index, copied once
    const int nsk = sk_entries(a.m);
    typedef typename Window<HALF>::Entry Entry;
    const size_t per_warp = lloyd_warp_bytes(a.m, HALF);
    Entry *gi = reinterpret_cast<Entry *>(gi_all + (size_t)warp * per_warp);
    double2 *segs = reinterpret_cast<double2 *>(gi_all + (size_t)warp * per_warp + (((size_t)nsk * sizeof(Entry) + 15) & ~(size_t)15));
    {
        // the segment table's sums of g and g*x (one pair per segment, the row totals last)
        const RowRecord R = row_record(a.m, HALF);
        const double4 *seg = reinterpret_cast<const double4 *>(rec + R.seg);
        for (int i = lane; i <= R.nseg; i += 32) segs[i] = __ldg(reinterpret_cast<const double2 *>(seg + i));
        const float4 *src = reinterpret_cast<const float4 *>(rec + row_record(a.m, HALF).gi);
        for (int i = lane; i < nsk / 4; i += 32) {
            const float4 v = __ldg(src + i);
            if (HALF) {
                // exact: the entries are binary16 numbers (the padding, the largest binary32, becomes +inf)
                const __half2 lo = __floats2half2_rn(v.x, v.y), hi = __floats2half2_rn(v.z, v.w);
                reinterpret_cast<uint2 *>(gi)[i] = make_uint2(*reinterpret_cast<const uint32_t *>(&lo), *reinterpret_cast<const uint32_t *>(&hi));
            } else {
                reinterpret_cast<float4 *>(gi)[i] = v;
            }
        }
    }
    __syncwarp();
    lloyd_warp<HALF>(rec, gi, segs, nd, a, row, sm);
    if (!a.codes) return;
    __syncwarp();
    write_codes(a, row, sm);
}

}  // namespace

int skim_launch_lloyd(skim_ctx *ctx, const ClusterArgs &args, int64_t rows)
{
    const unsigned blocks = (unsigned)((rows + LLOYD_WARPS - 1) / LLOYD_WARPS);
    const size_t smem = (size_t)LLOYD_WARPS * lloyd_warp_bytes(args.m, args.rec_half != 0);
    // set on every launch: a host-side call of microseconds, and no state shared between contexts
    void (*kernel)(ClusterArgs, int) = args.rec_half ? skim_lloyd_kernel<true> : skim_lloyd_kernel<false>;
    SKIM_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    kernel<<<blocks, LLOYD_WARPS * 32, smem, ctx->stream>>>(args, (int)rows);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    return SKIM_OK;
}
