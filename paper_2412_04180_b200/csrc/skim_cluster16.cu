// fp16-key row-sorting kernel, the first half of the row clustering (SKIM Algorithm 3, error pre-recording loop; objective of
// Section 3.2, diagonal form) for the common case: no scale vector installed, rows 16-byte aligned.
//
// With no scale the clustered value IS the fp16 weight, so a 16-bit order-preserving key is exact
// and the sort moves one 32-bit word per element: (key << 16) | column.
//
//   load    128-bit loads of the fp16 row straight into keys.
//   pass 0  low 12 key bits, 4096 block-wide counters; the counting atomic already hands every item
//           its slot inside its bin.
//           The first pass of an LSD sort need not be stable, so no ranking is needed.  The
//           scatter also counts, per owner thread of pass 1 and high digit, how many items land
//           in that thread's stretch of positions.
//   pass 1  high 4 key bits, stable without any warp-wide ranking: a thread owns a contiguous
//           stretch of positions, takes its items in position order and numbers them with
//           counters of its own (one 16-bit counter per thread and digit, prefix-summed across
//           threads per digit), so the order inside a digit is the order of pass 0.
//   then    one pass over the sorted items (skim_cluster_phases.cuh) writes the row record -- group
//           records with prefix sums, group index, segment table -- to global memory, from which
//           the Lloyd kernel (skim_lloyd.cu) iterates with one warp per row.  The pass fetches every
//           element's importance through the column index the item carries, so the importance
//           row is never rearranged in shared memory.
// The fp32 importance row is fetched by one bulk asynchronous copy (cp.async.bulk + mbarrier) that
// is issued once pass 0 is over (its landing area holds the pass-0 counters until then) and runs
// under pass 1.
//
// Shared memory per 11 008-column row is about 105 KB and the kernel is held to 64 registers, so two
// rows are resident per SM.
#include "skim_cluster_phases.cuh"

namespace {

using namespace skimk;

constexpr int D0_BITS = 12, D0 = 1 << D0_BITS;
constexpr int D1_BITS = 4, D1 = 1 << D1_BITS;
constexpr int MBAR_SPIN_LIMIT = 1 << 22;
constexpr uint32_t NO_ITEM = 0xffffffffu;    // slot of a thread beyond the row's end (no column is 65 535)
constexpr uint32_t PAD_ITEM = 0xffff0000u;   // largest key, column 0: fills the last group of the sorted row

struct Layout16 {
    size_t buf, graw, cnt1, dbase1, phase, mbar, total;
};

// buf:   the packed items, padded to a whole group of 8
// graw:  the raw importance row; the pass-0 counters (D0 words) until the copy is issued
// cnt1:  pass-1 counters, [D1][threads] 16-bit
__host__ __device__ inline Layout16 layout16(int m, int threads)
{
    Layout16 L;
    size_t off = 0;
    auto take = [&](size_t b) { size_t o = off; off += (b + 15) & ~(size_t)15; return o; };
    const size_t row = ((size_t)m + 7) / 8 * 8 * 4;
    L.buf = take(row);
    L.graw = take(row > (size_t)D0 * 4 ? row : (size_t)D0 * 4);
    L.cnt1 = take((size_t)D1 * threads * 2);
    L.dbase1 = take(D1 * 4);
    L.phase = take(sizeof(PhaseSmem));
    L.mbar = take(16);
    L.total = off;
    return L;
}

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, int count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}

__device__ __forceinline__ void bulk_load(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_addr(dst)),
                 "l"(src), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok)
                 : "r"(smem_addr(bar)), "r"(parity)
                 : "memory");
    return ok != 0;
}

// Bounded wait: false if the copy has not landed after MBAR_SPIN_LIMIT polls.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t *bar, uint32_t parity)
{
    for (int spin = 0; spin < MBAR_SPIN_LIMIT; ++spin)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

// The sorted row of this kernel: packed items (key << 16 | column) in sorted order, and the raw
// importance row, which the record pass reads through the column index.
struct SortedItems16 {
    const uint32_t *items;
    const float *graw;
    unsigned long long *status;
    __device__ __forceinline__ unsigned group(int e, int m, uint16_t *ks, float *gs) const
    {
        const uint4 a = *reinterpret_cast<const uint4 *>(items + e), b = *reinterpret_cast<const uint4 *>(items + e + 4);
        const uint32_t it[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
        unsigned bits = 0u;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            ks[u] = (uint16_t)(it[u] >> 16);
            const float g = (e + u < m && SKIM_IDX(it[u] & 0xffffu, m, status)) ? graw[it[u] & 0xffffu] : 0.0f;
            bits |= __float_as_uint(g);
            gs[u] = g;
        }
        return bits;      // not validated here
    }
    __device__ __forceinline__ uint16_t key_at(int p) const { return (uint16_t)(items[p] >> 16); }
};

template <int THREADS, int VEC>
__global__ void __launch_bounds__(THREADS, (THREADS <= 512 ? 2 : 1)) skim_sort16_kernel(ClusterArgs a)
{
    using K = KeyOps<uint16_t>;
    constexpr int ITEMS = VEC * 8;
    constexpr int EPT = D0 / THREADS;           // pass-0 counters scanned per thread
    constexpr int WPL = THREADS / 64;           // pass-1 counter words (two counters each) scanned per lane
    constexpr int NW = THREADS / 32;
    static_assert(D0 % THREADS == 0 && THREADS % 64 == 0, "thread count must divide 4096 and be a multiple of 64");
    extern __shared__ __align__(16) unsigned char smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int m = a.m;
    const int mpad = (m + 7) & ~7;
    const Layout16 L = layout16(m, THREADS);
    uint32_t *buf = reinterpret_cast<uint32_t *>(smem + L.buf);
    float *graw = reinterpret_cast<float *>(smem + L.graw);
    uint32_t *C0 = reinterpret_cast<uint32_t *>(smem + L.graw);
    uint32_t *cnt1w = reinterpret_cast<uint32_t *>(smem + L.cnt1);
    uint16_t *cnt1 = reinterpret_cast<uint16_t *>(smem + L.cnt1);
    uint32_t *dbase1 = reinterpret_cast<uint32_t *>(smem + L.dbase1);
    PhaseSmem &ps = *reinterpret_cast<PhaseSmem *>(smem + L.phase);
    uint64_t *mbar = reinterpret_cast<uint64_t *>(smem + L.mbar);
    uint32_t *scratch = reinterpret_cast<uint32_t *>(ps.segtot);   // free until the record pass

    const int64_t row = a.row0 + blockIdx.x;
    const uint16_t *Wr = a.W + row * a.ld;
    const float *Gr = a.G + row * a.ld;

    // ---------------------------------------------------------------- set-up
    if (tid == 0) {
        mbar_init(mbar, 1);
        ps.misc[0] = 0;
        ps.misc[1] = 0;
    }
    for (int d = tid; d < D0; d += THREADS) C0[d] = 0u;
    for (int d = tid; d < D1 * THREADS / 2; d += THREADS) cnt1w[d] = 0u;
    if (tid < mpad - m) buf[m + tid] = PAD_ITEM;
    __syncthreads();

    // ---------------------------------------------------------------- load, keys, pass-0 histogram
    uint32_t item[ITEMS];
    unsigned bad = 0;
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
        const int e0 = (j * THREADS + tid) * 8;
        uint32_t w[4];
        if (e0 + 8 <= m) {
            const uint4 raw = *reinterpret_cast<const uint4 *>(Wr + e0);
            w[0] = raw.x; w[1] = raw.y; w[2] = raw.z; w[3] = raw.w;
        } else {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t lo = (e0 + 2 * u < m) ? Wr[e0 + 2 * u] : 0u;
                const uint32_t hi = (e0 + 2 * u + 1 < m) ? Wr[e0 + 2 * u + 1] : 0u;
                w[u] = lo | (hi << 16);
            }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            uint16_t h = (uint16_t)((u & 1) ? (w[u >> 1] >> 16) : (w[u >> 1] & 0xffffu));
            const bool real = e0 + u < m;
            if (real && (h & 0x7c00u) == 0x7c00u) bad |= 1u;
            if (h == 0x8000u) h = 0;                      // -0 and +0 are one value
            const uint32_t key = (uint32_t)K::from_half_bits(h);
            // the count's old value is the item's slot inside its bin; it rides in the low half until the
            // scatter puts the column there (the column follows from the item's place in the thread)
            item[j * 8 + u] = real ? ((key << 16) | atomicAdd(&C0[key & (D0 - 1)], 1u)) : NO_ITEM;
        }
    }
    if (bad) atomicOr(a.status, (unsigned long long)bad);
    __syncthreads();

    // ---------------------------------------------------------------- pass 0: scan, claim slots, scatter
    {
        // a thread's EPT consecutive counters go through 128-bit accesses (scalar ones would hit one bank 8 ways)
        uint32_t loc[EPT], s = 0, occupied = 0;
        uint4 *C04 = reinterpret_cast<uint4 *>(C0 + tid * EPT);
#pragma unroll
        for (int u = 0; u < EPT / 4; ++u) {
            const uint4 v = C04[u];
            loc[4 * u] = v.x; loc[4 * u + 1] = v.y; loc[4 * u + 2] = v.z; loc[4 * u + 3] = v.w;
        }
#pragma unroll
        for (int u = 0; u < EPT; ++u) { s += loc[u]; occupied += loc[u] ? 1u : 0u; }
        // occupied low-digit bins: a lower bound of the number of distinct values
        occupied = __reduce_add_sync(0xffffffffu, occupied);
        if (lane == 0 && occupied) atomicAdd(&ps.misc[0], (int)occupied);
        uint32_t inc = s;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, inc, off);
            if (lane >= off) inc += t;
        }
        if (lane == 31) scratch[warp] = inc;
        __syncthreads();
        uint32_t run = inc - s;
        for (int w = 0; w < warp; ++w) run += scratch[w];
#pragma unroll
        for (int u = 0; u < EPT / 4; ++u) {
            uint4 v;
            v.x = run; run += loc[4 * u];
            v.y = run; run += loc[4 * u + 1];
            v.z = run; run += loc[4 * u + 2];
            v.w = run; run += loc[4 * u + 3];
            C04[u] = v;
        }
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
        if (item[i] != NO_ITEM) {
            const uint32_t key = item[i] >> 16;
            const uint32_t pos = C0[key & (D0 - 1)] + (item[i] & 0xffffu);      // bin base + slot
            const uint32_t col = (uint32_t)(((i >> 3) * THREADS + tid) * 8 + (i & 7));
            if (SKIM_IDX(pos, m, a.status)) buf[pos] = (key << 16) | col;
            // one more item of digit key >> 12 in the stretch of pass-1 owner pos / ITEMS
            const uint32_t owner = pos / ITEMS;
            if (SKIM_IDX(owner, THREADS, a.status))
                atomicAdd(&cnt1w[((key >> D0_BITS) * THREADS + owner) >> 1], (owner & 1u) ? 0x10000u : 1u);
        }
    }
    // the pass-0 counters are dead: their place takes the importance row, by the asynchronous proxy
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    if (tid == 0) {
        const uint32_t bytes = (uint32_t)m * 4u;
        mbar_expect_tx(mbar, bytes);
        for (uint32_t o = 0; o < bytes; o += 32768u)
            bulk_load(reinterpret_cast<unsigned char *>(graw) + o, reinterpret_cast<const unsigned char *>(Gr) + o,
                      min(32768u, bytes - o), mbar);
    }

    // ---------------------------------------------------------------- pass 1: counters -> positions
    // per digit, an exclusive prefix sum over the owner threads (a lane takes 2 * WPL consecutive owners)
    for (int d = warp; d < D1; d += NW) {
        uint32_t *cw = cnt1w + (d * THREADS) / 2 + lane * WPL;
        uint32_t wv[WPL], s = 0;
        if constexpr (WPL % 4 == 0) {
#pragma unroll
            for (int u = 0; u < WPL / 4; ++u) {
                const uint4 v = reinterpret_cast<const uint4 *>(cw)[u];
                wv[4 * u] = v.x; wv[4 * u + 1] = v.y; wv[4 * u + 2] = v.z; wv[4 * u + 3] = v.w;
            }
        } else {
#pragma unroll
            for (int u = 0; u < WPL; ++u) wv[u] = cw[u];
        }
#pragma unroll
        for (int u = 0; u < WPL; ++u) s += (wv[u] & 0xffffu) + (wv[u] >> 16);
        uint32_t inc = s;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, inc, off);
            if (lane >= off) inc += t;
        }
        if (lane == 31) dbase1[d] = inc;          // the digit's total
        uint32_t run = inc - s;
#pragma unroll
        for (int u = 0; u < WPL; ++u) {
            const uint32_t lo = wv[u] & 0xffffu, hi = wv[u] >> 16;
            wv[u] = run | ((run + lo) << 16);
            run += lo + hi;
        }
        if constexpr (WPL % 4 == 0) {
#pragma unroll
            for (int u = 0; u < WPL / 4; ++u)
                reinterpret_cast<uint4 *>(cw)[u] = make_uint4(wv[4 * u], wv[4 * u + 1], wv[4 * u + 2], wv[4 * u + 3]);
        } else {
#pragma unroll
            for (int u = 0; u < WPL; ++u) cw[u] = wv[u];
        }
    }
    // my stretch of positions, in order
#pragma unroll
    for (int i = 0; i < ITEMS; i += 4) {
        const int p = tid * ITEMS + i;
        uint4 v = make_uint4(NO_ITEM, NO_ITEM, NO_ITEM, NO_ITEM);
        if (p < m) v = *reinterpret_cast<const uint4 *>(buf + p);     // m is a multiple of 4 here
        item[i] = v.x; item[i + 1] = v.y; item[i + 2] = v.z; item[i + 3] = v.w;
    }
    __syncthreads();
    if (warp == 0) {
        // digit totals -> digit bases
        const uint32_t tot = lane < D1 ? dbase1[lane] : 0u;
        uint32_t inc = tot;
#pragma unroll
        for (int off = 1; off < D1; off <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, inc, off);
            if (lane >= off) inc += t;
        }
        if (lane < D1) dbase1[lane] = inc - tot;
    }
    __syncthreads();
    // positions = digit base + prefix over the owners before me; then number my items in order
#pragma unroll 4
    for (int d = 0; d < D1; ++d) cnt1[d * THREADS + tid] = (uint16_t)(cnt1[d * THREADS + tid] + dbase1[d]);
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
        if (tid * ITEMS + i < m) {
            uint16_t *c = cnt1 + (item[i] >> (16 + D0_BITS)) * THREADS + tid;
            const uint32_t pos = *c;
            *c = (uint16_t)(pos + 1u);
            if (SKIM_IDX(pos, m, a.status)) buf[pos] = item[i];
        }
    }

    // ---------------------------------------------------------------- the importance row must have landed
    // (the vote below is also the barrier that ends pass 1)
    {
        const bool landed = mbar_wait_bounded(mbar, 0);
        if (!__syncthreads_and(landed ? 1 : 0)) {
            // the copy never arrived: flag it, give it one more bounded chance to drain, leave
            // and mark the row record invalid, so that the Lloyd kernel skips the row
            if (tid == 0) {
                atomicOr(a.status, (unsigned long long)SKIM_STATUS_TIMEOUT);
                *reinterpret_cast<int *>(a.scratch + (size_t)blockIdx.x * (size_t)a.rec_stride) = -1;
            }
            mbar_wait_bounded(mbar, 0);
            return;
        }
    }
    // ---------------------------------------------------------------- row record
    const SortedItems16 src{buf, graw, a.status};
    int nd = ps.misc[0];                     // more than 16 occupied bins: more than 16 distinct values
    if (nd <= 16) {
        // few bins: count the distinct values themselves
        __syncthreads();
        if (tid == 0) ps.misc[0] = 0;
        __syncthreads();
        int dcount = 0;
        for (int p = tid; p < m; p += THREADS) dcount += (p == 0 || src.key_at(p) != src.key_at(p - 1)) ? 1 : 0;
        dcount = __reduce_add_sync(0xffffffffu, dcount);
        if (lane == 0 && dcount) atomicAdd(&ps.misc[0], dcount);
        __syncthreads();
        nd = ps.misc[0];
    }
    write_row_record_half<THREADS>(a, src, ps, nd, (int)blockIdx.x);
    if (nd <= 16) {
        collect_distinct<uint16_t, THREADS>(src, m, nd, ps);
        write_distinct_values(a, nd, ps.dvals, (int)blockIdx.x);
    }
}

struct Variant16 {
    int cap;
    int threads;
    void (*kernel)(ClusterArgs);
};

#define SKIM_V16(T, V) {T * V * 8, T, skim_sort16_kernel<T, V>}

const Variant16 kVariants[] = {
    SKIM_V16(128, 1), SKIM_V16(256, 1), SKIM_V16(512, 1), SKIM_V16(512, 2), SKIM_V16(512, 3), SKIM_V16(1024, 2),
    SKIM_V16(1024, 3),
};

}  // namespace

int skim_launch_sort16(skim_ctx *ctx, ClusterArgs &args, int64_t rows, bool launch)
{
    const int64_t cols = args.m;
    // 128-bit loads of W rows and the bulk copy of importance rows need 16-byte aligned rows
    if ((reinterpret_cast<uintptr_t>(args.W) & 15u) || (args.ld % 8) != 0) return 1;
    if ((reinterpret_cast<uintptr_t>(args.G) & 15u) || (cols % 4) != 0) return 1;
    for (const Variant16 &v : kVariants) {
        if (v.cap < cols) continue;
        const Layout16 L = layout16((int)cols, v.threads);
        if (L.total > (size_t)ctx->max_smem_optin) continue;
        args.rec_stride = (long long)row_record(args.m, true).total;
        args.rec_half = 1;
        if (!launch) return SKIM_OK;
        const ClusterArgs a = args;
        // set on every launch: a host-side call of microseconds, and no state shared between contexts
        SKIM_CUDA_OK(cudaFuncSetAttribute(v.kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L.total));
        v.kernel<<<(unsigned)rows, v.threads, L.total, ctx->stream>>>(a);
        SKIM_CUDA_OK(cudaGetLastError());
        ctx->launches += 1;
        return SKIM_OK;
    }
    return 1;
}
