// fp16-key row-sorting kernel, the first half of the row clustering (SKIM Algorithm 3, error pre-recording loop; objective of
// Section 3.2, diagonal form) for the common case: no scale vector installed, rows 16-byte aligned.
//
// With no scale the clustered value IS the fp16 weight, so a 16-bit order-preserving key is exact
// and the sort moves one 32-bit word per element: (key << 16) | column.
//
//   load    128-bit loads of the fp16 row straight into keys; the fp32 importance row is fetched
//           by one bulk asynchronous copy (cp.async.bulk + mbarrier) that runs under the sort.
//   pass 0  low 10 key bits, 1024 block-wide counters, slots claimed with shared-memory atomics.
//           The first pass of an LSD sort need not be stable, so no ranking is needed; the same
//           loop also builds the per-warp histogram of the next pass (the element's owner warp in
//           pass 1 follows from its slot).
//   pass 1  high 6 key bits, stable: lanes holding the same digit are found with 6 ballots.
//   then    one pass over the sorted items (skim_cluster_phases.cuh) writes the row record -- group
//           records with prefix sums, group index, segment table -- to global memory, from which
//           the Lloyd kernel (skim_lloyd.cu) iterates with one warp per row.  The pass fetches every
//           element's importance through the column index the item carries, so the importance
//           row is never rearranged in shared memory.
//
// Shared memory per 11 008-column row is about 107 KB and the kernel is held to 64 registers, so two
// rows are resident per SM.
#include "skim_cluster_phases.cuh"

namespace {

using namespace skimk;

constexpr int D0_BITS = 10, D0 = 1 << D0_BITS;
constexpr int D1_BITS = 6, D1 = 1 << D1_BITS;
constexpr int MBAR_SPIN_LIMIT = 1 << 22;

struct Layout16 {
    size_t buf, graw, uni, dbase1, phase, mbar, total;
};

// buf:  CAP words: packed items
// graw: CAP floats: the raw importance row
// uni:  pass counters
__host__ __device__ inline Layout16 layout16(int cap, int nwarps)
{
    Layout16 L;
    size_t off = 0;
    auto take = [&](size_t b) { size_t o = off; off += (b + 15) & ~(size_t)15; return o; };
    L.buf = take((size_t)cap * 4);
    L.graw = take((size_t)cap * 4);
    L.uni = take((size_t)D0 * 4 + (size_t)nwarps * D1 * 4);
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
    __device__ __forceinline__ unsigned group(int e, int m, uint16_t *ks, float *gs) const
    {
        const uint4 a = *reinterpret_cast<const uint4 *>(items + e), b = *reinterpret_cast<const uint4 *>(items + e + 4);
        const uint32_t it[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
        unsigned bad = 0u;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            ks[u] = (uint16_t)(it[u] >> 16);
            float g = 0.0f;
            if (e + u < m) {
                g = graw[it[u] & 0xffffu];
                if (!(g >= 0.0f) || g > 3.0e38f) bad |= 2u;
            }
            gs[u] = g;
        }
        return bad;
    }
    __device__ __forceinline__ uint16_t key_at(int p) const { return (uint16_t)(items[p] >> 16); }
};

template <int THREADS, int VEC>
__global__ void __launch_bounds__(THREADS, (THREADS <= 512 ? 2 : 1)) skim_sort16_kernel(ClusterArgs a)
{
    using K = KeyOps<uint16_t>;
    constexpr int ITEMS = VEC * 8;
    constexpr int CAP = THREADS * ITEMS;
    constexpr int NW = THREADS / 32;
    constexpr int WCHUNK = ITEMS * 32;          // positions owned by one warp in pass 1
    constexpr int EPT = D0 / THREADS;           // pass-0 counters scanned per thread
    static_assert(D0 % THREADS == 0 && THREADS >= D1, "thread count must divide 1024 and be >= 64");
    extern __shared__ __align__(16) unsigned char smem[];
    const Layout16 L = layout16(CAP, NW);
    uint32_t *buf = reinterpret_cast<uint32_t *>(smem + L.buf);
    float *graw = reinterpret_cast<float *>(smem + L.graw);
    uint32_t *C0 = reinterpret_cast<uint32_t *>(smem + L.uni);
    uint32_t *cnt1 = C0 + D0;
    uint32_t *dbase1 = reinterpret_cast<uint32_t *>(smem + L.dbase1);
    PhaseSmem &ps = *reinterpret_cast<PhaseSmem *>(smem + L.phase);
    uint64_t *mbar = reinterpret_cast<uint64_t *>(smem + L.mbar);
    uint32_t *scratch = reinterpret_cast<uint32_t *>(ps.segtot);   // free until the record pass

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int m = a.m;
    const int64_t row = a.row0 + blockIdx.x;
    const uint16_t *Wr = a.W + row * a.ld;
    const float *Gr = a.G + row * a.ld;

    // ---------------------------------------------------------------- set-up, importance row in flight
    if (tid == 0) {
        mbar_init(mbar, 1);
        ps.misc[0] = 0;
        ps.misc[1] = 0;
    }
    for (int d = tid; d < D0 + NW * D1; d += THREADS) C0[d] = 0u;
    __syncthreads();
    if (tid == 0) {
        const uint32_t bytes = (uint32_t)m * 4u;
        mbar_expect_tx(mbar, bytes);
        for (uint32_t o = 0; o < bytes; o += 32768u)
            bulk_load(reinterpret_cast<unsigned char *>(graw) + o, reinterpret_cast<const unsigned char *>(Gr) + o,
                      min(32768u, bytes - o), mbar);
    }

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
                const uint32_t lo = (e0 + 2 * u < m) ? Wr[e0 + 2 * u] : 0x7fffu;         // 0x7fff -> key 0xffff (padding)
                const uint32_t hi = (e0 + 2 * u + 1 < m) ? Wr[e0 + 2 * u + 1] : 0x7fffu;
                w[u] = lo | (hi << 16);
            }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            uint16_t h = (uint16_t)((u & 1) ? (w[u >> 1] >> 16) : (w[u >> 1] & 0xffffu));
            const bool real = e0 + u < m;
            if (real && (h & 0x7c00u) == 0x7c00u) bad |= 1u;
            if (h == 0x8000u) h = 0;                      // -0 and +0 are one value
            const uint32_t key = real ? (uint32_t)K::from_half_bits(h) : 0xffffu;
            item[j * 8 + u] = (key << 16) | (uint32_t)(real ? e0 + u : 0);
            atomicAdd(&C0[key & (D0 - 1)], 1u);
        }
    }
    if (bad) atomicOr(a.status, (unsigned long long)bad);
    __syncthreads();

    // ---------------------------------------------------------------- pass 0: scan, claim slots, scatter
    {
        uint32_t loc[EPT], s = 0;
#pragma unroll
        for (int u = 0; u < EPT; ++u) { loc[u] = C0[tid * EPT + u]; s += loc[u]; }
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
        for (int u = 0; u < EPT; ++u) { C0[tid * EPT + u] = run; run += loc[u]; }
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
        const uint32_t key = item[i] >> 16;
        const uint32_t pos = atomicAdd(&C0[key & (D0 - 1)], 1u);
        buf[pos] = item[i];
        atomicAdd(&cnt1[(pos / WCHUNK) * D1 + (key >> D0_BITS)], 1u);
    }
    __syncthreads();

    // ---------------------------------------------------------------- pass 1: scan, stable rank, scatter
    if (tid < D1) {
        uint32_t run = 0;
        for (int w = 0; w < NW; ++w) {
            const uint32_t c = cnt1[w * D1 + tid];
            cnt1[w * D1 + tid] = run;
            run += c;
        }
        // exclusive scan of the 64 digit totals by the first two warps
        uint32_t inc = run;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, inc, off);
            if (lane >= off) inc += t;
        }
        if (tid == 31) scratch[0] = inc;
        __syncwarp();
        dbase1[tid] = inc - run;
    }
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) item[i] = buf[warp * WCHUNK + i * 32 + lane];
    __syncthreads();
    if (tid >= 32 && tid < D1) dbase1[tid] += scratch[0];
    __syncthreads();
    {
        const unsigned lt_mask = (1u << lane) - 1u;
#pragma unroll
        for (int i = 0; i < ITEMS; ++i) {
            const uint32_t d = item[i] >> (16 + D0_BITS);
            unsigned peers = 0xffffffffu;
#pragma unroll
            for (int b = 0; b < D1_BITS; ++b) {
                const bool bit = (d >> b) & 1u;
                const unsigned bal = __ballot_sync(0xffffffffu, bit);
                peers &= bit ? bal : ~bal;
            }
            const uint32_t base = cnt1[warp * D1 + d];
            const unsigned rank = __popc(peers & lt_mask);
            __syncwarp();
            if (rank == 0) cnt1[warp * D1 + d] = base + __popc(peers);
            __syncwarp();
            buf[dbase1[d] + base + rank] = item[i];
        }
    }

    // ---------------------------------------------------------------- the importance row must have landed
    // (the vote below is also the barrier that ends pass 1)
    {
        const bool landed = mbar_wait_bounded(mbar, 0);
        if (!__syncthreads_and(landed ? 1 : 0)) {
            // the copy never arrived: flag it, give it one more bounded chance to drain, leave
            if (tid == 0) atomicOr(a.status, (unsigned long long)SKIM_STATUS_TIMEOUT);
            mbar_wait_bounded(mbar, 0);
            return;
        }
    }
    // ---------------------------------------------------------------- row record
    const SortedItems16 src{buf, graw};
    const int nd = write_row_record<uint16_t, THREADS>(a, src, ps);
    if (nd <= 16) {
        collect_distinct<uint16_t, THREADS>(src, m, nd, ps);
        write_distinct_values(a, nd, ps.dvals);
    }
}

struct Variant16 {
    int cap;
    int threads;
    void (*kernel)(ClusterArgs);
    int dev_set;    // device on which the shared-memory attribute below was last set (-1: none)
    int smem_set;
};

#define SKIM_V16(T, V) {T * V * 8, T, skim_sort16_kernel<T, V>, -1, 0}

Variant16 kVariants[] = {
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
    for (Variant16 &v : kVariants) {
        if (v.cap < cols) continue;
        const Layout16 L = layout16(v.cap, v.threads / 32);
        if (L.total > (size_t)ctx->max_smem_optin) continue;
        args.rec_stride = (long long)row_record(args.m).total;
        if (!launch) return SKIM_OK;
        const ClusterArgs a = args;
        if (v.dev_set != ctx->device || v.smem_set != (int)L.total) {
            SKIM_CUDA_OK(cudaFuncSetAttribute(v.kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L.total));
            v.dev_set = ctx->device;
            v.smem_set = (int)L.total;
        }
        v.kernel<<<(unsigned)rows, v.threads, L.total, ctx->stream>>>(a);
        SKIM_CUDA_OK(cudaGetLastError());
        ctx->launches += 1;
        return SKIM_OK;
    }
    return 1;
}
