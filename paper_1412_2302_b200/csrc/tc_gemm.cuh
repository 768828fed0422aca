// tcgen05 / TMEM / TMA GEMM core for sm_100a.
//
// A persistent kernel: each CTA (one per SM) walks a strided list of 128 x BN
// output tiles.  bf16 operands are staged in shared memory by TMA (128-byte
// swizzle) through a ring of `stages` buffers; fp32 accumulators live in tensor
// memory, double buffered, so the epilogue of tile i overlaps the main loop of
// tile i+1.  Warp roles: warp 0 = TMA producer (one lane), warp 1 = MMA issuer
// (the whole warp runs the loop, an elected lane issues) and TMEM owner, warps
// 2..5 = epilogue (each reads the 32 TMEM lanes of its quadrant and stores its
// rows through a swizzled shared-memory tile and TMA).  The producer and issuer
// loops carry no division or modulo: stage, phase, tap and chunk counters
// advance incrementally.  This file holds three kernels: gemm_kernel (FC
// backward), conv_kernel (convolution forward / backward-data, FC forward) and
// wgrad_kernel (convolution weight gradients).
// Three operand arrangements:
//   MODE_KK   A K-major, B K-major   conv fwd, conv bwd-data, FC fwd
//   MODE_KMN  A K-major, B MN-major  FC bwd-data (weights read untransposed)
//   MODE_MNMN A MN-major, B MN-major weight gradients (reduction over rows)
// A convolution is an implicit GEMM over a zero-padded flat NHWC grid: filter
// tap t reads the input rows of the output tile shifted by shift[t] rows, so
// every A tile is a plain 2-D TMA box; out-of-range rows are zero-filled by TMA.
// Every wait is bounded: on expiry the CTA raises *status and drains.
// conv_kernel also runs as CTA pairs (clusters of two, tcgen05.mma.cta_group::2: one instruction of the leader covers 128
// rows of each CTA), and gemm_kernel can apply the momentum update to the FC weights in its weight-gradient epilogue.
// All kernels are launched with programmatic stream serialization: they let the next launch of the stream start early
// (griddepcontrol.launch_dependents first thing) and wait for their predecessors (griddepcontrol.wait) after their
// barriers, tensor memory and descriptors are set up and before they touch global memory.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace tc {

// Optional per-role timeline of conv_kernel (compiled in only with -DALEXNET_TIMELINE, a separate build of the library for
// `python -m paper_1412_2302_b200.timeline`): every CTA records when it started, when its set-up was done, when its issuer
// entered and left the main loop and how many cycles it spent in each kind of wait, when its last store had completed and
// when it left.  16 slots per CTA; a launch overwrites the record of the launch before.
#ifdef ALEXNET_TIMELINE
__device__ long long g_timeline[160 * 16];
__device__ __forceinline__ long long gtime_ns() { long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
#define TL(...) __VA_ARGS__
#else
#define TL(...)
#endif

enum { MODE_KK = 0, MODE_KMN = 1, MODE_MNMN = 2 };
enum { EPI_BF16 = 0, EPI_F32 = 1 };
constexpr int kThreads = 192;
constexpr int kMaxTaps = 25;
constexpr int kMaxStages = 8;
constexpr long long kWaitBudgetCycles = 400000000LL;  // ~0.2 s at 2 GHz

struct GemmParams {
    CUtensorMap tmA, tmB, tmOut;   // tmOut: output as {columns, rows, splits}, box {128 bytes, 32, 1}, when tma_store
    int tma_store;
    // MODE_MNMN with fuse_update: the tile is an FC weight gradient and the epilogue applies the momentum update to the
    // weights in place instead of storing the gradient: tmW / tmV = fp32 weights and momentum ({32, 32, 1} boxes, 128-byte
    // swizzle), tmS = bf16 copy of the weights ({32, 32, 1} boxes, no swizzle); upd_d = lr * weight decay
    CUtensorMap tmW, tmV, tmS;
    int fuse_update;
    float upd_lr, upd_mu, upd_d;
    int mode, epi;
    int m_tiles, n_tiles, groups, taps_grid, splits;  // tile decomposition (m fastest)
    int tiles_total;
    int BN;            // MMA N (multiple of 16, <= 256)
    int kk;            // K=16 MMAs per stage (<= 4)
    int chunks;        // MODE_KK: 64-element K chunks per tap
    int steps_total;   // k-steps over the whole reduction (split evenly over `splits`)
    int steps_per_split;
    int stages;        // smem ring depth
    int a_x0, a_gx;    // A column origin and per-group column stride
    int b_gx;          // MODE_MNMN: B per-group column stride
    int b_tap_rows, b_g_rows;  // MODE_KK: B row = tap*b_tap_rows + g*b_g_rows + n0
    int shift[kMaxTaps];
    // epilogue
    int M_total;       // valid rows (MODE_KK/KMN); MODE_MNMN: valid rows per group (m_valid)
    int n_valid;       // valid columns per group
    int ldo;           // output row pitch (elements)
    int out_gx;        // per-group output column offset (MODE_KK/KMN) or row offset (MODE_MNMN)
    long long split_stride, tap_stride;  // EPI_F32 partial strides (elements)
    int Hp, Wp, H, W;  // flat-grid geometry for zeroing pad rows (Hp = 0: none)
    int relu;
    float mask_scale;
    const float* bias;           // [groups*n_valid...] indexed by output column, or nullptr
    const __nv_bfloat16* mask;   // same layout as out; out = mask>0 ? v*mask_scale : 0
    void* out;
    int* status;
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// bounded wait: returns false when the cycle budget ran out or another role aborted.  It polls with the
// non-blocking test_wait first: a thread suspended inside try_wait was seen to resume late, which starves the
// producer / issuer hand-over of a pipelined ring; only a long wait falls back to the suspending form.
__device__ __forceinline__ bool mbar_wait_budget(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long budget) {
    #pragma unroll 1
    for (int i = 0; i < 4096; ++i)
        if (mbar_test_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        #pragma unroll 1
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > budget) { *abort_flag = 1; return false; }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    return mbar_wait_budget(bar, parity, abort_flag, kWaitBudgetCycles);
}
// the same for a whole warp that must take one decision (all lanes wait; any failure fails all)
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                               long long budget = kWaitBudgetCycles) {
    return __all_sync(0xffffffffu, mbar_wait_budget(bar, parity, abort_flag, budget));
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, int x, int y, int z, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* tm) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(tm) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// The issuer WARP runs its loop convergently (uniform operands stay in uniform registers) and one elected lane
// issues.  In straight-line groups one warp issues at the tensor pipe's rate (measured 64 cycles per instruction at
// N = 128, 128 at N = 256); what an instruction costs is max(N / 2, (4096 + 32 N) / 128) cycles: its A slice (4 KB) and
// B slice are read from shared memory at 128 bytes per cycle, so N < 128 does not get faster than about 45 cycles and
// N = 128 leaves the shared memory no bandwidth for the TMA writes that run beside it.
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %4, 0;\n\telect.sync _|q, 0xffffffff;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("{\n\t.reg .pred q;\n\telect.sync _|q, 0xffffffff;\n\t"
                 "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(bar) : "memory");
}
// ---- CTA pairs (cta_group::2): one instruction of the leader CTA (cluster rank 0) multiplies a 256-row A (128 rows
// from each CTA's shared memory) by an N-column B (N/2 columns from each CTA) into 128 TMEM lanes of each CTA.
__device__ __forceinline__ uint32_t cluster_ctarank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
// shared::cluster address of the same shared-memory offset in the CTA of the given cluster rank
__device__ __forceinline__ uint32_t mapa_u32(uint32_t addr, uint32_t rank) {
    uint32_t r; asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank)); return r;
}
// all threads of all CTAs of the cluster
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void fence_acq_rel_cluster() { asm volatile("fence.acq_rel.cluster;" ::: "memory"); }
// load into this CTA's shared memory, completion counted on a barrier of either CTA of the pair (cluster address)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t cluster_bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
template <int CG>
__device__ __forceinline__ void umma_cg(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
    if (CG == 1) { umma(d_tmem, adesc, bdesc, idesc, accum); return; }
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %4, 0;\n\telect.sync _|q, 0xffffffff;\n\t"
        "@q tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum) : "memory");
}
// completion of the issuing thread's MMAs arrives on the barrier at this shared-memory offset in both CTAs of the pair
template <int CG>
__device__ __forceinline__ void umma_commit_cg(uint32_t bar) {
    if (CG == 1) { umma_commit(bar); return; }
    const uint16_t both = 3;
    asm volatile("{\n\t.reg .pred q;\n\telect.sync _|q, 0xffffffff;\n\t"
                 "@q tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;\n\t}"
                 ::"r"(bar), "h"(both) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
// TMA store of one box from shared memory (bulk async-group completion)
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* tm, uint32_t src, int x, int y, int z) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
                 ::"l"(tm), "r"(src), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor version 1
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFF) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// instruction descriptor: bf16 x bf16 -> fp32, M = 128 (256 for a CTA pair: 128 rows per CTA)
__device__ __forceinline__ uint32_t instr_desc(int N, int a_mn, int b_mn, int M = 128) {
    uint32_t d = 0;
    d |= 1u << 4;                 // D format fp32
    d |= 1u << 7;                 // A bf16
    d |= 1u << 10;                // B bf16
    d |= (uint32_t)a_mn << 15;    // A major (0 = K)
    d |= (uint32_t)b_mn << 16;    // B major
    d |= (uint32_t)(N >> 3) << 17;
    d |= (uint32_t)(M >> 4) << 24;
    return d;
}

// One 16-column slice of an accumulator row: bias, ReLU, pad-row zeroing, ReLU/dropout
// mask, conversion and store.  P is a parameter struct with the epilogue fields.
template <typename P>
__device__ __forceinline__ void epi_chunk(const P& p, uint32_t* v, bool zero, bool pad_row, long long row_off, int col0, int g) {
    if (zero) {
        #pragma unroll
        for (int k = 0; k < 16; ++k) v[k] = 0u;
    }
    if (p.epi == EPI_F32) {
        float* o = (float*)p.out + row_off + col0;
        if (col0 + 16 <= p.n_valid) {
            #pragma unroll
            for (int k = 0; k < 16; k += 4)
                *(float4*)(o + k) = make_float4(__uint_as_float(v[k]), __uint_as_float(v[k + 1]),
                                                __uint_as_float(v[k + 2]), __uint_as_float(v[k + 3]));
        } else {
            for (int k = 0; k < 16; ++k)
                if (col0 + k < p.n_valid) o[k] = __uint_as_float(v[k]);
        }
        return;
    }
    __nv_bfloat16* o = (__nv_bfloat16*)p.out + row_off + col0;
    float f[16];
    #pragma unroll
    for (int k = 0; k < 16; ++k) {
        float t = __uint_as_float(v[k]);
        if (p.bias) t += p.bias[g * p.out_gx + min(col0 + k, p.n_valid - 1)];
        if (p.relu) t = fmaxf(t, 0.f);
        f[k] = pad_row ? 0.f : t;
    }
    if (p.mask) {
        const __nv_bfloat16* mk = p.mask + row_off + col0;
        if (col0 + 16 <= p.n_valid) {
            uint4 m0v = *(const uint4*)mk, m1v = *(const uint4*)(mk + 8);
            const __nv_bfloat16* mm = (const __nv_bfloat16*)&m0v;
            const __nv_bfloat16* mn = (const __nv_bfloat16*)&m1v;
            #pragma unroll
            for (int k = 0; k < 8; ++k) {
                f[k] = __bfloat162float(mm[k]) > 0.f ? f[k] * p.mask_scale : 0.f;
                f[k + 8] = __bfloat162float(mn[k]) > 0.f ? f[k + 8] * p.mask_scale : 0.f;
            }
        } else {
            for (int k = 0; k < 16; ++k)
                if (col0 + k < p.n_valid)
                    f[k] = __bfloat162float(mk[k]) > 0.f ? f[k] * p.mask_scale : 0.f;
        }
    }
    if (col0 + 16 <= p.n_valid) {
        uint32_t w[8];
        #pragma unroll
        for (int k = 0; k < 8; ++k) {
            __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * k], f[2 * k + 1]);
            w[k] = *(uint32_t*)&h;
        }
        *(uint4*)o = make_uint4(w[0], w[1], w[2], w[3]);
        *(uint4*)(o + 8) = make_uint4(w[4], w[5], w[6], w[7]);
    } else {
        for (int k = 0; k < 16; ++k)
            if (col0 + k < p.n_valid) o[k] = __float2bfloat16_rn(f[k]);
    }
}

// Staged epilogue: one warp turns 32 accumulator rows x one 128-byte slab (64 bf16 or 32 fp32 columns) into a
// 128-byte-swizzled 4 KB tile in shared memory and stores it with one TMA box; rows and columns outside the output
// tensor are clipped by TMA.  Each epilogue warp owns one kEpiStageBytes tile: before rewriting it the warp waits
// until the previous store has finished reading it (wait_group.read 0), which the TMEM loads and the arithmetic of
// the next slab overlap.
constexpr uint32_t kEpiStageBytes = 4096;
template <typename P>
__device__ __forceinline__ void epi_slab(const P& p, uint32_t tmem_addr, bool pad_row, long long row_off, int col0, int g,
                                         int x, int y, int z, uint32_t stage, int lane) {
    uint32_t w[32];   // the packed 128-byte row
    if (p.epi == EPI_F32) {
        tmem_ld32(tmem_addr, w);
        tmem_ld_wait();
    } else {
        const float* bp = p.bias ? p.bias + g * p.out_gx + col0 : nullptr;
        const uint4* mp = p.mask ? (const uint4*)(p.mask + row_off + col0) : nullptr;
        #pragma unroll
        for (int half = 0; half < 2; ++half) {
            uint32_t v[32];
            tmem_ld32(tmem_addr + 32u * half, v);
            tmem_ld_wait();
            #pragma unroll
            for (int qq = 0; qq < 4; ++qq) {       // four 16-byte chunks of eight columns
                const int q = 4 * half + qq;
                float f[8];
                #pragma unroll
                for (int k = 0; k < 8; ++k) f[k] = __uint_as_float(v[8 * qq + k]);
                if (bp) {
                    const float4 b0 = __ldg((const float4*)(bp + 8 * q)), b1 = __ldg((const float4*)(bp + 8 * q + 4));
                    f[0] += b0.x; f[1] += b0.y; f[2] += b0.z; f[3] += b0.w; f[4] += b1.x; f[5] += b1.y; f[6] += b1.z; f[7] += b1.w;
                }
                if (p.relu) {
                    #pragma unroll
                    for (int k = 0; k < 8; ++k) f[k] = fmaxf(f[k], 0.f);
                }
                if (mp) {
                    const uint4 mv = __ldg(mp + q);
                    const __nv_bfloat162* mh = (const __nv_bfloat162*)&mv;
                    #pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const float2 m2 = __bfloat1622float2(mh[k]);
                        f[2 * k] = m2.x > 0.f ? f[2 * k] * p.mask_scale : 0.f;
                        f[2 * k + 1] = m2.y > 0.f ? f[2 * k + 1] * p.mask_scale : 0.f;
                    }
                }
                #pragma unroll
                for (int k = 0; k < 4; ++k) {
                    __nv_bfloat162 hh = __floats2bfloat162_rn(pad_row ? 0.f : f[2 * k], pad_row ? 0.f : f[2 * k + 1]);
                    w[4 * q + k] = *(uint32_t*)&hh;
                }
            }
        }
    }
    if (lane == 0) bulk_wait_read_0();
    __syncwarp();
    const uint32_t rowp = stage + (uint32_t)lane * 128u;
    #pragma unroll
    for (int q = 0; q < 8; ++q)
        st_shared_v4(rowp + (uint32_t)((q ^ (lane & 7)) << 4), w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
    fence_async_smem();
    __syncwarp();
    if (lane == 0) { tma_store_3d(&p.tmOut, stage, x, y, z); bulk_commit(); }
}

// Failure-detection self-test: one warp waits, through the bounded wait above, on a barrier nothing arrives on.  The
// wait runs out after `budget` cycles, the warp raises the status word as the GEMM kernels do, and returns.
__global__ void __launch_bounds__(32) wait_probe_kernel(int* status, long long budget) {
    kn::pdl_sync();
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const bool ok = mbar_wait_warp(smem_u32(&bar), 0u, &abort_flag, budget);
    if (!ok && threadIdx.x == 0 && status) atomicExch(status, 1);
}

constexpr int kABytes = 128 * 128;  // 128 rows x 64 bf16, or 2 boxes of 64 x 64

__host__ __device__ inline int b_stage_bytes(int mode, int BN) {
    return mode == MODE_KK ? BN * 128 : ((BN + 63) / 64) * 8192;
}
// per epilogue warp of a fused-update kernel: kUpdBufs {w tile, v tile} pairs of 4 KB each and two 2 KB bf16 tiles
constexpr int kUpdBufs = 5;
constexpr uint32_t kUpdWarpBytes = kUpdBufs * 8192 + 2 * 2048;
inline size_t smem_bytes(int mode, int BN, int stages, bool fuse_update = false) {
    return 1024 + (size_t)stages * (kABytes + b_stage_bytes(mode, BN)) + (fuse_update ? 4 * kUpdWarpBytes : 4 * kEpiStageBytes) + 512;
}

// position of a CTA in the tile list; tiles are numbered with m fastest, then
// n tile, group, tap (weight gradients), k split
struct TileCursor {
    int m_tile, rest;          // rest = tile / m_tiles
    int n_tile, g, tap_g, z;   // decoded from rest
    __device__ __forceinline__ void decode(const GemmParams& p) {
        int r = rest;
        n_tile = r % p.n_tiles; r /= p.n_tiles;
        g = r % p.groups; r /= p.groups;
        tap_g = r % p.taps_grid;
        z = r / p.taps_grid;
    }
    __device__ __forceinline__ void init(const GemmParams& p) {
        m_tile = blockIdx.x % p.m_tiles;
        rest = blockIdx.x / p.m_tiles;
        decode(p);
    }
    __device__ __forceinline__ void next(const GemmParams& p) {
        m_tile += gridDim.x;
        if (m_tile >= p.m_tiles) {
            do { m_tile -= p.m_tiles; ++rest; } while (m_tile >= p.m_tiles);
            decode(p);
        }
    }
};

__global__ void __launch_bounds__(kThreads, 1) gemm_kernel(const __grid_constant__ GemmParams p) {
    kn::pdl_trigger();
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const int bbytes = b_stage_bytes(p.mode, p.BN);
    const int stage_bytes = kABytes + bbytes;
    const int stages = p.stages;
    // epilogue staging (4 warps x kEpiStageBytes), then barriers: full[8] @0, empty[8] @64, acc_full[2] @128,
    // acc_empty[2] @144, tmem slot @160, abort flag @168
    const uint32_t epi_stage0 = base + stages * stage_bytes;
    const uint32_t upd0 = epi_stage0 + (p.fuse_update ? 0u : 4u * kEpiStageBytes);   // fused update: per-warp tiles instead of the staging
    const uint32_t bar_base = upd0 + (p.fuse_update ? 4u * kUpdWarpBytes : 0u);  // ... + per-warp load barriers [4][kUpdBufs] @176
    uint8_t* gen = smem_raw + (bar_base - raw);
    volatile int* abort_flag = (volatile int*)(gen + 168);
    volatile uint32_t* tmem_slot = (volatile uint32_t*)(gen + 160);
    const uint32_t full0 = bar_base, empty0 = bar_base + 64u, accf0 = bar_base + 128u, acce0 = bar_base + 144u;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    uint32_t ncols = 32;
    while ((int)ncols < 2 * p.BN) ncols <<= 1;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < stages; ++s) { mbar_init(full0 + 8u * s, 1); mbar_init(empty0 + 8u * s, 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(accf0 + 8u * s, 1); mbar_init(acce0 + 8u * s, 128); }
        for (int s = 0; s < 4 * kUpdBufs; ++s) mbar_init(bar_base + 176u + 8u * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tma_prefetch_desc(&p.tmA);
        tma_prefetch_desc(&p.tmB);
    }
    if (warp == 1) tmem_alloc(smem_u32((const void*)tmem_slot), ncols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    kn::pdl_wait();        // barriers, TMEM and descriptors are set up; global memory is touched from here on
    const int per = p.steps_per_split;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const uint32_t tx = (uint32_t)stage_bytes;
            const int nb = (p.BN + 63) >> 6;
            TileCursor tc; tc.init(p);
            int st = 0; uint32_t ph = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.tiles_total && ok; tile += gridDim.x, tc.next(p)) {
                const int m0 = tc.m_tile * 128, n0 = tc.n_tile * p.BN;
                const int s_begin = tc.z * per;
                const int nsteps = min(p.steps_total, s_begin + per) - s_begin;
                if (p.mode == MODE_KK) {
                    int tap = 0, ch = s_begin;
                    if (p.chunks < p.steps_total && s_begin > 0) { tap = s_begin / p.chunks; ch = s_begin - tap * p.chunks; }
                    const int xa = p.a_x0 + tc.g * p.a_gx, yb = tc.g * p.b_g_rows + n0;
                    for (int i = 0; i < nsteps; ++i) {
                        if (!(ok = mbar_wait(empty0 + 8u * st, ph ^ 1u, abort_flag))) break;
                        const uint32_t sa = base + st * stage_bytes, fb = full0 + 8u * st;
                        mbar_expect_tx(fb, tx);
                        tma_load_2d(sa, &p.tmA, xa + ch * 64, m0 + p.shift[tap], fb);
                        tma_load_2d(sa + kABytes, &p.tmB, ch * 64, tap * p.b_tap_rows + yb, fb);
                        if (++ch == p.chunks) { ch = 0; ++tap; }
                        if (++st == stages) { st = 0; ph ^= 1u; }
                    }
                } else if (p.mode == MODE_KMN) {
                    for (int i = 0; i < nsteps; ++i) {
                        if (!(ok = mbar_wait(empty0 + 8u * st, ph ^ 1u, abort_flag))) break;
                        const uint32_t sa = base + st * stage_bytes, fb = full0 + 8u * st;
                        const int q = (s_begin + i) * 64;
                        mbar_expect_tx(fb, tx);
                        tma_load_2d(sa, &p.tmA, q, m0, fb);
                        for (int j = 0; j < nb; ++j) tma_load_2d(sa + kABytes + j * 8192, &p.tmB, n0 + 64 * j, q, fb);
                        if (++st == stages) { st = 0; ph ^= 1u; }
                    }
                } else {
                    const int xa = tc.g * p.a_gx + m0, xb = tc.g * p.b_gx + n0, sh = p.shift[tc.tap_g];
                    for (int i = 0; i < nsteps; ++i) {
                        if (!(ok = mbar_wait(empty0 + 8u * st, ph ^ 1u, abort_flag))) break;
                        const uint32_t sa = base + st * stage_bytes, fb = full0 + 8u * st;
                        const int q = (s_begin + i) * 64;
                        mbar_expect_tx(fb, tx);
                        tma_load_2d(sa, &p.tmA, xa, q, fb);
                        tma_load_2d(sa + 8192, &p.tmA, xa + 64, q, fb);
                        for (int j = 0; j < nb; ++j) tma_load_2d(sa + kABytes + j * 8192, &p.tmB, xb + 64 * j, q + sh, fb);
                        if (++st == stages) { st = 0; ph ^= 1u; }
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (whole warp, one elected lane issues)
        {
            const int a_mn = p.mode == MODE_MNMN, b_mn = p.mode != MODE_KK;
            const uint32_t idesc = instr_desc(p.BN, a_mn, b_mn);
            const uint32_t a_adv = a_mn ? 2048u : 32u, b_adv = b_mn ? 2048u : 32u;
            const uint32_t a_lbo = a_mn ? 8192u : 16u, b_lbo = b_mn ? 8192u : 16u;
            const int kk = p.kk;
            TileCursor tc; tc.init(p);
            int st = 0; uint32_t ph = 0;
            int ab = 0; uint32_t aph = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.tiles_total && ok; tile += gridDim.x, tc.next(p)) {
                const int s_begin = tc.z * per;
                const int nsteps = min(p.steps_total, s_begin + per) - s_begin;
                if (!(ok = mbar_wait_warp(acce0 + 8u * ab, aph ^ 1u, abort_flag))) break;
                tc_fence_after();
                const uint32_t d = tmem + (uint32_t)(ab * p.BN);
                for (int i = 0; i < nsteps; ++i) {
                    if (!(ok = mbar_wait_warp(full0 + 8u * st, ph, abort_flag))) break;
                    tc_fence_after();
                    const uint32_t sa = base + st * stage_bytes, sb = sa + kABytes;
                    #pragma unroll 4
                    for (int j = 0; j < kk; ++j)
                        umma(d, smem_desc(sa + j * a_adv, a_lbo, 1024), smem_desc(sb + j * b_adv, b_lbo, 1024),
                             idesc, (i > 0 || j > 0) ? 1u : 0u);
                    umma_commit(empty0 + 8u * st);
                    if (++st == stages) { st = 0; ph ^= 1u; }
                }
                if (!ok) break;
                umma_commit(accf0 + 8u * ab);
                if (++ab == 2) { ab = 0; aph ^= 1u; }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue
        const int quad = warp & 3;
        const int r = quad * 32 + lane;          // row within the tile = TMEM lane
        TileCursor tc; tc.init(p);
        int ab = 0; uint32_t aph = 0;
        bool ok = true;
        if (p.fuse_update) {
            // FC weight gradient consumed in place: for every 32 x 32 slab of the tile this warp loads the weights and the
            // momentum by TMA (kUpdBufs - 2 = three slabs ahead of the arithmetic), applies v <- mu v - d w - lr g, w <- w + v to the
            // accumulator values and stores w, v and the bf16 copy of w by TMA.  A buffer (of kUpdBufs = 5) is reloaded
            // only after the stores issued from it two slabs earlier have finished reading (wait_group.read 1).
            const uint32_t ureg = upd0 + (uint32_t)quad * kUpdWarpBytes, ub0 = bar_base + 176u + (uint32_t)quad * (8u * kUpdBufs);
            TileCursor tp = tc;                      // prefetch cursor
            int tile = blockIdx.x, c = 0, q = 0;     // tile, column and count of the slab being processed
            int ptile = blockIdx.x, pc = 0, pq = 0;  // the same for the slab whose loads are issued next
            auto issue_loads = [&]() {
                const uint32_t bar = ub0 + 8u * (uint32_t)(pq % kUpdBufs), dst = ureg + (uint32_t)(pq % kUpdBufs) * 8192u;
                const int x = tp.n_tile * p.BN + pc, y = tp.m_tile * 128 + quad * 32;
                mbar_expect_tx(bar, 8192u);
                tma_load_3d(dst, &p.tmW, x, y, 0, bar);
                tma_load_3d(dst + 4096u, &p.tmV, x, y, 0, bar);
                ++pq; pc += 32;
                if (pc == p.BN) { pc = 0; ptile += gridDim.x; tp.next(p); }
            };
            if (lane == 0) {
                #pragma unroll 1
                for (int i = 0; i < kUpdBufs - 2 && ptile < p.tiles_total; ++i) issue_loads();
            }
            __syncwarp();
            while (tile < p.tiles_total) {
                if (lane == 0) { bulk_wait_read_1(); if (ptile < p.tiles_total) issue_loads(); }
                __syncwarp();
                if (c == 0) {
                    if (!(ok = mbar_wait(accf0 + 8u * ab, aph, abort_flag))) break;
                    tc_fence_after();
                }
                uint32_t g[32];
                tmem_ld32(tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)(ab * p.BN + c), g);
                tmem_ld_wait();
                if (!(ok = mbar_wait(ub0 + 8u * (uint32_t)(q % kUpdBufs), (uint32_t)((q / kUpdBufs) & 1), abort_flag))) break;
                const uint32_t buf = ureg + (uint32_t)(q % kUpdBufs) * 8192u, rowp = buf + (uint32_t)lane * 128u;
                const uint32_t sbuf = ureg + (uint32_t)kUpdBufs * 8192u + (uint32_t)(q & 1) * 2048u;
                uint32_t sh[16];
                #pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint32_t ch = (uint32_t)((j ^ (lane & 7)) << 4);
                    float4 w4, v4;
                    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(w4.x), "=f"(w4.y), "=f"(w4.z), "=f"(w4.w) : "r"(rowp + ch));
                    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v4.x), "=f"(v4.y), "=f"(v4.z), "=f"(v4.w) : "r"(rowp + 4096u + ch));
                    kn::sgd_step(w4.x, v4.x, __uint_as_float(g[4 * j]), p.upd_d, p.upd_lr, p.upd_mu);
                    kn::sgd_step(w4.y, v4.y, __uint_as_float(g[4 * j + 1]), p.upd_d, p.upd_lr, p.upd_mu);
                    kn::sgd_step(w4.z, v4.z, __uint_as_float(g[4 * j + 2]), p.upd_d, p.upd_lr, p.upd_mu);
                    kn::sgd_step(w4.w, v4.w, __uint_as_float(g[4 * j + 3]), p.upd_d, p.upd_lr, p.upd_mu);
                    st_shared_v4(rowp + ch, __float_as_uint(w4.x), __float_as_uint(w4.y), __float_as_uint(w4.z), __float_as_uint(w4.w));
                    st_shared_v4(rowp + 4096u + ch, __float_as_uint(v4.x), __float_as_uint(v4.y), __float_as_uint(v4.z), __float_as_uint(v4.w));
                    __nv_bfloat162 lo = __floats2bfloat162_rn(w4.x, w4.y), hi = __floats2bfloat162_rn(w4.z, w4.w);
                    sh[2 * j] = *(uint32_t*)&lo; sh[2 * j + 1] = *(uint32_t*)&hi;
                }
                #pragma unroll
                for (int j = 0; j < 4; ++j)
                    st_shared_v4(sbuf + (uint32_t)lane * 64u + 16u * j, sh[4 * j], sh[4 * j + 1], sh[4 * j + 2], sh[4 * j + 3]);
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                    const int x = tc.n_tile * p.BN + c, y = tc.m_tile * 128 + quad * 32;
                    tma_store_3d(&p.tmW, buf, x, y, 0);
                    tma_store_3d(&p.tmV, buf + 4096u, x, y, 0);
                    tma_store_3d(&p.tmS, sbuf, x, y, 0);
                    bulk_commit();
                }
                ++q; c += 32;
                if (c == p.BN) {
                    tc_fence_before();
                    mbar_arrive(acce0 + 8u * ab);
                    if (++ab == 2) { ab = 0; aph ^= 1u; }
                    c = 0; tile += gridDim.x; tc.next(p);
                }
            }
            if (lane == 0) bulk_wait_all();
        } else
        for (int tile = blockIdx.x; tile < p.tiles_total && ok; tile += gridDim.x, tc.next(p)) {
            const int m0 = tc.m_tile * 128, n0 = tc.n_tile * p.BN, g = tc.g;
            const int s_begin = tc.z * per;
            const int nsteps = min(p.steps_total, s_begin + per) - s_begin;
            bool row_ok, pad_row = false;
            long long row_off;
            if (p.mode == MODE_MNMN) {
                row_ok = (m0 + r) < p.M_total;
                row_off = (long long)tc.z * p.split_stride + (long long)tc.tap_g * p.tap_stride +
                          (long long)(g * p.out_gx + m0 + r) * p.ldo;
            } else {
                const int row = m0 + r;
                row_ok = row < p.M_total;
                if (p.Hp > 0) {
                    const int x = row % p.Wp, y = (row / p.Wp) % p.Hp;
                    pad_row = (x >= p.W) || (y >= p.H);
                }
                row_off = (long long)tc.z * p.split_stride + (long long)row * p.ldo + g * p.out_gx;
            }
            if (!(ok = mbar_wait(accf0 + 8u * ab, aph, abort_flag))) break;
            tc_fence_after();
            const uint32_t t0 = tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)(ab * p.BN);
            if (p.tma_store) {
                const int slab = p.epi == EPI_F32 ? 32 : 64;
                for (int c = 0; c < p.BN; c += slab) {
                    epi_slab(p, t0 + (uint32_t)c, pad_row, row_off, n0 + c, g, g * p.out_gx * (p.mode != MODE_MNMN) + n0 + c,
                             m0 + quad * 32 + (p.mode == MODE_MNMN ? g * p.out_gx : 0), tc.z,
                             epi_stage0 + (uint32_t)quad * kEpiStageBytes, lane);
                }
            } else {
                for (int c = 0; c < p.BN; c += 16) {
                    uint32_t v[16];
                    tmem_ld16(t0 + (uint32_t)c, v);
                    tmem_ld_wait();
                    if (!row_ok) continue;
                    epi_chunk(p, v, nsteps <= 0, pad_row, row_off, n0 + c, g);
                }
            }
            // this accumulator buffer may be overwritten by the next tile but one
            tc_fence_before();
            mbar_arrive(acce0 + 8u * ab);
            if (++ab == 2) { ab = 0; aph ^= 1u; }
        }
        if (!p.fuse_update && p.tma_store && lane == 0) bulk_wait_all();
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // a wait expired: give in-flight copies time to land before the block retires
        if (threadIdx.x == 0 && p.status) atomicExch(p.status, 1);
        long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) { }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, ncols);
    }
}

// ===========================================================================
// Convolution / FC-forward kernel (both operands K-major) with operand reuse.
//
// One tile = MH x 128 output rows by BN output channels (MH = 1, 2 or 4).  For
// each filter row ky and each 64-channel chunk the producer loads ONE "halo" of
// activation rows (MH boxes of a_box_rows rows, covering MH*128 + kw - 1
// consecutive rows of the flat grid); the kw taps of that filter row read it at
// row offsets tap_off[kx] through shared-memory descriptors whose start address
// is advanced by whole 128-byte rows.  Every weight tile (BN rows x 64 channels
// of one tap) is used by the MH row halves.  Activations and weights therefore
// travel in separate rings: an A stage lives for kw B stages.
// Each 128-row half has its own issuer warp (they write disjoint accumulators
// and share the weight tiles, which halves the weight traffic into shared
// memory per instruction).
// Warps: 0 and 1 = TMA producers (halos, weight groups), 2..MH+1 = MMA issuers, then four epilogue warps.
// Accumulators: MH x BN columns per buffer, two buffers when they fit in the
// 512 TMEM columns.
struct ConvParams {
    CUtensorMap tmA, tmB, tmOut;   // tmOut: output as {columns, rows, splits}, box {128 bytes, 32, 1}, when tma_store
    int tma_store;
    int m_tiles, n_tiles, groups, splits;   // tile decomposition (m fastest, then n, group, k split)
    int tiles_total;
    int b_res;          // 1: all kh*kw weight tiles of the layer fit in one group slot and stay there for the whole CTA (one
                        // n tile, one group, one chunk, no split: conv1), loaded once instead of once per tile
    int cg;             // 1, or 2: CTA pairs (clusters of two) work on tiles of 2 x MH halves with cta_group::2 instructions
    int MH;             // 128-row halves per tile and CTA (1, 2 or 4)
    int BN, kk;         // MMA N (multiple of 16, <= 256); K=16 MMAs per weight stage (<= 4)
    int kh, kw;         // filter rows; taps per filter row
    int cpg;            // 64-channel chunks per A stage: 1 for convolutions; 2 for FC layers (kw = 1), whose A stage then holds
                        // cpg activation boxes side by side and whose weight group holds the cpg matching weight tiles
    int tpg;            // taps per weight group (one barrier pair per group): kw, or 3 for a five-tap row (groups 3 + 2)
    int chunks;         // 64-channel chunks
    int asteps_total;   // kh * chunks, split evenly over `splits`
    int asteps_per_split;
    int epi_sets;       // 1 or 2 sets of four epilogue warps; with two, the (row half, column slab) units of a tile alternate between them
    int a_stages, b_stages, acc_stages;   // b_stages counts groups of kw weight tiles (one barrier pair per group)
    int a_box_rows;     // rows per activation box (128, or 136 when kw > 1)
    int a_x0, a_gx;     // A column origin and per-group column stride
    int b_tap_rows, b_g_rows;   // B row = (ky*kw+kx)*b_tap_rows + g*b_g_rows + n0
    int halo_shift[5];  // per ky: first halo row relative to the tile's first output row
    int tap_off[5];     // per kx: row offset of the tap inside the halo
    // epilogue (same meaning as in GemmParams)
    int epi, M_total, n_valid, ldo, out_gx;
    long long split_stride;
    int Hp, Wp, H, W, relu;
    float mask_scale;
    const float* bias;
    const __nv_bfloat16* mask;
    void* out;
    int* status;
    // FC forward with the split-K reduction inside the kernel: the `zcluster` CTAs of a thread-block cluster are the k splits
    // of one 128-row x BN tile (one tile per CTA, m_tiles == 1).  Each leaves its fp32 partial tile in its own shared
    // memory; after a cluster barrier CTA z adds rows [z * 128 / zcluster, ...) of all partials in split order through
    // distributed shared memory and applies bias, ReLU and dropout (the arithmetic of fc_reduce_fwd_kernel, so the result
    // is bit-identical to the two-launch form), writing the layer's bf16 output and its keep mask.  0: off.
    int zcluster;
    int fc_relu, fc_dropout;       // fc_dropout: 0 none, 1 mask from the hash, 2 evaluation (expectation of the mask)
    uint64_t fc_key; uint32_t fc_thr24; float fc_scale;
    __nv_bfloat16* fc_out; uint8_t* fc_keep;
    // 1: the weight producer does not wait for the kernel before this one in the stream (programmatic dependent launch):
    // the caller knows that no kernel that may still be running writes the weights, so their first stages load while
    // the predecessor drains.  Every other role waits as usual.
    int early_b;
};
constexpr int kZcPitch = 132;      // floats per row of the partial tile in shared memory (128 + 4: conflict-free float4 rows)

constexpr int kConvMaxThreads = 32 * 12;
inline int conv_threads(const ConvParams& p) { return 32 * (2 + p.MH + 4 * p.epi_sets); }
inline size_t conv_smem_bytes(const ConvParams& p) {
    return 1024 + (size_t)p.a_stages * p.MH * p.cpg * p.a_box_rows * 128 + (size_t)p.b_stages * p.tpg * (p.BN / p.cg) * 128 + 4 * p.epi_sets * kEpiStageBytes + 512;
}

// tile cursor shared by the roles (m fastest, then n tile, group, split)
struct ConvCursor {
    int m_tile, rest, n_tile, g, z;
    __device__ __forceinline__ void decode(const ConvParams& q) {
        int r = rest;
        n_tile = r % q.n_tiles; r /= q.n_tiles;
        g = r % q.groups;
        z = r / q.groups;
    }
    int stride;      // tile-list stride: CTAs of the grid, or CTA pairs
    __device__ __forceinline__ void init(const ConvParams& q, int first, int step) {
        stride = step;
        m_tile = first % q.m_tiles; rest = first / q.m_tiles; decode(q);
    }
    __device__ __forceinline__ void next(const ConvParams& q) {
        m_tile += stride;
        if (m_tile >= q.m_tiles) {
            do { m_tile -= q.m_tiles; ++rest; } while (m_tile >= q.m_tiles);
            decode(q);
        }
    }
};

// MMAs of one filter row (KW taps x KK K=16 steps) on one accumulator, fully unrolled; descriptors in 16-byte units
template <int KW, int KK, int CG>
__device__ __forceinline__ void issue_row(uint32_t d, uint64_t ad, uint64_t bd, uint32_t b_tile16, const int* tap_off,
                                          uint32_t idesc, uint32_t accum) {
    #pragma unroll
    for (int kx = 0; kx < KW; ++kx) {
        const uint64_t a_tap = ad + (uint64_t)(tap_off[kx] * 8);      // one row = 128 bytes = 8 units
        #pragma unroll
        for (int j = 0; j < KK; ++j)
            umma_cg<CG>(d, a_tap + (uint64_t)(2 * j), bd + (uint64_t)(kx * b_tile16 + 2 * j), idesc, (kx == 0 && j == 0) ? accum : 1u);
    }
}

// CG = 2: the CTAs of a pair (cluster of two) share one tile list.  A tile is 2 x MH x 128 rows; CTA `rank` owns the
// halves rank*MH .. rank*MH+MH-1, loads their halos and BN/2 rows of every weight tile into its own shared memory
// (completion counted on the leader's barriers), and runs the epilogue of its halves from its own TMEM.  Only the leader
// (rank 0) issues: one instruction covers half h of both CTAs, and its commits arrive on the barriers of both.
template <int CG>
__global__ void __launch_bounds__(kConvMaxThreads, 1) conv_kernel(const __grid_constant__ ConvParams p) {
    TL(long long* tl = g_timeline + (blockIdx.x % 160) * 16; if (threadIdx.x == 0) { tl[0] = gtime_ns(); tl[8] = 0; tl[10] = 0; tl[11] = 0; tl[7] = 0; })
    kn::pdl_trigger();
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const int MH = p.MH, BN = p.BN;
    const int rank = CG == 2 ? (int)cluster_ctarank() : 0;
    int vb = CG == 2 ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;       // position and stride in the tile list
    int vgrid = CG == 2 ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    const int zc = CG == 1 ? p.zcluster : 0;
    const int zrank = zc ? (int)cluster_ctarank() : 0;
    const int zdiv = zc ? zc : 1;
    if (zc) { vb = zrank * p.n_tiles + (int)blockIdx.x / zdiv; vgrid = p.tiles_total; }    // split zrank of n tile blockIdx / zc; one tile
    const int tile_rows = 128 * MH * CG, row0 = rank * 128 * MH;
    const int cpg = p.cpg, gw = cpg > 1 ? cpg : p.kw;            // weight tiles per A stage
    const uint32_t a_box_bytes = (uint32_t)p.a_box_rows * 128u, a_bytes = a_box_bytes * MH * cpg, b_bytes = (uint32_t)(BN / CG) * 128u;
    const int a_stages = p.a_stages, b_stages = p.b_stages;
    const uint32_t ring_a = base, ring_b = base + a_stages * a_bytes;
    // epilogue staging (4 * epi_sets warps x kEpiStageBytes), then barriers: fullA[8] @0, emptyA[8] @64, fullB[8] @128,
    // emptyB[8] @192, acc_full[2] @256, acc_empty[2] @272, tmem slot @288, abort flag @296
    const uint32_t g_bytes = b_bytes * (uint32_t)p.tpg;         // one group slot holds up to tpg weight tiles of a filter row
    const uint32_t epi_stage0 = ring_b + b_stages * g_bytes;
    const uint32_t bar_base = epi_stage0 + 4u * (uint32_t)p.epi_sets * kEpiStageBytes;
    uint8_t* gen = smem_raw + (bar_base - raw);
    volatile int* abort_flag = (volatile int*)(gen + 296);
    volatile uint32_t* tmem_slot = (volatile uint32_t*)(gen + 288);
    const uint32_t fullA = bar_base, emptyA = bar_base + 64u, fullB = bar_base + 128u, emptyB = bar_base + 192u;
    const uint32_t accf0 = bar_base + 256u, acce0 = bar_base + 272u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int acc_stages = p.acc_stages, acc_cols = MH * BN;
    uint32_t ncols = 32;
    while ((int)ncols < acc_stages * acc_cols) ncols <<= 1;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < a_stages; ++s) { mbar_init(fullA + 8u * s, 1); mbar_init(emptyA + 8u * s, MH); }
        for (int s = 0; s < b_stages; ++s) { mbar_init(fullB + 8u * s, 1); mbar_init(emptyB + 8u * s, MH); }
        for (int s = 0; s < 2; ++s) { mbar_init(accf0 + 8u * s, MH); mbar_init(acce0 + 8u * s, 128 * p.epi_sets * CG); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tma_prefetch_desc(&p.tmA);
        tma_prefetch_desc(&p.tmB);
    }
    if (warp == 2) {
        if (CG == 2) tmem_alloc_pair(smem_u32((const void*)tmem_slot), ncols);
        else tmem_alloc(smem_u32((const void*)tmem_slot), ncols);
    }
    tc_fence_before();
    __syncthreads();
    __syncwarp();
    if (CG == 2) cluster_sync_all();          // the peer's barriers exist before anything arrives on them
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    TL(if (threadIdx.x == 0) tl[12] = gtime_ns();)
    // barriers, TMEM and descriptors are set up; global memory is touched from here on (the weights possibly earlier)
    if (!(p.early_b && warp == 1)) kn::pdl_wait();
    TL(if (threadIdx.x == 0) tl[1] = gtime_ns();)
    const int per = p.asteps_per_split, kw = p.kw;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producers: lane 0 of warp 0 feeds the ring of
        // activation halos, lane 0 of warp 1 the ring of weight groups, so that neither ring waits for the other
        if (lane == 0) {
            ConvCursor tc; tc.init(p, vb, vgrid);
            int sa = 0; uint32_t pha = 0;
            bool ok = true;
            for (int tile = vb; tile < p.tiles_total && ok; tile += vgrid, tc.next(p)) {
                const int m0 = tc.m_tile * tile_rows + row0;
                const int a_begin = tc.z * per;
                const int nsteps = min(p.asteps_total, a_begin + per) - a_begin;
                // the reduction order is free: every CTA starts at a different (filter row, chunk) so that the SMs do not
                // all ask L2 for the same weight tile at the same moment
                const int a_end = a_begin + nsteps;
                int a = a_begin + (int)((unsigned)vb % (unsigned)nsteps);
                int ky = a / p.chunks, ch = a - ky * p.chunks;
                const int ky0 = a_begin / p.chunks, ch0 = a_begin - ky0 * p.chunks;
                const int xa = p.a_x0 + tc.g * p.a_gx;
                for (int i = 0; i < nsteps && ok; ++i) {
                    TL(const long long c0 = clock64();)
                    ok = mbar_wait(emptyA + 8u * sa, pha ^ 1u, abort_flag);
                    TL(tl[10] += clock64() - c0;)
                    if (!ok) break;
                    {
                        const uint32_t dst = ring_a + sa * a_bytes, fb = fullA + 8u * sa;
                        const int y = m0 + p.halo_shift[ky];
                        if (rank == 0) mbar_expect_tx(fb, a_bytes * CG);
                        const uint32_t fbc = CG == 2 ? mapa_u32(fb, 0) : fb;
                        for (int c = 0; c < cpg; ++c)
                            for (int h = 0; h < MH; ++h) {
                                if (CG == 2) tma_load_2d_pair(dst + (c * MH + h) * a_box_bytes, &p.tmA, xa + (ch * cpg + c) * 64, y + h * p.a_box_rows, fbc);
                                else tma_load_2d(dst + (c * MH + h) * a_box_bytes, &p.tmA, xa + (ch * cpg + c) * 64, y + h * p.a_box_rows, fb);
                            }
                    }
                    if (++sa == a_stages) { sa = 0; pha ^= 1u; }
                    if (++a == a_end) { a = a_begin; ky = ky0; ch = ch0; } else if (++ch == p.chunks) { ch = 0; ++ky; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && p.b_res) {
            // the whole filter, once: tile t = ky * kw + kx
            if (vb < p.tiles_total) {
                mbar_expect_tx(fullB, (uint32_t)(p.kh * kw) * b_bytes);
                for (int t = 0; t < p.kh * kw; ++t) tma_load_2d(ring_b + t * b_bytes, &p.tmB, 0, t * p.b_tap_rows, fullB);
            }
        } else if (lane == 0) {
            ConvCursor tc; tc.init(p, vb, vgrid);
            int sb = 0; uint32_t phb = 0;
            bool ok = true;
            for (int tile = vb; tile < p.tiles_total && ok; tile += vgrid, tc.next(p)) {
                const int n0 = tc.n_tile * BN + rank * (BN / CG);       // this CTA's rows of the weight tile
                const int a_begin = tc.z * per;
                const int nsteps = min(p.asteps_total, a_begin + per) - a_begin;
                // the reduction order is free: every CTA starts at a different (filter row, chunk) so that the SMs do not
                // all ask L2 for the same weight tile at the same moment
                const int a_end = a_begin + nsteps;
                int a = a_begin + (int)((unsigned)vb % (unsigned)nsteps);
                int ky = a / p.chunks, ch = a - ky * p.chunks;
                const int ky0 = a_begin / p.chunks, ch0 = a_begin - ky0 * p.chunks;
                const int yb = tc.g * p.b_g_rows + n0;
                for (int i = 0; i < nsteps && ok; ++i) {
                    int brow = ky * kw * p.b_tap_rows + yb, bcol = ch * cpg * 64;
                    const int brow_step = cpg > 1 ? 0 : p.b_tap_rows, bcol_step = cpg > 1 ? 64 : 0;
                    for (int kx0 = 0; kx0 < gw; kx0 += p.tpg) {
                        TL(const long long c0 = clock64();)
                        ok = mbar_wait(emptyB + 8u * sb, phb ^ 1u, abort_flag);
                        TL(tl[11] += clock64() - c0;)
                        if (!ok) break;
                        const uint32_t fb = fullB + 8u * sb, dst = ring_b + sb * g_bytes;
                        const int taps = min(p.tpg, gw - kx0);
                        if (rank == 0) mbar_expect_tx(fb, (uint32_t)taps * b_bytes * CG);
                        const uint32_t fbc = CG == 2 ? mapa_u32(fb, 0) : fb;
                        for (int t = 0; t < taps; ++t, brow += brow_step, bcol += bcol_step) {
                            if (CG == 2) tma_load_2d_pair(dst + t * b_bytes, &p.tmB, bcol, brow, fbc);
                            else tma_load_2d(dst + t * b_bytes, &p.tmB, bcol, brow, fb);
                        }
                        if (++sb == b_stages) { sb = 0; phb ^= 1u; }
                    }
                    if (++a == a_end) { a = a_begin; ky = ky0; ch = ch0; } else if (++ch == p.chunks) { ch = 0; ++ky; }
                }
            }
        }
    } else if (warp <= MH + 1) {
        // ------------------------------------------------------------ MMA issuer of row half h (whole warp)
        if (rank == 0) {
            const int h = warp - 2;
            const uint32_t idesc = instr_desc(BN, 0, 0, 128 * CG);
            const uint64_t dbase = smem_desc(0, 16, 1024);
            const int kk = p.kk;
            int sa = 0, sb = 0; uint32_t pha = 0, phb = 0;
            int ab = 0; uint32_t aph = 0;
            bool ok = true;
            int z = vb / (p.m_tiles * p.n_tiles * p.groups);     // only the split index matters here
            int in_split = vb - z * (p.m_tiles * p.n_tiles * p.groups);
            const int tiles_per_split = p.m_tiles * p.n_tiles * p.groups;
            const bool b_res = p.b_res != 0;
            if (b_res && vb < p.tiles_total) ok = mbar_wait_warp(fullB, 0u, abort_flag);      // the resident filter has arrived
            TL(long long wA = 0, wB = 0, wC = 0, nm = 0; const long long tl0 = clock64(), gl0 = gtime_ns();)
            for (int tile = vb; tile < p.tiles_total && ok; tile += vgrid) {
                const int a_begin = z * per;
                const int nsteps = min(p.asteps_total, a_begin + per) - a_begin;
                int ares = a_begin + (int)((unsigned)vb % (unsigned)nsteps);      // resident filter: the producer's rotation of the filter rows
                TL(const long long cc0 = clock64();)
                ok = mbar_wait_warp(acce0 + 8u * ab, aph ^ 1u, abort_flag);
                TL(wC += clock64() - cc0;)
                if (!ok) break;
                if (CG == 2) fence_acq_rel_cluster();      // the peer's epilogue arrived from the other CTA
                tc_fence_after();
                const uint32_t d = tmem + (uint32_t)(ab * acc_cols + h * BN);
                uint32_t accum = 0;
                for (int i = 0; i < nsteps && ok; ++i) {
                    TL(const long long ca0 = clock64();)
                    ok = mbar_wait_warp(fullA + 8u * sa, pha, abort_flag);
                    TL(wA += clock64() - ca0;)
                    if (!ok) break;
                    const uint64_t ad = dbase + (uint64_t)((ring_a + sa * a_bytes + (uint32_t)h * 16384u) >> 4);
                    // the MMAs of a weight group in straight-line code: the fixed cost of a loop trip with a barrier wait
                    // (a few hundred cycles) is paid once per taps*kk instructions
                    for (int kx0 = 0; kx0 < gw; kx0 += p.tpg) {
                        TL(const long long cb0 = clock64();)
                        if (!b_res && !(ok = mbar_wait_warp(fullB + 8u * sb, phb, abort_flag))) break;
                        TL(wB += clock64() - cb0; nm += (long long)min(p.tpg, gw - kx0) * kk;)
                        const uint64_t bd = dbase + (uint64_t)((b_res ? ring_b + (uint32_t)(ares * kw) * b_bytes : ring_b + sb * g_bytes) >> 4);
                        const int taps = min(p.tpg, gw - kx0);
                        const int* toff = p.tap_off + kx0;
                        if (kk == 4) {
                            if (taps == 3) issue_row<3, 4, CG>(d, ad, bd, b_bytes >> 4, toff, idesc, accum);
                            else if (taps == 2) issue_row<2, 4, CG>(d, ad, bd, b_bytes >> 4, toff, idesc, accum);
                            else issue_row<1, 4, CG>(d, ad, bd, b_bytes >> 4, toff, idesc, accum);
                        } else {
                            if (taps == 3) issue_row<3, 3, CG>(d, ad, bd, b_bytes >> 4, toff, idesc, accum);
                            else if (taps == 2) issue_row<2, 3, CG>(d, ad, bd, b_bytes >> 4, toff, idesc, accum);
                            else issue_row<1, 3, CG>(d, ad, bd, b_bytes >> 4, toff, idesc, accum);
                        }
                        accum = 1;
                        if (!b_res) {
                            umma_commit_cg<CG>(emptyB + 8u * sb);
                            if (++sb == b_stages) { sb = 0; phb ^= 1u; }
                        }
                    }
                    if (++ares == a_begin + nsteps) ares = a_begin;
                    if (!ok) break;
                    umma_commit_cg<CG>(emptyA + 8u * sa);
                    if (++sa == a_stages) { sa = 0; pha ^= 1u; }
                }
                if (!ok) break;
                umma_commit_cg<CG>(accf0 + 8u * ab);
                if (++ab == acc_stages) { ab = 0; aph ^= 1u; }
                in_split += vgrid;
                while (in_split >= tiles_per_split) { in_split -= tiles_per_split; ++z; }
            }
            TL(if (h == 0 && lane == 0) { tl[3] = wA; tl[4] = wB; tl[5] = wC; tl[6] = clock64() - tl0; tl[7] = nm; tl[13] = gl0; tl[14] = gtime_ns(); })
        }
    } else {
        // ------------------------------------------------------------ epilogue
        const int quad = warp & 3;
        const int ew = warp - (MH + 2), eset = ew >> 2, E = p.epi_sets;     // epilogue warp index and its set
        const int r = quad * 32 + lane;          // row within a 128-row half = TMEM lane
        ConvCursor tc; tc.init(p, vb, vgrid);
        int ab = 0; uint32_t aph = 0;
        bool ok = true;
        const uint32_t acce_leader = CG == 2 ? mapa_u32(acce0, 0) : acce0;
        for (int tile = vb; tile < p.tiles_total && ok; tile += vgrid, tc.next(p)) {
            const int m0 = tc.m_tile * tile_rows + row0, n0 = tc.n_tile * BN, g = tc.g;
            const int a_begin = tc.z * per;
            const int nsteps = min(p.asteps_total, a_begin + per) - a_begin;
            TL(const long long ce0 = clock64();)
            ok = mbar_wait(accf0 + 8u * ab, aph, abort_flag);
            TL(if (ew == 0 && lane == 0) tl[8] += clock64() - ce0;)
            if (!ok) break;
            tc_fence_after();
            // with two sets of epilogue warps, the (row half, slab) units of the tile alternate between the sets
            int unit = 0;
            #pragma unroll 1
            for (int h = 0; h < MH; ++h) {
                const int row = m0 + h * 128 + r;
                const bool row_ok = row < p.M_total;
                bool pad_row = false;
                if (p.Hp > 0) {
                    const int x = row % p.Wp, y = (row / p.Wp) % p.Hp;
                    pad_row = (x >= p.W) || (y >= p.H);
                }
                const long long row_off = (long long)tc.z * p.split_stride + (long long)row * p.ldo + g * p.out_gx;
                const uint32_t t0 = tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)(ab * acc_cols + h * BN);
                if (zc) {
                    // the partial tile stays on chip: row r of the tile to the (idle) operand ring, 32 columns per unit
                    for (int c = 0; c < BN; c += 32, ++unit) {
                        if (E == 2 && (unit & 1) != eset) continue;
                        uint32_t v[32];
                        tmem_ld32(t0 + (uint32_t)c, v);
                        tmem_ld_wait();
                        const uint32_t rowp = ring_a + (uint32_t)(r * kZcPitch + c) * 4u;
                        #pragma unroll
                        for (int q = 0; q < 8; ++q) st_shared_v4(rowp + 16u * q, v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                    }
                } else if (p.tma_store) {
                    const int slab = p.epi == EPI_F32 ? 32 : 64;
                    for (int c = 0; c < BN; c += slab, ++unit) {
                        if (E == 2 && (unit & 1) != eset) continue;
                        epi_slab(p, t0 + (uint32_t)c, pad_row, row_off, n0 + c, g, g * p.out_gx + n0 + c, m0 + h * 128 + quad * 32,
                                 tc.z, epi_stage0 + (uint32_t)ew * kEpiStageBytes, lane);
                    }
                } else {
                    for (int c = 0; c < BN; c += 16, ++unit) {
                        if (E == 2 && (unit & 1) != eset) continue;
                        uint32_t v[16];
                        tmem_ld16(t0 + (uint32_t)c, v);
                        tmem_ld_wait();
                        if (!row_ok) continue;
                        epi_chunk(p, v, nsteps <= 0, pad_row, row_off, n0 + c, g);
                    }
                }
            }
            tc_fence_before();
            if (CG == 2) mbar_arrive_cluster(acce_leader + 8u * ab);
            else mbar_arrive(acce0 + 8u * ab);
            if (++ab == acc_stages) { ab = 0; aph ^= 1u; }
        }
        if (p.tma_store && !zc && lane == 0) bulk_wait_all();
        TL(if (ew == 0 && lane == 0) tl[15] = gtime_ns();)
    }
    if (zc) {
        // every CTA of the cluster has its partial tile in shared memory (all threads arrive: the barrier also orders the
        // epilogue warps' stores before the peers' reads); then the epilogue warps reduce this CTA's rows across the cluster
        __syncwarp();
        cluster_sync_all();
        if (warp > MH + 1) {
            const int T = 128 * p.epi_sets, t = (warp - (MH + 2)) * 32 + lane;
            const int rows_per = 128 / zdiv, n0 = ((int)blockIdx.x / zdiv) * BN;
            for (int idx = t; idx < rows_per * 32; idx += T) {
                const int row = zrank * rows_per + (idx >> 5), c4 = idx & 31;
                const uint32_t local = ring_a + (uint32_t)(row * kZcPitch + 4 * c4) * 4u;
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
                for (int q = 0; q < zc; ++q) {
                    float4 v;
                    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(mapa_u32(local, (uint32_t)q)) : "memory");
                    acc[0] += v.x; acc[1] += v.y; acc[2] += v.z; acc[3] += v.w;
                }
                if (row >= p.M_total) continue;
                const int n = n0 + 4 * c4;
                if (n >= p.n_valid) continue;                      // n_valid is a multiple of 4 in the layers that run this way
                const long long tt = (long long)row * p.n_valid + n;
                uint32_t keepw = 0x01010101u;
                #pragma unroll
                for (int k = 0; k < 4; ++k) {
                    float v = acc[k] + p.bias[n + k];
                    if (p.fc_relu) v = fmaxf(v, 0.f);
                    if (p.fc_dropout == 2) v *= p.fc_scale;
                    else if (p.fc_dropout) {
                        const bool keep = (uint32_t)(kn::draw(p.fc_key, (uint64_t)(tt + k)) >> 40) >= p.fc_thr24;
                        if (!keep) keepw &= ~(0xFFu << (8 * k));
                        v = keep ? v * p.fc_scale : 0.f;
                    }
                    acc[k] = v;
                }
                const __nv_bfloat162 lo = __floats2bfloat162_rn(acc[0], acc[1]), hi = __floats2bfloat162_rn(acc[2], acc[3]);
                *(uint2*)(p.fc_out + tt) = make_uint2(*(const uint32_t*)&lo, *(const uint32_t*)&hi);
                if (p.fc_keep) *(uint32_t*)(p.fc_keep + tt) = keepw;
            }
        }
        __syncwarp();
        cluster_sync_all();          // no CTA leaves (and frees its shared memory) while a peer may still read its partial tile
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0 && p.status) atomicExch(p.status, 1);
        long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) { }
        __syncthreads();
    }
    __syncwarp();
    if (CG == 2) cluster_sync_all();          // no CTA leaves while its peer may still arrive on its barriers
    TL(if (threadIdx.x == 0) tl[2] = gtime_ns();)
    if (warp == 2) {
        tc_fence_after();
        if (CG == 2) tmem_dealloc_pair(tmem, ncols);
        else tmem_dealloc(tmem, ncols);
    }
}

// ===========================================================================
// FC forward chain: the three fully connected layers of the forward pass in ONE launch.
//
// At batch <= 128 an FC layer is a stream of weights (117 MB of bf16 for the three layers) against one 128-row tile of
// activations, and a launch per layer spends as long on its set-up, first loads and exposed epilogue as on the stream.
// Here the grid (128 CTAs, clusters of four) walks fc6 -> fc7 -> fc8 with one (128-column tile, k split) unit per CTA and
// layer.  The weight producer never waits for a layer boundary: while a layer's epilogue and the hand-over run, the
// ring already fills with the next layer's weights, so HBM stays busy.  Only the activation producer waits: a layer's
// input is the previous layer's output, stored by every CTA, so the CTAs count themselves on a grid-wide gate (a counter
// in global memory; the launch is cooperative, all CTAs are resident) and the producer reads past it with an
// acquire load and a proxy fence before its TMA loads.  All waits are bounded.
// fc6 / fc7: the four splits of a tile are one cluster and reduce their fp32 partial tiles through distributed shared
// memory with bias, ReLU and dropout applied (the arithmetic and order of conv_kernel's cluster form: bit-identical);
// fc8: fp32 partials per split to global memory, reduced by the softmax kernel that follows.
// Unit -> (tile, split) and the rotation of the reduction order are those of the per-layer launches.
// Warps: 0 = activation producer, 1 = weight producer, 2 = MMA issuer, 3..10 = two sets of four epilogue warps.
struct FcChainLayer {
    CUtensorMap tmA, tmB;        // activations [B][K], box {64, 128}; weights [N][K], box {64, 128}
    int n_tiles, splits, per;    // 128-column tiles; k splits; steps (of 128 channels) per split
    int asteps_total, n_valid;
    int cluster_reduce;          // 1: the splits of a tile are the CTAs of a cluster (splits == kChainCluster)
    int relu, dropout;           // dropout: 0 none, 1 mask from the hash, 2 evaluation (expectation of the mask)
    uint32_t thr24; float scale; uint64_t key;
    const float* bias; __nv_bfloat16* out; uint8_t* keep;     // cluster_reduce layers
    float* partial; long long split_stride;                   // other layers: [split][B][n_valid] fp32
};
struct FcChainParams {
    FcChainLayer L[3];
    int nlayers, M_total;
    int* status;
    unsigned* gate; unsigned gate_base;     // grid gate: counter and its value when the launch starts
};
constexpr int kChainThreads = 32 * 11, kChainCluster = 4, kChainAStages = 3, kChainBStages = 4;
constexpr uint32_t kChainStageBytes = 32768;      // two 64-channel boxes of 128 rows
inline size_t fc_chain_smem_bytes() { return 1024 + (size_t)(kChainAStages + kChainBStages) * kChainStageBytes + 512; }

__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned* p) {
    unsigned v; asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory"); return v;
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

__global__ void __launch_bounds__(kChainThreads, 1) fc_chain_kernel(const __grid_constant__ FcChainParams p) {
    // timeline slots (ns): 0 start, 1 set up, 2 end; issuer: 3 + 2 l first operands of layer l, 4 + 2 l its last commit;
    // first epilogue thread: 9 + 3 l accumulator of layer l ready, 10 + 3 l partial tiles of the cluster ready, 11 + 3 l stored
    // and counted on the gate (l = 0, 1); 15: the activation producer passed the first gate
    TL(long long* tl = g_timeline + (blockIdx.x % 160) * 16; if (threadIdx.x == 0) tl[0] = gtime_ns();)
    kn::pdl_trigger();
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const uint32_t ring_a = base, ring_b = base + kChainAStages * kChainStageBytes;
    const uint32_t bar_base = ring_b + kChainBStages * kChainStageBytes;
    // barriers: fullA[3] @0, emptyA[3] @24, fullB[4] @48, emptyB[4] @80, acc_full[2] @112, acc_empty[2] @128,
    // partials-ready (cluster) @144, stored (gate) @152; tmem slot @160, abort flag @168
    uint8_t* gen = smem_raw + (bar_base - raw);
    volatile int* abort_flag = (volatile int*)(gen + 168);
    volatile uint32_t* tmem_slot = (volatile uint32_t*)(gen + 160);
    const uint32_t fullA = bar_base, emptyA = bar_base + 24u, fullB = bar_base + 48u, emptyB = bar_base + 80u;
    const uint32_t accf0 = bar_base + 112u, acce0 = bar_base + 128u, xbar = bar_base + 144u, gbar = bar_base + 152u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int zrank = (int)cluster_ctarank(), cid = (int)blockIdx.x / kChainCluster;
    constexpr uint32_t kCols = 256;      // two accumulators of 128 columns

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < kChainAStages; ++s) { mbar_init(fullA + 8u * s, 1); mbar_init(emptyA + 8u * s, 1); }
        for (int s = 0; s < kChainBStages; ++s) { mbar_init(fullB + 8u * s, 1); mbar_init(emptyB + 8u * s, 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(accf0 + 8u * s, 1); mbar_init(acce0 + 8u * s, 256); }
        mbar_init(xbar, 8 * kChainCluster);
        mbar_init(gbar, 8);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        for (int l = 0; l < p.nlayers; ++l) { tma_prefetch_desc(&p.L[l].tmA); tma_prefetch_desc(&p.L[l].tmB); }
    }
    if (warp == 2) tmem_alloc(smem_u32((const void*)tmem_slot), kCols);
    tc_fence_before();
    __syncthreads();
    __syncwarp();
    cluster_sync_all();          // the peers' barriers exist before anything arrives on them
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    kn::pdl_wait();
    TL(if (threadIdx.x == 0) tl[1] = gtime_ns();)

    // this CTA's unit of layer l: position vb in the layer's tile list (split-major), tile and split
    #define CHAIN_UNIT(L) \
        int vb, n_tile, z; \
        if ((L).cluster_reduce) { n_tile = cid; z = zrank; vb = z * (L).n_tiles + n_tile; } \
        else { vb = (int)blockIdx.x; n_tile = vb % (L).n_tiles; z = vb / (L).n_tiles; } \
        const int a_begin = z * (L).per; \
        const int nsteps = min((L).asteps_total, a_begin + (L).per) - a_begin; \
        (void)vb; (void)n_tile;

    if (warp == 0) {
        if (lane == 0) {
            // ------------------------------------------------------------ activations
            int sa = 0; uint32_t pha = 0;
            bool ok = true;
            for (int l = 0; l < p.nlayers && ok; ++l) {
                const FcChainLayer& L = p.L[l];
                CHAIN_UNIT(L)
                if (l > 0) {
                    // the gate: every CTA has stored its part of the previous layer's output
                    const unsigned target = p.gate_base + (unsigned)l * gridDim.x;
                    const long long t0 = clock64();
                    while ((int)(ld_acquire_gpu(p.gate) - target) < 0) {
                        if (*abort_flag) { ok = false; break; }
                        if (clock64() - t0 > kWaitBudgetCycles) { *abort_flag = 1; ok = false; break; }
                    }
                    if (!ok) break;
                    TL(if (l == 1) tl[15] = gtime_ns();)
                    fence_proxy_async_all();     // those stores (generic proxy) before this thread's TMA reads (async proxy)
                }
                int a = a_begin + (int)((unsigned)vb % (unsigned)nsteps);
                for (int i = 0; i < nsteps && ok; ++i) {
                    ok = mbar_wait(emptyA + 8u * sa, pha ^ 1u, abort_flag);
                    if (!ok) break;
                    const uint32_t dst = ring_a + sa * kChainStageBytes, fb = fullA + 8u * sa;
                    mbar_expect_tx(fb, kChainStageBytes);
                    tma_load_2d(dst, &L.tmA, a * 128, 0, fb);
                    tma_load_2d(dst + 16384u, &L.tmA, a * 128 + 64, 0, fb);
                    if (++sa == kChainAStages) { sa = 0; pha ^= 1u; }
                    if (++a == a_begin + nsteps) a = a_begin;
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ------------------------------------------------------------ weights: no layer boundary
            int sb = 0; uint32_t phb = 0;
            bool ok = true;
            for (int l = 0; l < p.nlayers && ok; ++l) {
                const FcChainLayer& L = p.L[l];
                CHAIN_UNIT(L)
                int a = a_begin + (int)((unsigned)vb % (unsigned)nsteps);
                for (int i = 0; i < nsteps && ok; ++i) {
                    ok = mbar_wait(emptyB + 8u * sb, phb ^ 1u, abort_flag);
                    if (!ok) break;
                    const uint32_t dst = ring_b + sb * kChainStageBytes, fb = fullB + 8u * sb;
                    mbar_expect_tx(fb, kChainStageBytes);
                    tma_load_2d(dst, &L.tmB, a * 128, n_tile * 128, fb);
                    tma_load_2d(dst + 16384u, &L.tmB, a * 128 + 64, n_tile * 128, fb);
                    if (++sb == kChainBStages) { sb = 0; phb ^= 1u; }
                    if (++a == a_begin + nsteps) a = a_begin;
                }
            }
        }
    } else if (warp == 2) {
        // ---------------------------------------------------------------- MMA issuer (whole warp)
        const uint32_t idesc = instr_desc(128, 0, 0, 128);
        const uint64_t dbase = smem_desc(0, 16, 1024);
        int sa = 0, sb = 0; uint32_t pha = 0, phb = 0;
        int ab = 0; uint32_t aph = 0;
        bool ok = true;
        for (int l = 0; l < p.nlayers && ok; ++l) {
            const FcChainLayer& L = p.L[l];
            CHAIN_UNIT(L)
            ok = mbar_wait_warp(acce0 + 8u * ab, aph ^ 1u, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d = tmem + (uint32_t)(ab * 128);
            uint32_t accum = 0;
            for (int i = 0; i < nsteps && ok; ++i) {
                ok = mbar_wait_warp(fullA + 8u * sa, pha, abort_flag) && mbar_wait_warp(fullB + 8u * sb, phb, abort_flag);
                if (!ok) break;
                TL(if (i == 0 && lane == 0) tl[3 + 2 * l] = gtime_ns();)
                const uint64_t ad = dbase + (uint64_t)((ring_a + sa * kChainStageBytes) >> 4);
                const uint64_t bd = dbase + (uint64_t)((ring_b + sb * kChainStageBytes) >> 4);
                #pragma unroll
                for (int c = 0; c < 2; ++c)          // the stage's two 64-channel boxes, four K = 16 steps each
                    #pragma unroll
                    for (int j = 0; j < 4; ++j)
                        umma(d, ad + (uint64_t)(c * 1024 + 2 * j), bd + (uint64_t)(c * 1024 + 2 * j), idesc, (c == 0 && j == 0) ? accum : 1u);
                accum = 1;
                umma_commit(emptyB + 8u * sb);
                umma_commit(emptyA + 8u * sa);
                if (++sa == kChainAStages) { sa = 0; pha ^= 1u; }
                if (++sb == kChainBStages) { sb = 0; phb ^= 1u; }
            }
            if (!ok) break;
            umma_commit(accf0 + 8u * ab);
            TL(if (lane == 0) tl[4 + 2 * l] = gtime_ns();)
            if (++ab == 2) { ab = 0; aph ^= 1u; }
        }
    } else {
        // ---------------------------------------------------------------- epilogue
        const int quad = warp & 3, ew = warp - 3, eset = ew >> 2;
        const int r = quad * 32 + lane;          // row of the tile = TMEM lane
        const int et = ew * 32 + lane;           // 0..255
        int ab = 0; uint32_t aph = 0, xph = 0, gph = 0;
        bool ok = true;
        for (int l = 0; l < p.nlayers && ok; ++l) {
            const FcChainLayer& L = p.L[l];
            CHAIN_UNIT(L)
            ok = mbar_wait(accf0 + 8u * ab, aph, abort_flag);
            if (!ok) break;
            TL(if (et == 0 && l < 2) tl[9 + 3 * l] = gtime_ns();)
            tc_fence_after();
            const uint32_t t0 = tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)(ab * 128);
            const int n0 = n_tile * 128;
            #pragma unroll 1
            for (int unit = 0; unit < 4; ++unit) {       // 32-column units alternate between the two sets of warps
                if ((unit & 1) != eset) continue;
                const int c = unit * 32;
                uint32_t v[32];
                tmem_ld32(t0 + (uint32_t)c, v);
                tmem_ld_wait();
                if (nsteps <= 0) {
                    #pragma unroll
                    for (int k = 0; k < 32; ++k) v[k] = 0u;
                }
                if (L.cluster_reduce) {
                    // the partial tile stays on chip: in the activation ring, idle until the next layer's gate opens
                    const uint32_t rowp = ring_a + (uint32_t)(r * kZcPitch + c) * 4u;
                    #pragma unroll
                    for (int q = 0; q < 8; ++q) st_shared_v4(rowp + 16u * q, v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                } else if (r < p.M_total) {
                    float* o = L.partial + (long long)z * L.split_stride + (long long)r * L.n_valid + n0 + c;
                    #pragma unroll
                    for (int q = 0; q < 8; ++q)
                        if (n0 + c + 4 * q < L.n_valid)      // n_valid is a multiple of 4
                            *(float4*)(o + 4 * q) = make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]),
                                                                __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
                }
            }
            tc_fence_before();
            mbar_arrive(acce0 + 8u * ab);
            if (++ab == 2) { ab = 0; aph ^= 1u; }
            if (L.cluster_reduce) {
                // the four output columns this thread finishes, and their bias (fetched while the cluster gathers)
                const int c4 = et & 31, n = n0 + 4 * c4;
                const float4 b4 = n < L.n_valid ? __ldg((const float4*)(L.bias + n)) : make_float4(0.f, 0.f, 0.f, 0.f);
                // every epilogue warp of the cluster tells all four CTAs that its rows of a partial tile are written (one
                // arrival per warp: arrivals on one barrier are serialised, a thousand of them cost microseconds)
                __syncwarp();
                if (lane == 0) {
                    #pragma unroll
                    for (int q = 0; q < kChainCluster; ++q) mbar_arrive_cluster(mapa_u32(xbar, (uint32_t)q));
                }
                ok = mbar_wait(xbar, xph, abort_flag);
                xph ^= 1u;
                if (!ok) break;
                TL(if (et == 0 && l < 2) tl[10 + 3 * l] = gtime_ns();)
                fence_acq_rel_cluster();
                // this CTA's 32 rows of the four partial tiles: all sixteen remote loads of a thread are in flight together
                constexpr int rows_per = 128 / kChainCluster, items = rows_per * 32 / 256;
                float4 part[items][kChainCluster];
                #pragma unroll
                for (int it = 0; it < items; ++it) {
                    const int row = zrank * rows_per + (et >> 5) + 8 * it;
                    const uint32_t local = ring_a + (uint32_t)(row * kZcPitch + 4 * c4) * 4u;
                    #pragma unroll
                    for (int q = 0; q < kChainCluster; ++q)
                        asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                                     : "=f"(part[it][q].x), "=f"(part[it][q].y), "=f"(part[it][q].z), "=f"(part[it][q].w)
                                     : "r"(mapa_u32(local, (uint32_t)q)) : "memory");
                }
                #pragma unroll
                for (int it = 0; it < items; ++it) {
                    const int row = zrank * rows_per + (et >> 5) + 8 * it;
                    float acc[4] = {0.f, 0.f, 0.f, 0.f};
                    #pragma unroll
                    for (int q = 0; q < kChainCluster; ++q) {       // in split order
                        acc[0] += part[it][q].x; acc[1] += part[it][q].y; acc[2] += part[it][q].z; acc[3] += part[it][q].w;
                    }
                    if (row >= p.M_total || n >= L.n_valid) continue;
                    const long long tt = (long long)row * L.n_valid + n;
                    const float bb[4] = {b4.x, b4.y, b4.z, b4.w};
                    uint32_t keepw = 0x01010101u;
                    #pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        float y = acc[k] + bb[k];
                        if (L.relu) y = fmaxf(y, 0.f);
                        if (L.dropout == 2) y *= L.scale;
                        else if (L.dropout) {
                            const bool keep = (uint32_t)(kn::draw(L.key, (uint64_t)(tt + k)) >> 40) >= L.thr24;
                            if (!keep) keepw &= ~(0xFFu << (8 * k));
                            y = keep ? y * L.scale : 0.f;
                        }
                        acc[k] = y;
                    }
                    const __nv_bfloat162 lo = __floats2bfloat162_rn(acc[0], acc[1]), hi = __floats2bfloat162_rn(acc[2], acc[3]);
                    *(uint2*)(L.out + tt) = make_uint2(*(const uint32_t*)&lo, *(const uint32_t*)&hi);
                    if (L.keep) *(uint32_t*)(L.keep + tt) = keepw;
                }
            }
            if (l + 1 < p.nlayers) {
                // this thread's shared-memory accesses (its rows of the tile, the peers' tiles) come before the TMA
                // writes of the next layer's activations into the same ring; its global stores before the gate
                fence_proxy_async_all();
                __threadfence();
                __syncwarp();
                if (lane == 0) mbar_arrive(gbar);
                if (et == 0) {
                    ok = mbar_wait(gbar, gph, abort_flag);
                    if (ok) { __threadfence(); atomicAdd(p.gate, 1u); }
                    TL(if (l < 2) tl[11 + 3 * l] = gtime_ns();)
                }
                gph ^= 1u;
            }
        }
    }
    #undef CHAIN_UNIT
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0 && p.status) atomicExch(p.status, 1);
        long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) { }
        __syncthreads();
    }
    __syncwarp();
    cluster_sync_all();          // no CTA leaves while a peer may still read its partial tile or arrive on its barriers
    TL(if (threadIdx.x == 0) tl[2] = gtime_ns();)
    if (warp == 2) {
        tc_fence_after();
        tmem_dealloc(tmem, kCols);
    }
}

// ===========================================================================
// Convolution weight-gradient kernel.
//
//   dW[ky][kx][co][ci] = sum_m dy[m][co] * x[m + shift(ky,kx)][ci]
//
// Both operands are MN-major (the reduction runs over the rows m of the flat
// grid).  One CTA owns one filter row ky, one block of 128 output channels, one
// block of 64 input channels and one range of rows; per 64-row step it loads
// the dy tile (two 64 x 64 boxes) and ONE halo of x rows (72 rows x 64
// channels).  The kw taps of the filter row are the same halo shifted by whole
// rows, so they are fed to the tensor core as consecutive 64-wide N blocks of a
// single instruction: the B descriptor's leading-dimension offset is one row
// (128 bytes), which makes N block j read the halo from row j on.  One
// instruction therefore covers up to four taps (N = 64 * taps <= 256); a
// five-tap row takes two accumulators with an issuer warp each.
// Each CTA writes fp32 partial sums [split][tap][co][ci]; a reduction kernel
// adds the splits in a fixed order.
// Warps: 0 = TMA producer, 1..NI = MMA issuers, NI+1..NI+4 = epilogue.
struct WgradParams {
    CUtensorMap tmA, tmB;       // dy [M][cout] box {64, kWgRows}; x [M][cin] box {64, kWgRows + 8}
    int m_tiles, n_tiles, groups, kh, splits;   // tile decomposition (m fastest, then n, group, ky, split)
    int tiles_total;
    int kw;                     // taps per filter row
    int NI;                     // accumulators = issuers (1 or 2)
    int acc_kx0[2], acc_taps[2];  // first tap and tap count of each accumulator
    int steps_total, steps_per_split, stages;
    int a_gx, b_gx;             // per-group column strides of dy and x
    int halo_shift[5];          // per ky: first halo row relative to the dy row
    // output
    int M_total;                // valid output channels per group
    int n_valid;                // valid input channels per group
    int ldo, out_gx;            // row pitch (= input channels per group), per-group row offset
    long long split_stride, tap_stride;
    int epi, relu; float mask_scale; const float* bias; const __nv_bfloat16* mask;   // fixed: EPI_F32, unused
    void* out;
    float* bias_partial;        // [split][all output channels] column sums of dy, or nullptr
    int bias_ld;                // output channels over all groups
    int* status;
};
constexpr int kWgRows = 128;                           // rows of the flat grid per step: 8 MMAs (K = 16 each) per barrier wait
constexpr int kWgABytes = 2 * kWgRows * 128, kWgBBytes = (kWgRows + 8) * 128;
inline int wgrad_threads(const WgradParams& p) { return 32 * (5 + p.NI); }
inline size_t wgrad_smem_bytes(const WgradParams& p) { return 1024 + (size_t)p.stages * (kWgABytes + kWgBBytes) + 4096 + 256; }

__global__ void __launch_bounds__(32 * 7, 1) wgrad_kernel(const __grid_constant__ WgradParams p) {
    kn::pdl_trigger();
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const int stages = p.stages, NI = p.NI;
    constexpr uint32_t stage_bytes = kWgABytes + kWgBBytes;
    // 4 KB for the bias-gradient reduction, then barriers: full[8] @0, empty[8] @64, acc_full @128, tmem slot @136,
    // abort flag @144
    const uint32_t red_base = base + stages * stage_bytes;
    const uint32_t bar_base = red_base + 4096u;
    uint8_t* gen = smem_raw + (bar_base - raw);
    volatile int* abort_flag = (volatile int*)(gen + 144);
    volatile uint32_t* tmem_slot = (volatile uint32_t*)(gen + 136);
    const uint32_t full0 = bar_base, empty0 = bar_base + 64u, accf = bar_base + 128u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int acc_cols = 64 * p.kw;
    uint32_t ncols = 32;
    while ((int)ncols < acc_cols) ncols <<= 1;

    // this CTA's tile (one per CTA: the grid equals the tile count)
    int r = blockIdx.x;
    const int m_tile = r % p.m_tiles; r /= p.m_tiles;
    const int n_tile = r % p.n_tiles; r /= p.n_tiles;
    const int g = r % p.groups; r /= p.groups;
    const int ky = r % p.kh;
    const int z = r / p.kh;
    const int s_begin = z * p.steps_per_split;
    const int nsteps = min(p.steps_total, s_begin + p.steps_per_split) - s_begin;

    // the CTAs of filter row 0 and input block 0 also sum the dy tile over the rows (the bias gradient): their four
    // epilogue warps read every A stage and release it together with the issuers
    const bool do_bias = p.bias_partial != nullptr && ky == 0 && n_tile == 0;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < stages; ++s) { mbar_init(full0 + 8u * s, 1); mbar_init(empty0 + 8u * s, NI + (do_bias ? 4 : 0)); }
        mbar_init(accf, NI);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tma_prefetch_desc(&p.tmA);
        tma_prefetch_desc(&p.tmB);
    }
    if (warp == 1) tmem_alloc(smem_u32((const void*)tmem_slot), ncols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    kn::pdl_wait();        // barriers, TMEM and descriptors are set up; global memory is touched from here on

    if (warp == 0) {
        if (lane == 0) {
            const int xa = g * p.a_gx + m_tile * 128, xb = g * p.b_gx + n_tile * 64, sh = p.halo_shift[ky];
            int st = 0; uint32_t ph = 0;
            for (int i = 0; i < nsteps; ++i) {
                if (!mbar_wait(empty0 + 8u * st, ph ^ 1u, abort_flag)) break;
                const uint32_t sa = base + st * stage_bytes, fb = full0 + 8u * st;
                const int q = (s_begin + i) * kWgRows;
                mbar_expect_tx(fb, stage_bytes);
                tma_load_2d(sa, &p.tmA, xa, q, fb);
                tma_load_2d(sa + kWgRows * 128, &p.tmA, xa + 64, q, fb);
                tma_load_2d(sa + kWgABytes, &p.tmB, xb, q + sh, fb);
                if (++st == stages) { st = 0; ph ^= 1u; }
            }
        }
    } else if (warp <= NI) {
        {
            const int a = warp - 1;
            const int taps = p.acc_taps[a], kx0 = p.acc_kx0[a];
            const uint32_t idesc = instr_desc(64 * taps, 1, 1);
            const uint64_t adesc0 = smem_desc(0, kWgRows * 128, 1024), bdesc0 = smem_desc(0, 128, 1024);
            const uint32_t d = tmem + (uint32_t)(kx0 * 64);
            int st = 0; uint32_t ph = 0;
            bool ok = true;
            for (int i = 0; i < nsteps; ++i) {
                if (!(ok = mbar_wait_warp(full0 + 8u * st, ph, abort_flag))) break;
                tc_fence_after();
                const uint32_t sa = base + st * stage_bytes;
                const uint64_t ad = adesc0 + (uint64_t)(sa >> 4);
                const uint64_t bd = bdesc0 + (uint64_t)((sa + kWgABytes + (uint32_t)kx0 * 128u) >> 4);
                #pragma unroll
                for (int j = 0; j < kWgRows / 16; ++j)
                    umma(d, ad + (uint64_t)(128 * j), bd + (uint64_t)(128 * j), idesc, (i > 0 || j > 0) ? 1u : 0u);
                umma_commit(empty0 + 8u * st);
                if (++st == stages) { st = 0; ph ^= 1u; }
            }
            if (ok) umma_commit(accf);
        }
    } else {
        const int quad = warp & 3;
        const int row = m_tile * 128 + quad * 32 + lane;     // output channel within the group
        const bool row_ok = row < p.M_total;
        if (do_bias) {
            // thread te: eight output channels (16-byte chunk cc of the 128-channel tile) of rows rg*16 .. rg*16+15 of a stage
            const int te = (warp - NI - 1) * 32 + lane, cc = te & 15, rg = te >> 4;
            float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
            int st = 0; uint32_t ph = 0;
            bool ok = true;
            for (int i = 0; i < nsteps; ++i) {
                if (!(ok = mbar_wait(full0 + 8u * st, ph, abort_flag))) break;
                const uint32_t a0 = base + st * stage_bytes + (uint32_t)(cc >> 3) * (kWgRows * 128u) + (uint32_t)rg * (kWgRows / 8 * 128u);
                #pragma unroll
                for (int rr = 0; rr < kWgRows / 8; ++rr) {
                    uint4 u;
                    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(u.x), "=r"(u.y), "=r"(u.z), "=r"(u.w)
                                 : "r"(a0 + (uint32_t)rr * 128u + (uint32_t)(((cc & 7) ^ (rr & 7)) << 4)));
                    const __nv_bfloat162* hh = (const __nv_bfloat162*)&u;
                    #pragma unroll
                    for (int k = 0; k < 4; ++k) { const float2 f = __bfloat1622float2(hh[k]); acc[2 * k] += f.x; acc[2 * k + 1] += f.y; }
                }
                // these were generic-proxy reads of a stage that TMA (the async proxy) overwrites once it is released: without
                // a proxy fence between the reads and the release the refill may overtake reads still in flight (seen as a
                // wrong bias partial in a few per cent of the steps, only when other kernels shared the GPU)
                fence_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(empty0 + 8u * st);
                if (++st == stages) { st = 0; ph ^= 1u; }
            }
            float* red = (float*)(smem_raw + (red_base - raw));     // [8 row groups][128 channels]
            #pragma unroll
            for (int k = 0; k < 8; ++k) red[rg * 128 + cc * 8 + k] = acc[k];
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (ok && te + m_tile * 128 < p.M_total) {
                float sum = 0.f;
                #pragma unroll
                for (int q = 0; q < 8; ++q) sum += red[q * 128 + te];
                p.bias_partial[(size_t)z * p.bias_ld + g * p.out_gx + m_tile * 128 + te] = sum;
            }
        }
        if (mbar_wait(accf, 0, abort_flag)) {
            tc_fence_after();
            const uint32_t t0 = tmem + ((uint32_t)(quad * 32) << 16);
            for (int kx = 0; kx < p.kw; ++kx) {
                const long long row_off = (long long)z * p.split_stride + (long long)(ky * p.kw + kx) * p.tap_stride +
                                          (long long)(g * p.out_gx + row) * p.ldo;
                for (int c = 0; c < 64; c += 16) {
                    uint32_t v[16];
                    tmem_ld16(t0 + (uint32_t)(kx * 64 + c), v);
                    tmem_ld_wait();
                    if (!row_ok) continue;
                    epi_chunk(p, v, nsteps <= 0, false, row_off, n_tile * 64 + c, g);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (threadIdx.x == 0 && p.status) atomicExch(p.status, 1);
        long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) { }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, ncols);
    }
}

}  // namespace tc
