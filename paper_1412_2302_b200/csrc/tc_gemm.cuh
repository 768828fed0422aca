// tcgen05 / TMEM / TMA GEMM core for sm_100a.
//
// One CTA computes one 128 x BN fp32 accumulator tile in tensor memory from
// bf16 operands staged in shared memory by TMA (128-byte swizzle), through a
// ring of STAGES buffers.  Warp roles: warp 0 = TMA producer, warp 1 = MMA
// issuer (one elected lane) and TMEM owner, warps 2..5 = epilogue (each reads
// the 32 TMEM lanes of its quadrant).  Three operand arrangements:
//   MODE_KK   A K-major, B K-major   conv fwd, conv bwd-data, FC fwd
//   MODE_KMN  A K-major, B MN-major  FC bwd-data (weights read untransposed)
//   MODE_MNMN A MN-major, B MN-major weight gradients (reduction over rows)
// A convolution is an implicit GEMM over a zero-padded flat NHWC grid: filter
// tap t reads the input rows of the output tile shifted by shift[t] rows, so
// every A tile is a plain 2-D TMA box; out-of-range rows are zero-filled by TMA.
// Every wait is bounded: on expiry the CTA raises *status and drains.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace tc {

enum { MODE_KK = 0, MODE_KMN = 1, MODE_MNMN = 2 };
enum { EPI_BF16 = 0, EPI_F32 = 1 };
constexpr int kThreads = 192;
constexpr int kMaxTaps = 25;
constexpr long long kWaitBudgetCycles = 400000000LL;  // ~0.2 s at 2 GHz

struct GemmParams {
    CUtensorMap tmA, tmB;
    int mode, epi;
    int m_tiles, n_tiles, groups, taps_grid, splits;  // grid decomposition (m fastest)
    int BN;            // MMA N (multiple of 16, <= 256)
    int kk;            // K=16 MMAs per stage (<= 4)
    int chunks;        // MODE_KK: 64-element K chunks per tap
    int steps_total;   // k-steps over the whole reduction (split evenly over `splits`)
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
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// bounded wait: returns false when the cycle budget ran out or another role aborted
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    long long t0 = clock64();
    while (true) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitBudgetCycles) { *abort_flag = 1; return false; }
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(bar) : "memory");
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
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
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
// instruction descriptor: bf16 x bf16 -> fp32, M = 128
__device__ __forceinline__ uint32_t instr_desc(int N, int a_mn, int b_mn) {
    uint32_t d = 0;
    d |= 1u << 4;                 // D format fp32
    d |= 1u << 7;                 // A bf16
    d |= 1u << 10;                // B bf16
    d |= (uint32_t)a_mn << 15;    // A major (0 = K)
    d |= (uint32_t)b_mn << 16;    // B major
    d |= (uint32_t)(N >> 3) << 17;
    d |= (uint32_t)(128 >> 4) << 24;
    return d;
}

constexpr int kABytes = 128 * 128;  // 128 rows x 64 bf16, or 2 boxes of 64 x 64

__host__ __device__ inline int b_stage_bytes(int mode, int BN) {
    return mode == MODE_KK ? BN * 128 : ((BN + 63) / 64) * 8192;
}
inline size_t smem_bytes(int mode, int BN, int stages) {
    return 1024 + (size_t)stages * (kABytes + b_stage_bytes(mode, BN)) + 256;
}

__global__ void __launch_bounds__(kThreads, 1) gemm_kernel(const __grid_constant__ GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const int bbytes = b_stage_bytes(p.mode, p.BN);
    const int stage_bytes = kABytes + bbytes;
    const uint32_t bar_base = base + p.stages * stage_bytes;       // full[8], empty[8], accum, tmem slot
    uint8_t* gen = smem_raw + (base - raw) + p.stages * stage_bytes;
    volatile int* abort_flag = (volatile int*)(gen + 160);
    volatile uint32_t* tmem_slot = (volatile uint32_t*)(gen + 144);
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 64u + 8u * s; };
    const uint32_t accum_bar = bar_base + 128u;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // tile decode (m fastest)
    int idx = blockIdx.x;
    const int m_tile = idx % p.m_tiles; idx /= p.m_tiles;
    const int n_tile = idx % p.n_tiles; idx /= p.n_tiles;
    const int g = idx % p.groups; idx /= p.groups;
    const int tap_g = idx % p.taps_grid; idx /= p.taps_grid;
    const int z = idx;
    const int m0 = m_tile * 128, n0 = n_tile * p.BN;
    const int per = (p.steps_total + p.splits - 1) / p.splits;
    const int s_begin = z * per;
    const int s_end = min(p.steps_total, s_begin + per);
    const int nsteps = max(0, s_end - s_begin);

    uint32_t ncols = 32;
    while ((int)ncols < p.BN) ncols <<= 1;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(accum_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32((const void*)tmem_slot), ncols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const uint32_t tx = (uint32_t)stage_bytes;
            for (int i = 0; i < nsteps; ++i) {
                const int s = s_begin + i, st = i % p.stages;
                if (!mbar_wait(empty_bar(st), ((i / p.stages) & 1) ^ 1, abort_flag)) break;
                const uint32_t sa = base + st * stage_bytes, sb = sa + kABytes;
                mbar_expect_tx(full_bar(st), tx);
                if (p.mode == MODE_KK) {
                    const int tap = s / p.chunks, ch = s - tap * p.chunks;
                    tma_load_2d(sa, &p.tmA, p.a_x0 + g * p.a_gx + ch * 64, m0 + p.shift[tap], full_bar(st));
                    tma_load_2d(sb, &p.tmB, ch * 64, tap * p.b_tap_rows + g * p.b_g_rows + n0, full_bar(st));
                } else if (p.mode == MODE_KMN) {
                    tma_load_2d(sa, &p.tmA, s * 64, m0, full_bar(st));
                    for (int j = 0; j < (p.BN + 63) / 64; ++j)
                        tma_load_2d(sb + j * 8192, &p.tmB, n0 + 64 * j, s * 64, full_bar(st));
                } else {
                    const int q = s * 64;
                    for (int j = 0; j < 2; ++j)
                        tma_load_2d(sa + j * 8192, &p.tmA, g * p.a_gx + m0 + 64 * j, q, full_bar(st));
                    for (int j = 0; j < (p.BN + 63) / 64; ++j)
                        tma_load_2d(sb + j * 8192, &p.tmB, g * p.b_gx + n0 + 64 * j, q + p.shift[tap_g], full_bar(st));
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const int a_mn = p.mode == MODE_MNMN, b_mn = p.mode != MODE_KK;
            const uint32_t idesc = instr_desc(p.BN, a_mn, b_mn);
            const uint32_t a_adv = a_mn ? 2048u : 32u, b_adv = b_mn ? 2048u : 32u;
            const uint32_t a_lbo = a_mn ? 8192u : 16u, b_lbo = b_mn ? 8192u : 16u;
            bool ok = true;
            for (int i = 0; i < nsteps && ok; ++i) {
                const int st = i % p.stages;
                ok = mbar_wait(full_bar(st), (i / p.stages) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t sa = base + st * stage_bytes, sb = sa + kABytes;
                for (int j = 0; j < p.kk; ++j)
                    umma(tmem, smem_desc(sa + j * a_adv, a_lbo, 1024), smem_desc(sb + j * b_adv, b_lbo, 1024),
                         idesc, (i > 0 || j > 0) ? 1u : 0u);
                umma_commit(empty_bar(st));
            }
            umma_commit(accum_bar);
        }
    } else {
        // ------------------------------------------------------------ epilogue
        const int quad = warp & 3;
        const int r = quad * 32 + lane;          // row within the tile = TMEM lane
        bool ok = mbar_wait(accum_bar, 0, abort_flag);
        tc_fence_after();
        if (ok) {
            bool row_ok, pad_row = false;
            long long row_off;
            if (p.mode == MODE_MNMN) {
                row_ok = (m0 + r) < p.M_total;
                row_off = (long long)z * p.split_stride + (long long)tap_g * p.tap_stride +
                          (long long)(g * p.out_gx + m0 + r) * p.ldo;
            } else {
                const int row = m0 + r;
                row_ok = row < p.M_total;
                if (p.Hp > 0) {
                    const int x = row % p.Wp, y = (row / p.Wp) % p.Hp;
                    pad_row = (x >= p.W) || (y >= p.H);
                }
                row_off = (long long)z * p.split_stride + (long long)row * p.ldo + g * p.out_gx;
            }
            for (int c = 0; c < p.BN; c += 16) {
                uint32_t v[16];
                tmem_ld16(tmem + ((uint32_t)(quad * 32) << 16) + (uint32_t)c, v);
                tmem_ld_wait();
                if (!row_ok) continue;
                const int col0 = n0 + c;
                if (nsteps == 0) {
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
                } else {
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
            }
        }
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

}  // namespace tc
