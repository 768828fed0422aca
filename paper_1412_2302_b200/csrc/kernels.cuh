// HBM-bound kernels of the AlexNet training step: preprocessing gather, LRN,
// max-pool, split-K reductions with fused bias/ReLU/dropout, softmax
// cross-entropy, bias gradients, momentum update, replica average, layout
// permutations.  Activations are bf16 in a zero-padded flat NHWC grid
// [B][Hp][Wp][C] whose valid region is the top-left H x W of every image; pad
// positions always hold zero.  All accesses are 16-byte vectors along C.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace kn {

// Programmatic dependent launch: every kernel of the step lets the next launch of its stream start its blocks early
// (they become resident as the SMs drain) and itself waits here, before its first access to global memory, until the
// kernels before it have completed and their writes are visible.  Without the launch attribute both are no-ops.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_sync() { pdl_trigger(); pdl_wait(); }

// ---------------------------------------------------------------- counter hash
// SplitMix64 finaliser over key + golden*(idx+1); key = finalise(seed ^ stream<<56 ^ replica<<48 ^ step).
__host__ __device__ __forceinline__ uint64_t mix64(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}
__host__ __device__ __forceinline__ uint64_t stream_key(uint64_t seed, uint64_t stream, uint64_t replica, uint64_t step) {
    return mix64(seed ^ (stream << 56) ^ (replica << 48) ^ step);
}
__host__ __device__ __forceinline__ uint64_t draw(uint64_t key, uint64_t idx) {
    return mix64(key + 0x9E3779B97F4A7C15ULL * (idx + 1));
}

__device__ __forceinline__ void unpack8(const uint4& u, float* f) {
    const __nv_bfloat162* h = (const __nv_bfloat162*)&u;
    #pragma unroll
    for (int i = 0; i < 4; ++i) { float2 t = __bfloat1622float2(h[i]); f[2 * i] = t.x; f[2 * i + 1] = t.y; }
}
__device__ __forceinline__ uint4 pack8(const float* f) {
    uint4 u;
    __nv_bfloat162* h = (__nv_bfloat162*)&u;
    #pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
    return u;
}

// ------------------------------------------------------------- preprocessing
// Per image: crop offset (ox, oy) in [0,29]^2 and flip bit from the hash
// (stream 1, idx = image).  out = u8[sy][sx][c] - mean[sy][sx][c] with
// sy = oy + Y, sx = ox + (flip ? 226 - X : X), written as bf16 in the 4x4
// space-to-depth layout [B][57][57][48], channel = ((Y%4)*4 + X%4)*3 + c,
// with row/column 227 of the 228-padded image set to zero.
// Optional intensity augmentation (Krizhevsky et al. 2012, section 4.1; the paper's experiments leave it out): every
// pixel of image n gets the RGB offset d = sum_i pl[.][i] * alpha_i with pl[c][i] = eigvec[c][i] * eigval[i] and
// alpha_i = sigma * z_i, z_i standard normal from the hash (stream 10, index 3 n + i, Box-Muller as in the init kernel).
struct ColorAug { float pl[9]; float sigma; uint64_t key; };
__device__ __forceinline__ float normal_draw(uint64_t key, uint64_t idx) {
    const uint64_t r = draw(key, idx);
    const float u1 = ((float)(r >> 40) + 1.f) * (1.f / 16777216.f);
    const float u2 = (float)((r >> 16) & 0xFFFFFF) * (1.f / 16777216.f);
    return sqrtf(-2.f * logf(u1)) * cospif(2.f * u2);
}
// One block = one image and four rows of the 228-padded crop (one row `by` of the space-to-depth grid): the four source rows
// of the uint8 image (768 bytes each) and of the mean image (768 floats each) come to shared memory in coalesced loads, then
// thread (bx, dy) forms its 12 values (4 pixels x 3 colours) from there and stores 24 contiguous bytes; a warp writes 768
// contiguous bytes.  grid: (57, B), 256 threads.
template <bool AUG>
__global__ void __launch_bounds__(256) preprocess_kernel(const uint8_t* __restrict__ img, const float* __restrict__ mean,
                                                         __nv_bfloat16* __restrict__ out, int32_t* __restrict__ cf_out,
                                                         int B, uint64_t key, int eval_mode, const ColorAug aug) {
    pdl_sync();
    __shared__ uint4 s_img[4][49];        // rows padded by 16 bytes: the four rows start in different banks
    __shared__ float s_mean[4][769];      // row pitch = 1 mod 32 words: the warp's 8 bx x 4 dy reads (12 words apart per bx) hit 32 banks
    const int by = blockIdx.x, n = blockIdx.y, tid = threadIdx.x;
    const uint64_t r = draw(key, (uint64_t)n);
    // evaluation: the centre 227 x 227 window, never flipped
    const int ox = eval_mode ? 14 : (int)((r & 0xFFFF) % 30), oy = eval_mode ? 14 : (int)(((r >> 16) & 0xFFFF) % 30);
    const int flip = eval_mode ? 0 : (int)((r >> 32) & 1);
    if (cf_out && by == 0 && tid == 0) { cf_out[3 * n] = ox; cf_out[3 * n + 1] = oy; cf_out[3 * n + 2] = flip; }
    for (int i = tid; i < 4 * 48; i += 256) {
        const int dy = i / 48, j = i - dy * 48, Y = by * 4 + dy;
        if (Y < 227) s_img[dy][j] = __ldg((const uint4*)(img + (size_t)n * 196608 + (size_t)(oy + Y) * 768) + j);
    }
    #pragma unroll
    for (int i = tid; i < 4 * 768; i += 256) {     // one float per lane: conflict-free stores at the odd row pitch
        const int dy = i / 768, j = i - dy * 768, Y = by * 4 + dy;
        if (Y < 227) s_mean[dy][j] = __ldg(mean + (size_t)(oy + Y) * 768 + j);
    }
    __syncthreads();
    if (tid >= 228) return;
    const int dy = tid & 3, bx = tid >> 2;
    float shift[3] = {0.f, 0.f, 0.f};
    if (AUG && !eval_mode) {
        const float a0 = aug.sigma * normal_draw(aug.key, 3ull * n), a1 = aug.sigma * normal_draw(aug.key, 3ull * n + 1),
                    a2 = aug.sigma * normal_draw(aug.key, 3ull * n + 2);
        #pragma unroll
        for (int c = 0; c < 3; ++c) shift[c] = aug.pl[3 * c] * a0 + aug.pl[3 * c + 1] * a1 + aug.pl[3 * c + 2] * a2;
    }
    const int Y = by * 4 + dy;
    const uint8_t* ib = (const uint8_t*)s_img[dy];
    const float* mb = s_mean[dy];
    float v[12];
    #pragma unroll
    for (int dx = 0; dx < 4; ++dx) {
        const int X = bx * 4 + dx;
        if (Y < 227 && X < 227) {
            const int s3 = (ox + (flip ? 226 - X : X)) * 3;
            #pragma unroll
            for (int c = 0; c < 3; ++c) v[dx * 3 + c] = ((float)ib[s3 + c] - mb[s3 + c]) + shift[c];
        } else {
            v[dx * 3] = v[dx * 3 + 1] = v[dx * 3 + 2] = 0.f;
        }
    }
    uint2* o = (uint2*)(out + ((size_t)(n * 57 + by) * 57 + bx) * 48 + dy * 12);
    #pragma unroll
    for (int i = 0; i < 3; ++i) {
        const __nv_bfloat162 lo = __floats2bfloat162_rn(v[4 * i], v[4 * i + 1]), hi = __floats2bfloat162_rn(v[4 * i + 2], v[4 * i + 3]);
        o[i] = make_uint2(*(const uint32_t*)&lo, *(const uint32_t*)&hi);
    }
}

// ----------------------------------------------------------------------- LRN
// All index arithmetic below is 32-bit: the largest activation tensor of a batch of 1024 has
// 1024*57*57*12 < 2^31 sixteen-byte vectors.
__device__ __forceinline__ float rsqrt_fast(float x) { float y; asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ float sqrt_fast(float x) { float y; asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
// s^-beta and 1/s; the exponent 0.75 of the paper's network costs two special-function instructions
// B75: the exponent is known to be 0.75 at compile time (the fused kernels of the training step are instantiated both ways,
// so that their inner loops carry no test of beta)
template <bool B75>
__device__ __forceinline__ void pow_neg_t(float s, float beta, float& sp, float& rs) {
    if (B75) { const float r = rsqrt_fast(s); sp = r * sqrt_fast(r); rs = r * r; }
    else { sp = exp2f(-beta * __log2f(s)); rs = __fdividef(1.f, s); }
}
__device__ __forceinline__ void pow_neg(float s, float beta, float& sp, float& rs) {
    if (beta == 0.75f) pow_neg_t<true>(s, beta, sp, rs); else pow_neg_t<false>(s, beta, sp, rs);
}
// b_c = a_c * (k + alpha * sum_{c' in [c-2,c+2] clipped} a_c'^2)^(-beta); one thread = 8 channels of one pixel.
template <bool B75>
__device__ __forceinline__ uint4 lrn_fwd8_t(const uint4* ap, bool has_l, bool has_r, float alpha, float beta, float k) {
    const uint4 zero = make_uint4(0, 0, 0, 0);
    float f[24];
    unpack8(has_l ? __ldg(ap - 1) : zero, f);
    unpack8(__ldg(ap), f + 8);
    unpack8(has_r ? __ldg(ap + 1) : zero, f + 16);
    float sq[12];
    #pragma unroll
    for (int i = 0; i < 12; ++i) sq[i] = f[6 + i] * f[6 + i];
    float o[8];
    #pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float ss = (sq[i] + sq[i + 1]) + (sq[i + 2] + sq[i + 3]) + sq[i + 4];
        float sp, rs;
        pow_neg_t<B75>(fmaf(alpha, ss, k), beta, sp, rs);
        o[i] = f[8 + i] * sp;
    }
    return pack8(o);
}
__device__ __forceinline__ uint4 lrn_fwd8(const uint4* ap, bool has_l, bool has_r, float alpha, float beta, float k) {
    return beta == 0.75f ? lrn_fwd8_t<true>(ap, has_l, has_r, alpha, beta, k) : lrn_fwd8_t<false>(ap, has_l, has_r, alpha, beta, k);
}
__global__ void __launch_bounds__(256) lrn_fwd_kernel(const __nv_bfloat16* __restrict__ a, __nv_bfloat16* __restrict__ b,
                                                      unsigned total, unsigned cpr, float alpha, float beta, float k) {
    pdl_sync();
    const unsigned t = blockIdx.x * 256u + threadIdx.x;
    if (t >= total) return;
    const unsigned ch = t % cpr;
    ((uint4*)b)[t] = lrn_fwd8((const uint4*)a + t, ch > 0, ch < cpr - 1, alpha, beta, k);
}
// da_m = [a_m > 0] * ( g_m s_m^-beta - 2 alpha beta a_m sum_{c in [m-2,m+2]} g_c a_c s_c^(-beta-1) )
// (the ReLU mask of the convolution that produced a is applied here).  One thread = 8 channels of one
// pixel; it needs s for the 12 channels c0-2 .. c0+9 and a for c0-4 .. c0+11.
__device__ __forceinline__ uint4 lrn_bwd8(const float* fa, const float* fg, float alpha, float beta, float k) {
    float sq[16];
    #pragma unroll
    for (int i = 0; i < 16; ++i) sq[i] = fa[4 + i] * fa[4 + i];
    float sp[12], tt[12];   // channels c0-2 .. c0+9
    #pragma unroll
    for (int i = 0; i < 12; ++i) {
        const float ss = (sq[i] + sq[i + 1]) + (sq[i + 2] + sq[i + 3]) + sq[i + 4];
        float rs;
        pow_neg(fmaf(alpha, ss, k), beta, sp[i], rs);
        tt[i] = fg[6 + i] * fa[6 + i] * sp[i] * rs;
    }
    const float c2 = 2.f * alpha * beta;
    float o[8];
    #pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float acc = (tt[i] + tt[i + 1]) + (tt[i + 2] + tt[i + 3]) + tt[i + 4];
        const float am = fa[8 + i];
        const float v = fmaf(fg[8 + i], sp[i + 2], -c2 * am * acc);
        o[i] = am > 0.f ? v : 0.f;
    }
    return pack8(o);
}
__global__ void __launch_bounds__(256) lrn_bwd_kernel(const __nv_bfloat16* __restrict__ a, const __nv_bfloat16* __restrict__ g,
                                                      __nv_bfloat16* __restrict__ da, unsigned total, unsigned cpr,
                                                      float alpha, float beta, float k) {
    pdl_sync();
    const unsigned t = blockIdx.x * 256u + threadIdx.x;
    if (t >= total) return;
    const unsigned ch = t % cpr;
    const uint4* ap = (const uint4*)a + t;
    const uint4* gp = (const uint4*)g + t;
    const uint4 zero = make_uint4(0, 0, 0, 0);
    const bool has_l = ch > 0, has_r = ch < cpr - 1;
    float fa[24], fg[24];
    unpack8(has_l ? __ldg(ap - 1) : zero, fa);
    unpack8(__ldg(ap), fa + 8);
    unpack8(has_r ? __ldg(ap + 1) : zero, fa + 16);
    unpack8(has_l ? __ldg(gp - 1) : zero, fg);
    unpack8(__ldg(gp), fg + 8);
    unpack8(has_r ? __ldg(gp + 1) : zero, fg + 16);
    ((uint4*)da)[t] = lrn_bwd8(fa, fg, alpha, beta, k);
}

// ------------------------------------------------------------------ max pool
// 3x3 stride 2, no padding; first maximum in (ky,kx) row-major order wins; argmax = ky*3+kx.
// grid: (ceil(Wo*cpr / 256), Ho, B); one thread = 8 channels of one output pixel.
__global__ void __launch_bounds__(256) pool_fwd_kernel(const __nv_bfloat16* __restrict__ x, __nv_bfloat16* __restrict__ y,
                                                       uint8_t* __restrict__ arg, int cpr, int Hpi, int Wpi,
                                                       int Ho, int Wo, int Hpo, int Wpo) {
    pdl_sync();
    const unsigned i = blockIdx.x * 256u + threadIdx.x;
    if (i >= (unsigned)(Wo * cpr)) return;
    const int ox = i / cpr, ch = i - ox * cpr;
    const int oy = blockIdx.y, n = blockIdx.z;
    float best[8]; int bi[8];
    const uint4* xp = (const uint4*)x + ((size_t)(n * Hpi + 2 * oy) * Wpi + 2 * ox) * cpr + ch;
    #pragma unroll
    for (int ky = 0; ky < 3; ++ky)
        #pragma unroll
        for (int kx = 0; kx < 3; ++kx) {
            float f[8];
            unpack8(__ldg(xp + (ky * Wpi + kx) * cpr), f);
            #pragma unroll
            for (int q = 0; q < 8; ++q)
                if ((ky == 0 && kx == 0) || f[q] > best[q]) { best[q] = f[q]; bi[q] = ky * 3 + kx; }
        }
    ((uint4*)y)[((size_t)(n * Hpo + oy) * Wpo + ox) * cpr + ch] = pack8(best);
    uint2 ab;
    ab.x = bi[0] | (bi[1] << 8) | (bi[2] << 16) | (bi[3] << 24);
    ab.y = bi[4] | (bi[5] << 8) | (bi[6] << 16) | (bi[7] << 24);
    ((uint2*)arg)[((size_t)(n * Ho + oy) * Wo + ox) * cpr + ch] = ab;
}
// dx[y][x] = sum over the (up to 4) windows containing (y,x) whose argmax points at it; optional ReLU mask.
// grid: (ceil(Wpi*cpr / 256), Hpi, B); one thread = 8 channels of one input pixel (pad pixels get zero).
__device__ __forceinline__ void pool_bwd8(const __nv_bfloat16* __restrict__ dy, const uint8_t* __restrict__ arg, float* acc,
                                          int n, int y, int x, int ch, int cpr, int Ho, int Wo, int Hpo, int Wpo) {
    const int oy_lo = max(0, (y - 1) >> 1), oy_hi = min(Ho - 1, y >> 1);
    const int ox_lo = max(0, (x - 1) >> 1), ox_hi = min(Wo - 1, x >> 1);
    for (int oy = oy_lo; oy <= oy_hi; ++oy)
        for (int ox = ox_lo; ox <= ox_hi; ++ox) {
            const unsigned code = (unsigned)((y - 2 * oy) * 3 + (x - 2 * ox)) * 0x01010101u;
            const uint2 ab = __ldg((const uint2*)arg + ((size_t)(n * Ho + oy) * Wo + ox) * cpr + ch);
            float f[8];
            unpack8(__ldg((const uint4*)dy + ((size_t)(n * Hpo + oy) * Wpo + ox) * cpr + ch), f);
            // byte-wise equality of the eight argmax codes with this pixel's code
            const unsigned e0 = ab.x ^ code, e1 = ab.y ^ code;
            #pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (((e0 >> (8 * q)) & 0xFFu) == 0u) acc[q] += f[q];
                if (((e1 >> (8 * q)) & 0xFFu) == 0u) acc[q + 4] += f[q + 4];
            }
        }
}
__global__ void __launch_bounds__(256) pool_bwd_kernel(const __nv_bfloat16* __restrict__ dy, const uint8_t* __restrict__ arg,
                                                       const __nv_bfloat16* __restrict__ relu_src, __nv_bfloat16* __restrict__ dx,
                                                       int cpr, int Hpi, int Wpi, int Hi, int Wi, int Ho, int Wo, int Hpo, int Wpo) {
    pdl_sync();
    const unsigned i = blockIdx.x * 256u + threadIdx.x;
    if (i >= (unsigned)(Wpi * cpr)) return;
    const int x = i / cpr, ch = i - x * cpr;
    const int y = blockIdx.y, n = blockIdx.z;
    const size_t t = ((size_t)(n * Hpi + y) * Wpi + x) * cpr + ch;
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (y < Hi && x < Wi) {
        pool_bwd8(dy, arg, acc, n, y, x, ch, cpr, Ho, Wo, Hpo, Wpo);
        if (relu_src) {
            float m[8];
            unpack8(__ldg((const uint4*)relu_src + t), m);
            #pragma unroll
            for (int q = 0; q < 8; ++q) acc[q] = m[q] > 0.f ? acc[q] : 0.f;
        }
    }
    ((uint4*)dx)[t] = pack8(acc);
}

// ------------------------------------------------- LRN + pool fused (the training step)
// Geometry is a template parameter (the network's two LRN layers): CPR 16-byte vectors per pixel, input WI x HI.
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d; asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel)); return d;
}
// Forward: p = maxpool(LRN(a)) without writing the normalised tensor.  One block = one image, OPR output rows and CV
// of the CPR channel vectors: the 2*OPR+1 input rows they cover are normalised once into shared memory as bf16 (the
// same rounding as lrn_fwd_kernel's output; channel neighbours outside the block's range come from global memory),
// then pooled from there.  The normalised values are non-negative (a is a ReLU output; the sign bit is cleared so that
// a -0 cannot occur), so bf16 bit patterns order like the values: each candidate becomes the 32-bit key
// (bits << 16) | (8 - tap) and the window's maximum key carries the largest value and, among equal values, the first
// tap in scan order - pool_fwd_kernel's tie rule.
// grid: (ceil(HO / OPR), CPR / CV, B); dynamic shared memory (2*OPR+1) * WI * CV * 16 bytes.
template <int CPR, int CV, int WI, int HI, int OPR, int NT, bool B75>
__global__ void __launch_bounds__(NT) lrn_pool_fwd_kernel(const __nv_bfloat16* __restrict__ a, __nv_bfloat16* __restrict__ y,
                                                          uint8_t* __restrict__ arg, int Hpi, int Wpi, int Hpo, int Wpo,
                                                          float alpha, float beta, float k) {
    pdl_sync();
    constexpr int RV = WI * CV, NR = 2 * OPR + 1, WO = (WI - 3) / 2 + 1, HO = (HI - 3) / 2 + 1;
    extern __shared__ uint4 nrm[];            // [row][x][vector]
    const int n = blockIdx.z, c0 = blockIdx.y * CV, oy0 = OPR * blockIdx.x, iy0 = 2 * oy0;
    const int nrows = min(NR, HI - iy0);
    for (int q = threadIdx.x; q < RV; q += NT) {
        const int x = q / CV, ch = c0 + q % CV;
        const uint4* ap = (const uint4*)a + ((size_t)(n * Hpi + iy0) * Wpi + x) * CPR + ch;
        for (int r = 0; r < nrows; ++r) {
            uint4 v = lrn_fwd8_t<B75>(ap + (size_t)r * Wpi * CPR, ch > 0, ch < CPR - 1, alpha, beta, k);
            v.x &= 0x7fff7fffu; v.y &= 0x7fff7fffu; v.z &= 0x7fff7fffu; v.w &= 0x7fff7fffu;
            nrm[r * RV + q] = v;
        }
    }
    __syncthreads();
    const int orows = min(OPR, HO - oy0);
    for (int t = threadIdx.x; t < orows * WO * CV; t += NT) {
        const int oyl = t / (WO * CV), q = t - oyl * (WO * CV);
        const int ox = q / CV, cv = q - ox * CV;
        const uint4* src = nrm + (2 * oyl * WI + 2 * ox) * CV + cv;
        uint32_t best[8];
        #pragma unroll
        for (int ky = 0; ky < 3; ++ky)
            #pragma unroll
            for (int kx = 0; kx < 3; ++kx) {
                const uint4 v = src[(ky * WI + kx) * CV];
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
                const uint32_t code = 8u - (uint32_t)(ky * 3 + kx);
                #pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t lo = prmt(w[i], code, 0x1054u);      // (low bf16 << 16) | code
                    const uint32_t hi = prmt(w[i], code, 0x3254u);      // (high bf16 << 16) | code
                    if (ky == 0 && kx == 0) { best[2 * i] = lo; best[2 * i + 1] = hi; }
                    else { best[2 * i] = max(best[2 * i], lo); best[2 * i + 1] = max(best[2 * i + 1], hi); }
                }
            }
        const int oy = oy0 + oyl;
        uint4 o;
        o.x = prmt(best[0], best[1], 0x7632u); o.y = prmt(best[2], best[3], 0x7632u);
        o.z = prmt(best[4], best[5], 0x7632u); o.w = prmt(best[6], best[7], 0x7632u);
        ((uint4*)y)[((size_t)(n * Hpo + oy) * Wpo + ox) * CPR + c0 + cv] = o;
        uint2 ab;     // tap = 8 - low byte of the key
        ab.x = 0x08080808u - prmt(prmt(best[0], best[1], 0x4040u), prmt(best[2], best[3], 0x4040u), 0x5410u);
        ab.y = 0x08080808u - prmt(prmt(best[4], best[5], 0x4040u), prmt(best[6], best[7], 0x4040u), 0x5410u);
        ((uint2*)arg)[((size_t)(n * HO + oy) * WO + ox) * CPR + c0 + cv] = ab;
    }
}
// Backward: da = LRN'(a, dn) with dn = maxpool'(dp, arg) formed in shared memory.  One block = one image and the two
// input rows 2j, 2j+1.  The pooling windows that reach these rows lie in the window rows j-1 (its last filter row) and
// j (its first two); windows of one row and one column parity do not overlap, so four passes (window row x parity),
// each thread adding the eight gradients of one window vector to the fp32 pixels its argmax codes name, form dn
// without atomics and in a fixed order.  Then one thread = 8 channels of one pixel (PPB pixels at a time): dn rounded
// to bf16 (as pool_bwd_kernel stores it), s^-beta, tt = dn a s^(-beta-1), the tt of the two channels on either side
// from the neighbouring threads through shared memory, and da with the ReLU mask of the convolution that produced a.
// Pad pixels of the grid get zero.  grid: (ceil(Hpi / 2), B); dynamic shared memory 2 * WI * CPR * 48 bytes.
template <int CPR, int WI, int HI, int PPB, int NT, bool B75, bool STAGE_A>
__global__ void __launch_bounds__(NT) pool_lrn_bwd_kernel(const __nv_bfloat16* __restrict__ a, const __nv_bfloat16* __restrict__ dp,
                                                          const uint8_t* __restrict__ arg, __nv_bfloat16* __restrict__ da,
                                                          int Hpi, int Wpi, int Hpo, int Wpo, float alpha, float beta, float k) {
    pdl_sync();
    static_assert(PPB * CPR <= NT, "one thread per vector of PPB pixels");
    constexpr int RV = WI * CPR, WO = (WI - 3) / 2 + 1, HO = (HI - 3) / 2 + 1;
    __shared__ float4 edge[2][NT];    // tt of the two lowest and two highest channels of every thread, for its neighbours
    extern __shared__ float dn[];     // [2 planes: channels 0-3 / 4-7 of a vector][2 rows][WI][CPR] float4 (conflict-free reads)
    constexpr int PLANE = 2 * RV * 4; // floats per plane
    uint4* const as = (uint4*)(dn + 2 * PLANE);     // then the block's two rows of a, [2][WI][CPR] vectors
    const int j = blockIdx.x, n = blockIdx.y, y0 = 2 * j;
    const uint4 zero4 = make_uint4(0, 0, 0, 0);
    if (y0 >= HI) {                   // pad rows of the grid
        for (int row = 0; row < 2 && y0 + row < Hpi; ++row)
            for (int i = threadIdx.x; i < Wpi * CPR; i += NT) ((uint4*)da)[(size_t)(n * Hpi + y0 + row) * Wpi * CPR + i] = zero4;
        return;
    }
    // every thread first fetches the (up to four) window vectors it will scatter: window rows j-1 and j, even and odd
    // columns; the loads are in flight while the tile is cleared
    static_assert(((WO + 1) / 2) * CPR <= NT, "one thread per window vector of a pass");
    const int wq = threadIdx.x / CPR, wch = threadIdx.x - wq * CPR;
    uint4 wdp[4]; uint2 warg[4]; bool has[4];
    #pragma unroll
    for (int pass = 0; pass < 4; ++pass) {
        const int oy = j - 1 + (pass >> 1), ox = 2 * wq + (pass & 1);
        has[pass] = oy >= 0 && oy < HO && ox < WO;
        if (has[pass]) {
            warg[pass] = __ldg((const uint2*)arg + ((size_t)(n * HO + oy) * WO + ox) * CPR + wch);
            wdp[pass] = __ldg((const uint4*)dp + ((size_t)(n * Hpo + oy) * Wpo + ox) * CPR + wch);
        }
    }
    // the two rows of a travel to shared memory asynchronously, behind the scatter passes (the LRN part then reads a and
    // its channel neighbours from there instead of waiting for global memory three times per vector)
    for (int i = threadIdx.x; STAGE_A && i < 2 * RV; i += NT) {
        const int row = i / RV, q = i - row * RV;
        if (y0 + row < HI) {
            const uint4* src = (const uint4*)a + (size_t)(n * Hpi + y0 + row) * Wpi * CPR + q;
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(as + i)), "l"(src) : "memory");
        }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    for (int i = threadIdx.x; i < 4 * RV; i += NT) ((float4*)dn)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    __syncthreads();
    #pragma unroll
    for (int pass = 0; pass < 4; ++pass) {
        const int oy = j - 1 + (pass >> 1), par = pass & 1;
        if (pass == 3) asm volatile("cp.async.wait_group 0;" ::: "memory");     // before the last barrier of the passes
        if (has[pass]) {
            const int ox = 2 * wq + par;
            float f[8];
            unpack8(wdp[pass], f);
            float* base = dn + ((2 * ox) * CPR + wch) * 4;
            const int r0 = 2 * oy - y0;            // window row 0 relative to the block's first row: -2 or 0
            #pragma unroll
            for (int q = 0; q < 8; ++q) {
                const int tap = (int)(((q < 4 ? warg[pass].x : warg[pass].y) >> (8 * (q & 3))) & 0xFFu);
                const int ky = (tap * 11) >> 5, kx = tap - 3 * ky;
                const int row = r0 + ky;
                if ((unsigned)row < 2u) base[(q >> 2) * PLANE + (row * WI + kx) * (CPR * 4) + (q & 3)] += f[q];
            }
        }
        __syncthreads();
    }
    const int px = threadIdx.x / CPR, ch = threadIdx.x - px * CPR;
    int it = 0;
    #pragma unroll 1
    for (int row = 0; row < 2; ++row) {
        const int yy = y0 + row;
        if (yy >= Hpi) break;
        uint4* out_row = (uint4*)da + (size_t)(n * Hpi + yy) * Wpi * CPR;
        if (yy >= HI) {
            for (int i = threadIdx.x; i < Wpi * CPR; i += NT) out_row[i] = zero4;
            continue;
        }
        for (int i = threadIdx.x; i < (Wpi - WI) * CPR; i += NT) out_row[WI * CPR + i] = zero4;     // pad columns
        #pragma unroll 1
        for (int p0 = 0; p0 < WI; p0 += PPB, ++it) {
            const int x = p0 + px;
            const bool valid = px < PPB && x < WI;
            float fa[24], g8[8], sp[8], tt[8];
            if (valid) {
                const float4* gp = (const float4*)dn + (row * WI + x) * CPR + ch;
                const float4 g0 = gp[0], g1 = gp[PLANE / 4];
                const float acc[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
                unpack8(pack8(acc), g8);
                if (STAGE_A) {
                    const uint4* ap = as + (row * WI + x) * CPR + ch;
                    unpack8(ch > 0 ? ap[-1] : zero4, fa);
                    unpack8(ap[0], fa + 8);
                    unpack8(ch < CPR - 1 ? ap[1] : zero4, fa + 16);
                } else {
                    const uint4* ap = (const uint4*)a + ((size_t)(n * Hpi + yy) * Wpi + x) * CPR + ch;
                    unpack8(ch > 0 ? __ldg(ap - 1) : zero4, fa);
                    unpack8(__ldg(ap), fa + 8);
                    unpack8(ch < CPR - 1 ? __ldg(ap + 1) : zero4, fa + 16);
                }
                float sq[12];
                #pragma unroll
                for (int i = 0; i < 12; ++i) sq[i] = fa[6 + i] * fa[6 + i];
                #pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float ss = (sq[i] + sq[i + 1]) + (sq[i + 2] + sq[i + 3]) + sq[i + 4];
                    float rs;
                    pow_neg_t<B75>(fmaf(alpha, ss, k), beta, sp[i], rs);
                    tt[i] = g8[i] * fa[8 + i] * sp[i] * rs;
                }
            } else {
                #pragma unroll
                for (int i = 0; i < 8; ++i) tt[i] = 0.f;
            }
            // tt of channels c0-2, c0-1 (left neighbour's two highest) and c0+8, c0+9 (right neighbour's two lowest)
            float4 l, r;
            if (CPR == 32) {
                // a pixel is exactly one warp: the neighbours are the adjacent lanes, no shared memory and no block barrier
                l.z = __shfl_up_sync(0xffffffffu, tt[6], 1); l.w = __shfl_up_sync(0xffffffffu, tt[7], 1);
                r.x = __shfl_down_sync(0xffffffffu, tt[0], 1); r.y = __shfl_down_sync(0xffffffffu, tt[1], 1);
                if (ch == 0) { l.z = 0.f; l.w = 0.f; }
                if (ch == CPR - 1) { r.x = 0.f; r.y = 0.f; }
            } else {
                float4* eb = edge[it & 1];
                eb[threadIdx.x] = make_float4(tt[0], tt[1], tt[6], tt[7]);
                __syncthreads();
                l = ch > 0 ? eb[threadIdx.x - 1] : make_float4(0, 0, 0, 0);
                r = ch < CPR - 1 ? eb[threadIdx.x + 1] : make_float4(0, 0, 0, 0);
            }
            if (valid) {
                float te[12];
                te[0] = l.z; te[1] = l.w; te[10] = r.x; te[11] = r.y;
                #pragma unroll
                for (int i = 0; i < 8; ++i) te[2 + i] = tt[i];
                const float c2 = 2.f * alpha * beta;
                float o[8];
                #pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float acc = (te[i] + te[i + 1]) + (te[i + 2] + te[i + 3]) + te[i + 4];
                    const float am = fa[8 + i];
                    const float v = fmaf(g8[i], sp[i], -c2 * am * acc);
                    o[i] = am > 0.f ? v : 0.f;
                }
                out_row[x * CPR + ch] = pack8(o);
            }
        }
    }
}

// ------------------------------------------------- split-K reductions (FC, wgrad)
// y[b][n] = act( sum_z ws[z][b][n] + bias[n] ) * keep(b*N + n) * scale -> bf16, or fp32 logits when out_f32.
__global__ void fc_reduce_fwd_kernel(const float* __restrict__ ws, int splits, long long split_stride,
                                     const float* __restrict__ bias, int B, int N, int relu,
                                     int use_dropout, uint64_t key, uint32_t thr24, float scale,
                                     __nv_bfloat16* __restrict__ out_bf16, float* __restrict__ out_f32,
                                     uint8_t* __restrict__ keep_out) {
    pdl_sync();
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= (long long)B * N) return;
    const int n = (int)(t % N);
    float v = 0.f;
    for (int z = 0; z < splits; ++z) v += ws[z * split_stride + t];
    v += bias[n];
    if (relu) v = fmaxf(v, 0.f);
    if (use_dropout == 2) {            // evaluation: the expectation of the mask instead of a mask
        v *= scale;
        if (keep_out) keep_out[t] = 1;
    } else if (use_dropout) {
        const bool keep = (uint32_t)(draw(key, (uint64_t)t) >> 40) >= thr24;
        if (keep_out) keep_out[t] = keep ? 1 : 0;
        v = keep ? v * scale : 0.f;
    } else if (keep_out) {
        keep_out[t] = 1;
    }
    if (out_f32) out_f32[t] = v; else out_bf16[t] = __float2bfloat16_rn(v);
}
// dx[b][k] = [mask[b][k] > 0] * scale * sum_z ws[z][b][k] -> bf16 (mask = the layer input, post ReLU and dropout);
// db[k] = sum_b dx[b][k] (of the bf16-rounded values: the bias gradient of the layer below), when db != nullptr.
// grid: K/32 blocks of 256 threads = 8 column quads x 32 row lanes; a thread owns four columns of the rows rl, rl + 32, ...
// (batch <= 128: at most four) and has all its loads in flight together.  K is a multiple of 4; larger batches take the
// rows in rounds of 128.
__global__ void __launch_bounds__(256) fc_reduce_bwd_kernel(const float* __restrict__ ws, int splits, long long split_stride,
                                                            const __nv_bfloat16* __restrict__ mask, float scale, int B, int K,
                                                            __nv_bfloat16* __restrict__ out, float* __restrict__ db) {
    pdl_sync();
    __shared__ float red[32][33];
    const int cq = threadIdx.x & 7, rl = threadIdx.x >> 3;
    const int c = blockIdx.x * 32 + 4 * cq;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    if (c < K) {
        for (int b0 = 0; b0 < B; b0 += 128) {
            float4 v[4];
            uint2 mk[4];
            #pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int b = b0 + rl + 32 * i;
                v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                mk[i] = make_uint2(0u, 0u);
                if (b < B) {
                    const size_t t = (size_t)b * K + c;
                    if (mask) mk[i] = __ldg((const uint2*)(mask + t));
                    for (int z = 0; z < splits; ++z) {
                        const float4 w = __ldg((const float4*)(ws + z * split_stride + t));
                        v[i].x += w.x; v[i].y += w.y; v[i].z += w.z; v[i].w += w.w;
                    }
                }
            }
            #pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int b = b0 + rl + 32 * i;
                if (b >= B) continue;
                float f[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
                if (mask) {
                    const __nv_bfloat162* m2 = (const __nv_bfloat162*)&mk[i];
                    const float2 ma = __bfloat1622float2(m2[0]), mb = __bfloat1622float2(m2[1]);
                    f[0] = ma.x > 0.f ? f[0] * scale : 0.f; f[1] = ma.y > 0.f ? f[1] * scale : 0.f;
                    f[2] = mb.x > 0.f ? f[2] * scale : 0.f; f[3] = mb.y > 0.f ? f[3] * scale : 0.f;
                }
                const __nv_bfloat162 lo = __floats2bfloat162_rn(f[0], f[1]), hi = __floats2bfloat162_rn(f[2], f[3]);
                *(uint2*)(out + (size_t)b * K + c) = make_uint2(*(const uint32_t*)&lo, *(const uint32_t*)&hi);
                const float2 ra = __bfloat1622float2(lo), rb = __bfloat1622float2(hi);
                acc[0] += ra.x; acc[1] += ra.y; acc[2] += rb.x; acc[3] += rb.y;
            }
        }
    }
    if (!db) return;
    #pragma unroll
    for (int k = 0; k < 4; ++k) red[rl][4 * cq + k] = acc[k];
    __syncthreads();
    if (threadIdx.x < 32 && blockIdx.x * 32 + threadIdx.x < K) {
        float s = 0.f;
        #pragma unroll
        for (int q = 0; q < 32; ++q) s += red[q][threadIdx.x];
        db[blockIdx.x * 32 + threadIdx.x] = s;
    }
}
// g[i] = sum_z ws[z][i]; conv1: entries of the 12x12 zero-padded filter outside 11x11 stay zero.
// The first `cout` threads also add the per-split bias-gradient partials: db[c] = sum_z bias_partial[z][c].
__global__ void wgrad_reduce_kernel(const float* __restrict__ ws, int splits, long long split_stride,
                                    long long total, float* __restrict__ g, int conv1_pad_mask,
                                    const float* __restrict__ bias_partial, int cout, float* __restrict__ db) {
    pdl_sync();
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= total) return;
    float v = 0.f;
    for (int z = 0; z < splits; ++z) v += ws[z * split_stride + t];
    if (conv1_pad_mask) {
        const int ch = (int)(t % 48), tap = (int)(t / (48 * 96));
        const int ky = (tap / 3) * 4 + (ch / 3) / 4, kx = (tap % 3) * 4 + (ch / 3) % 4;
        if (ky > 10 || kx > 10) v = 0.f;
    }
    g[t] = v;
    if (bias_partial && t < cout) {
        float b = 0.f;
        for (int z = 0; z < splits; ++z) b += bias_partial[(size_t)z * cout + t];
        db[t] = b;
    }
}

// db[c] = sum over rows of dy[row][c] (bf16 in, fp32 out), two stages: grid (ceil(C/64), row_splits)
// writes partial[split][C]; colsum_final_kernel adds the splits in a fixed order.
__global__ void colsum_kernel(const __nv_bfloat16* __restrict__ dy, long long rows, int C, float* __restrict__ partial) {
    pdl_sync();
    // block: 256 threads = 32 row-lanes x 8 column-chunks (8 channels each) -> 64 columns per block
    __shared__ float red[32][65];
    const int cc = threadIdx.x & 7, rl = threadIdx.x >> 3;
    const int c0 = blockIdx.x * 64 + cc * 8;
    const long long per = (rows + gridDim.y - 1) / gridDim.y;
    const long long r0 = (long long)blockIdx.y * per, r1 = min(rows, r0 + per);
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (c0 < C) {
        for (long long r = r0 + rl; r < r1; r += 32) {
            float f[8];
            unpack8(*(const uint4*)(dy + r * C + c0), f);
            #pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] += f[i];
        }
    }
    #pragma unroll
    for (int i = 0; i < 8; ++i) red[rl][cc * 8 + i] = acc[i];
    __syncthreads();
    if (threadIdx.x < 64) {
        float s = 0.f;
        for (int r = 0; r < 32; ++r) s += red[r][threadIdx.x];
        const int c = blockIdx.x * 64 + threadIdx.x;
        if (c < C) partial[(size_t)blockIdx.y * C + c] = s;
    }
}
__global__ void colsum_final_kernel(const float* __restrict__ partial, int splits, int C, float* __restrict__ db) {
    pdl_sync();
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    float s = 0.f;
    for (int z = 0; z < splits; ++z) s += partial[(size_t)z * C + c];
    db[c] = s;
}
// same for a row pitch that is not a multiple of 8 elements (the 1000-wide logits gradient)
__global__ void colsum_scalar_kernel(const __nv_bfloat16* __restrict__ dy, int rows, int C, float* __restrict__ db) {
    pdl_sync();
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    float s = 0.f;
    for (int r = 0; r < rows; ++r) s += __bfloat162float(dy[(size_t)r * C + c]);
    db[c] = s;
}

// ------------------------------------------------------ softmax cross-entropy
// one block per sample: p = softmax(z), loss_n = -log p[label], dz = (p - onehot)/B as bf16
__global__ void softmax_xent_kernel(const float* __restrict__ z, const int32_t* __restrict__ labels,
                                    __nv_bfloat16* __restrict__ dz, float* __restrict__ loss_n, int B, int N) {
    pdl_sync();
    __shared__ float red[32];
    const int n = blockIdx.x, tid = threadIdx.x;
    const float* zr = z + (size_t)n * N;
    float mx = -INFINITY;
    for (int j = tid; j < N; j += blockDim.x) mx = fmaxf(mx, zr[j]);
    for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(~0u, mx, o));
    if ((tid & 31) == 0) red[tid >> 5] = mx;
    __syncthreads();
    mx = red[0];
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w) mx = fmaxf(mx, red[w]);
    __syncthreads();
    float sum = 0.f;
    for (int j = tid; j < N; j += blockDim.x) sum += expf(zr[j] - mx);
    for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(~0u, sum, o);
    if ((tid & 31) == 0) red[tid >> 5] = sum;
    __syncthreads();
    sum = 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) sum += red[w];
    const int lab = labels[n];
    const float inv = 1.f / sum, invB = 1.f / (float)B;
    for (int j = tid; j < N; j += blockDim.x) {
        const float pj = expf(zr[j] - mx) * inv;
        dz[(size_t)n * N + j] = __float2bfloat16_rn((pj - (j == lab ? 1.f : 0.f)) * invB);
    }
    if (tid == 0) loss_n[n] = -(zr[lab] - mx - logf(sum));
}
// The training step's form of the three kernels fc_reduce_fwd (fc8), softmax_xent and mean in one launch: block n adds the
// split-K partials of its row of logits in split order, adds the bias, stores z (fp32 logits), then softmax, loss_n and dz as
// above; the block that finishes last (a counter in global memory, reset for the next launch) averages loss_n in index order,
// so the result does not depend on which block that is.  Same arithmetic as the separate kernels.
__global__ void __launch_bounds__(256) fc8_softmax_xent_kernel(const float* __restrict__ ws, int splits, long long split_stride,
                                                               const float* __restrict__ bias, float* __restrict__ z,
                                                               const int32_t* __restrict__ labels, __nv_bfloat16* __restrict__ dz,
                                                               float* __restrict__ loss_n, float* __restrict__ loss_mean,
                                                               int* __restrict__ done_counter, int B, int N) {
    pdl_sync();
    __shared__ float red[32];
    __shared__ __align__(16) float zs[1024];
    __shared__ int last;
    const int n = blockIdx.x, tid = threadIdx.x;
    float mx = -INFINITY;
    if ((N & 3) == 0) {
        // four columns per thread, the loads of all splits in flight together (the maximum does not depend on which thread
        // sees which column; the sums below keep the column -> thread mapping of softmax_xent_kernel)
        for (int j = 4 * tid; j < N; j += 1024) {
            const long long t = (long long)n * N + j;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            #pragma unroll 4
            for (int q = 0; q < splits; ++q) {
                const float4 w = __ldg((const float4*)(ws + q * split_stride + t));
                v.x += w.x; v.y += w.y; v.z += w.z; v.w += w.w;
            }
            const float4 b4 = __ldg((const float4*)(bias + j));
            v.x += b4.x; v.y += b4.y; v.z += b4.z; v.w += b4.w;
            *(float4*)(z + t) = v;
            *(float4*)(zs + j) = v;
            mx = fmaxf(fmaxf(mx, fmaxf(v.x, v.y)), fmaxf(v.z, v.w));
        }
    } else {
        for (int j = tid; j < N; j += 256) {
            const long long t = (long long)n * N + j;
            float v = 0.f;
            for (int q = 0; q < splits; ++q) v += ws[q * split_stride + t];
            v += bias[j];
            z[t] = v;
            zs[j] = v;
            mx = fmaxf(mx, v);
        }
    }
    for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(~0u, mx, o));
    if ((tid & 31) == 0) red[tid >> 5] = mx;
    __syncthreads();
    mx = red[0];
    for (int w = 1; w < 8; ++w) mx = fmaxf(mx, red[w]);
    __syncthreads();
    float sum = 0.f;
    for (int j = tid; j < N; j += 256) sum += expf(zs[j] - mx);
    for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(~0u, sum, o);
    if ((tid & 31) == 0) red[tid >> 5] = sum;
    __syncthreads();
    sum = 0.f;
    for (int w = 0; w < 8; ++w) sum += red[w];
    const int lab = labels[n];
    const float inv = 1.f / sum, invB = 1.f / (float)B;
    for (int j = tid; j < N; j += 256) {
        const float pj = expf(zs[j] - mx) * inv;
        dz[(size_t)n * N + j] = __float2bfloat16_rn((pj - (j == lab ? 1.f : 0.f)) * invB);
    }
    if (tid == 0) {
        loss_n[n] = -(zs[lab] - mx - logf(sum));
        __threadfence();
        last = atomicAdd(done_counter, 1) == B - 1;
    }
    __syncthreads();
    if (!last) return;
    __threadfence();
    float s = 0.f;
    for (int i = tid; i < B; i += 256) s += __ldcg(loss_n + i);
    for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(~0u, s, o);
    __syncthreads();
    if ((tid & 31) == 0) red[tid >> 5] = s;
    __syncthreads();
    if (tid == 0) {
        float t = 0.f;
        for (int w = 0; w < 8; ++w) t += red[w];
        *loss_mean = t / (float)B;
        *done_counter = 0;
    }
}
// one float to wherever dst points (device memory, or pinned host memory mapped into the device's address space): the
// loss read-back without a copy engine, whose queue a batch upload of 25 MB may occupy
__global__ void store_value_kernel(const float* __restrict__ src, float* __restrict__ dst) {
    pdl_sync();
    *dst = *src;
    __threadfence_system();
}
__global__ void mean_kernel(const float* __restrict__ v, int n, float* __restrict__ out) {
    pdl_sync();
    __shared__ float red[32];
    float s = 0.f;
    for (int i = threadIdx.x; i < n; i += blockDim.x) s += v[i];
    for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(~0u, s, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += red[w];
        *out = t / (float)n;
    }
}

// top-1 / top-5 counting: one block per sample.  rank of the label = logits strictly greater than it plus equal
// logits with a smaller class index; the sample counts for top-k when rank < k.  counts[0] += top-1, counts[1] += top-5
// (integer atomics: the result does not depend on the order).
__global__ void topk_count_kernel(const float* __restrict__ z, const int32_t* __restrict__ labels, int N, int32_t* __restrict__ counts) {
    pdl_sync();
    __shared__ int red[32];
    const int n = blockIdx.x, lab = labels[n];
    const float* zr = z + (size_t)n * N;
    const float zl = zr[lab];
    int c = 0;
    for (int j = threadIdx.x; j < N; j += blockDim.x) {
        const float v = zr[j];
        c += (v > zl) || (v == zl && j < lab);
    }
    for (int o = 16; o; o >>= 1) c += __shfl_xor_sync(~0u, c, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        int rank = 0;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) rank += red[w];
        if (rank < 1) atomicAdd(counts, 1);
        if (rank < 5) atomicAdd(counts + 1, 1);
    }
}

// ------------------------------------------------ momentum update and average
// transposed bf16 copies of the grouped conv filters for the backward-data pass:
// wt[tap][g*cig + ci][co'] = wf[tap][g*cog + co'][ci]
struct TransposeJob { long long src_off, dst_off; int taps, cout, cig, groups; long long count; };
struct TransposeJobs { TransposeJob j[5]; int n; int tile0[6]; };   // tile0: first 32 x 32 tile of each job in sgd_update_conv_kernel's grid
// one parameter of the momentum update: v <- mu v - d w - lr g (d = lr * weight decay, or 0); w <- w + v.
// Used by the update kernel and by the FC weight-gradient epilogue that applies the update in place, so that both
// give bit-identical results.
__device__ __forceinline__ void sgd_step(float& w, float& v, float g, float d, float lr, float mu) {
    v = fmaf(mu, v, fmaf(-d, w, -lr * g));
    w += v;
}
// v <- mu v - lr wd w [i < n_decay] - lr g ; w <- w + v ; bf16 shadow of w.  22 bytes per parameter.
// Updates the 16-byte vectors [begin4, n4) of the internal order: everything after the conv filters (which
// sgd_update_conv_kernel takes), or only the biases when the FC weight-gradient kernel has already updated the FC weights.
// gscale multiplies the gradient first (1 for a single replica: exact; 1/R for a gradient summed over R replicas).
__global__ void sgd_update_kernel(float* __restrict__ w, float* __restrict__ v, const float* __restrict__ g,
                                  __nv_bfloat16* __restrict__ shadow, long long begin4, long long n4, long long n_decay4,
                                  float lr, float mu, float wd, float gscale) {
    pdl_sync();
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = begin4 + (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
        float4 wv = ((float4*)w)[i], vv = ((float4*)v)[i];
        const float4 gv = ((const float4*)g)[i];
        const float d = i < n_decay4 ? lr * wd : 0.f;
        sgd_step(wv.x, vv.x, gscale * gv.x, d, lr, mu);
        sgd_step(wv.y, vv.y, gscale * gv.y, d, lr, mu);
        sgd_step(wv.z, vv.z, gscale * gv.z, d, lr, mu);
        sgd_step(wv.w, vv.w, gscale * gv.w, d, lr, mu);
        ((float4*)w)[i] = wv;
        ((float4*)v)[i] = vv;
        __nv_bfloat162 lo2 = __floats2bfloat162_rn(wv.x, wv.y), hi2 = __floats2bfloat162_rn(wv.z, wv.w);
        ((uint2*)shadow)[i] = make_uint2(*(uint32_t*)&lo2, *(uint32_t*)&hi2);
    }
}
// The same update for the conv filters, tiled so that the transposed bf16 copies are written in runs: one block = one tap,
// 32 output channels and 32 input channels of one layer.  Thread (r, c4) updates the four consecutive input channels
// 4*c4 .. 4*c4+3 of output channel r (the source order [tap][cout][cig]: 128-byte runs per row), the bf16 values cross a
// shared-memory tile, and thread (ci, q) writes four consecutive output channels of input channel ci to the transposed copy
// [tap][cin][cog] (64-byte runs; a thread that walked the source order would write single elements).  Same arithmetic as sgd_update_kernel.
// With src.on the kernel also forms the conv gradients it consumes: the weight-gradient kernels leave fp32 partials per row
// split (and bias-gradient partials), and instead of a reduction launch per layer the update adds them here, in split
// order and with conv1's pad entries zeroed - wgrad_reduce_kernel's arithmetic - and stores the sums to g as that kernel does.
struct ConvSplitSrc {
    int on;
    int splits[5], cout[5];
    const float* ws[5]; long long stride[5];       // layer l: ws[l][z * stride[l] + index within the layer's filters]
    const float* bpart[5]; long long b_off4[5];    // bias partials [z][cout]; first 16-byte vector of the layer's biases
};
__global__ void __launch_bounds__(256) sgd_update_conv_kernel(float* __restrict__ w, float* __restrict__ v, float* __restrict__ g,
                                                              __nv_bfloat16* __restrict__ shadow, float d, float lr, float mu,
                                                              __nv_bfloat16* __restrict__ wt, const TransposeJobs jobs, float gscale,
                                                              long long tail_begin4, long long tail_end4, float tail_d,
                                                              const ConvSplitSrc src) {
    pdl_sync();
    __shared__ __nv_bfloat16 tile[32][36];       // [input channel][output channel], padded
    if ((int)blockIdx.x >= jobs.tile0[jobs.n]) {
        // blocks past the filter tiles: the plain update of the 16-byte vectors [tail_begin4, tail_end4) (the biases, when the
        // FC weights have been updated by their weight-gradient kernels), sgd_update_kernel's arithmetic, one launch less
        const long long i = tail_begin4 + (long long)((int)blockIdx.x - jobs.tile0[jobs.n]) * 256 + threadIdx.x;
        if (i < tail_end4) {
            float4 wv = ((float4*)w)[i], vv = ((float4*)v)[i];
            float4 gv;
            int lb = -1;
            if (src.on) {
                #pragma unroll
                for (int l = 0; l < 5; ++l)
                    if (i >= src.b_off4[l] && i < src.b_off4[l] + src.cout[l] / 4) lb = l;
            }
            if (lb >= 0) {                       // a conv layer's bias gradient from its partials
                const float* bp = src.bpart[lb] + 4 * (i - src.b_off4[lb]);
                gv = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int z = 0; z < src.splits[lb]; ++z) {
                    const float4 t4 = __ldg((const float4*)(bp + (size_t)z * src.cout[lb]));
                    gv.x += t4.x; gv.y += t4.y; gv.z += t4.z; gv.w += t4.w;
                }
                ((float4*)g)[i] = gv;
            } else {
                gv = ((const float4*)g)[i];
            }
            sgd_step(wv.x, vv.x, gscale * gv.x, tail_d, lr, mu);
            sgd_step(wv.y, vv.y, gscale * gv.y, tail_d, lr, mu);
            sgd_step(wv.z, vv.z, gscale * gv.z, tail_d, lr, mu);
            sgd_step(wv.w, vv.w, gscale * gv.w, tail_d, lr, mu);
            ((float4*)w)[i] = wv;
            ((float4*)v)[i] = vv;
            __nv_bfloat162 lo2 = __floats2bfloat162_rn(wv.x, wv.y), hi2 = __floats2bfloat162_rn(wv.z, wv.w);
            ((uint2*)shadow)[i] = make_uint2(*(uint32_t*)&lo2, *(uint32_t*)&hi2);
        }
        return;
    }
    int q = 0;
    while (q + 1 < jobs.n && (int)blockIdx.x >= jobs.tile0[q + 1]) ++q;
    const TransposeJob J = jobs.j[q];
    const int cog = J.cout / J.groups;
    const int ci_blocks = (J.cig + 31) / 32, co_blocks = J.cout / 32;     // cout is a multiple of 32 in every layer
    int t = (int)blockIdx.x - jobs.tile0[q];
    const int cib = t % ci_blocks; t /= ci_blocks;
    const int cob = t % co_blocks, tap = t / co_blocks;
    const int r = threadIdx.x >> 3, c4 = threadIdx.x & 7;
    const int co = cob * 32 + r, ci = cib * 32 + 4 * c4;
    if (ci < J.cig) {                            // cig is a multiple of 4
        const long long e = J.src_off + ((long long)tap * J.cout + co) * J.cig + ci;
        float4 wv = *(float4*)(w + e), vv = *(float4*)(v + e);
        float4 gv;
        if (src.on) {
            const long long t = e - J.src_off;
            const float* sp = src.ws[q] + t;
            gv = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int z = 0; z < src.splits[q]; ++z) {
                const float4 t4 = __ldg((const float4*)(sp + z * src.stride[q]));
                gv.x += t4.x; gv.y += t4.y; gv.z += t4.z; gv.w += t4.w;
            }
            if (q == 0) {                        // conv1: entries of the 12 x 12 zero-padded filter outside 11 x 11 stay zero
                float* gp = &gv.x;
                #pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int ch = (int)((t + k) % 48), tp = (int)((t + k) / (48 * 96));
                    const int ky = (tp / 3) * 4 + (ch / 3) / 4, kx = (tp % 3) * 4 + (ch / 3) % 4;
                    if (ky > 10 || kx > 10) gp[k] = 0.f;
                }
            }
            *(float4*)(g + e) = gv;
        } else {
            gv = *(const float4*)(g + e);
        }
        sgd_step(wv.x, vv.x, gscale * gv.x, d, lr, mu);
        sgd_step(wv.y, vv.y, gscale * gv.y, d, lr, mu);
        sgd_step(wv.z, vv.z, gscale * gv.z, d, lr, mu);
        sgd_step(wv.w, vv.w, gscale * gv.w, d, lr, mu);
        *(float4*)(w + e) = wv;
        *(float4*)(v + e) = vv;
        const __nv_bfloat162 lo2 = __floats2bfloat162_rn(wv.x, wv.y), hi2 = __floats2bfloat162_rn(wv.z, wv.w);
        *(uint2*)(shadow + e) = make_uint2(*(const uint32_t*)&lo2, *(const uint32_t*)&hi2);
        tile[4 * c4][r] = lo2.x; tile[4 * c4 + 1][r] = lo2.y; tile[4 * c4 + 2][r] = hi2.x; tile[4 * c4 + 3][r] = hi2.y;
    }
    __syncthreads();
    const int ci2 = cib * 32 + r, cq = 4 * c4;   // now: thread (input channel r of the tile, four output channels from cq)
    if (ci2 < J.cig) {
        const int co0 = cob * 32 + cq, grp = co0 / cog, col = co0 - grp * cog;
        __nv_bfloat16* dst = wt + J.dst_off + ((long long)tap * J.cig * J.groups + grp * J.cig + ci2) * cog + col;
        const __nv_bfloat162 a = __halves2bfloat162(tile[r][cq], tile[r][cq + 1]), b = __halves2bfloat162(tile[r][cq + 2], tile[r][cq + 3]);
        *(uint2*)dst = make_uint2(*(const uint32_t*)&a, *(const uint32_t*)&b);
    }
}
// exchange-and-average with both replicas in one HBM: w_a = w_b = (w_a+w_b)/2, same for momentum; refresh both shadows.
__global__ void replica_average_kernel(float* __restrict__ wa, float* __restrict__ wb, float* __restrict__ va,
                                       float* __restrict__ vb, __nv_bfloat16* __restrict__ sa,
                                       __nv_bfloat16* __restrict__ sb, long long n4) {
    pdl_sync();
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
        const float4 a = ((float4*)wa)[i], b = ((float4*)wb)[i];
        const float4 c = ((float4*)va)[i], d = ((float4*)vb)[i];
        const float4 w = make_float4(0.5f * (a.x + b.x), 0.5f * (a.y + b.y), 0.5f * (a.z + b.z), 0.5f * (a.w + b.w));
        const float4 v = make_float4(0.5f * (c.x + d.x), 0.5f * (c.y + d.y), 0.5f * (c.z + d.z), 0.5f * (c.w + d.w));
        ((float4*)wa)[i] = w; ((float4*)wb)[i] = w;
        ((float4*)va)[i] = v; ((float4*)vb)[i] = v;
        __nv_bfloat162 lo = __floats2bfloat162_rn(w.x, w.y), hi = __floats2bfloat162_rn(w.z, w.w);
        const uint2 s = make_uint2(*(uint32_t*)&lo, *(uint32_t*)&hi);
        ((uint2*)sa)[i] = s; ((uint2*)sb)[i] = s;
    }
}
// Momentum update of two replicas and their exchange-and-average in one pass: each replica's own (w, v, g) goes through
// sgd_step (the update kernels' arithmetic), then w and v of both are replaced by 0.5 * (a + b) (replica_average_kernel's
// arithmetic) and both bf16 copies are written: six 16-byte loads and six stores per four parameter indices, 44 bytes per
// index, against 22 + 22 + 36 for the three separate passes, with bit-identical results.
__device__ __forceinline__ float4 ld_stream(const float* p) {       // read once, do not keep in L1
    float4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "l"(p));
    return r;
}
__global__ void __launch_bounds__(256) sgd_update_average_kernel(float* __restrict__ wa, float* __restrict__ va, const float* __restrict__ ga,
                                                                 float* __restrict__ wb, float* __restrict__ vb, const float* __restrict__ gb,
                                                                 __nv_bfloat16* __restrict__ sa, __nv_bfloat16* __restrict__ sb,
                                                                 long long n4, long long n_decay4, float lr, float mu, float wd) {
    pdl_sync();
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
        float4 a = ((const float4*)wa)[i], c = ((const float4*)va)[i];
        float4 b = ((const float4*)wb)[i], e = ((const float4*)vb)[i];
        const float4 g0 = ld_stream(ga + 4 * i), g1 = ld_stream(gb + 4 * i);
        const float d = i < n_decay4 ? lr * wd : 0.f;
        sgd_step(a.x, c.x, g0.x, d, lr, mu); sgd_step(a.y, c.y, g0.y, d, lr, mu);
        sgd_step(a.z, c.z, g0.z, d, lr, mu); sgd_step(a.w, c.w, g0.w, d, lr, mu);
        sgd_step(b.x, e.x, g1.x, d, lr, mu); sgd_step(b.y, e.y, g1.y, d, lr, mu);
        sgd_step(b.z, e.z, g1.z, d, lr, mu); sgd_step(b.w, e.w, g1.w, d, lr, mu);
        const float4 w = make_float4(0.5f * (a.x + b.x), 0.5f * (a.y + b.y), 0.5f * (a.z + b.z), 0.5f * (a.w + b.w));
        const float4 v = make_float4(0.5f * (c.x + e.x), 0.5f * (c.y + e.y), 0.5f * (c.z + e.z), 0.5f * (c.w + e.w));
        ((float4*)wa)[i] = w; ((float4*)wb)[i] = w;
        ((float4*)va)[i] = v; ((float4*)vb)[i] = v;
        __nv_bfloat162 lo = __floats2bfloat162_rn(w.x, w.y), hi = __floats2bfloat162_rn(w.z, w.w);
        const uint2 s = make_uint2(*(uint32_t*)&lo, *(uint32_t*)&hi);
        ((uint2*)sa)[i] = s; ((uint2*)sb)[i] = s;
    }
}
// The same for two replicas that SHARE one copy of parameters and momentum (they are identical at the start of every
// iteration: identical initialisation, and every exchange makes them equal again, so one copy holds both): each replica's
// update starts from the shared (w, v) with its own gradient, the averages go back to the shared arrays.  Same arithmetic in
// the same order as above, hence the same bits; 16 bytes read and 10 written per index (26 instead of 44).
__global__ void __launch_bounds__(256) sgd_update_average_shared_kernel(float* __restrict__ w, float* __restrict__ v, const float* __restrict__ ga,
                                                                        const float* __restrict__ gb, __nv_bfloat16* __restrict__ shadow,
                                                                        long long n4, long long n_decay4, float lr, float mu, float wd) {
    pdl_sync();
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
        float4 a = ((const float4*)w)[i], c = ((const float4*)v)[i];
        float4 b = a, e = c;
        const float4 g0 = ld_stream(ga + 4 * i), g1 = ld_stream(gb + 4 * i);
        const float d = i < n_decay4 ? lr * wd : 0.f;
        sgd_step(a.x, c.x, g0.x, d, lr, mu); sgd_step(a.y, c.y, g0.y, d, lr, mu);
        sgd_step(a.z, c.z, g0.z, d, lr, mu); sgd_step(a.w, c.w, g0.w, d, lr, mu);
        sgd_step(b.x, e.x, g1.x, d, lr, mu); sgd_step(b.y, e.y, g1.y, d, lr, mu);
        sgd_step(b.z, e.z, g1.z, d, lr, mu); sgd_step(b.w, e.w, g1.w, d, lr, mu);
        const float4 wn = make_float4(0.5f * (a.x + b.x), 0.5f * (a.y + b.y), 0.5f * (a.z + b.z), 0.5f * (a.w + b.w));
        const float4 vn = make_float4(0.5f * (c.x + e.x), 0.5f * (c.y + e.y), 0.5f * (c.z + e.z), 0.5f * (c.w + e.w));
        ((float4*)w)[i] = wn; ((float4*)v)[i] = vn;
        __nv_bfloat162 lo = __floats2bfloat162_rn(wn.x, wn.y), hi = __floats2bfloat162_rn(wn.z, wn.w);
        ((uint2*)shadow)[i] = make_uint2(*(uint32_t*)&lo, *(uint32_t*)&hi);
    }
}
// After an all-reduce(sum) of parameters and momentum over R replicas on R GPUs: w <- scale w, v <- scale v (scale = 1/R:
// the average) and the bf16 copy of w: 8 bytes read and 10 written per index.
__global__ void __launch_bounds__(256) scale_refresh_kernel(float* __restrict__ w, float* __restrict__ v,
                                                            __nv_bfloat16* __restrict__ shadow, long long n4, float scale) {
    pdl_sync();
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
        float4 a = ((const float4*)w)[i], c = ((const float4*)v)[i];
        a.x *= scale; a.y *= scale; a.z *= scale; a.w *= scale;
        c.x *= scale; c.y *= scale; c.z *= scale; c.w *= scale;
        ((float4*)w)[i] = a; ((float4*)v)[i] = c;
        __nv_bfloat162 lo = __floats2bfloat162_rn(a.x, a.y), hi = __floats2bfloat162_rn(a.z, a.w);
        ((uint2*)shadow)[i] = make_uint2(*(uint32_t*)&lo, *(uint32_t*)&hi);
    }
}
// The paper's own form of the exchange ("Data parallelism" figure, steps 2 and 3): every replica has RECEIVED the other
// replicas' parameters and momenta into buffers of its own GPU (peer copies or an all-gather: the caller's) and now averages.
// slot[r] = the arrays of the replica of rank r in rank order, the local replica's own arrays at r = self (so every rank adds
// in the same order and all ranks end bit-identical); w, v = the local arrays, overwritten; also writes the bf16 copy.
struct RecvList { const float* w[8]; const float* v[8]; int count; };
__global__ void __launch_bounds__(256) average_received_kernel(float* __restrict__ w, float* __restrict__ v, __nv_bfloat16* __restrict__ shadow,
                                                               const RecvList rl, long long n4, float inv_count) {
    pdl_sync();
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
        float4 a = ((const float4*)rl.w[0])[i], c = ((const float4*)rl.v[0])[i];
        #pragma unroll 1
        for (int r = 1; r < rl.count; ++r) {
            const float4 b = ((const float4*)rl.w[r])[i], d = ((const float4*)rl.v[r])[i];
            a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
            c.x += d.x; c.y += d.y; c.z += d.z; c.w += d.w;
        }
        a.x *= inv_count; a.y *= inv_count; a.z *= inv_count; a.w *= inv_count;
        c.x *= inv_count; c.y *= inv_count; c.z *= inv_count; c.w *= inv_count;
        ((float4*)w)[i] = a; ((float4*)v)[i] = c;
        __nv_bfloat162 lo = __floats2bfloat162_rn(a.x, a.y), hi = __floats2bfloat162_rn(a.z, a.w);
        ((uint2*)shadow)[i] = make_uint2(*(uint32_t*)&lo, *(uint32_t*)&hi);
    }
}
__global__ void shadow_kernel(const float* __restrict__ w, __nv_bfloat16* __restrict__ shadow, long long n4) {
    pdl_sync();
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
        const float4 wv = ((const float4*)w)[i];
        __nv_bfloat162 lo = __floats2bfloat162_rn(wv.x, wv.y), hi = __floats2bfloat162_rn(wv.z, wv.w);
        ((uint2*)shadow)[i] = make_uint2(*(uint32_t*)&lo, *(uint32_t*)&hi);
    }
}

// Transposed bf16 copies of the conv filters from the bf16 copy of the weights, in the 32 x 32 tiles of
// sgd_update_conv_kernel (8-byte reads along the input channels, 8-byte writes along the output channels through a
// shared-memory tile); wt2 != nullptr: a second destination (the other replica's copy after an average, when both are equal).
__global__ void __launch_bounds__(256) conv_transpose_shadow_kernel(const __nv_bfloat16* __restrict__ shadow, __nv_bfloat16* __restrict__ wt,
                                                                    __nv_bfloat16* __restrict__ wt2, const TransposeJobs jobs) {
    pdl_sync();
    __shared__ __nv_bfloat16 tile[32][36];       // [input channel][output channel], padded
    int q = 0;
    while (q + 1 < jobs.n && (int)blockIdx.x >= jobs.tile0[q + 1]) ++q;
    const TransposeJob J = jobs.j[q];
    const int cog = J.cout / J.groups;
    const int ci_blocks = (J.cig + 31) / 32, co_blocks = J.cout / 32;
    int t = (int)blockIdx.x - jobs.tile0[q];
    const int cib = t % ci_blocks; t /= ci_blocks;
    const int cob = t % co_blocks, tap = t / co_blocks;
    const int r = threadIdx.x >> 3, c4 = threadIdx.x & 7;
    const int co = cob * 32 + r, ci = cib * 32 + 4 * c4;
    if (ci < J.cig) {                            // cig is a multiple of 4
        const uint2 u = *(const uint2*)(shadow + J.src_off + ((long long)tap * J.cout + co) * J.cig + ci);
        const __nv_bfloat162 lo2 = *(const __nv_bfloat162*)&u.x, hi2 = *(const __nv_bfloat162*)&u.y;
        tile[4 * c4][r] = lo2.x; tile[4 * c4 + 1][r] = lo2.y; tile[4 * c4 + 2][r] = hi2.x; tile[4 * c4 + 3][r] = hi2.y;
    }
    __syncthreads();
    const int ci2 = cib * 32 + r, cq = 4 * c4;   // now: thread (input channel r of the tile, four output channels from cq)
    if (ci2 < J.cig) {
        const int co0 = cob * 32 + cq, grp = co0 / cog, col = co0 - grp * cog;
        const long long d = J.dst_off + ((long long)tap * J.cig * J.groups + grp * J.cig + ci2) * cog + col;
        const __nv_bfloat162 a = __halves2bfloat162(tile[r][cq], tile[r][cq + 1]), b2 = __halves2bfloat162(tile[r][cq + 2], tile[r][cq + 3]);
        const uint2 o = make_uint2(*(const uint32_t*)&a, *(const uint32_t*)&b2);
        *(uint2*)(wt + d) = o;
        if (wt2) *(uint2*)(wt2 + d) = o;
    }
}

// ------------------------------------------- canonical <-> internal parameter order
struct ParamSeg { long long canon_off, int_off, count; int kind, a, b, c; };  // kind 0 copy, 1 conv [co][ci][k][k], 2 conv1 s2d, 3 fc6
struct ParamSegs { ParamSeg s[16]; };
__device__ __forceinline__ long long canon_to_internal(const ParamSeg& S, long long i) {
    if (S.kind == 0) return S.int_off + i;
    if (S.kind == 1) {          // a = cout, b = cig, c = k : canonical ((co*cig+ci)*k+ky)*k+kx -> (tap*cout+co)*cig+ci
        const int kk2 = S.c * S.c;
        const int tap = (int)(i % kk2);
        long long r = i / kk2;
        const int ci = (int)(r % S.b), co = (int)(r / S.b);
        return S.int_off + ((long long)tap * S.a + co) * S.b + ci;
    }
    if (S.kind == 2) {          // conv1: [96][3][11][11] -> [tap 3x3][96][48], channel ((ky%4)*4 + kx%4)*3 + c
        const int kx = (int)(i % 11), ky = (int)((i / 11) % 11), c = (int)((i / 121) % 3), co = (int)(i / 363);
        const int tap = (ky >> 2) * 3 + (kx >> 2), ch = ((ky & 3) * 4 + (kx & 3)) * 3 + c;
        return S.int_off + ((long long)tap * 96 + co) * 48 + ch;
    }
    // fc6: [4096][c*36 + hw] -> [4096][hw*256 + c]
    const int k = (int)(i % 9216), n = (int)(i / 9216);
    return S.int_off + (long long)n * 9216 + (k % 36) * 256 + k / 36;
}
__global__ void params_gather_kernel(const float* __restrict__ arena, float* __restrict__ canon, const ParamSegs segs,
                                     long long total) {
    pdl_sync();
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        int s = 0;
        while (s < 15 && i >= segs.s[s + 1].canon_off) ++s;
        canon[i] = arena[canon_to_internal(segs.s[s], i - segs.s[s].canon_off)];
    }
}
__global__ void params_scatter_kernel(float* __restrict__ arena, const float* __restrict__ canon, const ParamSegs segs,
                                      long long total) {
    pdl_sync();
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        int s = 0;
        while (s < 15 && i >= segs.s[s + 1].canon_off) ++s;
        arena[canon_to_internal(segs.s[s], i - segs.s[s].canon_off)] = canon[i];
    }
}

}  // namespace kn
