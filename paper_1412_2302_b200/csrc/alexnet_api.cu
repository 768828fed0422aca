// Host side of the C ABI declared in include/alexnet.h: arena layout, tensor
// maps and GEMM plans, the two-stream step schedule, parameter / tensor access.
#include "../../include/alexnet.h"

#include <cudaTypedefs.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <string>
#include <utility>
#include <vector>

#include "kernels.cuh"
#include "tc_gemm.cuh"

// Every kernel is launched with programmatic stream serialization: its blocks may become resident while the kernel
// before it in the stream drains, and run their set-up; each kernel waits (griddepcontrol.wait) before it touches
// global memory, so the data dependencies of the stream order are kept.
template <typename... KArgs, typename... Args>
void launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t lc{};
    lc.gridDim = grid; lc.blockDim = block; lc.dynamicSmemBytes = smem; lc.stream = st;
    cudaLaunchAttribute at{};
    at.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at.val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = &at; lc.numAttrs = 1;
    cudaLaunchKernelEx(&lc, kernel, std::forward<Args>(args)...);
}

namespace {

typedef __nv_bfloat16 bf16;

// ------------------------------------------------------------------ geometry
struct Grid { int Hp, Wp, H, W, C; };
struct ConvL {
    int k, pad, cin, cout, groups, cig, cog, taps;
    Grid gin, gout;
    long long w_off, b_off, wt_off, canon_w, canon_b;
    int shift[25];
};
struct FcL { int K, N; long long w_off, b_off, canon_w, canon_b; };

struct Layout {
    ConvL conv[5];
    FcL fc[3];
    long long n_weights;   // internal floats holding weights (decay region), multiple of 64
    long long n_total;     // internal floats in total, multiple of 64
    long long wt_total;    // bf16 elements of the transposed conv filters
    kn::ParamSegs segs;
    kn::TransposeJobs tjobs;
};

long long align_up(long long x, long long a) { return (x + a - 1) / a * a; }

Layout make_layout() {
    Layout L;
    memset(&L, 0, sizeof(L));
    // conv1 runs as a stride-1 3x3 convolution over the 4x4 space-to-depth input (48 channels on a 57x57 grid)
    const int spec[5][6] = {  // k, pad, cin, cout, groups, grid
        {3, 0, 48, 96, 1, 57}, {5, 2, 96, 256, 2, 29}, {3, 1, 256, 384, 1, 14}, {3, 1, 384, 384, 2, 14}, {3, 1, 384, 256, 2, 14}};
    const int valid[5] = {55, 27, 13, 13, 13};
    long long off = 0, canon = 0, wt = 0;
    const long long canon_wcount[5] = {34848, 307200, 884736, 663552, 442368};
    for (int l = 0; l < 5; ++l) {
        ConvL& c = L.conv[l];
        c.k = spec[l][0]; c.pad = spec[l][1]; c.cin = spec[l][2]; c.cout = spec[l][3]; c.groups = spec[l][4];
        c.cig = c.cin / c.groups; c.cog = c.cout / c.groups; c.taps = c.k * c.k;
        const int gp = spec[l][5];
        c.gin = Grid{gp, gp, l == 0 ? 57 : valid[l], l == 0 ? 57 : valid[l], c.cin};
        c.gout = Grid{gp, gp, valid[l], valid[l], c.cout};
        for (int t = 0; t < c.taps; ++t) c.shift[t] = (t / c.k - c.pad) * gp + (t % c.k - c.pad);
        c.w_off = off; off = align_up(off + (long long)c.taps * c.cout * c.cig, 64);
        c.canon_w = canon; canon += canon_wcount[l];
        c.canon_b = canon; canon += c.cout;
        c.wt_off = wt; wt = align_up(wt + (long long)c.taps * c.cin * c.cog, 64);
    }
    const int fcs[3][2] = {{9216, 4096}, {4096, 4096}, {4096, 1000}};
    for (int l = 0; l < 3; ++l) {
        FcL& f = L.fc[l];
        f.K = fcs[l][0]; f.N = fcs[l][1];
        f.w_off = off; off = align_up(off + (long long)f.K * f.N, 64);
        f.canon_w = canon; canon += (long long)f.K * f.N;
        f.canon_b = canon; canon += f.N;
    }
    L.n_weights = off;
    for (int l = 0; l < 5; ++l) { L.conv[l].b_off = off; off = align_up(off + L.conv[l].cout, 64); }
    for (int l = 0; l < 3; ++l) { L.fc[l].b_off = off; off = align_up(off + L.fc[l].N, 64); }
    L.n_total = off;
    L.wt_total = wt;
    // canonical -> internal segments, in canonical order
    int s = 0;
    for (int l = 0; l < 5; ++l) {
        const ConvL& c = L.conv[l];
        if (l == 0) L.segs.s[s++] = kn::ParamSeg{c.canon_w, c.w_off, 34848, 2, 0, 0, 0};
        else L.segs.s[s++] = kn::ParamSeg{c.canon_w, c.w_off, canon_wcount[l], 1, c.cout, c.cig, c.k};
        L.segs.s[s++] = kn::ParamSeg{c.canon_b, c.b_off, c.cout, 0, 0, 0, 0};
    }
    for (int l = 0; l < 3; ++l) {
        const FcL& f = L.fc[l];
        L.segs.s[s++] = kn::ParamSeg{f.canon_w, f.w_off, (long long)f.K * f.N, l == 0 ? 3 : 0, 0, 0, 0};
        L.segs.s[s++] = kn::ParamSeg{f.canon_b, f.b_off, f.N, 0, 0, 0, 0};
    }
    L.tjobs.n = 5;
    for (int l = 0; l < 5; ++l) {
        const ConvL& c = L.conv[l];
        L.tjobs.j[l] = kn::TransposeJob{c.w_off, c.wt_off, c.taps, c.cout, c.cig, c.groups, (long long)c.taps * c.cin * c.cog};
    }
    L.tjobs.tile0[0] = 0;
    for (int l = 0; l < 5; ++l) {
        const ConvL& c = L.conv[l];
        L.tjobs.tile0[l + 1] = L.tjobs.tile0[l] + c.taps * (c.cout / 32) * ((c.cig + 31) / 32);
    }
    return L;
}
const long long kCanonCount = 60965224;

// ------------------------------------------------------------------- handle
constexpr size_t kBiasPartial = 65536;    // floats per conv layer: row splits (<= 148) x output channels (<= 384)
struct Plan { tc::GemmParams p; tc::ConvParams c; tc::WgradParams w; bool conv, wgrad; int grid; size_t smem; bool valid; };

struct Tensor {  // description of one exportable device tensor
    void* ptr; int kind; int C, Hp, Wp, H, W; long long N;
};  // kind: 0 bf16 grid, 1 u8 compact NHWC, 2 bf16 [B][N], 3 f32 [B][N], 4 u8 [B][N], 5 s2d input, 6 int32 [B][3], 7 f32 [B]

struct Replica {
    float *w, *v, *g;
    bf16 *shadow, *wt;
    uint8_t* stage[2]; int32_t* labels[2]; bf16* x0[2]; int32_t* cf[2];
    bf16 *a1, *n1, *p1, *a2, *n2, *p2, *a3, *a4, *a5, *p5, *f6, *f7;
    float* z;
    uint8_t *arg1, *arg2, *arg5, *m6, *m7;
    bf16 *dz, *df7, *df6, *dp5, *da5, *da4, *da3, *dp2, *dn2, *da2, *dp1, *dn1, *da1, *dx0;
    float *loss_n, *loss;
    // batch slots
    cudaEvent_t ready[2], consumed[2];
    bool consumed_valid[2];
    uint64_t slot_step[2];
    int next_load, next_train, loaded, last_slot;
    // the step fuses LRN with pooling and never writes n1/n2 or dn1/dn2; get_tensor fills them in on demand
    bool n_stale[2], dn_stale[2];
    // plans
    Plan conv_fwd[5][2], conv_bwd[5], conv_wg[5][2], fc_fwd[3], fc_bwd[3], fc_wg[3];
    Plan fc_wg_plain[3];    // the FC weight gradient stored, never fused with the update (alexnet_forward_backward)
    bool grad_pending;      // forward_backward has left a gradient that no update has consumed yet
    // fc6 -> fc7 -> fc8 forward as one cooperative launch (tc::fc_chain_kernel); chain_mode: 0 off, 1 with programmatic
    // dependent launch, 2 without (the launch attributes the driver accepted); chain_gate: value of the grid gate
    tc::FcChainParams chain; int chain_mode; unsigned chain_gate;
};

}  // namespace

struct alexnet {
    alexnet_config_t cfg;
    Layout L;
    int B;
    cudaStream_t cs, ls;   // compute, loader
    // The independent branches of the backward pass - the weight gradient (+ update) of FC layer l (branch l) and the weight
    // gradient + split reduction of conv layer l (branch 3 + l) - each run on a stream of their own (owned by the handle),
    // forked from the compute stream when their inputs exist and joined before the update.
    static const int kBranches = 8;
    cudaStream_t side[kBranches] = {};
    cudaEvent_t ev_side_done[kBranches] = {};
    cudaEvent_t ev_fork[kBranches] = {};   // the inputs of branch b are ready on the compute stream
    bool fc_grads_on_branches = false;     // the last backward pass ran the FC weight gradients on branches 0-2: ev_side_done[0..2]
                                           // then complete as soon as those gradients exist, long before the pass ends
    cudaEvent_t ev_backward_done = nullptr;   // recorded on the compute stream after every backward pass
    size_t ws_conv_off[5] = {};            // floats: each conv layer's split partials have their own region of the workspace
    float* bias_partial = nullptr;         // [5][kBiasPartial] bias-gradient partials of the conv weight-gradient kernels
    uint8_t* arena; size_t arena_bytes;
    Replica rep[2];
    float* mean; float* ws; float* cs_partial; float* canon_tmp; int* status;
    size_t ws_floats;
    std::string err;
    uint64_t launches;
    int latched;
    float alpha_eff, drop_scale; uint32_t thr24;
    kn::ColorAug color = {};      // sigma == 0: no intensity augmentation (the paper's setting)
    int sm_count;
    PFN_cuTensorMapEncodeTiled_v12000 encode;
    // optional per-launch timing of the GEMM kernel (event pairs on the launching stream)
    bool prof;
    std::vector<cudaEvent_t> prof_ev;
    std::vector<int> prof_kind;     // kernel of each recorded pair: 0 conv_kernel (convolutions), 1 wgrad_kernel, 2 gemm_kernel,
                                    // 3 conv_kernel (FC forward)
    size_t prof_used;
};

namespace {

int fail(alexnet* h, int code, const std::string& msg) { if (h) h->err = msg; return code; }
#define CK(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return fail(h, ALEXNET_ERR_CUDA, std::string(#call) + ": " + cudaGetErrorString(e_)); } while (0)

struct Carver {
    uint8_t* base; size_t off;
    template <typename T> T* take(size_t count) {
        off = (off + 1023) / 1024 * 1024;
        T* p = base ? (T*)(base + off) : nullptr;
        off += count * sizeof(T);
        return p;
    }
};

// k splits of a GEMM with `tiles` output tiles and `steps` k-steps: fill one wave of 148 CTAs, never more (a second,
// nearly empty round costs a whole tile time), and keep at least two k-steps per split
int pick_splits(int tiles, int steps) {
    int s = 148 / tiles;
    if (s > steps / 2) s = steps / 2;
    if (s < 1) s = 1;
    return s;
}
int conv_wg_splits(const ConvL& c, int B, int sm_count = 148) {
    // one wave: (filter rows x 64-channel input blocks x 128-channel output blocks x groups) units times the row splits
    const long long M = (long long)B * c.gin.Hp * c.gin.Wp;
    const int steps = (int)((M + tc::kWgRows - 1) / tc::kWgRows);
    const int units = ((c.cog + 127) / 128) * ((c.cig + 63) / 64) * c.groups * c.k;
    int s = sm_count / units;
    if (s > steps) s = steps;
    if (s < 1) s = 1;
    return s;
}
int fc_fwd_bn(const FcL&) { return 128; }
int fc_fwd_splits(const FcL& f, int B) {
    const int tiles = ((B + 127) / 128) * ((f.N + 127) / 128);
    return pick_splits(tiles, f.K / 128);    // k-steps of two 64-channel chunks
}
int fc_bwd_splits(const FcL& f, int B) {
    const int tiles = ((B + 127) / 128) * (f.K / 256);
    return pick_splits(tiles, (f.N + 63) / 64);
}
// split-K workspace in floats: one region shared by the FC passes (they follow one another on the compute stream), then one
// region per conv layer's weight-gradient partials (those kernels run side by side); conv_off receives the conv regions' offsets
size_t ws_need(const Layout& L, int B, size_t* conv_off = nullptr) {
    size_t need = 0;
    for (int l = 0; l < 3; ++l) {
        need = std::max(need, (size_t)fc_fwd_splits(L.fc[l], B) * B * L.fc[l].N);
        need = std::max(need, (size_t)fc_bwd_splits(L.fc[l], B) * B * L.fc[l].K);
    }
    for (int l = 0; l < 5; ++l) {
        const ConvL& c = L.conv[l];
        need = (need + 63) / 64 * 64;
        if (conv_off) conv_off[l] = need;
        need += (size_t)conv_wg_splits(c, B) * c.taps * c.cout * c.cig;
    }
    return need;
}

// carve the arena; with base == nullptr only the size is computed
size_t carve(alexnet* h, uint8_t* base) {
    Carver c{base, 0};
    const Layout& L = h->L;
    const int B = h->B;
    auto rows = [&](const Grid& g) { return (size_t)B * g.Hp * g.Wp; };
    h->mean = c.take<float>(256 * 256 * 3);
    h->ws_floats = ws_need(L, B, h->ws_conv_off);
    h->ws = c.take<float>(h->ws_floats);
    h->cs_partial = c.take<float>(256 * 4096);
    h->bias_partial = c.take<float>(5 * kBiasPartial);
    h->canon_tmp = c.take<float>(kCanonCount);
    h->status = c.take<int>(16);
    for (int r = 0; r < h->cfg.replicas; ++r) {
        Replica& R = h->rep[r];
        if (r == 1 && (h->cfg.flags & ALEXNET_FLAG_SHARED_REPLICA_WEIGHTS)) {
            // one copy of parameters, momentum and their bf16 forms for both replicas; gradients stay per replica
            R.w = h->rep[0].w; R.v = h->rep[0].v; R.shadow = h->rep[0].shadow; R.wt = h->rep[0].wt;
            R.g = c.take<float>(L.n_total);
        } else {
            R.w = c.take<float>(L.n_total); R.v = c.take<float>(L.n_total); R.g = c.take<float>(L.n_total);
            R.shadow = c.take<bf16>(L.n_total); R.wt = c.take<bf16>(L.wt_total);
        }
        for (int s = 0; s < 2; ++s) {
            R.stage[s] = c.take<uint8_t>((size_t)B * 196608);
            R.labels[s] = c.take<int32_t>(B);
            R.x0[s] = c.take<bf16>(rows(L.conv[0].gin) * 48);
            R.cf[s] = c.take<int32_t>(3 * B);
        }
        const size_t r1 = rows(L.conv[0].gout), r2 = rows(L.conv[1].gout), r3 = rows(L.conv[2].gout);
        R.a1 = c.take<bf16>(r1 * 96); R.n1 = c.take<bf16>(r1 * 96); R.p1 = c.take<bf16>(r2 * 96);
        R.a2 = c.take<bf16>(r2 * 256); R.n2 = c.take<bf16>(r2 * 256); R.p2 = c.take<bf16>(r3 * 256);
        R.a3 = c.take<bf16>(r3 * 384); R.a4 = c.take<bf16>(r3 * 384); R.a5 = c.take<bf16>(r3 * 256);
        R.p5 = c.take<bf16>((size_t)B * 9216); R.f6 = c.take<bf16>((size_t)B * 4096); R.f7 = c.take<bf16>((size_t)B * 4096);
        R.z = c.take<float>((size_t)B * 1000);
        R.arg1 = c.take<uint8_t>((size_t)B * 27 * 27 * 96); R.arg2 = c.take<uint8_t>((size_t)B * 13 * 13 * 256);
        R.arg5 = c.take<uint8_t>((size_t)B * 9216);
        R.m6 = c.take<uint8_t>((size_t)B * 4096); R.m7 = c.take<uint8_t>((size_t)B * 4096);
        R.dz = c.take<bf16>((size_t)B * 1000); R.df7 = c.take<bf16>((size_t)B * 4096); R.df6 = c.take<bf16>((size_t)B * 4096);
        R.dp5 = c.take<bf16>((size_t)B * 9216);
        R.da5 = c.take<bf16>(r3 * 256); R.da4 = c.take<bf16>(r3 * 384); R.da3 = c.take<bf16>(r3 * 384);
        R.dp2 = c.take<bf16>(r3 * 256); R.dn2 = c.take<bf16>(r2 * 256); R.da2 = c.take<bf16>(r2 * 256);
        R.dp1 = c.take<bf16>(r2 * 96); R.dn1 = c.take<bf16>(r1 * 96); R.da1 = c.take<bf16>(r1 * 96);
        R.dx0 = c.take<bf16>(rows(L.conv[0].gin) * 48);
        R.loss_n = c.take<float>(B); R.loss = c.take<float>(16);
    }
    return (c.off + 1023) / 1024 * 1024;
}

int check_cfg(const alexnet_config_t* c) {
    if (!c) return 0;
    if (c->batch < 1 || c->batch > 1024) return 0;
    if (c->replicas < 1 || c->replicas > 2) return 0;
    if (c->lrn_size != 5) return 0;
    if (!(c->dropout_p >= 0.f && c->dropout_p < 1.f)) return 0;
    if (!(c->lrn_k > 0.f)) return 0;
    return 1;
}

// ------------------------------------------------------------------- plans
int make_tm(alexnet* h, CUtensorMap* tm, const void* ptr, uint64_t cols, uint64_t rows, uint64_t pitch_bytes, uint32_t box_rows) {
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {pitch_bytes};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t es[2] = {1, 1};
    CUresult r = h->encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void*)ptr, dims, strides, box, es,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(h, ALEXNET_ERR_CUDA, "cuTensorMapEncodeTiled failed with code " + std::to_string((int)r));
    return ALEXNET_OK;
}

// output tensor map of the staged epilogue: {columns, rows, splits}, box = {128 bytes of columns, 32 rows, 1}
int make_tm_out(alexnet* h, CUtensorMap* tm, const void* ptr, bool f32, uint64_t cols, uint64_t rows, uint64_t nz,
                uint64_t row_pitch_bytes, uint64_t z_pitch_bytes, bool narrow_plain = false) {
    // narrow_plain: bf16 box of 32 columns (64 bytes) without swizzle, the bf16 copy written by the fused FC update
    cuuint64_t dims[3] = {cols, rows, nz};
    cuuint64_t strides[2] = {row_pitch_bytes, z_pitch_bytes};
    cuuint32_t box[3] = {(f32 || narrow_plain) ? 32u : 64u, 32u, 1u};
    cuuint32_t es[3] = {1, 1, 1};
    CUresult r = h->encode(tm, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, (void*)ptr, dims, strides,
                           box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, narrow_plain ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_NONE,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(h, ALEXNET_ERR_CUDA, "cuTensorMapEncodeTiled (output) failed with code " + std::to_string((int)r));
    return ALEXNET_OK;
}

void finish_plan(const alexnet* h, Plan& P) {
    tc::GemmParams& p = P.p;
    const int stage_bytes = tc::kABytes + tc::b_stage_bytes(p.mode, p.BN);
    int stages = (227 * 1024 - 2048 - 4 * (int)tc::kEpiStageBytes) / stage_bytes;
    if (stages > tc::kMaxStages) stages = tc::kMaxStages;
    p.stages = stages;
    // every split gets at least one k-step
    const int per = (p.steps_total + p.splits - 1) / p.splits;
    p.splits = (p.steps_total + per - 1) / per;
    p.steps_per_split = per;
    p.tiles_total = p.m_tiles * p.n_tiles * p.groups * p.taps_grid * p.splits;
    if (p.fuse_update) p.stages = stages = 1;      // two k-steps per tile, hidden behind the epilogue of the tile before; the epilogue tiles need the room
    P.smem = tc::smem_bytes(p.mode, p.BN, stages, p.fuse_update != 0);
    P.grid = std::min(p.tiles_total, h->sm_count);   // persistent: one CTA per SM walks the tile list
    P.valid = true;
}

// Tile shape of the convolution kernel for a problem of M rows, N output channels per group, `groups`
// groups, a kh x kw filter over `chunks` 64-channel chunks: the (row halves, BN) pair with the lowest
// modelled time.  Per weight stage the tensor pipe needs MH*kk*BN/2 cycles; TMA brings about 64 bytes
// per cycle per SM from L2; tiles are dealt to the SMs in rounds.
struct ConvShape { int MH, BN, acc_stages, epi_sets, cg; };
ConvShape choose_conv_shape(const alexnet* h, long long M, int N, int groups, int kh, int kw, int chunks, int kk, bool masked = false) {
    ConvShape best{1, N <= 256 ? N : 128, 1, 1, 1};
    double best_t = 1e30;
    const int a_rows = kw > 1 ? 136 : 128;
    const size_t budget = 227 * 1024 - 2048 - 4 * tc::kEpiStageBytes;
    const int cg_lo = (h->cfg.flags & ALEXNET_FLAG_ALL_CTA_PAIRS) ? 2 : 1, cg_hi = (h->cfg.flags & ALEXNET_FLAG_NO_CTA_PAIRS) ? 1 : 2;
    // a reduction of fewer than four (filter row, chunk) steps per tile (conv1) cannot amortise the accumulator hand-over
    // across the pair: measured slower in pairs (55 -> 61 us), so such layers stay on single CTAs unless forced
    const int cg_auto_hi = kh * chunks >= 4 ? 2 : 1;
    for (int cg = cg_lo; cg <= (cg_lo == 2 ? 2 : std::min(cg_hi, cg_auto_hi)); ++cg)
    for (int MH = 1; MH <= 4; MH *= 2) {
        for (int BN = 16; BN <= 256 && BN <= N; BN += 16) {
            if (N % BN) continue;
            if (MH * BN > 512) continue;
            const size_t g_tiles = kw <= 3 ? kw : 2;     // weight tiles per group (see finish_conv_plan)
            if (2 * (size_t)MH * a_rows * 128 + 2 * g_tiles * (BN / cg) * 128 > budget) continue;
            const int acc = 2 * MH * BN <= 512 ? 2 : 1;
            const long long tiles = ((M + 128 * MH * cg - 1) / (128 * MH * cg)) * (N / BN) * groups;
            const int slots = h->sm_count / cg;
            const long long rounds = (tiles + slots - 1) / slots;
            // per filter row and chunk: the pipe needs kw*kk*MH*BN/2 cycles; each issuer warp pays about 330 cycles per
            // weight group plus 50 per instruction; all issuers together get about one instruction per 40 cycles
            // dispatched (measured: 4 issuers of N = 64 are slower than one of N = 192); TMA brings about 72 B/cycle,
            // and a ring of only two halos (large MH) cannot hide its latency
            const int ngroups = kw <= 3 ? 1 : (kw + 1) / 2;
            const double n_mma = (double)kw * kk;
            const double mma = std::max(std::max(n_mma * MH * BN / 2.0, ngroups * 330.0 + n_mma * 50.0), n_mma * MH * 40.0);
            const bool shallow = 3 * (size_t)MH * a_rows * 128 + 2 * g_tiles * (BN / cg) * 128 > budget;
            const double tma = ((double)MH * a_rows * 128 + (double)kw * (BN / cg) * 128) / 72.0;
            // a CTA pair issues one instruction for both SMs: measured, its issuers run at about 100 cycles per instruction
            // where two issuers of one CTA (N = 128) hold each other up at about 150; worth a tenth of the main loop
            const double pair_gain = cg == 2 ? 0.9 : 1.0;
            double tile_t = (double)kh * chunks * (std::max(mma, tma) * pair_gain + (shallow ? 600.0 : 0.0)) + 800.0;
            // epilogue per 16 columns and row half: about 450 cycles through the staged TMA store (single staging tile per warp), about 1000 with direct
            // stores (tiles whose 64-column slabs would not fit the group's channel range)
            const bool staged = BN % 64 == 0 || (groups == 1 && N == BN);
            // (a ReLU mask read from global memory in the epilogue adds its load latency: measured, the issuer of a masked
            // backward-data layer waits a quarter of its time for a free accumulator)
            const double epi = MH * (BN / 16) * (staged ? (masked ? 1000.0 : 450.0) : 1000.0);
            // a second set of epilogue warps (the sets alternate over the tile's row halves x 64-column slabs) when the
            // epilogue is the longer side
            for (int E = 1; E <= (staged && MH * ((BN + 63) / 64) >= 2 ? 2 : 1); ++E) {
                if (32 * (2 + MH + 4 * E) > tc::kConvMaxThreads) continue;     // warps: 2 producers, MH issuers, 4 E epilogue
                if (E == 2 && 2 * (size_t)MH * a_rows * 128 + 2 * g_tiles * (BN / cg) * 128 + 4 * tc::kEpiStageBytes > budget) continue;
                double tt = tile_t;
                if (acc == 1) tt += epi / E; else tt = std::max(tt, epi / E + 300.0);
                const double t = rounds * tt + (E == 2 ? 1.0 : 0.0);     // ties go to the smaller block
                if (t < best_t) { best_t = t; best = ConvShape{MH, BN, acc, E, cg}; }
            }
        }
    }
    return best;
}

void finish_conv_plan(const alexnet* h, Plan& P) {
    tc::ConvParams& c = P.c;
    const int per = (c.asteps_total + c.splits - 1) / c.splits;
    c.splits = (c.asteps_total + per - 1) / per;
    c.asteps_per_split = per;
    c.tiles_total = c.m_tiles * c.n_tiles * c.groups * c.splits;
    if (c.cpg < 1) c.cpg = 1;
    if (c.cg < 1) c.cg = 1;
    const size_t a_bytes = (size_t)c.MH * c.cpg * c.a_box_rows * 128, b_bytes = (size_t)(c.BN / c.cg) * 128;
    if (c.epi_sets < 1) c.epi_sets = 1;
    const size_t budget = 227 * 1024 - 2048 - 4 * c.epi_sets * tc::kEpiStageBytes;
    c.tpg = c.b_res ? c.kh * c.kw : c.cpg > 1 ? c.cpg : (c.kw <= 3 ? c.kw : 2);   // weight tiles travel in groups: a filter row (2 + 2 + 1 taps of a five-tap row, which keeps
                                                          // four groups in flight), or the chunks of an FC stage
    const size_t g_bytes = b_bytes * c.tpg;
    if (c.kw == 1) {
        int st = (int)(budget / (a_bytes + g_bytes));
        st = std::min(st, 8);
        c.a_stages = c.b_stages = st;
    } else {
        c.a_stages = (budget >= 3 * a_bytes + 2 * g_bytes) ? 3 : 2;
        c.b_stages = (int)std::min<size_t>(8, (budget - c.a_stages * a_bytes) / g_bytes);
    }
    P.conv = true;
    P.smem = tc::conv_smem_bytes(c);
    P.grid = c.cg * std::min(c.tiles_total, h->sm_count / c.cg);     // persistent: CTAs (or CTA pairs) walk the tile list
    P.valid = true;
}

// bf16 convolution output through the staged epilogue when whole 64-column slabs tile the channel range of a
// group, or when the tile ends at the tensor's last column (TMA clips the rest) and the over-read stays inside the
// TMEM allocation; otherwise the epilogue stores rows directly
int conv_out_map(alexnet* h, tc::ConvParams& p, const void* out, int ldo, long long M) {
    const int used = p.acc_stages * p.MH * p.BN;
    int alloc = 32;
    while (alloc < used) alloc <<= 1;
    const bool whole = p.BN % 64 == 0;
    const bool clipped = p.groups == 1 && p.n_tiles == 1 && used - p.BN + (p.BN + 63) / 64 * 64 <= alloc;
    p.tma_store = (whole || clipped) ? 1 : 0;
    if (!p.tma_store) return ALEXNET_OK;
    return make_tm_out(h, &p.tmOut, out, false, (uint64_t)ldo, (uint64_t)M, 1, (uint64_t)ldo * 2, (uint64_t)ldo * 2 * (uint64_t)M);
}

int plan_conv_fwd(alexnet* h, Plan& P, const ConvL& c, const bf16* in, const bf16* wsh, const float* bias, bf16* out) {
    memset(&P, 0, sizeof(P));
    tc::ConvParams& p = P.c;
    const long long M = (long long)h->B * c.gin.Hp * c.gin.Wp;
    const int gp = c.gin.Wp;
    p.kh = p.kw = c.k; p.chunks = (c.cig + 63) / 64; p.kk = c.cig == 48 ? 3 : 4;
    const ConvShape sh = choose_conv_shape(h, M, c.cog, c.groups, p.kh, p.kw, p.chunks, p.kk);
    p.MH = sh.MH; p.BN = sh.BN; p.acc_stages = sh.acc_stages; p.epi_sets = sh.epi_sets; p.cg = sh.cg;
    p.M_total = (int)M; p.m_tiles = (int)((M + 128 * p.MH * p.cg - 1) / (128 * p.MH * p.cg));
    p.n_tiles = c.cog / p.BN; p.groups = c.groups; p.splits = 1;
    p.asteps_total = p.kh * p.chunks;
    p.a_box_rows = p.kw > 1 ? 136 : 128;
    p.a_x0 = 0; p.a_gx = c.cig; p.b_tap_rows = c.cout; p.b_g_rows = c.cog;
    for (int ky = 0; ky < c.k; ++ky) p.halo_shift[ky] = (ky - c.pad) * gp - c.pad;
    for (int kx = 0; kx < c.k; ++kx) p.tap_off[kx] = kx;
    p.epi = tc::EPI_BF16; p.n_valid = c.cog; p.ldo = c.cout; p.out_gx = c.cog;
    p.Hp = c.gout.Hp; p.Wp = c.gout.Wp; p.H = c.gout.H; p.W = c.gout.W;
    p.relu = 1; p.mask_scale = 1.f; p.bias = bias; p.mask = nullptr; p.out = out; p.status = h->status;
    int rc;
    if ((rc = make_tm(h, &p.tmA, in, c.cin, M, (uint64_t)c.cin * 2, p.a_box_rows))) return rc;
    if ((rc = make_tm(h, &p.tmB, wsh, c.cig, (uint64_t)c.taps * c.cout, (uint64_t)c.cig * 2, p.BN / p.cg))) return rc;
    if ((rc = conv_out_map(h, p, out, c.cout, M))) return rc;
    // a layer whose whole filter is one n tile of one chunk (conv1: 9 taps x 96 rows x 128 bytes = 108 KB) keeps it in
    // shared memory for all the tiles of a CTA; the halo ring gets two stages
    p.b_res = (p.cg == 1 && p.groups == 1 && p.n_tiles == 1 && p.chunks == 1 && (size_t)p.kh * p.kw * p.BN * 128 <= 112 * 1024) ? 1 : 0;
    finish_conv_plan(h, P);
    return ALEXNET_OK;
}
int plan_conv_bwd(alexnet* h, Plan& P, const ConvL& c, const bf16* dy, const bf16* wt, const bf16* mask, bf16* dx) {
    memset(&P, 0, sizeof(P));
    tc::ConvParams& p = P.c;
    const long long M = (long long)h->B * c.gin.Hp * c.gin.Wp;
    const int gp = c.gin.Wp;
    p.kh = p.kw = c.k; p.chunks = (c.cog + 63) / 64; p.kk = 4;      // conv1: 96 channels, the second chunk is half zero fill
    const ConvShape sh = choose_conv_shape(h, M, c.cig, c.groups, p.kh, p.kw, p.chunks, p.kk, mask != nullptr);
    p.MH = sh.MH; p.BN = sh.BN; p.acc_stages = sh.acc_stages; p.epi_sets = sh.epi_sets; p.cg = sh.cg;
    p.M_total = (int)M; p.m_tiles = (int)((M + 128 * p.MH * p.cg - 1) / (128 * p.MH * p.cg));
    p.n_tiles = c.cig / p.BN; p.groups = c.groups; p.splits = 1;
    p.asteps_total = p.kh * p.chunks;
    p.a_box_rows = p.kw > 1 ? 136 : 128;
    p.a_x0 = 0; p.a_gx = c.cog; p.b_tap_rows = c.cin; p.b_g_rows = c.cig;
    // the gradient at input row m gathers dy at m - shift(ky,kx): per filter row the taps read descending rows
    for (int ky = 0; ky < c.k; ++ky) p.halo_shift[ky] = -(ky - c.pad) * gp + c.pad - (c.k - 1);
    for (int kx = 0; kx < c.k; ++kx) p.tap_off[kx] = c.k - 1 - kx;
    p.epi = tc::EPI_BF16; p.n_valid = c.cig; p.ldo = c.cin; p.out_gx = c.cig;
    p.Hp = c.gin.Hp; p.Wp = c.gin.Wp; p.H = c.gin.H; p.W = c.gin.W;
    p.relu = 0; p.mask_scale = 1.f; p.bias = nullptr; p.mask = mask; p.out = dx; p.status = h->status;
    int rc;
    if ((rc = make_tm(h, &p.tmA, dy, c.cout, M, (uint64_t)c.cout * 2, p.a_box_rows))) return rc;
    if ((rc = make_tm(h, &p.tmB, wt, c.cog, (uint64_t)c.taps * c.cin, (uint64_t)c.cog * 2, p.BN / p.cg))) return rc;
    if ((rc = conv_out_map(h, p, dx, c.cin, M))) return rc;
    finish_conv_plan(h, P);
    return ALEXNET_OK;
}
int plan_conv_wg(alexnet* h, Plan& P, int l, const ConvL& c, const bf16* dy, const bf16* xin) {
    memset(&P, 0, sizeof(P));
    tc::WgradParams& p = P.w;
    const long long M = (long long)h->B * c.gin.Hp * c.gin.Wp;
    p.m_tiles = (c.cog + 127) / 128; p.n_tiles = (c.cig + 63) / 64; p.groups = c.groups; p.kh = c.k; p.kw = c.k;
    p.steps_total = (int)((M + tc::kWgRows - 1) / tc::kWgRows);
    p.splits = conv_wg_splits(c, h->B, std::min(h->sm_count, 148));   // never more than the workspace was sized for
    p.steps_per_split = (p.steps_total + p.splits - 1) / p.splits;
    p.splits = (p.steps_total + p.steps_per_split - 1) / p.steps_per_split;
    p.tiles_total = p.m_tiles * p.n_tiles * p.groups * p.kh * p.splits;
    if (c.k <= 4) { p.NI = 1; p.acc_kx0[0] = 0; p.acc_taps[0] = c.k; }
    else { p.NI = 2; p.acc_kx0[0] = 0; p.acc_taps[0] = 3; p.acc_kx0[1] = 3; p.acc_taps[1] = c.k - 3; }
    p.stages = std::min(8, (int)((227 * 1024 - 2048) / (tc::kWgABytes + tc::kWgBBytes)));
    p.a_gx = c.cog; p.b_gx = c.cig;
    for (int ky = 0; ky < c.k; ++ky) p.halo_shift[ky] = (ky - c.pad) * c.gin.Wp - c.pad;
    p.M_total = c.cog; p.n_valid = c.cig; p.ldo = c.cig; p.out_gx = c.cog;
    p.tap_stride = (long long)c.cout * c.cig; p.split_stride = (long long)c.taps * c.cout * c.cig;
    p.epi = tc::EPI_F32; p.mask_scale = 1.f;
    p.out = h->ws + h->ws_conv_off[l]; p.status = h->status;
    p.bias_partial = h->bias_partial + (size_t)l * kBiasPartial; p.bias_ld = c.cout;
    int rc;
    if ((rc = make_tm(h, &p.tmA, dy, c.cout, M, (uint64_t)c.cout * 2, tc::kWgRows))) return rc;
    if ((rc = make_tm(h, &p.tmB, xin, c.cin, M, (uint64_t)c.cin * 2, tc::kWgRows + 8))) return rc;
    P.wgrad = true;
    P.smem = tc::wgrad_smem_bytes(p);
    P.grid = p.tiles_total;
    P.valid = true;
    return ALEXNET_OK;
}
int plan_fc_fwd(alexnet* h, Plan& P, const FcL& f, const bf16* x, const bf16* wsh, const float* bias, bool with_epilogue) {
    memset(&P, 0, sizeof(P));
    tc::ConvParams& p = P.c;
    const int B = h->B;
    p.kh = p.kw = 1; p.cpg = 2; p.chunks = f.K / 64 / p.cpg; p.kk = 4;   // K is a multiple of 128 in all three layers
    p.MH = 1; p.BN = fc_fwd_bn(f); p.acc_stages = 2; p.cg = 1;
    p.epi_sets = 2;     // one tile per CTA: its epilogue is never hidden behind a next tile, so two sets of warps share the four slabs
    p.M_total = B; p.m_tiles = (B + 127) / 128; p.n_tiles = (f.N + p.BN - 1) / p.BN;
    p.groups = 1; p.splits = fc_fwd_splits(f, B);
    p.asteps_total = p.chunks;
    p.a_box_rows = 128;
    p.halo_shift[0] = 0; p.tap_off[0] = 0; p.tap_off[1] = 128;   // the second chunk's box follows the first in the stage
    p.epi = tc::EPI_F32; p.n_valid = f.N; p.ldo = f.N; p.split_stride = (long long)B * f.N;
    p.mask_scale = 1.f; p.out = h->ws; p.status = h->status;
    int rc;
    if ((rc = make_tm(h, &p.tmA, x, f.K, B, (uint64_t)f.K * 2, 128))) return rc;
    if ((rc = make_tm(h, &p.tmB, wsh, f.K, f.N, (uint64_t)f.K * 2, p.BN))) return rc;
    p.tma_store = 1;
    if ((rc = make_tm_out(h, &p.tmOut, h->ws, true, (uint64_t)f.N, (uint64_t)B, (uint64_t)p.splits, (uint64_t)f.N * 4,
                          (uint64_t)B * f.N * 4))) return rc;
    finish_conv_plan(h, P);
    // fc6 / fc7 with one row tile (batch <= 128) and 2, 4 or 8 splits: the splits of a tile form a thread-block cluster and
    // reduce their partial tiles through distributed shared memory, with bias, ReLU and dropout applied there (no partials in
    // HBM, no second launch).  fc8 keeps its partials: its reduction is part of the softmax kernel.
    const int S = p.splits;
    if (with_epilogue && p.m_tiles == 1 && (S == 2 || S == 4 || S == 8) && p.tiles_total <= h->sm_count && f.N % 4 == 0 &&
        (size_t)128 * tc::kZcPitch * 4 <= (size_t)p.a_stages * p.MH * p.cpg * p.a_box_rows * 128 + (size_t)p.b_stages * p.tpg * p.BN * 128) {
        p.zcluster = S;
        p.bias = bias;
        P.grid = p.tiles_total;
    }
    return ALEXNET_OK;
}
int plan_fc_bwd(alexnet* h, Plan& P, const FcL& f, const bf16* dy, const bf16* wsh) {
    memset(&P, 0, sizeof(P));
    tc::GemmParams& p = P.p;
    const int B = h->B;
    p.mode = tc::MODE_KMN; p.epi = tc::EPI_F32;
    p.M_total = B; p.m_tiles = (B + 127) / 128; p.BN = 256; p.n_tiles = f.K / 256;
    p.groups = 1; p.taps_grid = 1; p.splits = fc_bwd_splits(f, B);
    p.kk = 4; p.chunks = 1; p.steps_total = (f.N + 63) / 64;
    p.n_valid = f.K; p.ldo = f.K; p.split_stride = (long long)B * f.K;
    p.out = h->ws; p.status = h->status;
    int rc;
    if ((rc = make_tm(h, &p.tmA, dy, f.N, B, (uint64_t)f.N * 2, 128))) return rc;
    if ((rc = make_tm(h, &p.tmB, wsh, f.K, f.N, (uint64_t)f.K * 2, 64))) return rc;
    p.tma_store = 1;
    if ((rc = make_tm_out(h, &p.tmOut, h->ws, true, (uint64_t)f.K, (uint64_t)B, (uint64_t)p.splits, (uint64_t)f.K * 4,
                          (uint64_t)B * f.K * 4))) return rc;
    finish_plan(h, P);
    return ALEXNET_OK;
}
int plan_fc_wg(alexnet* h, Plan& P, const FcL& f, const bf16* dy, const bf16* x, float* gout, float* w, float* v, bf16* shadow,
               bool fuse) {
    memset(&P, 0, sizeof(P));
    tc::GemmParams& p = P.p;
    const int B = h->B;
    p.mode = tc::MODE_MNMN; p.epi = tc::EPI_F32;
    p.M_total = f.N; p.m_tiles = (f.N + 127) / 128; p.BN = 256; p.n_tiles = f.K / 256;
    p.groups = 1; p.taps_grid = 1; p.splits = 1; p.kk = 4; p.chunks = 1; p.steps_total = (B + 63) / 64;
    p.n_valid = f.K; p.ldo = f.K;
    p.out = gout; p.status = h->status;
    int rc;
    if ((rc = make_tm(h, &p.tmA, dy, f.N, B, (uint64_t)f.N * 2, 64))) return rc;
    if ((rc = make_tm(h, &p.tmB, x, f.K, B, (uint64_t)f.K * 2, 64))) return rc;
    p.tma_store = 1;
    if ((rc = make_tm_out(h, &p.tmOut, gout, true, (uint64_t)f.K, (uint64_t)f.N, 1, (uint64_t)f.K * 4, (uint64_t)f.K * 4 * f.N))) return rc;
    if (fuse) {
        p.fuse_update = 1;
        p.BN = 128; p.n_tiles = f.K / 128;   // narrower tiles leave room for four {w, v} buffers per epilogue warp
        p.upd_lr = h->cfg.lr; p.upd_mu = h->cfg.momentum; p.upd_d = h->cfg.lr * h->cfg.weight_decay;
        if ((rc = make_tm_out(h, &p.tmW, w, true, (uint64_t)f.K, (uint64_t)f.N, 1, (uint64_t)f.K * 4, (uint64_t)f.K * 4 * f.N))) return rc;
        if ((rc = make_tm_out(h, &p.tmV, v, true, (uint64_t)f.K, (uint64_t)f.N, 1, (uint64_t)f.K * 4, (uint64_t)f.K * 4 * f.N))) return rc;
        if ((rc = make_tm_out(h, &p.tmS, shadow, false, (uint64_t)f.K, (uint64_t)f.N, 1, (uint64_t)f.K * 2, (uint64_t)f.K * 2 * f.N, true))) return rc;
    }
    finish_plan(h, P);
    return ALEXNET_OK;
}

// The three FC forward passes as one launch (ALEXNET_FLAG_FC_CHAIN), when every layer is one unit per CTA of the same grid: one row tile (batch
// <= 128), 128-column tiles, fc6 / fc7 as clusters of their four splits, fc8's tiles x splits filling the same grid, and
// the device able to hold all clusters at once (the CTAs wait for one another at the layer boundaries).
void plan_fc_chain(alexnet* h, int r) {
    Replica& R = h->rep[r];
    R.chain_mode = 0; R.chain_gate = 0;
    if (!(h->cfg.flags & ALEXNET_FLAG_FC_CHAIN)) return;
    tc::FcChainParams& q = R.chain;
    memset(&q, 0, sizeof(q));
    const int grid = R.fc_fwd[0].c.tiles_total;
    bf16* outs[3] = {R.f6, R.f7, nullptr};
    uint8_t* keeps[3] = {R.m6, R.m7, nullptr};
    for (int l = 0; l < 3; ++l) {
        const tc::ConvParams& c = R.fc_fwd[l].c;
        const FcL& f = h->L.fc[l];
        if (!R.fc_fwd[l].valid || c.m_tiles != 1 || c.BN != 128 || c.cpg != 2 || c.kk != 4 || c.kh != 1 || c.tiles_total != grid ||
            c.n_valid % 4 || (l < 2 ? c.zcluster != tc::kChainCluster : c.zcluster != 0)) return;
        tc::FcChainLayer& y = q.L[l];
        y.tmA = c.tmA; y.tmB = c.tmB;
        y.n_tiles = c.n_tiles; y.splits = c.splits; y.per = c.asteps_per_split; y.asteps_total = c.asteps_total; y.n_valid = c.n_valid;
        y.cluster_reduce = l < 2;
        y.relu = l < 2; y.bias = R.w + f.b_off; y.out = outs[l]; y.keep = keeps[l];
        y.partial = h->ws; y.split_stride = c.split_stride;
    }
    if (grid % tc::kChainCluster || grid > h->sm_count) return;
    q.nlayers = 3; q.M_total = h->B; q.status = h->status; q.gate = (unsigned*)(h->status + 12 + r);
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(grid); lc.blockDim = dim3(tc::kChainThreads); lc.dynamicSmemBytes = tc::fc_chain_smem_bytes();
    cudaLaunchAttribute at[1] = {};
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = tc::kChainCluster; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    lc.attrs = at; lc.numAttrs = 1;
    int clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&clusters, tc::fc_chain_kernel, &lc) != cudaSuccess) { cudaGetLastError(); return; }
    if (clusters * tc::kChainCluster < grid) return;
    R.chain_mode = 1;
}

int build_plans(alexnet* h, int r) {
    Replica& R = h->rep[r];
    const Layout& L = h->L;
    const bf16* in[5] = {nullptr, R.p1, R.p2, R.a3, R.a4};
    bf16* out[5] = {R.a1, R.a2, R.a3, R.a4, R.a5};
    bf16* dyv[5] = {R.da1, R.da2, R.da3, R.da4, R.da5};
    bf16* dxv[5] = {R.dx0, R.dp1, R.dp2, R.da3, R.da4};
    const bf16* maskv[5] = {nullptr, nullptr, nullptr, R.a3, R.a4};
    int rc;
    for (int l = 0; l < 5; ++l) {
        const ConvL& c = L.conv[l];
        for (int s = 0; s < 2; ++s) {
            const bf16* x = l == 0 ? R.x0[s] : in[l];
            if ((rc = plan_conv_fwd(h, R.conv_fwd[l][s], c, x, R.shadow + c.w_off, R.w + c.b_off, out[l]))) return rc;
            if ((rc = plan_conv_wg(h, R.conv_wg[l][s], l, c, dyv[l], x))) return rc;
        }
        if ((rc = plan_conv_bwd(h, R.conv_bwd[l], c, dyv[l], R.wt + c.wt_off, maskv[l], dxv[l]))) return rc;
    }
    const bf16* fx[3] = {R.p5, R.f6, R.f7};
    const bf16* fdy[3] = {R.df6, R.df7, R.dz};
    for (int l = 0; l < 3; ++l) {
        const FcL& f = L.fc[l];
        if ((rc = plan_fc_fwd(h, R.fc_fwd[l], f, fx[l], R.shadow + f.w_off, R.w + f.b_off, l < 2))) return rc;
        if ((rc = plan_fc_bwd(h, R.fc_bwd[l], f, fdy[l], R.shadow + f.w_off))) return rc;
        const bool fuse = (h->cfg.flags & ALEXNET_FLAG_FUSED_FC_UPDATE) != 0;
        if ((rc = plan_fc_wg(h, R.fc_wg[l], f, fdy[l], fx[l], R.g + f.w_off, R.w + f.w_off, R.v + f.w_off, R.shadow + f.w_off, fuse))) return rc;
        if ((rc = plan_fc_wg(h, R.fc_wg_plain[l], f, fdy[l], fx[l], R.g + f.w_off, R.w + f.w_off, R.v + f.w_off, R.shadow + f.w_off, false))) return rc;
    }
    plan_fc_chain(h, r);
    return ALEXNET_OK;
}

// ---------------------------------------------------------------- launches
inline int nblk(long long n, int t) { return (int)((n + t - 1) / t); }

// early_weights: the launch is part of a forward or backward pass whose earlier kernels (and whatever may still run beside
// them) never write this layer's bf16 weights, so conv_kernel may load them before its predecessor has finished
void launch_gemm(alexnet* h, const Plan& P0, cudaStream_t st, bool early_weights = false) {
    Plan Pl;
    const Plan* Pp = &P0;
    if (early_weights && P0.conv) { Pl = P0; Pl.c.early_b = 1; Pp = &Pl; }
    const Plan& P = *Pp;
    if (h->prof) {
        while (h->prof_ev.size() < h->prof_used + 2) {
            cudaEvent_t e;
            if (cudaEventCreate(&e) != cudaSuccess) { h->prof = false; break; }
            h->prof_ev.push_back(e);
        }
    }
    if (h->prof) cudaEventRecord(h->prof_ev[h->prof_used], st);
    if (P.wgrad) launch_k(tc::wgrad_kernel, P.grid, tc::wgrad_threads(P.w), P.smem, st, P.w);
    else if (P.conv && P.c.cg == 2) {
        cudaLaunchConfig_t lc{};
        lc.gridDim = dim3(P.grid); lc.blockDim = dim3(tc::conv_threads(P.c)); lc.dynamicSmemBytes = P.smem; lc.stream = st;
        cudaLaunchAttribute at[2] = {};
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[1].val.programmaticStreamSerializationAllowed = 1;
        lc.attrs = at; lc.numAttrs = 2;
        cudaLaunchKernelEx(&lc, tc::conv_kernel<2>, P.c);
    }
    else if (P.conv && P.c.zcluster) {
        cudaLaunchConfig_t lc{};
        lc.gridDim = dim3(P.grid); lc.blockDim = dim3(tc::conv_threads(P.c)); lc.dynamicSmemBytes = P.smem; lc.stream = st;
        cudaLaunchAttribute at[2] = {};
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = P.c.zcluster; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[1].val.programmaticStreamSerializationAllowed = 1;
        lc.attrs = at; lc.numAttrs = 2;
        cudaLaunchKernelEx(&lc, tc::conv_kernel<1>, P.c);
    }
    else if (P.conv) launch_k(tc::conv_kernel<1>, P.grid, tc::conv_threads(P.c), P.smem, st, P.c);
    else launch_k(tc::gemm_kernel, P.grid, tc::kThreads, P.smem, st, P.p);
    if (h->prof) {
        cudaEventRecord(h->prof_ev[h->prof_used + 1], st);
        h->prof_kind.push_back(P.conv ? (P.c.kh == 1 && P.c.cpg > 1 ? 3 : 0) : P.wgrad ? 1 : 2);
        h->prof_used += 2;
    }
    h->launches++;
}
void colsum(alexnet* h, const bf16* dy, long long rows, int C, float* db, cudaStream_t st) {
    if (C % 8 || rows < 512) {     // few rows: one thread per column, one launch (the two-stage form would use a single split)
        launch_k(kn::colsum_scalar_kernel, nblk(C, 128), 128, 0, st, dy, (int)rows, C, db);
        h->launches++;
        return;
    }
    int splits = (int)std::min<long long>(256, std::max<long long>(1, rows / 256));
    dim3 grid((C + 63) / 64, splits);
    launch_k(kn::colsum_kernel, grid, 256, 0, st, dy, rows, C, h->cs_partial);
    launch_k(kn::colsum_final_kernel, nblk(C, 128), 128, 0, st, h->cs_partial, splits, C, db);
    h->launches += 2;
}
void refresh_shadows(alexnet* h, int r, bool whole, cudaStream_t st) {
    Replica& R = h->rep[r];
    if (whole) {
        launch_k(kn::shadow_kernel, 1184, 256, 0, st, R.w, R.shadow, h->L.n_total / 4);
        h->launches++;
    }
    launch_k(kn::conv_transpose_shadow_kernel, h->L.tjobs.tile0[5], 256, 0, st, R.shadow, R.wt, (bf16*)nullptr, h->L.tjobs);
    h->launches++;
}
// after an average both replicas hold the same parameters: one launch writes both transposed copies
void refresh_transposed_both(alexnet* h, cudaStream_t st) {
    launch_k(kn::conv_transpose_shadow_kernel, h->L.tjobs.tile0[5], 256, 0, st, h->rep[0].shadow, h->rep[0].wt, h->rep[1].wt, h->L.tjobs);
    h->launches++;
}

void op_conv_fwd(alexnet* h, int r, int l, int slot, cudaStream_t st, bool early_weights = false) {
    launch_gemm(h, h->rep[r].conv_fwd[l][slot], st, early_weights);
}
void op_conv_bwd(alexnet* h, int r, int l, cudaStream_t st, bool early_weights = false) { launch_gemm(h, h->rep[r].conv_bwd[l], st, early_weights); }
// reduce == false: the split partials stay as they are; the update that follows the pass adds them (op_update with a slot)
void op_conv_wg(alexnet* h, int r, int l, int slot, cudaStream_t st, bool reduce = true) {
    Replica& R = h->rep[r];
    const ConvL& c = h->L.conv[l];
    const Plan& P = R.conv_wg[l][slot];
    launch_gemm(h, P, st);     // weight-gradient partials per row split, and the bias-gradient partials
    if (!reduce) return;
    const long long total = (long long)c.taps * c.cout * c.cig;
    launch_k(kn::wgrad_reduce_kernel, nblk(total, 256), 256, 0, st, h->ws + h->ws_conv_off[l], P.w.splits, P.w.split_stride, total,
             R.g + c.w_off, l == 0, h->bias_partial + (size_t)l * kBiasPartial, c.cout, R.g + c.b_off);
    h->launches++;
}
void op_fc_fwd(alexnet* h, int r, int l, uint64_t step, cudaStream_t st, bool eval = false, bool gemm_only = false,
               bool early_weights = false) {
    Replica& R = h->rep[r];
    const FcL& f = h->L.fc[l];
    Plan& P = R.fc_fwd[l];
    bf16* outs[3] = {R.f6, R.f7, nullptr};
    uint8_t* keeps[3] = {R.m6, R.m7, nullptr};
    int drop = l < 2 && h->cfg.dropout_p > 0.f;
    float scale = h->drop_scale;
    if (eval && drop) {    // no mask at evaluation: its expectation, unless training already rescales (inverted dropout)
        drop = 2;
        scale = (h->cfg.flags & ALEXNET_FLAG_INVERTED_DROPOUT) ? 1.f : 1.f - h->cfg.dropout_p;
    }
    const uint64_t key = kn::stream_key(h->cfg.seed, 2 + l, r, step);
    if (P.c.zcluster) {      // reduction, bias, ReLU and dropout inside the GEMM kernel (a cluster per tile)
        P.c.fc_relu = 1; P.c.fc_dropout = drop; P.c.fc_key = key; P.c.fc_thr24 = h->thr24; P.c.fc_scale = scale;
        P.c.fc_out = outs[l]; P.c.fc_keep = keeps[l];
        launch_gemm(h, P, st, early_weights);
        return;
    }
    launch_gemm(h, P, st, early_weights);
    if (gemm_only) return;     // the split reduction is part of the kernel that follows (fc8 inside the step)
    const long long total = (long long)h->B * f.N;
    launch_k(kn::fc_reduce_fwd_kernel, nblk(total, 256), 256, 0, st, h->ws, P.c.splits, P.c.split_stride, R.w + f.b_off, h->B, f.N,
                                                                l < 2, drop, key, h->thr24, scale, outs[l],
                                                                l == 2 ? R.z : nullptr, keeps[l]);
    h->launches++;
}
void op_fc_bwd(alexnet* h, int r, int l, cudaStream_t st) {
    Replica& R = h->rep[r];
    const FcL& f = h->L.fc[l];
    const Plan& P = R.fc_bwd[l];
    launch_gemm(h, P, st);
    const bf16* masks[3] = {nullptr, R.f6, R.f7};
    bf16* outs[3] = {R.dp5, R.df6, R.df7};
    // the data gradient of layer l is the output gradient of layer l-1: its column sums are that layer's bias gradient
    float* db = l > 0 ? R.g + h->L.fc[l - 1].b_off : nullptr;
    launch_k(kn::fc_reduce_bwd_kernel, nblk(f.K, 32), 256, 0, st, h->ws, P.p.splits, P.p.split_stride, masks[l], h->drop_scale, h->B, f.K,
                                                           outs[l], db);
    h->launches++;
}
void op_fc_wg(alexnet* h, int r, int l, bool with_bias, cudaStream_t st, bool plain = false) {
    Replica& R = h->rep[r];
    const FcL& f = h->L.fc[l];
    launch_gemm(h, plain ? R.fc_wg_plain[l] : R.fc_wg[l], st);
    if (with_bias) {    // in the step only fc8 needs this: fc6 / fc7 get theirs from the data-gradient reduction above them
        const bf16* dyv[3] = {R.df6, R.df7, R.dz};
        colsum(h, dyv[l], h->B, f.N, R.g + f.b_off, st);
    }
}
void op_lrn_fwd(alexnet* h, int r, int which, cudaStream_t st) {
    Replica& R = h->rep[r];
    R.n_stale[which] = false;
    const Grid& g = h->L.conv[which].gout;
    const long long rows = (long long)h->B * g.Hp * g.Wp;
    launch_k(kn::lrn_fwd_kernel, nblk(rows * (g.C / 8), 256), 256, 0, st, which ? R.a2 : R.a1, which ? R.n2 : R.n1,
                                                                   (unsigned)(rows * (g.C / 8)), (unsigned)(g.C / 8),
                                                                   h->alpha_eff, h->cfg.lrn_beta, h->cfg.lrn_k);
    h->launches++;
}
void op_lrn_bwd(alexnet* h, int r, int which, cudaStream_t st) {
    Replica& R = h->rep[r];
    const Grid& g = h->L.conv[which].gout;
    const long long rows = (long long)h->B * g.Hp * g.Wp;
    launch_k(kn::lrn_bwd_kernel, nblk(rows * (g.C / 8), 256), 256, 0, st, which ? R.a2 : R.a1, which ? R.dn2 : R.dn1,
                                                                   which ? R.da2 : R.da1, (unsigned)(rows * (g.C / 8)),
                                                                   (unsigned)(g.C / 8), h->alpha_eff, h->cfg.lrn_beta, h->cfg.lrn_k);
    h->launches++;
}
struct PoolGeo { int C, Hpi, Wpi, Hi, Wi, Ho, Wo, Hpo, Wpo; };
const PoolGeo kPool[3] = {{96, 57, 57, 55, 55, 27, 27, 29, 29}, {256, 29, 29, 27, 27, 13, 13, 14, 14}, {256, 14, 14, 13, 13, 6, 6, 6, 6}};
void op_pool_fwd(alexnet* h, int r, int which, cudaStream_t st) {
    Replica& R = h->rep[r];
    const PoolGeo& g = kPool[which];
    const bf16* x[3] = {R.n1, R.n2, R.a5};
    bf16* y[3] = {R.p1, R.p2, R.p5};
    uint8_t* a[3] = {R.arg1, R.arg2, R.arg5};
    const dim3 grid(nblk((long long)g.Wo * (g.C / 8), 256), g.Ho, h->B);
    launch_k(kn::pool_fwd_kernel, grid, 256, 0, st, x[which], y[which], a[which], g.C / 8, g.Hpi, g.Wpi, g.Ho, g.Wo, g.Hpo, g.Wpo);
    h->launches++;
}
void op_pool_bwd(alexnet* h, int r, int which, cudaStream_t st) {
    Replica& R = h->rep[r];
    if (which < 2) R.dn_stale[which] = false;
    const PoolGeo& g = kPool[which];
    const bf16* dy[3] = {R.dp1, R.dp2, R.dp5};
    const uint8_t* a[3] = {R.arg1, R.arg2, R.arg5};
    const bf16* relu[3] = {nullptr, nullptr, R.a5};
    bf16* dx[3] = {R.dn1, R.dn2, R.da5};
    const dim3 grid(nblk((long long)g.Wpi * (g.C / 8), 256), g.Hpi, h->B);
    launch_k(kn::pool_bwd_kernel, grid, 256, 0, st, dy[which], a[which], relu[which], dx[which], g.C / 8, g.Hpi, g.Wpi,
                                              g.Hi, g.Wi, g.Ho, g.Wo, g.Hpo, g.Wpo);
    h->launches++;
}
// fused LRN + pool kernels, instantiated for the two LRN layers: {vectors per pixel, vectors per block, W, H, output rows
// per block, threads} forward; {vectors per pixel, W, H, pixels per pass, threads} backward
// (the last parameter: exponent beta = 0.75 known at compile time)
#define LRN_POOL_FWD_1(B75) kn::lrn_pool_fwd_kernel<12, 6, 55, 55, 3, 352, B75>
#define LRN_POOL_FWD_2(B75) kn::lrn_pool_fwd_kernel<32, 8, 27, 27, 3, 224, B75>
#define POOL_LRN_BWD_1(B75) kn::pool_lrn_bwd_kernel<12, 55, 55, 28, 352, B75, true>
#define POOL_LRN_BWD_2(B75) kn::pool_lrn_bwd_kernel<32, 27, 27, 9, 288, B75, false>
void op_lrn_pool_fwd(alexnet* h, int r, int which, cudaStream_t st) {
    Replica& R = h->rep[r];
    const PoolGeo& g = kPool[which];
    const bool b75 = h->cfg.lrn_beta == 0.75f;
    const dim3 grid((g.Ho + 2) / 3, which == 0 ? 2 : 4, h->B);
    const size_t smem = which == 0 ? (size_t)7 * 55 * 6 * 16 : (size_t)7 * 27 * 8 * 16;
    auto k = which == 0 ? (b75 ? LRN_POOL_FWD_1(true) : LRN_POOL_FWD_1(false)) : (b75 ? LRN_POOL_FWD_2(true) : LRN_POOL_FWD_2(false));
    launch_k(k, grid, which == 0 ? 352 : 224, smem, st, which ? R.a2 : R.a1, which ? R.p2 : R.p1, which ? R.arg2 : R.arg1, g.Hpi, g.Wpi,
             g.Hpo, g.Wpo, h->alpha_eff, h->cfg.lrn_beta, h->cfg.lrn_k);
    h->launches++;
    R.n_stale[which] = true;
}
void op_pool_lrn_bwd(alexnet* h, int r, int which, cudaStream_t st) {
    Replica& R = h->rep[r];
    const PoolGeo& g = kPool[which];
    const bool b75 = h->cfg.lrn_beta == 0.75f;
    const size_t smem = which == 0 ? (size_t)2 * 55 * 12 * 48 : (size_t)2 * 27 * 32 * 32;     // gradient tile (fp32) (+ two rows of a: LRN1)
    auto k = which == 0 ? (b75 ? POOL_LRN_BWD_1(true) : POOL_LRN_BWD_1(false)) : (b75 ? POOL_LRN_BWD_2(true) : POOL_LRN_BWD_2(false));
    launch_k(k, dim3((g.Hpi + 1) / 2, h->B), which == 0 ? 352 : 288, smem, st, which ? R.a2 : R.a1, which ? R.dp2 : R.dp1,
             which ? R.arg2 : R.arg1, which ? R.da2 : R.da1, g.Hpi, g.Wpi, g.Hpo, g.Wpo, h->alpha_eff, h->cfg.lrn_beta, h->cfg.lrn_k);
    h->launches++;
    R.dn_stale[which] = true;
}
void op_softmax(alexnet* h, int r, int slot, cudaStream_t st) {
    Replica& R = h->rep[r];
    launch_k(kn::softmax_xent_kernel, h->B, 256, 0, st, R.z, R.labels[slot], R.dz, R.loss_n, h->B, 1000);
    launch_k(kn::mean_kernel, 1, 256, 0, st, R.loss_n, h->B, R.loss);
    h->launches += 2;
}
// fc8's split reduction + bias, softmax cross-entropy and the mean loss in one launch (the step's form; N <= 1024)
// fc6 -> fc7 -> fc8 (partials) in one cooperative launch; false when the driver refuses the launch (the caller then runs the
// three layers one by one, and the chain stays off)
bool op_fc_chain(alexnet* h, int r, uint64_t step, cudaStream_t st, bool eval) {
    Replica& R = h->rep[r];
    tc::FcChainParams& q = R.chain;
    for (int l = 0; l < 2; ++l) {
        int drop = h->cfg.dropout_p > 0.f;
        float scale = h->drop_scale;
        if (eval && drop) { drop = 2; scale = (h->cfg.flags & ALEXNET_FLAG_INVERTED_DROPOUT) ? 1.f : 1.f - h->cfg.dropout_p; }
        q.L[l].dropout = drop; q.L[l].scale = scale; q.L[l].thr24 = h->thr24;
        q.L[l].key = kn::stream_key(h->cfg.seed, 2 + l, r, step);
    }
    q.gate_base = R.chain_gate;
    const int grid = R.fc_fwd[0].c.tiles_total;
    if (h->prof) {
        while (h->prof_ev.size() < h->prof_used + 2) {
            cudaEvent_t e;
            if (cudaEventCreate(&e) != cudaSuccess) { h->prof = false; break; }
            h->prof_ev.push_back(e);
        }
    }
    if (h->prof) cudaEventRecord(h->prof_ev[h->prof_used], st);
    cudaError_t e = cudaErrorUnknown;
    for (; R.chain_mode && R.chain_mode <= 2; ++R.chain_mode) {
        cudaLaunchConfig_t lc{};
        lc.gridDim = dim3(grid); lc.blockDim = dim3(tc::kChainThreads); lc.dynamicSmemBytes = tc::fc_chain_smem_bytes(); lc.stream = st;
        cudaLaunchAttribute at[3] = {};
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = tc::kChainCluster; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        at[1].id = cudaLaunchAttributeCooperative;
        at[1].val.cooperative = 1;
        at[2].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[2].val.programmaticStreamSerializationAllowed = 1;
        lc.attrs = at; lc.numAttrs = R.chain_mode == 1 ? 3 : 2;
        e = cudaLaunchKernelEx(&lc, tc::fc_chain_kernel, q);
        if (e == cudaSuccess) break;
        cudaGetLastError();      // a refused launch configuration is not sticky: try the next form
    }
    if (e != cudaSuccess) { R.chain_mode = 0; return false; }
    R.chain_gate += (unsigned)(q.nlayers - 1) * (unsigned)grid;
    if (h->prof) {
        cudaEventRecord(h->prof_ev[h->prof_used + 1], st);
        h->prof_kind.push_back(3);
        h->prof_used += 2;
    }
    h->launches++;
    return true;
}
void op_fc8_softmax(alexnet* h, int r, int slot, cudaStream_t st) {
    Replica& R = h->rep[r];
    const FcL& f = h->L.fc[2];
    const Plan& P = R.fc_fwd[2];
    launch_k(kn::fc8_softmax_xent_kernel, h->B, 256, 0, st, h->ws, P.c.splits, P.c.split_stride, R.w + f.b_off, R.z, R.labels[slot], R.dz,
             R.loss_n, R.loss, h->status + 8, h->B, f.N);
    h->launches++;
}
// The conv split reduction may ride in the update launch when that launch takes the conv filters and every bias in one go
bool update_can_reduce_conv(const alexnet* h) {
    return (h->cfg.flags & ALEXNET_FLAG_FUSED_FC_UPDATE) && !(h->cfg.flags & ALEXNET_FLAG_WD_ON_BIASES);
}
// reduce_slot >= 0: the conv weight-gradient kernels of that batch slot left their split partials unreduced (see op_conv_wg)
void op_update(alexnet* h, int r, cudaStream_t st, bool full = false, float gscale = 1.f, int reduce_slot = -1) {
    Replica& R = h->rep[r];
    const Layout& L = h->L;
    const long long nd = (h->cfg.flags & ALEXNET_FLAG_WD_ON_BIASES) ? L.n_total : L.n_weights;
    // internal order: conv filters, FC weights, biases.  The conv filters (with their transposed bf16 copies) have a tiled
    // kernel of their own; the one-pass kernel takes the rest, minus the FC weights when the fused FC update has done them.
    const bool fused = (h->cfg.flags & ALEXNET_FLAG_FUSED_FC_UPDATE) != 0 && !full;
    const float d = h->cfg.lr * h->cfg.weight_decay;
    if (fused && nd == L.n_weights) {
        // only the biases are left beside the conv filters: extra blocks of the filter kernel take them (no decay on biases)
        const long long b4 = L.n_weights / 4, e4 = L.n_total / 4;
        kn::ConvSplitSrc src;
        memset(&src, 0, sizeof(src));
        if (reduce_slot >= 0) {
            src.on = 1;
            for (int l = 0; l < 5; ++l) {
                const tc::WgradParams& wp = R.conv_wg[l][reduce_slot].w;
                src.splits[l] = wp.splits; src.cout[l] = L.conv[l].cout;
                src.ws[l] = h->ws + h->ws_conv_off[l]; src.stride[l] = wp.split_stride;
                src.bpart[l] = h->bias_partial + (size_t)l * kBiasPartial; src.b_off4[l] = L.conv[l].b_off / 4;
            }
        }
        launch_k(kn::sgd_update_conv_kernel, L.tjobs.tile0[5] + nblk(e4 - b4, 256), 256, 0, st, R.w, R.v, R.g, R.shadow, d,
                 h->cfg.lr, h->cfg.momentum, R.wt, L.tjobs, gscale, b4, e4, 0.f, src);
        h->launches++;
        return;
    }
    kn::ConvSplitSrc none;
    memset(&none, 0, sizeof(none));
    launch_k(kn::sgd_update_conv_kernel, L.tjobs.tile0[5], 256, 0, st, R.w, R.v, R.g, R.shadow, d,
             h->cfg.lr, h->cfg.momentum, R.wt, L.tjobs, gscale, 0LL, 0LL, 0.f, none);
    launch_k(kn::sgd_update_kernel, fused ? 148 : 1184, 256, 0, st, R.w, R.v, R.g, R.shadow, (fused ? L.n_weights : L.fc[0].w_off) / 4,
             L.n_total / 4, nd / 4, h->cfg.lr, h->cfg.momentum, h->cfg.weight_decay, gscale);
    h->launches += 2;
}
// both replicas: update from each one's own gradient, then average, in one pass; then the transposed conv filters
void op_update_average(alexnet* h, cudaStream_t st) {
    Replica &A = h->rep[0], &Bq = h->rep[1];
    const Layout& L = h->L;
    const long long nd = (h->cfg.flags & ALEXNET_FLAG_WD_ON_BIASES) ? L.n_total : L.n_weights;
    if (A.w == Bq.w) {      // shared copy
        launch_k(kn::sgd_update_average_shared_kernel, 1184, 256, 0, st, A.w, A.v, A.g, Bq.g, A.shadow, L.n_total / 4, nd / 4,
                 h->cfg.lr, h->cfg.momentum, h->cfg.weight_decay);
        h->launches++;
        refresh_shadows(h, 0, false, st);
        return;
    }
    launch_k(kn::sgd_update_average_kernel, 1184, 256, 0, st, A.w, A.v, A.g, Bq.w, Bq.v, Bq.g, A.shadow, Bq.shadow, L.n_total / 4,
             nd / 4, h->cfg.lr, h->cfg.momentum, h->cfg.weight_decay);
    h->launches++;
    refresh_transposed_both(h, st);
}
void op_scale_refresh(alexnet* h, int r, float scale, cudaStream_t st) {
    Replica& R = h->rep[r];
    if (scale == 1.f) { refresh_shadows(h, r, true, st); return; }
    launch_k(kn::scale_refresh_kernel, 1184, 256, 0, st, R.w, R.v, R.shadow, h->L.n_total / 4, scale);
    h->launches++;
    refresh_shadows(h, r, false, st);
}
void op_average(alexnet* h, cudaStream_t st) {
    Replica &A = h->rep[0], &Bq = h->rep[1];
    launch_k(kn::replica_average_kernel, 1184, 256, 0, st, A.w, Bq.w, A.v, Bq.v, A.shadow, Bq.shadow, h->L.n_total / 4);
    h->launches++;
    refresh_transposed_both(h, st);
}
void op_preprocess(alexnet* h, int r, int slot, uint64_t step, cudaStream_t st, bool eval = false) {
    Replica& R = h->rep[r];
    kn::ColorAug aug = h->color;
    aug.key = kn::stream_key(h->cfg.seed, 10, r, step);
    const dim3 grid(57, h->B);
    if (aug.sigma != 0.f && !eval)
        launch_k(kn::preprocess_kernel<true>, grid, 256, 0, st, R.stage[slot], h->mean, R.x0[slot], R.cf[slot], h->B,
                 kn::stream_key(h->cfg.seed, 1, r, step), 0, aug);
    else
        launch_k(kn::preprocess_kernel<false>, grid, 256, 0, st, R.stage[slot], h->mean, R.x0[slot], R.cf[slot], h->B,
                 kn::stream_key(h->cfg.seed, 1, r, step), eval ? 1 : 0, aug);
    h->launches++;
}

void forward(alexnet* h, int r, int slot, cudaStream_t st, bool eval) {
    Replica& R = h->rep[r];
    const uint64_t step = R.slot_step[slot];
    // conv1 may directly follow the kernel that wrote its weights (the update of the step before): it waits in full.  Its
    // CTAs hold every SM until it ends, so no later kernel of the pass can start (and read weights) before that writer is done.
    op_conv_fwd(h, r, 0, slot, st); op_lrn_pool_fwd(h, r, 0, st);
    op_conv_fwd(h, r, 1, slot, st, true); op_lrn_pool_fwd(h, r, 1, st);
    op_conv_fwd(h, r, 2, slot, st, true); op_conv_fwd(h, r, 3, slot, st, true); op_conv_fwd(h, r, 4, slot, st, true);
    op_pool_fwd(h, r, 2, st);
    if (!R.chain_mode || !op_fc_chain(h, r, step, st, eval)) {
        op_fc_fwd(h, r, 0, step, st, eval, false, true); op_fc_fwd(h, r, 1, step, st, eval, false, true);
        op_fc_fwd(h, r, 2, step, st, eval, true, true);
    }
    op_fc8_softmax(h, r, slot, st);
}
void forward_backward(alexnet* h, int r, int slot, cudaStream_t st, bool plain_fc = false, bool defer_conv_reduce = false) {
    forward(h, r, slot, st, false);
    // the data gradient reads the layer's weights, so it comes first when the weight-gradient kernel updates them in place
    const bool fused = (h->cfg.flags & ALEXNET_FLAG_FUSED_FC_UPDATE) != 0 && !plain_fc;
    // Every independent branch of the backward pass runs on its own stream: with the fused update the weight-gradient kernel
    // of an FC layer (HBM-bound: it streams the layer's weights and momentum) once the layer's data gradient has read the old
    // weights, and the weight gradient of a conv layer (kernel, then split reduction) once the layer's dy exists.  The chain
    // of data gradients stays on `st`.  The kernels of the branches fill the SMs that the chain leaves idle (small split
    // GEMMs and reductions of the FC layers, last rounds and tails of the conv kernels) and overlap HBM-bound with
    // tensor-bound work; each branch has its own region of the split workspace and of the bias partials.  `st` joins all
    // branches before it returns.  Per-kernel profiling keeps everything on one stream.
    const bool fork = h->side[0] != nullptr && !h->prof;
    bool used[alexnet::kBranches] = {};
    auto branch = [&](int b) -> cudaStream_t {       // fork branch b from `st` here
        if (!fork) return st;
        cudaEventRecord(h->ev_fork[b], st);
        cudaStreamWaitEvent(h->side[b], h->ev_fork[b], 0);
        used[b] = true;
        return h->side[b];
    };
    for (int l = 2; l >= 0; --l) {
        if (fused) { op_fc_bwd(h, r, l, st); op_fc_wg(h, r, l, l == 2, branch(l)); }
        else if (plain_fc) { op_fc_wg(h, r, l, l == 2, branch(l), true); op_fc_bwd(h, r, l, st); }
        else { op_fc_wg(h, r, l, l == 2, st); op_fc_bwd(h, r, l, st); }
    }
    op_pool_bwd(h, r, 2, st);
    // (the transposed bf16 filters that the data gradients read are written between steps only: they may load early)
    op_conv_wg(h, r, 4, slot, branch(3 + 4), !defer_conv_reduce); op_conv_bwd(h, r, 4, st, true);
    op_conv_wg(h, r, 3, slot, branch(3 + 3), !defer_conv_reduce); op_conv_bwd(h, r, 3, st, true);
    op_conv_wg(h, r, 2, slot, branch(3 + 2), !defer_conv_reduce); op_conv_bwd(h, r, 2, st, true);
    op_pool_lrn_bwd(h, r, 1, st);
    op_conv_wg(h, r, 1, slot, branch(3 + 1), !defer_conv_reduce); op_conv_bwd(h, r, 1, st, true);
    op_pool_lrn_bwd(h, r, 0, st);
    op_conv_wg(h, r, 0, slot, branch(3 + 0), !defer_conv_reduce);
    for (int b = 0; b < alexnet::kBranches; ++b)
        if (used[b]) {
            cudaEventRecord(h->ev_side_done[b], h->side[b]);
            cudaStreamWaitEvent(st, h->ev_side_done[b], 0);
        }
    h->fc_grads_on_branches = used[0] && used[1] && used[2] && !fused;
    if (h->ev_backward_done) cudaEventRecord(h->ev_backward_done, st);
}

int check_status(alexnet* h) {
    if (h->latched) return h->latched;
    return ALEXNET_OK;
}
int poll_status(alexnet* h) {  // after a synchronisation
    int st = 0;
    cudaError_t e = cudaMemcpy(&st, h->status, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return fail(h, ALEXNET_ERR_CUDA, std::string("status read: ") + cudaGetErrorString(e));
    if (st) { h->latched = ALEXNET_ERR_DEVICE_TIMEOUT; return fail(h, ALEXNET_ERR_DEVICE_TIMEOUT, "a bounded device-side wait expired"); }
    return ALEXNET_OK;
}

// N(0, std^2) init from the hash (stream 6), identical in every replica; written at internal positions
__global__ void init_kernel(float* arena, const kn::ParamSegs segs, uint64_t key, float std_) {
    kn::pdl_sync();
    const long long stride = (long long)gridDim.x * blockDim.x;
    const long long total = 60965224;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        int s = 0;
        while (s < 15 && i >= segs.s[s + 1].canon_off) ++s;
        float val = 0.f;
        if ((s & 1) == 0) {  // weight segments
            const uint64_t r = kn::draw(key, (uint64_t)i);
            const float u1 = ((float)(r >> 40) + 1.f) * (1.f / 16777216.f);
            const float u2 = (float)((r >> 16) & 0xFFFFFF) * (1.f / 16777216.f);
            val = std_ * sqrtf(-2.f * logf(u1)) * cospif(2.f * u2);
        }
        arena[kn::canon_to_internal(segs.s[s], i - segs.s[s].canon_off)] = val;
    }
}

// -------------------------------------------------------------- tensor table
bool tensor_desc(alexnet* h, int r, int id, Tensor* T) {
    Replica& R = h->rep[r];
    const int ls = R.last_slot;
    auto grid = [&](void* p, const Grid& g, int C) { *T = Tensor{p, 0, C, g.Hp, g.Wp, g.H, g.W, 0}; };
    const Grid g1 = h->L.conv[0].gout, g2 = h->L.conv[1].gout, g3 = h->L.conv[2].gout;
    const Grid gp5 = Grid{6, 6, 6, 6, 256};
    switch (id) {
        case ALEXNET_T_CROPFLIP: *T = Tensor{R.cf[ls], 6, 0, 0, 0, 0, 0, 3}; return true;
        case ALEXNET_T_X0: *T = Tensor{R.x0[ls], 5, 3, 57, 57, 227, 227, 0}; return true;
        case ALEXNET_T_A1: grid(R.a1, g1, 96); return true;
        case ALEXNET_T_N1: grid(R.n1, g1, 96); return true;
        case ALEXNET_T_P1: grid(R.p1, g2, 96); return true;
        case ALEXNET_T_ARG1: *T = Tensor{R.arg1, 1, 96, 27, 27, 27, 27, 0}; return true;
        case ALEXNET_T_A2: grid(R.a2, g2, 256); return true;
        case ALEXNET_T_N2: grid(R.n2, g2, 256); return true;
        case ALEXNET_T_P2: grid(R.p2, g3, 256); return true;
        case ALEXNET_T_ARG2: *T = Tensor{R.arg2, 1, 256, 13, 13, 13, 13, 0}; return true;
        case ALEXNET_T_A3: grid(R.a3, g3, 384); return true;
        case ALEXNET_T_A4: grid(R.a4, g3, 384); return true;
        case ALEXNET_T_A5: grid(R.a5, g3, 256); return true;
        case ALEXNET_T_P5: grid(R.p5, gp5, 256); return true;
        case ALEXNET_T_ARG5: *T = Tensor{R.arg5, 1, 256, 6, 6, 6, 6, 0}; return true;
        case ALEXNET_T_F6: *T = Tensor{R.f6, 2, 0, 0, 0, 0, 0, 4096}; return true;
        case ALEXNET_T_F7: *T = Tensor{R.f7, 2, 0, 0, 0, 0, 0, 4096}; return true;
        case ALEXNET_T_Z: *T = Tensor{R.z, 3, 0, 0, 0, 0, 0, 1000}; return true;
        case ALEXNET_T_M6: *T = Tensor{R.m6, 4, 0, 0, 0, 0, 0, 4096}; return true;
        case ALEXNET_T_M7: *T = Tensor{R.m7, 4, 0, 0, 0, 0, 0, 4096}; return true;
        case ALEXNET_T_DZ: *T = Tensor{R.dz, 2, 0, 0, 0, 0, 0, 1000}; return true;
        case ALEXNET_T_DF7: *T = Tensor{R.df7, 2, 0, 0, 0, 0, 0, 4096}; return true;
        case ALEXNET_T_DF6: *T = Tensor{R.df6, 2, 0, 0, 0, 0, 0, 4096}; return true;
        case ALEXNET_T_DP5: grid(R.dp5, gp5, 256); return true;
        case ALEXNET_T_DA5: grid(R.da5, g3, 256); return true;
        case ALEXNET_T_DA4: grid(R.da4, g3, 384); return true;
        case ALEXNET_T_DA3: grid(R.da3, g3, 384); return true;
        case ALEXNET_T_DP2: grid(R.dp2, g3, 256); return true;
        case ALEXNET_T_DN2: grid(R.dn2, g2, 256); return true;
        case ALEXNET_T_DA2: grid(R.da2, g2, 256); return true;
        case ALEXNET_T_DP1: grid(R.dp1, g2, 96); return true;
        case ALEXNET_T_DN1: grid(R.dn1, g1, 96); return true;
        case ALEXNET_T_DA1: grid(R.da1, g1, 96); return true;
        case ALEXNET_T_LOSS: *T = Tensor{R.loss_n, 7, 0, 0, 0, 0, 0, 1}; return true;
        case ALEXNET_T_DX0: *T = Tensor{R.dx0, 5, 3, 57, 57, 227, 227, 0}; return true;
    }
    return false;
}
size_t tensor_elems(const Tensor& T, int B) {  // canonical element count
    switch (T.kind) {
        case 0: case 1: return (size_t)B * T.C * T.H * T.W;
        case 5: return (size_t)B * 3 * 227 * 227;
        default: return (size_t)B * T.N;
    }
}
size_t tensor_dev_bytes(const Tensor& T, int B) {
    switch (T.kind) {
        case 0: return (size_t)B * T.Hp * T.Wp * T.C * 2;
        case 1: return (size_t)B * T.H * T.W * T.C;
        case 2: return (size_t)B * T.N * 2;
        case 3: case 7: return (size_t)B * T.N * 4;
        case 4: return (size_t)B * T.N;
        case 5: return (size_t)B * 57 * 57 * 48 * 2;
        case 6: return (size_t)B * 3 * 4;
    }
    return 0;
}
inline float bf2f(uint16_t b) { uint32_t u = (uint32_t)b << 16; float f; memcpy(&f, &u, 4); return f; }
inline uint16_t f2bf(float f) {
    uint32_t u; memcpy(&u, &f, 4);
    u = u + 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

// everything the handle owns: streams, events (null where never created); shared by alexnet_destroy and the failure paths
// of alexnet_create
void teardown(alexnet* h) {
    for (int b = 0; b < alexnet::kBranches; ++b) {
        if (h->side[b]) { cudaStreamSynchronize(h->side[b]); cudaStreamDestroy(h->side[b]); }
        if (h->ev_side_done[b]) cudaEventDestroy(h->ev_side_done[b]);
        if (h->ev_fork[b]) cudaEventDestroy(h->ev_fork[b]);
    }
    for (cudaEvent_t e : h->prof_ev) cudaEventDestroy(e);
    if (h->ev_backward_done) cudaEventDestroy(h->ev_backward_done);
    for (int r = 0; r < h->cfg.replicas; ++r)
        for (int s = 0; s < 2; ++s) {
            if (h->rep[r].ready[s]) cudaEventDestroy(h->rep[r].ready[s]);
            if (h->rep[r].consumed[s]) cudaEventDestroy(h->rep[r].consumed[s]);
        }
    delete h;
}
thread_local std::string g_create_err;
int create_fail(alexnet* h, int code, const std::string& msg) {
    g_create_err = msg;
    if (h) teardown(h);
    return code;
}

}  // namespace

// =========================================================================== C ABI
extern "C" {

const char* alexnet_create_error(void) { return g_create_err.c_str(); }

size_t alexnet_param_count(void) { return (size_t)kCanonCount; }

size_t alexnet_workspace_bytes(const alexnet_config_t* cfg) {
    if (!check_cfg(cfg)) return 0;
    alexnet tmp;
    tmp.cfg = *cfg; tmp.B = cfg->batch; tmp.L = make_layout();
    return carve(&tmp, nullptr);
}

int alexnet_create(const alexnet_config_t* cfg, void* dev_arena, size_t arena_bytes, const float* host_mean_image,
                   void* compute_stream, void* copy_stream, alexnet_t** out) {
    if (!out) return create_fail(nullptr, ALEXNET_ERR_ARG, "alexnet_create: out is NULL");
    *out = nullptr;
    if (!check_cfg(cfg)) return create_fail(nullptr, ALEXNET_ERR_ARG, "alexnet_create: invalid configuration");
    if (!dev_arena || ((uintptr_t)dev_arena & 1023)) return create_fail(nullptr, ALEXNET_ERR_ARG, "alexnet_create: arena is NULL or not 1024-byte aligned");
    alexnet* h = new alexnet();
    h->cfg = *cfg; h->B = cfg->batch; h->L = make_layout();
    h->cs = (cudaStream_t)compute_stream; h->ls = (cudaStream_t)copy_stream;
    h->launches = 0; h->latched = 0; h->prof = false; h->prof_used = 0;
    h->alpha_eff = (cfg->flags & ALEXNET_FLAG_LRN_ALPHA_DIV_N) ? cfg->lrn_alpha / 5.f : cfg->lrn_alpha;
    h->drop_scale = ((cfg->flags & ALEXNET_FLAG_INVERTED_DROPOUT) && cfg->dropout_p > 0.f) ? 1.f / (1.f - cfg->dropout_p) : 1.f;
    h->thr24 = (uint32_t)floor((double)cfg->dropout_p * 16777216.0);
    for (int r = 0; r < 2; ++r)
        for (int s = 0; s < 2; ++s) { h->rep[r].ready[s] = nullptr; h->rep[r].consumed[s] = nullptr; }
    // nothing is created before the size check: a caller probing arena sizes leaves nothing behind
    const size_t need = carve(h, nullptr);
    if (arena_bytes < need)
        return create_fail(h, ALEXNET_ERR_NOMEM, "alexnet_create: arena of " + std::to_string(arena_bytes) + " bytes, " + std::to_string(need) + " needed");
    h->arena = (uint8_t*)dev_arena; h->arena_bytes = arena_bytes;
    carve(h, h->arena);
#define CKC(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return create_fail(h, ALEXNET_ERR_CUDA, std::string("alexnet_create: ") + #call + ": " + cudaGetErrorString(e_)); } while (0)
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    CKC(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
    if (!fn || qres != cudaDriverEntryPointSuccess) return create_fail(h, ALEXNET_ERR_CUDA, "alexnet_create: the driver has no cuTensorMapEncodeTiled");
    h->encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
    CKC(cudaFuncSetAttribute(tc::gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    CKC(cudaFuncSetAttribute(tc::conv_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    CKC(cudaFuncSetAttribute(tc::conv_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    CKC(cudaFuncSetAttribute(tc::wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    CKC(cudaFuncSetAttribute(tc::fc_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    // (static + dynamic shared memory of both exceeds the 48 KB that need no opt-in)
    CKC(cudaFuncSetAttribute(POOL_LRN_BWD_1(true), cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * 55 * 12 * 48));
    CKC(cudaFuncSetAttribute(POOL_LRN_BWD_1(false), cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * 55 * 12 * 48));
    CKC(cudaFuncSetAttribute(POOL_LRN_BWD_2(true), cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * 27 * 32 * 32));
    CKC(cudaFuncSetAttribute(POOL_LRN_BWD_2(false), cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * 27 * 32 * 32));
    {
        int dev = 0;
        CKC(cudaGetDevice(&dev));
        CKC(cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, dev));
    }
    for (int b = 0; b < alexnet::kBranches; ++b) {
        CKC(cudaStreamCreateWithFlags(&h->side[b], cudaStreamNonBlocking));
        CKC(cudaEventCreateWithFlags(&h->ev_side_done[b], cudaEventDisableTiming));
        CKC(cudaEventCreateWithFlags(&h->ev_fork[b], cudaEventDisableTiming));
    }
    CKC(cudaEventCreateWithFlags(&h->ev_backward_done, cudaEventDisableTiming));
    // pad positions of every grid must be zero from the start; gradients and momentum start at zero
    CKC(cudaMemsetAsync(h->arena, 0, need, h->cs));
    if (host_mean_image) CKC(cudaMemcpyAsync(h->mean, host_mean_image, 256 * 256 * 3 * sizeof(float), cudaMemcpyHostToDevice, h->cs));
    for (int r = 0; r < cfg->replicas; ++r) {
        Replica& R = h->rep[r];
        R.next_load = R.next_train = R.loaded = R.last_slot = 0;
        R.n_stale[0] = R.n_stale[1] = R.dn_stale[0] = R.dn_stale[1] = false;
        R.grad_pending = false;
        for (int s = 0; s < 2; ++s) {
            CKC(cudaEventCreateWithFlags(&R.ready[s], cudaEventDisableTiming));
            CKC(cudaEventCreateWithFlags(&R.consumed[s], cudaEventDisableTiming));
            R.consumed_valid[s] = false; R.slot_step[s] = 0;
        }
        if (cfg->init_std > 0.f) {
            launch_k(init_kernel, 1184, 256, 0, h->cs, R.w, h->L.segs, kn::stream_key(cfg->seed, 6, 0, 0), cfg->init_std);
            h->launches++;
        }
        refresh_shadows(h, r, true, h->cs);
        int rc = build_plans(h, r);
        if (rc) return create_fail(h, rc, "alexnet_create: " + h->err);
    }
    CKC(cudaStreamSynchronize(h->cs));
    CKC(cudaGetLastError());
    *out = h;
    return ALEXNET_OK;
}

int alexnet_destroy(alexnet_t* h) {
    if (!h) return ALEXNET_ERR_ARG;
    cudaStreamSynchronize(h->cs);
    cudaStreamSynchronize(h->ls);
    teardown(h);
    return ALEXNET_OK;
}

int alexnet_load_batch_async(alexnet_t* h, int replica, const uint8_t* images, const int32_t* labels, uint64_t step) {
    if (!h) return ALEXNET_ERR_ARG;
    if (replica < 0 || replica >= h->cfg.replicas || !images || !labels) return fail(h, ALEXNET_ERR_ARG, "load_batch_async: bad argument");
    if (int rc = check_status(h)) return rc;
    Replica& R = h->rep[replica];
    if (R.loaded == 2) return fail(h, ALEXNET_ERR_STATE, "load_batch_async: both batch slots hold unconsumed batches");
    const int s = R.next_load;
    if (R.consumed_valid[s]) CK(cudaStreamWaitEvent(h->ls, R.consumed[s], 0));
    CK(cudaMemcpyAsync(R.stage[s], images, (size_t)h->B * 196608, cudaMemcpyDefault, h->ls));
    CK(cudaMemcpyAsync(R.labels[s], labels, (size_t)h->B * sizeof(int32_t), cudaMemcpyDefault, h->ls));
    op_preprocess(h, replica, s, step, h->ls);
    CK(cudaEventRecord(R.ready[s], h->ls));
    R.slot_step[s] = step;
    R.last_slot = s; R.next_load ^= 1; R.loaded++;
    return ALEXNET_OK;
}

static bool shared_weights(const alexnet_t* h) { return h->cfg.replicas == 2 && (h->cfg.flags & ALEXNET_FLAG_SHARED_REPLICA_WEIGHTS); }

static int step_impl(alexnet_t* h, int replica, float* host_loss, bool with_update) {
    if (!h) return ALEXNET_ERR_ARG;
    if (replica < 0 || replica >= h->cfg.replicas) return fail(h, ALEXNET_ERR_ARG, "train_step: bad replica");
    if (with_update && shared_weights(h))
        return fail(h, ALEXNET_ERR_STATE, "train_step: the replicas share one copy of the parameters; use alexnet_forward_backward on both and alexnet_update_and_average");
    if (int rc = check_status(h)) return rc;
    Replica& R = h->rep[replica];
    if (R.loaded == 0) return fail(h, ALEXNET_ERR_STATE, "train_step: no loaded batch");
    const int s = R.next_train;
    CK(cudaStreamWaitEvent(h->cs, R.ready[s], 0));
    // a step with its update: the conv split partials are added by the update launch (five reduction launches fewer)
    const bool defer = with_update && update_can_reduce_conv(h);
    forward_backward(h, replica, s, h->cs, !with_update, defer);
    CK(cudaEventRecord(R.consumed[s], h->cs));
    R.consumed_valid[s] = true;
    if (with_update) op_update(h, replica, h->cs, false, 1.f, defer ? s : -1);
    R.grad_pending = !with_update;
    R.last_slot = s; R.next_train ^= 1; R.loaded--;
    CK(cudaGetLastError());
    if (host_loss) {
        CK(cudaMemcpyAsync(host_loss, R.loss, sizeof(float), cudaMemcpyDeviceToHost, h->cs));
        CK(cudaStreamSynchronize(h->cs));
        return poll_status(h);
    }
    return ALEXNET_OK;
}

int alexnet_train_step(alexnet_t* h, int replica, float* host_loss) { return step_impl(h, replica, host_loss, true); }
int alexnet_forward_backward(alexnet_t* h, int replica, float* host_loss) { return step_impl(h, replica, host_loss, false); }

int alexnet_apply_update(alexnet_t* h, int replica, float grad_scale) {
    if (!h) return ALEXNET_ERR_ARG;
    if (replica < 0 || replica >= h->cfg.replicas || !(grad_scale == grad_scale))
        return fail(h, ALEXNET_ERR_ARG, "apply_update: bad argument");
    if (int rc = check_status(h)) return rc;
    Replica& R = h->rep[replica];
    if (shared_weights(h)) return fail(h, ALEXNET_ERR_STATE, "apply_update: the replicas share one copy of the parameters; use alexnet_update_and_average");
    if (!R.grad_pending) return fail(h, ALEXNET_ERR_STATE, "apply_update: no pending gradient (call alexnet_forward_backward first)");
    op_update(h, replica, h->cs, true, grad_scale);
    R.grad_pending = false;
    CK(cudaGetLastError());
    return ALEXNET_OK;
}

int alexnet_update_and_average(alexnet_t* h) {
    if (!h) return ALEXNET_ERR_ARG;
    if (int rc = check_status(h)) return rc;
    if (h->cfg.replicas != 2) return fail(h, ALEXNET_ERR_STATE, "update_and_average: needs two replicas");
    if (!h->rep[0].grad_pending || !h->rep[1].grad_pending)
        return fail(h, ALEXNET_ERR_STATE, "update_and_average: both replicas need a pending gradient (alexnet_forward_backward)");
    op_update_average(h, h->cs);
    h->rep[0].grad_pending = h->rep[1].grad_pending = false;
    CK(cudaGetLastError());
    return ALEXNET_OK;
}

int alexnet_param_regions(alexnet_t* h, int replica, float** dev_w, float** dev_v, float** dev_g, size_t* n_floats) {
    if (!h) return ALEXNET_ERR_ARG;
    if (replica < 0 || replica >= h->cfg.replicas) return fail(h, ALEXNET_ERR_ARG, "param_regions: bad replica");
    Replica& R = h->rep[replica];
    if (dev_w) *dev_w = R.w;
    if (dev_v) *dev_v = R.v;
    if (dev_g) *dev_g = R.g;
    if (n_floats) *n_floats = (size_t)h->L.n_total;
    return ALEXNET_OK;
}

int alexnet_param_layout(const alexnet_t* h, size_t* fc_weights_begin, size_t* fc_weights_end, size_t* n_floats) {
    if (!h) return ALEXNET_ERR_ARG;
    if (fc_weights_begin) *fc_weights_begin = (size_t)h->L.fc[0].w_off;
    if (fc_weights_end) *fc_weights_end = (size_t)h->L.n_weights;
    if (n_floats) *n_floats = (size_t)h->L.n_total;
    return ALEXNET_OK;
}

int alexnet_stream_wait_fc_gradients(alexnet_t* h, void* stream) {
    if (!h) return ALEXNET_ERR_ARG;
    if (int rc = check_status(h)) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    if (h->fc_grads_on_branches) {
        for (int b = 0; b < 3; ++b) CK(cudaStreamWaitEvent(st, h->ev_side_done[b], 0));
    } else {
        CK(cudaStreamWaitEvent(st, h->ev_backward_done, 0));
    }
    return ALEXNET_OK;
}

int alexnet_scale_and_refresh(alexnet_t* h, int replica, float scale) {
    if (!h) return ALEXNET_ERR_ARG;
    if (replica < 0 || replica >= h->cfg.replicas || !(scale == scale)) return fail(h, ALEXNET_ERR_ARG, "scale_and_refresh: bad argument");
    if (int rc = check_status(h)) return rc;
    if (shared_weights(h) && replica == 1) return ALEXNET_OK;      // replica 0's call has done the shared copy
    op_scale_refresh(h, replica, scale, h->cs);
    CK(cudaGetLastError());
    return ALEXNET_OK;
}

int alexnet_set_color_augmentation(alexnet_t* h, const float* host_eigvec, const float* host_eigval, float sigma) {
    if (!h) return ALEXNET_ERR_ARG;
    if (!(sigma >= 0.f) || (sigma > 0.f && (!host_eigvec || !host_eigval))) return fail(h, ALEXNET_ERR_ARG, "set_color_augmentation: bad argument");
    h->color.sigma = sigma;
    for (int c = 0; c < 3 && sigma > 0.f; ++c)
        for (int i = 0; i < 3; ++i) h->color.pl[3 * c + i] = host_eigvec[3 * c + i] * host_eigval[i];
    return ALEXNET_OK;
}

int alexnet_average_received(alexnet_t* h, int replica, const float* const* dev_w, const float* const* dev_v, int count, int self) {
    if (!h) return ALEXNET_ERR_ARG;
    if (replica < 0 || replica >= h->cfg.replicas || count < 1 || count > 8 || self < 0 || self >= count || !dev_w || !dev_v)
        return fail(h, ALEXNET_ERR_ARG, "average_received: bad argument (1 <= count <= 8, 0 <= self < count)");
    if (int rc = check_status(h)) return rc;
    if (shared_weights(h) && replica == 1) return ALEXNET_OK;      // replica 0's call has done the shared copy
    Replica& R = h->rep[replica];
    kn::RecvList rl{};
    rl.count = count;
    for (int r = 0; r < count; ++r) {
        rl.w[r] = r == self ? R.w : dev_w[r];
        rl.v[r] = r == self ? R.v : dev_v[r];
        if (!rl.w[r] || !rl.v[r] || ((uintptr_t)rl.w[r] & 15) || ((uintptr_t)rl.v[r] & 15))
            return fail(h, ALEXNET_ERR_ARG, "average_received: NULL or misaligned buffer");
    }
    launch_k(kn::average_received_kernel, 1184, 256, 0, h->cs, R.w, R.v, R.shadow, rl, h->L.n_total / 4, 1.f / (float)count);
    h->launches++;
    refresh_shadows(h, replica, false, h->cs);
    CK(cudaGetLastError());
    return ALEXNET_OK;
}

int alexnet_debug_expire_wait(alexnet_t* h, long long budget_cycles) {
    if (!h) return ALEXNET_ERR_ARG;
    if (int rc = check_status(h)) return rc;
    const long long budget = std::min<long long>(200000000LL, std::max<long long>(10000LL, budget_cycles));
    launch_k(tc::wait_probe_kernel, 1, 32, 0, h->cs, h->status, budget);
    h->launches++;
    CK(cudaGetLastError());
    return ALEXNET_OK;
}

int alexnet_loss_async(alexnet_t* h, int replica, float* loss_out) {
    if (!h) return ALEXNET_ERR_ARG;
    if (replica < 0 || replica >= h->cfg.replicas || !loss_out) return fail(h, ALEXNET_ERR_ARG, "loss_async: bad argument");
    if (int rc = check_status(h)) return rc;
    // A 4-byte cudaMemcpyAsync shares the copy engines with the 25 MB batch uploads of the loader stream and was seen to hold
    // the compute stream up by 35 us per step behind one.  Where the destination is visible to the device (device memory, or
    // pinned / registered host memory: the cases the header allows) a one-thread kernel stores the value instead.
    cudaPointerAttributes at{};
    if (cudaPointerGetAttributes(&at, loss_out) == cudaSuccess && at.devicePointer != nullptr &&
        (at.type == cudaMemoryTypeHost || at.type == cudaMemoryTypeDevice || at.type == cudaMemoryTypeManaged)) {
        launch_k(kn::store_value_kernel, 1, 1, 0, h->cs, (const float*)h->rep[replica].loss, (float*)at.devicePointer);
        h->launches++;
        CK(cudaGetLastError());
        return ALEXNET_OK;
    }
    cudaGetLastError();      // (an unregistered host pointer makes the query fail on some drivers: not an error here)
    CK(cudaMemcpyAsync(loss_out, h->rep[replica].loss, sizeof(float), cudaMemcpyDefault, h->cs));
    return ALEXNET_OK;
}

int alexnet_eval_batch(alexnet_t* h, int replica, const uint8_t* images, const int32_t* labels, int32_t* host_top1,
                       int32_t* host_top5, float* host_loss) {
    if (!h) return ALEXNET_ERR_ARG;
    if (replica < 0 || replica >= h->cfg.replicas || !images || !labels) return fail(h, ALEXNET_ERR_ARG, "eval_batch: bad argument");
    if (int rc = check_status(h)) return rc;
    Replica& R = h->rep[replica];
    if (R.loaded != 0) return fail(h, ALEXNET_ERR_STATE, "eval_batch: a loaded training batch is waiting for its train_step");
    const int s = R.next_load;      // the free slot the next training load would use; it stays free afterwards
    if (R.consumed_valid[s]) CK(cudaStreamWaitEvent(h->ls, R.consumed[s], 0));
    CK(cudaMemcpyAsync(R.stage[s], images, (size_t)h->B * 196608, cudaMemcpyDefault, h->ls));
    CK(cudaMemcpyAsync(R.labels[s], labels, (size_t)h->B * sizeof(int32_t), cudaMemcpyDefault, h->ls));
    op_preprocess(h, replica, s, 0, h->ls, true);
    CK(cudaEventRecord(R.ready[s], h->ls));
    R.slot_step[s] = 0; R.last_slot = s;
    CK(cudaStreamWaitEvent(h->cs, R.ready[s], 0));
    forward(h, replica, s, h->cs, true);
    int32_t* counts = (int32_t*)(h->status + 4);    // two counters in the status block
    CK(cudaMemsetAsync(counts, 0, 2 * sizeof(int32_t), h->cs));
    launch_k(kn::topk_count_kernel, h->B, 256, 0, h->cs, R.z, R.labels[s], 1000, counts);
    h->launches++;
    CK(cudaEventRecord(R.consumed[s], h->cs));
    R.consumed_valid[s] = true;
    int32_t hc[2] = {0, 0};
    float loss = 0.f;
    CK(cudaMemcpyAsync(hc, counts, sizeof(hc), cudaMemcpyDeviceToHost, h->cs));
    CK(cudaMemcpyAsync(&loss, R.loss, sizeof(float), cudaMemcpyDeviceToHost, h->cs));
    CK(cudaStreamSynchronize(h->cs));
    CK(cudaGetLastError());
    if (host_top1) *host_top1 = hc[0];
    if (host_top5) *host_top5 = hc[1];
    if (host_loss) *host_loss = loss;
    return poll_status(h);
}

int alexnet_replica_average(alexnet_t* h) {
    if (!h) return ALEXNET_ERR_ARG;
    if (int rc = check_status(h)) return rc;
    if (h->cfg.replicas < 2 || shared_weights(h)) return ALEXNET_OK;     // one copy: nothing to average
    op_average(h, h->cs);
    CK(cudaGetLastError());
    return ALEXNET_OK;
}

int alexnet_get_params(alexnet_t* h, int replica, int which, float* host_out, size_t n) {
    if (!h) return ALEXNET_ERR_ARG;
    if (replica < 0 || replica >= h->cfg.replicas || which < 0 || which > 2 || !host_out || n != (size_t)kCanonCount)
        return fail(h, ALEXNET_ERR_ARG, "get_params: bad argument");
    Replica& R = h->rep[replica];
    const float* src = which == 0 ? R.w : which == 1 ? R.v : R.g;
    launch_k(kn::params_gather_kernel, 1184, 256, 0, h->cs, src, h->canon_tmp, h->L.segs, kCanonCount);
    h->launches++;
    CK(cudaMemcpyAsync(host_out, h->canon_tmp, n * sizeof(float), cudaMemcpyDeviceToHost, h->cs));
    CK(cudaStreamSynchronize(h->cs));
    return poll_status(h);
}

int alexnet_set_params(alexnet_t* h, int replica, int which, const float* host_in, size_t n) {
    if (!h) return ALEXNET_ERR_ARG;
    if (replica < 0 || replica >= h->cfg.replicas || which < 0 || which > 1 || !host_in || n != (size_t)kCanonCount)
        return fail(h, ALEXNET_ERR_ARG, "set_params: bad argument");
    Replica& R = h->rep[replica];
    float* dst = which == 0 ? R.w : R.v;
    CK(cudaMemcpyAsync(h->canon_tmp, host_in, n * sizeof(float), cudaMemcpyHostToDevice, h->cs));
    CK(cudaMemsetAsync(dst, 0, h->L.n_total * sizeof(float), h->cs));
    launch_k(kn::params_scatter_kernel, 1184, 256, 0, h->cs, dst, h->canon_tmp, h->L.segs, kCanonCount);
    h->launches++;
    if (which == 0) refresh_shadows(h, replica, true, h->cs);
    CK(cudaStreamSynchronize(h->cs));
    return ALEXNET_OK;
}

size_t alexnet_tensor_size(const alexnet_t* h, int tensor_id) {
    if (!h) return 0;
    Tensor T;
    if (!tensor_desc((alexnet*)h, 0, tensor_id, &T)) return 0;
    return tensor_elems(T, h->B);
}

int alexnet_get_tensor(alexnet_t* h, int replica, int tensor_id, float* out, size_t n) {
    if (!h) return ALEXNET_ERR_ARG;
    Tensor T;
    if (replica < 0 || replica >= h->cfg.replicas || !out || !tensor_desc(h, replica, tensor_id, &T) || n != tensor_elems(T, h->B))
        return fail(h, ALEXNET_ERR_ARG, "get_tensor: bad argument");
    const int B = h->B;
    {
        Replica& R = h->rep[replica];
        if (tensor_id == ALEXNET_T_N1 && R.n_stale[0]) op_lrn_fwd(h, replica, 0, h->cs);
        if (tensor_id == ALEXNET_T_N2 && R.n_stale[1]) op_lrn_fwd(h, replica, 1, h->cs);
        if (tensor_id == ALEXNET_T_DN1 && R.dn_stale[0]) op_pool_bwd(h, replica, 0, h->cs);
        if (tensor_id == ALEXNET_T_DN2 && R.dn_stale[1]) op_pool_bwd(h, replica, 1, h->cs);
    }
    std::vector<uint8_t> raw(tensor_dev_bytes(T, B));
    CK(cudaStreamSynchronize(h->cs));
    CK(cudaStreamSynchronize(h->ls));
    CK(cudaMemcpy(raw.data(), T.ptr, raw.size(), cudaMemcpyDeviceToHost));
    const uint16_t* hb = (const uint16_t*)raw.data();
    switch (T.kind) {
        case 0:
            for (int b = 0; b < B; ++b) for (int c = 0; c < T.C; ++c) for (int y = 0; y < T.H; ++y) for (int x = 0; x < T.W; ++x)
                out[(((size_t)b * T.C + c) * T.H + y) * T.W + x] = bf2f(hb[(((size_t)b * T.Hp + y) * T.Wp + x) * T.C + c]);
            break;
        case 1:
            for (int b = 0; b < B; ++b) for (int c = 0; c < T.C; ++c) for (int y = 0; y < T.H; ++y) for (int x = 0; x < T.W; ++x)
                out[(((size_t)b * T.C + c) * T.H + y) * T.W + x] = (float)raw[(((size_t)b * T.H + y) * T.W + x) * T.C + c];
            break;
        case 2: for (size_t i = 0; i < n; ++i) out[i] = bf2f(hb[i]); break;
        case 3: case 7: memcpy(out, raw.data(), n * 4); break;
        case 4: for (size_t i = 0; i < n; ++i) out[i] = (float)raw[i]; break;
        case 5:
            for (int b = 0; b < B; ++b) for (int c = 0; c < 3; ++c) for (int y = 0; y < 227; ++y) for (int x = 0; x < 227; ++x)
                out[(((size_t)b * 3 + c) * 227 + y) * 227 + x] =
                    bf2f(hb[(((size_t)b * 57 + y / 4) * 57 + x / 4) * 48 + ((y % 4) * 4 + x % 4) * 3 + c]);
            break;
        case 6: for (size_t i = 0; i < n; ++i) out[i] = (float)((const int32_t*)raw.data())[i]; break;
    }
    return ALEXNET_OK;
}

int alexnet_set_tensor(alexnet_t* h, int replica, int tensor_id, const float* in, size_t n) {
    if (!h) return ALEXNET_ERR_ARG;
    Tensor T;
    if (replica < 0 || replica >= h->cfg.replicas || !in || !tensor_desc(h, replica, tensor_id, &T) || n != tensor_elems(T, h->B))
        return fail(h, ALEXNET_ERR_ARG, "set_tensor: bad argument");
    const int B = h->B;
    std::vector<uint8_t> raw(tensor_dev_bytes(T, B), 0);
    uint16_t* hb = (uint16_t*)raw.data();
    switch (T.kind) {
        case 0:
            for (int b = 0; b < B; ++b) for (int c = 0; c < T.C; ++c) for (int y = 0; y < T.H; ++y) for (int x = 0; x < T.W; ++x)
                hb[(((size_t)b * T.Hp + y) * T.Wp + x) * T.C + c] = f2bf(in[(((size_t)b * T.C + c) * T.H + y) * T.W + x]);
            break;
        case 1:
            for (int b = 0; b < B; ++b) for (int c = 0; c < T.C; ++c) for (int y = 0; y < T.H; ++y) for (int x = 0; x < T.W; ++x)
                raw[(((size_t)b * T.H + y) * T.W + x) * T.C + c] = (uint8_t)in[(((size_t)b * T.C + c) * T.H + y) * T.W + x];
            break;
        case 2: for (size_t i = 0; i < n; ++i) hb[i] = f2bf(in[i]); break;
        case 3: case 7: memcpy(raw.data(), in, n * 4); break;
        case 4: for (size_t i = 0; i < n; ++i) raw[i] = (uint8_t)in[i]; break;
        case 5:
            for (int b = 0; b < B; ++b) for (int c = 0; c < 3; ++c) for (int y = 0; y < 227; ++y) for (int x = 0; x < 227; ++x)
                hb[(((size_t)b * 57 + y / 4) * 57 + x / 4) * 48 + ((y % 4) * 4 + x % 4) * 3 + c] =
                    f2bf(in[(((size_t)b * 3 + c) * 227 + y) * 227 + x]);
            break;
        case 6: for (size_t i = 0; i < n; ++i) ((int32_t*)raw.data())[i] = (int32_t)in[i]; break;
    }
    CK(cudaStreamSynchronize(h->cs));
    CK(cudaStreamSynchronize(h->ls));
    CK(cudaMemcpy(T.ptr, raw.data(), raw.size(), cudaMemcpyHostToDevice));
    {
        Replica& R = h->rep[replica];
        if (tensor_id == ALEXNET_T_N1) R.n_stale[0] = false;
        if (tensor_id == ALEXNET_T_N2) R.n_stale[1] = false;
        if (tensor_id == ALEXNET_T_DN1) R.dn_stale[0] = false;
        if (tensor_id == ALEXNET_T_DN2) R.dn_stale[1] = false;
    }
    return ALEXNET_OK;
}

int alexnet_run_op(alexnet_t* h, int replica, int op, int iters) {
    if (!h) return ALEXNET_ERR_ARG;
    if (replica < 0 || replica >= h->cfg.replicas || op < 0 || op >= ALEXNET_OP_COUNT || iters < 1)
        return fail(h, ALEXNET_ERR_ARG, "run_op: bad argument");
    if ((op == ALEXNET_OP_AVERAGE || op == ALEXNET_OP_UPDATE_AVERAGE) && h->cfg.replicas < 2)
        return fail(h, ALEXNET_ERR_ARG, "run_op: average needs two replicas");
    if (shared_weights(h) && (op == ALEXNET_OP_AVERAGE || op == ALEXNET_OP_UPDATE))
        return fail(h, ALEXNET_ERR_STATE, "run_op: not while the replicas share one copy of the parameters");
    if (int rc = check_status(h)) return rc;
    Replica& R = h->rep[replica];
    const int slot = R.last_slot;
    cudaStream_t st = h->cs;
    for (int it = 0; it < iters; ++it) {
        if (op <= ALEXNET_OP_CONV5_FWD) op_conv_fwd(h, replica, op - ALEXNET_OP_CONV1_FWD, slot, st);
        else if (op <= ALEXNET_OP_CONV5_BWD_DATA) op_conv_bwd(h, replica, op - ALEXNET_OP_CONV2_BWD_DATA + 1, st);
        else if (op <= ALEXNET_OP_CONV5_BWD_WEIGHT) op_conv_wg(h, replica, op - ALEXNET_OP_CONV1_BWD_WEIGHT, slot, st);
        else if (op <= ALEXNET_OP_FC8_FWD) op_fc_fwd(h, replica, op - ALEXNET_OP_FC6_FWD, R.slot_step[slot], st);
        else if (op <= ALEXNET_OP_FC8_BWD_DATA) op_fc_bwd(h, replica, op - ALEXNET_OP_FC6_BWD_DATA, st);
        else if (op <= ALEXNET_OP_FC8_BWD_WEIGHT) op_fc_wg(h, replica, op - ALEXNET_OP_FC6_BWD_WEIGHT, true, st);
        else if (op <= ALEXNET_OP_LRN2_FWD) op_lrn_fwd(h, replica, op - ALEXNET_OP_LRN1_FWD, st);
        else if (op <= ALEXNET_OP_LRN2_BWD) op_lrn_bwd(h, replica, op - ALEXNET_OP_LRN1_BWD, st);
        else if (op <= ALEXNET_OP_POOL5_FWD) op_pool_fwd(h, replica, op - ALEXNET_OP_POOL1_FWD, st);
        else if (op <= ALEXNET_OP_POOL5_BWD) op_pool_bwd(h, replica, op - ALEXNET_OP_POOL1_BWD, st);
        else if (op == ALEXNET_OP_SOFTMAX) op_softmax(h, replica, slot, st);
        else if (op == ALEXNET_OP_UPDATE) op_update(h, replica, st, true);
        else if (op == ALEXNET_OP_AVERAGE) op_average(h, st);
        else if (op == ALEXNET_OP_PREPROCESS) op_preprocess(h, replica, slot, R.slot_step[slot], st);
        else if (op == ALEXNET_OP_CONV1_BWD_DATA) op_conv_bwd(h, replica, 0, st);
        else if (op == ALEXNET_OP_LRN1_POOL1_FWD || op == ALEXNET_OP_LRN2_POOL2_FWD) op_lrn_pool_fwd(h, replica, op - ALEXNET_OP_LRN1_POOL1_FWD, st);
        else if (op == ALEXNET_OP_POOL1_LRN1_BWD || op == ALEXNET_OP_POOL2_LRN2_BWD) op_pool_lrn_bwd(h, replica, op - ALEXNET_OP_POOL1_LRN1_BWD, st);
        else if (op == ALEXNET_OP_UPDATE_AVERAGE) op_update_average(h, st);
        else if (op == ALEXNET_OP_SCALE_REFRESH) op_scale_refresh(h, replica, 1.f, st);
        else if (op == ALEXNET_OP_FC_CHAIN_FWD) {
            if (!R.chain_mode || !op_fc_chain(h, replica, R.slot_step[slot], st, false))
                return fail(h, ALEXNET_ERR_STATE, "the FC forward chain is not available in this configuration");
        }
    }
    CK(cudaGetLastError());
    return ALEXNET_OK;
}

uint64_t alexnet_launch_count(const alexnet_t* h) { return h ? h->launches : 0; }

int alexnet_timeline_read(long long* host_out, int clear) {
#ifdef ALEXNET_TIMELINE
    if (cudaDeviceSynchronize() != cudaSuccess) return ALEXNET_ERR_CUDA;
    if (host_out && cudaMemcpyFromSymbol(host_out, tc::g_timeline, sizeof(long long) * 160 * 16) != cudaSuccess) return ALEXNET_ERR_CUDA;
    if (clear) {
        static const long long zeros[160 * 16] = {0};
        if (cudaMemcpyToSymbol(tc::g_timeline, zeros, sizeof(zeros)) != cudaSuccess) return ALEXNET_ERR_CUDA;
    }
    return ALEXNET_OK;
#else
    (void)host_out; (void)clear;
    return ALEXNET_ERR_STATE;      // this build of the library carries no timeline instrumentation
#endif
}

int alexnet_profile(alexnet_t* h, int enable) {
    if (!h) return ALEXNET_ERR_ARG;
    h->prof = enable != 0;
    return ALEXNET_OK;
}

int alexnet_profile_read(alexnet_t* h, double* ms3, uint64_t* launches3) {
    if (!h || !ms3 || !launches3) return ALEXNET_ERR_ARG;
    CK(cudaStreamSynchronize(h->ls));
    CK(cudaStreamSynchronize(h->cs));
    for (int k = 0; k < 4; ++k) { ms3[k] = 0.0; launches3[k] = 0; }
    for (size_t i = 0; i + 1 < h->prof_used; i += 2) {
        float t = 0.f;
        CK(cudaEventElapsedTime(&t, h->prof_ev[i], h->prof_ev[i + 1]));
        const int k = h->prof_kind[i / 2];
        ms3[k] += t;
        launches3[k]++;
    }
    h->prof_used = 0;
    h->prof_kind.clear();
    return ALEXNET_OK;
}

int alexnet_sync(alexnet_t* h) {
    if (!h) return ALEXNET_ERR_ARG;
    CK(cudaStreamSynchronize(h->ls));
    CK(cudaStreamSynchronize(h->cs));
    if (int rc = check_status(h)) return rc;
    return poll_status(h);
}

const char* alexnet_last_error(const alexnet_t* h) { return h ? h->err.c_str() : "null handle"; }

}  // extern "C"

// ===================================================================================
// Bias gradient without any allocation.
//
// Some users of this library cannot allocate device memory at the moment they
// need a bias gradient: a training loop that is in the middle of overlapped
// steps (cudaMalloc and cudaFree synchronise the whole device, which would
// serialise the loader stream with the compute stream), or a process that has
// already given every free byte of HBM to the arena it passed to
// alexnet_create.  For them this entry point keeps its scratch -- the per-split
// partial column sums of the two-stage reduction -- in a fixed array that is
// part of the loaded library image.  Every GPU that loads the library holds
// that array (kNoAllocSplits * kNoAllocMaxC floats = 1 MiB) until the process
// exits.
//
// The array's name is only a host-side stand-in for the symbol, not a device
// address, so host code never passes it to a kernel: once per device, with that
// device current, the address is fetched with cudaGetSymbolAddress and cached.
// That set-up happens inside the first call on each device, so make that first
// call before starting any stream capture on that device.
//
// All calls share the one array and it keeps whatever the last call left in it.
// Nothing in it has to start at zero: the first stage writes every partial the
// second stage reads, in the same call.  Two calls whose kernels overlap on the
// GPU (different streams, no dependency) race on it; order them.
namespace {
constexpr int kNoAllocSplits = 64;
constexpr int kNoAllocMaxC = 4096;
static __device__ __align__(256) float g_noalloc_partials[kNoAllocSplits * kNoAllocMaxC];

constexpr int kMaxDevices = 64;
float* g_noalloc_ptr[kMaxDevices] = {nullptr};

void put_err(char* buf, size_t len, const char* msg) {
    if (buf && len) { snprintf(buf, len, "%s", msg); }
}
}  // namespace

extern "C" int alexnet_bias_grad_noalloc(const void* dev_dy, int64_t rows, int32_t channels, float* dev_db,
                                         void* stream, char* err, size_t err_len) {
    if (!dev_dy || !dev_db) { put_err(err, err_len, "bias_grad_noalloc: NULL pointer"); return ALEXNET_ERR_ARG; }
    if (rows < 1) { put_err(err, err_len, "bias_grad_noalloc: rows must be >= 1"); return ALEXNET_ERR_ARG; }
    if (channels < 8 || channels % 8 != 0) {
        put_err(err, err_len, "bias_grad_noalloc: channels must be a positive multiple of 8");
        return ALEXNET_ERR_ARG;
    }
    if (channels > kNoAllocMaxC) {
        put_err(err, err_len, "bias_grad_noalloc: channels exceeds the fixed scratch (maximum 4096)");
        return ALEXNET_ERR_ARG;
    }
    if (((uintptr_t)dev_dy & 15) != 0) { put_err(err, err_len, "bias_grad_noalloc: dy must be 16-byte aligned"); return ALEXNET_ERR_ARG; }
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) { put_err(err, err_len, "bias_grad_noalloc: cudaGetDevice failed"); return ALEXNET_ERR_CUDA; }
    if (!g_noalloc_ptr[dev]) {
        float* p = nullptr;
        e = cudaGetSymbolAddress((void**)&p, g_noalloc_partials);
        if (e != cudaSuccess || !p) {
            put_err(err, err_len, cudaGetErrorString(e));
            return ALEXNET_ERR_CUDA;
        }
        g_noalloc_ptr[dev] = p;
    }
    float* scratch = g_noalloc_ptr[dev];
    cudaStream_t st = (cudaStream_t)stream;
    int splits = (int)std::min<int64_t>(kNoAllocSplits, std::max<int64_t>(1, rows / 256));
    dim3 grid((channels + 63) / 64, splits);
    launch_k(kn::colsum_kernel, grid, 256, 0, st, (const bf16*)dev_dy, (long long)rows, channels, scratch);
    launch_k(kn::colsum_final_kernel, (channels + 127) / 128, 128, 0, st, scratch, splits, channels, dev_db);
    e = cudaGetLastError();
    if (e != cudaSuccess) { put_err(err, err_len, cudaGetErrorString(e)); return ALEXNET_ERR_CUDA; }
    return ALEXNET_OK;
}
