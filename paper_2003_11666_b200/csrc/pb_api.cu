// C interface of the Pipelined Backpropagation engine: layer-list parsing,
// stage schedule constants, device memory layout and the per-tick launches.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>

#include "conv_gemm.cuh"
#include "conv_stage.cuh"
#include "fc_kernels.cuh"
#include "microbench.cuh"
#include "pb_engine.h"

using namespace pb;

namespace {

std::string g_create_error;

int fail(pb_handle* h, int code, const std::string& msg) {
    if (h) h->err = msg; else g_create_error = msg;
    return code;
}

#define PB_CUDA(h, call)                                                              \
    do {                                                                              \
        cudaError_t e_ = (call);                                                      \
        if (e_ != cudaSuccess)                                                        \
            return fail(h, PB_E_CUDA, std::string(#call) + ": " + cudaGetErrorString(e_)); \
    } while (0)

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int conv_out(int n, int k, int stride, int pad) { return (n + 2 * pad - k) / stride + 1; }

// ---------------------------------------------------------------- parsing
int parse_layers(pb_handle* h, const pb_layer* layers, int n_layers, const int32_t* stage_of) {
    std::vector<StageHost>& st = h->stages;
    size_t user_off = 0;
    for (int q = 0; q < n_layers; ++q) {
        const pb_layer& L = layers[q];
        const int s = stage_of[q];
        if (L.op == PB_FC || L.op == PB_CONV2D) {
            if (s != (int)st.size()) return fail(nullptr, PB_E_ARG, "a stage must start with its FC/CONV2D layer and stages must be numbered 0,1,2,...");
            StageHost x;
            x.index = s;
            x.head_op = L.op;
            x.head = L;
            x.src = L.src >= 0 ? L.src : s - 1;
            if (x.src >= s) return fail(nullptr, PB_E_ARG, "a stage may only read an earlier stage");
            x.in = x.src < 0 ? h->in_shape : st[x.src].out;
            if (L.op == PB_FC) {
                if (L.c_in <= 0 || L.c_out <= 0 || x.in.elems() != L.c_in)
                    return fail(nullptr, PB_E_SHAPE, "FC input size does not match its source at stage " + std::to_string(s));
                x.z = Shape{L.c_out, 1, 1};
                x.n_params = (size_t)L.c_in * L.c_out + L.c_out;
            } else {
                if (L.c_in <= 0 || L.c_out <= 0 || L.k <= 0 || L.stride <= 0 || L.pad < 0 || x.in.c != L.c_in)
                    return fail(nullptr, PB_E_SHAPE, "CONV2D channels do not match its source at stage " + std::to_string(s));
                x.z = Shape{L.c_out, conv_out(x.in.h, L.k, L.stride, L.pad), conv_out(x.in.w, L.k, L.stride, L.pad)};
                if (x.z.h <= 0 || x.z.w <= 0) return fail(nullptr, PB_E_SHAPE, "CONV2D output is empty");
                x.n_params = (size_t)L.c_out * L.c_in * L.k * L.k;
            }
            x.out = x.z;
            x.user_off = user_off;
            st.push_back(x);
            user_off += x.n_params;
            continue;
        }
        if (st.empty() || s != (int)st.size() - 1) return fail(nullptr, PB_E_ARG, "layer " + std::to_string(q) + " does not follow the head of its stage");
        StageHost& x = st.back();
        switch (L.op) {
            case PB_GROUPNORM:
                if (x.head_op != PB_CONV2D || L.groups <= 0 || x.z.c % L.groups) return fail(nullptr, PB_E_SHAPE, "bad GROUPNORM");
                x.gn_groups = L.groups;
                x.n_params += 2 * (size_t)x.z.c;
                user_off += 2 * (size_t)x.z.c;
                break;
            case PB_ADD_SKIP:
                if (L.src < 0 || L.src >= s) return fail(nullptr, PB_E_ARG, "ADD_SKIP needs an earlier stage");
                if (L.skip_mode < 0 || L.skip_mode > 3) return fail(nullptr, PB_E_ARG, "unknown skip mode");
                x.has_skip = true; x.skip_src = L.src; x.skip_mode = L.skip_mode & 1; x.skip_pre = (L.skip_mode & 2) != 0;
                if (x.skip_pre && (x.head_op != PB_CONV2D || st[L.src].head_op != PB_CONV2D))
                    return fail(nullptr, PB_E_ARG, "a pre-normalisation skip joins two CONV2D stages");
                if (x.skip_pre && x.gn_groups > 0)
                    return fail(nullptr, PB_E_ARG, "a pre-normalisation ADD_SKIP comes before the stage's GROUPNORM in the layer list");
                {
                    const Shape& sk = x.skip_pre ? st[L.src].z : st[L.src].out;
                    bool ok = x.skip_mode == 0 ? (sk.c == x.z.c && sk.h == x.z.h && sk.w == x.z.w)
                                               : (sk.c <= x.z.c && (sk.h + 1) / 2 == x.z.h && (sk.w + 1) / 2 == x.z.w);
                    if (!ok) return fail(nullptr, PB_E_SHAPE, "ADD_SKIP shapes do not match at stage " + std::to_string(s));
                }
                break;
            case PB_RELU: x.relu = true; break;
            case PB_MAXPOOL:
                if (L.k <= 0 || L.stride <= 0 || L.pad < 0 || 2 * L.pad > L.k) return fail(nullptr, PB_E_ARG, "bad MAXPOOL");
                x.has_pool = true; x.pool_k = L.k; x.pool_stride = L.stride; x.pool_pad = L.pad;
                x.out = Shape{x.z.c, conv_out(x.z.h, L.k, L.stride, L.pad), conv_out(x.z.w, L.k, L.stride, L.pad)};
                break;
            case PB_AVGPOOL_GLOBAL: x.avgpool = true; x.out = Shape{x.z.c, 1, 1}; break;
            case PB_SOFTMAX_CE: x.loss = true; break;
            default: return fail(nullptr, PB_E_ARG, "unknown op");
        }
    }
    if (st.empty()) return fail(nullptr, PB_E_ARG, "empty layer list");
    if (!st.back().loss || st.back().head_op != PB_FC || st.back().relu)
        return fail(nullptr, PB_E_ARG, "the last stage must be FC + SOFTMAX_CE");
    if (st.back().out.elems() != h->n_classes) return fail(nullptr, PB_E_SHAPE, "n_classes does not match the last FC");
    for (size_t s = 0; s + 1 < st.size(); ++s)
        if (st[s].loss) return fail(nullptr, PB_E_ARG, "SOFTMAX_CE before the last stage");
    h->S = (int)st.size();
    h->n_params = user_off;
    return PB_OK;
}

// SC coefficients for the delay alpha_sc * D and LWP horizon alpha_T * D of one stage
// (alpha = 1: SC_D and LWP_D; alpha = 2: the over-compensating SC_2D / LWP_2D variants).
void mitigation_constants(const pb_handle* h, StageHost& x) {
    const double m = h->momentum;
    double a = 1.0, b = 0.0;
    if (h->flags & PB_SC) {
        const double d = (double)h->sc_delay_scale * x.delay;
        a = std::pow(m, d);
        b = (1.0 - a) / (1.0 - m);            // 0 <= m < 1 is checked at pb_create
    }
    x.a = (float)a; x.b = (float)b;
    x.T = (h->flags & PB_LWP) ? h->horizon_scale * (float)x.delay : 0.f;
    if (h->update_size > 0) {
        // fill and drain: forward and backward of a sample see the same weights; plain SGDM
        x.a = 1.f; x.b = 0.f; x.T = 0.f;
    }
}

// Resets the device-side tick state (tick 0, no error) and files the training mode.
int reset_tick_state(pb_handle* h) {
    TickState ts{};
    ts.fd_n = h->update_size;
    ts.fd_cycle = h->update_size > 0 ? h->update_size + 2 * (h->S - 1) : 0;
    cudaError_t e = cudaMemcpyAsync(h->d_ts, &ts, sizeof(ts), cudaMemcpyHostToDevice, h->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);      // ts is a stack variable
    return e == cudaSuccess ? PB_OK : PB_E_CUDA;
}

// Per-stage constants: delay (Eq. F_i), SC_D coefficients, LWP horizon.
void schedule_constants(pb_handle* h) {
    const int S = h->S;
    size_t dev_off = 0;
    h->all_fc = true;
    for (StageHost& x : h->stages) {
        x.delay = 2 * (S - 1 - x.index);
        mitigation_constants(h, x);
        x.dev_off = dev_off;
        dev_off += align_up(x.n_params, 64);
        if (x.head_op != PB_FC) h->all_fc = false;
        if (x.src >= 0) h->stages[x.src].consumers_main.push_back(x.index);
        if (x.has_skip) (x.skip_pre ? h->stages[x.skip_src].consumers_res : h->stages[x.skip_src].consumers_skip).push_back(x.index);
    }
    h->dev_params = dev_off;
}

// Split FC stages into row bands, one or more per thread block, of equal bytes:
// block k owns the rows whose cumulative byte offset falls in [k*B, (k+1)*B), so
// the first wave is exact and balanced.  Networks whose weights are far larger than
// the cache also get a second wave of short blocks (see below).
void partition_fc(pb_handle* h, const std::vector<int>& fc_ids, std::vector<FcSeg>& segs,
                  std::vector<int>& cta_begin, std::vector<int>& nparts, bool fuse_last) {
    segs.clear(); cta_begin.clear();
    cta_begin.push_back(0);
    // a small last stage runs whole in one block (forward, loss, backward, update),
    // placed first so that it overlaps the long bands of the other stages
    int fused_ctas = 0;
    for (int f : fc_ids) {
        const FcStage& st = h->h_fc[f];
        if (!fuse_last || !st.is_last) continue;
        segs.push_back(FcSeg{f, 0, st.out_dim, 0, 1});
        cta_begin.push_back((int)segs.size());
        nparts[f] = 1;
        ++fused_ctas;
    }
    // The first wave (two resident blocks per SM) takes all but a small share of every
    // stage's rows; the rest goes to short blocks of kFcTailRows rows that the hardware
    // hands to whichever SM finishes its band first, which evens out the SMs' speeds.
    const double tail_frac = kFcTailFraction;
    const int tail_rows = kFcTailRows;
    std::vector<int> main_rows(h->h_fc.size(), 0);
    double total = 0, all_bytes = 0;
    for (int f : fc_ids) {
        const FcStage& st = h->h_fc[f];
        if (fuse_last && st.is_last) continue;
        all_bytes += (double)st.out_dim * st.in_dim * 8.0;
    }
    const bool with_tail = tail_frac > 0 && all_bytes >= 2.0 * h->num_sms * 1024.0 * 1024.0;
    for (int f : fc_ids) {
        const FcStage& st = h->h_fc[f];
        if (fuse_last && st.is_last) continue;
        int tail = with_tail ? (int)(st.out_dim * tail_frac / tail_rows + 0.5) * tail_rows : 0;
        if (tail > st.out_dim - 1) tail = 0;
        main_rows[f] = st.out_dim - tail;
        total += (double)main_rows[f] * st.in_dim * 8.0;
    }
    if (total <= 0) return;
    int ncta = kFcBlocksPerSM * h->num_sms - fused_ctas;       // one wave of resident blocks
    const int by_size = (int)(total / (48.0 * 1024)) + 1;      // at least 48 KB of weights per block
    if (ncta > by_size) ncta = by_size;
    if (ncta < 1) ncta = 1;
    const double budget = total / ncta;
    double acc = 0;
    int cur = 0;                        // block that owns the bytes at offset acc
    for (int f : fc_ids) {
        const FcStage& st = h->h_fc[f];
        if (fuse_last && st.is_last) continue;
        const double row_bytes = st.in_dim * 8.0;
        int r = 0, part = 0;
        while (r < main_rows[f]) {
            // rows until the next block boundary (at least one), capped by the segment limit
            const double room = (cur + 1) * budget - acc;
            int n = (int)(room / row_bytes + 0.5);
            if (n < 1) n = 1;
            if (n > kFcMaxSegRows) n = kFcMaxSegRows;
            if (n > main_rows[f] - r) n = main_rows[f] - r;
            segs.push_back(FcSeg{f, r, r + n, part++, 0});
            r += n;
            acc += n * row_bytes;
            const int owner = std::min(ncta - 1, (int)((acc + 0.5 * row_bytes) / budget));
            if (owner != cur) { cta_begin.push_back((int)segs.size()); cur = owner; }
        }
        nparts[f] = part;
    }
    if (cta_begin.back() != (int)segs.size()) cta_begin.push_back((int)segs.size());
    for (int f : fc_ids) {
        const FcStage& st = h->h_fc[f];
        if (fuse_last && st.is_last) continue;
        for (int r = main_rows[f]; r < st.out_dim; r += kFcTailRows) {
            segs.push_back(FcSeg{f, r, std::min(st.out_dim, r + kFcTailRows), nparts[f]++, 0});
            cta_begin.push_back((int)segs.size());
        }
    }
}

// FC stage descriptors and their partition into thread blocks.  w_base / v_base: where the
// flat parameter vectors start when they are the caller's memory (their alignment then
// decides whether rows can be read 16 bytes at a time); nullptr for the engine's own arena,
// whose stage blocks are 256-byte aligned.
void build_fc_tables(pb_handle* h, const float* w_base, const float* v_base) {
    std::vector<int> idsA, idsB;
    for (const StageHost& x : h->stages) {
        if (x.head_op != PB_FC || !h->owns(x.index)) continue;
        FcStage f{};
        f.in_dim = x.head.c_in; f.out_dim = x.head.c_out; f.s = x.index;
        f.relu = x.relu; f.is_last = x.loss; f.need_dx = x.src >= 0;
        bool aligned = true;
        if (w_base)
            aligned = ((reinterpret_cast<uintptr_t>(w_base + x.dev_off) | reinterpret_cast<uintptr_t>(v_base + x.dev_off)) & 15) == 0;
        f.vec = (f.in_dim % 4 == 0 && aligned) ? 4 : 1;
        f.neg_lr_T = -h->lr * x.T; f.m = h->momentum; f.neg_lr_a = -h->lr * x.a; f.neg_lr_b = -h->lr * x.b;
        idsA.push_back((int)h->h_fc.size());
        if (x.loss) idsB.push_back((int)h->h_fc.size());
        h->h_fc.push_back(f);
    }
    std::vector<int> npartsA(h->h_fc.size(), 1), npartsB(h->h_fc.size(), 1);
    // a last stage of at most 256 rows and 64 K weights is fused into the phase-0 launch
    bool fuse_last = false;
    for (int f : idsB) fuse_last = h->h_fc[f].out_dim <= kFcMaxSegRows && (long long)h->h_fc[f].out_dim * h->h_fc[f].in_dim <= 65536;
    partition_fc(h, idsA, h->h_segA, h->h_ctaA, npartsA, fuse_last);
    if (fuse_last) { h->h_segB.clear(); h->h_ctaB.assign(1, 0); }
    else partition_fc(h, idsB, h->h_segB, h->h_ctaB, npartsB, false);
    for (size_t f = 0; f < h->h_fc.size(); ++f) {
        StageHost& x = h->stages[h->h_fc[f].s];
        x.dx_nparts = (x.loss && !fuse_last) ? npartsB[f] : npartsA[f];
    }
    h->nctaA = (int)h->h_ctaA.size() - 1;
    h->nctaB = (int)h->h_ctaB.size() - 1;
}

// ---------------------------------------------------------------- convolution planning
void choose_split(int M, int N, int K, int num_sms, int& nsplit, int& kps) {
    // as for the tensor-core path: slices only bound the K loop of one tile
    (void)M; (void)N; (void)num_sms;
    nsplit = std::max(1, std::min(ceil_div(K, kSimtMaxK), 64));
    kps = ceil_div(ceil_div(K, nsplit), kBK) * kBK;
    nsplit = ceil_div(K, kps);
}

void choose_split_tc(int K, int max_k, int& nsplit, int& kps) {
    // The grouped launch already holds thousands of tiles, so K is sliced only to bound the
    // length of one tile's K loop (every slice costs a partial result that must be written
    // and read back): at most max_k elements of K per slice.
    nsplit = std::max(1, std::min(ceil_div(K, max_k), 16));
    kps = ceil_div(ceil_div(K, nsplit), kTcChunk) * kTcChunk;
    nsplit = ceil_div(K, kps);
}

int tc_bn(int N) { return N <= 64 ? 64 : 128; }

// Column tiles made of whole image rows (for operands fetched as boxes of the image): the
// largest number of rows whose pixels fit one tile and are a multiple of 16 (the MMA's N
// granularity); a small image is one tile.  Returns the rows of a box (0: no such tiling)
// and the tile width in bn.
int rect_rows(int w, int hgt, int& bn) {
    if (w > 128) return 0;
    if (w * hgt <= 64) { bn = 64; return hgt; }
    for (int r = 128 / w; r >= 1; --r)
        if ((r * w) % 16 == 0) { bn = r * w; return r; }
    return 0;
}
// 3x3 stride-1 convolutions whose channel count lets a K chunk of 64 sit inside one tap
bool rect_conv(const pb_layer& L, int channels) { return L.k == 3 && L.stride == 1 && L.pad == 1 && channels % 64 == 0; }

void plan_conv(pb_handle* h) {
    {
        // first-step blocks of the normalisation launches over the whole network
        long long chunks = 0;
        for (const StageHost& x : h->stages) {
            if (x.head_op != PB_CONV2D) continue;
            const int hw = x.z.h * x.z.w, cpg = x.head.c_out / x.gn_groups;
            chunks += (long long)x.gn_groups * (hw <= kPostChunk ? ceil_div(cpg, std::max(1, kPostChunk / hw)) : cpg * ceil_div(hw, kPostChunk));
        }
        h->post_fuse = chunks <= 8LL * h->num_sms;       // under two waves of four blocks per SM
    }
    for (StageHost& x : h->stages) {
        if (x.head_op != PB_CONV2D) continue;
        const int k2 = x.head.k * x.head.k;
        {
            const int hw = x.z.h * x.z.w, cpg = x.head.c_out / x.gn_groups;
            x.npieces = hw <= kPostChunk ? 1 : ceil_div(hw, kPostChunk);
            x.fstat_stride = hw <= kPostChunk ? ceil_div(cpg, std::max(1, kPostChunk / hw)) : cpg * x.npieces;
        }
        x.tc = (h->flags & PB_CONV_BF16) && x.src >= 0 && x.head.c_in % 8 == 0 && x.head.c_out % 8 == 0 &&
               h->stages[x.src].head_op == PB_CONV2D;
        if (x.tc) {
            const int opix = x.z.h * x.z.w, ipix = x.in.h * x.in.w;
            (void)ipix;
            choose_split_tc(x.head.c_in * k2, kTcMaxKFprop, x.split_f, x.kps_f);
            choose_split_tc(x.head.c_out * k2, kTcMaxK, x.split_d, x.kps_d);
            choose_split_tc(opix, kTcMaxK, x.split_w, x.kps_w);
            x.dx_nparts = x.split_d;
            // Large networks: a forward GEMM with one K slice writes the conv output into its ring
            // and the per-(channel, column tile) statistics itself, so the first normalisation
            // step is not run for that stage.
            {
                int bn = tc_bn(opix), rbn = 0;
                if (rect_conv(x.head, x.head.c_in) && rect_rows(x.z.w, x.z.h, rbn) > 0) bn = rbn;
                x.ntn = ceil_div(opix, bn);
            }
            x.fuse_stats = !h->post_fuse && x.split_f == 1;
            if (x.fuse_stats) x.fstat_stride = (x.head.c_out / x.gn_groups) * x.ntn;
            continue;
        }
        choose_split(x.head.c_out, x.z.h * x.z.w, x.head.c_in * k2, h->num_sms, x.split_f, x.kps_f);
        choose_split(x.head.c_in, x.in.h * x.in.w, x.head.c_out * k2, h->num_sms, x.split_d, x.kps_d);
        choose_split(x.head.c_out, x.head.c_in * k2, x.z.h * x.z.w, h->num_sms, x.split_w, x.kps_w);
        x.dx_nparts = x.split_d;
        // 3x3 / stride 1 / pad 1 on a 4x4 or 2x2 image: a weight-streaming problem, run by the fused
        // tick kernel of conv_gemv.cuh (forward, both gradients and the update in one pass over w, v)
        x.gemv = x.head.k == 3 && x.head.stride == 1 && x.head.pad == 1 && x.src >= 0 && x.in.h == x.in.w &&
                 (x.in.h == 4 || x.in.h == 2) && x.z.h == x.in.h && x.head.c_in % 32 == 0 &&
                 !(h->flags & (PB_LWP_WFORM | PB_WEIGHT_STASH)) && !x.skip_pre && x.consumers_res.empty();
        if (x.gemv) {
            x.split_f = 1; x.kps_f = ceil_div(x.head.c_in * k2, kBK) * kBK;
            x.split_w = 1; x.kps_w = ceil_div(x.z.h * x.z.w, kBK) * kBK;
            x.dx_nparts = ceil_div(x.head.c_out, kGemvRows);
        }
    }
}

// Weight stashing: ring geometry of the weight versions a stage keeps (D_s + 1 of them; a stage
// with delay 0 takes forward and backward of a sample in the same tick and keeps nothing).
void plan_stash(pb_handle* h) {
    if (!(h->flags & PB_WEIGHT_STASH)) return;
    for (StageHost& x : h->stages) {
        if (x.delay <= 0) continue;
        x.stash_slots = x.delay + 1;
        const size_t nw = x.head_op == PB_FC ? (size_t)x.head.c_in * x.head.c_out
                                             : (size_t)x.head.c_out * x.head.c_in * x.head.k * x.head.k;
        x.wstash_stride = x.head_op == PB_FC ? nw * 4 : align_up(nw * (x.tc ? 2 : 4), 16);
        if (x.head_op == PB_CONV2D) x.gstash_stride = (size_t)x.head.c_out * 4;       // slots of exactly c_out floats
    }
}

void add_tiles(std::vector<GemmTile>& tiles, int gemm, int M, int N, int nsplit, int bm = kBM, int bn = kBN) {
    for (int q = 0; q < nsplit; ++q)
        for (int m0 = 0; m0 < M; m0 += bm)
            for (int n0 = 0; n0 < N; n0 += bn) tiles.push_back(GemmTile{gemm, m0, n0, q});
}

// Tensor map (descriptor of a bulk tensor copy) of a bfloat16 matrix with up to three
// dimensions, innermost first; strides in bytes for dimensions 1.., 128-byte swizzle, zero
// fill outside the matrix.  With a null base (the sizing pass before the arena exists) an
// empty placeholder is filed so that table sizes do not change between the passes.
typedef CUresult (*TensorMapEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                      const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                      CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
TensorMapEncodeFn tensor_map_encoder() {
    static TensorMapEncodeFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess && qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<TensorMapEncodeFn>(p);
    }
    return fn;
}

int add_tensor_map(pb_handle* h, const void* base, int rank, const unsigned long long* dims, const unsigned long long* strides_bytes,
                   const unsigned* box, bool* all_ok) {
    bool this_ok = true;
    bool* ok = &this_ok;
    struct Note { bool* all; bool* one; ~Note() { if (!*one) *all = false; } } note{all_ok, &this_ok};
    CUtensorMap tm;
    std::memset(&tm, 0, sizeof(tm));
    if (base) {
        TensorMapEncodeFn enc = tensor_map_encoder();
        cuuint64_t gd[3] = {1, 1, 1}, gs[2] = {0, 0};
        cuuint32_t bx[3] = {1, 1, 1}, es[3] = {1, 1, 1};
        for (int q = 0; q < rank; ++q) { gd[q] = dims[q]; bx[q] = box[q]; }
        for (int q = 0; q + 1 < rank; ++q) gs[q] = strides_bytes[q];
        if (!enc || enc(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gd, gs, bx, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            *ok = false;
    }
    h->h_tmaps.push_back(tm);
    return *ok ? (int)h->h_tmaps.size() - 1 : -1;       // an operand without a map is gathered instead
}

// Tiles of one grouped tensor-core launch handed to persistent blocks: longest first, each
// to the block with the least work so far (cost = K chunks plus a constant for the epilogue).
void balance_tc_tiles(const pb_handle* h, const std::vector<ConvGemmTC>& gemms, std::vector<GemmTile>& tiles, std::vector<int>& begin) {
    const int nb = std::max(1, std::min((int)tiles.size(), 2 * h->num_sms));       // two resident blocks per SM
    auto cost = [&](const GemmTile& t) {
        const ConvGemmTC& g = gemms[t.gemm];
        const int kb = t.split * g.k_per_split, ke = std::min(g.K, kb + g.k_per_split);
        return ceil_div(ke - kb, kTcChunk) + 3;
    };
    std::vector<int> order(tiles.size());
    for (size_t q = 0; q < order.size(); ++q) order[q] = (int)q;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return cost(tiles[a]) > cost(tiles[b]); });
    std::vector<long long> load(nb, 0);
    std::vector<std::vector<int>> mine(nb);
    for (int q : order) {
        int best = 0;
        for (int b = 1; b < nb; ++b) if (load[b] < load[best]) best = b;
        load[best] += cost(tiles[q]);
        mine[best].push_back(q);
    }
    std::vector<GemmTile> out;
    begin.assign(1, 0);
    for (int b = 0; b < nb; ++b) {
        for (int q : mine[b]) out.push_back(tiles[q]);
        begin.push_back((int)out.size());
    }
    tiles.swap(out);
}

bool fill_conv_tables(pb_handle* h) {
    bool maps_ok = true;
    h->h_gemms.clear(); h->h_cs.clear(); h->h_pchunks.clear(); h->h_bundles.clear(); h->h_groups.clear(); h->h_ptiles[0].clear(); h->h_ptiles[1].clear(); h->h_dtiles[0].clear(); h->h_dtiles[1].clear(); h->h_upd.clear(); h->h_chunks.clear(); h->h_tc.clear(); h->h_tmaps.clear(); h->h_fchunks.clear(); h->h_stash.clear(); h->h_stashchunks.clear(); h->h_gblocks.clear(); h->h_gemv.clear(); h->h_gemvblocks.clear();
    for (auto& t : h->h_tiles) t.clear();
    for (auto& t : h->h_tctiles) t.clear();
    const int bf = (h->flags & PB_CONV_BF16) ? 1 : 0;
    for (const StageHost& x : h->stages) {
        if (x.head_op != PB_CONV2D) continue;
        const pb_layer& L = x.head;
        const int k2 = L.k * L.k, opix = x.z.h * x.z.w, ipix = x.in.h * x.in.w, nw = L.c_out * L.c_in * k2;
        const float* xin = x.src < 0 ? h->in_ring : h->stages[x.src].out_ring;
        const int xin_slots = x.src < 0 ? h->in_slots : h->stages[x.src].out_slots;
        if (x.tc) {
            const StageHost& y = h->stages[x.src];
            ConvGemmTC t{};
            t.ci = L.c_in; t.co = L.c_out; t.k = L.k; t.stride = L.stride; t.pad = L.pad;
            t.ih = x.in.h; t.iw = x.in.w; t.oh = x.z.h; t.ow = x.z.w; t.s = x.index;
            t.a_slots = 1; t.a_elems = 0;
            const bool plain = L.k == 1 && L.stride == 1 && L.pad == 0;     // the activations / dz are then plain [pixel][channel] matrices
            const __nv_bfloat16* none = nullptr;
            const bool live = h->arena != nullptr;
            // fprop: D[c_out, out pixel]
            t.mode = kFprop; t.M = L.c_out; t.N = opix; t.K = L.c_in * k2; t.bn = tc_bn(t.N);
            t.nsplit = x.split_f; t.k_per_split = x.kps_f;
            t.a = h->d_wh16 + x.dev_off; t.b = y.out16; t.b_slots = y.out_slots; t.b_elems = x.in.elems();
            t.c = x.zpart; t.c_slots = 1;
            t.fuse = x.fuse_stats ? 1 : 0; t.cpg = L.c_out / x.gn_groups; t.ntn = x.ntn; t.fstat = x.fstat;
            if (t.fuse) { t.c = x.z_ring; t.c_slots = x.out_slots; }
            {
                const unsigned long long d[2] = {(unsigned long long)t.K, (unsigned long long)t.M}, sb[1] = {(unsigned long long)t.K * 2};
                const unsigned bx[2] = {64, 128};
                t.a_tmap = add_tensor_map(h, live ? t.a : none, 2, d, sb, bx, &maps_ok);
            }
            t.b_tmap = -1; t.b_rect = 0; t.b_bytes = t.bn * 128;
            if (plain) {
                const unsigned long long d[3] = {(unsigned long long)L.c_in, (unsigned long long)ipix, (unsigned long long)y.out_slots},
                                         sb[2] = {(unsigned long long)L.c_in * 2, (unsigned long long)x.in.elems() * 2};
                const unsigned bx[3] = {64, (unsigned)t.bn, 1};
                t.b_tmap = add_tensor_map(h, live ? t.b : none, 3, d, sb, bx, &maps_ok);
            } else {
                int rbn = 0;
                const int rows = rect_conv(L, L.c_in) ? rect_rows(x.z.w, x.z.h, rbn) : 0;
                if (rows > 0) {
                    // input image [slot][y][x][c_in] (same size as the output: stride 1, pad 1)
                    const unsigned long long d[4] = {(unsigned long long)L.c_in, (unsigned long long)x.in.w, (unsigned long long)x.in.h, (unsigned long long)y.out_slots},
                                             sb[3] = {(unsigned long long)L.c_in * 2, (unsigned long long)x.in.w * L.c_in * 2, (unsigned long long)x.in.elems() * 2};
                    const unsigned bx[4] = {64, (unsigned)x.in.w, (unsigned)rows, 1};
                    const int m = add_tensor_map(h, live ? t.b : none, 4, d, sb, bx, &maps_ok);
                    t.bn = rbn;                                  // the tiling holds whether or not the map could be made
                    if (m >= 0) { t.b_tmap = m; t.b_rect = x.in.w; t.b_bytes = 128 * x.in.w * rows; }
                }
            }
            add_tiles(h->h_tctiles[0], (int)h->h_tc.size(), t.M, t.N, t.nsplit, kTcBM, t.bn);
            h->h_tc.push_back(t);
            t.fuse = 0; t.fstat = nullptr;
            // dgrad: D[c_in, in pixel]
            t.mode = kDgrad; t.M = L.c_in; t.N = ipix; t.K = L.c_out * k2; t.bn = tc_bn(t.N);
            t.nsplit = x.split_d; t.k_per_split = x.kps_d;
            t.a = h->d_w16 + x.dev_off; t.b = x.dz16; t.b_slots = 1; t.b_elems = x.z.elems();
            t.c = x.dx; t.c_slots = x.dx_slots;
            t.a_tmap = -1; t.b_tmap = -1;
            if (x.stash_slots > 0) {
                // the weights of the sample's forward, one ring slot per sample: gathered
                t.a = x.wstash16; t.a_slots = x.stash_slots; t.a_elems = (int)(x.wstash_stride / 2);
            } else if (L.c_out % 64 == 0) {
                // weights [c_out][tap][c_in]: a K chunk is 64 output channels of one tap
                const unsigned long long d[3] = {(unsigned long long)L.c_in, (unsigned long long)k2, (unsigned long long)L.c_out},
                                         sb[2] = {(unsigned long long)L.c_in * 2, (unsigned long long)k2 * L.c_in * 2};
                const unsigned bx[3] = {64, 1, 64};
                t.a_tmap = add_tensor_map(h, live ? t.a : none, 3, d, sb, bx, &maps_ok);
            }
            t.b_rect = 0; t.b_bytes = t.bn * 128;
            if (plain) {
                const unsigned long long d[2] = {(unsigned long long)L.c_out, (unsigned long long)opix}, sb[1] = {(unsigned long long)L.c_out * 2};
                const unsigned bx[2] = {64, (unsigned)t.bn};
                t.b_tmap = add_tensor_map(h, live ? t.b : none, 2, d, sb, bx, &maps_ok);
            } else {
                int rbn = 0;
                const int rows = rect_conv(L, L.c_out) ? rect_rows(x.in.w, x.in.h, rbn) : 0;
                if (rows > 0) {
                    // gradient image [y][x][c_out] (same size as the input: stride 1, pad 1)
                    const unsigned long long d[3] = {(unsigned long long)L.c_out, (unsigned long long)x.z.w, (unsigned long long)x.z.h},
                                             sb[2] = {(unsigned long long)L.c_out * 2, (unsigned long long)x.z.w * L.c_out * 2};
                    const unsigned bx[3] = {64, (unsigned)x.z.w, (unsigned)rows};
                    const int m = add_tensor_map(h, live ? t.b : none, 3, d, sb, bx, &maps_ok);
                    t.bn = rbn;
                    if (m >= 0) { t.b_tmap = m; t.b_rect = x.z.w; t.b_bytes = 128 * x.z.w * rows; }
                }
            }
            add_tiles(h->h_tctiles[1], (int)h->h_tc.size(), t.M, t.N, t.nsplit, kTcBM, t.bn);
            h->h_tc.push_back(t);
            // wgrad: D[c_out, (r, s, c_in)]
            t.a_slots = 1; t.a_elems = 0; t.b_rect = 0;
            t.mode = kWgrad; t.M = L.c_out; t.N = L.c_in * k2; t.K = opix; t.bn = tc_bn(t.N);
            t.nsplit = x.split_w; t.k_per_split = x.kps_w;
            t.a = x.dz16; t.b = y.out16; t.b_slots = y.out_slots; t.b_elems = x.in.elems();
            t.c = x.gpart; t.c_slots = 1;
            {
                const unsigned long long d[2] = {(unsigned long long)L.c_out, (unsigned long long)opix}, sb[1] = {(unsigned long long)L.c_out * 2};
                const unsigned bx[2] = {64, 64};
                t.a_tmap = add_tensor_map(h, live ? t.a : none, 2, d, sb, bx, &maps_ok);
            }
            t.b_tmap = -1;
            if (plain) {
                const unsigned long long d[3] = {(unsigned long long)L.c_in, (unsigned long long)ipix, (unsigned long long)y.out_slots},
                                         sb[2] = {(unsigned long long)L.c_in * 2, (unsigned long long)x.in.elems() * 2};
                const unsigned bx[3] = {64, 64, 1};
                t.b_tmap = add_tensor_map(h, live ? t.b : none, 3, d, sb, bx, &maps_ok);
            }
            add_tiles(h->h_tctiles[2], (int)h->h_tc.size(), t.M, t.N, t.nsplit, kTcBM, t.bn);
            h->h_tc.push_back(t);
        }
        ConvGemm g{};
        g.ci = L.c_in; g.co = L.c_out; g.k = L.k; g.stride = L.stride; g.pad = L.pad;
        g.ih = x.in.h; g.iw = x.in.w; g.oh = x.z.h; g.ow = x.z.w; g.s = x.index; g.bf16 = bf;
        // fprop
        g.mode = kFprop; g.M = L.c_out; g.N = opix; g.K = L.c_in * k2; g.nsplit = x.split_f; g.k_per_split = x.kps_f;
        g.a = h->d_wh + x.dev_off; g.b = xin; g.b_slots = xin_slots; g.b_elems = x.in.elems();
        g.c = x.zpart; g.c_slots = 1;
        g.a_slots = 1; g.a_elems = 0;
        g.tm = g.M <= 16 ? 1 : 4; g.tn = g.N <= 16 ? 1 : 4;        // small problems take small tiles
        if (!x.tc && !x.gemv) add_tiles(h->h_tiles[0], (int)h->h_gemms.size(), g.M, g.N, g.nsplit, 16 * g.tm, 16 * g.tn);
        h->h_gemms.push_back(g);
        // dgrad (not for the first stage: nobody needs the gradient of the input)
        if (x.src >= 0) {
            g.mode = kDgrad; g.M = L.c_in; g.N = ipix; g.K = L.c_out * k2; g.nsplit = x.split_d; g.k_per_split = x.kps_d;
            g.a = h->d_w + x.dev_off; g.b = x.dz; g.b_slots = 1; g.b_elems = x.z.elems();
            if (!x.tc && x.stash_slots > 0) { g.a = x.wstash; g.a_slots = x.stash_slots; g.a_elems = (int)(x.wstash_stride / 4); }   // the forward's weights
            g.c = x.dx; g.c_slots = x.dx_slots;
            g.tm = g.M <= 16 ? 1 : 4; g.tn = g.N <= 16 ? 1 : 4;
            if (!x.tc && !x.gemv) add_tiles(h->h_tiles[1], (int)h->h_gemms.size(), g.M, g.N, g.nsplit, 16 * g.tm, 16 * g.tn);
            h->h_gemms.push_back(g);
        }
        // wgrad
        g.mode = kWgrad; g.M = L.c_out; g.N = L.c_in * k2; g.K = opix; g.nsplit = x.split_w; g.k_per_split = x.kps_w;
        g.a = x.dz; g.b = xin; g.b_slots = xin_slots; g.b_elems = x.in.elems();
        g.a_slots = 1; g.a_elems = 0;
        g.c = x.gpart; g.c_slots = 1;
        g.tm = g.M <= 16 ? 1 : 4; g.tn = g.N <= 16 ? 1 : 4;
        if (!x.tc && !x.gemv) add_tiles(h->h_tiles[2], (int)h->h_gemms.size(), g.M, g.N, g.nsplit, 16 * g.tm, 16 * g.tn);
        h->h_gemms.push_back(g);

        ConvStage c{};
        c.s = x.index; c.co = L.c_out; c.oh = x.z.h; c.ow = x.z.w;
        c.groups = x.gn_groups; c.cpg = L.c_out / x.gn_groups;
        c.relu = x.relu; c.avgpool = x.avgpool;
        c.need_out32 = x.consumers_skip.empty() ? 0 : 1;
        for (int q : x.consumers_main) if (!h->stages[q].tc) c.need_out32 = 1;
        c.vec4 = ((x.z.h * x.z.w) % 4 == 0) ? 1 : 0;
        c.pool_k = x.has_pool ? x.pool_k : 0; c.pool_stride = x.pool_stride; c.pool_pad = x.pool_pad;
        c.out_h = x.out.h; c.out_w = x.out.w;
        c.zpart = x.zpart; c.z_nsplit = x.split_f;
        c.z_ring = x.z_ring; c.stat_ring = x.stat_ring; c.code_ring = x.code_ring; c.arg_ring = x.arg_ring;
        c.out_ring = x.out_ring; c.slots = x.out_slots;
        c.out16 = x.out16; c.dz16 = x.tc ? x.dz16 : nullptr;     // only tensor-core stages read the bfloat16 gradient
        c.wh = h->d_wh + x.dev_off; c.w = h->d_w + x.dev_off; c.g = h->d_g + x.dev_off; c.nw = nw;
        if (x.has_skip) {
            const StageHost& y = h->stages[x.skip_src];
            c.skip_ring = x.skip_pre ? y.z_ring : y.out_ring; c.skip_slots = y.out_slots; c.skip_mode = x.skip_mode;
            c.skip_pre = x.skip_pre ? 1 : 0;
            const Shape& ys = x.skip_pre ? y.z : y.out;
            c.skip_c = ys.c; c.skip_h = ys.h; c.skip_w = ys.w;
            c.dskip = x.dskip; c.dskip_slots = x.dskip_slots;
        }
        c.n_dsrc = 0;
        for (int q : x.consumers_main) { const StageHost& y = h->stages[q]; c.dsrc[c.n_dsrc++] = DeltaSrc{y.dx, y.dx_slots, y.dx_nparts}; }
        for (int q : x.consumers_skip) { const StageHost& y = h->stages[q]; c.dsrc[c.n_dsrc++] = DeltaSrc{y.dskip, y.dskip_slots, 1}; }
        c.n_rsrc = 0;
        for (int q : x.consumers_res) { const StageHost& y = h->stages[q]; c.rsrc[c.n_rsrc++] = DeltaSrc{y.dskip, y.dskip_slots, 1}; }
        c.dz = x.dz;
        c.gstash = x.gstash; c.gstash_slots = x.stash_slots;
        c.fstat = x.fstat; c.fstat_stride = x.fstat_stride; c.fused = x.fuse_stats ? 1 : 0; c.bsum = x.bsum; c.npieces = x.npieces; c.gsum = x.gsum;
        {
            // Chunks of the first step: whole channels while they fit, else pieces of one channel.
            // Tiles of the second step: (a multiple of 8 channels) x pixels, up to kPostChunk
            // elements; the forward of a pooling stage works on the group chunks instead.
            // In small networks (the first step is under two waves of blocks, so launch latency
            // dominates) stages are FUSED: their groups are bundled (whole groups, at least 8
            // channels where bfloat16 copies are written, whose 16-byte runs hold 8 channels of a
            // pixel), tiles stay inside a bundle and the block that closes a bundle finishes it.
            // Elsewhere, and for a stage with a bundle of more than kPostFuseTiles tiles, the
            // three-launch form stays (closing blocks working through several tiles each would
            // be the tail of a launch that is already many waves long).
            const int hw = x.z.h * x.z.w, cpg = c.cpg, stage_idx = (int)h->h_cs.size();
            const bool need16 = x.tc && L.c_out % 8 == 0 && 8 % cpg == 0;
            const int gpb = need16 && cpg < 8 ? 8 / cpg : 1;           // groups per bundle
            // Large networks: a tensor-core stage whose bundles fit in shared memory is normalised by
            // one block per bundle, forward and backward (conv_group.cuh), and leaves the lists below.
            // (a bundle spans whole 8-channel units: groups of 1, 2, 4 channels are bundled, groups of 8, 16, ... stand alone)
            const bool units_ok = x.tc && L.c_out % 8 == 0 && (cpg < 8 ? 8 % cpg == 0 : cpg % 8 == 0);
            // small groups are bundled further (a block pays its chain of memory latencies whatever its size)
            int rgpb = gpb;
            const long long target = x.fuse_stats ? kGroupTargetElems : kGroupSliceTarget;
            while (x.gn_groups % (2 * rgpb) == 0 && 2 * rgpb * cpg <= kGroupMaxChannels && 2LL * rgpb * cpg * hw <= target) rgpb *= 2;
            // (a stage whose forward GEMM left K slices keeps the float32 sum of a bundle in shared memory)
            const bool resident = x.tc && !h->post_fuse && units_ok && !x.has_pool && !x.avgpool && x.gn_groups % rgpb == 0 &&
                                  rgpb * cpg <= kGroupMaxChannels && (long long)rgpb * cpg * hw <= (x.fuse_stats ? kGroupMaxElems : kGroupSliceElems);
            if (resident) {
                for (int g0 = 0; g0 < x.gn_groups; g0 += rgpb) h->h_gblocks.push_back(GroupBlock{stage_idx, g0, rgpb});
                // each of the kGroupSplit blocks of a bundle holds a quarter of the pixels (rounded up to whole units of 4)
                const size_t np = (size_t)(ceil_div(ceil_div(hw, 4), kGroupSplit) + 1) * 4;
                const size_t t16_bytes = align_up((size_t)rgpb * cpg * (np + 2) * 2, 16);
                h->group_smem_fwd = std::max(h->group_smem_fwd, t16_bytes + (x.fuse_stats ? 0 : (size_t)rgpb * cpg * hw * 4));
                h->group_smem_bwd = std::max(h->group_smem_bwd, (size_t)2 * rgpb * cpg * (np + 5) * 4);      // dn and zhat (pitch np + 4, made odd for short rows)
            }
            if (!resident) {
            const bool pooled = x.has_pool || x.avgpool;
            auto tile_shape = [&](int channels, int& CT, int& PT) {
                CT = std::min(kPostTileChannels, std::max(8, (kPostChunk / std::min(hw, kPostTilePixels)) / 8 * 8));
                CT = std::min(CT, channels);
                PT = CT * hw <= kPostChunk ? hw : std::min(hw, std::max(4, (kPostChunk / CT) / 4 * 4));
            };
            auto chunks_of_group = [&](int gq) {
                int n = 0;
                if (hw <= kPostChunk) n = ceil_div(cpg, std::max(1, kPostChunk / hw));
                else n = cpg * ceil_div(hw, kPostChunk);
                return n;
            };
            bool fuse = h->post_fuse;
            if (fuse) {
                int CT, PT;
                tile_shape(gpb * cpg, CT, PT);
                const int btiles = ceil_div(gpb * cpg, CT) * ceil_div(hw, PT);
                const int ftiles = pooled ? gpb * chunks_of_group(0) : btiles;
                fuse = btiles <= kPostFuseTiles && ftiles <= kPostFuseTiles;
            }
            for (int g0 = 0; g0 < x.gn_groups; g0 += gpb) {
                PostBundle bd{};
                bd.stage = stage_idx; bd.grp0 = g0; bd.ngrp = std::min(gpb, x.gn_groups - g0);
                const int bundle_idx = fuse ? (int)h->h_bundles.size() : -1;
                bd.ftile0 = (int)h->h_ptiles[0].size(); bd.btile0 = (int)h->h_ptiles[1].size();
                for (int gq = g0; gq < g0 + bd.ngrp; ++gq) {
                    if (!fuse) h->h_groups.push_back(GroupRef{stage_idx, gq});
                    const size_t first = h->h_pchunks.size();
                    if (hw <= kPostChunk) {
                        const int per = std::max(1, kPostChunk / hw);
                        for (int cl = 0; cl < cpg; cl += per)
                            h->h_pchunks.push_back(PostChunk{stage_idx, gq, cl, std::min(per, cpg - cl), 0, hw, 0, 0, bundle_idx});
                    } else {
                        for (int cl = 0; cl < cpg; ++cl)
                            for (int p0 = 0; p0 < hw; p0 += kPostChunk)
                                h->h_pchunks.push_back(PostChunk{stage_idx, gq, cl, 1, p0, std::min(kPostChunk, hw - p0), 0, 0, bundle_idx});
                    }
                    const int nidx = (int)(h->h_pchunks.size() - first);
                    for (int q = 0; q < nidx; ++q) { h->h_pchunks[first + q].idx = q; h->h_pchunks[first + q].nidx = nidx; }
                    bd.nchunks += nidx;
                    if (pooled)
                        for (int q = 0; q < nidx; ++q) {
                            PostChunk tch = h->h_pchunks[first + q];
                            tch.cl0 += gq * cpg; tch.grp = -1;
                            (fuse ? h->h_ptiles[0] : h->h_dtiles[0]).push_back(tch);
                        }
                }
                if (!fuse) continue;
                const int c_lo = g0 * cpg, c_hi = (g0 + bd.ngrp) * cpg;
                int CT, PT;
                tile_shape(c_hi - c_lo, CT, PT);
                for (int c0 = c_lo; c0 < c_hi; c0 += CT)
                    for (int p0 = 0; p0 < hw; p0 += PT) {
                        const PostChunk tch{stage_idx, -1, c0, std::min(CT, c_hi - c0), p0, std::min(PT, hw - p0), 0, 0, bundle_idx};
                        if (!pooled) h->h_ptiles[0].push_back(tch);
                        h->h_ptiles[1].push_back(tch);
                    }
                bd.nftiles = (int)h->h_ptiles[0].size() - bd.ftile0;
                bd.nbtiles = (int)h->h_ptiles[1].size() - bd.btile0;
                h->h_bundles.push_back(bd);
            }
            if (!fuse) {
                // stage-wide tiles for the launches of their own
                int CT, PT;
                tile_shape(L.c_out, CT, PT);
                for (int c0 = 0; c0 < L.c_out; c0 += CT)
                    for (int p0 = 0; p0 < hw; p0 += PT) {
                        const PostChunk tch{stage_idx, -1, c0, std::min(CT, (int)L.c_out - c0), p0, std::min(PT, hw - p0), 0, 0, -1};
                        if (!pooled) h->h_dtiles[0].push_back(tch);
                        h->h_dtiles[1].push_back(tch);
                    }
            }
            }   // !resident
        }
        h->h_cs.push_back(c);

        UpdRange r{};
        r.s = x.index; r.neg_lr_T = -h->lr * x.T; r.m = h->momentum; r.neg_lr_a = -h->lr * x.a; r.neg_lr_b = -h->lr * x.b;
        r.T_w = x.T; r.wform = (h->flags & PB_LWP_WFORM) ? 1 : 0;
        r.w = h->d_w + x.dev_off; r.v = h->d_v + x.dev_off; r.wh = h->d_wh + x.dev_off;
        r.g = x.gpart; r.nparts = x.split_w; r.part_stride = nw; r.n = nw;
        if (x.tc) { r.w16 = h->d_w16 + x.dev_off; r.wh16 = h->d_wh16 + x.dev_off; }
        if (x.gemv) {
            // its conv weights are updated inside the fused kernel (and predicted on the fly)
            ConvGemvStage gs{};
            gs.w = h->d_w + x.dev_off; gs.v = h->d_v + x.dev_off;
            gs.ci = L.c_in; gs.co = L.c_out; gs.hw = x.in.h; gs.s = x.index;
            gs.xin = xin; gs.xin_slots = xin_slots;
            gs.dz = x.dz; gs.z = x.zpart;
            gs.dx = x.dx; gs.dx_slots = x.dx_slots; gs.dx_nparts = x.dx_nparts;
            gs.neg_lr_T = -h->lr * x.T; gs.m = h->momentum; gs.neg_lr_a = -h->lr * x.a; gs.neg_lr_b = -h->lr * x.b;
            for (int r0 = 0, part = 0; r0 < L.c_out; r0 += kGemvRows, ++part) h->h_gemvblocks.push_back(GemvBlock{(int)h->h_gemv.size(), r0, part});
            h->h_gemv.push_back(gs);
            const int P = x.in.h * x.in.w;
            h->gemv_smem = std::max(h->gemv_smem, sizeof(float) * ((size_t)2 * L.c_in * (P + 1) + (size_t)(1 + kGemvWarps) * kGemvRows * P + (size_t)kGemvWarps * 576 + 4));
        } else {
        for (int st = 0; st < r.n; st += kUpdChunk) h->h_chunks.push_back(UpdChunk{(int)h->h_upd.size(), st});
        h->h_upd.push_back(r);
        }
        r.w += nw; r.v += nw; r.wh += nw; r.w16 = nullptr; r.wh16 = nullptr;
        r.g = h->d_g + x.dev_off + nw; r.nparts = 1; r.part_stride = 0; r.n = 2 * L.c_out;
        for (int st = 0; st < r.n; st += kUpdChunk) h->h_chunks.push_back(UpdChunk{(int)h->h_upd.size(), st});
        h->h_upd.push_back(r);
        if (x.stash_slots > 0) {
            auto add = [&](const void* src, void* ring, int esize, long long n, size_t stride) {
                for (long long b0 = 0; b0 < n * esize; b0 += kStashChunkBytes) h->h_stashchunks.push_back(StashChunk{(int)h->h_stash.size(), b0});
                h->h_stash.push_back(StashRange{src, ring, x.stash_slots, x.index, esize, n, (long long)stride});
            };
            if (x.tc) add(h->d_wh16 + x.dev_off, x.wstash16, 2, nw, x.wstash_stride);
            else add(h->d_wh + x.dev_off, x.wstash, 4, nw, x.wstash_stride);
            add(h->d_wh + x.dev_off + nw, x.gstash, 4, L.c_out, x.gstash_stride);
        }
    }
    // Data-gradient and weight-gradient GEMMs both start from dz and write different buffers: one
    // launch takes the tiles of both (one start-up and one tail instead of two, and the long K loops
    // of the data gradients balance against the many short tiles of the weight gradients).
    h->h_tctiles[1].insert(h->h_tctiles[1].end(), h->h_tctiles[2].begin(), h->h_tctiles[2].end());
    h->h_tctiles[2].clear();
    for (int q = 0; q < 3; ++q) balance_tc_tiles(h, h->h_tc, h->h_tctiles[q], h->h_tcbegin[q]);
    // the first forward normalisation step skips the stages whose GEMM epilogue has done it
    {
        std::vector<char> fused;
        for (const StageHost& x : h->stages) if (x.head_op == PB_CONV2D) fused.push_back(x.fuse_stats ? 1 : 0);
        for (const PostChunk& ch : h->h_pchunks) if (!fused[ch.stage]) h->h_fchunks.push_back(ch);
    }
    return maps_ok;
}

int validate_conv(pb_handle* h) {
    for (const StageHost& x : h->stages) {
        if (x.head_op != PB_CONV2D) continue;
        if (x.gn_groups <= 0) return fail(nullptr, PB_E_UNSUPPORTED, "a CONV2D stage needs a GROUPNORM layer");
        if (x.head.c_out / x.gn_groups > kMaxGroupChannels) return fail(nullptr, PB_E_UNSUPPORTED, "more than 64 channels per normalisation group");
        if (x.has_pool && x.avgpool) return fail(nullptr, PB_E_UNSUPPORTED, "max-pool and average pool in one stage");
        if (x.avgpool && x.z.h * x.z.w > kPostChunk) return fail(nullptr, PB_E_UNSUPPORTED, "global average pool over more than 2048 pixels");
        if ((int)(x.consumers_main.size() + x.consumers_skip.size()) > kMaxDeltaSrc) return fail(nullptr, PB_E_UNSUPPORTED, "too many consumers of one stage");
        if ((int)x.consumers_res.size() > kMaxDeltaSrc) return fail(nullptr, PB_E_UNSUPPORTED, "too many stages add one stage's pre-normalisation sum");
        if ((x.skip_pre || !x.consumers_res.empty()) && (h->flags & PB_CONV_BF16))
            return fail(nullptr, PB_E_UNSUPPORTED, "pre-normalisation skips run on the float32 convolution path only");
    }
    for (const StageHost& x : h->stages)
        if (x.head_op == PB_FC && (x.has_skip || x.has_pool || x.avgpool || x.gn_groups)) return fail(nullptr, PB_E_UNSUPPORTED, "FC stages take only RELU or SOFTMAX_CE");
    return PB_OK;
}

__global__ void ingest_kernel(const TickState* __restrict__ ts, int par, const float* __restrict__ xs,
                              const int* __restrict__ labels, int label_value, float* __restrict__ in_ring,
                              int in_slots, int elems, int* __restrict__ label_ring, int S, long long t_base) {
    const long long t = ts->cnt[par];
    const float* src = xs + (size_t)(t - t_base) * elems;
    float* dst = in_ring + (size_t)(t % in_slots) * elems;
    for (int k = blockIdx.x * blockDim.x + threadIdx.x; k < elems; k += gridDim.x * blockDim.x) dst[k] = src[k];
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        label_ring[t % S] = labels ? labels[t - t_base] : label_value;
    }
}

// ---------------------------------------------------------------- memory layout
struct Carver {
    char* base; size_t off = 0;
    template <class T> T* take(size_t n) {
        T* p = reinterpret_cast<T*>(base + off);
        off += align_up(n * sizeof(T), 256);
        return p;
    }
};

size_t layout(pb_handle* h, char* base, size_t* zero_from) {
    Carver c{base};
    h->d_ts = c.take<TickState>(1);
    h->d_fc = c.take<FcStage>(h->h_fc.size() + 1);
    h->d_segA = c.take<FcSeg>(h->h_segA.size() + 1);
    h->d_segB = c.take<FcSeg>(h->h_segB.size() + 1);
    h->d_ctaA = c.take<int>(h->h_ctaA.size() + 1);
    h->d_ctaB = c.take<int>(h->h_ctaB.size() + 1);
    h->d_gemms = c.take<ConvGemm>(h->h_gemms.size() + 1);
    for (int q = 0; q < 3; ++q) h->d_tiles[q] = c.take<GemmTile>(h->h_tiles[q].size() + 1);
    h->d_cs = c.take<ConvStage>(h->h_cs.size() + 1);
    h->d_pchunks = c.take<PostChunk>(h->h_pchunks.size() + 1);
    h->d_bundles = c.take<PostBundle>(h->h_bundles.size() + 1);
    h->d_groups = c.take<GroupRef>(h->h_groups.size() + 1);
    for (int q = 0; q < 2; ++q) h->d_ptiles[q] = c.take<PostChunk>(h->h_ptiles[q].size() + 1);
    for (int q = 0; q < 2; ++q) h->d_dtiles[q] = c.take<PostChunk>(h->h_dtiles[q].size() + 1);
    h->d_upd = c.take<UpdRange>(h->h_upd.size() + 1);
    h->d_chunks = c.take<UpdChunk>(h->h_chunks.size() + 1);
    h->d_gblocks = c.take<GroupBlock>(h->h_gblocks.size() + 1);
    h->d_gemv = c.take<ConvGemvStage>(h->h_gemv.size() + 1);
    h->d_gemvblocks = c.take<GemvBlock>(h->h_gemvblocks.size() + 1);
    h->d_stash = c.take<StashRange>(h->h_stash.size() + 1);
    h->d_stashchunks = c.take<StashChunk>(h->h_stashchunks.size() + 1);
    h->d_tc = c.take<ConvGemmTC>(h->h_tc.size() + 1);
    for (int q = 0; q < 3; ++q) h->d_tctiles[q] = c.take<GemmTile>(h->h_tctiles[q].size() + 1);
    for (int q = 0; q < 3; ++q) h->d_tcbegin[q] = c.take<int>(h->h_tcbegin[q].size() + 1);
    h->d_tmaps = c.take<CUtensorMap>(h->h_tmaps.size() + 1);
    h->d_fchunks = c.take<PostChunk>(h->h_fchunks.size() + 1);
    h->d_w = c.take<float>(h->dev_params);
    if (!h->all_fc || (h->flags & PB_LWP_WFORM)) h->d_wh = c.take<float>(h->dev_params);
    *zero_from = c.off;
    h->d_stamps = c.take<long long>(2);
    h->d_v = c.take<float>(h->dev_params);
    for (int q = 0; q < 2; ++q) h->d_bcnt[q] = c.take<int>(h->h_bundles.size() + 1);   // bundle counters (zero between launches)
    if (!h->all_fc) h->d_g = c.take<float>(h->dev_params);
    if (h->flags & PB_CONV_BF16) {
        h->d_w16 = c.take<__nv_bfloat16>(h->dev_params);
        h->d_wh16 = c.take<__nv_bfloat16>(h->dev_params);
    }
    h->in_slots = 2 * (h->S - 1) + 1;
    h->in_ring = c.take<float>((size_t)h->in_slots * h->in_shape.elems());
    h->label_ring = c.take<int>(h->S);
    h->d_loss1 = c.take<float>(1);
    for (StageHost& x : h->stages) {
        x.out_slots = x.delay + 1;
        x.out_ring = c.take<float>((size_t)x.out_slots * x.out.elems());
        if (x.src >= 0) {
            x.dx_slots = x.index - x.src + 1;
            x.dx = c.take<float>((size_t)x.dx_slots * x.dx_nparts * x.in.elems());
        }
        if (x.has_skip) {
            x.dskip_slots = x.index - x.skip_src + 1;
            x.dskip = c.take<float>((size_t)x.dskip_slots * (x.skip_pre ? h->stages[x.skip_src].z.elems() : h->stages[x.skip_src].out.elems()));
        }
        if (x.head_op == PB_CONV2D) {
            const size_t ze = x.z.elems(), nw = (size_t)x.head.c_out * x.head.c_in * x.head.k * x.head.k;
            x.z_ring = c.take<float>((size_t)x.out_slots * ze);
            x.stat_ring = c.take<float>((size_t)x.out_slots * 2 * x.gn_groups);
            x.code_ring = c.take<unsigned char>((size_t)x.out_slots * ze);
            x.arg_ring = x.has_pool ? c.take<unsigned char>((size_t)x.out_slots * x.out.elems()) : nullptr;
            x.zpart = c.take<float>((size_t)x.split_f * ze);
            x.dz = c.take<float>(ze);
            x.gpart = c.take<float>((size_t)x.split_w * nw);
            x.fstat = c.take<float>((size_t)x.gn_groups * x.fstat_stride * 3);
            x.bsum = c.take<float>((size_t)x.head.c_out * x.npieces * 2);
            x.gsum = c.take<float>((size_t)x.gn_groups * 2);
            if (h->flags & PB_CONV_BF16) {
                x.out16 = c.take<__nv_bfloat16>((size_t)x.out_slots * x.out.elems());
                x.dz16 = c.take<__nv_bfloat16>(ze);
            }
        }
        if (x.stash_slots > 0) {
            if (x.tc) x.wstash16 = reinterpret_cast<__nv_bfloat16*>(c.take<char>(x.wstash_stride * x.stash_slots));
            else x.wstash = reinterpret_cast<float*>(c.take<char>(x.wstash_stride * x.stash_slots));
            if (x.head_op == PB_CONV2D) x.gstash = reinterpret_cast<float*>(c.take<char>(x.gstash_stride * x.stash_slots));
        }
    }
    return c.off;
}

void fill_fc_tables(pb_handle* h) {
    for (FcStage& f : h->h_fc) {
        const StageHost& x = h->stages[f.s];
        f.w = h->d_w + x.dev_off;
        f.v = h->d_v + x.dev_off;
        f.neg_lr_T = -h->lr * x.T; f.m = h->momentum; f.neg_lr_a = -h->lr * x.a; f.neg_lr_b = -h->lr * x.b;
        f.T_w = x.T;
        f.wh = ((h->flags & PB_LWP_WFORM) && h->d_wh) ? h->d_wh + x.dev_off : nullptr;
        f.stash = x.wstash; f.stash_slots = x.stash_slots;      // slots of exactly out*in floats
        if (x.src < 0) { f.xin = h->in_ring; f.xin_slots = h->in_slots; }
        else { f.xin = h->stages[x.src].out_ring; f.xin_slots = h->stages[x.src].out_slots; }
        f.out = x.out_ring; f.out_slots = x.out_slots;
        f.dx = x.dx; f.dx_slots = x.dx_slots; f.dx_nparts = x.dx_nparts;
        f.n_dsrc = 0;
        for (int c : x.consumers_main) {
            const StageHost& y = h->stages[c];
            f.dsrc[f.n_dsrc++] = DeltaSrc{y.dx, y.dx_slots, y.dx_nparts};
        }
        for (int c : x.consumers_skip) {
            const StageHost& y = h->stages[c];
            f.dsrc[f.n_dsrc++] = DeltaSrc{y.dskip, y.dskip_slots, 1};
        }
    }
}

// ---------------------------------------------------------------- profiling helpers
void prof_begin(pb_handle* h, int cls, cudaStream_t st = nullptr) {
    if (!st) st = h->stream;
    if (!h->profile) return;
    if (h->ev_used + 2 > h->ev_pool.size()) {
        for (int k = 0; k < 2; ++k) { cudaEvent_t e; cudaEventCreate(&e); h->ev_pool.push_back(e); }
    }
    h->ev_class.push_back(cls);
    cudaEventRecord(h->ev_pool[h->ev_used], st);
}
void prof_end(pb_handle* h, cudaStream_t st = nullptr) {
    if (!st) st = h->stream;
    if (!h->profile) return;
    cudaEventRecord(h->ev_pool[h->ev_used + 1], st);
    h->ev_used += 2;
}
void prof_collect(pb_handle* h) {
    if (!h->profile) return;
    cudaStreamSynchronize(h->stream);
    for (size_t k = 0; k < h->ev_class.size(); ++k) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, h->ev_pool[2 * k], h->ev_pool[2 * k + 1]) == cudaSuccess) {
            h->prof[h->ev_class[k]].ms += ms;
            h->prof[h->ev_class[k]].launches += 1;
        }
    }
    h->ev_class.clear();
    h->ev_used = 0;
}

// ---------------------------------------------------------------- stage split
// Contiguous ranges of stages for n ranks that minimise the largest per-rank sum of `cost`
// (dynamic programme over the cut positions; every rank gets at least one stage).
bool split_ranges(const std::vector<double>& cost, int n, std::vector<int>& lo, std::vector<int>& hi) {
    const int S = (int)cost.size();
    if (n < 1 || n > S) return false;
    std::vector<double> pre(S + 1, 0.0);
    for (int s = 0; s < S; ++s) pre[s + 1] = pre[s] + cost[s];
    const double inf = 1e300;
    std::vector<std::vector<double>> best(n + 1, std::vector<double>(S + 1, inf));
    std::vector<std::vector<int>> cut(n + 1, std::vector<int>(S + 1, 0));
    best[0][0] = 0.0;
    for (int r = 1; r <= n; ++r)
        for (int e = r; e <= S; ++e)
            for (int b = r - 1; b < e; ++b) {
                const double v = std::max(best[r - 1][b], pre[e] - pre[b]);
                if (v < best[r][e]) { best[r][e] = v; cut[r][e] = b; }
            }
    lo.assign(n, 0); hi.assign(n, 0);
    int e = S;
    for (int r = n; r >= 1; --r) { hi[r - 1] = e; lo[r - 1] = cut[r][e]; e = cut[r][e]; }
    return true;
}

int plan_split(pb_handle* h, int n_ranks, std::vector<int>& lo, std::vector<int>& hi) {
    for (const StageHost& x : h->stages) {
        if (x.head_op != PB_FC || x.has_skip) return fail(nullptr, PB_E_UNSUPPORTED, "the stage split supports fully connected networks only");
        if (x.src != x.index - 1) return fail(nullptr, PB_E_UNSUPPORTED, "the stage split needs every stage to read the stage before it");
    }
    std::vector<double> cost;
    for (const StageHost& x : h->stages) cost.push_back(16.0 * (double)x.n_params);      // one read and one write of w and v per tick
    if (!split_ranges(cost, n_ranks, lo, hi)) return fail(nullptr, PB_E_ARG, "need 1 <= n_ranks <= number of stages");
    return PB_OK;
}

// ---------------------------------------------------------------- ticks
int run_ticks(pb_handle* h, const float* dev_xs, const int32_t* dev_labels, int label_value,
              int n_ticks, float* dev_losses) {
    const int elems = h->in_shape.elems();
    const int ingest_blocks = std::min(ceil_div(elems, 1024), 2 * h->num_sms);
    const long long t_base = h->tick;
    h->last_launches = 0;
    // Fully connected pipelines read the current sample straight from the caller's buffer,
    // 16 bytes at a time when the sample length is a multiple of 4: the buffer must then be
    // 16-byte aligned (checked here, on the host, before anything is launched).
    const bool split = h->split_n > 1;
    if (split && !h->split_connected) return fail(h, PB_E_ARG, "a split handle must be connected to its neighbours first (pb_split_connect)");
    if (h->all_fc && h->owns(0) && !h->h_fc.empty() && h->h_fc[0].vec == 4 && (reinterpret_cast<uintptr_t>(dev_xs) & 15) != 0)
        return fail(h, PB_E_ARG, "the sample buffer must be 16-byte aligned when the sample length is a multiple of 4");
    if (h->profile) for (auto& p : h->prof) p = ProfileClass{};
    const bool fused_last = h->nctaB == 0;      // the last stage rides in the phase-0 launch
    const int npc = (int)h->h_pchunks.size();
    const int ngb = (int)h->h_gblocks.size();             // bundles normalised by one block each (large networks)
    const int nfc = (int)h->h_fchunks.size();            // forward first-step blocks (stages whose GEMM has not done that step)
    const int post_grid = std::max(1, npc);              // one block per chunk
    const int ngr = (int)h->h_groups.size();             // groups of the stages that keep the three-launch form
    for (int k = 0; k < n_ticks; ++k) {
        const int par = (int)((t_base + k) & 1);
        if (h->all_fc) {
            // one launch: ingest + every stage (two when the last stage needs its own)
            const float* xs_mine = h->owns(0) ? dev_xs : nullptr;       // only the rank with stage 0 ingests the sample
            if (split) {
                // wait for the neighbours' previous tick; ranks without stage 0 file the label here,
                // ranks without the last stage report NaN as this tick's loss
                split_wait_kernel<<<1, 32, 0, h->stream>>>(h->links, h->d_ts, par, h->owns(0) ? nullptr : h->label_ring, h->S,
                                                           dev_labels, label_value, t_base,
                                                           (!h->owns(h->S - 1) && dev_losses) ? dev_losses : nullptr);
                h->last_launches += 1;
            }
            prof_begin(h, 0);
            {
                // consecutive ticks overlap their launch latency (see the kernel's first lines)
                cudaLaunchConfig_t cfg = {};
                cfg.gridDim = dim3(h->nctaA); cfg.blockDim = dim3(kFcThreads); cfg.dynamicSmemBytes = 0; cfg.stream = h->stream;
                cudaLaunchAttribute attr[1];
                attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
                attr[0].val.programmaticStreamSerializationAllowed = 1;
                cfg.attrs = attr; cfg.numAttrs = (fused_last && !h->profile && !split) ? 1 : 0;
                cudaLaunchKernelEx(&cfg, fc_tick_kernel, (const FcStage*)h->d_fc, (const FcSeg*)h->d_segA, (const int*)h->d_ctaA, h->d_ts,
                                   h->S, 0, par, fused_last ? 1 : 0, h->label_ring, dev_losses, t_base,
                                   xs_mine, dev_labels, label_value, h->in_ring, h->in_slots, elems);
            }
            prof_end(h);
            h->last_launches += 1;
            if (!fused_last) {
                prof_begin(h, 1);
                fc_tick_kernel<<<h->nctaB, kFcThreads, 0, h->stream>>>(h->d_fc, h->d_segB, h->d_ctaB, h->d_ts, h->S, 1, par, 1,
                                                                      h->label_ring, dev_losses, t_base,
                                                                      nullptr, nullptr, 0, nullptr, 0, 0);
                prof_end(h);
                h->last_launches += 1;
            }
            if (split) {
                split_handoff_kernel<<<1, 256, 0, h->stream>>>(h->links, h->d_ts, par, h->S);
                h->last_launches += 1;
            }
        } else {
            // The new sample goes into the ring slot that the previous tick's weight gradient of
            // stage 0 was the last to read, and its label into the slot the previous tick's loss
            // read: the copy waits for those two only (side stream, after the FC stage of the
            // previous tick) and so runs beside the previous tick's update.  The caller's buffers
            // are ordered behind the caller's stream once per call.
            cudaStream_t fs = h->side ? h->side : h->stream;
            if (kEarlyIngest && h->side && h->ev_inputs) {
                if (k == 0) {
                    cudaEventRecord(h->ev_inputs, h->stream);
                    cudaStreamWaitEvent(fs, h->ev_inputs, 0);
                }
                cudaStreamWaitEvent(fs, h->ev_wjoin, 0);         // as recorded by the previous tick
                ingest_kernel<<<ingest_blocks, 256, 0, fs>>>(h->d_ts, par, dev_xs, dev_labels, label_value, h->in_ring,
                                                             h->in_slots, elems, h->label_ring, h->S, t_base);
                cudaEventRecord(h->ev_ingest, fs);
                cudaStreamWaitEvent(h->stream, h->ev_ingest, 0);
            } else {
                ingest_kernel<<<ingest_blocks, 256, 0, h->stream>>>(h->d_ts, par, dev_xs, dev_labels, label_value, h->in_ring,
                                                                    h->in_slots, elems, h->label_ring, h->S, t_base);
            }
            // The FC stages of this tick depend only on what earlier ticks left in the rings
            // (and on the label just ingested): they run on a side stream beside the conv chain.
            cudaEventRecord(h->ev_fork, h->stream);
            cudaStreamWaitEvent(fs, h->ev_fork, 0);
            prof_begin(h, 0, fs);
            fc_tick_kernel<<<h->nctaA, kFcThreads, 0, fs>>>(h->d_fc, h->d_segA, h->d_ctaA, h->d_ts, h->S, 0, par,
                                                           fused_last ? 1 : 0, h->label_ring, dev_losses, t_base,
                                                           nullptr, nullptr, 0, nullptr, 0, 0);
            prof_end(h, fs);
            if (!fused_last) {
                prof_begin(h, 1, fs);
                fc_tick_kernel<<<h->nctaB, kFcThreads, 0, fs>>>(h->d_fc, h->d_segB, h->d_ctaB, h->d_ts, h->S, 1, par, 1,
                                                               h->label_ring, dev_losses, t_base,
                                                               nullptr, nullptr, 0, nullptr, 0, 0);
                prof_end(h, fs);
            }
            // forward chain: convolutions -> normalise/activate/pool
            if (!h->h_tiles[0].empty()) {
                prof_begin(h, 3);
                conv_gemm_kernel<<<(int)h->h_tiles[0].size(), kGemmThreads, 0, h->stream>>>(h->d_gemms, h->d_tiles[0], h->d_ts, h->S, par);
                prof_end(h);
            }
            if (!h->h_tctiles[0].empty()) {
                prof_begin(h, 4);
                conv_tc_kernel<<<(int)h->h_tcbegin[0].size() - 1, kTcThreads, kTcSmemBytes, h->stream>>>(
                    h->d_tc, TcLaunch{h->d_tctiles[0], h->d_tcbegin[0]}, h->d_tmaps, h->d_ts, h->S, par);
                prof_end(h);
            }
            // Backward chain: through pool/ReLU/GroupNorm -> data and weight gradients.  It reads
            // what earlier ticks stored (other ring slots than the forward chain writes) and the
            // current weights, so it runs on its own stream beside the forward chain; only the
            // update, which overwrites the predicted weights the forward reads, waits for both.
            cudaStream_t bs = h->bwd ? h->bwd : h->stream;
            // In the three-launch form the first backward step touches no parameter and no
            // gradient table: it reads rings that were filled at least two ticks ago, the
            // hand-offs that the previous tick's backward chain (this stream), its FC stage (side
            // stream) and nobody else wrote, and it overwrites the scratch that the previous
            // tick's weight gradients (third stream) were the last to read.  So it need not wait
            // for the previous tick's update: it starts as soon as those two streams are done and
            // runs beside the update and the ingest; the merge that follows waits for the fork.
            const bool early_bwd = !h->post_fuse && kEarlyBackward && h->bwd && h->aux && h->side;
            if (early_bwd) {
                cudaStreamWaitEvent(bs, h->ev_join, 0);      // as recorded by the previous tick
                cudaStreamWaitEvent(bs, h->ev_wjoin, 0);
            } else {
                cudaStreamWaitEvent(bs, h->ev_fork, 0);
            }
            prof_begin(h, 6, bs);
            conv_bwd_post_kernel<<<post_grid, kPostThreads, 0, bs>>>(h->d_cs, h->d_pchunks, npc, h->d_bundles, h->d_ptiles[1], h->d_bcnt[1], h->d_ts, h->S, par);
            if (early_bwd) cudaStreamWaitEvent(bs, h->ev_fork, 0);
            if (ngr > 0)
                conv_group_merge_kernel<<<ceil_div(ngr, 8), 256, 0, bs>>>(h->d_cs, h->d_groups, ngr, h->d_ts, h->S, par, 1);
            if (!h->h_dtiles[1].empty())
                conv_bwd_dz_kernel<<<(int)h->h_dtiles[1].size(), kPostThreads, 0, bs>>>(h->d_cs, h->d_dtiles[1], (int)h->h_dtiles[1].size(), h->d_ts, h->S, par);
            if (ngb > 0)
                conv_group_bwd_kernel<<<ngb * kGroupSplit, kGroupThreads, h->group_smem_bwd, bs>>>(h->d_cs, h->d_gblocks, ngb, h->d_ts, h->S, par);     // clusters of kGroupSplit
            prof_end(h, bs);
            const int ngv_ = (int)h->h_gemvblocks.size();
            if (ngv_ > 0) {
                // 3x3 stages on tiny images: forward, both gradients and the update in one pass over (w, v)
                prof_begin(h, 3, bs);
                conv_gemv_kernel<<<ngv_, kGemvThreads, h->gemv_smem, bs>>>(h->d_gemv, h->d_gemvblocks, h->d_ts, h->S, par);
                prof_end(h, bs);
                cudaEventRecord(h->ev_gemv, bs);
                h->last_launches += 1;
            }
            // forward normalisation (issued here, after the kernel above has been queued: it waits for it)
            const int ngv = (int)h->h_gemvblocks.size();
            prof_begin(h, 5);
            // (stages run by the fused tiny-image kernel get their conv output from it: that kernel sits
            //  in the backward chain, behind the gradient it also needs, so the forward normalisation waits for it)
            if (ngv > 0) cudaStreamWaitEvent(h->stream, h->ev_gemv, 0);
            if (nfc > 0)
                conv_fwd_post_kernel<<<nfc, kPostThreads, 0, h->stream>>>(h->d_cs, h->d_fchunks, nfc, h->d_bundles, h->d_ptiles[0], h->d_bcnt[0], h->d_ts, h->S, par);
            if (ngr > 0)
                conv_group_merge_kernel<<<ceil_div(ngr, 8), 256, 0, h->stream>>>(h->d_cs, h->d_groups, ngr, h->d_ts, h->S, par, 0);
            if (!h->h_dtiles[0].empty())
                conv_apply_fwd_kernel<<<(int)h->h_dtiles[0].size(), kPostThreads, 0, h->stream>>>(h->d_cs, h->d_dtiles[0], (int)h->h_dtiles[0].size(), h->d_ts, h->S, par);
            if (ngb > 0)
                conv_group_fwd_kernel<<<ngb * kGroupSplit, kGroupThreads, h->group_smem_fwd, h->stream>>>(h->d_cs, h->d_gblocks, ngb, h->d_ts, h->S, par);
            prof_end(h);
            // data gradients (dgrad) and weight gradients (wgrad) both start from dz and write
            // different buffers: wgrad goes to a stream of its own
            cudaStream_t ws = h->aux ? h->aux : bs;
            cudaEventRecord(h->ev_dz, bs);
            cudaStreamWaitEvent(ws, h->ev_dz, 0);
            for (int q = 1; q < 3; ++q) {
                cudaStream_t qs = q == 1 ? bs : ws;
                if (!h->h_tiles[q].empty()) {
                    prof_begin(h, 3, qs);
                    conv_gemm_kernel<<<(int)h->h_tiles[q].size(), kGemmThreads, 0, qs>>>(h->d_gemms, h->d_tiles[q], h->d_ts, h->S, par);
                    prof_end(h, qs);
                }
                if (!h->h_tctiles[q].empty()) {
                    prof_begin(h, q == 1 ? 8 : 7, qs);
                    conv_tc_kernel<<<(int)h->h_tcbegin[q].size() - 1, kTcThreads, kTcSmemBytes, qs>>>(
                        h->d_tc, TcLaunch{h->d_tctiles[q], h->d_tcbegin[q]}, h->d_tmaps, h->d_ts, h->S, par);
                    prof_end(h, qs);
                }
            }
            cudaEventRecord(h->ev_wjoin, ws);
            cudaStreamWaitEvent(h->stream, h->ev_wjoin, 0);
            cudaEventRecord(h->ev_bjoin, bs);
            cudaStreamWaitEvent(h->stream, h->ev_bjoin, 0);
            if (!h->h_stashchunks.empty()) {
                // weight stashing: this tick's forward weights go to their sample's slot before the update replaces them
                stash_copy_kernel<<<(int)h->h_stashchunks.size(), 256, 0, h->stream>>>(h->d_stash, h->d_stashchunks, h->d_ts, par);
                h->last_launches += 1;
            }
            prof_begin(h, 2);
            update_kernel<<<(int)h->h_chunks.size(), 256, 0, h->stream>>>(h->d_upd, h->d_chunks, h->d_ts, h->S, par);
            prof_end(h);
            // the conv chain waits for the FC stages before the tick ends
            cudaEventRecord(h->ev_join, fs);
            cudaStreamWaitEvent(h->stream, h->ev_join, 0);
            h->last_launches += 4 + (nfc > 0 ? 1 : 0) + (fused_last ? 0 : 1);      // ingest, the normalisation kernels, update, FC
            h->last_launches += (ngb > 0 ? 2 : 0);
            h->last_launches += (h->h_dtiles[0].empty() ? 0 : 1) + (h->h_dtiles[1].empty() ? 0 : 1) + (ngr > 0 ? 2 : 0);
            for (int q = 0; q < 3; ++q) h->last_launches += (h->h_tiles[q].empty() ? 0 : 1) + (h->h_tctiles[q].empty() ? 0 : 1);
        }
    }
    PB_CUDA(h, cudaGetLastError());
    h->tick += n_ticks;
    prof_collect(h);
    return PB_OK;
}

int check_device_error(pb_handle* h) {
    TickState ts;
    PB_CUDA(h, cudaMemcpyAsync(&ts, h->d_ts, sizeof(ts), cudaMemcpyDeviceToHost, h->stream));
    PB_CUDA(h, cudaStreamSynchronize(h->stream));
    if (ts.error != kErrNone)
        return fail(h, PB_E_DEVICE, "device index check failed: code " + std::to_string(ts.error) + " info " + std::to_string(ts.error_info));
    return PB_OK;
}

}  // namespace

// ---------------------------------------------------------------- C interface
namespace {
int create_engine(const pb_layer* layers, int n_layers, const int32_t* stage_of_layer, int in_c, int in_h,
                  int in_w, int n_classes, float lr, float momentum, unsigned flags, void* stream,
                  int rank, int n_ranks, pb_handle** out) {
    if (out) *out = nullptr;
    if (!layers || !stage_of_layer || !out || n_layers <= 0 || in_c <= 0 || in_h <= 0 || in_w <= 0 || n_classes <= 0)
        return fail(nullptr, PB_E_ARG, "pb_create: NULL pointer or non-positive size");
    if (!(momentum >= 0.f && momentum < 1.f) || !(lr >= 0.f)) return fail(nullptr, PB_E_ARG, "pb_create: need 0 <= momentum < 1 and lr >= 0");
    if (flags & ~(unsigned)(PB_SC | PB_LWP | PB_LWP_WFORM | PB_CONV_BF16 | PB_WEIGHT_STASH)) return fail(nullptr, PB_E_ARG, "pb_create: unknown flag");
    if ((flags & PB_LWP_WFORM) && !(flags & PB_LWP)) return fail(nullptr, PB_E_ARG, "pb_create: PB_LWP_WFORM needs PB_LWP");
    for (int q = 1; q < n_layers; ++q)
        if (stage_of_layer[q] < stage_of_layer[q - 1]) return fail(nullptr, PB_E_ARG, "pb_create: stage indices must not decrease");
    pb_handle* h = new (std::nothrow) pb_handle();
    if (!h) return fail(nullptr, PB_E_ALLOC, "pb_create: out of host memory");
    h->stream = (cudaStream_t)stream;
    h->flags = flags; h->lr = lr; h->momentum = momentum; h->n_classes = n_classes;
    h->in_shape = Shape{in_c, in_h, in_w};
    int rc = parse_layers(h, layers, n_layers, stage_of_layer);
    if (rc != PB_OK) { delete h; return rc; }
    schedule_constants(h);
    h->s_lo = 0; h->s_hi = h->S;
    if (n_ranks > 1) {
        std::vector<int> lo, hi;
        rc = plan_split(h, n_ranks, lo, hi);
        if (rc != PB_OK) { delete h; return rc; }
        h->split_rank = rank; h->split_n = n_ranks; h->s_lo = lo[rank]; h->s_hi = hi[rank];
    }
    cudaError_t e = cudaGetDevice(&h->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->num_sms, cudaDevAttrMultiProcessorCount, h->device);
    if (e != cudaSuccess) { std::string m = cudaGetErrorString(e); delete h; return fail(nullptr, PB_E_CUDA, "pb_create: no CUDA device: " + m); }

    build_fc_tables(h, nullptr, nullptr);

    rc = validate_conv(h);
    if (rc != PB_OK) { delete h; return rc; }
    plan_conv(h);
    plan_stash(h);
    fill_conv_tables(h);     // sizes only; pointers are filled in after the layout
    size_t zero_from = 0;
    h->arena_bytes = layout(h, nullptr, &zero_from);
    if (flags & PB_WEIGHT_STASH) {
        size_t stash_bytes = 0;
        for (const StageHost& x : h->stages) stash_bytes += (x.wstash_stride + x.gstash_stride) * (size_t)x.stash_slots;
        if (stash_bytes > (16ull << 30)) {
            std::string m = "pb_create: weight stashing would keep " + std::to_string(stash_bytes) + " bytes of weight versions (limit 16 GiB)";
            delete h; return fail(nullptr, PB_E_UNSUPPORTED, m);
        }
    }
    e = cudaMalloc((void**)&h->arena, h->arena_bytes);
    if (e != cudaSuccess) {
        std::string m = "pb_create: cudaMalloc of " + std::to_string(h->arena_bytes) + " bytes failed: " + cudaGetErrorString(e);
        delete h; return fail(nullptr, PB_E_ALLOC, m);
    }
    layout(h, h->arena, &zero_from);
    h->zero_from = zero_from;
    fill_fc_tables(h);
    fill_conv_tables(h);
    e = cudaMemsetAsync(h->arena, 0, h->arena_bytes, h->stream);
    auto up = [&](void* d, const void* s, size_t n) { if (e == cudaSuccess && n) e = cudaMemcpyAsync(d, s, n, cudaMemcpyHostToDevice, h->stream); };
    up(h->d_fc, h->h_fc.data(), h->h_fc.size() * sizeof(FcStage));
    up(h->d_segA, h->h_segA.data(), h->h_segA.size() * sizeof(FcSeg));
    up(h->d_segB, h->h_segB.data(), h->h_segB.size() * sizeof(FcSeg));
    up(h->d_ctaA, h->h_ctaA.data(), h->h_ctaA.size() * sizeof(int));
    up(h->d_ctaB, h->h_ctaB.data(), h->h_ctaB.size() * sizeof(int));
    up(h->d_gemms, h->h_gemms.data(), h->h_gemms.size() * sizeof(ConvGemm));
    for (int q = 0; q < 3; ++q) up(h->d_tiles[q], h->h_tiles[q].data(), h->h_tiles[q].size() * sizeof(GemmTile));
    up(h->d_cs, h->h_cs.data(), h->h_cs.size() * sizeof(ConvStage));
    up(h->d_pchunks, h->h_pchunks.data(), h->h_pchunks.size() * sizeof(PostChunk));
    up(h->d_bundles, h->h_bundles.data(), h->h_bundles.size() * sizeof(PostBundle));
    up(h->d_groups, h->h_groups.data(), h->h_groups.size() * sizeof(GroupRef));
    for (int q = 0; q < 2; ++q) up(h->d_ptiles[q], h->h_ptiles[q].data(), h->h_ptiles[q].size() * sizeof(PostChunk));
    for (int q = 0; q < 2; ++q) up(h->d_dtiles[q], h->h_dtiles[q].data(), h->h_dtiles[q].size() * sizeof(PostChunk));
    up(h->d_upd, h->h_upd.data(), h->h_upd.size() * sizeof(UpdRange));
    up(h->d_chunks, h->h_chunks.data(), h->h_chunks.size() * sizeof(UpdChunk));
    up(h->d_gblocks, h->h_gblocks.data(), h->h_gblocks.size() * sizeof(GroupBlock));
    up(h->d_gemv, h->h_gemv.data(), h->h_gemv.size() * sizeof(ConvGemvStage));
    up(h->d_gemvblocks, h->h_gemvblocks.data(), h->h_gemvblocks.size() * sizeof(GemvBlock));
    up(h->d_stash, h->h_stash.data(), h->h_stash.size() * sizeof(StashRange));
    up(h->d_stashchunks, h->h_stashchunks.data(), h->h_stashchunks.size() * sizeof(StashChunk));
    up(h->d_tc, h->h_tc.data(), h->h_tc.size() * sizeof(ConvGemmTC));
    for (int q = 0; q < 3; ++q) up(h->d_tctiles[q], h->h_tctiles[q].data(), h->h_tctiles[q].size() * sizeof(GemmTile));
    for (int q = 0; q < 3; ++q) up(h->d_tcbegin[q], h->h_tcbegin[q].data(), h->h_tcbegin[q].size() * sizeof(int));
    up(h->d_tmaps, h->h_tmaps.data(), h->h_tmaps.size() * sizeof(CUtensorMap));
    up(h->d_fchunks, h->h_fchunks.data(), h->h_fchunks.size() * sizeof(PostChunk));
    if (e == cudaSuccess && !h->all_fc) {
        // The backward chain (normalisation backward -> data gradients) is the longest of the
        // tick's chains and the update waits for it.  In small networks, whose launches do not
        // fill the GPU, giving its streams the higher priority shortens the tick (measured:
        // VGG-11 200 -> 186 us, ResNet-20 69 -> 66 us); in ResNet-50 it starves the forward
        // convolutions (597 -> 613 us), so large networks keep equal priorities.
        int prio_least = 0, prio_greatest = 0;
        cudaDeviceGetStreamPriorityRange(&prio_least, &prio_greatest);
        auto prio = [&](int level) { return (level && h->post_fuse) ? prio_greatest : prio_least; };
        e = cudaStreamCreateWithPriority(&h->side, cudaStreamNonBlocking, prio(kPrioSide));
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_inputs, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_ingest, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&h->bwd, cudaStreamNonBlocking, prio(kPrioBwd));
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_bjoin, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&h->aux, cudaStreamNonBlocking, prio(kPrioAux));
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_dz, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_wjoin, cudaEventDisableTiming);
    }
    if (e == cudaSuccess && !h->h_tc.empty())
        e = cudaFuncSetAttribute(conv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmemBytes);
    if (e == cudaSuccess && !h->h_gemvblocks.empty()) {
        e = cudaFuncSetAttribute(conv_gemv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)h->gemv_smem);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_gemv, cudaEventDisableTiming);
    }
    if (e == cudaSuccess && !h->h_gblocks.empty()) {
        e = cudaFuncSetAttribute(conv_group_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)h->group_smem_fwd);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(conv_group_bwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)h->group_smem_bwd);
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
    if (e != cudaSuccess) {
        std::string m = std::string("pb_create: upload failed: ") + cudaGetErrorString(e);
        pb_destroy(h);          // frees the arena and whatever streams and events exist by now
        return fail(nullptr, PB_E_CUDA, m);
    }
    *out = h;
    return PB_OK;
}
}  // namespace

extern "C" {

int pb_create(const pb_layer* layers, int n_layers, const int32_t* stage_of_layer, int in_c, int in_h,
              int in_w, int n_classes, float lr, float momentum, unsigned flags, void* stream,
              pb_handle** out) {
    return create_engine(layers, n_layers, stage_of_layer, in_c, in_h, in_w, n_classes, lr, momentum, flags, stream, 0, 1, out);
}

int pb_create_split(const pb_layer* layers, int n_layers, const int32_t* stage_of_layer, int in_c, int in_h,
                    int in_w, int n_classes, float lr, float momentum, unsigned flags, void* stream,
                    int rank, int n_ranks, pb_handle** out) {
    if (out) *out = nullptr;
    if (n_ranks < 1 || rank < 0 || rank >= n_ranks) return fail(nullptr, PB_E_ARG, "pb_create_split: need 0 <= rank < n_ranks");
    return create_engine(layers, n_layers, stage_of_layer, in_c, in_h, in_w, n_classes, lr, momentum, flags, stream, rank, n_ranks, out);
}

int pb_split_plan(const pb_layer* layers, int n_layers, const int32_t* stage_of_layer, int in_c, int in_h, int in_w,
                  int n_classes, int n_ranks, int32_t* lo, int32_t* hi) {
    if (!layers || !stage_of_layer || !lo || !hi || n_layers <= 0 || in_c <= 0 || in_h <= 0 || in_w <= 0 || n_classes <= 0)
        return fail(nullptr, PB_E_ARG, "pb_split_plan: NULL pointer or non-positive size");
    for (int q = 1; q < n_layers; ++q)
        if (stage_of_layer[q] < stage_of_layer[q - 1]) return fail(nullptr, PB_E_ARG, "pb_split_plan: stage indices must not decrease");
    pb_handle hs;                       // host bookkeeping only
    hs.n_classes = n_classes; hs.in_shape = Shape{in_c, in_h, in_w};
    int rc = parse_layers(&hs, layers, n_layers, stage_of_layer);
    if (rc != PB_OK) return rc;
    std::vector<int> l, u;
    rc = plan_split(&hs, n_ranks, l, u);
    if (rc != PB_OK) return rc;
    for (int r = 0; r < n_ranks; ++r) { lo[r] = l[r]; hi[r] = u[r]; }
    return PB_OK;
}

int pb_split_range(const pb_handle* h, int32_t* lo, int32_t* hi) {
    if (!h || !lo || !hi) return PB_E_ARG;
    *lo = h->split_n > 1 ? h->s_lo : 0; *hi = h->split_n > 1 ? h->s_hi : h->S;
    return PB_OK;
}

int pb_split_ports(pb_handle* h, pb_split_port* mine) {
    if (!h || !mine) return PB_E_ARG;
    if (h->split_n <= 1) return fail(h, PB_E_ARG, "pb_split_ports: not a split handle");
    // the neighbours' boundary tensors land in this handle's own copies of the neighbour stages' rings
    mine->act = h->s_lo > 0 ? (void*)h->stages[h->s_lo - 1].out_ring : nullptr;
    mine->act_stamp = h->s_lo > 0 ? (void*)(h->d_stamps + 0) : nullptr;
    mine->grad = h->s_hi < h->S ? (void*)h->stages[h->s_hi].dx : nullptr;
    mine->grad_stamp = h->s_hi < h->S ? (void*)(h->d_stamps + 1) : nullptr;
    return PB_OK;
}

int pb_split_connect(pb_handle* h, const pb_split_port* prev_rank, const pb_split_port* next_rank) {
    if (!h) return PB_E_ARG;
    if (h->split_n <= 1) return fail(h, PB_E_ARG, "pb_split_connect: not a split handle");
    if ((h->s_lo > 0) != (prev_rank != nullptr) || (h->s_hi < h->S) != (next_rank != nullptr))
        return fail(h, PB_E_ARG, "pb_split_connect: a port is needed for exactly the neighbours that exist");
    SplitLinks L{};
    if (prev_rank) {
        if (!prev_rank->grad || !prev_rank->grad_stamp) return fail(h, PB_E_ARG, "pb_split_connect: the previous rank's gradient port is empty");
        const StageHost& x = h->stages[h->s_lo];                 // own first stage: its input gradient goes back
        L.act_stamp = h->d_stamps + 0;
        L.grad_src = x.dx; L.grad_slots = x.dx_slots; L.grad_nparts = x.dx_nparts; L.grad_dim = x.in.elems(); L.grad_stage = x.index;
        L.grad_dst = static_cast<float*>(prev_rank->grad); L.grad_dst_stamp = static_cast<long long*>(prev_rank->grad_stamp);
    }
    if (next_rank) {
        if (!next_rank->act || !next_rank->act_stamp) return fail(h, PB_E_ARG, "pb_split_connect: the next rank's activation port is empty");
        const StageHost& x = h->stages[h->s_hi - 1];             // own last stage: its output goes forward
        L.grad_stamp = h->d_stamps + 1;
        L.act_src = x.out_ring; L.act_slots = x.out_slots; L.act_dim = x.out.elems(); L.act_stage = x.index;
        L.act_dst = static_cast<float*>(next_rank->act); L.act_dst_stamp = static_cast<long long*>(next_rank->act_stamp);
    }
    h->links = L;
    h->split_connected = true;
    return PB_OK;
}

int pb_set_weights(pb_handle* h, const float* host_w, size_t n) {
    if (!h) return PB_E_ARG;
    if (!host_w || n != h->n_params) return fail(h, PB_E_ARG, "pb_set_weights: need pb_num_params() floats");
    PB_CUDA(h, cudaMemsetAsync(h->arena + h->zero_from, 0, h->arena_bytes - h->zero_from, h->stream));
    if (reset_tick_state(h) != PB_OK) return fail(h, PB_E_CUDA, "pb_set_weights: could not reset the tick state");
    std::vector<float> tmp;
    for (const StageHost& x : h->stages) {
        const float* src = host_w + x.user_off;
        if (x.tc) {
            // tensor-core stages keep conv weights as [c_out][r][s][c_in]
            tmp.assign(src, src + x.n_params);
            const int CI = x.head.c_in, k2 = x.head.k * x.head.k;
            for (int co = 0; co < x.head.c_out; ++co)
                for (int ci = 0; ci < CI; ++ci)
                    for (int rs = 0; rs < k2; ++rs) tmp[((size_t)co * k2 + rs) * CI + ci] = src[((size_t)co * CI + ci) * k2 + rs];
            src = tmp.data();
        }
        PB_CUDA(h, cudaMemcpyAsync(h->d_w + x.dev_off, src, x.n_params * sizeof(float), cudaMemcpyHostToDevice, h->stream));
        if (x.tc) PB_CUDA(h, cudaStreamSynchronize(h->stream));     // tmp is reused
    }
    // zero velocity: the predicted weights start equal to the weights
    if (h->d_wh) PB_CUDA(h, cudaMemcpyAsync(h->d_wh, h->d_w, h->dev_params * sizeof(float), cudaMemcpyDeviceToDevice, h->stream));
    if (h->d_w16 && !h->h_chunks.empty())
        cast_weights_kernel<<<(int)h->h_chunks.size(), 256, 0, h->stream>>>(h->d_upd, h->d_chunks);
    PB_CUDA(h, cudaStreamSynchronize(h->stream));
    h->tick = 0;
    return PB_OK;
}

int pb_set_mitigation(pb_handle* h, float sc_delay_scale, float horizon_scale) {
    if (!h) return PB_E_ARG;
    if (!(sc_delay_scale >= 0.f) || !(horizon_scale >= 0.f)) return fail(h, PB_E_ARG, "pb_set_mitigation: scales must be >= 0");
    if ((h->flags & PB_LWP_WFORM) && h->tick != 0)
        return fail(h, PB_E_UNSUPPORTED, "pb_set_mitigation: with PB_LWP_WFORM the scales can only be set before the first tick "
                                         "(the stored prediction cannot be re-made without the previous weights)");
    h->sc_delay_scale = sc_delay_scale;
    h->horizon_scale = horizon_scale;
    for (StageHost& x : h->stages) mitigation_constants(h, x);
    fill_fc_tables(h);
    fill_conv_tables(h);
    // the tables take effect for launches issued after this call (stream order)
    PB_CUDA(h, cudaStreamSynchronize(h->stream));
    if (!h->h_fc.empty())
        PB_CUDA(h, cudaMemcpyAsync(h->d_fc, h->h_fc.data(), h->h_fc.size() * sizeof(FcStage), cudaMemcpyHostToDevice, h->stream));
    if (!h->h_gemv.empty())
        PB_CUDA(h, cudaMemcpyAsync(h->d_gemv, h->h_gemv.data(), h->h_gemv.size() * sizeof(ConvGemvStage), cudaMemcpyHostToDevice, h->stream));
    if (!h->h_upd.empty()) {
        PB_CUDA(h, cudaMemcpyAsync(h->d_upd, h->h_upd.data(), h->h_upd.size() * sizeof(UpdRange), cudaMemcpyHostToDevice, h->stream));
        // Conv stages read STORED predicted weights, written by their last update with the old
        // horizon: re-make them from (w, v) so that the next forward of every stage, FC or
        // conv, uses the new T.  (Velocity form only; see the check above.)
        if (!(h->flags & PB_LWP_WFORM) && !h->h_chunks.empty()) {
            repredict_kernel<<<(int)h->h_chunks.size(), 256, 0, h->stream>>>(h->d_upd, h->d_chunks);
            PB_CUDA(h, cudaGetLastError());
        }
    }
    PB_CUDA(h, cudaStreamSynchronize(h->stream));
    return PB_OK;
}

int pb_set_update_size(pb_handle* h, int n_samples) {
    if (!h) return PB_E_ARG;
    if (n_samples < 0) return fail(h, PB_E_ARG, "pb_set_update_size: negative update size");
    if (h->tick != 0) return fail(h, PB_E_ARG, "pb_set_update_size: call it before the first tick (after pb_set_weights)");
    h->update_size = n_samples;
    for (StageHost& x : h->stages) mitigation_constants(h, x);
    fill_fc_tables(h);
    fill_conv_tables(h);
    PB_CUDA(h, cudaStreamSynchronize(h->stream));
    if (!h->h_fc.empty())
        PB_CUDA(h, cudaMemcpyAsync(h->d_fc, h->h_fc.data(), h->h_fc.size() * sizeof(FcStage), cudaMemcpyHostToDevice, h->stream));
    if (!h->h_gemv.empty())
        PB_CUDA(h, cudaMemcpyAsync(h->d_gemv, h->h_gemv.data(), h->h_gemv.size() * sizeof(ConvGemvStage), cudaMemcpyHostToDevice, h->stream));
    if (!h->h_upd.empty())
        PB_CUDA(h, cudaMemcpyAsync(h->d_upd, h->h_upd.data(), h->h_upd.size() * sizeof(UpdRange), cudaMemcpyHostToDevice, h->stream));
    if (reset_tick_state(h) != PB_OK) return fail(h, PB_E_CUDA, "pb_set_update_size: could not write the tick state");
    return PB_OK;
}

int pb_tick(pb_handle* h, const float* dev_x, int label, float* host_loss) {
    if (!h) return PB_E_ARG;
    if ((!dev_x && h->owns(0)) || label < 0 || label >= h->n_classes) return fail(h, PB_E_ARG, "pb_tick: NULL input or label out of range");
    int rc = run_ticks(h, dev_x, nullptr, label, 1, h->d_loss1);
    if (rc != PB_OK) return rc;
    if (host_loss) {
        PB_CUDA(h, cudaMemcpyAsync(host_loss, h->d_loss1, sizeof(float), cudaMemcpyDeviceToHost, h->stream));
        return check_device_error(h);
    }
    return PB_OK;
}

int pb_run(pb_handle* h, const float* dev_xs, const int32_t* dev_labels, int n_ticks, float* dev_losses) {
    if (!h) return PB_E_ARG;
    if (n_ticks == 0) return PB_OK;         // nothing to do; the pointers are not looked at
    if ((!dev_xs && h->owns(0)) || !dev_labels || n_ticks < 0) return fail(h, PB_E_ARG, "pb_run: NULL pointer or negative count");
    return run_ticks(h, dev_xs, dev_labels, 0, n_ticks, dev_losses);
}

int pb_run_host(pb_handle* h, const float* host_xs, const int32_t* host_labels, int n_ticks, float* host_losses) {
    if (!h) return PB_E_ARG;
    if (n_ticks == 0) return PB_OK;
    if (!host_xs || !host_labels || n_ticks < 0) return fail(h, PB_E_ARG, "pb_run_host: NULL pointer or negative count");
    const size_t xb = (size_t)n_ticks * h->in_shape.elems() * sizeof(float);
    const size_t lb = (size_t)n_ticks * sizeof(int32_t), fb = (size_t)n_ticks * sizeof(float);
    const size_t o1 = align_up(xb, 256), o2 = o1 + align_up(lb, 256), need = o2 + align_up(fb, 256);
    cudaError_t e = cudaSuccess;
    if (need > h->staging_bytes) {   // grow-only staging buffer, kept for later calls
        PB_CUDA(h, cudaStreamSynchronize(h->stream));
        if (h->staging) cudaFree(h->staging);
        h->staging = nullptr; h->staging_bytes = 0;
        e = cudaMalloc((void**)&h->staging, need);
        if (e != cudaSuccess) return fail(h, PB_E_ALLOC, std::string("pb_run_host: staging allocation failed: ") + cudaGetErrorString(e));
        h->staging_bytes = need;
    }
    char* stage = h->staging;
    int rc = PB_OK;
    e = cudaMemcpyAsync(stage, host_xs, xb, cudaMemcpyHostToDevice, h->stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(stage + o1, host_labels, lb, cudaMemcpyHostToDevice, h->stream);
    if (e == cudaSuccess) rc = run_ticks(h, (const float*)stage, (const int32_t*)(stage + o1), 0, n_ticks, (float*)(stage + o2));
    if (e == cudaSuccess && rc == PB_OK && host_losses) e = cudaMemcpyAsync(host_losses, stage + o2, fb, cudaMemcpyDeviceToHost, h->stream);
    cudaError_t e2 = cudaStreamSynchronize(h->stream);
    if (rc != PB_OK) return rc;
    if (e != cudaSuccess || e2 != cudaSuccess) return fail(h, PB_E_CUDA, std::string("pb_run_host: ") + cudaGetErrorString(e != cudaSuccess ? e : e2));
    return check_device_error(h);
}

static int get_params(pb_handle* h, const float* dev, float* host, size_t n, const char* who) {
    if (!h) return PB_E_ARG;
    if (!host || n != h->n_params) return fail(h, PB_E_ARG, std::string(who) + ": need pb_num_params() floats");
    for (const StageHost& x : h->stages) {
        if (!h->owns(x.index)) { std::memset(host + x.user_off, 0, x.n_params * sizeof(float)); continue; }   // that stage lives on another rank
        PB_CUDA(h, cudaMemcpyAsync(host + x.user_off, dev + x.dev_off, x.n_params * sizeof(float), cudaMemcpyDeviceToHost, h->stream));
    }
    int rc = check_device_error(h);
    if (rc != PB_OK) return rc;
    std::vector<float> tmp;
    for (const StageHost& x : h->stages) {
        if (!x.tc) continue;
        // back from [c_out][r][s][c_in] to the caller's [c_out][c_in][r][s]
        float* dst = host + x.user_off;
        const int CI = x.head.c_in, k2 = x.head.k * x.head.k;
        const size_t nw = (size_t)x.head.c_out * CI * k2;
        tmp.assign(dst, dst + nw);
        for (int co = 0; co < x.head.c_out; ++co)
            for (int ci = 0; ci < CI; ++ci)
                for (int rs = 0; rs < k2; ++rs) dst[((size_t)co * CI + ci) * k2 + rs] = tmp[((size_t)co * k2 + rs) * CI + ci];
    }
    return PB_OK;
}

int pb_get_weights(pb_handle* h, float* host_w, size_t n) { return get_params(h, h ? h->d_w : nullptr, host_w, n, "pb_get_weights"); }
int pb_get_velocity(pb_handle* h, float* host_v, size_t n) { return get_params(h, h ? h->d_v : nullptr, host_v, n, "pb_get_velocity"); }

int pb_sync(pb_handle* h) { return h ? check_device_error(h) : PB_E_ARG; }
size_t pb_num_params(const pb_handle* h) { return h ? h->n_params : 0; }
int pb_num_stages(const pb_handle* h) { return h ? h->S : PB_E_ARG; }
int pb_stage_delay(const pb_handle* h, int s) { return (h && s >= 0 && s < h->S) ? h->stages[s].delay : PB_E_ARG; }
long long pb_tick_count(const pb_handle* h) { return h ? h->tick : -1; }
long long pb_last_launch_count(const pb_handle* h) { return h ? h->last_launches : -1; }
size_t pb_device_bytes(const pb_handle* h) { return h ? h->arena_bytes : 0; }

double pb_kernel_min_bytes(const pb_handle* h, int which) {
    if (!h) return -1.0;
    double bytes = 0.0;
    if (which == 0) {
        // FC tick kernel: w and v read once and written once; the weight-difference form
        // also reads and writes its stored prediction
        const double per = ((h->flags & PB_LWP_WFORM) ? 24.0 : 16.0) + ((h->flags & PB_WEIGHT_STASH) ? 8.0 : 0.0);
        for (const pb::FcStage& f : h->h_fc) bytes += per * ((double)f.in_dim * f.out_dim + f.out_dim);
        return bytes;
    }
    if (which == 2) {
        // update kernel: reads w, v and every gradient slice (4 B each), writes w, v (8 B) and
        // the prediction (4 B as float32, or two bfloat16 copies of w and w_hat)
        for (const pb::UpdRange& r : h->h_upd) bytes += (double)r.n * (24.0 + 4.0 * (r.nparts - 1));
        return bytes;
    }
    return -1.0;
}

int pb_bench_l2_bandwidth(size_t bytes, int iters, void* stream, double* gbs) {
    if (!gbs || bytes < 4096 || iters <= 0) return fail(nullptr, PB_E_ARG, "pb_bench_l2_bandwidth: bad argument");
    cudaStream_t st = (cudaStream_t)stream;
    const size_t n = bytes / sizeof(float4);
    float4* buf = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    int sms = 0, dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaMalloc((void**)&buf, n * sizeof(float4));
    if (e == cudaSuccess) e = cudaMemsetAsync(buf, 0, n * sizeof(float4), st);
    if (e == cudaSuccess) e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    float ms = 0.f;
    if (e == cudaSuccess) {
        const int grid = sms * 8;
        for (int k = 0; k < 3; ++k) l2_sweep_kernel<<<grid, 256, 0, st>>>(buf, n, 0.5f, 1.0f);     // warm: the buffer is now cached
        cudaEventRecord(e0, st);
        for (int k = 0; k < iters; ++k) l2_sweep_kernel<<<grid, 256, 0, st>>>(buf, n, 0.5f, 1.0f);
        cudaEventRecord(e1, st);
        e = cudaEventSynchronize(e1);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
        if (e == cudaSuccess) e = cudaGetLastError();
    }
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    if (buf) cudaFree(buf);
    if (e != cudaSuccess) return fail(nullptr, PB_E_CUDA, std::string("pb_bench_l2_bandwidth: ") + cudaGetErrorString(e));
    *gbs = 2.0 * (double)(n * sizeof(float4)) * iters / (ms * 1e-3) / 1e9;
    return PB_OK;
}

int pb_bench_fp32_fma(int iters, void* stream, double* tflops) {
    if (!tflops || iters <= 0) return fail(nullptr, PB_E_ARG, "pb_bench_fp32_fma: bad argument");
    cudaStream_t st = (cudaStream_t)stream;
    float* out = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    int sms = 0, dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int grid = sms * 8, threads = 256;
    if (e == cudaSuccess) e = cudaMalloc((void**)&out, (size_t)grid * threads * sizeof(float));
    if (e == cudaSuccess) e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    float ms = 0.f;
    if (e == cudaSuccess) {
        fma_chain_kernel<<<grid, threads, 0, st>>>(out, 64, 0.999f, 1e-3f);
        cudaEventRecord(e0, st);
        fma_chain_kernel<<<grid, threads, 0, st>>>(out, iters, 0.999f, 1e-3f);
        cudaEventRecord(e1, st);
        e = cudaEventSynchronize(e1);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
        if (e == cudaSuccess) e = cudaGetLastError();
    }
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    if (out) cudaFree(out);
    if (e != cudaSuccess) return fail(nullptr, PB_E_CUDA, std::string("pb_bench_fp32_fma: ") + cudaGetErrorString(e));
    *tflops = 2.0 * 16.0 * (double)iters * grid * threads / (ms * 1e-3) / 1e12;
    return PB_OK;
}

int pb_profile_enable(pb_handle* h, int enable) {
    if (!h) return PB_E_ARG;
    h->profile = enable != 0;
    return PB_OK;
}

double pb_profile_ms(pb_handle* h, int which, long long* launches) {
    if (!h || which < 0 || which >= 9 || h->prof[which].launches == 0) { if (launches) *launches = 0; return -1.0; }
    if (launches) *launches = h->prof[which].launches;
    return h->prof[which].ms;
}

const char* pb_last_error(const pb_handle* h) { return h ? h->err.c_str() : g_create_error.c_str(); }

void pb_destroy(pb_handle* h) {
    if (!h) return;
    cudaStreamSynchronize(h->stream);
    for (cudaEvent_t e : h->ev_pool) cudaEventDestroy(e);
    if (h->side) { cudaStreamSynchronize(h->side); cudaStreamDestroy(h->side); }
    if (h->bwd) { cudaStreamSynchronize(h->bwd); cudaStreamDestroy(h->bwd); }
    if (h->ev_bjoin) cudaEventDestroy(h->ev_bjoin);
    if (h->aux) { cudaStreamSynchronize(h->aux); cudaStreamDestroy(h->aux); }
    if (h->ev_dz) cudaEventDestroy(h->ev_dz);
    if (h->ev_gemv) cudaEventDestroy(h->ev_gemv);
    if (h->ev_wjoin) cudaEventDestroy(h->ev_wjoin);
    if (h->ev_fork) cudaEventDestroy(h->ev_fork);
    if (h->ev_inputs) cudaEventDestroy(h->ev_inputs);
    if (h->ev_ingest) cudaEventDestroy(h->ev_ingest);
    if (h->ev_join) cudaEventDestroy(h->ev_join);
    if (h->staging) cudaFree(h->staging);
    cudaFree(h->arena);
    delete h;
}

}  // extern "C"

// ---------------------------------------------------------------- allocation-free entry point
namespace {

constexpr size_t kStaticScratchBytes = 4u << 20;   // 4 MiB, held by every GPU that loads the library
constexpr int kStaticMaxStages = 16;
constexpr int kStaticMaxDevices = 64;

// Scratch of pb_mlp_run_static: tick state, stage tables, activation rings and
// gradient hand-off buffers are carved out of this array instead of cudaMalloc'd
// memory.  In host code this name is only a handle for the runtime, not a
// device address: the address is looked up once per device below.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
void* g_static_scratch_addr[kStaticMaxDevices] = {nullptr};

}  // namespace

extern "C" int pb_mlp_run_static(const int32_t* sizes, int n_sizes, float lr, float momentum, unsigned flags,
                                 float* dev_w, float* dev_v, const float* dev_xs, const int32_t* dev_labels,
                                 int n_ticks, float* dev_losses, void* stream) {
    if (!sizes || !dev_w || !dev_v || !dev_xs || !dev_labels || n_ticks < 0)
        return fail(nullptr, PB_E_ARG, "pb_mlp_run_static: NULL pointer or negative tick count");
    if (n_sizes < 2 || n_sizes > kStaticMaxStages + 1)
        return fail(nullptr, PB_E_ARG, "pb_mlp_run_static: between 1 and 16 FC stages are supported");
    if (!(momentum >= 0.f && momentum < 1.f) || !(lr >= 0.f) || (flags & ~(unsigned)(PB_SC | PB_LWP)))
        return fail(nullptr, PB_E_ARG, "pb_mlp_run_static: need 0 <= momentum < 1, lr >= 0, flags within PB_SC|PB_LWP");
    pb_layer layers[2 * kStaticMaxStages];
    int32_t stage_of[2 * kStaticMaxStages];
    int nl = 0;
    for (int q = 0; q + 1 < n_sizes; ++q) {
        if (sizes[q] <= 0 || sizes[q + 1] <= 0) return fail(nullptr, PB_E_ARG, "pb_mlp_run_static: layer sizes must be positive");
        pb_layer fc{}; fc.op = PB_FC; fc.c_in = sizes[q]; fc.c_out = sizes[q + 1]; fc.src = -1;
        pb_layer tail{}; tail.op = (q + 2 == n_sizes) ? PB_SOFTMAX_CE : PB_RELU; tail.src = -1;
        layers[nl] = fc; stage_of[nl++] = q;
        layers[nl] = tail; stage_of[nl++] = q;
    }
    pb_handle hs;                       // host bookkeeping only; owns no device memory
    pb_handle* h = &hs;
    h->stream = (cudaStream_t)stream;
    h->flags = flags; h->lr = lr; h->momentum = momentum; h->n_classes = sizes[n_sizes - 1];
    h->in_shape = Shape{sizes[0], 1, 1};
    int rc = parse_layers(h, layers, nl, stage_of);
    if (rc != PB_OK) return rc;
    schedule_constants(h);
    cudaError_t e = cudaGetDevice(&h->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->num_sms, cudaDevAttrMultiProcessorCount, h->device);
    if (e != cudaSuccess) return fail(nullptr, PB_E_CUDA, std::string("pb_mlp_run_static: no CUDA device: ") + cudaGetErrorString(e));
    if (h->device < 0 || h->device >= kStaticMaxDevices) return fail(nullptr, PB_E_UNSUPPORTED, "pb_mlp_run_static: device ordinal above 63");
    if (!g_static_scratch_addr[h->device]) {
        // set-up, once per device, with that device current
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p) return fail(nullptr, PB_E_CUDA, std::string("pb_mlp_run_static: cudaGetSymbolAddress: ") + cudaGetErrorString(e));
        g_static_scratch_addr[h->device] = p;
    }
    char* base = static_cast<char*>(g_static_scratch_addr[h->device]);

    // the caller's flat vectors are the master weights and velocities
    h->d_w = dev_w; h->d_v = dev_v;
    for (StageHost& x : h->stages) x.dev_off = x.user_off;
    build_fc_tables(h, dev_w, dev_v);

    // carve the static array
    Carver c{base};
    h->d_ts = c.take<TickState>(1);
    h->d_fc = c.take<FcStage>(h->h_fc.size());
    h->d_segA = c.take<FcSeg>(h->h_segA.size());
    h->d_segB = c.take<FcSeg>(h->h_segB.size());
    h->d_ctaA = c.take<int>(h->h_ctaA.size());
    h->d_ctaB = c.take<int>(h->h_ctaB.size());
    h->in_slots = 2 * (h->S - 1) + 1;
    h->in_ring = c.take<float>((size_t)h->in_slots * h->in_shape.elems());
    h->label_ring = c.take<int>(h->S);
    for (StageHost& x : h->stages) {
        x.out_slots = x.delay + 1;
        x.out_ring = c.take<float>((size_t)x.out_slots * x.out.elems());
        if (x.src >= 0) {
            x.dx_slots = x.index - x.src + 1;
            x.dx = c.take<float>((size_t)x.dx_slots * x.dx_nparts * x.in.elems());
        }
    }
    if (c.off > kStaticScratchBytes)
        return fail(nullptr, PB_E_ARG, "pb_mlp_run_static: this network needs " + std::to_string(c.off) +
                                           " bytes of scratch, the static array holds " + std::to_string(kStaticScratchBytes));
    fill_fc_tables(h);
    // the array keeps the previous call's contents: clear what this call uses
    e = cudaMemsetAsync(base, 0, c.off, h->stream);
    auto up = [&](void* d, const void* s, size_t n) { if (e == cudaSuccess && n) e = cudaMemcpyAsync(d, s, n, cudaMemcpyHostToDevice, h->stream); };
    up(h->d_fc, h->h_fc.data(), h->h_fc.size() * sizeof(FcStage));
    up(h->d_segA, h->h_segA.data(), h->h_segA.size() * sizeof(FcSeg));
    up(h->d_segB, h->h_segB.data(), h->h_segB.size() * sizeof(FcSeg));
    up(h->d_ctaA, h->h_ctaA.data(), h->h_ctaA.size() * sizeof(int));
    up(h->d_ctaB, h->h_ctaB.data(), h->h_ctaB.size() * sizeof(int));
    if (e != cudaSuccess) return fail(nullptr, PB_E_CUDA, std::string("pb_mlp_run_static: table upload: ") + cudaGetErrorString(e));
    h->all_fc = true;
    if (n_ticks > 0) {
        rc = run_ticks(h, dev_xs, dev_labels, 0, n_ticks, dev_losses);
        if (rc != PB_OK) return fail(nullptr, rc, "pb_mlp_run_static: " + h->err);
    }
    rc = check_device_error(h);          // waits for the stream; the host tables may go after this
    if (rc != PB_OK) return fail(nullptr, rc, "pb_mlp_run_static: " + h->err);
    return PB_OK;
}
