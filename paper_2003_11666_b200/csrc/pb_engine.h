// Host-side engine state behind pb_handle.
#pragma once
#include <string>
#include <vector>

#include "../../include/pb.h"
#include "pb_internal.h"
#include "conv_types.h"
#include "conv_tc.cuh"
#include "conv_group.cuh"
#include "split.cuh"
#include "conv_gemv.cuh"

namespace pb {

struct Shape { int c = 0, h = 0, w = 0; int elems() const { return c * h * w; } };

// Host description of one pipeline stage.
struct StageHost {
    int index = 0;
    int head_op = PB_FC;            // PB_FC or PB_CONV2D
    pb_layer head{};
    int gn_groups = 0;
    int skip_src = -1, skip_mode = 0;
    bool skip_pre = false;                                          // the skip joins before the normalisation (and reads the source's pre-normalisation sum)
    bool has_skip = false, relu = false, avgpool = false, loss = false;
    bool has_pool = false;
    int pool_k = 0, pool_stride = 0, pool_pad = 0;
    int src = -1;                   // producing stage (-1: network input)
    Shape in, z, out;               // input, head output (pre-pool), stage output
    size_t n_params = 0;
    size_t user_off = 0;            // offset in the caller's flat parameter vector
    size_t dev_off = 0;             // offset (floats) in the padded device arrays
    int delay = 0;                  // D_s = 2 (S-1-s)
    float a = 1.f, b = 0.f, T = 0.f;
    // rings (device pointers into the arena)
    float* out_ring = nullptr; int out_slots = 0;
    float* dx = nullptr; int dx_slots = 0, dx_nparts = 1;          // gradient w.r.t. main input
    float* dskip = nullptr; int dskip_slots = 0;                   // gradient w.r.t. skip input
    std::vector<int> consumers_main, consumers_skip;               // stages reading this output
    std::vector<int> consumers_res;                                 // stages adding this stage's pre-normalisation sum to theirs
    // convolution stages only
    float *z_ring = nullptr, *stat_ring = nullptr, *zpart = nullptr, *dz = nullptr, *gpart = nullptr;
    unsigned char *code_ring = nullptr, *arg_ring = nullptr;
    float *fstat = nullptr, *bsum = nullptr, *gsum = nullptr; int fstat_stride = 1, npieces = 1;
    int split_f = 1, split_d = 1, split_w = 1;                     // K-slices of fprop / dgrad / wgrad
    int kps_f = 0, kps_d = 0, kps_w = 0;                           // K per slice
    bool tc = false;                                               // tensor-core path, weights kept as [co][r][s][ci]
    // weight stashing: rings of the weights (and normalisation scale) each forward used
    float* wstash = nullptr; __nv_bfloat16* wstash16 = nullptr; float* gstash = nullptr;
    int stash_slots = 0; size_t wstash_stride = 0, gstash_stride = 0;       // strides in bytes, multiples of 16
    bool gemv = false;                                             // 3x3 stage on a tiny image: one fused pass over (w, v) per tick
    bool fuse_stats = false;                                       // its forward GEMM writes the conv output and the chunk statistics
    int ntn = 1;                                                   // column tiles of that GEMM
    __nv_bfloat16 *out16 = nullptr, *dz16 = nullptr;
};

struct ProfileClass { double ms = 0; long long launches = 0; };

}  // namespace pb

struct pb_handle {
    cudaStream_t stream = nullptr;
    cudaStream_t side = nullptr;                // FC stages of conv nets run beside the conv chain of the same tick
    cudaStream_t bwd = nullptr;                 // backward chain of a tick, beside its forward chain
    cudaStream_t aux = nullptr;                 // weight gradients, beside the data gradients
    cudaEvent_t ev_dz = nullptr, ev_wjoin = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr, ev_bjoin = nullptr;
    cudaEvent_t ev_inputs = nullptr, ev_ingest = nullptr;   // caller's inputs ordered once per call; the sample's copy done
    int device = 0, num_sms = 0;
    unsigned flags = 0;
    float lr = 0, momentum = 0;
    float sc_delay_scale = 1.f, horizon_scale = 1.f;     // SC with alpha*D, LWP horizon alpha*D
    int update_size = 0;                        // > 0: fill-and-drain mini-batch SGD with that many samples per update
    int S = 0, n_classes = 0;
    pb::Shape in_shape;
    size_t n_params = 0, dev_params = 0;
    std::vector<pb::StageHost> stages;
    bool all_fc = true;

    // device memory (one arena)
    char* arena = nullptr; size_t arena_bytes = 0, zero_from = 0;
    char* staging = nullptr; size_t staging_bytes = 0;   // pb_run_host, grow-only
    float *d_w = nullptr, *d_v = nullptr;
    float* in_ring = nullptr; int in_slots = 0;
    int* label_ring = nullptr;
    pb::TickState* d_ts = nullptr;
    float* d_loss1 = nullptr;
    // FC tables
    pb::FcStage* d_fc = nullptr; int n_fc = 0;
    pb::FcSeg *d_segA = nullptr, *d_segB = nullptr;
    int *d_ctaA = nullptr, *d_ctaB = nullptr;
    int nctaA = 0, nctaB = 0;
    std::vector<pb::FcStage> h_fc;
    std::vector<pb::FcSeg> h_segA, h_segB;
    std::vector<int> h_ctaA, h_ctaB;
    // convolution tables
    float *d_wh = nullptr, *d_g = nullptr;
    __nv_bfloat16 *d_w16 = nullptr, *d_wh16 = nullptr;
    std::vector<pb::ConvGemmTC> h_tc; pb::ConvGemmTC* d_tc = nullptr;
    std::vector<pb::GemmTile> h_tctiles[3]; pb::GemmTile* d_tctiles[3] = {nullptr, nullptr, nullptr};
    std::vector<int> h_tcbegin[3]; int* d_tcbegin[3] = {nullptr, nullptr, nullptr};        // tiles of each persistent block
    std::vector<CUtensorMap> h_tmaps; CUtensorMap* d_tmaps = nullptr;                        // operand matrices fetched by bulk tensor copies
    std::vector<pb::PostChunk> h_fchunks; pb::PostChunk* d_fchunks = nullptr;                // first forward normalisation step (stages whose GEMM has not done it)
    std::vector<pb::ConvGemm> h_gemms; pb::ConvGemm* d_gemms = nullptr;
    std::vector<pb::GemmTile> h_tiles[3]; pb::GemmTile* d_tiles[3] = {nullptr, nullptr, nullptr};
    std::vector<pb::ConvStage> h_cs; pb::ConvStage* d_cs = nullptr;
    std::vector<pb::PostChunk> h_pchunks; pb::PostChunk* d_pchunks = nullptr;
    std::vector<pb::PostChunk> h_dtiles[2]; pb::PostChunk* d_dtiles[2] = {nullptr, nullptr};   // tiles of large bundles: launches of their own
    std::vector<pb::GroupRef> h_groups; pb::GroupRef* d_groups = nullptr;      // groups merged by the merge kernel
    bool post_fuse = false;                     // normalisation steps of a stage fused into one launch
    std::vector<pb::PostBundle> h_bundles; pb::PostBundle* d_bundles = nullptr;
    int* d_bcnt[2] = {nullptr, nullptr};        // bundle counters of the forward / backward launch
    std::vector<pb::PostChunk> h_ptiles[2]; pb::PostChunk* d_ptiles[2] = {nullptr, nullptr};   // tiles of the elementwise kernels: forward, backward
    std::vector<pb::UpdRange> h_upd; pb::UpdRange* d_upd = nullptr;
    std::vector<pb::UpdChunk> h_chunks; pb::UpdChunk* d_chunks = nullptr;
    std::vector<pb::ConvGemvStage> h_gemv; pb::ConvGemvStage* d_gemv = nullptr;             // stages run by the fused tiny-image kernel
    std::vector<pb::GemvBlock> h_gemvblocks; pb::GemvBlock* d_gemvblocks = nullptr;
    size_t gemv_smem = 0;
    cudaEvent_t ev_gemv = nullptr;
    std::vector<pb::GroupBlock> h_gblocks; pb::GroupBlock* d_gblocks = nullptr;             // bundles normalised by one block each
    size_t group_smem_fwd = 0, group_smem_bwd = 0;
    std::vector<pb::StashRange> h_stash; pb::StashRange* d_stash = nullptr;
    std::vector<pb::StashChunk> h_stashchunks; pb::StashChunk* d_stashchunks = nullptr;

    // stage split over several GPUs: this handle runs stages [s_lo, s_hi) (the whole network when n_ranks == 1)
    int split_rank = 0, split_n = 1, s_lo = 0, s_hi = 0;
    long long* d_stamps = nullptr;              // [0]: previous rank's activation stamp, [1]: next rank's gradient stamp
    pb::SplitLinks links{};
    bool split_connected = false;
    bool owns(int s) const { return split_n <= 1 || (s >= s_lo && s < s_hi); }

    long long tick = 0, last_launches = 0;
    bool profile = false;
    pb::ProfileClass prof[9];
    std::vector<cudaEvent_t> ev_pool; size_t ev_used = 0;
    std::vector<int> ev_class;
    std::string err;
};
