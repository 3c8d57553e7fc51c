// Host side of the C ABI (include/splitbrain.h): validation, the arena carve-up, the per-layer
// launch plan for forward / backward / update, and tensor introspection.
//
// Partitioning as data layout (one GPU, R logical replicas, K logical shards):
//  * every conv-side activation buffer is [B = R*b, H, W, C]; replica r owns the image rows
//    [r*b, (r+1)*b).  The last conv-side buffer reinterpreted as [B, H*W*C] *is* the gathered
//    input of the first FC layer (modulo layer, forward), and the FC input gradient written in
//    the same buffer shape *is* the scatter back to the replicas (modulo layer, backward).
//  * an FC weight is [out, in]; shard j is the row block [c_j, c_{j+1}), c_j = floor(j*out/K),
//    and owns the output columns with the same indices (shard layer, forward = column concat by
//    addressing).  The FC kernels take (shard_dim, K) and never let a tile straddle two shards.
#include "../../include/splitbrain.h"
#include "sb_internal.h"
#include "sb_umma.h"

#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <algorithm>
#include <vector>

using namespace sb;

static thread_local char g_err[512] = "";
static sb_status fail(sb_status s, const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return s;
}
extern "C" const char* sb_last_error(void) { return g_err; }

#define CU_TRY(expr)                                                                             \
    do {                                                                                         \
        cudaError_t e_ = (expr);                                                                 \
        if (e_ != cudaSuccess) return fail(SB_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e_)); \
    } while (0)

namespace {

struct Layer {
    int kind = 0, out = 0;
    int H = 0, W = 0, Cin = 0, Cout = 0;  // conv: input H,W,Cin -> Cout ; pool: input H,W,C=Cin=Cout
    int in_f = 0, out_f = 0;              // fc
    bool relu = false;
    size_t p_w = 0, p_b = 0, n_w = 0, n_b = 0;  // element offsets/counts in the parameter regions
    size_t out_per_img = 0;                     // elements of the layer output per image (row)
    char* act = nullptr;                        // [B, out_per_img] activation dtype (float for the logits layer)
    char* dact = nullptr;                       // same shape, activation dtype
    uint8_t* idx = nullptr;                     // pool argmax
    int wg_splits = 1;                          // conv wgrad pixel-range splits (CUDA-core kernel)
    int bg_splits = 1;                          // conv bias-gradient row splits
    bool thin_input = false;                    // conv with Cin of 1/3/4: dedicated input-layer kernels
    bool narrow = false;                        // FC with out <= 16: dedicated narrow kernels
    int K = 1;                                  // FC: column shards of this layer (the model's K, or 1 for a layer kept whole)
    int act_dt = SB_DT_F32;
    UmmaLayer um;                               // tensor-core plan of this layer (tcgen05 path)
    // Sub-batch copies of the first FC layer (modulo schedule): where its input comes from and where its input
    // gradient goes, instead of the layer below's buffers
    char* in_override = nullptr;
    char* dbelow_override = nullptr;
};

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace

struct sb_model {
    sb_config cfg{};
    std::vector<Layer> L;
    bool bf16 = false;
    int B = 0, first_fc = 0, n_layers = 0;
    size_t in_per_img = 0, esz = 4;
    char* arena = nullptr;
    size_t arena_bytes = 0;
    size_t P = 0;  // padded parameter element count
    float *Wm = nullptr, *Vm = nullptr, *Gm = nullptr;
    __nv_bfloat16* Sm = nullptr;
    float* ws = nullptr;    // scratch of the data-side kernels (split partial sums of forward / data gradient)
    float* ws_wk[8] = {};   // one weight-side scratch region per weight stream
    float* ws_w = nullptr;  // scratch of the weight-side kernels (split partial sums of weight / bias gradients), so that
                            // the two sides can run concurrently in the backward pass
    size_t ws_floats = 0;
    // backward-pass concurrency: weight-gradient work runs on a second stream, ordered by events
    static constexpr int MAX_WSTREAMS = 8;
    int n_wstreams = 0;                          // weight-gradient work of layer i runs on wstreams[i % n_wstreams]
    cudaStream_t wstreams[MAX_WSTREAMS] = {};
    cudaEvent_t ev_wjoin[MAX_WSTREAMS] = {};
    cudaStream_t ustream = nullptr;   // parameter updates folded into the backward pass
    cudaEvent_t ev_join = nullptr, ev_ujoin = nullptr;
    std::vector<cudaEvent_t> ev_ready;   // one per layer: "the gradient w.r.t. this layer's output is ready"
    std::vector<cudaEvent_t> ev_dgrad;   // one per layer: "this layer's input gradient has been computed"
    std::vector<cudaEvent_t> ev_wdone;   // one per layer: "this layer's weight and bias gradients are complete"
    float *row_loss = nullptr, *loss = nullptr;
    unsigned int* counter = nullptr;
    uint32_t* status = nullptr;
    uint32_t* drop_state = nullptr;   // dropout: {seed lo, seed hi, iteration, 0} (device words, kept between calls)
    int last_dropout = -1;            // index of the network's last dropout layer: its forward kernel is followed by the iteration bump
    bool st_clean = false;     // the chain stream's last kernel belongs to the current forward / backward pass (it cannot have written weights)
    int pooled_by_conv = -1;   // index of the pool layer whose output the conv kernel just before it has already written (same forward call)
    // Set by the multi-stream backward pass while it enqueues the weight side of one conv layer: the layer's split
    // reduces then apply the update themselves (launch_reduce_sgd) once `ev` (the layer's input-gradient kernel, which
    // reads the weights) has passed; `covered` counts the parameters updated that way.
    struct { bool on = false; float lr = 0.f, mu = 0.f; cudaEvent_t ev = nullptr; bool waited = false; size_t covered = 0; } fuse;
    char* stage_x = nullptr;
    int32_t* stage_labels = nullptr;
    // Input prefetch (sb_prefetch_host): a second staging area, so that the copy of the next iteration's inputs runs on a
    // copy stream while the current iteration computes.  Staged batches are consumed in order by sb_train_step_host.
    char* stage_xb[2] = {nullptr, nullptr};          // [0] = stage_x
    int32_t* stage_lb[2] = {nullptr, nullptr};       // [0] = stage_labels
    struct Staged { const void* host_x; const void* host_labels; int buf; };
    Staged staged[2];
    int n_staged = 0, stage_next = 0;
    cudaStream_t cpstream = nullptr;
    cudaEvent_t ev_staged[2] = {nullptr, nullptr};
    // Iterations in flight (sb_train_step_host_async): at most one per staging area; each writes its loss and the device
    // status word into its own pair of words of a small pinned host buffer and records ev_done[area].
    struct Flight { int slot; bool finished; float loss; sb_status status; char msg[160]; };
    Flight flights[2];
    int n_flights = 0;
    bool slot_busy[2] = {false, false};
    cudaEvent_t ev_done[2] = {nullptr, nullptr};
    uint32_t* host_res = nullptr;      // pinned host memory: [3][2] words (areas 0, 1; 2 = the call that copies its inputs itself)
    char* input_grad = nullptr;
    PtrTab x_tab{}, label_tab{};
    bool have_x = false, have_labels = false, have_fwd = false;
    // Modulo schedule (SB_FLAG_MODULO_SCHEDULE): the FC input / its gradient in sub-iteration order, the labels in
    // that order, and per sub-iteration a copy of the layer table whose FC layers address B/K rows of the buffers.
    // While a sub-iteration runs, L and B are those of the sub-batch (sub_active, sub_row0 say so).
    char *mod_x = nullptr, *mod_dx = nullptr;
    int32_t* mod_labels = nullptr;
    std::vector<std::vector<Layer>> mod_L;
    bool sub_active = false;
    int sub_row0 = 0, full_B = 0;
    int64_t launches = 0, last_step_launches = 0;
    // CUDA graphs of a whole iteration (sb_graph_step, sb_train_step_host), re-captured when their key changes
    struct StepGraph {
        cudaGraphExec_t exec = nullptr;
        PtrTab x{}, labels{};
        const void* host_x = nullptr;
        const void* host_labels = nullptr;
        float* host_loss = nullptr;
        float lr = 0.f, mu = 0.f;
        bool warmed = false;
    };
    StepGraph g_dev, g_host, g_mod;
    StepGraph g_pre[2];      // sb_train_step_host on inputs staged by sb_prefetch_host: one graph per staging area
    // Debug aids that stand in for a memory checker: every arena region is followed by a 256-byte guard holding a fixed
    // pattern (sb_debug_check_guards), and the regions a step overwrites are listed so that they can be filled with NaN
    // bit patterns before a step (sb_debug_poison).
    struct Region { size_t off, bytes; bool scratch; };
    std::vector<Region> regions;
    // per-launch event recording (sb_profile_begin / sb_profile_end)
    struct Rec { const char* tag; cudaEvent_t e0, e1; double flops, bytes; int layer; };
    int cur_layer = -1;   // layer whose kernels are being enqueued (profiling detail)
    bool debug_sync = false;   // SB_DEBUG_SYNC=1 in the environment: synchronise and check after every launch
    bool profiling = false;
    std::vector<Rec> recs;
    std::vector<cudaEvent_t> ev_pool;
    size_t ev_used = 0;
    cudaEvent_t next_event()
    {
        if (ev_used == ev_pool.size()) {
            cudaEvent_t e;
            if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
            ev_pool.push_back(e);
        }
        return ev_pool[ev_used++];
    }
    ~sb_model()
    {
        for (cudaEvent_t e : ev_pool) cudaEventDestroy(e);
        for (cudaEvent_t e : ev_ready) cudaEventDestroy(e);
        for (cudaEvent_t e : ev_dgrad) cudaEventDestroy(e);
        for (cudaEvent_t e : ev_wdone) cudaEventDestroy(e);
        if (ev_ujoin) cudaEventDestroy(ev_ujoin);
        if (ustream) cudaStreamDestroy(ustream);
        if (ev_join) cudaEventDestroy(ev_join);
        for (int k = 0; k < MAX_WSTREAMS; ++k) { if (wstreams[k]) cudaStreamDestroy(wstreams[k]); if (ev_wjoin[k]) cudaEventDestroy(ev_wjoin[k]); }
        if (g_dev.exec) cudaGraphExecDestroy(g_dev.exec);
        if (g_host.exec) cudaGraphExecDestroy(g_host.exec);
        if (g_mod.exec) cudaGraphExecDestroy(g_mod.exec);
        for (int k = 0; k < 2; ++k) {
            if (g_pre[k].exec) cudaGraphExecDestroy(g_pre[k].exec);
            if (ev_staged[k]) cudaEventDestroy(ev_staged[k]);
            if (ev_done[k]) cudaEventDestroy(ev_done[k]);
        }
        if (host_res) cudaFreeHost(host_res);
        if (cpstream) cudaStreamDestroy(cpstream);
    }
};

namespace {

// Walks the layer list, fills shapes, and assigns arena offsets (relative to base, which may be
// null for a pure size computation).  Returns SB_OK and the total size.
sb_status plan(const sb_layer* layers, int n, const sb_config* cfg, sb_model* m, char* base, size_t* total)
{
    if (!layers || !cfg || n <= 0) return fail(SB_ERR_INVALID_ARG, "null layers/config or empty layer list");
    if (cfg->precision != SB_FP32 && cfg->precision != SB_BF16) return fail(SB_ERR_INVALID_ARG, "precision must be SB_FP32 or SB_BF16");
    if (cfg->R < 1 || cfg->R > MAX_PARTS || cfg->K < 1 || cfg->K > MAX_PARTS) return fail(SB_ERR_SHAPE, "R and K must be in 1..%d", MAX_PARTS);
    if (cfg->H < 1 || cfg->W < 1 || cfg->C < 1 || cfg->batch_per_replica < 1) return fail(SB_ERR_SHAPE, "H, W, C and batch_per_replica must be positive");
    m->cfg = *cfg;
    m->bf16 = cfg->precision == SB_BF16;
    m->esz = m->bf16 ? 2 : 4;
    m->B = cfg->R * cfg->batch_per_replica;
    m->n_layers = n;
    m->L.assign(n, Layer());
    m->in_per_img = (size_t)cfg->H * cfg->W * cfg->C;
    if ((m->in_per_img * m->esz) % 16 != 0) return fail(SB_ERR_SHAPE, "one input image must be a multiple of 16 bytes");
    int H = cfg->H, W = cfg->W, C = cfg->C;
    long feat = -1;
    size_t P = 0;
    int first_fc = -1;
    for (int i = 0; i < n; ++i) {
        Layer& l = m->L[i];
        l.kind = layers[i].kind;
        l.out = layers[i].out;
        l.act_dt = m->bf16 ? SB_DT_BF16 : SB_DT_F32;
        // an FC layer kept whole is the same layer with one shard: from here on only the shard count tells them apart
        const bool whole = l.kind == SB_FC_RELU_WHOLE || l.kind == SB_FC_WHOLE;
        if (whole) l.kind = l.kind == SB_FC_RELU_WHOLE ? SB_FC_RELU : SB_FC;
        switch (l.kind) {
        case SB_CONV3X3_RELU:
            if (feat >= 0) return fail(SB_ERR_SHAPE, "layer %d: convolution after a fully-connected layer", i);
            if (l.out < 1) return fail(SB_ERR_SHAPE, "layer %d: Cout must be positive", i);
            l.H = H; l.W = W; l.Cin = C; l.Cout = l.out; l.relu = true;
            l.n_w = (size_t)l.Cout * 9 * l.Cin; l.n_b = l.Cout;
            C = l.out;
            l.out_per_img = (size_t)H * W * C;
            break;
        case SB_MAXPOOL2:
            if (feat >= 0) return fail(SB_ERR_SHAPE, "layer %d: pooling after a fully-connected layer", i);
            if (H % 2 || W % 2) return fail(SB_ERR_SHAPE, "layer %d: pooling needs even H and W (got %dx%d)", i, H, W);
            if (i == 0) return fail(SB_ERR_UNSUPPORTED, "layer 0 cannot be a pooling layer");
            l.H = H; l.W = W; l.Cin = l.Cout = C;
            H /= 2; W /= 2;
            l.out_per_img = (size_t)H * W * C;
            break;
        case SB_FC_RELU:
        case SB_FC:
            if (l.out < 1) return fail(SB_ERR_SHAPE, "layer %d: FC width must be positive", i);
            if (!whole && cfg->K > l.out) return fail(SB_ERR_SHAPE, "layer %d: K=%d exceeds the FC width %d", i, cfg->K, l.out);
            if (feat < 0) { feat = (long)H * W * C; first_fc = i; }
            l.in_f = (int)feat; l.out_f = l.out; l.relu = l.kind == SB_FC_RELU;
            l.n_w = (size_t)l.in_f * l.out_f; l.n_b = l.out_f;
            feat = l.out;
            l.out_per_img = l.out;
            if (l.kind == SB_FC) l.act_dt = SB_DT_F32;
            break;
        case SB_DROPOUT:
            // one-to-one layer on the output of the FC + ReLU layer below [Listing 1, case DROPOUT | RELU]; out = p * 65536
            if (i == 0 || m->L[i - 1].kind != SB_FC_RELU) return fail(SB_ERR_UNSUPPORTED, "layer %d: dropout must follow an FC + ReLU layer", i);
            if (l.out < 1 || l.out > 65535) return fail(SB_ERR_SHAPE, "layer %d: drop probability must be 1..65535 (units of 1/65536)", i);
            l.in_f = l.out_f = (int)feat;
            l.out_per_img = (size_t)feat;
            m->last_dropout = i;
            break;
        case SB_SOFTMAX_XENT:
            if (i != n - 1) return fail(SB_ERR_SHAPE, "the loss must be the last layer");
            if (i == 0 || m->L[i - 1].kind != SB_FC) return fail(SB_ERR_SHAPE, "the loss must follow an SB_FC (logits) layer");
            if (l.out != feat) return fail(SB_ERR_SHAPE, "loss classes (%d) != last FC width (%ld)", l.out, feat);
            break;
        default:
            return fail(SB_ERR_INVALID_ARG, "layer %d: unknown kind %d", i, l.kind);
        }
        if (l.kind == SB_FC && (i + 1 >= n || layers[i + 1].kind != SB_SOFTMAX_XENT))
            return fail(SB_ERR_SHAPE, "layer %d: SB_FC (no ReLU) is the logits layer and must be followed by the loss", i);
        if (l.n_w) {
            l.p_w = P; P += align_up(l.n_w, 64);
            l.p_b = P; P += align_up(l.n_b, 64);
        }
    }
    if (m->L[n - 1].kind != SB_SOFTMAX_XENT) return fail(SB_ERR_SHAPE, "the last layer must be SB_SOFTMAX_XENT");
    {
        // The partitioning table [Listing 1] decides how many column shards every layer has.  On one GPU its MODULO and SHARD
        // nodes are addressing inside one device buffer (row g of the gathered matrix is row g of the batch-major activation
        // buffer, a column slice is a column range), so only the per-layer shard counts are consumed here.
        std::vector<sb_plan_node> nodes((size_t)2 * n + 2);
        int32_t nn = 0;
        sb_status ps = sb_partition(layers, n, cfg, nodes.data(), (int32_t)nodes.size(), &nn);
        if (ps != SB_OK) return fail(ps, "%s", sb_partition_last_error());
        for (int32_t k = 0; k < nn; ++k)
            if (nodes[k].node == SB_NODE_LAYER) m->L[nodes[k].layer].K = nodes[k].shards;
    }
    m->first_fc = first_fc;
    m->P = P;

    // ---- arena carve-up -------------------------------------------------------------------
    size_t off = 0;
    // every region starts on a 256-byte boundary and is followed by at least 256 guard bytes that no kernel may touch
    bool scratch_region = false;
    m->regions.clear();
    auto take = [&](size_t bytes) {
        size_t o = off;
        m->regions.push_back({o, bytes, scratch_region});
        off = align_up(off + bytes, 256) + 256;
        return base ? base + o : (char*)nullptr;
    };
    m->Wm = (float*)take(P * 4);
    m->Vm = (float*)take(P * 4);
    m->Gm = (float*)take(P * 4);
    m->Sm = m->bf16 ? (__nv_bfloat16*)take(P * 2) : nullptr;
    scratch_region = true;      // from here on: activations, gradients of activations, scratch -- everything a step rewrites
    const size_t B = m->B;
    size_t ws_floats = 1024;
    for (int i = 0; i < n; ++i) {
        Layer& l = m->L[i];
        if (l.kind == SB_SOFTMAX_XENT) continue;
        size_t e = (l.kind == SB_FC) ? 4 : m->esz;
        l.act = take(B * l.out_per_img * e);
        l.dact = take(B * l.out_per_img * m->esz);
        if (l.kind == SB_MAXPOOL2) l.idx = (uint8_t*)take(B * l.out_per_img);
        if (l.kind == SB_FC_RELU || l.kind == SB_FC) l.narrow = fc_narrow_supported(l.out_f, (int)B);
        if (l.kind == SB_CONV3X3_RELU) {
            // pixel-range splits of the weight gradient: enough blocks to fill the machine, each
            // split a whole number of images
            long tiles = (long)((l.Cout + 31) / 32) * ((l.Cin + 31) / 32) * 9;
            int s = 1;
            while (tiles * s < 148 * 4 && s * 2 <= (int)B && B % (s * 2) == 0) s *= 2;
            l.wg_splits = s;
            size_t need = (size_t)s * l.n_w;
            if (need > ws_floats) ws_floats = need;
            int sb_ = 1;
            while (sb_ * 2 <= (int)B && B % (sb_ * 2) == 0 && (long)sb_ * ((l.Cout + 31) / 32) < 148 * 2) sb_ *= 2;
            l.bg_splits = sb_;
            if ((size_t)sb_ * l.n_b > ws_floats) ws_floats = (size_t)sb_ * l.n_b;
            l.thin_input = conv_in_supported(l.Cin, l.Cout);
            if (l.thin_input) {
                const int nblk = std::max(conv_in_wgrad_blocks((int)B, l.H, l.W), conv_in_umma_wgrad_blocks((long)B * l.H * l.W));
                size_t nd = (size_t)nblk * (l.n_w + l.n_b);
                if (nd > ws_floats) ws_floats = nd;
            }
        }
    }
    size_t um_ws = 0;
    sb_status us = umma_plan_scratch(m, &um_ws);
    if (us != SB_OK) return us;
    if (um_ws > ws_floats) ws_floats = um_ws;
    m->ws_floats = ws_floats;
    m->ws = (float*)take(ws_floats * 4);
    for (int k = 0; k < sb_model::MAX_WSTREAMS; ++k) m->ws_wk[k] = (float*)take(ws_floats * 4);
    m->ws_w = m->ws_wk[0];
    m->row_loss = (float*)take(B * 4);
    scratch_region = false;     // (loss, counter and status words keep their values between calls)
    m->loss = (float*)take(256);              // [0] = mean loss, [1] = device status word: adjacent, so that one copy reads both back
    m->status = base ? (uint32_t*)(m->loss + 1) : nullptr;
    m->counter = (unsigned int*)take(256);
    m->drop_state = (uint32_t*)take(256);
    m->stage_x = take(B * m->in_per_img * m->esz);
    m->stage_labels = (int32_t*)take(B * 4);
    m->stage_xb[0] = m->stage_x; m->stage_lb[0] = m->stage_labels;
    m->stage_xb[1] = take(B * m->in_per_img * m->esz);
    m->stage_lb[1] = (int32_t*)take(B * 4);
    m->input_grad = (cfg->flags & SB_FLAG_INPUT_GRAD) ? take(B * m->in_per_img * m->esz) : nullptr;
    if (cfg->flags & SB_FLAG_MODULO_SCHEDULE) {
        if (m->first_fc == 0) return fail(SB_ERR_UNSUPPORTED, "the modulo schedule needs a conv-side stack below the FC stack");
        if (cfg->batch_per_replica % cfg->K != 0) return fail(SB_ERR_UNSUPPORTED, "the modulo schedule needs batch_per_replica divisible by K");
        const size_t D = (size_t)m->L[m->first_fc].in_f;
        if ((D * m->esz) % 16 != 0) return fail(SB_ERR_UNSUPPORTED, "the modulo schedule needs feature rows of a multiple of 16 bytes");
        m->mod_x = take(B * D * m->esz);
        m->mod_dx = take(B * D * m->esz);
        m->mod_labels = (int32_t*)take(B * sizeof(int32_t));
    }
    *total = off;
    return SB_OK;
}

inline int shard_lo(int j, int total, int K) { return (int)(((long)j * total) / K); }

// Every kernel launch goes through here: counts it and, when profiling, brackets it with events.
// `tag` names the kernel class; flops/bytes are the algorithmic work of this launch.
#define L_TRY(tag, flops, bytes, expr)                                                            \
    do {                                                                                          \
        sb_model::Rec rec_{tag, nullptr, nullptr, (double)(flops), (double)(bytes), m->cur_layer}; \
        if (m->profiling) { rec_.e0 = m->next_event(); rec_.e1 = m->next_event();                 \
                            if (rec_.e0) cudaEventRecord(rec_.e0, st); }                          \
        cudaError_t e_ = (expr);                                                                  \
        ++m->launches;                                                                            \
        if (e_ != cudaSuccess) return fail(SB_ERR_CUDA, "launch failed in %s: %s", #expr, cudaGetErrorString(e_)); \
        if (m->profiling && rec_.e1) { cudaEventRecord(rec_.e1, st); m->recs.push_back(rec_); }   \
        if (m->debug_sync) {                                                                      \
            cudaError_t d_ = cudaStreamSynchronize(st);                                           \
            if (d_ != cudaSuccess) return fail(SB_ERR_CUDA, "kernel %s (layer call %s) failed: %s", tag, #expr, cudaGetErrorString(d_)); \
        }                                                                                         \
    } while (0)
// Same bracket for the tensor-core launchers, which return sb_status.
#define U_TRY(tag, flops, bytes, expr)                                                            \
    do {                                                                                          \
        sb_model::Rec rec_{tag, nullptr, nullptr, (double)(flops), (double)(bytes), m->cur_layer}; \
        if (m->profiling) { rec_.e0 = m->next_event(); rec_.e1 = m->next_event();                 \
                            if (rec_.e0) cudaEventRecord(rec_.e0, st); }                          \
        sb_status s_ = (expr);                                                                    \
        if (s_ != SB_OK) return fail(s_, "%s", umma_last_error());                                                            \
        if (m->profiling && rec_.e1) { cudaEventRecord(rec_.e1, st); m->recs.push_back(rec_); }   \
        if (m->debug_sync) {                                                                      \
            cudaError_t d_ = cudaStreamSynchronize(st);                                           \
            if (d_ != cudaSuccess) return fail(SB_ERR_CUDA, "kernel %s failed: %s", tag, cudaGetErrorString(d_)); \
        }                                                                                         \
    } while (0)

// Which buffer holds the input of layer i: the previous layer's output, or the caller's images.
inline const char* layer_input(const sb_model* m, int i) { return m->L[i].in_override ? m->L[i].in_override : (i > 0 ? m->L[i - 1].act : nullptr); }

sb_status forward_layer(sb_model* m, int i, cudaStream_t st)
{
    Layer& l = m->L[i];
    m->cur_layer = i;
    const bool bf = m->bf16;
    const int B = m->B, b = m->cfg.batch_per_replica;
    const double e = (double)m->esz;
    const void* wts = bf ? (const void*)(m->Sm + l.p_w) : (const void*)(m->Wm + l.p_w);
    switch (l.kind) {
    case SB_CONV3X3_RELU: {
        if (i == 0 && !m->have_x) return fail(SB_ERR_STATE, "layer 0 needs input pointers");
        const double pix = (double)B * l.H * l.W;
        const double flops = 2.0 * pix * l.Cout * 9.0 * l.Cin;
        const double bytes = pix * l.Cin * e + (double)l.n_w * e + pix * l.Cout * e;
        if (l.um.fwd.enabled) {
            const double pool_bytes = l.um.pool_fused ? pix / 4.0 * l.Cout * (e + 1.0) : 0.0;
            U_TRY("conv_fwd_umma", flops, bytes + pool_bytes, umma_conv_fwd(m, i, st));
            ++m->launches;
            if (l.um.pool_fused) m->pooled_by_conv = i + 1;
            break;
        }
        ConvSimtArgs a{};
        a.in = layer_input(m, i); a.tab = i == 0 ? &m->x_tab : nullptr; a.b_per_rep = b;
        a.w = wts; a.bias = m->Wm + l.p_b; a.out = l.act; a.mask_ref = nullptr;
        a.B = B; a.H = l.H; a.W = l.W; a.Cin = l.Cin; a.Cout = l.Cout; a.dgrad = 0; a.relu = 1;
        if (l.thin_input && l.um.conv_in) L_TRY("conv_in_fwd_umma", flops, bytes, launch_conv_in_fwd_umma(a, &l.um.fwd.mapA, m->status, st));
        else if (l.thin_input) L_TRY("conv_in_fwd", flops, bytes, launch_conv_in_fwd(a, bf, st));
        else L_TRY("conv_fwd_simt", flops, bytes, launch_conv_simt(a, bf, st));
        break;
    }
    case SB_MAXPOOL2: {
        if (m->pooled_by_conv == i) { m->pooled_by_conv = -1; break; }   // the conv kernel below has written this layer's output
        PoolArgs a{layer_input(m, i), l.act, l.idx, B, l.H, l.W, l.Cin};
        const double pooled = (double)B * l.out_per_img;
        L_TRY("pool_fwd", 0.0, pooled * (4 * e + e + 1), launch_pool_fwd(a, bf, st));
        break;
    }
    case SB_FC_RELU:
    case SB_FC: {
        if (i == 0 && !m->have_x) return fail(SB_ERR_STATE, "layer 0 needs input pointers");
        const double flops = 2.0 * B * (double)l.in_f * l.out_f;
        const double bytes = (double)B * l.in_f * e + (double)l.n_w * e + (double)B * l.out_f * (l.kind == SB_FC ? 4.0 : e);
        if (l.um.fwd.enabled) {
            if (i == 0) {
                // The tensor-core kernel reads the gathered input through one tensor map: replica buffers that
                // already lie back to back are used in place; scattered ones are first copied into the staging area.
                bool contiguous = true;
                const size_t rep_bytes = (size_t)b * m->in_per_img * m->esz;
                for (int r = 1; r < m->cfg.R; ++r)
                    contiguous = contiguous && (const char*)m->x_tab.p[r] == (const char*)m->x_tab.p[0] + (size_t)r * rep_bytes;
                const void* src = m->x_tab.p[0];
                if (!contiguous) {
                    if (m->n_staged > 0) return fail(SB_ERR_STATE, "a batch staged by sb_prefetch_host occupies the staging area: consume it first");
                    for (int r = 0; r < m->cfg.R; ++r)
                        if (m->x_tab.p[r] != m->stage_x + (size_t)r * rep_bytes)
                            CU_TRY(cudaMemcpyAsync(m->stage_x + (size_t)r * rep_bytes, m->x_tab.p[r], rep_bytes, cudaMemcpyDeviceToDevice, st));
                    src = m->stage_x;
                }
                sb_status bs = umma_bind_input(m, src);
                if (bs != SB_OK) return fail(bs, "%s", umma_last_error());
            }
            U_TRY("fc_fwd_umma", flops, bytes, umma_fc_fwd(m, i, st));
            ++m->launches;
            break;
        }
        if (l.narrow) {
            FcNarrowArgs a{};
            a.pass = 0; a.X = layer_input(m, i); a.tab = i == 0 ? &m->x_tab : nullptr; a.tab_b = b; a.W = wts;
            a.bias = m->Wm + l.p_b; a.relu = l.relu; a.B = B; a.in_f = l.in_f; a.out_f = l.out_f;
            if (l.kind == SB_FC) a.Y32 = (float*)l.act; else a.Y = l.act;
            L_TRY("fc_narrow_fwd", flops, bytes, launch_fc_narrow(a, bf, st));
            break;
        }
        GemmSimtArgs a{};
        a.A = layer_input(m, i); a.sAm = l.in_f; a.sAk = 1;
        a.B = wts; a.sBn = l.in_f; a.sBk = 1;
        a.M = B; a.N = l.out_f; a.K = l.in_f;
        a.epi = EPI_BIAS_ACT; a.ldc = l.out_f; a.bias = m->Wm + l.p_b; a.relu = l.relu;
        if (l.kind == SB_FC) { a.C = nullptr; a.C32 = (float*)l.act; } else { a.C = l.act; a.C32 = nullptr; }
        a.shard_dim = 1; a.shards = l.K;
        if (i == 0) { a.tab = &m->x_tab; a.tab_mode = 1; a.tab_b = b; }
        L_TRY("fc_fwd_simt", flops, bytes, launch_gemm_simt(a, bf, st));
        break;
    }
    case SB_DROPOUT: {
        const double n = (double)B * l.out_f;
        // (a sub-iteration of the modulo schedule works on b/K rows of every replica: the masks are those of the batch rows,
        // and the iteration counter moves on after the last sub-iteration)
        const int sub_bk = m->sub_active ? b / m->cfg.K : 0, sub_k = m->sub_active ? m->sub_row0 / B : 0;
        L_TRY("dropout_fwd", 0.0, 2.0 * n * e, launch_dropout_fwd(layer_input(m, i), l.act, (size_t)B, l.out_f, m->drop_state, i, l.out, bf, st, sub_bk, b, sub_k));
        if (i == m->last_dropout && (!m->sub_active || m->sub_row0 + B == m->full_B))
            L_TRY("dropout_state", 0.0, 8.0, launch_dropout_state(m->drop_state, 1, 0, 0, st));
        break;
    }
    case SB_SOFTMAX_XENT: {
        if (!m->have_labels) return fail(SB_ERR_STATE, "the loss layer needs label pointers");
        Layer& fc = m->L[i - 1];
        XentArgs a{};
        a.logits = (const float*)fc.act; a.labels = m->label_tab; a.b_per_rep = b;
        a.row_loss = m->row_loss; a.loss = m->loss; a.dZ = fc.dact; a.counter = m->counter;
        a.B = B; a.C = l.out;
        if (m->sub_active) {
            // rows [sub_row0, sub_row0 + B) of the full batch, labels already in sub-iteration order; every row's
            // gradient carries 1/full_B and the mean loss is taken over all rows written so far and before
            a.labels = PtrTab{};
            a.labels.p[0] = m->mod_labels + m->sub_row0;
            a.b_per_rep = B;
            a.row_loss = m->row_loss + m->sub_row0;
            a.scale_B = m->full_B; a.loss_base = m->row_loss; a.loss_rows = m->full_B;
        }
        L_TRY("softmax_xent", 0.0, (double)B * l.out * (4.0 + e) + 8.0 * B, launch_softmax_xent(a, bf, st));
        break;
    }
    }
    return SB_OK;
}

// part: 1 = weight-side work (weight / bias gradients), 2 = data-side work (input gradient), 3 = both.
// The two sides of a layer only share read-only inputs, so they may run on different streams.
enum { SIDE_W = 1, SIDE_D = 2, SIDE_BOTH = 3 };
sb_status backward_layer(sb_model* m, int i, cudaStream_t st, int part = SIDE_BOTH)
{
    Layer& l = m->L[i];
    m->cur_layer = i;
    const bool bf = m->bf16;
    const int B = m->B, b = m->cfg.batch_per_replica;
    const double e = (double)m->esz;
    const bool want_in_grad = i > 0 || (m->cfg.flags & SB_FLAG_INPUT_GRAD);
    // where the gradient w.r.t. this layer's input goes, and whether the layer below applied a ReLU
    char* d_below = l.dbelow_override ? l.dbelow_override : (i > 0 ? m->L[i - 1].dact : m->input_grad);
    const bool below_relu = i > 0 && (m->L[i - 1].kind == SB_CONV3X3_RELU || m->L[i - 1].kind == SB_FC_RELU || m->L[i - 1].kind == SB_DROPOUT);
    const void* wts = bf ? (const void*)(m->Sm + l.p_w) : (const void*)(m->Wm + l.p_w);
    // this layer's weight-side scratch: one region per weight stream, so two layers that share a region are
    // ordered by the stream they share
    float* const ws_w = m->ws_wk[m->n_wstreams > 0 ? i % m->n_wstreams : 0];
    switch (l.kind) {
    case SB_SOFTMAX_XENT:
        break;  // dZ was produced by the forward loss kernel
    case SB_FC_RELU:
    case SB_FC: {
        if (i == 0 && !m->have_x) return fail(SB_ERR_STATE, "layer 0 needs input pointers");
        const double flops = 2.0 * B * (double)l.in_f * l.out_f;
        const double act_bytes = (double)B * (l.in_f + l.out_f) * e;
        // weight gradient per shard: dW_j = dY_j^T X   (rows c_j..c_{j+1} of the [out,in] gradient)
        if (l.narrow) {
            FcNarrowArgs a{};
            a.pass = 1; a.X = layer_input(m, i); a.tab = i == 0 ? &m->x_tab : nullptr; a.tab_b = b;
            a.dY = l.dact; a.dW = m->Gm + l.p_w; a.db = m->Gm + l.p_b; a.B = B; a.in_f = l.in_f; a.out_f = l.out_f;
            if (part & SIDE_W) L_TRY("fc_narrow_wgrad", flops, act_bytes + (double)l.n_w * 4.0, launch_fc_narrow(a, bf, st));
            if (want_in_grad && (part & SIDE_D)) {
                a.pass = 2; a.W = wts; a.ref = below_relu ? layer_input(m, i) : nullptr; a.dX = d_below;
                L_TRY("fc_narrow_dgrad", flops, act_bytes + (double)l.n_w * e + (below_relu ? (double)B * l.in_f * e : 0.0), launch_fc_narrow(a, bf, st));
            }
            break;
        }
        if (!(part & SIDE_W)) {
        } else if (l.um.wgrad.enabled && m->fuse.on && !(part & SIDE_D) && umma_fc_wgrad_can_update(m, i)) {
            // fused pass: the update is applied by the weight-gradient kernel's epilogue (after the layer's input-gradient
            // kernel, which reads the weights); the gradient itself is never stored
            if (!m->fuse.waited) { CU_TRY(cudaStreamWaitEvent(st, m->fuse.ev, 0)); m->fuse.waited = true; }
            U_TRY("fc_wgrad_umma", flops, act_bytes + (double)(l.n_w + l.n_b) * (m->bf16 ? 18.0 : 16.0), umma_fc_wgrad_update(m, i, m->fuse.lr, m->fuse.mu, st));
            ++m->launches;
            m->fuse.covered = l.n_w + l.n_b;
        } else if (l.um.wgrad.enabled) {
            U_TRY("fc_wgrad_umma", flops, act_bytes + (double)l.n_w * 4.0, umma_fc_wgrad(m, i, st));
            ++m->launches;
        } else {
            GemmSimtArgs a{};
            a.A = l.dact; a.sAm = 1; a.sAk = l.out_f;
            a.B = layer_input(m, i); a.sBn = 1; a.sBk = l.in_f;
            a.M = l.out_f; a.N = l.in_f; a.K = B;
            a.epi = EPI_F32; a.C = m->Gm + l.p_w; a.ldc = l.in_f;
            a.shard_dim = 3; a.shards = l.K;
            if (i == 0) { a.tab = &m->x_tab; a.tab_mode = 2; a.tab_b = b; }
            L_TRY("fc_wgrad_simt", flops, act_bytes + (double)l.n_w * 4.0, launch_gemm_simt(a, bf, st));
        }
        if (!l.um.wgrad.enabled && (part & SIDE_W))   // the tensor-core weight-gradient kernel also produces the bias gradient
            L_TRY("bias_grad", 0.0, (double)B * l.out_f * e + 4.0 * l.out_f, launch_colsum(l.dact, bf, m->Gm + l.p_b, B, l.out_f, 1, st));
        if (want_in_grad && (part & SIDE_D)) {
            // shard-layer / modulo-layer backward: dX = sum_j dY_j W_j, rows stay with their replica
            const double bytes = act_bytes + (double)l.n_w * e + (below_relu ? (double)B * l.in_f * e : 0.0);
            if (l.um.dgrad.enabled) {
                U_TRY("fc_dgrad_umma", flops, bytes, umma_fc_dgrad(m, i, st));
                ++m->launches;
            } else {
                GemmSimtArgs a{};
                a.A = l.dact; a.sAm = l.out_f; a.sAk = 1;
                a.B = wts; a.sBn = 1; a.sBk = l.in_f;
                a.M = B; a.N = l.in_f; a.K = l.out_f;
                a.epi = EPI_MASK; a.C = d_below; a.ldc = l.in_f;
                a.ref = below_relu ? layer_input(m, i) : nullptr; a.ldref = l.in_f;
                a.shard_dim = 2; a.shards = l.K;
                L_TRY("fc_dgrad_simt", flops, bytes, launch_gemm_simt(a, bf, st));
            }
        }
        break;
    }
    case SB_DROPOUT: {
        // the layer above wrote the gradient w.r.t. this layer's output, zeroed wherever the output is zero (dropped, or the
        // ReLU below was inactive): what is left is the scale of the kept elements, and the result is the gradient w.r.t. the
        // pre-activation output of the FC + ReLU layer below
        if (!(part & SIDE_D)) break;
        const double n = (double)B * l.out_f;
        L_TRY("dropout_bwd", 0.0, 2.0 * n * e, launch_dropout_bwd(l.dact, d_below, (size_t)B * l.out_f, l.out, bf, st));
        break;
    }
    case SB_MAXPOOL2: {
        if (!(part & SIDE_D)) break;
        PoolBwdArgs a{l.dact, l.idx, below_relu ? l.act : nullptr, d_below, B, l.H, l.W, l.Cin};
        const double pooled = (double)B * l.out_per_img;
        L_TRY("pool_bwd", 0.0, pooled * (e + 1 + (below_relu ? e : 0.0) + 4 * e), launch_pool_bwd(a, bf, st));
        break;
    }
    case SB_CONV3X3_RELU: {
        if (i == 0 && !m->have_x) return fail(SB_ERR_STATE, "layer 0 needs input pointers");
        const double pix = (double)B * l.H * l.W;
        const double flops = 2.0 * pix * l.Cout * 9.0 * l.Cin;
        // End of a gradient range [goff, goff + n) of this layer: S > 1 partial copies at `src` are reduced in order into
        // the gradient arena -- or, when the backward pass folds the update in, reduced and applied in one kernel (S = 1:
        // the gradient is already in the arena and takes a plain update).
        const bool fuse = m->fuse.on && (part & SIDE_W) && !(part & SIDE_D) && l.n_w % 4 == 0 && l.n_b % 4 == 0 && l.p_w % 4 == 0 && l.p_b % 4 == 0;
        // (in_place: with S = 1 the kernel wrote the gradient into the arena itself; the input-layer kernels always write
        // partial buffers, so a single one still has to be carried over)
        auto finish = [&](const float* src, size_t stride, size_t goff, size_t n, int S, bool in_place = true) -> sb_status {
            const bool reduce = S > 1 || !in_place;
            if (!fuse) {
                if (reduce) L_TRY("split_reduce", 0.0, (double)n * 4.0 * (S + 1), launch_reduce_partials(src, stride, m->Gm + goff, n, S, st));
                return SB_OK;
            }
            if (!m->fuse.waited) { CU_TRY(cudaStreamWaitEvent(st, m->fuse.ev, 0)); m->fuse.waited = true; }
            __nv_bfloat16* sh = m->Sm ? m->Sm + goff : nullptr;
            if (reduce)
                L_TRY("split_reduce_sgd", 0.0, (double)n * (4.0 * S + (m->bf16 ? 18.0 : 16.0)),
                      launch_reduce_sgd(src, stride, n, S, m->Wm + goff, m->Vm + goff, sh, m->fuse.lr, m->fuse.mu, st));
            else
                L_TRY("sgd", 0.0, (double)n * (m->bf16 ? 22.0 : 20.0), launch_sgd(m->Wm + goff, m->Vm + goff, m->Gm + goff, sh, n, m->fuse.lr, m->fuse.mu, st));
            m->fuse.covered += n;
            return SB_OK;
        };
        sb_status fs = SB_OK;
        // weight gradient over all replicas' pixels (the DP reduce is the sum over image ranges)
        if (!(part & SIDE_W)) {
        } else if (l.thin_input) {
            // input-layer kernel: weight and bias partial sums per block, then one ordered reduce each
            WgradSimtArgs a{};
            a.x = layer_input(m, i); a.tab = i == 0 ? &m->x_tab : nullptr; a.b_per_rep = b;
            a.dy = l.dact; a.part = ws_w; a.B = B; a.H = l.H; a.W = l.W; a.Cin = l.Cin; a.Cout = l.Cout;
            const int nb = l.um.conv_in ? conv_in_umma_wgrad_blocks((long)B * l.H * l.W) : conv_in_wgrad_blocks(B, l.H, l.W);
            const size_t stride = l.n_w + l.n_b;
            if (l.um.conv_in)
                L_TRY("conv_in_wgrad_umma", flops, pix * (l.Cin + l.Cout) * e + (double)l.n_w * 4.0, launch_conv_in_wgrad_umma(a, l.um.wgrad.mapA, m->status, st));
            else
                L_TRY("conv_in_wgrad", flops, pix * (l.Cin + l.Cout) * e + (double)l.n_w * 4.0, launch_conv_in_wgrad(a, bf, st));
            if (l.p_b == l.p_w + l.n_w) {
                // the bias vector directly follows the weights in the gradient arena, as it does in a partial buffer
                if ((fs = finish(ws_w, stride, l.p_w, stride, nb, false)) != SB_OK) return fs;
            } else {
                if ((fs = finish(ws_w, stride, l.p_w, l.n_w, nb, false)) != SB_OK) return fs;
                if ((fs = finish(ws_w + l.n_w, stride, l.p_b, l.n_b, nb, false)) != SB_OK) return fs;
            }
        } else if (l.um.wgrad.enabled) {
            int S = 1;
            float* part = nullptr;
            U_TRY("conv_wgrad_umma", flops, pix * (l.Cin + l.Cout) * e + (double)l.n_w * 4.0, umma_conv_wgrad_launch(m, i, st, &S, &part));
            ++m->launches;
            // weights and bias gradient reduce together (same layout in the split buffers and in the arena); a kernel
            // that leaves the bias gradient to the column-sum pass below reduces (or updates) the weights only
            const bool with_bias = umma_wgrad_bias_fused(m, i) && l.p_b == l.p_w + l.n_w;
            if (with_bias || S > 1 || fuse) {
                if (with_bias || !fuse) { if ((fs = finish(part, l.n_w + l.n_b, l.p_w, l.n_w + l.n_b, S)) != SB_OK) return fs; }
                else if ((fs = finish(part, l.n_w + l.n_b, l.p_w, l.n_w, S)) != SB_OK) return fs;
            }
        } else {
            const int S = l.wg_splits;
            WgradSimtArgs a{};
            a.x = layer_input(m, i); a.tab = i == 0 ? &m->x_tab : nullptr; a.b_per_rep = b;
            a.dy = l.dact; a.part = S > 1 ? ws_w : m->Gm + l.p_w;
            a.B = B; a.H = l.H; a.W = l.W; a.Cin = l.Cin; a.Cout = l.Cout; a.splits = S;
            L_TRY("conv_wgrad_simt", flops, pix * (l.Cin + l.Cout) * e + (double)l.n_w * 4.0, launch_wgrad_simt(a, bf, st));
            if ((fs = finish(ws_w, l.n_w, l.p_w, l.n_w, S)) != SB_OK) return fs;
        }
        if (!l.thin_input && (part & SIDE_W) && (!l.um.wgrad.enabled || !umma_wgrad_bias_fused(m, i))) {
            // bias gradient: column sums of dY over image-range splits, then the same ordered reduce
            const long M = (long)B * l.H * l.W;
            // (stream order makes it safe to reuse the scratch the weight-gradient reduce just read)
            int S = l.bg_splits;
            if (bf && l.Cout % 8 == 0) {
                // the vectorised column-sum kernel covers 256 columns per block column: split the rows finely enough to
                // fill the machine (its splits need not be whole images), within the scratch
                long want = 592 / ((l.Cout / 8 + 31) / 32);
                if (want > M / 64) want = M / 64;
                if (want > (long)(m->ws_floats / l.n_b)) want = (long)(m->ws_floats / l.n_b);
                S = want < 1 ? 1 : (int)want;
            }
            float* part = S > 1 ? ws_w : m->Gm + l.p_b;
            L_TRY("bias_grad", 0.0, pix * l.Cout * e, launch_colsum(l.dact, bf, part, (int)M, l.Cout, S, st));
            if ((fs = finish(part, l.n_b, l.p_b, l.n_b, S)) != SB_OK) return fs;
        }
        if (want_in_grad && (part & SIDE_D)) {
            const double bytes = pix * (l.Cin + l.Cout) * e + (double)l.n_w * e + (below_relu ? pix * l.Cin * e : 0.0);
            if (l.um.dgrad.enabled) {
                U_TRY("conv_dgrad_umma", flops, bytes, umma_conv_dgrad(m, i, st));
                ++m->launches;
            } else {
                ConvSimtArgs a{};
                a.in = l.dact; a.tab = nullptr; a.b_per_rep = b;
                a.w = wts; a.bias = nullptr; a.out = d_below;
                a.mask_ref = below_relu ? m->L[i - 1].act : nullptr;
                a.B = B; a.H = l.H; a.W = l.W; a.Cin = l.Cin; a.Cout = l.Cout; a.dgrad = 1; a.relu = 0;
                L_TRY("conv_dgrad_simt", flops, bytes, launch_conv_simt(a, bf, st));
            }
        }
        break;
    }
    }
    return SB_OK;
}

sb_status set_inputs(sb_model* m, const void* const* x, const int32_t* const* labels)
{
    for (int r = 0; r < m->cfg.R; ++r) {
        if (x) {
            if (!x[r] || ((uintptr_t)x[r] & 15)) return fail(SB_ERR_INVALID_ARG, "x[%d] is null or not 16-byte aligned", r);
            m->x_tab.p[r] = x[r];
        }
        if (labels) {
            if (!labels[r] || ((uintptr_t)labels[r] & 3)) return fail(SB_ERR_INVALID_ARG, "labels[%d] is null or misaligned", r);
            m->label_tab.p[r] = labels[r];
        }
    }
    if (x) m->have_x = true;
    if (labels) m->have_labels = true;
    return SB_OK;
}

// Resolves (what, layer, part) to a device pointer, shape and dtype.
sb_status resolve(sb_model* m, int what, int li, int part, char** ptr, int64_t shape[4], int* dtype, size_t* bytes)
{
    if (!m) return fail(SB_ERR_INVALID_ARG, "null model");
    if (li < 0 || li >= m->n_layers) return fail(SB_ERR_INVALID_ARG, "layer %d out of range", li);
    Layer& l = m->L[li];
    const int b = m->cfg.batch_per_replica, R = m->cfg.R, K = l.K;      // (K: this layer's own shard count)
    int64_t sh[4] = {1, 1, 1, 1};
    char* p = nullptr;
    int dt = SB_DT_F32;
    const bool is_conv = l.kind == SB_CONV3X3_RELU, is_fc = l.kind == SB_FC_RELU || l.kind == SB_FC, is_pool = l.kind == SB_MAXPOOL2;
    const bool is_flat = is_fc || l.kind == SB_DROPOUT;   // [B, width] activations
    auto param = [&](float* region, bool weight) -> sb_status {
        if (!is_conv && !is_fc) return fail(SB_ERR_INVALID_ARG, "layer %d has no parameters", li);
        if (is_conv) {
            if (part != 0) return fail(SB_ERR_INVALID_ARG, "conv parameters are replicated: part must be 0");
            if (weight) { p = (char*)(region + l.p_w); sh[0] = l.Cout; sh[1] = 3; sh[2] = 3; sh[3] = l.Cin; }
            else { p = (char*)(region + l.p_b); sh[0] = l.Cout; }
        } else {
            if (part < 0 || part >= K) return fail(SB_ERR_INVALID_ARG, "shard %d out of range", part);
            int lo = shard_lo(part, l.out_f, K), hi = shard_lo(part + 1, l.out_f, K);
            if (weight) { p = (char*)(region + l.p_w + (size_t)lo * l.in_f); sh[0] = hi - lo; sh[1] = l.in_f; }
            else { p = (char*)(region + l.p_b + lo); sh[0] = hi - lo; }
        }
        return SB_OK;
    };
    sb_status s = SB_OK;
    switch (what) {
    case SB_T_WEIGHT: s = param(m->Wm, true); break;
    case SB_T_BIAS: s = param(m->Wm, false); break;
    case SB_T_GRAD_W: s = param(m->Gm, true); break;
    case SB_T_GRAD_B: s = param(m->Gm, false); break;
    case SB_T_MOM_W: s = param(m->Vm, true); break;
    case SB_T_MOM_B: s = param(m->Vm, false); break;
    case SB_T_SHADOW_W:
        if (!m->bf16) return fail(SB_ERR_INVALID_ARG, "no bf16 weight copies in SB_FP32 mode");
        s = param(m->Wm, true);
        if (s == SB_OK) { p = (char*)(m->Sm + ((float*)p - m->Wm)); dt = SB_DT_BF16; }
        break;
    case SB_T_ACT:
    case SB_T_DACT: {
        if (l.kind == SB_SOFTMAX_XENT) return fail(SB_ERR_INVALID_ARG, "the loss layer has no activation tensor");
        char* basep = what == SB_T_ACT ? l.act : l.dact;
        dt = what == SB_T_ACT ? l.act_dt : (m->bf16 ? SB_DT_BF16 : SB_DT_F32);
        size_t e = dt == SB_DT_BF16 ? 2 : 4;
        if (is_flat) { p = basep; sh[0] = m->B; sh[1] = l.out_f; }
        else {
            if (part < 0 || part >= R) return fail(SB_ERR_INVALID_ARG, "replica %d out of range", part);
            p = basep + (size_t)part * b * l.out_per_img * e;
            int Ho = is_pool ? l.H / 2 : l.H, Wo = is_pool ? l.W / 2 : l.W;
            sh[0] = b; sh[1] = Ho; sh[2] = Wo; sh[3] = l.Cout;
        }
        break;
    }
    case SB_T_POOL_IDX:
        if (!is_pool) return fail(SB_ERR_INVALID_ARG, "layer %d is not a pooling layer", li);
        if (part < 0 || part >= R) return fail(SB_ERR_INVALID_ARG, "replica %d out of range", part);
        p = (char*)l.idx + (size_t)part * b * l.out_per_img;
        sh[0] = b; sh[1] = l.H / 2; sh[2] = l.W / 2; sh[3] = l.Cout; dt = SB_DT_U8;
        break;
    case SB_T_ROW_LOSS:
        p = (char*)m->row_loss; sh[0] = m->B;
        break;
    case SB_T_INPUT_GRAD:
        if (!m->input_grad) return fail(SB_ERR_INVALID_ARG, "model was created without SB_FLAG_INPUT_GRAD");
        if (part < 0 || part >= R) return fail(SB_ERR_INVALID_ARG, "replica %d out of range", part);
        dt = m->bf16 ? SB_DT_BF16 : SB_DT_F32;
        p = m->input_grad + (size_t)part * b * m->in_per_img * m->esz;
        sh[0] = b; sh[1] = m->cfg.H; sh[2] = m->cfg.W; sh[3] = m->cfg.C;
        break;
    default:
        return fail(SB_ERR_INVALID_ARG, "unknown tensor selector %d", what);
    }
    if (s != SB_OK) return s;
    if (ptr) *ptr = p;
    if (shape) memcpy(shape, sh, sizeof(sh));
    if (dtype) *dtype = dt;
    if (bytes) {
        size_t e = dt == SB_DT_F32 || dt == SB_DT_I32 ? 4 : dt == SB_DT_BF16 ? 2 : 1;
        *bytes = (size_t)(sh[0] * sh[1] * sh[2] * sh[3]) * e;
    }
    return SB_OK;
}

}  // namespace

// Accessors used by the tensor-core planner (sb_umma.cu), which cannot see the struct layout.
namespace sb {
ModelView model_view(sb_model* m)
{
    ModelView v{};
    v.cfg = &m->cfg; v.bf16 = m->bf16; v.B = m->B; v.n_layers = m->n_layers; v.first_fc = m->first_fc;
    v.Wm = m->Wm; v.Gm = m->Gm; v.Vm = m->Vm; v.Sm = m->Sm; v.ws = m->ws; for (int k = 0; k < sb_model::MAX_WSTREAMS; ++k) v.ws_wk[k] = m->ws_wk[k]; v.ws_floats = m->ws_floats; v.n_wstreams = m->n_wstreams; v.status = m->status;
    v.input_grad = m->input_grad; v.x_tab = &m->x_tab; v.stage_x = m->stage_x;
    return v;
}
LayerView layer_view(sb_model* m, int i)
{
    Layer& l = m->L[i];
    LayerView v{};
    v.K = l.K;
    v.kind = l.kind; v.H = l.H; v.W = l.W; v.Cin = l.Cin; v.Cout = l.Cout; v.in_f = l.in_f; v.out_f = l.out_f; v.relu = l.relu;
    v.p_w = l.p_w; v.p_b = l.p_b; v.n_w = l.n_w; v.n_b = l.n_b;
    v.act = l.act; v.dact = l.dact; v.um = &l.um; v.pool_idx = l.idx;
    v.in_act = l.in_override ? l.in_override : (i > 0 ? m->L[i - 1].act : nullptr);
    v.d_below = l.dbelow_override ? l.dbelow_override : (i > 0 ? m->L[i - 1].dact : m->input_grad);
    v.below_relu = i > 0 && (m->L[i - 1].kind == SB_CONV3X3_RELU || m->L[i - 1].kind == SB_FC_RELU || m->L[i - 1].kind == SB_DROPOUT);
    return v;
}
int64_t* launch_counter(sb_model* m) { return &m->launches; }
}  // namespace sb

// =================================================================================================
extern "C" {

sb_status sb_model_bytes(const sb_layer* layers, int32_t n, const sb_config* cfg, size_t* arena_bytes)
{
    if (!arena_bytes) return fail(SB_ERR_INVALID_ARG, "arena_bytes is null");
    sb_model tmp;
    return plan(layers, n, cfg, &tmp, nullptr, arena_bytes);
}

sb_status sb_model_create(const sb_layer* layers, int32_t n, const sb_config* cfg, void* arena, size_t arena_bytes, sb_model** out)
{
    if (!out) return fail(SB_ERR_INVALID_ARG, "out is null");
    *out = nullptr;
    if (!arena || ((uintptr_t)arena & 255)) return fail(SB_ERR_INVALID_ARG, "arena is null or not 256-byte aligned");
    sb_model* m = new (std::nothrow) sb_model;
    if (!m) return fail(SB_ERR_INVALID_ARG, "out of host memory");
    size_t need = 0;
    sb_status s = plan(layers, n, cfg, m, (char*)arena, &need);
    if (s != SB_OK) { delete m; return s; }
    if (need > arena_bytes) { delete m; return fail(SB_ERR_ARENA_TOO_SMALL, "arena has %zu bytes, model needs %zu", arena_bytes, need); }
    m->arena = (char*)arena;
    m->arena_bytes = need;
    const char* dbg = getenv("SB_DEBUG_SYNC");
    m->debug_sync = dbg && dbg[0] == '1';
    const char* one = getenv("SB_ONE_STREAM");
    if (!(one && one[0] == '1')) {
        // second stream + ordering events for the backward pass (host objects; no device memory)
        m->n_wstreams = (int)tune("SB_WSTREAMS", 6);
        if (m->n_wstreams < 1) m->n_wstreams = 1;
        if (m->n_wstreams > sb_model::MAX_WSTREAMS) m->n_wstreams = sb_model::MAX_WSTREAMS;
        bool ok_ = true;
        for (int k = 0; ok_ && k < m->n_wstreams; ++k)
            ok_ = cudaStreamCreateWithFlags(&m->wstreams[k], cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&m->ev_wjoin[k], cudaEventDisableTiming) == cudaSuccess;
        ok_ = ok_ && cudaStreamCreateWithFlags(&m->ustream, cudaStreamNonBlocking) == cudaSuccess &&
                   cudaEventCreateWithFlags(&m->ev_join, cudaEventDisableTiming) == cudaSuccess &&
                   cudaEventCreateWithFlags(&m->ev_ujoin, cudaEventDisableTiming) == cudaSuccess;
        m->ev_ready.assign(n, nullptr);
        m->ev_dgrad.assign(n, nullptr);
        m->ev_wdone.assign(n, nullptr);
        for (int i = 0; ok_ && i < n; ++i)
            ok_ = cudaEventCreateWithFlags(&m->ev_ready[i], cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&m->ev_dgrad[i], cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&m->ev_wdone[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok_) { delete m; return fail(SB_ERR_CUDA, "creating the backward-pass stream / events failed"); }
    }
    cudaError_t e = cudaMemset(arena, 0, need);
    // the guard bytes behind every region (checked by sb_debug_check_guards)
    for (size_t k = 0; e == cudaSuccess && k < m->regions.size(); ++k) {
        const size_t g0 = m->regions[k].off + m->regions[k].bytes, g1 = align_up(g0, 256) + 256;
        e = cudaMemset((char*)arena + g0, 0xA5, g1 - g0);
    }
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) { delete m; return fail(SB_ERR_CUDA, "clearing the arena: %s", cudaGetErrorString(e)); }
    s = umma_plan_layers(m, 0);
    if (s != SB_OK) { delete m; return fail(s, "tensor-core planning failed: %s", umma_last_error()); }
    if (m->cfg.flags & SB_FLAG_MODULO_SCHEDULE) {
        // One layer table per sub-iteration: its FC layers address rows [k*B/K, (k+1)*B/K) of the same buffers, the
        // first of them reads / writes the permuted feature buffers; their tensor-core ops are planned for B/K rows.
        const int K = m->cfg.K, Bk = m->B / K;
        const size_t D = (size_t)m->L[m->first_fc].in_f;
        m->full_B = m->B;
        for (int k = 0; k < K; ++k) {
            std::vector<Layer> Lk = m->L;
            const size_t row0 = (size_t)k * Bk;
            for (int i = m->first_fc; i < m->n_layers; ++i) {
                Layer& l = Lk[i];
                if (l.kind != SB_FC_RELU && l.kind != SB_FC && l.kind != SB_DROPOUT) continue;
                l.act += row0 * l.out_per_img * (l.act_dt == SB_DT_F32 ? 4 : m->esz);
                l.dact += row0 * l.out_per_img * m->esz;
                l.um = UmmaLayer{};
            }
            Lk[m->first_fc].in_override = m->mod_x + row0 * D * m->esz;
            Lk[m->first_fc].dbelow_override = m->mod_dx + row0 * D * m->esz;
            m->mod_L.push_back(std::move(Lk));
        }
        for (int k = 0; k < K && s == SB_OK; ++k) {
            std::swap(m->L, m->mod_L[k]);
            m->B = Bk;
            s = umma_plan_layers(m, m->first_fc);
            m->B = m->full_B;
            std::swap(m->L, m->mod_L[k]);
        }
        if (s != SB_OK) { delete m; return fail(s, "tensor-core planning of the sub-batches failed: %s", umma_last_error()); }
    }
    *out = m;
    return SB_OK;
}

sb_status sb_model_destroy(sb_model* m)
{
    if (!m) return fail(SB_ERR_INVALID_ARG, "null model");
    delete m;
    return SB_OK;
}

// One layer's kernels on the chain stream of a pass.  Once a kernel of the same pass precedes it on that stream, a tensor-core
// forward / data-gradient kernel may fetch its weights before it waits for that predecessor (weights_first()): within a pass
// nothing on the chain stream writes parameters -- updates run on other streams behind events, or after the pass.
static sb_status chain_fwd(sb_model* m, int i, cudaStream_t st)
{
    weights_first() = m->st_clean ? 1 : 0;
    const int64_t l0 = m->launches;
    const sb_status s = forward_layer(m, i, st);
    weights_first() = 0;
    if (m->launches > l0) m->st_clean = true;
    return s;
}
static sb_status chain_bwd(sb_model* m, int i, cudaStream_t st, int part)
{
    weights_first() = m->st_clean ? 1 : 0;
    const int64_t l0 = m->launches;
    const sb_status s = backward_layer(m, i, st, part);
    weights_first() = 0;
    if (m->launches > l0) m->st_clean = true;
    return s;
}

sb_status sb_forward_layers(sb_model* m, int32_t first, int32_t last, const void* const* x, const int32_t* const* labels, void* stream)
{
    if (!m) return fail(SB_ERR_INVALID_ARG, "null model");
    if (first < 0 || last >= m->n_layers || first > last) return fail(SB_ERR_INVALID_ARG, "bad layer range %d..%d", first, last);
    if (x || labels) {
        sb_status s = set_inputs(m, x, labels);
        if (s != SB_OK) return s;
    }
    m->pooled_by_conv = -1;     // a pool layer run on its own (or first in the range) computes its output itself
    m->st_clean = false;
    for (int i = first; i <= last; ++i) {
        sb_status s = chain_fwd(m, i, (cudaStream_t)stream);
        if (s != SB_OK) return s;
    }
    m->st_clean = false;
    m->pooled_by_conv = -1;
    return SB_OK;
}

sb_status sb_backward_layers(sb_model* m, int32_t last, int32_t first, void* stream)
{
    if (!m) return fail(SB_ERR_INVALID_ARG, "null model");
    if (first < 0 || last >= m->n_layers || first > last) return fail(SB_ERR_INVALID_ARG, "bad layer range %d..%d", last, first);
    m->st_clean = false;
    for (int i = last; i >= first; --i) {
        sb_status s = chain_bwd(m, i, (cudaStream_t)stream, SIDE_BOTH);
        if (s != SB_OK) return s;
    }
    m->st_clean = false;
    return SB_OK;
}

sb_status sb_forward(sb_model* m, const void* const* x, const int32_t* const* labels, void* stream)
{
    if (!m) return fail(SB_ERR_INVALID_ARG, "null model");
    if (!x || !labels) return fail(SB_ERR_INVALID_ARG, "x or labels is null");
    sb_status s = set_inputs(m, x, labels);
    if (s != SB_OK) return s;
    m->launches = 0;
    m->pooled_by_conv = -1;
    m->st_clean = false;
    for (int i = 0; i < m->n_layers; ++i) {
        s = chain_fwd(m, i, (cudaStream_t)stream);
        if (s != SB_OK) return s;
    }
    m->st_clean = false;
    m->pooled_by_conv = -1;
    m->have_fwd = true;
    return SB_OK;
}

// The weight-side work of layer i (weight / bias gradient, split reduces, folded update) on `wst`; classic = without the
// programmatic-dependent-launch attribute.
static sb_status weight_side(sb_model* m, int i, cudaStream_t wst, bool classic)
{
    pdl_classic() = classic ? 1 : 0;
    const sb_status s = backward_layer(m, i, wst, SIDE_W);
    pdl_classic() = 0;
    return s;
}

// Backward pass; with `fuse_update` the SGD update of each layer's parameters is enqueued on the weight-side
// stream as soon as that layer's gradients are complete and its input gradient (which reads the weights) has
// been computed, so the bandwidth-bound update overlaps the rest of the backward pass.  Element for element the
// update is the one sb_sgd_step does.  Returns *updated = true if the update was done here.
static sb_status backward_pass(sb_model* m, cudaStream_t st, bool fuse_update, float lr, float mu, bool* updated, int hi = -1, int lo = 0)
{
    if (hi < 0) hi = m->n_layers - 1;     // layers hi .. lo, top down
    // The weight-gradient work of a layer (and its split reduce) only has to be finished before the update,
    // while the input-gradient chain is the critical path: the former runs on the model's second stream,
    // ordered by one event per layer ("the gradient w.r.t. this layer's output is ready") and joined at the
    // end.  Profiling and debug-sync modes keep everything on one stream.
    const bool two_streams = m->n_wstreams > 0 && !m->profiling && !m->debug_sync;
    const bool fuse = fuse_update && two_streams;
    if (updated) *updated = fuse;
    m->st_clean = false;
    unsigned used_streams = 0;   // weight streams that received work in this pass (only those are joined)
    bool used_ustream = false;   // likewise the update stream
    for (int i = hi; i >= lo; --i) {
        Layer& l = m->L[i];
        const bool has_params = l.kind == SB_CONV3X3_RELU || l.kind == SB_FC_RELU || l.kind == SB_FC;
        if (two_streams && has_params) {
            // Weight-side kernels of short reductions (FC layers, the 2x2 and 4x4 conv layers) are launched the classic way:
            // launched early, their CTAs sit on SMs waiting for the stream's previous kernel while the input-gradient chain
            // needs those SMs (batch 128 / 256 at CIFAR size: -1.9 % step, the 7-conv net -3.9 %; layers of 8192+ rows: +-0 to +1.9 %
            // without the early launch, so those keep it; so does every layer of a step of long kernels -- ImageNet-size inputs:
            // +0.6 to +1 % without).
            static const long classic_max_rows = (long)tune("SB_WSIDE_CLASSIC_MAX_ROWS", 5000);
            static const long classic_max_input = (long)tune("SB_WSIDE_CLASSIC_MAX_INPUT", 1L << 20);
            const bool classic = (l.kind == SB_CONV3X3_RELU ? (long)m->B * l.H * l.W : (long)m->B) <= classic_max_rows &&
                                 (long)m->B * m->cfg.H * m->cfg.W <= classic_max_input;
            cudaStream_t wst = m->wstreams[i % m->n_wstreams];
            used_streams |= 1u << (i % m->n_wstreams);
            CU_TRY(cudaEventRecord(m->ev_ready[i], st));
            CU_TRY(cudaStreamWaitEvent(wst, m->ev_ready[i], 0));
            // Conv layers in a fused pass: the input-gradient kernel is enqueued first and its event recorded, so that the
            // layer's split reduces on the weight stream can wait for it and apply the update themselves.
            static const bool reduce_updates = tune("SB_REDUCE_SGD", 1) != 0;
            // FC layers whose weight-gradient kernel can carry the update take the same order (SB_FC_WGRAD_UPDATE=0: separate update)
            static const bool fc_wgrad_update = tune("SB_FC_WGRAD_UPDATE", 1) != 0;
            const bool in_reduce = fuse && ((reduce_updates && l.kind == SB_CONV3X3_RELU) ||
                                            (fc_wgrad_update && l.kind != SB_CONV3X3_RELU && !l.narrow && umma_fc_wgrad_can_update(m, i)));
            sb_status s = SB_OK;
            if (in_reduce) {
                s = chain_bwd(m, i, st, SIDE_D);
                if (s != SB_OK) return s;
                CU_TRY(cudaEventRecord(m->ev_dgrad[i], st));
                m->fuse.on = true; m->fuse.lr = lr; m->fuse.mu = mu; m->fuse.ev = m->ev_dgrad[i]; m->fuse.waited = false; m->fuse.covered = 0;
                s = weight_side(m, i, wst, classic);
                m->fuse.on = false;
                if (s != SB_OK) return s;
                if (m->fuse.covered == l.n_w + l.n_b) continue;     // every parameter of the layer has taken its update
                if (m->fuse.covered != 0) return fail(SB_ERR_STATE, "layer %d: update folded into part of its reduces only", i);
            } else {
                s = weight_side(m, i, wst, classic);
                if (s != SB_OK) return s;
                s = chain_bwd(m, i, st, SIDE_D);
                if (s != SB_OK) return s;
            }
            if (fuse) {
                // The update of this layer runs on a third stream: after the layer's gradients are complete (weight
                // stream) and after its input-gradient kernel, which reads the weights the update rewrites (main stream).
                if (!in_reduce) CU_TRY(cudaEventRecord(m->ev_dgrad[i], st));
                CU_TRY(cudaEventRecord(m->ev_wdone[i], wst));
                CU_TRY(cudaStreamWaitEvent(m->ustream, m->ev_dgrad[i], 0));
                CU_TRY(cudaStreamWaitEvent(m->ustream, m->ev_wdone[i], 0));
                used_ustream = true;
                const size_t off = l.p_w, cnt = (l.p_b - l.p_w) + align_up(l.n_b, 64);
                {
                    cudaStream_t st = m->ustream;   // the launch bracket below records on the stream it launches on
                    m->cur_layer = i;
                    L_TRY("sgd", 0.0, (double)cnt * (m->bf16 ? 22.0 : 20.0),
                          launch_sgd(m->Wm + off, m->Vm + off, m->Gm + off, m->Sm ? m->Sm + off : nullptr, cnt, lr, mu, st));
                }
            }
        } else {
            sb_status s = chain_bwd(m, i, st, SIDE_BOTH);
            if (s != SB_OK) return s;
        }
    }
    m->st_clean = false;
    if (two_streams) {
        for (int k = 0; k < m->n_wstreams; ++k) {
            if (!(used_streams & (1u << k))) continue;
            CU_TRY(cudaEventRecord(m->ev_wjoin[k], m->wstreams[k]));
            CU_TRY(cudaStreamWaitEvent(st, m->ev_wjoin[k], 0));
        }
    }
    if (fuse) {
        if (used_ustream) {
            CU_TRY(cudaEventRecord(m->ev_ujoin, m->ustream));
            CU_TRY(cudaStreamWaitEvent(st, m->ev_ujoin, 0));
        }
        m->last_step_launches = m->launches;
    }
    return SB_OK;
}

sb_status sb_backward(sb_model* m, void* stream)
{
    if (!m) return fail(SB_ERR_INVALID_ARG, "null model");
    if (!m->have_fwd) return fail(SB_ERR_STATE, "sb_backward needs a preceding sb_forward");
    return backward_pass(m, (cudaStream_t)stream, false, 0.f, 0.f, nullptr);
}

// forward + backward + update of one iteration, with the update folded into the backward pass when possible
static sb_status whole_step(sb_model* m, const void* const* x, const int32_t* const* labels, float lr, float mu, void* stream)
{
    sb_status s = sb_forward(m, x, labels, stream);
    if (s != SB_OK) return s;
    bool updated = false;
    s = backward_pass(m, (cudaStream_t)stream, true, lr, mu, &updated);
    if (s != SB_OK) return s;
    if (!updated) s = sb_sgd_step(m, lr, mu, stream);
    return s;
}

// One iteration in the modulo layer's own schedule [Modulo Layer]: the conv-side stack runs forward once on all
// R*b rows; the modulo layer copies the feature rows into sub-iteration order (replica r's k-th slice of b/K rows
// -> rows k*B/K + r*b/K ...); the FC stack then runs K sub-iterations (forward, loss with 1/B per row, backward,
// SGD update of the FC parameters), each on B/K rows; the input gradients are copied back into row order and the
// conv-side stack back-propagates once and takes its update.  Everything runs on the caller's stream.
static sb_status modulo_step_direct(sb_model* m, const void* const* x, const int32_t* const* labels, float lr, float momentum, void* stream)
{
    if (!m) return fail(SB_ERR_INVALID_ARG, "null model");
    if (!(m->cfg.flags & SB_FLAG_MODULO_SCHEDULE)) return fail(SB_ERR_STATE, "the model was created without SB_FLAG_MODULO_SCHEDULE");
    if (!x || !labels) return fail(SB_ERR_INVALID_ARG, "x or labels is null");
    if (m->sub_active) return fail(SB_ERR_STATE, "a sub-iteration is in progress");
    cudaStream_t st = (cudaStream_t)stream;
    sb_status s = set_inputs(m, x, labels);
    if (s != SB_OK) return s;
    m->launches = 0;
    m->pooled_by_conv = -1;
    const int ff = m->first_fc, K = m->cfg.K, R = m->cfg.R, b = m->cfg.batch_per_replica, Bk = m->B / K;
    const size_t D = (size_t)m->L[ff].in_f;
    m->st_clean = false;
    for (int i = 0; i < ff; ++i) {
        s = chain_fwd(m, i, st);
        if (s != SB_OK) return s;
    }
    m->cur_layer = ff;
    {
        ModuloCopyArgs a{m->L[ff - 1].act, m->mod_x, D * m->esz, R, b, K, 0, &m->label_tab, m->mod_labels};
        L_TRY("modulo_gather", 0.0, 2.0 * m->B * D * m->esz, launch_modulo_copy(a, st));
    }
    const size_t fc_off = m->L[ff].p_w, fc_cnt = m->P - fc_off;
    for (int k = 0; k < K; ++k) {
        std::swap(m->L, m->mod_L[k]);
        m->B = Bk; m->sub_active = true; m->sub_row0 = k * Bk;
        s = SB_OK;
        m->st_clean = k == 0;     // (the modulo copy precedes the first sub-iteration; the FC update of the one before, every other)
        for (int i = ff; i < m->n_layers && s == SB_OK; ++i) s = chain_fwd(m, i, st);
        for (int i = m->n_layers - 1; i >= ff && s == SB_OK; --i) s = chain_bwd(m, i, st, SIDE_BOTH);
        m->st_clean = false;
        m->B = m->full_B; m->sub_active = false; m->sub_row0 = 0;
        std::swap(m->L, m->mod_L[k]);
        if (s != SB_OK) return s;
        m->cur_layer = -1;
        L_TRY("sgd", 0.0, (double)fc_cnt * (m->bf16 ? 22.0 : 20.0),
              launch_sgd(m->Wm + fc_off, m->Vm + fc_off, m->Gm + fc_off, m->Sm ? m->Sm + fc_off : nullptr, fc_cnt, lr, momentum, st));
    }
    m->cur_layer = ff;
    {
        ModuloCopyArgs a{m->mod_dx, m->L[ff - 1].dact, D * m->esz, R, b, K, 1, nullptr, nullptr};
        L_TRY("modulo_scatter", 0.0, 2.0 * m->B * D * m->esz, launch_modulo_copy(a, st));
    }
    // conv-side stack: the multi-stream backward pass with the per-layer updates folded in, as in the synchronous step
    bool updated = false;
    s = backward_pass(m, st, true, lr, momentum, &updated, ff - 1, 0);
    if (s != SB_OK) return s;
    m->cur_layer = -1;
    if (!updated) L_TRY("sgd", 0.0, (double)fc_off * (m->bf16 ? 22.0 : 20.0), launch_sgd(m->Wm, m->Vm, m->Gm, m->Sm, fc_off, lr, momentum, st));
    m->have_fwd = false;   // the FC activations hold the last sub-iteration only: sb_backward has nothing consistent to use
    m->last_step_launches = m->launches;
    return SB_OK;
}

sb_status sb_sgd_step(sb_model* m, float lr, float momentum, void* stream)
{
    if (!m) return fail(SB_ERR_INVALID_ARG, "null model");
    cudaStream_t st = (cudaStream_t)stream;
    m->cur_layer = -1;
    L_TRY("sgd", 0.0, (double)m->P * (m->bf16 ? 22.0 : 20.0), launch_sgd(m->Wm, m->Vm, m->Gm, m->Sm, m->P, lr, momentum, st));
    m->last_step_launches = m->launches;
    return SB_OK;
}

sb_status sb_refresh_shadow(sb_model* m, void* stream)
{
    if (!m) return fail(SB_ERR_INVALID_ARG, "null model");
    cudaStream_t st = (cudaStream_t)stream;
    if (m->bf16) L_TRY("to_bf16", 0.0, (double)m->P * 6.0, launch_to_bf16(m->Wm, m->Sm, m->P, st));
    return SB_OK;
}

sb_status sb_dropout_seed(sb_model* m, uint64_t seed, uint64_t iteration, void* stream)
{
    if (!m) return fail(SB_ERR_INVALID_ARG, "null model");
    cudaStream_t st = (cudaStream_t)stream;
    m->cur_layer = -1;
    L_TRY("dropout_state", 0.0, 16.0, launch_dropout_state(m->drop_state, 0, seed, (uint32_t)iteration, st));
    return SB_OK;
}

sb_status sb_loss(sb_model* m, void* stream, float* host_loss)
{
    if (!m || !host_loss) return fail(SB_ERR_INVALID_ARG, "null model or host_loss");
    struct { float loss; uint32_t status; } r;
    CU_TRY(cudaMemcpyAsync(&r.loss, m->loss, 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    CU_TRY(cudaMemcpyAsync(&r.status, m->status, 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    CU_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    *host_loss = r.loss;
    if (r.status != DEV_OK) {
        cudaMemsetAsync(m->status, 0, 4, (cudaStream_t)stream);
        cudaStreamSynchronize((cudaStream_t)stream);
        return fail(SB_ERR_TIMEOUT, "a kernel gave up on a bounded wait (device status %u)", r.status);
    }
    return SB_OK;
}

static bool same_ptrs(const PtrTab& a, const PtrTab& b, int n)
{
    for (int i = 0; i < n; ++i)
        if (a.p[i] != b.p[i]) return false;
    return true;
}

// Ends a capture that failed half-way so that the stream is usable again.
static void abandon_capture(cudaStream_t st)
{
    cudaGraph_t g = nullptr;
    cudaStreamEndCapture(st, &g);
    if (g) cudaGraphDestroy(g);
    cudaGetLastError();
}

// An iteration on device-resident inputs replayed as a CUDA graph: the first call runs `step` directly, the second
// captures it, later calls with the same pointers and hyper-parameters are one graph launch.
typedef sb_status (*StepFn)(sb_model*, const void* const*, const int32_t* const*, float, float, void*);
static sb_status graph_replay(sb_model* m, sb_model::StepGraph& G, StepFn step, const void* const* x, const int32_t* const* labels,
                              float lr, float momentum, void* stream)
{
    if (!m) return fail(SB_ERR_INVALID_ARG, "null model");
    if (!x || !labels) return fail(SB_ERR_INVALID_ARG, "x or labels is null");
    cudaStream_t st = (cudaStream_t)stream;
    PtrTab xt{}, lt{};
    for (int r = 0; r < m->cfg.R; ++r) { xt.p[r] = x[r]; lt.p[r] = labels[r]; }
    const bool eager = m->profiling || m->debug_sync || !G.warmed || st == nullptr;
    if (eager) {
        // first use (one-time function attributes are set by the first launches), or a mode that needs every launch visible
        sb_status s = step(m, x, labels, lr, momentum, stream);
        if (s == SB_OK) G.warmed = true;
        return s;
    }
    const bool hit = G.exec && same_ptrs(G.x, xt, m->cfg.R) && same_ptrs(G.labels, lt, m->cfg.R) && G.lr == lr && G.mu == momentum;
    if (!hit) {
        if (G.exec) { cudaGraphExecDestroy(G.exec); G.exec = nullptr; }
        CU_TRY(cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
        sb_status s = step(m, x, labels, lr, momentum, stream);
        if (s != SB_OK) { abandon_capture(st); return s; }
        cudaGraph_t graph = nullptr;
        CU_TRY(cudaStreamEndCapture(st, &graph));
        cudaError_t e = cudaGraphInstantiate(&G.exec, graph, 0);
        cudaGraphDestroy(graph);
        if (e != cudaSuccess) { G.exec = nullptr; return fail(SB_ERR_CUDA, "cudaGraphInstantiate: %s", cudaGetErrorString(e)); }
        G.x = xt; G.labels = lt; G.lr = lr; G.mu = momentum;
    }
    CU_TRY(cudaGraphLaunch(G.exec, st));
    return SB_OK;
}

sb_status sb_graph_step(sb_model* m, const void* const* x, const int32_t* const* labels, float lr, float momentum, void* stream)
{
    if (!m) return fail(SB_ERR_INVALID_ARG, "null model");
    sb_status s = graph_replay(m, m->g_dev, whole_step, x, labels, lr, momentum, stream);
    if (s == SB_OK) m->have_fwd = true;
    return s;
}

sb_status sb_modulo_step(sb_model* m, const void* const* x, const int32_t* const* labels, float lr, float momentum, void* stream)
{
    if (!m) return fail(SB_ERR_INVALID_ARG, "null model");
    if (!(m->cfg.flags & SB_FLAG_MODULO_SCHEDULE)) return fail(SB_ERR_STATE, "the model was created without SB_FLAG_MODULO_SCHEDULE");
    sb_status s = graph_replay(m, m->g_mod, modulo_step_direct, x, labels, lr, momentum, stream);
    if (s == SB_OK) m->have_fwd = false;
    return s;
}

namespace {
// pinned result words, the copy stream and its events: host-side objects made on first use (no device memory)
sb_status host_step_objects(sb_model* m)
{
    if (m->host_res) return SB_OK;
    CU_TRY(cudaHostAlloc((void**)&m->host_res, 6 * sizeof(uint32_t), cudaHostAllocDefault));
    memset(m->host_res, 0, 6 * sizeof(uint32_t));
    CU_TRY(cudaStreamCreateWithFlags(&m->cpstream, cudaStreamNonBlocking));
    for (int k = 0; k < 2; ++k) {
        CU_TRY(cudaEventCreateWithFlags(&m->ev_staged[k], cudaEventDisableTiming));
        CU_TRY(cudaEventCreateWithFlags(&m->ev_done[k], cudaEventDisableTiming));
    }
    return SB_OK;
}
sb_status read_result(sb_model* m, int slot, cudaStream_t st, float* host_loss)
{
    uint32_t status_word;
    memcpy(host_loss, &m->host_res[2 * slot], 4);
    memcpy(&status_word, &m->host_res[2 * slot + 1], 4);
    if (status_word != DEV_OK) {
        cudaMemsetAsync(m->status, 0, 4, st);
        cudaStreamSynchronize(st);
        return fail(SB_ERR_TIMEOUT, "a kernel gave up on a bounded wait (device status %u)", status_word);
    }
    return SB_OK;
}
}  // namespace

sb_status sb_prefetch_host(sb_model* m, const void* host_x, const int32_t* host_labels)
{
    if (!m || !host_x || !host_labels) return fail(SB_ERR_INVALID_ARG, "null argument");
    if (m->n_staged >= 2) return fail(SB_ERR_STATE, "two batches are staged already: consume one with sb_train_step_host first");
    sb_status hs = host_step_objects(m);
    if (hs != SB_OK) return hs;
    // The staging area chosen here is free on the host's side (the iteration that last read it has been launched); on the
    // device the copy waits for that iteration to finish.
    const int buf = m->stage_next;
    const size_t xb = (size_t)m->B * m->in_per_img * m->esz;
    CU_TRY(cudaStreamWaitEvent(m->cpstream, m->ev_done[buf], 0));      // (an event never recorded counts as complete)
    CU_TRY(cudaMemcpyAsync(m->stage_xb[buf], host_x, xb, cudaMemcpyHostToDevice, m->cpstream));
    CU_TRY(cudaMemcpyAsync(m->stage_lb[buf], host_labels, (size_t)m->B * 4, cudaMemcpyHostToDevice, m->cpstream));
    CU_TRY(cudaEventRecord(m->ev_staged[buf], m->cpstream));
    m->staged[m->n_staged++] = sb_model::Staged{host_x, (const void*)host_labels, buf};
    m->stage_next = buf ^ 1;
    return SB_OK;
}

// Launches one iteration from host buffers.  wait = true: synchronises and returns the loss (sb_train_step_host);
// wait = false: returns after the launch and appends the iteration to the flights (sb_train_step_host_async).
static sb_status host_step(sb_model* m, const void* host_x, const int32_t* host_labels, float lr, float momentum, void* stream, bool wait,
                           float* host_loss)
{
    cudaStream_t st = (cudaStream_t)stream;
    sb_status hs = host_step_objects(m);
    if (hs != SB_OK) return hs;
    const size_t xb = (size_t)m->B * m->in_per_img * m->esz;
    // a batch staged by sb_prefetch_host is consumed by the next call, which must name the same host buffers
    const bool pre = m->n_staged > 0;
    int buf = 0;
    if (pre) {
        if (m->staged[0].host_x != host_x || m->staged[0].host_labels != (const void*)host_labels)
            return fail(SB_ERR_STATE, "a batch staged by sb_prefetch_host is pending: the next sb_train_step_host must name its host buffers");
        buf = m->staged[0].buf;
        if (m->slot_busy[buf]) return fail(SB_ERR_STATE, "the iteration that used this staging area has not been collected (sb_train_step_host_wait)");
        m->staged[0] = m->staged[1];
        --m->n_staged;
        CU_TRY(cudaStreamWaitEvent(st, m->ev_staged[buf], 0));
    } else {
        if (m->n_flights > 0) return fail(SB_ERR_STATE, "iterations are in flight: only staged batches may be launched behind them");
        m->stage_next = 1;      // (this call copies into staging area 0 itself: the next prefetch goes to area 1)
    }
    const int slot = pre ? buf : 2;
    const void* xp[MAX_PARTS];
    const int32_t* lp[MAX_PARTS];
    const int b = m->cfg.batch_per_replica;
    for (int r = 0; r < m->cfg.R; ++r) {
        xp[r] = m->stage_xb[buf] + (size_t)r * b * m->in_per_img * m->esz;
        lp[r] = m->stage_lb[buf] + (size_t)r * b;
    }
    sb_model::StepGraph& G = pre ? m->g_pre[buf] : m->g_host;
    const bool eager = m->profiling || m->debug_sync || !m->g_host.warmed || st == nullptr;
    sb_status s = SB_OK;
    bool finished = false;
    float loss = 0.f;
    if (eager) {
        if (!pre) {
            CU_TRY(cudaMemcpyAsync(m->stage_x, host_x, xb, cudaMemcpyHostToDevice, st));
            CU_TRY(cudaMemcpyAsync(m->stage_labels, host_labels, (size_t)m->B * 4, cudaMemcpyHostToDevice, st));
        }
        s = whole_step(m, xp, lp, lr, momentum, stream);
        if (s != SB_OK) return s;
        m->g_host.warmed = true;
        if (pre) CU_TRY(cudaEventRecord(m->ev_done[buf], st));
        s = sb_loss(m, stream, &loss);       // (synchronises: the direct path is the first call and the diagnostic modes)
        finished = true;
    } else {
        // One graph per (host buffers, lr, momentum): H2D copies (unless staged beforehand), the whole iteration, and the
        // loss / status read-back.  A staged batch has one graph per staging area, keyed by lr and momentum only.
        const bool hit = G.exec && (pre || (G.host_x == host_x && G.host_labels == (const void*)host_labels)) && G.lr == lr && G.mu == momentum;
        if (!hit) {
            if (G.exec) { cudaGraphExecDestroy(G.exec); G.exec = nullptr; }
            CU_TRY(cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
            cudaError_t e = cudaSuccess;
            if (!pre) {
                e = cudaMemcpyAsync(m->stage_x, host_x, xb, cudaMemcpyHostToDevice, st);
                if (e == cudaSuccess) e = cudaMemcpyAsync(m->stage_labels, host_labels, (size_t)m->B * 4, cudaMemcpyHostToDevice, st);
            }
            s = e == cudaSuccess ? SB_OK : fail(SB_ERR_CUDA, "capturing the input copies: %s", cudaGetErrorString(e));
            if (s == SB_OK) s = whole_step(m, xp, lp, lr, momentum, stream);
            if (s == SB_OK) {
                e = cudaMemcpyAsync(&m->host_res[2 * slot], m->loss, 8, cudaMemcpyDeviceToHost, st);      // loss and status word
                if (e != cudaSuccess) s = fail(SB_ERR_CUDA, "capturing the read-back: %s", cudaGetErrorString(e));
            }
            if (s != SB_OK) { abandon_capture(st); return s; }
            cudaGraph_t graph = nullptr;
            CU_TRY(cudaStreamEndCapture(st, &graph));
            e = cudaGraphInstantiate(&G.exec, graph, 0);
            cudaGraphDestroy(graph);
            if (e != cudaSuccess) { G.exec = nullptr; return fail(SB_ERR_CUDA, "cudaGraphInstantiate: %s", cudaGetErrorString(e)); }
            G.host_x = host_x; G.host_labels = host_labels; G.lr = lr; G.mu = momentum;
        }
        CU_TRY(cudaGraphLaunch(G.exec, st));
        if (pre) CU_TRY(cudaEventRecord(m->ev_done[buf], st));
        m->have_fwd = true;
        if (wait || !pre) {
            CU_TRY(cudaStreamSynchronize(st));
            s = read_result(m, slot, st, &loss);
            finished = true;
        }
    }
    if (wait) {
        if (host_loss) *host_loss = loss;
        return s;
    }
    sb_model::Flight& f = m->flights[m->n_flights++];
    f.slot = slot; f.finished = finished; f.loss = loss; f.status = s;
    snprintf(f.msg, sizeof(f.msg), "%s", finished && s != SB_OK ? sb_last_error() : "");
    if (!finished) m->slot_busy[slot] = true;
    return SB_OK;
}

sb_status sb_train_step_host(sb_model* m, const void* host_x, const int32_t* host_labels, float lr, float momentum,
                             void* stream, float* host_loss)
{
    if (!m || !host_x || !host_labels || !host_loss) return fail(SB_ERR_INVALID_ARG, "null argument");
    if (m->n_flights > 0) return fail(SB_ERR_STATE, "iterations are in flight: collect them with sb_train_step_host_wait first");
    return host_step(m, host_x, host_labels, lr, momentum, stream, true, host_loss);
}

sb_status sb_train_step_host_async(sb_model* m, const void* host_x, const int32_t* host_labels, float lr, float momentum, void* stream)
{
    if (!m || !host_x || !host_labels) return fail(SB_ERR_INVALID_ARG, "null argument");
    if (m->n_flights >= 2) return fail(SB_ERR_STATE, "two iterations are in flight: collect one with sb_train_step_host_wait first");
    return host_step(m, host_x, host_labels, lr, momentum, stream, false, nullptr);
}

sb_status sb_train_step_host_wait(sb_model* m, void* stream, float* host_loss)
{
    if (!m || !host_loss) return fail(SB_ERR_INVALID_ARG, "null argument");
    if (m->n_flights == 0) return fail(SB_ERR_STATE, "no iteration in flight");
    sb_model::Flight f = m->flights[0];
    m->flights[0] = m->flights[1];
    --m->n_flights;
    if (f.finished) {
        *host_loss = f.loss;
        return f.status == SB_OK ? SB_OK : fail(f.status, "%s", f.msg);
    }
    CU_TRY(cudaEventSynchronize(m->ev_done[f.slot]));
    m->slot_busy[f.slot] = false;
    return read_result(m, f.slot, (cudaStream_t)stream, host_loss);
}

sb_status sb_tensor(sb_model* m, int32_t what, int32_t layer, int32_t part, void** dev_ptr, int64_t shape[4], int32_t* dtype)
{
    char* p = nullptr;
    sb_status s = resolve(m, what, layer, part, &p, shape, dtype, nullptr);
    if (s == SB_OK && dev_ptr) *dev_ptr = p;
    return s;
}

sb_status sb_tensor_read(sb_model* m, int32_t what, int32_t layer, int32_t part, void* host_dst, size_t bytes)
{
    char* p = nullptr;
    size_t nb = 0;
    sb_status s = resolve(m, what, layer, part, &p, nullptr, nullptr, &nb);
    if (s != SB_OK) return s;
    if (!host_dst || bytes != nb) return fail(SB_ERR_INVALID_ARG, "host buffer is null or %zu bytes (tensor has %zu)", bytes, nb);
    CU_TRY(cudaDeviceSynchronize());
    CU_TRY(cudaMemcpy(host_dst, p, nb, cudaMemcpyDeviceToHost));
    return SB_OK;
}

sb_status sb_tensor_write(sb_model* m, int32_t what, int32_t layer, int32_t part, const void* host_src, size_t bytes)
{
    char* p = nullptr;
    size_t nb = 0;
    sb_status s = resolve(m, what, layer, part, &p, nullptr, nullptr, &nb);
    if (s != SB_OK) return s;
    if (!host_src || bytes != nb) return fail(SB_ERR_INVALID_ARG, "host buffer is null or %zu bytes (tensor has %zu)", bytes, nb);
    CU_TRY(cudaDeviceSynchronize());
    CU_TRY(cudaMemcpy(p, host_src, nb, cudaMemcpyHostToDevice));
    return SB_OK;
}

sb_status sb_param_bytes(const sb_model* m, int32_t shard, size_t* bytes)
{
    if (!m || !bytes) return fail(SB_ERR_INVALID_ARG, "null argument");
    if (shard < 0 || shard >= m->cfg.K) return fail(SB_ERR_INVALID_ARG, "shard %d out of range", shard);
    size_t n = 0;
    for (const Layer& l : m->L) {
        if (l.kind == SB_CONV3X3_RELU) n += l.n_w + l.n_b;
        else if (l.kind == SB_FC_RELU || l.kind == SB_FC) {
            // a layer kept whole is held in full by every worker
            size_t rows = l.K == 1 ? (size_t)l.out_f : (size_t)(shard_lo(shard + 1, l.out_f, l.K) - shard_lo(shard, l.out_f, l.K));
            n += rows * l.in_f + rows;
        }
    }
    *bytes = n * 4;
    return SB_OK;
}

sb_status sb_profile_begin(sb_model* m, void* stream)
{
    if (!m) return fail(SB_ERR_INVALID_ARG, "null model");
    (void)stream;
    m->profiling = true;
    m->recs.clear();
    m->ev_used = 0;
    return SB_OK;
}

sb_status sb_profile_end(sb_model* m, void* stream, sb_profile_entry* out, int32_t max_entries, int32_t* n)
{
    if (!m || !out || !n || max_entries < 1) return fail(SB_ERR_INVALID_ARG, "null argument");
    m->profiling = false;
    CU_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    int cnt = 0;
    for (const sb_model::Rec& r : m->recs) {
        float ms = 0.f;
        CU_TRY(cudaEventElapsedTime(&ms, r.e0, r.e1));
        char name[32];
        if ((m->cfg.flags & SB_FLAG_PROFILE_LAYERS) && r.layer >= 0) snprintf(name, sizeof(name), "%.24s#%d", r.tag, r.layer);
        else snprintf(name, sizeof(name), "%.31s", r.tag);
        int k = 0;
        for (; k < cnt; ++k)
            if (strncmp(out[k].name, name, sizeof(out[k].name)) == 0) break;
        if (k == cnt) {
            if (cnt == max_entries) continue;
            memset(&out[k], 0, sizeof(out[k]));
            strncpy(out[k].name, name, sizeof(out[k].name) - 1);
            ++cnt;
        }
        out[k].launches += 1;
        out[k].ms_total += ms;
        out[k].flops += r.flops;
        out[k].bytes += r.bytes;
    }
    m->recs.clear();
    m->ev_used = 0;
    *n = cnt;
    return SB_OK;
}

#ifdef SB_CTA_TIMING
// development builds only (not in the public header): hands the tensor-core kernels a device buffer for per-CTA clock stamps
extern "C" sb_status sb_debug_cta_timing(void* dev_buffer)
{
    umma_set_timing_buffer(dev_buffer);
    return SB_OK;
}
extern "C" sb_status sb_debug_cta_trace(void* dev_buffer)
{
    umma_set_trace_buffer(dev_buffer);
    return SB_OK;
}
#endif

sb_status sb_debug_wait_probe(sb_model* m, int32_t limit_ms, void* stream)
{
    if (!m) return fail(SB_ERR_INVALID_ARG, "null model");
    if (limit_ms < 1 || limit_ms > 1000) return fail(SB_ERR_INVALID_ARG, "limit_ms must be in 1..1000");
    CU_TRY(launch_wait_probe(m->status, (unsigned long long)limit_ms * 1000000ull, (cudaStream_t)stream));
    return SB_OK;
}

sb_status sb_debug_poison(sb_model* m, void* stream)
{
    if (!m) return fail(SB_ERR_INVALID_ARG, "null model");
    // 0xFF bytes are NaN in float and in bfloat16, and an impossible argmax byte
    for (const sb_model::Region& r : m->regions)
        if (r.scratch && r.bytes) CU_TRY(cudaMemsetAsync(m->arena + r.off, 0xFF, r.bytes, (cudaStream_t)stream));
    m->have_fwd = false;
    return SB_OK;
}

sb_status sb_debug_check_guards(sb_model* m, void* stream, int32_t* n_bad, int64_t* first_bad_offset)
{
    if (!m || !n_bad) return fail(SB_ERR_INVALID_ARG, "null argument");
    CU_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    *n_bad = 0;
    if (first_bad_offset) *first_bad_offset = -1;
    std::vector<unsigned char> h;
    for (const sb_model::Region& r : m->regions) {
        const size_t g0 = r.off + r.bytes, g1 = align_up(r.off + r.bytes, 256) + 256;
        h.resize(g1 - g0);
        CU_TRY(cudaMemcpy(h.data(), m->arena + g0, g1 - g0, cudaMemcpyDeviceToHost));
        for (size_t k = 0; k < h.size(); ++k)
            if (h[k] != 0xA5) {
                if (*n_bad == 0 && first_bad_offset) *first_bad_offset = (int64_t)(g0 + k);
                ++*n_bad;
                break;
            }
    }
    return SB_OK;
}

sb_status sb_launch_count(const sb_model* m, int64_t* launches)
{
    if (!m || !launches) return fail(SB_ERR_INVALID_ARG, "null argument");
    *launches = m->last_step_launches;
    return SB_OK;
}

}  // extern "C"
