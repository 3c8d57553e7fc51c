// Host-side partitioning of a sequential CNN for hybrid data / model parallelism, and the exchange schedule of one
// MP group.  No CUDA call is made here: both entry points run on a machine without a GPU.
//
// sb_partition restates the paper's layer-partitioning walk [Listing 1 "Layer Partitioning"; Layer Partitioning
// paragraph]: it tracks the width of the previous layer's output as one worker holds it (dim) and in full (dimF),
// leaves reshape / convolution / pooling layers whole (they only pass their output size on, and refuse a partitioned
// input), splits fully-connected layers by output column into K shards unless the layer is marked "whole" (the
// outcome of the paper's computation-to-communication test, for which it gives no formula), puts a MODULO node in
// front of the first split layer whose input is whole and a SHARD node in front of every layer -- the loss included --
// whose input arrives partitioned.  ReLU is part of the FC kinds here and follows the partitioned width; so does a
// dropout layer (the listing's DROPOUT | RELU case: dim and dimF pass through unchanged).
//
// Reading of the listing's LINEAR case: as printed it overwrites dimF with the layer's output width BEFORE comparing
// dim with dimF; the surrounding text compares the two widths of the layer's INPUT ("if the input dimension has been
// partitioned, a shard layer is inserted"), which is what is done here.
//
// sb_exchange_plan lists, for N = R workers arranged in R / K MP groups of K = mp workers each [Group MP Extension], every
// block of every matrix that has to travel between two workers in one synchronous iteration [Modulo Layer and Shard
// Layer paragraphs and their figures]: the modulo layer's gather of feature rows and the return of gradient rows, the
// shard layer's gather of column slices and the reduce of gradient column slices -- all of them inside one group --
// and the two parameter reduces [Distributed Machine Learning: reduce; Implementation]: the conv stack over all N
// workers, and each FC shard over the workers that hold the same shard in the other groups.  Worker p belongs to group
// gid = p / mp and is data replica p and model shard off = p % mp of that group (the lost figure's mapping, taken from
// the text: the group a worker belongs to, and its offset inside it); with R = K there is a single group, with K = 1
// the schedule is pure data parallelism.
#include "../../include/splitbrain.h"

#include <cstdarg>
#include <cstdio>
#include <vector>

namespace {

thread_local char g_msg[256] = "";
sb_status fail(sb_status s, const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_msg, sizeof(g_msg), fmt, ap);
    va_end(ap);
    return s;
}

bool is_fc(int kind) { return kind == SB_FC_RELU || kind == SB_FC || kind == SB_FC_RELU_WHOLE || kind == SB_FC_WHOLE; }
bool is_whole(int kind) { return kind == SB_FC_RELU_WHOLE || kind == SB_FC_WHOLE; }
int64_t lo(int j, int64_t out, int K) { return ((int64_t)j * out) / K; }     // c_j = floor(j * out / K)

sb_status walk(const sb_layer* layers, int32_t n, const sb_config* cfg, std::vector<sb_plan_node>& net)
{
    if (!layers || !cfg || n <= 0) return fail(SB_ERR_INVALID_ARG, "null layers/config or empty layer list");
    if (cfg->K < 1 || cfg->H < 1 || cfg->W < 1 || cfg->C < 1) return fail(SB_ERR_SHAPE, "H, W, C and K must be positive");
    const int K = cfg->K;
    int H = cfg->H, W = cfg->W, C = cfg->C;
    bool flat = false;                          // a fully-connected layer has flattened the feature map
    bool gathered = false;                      // a modulo node has been placed: every worker sees all rows from there on
    int64_t dim = (int64_t)H * W * C, dimF = dim;
    auto push = [&](int node, int layer, int shards, int64_t d, int64_t dF) {
        sb_plan_node nd{};
        nd.node = node; nd.layer = layer; nd.shards = shards; nd.dim = d; nd.dimF = dF;
        net.push_back(nd);
    };
    for (int i = 0; i < n; ++i) {
        const int kind = layers[i].kind, out = layers[i].out;
        if (kind == SB_CONV3X3_RELU || kind == SB_MAXPOOL2) {
            // never partitioned: passes its output size on, and cannot take a partitioned input
            if (flat) return fail(SB_ERR_SHAPE, "layer %d: convolution / pooling after a fully-connected layer", i);
            if (dim != dimF) return fail(SB_ERR_UNSUPPORTED, "layer %d: partitioned input unsupported", i);
            if (kind == SB_CONV3X3_RELU) {
                if (out < 1) return fail(SB_ERR_SHAPE, "layer %d: Cout must be positive", i);
                C = out;
            } else {
                if (H % 2 || W % 2) return fail(SB_ERR_SHAPE, "layer %d: pooling needs even H and W (got %dx%d)", i, H, W);
                H /= 2; W /= 2;
            }
            dim = dimF = (int64_t)H * W * C;
            push(SB_NODE_LAYER, i, 1, dim, dimF);
        } else if (is_fc(kind)) {
            if (out < 1) return fail(SB_ERR_SHAPE, "layer %d: FC width must be positive", i);
            const bool split = K > 1 && !is_whole(kind);
            if (split && K > out) return fail(SB_ERR_SHAPE, "layer %d: K=%d exceeds the FC width %d", i, K, out);
            if (dim == dimF) {
                if (split && !gathered) { push(SB_NODE_MODULO, i, K, dimF, dimF); gathered = true; }   // first split layer on a whole input
            } else {
                push(SB_NODE_SHARD, i, K, dimF, dimF);                   // input arrives as column slices: gather it
            }
            flat = true;
            dimF = out;
            dim = split ? (out + K - 1) / K : out;                       // one K-th of the width (the widest shard when K does not divide out)
            push(SB_NODE_LAYER, i, split ? K : 1, dim, dimF);
        } else if (kind == SB_DROPOUT) {
            // one-to-one functional layer: adapts to the (partitioned) width of the layer below, dim and dimF pass through,
            // no modulo or shard node in front of it
            if (i == 0 || !(layers[i - 1].kind == SB_FC_RELU || layers[i - 1].kind == SB_FC_RELU_WHOLE))
                return fail(SB_ERR_UNSUPPORTED, "layer %d: dropout must follow an FC + ReLU layer", i);
            if (out < 1 || out > 65535) return fail(SB_ERR_SHAPE, "layer %d: drop probability must be 1..65535 (units of 1/65536)", i);
            push(SB_NODE_LAYER, i, dim != dimF ? K : 1, dim, dimF);
        } else if (kind == SB_SOFTMAX_XENT) {
            if (dim != dimF) push(SB_NODE_SHARD, i, K, dimF, dimF);      // the loss needs the full width
            dim = dimF;
            push(SB_NODE_LAYER, i, 1, dim, dimF);
        } else {
            return fail(SB_ERR_INVALID_ARG, "layer %d: unknown kind %d", i, kind);
        }
    }
    return SB_OK;
}

}  // namespace

extern "C" const char* sb_partition_last_error(void) { return g_msg; }

extern "C" sb_status sb_partition(const sb_layer* layers, int32_t n, const sb_config* cfg, sb_plan_node* out, int32_t max_nodes,
                                  int32_t* n_nodes)
{
    if (!n_nodes) return fail(SB_ERR_INVALID_ARG, "null n_nodes");
    std::vector<sb_plan_node> net;
    sb_status s = walk(layers, n, cfg, net);
    if (s != SB_OK) return s;
    *n_nodes = (int32_t)net.size();
    if (!out) return SB_OK;                                              // size query
    if ((int32_t)net.size() > max_nodes) return fail(SB_ERR_INVALID_ARG, "plan has %zu nodes, room for %d", net.size(), max_nodes);
    for (size_t k = 0; k < net.size(); ++k) out[k] = net[k];
    return SB_OK;
}

extern "C" sb_status sb_exchange_plan(const sb_layer* layers, int32_t n, const sb_config* cfg, sb_exchange_msg* out, int32_t max_msgs,
                                      int32_t* n_msgs)
{
    if (!n_msgs) return fail(SB_ERR_INVALID_ARG, "null n_msgs");
    std::vector<sb_plan_node> net;
    sb_status s = walk(layers, n, cfg, net);
    if (s != SB_OK) return s;
    if (cfg->R < 1 || cfg->R % cfg->K != 0)
        return fail(SB_ERR_UNSUPPORTED, "the R (%d) workers form groups of K (%d): R must be a multiple of K", cfg->R, cfg->K);
    if (cfg->batch_per_replica < 1) return fail(SB_ERR_SHAPE, "batch_per_replica must be positive");
    const int mp = cfg->K, N = cfg->R, G = N / mp;                    // group size, workers, groups
    const int64_t b = cfg->batch_per_replica, Bg = b * mp;             // rows one worker owns, rows one group works on
    std::vector<sb_exchange_msg> fwd;
    std::vector<std::vector<sb_exchange_msg>> bwd_blocks;      // one block per node, in forward order
    auto msg = [&](int kind, int layer, int pass, int src, int dst, int64_t r0, int64_t r1, int64_t c0, int64_t c1, int64_t width) {
        sb_exchange_msg m{};
        m.kind = kind; m.layer = layer; m.pass = pass; m.src = src; m.dst = dst;
        m.row0 = r0; m.row1 = r1; m.col0 = c0; m.col1 = c1; m.width = width;
        return m;
    };
    bool gathered = false;      // the modulo layer has run: every worker holds all rows of its group from here on
    for (size_t k = 0; k < net.size(); ++k) {
        const sb_plan_node& nd = net[k];
        bwd_blocks.emplace_back();
        std::vector<sb_exchange_msg>& bwd_rev = bwd_blocks.back();
        if (nd.node == SB_NODE_MODULO) {
            // forward: worker p owns rows [p*b, (p+1)*b) of the feature matrix and sends them to every other worker of its
            // group; backward: worker src holds a full-width partial gradient for ALL rows of the group and returns dst's rows
            // to their owner, which sums the mp partial results in worker order
            for (int gid = 0; gid < G; ++gid)
                for (int so = 0; so < mp; ++so)
                    for (int d_o = 0; d_o < mp; ++d_o) {
                        if (so == d_o) continue;
                        const int src = gid * mp + so, dst = gid * mp + d_o;
                        fwd.push_back(msg(SB_X_GATHER_ROWS, nd.layer, 0, src, dst, src * b, (src + 1) * b, 0, nd.dimF, nd.dimF));
                        bwd_rev.push_back(msg(SB_X_REDUCE_ROWS, nd.layer, 1, src, dst, dst * b, (dst + 1) * b, 0, nd.dimF, nd.dimF));
                    }
            gathered = true;
        } else if (nd.node == SB_NODE_SHARD) {
            // the layer below (nd.layer - 1) is split: the worker at offset o holds columns [c_o, c_{o+1}) of its group's
            // [Bg, width] output
            const int below = nd.layer - 1;
            const int64_t width = nd.dimF;
            const bool consumer_split = layers[nd.layer].kind == SB_FC_RELU || layers[nd.layer].kind == SB_FC;
            for (int gid = 0; gid < G; ++gid)
                for (int so = 0; so < mp; ++so)
                    for (int d_o = 0; d_o < mp; ++d_o) {
                        if (so == d_o) continue;
                        const int src = gid * mp + so, dst = gid * mp + d_o;
                        const int64_t r0 = gid * Bg, r1 = (gid + 1) * Bg;
                        fwd.push_back(msg(SB_X_GATHER_COLS, below, 0, src, dst, r0, r1, lo(so, width, mp), lo(so + 1, width, mp), width));
                        // backward: a split consumer computes a full-width partial input gradient on every worker; the slice that
                        // belongs to worker dst travels there and is summed in worker order.  A whole consumer (and the loss, which
                        // every worker evaluates on the full logits) yields the same full gradient everywhere in the group: each
                        // worker just keeps its own column slice, nothing travels.
                        if (consumer_split)
                            bwd_rev.push_back(msg(SB_X_REDUCE_COLS, below, 1, src, dst, r0, r1, lo(d_o, width, mp), lo(d_o + 1, width, mp), width));
                    }
        } else {
            const int kind = layers[nd.layer].kind;
            // parameters that every worker holds AND trains on its own rows are reduced over all N workers: the conv stack, and
            // an FC layer kept whole below the modulo layer (every FC layer when K = 1).
            const bool dp_params = kind == SB_CONV3X3_RELU || (is_fc(kind) && nd.shards == 1 && !gathered);
            if (dp_params && N > 1) bwd_rev.push_back(msg(SB_X_ALLREDUCE, nd.layer, 1, -1, -1, 0, 0, 0, 0, 0));
            // above the modulo layer a group trains its FC parameters on the group's rows only: shard o is summed over the
            // workers at offset o of every group (src = o); a layer kept whole there is equal on all workers of a group and
            // is summed over the groups likewise (src = -1: every offset)
            if (is_fc(kind) && !dp_params && G > 1) {
                if (nd.shards > 1)
                    for (int o = 0; o < mp; ++o)
                        bwd_rev.push_back(msg(SB_X_ALLREDUCE_GROUPS, nd.layer, 1, o, -1, 0, 0, lo(o, nd.dimF, mp), lo(o + 1, nd.dimF, mp), nd.dimF));
                else
                    bwd_rev.push_back(msg(SB_X_ALLREDUCE_GROUPS, nd.layer, 1, -1, -1, 0, 0, 0, nd.dimF, nd.dimF));
            }
        }
    }
    std::vector<sb_exchange_msg> all(fwd);
    for (size_t k = bwd_blocks.size(); k-- > 0;)                              // the backward pass visits the nodes in reverse
        for (const sb_exchange_msg& m : bwd_blocks[k]) all.push_back(m);
    *n_msgs = (int32_t)all.size();
    if (!out) return SB_OK;
    if ((int32_t)all.size() > max_msgs) return fail(SB_ERR_INVALID_ARG, "plan has %zu messages, room for %d", all.size(), max_msgs);
    for (size_t k = 0; k < all.size(); ++k) out[k] = all[k];
    return SB_OK;
}
