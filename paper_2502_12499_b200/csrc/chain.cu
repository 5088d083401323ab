// Layer-chain description, workspace layout and the step executor (Algorithms 1, 2 and 4).
//
// The executor is host control flow only: it walks the units, asks the arena where each d_i lives,
// and launches kernels.  The same walk with launches disabled is the arena dry run.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstring>

#include "internal.h"

namespace ckpt {

struct Shape { int h, w, c; };

struct Unit {
    ckpt_unit_desc desc;
    Shape in, out;
    int param_first = 0, n_params = 0;
    int64_t stats_off = 0;       // float offset of this unit's saved batch statistics
    bool in_pending = false;     // the unit's input is a conv+BN+ReLU unit's stored output (normalisation applied on the way in)
    int64_t blk_off = 0;         // residual block: offset of a region of its own when every block keeps its interiors
    ConvGeom geom;               // conv / fc as a convolution
    // bottleneck block: its four convolutions (1x1, 3x3 with the stride, 1x1, projection 1x1 with the stride)
    ConvGeom g1, g2, g3, gp;
};

struct ParamInfo { int64_t unit, elems; int32_t dtype; };

// One captured step: the launch sequence of run_step for a fixed set of arguments.
struct StepGraph {
    uint64_t key = 0;
    std::vector<uint64_t> args;          // the argument set itself: a recording is replayed only for an exact match
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    int64_t peak = 0, extent = 0, launches = 0, recomputed = 0;
    uint64_t last_use = 0;
};

}  // namespace ckpt

struct ckpt_chain {
    std::vector<ckpt::Unit> units;       // units[0] is unit 1
    std::vector<int64_t> d;              // d_0..d_n, bytes
    std::vector<ckpt::Shape> shapes;
    std::vector<ckpt::ParamInfo> params;
    int64_t batch = 0;
    int dtype = 0, loss = 0, impl = 0;
    // workspace layout (byte offsets)
    int64_t max_d = 0, off_g0 = 0, off_g1 = 0, off_z = 0, off_scr = 0, scr_bytes = 0, off_stats = 0,
            off_misc = 0, off_blk = 0, blk_bytes = 0, blk_lean_bytes = 0, ws_bytes = 0;
    // Algorithm 1 taken literally (ckpt_chain_set_keep_interiors): every residual block keeps its interior tensors
    // from the forward to the backward pass in a region of its own, blk_sum bytes in all
    int keep_interiors = 0;
    int64_t blk_sum = 0, z_bytes = 0;
    // graph replay: steps captured once per distinct argument set (pointers, plan, policy)
    int use_graph = 0;
    std::vector<ckpt::StepGraph> graphs;
    std::vector<uint64_t> seen_keys;     // argument sets that have run once without capture
    uint64_t use_clock = 0;              // least-recently-used order of the recordings
    // verification aids (off by default)
    char* tap = nullptr;                 // device: where the step leaves every inter-unit gradient (ckpt_chain_set_gradient_tap)
    int64_t tap_bytes = 0;
    int selftest_wait = 0;               // the next steps include one kernel whose bounded wait runs out
    float sgd_lr = 0.f;                  // != 0: every parameter takes w - lr * g as soon as its gradient is complete
    void* host_result = nullptr;         // pinned: loss (8 bytes) and status word of the last step
    cudaStream_t capture_stream = nullptr;   // recording happens here (the caller's stream may be the default one,
                                             // which cannot record); replays run on the caller's stream
    // input staging (ckpt_chain_stage_batch): copies run on a stream of the chain's own, the step that is given a
    // staged batch waits for the copy's event on its stream
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t stage_event[2] = {nullptr, nullptr};
    const void* stage_batch[2] = {nullptr, nullptr};
    bool stage_pending[2] = {false, false};
    ~ckpt_chain();
};

namespace ckpt {

static int out_size(int h, int k, int stride, int pad) { return (h + 2 * pad - k) / stride + 1; }

static int check_conv(const ckpt_unit_desc& u, const Shape& in, int64_t idx) {
    if (u.k < 1 || u.stride < 1 || u.pad < 0 || u.c_out < 1) { set_error("unit %lld: bad conv parameters", (long long)idx); return CKPT_E_BAD_ARG; }
    if (u.c_in != in.c) { set_error("unit %lld: c_in %d != incoming channels %d", (long long)idx, u.c_in, in.c); return CKPT_E_BAD_ARG; }
    if (in.h + 2 * u.pad < u.k || in.w + 2 * u.pad < u.k) { set_error("unit %lld: window larger than input", (long long)idx); return CKPT_E_BAD_ARG; }
    return CKPT_OK;
}

static bool use_tc(const ckpt_chain* ch, const ConvGeom& g) {
    return ch->impl == 0 && tc_conv_supported(ch->dtype, g);
}

// ------------------------------------------------------------------------------------------------
// executor
// ------------------------------------------------------------------------------------------------
struct StepCtx {
    ckpt_chain* ch;
    const uint8_t* is_ckpt;
    int policy;
    bool dry;
    char* arena_base;
    char* ws;
    void* const* params;
    void* const* grads;
    const void* batch;
    const int32_t* labels;
    cudaStream_t stream;
    Arena* arena;
    int64_t recomputed = 0;
    int64_t* stage_trace = nullptr;     // optional: live arena bytes at the end of each of the 2n+2 stages
    void* host_result = nullptr;        // capture: pinned destination of the loss and the status word (no wait)
    char* act_buf = nullptr;            // where the activated copy of a unit's input goes (null: the workspace's own buffer)
    int64_t act_cap = 0;                // its capacity in bytes
    int* status() const { return (int*)(ws + ch->off_misc + 64); }
};

static const int64_t kGradId = 1000000007;   // arena id of the per-segment gradient buffer

// Workspace layout per schedule: Algorithm 4's schedule stops before the tail of the block region and the buffer of
// the activated copy; a store-all step that keeps block interiors has one block region per residual block.
static bool keeps_interiors(const ckpt_chain* ch, int policy) { return ch->keep_interiors && policy == CKPT_POLICY_STORE_ALL; }
static int64_t z_offset(const ckpt_chain* ch, int policy) { return keeps_interiors(ch, policy) ? ch->off_blk + ch->blk_sum : ch->off_z; }
static int64_t workspace_need(const ckpt_chain* ch, int policy) {
    if (policy == CKPT_POLICY_DYNAMIC) return ch->off_blk + ch->blk_lean_bytes;
    return z_offset(ch, policy) + ch->z_bytes;
}

static int conv_forward_any(StepCtx& c, const ConvGeom& g, const void* x, const void* w, void* z,
                            const float* bias, int relu) {
    if (use_tc(c.ch, g))
        return tc_conv_fwd(g, x, w, z, bias, relu, c.ws + c.ch->off_scr, c.ch->scr_bytes, c.status(), c.stream);
    if (c.ch->impl == 0 && !bias && !relu && tc_first_conv_supported(c.ch->dtype, g))
        return tc_first_conv_fwd(g, x, w, z, c.status(), c.stream);
    if (c.ch->impl == 0 && !bias && !relu && stem_conv_supported(c.ch->dtype, g))
        return stem_conv_fwd(g, x, w, z, c.status(), c.stream);
    return simt_conv_fwd(c.ch->dtype, g, x, w, z, bias, relu, c.stream);
}
static int conv_dgrad_any(StepCtx& c, const ConvGeom& g, const void* dz, const void* w, void* dx) {
    if (use_tc(c.ch, g))
        return tc_conv_dgrad(g, dz, w, dx, c.ws + c.ch->off_scr, c.ch->scr_bytes, c.status(), c.stream);
    return simt_conv_dgrad(c.ch->dtype, g, dz, w, dx, c.stream);
}
static int conv_wgrad_any(StepCtx& c, const ConvGeom& g, const void* dz, const void* x, float* dw) {
    if (c.ch->impl == 0 && small_conv_supported(c.ch->dtype, g))
        return small_conv_wgrad(g, dz, x, dw, c.ws + c.ch->off_scr, c.ch->scr_bytes, c.status(), c.stream);
    if (c.ch->impl == 0 && stem_conv_supported(c.ch->dtype, g))
        return stem_conv_wgrad(g, dz, x, dw, c.ws + c.ch->off_scr, c.ch->scr_bytes, c.status(), c.stream);
    if (use_tc(c.ch, g))
        return tc_conv_wgrad(g, dz, x, dw, c.ws + c.ch->off_scr, c.ch->scr_bytes, c.status(), c.stream);
    return simt_conv_wgrad(c.ch->dtype, g, dz, x, dw, c.ws + c.ch->off_scr, c.ch->scr_bytes, c.stream);
}

// "Update w_i with g_i" (Algorithms 1, 2, 4), when a learning rate is set.  param = index of the parameter tensor.
static SgdUpdate sgd_of(StepCtx& c, int param) {
    SgdUpdate u;
    if (c.ch->sgd_lr != 0.f) { u.w = c.params[param]; u.lr = c.ch->sgd_lr; u.dtype = c.ch->params[param].dtype; }
    return u;
}
static int sgd_step(StepCtx& c, int param) {
    if (c.ch->sgd_lr == 0.f) return CKPT_OK;
    return sgd_update(sgd_of(c, param), (const float*)c.grads[param], c.ch->params[param].elems, c.stream);
}
// Weight gradient and input gradient of one convolution.  Without an update: wgrad, then dgrad.  With one the filter
// changes as soon as its gradient is summed, so the input gradient (which reads the filter) runs first.
static int conv_backward_pair(StepCtx& c, const ConvGeom& g, const void* dz, const void* x, const void* w, int param, void* dx) {
    int rc;
    const bool sgd = c.ch->sgd_lr != 0.f;
    if (sgd && dx && (rc = conv_dgrad_any(c, g, dz, w, dx))) return rc;
    const bool stem = c.ch->impl == 0 && stem_conv_supported(c.ch->dtype, g);
    const bool tc_path = !(c.ch->impl == 0 && small_conv_supported(c.ch->dtype, g)) && !stem && use_tc(c.ch, g);
    if (sgd && stem) {
        rc = stem_conv_wgrad(g, dz, x, (float*)c.grads[param], c.ws + c.ch->off_scr, c.ch->scr_bytes, c.status(), c.stream, sgd_of(c, param));
        if (rc) return rc;
    } else if (sgd && tc_path) {
        rc = tc_conv_wgrad(g, dz, x, (float*)c.grads[param], c.ws + c.ch->off_scr, c.ch->scr_bytes, c.status(), c.stream, sgd_of(c, param));
        if (rc) return rc;
    } else {
        if ((rc = conv_wgrad_any(c, g, dz, x, (float*)c.grads[param]))) return rc;
        if ((rc = sgd_step(c, param))) return rc;
    }
    if (!sgd && dx && (rc = conv_dgrad_any(c, g, dz, w, dx))) return rc;
    return CKPT_OK;
}

// Convolution followed by the batch statistics of its stored output.  The tensor-core kernels gather the
// partial sums in their epilogue; every other shape takes a separate pass over z.
static int conv_with_statistics(StepCtx& c, const ConvGeom& g, const void* x, const void* w, void* z, const float* gamma,
                                const float* beta, float* stats) {
    const int dt = c.ch->dtype;
    const int64_t rows = (int64_t)g.n * g.ho * g.wo;
    char* scr = c.ws + c.ch->off_scr;
    int rc;
    if (use_tc(c.ch, g) || (c.ch->impl == 0 && (tc_first_conv_supported(dt, g) || stem_conv_supported(dt, g)))) {
        int blocks = 0;
        if (use_tc(c.ch, g)) rc = tc_conv_fwd_stats(g, x, w, z, (float*)scr, &blocks, c.status(), c.stream, c.ch->scr_bytes);
        else if (stem_conv_supported(dt, g)) rc = stem_conv_fwd(g, x, w, z, c.status(), c.stream, (float*)scr, &blocks);
        else rc = tc_first_conv_fwd(g, x, w, z, c.status(), c.stream, (float*)scr, &blocks);
        if (rc) return rc;
        if (blocks > 0) return bn_statistics_from_partials((const float*)scr, blocks, rows, g.cout, gamma, beta, stats, c.stream);
    } else if ((rc = conv_forward_any(c, g, x, w, z, nullptr, 0))) {
        return rc;
    }
    return bn_statistics(dt, rows, g.cout, z, gamma, beta, stats, scr, c.stream);
}

// A conv+BN+ReLU unit stores its convolution output *before* normalisation as d_i; normalisation and
// ReLU (fixed by the batch statistics saved next to the parameters) are applied by whoever reads
// d_i.  The unit's backward then has everything it needs - its input, its own pre-normalisation
// tensor - without re-running the convolution, and d_i keeps the size the planner was given.
static bool pending_act(const ckpt_chain* ch, int64_t j) {
    return j >= 1 && ch->units[j - 1].desc.kind == CKPT_UNIT_CONV_BN_RELU;
}
static float* stats_of(StepCtx& c, int64_t j) {
    return (float*)(c.ws + c.ch->off_stats) + c.ch->units[j - 1].stats_off;
}
static int64_t rows_of(const ckpt_chain* ch, int64_t j) { return ch->batch * ch->shapes[j].h * ch->shapes[j].w; }

// The activated form of d_j: d_j itself, or a materialised copy in the workspace.
static int activated(StepCtx& c, int64_t j, const void* raw, const void** out) {
    *out = raw;
    if (!pending_act(c.ch, j)) return CKPT_OK;
    void* xbuf = c.act_buf ? c.act_buf : c.ws + z_offset(c.ch, c.policy);
    *out = xbuf;
    return bn_apply(c.ch->dtype, rows_of(c.ch, j), c.ch->shapes[j].c, raw, stats_of(c, j), 1, xbuf, c.stream);
}

// ---------------------------------------------------------------------------------------------
// Bottleneck block (ResNet v1.5): z1 = conv1x1(x), a = relu(bn1(z1)), z2 = conv3x3_stride(a),
// b = relu(bn2(z2)), z3 = conv1x1(b), shortcut = x or bn_p(conv1x1_stride(x)), y = relu(bn3(z3) + shortcut).
// Only y is chain data; every interior tensor lives in the block region of the workspace and is
// re-derived from x at the start of the block's backward.
// ---------------------------------------------------------------------------------------------
struct BlockBuffers {
    char *z1, *a, *da, *z2, *b, *db, *z3, *zp, *t0, *t1, *dxs;
    float *s1, *s2, *s3, *sp;       // statistics blocks of the four normalisations
};
static BlockBuffers block_buffers(StepCtx& c, const Unit& u) {
    const int64_t es = dtype_size(c.ch->dtype);
    const int64_t in_px = c.ch->batch * u.in.h * u.in.w, out_px = c.ch->batch * u.out.h * u.out.w;
    const int64_t m_in = align_up(in_px * u.desc.mid * es, 256), m_out = align_up(out_px * u.desc.mid * es, 256);
    const int64_t c_out = align_up(out_px * u.out.c * es, 256);
    BlockBuffers B;
    char* p = c.ws + c.ch->off_blk + (keeps_interiors(c.ch, c.policy) ? u.blk_off : 0);
    const bool project = (u.desc.flags & 2) != 0;
    B.z1 = p; p += m_in; B.a = p; p += m_in; B.da = p; p += m_in;
    B.z2 = p; p += m_out; B.b = p; p += m_out; B.db = p; p += m_out;
    // projection branch: its pre-normalisation output and the gradient with respect to the block's input through it
    B.zp = project ? p : nullptr; if (project) p += c_out;
    B.dxs = project ? p : nullptr; if (project) p += align_up(in_px * u.in.c * es, 256);
    // z3 last: where an idle gradient buffer is at hand (Algorithm 4's schedule, see run_step) z3 lives there and
    // the block region ends here
    if (c.act_buf && !u.in_pending && c.act_cap >= c_out) B.z3 = c.act_buf;
    else B.z3 = p;
    // the gradients with respect to z3 and zp are written over z3 and zp themselves (the batch-norm backward reads an
    // element of z and of the incoming gradient and writes the same element; nothing reads z3 or zp afterwards)
    B.t1 = B.z3; B.t0 = B.zp;
    float* st = (float*)(c.ws + c.ch->off_stats) + u.stats_off;
    B.s1 = st; B.s2 = st + 4 * u.desc.mid; B.s3 = st + 8 * u.desc.mid; B.sp = B.s3 + 4 * u.out.c;
    return B;
}

// z1, a, z2, b, z3 (and zp) with their statistics; the residual join is left to the caller.
// have_stats: the block's four statistics blocks are those of this very input (they were written by the unit's last
// forward, original or recomputed, and every unit has a block of its own), so the backward's re-derivation of the
// interior tensors runs the convolutions without gathering sums and skips the finalize steps; the tensors come out
// bit-identical (same kernels, same reduction order).
static int block_interiors(StepCtx& c, const Unit& u, const void* x, const BlockBuffers& B, bool have_stats = false) {
    const int dt = c.ch->dtype;
    void* const* p = c.params + u.param_first;
    const int64_t in_px = c.ch->batch * u.in.h * u.in.w, out_px = c.ch->batch * u.out.h * u.out.w;
    const int mid = u.desc.mid;
    int rc;
    auto conv = [&](const ConvGeom& g, const void* in, int w_index, void* z, float* stats) {
        if (have_stats) return conv_forward_any(c, g, in, p[w_index], z, nullptr, 0);
        return conv_with_statistics(c, g, in, p[w_index], z, (const float*)p[w_index + 1], (const float*)p[w_index + 2], stats);
    };
    if ((rc = conv(u.g1, x, 0, B.z1, B.s1))) return rc;
    if ((rc = bn_apply(dt, in_px, mid, B.z1, B.s1, 1, B.a, c.stream))) return rc;
    if ((rc = conv(u.g2, B.a, 3, B.z2, B.s2))) return rc;
    if ((rc = bn_apply(dt, out_px, mid, B.z2, B.s2, 1, B.b, c.stream))) return rc;
    if ((rc = conv(u.g3, B.b, 6, B.z3, B.s3))) return rc;
    if (u.desc.flags & 2) {
        if ((rc = conv(u.gp, x, 9, B.zp, B.sp))) return rc;
    }
    return CKPT_OK;
}

static int block_forward(StepCtx& c, const Unit& u, const void* x, void* y, bool have_stats = false) {
    const BlockBuffers B = block_buffers(c, u);
    int rc = block_interiors(c, u, x, B, have_stats);
    if (rc) return rc;
    const bool project = (u.desc.flags & 2) != 0;
    return bn_add_relu(c.ch->dtype, c.ch->batch * u.out.h * u.out.w, u.out.c, B.z3, B.s3, project ? (const void*)B.zp : x,
                       project ? B.sp : nullptr, y, c.stream);
}

// g_in = dL/dy (overwritten), g_out = dL/dx or null.
static int block_backward(StepCtx& c, const Unit& u, const void* x, const void* y, void* g_in, void* g_out) {
    const int dt = c.ch->dtype;
    const BlockBuffers B = block_buffers(c, u);
    void* const* p = c.params + u.param_first;
    void* const* g = c.grads + u.param_first;
    const int pf = u.param_first;
    char* scr = c.ws + c.ch->off_scr;
    const int64_t in_px = c.ch->batch * u.in.h * u.in.w, out_px = c.ch->batch * u.out.h * u.out.w;
    const int mid = u.desc.mid, co = u.out.c;
    const bool project = (u.desc.flags & 2) != 0;
    int rc;
    // the interiors are re-derived from x, unless every block kept its own since the forward pass (store-all, literally)
    if (!keeps_interiors(c.ch, c.policy) && (rc = block_interiors(c, u, x, B, true))) return rc;
    // through the final ReLU: g_in <- dL/d(bn3 + shortcut)
    if ((rc = relu_mask_inplace(dt, out_px * co, g_in, y, c.stream))) return rc;
    const void* dx_shortcut = g_in;                       // identity shortcut: the same gradient flows to x
    if (project) {
        if ((rc = bn_relu_backward(dt, out_px, co, g_in, B.zp, (const float*)p[10], B.sp, 0, B.t0, (float*)g[10], (float*)g[11], scr, c.stream))) return rc;
        if ((rc = sgd_step(c, pf + 10)) || (rc = sgd_step(c, pf + 11))) return rc;
        if ((rc = conv_backward_pair(c, u.gp, B.t0, x, p[9], pf + 9, g_out ? B.dxs : nullptr))) return rc;
        dx_shortcut = B.dxs;
    }
    if ((rc = bn_relu_backward(dt, out_px, co, g_in, B.z3, (const float*)p[7], B.s3, 0, B.t1, (float*)g[7], (float*)g[8], scr, c.stream))) return rc;
    if ((rc = sgd_step(c, pf + 7)) || (rc = sgd_step(c, pf + 8))) return rc;
    if ((rc = conv_backward_pair(c, u.g3, B.t1, B.b, p[6], pf + 6, B.db))) return rc;
    if ((rc = bn_relu_backward(dt, out_px, mid, B.db, B.z2, (const float*)p[4], B.s2, 1, B.db, (float*)g[4], (float*)g[5], scr, c.stream))) return rc;
    if ((rc = sgd_step(c, pf + 4)) || (rc = sgd_step(c, pf + 5))) return rc;
    if ((rc = conv_backward_pair(c, u.g2, B.db, B.a, p[3], pf + 3, B.da))) return rc;
    if ((rc = bn_relu_backward(dt, in_px, mid, B.da, B.z1, (const float*)p[1], B.s1, 1, B.da, (float*)g[1], (float*)g[2], scr, c.stream))) return rc;
    if ((rc = sgd_step(c, pf + 1)) || (rc = sgd_step(c, pf + 2))) return rc;
    if ((rc = conv_backward_pair(c, u.g1, B.da, x, p[0], pf, g_out))) return rc;
    if (!g_out) return CKPT_OK;
    return add_tensors(dt, in_px * u.in.c, g_out, dx_shortcut, g_out, c.stream);
}

// d_i = f_i(d_{i-1}, w_i)  (Eq. (1)); i is 1-based.
// recompute: the unit ran before in this step (segment recomputation of Algorithms 2 and 4).  Its output is a function of
// the same inputs and parameters, so the batch statistics saved by its first run are the ones a second pass over the
// output would find: the convolutions skip the sums in their epilogues and no finalize kernel runs.
static int unit_forward(StepCtx& c, int64_t i, const void* x_raw, void* y, bool recompute = false) {
    if (c.dry) return CKPT_OK;
    const Unit& u = c.ch->units[i - 1];
    const int dt = c.ch->dtype;
    void* const* p = c.params + u.param_first;
    char* ws = c.ws;
    const void* x = x_raw;
    int rc;
    switch (u.desc.kind) {
        case CKPT_UNIT_CONV_BN_RELU:
            if ((rc = activated(c, i - 1, x_raw, &x))) return rc;
            if (recompute) return conv_forward_any(c, u.geom, x, p[0], y, nullptr, 0);
            return conv_with_statistics(c, u.geom, x, p[0], y, (const float*)p[1], (const float*)p[2], stats_of(c, i));
        case CKPT_UNIT_CONV:
            if ((rc = activated(c, i - 1, x_raw, &x))) return rc;
            return conv_forward_any(c, u.geom, x, p[0], y, nullptr, 0);
        case CKPT_UNIT_BN:
            if ((rc = activated(c, i - 1, x_raw, &x))) return rc;
            if (!recompute && (rc = bn_statistics(dt, rows_of(c.ch, i), u.out.c, x, (const float*)p[0], (const float*)p[1], stats_of(c, i),
                                                  ws + c.ch->off_scr, c.stream))) return rc;
            return bn_apply(dt, rows_of(c.ch, i), u.out.c, x, stats_of(c, i), 0, y, c.stream);
        case CKPT_UNIT_RELU:
            if ((rc = activated(c, i - 1, x_raw, &x))) return rc;
            return relu_forward(dt, rows_of(c.ch, i) * u.out.c, x, y, c.stream);
        case CKPT_UNIT_MAXPOOL: {
            const float* act = nullptr;
            if (pending_act(c.ch, i - 1)) {
                if (maxpool_fuses_activation(dt, u.in.h, u.in.w, u.in.c, u.desc.k, u.desc.stride, u.desc.pad)) act = stats_of(c, i - 1);
                else if ((rc = activated(c, i - 1, x_raw, &x))) return rc;
            }
            return maxpool_forward(dt, (int)c.ch->batch, u.in.h, u.in.w, u.in.c, u.desc.k, u.desc.stride, u.desc.pad, x, y, act,
                                   c.stream);
        }
        case CKPT_UNIT_AVGPOOL:
            if ((rc = activated(c, i - 1, x_raw, &x))) return rc;
            return avgpool_forward(dt, (int)c.ch->batch, u.in.h, u.in.w, u.in.c, x, y, c.stream);
        case CKPT_UNIT_FC:
            if ((rc = activated(c, i - 1, x_raw, &x))) return rc;
            return conv_forward_any(c, u.geom, x, p[0], y, (const float*)p[1], u.desc.flags & 1);
        case CKPT_UNIT_BOTTLENECK:
            if ((rc = activated(c, i - 1, x_raw, &x))) return rc;
            return block_forward(c, u, x, y, recompute);
    }
    set_error("unit kind %d has no forward kernel", u.desc.kind);
    return CKPT_E_UNSUPPORTED;
}

// Turns dL/d(activated d_j) into dL/d(d_j) in place when d_j carries a pending normalisation, and
// writes the gradients of that normalisation's scale and shift.
// sum_blocks > 0: the kernel that wrote g has already left that many partial row pairs of the backward sums
// in the scratch region.
static int through_pending_act(StepCtx& c, int64_t j, const void* d_j, void* g, int sum_blocks = 0) {
    if (!pending_act(c.ch, j)) return CKPT_OK;
    const Unit& uj = c.ch->units[j - 1];
    void* const* p = c.params + uj.param_first;
    void* const* gr = c.grads + uj.param_first;
    int rc;
    if (sum_blocks > 0)
        rc = bn_relu_backward_from_partials(c.ch->dtype, rows_of(c.ch, j), uj.out.c, g, d_j, stats_of(c, j), 1, g,
                                            (float*)gr[1], (float*)gr[2], c.ws + c.ch->off_scr, sum_blocks, c.stream);
    else
        rc = bn_relu_backward(c.ch->dtype, rows_of(c.ch, j), uj.out.c, g, d_j, (const float*)p[1], stats_of(c, j), 1, g,
                              (float*)gr[1], (float*)gr[2], c.ws + c.ch->off_scr, c.stream);
    // scale and shift of unit j are not read again in this step: the saved statistics block holds what forward and
    // backward need of them
    if (!rc) rc = sgd_step(c, uj.param_first + 1);
    if (!rc) rc = sgd_step(c, uj.param_first + 2);
    return rc;
}

// r_i and g_i (Eqs. (3) and (5)): g_in = dL/dd_i (may be overwritten), g_out = dL/dd_{i-1} or null.
static int unit_backward(StepCtx& c, int64_t i, const void* x_raw, const void* y, void* g_in, void* g_out) {
    if (c.dry) return CKPT_OK;
    const Unit& u = c.ch->units[i - 1];
    const int dt = c.ch->dtype;
    void* const* p = c.params + u.param_first;
    void* const* g = c.grads + u.param_first;
    const void* x = x_raw;
    int rc, sum_blocks = 0;
    switch (u.desc.kind) {
        case CKPT_UNIT_CONV_BN_RELU:
        case CKPT_UNIT_CONV:
            if ((rc = activated(c, i - 1, x_raw, &x))) return rc;
            if ((rc = conv_backward_pair(c, u.geom, g_in, x, p[0], u.param_first, g_out))) return rc;
            break;
        case CKPT_UNIT_BN:
            // the statistics saved by this unit's (re)computed forward are those of its input
            if ((rc = activated(c, i - 1, x_raw, &x))) return rc;
            if ((rc = bn_relu_backward(dt, rows_of(c.ch, i), u.out.c, g_in, x, (const float*)p[0], stats_of(c, i), 0,
                                       g_out ? g_out : g_in, (float*)g[0], (float*)g[1], c.ws + c.ch->off_scr, c.stream))) return rc;
            if ((rc = sgd_step(c, u.param_first)) || (rc = sgd_step(c, u.param_first + 1))) return rc;
            break;
        case CKPT_UNIT_RELU:
            if (g_out && (rc = relu_backward(dt, rows_of(c.ch, i) * u.out.c, g_in, y, g_out, c.stream))) return rc;
            break;
        case CKPT_UNIT_MAXPOOL: {
            if (!g_out) break;
            const float* act = nullptr;
            if (pending_act(c.ch, i - 1)) {
                if (maxpool_fuses_activation(dt, u.in.h, u.in.w, u.in.c, u.desc.k, u.desc.stride, u.desc.pad)) act = stats_of(c, i - 1);
                else if ((rc = activated(c, i - 1, x_raw, &x))) return rc;
            }
            if ((rc = maxpool_backward(dt, (int)c.ch->batch, u.in.h, u.in.w, u.in.c, u.desc.k, u.desc.stride, u.desc.pad, x, g_in,
                                       g_out, act, c.stream, act ? (float*)(c.ws + c.ch->off_scr) : nullptr, &sum_blocks,
                                       c.ws + c.ch->off_scr, c.ch->scr_bytes))) return rc;
            break;
        }
        case CKPT_UNIT_AVGPOOL:
            if (!g_out) break;
            if ((rc = avgpool_backward(dt, (int)c.ch->batch, u.in.h, u.in.w, u.in.c, g_in, g_out, c.stream))) return rc;
            break;
        case CKPT_UNIT_FC: {
            const int64_t elems = c.ch->batch * u.out.c;
            if ((rc = activated(c, i - 1, x_raw, &x))) return rc;
            if (u.desc.flags & 1)
                if ((rc = relu_mask_inplace(dt, elems, g_in, y, c.stream))) return rc;
            if ((rc = column_sums(dt, c.ch->batch, u.out.c, g_in, (float*)g[1], c.stream))) return rc;
            if ((rc = sgd_step(c, u.param_first + 1))) return rc;
            if ((rc = conv_backward_pair(c, u.geom, g_in, x, p[0], u.param_first, g_out))) return rc;
            break;
        }
        case CKPT_UNIT_BOTTLENECK:
            if ((rc = activated(c, i - 1, x_raw, &x))) return rc;
            if ((rc = block_backward(c, u, x, y, g_in, g_out))) return rc;
            break;
        default:
            set_error("unit kind %d has no backward kernel", u.desc.kind);
            return CKPT_E_UNSUPPORTED;
    }
    // the producer of d_{i-1} may have left its normalisation pending: finish the chain rule through it
    if (g_out) return through_pending_act(c, i - 1, x_raw, g_out, sum_blocks);
    return CKPT_OK;
}

// loss (float for softmax cross-entropy, double for the sum loss) at byte 0, device status word at byte 8
static int decode_result(const ckpt_chain* ch, const void* result, double* loss_out) {
    int status = 0;
    memcpy(&status, (const char*)result + 8, sizeof(int));
    if (ch->loss == CKPT_LOSS_SOFTMAX_CE) { float l; memcpy(&l, result, sizeof(float)); *loss_out = l; }
    else { double l; memcpy(&l, result, sizeof(double)); *loss_out = l; }
    if (status != 0) { set_error("a device-side wait gave up (status %d)", status); return CKPT_E_DEVICE_TIMEOUT; }
    return CKPT_OK;
}

// Verification aid: r_i = dL/dd_i (Eq. (3)) as it enters unit i's backward, copied to the tap at the offset of d_i
// among d_1..d_n.
static int tap_gradient(StepCtx& c, int64_t i, const void* g) {
    if (c.dry || !c.ch->tap || i < 1) return CKPT_OK;
    int64_t off = 0;
    for (int64_t k = 1; k < i; ++k) off += c.ch->d[k];
    return device_copy(c.ch->tap + off, g, c.ch->d[i], c.stream);
}

static int run_step(StepCtx& c, double* loss_out) {
    ckpt_chain* ch = c.ch;
    const int64_t n = (int64_t)ch->units.size();
    const std::vector<int64_t>& d = ch->d;
    Arena& A = *c.arena;
    const bool store_all = c.policy == CKPT_POLICY_STORE_ALL;
    auto ck = [&](int64_t i) { return store_all || c.is_ckpt[i] != 0; };
    auto ptr = [&](int64_t id) -> void* {
        int64_t off = A.offset_of(id);
        return (c.dry || off < 0) ? nullptr : (void*)(c.arena_base + off);
    };
    int rc;
    int64_t off;

    // Activated copies under Algorithm 4: a backward hop has its gradient in one of {segment buffer, carry 0, carry 1}
    // and writes the next one into another, so the third is idle and takes the activated copy of the unit's input
    // (the segment's buffer is at least as large as every tensor of the segment, the carry buffers as the largest
    // tensor of the chain); forward and recomputation have at most one gradient alive.  The workspace's own buffer
    // for that copy is then never touched.
    const bool lean = c.policy == CKPT_POLICY_DYNAMIC && !c.dry;
    char* const carry[2] = {c.dry ? nullptr : c.ws + ch->off_g0, c.dry ? nullptr : c.ws + ch->off_g1};
    auto idle_buffer = [&](const void* busy_a, const void* busy_b, char* segment_buffer) -> char* {
        for (char* cand : {carry[1], carry[0]})
            if (cand != busy_a && cand != busy_b) return cand;
        return segment_buffer;
    };
    if (lean) { c.act_buf = carry[1]; c.act_cap = ch->max_d; }

    // ---------------- forward phase
    if ((rc = A.alloc_stack(0, d[0], &off))) return rc;
    if (c.stage_trace) c.stage_trace[0] = A.live_bytes();
    if (!c.dry) {
        const int64_t payload = ch->batch * ch->shapes[0].h * ch->shapes[0].w * ch->shapes[0].c * dtype_size(ch->dtype);
        cudaError_t e = cudaMemcpyAsync(c.arena_base + off, c.batch, payload, cudaMemcpyDefault, c.stream);
        if (e != cudaSuccess) return cuda_fail(e, "copy of the input batch into the arena");
    }
    // Side of each forward temporary: the one just before a checkpoint sits at the top of the slab,
    // the one before it on the stack, and so on alternately.
    std::vector<uint8_t> top_side(n + 1, 0);
    for (int64_t i = n, dist = 0; i >= 1; --i) {
        if (ck(i)) dist = 0; else { top_side[i] = (dist % 2 == 0); ++dist; }
    }
    if (store_all) {
        for (int64_t i = 1; i <= n; ++i) if ((rc = A.alloc_stack(i, d[i], &off))) return rc;
    }
    for (int64_t i = 1; i <= n; ++i) {
        if (!store_all) {
            if (ck(i) || !top_side[i]) rc = A.alloc_stack(i, d[i], &off);
            else rc = A.alloc_top(i, d[i], &off);
            if (rc) return rc;
        }
        if ((rc = unit_forward(c, i, ptr(i - 1), ptr(i)))) return rc;
        if (!ck(i - 1)) if ((rc = A.release(i - 1))) return rc;
        if (c.stage_trace) c.stage_trace[i] = A.live_bytes();
    }

    // ---------------- loss and dL/dd_n
    char* gbuf[2] = {c.dry ? nullptr : c.ws + ch->off_g0, c.dry ? nullptr : c.ws + ch->off_g1};
    void* g_cur = gbuf[0];
    if (!c.dry) {
        const Shape& so = ch->shapes[n];
        const void* out_act = nullptr;
        if ((rc = activated(c, n, ptr(n), &out_act))) return rc;
        if (ch->loss == CKPT_LOSS_SOFTMAX_CE) {
            const int32_t* lab = (const int32_t*)(c.ws + ch->off_misc + 128 + 256);
            cudaError_t e = cudaMemcpyAsync((void*)lab, c.labels, ch->batch * sizeof(int32_t), cudaMemcpyDefault, c.stream);
            if (e != cudaSuccess) return cuda_fail(e, "copy of the labels");
            rc = softmax_ce(ch->dtype, (int)ch->batch, so.h * so.w * so.c, out_act, lab,
                            (float*)(c.ws + ch->off_misc), g_cur, (float*)(c.ws + ch->off_scr), c.stream);
        } else {
            rc = sum_loss(ch->dtype, ch->batch * so.h * so.w * so.c, out_act, (double*)(c.ws + ch->off_misc),
                          g_cur, (double*)(c.ws + ch->off_scr), c.stream);
        }
        if (rc) return rc;
        if ((rc = through_pending_act(c, n, ptr(n), g_cur))) return rc;
        if ((rc = tap_gradient(c, n, g_cur))) return rc;
        if (ch->selftest_wait && (rc = tc_selftest_wait(200000, c.status(), c.stream))) return rc;
    }

    // ---------------- backward phase
    bool have_r = false;            // Algorithm 4: a per-segment gradient buffer is live in the arena
    int64_t r_bytes = 0;            // its size
    bool g_in_r = false;            // the current gradient lives in that buffer
    bool bypass_r_once = false;     // first hop of a segment with an odd number of hops goes carry -> carry
    std::vector<int64_t> live_segment;
    for (int64_t i = n; i >= 1; --i) {
        if (!store_all && c.is_ckpt[i]) {
            int64_t h = i - 1;
            while (!c.is_ckpt[h]) --h;
            if (c.policy == CKPT_POLICY_DYNAMIC) {
                if (have_r) {
                    if (g_in_r) {
                        // the gradient entering the next segment must outlive the buffer it sits in
                        if (!c.dry && (rc = device_copy(gbuf[0], g_cur, d[i], c.stream))) return rc;
                        g_cur = gbuf[0];
                        g_in_r = false;
                    }
                    if ((rc = A.release(kGradId))) return rc;
                }
            } else {
                for (int64_t k : live_segment) if ((rc = A.release(k))) return rc;
                live_segment.clear();
            }
            if (lean) { c.act_buf = idle_buffer(g_cur, nullptr, nullptr); c.act_cap = ch->max_d; }
            for (int64_t k = h + 1; k < i; ++k) {
                if ((rc = A.alloc_stack(k, d[k], &off))) return rc;
                if ((rc = unit_forward(c, k, ptr(k - 1), ptr(k), true))) return rc;
                ++c.recomputed;
                if (c.policy == CKPT_POLICY_STATIC) live_segment.push_back(k);
            }
            if (c.policy == CKPT_POLICY_DYNAMIC) {
                int64_t r = 0;
                for (int64_t k = h; k < i; ++k) r = std::max(r, d[k]);
                if ((rc = A.alloc_stack(kGradId, r, &off))) return rc;
                have_r = true;
                r_bytes = r;
                // The gradient alternates between the segment's buffer and a carry buffer, one hop per
                // unit.  It has to sit in a carry buffer when the segment ends (its buffer is released
                // then), so a segment with an odd number of hops starts with one carry -> carry hop.
                bypass_r_once = h > 0 && ((i - h) % 2 == 1);
                // a carry -> carry hop leaves only the segment's buffer idle; a residual block keeps a tensor of its
                // output's size there, so the hop is taken only when that fits (otherwise the gradient is copied out
                // of the segment's buffer when the segment ends)
                if (bypass_r_once && ch->units[i - 1].desc.kind == CKPT_UNIT_BOTTLENECK && r < d[i]) bypass_r_once = false;
            }
        }
        // where the outgoing gradient goes: the segment's buffer (Algorithm 4) or the other carry buffer
        void* g_next;
        bool next_in_r = false;
        if (c.policy == CKPT_POLICY_DYNAMIC && !g_in_r && !bypass_r_once) { g_next = ptr(kGradId); next_in_r = true; }
        else if (c.policy == CKPT_POLICY_DYNAMIC && g_in_r) g_next = gbuf[0];
        else g_next = (g_cur == gbuf[0]) ? gbuf[1] : gbuf[0];
        bypass_r_once = false;
        const bool need_dx = i > 1;   // the gradient w.r.t. the input batch is never used
        if (lean) {
            c.act_buf = idle_buffer(g_cur, need_dx ? g_next : nullptr, have_r ? (char*)ptr(kGradId) : nullptr);
            c.act_cap = (c.act_buf == carry[0] || c.act_buf == carry[1]) ? ch->max_d : r_bytes;
        }
        if ((rc = unit_backward(c, i, ptr(i - 1), ptr(i), g_cur, need_dx ? g_next : nullptr))) return rc;
        if (need_dx) {
            g_cur = g_next; g_in_r = next_in_r;
            if ((rc = tap_gradient(c, i - 1, g_cur))) return rc;
        }
        if (c.policy == CKPT_POLICY_DYNAMIC) if ((rc = A.release(i))) return rc;
        if (c.stage_trace) c.stage_trace[2 * n + 1 - i] = A.live_bytes();
    }
    if (c.stage_trace) c.stage_trace[2 * n + 1] = d[0];

    if (!c.dry) {
        const size_t loss_bytes = ch->loss == CKPT_LOSS_SOFTMAX_CE ? sizeof(float) : sizeof(double);
        if (c.host_result) {
            // being captured: the results travel to pinned memory; whoever launches the graph waits and decodes
            cudaError_t e = cudaMemcpyAsync(c.host_result, c.ws + ch->off_misc, loss_bytes, cudaMemcpyDeviceToHost, c.stream);
            if (e == cudaSuccess) e = cudaMemcpyAsync((char*)c.host_result + 8, c.status(), sizeof(int), cudaMemcpyDeviceToHost, c.stream);
            if (e != cudaSuccess) return cuda_fail(e, "queueing the end-of-step copies");
            return CKPT_OK;
        }
        char result[16] = {0};
        cudaError_t e = cudaMemcpyAsync(result, c.ws + ch->off_misc, loss_bytes, cudaMemcpyDeviceToHost, c.stream);
        if (e == cudaSuccess) e = cudaMemcpyAsync(result + 8, c.status(), sizeof(int), cudaMemcpyDeviceToHost, c.stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(c.stream);
        if (e != cudaSuccess) return cuda_fail(e, "end-of-step synchronisation");
        return decode_result(ch, result, loss_out);
    }
    return CKPT_OK;
}

static int policy_model(int policy) {
    return policy == CKPT_POLICY_STORE_ALL ? CKPT_MODEL_STORE_ALL
         : policy == CKPT_POLICY_STATIC ? CKPT_MODEL_STATIC : CKPT_MODEL_DYNAMIC;
}

// ---------------------------------------------------------------------------------------------
// Graph replay.  Every launch of a step depends only on the chain, the plan, the policy and the
// pointers it is given (tensor maps and arena offsets are functions of those), so a step whose
// arguments repeat is recorded once as a CUDA graph and replayed: one submission instead of
// hundreds to tens of thousands of launches.
// ---------------------------------------------------------------------------------------------
static const size_t kMaxGraphs = 4;

static uint64_t mix(uint64_t h, uint64_t v) {
    h ^= v + 0x9E3779B97F4A7C15ull + (h << 6) + (h >> 2);
    return h * 0xFF51AFD7ED558CCDull;
}
// Everything a step's launch sequence depends on, as a list of words, and a hash of it.
static uint64_t step_key(const ckpt_chain* ch, const uint8_t* is_ckpt, int policy, const void* batch, const int32_t* labels,
                         void* const* params, void* const* grads, const void* arena, const void* ws, std::vector<uint64_t>* args) {
    args->clear();
    args->push_back((uint64_t)policy);
    args->push_back((uint64_t)(uintptr_t)batch); args->push_back((uint64_t)(uintptr_t)labels);
    args->push_back((uint64_t)(uintptr_t)arena); args->push_back((uint64_t)(uintptr_t)ws);
    args->push_back((uint64_t)ch->impl);
    args->push_back((uint64_t)(uintptr_t)ch->tap); args->push_back((uint64_t)ch->selftest_wait);
    args->push_back((uint64_t)ch->keep_interiors);
    { uint32_t bits; memcpy(&bits, &ch->sgd_lr, sizeof(bits)); args->push_back((uint64_t)bits); }
    for (size_t p = 0; p < ch->params.size(); ++p) { args->push_back((uint64_t)(uintptr_t)params[p]); args->push_back((uint64_t)(uintptr_t)grads[p]); }
    if (policy != CKPT_POLICY_STORE_ALL)
        for (size_t i = 0; i <= ch->units.size(); ++i) args->push_back((uint64_t)is_ckpt[i]);
    uint64_t h = 0x1234567ull;
    for (uint64_t v : *args) h = mix(h, v);
    return h;
}
// A copy from pageable host memory cannot be part of a captured sequence.
static bool graph_eligible(const void* batch, const int32_t* labels) {
    const void* ptrs[2] = {batch, labels};
    for (const void* p : ptrs) {
        if (!p) continue;
        cudaPointerAttributes a;
        if (cudaPointerGetAttributes(&a, p) != cudaSuccess) { cudaGetLastError(); return false; }
        if (a.type == cudaMemoryTypeUnregistered) return false;
    }
    return true;
}
static StepGraph* find_graph(ckpt_chain* ch, uint64_t key, const std::vector<uint64_t>& args) {
    for (StepGraph& g : ch->graphs)
        if (g.key == key && g.args == args) { g.last_use = ++ch->use_clock; return &g; }
    return nullptr;
}
static void destroy_graph(StepGraph& g) {
    if (g.exec) cudaGraphExecDestroy(g.exec);
    if (g.graph) cudaGraphDestroy(g.graph);
    g.exec = nullptr; g.graph = nullptr;
}
static void drop_graphs(ckpt_chain* ch) {
    for (StepGraph& g : ch->graphs) destroy_graph(g);
    ch->graphs.clear();
    ch->seen_keys.clear();
}
static int capture_step(ckpt_chain* ch, StepCtx c, uint64_t key, const std::vector<uint64_t>& args, StepGraph** out) {
    Arena ar(c.arena->capacity());
    c.arena = &ar;
    c.host_result = ch->host_result;
    c.recomputed = 0;
    cudaError_t e = cudaSuccess;
    if (!ch->capture_stream) {
        e = cudaStreamCreateWithFlags(&ch->capture_stream, cudaStreamNonBlocking);
        if (e != cudaSuccess) { ch->capture_stream = nullptr; return cuda_fail(e, "creating the recording stream"); }
    }
    c.stream = ch->capture_stream;
    e = cudaStreamBeginCapture(c.stream, cudaStreamCaptureModeThreadLocal);
    if (e != cudaSuccess) return cuda_fail(e, "beginning the capture of a step");
    const int64_t launches0 = g_launches;
    double unused = 0;
    int rc = CKPT_OK;
    e = cudaMemsetAsync(c.ws + ch->off_misc, 0, 128, c.stream);
    if (e != cudaSuccess) rc = cuda_fail(e, "clearing the status words");
    if (!rc) rc = run_step(c, &unused);
    StepGraph g;
    e = cudaStreamEndCapture(c.stream, &g.graph);
    if (rc) { if (g.graph) cudaGraphDestroy(g.graph); return rc; }
    if (e != cudaSuccess) return cuda_fail(e, "ending the capture of a step");
    e = cudaGraphInstantiate(&g.exec, g.graph, 0);
    if (e != cudaSuccess) { cudaGraphDestroy(g.graph); return cuda_fail(e, "instantiating the captured step"); }
    g.key = key;
    g.args = args;
    g.peak = ar.high_water(); g.extent = ar.extent();
    g.launches = g_launches - launches0; g.recomputed = c.recomputed;
    if (ch->graphs.size() >= kMaxGraphs) {
        size_t victim = 0;
        for (size_t i = 1; i < ch->graphs.size(); ++i) if (ch->graphs[i].last_use < ch->graphs[victim].last_use) victim = i;
        destroy_graph(ch->graphs[victim]);
        ch->graphs.erase(ch->graphs.begin() + victim);
    }
    ch->graphs.push_back(g);
    *out = find_graph(ch, key, args);
    return CKPT_OK;
}

}  // namespace ckpt

ckpt_chain::~ckpt_chain() {
    ckpt::drop_graphs(this);
    if (host_result) cudaFreeHost(host_result);
    if (capture_stream) cudaStreamDestroy(capture_stream);
    for (cudaEvent_t e : stage_event) if (e) cudaEventDestroy(e);
    if (copy_stream) cudaStreamDestroy(copy_stream);
}

using namespace ckpt;

extern "C" {

int ckpt_arena_dry_run(int policy, int64_t n, const int64_t* d, const uint8_t* is_ckpt, int64_t* events,
                       int64_t max_events, int64_t* n_events, int64_t* high_water_bytes, int64_t* extent_bytes) {
    if (policy < 0 || policy > 2) { set_error("unknown policy %d", policy); return CKPT_E_BAD_ARG; }
    int64_t predicted = 0;
    int rc = eval_model(policy_model(policy), n, d, is_ckpt, &predicted);
    if (rc) return rc;
    ckpt_chain fake;
    fake.units.resize(n);
    fake.d.assign(d, d + n + 1);
    fake.shapes.resize(n + 1);
    Arena arena(predicted);
    StepCtx c{};
    c.ch = &fake; c.is_ckpt = is_ckpt; c.policy = policy; c.dry = true; c.arena = &arena;
    double loss = 0;
    rc = run_step(c, &loss);
    if (rc) return rc;
    if (n_events) *n_events = (int64_t)arena.events.size();
    if (events) {
        int64_t m = std::min<int64_t>(max_events, (int64_t)arena.events.size());
        for (int64_t e = 0; e < m; ++e) {
            const ArenaEvent& ev = arena.events[e];
            events[4 * e + 0] = ev.kind;
            events[4 * e + 1] = ev.id == kGradId ? n + 1 : ev.id;
            events[4 * e + 2] = ev.offset;
            events[4 * e + 3] = ev.size;
        }
    }
    if (high_water_bytes) *high_water_bytes = arena.high_water();
    if (extent_bytes) *extent_bytes = arena.extent();
    return CKPT_OK;
}

int ckpt_arena_stage_trace(int policy, int64_t n, const int64_t* d, const uint8_t* is_ckpt, int64_t* trace) {
    if (policy < 0 || policy > 2) { set_error("unknown policy %d", policy); return CKPT_E_BAD_ARG; }
    if (!trace) { set_error("trace is null"); return CKPT_E_NULL; }
    int64_t predicted = 0;
    int rc = eval_model(policy_model(policy), n, d, is_ckpt, &predicted);
    if (rc) return rc;
    ckpt_chain fake;
    fake.units.resize(n);
    fake.d.assign(d, d + n + 1);
    fake.shapes.resize(n + 1);
    Arena arena(predicted);
    StepCtx c{};
    c.ch = &fake; c.is_ckpt = is_ckpt; c.policy = policy; c.dry = true; c.arena = &arena; c.stage_trace = trace;
    double loss = 0;
    return run_step(c, &loss);
}

int ckpt_chain_create(const ckpt_unit_desc* units, int64_t n, int64_t batch, int32_t in_h, int32_t in_w,
                      int32_t in_c, int dtype, int loss, ckpt_chain** out) {
    if (!units || !out) { set_error("null pointer"); return CKPT_E_NULL; }
    if (n < 1) { set_error("n < 1"); return CKPT_E_BAD_N; }
    if (batch < 1 || in_h < 1 || in_w < 1 || in_c < 1) { set_error("bad input shape"); return CKPT_E_BAD_ARG; }
    if (dtype != CKPT_DTYPE_F32 && dtype != CKPT_DTYPE_BF16) { set_error("unknown dtype %d", dtype); return CKPT_E_BAD_ARG; }
    if (loss != CKPT_LOSS_SUM && loss != CKPT_LOSS_SOFTMAX_CE) { set_error("unknown loss %d", loss); return CKPT_E_BAD_ARG; }
    ckpt_chain* ch = new ckpt_chain();
    ch->batch = batch; ch->dtype = dtype; ch->loss = loss;
    const int64_t es = dtype_size(dtype);
    Shape cur{in_h, in_w, in_c};
    ch->shapes.push_back(cur);
    ch->d.push_back(align_up(batch * cur.h * cur.w * cur.c * es, 256));
    int64_t stats_floats = 0, max_z = 0, scr = 256;
    for (int64_t i = 1; i <= n; ++i) {
        Unit u;
        u.desc = units[i - 1];
        u.in = cur;
        u.param_first = (int)ch->params.size();
        int rc = CKPT_OK;
        switch (u.desc.kind) {
            case CKPT_UNIT_CONV_BN_RELU: {
                rc = check_conv(u.desc, cur, i);
                if (rc) break;
                u.out = {out_size(cur.h, u.desc.k, u.desc.stride, u.desc.pad),
                         out_size(cur.w, u.desc.k, u.desc.stride, u.desc.pad), u.desc.c_out};
                u.geom = {(int)batch, cur.h, cur.w, cur.c, u.out.h, u.out.w, u.out.c, u.desc.k, u.desc.stride, u.desc.pad};
                ch->params.push_back({i, (int64_t)u.desc.c_out * u.desc.k * u.desc.k * u.desc.c_in, dtype});
                ch->params.push_back({i, u.desc.c_out, CKPT_DTYPE_F32});
                ch->params.push_back({i, u.desc.c_out, CKPT_DTYPE_F32});
                u.stats_off = stats_floats;
                stats_floats += 4 * (int64_t)u.desc.c_out;
                const int64_t rows = batch * u.out.h * u.out.w;
                max_z = std::max(max_z, align_up(rows * u.out.c * es, 256));
                scr = std::max(scr, bn_scratch_bytes(rows, u.out.c));
                scr = std::max(scr, simt_wgrad_scratch_bytes(u.geom));
                if (tc_conv_supported(dtype, u.geom)) scr = std::max(scr, tc_conv_scratch_bytes(u.geom));
                if (small_conv_supported(dtype, u.geom)) scr = std::max(scr, small_conv_scratch_bytes(u.geom));
                if (stem_conv_supported(dtype, u.geom)) scr = std::max(scr, stem_conv_scratch_bytes(u.geom));
                break;
            }
            case CKPT_UNIT_CONV: {
                rc = check_conv(u.desc, cur, i);
                if (rc) break;
                u.out = {out_size(cur.h, u.desc.k, u.desc.stride, u.desc.pad),
                         out_size(cur.w, u.desc.k, u.desc.stride, u.desc.pad), u.desc.c_out};
                u.geom = {(int)batch, cur.h, cur.w, cur.c, u.out.h, u.out.w, u.out.c, u.desc.k, u.desc.stride, u.desc.pad};
                ch->params.push_back({i, (int64_t)u.desc.c_out * u.desc.k * u.desc.k * u.desc.c_in, dtype});
                scr = std::max(scr, simt_wgrad_scratch_bytes(u.geom));
                if (tc_conv_supported(dtype, u.geom)) scr = std::max(scr, tc_conv_scratch_bytes(u.geom));
                if (small_conv_supported(dtype, u.geom)) scr = std::max(scr, small_conv_scratch_bytes(u.geom));
                if (stem_conv_supported(dtype, u.geom)) scr = std::max(scr, stem_conv_scratch_bytes(u.geom));
                break;
            }
            case CKPT_UNIT_BN:
                if (u.desc.c_in != cur.c || u.desc.c_out != cur.c) {
                    set_error("unit %lld: batch norm over %d channels on %d incoming channels", (long long)i, u.desc.c_out, cur.c);
                    rc = CKPT_E_BAD_ARG; break;
                }
                u.out = cur;
                ch->params.push_back({i, cur.c, CKPT_DTYPE_F32});
                ch->params.push_back({i, cur.c, CKPT_DTYPE_F32});
                u.stats_off = stats_floats;
                stats_floats += 4 * (int64_t)cur.c;
                scr = std::max(scr, bn_scratch_bytes(batch * cur.h * cur.w, cur.c));
                break;
            case CKPT_UNIT_RELU:
                u.out = cur;
                break;
            case CKPT_UNIT_MAXPOOL:
                if (u.desc.k < 1 || u.desc.stride < 1 || u.desc.pad < 0 || 2 * u.desc.pad > u.desc.k ||
                    cur.h + 2 * u.desc.pad < u.desc.k || cur.w + 2 * u.desc.pad < u.desc.k) {
                    set_error("unit %lld: bad pooling parameters", (long long)i); rc = CKPT_E_BAD_ARG; break;
                }
                u.out = {out_size(cur.h, u.desc.k, u.desc.stride, u.desc.pad),
                         out_size(cur.w, u.desc.k, u.desc.stride, u.desc.pad), cur.c};
                scr = std::max(scr, maxpool_backward_scratch_bytes(dtype, (int)batch, cur.h, cur.w, cur.c, u.desc.k, u.desc.stride, u.desc.pad));
                break;
            case CKPT_UNIT_AVGPOOL:
                u.out = {1, 1, cur.c};
                break;
            case CKPT_UNIT_FC: {
                if (u.desc.c_in != cur.h * cur.w * cur.c || u.desc.c_out < 1) {
                    set_error("unit %lld: fc c_in %d != flattened input %d", (long long)i, u.desc.c_in, cur.h * cur.w * cur.c);
                    rc = CKPT_E_BAD_ARG; break;
                }
                u.out = {1, 1, u.desc.c_out};
                u.geom = {(int)batch, 1, 1, u.desc.c_in, 1, 1, u.desc.c_out, 1, 1, 0};
                ch->params.push_back({i, (int64_t)u.desc.c_out * u.desc.c_in, dtype});
                ch->params.push_back({i, u.desc.c_out, CKPT_DTYPE_F32});
                scr = std::max(scr, simt_wgrad_scratch_bytes(u.geom));
                if (tc_conv_supported(dtype, u.geom)) scr = std::max(scr, tc_conv_scratch_bytes(u.geom));
                break;
            }
            case CKPT_UNIT_BOTTLENECK: {
                const int mid = u.desc.mid, st = u.desc.stride, co = u.desc.c_out;
                const bool project = (u.desc.flags & 2) != 0;
                if (u.desc.c_in != cur.c || mid < 1 || co < 1 || st < 1 || st > 2 || (!project && (co != cur.c || st != 1))) {
                    set_error("unit %lld: inconsistent bottleneck block", (long long)i); rc = CKPT_E_BAD_ARG; break;
                }
                const int ho = out_size(cur.h, 3, st, 1), wo = out_size(cur.w, 3, st, 1);
                u.out = {ho, wo, co};
                u.g1 = {(int)batch, cur.h, cur.w, cur.c, cur.h, cur.w, mid, 1, 1, 0};
                u.g2 = {(int)batch, cur.h, cur.w, mid, ho, wo, mid, 3, st, 1};
                u.g3 = {(int)batch, ho, wo, mid, ho, wo, co, 1, 1, 0};
                u.gp = {(int)batch, cur.h, cur.w, cur.c, out_size(cur.h, 1, st, 0), out_size(cur.w, 1, st, 0), co, 1, st, 0};
                if (project && (u.gp.ho != ho || u.gp.wo != wo)) { set_error("unit %lld: shortcut shape mismatch", (long long)i); rc = CKPT_E_BAD_ARG; break; }
                const ConvGeom* gs[4] = {&u.g1, &u.g2, &u.g3, &u.gp};
                for (int q = 0; q < (project ? 4 : 3); ++q) {
                    const ConvGeom& g = *gs[q];
                    ch->params.push_back({i, (int64_t)g.cout * g.k * g.k * g.cin, dtype});
                    ch->params.push_back({i, g.cout, CKPT_DTYPE_F32});
                    ch->params.push_back({i, g.cout, CKPT_DTYPE_F32});
                    const int64_t rows = batch * g.ho * g.wo;
                    scr = std::max(scr, bn_scratch_bytes(rows, g.cout));
                    scr = std::max(scr, simt_wgrad_scratch_bytes(g));
                    if (tc_conv_supported(dtype, g)) scr = std::max(scr, tc_conv_scratch_bytes(g));
                }
                u.stats_off = stats_floats;
                stats_floats += 4 * (int64_t)(2 * mid + 2 * co);
                // interiors and gradient temporaries of one block (see block_buffers)
                const int64_t in_px = batch * cur.h * cur.w, out_px = batch * ho * wo;
                const int64_t z3_bytes = align_up(out_px * co * es, 256);
                const int64_t blk = 3 * align_up(in_px * mid * es, 256) + 3 * align_up(out_px * mid * es, 256) + z3_bytes +
                                    (project ? z3_bytes + align_up(in_px * cur.c * es, 256) : 0);
                u.in_pending = i >= 2 && units[i - 2].kind == CKPT_UNIT_CONV_BN_RELU;
                u.blk_off = ch->blk_sum;
                ch->blk_sum += blk;
                ch->blk_bytes = std::max(ch->blk_bytes, blk);
                ch->blk_lean_bytes = std::max(ch->blk_lean_bytes, u.in_pending ? blk : blk - z3_bytes);
                break;
            }
            default:
                set_error("unit %lld: kind %d is not implemented", (long long)i, u.desc.kind);
                rc = CKPT_E_UNSUPPORTED;
        }
        if (rc) { delete ch; return rc; }
        u.n_params = (int)ch->params.size() - u.param_first;
        cur = u.out;
        ch->shapes.push_back(cur);
        ch->d.push_back(align_up(batch * cur.h * cur.w * cur.c * es, 256));
        ch->units.push_back(u);
    }
    scr = std::max<int64_t>(scr, std::max<int64_t>(sum_loss_scratch_bytes(), batch * (int64_t)sizeof(float)));
    ch->max_d = *std::max_element(ch->d.begin(), ch->d.end());
    int64_t o = 0;
    ch->off_g0 = o; o += ch->max_d;
    ch->off_g1 = o; o += ch->max_d;
    ch->off_scr = o; ch->scr_bytes = align_up(scr, 256); o += ch->scr_bytes;
    ch->off_stats = o; o += align_up(std::max<int64_t>(stats_floats, 1) * 4, 256);
    ch->off_misc = o; o += align_up(128 + 256 + batch * 4, 256);
    ch->off_blk = o; o += ch->blk_bytes;
    // last: the buffer of the activated copy.  Algorithm 4's schedule never needs it (see run_step) and takes a
    // workspace that ends here
    ch->z_bytes = std::max<int64_t>(max_z, 256);
    ch->off_z = o; o += ch->z_bytes;
    ch->ws_bytes = o;
    *out = ch;
    return CKPT_OK;
}

void ckpt_chain_destroy(ckpt_chain* chain) { delete chain; }

int ckpt_chain_sizes(const ckpt_chain* chain, int64_t* d, int32_t* shapes) {
    if (!chain || !d) { set_error("null pointer"); return CKPT_E_NULL; }
    for (size_t i = 0; i < chain->d.size(); ++i) {
        d[i] = chain->d[i];
        if (shapes) { shapes[3 * i] = chain->shapes[i].h; shapes[3 * i + 1] = chain->shapes[i].w; shapes[3 * i + 2] = chain->shapes[i].c; }
    }
    return CKPT_OK;
}

// Forward cost of every unit in nanoseconds from its arithmetic and its memory traffic at nominal rates (1.1 PFLOP/s
// for the contractions, 5.5 TB/s for everything that streams a tensor): what a recomputation of the unit costs, for
// ckpt_plan_min_recompute.  A model, not a measurement: only the order of magnitude between units matters.
int ckpt_chain_unit_costs(const ckpt_chain* chain, int64_t* cost_ns) {
    if (!chain || !cost_ns) { set_error("null pointer"); return CKPT_E_NULL; }
    const double flop_per_ns = 1.1e6, byte_per_ns = 5.5e3;
    auto conv_flops = [](const ConvGeom& g) { return 2.0 * g.n * g.ho * g.wo * g.cout * g.k * g.k * g.cin; };
    cost_ns[0] = 0;
    for (size_t i = 1; i < chain->d.size(); ++i) {
        const Unit& u = chain->units[i - 1];
        const double in_b = (double)chain->d[i - 1], out_b = (double)chain->d[i];
        const bool pending = pending_act(chain, (int64_t)i - 1);       // the producer's normalisation is applied on the way in
        double ns = 0;
        switch (u.desc.kind) {
            case CKPT_UNIT_CONV_BN_RELU:
            case CKPT_UNIT_CONV:
            case CKPT_UNIT_FC: {
                const double w_b = (double)u.geom.cout * u.geom.k * u.geom.k * u.geom.cin * dtype_size(chain->dtype);
                ns = conv_flops(u.geom) / flop_per_ns + ((pending ? 3.0 : 1.0) * in_b + out_b + w_b) / byte_per_ns;
                break;
            }
            case CKPT_UNIT_BOTTLENECK: {
                double fl = conv_flops(u.g1) + conv_flops(u.g2) + conv_flops(u.g3) + ((u.desc.flags & 2) ? conv_flops(u.gp) : 0.0);
                // the 1x1 layers stream their tensors: input, three interior pairs, output and the residual join
                ns = fl / flop_per_ns + (2.0 * in_b + 6.0 * out_b) / byte_per_ns;
                break;
            }
            default:
                ns = ((pending ? 1.0 : 1.0) * in_b + out_b) / byte_per_ns;
        }
        cost_ns[i] = (int64_t)(ns + 0.5) + 1000;        // plus a launch or two
    }
    return CKPT_OK;
}

int ckpt_chain_num_params(const ckpt_chain* chain, int64_t* count) {
    if (!chain || !count) { set_error("null pointer"); return CKPT_E_NULL; }
    *count = (int64_t)chain->params.size();
    return CKPT_OK;
}

int ckpt_chain_param_info(const ckpt_chain* chain, int64_t p, int64_t* unit, int64_t* elems, int32_t* dtype) {
    if (!chain) { set_error("null pointer"); return CKPT_E_NULL; }
    if (p < 0 || p >= (int64_t)chain->params.size()) { set_error("parameter index out of range"); return CKPT_E_BAD_ARG; }
    if (unit) *unit = chain->params[p].unit;
    if (elems) *elems = chain->params[p].elems;
    if (dtype) *dtype = chain->params[p].dtype;
    return CKPT_OK;
}

int ckpt_chain_workspace_bytes_for(const ckpt_chain* chain, int policy, int64_t* bytes) {
    if (!chain || !bytes) { set_error("null pointer"); return CKPT_E_NULL; }
    if (policy < 0 || policy > 2) { set_error("unknown policy %d", policy); return CKPT_E_BAD_ARG; }
    *bytes = workspace_need(chain, policy);
    return CKPT_OK;
}

int ckpt_chain_workspace_bytes(const ckpt_chain* chain, int64_t* bytes) {
    if (!chain || !bytes) { set_error("null pointer"); return CKPT_E_NULL; }
    *bytes = std::max(workspace_need(chain, CKPT_POLICY_STORE_ALL), workspace_need(chain, CKPT_POLICY_STATIC));
    return CKPT_OK;
}

int ckpt_chain_set_impl(ckpt_chain* chain, int impl) {
    if (!chain) { set_error("null pointer"); return CKPT_E_NULL; }
    if (impl != 0 && impl != 1) { set_error("impl must be 0 or 1"); return CKPT_E_BAD_ARG; }
    chain->impl = impl;
    return CKPT_OK;
}

int ckpt_train_step(ckpt_chain* chain, const uint8_t* is_ckpt, int policy, const void* batch,
                    const int32_t* labels, void* const* params, void* const* grads, void* arena,
                    int64_t arena_bytes, void* workspace, int64_t ws_bytes, void* stream,
                    ckpt_step_report* report) {
    if (!chain || !batch || !params || !grads || !arena || !workspace || !report) { set_error("null pointer"); return CKPT_E_NULL; }
    if (policy < 0 || policy > 2) { set_error("unknown policy %d", policy); return CKPT_E_BAD_ARG; }
    if (policy != CKPT_POLICY_STORE_ALL && !is_ckpt) { set_error("is_ckpt is null"); return CKPT_E_NULL; }
    if (chain->loss == CKPT_LOSS_SOFTMAX_CE && !labels) { set_error("labels are null"); return CKPT_E_NULL; }
    for (size_t p = 0; p < chain->params.size(); ++p)
        if (!params[p] || !grads[p]) { set_error("parameter or gradient pointer %zu is null", p); return CKPT_E_NULL; }
    const int64_t n = (int64_t)chain->units.size();
    memset(report, 0, sizeof(*report));
    int64_t predicted = 0;
    int rc = eval_model(policy_model(policy), n, chain->d.data(), is_ckpt, &predicted);
    if (rc) return rc;
    report->predicted_bytes = predicted;
    report->workspace_bytes = chain->ws_bytes;
    if (arena_bytes < predicted) {
        set_error("arena of %lld bytes is smaller than the plan's peak of %lld bytes", (long long)arena_bytes, (long long)predicted);
        return CKPT_E_ARENA_OOM;
    }
    const int64_t ws_need = workspace_need(chain, policy);
    report->workspace_bytes = ws_need;
    if (ws_bytes < ws_need) {
        set_error("workspace of %lld bytes, %lld needed", (long long)ws_bytes, (long long)ws_need);
        return CKPT_E_WORKSPACE;
    }
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) { set_error("no CUDA device"); return CKPT_E_NO_DEVICE; }
    Arena ar(predicted);
    StepCtx c{};
    c.ch = chain; c.is_ckpt = is_ckpt; c.policy = policy; c.dry = false;
    c.arena_base = (char*)arena; c.ws = (char*)workspace; c.params = params; c.grads = grads;
    c.batch = batch; c.labels = labels; c.stream = (cudaStream_t)stream; c.arena = &ar;
    double loss = 0;
    for (int slot = 0; slot < 2; ++slot) {
        if (chain->stage_pending[slot] && chain->stage_batch[slot] == batch) {
            // the batch was staged by ckpt_chain_stage_batch: its copy has to land before the step reads it
            cudaError_t se = cudaStreamWaitEvent(c.stream, chain->stage_event[slot], 0);
            if (se != cudaSuccess) return cuda_fail(se, "waiting for the staged batch");
            chain->stage_pending[slot] = false;
        }
    }
    if (chain->use_graph && graph_eligible(batch, labels)) {
        std::vector<uint64_t> args;
        const uint64_t key = step_key(chain, is_ckpt, policy, batch, labels, params, grads, arena, workspace, &args);
        StepGraph* g = find_graph(chain, key, args);
        const bool seen = std::find(chain->seen_keys.begin(), chain->seen_keys.end(), key) != chain->seen_keys.end();
        if (!g && seen) {
            // second step with these arguments: record its launch sequence
            rc = capture_step(chain, c, key, args, &g);
            if (rc) return rc;
        }
        if (g) {
            cudaError_t e = cudaGraphLaunch(g->exec, c.stream);
            if (e == cudaSuccess) e = cudaStreamSynchronize(c.stream);
            if (e != cudaSuccess) return cuda_fail(e, "replaying the captured step");
            rc = decode_result(chain, chain->host_result, &loss);
            report->peak_bytes = g->peak;
            report->extent_bytes = g->extent;
            report->launches = g->launches;
            report->recomputed_units = g->recomputed;
            report->loss = loss;
            report->replayed = 1;
            if (rc == CKPT_E_DEVICE_TIMEOUT) report->device_status = 1;
            return rc;
        }
        chain->seen_keys.push_back(key);       // first step with these arguments runs launch by launch
        if (chain->seen_keys.size() > 64) chain->seen_keys.erase(chain->seen_keys.begin());
    }
    cudaError_t e = cudaMemsetAsync(c.ws + chain->off_misc, 0, 128, c.stream);
    if (e != cudaSuccess) return cuda_fail(e, "clearing the status words");
    const int64_t launches0 = g_launches;
    rc = run_step(c, &loss);
    report->peak_bytes = ar.high_water();
    report->extent_bytes = ar.extent();
    report->launches = g_launches - launches0;
    report->recomputed_units = c.recomputed;
    report->loss = loss;
    if (rc == CKPT_E_DEVICE_TIMEOUT) report->device_status = 1;
    return rc;
}

int ckpt_chain_set_graph(ckpt_chain* chain, int enable) {
    if (!chain) { set_error("null pointer"); return CKPT_E_NULL; }
    if (enable && !chain->host_result) {
        cudaError_t e = cudaHostAlloc(&chain->host_result, 64, cudaHostAllocDefault);
        if (e != cudaSuccess) { chain->host_result = nullptr; return cuda_fail(e, "pinned result buffer of the captured step"); }
    }
    chain->use_graph = enable ? 1 : 0;
    if (!enable) drop_graphs(chain);
    return CKPT_OK;
}

static int64_t staging_slot_bytes(const ckpt_chain* chain) {
    return align_up(chain->d[0], 256) + align_up(chain->batch * (int64_t)sizeof(int32_t), 256);
}

int ckpt_chain_staging_bytes(const ckpt_chain* chain, int64_t* bytes) {
    if (!chain || !bytes) { set_error("null pointer"); return CKPT_E_NULL; }
    *bytes = 2 * staging_slot_bytes(chain);
    return CKPT_OK;
}

int ckpt_chain_stage_batch(ckpt_chain* chain, int slot, const void* batch, const int32_t* labels, void* staging, int64_t staging_bytes,
                           const void** batch_dev, const int32_t** labels_dev) {
    if (!chain || !batch || !staging || !batch_dev || !labels_dev) { set_error("null pointer"); return CKPT_E_NULL; }
    if (slot < 0 || slot > 1) { set_error("staging slot %d: 0 or 1", slot); return CKPT_E_BAD_ARG; }
    if (chain->loss == CKPT_LOSS_SOFTMAX_CE && !labels) { set_error("labels are null"); return CKPT_E_NULL; }
    if (staging_bytes < 2 * staging_slot_bytes(chain)) {
        set_error("staging buffer of %lld bytes, %lld needed", (long long)staging_bytes, (long long)(2 * staging_slot_bytes(chain)));
        return CKPT_E_WORKSPACE;
    }
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) { set_error("no CUDA device"); return CKPT_E_NO_DEVICE; }
    cudaError_t e = cudaSuccess;
    if (!chain->copy_stream) {
        e = cudaStreamCreateWithFlags(&chain->copy_stream, cudaStreamNonBlocking);
        if (e != cudaSuccess) { chain->copy_stream = nullptr; return cuda_fail(e, "creating the copy stream"); }
    }
    if (!chain->stage_event[slot]) {
        e = cudaEventCreateWithFlags(&chain->stage_event[slot], cudaEventDisableTiming);
        if (e != cudaSuccess) { chain->stage_event[slot] = nullptr; return cuda_fail(e, "creating the staging event"); }
    }
    char* base = (char*)staging + (int64_t)slot * staging_slot_bytes(chain);
    int32_t* lab = (int32_t*)(base + align_up(chain->d[0], 256));
    e = cudaMemcpyAsync(base, batch, (size_t)chain->d[0], cudaMemcpyDefault, chain->copy_stream);
    if (e == cudaSuccess && labels) e = cudaMemcpyAsync(lab, labels, (size_t)chain->batch * sizeof(int32_t), cudaMemcpyDefault, chain->copy_stream);
    if (e == cudaSuccess) e = cudaEventRecord(chain->stage_event[slot], chain->copy_stream);
    if (e != cudaSuccess) return cuda_fail(e, "staging a batch");
    chain->stage_batch[slot] = base;
    chain->stage_pending[slot] = true;
    *batch_dev = base;
    *labels_dev = labels ? lab : nullptr;
    return CKPT_OK;
}

int ckpt_chain_set_gradient_tap(ckpt_chain* chain, void* tap, int64_t tap_bytes) {
    if (!chain) { set_error("null pointer"); return CKPT_E_NULL; }
    int64_t need = 0;
    for (size_t i = 1; i < chain->d.size(); ++i) need += chain->d[i];
    if (tap && tap_bytes < need) { set_error("gradient tap of %lld bytes, %lld needed", (long long)tap_bytes, (long long)need); return CKPT_E_WORKSPACE; }
    chain->tap = (char*)tap;
    chain->tap_bytes = tap ? tap_bytes : 0;
    return CKPT_OK;
}

int ckpt_chain_set_sgd(ckpt_chain* chain, double learning_rate) {
    if (!chain) { set_error("null pointer"); return CKPT_E_NULL; }
    if (!(learning_rate == learning_rate) || learning_rate < 0) { set_error("learning rate must be >= 0"); return CKPT_E_BAD_ARG; }
    chain->sgd_lr = (float)learning_rate;
    return CKPT_OK;
}

int ckpt_chain_set_keep_interiors(ckpt_chain* chain, int enable) {
    if (!chain) { set_error("null pointer"); return CKPT_E_NULL; }
    chain->keep_interiors = enable ? 1 : 0;
    drop_graphs(chain);
    return CKPT_OK;
}

int ckpt_chain_set_selftest(ckpt_chain* chain, int wait_runs_out) {
    if (!chain) { set_error("null pointer"); return CKPT_E_NULL; }
    chain->selftest_wait = wait_runs_out ? 1 : 0;
    return CKPT_OK;
}

}  // extern "C"
