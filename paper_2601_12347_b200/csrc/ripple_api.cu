// C ABI of the ripple library: argument checks, device state set-up, and the per-batch launch
// chain.  See include/ripple.h for the contract of every entry point.
#include "device_utils.cuh"
#include "ripple_internal.cuh"

#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

using namespace rp;

static thread_local char g_create_err[512] = "";

static void set_err(Ctx* c, const char* fmt, ...) {
    char* dst = c ? c->err : g_create_err;
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(dst, 512, fmt, ap);
    va_end(ap);
}

#define CK(call)                                                                              \
    do {                                                                                      \
        cudaError_t e_ = (call);                                                              \
        if (e_ != cudaSuccess) {                                                              \
            set_err(c, "%s failed: %s", #call, cudaGetErrorString(e_));                       \
            st = e_ == cudaErrorMemoryAllocation ? RIPPLE_ERR_OOM : RIPPLE_ERR_CUDA;          \
            goto fail;                                                                        \
        }                                                                                     \
    } while (0)

template <typename T>
static cudaError_t dev_alloc(T** p, size_t count, int fill_byte = -2) {
    cudaError_t e = cudaMalloc(p, sizeof(T) * std::max<size_t>(count, 1));
    if (e) return e;
    if (fill_byte != -2) e = cudaMemset(*p, fill_byte, sizeof(T) * std::max<size_t>(count, 1));
    return e;
}

// params[0] = number of ops, params[1] = number of payload rows (device memory, so that a captured
// launch chain can be replayed for batches that differ in them)
__global__ void k_ctl_reset(Ctl* ctl, const int* params) {
    pdl_enter();
    d_ctl_reset(ctl, params);
}

static void destroy_ctx(Ctx* c) {
    if (!c) return;
    cudaSetDevice(c->device);
    if (c->stream) cudaStreamSynchronize(c->stream);
    for (int s = 0; s < 2; ++s) {
        Side& sd = c->side[s];
        cudaFree(sd.col); cudaFree(sd.w); cudaFree(sd.start); cudaFree(sd.cap); cudaFree(sd.deg);
        cudaFree(sd.cnt_del); cudaFree(sd.cnt_add); cudaFree(sd.tick_a); cudaFree(sd.tick_b); cudaFree(sd.touch);
        cudaFree(c->grow_list[s]); cudaFree(c->shrink_list[s]); cudaFree(c->D[s]); cudaFree(c->Clist[s]);
        cudaFree(sd.free_blk); cudaFree(sd.free_cnt);
    }
    for (int l = 0; l <= RP_MAXL; ++l) {
        cudaFree(c->att_s[l]); cudaFree(c->att_t[l]);
        cudaFree(c->H[l]); cudaFree(c->S[l]); cudaFree(c->dS[l]); cudaFree(c->Eb[l]); cudaFree(c->Z[l]); cudaFree(c->P[l]); cudaFree(c->A[l]);
        cudaFree(c->layer[l].W1); cudaFree(c->layer[l].b1); cudaFree(c->layer[l].W2); cudaFree(c->layer[l].b2);
        for (TcW* t : {&c->layer[l].tc_main, &c->layer[l].tc_nbr, &c->layer[l].tc_2, &c->layer[l].tc_self}) { cudaFree(t->hi); cudaFree(t->lo); }
    }
    cudaFree(c->att_so); cudaFree(c->att_items);
    cudaFree(c->halo_owner); cudaFree(c->halo_rid); cudaFree(c->silent_dev); cudaFree(c->rows_sent);
    free(c->halo_owner_h); free(c->halo_rid_h);
    for (int i = 0; i < c->n_ipc_opened; ++i) cudaIpcCloseMemHandle(c->ipc_opened[i]);
    cudaFree(c->T); cudaFree(c->Dt); cudaFree(c->coff); cudaFree(c->bitmap); cudaFree(c->bitmap2); cudaFree(c->old_idx); cudaFree(c->invmask); cudaFree(c->posmap); cudaFree(c->deg_out_old);
    cudaFree(c->feat_last); cudaFree(c->ups_dev); cudaFree(c->opw_dev); cudaFree(c->feat_dev); cudaFree(c->hkeys); cudaFree(c->hwin); cudaFree(c->op_seq); cudaFree(c->vdel_seq); cudaFree(c->vjobs);
    cudaFree(c->op_slot); cudaFree(c->rec); cudaFree(c->tile_sums); cudaFree(c->scan_done); cudaFree(c->ctl);
    cudaFree(c->moved_start); cudaFree(c->moved_cap);
    if (c->ctl_host) cudaFreeHost(c->ctl_host);
    if (c->params_host) cudaFreeHost(c->params_host);
    if (c->stage_host) cudaFreeHost(c->stage_host);
    cudaFree(c->stage_dev);
    cudaFree(c->params_dev);
    for (auto& g : c->graph_exec) if (g) cudaGraphExecDestroy(g);
    for (auto& e : c->ev) if (e) cudaEventDestroy(e);
    for (auto& e : c->ev_sc) if (e) cudaEventDestroy(e);
    for (auto& e : c->ev_rg) if (e) cudaEventDestroy(e);
    if (c->own_stream && c->stream) cudaStreamDestroy(c->stream);
    delete c;
}

static ripple_status sync_and_fetch_ctl(Ctx* c) {
    cudaError_t e = cudaMemcpyAsync(c->ctl_host, c->ctl, sizeof(Ctl), cudaMemcpyDeviceToHost, c->stream);
    if (!e) e = cudaStreamSynchronize(c->stream);
    if (!e) e = cudaGetLastError();
    if (e) {
        set_err(c, "CUDA error while running the batch: %s", cudaGetErrorString(e));
        return RIPPLE_ERR_CUDA;
    }
    return RIPPLE_OK;
}

// layer l of the full inference: cached aggregates and embeddings of every vertex
static void full_layer(Ctx* c, int l) {
    if (c->attention) { att_full(c, l); return; }
    if (rp_monotonic(c->agg)) max_full(c, l);
    else spmm_full(c, l);
    if (c->Eb[l]) cudaMemsetAsync(c->Eb[l], 0, sizeof(float) * (size_t)c->N, c->stream);   // every row freshly gathered
    self_project(c, l, true);
    update_rows(c, l, true);
}

// full layer-wise inference over the current graph (Eq. 1-2): bootstrap and recompute-all
static ripple_status run_full(Ctx* c) {
    c->launches = 0;
    c->debug_tc_withhold = 0;
    c->params_host[0] = 0; c->params_host[1] = 0;
    cudaMemcpyAsync(c->params_dev, c->params_host, 2 * sizeof(int), cudaMemcpyHostToDevice, c->stream);
    RP_LAUNCH(c, k_ctl_reset, 1, 1, 0, c->ctl, c->params_dev);
    if (c->timing) cudaEventRecord(c->ev[0], c->stream);
    for (int l = 1; l <= c->L; ++l) full_layer(c, l);
    if (c->timing) cudaEventRecord(c->ev[1], c->stream);
    ripple_status st = sync_and_fetch_ctl(c);
    if (st) return st;
    if (c->timing) cudaEventElapsedTime(&c->stats.ms_bootstrap, c->ev[0], c->ev[1]);
    c->stats.gpu_launches = c->launches;
    return RIPPLE_OK;
}

static std::vector<float> padded_matrix(const float* src, int rows, int cols, int rows_p, int cols_p) {
    std::vector<float> m((size_t)rows_p * cols_p, 0.f);
    if (src)
        for (int r = 0; r < rows; ++r) memcpy(&m[(size_t)r * cols_p], src + (size_t)r * cols, sizeof(float) * cols);
    return m;
}

extern "C" ripple_status ripple_create(const ripple_graph* g, const float* features, int32_t feat_mem,
                                       const ripple_layer* layers, int32_t L, int32_t agg,
                                       const ripple_options* opt, ripple_ctx** out) {
    Ctx* c = nullptr;
    ripple_status st = RIPPLE_ERR_INVALID_ARG;
    if (out) *out = nullptr;
    g_create_err[0] = 0;
    if (!g || !features || !layers || !out) { set_err(nullptr, "null argument"); return st; }
    if (L < 1 || L > RP_MAXL) { set_err(nullptr, "L must be in 1..%d", RP_MAXL); return st; }
    if (agg < 0 || agg > 5) { set_err(nullptr, "unknown aggregator %d", agg); return st; }
    if (rp_monotonic(agg) && layers[0].kind == RIPPLE_LAYER_GIN) {
        set_err(nullptr, "the max and min aggregators are built for GRAPHCONV and SAGE layers");
        return st;
    }
    if (g->num_vertices < 1 || g->num_vertices > 0x7fffffff - 64 || g->num_edges < 0 ||
        (g->num_edges > 0 && (!g->src || !g->dst))) {
        set_err(nullptr, "bad graph description");
        return st;
    }
    for (int l = 0; l < L; ++l) {
        const ripple_layer& y = layers[l];
        bool ok = y.kind >= 0 && y.kind <= 3 && y.d_in >= 1 && y.d_out >= 1 && y.d_in <= 1024 && y.d_out <= 1024 &&
                  (y.act == 0 || y.act == 1) && y.Wa && y.kind == layers[0].kind;
        if (y.kind == RIPPLE_LAYER_SAGE) ok = ok && y.Wb;
        if (y.kind == RIPPLE_LAYER_GIN) ok = ok && y.Wb && y.d_hidden >= 1 && y.d_hidden <= 1024;
        if (y.kind == RIPPLE_LAYER_GAT)
            ok = ok && y.ba && y.bb && y.d_hidden >= 1 && y.d_hidden <= 1024 && y.d_out == y.d_in && agg == RIPPLE_AGG_SUM;
        if (l > 0) ok = ok && y.d_in == layers[l - 1].d_out;
        if (!ok) { set_err(nullptr, "bad description of layer %d", l + 1); return st; }
    }
    {
        ripple_options o{};
        if (opt) o = *opt;
        if (o.slack <= 0) o.slack = 0.25;
        if (o.max_batch <= 0) o.max_batch = 16384;
        if (o.n_local != 0) {   // one worker of a partitioned execution
            const bool linear = agg == RIPPLE_AGG_SUM || agg == RIPPLE_AGG_MEAN || agg == RIPPLE_AGG_WSUM_GCN ||
                                agg == RIPPLE_AGG_WSUM_EDGE;
            if (o.n_local < 0 || (o.n_local & 31) || o.n_local > g->num_vertices || !linear ||
                layers[0].kind > RIPPLE_LAYER_GIN) {
                set_err(nullptr, "a partitioned context needs n_local a multiple of 32 within num_vertices, a linear aggregator and SAGE, GRAPHCONV or GIN layers");
                return st;
            }
            o.scatter_mode = RIPPLE_SCATTER_PUSH;   // rows cannot be gathered anew: remote in-neighbours' rows live elsewhere
            o.rebuild_budget = -1.f;
            o.no_graphs = 1;
        }
        if (o.pool_edges <= 0) o.pool_edges = std::max<int64_t>(g->num_edges / 4, 1 << 20);
        o.pool_edges = std::max<int64_t>(o.pool_edges, 4);
        c = new (std::nothrow) Ctx();
        if (!c) { set_err(nullptr, "host allocation failed"); return RIPPLE_ERR_OOM; }
        memset(static_cast<void*>(c), 0, sizeof(Ctx));
        int32_t *src_dev = nullptr, *dst_dev = nullptr;
        float* w_dev = nullptr;
        bool own_coo = false;
        const int N = (int)g->num_vertices;
        const int64_t E = g->num_edges;
        int max_ld = 0, max_hid = 0;

        if (o.device >= 0) CK(cudaSetDevice(o.device));
        CK(cudaGetDevice(&c->device));
        CK(cudaDeviceGetAttribute(&c->n_sm, cudaDevAttrMultiProcessorCount, c->device));
        if (o.stream) c->stream = (cudaStream_t)o.stream;
        else { CK(cudaStreamCreateWithFlags(&c->stream, cudaStreamNonBlocking)); c->own_stream = true; }
        c->N = N; c->L = L; c->agg = agg; c->E0 = E;
        c->max_batch = o.max_batch;
        c->scatter_mode = o.scatter_mode; c->gemm_mode = o.gemm_mode; c->timing = o.timing;
        c->rebuild_tau2 = o.rebuild_budget > 0.f ? o.rebuild_budget * o.rebuild_budget : 64.f;
        c->self_term = layers[0].kind != RIPPLE_LAYER_GRAPHCONV;
        c->src_norm = agg == RIPPLE_AGG_WSUM_GCN;
        c->weighted = agg == RIPPLE_AGG_WSUM_EDGE;
        c->attention = layers[0].kind == RIPPLE_LAYER_GAT;
        c->n_local = o.n_local;
        CK(dev_alloc(&c->ctl, 1, 0));
        CK(dev_alloc(&c->params_dev, 2, 0));
        CK(cudaMallocHost(&c->params_host, 2 * sizeof(int)));
        c->stage_bytes = 64 + (size_t)RP_GRAPH_MAX_BATCH * (sizeof(ripple_update) + sizeof(float) + sizeof(float) * (size_t)layers[0].d_in);
        CK(cudaMallocHost(&c->stage_host, c->stage_bytes));
        CK(dev_alloc(&c->stage_dev, c->stage_bytes));
        c->no_graphs = o.no_graphs;
        {
            const char* e = getenv("RIPPLE_NO_PDL");
            c->pdl = !(e && e[0] == '1');
        }
        {
            // Hops whose messages are at least this wide gather per sink once they carry a million messages
            // (measured on the dense graph, 256 floats: see scatter.cu); 0 = never.
            const char* e = getenv("RIPPLE_GATHER_MIN_WIDTH");
            c->gather_min_width = e ? atoi(e) : 128;
            c->gather_min_messages = 1 << 20;
        }
        tc_prepare();
        narrow_prepare();
        max_prepare();
        CK(cudaMallocHost(&c->ctl_host, sizeof(Ctl)));
        memset(c->ctl_host, 0, sizeof(Ctl));
        c->n_words = (N + 31) / 32;
        c->n_tile_sums = std::max(div_up(N, 1024) + 2, div_up(c->n_words, 256) + 2);
        CK(dev_alloc(&c->tile_sums, (size_t)c->n_tile_sums, 0));
        CK(dev_alloc(&c->scan_done, 1, 0));
        for (auto& e : c->ev) CK(cudaEventCreate(&e));
        for (auto& e : c->ev_sc) CK(cudaEventCreate(&e));
        for (auto& e : c->ev_rg) CK(cudaEventCreate(&e));

        // graph
        if (E > 0 && g->mem == RIPPLE_MEM_HOST) {
            own_coo = true;
            CK(dev_alloc(&src_dev, (size_t)E));
            CK(dev_alloc(&dst_dev, (size_t)E));
            CK(cudaMemcpyAsync(src_dev, g->src, sizeof(int32_t) * (size_t)E, cudaMemcpyHostToDevice, c->stream));
            CK(cudaMemcpyAsync(dst_dev, g->dst, sizeof(int32_t) * (size_t)E, cudaMemcpyHostToDevice, c->stream));
            if (c->weighted && g->weight) {
                CK(dev_alloc(&w_dev, (size_t)E));
                CK(cudaMemcpyAsync(w_dev, g->weight, sizeof(float) * (size_t)E, cudaMemcpyHostToDevice, c->stream));
            }
        } else {
            src_dev = const_cast<int32_t*>(g->src);
            dst_dev = const_cast<int32_t*>(g->dst);
            w_dev = c->weighted ? const_cast<float*>(g->weight) : nullptr;
        }
        {
            cudaError_t e = graph_build(c, src_dev, dst_dev, w_dev, E, o.slack, o.pool_edges);
            if (own_coo) { cudaFree(src_dev); cudaFree(dst_dev); cudaFree(w_dev); }
            CK(e);
            if (c->ctl_host->err) {
                set_err(nullptr, "an edge endpoint is outside [0, N)");
                st = RIPPLE_ERR_VERTEX_RANGE;
                goto fail;
            }
        }

        // model and cached state
        c->d[0] = layers[0].d_in; c->ld[0] = pad4(c->d[0]);
        for (int l = 1; l <= L; ++l) {
            const ripple_layer& y = layers[l - 1];
            LayerDev& ly = c->layer[l];
            c->d[l] = y.d_out; c->ld[l] = pad4(y.d_out);
            ly.kind = y.kind; ly.d_in = y.d_in; ly.d_hid = y.d_hidden; ly.d_out = y.d_out; ly.act = y.act; ly.eps = y.eps;
            ly.ld_in = pad4(y.d_in); ly.ld_hid = pad4(y.d_hidden); ly.ld_out = pad4(y.d_out);
            std::vector<float> w1, b1, w2, b2;
            if (y.kind == RIPPLE_LAYER_SAGE) {
                w1 = padded_matrix(y.Wa, y.d_in, y.d_out, ly.ld_in, ly.ld_out);
                std::vector<float> wn = padded_matrix(y.Wb, y.d_in, y.d_out, ly.ld_in, ly.ld_out);
                w1.insert(w1.end(), wn.begin(), wn.end());
                b1 = padded_matrix(y.ba, 1, y.d_out, 1, ly.ld_out);
            } else if (y.kind == RIPPLE_LAYER_GRAPHCONV) {
                w1 = padded_matrix(y.Wa, y.d_in, y.d_out, ly.ld_in, ly.ld_out);
                b1 = padded_matrix(y.ba, 1, y.d_out, 1, ly.ld_out);
            } else if (y.kind == RIPPLE_LAYER_GAT) {
                // a . (W h) = (W a) . h: the two halves of a are folded into W once (Wa is d_in x d_hidden, input-major)
                w1.assign((size_t)2 * ly.ld_in, 0.f);
                for (int k = 0; k < y.d_in; ++k) {
                    double qs = 0.0, qt = 0.0;
                    for (int j = 0; j < y.d_hidden; ++j) {
                        qs += (double)y.Wa[(size_t)k * y.d_hidden + j] * (double)y.ba[j];
                        qt += (double)y.Wa[(size_t)k * y.d_hidden + j] * (double)y.bb[j];
                    }
                    w1[k] = (float)qs;
                    w1[(size_t)ly.ld_in + k] = (float)qt;
                }
                b1.assign(1, 0.f);
            } else {
                w1 = padded_matrix(y.Wa, y.d_in, y.d_hidden, ly.ld_in, ly.ld_hid);
                b1 = padded_matrix(y.ba, 1, y.d_hidden, 1, ly.ld_hid);
                w2 = padded_matrix(y.Wb, y.d_hidden, y.d_out, ly.ld_hid, ly.ld_out);
                b2 = padded_matrix(y.bb, 1, y.d_out, 1, ly.ld_out);
                max_hid = std::max(max_hid, ly.ld_hid);
            }
            if (y.kind == RIPPLE_LAYER_GAT) {
                c->pre[l] = false;
                c->ws[l] = pad4(y.d_in + 1);   // numerator columns, then the denominator
                c->fused_fold[l] = false;
                c->regather_threshold[l] = -1.f;
            } else {
                // a layer narrower than its input transforms the few sender rows before the scatter
                const int target = y.kind == RIPPLE_LAYER_GIN ? ly.ld_hid : ly.ld_out;
                // Also for equal widths where nothing but the matrix product is left per affected row
                // (SAGE with its cached self projection, GraphConv): the product then runs over the
                // senders of the hop, the affected rows of the hop before, which are far fewer.
                // Not for max / min: a maximum does not commute with the matrix.
                c->pre[l] = o.pre_transform == 0 && !rp_monotonic(agg) &&
                            (target < ly.ld_in || (target == ly.ld_in && y.kind != RIPPLE_LAYER_GIN));
                c->ws[l] = c->pre[l] ? target : ly.ld_in;
                // Transformed aggregates are folded inside the update's epilogue, which sees a row in
                // pieces and keeps no rounding budget for it.  That is left to the normalised
                // aggregators, whose rows stay of one size; an unnormalised sum folds in a pass of its
                // own, with the budget.
                c->fused_fold[l] = c->pre[l] && agg != RIPPLE_AGG_SUM && agg != RIPPLE_AGG_WSUM_EDGE;
                // measured on the dense graph: rebuilding every aggregate costs 0.47 of pushing a message
                // along every edge at 256 floats per row (12.1 against 26 ms) and 0.54 at 48 (3.5 / 6.4 ms)
                c->regather_min_messages = o.regather_threshold > 0.f ? 0 : (4ll << 20);
                c->regather_threshold[l] = o.regather_threshold > 0.f ? o.regather_threshold
                                           : o.regather_threshold < 0.f ? -1.f
                                           : c->ws[l] >= 128 ? 0.5f : 0.55f;
                if (o.gemm_mode != RIPPLE_GEMM_FP32) {   // transposed, tf32-split copies for the tensor-core form
                    const float* wn = y.kind == RIPPLE_LAYER_SAGE ? w1.data() + (size_t)ly.ld_in * ly.ld_out : w1.data();
                    if (y.kind == RIPPLE_LAYER_SAGE)
                    {   // self part for the cached projection; neighbour part for the affected-row GEMM
                        CK(tc_weights_build(&ly.tc_self, w1.data(), ly.ld_in, ly.ld_out));
                        if (!c->pre[l]) CK(tc_weights_build(&ly.tc_main, wn, ly.ld_in, ly.ld_out));
                    }
                    else if (y.kind == RIPPLE_LAYER_GIN)
                        CK(tc_weights_build(&ly.tc_main, w1.data(), ly.ld_in, ly.ld_hid));
                    else if (!c->pre[l])
                        CK(tc_weights_build(&ly.tc_main, w1.data(), ly.ld_in, ly.ld_out));
                    if (c->pre[l]) CK(tc_weights_build(&ly.tc_nbr, wn, ly.ld_in, c->ws[l]));
                    if (y.kind == RIPPLE_LAYER_GIN) CK(tc_weights_build(&ly.tc_2, w2.data(), ly.ld_hid, ly.ld_out));
                }
            }
            CK(dev_alloc(&ly.W1, w1.size()));
            CK(cudaMemcpy(ly.W1, w1.data(), sizeof(float) * w1.size(), cudaMemcpyHostToDevice));
            CK(dev_alloc(&ly.b1, b1.size()));
            CK(cudaMemcpy(ly.b1, b1.data(), sizeof(float) * b1.size(), cudaMemcpyHostToDevice));
            if (!w2.empty()) {
                CK(dev_alloc(&ly.W2, w2.size()));
                CK(cudaMemcpy(ly.W2, w2.data(), sizeof(float) * w2.size(), cudaMemcpyHostToDevice));
                CK(dev_alloc(&ly.b2, b2.size()));
                CK(cudaMemcpy(ly.b2, b2.data(), sizeof(float) * b2.size(), cudaMemcpyHostToDevice));
            }
        }
        for (int l = 0; l <= L; ++l) {
            max_ld = std::max(max_ld, c->ld[l]);
            CK(dev_alloc(&c->H[l], (size_t)N * c->ld[l], 0));
            if (l > 0) { CK(dev_alloc(&c->S[l], (size_t)N * c->ws[l], 0));
                         if (!rp_monotonic(agg)) CK(dev_alloc(&c->dS[l], (size_t)N * c->ws[l], 0));
                         if (!rp_monotonic(agg) && !c->fused_fold[l] && o.rebuild_budget >= 0.f)
                             CK(dev_alloc(&c->Eb[l], (size_t)N, 0));
                         if (c->layer[l].kind == RIPPLE_LAYER_SAGE) CK(dev_alloc(&c->Z[l], (size_t)N * c->ld[l], 0));
                         if (c->pre[l]) CK(dev_alloc(&c->P[l], (size_t)N * c->ws[l], 0));
                         if (c->attention) { CK(dev_alloc(&c->att_s[l], (size_t)N, 0)); CK(dev_alloc(&c->att_t[l], (size_t)N, 0)); } }
            CK(dev_alloc(&c->A[l], (size_t)N + 32));
        }
        CK(cudaMemcpy2D(c->H[0], sizeof(float) * c->ld[0], features, sizeof(float) * c->d[0],
                        sizeof(float) * c->d[0], (size_t)N,
                        feat_mem == RIPPLE_MEM_DEVICE ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice));
        if (max_hid) CK(dev_alloc(&c->T, (size_t)N * max_hid));
        if (c->attention) {
            CK(dev_alloc(&c->att_so, (size_t)N + 32));
            CK(dev_alloc(&c->att_items, (size_t)N + (size_t)(c->side[1].col_size / RP_ATT_CHUNK) + 64));
        }
        CK(dev_alloc(&c->Dt, (size_t)N * max_ld));
        for (int s = 0; s < 2; ++s) {
            CK(dev_alloc(&c->D[s], (size_t)N * max_ld));
            CK(dev_alloc(&c->Clist[s], (size_t)N + 32));
            CK(dev_alloc(&c->grow_list[s], (size_t)o.max_batch));
            CK(dev_alloc(&c->shrink_list[s], (size_t)o.max_batch));
        }
        CK(dev_alloc(&c->moved_start, (size_t)4 * o.max_batch));
        CK(dev_alloc(&c->moved_cap, (size_t)4 * o.max_batch));
        // degree prefix of a sender list; also the (vertex, chunk) work items of long in-lists during a
        // gather: a row of more than 256 entries gives at most 2 items per 256 of them
        CK(dev_alloc(&c->coff, std::max((size_t)N + 2, (size_t)(c->side[1].col_size / 128) + 64), 0));
        CK(dev_alloc(&c->bitmap, (size_t)c->n_words + 256, 0));
        if (rp_monotonic(agg)) {
            CK(dev_alloc(&c->bitmap2, (size_t)c->n_words + 256, 0));
            CK(dev_alloc(&c->old_idx, (size_t)N + 32));
            c->mw = (max_ld + 31) / 32;
            CK(dev_alloc(&c->invmask, (size_t)N * c->mw, 0));
        }
        CK(dev_alloc(&c->posmap, (size_t)N, 0xFF));
        CK(dev_alloc(&c->deg_out_old, (size_t)N, 0xFF));
        CK(dev_alloc(&c->feat_last, (size_t)N, 0xFF));
        // batch staging
        CK(dev_alloc(&c->ups_dev, (size_t)o.max_batch));
        if (c->weighted) CK(dev_alloc(&c->opw_dev, (size_t)o.max_batch));
        CK(dev_alloc(&c->feat_dev, (size_t)o.max_batch * c->d[0]));
        c->hsize = 1024;
        while (c->hsize < 4 * o.max_batch) c->hsize <<= 1;
        CK(dev_alloc(&c->hkeys, (size_t)c->hsize, 0));
        CK(dev_alloc(&c->hwin, (size_t)c->hsize, 0));
        CK(dev_alloc(&c->op_seq, (size_t)o.max_batch));
        CK(dev_alloc(&c->vdel_seq, (size_t)N, 0xFF));
        CK(dev_alloc(&c->vjobs, (size_t)o.max_batch));
        CK(dev_alloc(&c->op_slot, (size_t)o.max_batch));
        CK(dev_alloc(&c->rec, (size_t)o.max_batch));
        if (c->n_local > 0) {
            CK(dev_alloc(&c->halo_owner, (size_t)(N - c->n_local), 0xFF));
            CK(dev_alloc(&c->halo_rid, (size_t)(N - c->n_local), 0xFF));
            CK(dev_alloc(&c->silent_dev, (size_t)o.max_batch, 0));
            CK(dev_alloc(&c->rows_sent, (size_t)RP_MAXL + 1, 0));
            c->halo_owner_h = static_cast<int32_t*>(malloc(sizeof(int32_t) * (size_t)std::max(N - c->n_local, 1)));
            c->halo_rid_h = static_cast<int32_t*>(malloc(sizeof(int32_t) * (size_t)std::max(N - c->n_local, 1)));
            if (!c->halo_owner_h || !c->halo_rid_h) { set_err(nullptr, "host allocation failed"); st = RIPPLE_ERR_OOM; goto fail; }
            for (int h = 0; h < N - c->n_local; ++h) c->halo_owner_h[h] = -1;
        }
        CK(cudaDeviceSynchronize());

        {
            const long long e0 = (long long)E;
            CK(cudaMemcpy(&c->ctl->num_edges, &e0, sizeof(e0), cudaMemcpyHostToDevice));
        }
        if (c->n_local == 0) {   // (a partitioned context is bootstrapped layer by layer, in step with its peers)
            st = run_full(c);
            if (st) { memcpy(g_create_err, c->err, sizeof(g_create_err)); goto fail_keep_msg; }
        }
        c->stats.num_layers = L;
        c->stats.num_edges = E;
        *out = reinterpret_cast<ripple_ctx*>(c);
        return RIPPLE_OK;
    }
fail:
    if (c && c->err[0]) memcpy(g_create_err, c->err, sizeof(g_create_err));
fail_keep_msg:
    destroy_ctx(c);
    return st;
}

// The launch chain of one batch: no host decision inside, every size read on the device.
static int enqueue_batch(Ctx* c, int nb, bool stamps) {
    const int L = c->L;
    int evi = 0;
#define STAMP() do { if (stamps) cudaEventRecord(c->ev[evi], c->stream); ++evi; } while (0)
    // A handful of updates: the whole of Apply and the hop-0 sender list in one block (the chain of a small batch
    // is bound by the number of dependent steps, not by their work); also the merged frontier kernel below.
    const bool tiny = nb >= 1 && nb <= RP_TINY_BATCH && !c->may_expand && !c->src_norm && !rp_monotonic(c->agg);
    if (nb >= 1 && nb <= RP_TINY_APPLY && !c->may_expand && !c->src_norm) {
        STAMP();  // 0
        graph_batch_apply_small(c, nb);
        if (rp_monotonic(c->agg)) max_senders_build(c, 0);
    } else {
        RP_LAUNCH(c, k_ctl_reset, 1, 1, 0, c->ctl, c->params_dev);
        STAMP();  // 0
        // Apply (Sec. 3.3): normalise the batch, mutate both adjacency directions, replace features
        graph_batch_classify(c, nb);
        graph_batch_mutate(c, nb);
        frontier_seed_features(c, nb);
        feature_rows(c, nb);
        if (rp_monotonic(c->agg)) max_senders_build(c, 0);
        else senders_build(c, 0, nb);
    }
    STAMP();  // 1
    if (rp_monotonic(c->agg)) {
        // hybrid-incremental hops of a monotonic aggregator (Sec. 3.4.2)
        for (int l = 1; l <= L; ++l) {
            STAMP();
            max_hop(c, l, nb);
            frontier_compact(c, l);
            senders_release(c, l - 1);
            STAMP();
            self_project(c, l, false);
            update_rows(c, l, false);
            if (l < L) max_senders_build(c, l);
            STAMP();
        }
    }
    if (c->attention) {
        // hybrid-incremental hops of attention layers (Sec. 3.4.1)
        for (int l = 1; l <= L; ++l) {
            const bool small = tiny && c->n_words <= RP_TINY_WORDS;
            STAMP();
            att_hop(c, l, nb, small);
            STAMP();
            att_update(c, l, false);
            if (l < L) { if (small) senders_build_small(c, l); else senders_build(c, l, nb); }
            STAMP();
        }
    }
    // one superstep per hop (Sec. 3.3.1): frontier, send + aggregate, compute + prepare
    for (int l = 1; l <= L && !rp_monotonic(c->agg) && !c->attention; ++l) {
        // The push scatter walks the same out-lists as the frontier and marks the sinks itself; the
        // gathering forms need the list A_l first, so the frontier walk is a pass of its own for them
        // (decided per hop on the device for the rebuilding form).
        const bool pull = c->pull_hop[l] != 0;
        choose_direction(c, l);
        frontier_mark(c, l, pull, nb);
        if (pull) frontier_compact(c, l);
        STAMP();
        scatter_layer(c, l, nb);
        // tiny batches on graphs whose frontier bitmap one block can sweep: A_l, and later the next hop's senders,
        // by one launch each instead of two
        const bool merged = tiny && !pull && c->n_words <= RP_TINY_WORDS;
        if (merged) frontier_compact_small(c, l);
        else if (!pull) frontier_compact(c, l);
        if (nb <= 0) senders_release(c, l - 1);   // (otherwise the last kernel of the hop's delta form clears them)
        fold_deltas(c, l);
        regather_layer(c, l);
        STAMP();
        self_project(c, l, false);
        update_rows(c, l, false);
        if (l < L) { if (merged) senders_build_small(c, l); else senders_build(c, l, nb); }
        STAMP();
    }
    graph_batch_cleanup(c, nb);
    STAMP();
#undef STAMP
    return evi;
}

// The choice between pushing and rebuilding a hop is taken on the device, but the kernels of the
// rebuilding form (bottom-up marking, gather) only need to be in the chain when the choice can
// fall on them.  A hop is armed if the last batch brought it within a factor two of the threshold,
// or if nothing comparable is known (first batch, much larger batch).  An unarmed hop pushes even
// if it turns out saturated: slower for that one batch, never wrong, and armed for the next.
static void arm_rebuild(Ctx* c, int nb) {
    const bool no_history = c->batches_done == 0 || nb > 4 * std::max(c->last_nb, 1);
    // the tensor-core update takes over from 1024 rows: in the chain if any frontier of the last batch came near
    c->tc_armed = no_history;
    for (int l = 0; l <= c->L; ++l) c->tc_armed |= c->stats.affected[l] >= 256 || c->stats.senders[l] >= 256;
    for (int l = 1; l <= c->L; ++l) {
        bool armed = false;
        if (rp_monotonic(c->agg) || c->attention) armed = false;
        else if (c->scatter_mode == RIPPLE_SCATTER_REGATHER) armed = true;
        else if (c->scatter_mode == RIPPLE_SCATTER_AUTO && c->regather_threshold[l] > 0.f)
            armed = (no_history || (double)c->stats.active_edges[l] >=
                                       0.5 * (double)c->regather_threshold[l] * (double)c->stats.num_edges) &&
                    c->stats.num_edges + c->max_batch >= c->regather_min_messages;
        c->rebuild_armed[l] = armed;
        // The gathering form of the delta scatter is chosen here, from what the hop carried in the batch before
        // (any choice is correct; a hop that turns out small gathers over a small frontier).
        bool gather = c->scatter_mode == RIPPLE_SCATTER_PULL;
        if (c->scatter_mode == RIPPLE_SCATTER_AUTO && !rp_monotonic(c->agg) && !c->attention && c->n_local == 0 &&
            c->gather_min_width > 0 && c->ws[l] >= c->gather_min_width && !no_history)
            gather = c->stats.active_edges[l] >= c->gather_min_messages && c->stats.scatter_pull[l] != 2 &&
                     // the senders' delta rows stay in L2 with room to spare, and a sink's one addition replaces many
                     (double)c->stats.senders[l - 1] * c->ws[l] * sizeof(float) <= 32.0 * (1 << 20) &&
                     c->stats.active_edges[l] >= 8 * c->stats.affected[l];
        c->pull_hop[l] = gather;
    }
}

// Small batches are launch-bound (about fifty short kernels): their chain is captured once per
// batch size into a CUDA graph and replayed.  Returns false if this batch must take the direct path.
static bool launch_batch_graph(Ctx* c, int nb) {
    if (c->no_graphs || c->timing || nb < 1 || nb > RP_GRAPH_MAX_BATCH) return false;
    // the captured chain differs with the expansion kernels and with the hops whose rebuilding form is enqueued
    int key = 4 * nb + (c->may_expand ? 1 : 0) + (c->has_opw ? 2 : 0);
    key = 2 * key + (c->tc_armed ? 1 : 0);
    key = 2 * key + (c->packed_now ? 1 : 0);   // (the chain holds the addresses its kernels read the batch from)
    for (int l = 1; l <= c->L; ++l) key = 4 * key + (c->rebuild_armed[l] ? 1 : 0) + (c->pull_hop[l] ? 2 : 0);
    int slot = -1;
    for (int i = 0; i < RP_GRAPH_SLOTS; ++i)
        if (c->graph_exec[i] && c->graph_n[i] == key) slot = i;
    if (slot < 0) {
        // Capturing costs a millisecond or more: only a chain that keeps coming back is worth it.  A
        // stream whose batch sizes never repeat is launched kernel by kernel.
        int seen = -1;
        for (int i = 0; i < RP_GRAPH_SEEN; ++i)
            if (c->seen_key[i] == key) seen = i;
        if (seen < 0) {
            seen = c->seen_next++ % RP_GRAPH_SEEN;
            c->seen_key[seen] = key;
            c->seen_count[seen] = 0;
        }
        if (++c->seen_count[seen] < 2) return false;
        slot = c->graph_next++ % RP_GRAPH_SLOTS;
        if (c->graph_exec[slot]) { cudaGraphExecDestroy(c->graph_exec[slot]); c->graph_exec[slot] = nullptr; }
        cudaGraph_t g = nullptr;
        if (cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) { c->no_graphs = 1; return false; }
        c->launches = 0;
        enqueue_batch(c, nb, false);
        cudaError_t e = cudaStreamEndCapture(c->stream, &g);
        if (e == cudaSuccess) e = cudaGraphInstantiate(&c->graph_exec[slot], g, 0);
        if (g) cudaGraphDestroy(g);
        if (e != cudaSuccess) { cudaGetLastError(); c->graph_exec[slot] = nullptr; c->no_graphs = 1; return false; }
        c->graph_n[slot] = key;
        c->graph_launches[slot] = c->launches;
    }
    c->launches = c->graph_launches[slot];
    return cudaGraphLaunch(c->graph_exec[slot], c->stream) == cudaSuccess;
}

extern "C" ripple_status ripple_apply_batch(ripple_ctx* ctx, const ripple_update* ups, int64_t n,
                                            const float* feat_rows, int64_t n_rows, int32_t mem) {
    return ripple_apply_batch_weighted(ctx, ups, n, feat_rows, n_rows, nullptr, mem);
}

extern "C" ripple_status ripple_apply_batch_weighted(ripple_ctx* ctx, const ripple_update* ups, int64_t n,
                                                     const float* feat_rows, int64_t n_rows,
                                                     const float* edge_weights, int32_t mem) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c) return RIPPLE_ERR_INVALID_ARG;
    ripple_status st = RIPPLE_OK;
    if (n < 0 || n_rows < 0 || (n > 0 && !ups) || (n_rows > 0 && !feat_rows) || (mem != 0 && mem != 1)) {
        set_err(c, "bad arguments to ripple_apply_batch");
        return RIPPLE_ERR_INVALID_ARG;
    }
    if (c->n_local > 0) {
        set_err(c, "a partitioned context applies its batches in phases: ripple_part_begin and so on");
        return RIPPLE_ERR_INVALID_ARG;
    }
    if (n > c->max_batch || n_rows > c->max_batch) {
        set_err(c, "batch of %lld updates exceeds max_batch = %lld", (long long)n, (long long)c->max_batch);
        return RIPPLE_ERR_CAPACITY;
    }
    cudaSetDevice(c->device);
    const int nb = (int)n, nr = (int)n_rows, L = c->L;
    if (nb == 0) {   // nothing to apply, nothing to propagate: no device work at all
        ripple_stats& s = c->stats;
        s.gpu_launches = 0;
        s.n_ops = s.n_added = s.n_deleted = s.n_noop_add = s.n_noop_del = s.n_superseded = s.n_feature = s.n_expanded = 0;
        for (int l = 0; l <= L; ++l) s.affected[l] = s.senders[l] = s.active_edges[l] = s.rows_rebuilt[l] = s.in_edges[l] = 0;
        s.ms_total = s.ms_graph = 0.f;
        return RIPPLE_OK;
    }
    float* own_feat = c->feat_dev;
    ripple_update* own_ups = c->ups_dev;
    float* own_opw = c->opw_dev;
    int* own_params = c->params_dev;
    c->launches = 0;
    int evi = 0;
    // A vertex deletion becomes one edge deletion per incident edge on the device.  Launches are
    // sized from the number of operations, so a host batch that holds one is given the geometry
    // of a full batch (device batches are not inspected and keep the geometry of n: still
    // correct, since every kernel strides over the counts it reads from the control block).
    bool wide = false;
    if (mem == RIPPLE_MEM_HOST)
        for (int i = 0; i < nb && !wide; ++i) wide = ups[i].op == RIPPLE_OP_DEL_VERTEX;
    const int ng = wide ? (int)c->max_batch : nb;
    c->may_expand = wide || mem != RIPPLE_MEM_HOST;
    {   // diagnostic: a wait that nothing ends, to exercise the time-out path without faulting the device
        const char* e = getenv("RIPPLE_DEBUG_TC_WITHHOLD");
        c->debug_tc_withhold = e && e[0] == '1';
    }
    arm_rebuild(c, nb);
    const bool try_graph = !wide && !c->no_graphs && !c->timing && nb >= 1 && nb <= RP_GRAPH_MAX_BATCH;
    const cudaMemcpyKind kind = mem == RIPPLE_MEM_HOST ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToDevice;
    c->has_opw = c->weighted && edge_weights && nb;
    // A small host batch without vertex deletions travels in one copy: sizes, operations, weights and payload
    // rows are packed into pinned memory at offsets that depend on the number of operations alone (a captured
    // chain holds them), and the kernels read them where they land.
    const bool packed = mem == RIPPLE_MEM_HOST && !wide && nb >= 1 && nb <= RP_GRAPH_MAX_BATCH && nr <= RP_GRAPH_MAX_BATCH;
    c->packed_now = packed;
    c->few_rows_form = nb <= 128;
    if (packed) {
        auto pad16 = [](size_t x) { return (x + 15) & ~(size_t)15; };
        const size_t off_ups = 16, off_w = off_ups + pad16(sizeof(ripple_update) * (size_t)nb);
        const size_t off_rows = off_w + (c->weighted ? pad16(sizeof(float) * (size_t)nb) : 0);
        const size_t total = off_rows + sizeof(float) * (size_t)nr * c->d[0];
        int* head = reinterpret_cast<int*>(c->stage_host);
        head[0] = nb; head[1] = nr;
        memcpy(c->stage_host + off_ups, ups, sizeof(ripple_update) * (size_t)nb);
        if (c->has_opw) memcpy(c->stage_host + off_w, edge_weights, sizeof(float) * (size_t)nb);
        if (nr) memcpy(c->stage_host + off_rows, feat_rows, sizeof(float) * (size_t)nr * c->d[0]);
        CK(cudaMemcpyAsync(c->stage_dev, c->stage_host, total, cudaMemcpyHostToDevice, c->stream));
        c->params_dev = reinterpret_cast<int*>(c->stage_dev);
        c->ups_dev = reinterpret_cast<ripple_update*>(c->stage_dev + off_ups);
        c->opw_dev = reinterpret_cast<float*>(c->stage_dev + off_w);
        c->feat_dev = reinterpret_cast<float*>(c->stage_dev + off_rows);
    } else {
        // operations are always staged: generated edge deletions are appended behind them
        if (nb) CK(cudaMemcpyAsync(c->ups_dev, ups, sizeof(ripple_update) * (size_t)nb, kind, c->stream));
        if (c->has_opw) CK(cudaMemcpyAsync(c->opw_dev, edge_weights, sizeof(float) * (size_t)nb, kind, c->stream));
        if (mem == RIPPLE_MEM_HOST || try_graph) {
            // a replayed graph reads the library's own staging buffers, so device payload rows are copied too
            if (nr) CK(cudaMemcpyAsync(c->feat_dev, feat_rows, sizeof(float) * (size_t)nr * c->d[0], kind, c->stream));
        } else {
            c->feat_dev = const_cast<float*>(feat_rows);   // device payload rows are read in place
        }
        c->params_host[0] = nb; c->params_host[1] = nr;
        CK(cudaMemcpyAsync(c->params_dev, c->params_host, 2 * sizeof(int), cudaMemcpyHostToDevice, c->stream));
    }
    if (!try_graph || !launch_batch_graph(c, nb)) {
        c->launches = 0;
        evi = enqueue_batch(c, ng, c->timing != 0);
    }
    c->feat_dev = own_feat; c->ups_dev = own_ups; c->opw_dev = own_opw; c->params_dev = own_params;
    st = sync_and_fetch_ctl(c);
    if (st) return st;
    {
        const Ctl& h = *c->ctl_host;
        ripple_stats& s = c->stats;
        s.gpu_launches = c->launches;
        s.n_ops = nb;
        if (h.err) {
            st = (ripple_status)h.err;
            set_err(c, st == RIPPLE_ERR_VERTEX_RANGE ? "batch rejected: vertex id or payload row out of range"
                       : st == RIPPLE_ERR_CAPACITY   ? (h.expand_failed ? "batch rejected: vertex deletions expand to more than max_batch operations"
                                                                         : "batch rejected: overflow edge pool exhausted")
                       : st == RIPPLE_ERR_TIMEOUT    ? "a bounded device-side wait gave up; the embeddings are no longer consistent: destroy the context"
                                                     : "batch rejected: unknown op code");
            s.n_added = s.n_deleted = s.n_noop_add = s.n_noop_del = s.n_superseded = s.n_feature = s.n_expanded = 0;
            for (int l = 0; l <= L; ++l) s.affected[l] = s.senders[l] = s.active_edges[l] = s.rows_rebuilt[l] = 0;
            return st;
        }
        s.n_added = h.n_add; s.n_deleted = h.n_del; s.n_noop_add = h.n_noop_add; s.n_noop_del = h.n_noop_del;
        s.n_superseded = h.n_superseded; s.n_feature = h.n_feat;
        c->batches_done++;
        c->last_nb = nb;
        s.n_expanded = (int64_t)h.n_extra;
        s.num_edges += h.n_add - h.n_del;
        for (int l = 0; l <= L; ++l) {
            s.affected[l] = h.nA[l];
            s.senders[l] = h.nC[l];
            s.active_edges[l] = l ? (int64_t)h.E[l] + h.n_rec : 0;
            s.scatter_pull[l] = h.regather[l] ? 2 : h.pull[l];
            s.in_edges[l] = (int64_t)h.pull_work[l];
            s.message_width[l] = l ? c->ws[l] : 0;
            s.rows_rebuilt[l] = h.n_rebuilt[l];
        }
        s.pool_used = (int64_t)h.pool_next[0] - c->side[0].base_end;
        s.pool_size = c->side[0].col_size - c->side[0].base_end;
        s.pool_free = (int64_t)h.pool_free[0];
        s.pool_lost = (int64_t)h.pool_lost[0];
        if (c->timing) {
            cudaEventElapsedTime(&s.ms_total, c->ev[0], c->ev[evi - 1]);
            cudaEventElapsedTime(&s.ms_graph, c->ev[0], c->ev[1]);
            for (int l = 1; l <= L; ++l) {
                int b = 1 + 3 * (l - 1);
                cudaEventElapsedTime(&s.ms_frontier[l], c->ev[b], c->ev[b + 1]);
                cudaEventElapsedTime(&s.ms_scatter[l], c->ev[b + 1], c->ev[b + 2]);
                cudaEventElapsedTime(&s.ms_update[l], c->ev[b + 2], c->ev[b + 3]);
                cudaEventElapsedTime(&s.ms_scatter_kernel[l], c->ev_sc[2 * l], c->ev_sc[2 * l + 1]);
                s.ms_regather[l] = 0.f;
                if (h.regather[l]) cudaEventElapsedTime(&s.ms_regather[l], c->ev_rg[2 * l], c->ev_rg[2 * l + 1]);
            }
        }
    }
    return RIPPLE_OK;
fail:
    c->feat_dev = own_feat; c->ups_dev = own_ups; c->opw_dev = own_opw; c->params_dev = own_params;
    return st;
}

extern "C" ripple_status ripple_get_embeddings(ripple_ctx* ctx, int32_t layer, const float** dev_ptr, int64_t* ld) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c || !dev_ptr || !ld || layer < 0 || layer > c->L) return RIPPLE_ERR_INVALID_ARG;
    *dev_ptr = c->H[layer];
    *ld = c->ld[layer];
    return RIPPLE_OK;
}

extern "C" ripple_status ripple_get_aggregate(ripple_ctx* ctx, int32_t layer, const float** dev_ptr, int64_t* ld,
                                              int32_t* width, int32_t* transformed) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c || !dev_ptr || !ld || layer < 1 || layer > c->L) return RIPPLE_ERR_INVALID_ARG;
    *dev_ptr = c->S[layer];
    *ld = c->ws[layer];
    const LayerDev& ly = c->layer[layer];
    if (width) *width = c->attention ? ly.d_in + 1 : c->pre[layer] ? (ly.kind == RIPPLE_LAYER_GIN ? ly.d_hid : ly.d_out) : ly.d_in;
    if (transformed) *transformed = c->pre[layer] ? 1 : 0;
    return RIPPLE_OK;
}

extern "C" ripple_status ripple_get_affected(ripple_ctx* ctx, int32_t layer, const int32_t** dev_ids, int64_t* count) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c || !dev_ids || !count || layer < 0 || layer > c->L) return RIPPLE_ERR_INVALID_ARG;
    *dev_ids = c->A[layer];
    *count = c->stats.affected[layer];
    return RIPPLE_OK;
}

extern "C" ripple_status ripple_export_graph(ripple_ctx* ctx, int64_t* rowptr, int32_t* col, int64_t col_capacity) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c || !rowptr || (!col && col_capacity > 0)) return RIPPLE_ERR_INVALID_ARG;
    cudaSetDevice(c->device);
    int64_t ne = 0;
    cudaError_t e = graph_export(c, rowptr, col, nullptr, col_capacity, &ne);
    if (e == cudaErrorInvalidValue) {
        set_err(c, "col_capacity %lld is smaller than the edge count %lld", (long long)col_capacity, (long long)ne);
        return RIPPLE_ERR_INVALID_ARG;
    }
    if (e) { set_err(c, "export failed: %s", cudaGetErrorString(e)); return RIPPLE_ERR_CUDA; }
    return RIPPLE_OK;
}

extern "C" ripple_status ripple_export_graph_weighted(ripple_ctx* ctx, int64_t* rowptr, int32_t* col, float* weight,
                                                      int64_t col_capacity) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c || !rowptr || ((!col || !weight) && col_capacity > 0)) return RIPPLE_ERR_INVALID_ARG;
    cudaSetDevice(c->device);
    int64_t ne = 0;
    cudaError_t e = graph_export(c, rowptr, col, weight, col_capacity, &ne);
    if (e == cudaErrorInvalidValue) {
        set_err(c, "col_capacity %lld is smaller than the edge count %lld", (long long)col_capacity, (long long)ne);
        return RIPPLE_ERR_INVALID_ARG;
    }
    if (e) { set_err(c, "export failed: %s", cudaGetErrorString(e)); return RIPPLE_ERR_CUDA; }
    return RIPPLE_OK;
}

extern "C" ripple_status ripple_get_degrees(ripple_ctx* ctx, const int32_t** deg_out, const int32_t** deg_in) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c || !deg_out || !deg_in) return RIPPLE_ERR_INVALID_ARG;
    *deg_out = c->side[0].deg;
    *deg_in = c->side[1].deg;
    return RIPPLE_OK;
}

extern "C" ripple_status ripple_recompute_full(ripple_ctx* ctx) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c || c->n_local > 0) return RIPPLE_ERR_INVALID_ARG;
    cudaSetDevice(c->device);
    return run_full(c);
}

// ---------------------------------------------------------------------------------------------
// growing the vertex set
// ---------------------------------------------------------------------------------------------
template <typename T>
static cudaError_t grow_array(T** p, size_t old_count, size_t new_count, int fill_byte) {
    if (!*p) return cudaSuccess;
    T* q = nullptr;
    cudaError_t e = cudaMalloc(&q, sizeof(T) * std::max<size_t>(new_count, 1));
    if (e) return e;
    if ((e = cudaMemset(q, fill_byte, sizeof(T) * new_count))) return e;
    if ((e = cudaMemcpy(q, *p, sizeof(T) * std::min(old_count, new_count), cudaMemcpyDeviceToDevice))) return e;
    cudaFree(*p);
    *p = q;
    return cudaSuccess;
}

// ids first .. first + count - 1 into every list a hop reads (A_l, the two sender lists), and their number
// into the control block: the new vertices are then rows of every hop's update
__global__ void k_list_new_vertices(Ctl* ctl, int L, int first, int count, int32_t* const* lists, int n_lists) {
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < count; i += gridDim.x * blockDim.x)
        for (int k = 0; k < n_lists; ++k) lists[k][i] = first + i;
    if (blockIdx.x == 0 && threadIdx.x == 0)
        for (int l = 0; l <= L; ++l) { ctl->nA[l] = count; ctl->nC[l] = count; }
}

extern "C" ripple_status ripple_reserve_vertices(ripple_ctx* ctx, int64_t num_vertices) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c) return RIPPLE_ERR_INVALID_ARG;
    if (c->n_local > 0 || num_vertices <= c->N || num_vertices > 0x7fffffff - 64) {
        set_err(c, "ripple_reserve_vertices: %lld is not above the present capacity %d (or the context is a worker of a partitioned execution)",
                (long long)num_vertices, c->N);
        return RIPPLE_ERR_INVALID_ARG;
    }
    cudaSetDevice(c->device);
    ripple_status st = RIPPLE_OK;
    const size_t N0 = (size_t)c->N, N1 = (size_t)num_vertices;
    const int L = c->L;
    int max_ld = 0, max_hid = 0;
    for (int l = 0; l <= L; ++l) max_ld = std::max(max_ld, c->ld[l]);
    for (int l = 1; l <= L; ++l) if (c->layer[l].kind == RIPPLE_LAYER_GIN) max_hid = std::max(max_hid, c->layer[l].ld_hid);
    CK(cudaStreamSynchronize(c->stream));
    for (auto& g : c->graph_exec) if (g) { cudaGraphExecDestroy(g); g = nullptr; }   // captured chains hold the old addresses
    memset(c->graph_n, 0, sizeof(c->graph_n));
    memset(c->seen_key, 0, sizeof(c->seen_key));
    memset(c->seen_count, 0, sizeof(c->seen_count));
    for (int l = 0; l <= L; ++l) {
        CK(grow_array(&c->H[l], N0 * c->ld[l], N1 * c->ld[l], 0));
        CK(grow_array(&c->A[l], N0 + 32, N1 + 32, 0));
        if (!l) continue;
        CK(grow_array(&c->S[l], N0 * c->ws[l], N1 * c->ws[l], 0));
        CK(grow_array(&c->dS[l], N0 * c->ws[l], N1 * c->ws[l], 0));
        CK(grow_array(&c->Eb[l], N0, N1, 0));
        CK(grow_array(&c->Z[l], N0 * c->ld[l], N1 * c->ld[l], 0));
        CK(grow_array(&c->P[l], N0 * c->ws[l], N1 * c->ws[l], 0));
        CK(grow_array(&c->att_s[l], N0, N1, 0));
        CK(grow_array(&c->att_t[l], N0, N1, 0));
    }
    CK(grow_array(&c->T, N0 * max_hid, N1 * max_hid, 0));
    CK(grow_array(&c->Dt, N0 * max_ld, N1 * max_ld, 0));
    for (int s = 0; s < 2; ++s) {
        CK(grow_array(&c->D[s], N0 * max_ld, N1 * max_ld, 0));
        CK(grow_array(&c->Clist[s], N0 + 32, N1 + 32, 0));
        Side& sd = c->side[s];
        CK(grow_array(&sd.start, N0 + 1, N1 + 1, 0));   // a new row is empty: capacity 0, its first edge takes a block of the pool
        for (int32_t** a : {&sd.cap, &sd.deg, &sd.cnt_del, &sd.cnt_add, &sd.tick_a, &sd.tick_b, &sd.touch}) CK(grow_array(a, N0, N1, 0));
    }
    CK(grow_array(&c->att_so, N0 + 32, N1 + 32, 0));
    if (c->att_items) CK(grow_array(&c->att_items, N0 + (size_t)(c->side[1].col_size / RP_ATT_CHUNK) + 64, N1 + (size_t)(c->side[1].col_size / RP_ATT_CHUNK) + 64, 0));
    {
        const size_t other = (size_t)(c->side[1].col_size / 128) + 64;
        CK(grow_array(&c->coff, std::max(N0 + 2, other), std::max(N1 + 2, other), 0));
    }
    {
        const size_t w0 = (size_t)c->n_words + 256, w1 = (N1 + 31) / 32 + 256;
        CK(grow_array(&c->bitmap, w0, w1, 0));
        CK(grow_array(&c->bitmap2, w0, w1, 0));
    }
    CK(grow_array(&c->old_idx, N0 + 32, N1 + 32, 0));
    CK(grow_array(&c->invmask, N0 * c->mw, N1 * c->mw, 0));
    CK(grow_array(&c->posmap, N0, N1, 0xFF));
    CK(grow_array(&c->deg_out_old, N0, N1, 0xFF));
    CK(grow_array(&c->feat_last, N0, N1, 0xFF));
    CK(grow_array(&c->vdel_seq, N0, N1, 0xFF));
    {
        const int nt = std::max(div_up((int64_t)N1, 1024) + 2, div_up((int64_t)((N1 + 31) / 32), 256) + 2);
        CK(grow_array(&c->tile_sums, (size_t)c->n_tile_sums, (size_t)nt, 0));
        c->n_tile_sums = nt;
    }
    c->N = (int)N1;
    c->n_words = (int)((N1 + 31) / 32);
    {
        // embeddings of the new, isolated vertices: every layer's update (and the cached projections it reads)
        // run over exactly those rows; their aggregates are zero already
        const int first = (int)N0, count = (int)(N1 - N0);
        std::vector<int32_t*> lists;
        for (int l = 0; l <= L; ++l) lists.push_back(c->A[l]);
        lists.push_back(c->Clist[0]);
        lists.push_back(c->Clist[1]);
        int32_t** lists_dev = nullptr;
        CK(cudaMalloc(&lists_dev, sizeof(int32_t*) * lists.size()));
        CK(cudaMemcpy(lists_dev, lists.data(), sizeof(int32_t*) * lists.size(), cudaMemcpyHostToDevice));
        c->launches = 0;
        c->debug_tc_withhold = 0;
        c->tc_armed = 1;
        c->few_rows_form = count <= 256;
        c->params_host[0] = 0; c->params_host[1] = 0;
        cudaMemcpyAsync(c->params_dev, c->params_host, 2 * sizeof(int), cudaMemcpyHostToDevice, c->stream);
        RP_LAUNCH(c, k_ctl_reset, 1, 1, 0, c->ctl, c->params_dev);
        k_list_new_vertices<<<std::min(div_up(count, 256), c->n_sm * 4), 256, 0, c->stream>>>(c->ctl, L, first, count, lists_dev, (int)lists.size());
        for (int l = 1; l <= L && !c->attention; ++l) {   // (attention: an isolated vertex outputs zeros and its logit halves are zero)
            if (c->pre[l]) sender_transform(c, l);
            self_project(c, l, false);
            update_rows(c, l, false);
        }
        RP_LAUNCH(c, k_ctl_reset, 1, 1, 0, c->ctl, c->params_dev);
        st = sync_and_fetch_ctl(c);
        cudaFree(lists_dev);
        if (st) return st;
    }
    return RIPPLE_OK;
fail:
    return st;
}

extern "C" ripple_status ripple_get_stats(ripple_ctx* ctx, ripple_stats* out) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c || !out) return RIPPLE_ERR_INVALID_ARG;
    *out = c->stats;
    return RIPPLE_OK;
}

extern "C" ripple_status ripple_set_timing(ripple_ctx* ctx, int32_t on) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    if (!c) return RIPPLE_ERR_INVALID_ARG;
    c->timing = on ? 1 : 0;
    return RIPPLE_OK;
}

extern "C" const char* ripple_last_error(ripple_ctx* ctx) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    return c ? c->err : g_create_err;
}

extern "C" void ripple_destroy(ripple_ctx* ctx) { destroy_ctx(reinterpret_cast<Ctx*>(ctx)); }

// ---------------------------------------------------------------------------------------------
// partitioned execution (Sec. 4): one worker's phases; see include/ripple_part.h
// ---------------------------------------------------------------------------------------------
static Ctx* worker(ripple_ctx* ctx) {
    Ctx* c = reinterpret_cast<Ctx*>(ctx);
    return (c && c->n_local > 0) ? c : nullptr;
}

// every worker that owns one of this worker's halo slots must have been registered: the exchange kernels
// dereference its buffers
static ripple_status peers_known(Ctx* c) {
    if (c->halo_owner_mask & ~c->peer_mask) {
        set_err(c, "halo slots name workers (mask 0x%x) whose buffers have not been registered (ripple_part_set_peer / ripple_part_ipc_open)",
                c->halo_owner_mask & ~c->peer_mask);
        return RIPPLE_ERR_INVALID_ARG;
    }
    if (c->halo_dirty) {   // no halo slot may name a vertex its owner does not have
        for (int h = 0; h < c->halo_hi; ++h) {
            const int o = c->halo_owner_h[h];
            if (o >= 0 && (int64_t)c->halo_rid_h[h] >= c->peer_n[o]) {
                set_err(c, "halo slot %d names vertex %d of worker %d, which has %lld", h, c->halo_rid_h[h], o, (long long)c->peer_n[o]);
                return RIPPLE_ERR_VERTEX_RANGE;
            }
        }
        c->halo_dirty = 0;
    }
    return RIPPLE_OK;
}

static ripple_status finish_phase(Ctx* c) {
    cudaError_t e = cudaStreamSynchronize(c->stream);
    if (!e) e = cudaGetLastError();
    if (e) {
        set_err(c, "CUDA error in a phase of a partitioned batch: %s", cudaGetErrorString(e));
        return RIPPLE_ERR_CUDA;
    }
    return RIPPLE_OK;
}

extern "C" ripple_status ripple_part_exports_get(ripple_ctx* ctx, ripple_part_exports* out) {
    Ctx* c = worker(ctx);
    if (!c || !out) return RIPPLE_ERR_INVALID_ARG;
    memset(out, 0, sizeof(*out));
    for (int l = 0; l <= c->L; ++l) {
        out->accumulator[l] = c->dS[l]; out->accumulator_ld[l] = l ? c->ws[l] : 0;
        out->embeddings[l] = c->H[l]; out->embeddings_ld[l] = c->ld[l];
    }
    out->frontier_bitmap = c->bitmap;
    out->out_degrees = c->side[0].deg;
    out->num_vertices = c->N;
    return RIPPLE_OK;
}

extern "C" ripple_status ripple_part_set_peer(ripple_ctx* ctx, int32_t rank, const ripple_part_exports* e) {
    Ctx* c = worker(ctx);
    if (!c || !e || rank < 0 || rank >= RIPPLE_MAX_PEERS) return RIPPLE_ERR_INVALID_ARG;
    for (int l = 0; l <= c->L; ++l) {
        if ((l && e->accumulator_ld[l] != c->ws[l]) || e->embeddings_ld[l] != c->ld[l]) {
            set_err(c, "peer %d runs another model: row widths differ at layer %d", rank, l);
            return RIPPLE_ERR_INVALID_ARG;
        }
        c->peer_dS[rank][l] = static_cast<float*>(e->accumulator[l]);
        c->peer_H[rank][l] = static_cast<float*>(e->embeddings[l]);
    }
    c->peer_bitmap[rank] = static_cast<uint32_t*>(e->frontier_bitmap);
    c->peer_deg_out[rank] = static_cast<int32_t*>(e->out_degrees);
    if (e->frontier_bitmap && e->out_degrees) c->peer_mask |= 1u << rank;
    c->peer_n[rank] = e->num_vertices;
    c->halo_dirty = 1;
    {   // a peer of the same process on another GPU: its memory must be opened to this device's kernels
        cudaPointerAttributes at;
        if (e->frontier_bitmap && cudaPointerGetAttributes(&at, e->frontier_bitmap) == cudaSuccess &&
            at.type == cudaMemoryTypeDevice && at.device != c->device) {
            cudaSetDevice(c->device);
            const cudaError_t pe = cudaDeviceEnablePeerAccess(at.device, 0);
            if (pe != cudaSuccess && pe != cudaErrorPeerAccessAlreadyEnabled) {
                set_err(c, "device %d cannot reach the memory of device %d: %s", c->device, at.device, cudaGetErrorString(pe));
                return RIPPLE_ERR_CUDA;
            }
        }
        cudaGetLastError();
    }
    return RIPPLE_OK;
}

extern "C" ripple_status ripple_part_ipc_export(ripple_ctx* ctx, ripple_part_ipc* out) {
    Ctx* c = worker(ctx);
    if (!c || !out) return RIPPLE_ERR_INVALID_ARG;
    static_assert(sizeof(cudaIpcMemHandle_t) == 64, "handle size");
    cudaSetDevice(c->device);
    memset(out, 0, sizeof(*out));
    out->num_layers = c->L;
    out->num_vertices = c->N;
    cudaError_t e = cudaIpcGetMemHandle(reinterpret_cast<cudaIpcMemHandle_t*>(out->frontier_bitmap), c->bitmap);
    if (!e) e = cudaIpcGetMemHandle(reinterpret_cast<cudaIpcMemHandle_t*>(out->out_degrees), c->side[0].deg);
    for (int l = 0; l <= c->L && !e; ++l) {
        out->accumulator_ld[l] = l ? c->ws[l] : 0;
        out->embeddings_ld[l] = c->ld[l];
        if (l) e = cudaIpcGetMemHandle(reinterpret_cast<cudaIpcMemHandle_t*>(out->accumulator[l]), c->dS[l]);
        if (!e) e = cudaIpcGetMemHandle(reinterpret_cast<cudaIpcMemHandle_t*>(out->embeddings[l]), c->H[l]);
    }
    if (e) { set_err(c, "cudaIpcGetMemHandle failed: %s", cudaGetErrorString(e)); return RIPPLE_ERR_CUDA; }
    return RIPPLE_OK;
}

extern "C" ripple_status ripple_part_ipc_open(ripple_ctx* ctx, int32_t rank, const ripple_part_ipc* in) {
    Ctx* c = worker(ctx);
    if (!c || !in || rank < 0 || rank >= RIPPLE_MAX_PEERS || in->num_layers != c->L) return RIPPLE_ERR_INVALID_ARG;
    cudaSetDevice(c->device);
    ripple_part_exports ex;
    memset(&ex, 0, sizeof(ex));
    auto open = [&](const unsigned char* h, void** p) {
        cudaIpcMemHandle_t hh;
        memcpy(&hh, h, sizeof(hh));
        cudaError_t e = cudaIpcOpenMemHandle(p, hh, cudaIpcMemLazyEnablePeerAccess);
        if (!e) c->ipc_opened[c->n_ipc_opened++] = *p;
        return e;
    };
    ex.num_vertices = in->num_vertices;
    cudaError_t e = open(in->frontier_bitmap, &ex.frontier_bitmap);
    if (!e) e = open(in->out_degrees, &ex.out_degrees);
    for (int l = 0; l <= c->L && !e; ++l) {
        ex.accumulator_ld[l] = in->accumulator_ld[l];
        ex.embeddings_ld[l] = in->embeddings_ld[l];
        if (l) e = open(in->accumulator[l], &ex.accumulator[l]);
        if (!e) e = open(in->embeddings[l], &ex.embeddings[l]);
    }
    if (e) { set_err(c, "cudaIpcOpenMemHandle failed: %s", cudaGetErrorString(e)); return RIPPLE_ERR_CUDA; }
    return ripple_part_set_peer(ctx, rank, &ex);
}

extern "C" ripple_status ripple_part_set_halos(ripple_ctx* ctx, int32_t first, int32_t count, const int32_t* owner,
                                               const int32_t* remote_id) {
    Ctx* c = worker(ctx);
    if (!c || first < 0 || count < 0 || (count > 0 && (!owner || !remote_id)) ||
        (int64_t)first + count > (int64_t)c->N - c->n_local)
        return RIPPLE_ERR_INVALID_ARG;
    if (count == 0) return RIPPLE_OK;
    for (int32_t i = 0; i < count; ++i) {
        if (owner[i] < 0 || owner[i] >= RIPPLE_MAX_PEERS || remote_id[i] < 0) {
            set_err(c, "halo slot %d names worker %d, vertex %d", first + i, owner[i], remote_id[i]);
            return RIPPLE_ERR_INVALID_ARG;
        }
        c->halo_owner_mask |= 1u << owner[i];
        c->halo_owner_h[first + i] = owner[i];
        c->halo_rid_h[first + i] = remote_id[i];
    }
    c->halo_hi = std::max(c->halo_hi, first + count);
    c->halo_dirty = 1;
    cudaSetDevice(c->device);
    cudaError_t e = cudaMemcpyAsync(c->halo_owner + first, owner, sizeof(int32_t) * (size_t)count, cudaMemcpyHostToDevice, c->stream);
    if (!e) e = cudaMemcpyAsync(c->halo_rid + first, remote_id, sizeof(int32_t) * (size_t)count, cudaMemcpyHostToDevice, c->stream);
    if (!e) e = cudaStreamSynchronize(c->stream);
    if (e) { set_err(c, "copying the halo table failed: %s", cudaGetErrorString(e)); return RIPPLE_ERR_CUDA; }
    return RIPPLE_OK;
}

extern "C" ripple_status ripple_part_bootstrap_layer(ripple_ctx* ctx, int32_t l) {
    Ctx* c = worker(ctx);
    if (!c || l < 1 || l > c->L) return RIPPLE_ERR_INVALID_ARG;
    if (ripple_status ps = peers_known(c)) return ps;
    cudaSetDevice(c->device);
    c->launches = 0;
    c->params_host[0] = 0; c->params_host[1] = 0;
    cudaMemcpyAsync(c->params_dev, c->params_host, 2 * sizeof(int), cudaMemcpyHostToDevice, c->stream);
    RP_LAUNCH(c, k_ctl_reset, 1, 1, 0, c->ctl, c->params_dev);
    part_fetch_halo_rows(c, l - 1);
    full_layer(c, l);
    c->stats.num_layers = c->L;
    return finish_phase(c);
}

extern "C" ripple_status ripple_part_begin(ripple_ctx* ctx, const ripple_update* ups, int64_t n, const float* feat_rows,
                                           int64_t n_rows, const uint8_t* no_compute, const float* edge_weights,
                                           int32_t mem) {
    Ctx* c = worker(ctx);
    if (!c || n < 0 || n_rows < 0 || (n > 0 && !ups) || (n_rows > 0 && !feat_rows) || (mem != 0 && mem != 1))
        return RIPPLE_ERR_INVALID_ARG;
    if (n > c->max_batch || n_rows > c->max_batch) {
        set_err(c, "batch of %lld updates exceeds max_batch = %lld", (long long)n, (long long)c->max_batch);
        return RIPPLE_ERR_CAPACITY;
    }
    if (mem == RIPPLE_MEM_HOST)
        for (int64_t i = 0; i < n; ++i)
            if (ups[i].op == RIPPLE_OP_DEL_VERTEX) {
                set_err(c, "a partitioned context does not take vertex deletions");
                return RIPPLE_ERR_INVALID_ARG;
            }
    cudaSetDevice(c->device);
    const int nb = (int)n, nr = (int)n_rows;
    const cudaMemcpyKind kind = mem == RIPPLE_MEM_HOST ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToDevice;
    c->launches = 0;
    c->may_expand = 0;
    c->has_opw = c->weighted && edge_weights && nb;
    c->debug_tc_withhold = 0;
    c->tc_armed = 1;
    c->few_rows_form = nb <= 128;
    for (int l = 0; l <= c->L; ++l) c->rebuild_armed[l] = 0;
    if (nb) cudaMemcpyAsync(c->ups_dev, ups, sizeof(ripple_update) * (size_t)nb, kind, c->stream);
    c->has_silent = no_compute && nb;
    if (c->has_silent) cudaMemcpyAsync(c->silent_dev, no_compute, (size_t)nb, kind, c->stream);
    if (c->has_opw) cudaMemcpyAsync(c->opw_dev, edge_weights, sizeof(float) * (size_t)nb, kind, c->stream);
    if (nr) cudaMemcpyAsync(c->feat_dev, feat_rows, sizeof(float) * (size_t)nr * c->d[0], kind, c->stream);
    c->params_host[0] = nb; c->params_host[1] = nr;
    cudaMemcpyAsync(c->params_dev, c->params_host, 2 * sizeof(int), cudaMemcpyHostToDevice, c->stream);
    cudaMemsetAsync(c->rows_sent, 0, sizeof(unsigned long long) * (RP_MAXL + 1), c->stream);
    // launch geometry for at least one operation: a worker with an empty share still takes part in every hop
    c->part_nb = std::max(nb, 1);
    RP_LAUNCH(c, k_ctl_reset, 1, 1, 0, c->ctl, c->params_dev);
    graph_batch_classify(c, c->part_nb);
    graph_batch_mutate(c, c->part_nb);
    frontier_seed_features(c, c->part_nb);
    feature_rows(c, c->part_nb);
    senders_build(c, 0, c->part_nb);
    ripple_status st = sync_and_fetch_ctl(c);
    if (st) return st;
    c->stats.n_ops = nb;
    if (c->ctl_host->err) {
        st = (ripple_status)c->ctl_host->err;
        set_err(c, "batch rejected by a worker (status %d)", (int)st);
        graph_batch_cleanup(c, c->part_nb);
        finish_phase(c);
        return st;
    }
    return RIPPLE_OK;
}

extern "C" ripple_status ripple_part_hop_send(ripple_ctx* ctx, int32_t l) {
    Ctx* c = worker(ctx);
    if (!c || l < 1 || l > c->L) return RIPPLE_ERR_INVALID_ARG;
    if (ripple_status ps = peers_known(c)) return ps;
    cudaSetDevice(c->device);
    scatter_layer(c, l, c->part_nb);
    part_ship(c, l);
    return finish_phase(c);
}

extern "C" ripple_status ripple_part_hop_compute(ripple_ctx* ctx, int32_t l) {
    Ctx* c = worker(ctx);
    if (!c || l < 1 || l > c->L) return RIPPLE_ERR_INVALID_ARG;
    cudaSetDevice(c->device);
    frontier_compact(c, l);
    fold_deltas(c, l);
    self_project(c, l, false);
    update_rows(c, l, false);
    if (l < c->L) senders_build(c, l, c->part_nb);
    return finish_phase(c);
}

extern "C" ripple_status ripple_part_end(ripple_ctx* ctx) {
    Ctx* c = worker(ctx);
    if (!c) return RIPPLE_ERR_INVALID_ARG;
    cudaSetDevice(c->device);
    graph_batch_cleanup(c, c->part_nb);
    ripple_status st = sync_and_fetch_ctl(c);
    if (st) return st;
    const Ctl& h = *c->ctl_host;
    ripple_stats& s = c->stats;
    s.gpu_launches = c->launches;
    s.n_added = h.n_add; s.n_deleted = h.n_del; s.n_noop_add = h.n_noop_add; s.n_noop_del = h.n_noop_del;
    s.n_superseded = h.n_superseded; s.n_feature = h.n_feat;
    s.num_edges += h.n_add - h.n_del;
    c->batches_done++;
    for (int l = 0; l <= c->L; ++l) {
        s.affected[l] = h.nA[l];
        s.senders[l] = h.nC[l];
        s.active_edges[l] = l ? (int64_t)h.E[l] + h.n_rec : 0;
        s.scatter_pull[l] = 0;
        s.message_width[l] = l ? c->ws[l] : 0;
    }
    return RIPPLE_OK;
}

extern "C" ripple_status ripple_part_rows_sent(ripple_ctx* ctx, int64_t* out) {
    Ctx* c = worker(ctx);
    if (!c || !out) return RIPPLE_ERR_INVALID_ARG;
    cudaSetDevice(c->device);
    unsigned long long tmp[RP_MAXL + 1];
    if (cudaMemcpy(tmp, c->rows_sent, sizeof(tmp), cudaMemcpyDeviceToHost) != cudaSuccess) return RIPPLE_ERR_CUDA;
    for (int l = 0; l <= RP_MAXL; ++l) out[l] = (int64_t)tmp[l];
    return RIPPLE_OK;
}

extern "C" const char* ripple_version(void) { return "ripple-b200 0.1 (sm_100a)"; }
