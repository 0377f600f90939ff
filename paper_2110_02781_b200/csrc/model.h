// Host-side model object: unit table, arena layout, execution and gradient-buffer plan.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <vector>
#include "common.h"
#include "kernels.h"

namespace ftp {

enum KernelId {
    K_CONV_FWD_F32 = 0, K_CONV_DGRAD_F32, K_CONV_WGRAD_F32, K_BN_STATS, K_BN_FINALIZE, K_BN_APPLY, K_BN_BWD_REDUCE,
    K_BN_BWD_FINALIZE, K_BN_BWD_APPLY, K_ACT_BIAS_BWD, K_DW_FWD, K_DW_DGRAD, K_DW_WGRAD, K_MAXPOOL_FWD,
    K_MAXPOOL_BWD, K_GAP_FWD, K_GAP_BWD, K_SOFTMAX_CE, K_SGD, K_ACT_FWD, K_ACT_BWD, K_COPY, K_GEMM_BF16_FWD,
    K_GEMM_BF16_DGRAD, K_GEMM_BF16_WGRAD, K_CONV_FWD_BF16_SIMT, K_CONV_DGRAD_BF16_SIMT, K_CONV_WGRAD_BF16_SIMT, K_TC32_FWD, K_TC32_DGRAD, K_TC32_WGRAD, K_COUNT
};

struct Op {
    ftp_layer_desc d;
    int N, H, W, C;          // input shape
    int Ho, Wo, Co;          // output shape
    long long in_elems, out_elems;
    ConvGeom g;
    long long w_off, w_cnt;  // first trainable array (conv / dw weights, BN gamma), floats, canonical order
    long long b_off, b_cnt;  // second trainable array (bias, BN beta)
    long long rm_off, rv_off;  // BN running mean / variance in the state arena
    void* out;               // internal output buffer
    bool out_f32;            // output kept in float whatever the precision (logits, loss)
    float *scale, *shift, *mean, *mean_lo, *rstd, *offset, *coef;   // BN per-channel tables
    FoldPlan fold;
    bool fused_add;          // BN whose normalised output goes straight through the following residual add
    bool skip;               // residual add folded into the preceding BN
    bool defer;              // BN whose normalised output is never stored: the next op of the unit applies it to what it loads
    int gslot;               // slot holding the gradient w.r.t. this op's output (-1 none, -2 dlogits)
    int galias;              // op whose output-gradient buffer this op's output gradient shares
    int addend_of;           // when writing the gradient of this op's input, add the gradient buffer of that op's output
};

struct Arena {
    float* w;
    float* m;
    float* run;
    __nv_bfloat16* wb;       // bf16 copy of w, same layout
    __nv_bfloat16* wbt;      // bf16 copy with every 1x1-convolution matrix transposed ([cout][cin]): the forward's K-major B operand
    // float models, for the split-tf32 tensor-core products: wl = w - trunc_tf32(w), same layout as w (data gradient);
    // wt / wtl = every 1x1-convolution matrix transposed, as it is and its lo part (forward)
    float* wl; float* wt; float* wtl;
};

struct TraceSlot { cudaEvent_t e0, e1; ftp_trace_rec rec; };

}  // namespace ftp

struct SidePending { const void* buf; cudaEvent_t done; };

struct ftp_model {
    ftp_model_cfg cfg;
    std::vector<ftp::Op> ops;
    int L;
    int esize;                                    // bytes per activation element
    std::vector<int> unit_first, unit_last;       // op index range of each unit
    std::vector<long long> unit_p_off, unit_p_cnt, unit_s_off, unit_s_cnt;
    long long P, R;
    std::vector<ftp::Arena> arena;
    float* grad;
    std::vector<int> owner;                       // unit -> arena of the worker that holds it
    std::vector<int> worker;                      // stage -> arena (a worker keeps its arena when failures renumber the stages)
    std::vector<int> points;
    int n_stages;
    std::vector<char> mom_init;                   // per unit: momentum buffer holds a value
    std::vector<void*> slots;
    size_t slot_bytes;
    float* red_scratch; size_t red_floats;
    double* fold_scratch; size_t fold_doubles;
    ftp::FinScratch fin; size_t fin_counter_bytes;
    // weight gradients run on a second stream beside the chain of input gradients; they have scratch of their own
    float* red_side; ftp::FinScratch fin_side;
    cudaStream_t side; std::vector<cudaEvent_t> ev_fork, ev_side; bool overlap; bool producer_stats; bool bwd_sums_on;
    float* dw_part[4]; int dw_rot = 0; bool dw_fin_side = true;   // partial sums of the fused depthwise backward kernels, in turn: their second pass runs on the second stream
    std::vector<SidePending> pending;             // buffers that weight gradients on the second stream still read, with the event that ends the read
    bool side_unjoined = false;                   // the second stream holds work the caller's stream has not waited for yet
    bool defer_join = false;                      // the training step joins the second stream once, before the update, instead of after every stage
    std::vector<ftp::TransposeEntryDev> tp_host; std::vector<int> tp_first;   // tp_first[u]: first entry of unit u (L + 1 values)
    ftp::TransposeEntryDev* tp_dev;
    void* dpre; size_t dpre_bytes;
    int* tc_err;                                  // device word set by a tensor-core kernel whose bounded wait ran out
    float* fc_in; float* fc_din;                  // bf16 models: the classifier's input and input gradient widened to float
    float* dlogits; float* per_sample; float* loss_dev; int32_t* labels_dev; void* input_dev; float* state_backup;
    float* pinned; size_t pinned_bytes;
    char* ws_base; std::vector<size_t> guards;    // device workspace and the offsets of its guard zones
    // run-time state of the last forward of each range
    std::vector<const void*> stage_in;            // act_in of the range starting at op i
    std::vector<void*> cur_out;                   // resolved output pointer of op i
    std::vector<char> fwd_done;
    // per-stage timing of ftp_train_step (Sec. III-B: a worker reports the execution time of its batch)
    bool stage_timing = false;
    std::vector<cudaEvent_t> ev_sf, ev_sb;        // forward / backward boundaries, max_stages + 1 each
    int timed_stages = 0;                         // stages of the last timed step (0: none yet)
    const int32_t* cur_labels;
    // trace
    bool trace;
    std::vector<ftp::TraceSlot> tr;
    size_t tr_used;
    // per-unit profiling events
    bool unit_events;
    std::vector<cudaEvent_t> ev_f, ev_b;
};
