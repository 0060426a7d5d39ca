// Shared device/host structures of the decode library.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "adadecode.h"

namespace ada {

constexpr int kMaxRows = 128;       // rows (tokens) one layer pass can carry (a block of a dense prompt pass)
constexpr int kAttnChunk = 128;     // attention split size; chunk c covers positions [128c, 128c+127]
constexpr int kMaxTape = 4096;
constexpr int kHeadLogCap = 1 << 16;

// One row = one token travelling through a layer pass.  Rebuilt by the begin kernels of every
// step (Algorithm 1: the rows of layer l are P[l] (+) t_i, a contiguous suffix of the sequence).
struct RowTable {
    int32_t n_rows;                 // rows with a valid entry
    int32_t seq[kMaxRows];
    int32_t pos[kMaxRows];          // absolute position in the sequence
    int32_t first_layer[kMaxRows];  // 0-based layer at which the row resumes; INT_MAX = idle
};

struct DevStats {
    long long steps, head_evals, early_exits, verify_steps, accepted, rejected, discarded, row_layers, truncated;
    long long exits_at_layer[ADA_MAX_LAYERS];
    long long layer_passes;              // counted on the device by the persistent kernel
    long long phase_ns[ADA_PROF_CLASSES];    // device time per phase class (persistent kernel, measured in CTA 0)
    long long phase_count[ADA_PROF_CLASSES];
};

// Device-resident decoding state of a session.
struct DevState {
    int32_t batch, slots, n_layers, max_seq;
    int32_t len[ADA_MAX_BATCH];         // tokens in the sequence, tentative tail and newest included
    int32_t base[ADA_MAX_BATCH];        // position held by row slot 0 (first token not complete at all layers)
    int32_t n_prompt[ADA_MAX_BATCH];
    int32_t target_len[ADA_MAX_BATCH];  // sequence length at which the current call ends
    int32_t climbing[ADA_MAX_BATCH];    // newest token still climbing in the current step
    int32_t done[ADA_MAX_BATCH];        // call finished for this sequence
    int32_t n_climbing, n_done;
    int32_t step_no;
    // parameters of the current adaptive call
    float gamma;
    int32_t max_early;
    int32_t eos_id;                     // end-of-sequence token of the current call (-1: none)
    int32_t eos_hit[ADA_MAX_BATCH];     // the call ended this sequence on a verified end-of-sequence token
    // debug: forced decisions (sequence 0), head log, logits capture
    int32_t tape_n, tape_i;
    uint8_t tape[kMaxTape];
    int32_t head_log_n;
    int32_t capture_cap, capture_n;     // final-logit capture (sequence 0)
    int32_t keep_rows;                  // rows of sequence 0 whose logits the last verification kept
    int32_t keep_row0;                  // first of those rows in the logits staging buffer
    int32_t pf_pos, pf_end;             // persistent-kernel prefill: next prompt position, prompt length (0: not prefilling)
    DevStats st;
};

struct HeadResult {
    int32_t token;
    float p;       // probability of `token` under the head (max softmax)
    float zmax;    // its (scaled) logit
    float sumexp;  // sum_v exp(z_v - zmax)
};

}  // namespace ada
