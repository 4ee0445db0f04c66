// Plan of the tensor-core scorer: the phase list built at plan time.
#pragma once
#include <stdint.h>
#include <vector>

constexpr int ASL_TC_KEY_TILE = 128;

// one pass over the 128-key tiles of one segment = (request, kv head, row chunk);
// its tiles are the global work items g0 .. g0 + ntiles - 1
// (T, t_off, tok_off: the request's past length, score offset and first token, copied here so that
// one record is all a role needs when it enters the phase)
// rows: query rows of the chunk that exist (the last chunk of a kv head may be padded up to NC)
// kscale: factor between the accumulator and q.k (1 for bf16 keys; k_scale[h] / 16 for FP8 keys, whose
// queries are scaled by 16 before they are split into two E4M3 terms)
struct TcPhase { int32_t g0, ntiles, pass, seg, b, h, chunk, ncontrib, T, t_off, tok_off, rows; float kscale; };

struct AslTcPlan {
  bool enabled = false;
  int NC = 0;           // query rows per chunk (MMA N in pass 2)
  int nchunk = 0;       // chunks per kv head
  int nseg = 0;         // segments
  int grid = 0;         // CTAs of the persistent kernel (one per SM)
  int group = 0;        // segments whose pass 1 runs before their pass 2
  int32_t total_items = 0;
  std::vector<TcPhase> phases;   // both passes
  TcPhase* d_phases = nullptr;
  int32_t n_phases2 = 0;         // the pass-2 phases alone (scoring with a supplied log-sum-exp)
  int32_t total_items2 = 0;
  TcPhase* d_phases2 = nullptr;
  uint32_t* d_sync = nullptr;   // [nseg] publish counters, [nseg] folded-row counters, launch number, exit ticket
  // device-side controller: the phase list of the next launch without the finished requests' phases,
  // written ahead of the launch (capacity: the longer of the two static lists), and its header
  // {phases, work items}
  TcPhase* d_live = nullptr;
  int32_t* d_live_hdr = nullptr;
};
