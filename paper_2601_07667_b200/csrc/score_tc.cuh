// Plan of the tensor-core scorer: work units and segments built at plan time.
#pragma once
#include <stdint.h>
#include <vector>

constexpr int ASL_TC_KEY_TILE = 128;

// a run of consecutive key tiles of one (request, kv head, row chunk)
struct TcUnit { int32_t b, h, chunk, tile0, ntiles, seg, split, pad; };
// all units of one (request, kv head, row chunk)
struct TcSeg { int32_t unit0, nunits, b, h, chunk, pad0, pad1, pad2; };

struct AslTcPlan {
  bool enabled = false;
  int NC = 0;         // query rows per chunk (MMA N in pass 2)
  int nchunk = 0;     // chunks per kv head
  std::vector<TcUnit> units1, units2;   // pass 1 (all keys), pass 2 (past keys)
  std::vector<TcSeg> segs1;
  TcUnit* d_units1 = nullptr;
  TcUnit* d_units2 = nullptr;
  TcSeg* d_segs1 = nullptr;
};
