// Time stamps of the roles of the tcgen05 decode kernel.  Compiled in only with -DCOOPT_TRACE (the separate
// library libcoopt_trace.so); the ordinary library contains none of this.  A stamp is the SM's cycle counter
// written to slot `s` of the CTA's record in a caller-supplied buffer (coopt_trace_set_buffer); two slots
// hold the global nanosecond timer at entry and exit so that the CTAs of a launch can be laid side by side.
#pragma once

#include <stdint.h>

namespace coopt {

enum TraceSlot {
  kTrEntry = 0,        // first instruction of the CTA (cycles; every other cycle stamp is read against this one)
  kTrEntryNs,          // global timer at entry
  kTrSetupDone,        // barriers initialised, tensor memory allocated, plan in shared memory
  kTrIdsStaged,        // block ids of the first round staged: the copy warp may start
  kTrFirstCopy,        // first tile requested
  kTrFirstLanded,      // first tile's bytes have landed (seen by the lane that issues the logits)
  kTrFirstProbs,       // probabilities of the first tile written (team 0)
  kTrLastCopy,         // last tile requested
  kTrLastLanded,       // last tile's bytes have landed
  kTrLastPv,           // last P V group committed
  kTrTeamsDone,        // team 0 has handed over its last piece
  kTrLastHandOff,      // epilogue warp has received the last segment
  kTrPieceStored,      // last piece written to the workspace (before the counter)
  kTrCounted,          // counter round trip done
  kTrEpilogueDone,     // last store / merge done
  kTrExit,             // behind the final barrier
  kTrExitNs,           // global timer at exit
  kTrWriteDone,        // fused step: the new tokens' granules are written
  kTrNumSeg,           // number of segments of the first round (a count, not a time)
  kTrNumTiles,         // tiles of the CTA (a count)
  kTrSmId,             // the SM the CTA ran on
  kTrProducerPlan,     // the copy warp has seen the plan
  kTrPrevExitNs,       // what kTrExitNs held at entry: the exit of this CTA's slot in the launch before
  kTrFirstCopyReady,   // the copy warp is about to request the first tile (rows worked out, byte count posted)
  kTrSegBase = 24,     // 24 + i: epilogue warp received segment i (i < 20)
  kTrTeamSegBase = 44, // 44 + i: team 0 began segment i (i < 20)
  kTrCopyTileBase = 64,    // 64 + i: tile i requested (i < 32)
  kTrProbsTileBase = 96,   // 96 + i: probabilities of tile i written by its team (i < 32)
  kTrSegTileBase = 128,    // 128 + i: 1 + number of the first tile of segment i (i < 20; a count)
  kTrLogitsTileBase = 148, // 148 + i: logits of tile i issued (i < 32)
  kTrPvTileBase = 180,     // 180 + i: P V of tile i issued (i < 32)
  kTraceSlots = 256
};
constexpr int kTraceMaxCtas = 1024;

#ifdef COOPT_TRACE
unsigned long long* trace_buffer();      // host: what coopt_trace_set_buffer registered (nullptr = none)
int trace_plan_rotate();                 // host: what coopt_trace_set_rotate registered
#ifdef __CUDACC__
__device__ __forceinline__ void trace_put(unsigned long long* buf, int slot, unsigned long long v) {
  if (buf != nullptr && blockIdx.x < kTraceMaxCtas && slot < kTraceSlots) buf[blockIdx.x * kTraceSlots + slot] = v;
}
__device__ __forceinline__ unsigned long long trace_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
#define COOPT_TRACE_CYCLES(buf, slot, cond) do { if (cond) ::coopt::trace_put((buf), (slot), static_cast<unsigned long long>(clock64())); } while (0)
#define COOPT_TRACE_NS(buf, slot, cond) do { if (cond) ::coopt::trace_put((buf), (slot), ::coopt::trace_ns()); } while (0)
#define COOPT_TRACE_VALUE(buf, slot, cond, v) do { if (cond) ::coopt::trace_put((buf), (slot), static_cast<unsigned long long>(v)); } while (0)
#endif
#else
#define COOPT_TRACE_CYCLES(buf, slot, cond) do { } while (0)
#define COOPT_TRACE_NS(buf, slot, cond) do { } while (0)
#define COOPT_TRACE_VALUE(buf, slot, cond, v) do { } while (0)
#endif

}  // namespace coopt
