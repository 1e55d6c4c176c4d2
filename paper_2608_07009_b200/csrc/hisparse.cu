// HiSparse selection resolution for B200 (sm_100a): kernels and the C-ABI declared in hisparse.h.
//
// Data layout in HBM (N requests, L layers in G = L / layers_per_group groups, B slots, k selections,
// E bytes per record):
//   pool      uint8  [L][N][B+1][E]   cache pools; slot B of each (r, l) is the reserved newest-record slot
//   slot_pos  int32  [N][G][B]        position held by each slot, -1 = empty
//   last_use  uint32 [N][G][B]        recency stamps: 2t+1 hit at resolve t, 2t fetched at resolve t, 0 unused
//   order     uint16 [N][G][B]        slots from least to most recent: equal to sorting the slots by (last_use,
//                                     slot) whenever order_t == t.  Kept so that victim choice is a prefix scan,
//                                     not a sort; resolves without misses leave it behind (rebuild_order)
//   order_t   uint32 [N][G]           resolve count the list is current for
//   pos2slot  int16  ragged [N][G][capacity[r] rounded up to 8]  the page table (Sec. 3.2), -1 = host-only; every
//                                     slice starts on a 16-byte boundary
//   plan_*    int32  [N][G][k]        miss plan of the last anchor resolve (Sec. 3.5)
// All step-dependent scalars (resolve counters, number of appends, plan sizes) live in device memory so
// that every launch is replayable from a CUDA graph.
//
// The Resolve kernel (Sec. 3.4, Phases 1-5) runs one thread-block cluster per request.  The cluster's first
// block does the metadata: bulk copies stage the selected row and (when it fits) the request's slice of the page table
// in shared memory; every thread looks its few row entries up in the page table, marks hit slots with a byte store,
// writes its part of the slot table and the block votes on "did anything miss?".  If nothing did, the hit stamps go
// out in slot order from the marks and the request is done (the recency list is left behind, see rebuild_order).
// Otherwise the misses are ranked in selection order (ballots), and as soon as their positions exist the records
// start travelling host -> shared memory -> cache slot with cp.async.bulk in both directions (Phase 4); while the
// first loads fly the block walks the recency order once to split the non-hit slots into the first m (victims, needed
// only when a record is stored) and the rest, and rewrites the order as (untouched ++ victims by slot ++ hits by
// slot); the plan is published to the other blocks of the cluster, which take their share of the records, so the
// fetch parallelism does not depend on the number of requests.
// The launch carries the programmatic-dependent-launch attribute: everything before griddepcontrol.wait depends on
// nothing an earlier kernel wrote.  Blocks have 1024 threads and an SM each; a grid of more blocks than SMs is
// launched as one resident wave of 512-thread blocks (three or two per SM) that loop over the requests.
#include "hisparse.h"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "device_common.cuh"
#include "resolve_kernel.cuh"
#include "aux_kernels.cuh"
#include "attention_kernel.cuh"
#include "host_api.inl"
#include "noalloc.inl"
