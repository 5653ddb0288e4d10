// Workspace layouts (host-side arithmetic only; used by the size query and by the launchers).
#pragma once

#include <stddef.h>
#include <stdint.h>

namespace bof4 {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---------------------------------------------------------------- EM workspace
// [0, kEmPartialBytes)            per-CTA partial records of the MSE / error reduction
// [kEmMaeOffset, +kEmMaeBytes)    weighted-median selection state and histograms (MAE)
constexpr int kEmGrid = 148;              // CTAs of the accumulation kernels (1 per SM)
constexpr int kEmRecordDoubles = 64;      // 16 s1 + 16 s0 + 16 count + sum w^2, padded to 512 B
constexpr int kEmRecords = kEmGrid + 1;    // one per CTA, and one for the short last blocks of ragged tensors
constexpr size_t kEmPartialBytes = (size_t)kEmRecords * kEmRecordDoubles * 8;
constexpr size_t kEmTicketOffset = kEmPartialBytes;  // arrival counter of the accumulation CTAs (4 bytes)
constexpr int kMaeDigitBits = 9;          // key bits resolved per selection pass
constexpr int kMaeBins = 1 << kMaeDigitBits;  // bins per level and selection pass
constexpr int kMaeMaxPasses = 4;          // 31 key bits / 9 bits per pass
constexpr size_t kEmMaeOffset = 512 * 1024;
constexpr size_t kEmMaeStateBytes = 4096;  // selection state (struct MaeState)
// bf16 first pass: 2 x kFineStride slots (see em_mae.cu); later passes: 16 x kMaeBins digit bins
constexpr int kFineScale = 2048;                 // fine bins per unit of the normalised weight
constexpr int kFineBins = 2 * kFineScale + 1;    // fine bin of x in [-1, 1]: RN(2048 x) + 2048
constexpr int kFineStride = 4112;                // slots per half (below / not below the bin's threshold)
constexpr int kFineSlots = 2 * kFineStride;
constexpr size_t kEmMaeHistBytes = 66048;        // weight histogram, then count histogram (>= 8 * kFineSlots)
static_assert(kEmMaeHistBytes >= (size_t)kFineSlots * 8 && kEmMaeHistBytes >= (size_t)16 * kMaeBins * 8, "histogram space");
constexpr int kMaeCand = 1 << 16;          // smallest candidate list per level (entries of 8 bytes)
constexpr int kMaeCandMax = 1 << 23;       // largest one a workspace is sized for (1 GiB for the 16 lists)
constexpr size_t kEmMaeCandBytes = (size_t)16 * kMaeCand * 8;
constexpr size_t kEmMaeBytes = kEmMaeStateBytes + 2 * kEmMaeHistBytes + kEmMaeCandBytes;

// Smallest workspace of the fit (any input size).
inline size_t em_workspace_bytes() { return kEmMaeOffset + align_up(kEmMaeBytes, 256); }
// Workspace for n_max weights in total: the candidate lists of the median selection grow with the
// data (n_max / 1024 entries per level, within [kMaeCand, kMaeCandMax]: n_max / 8 bytes in all) so
// that the pass after the first can collect a region's remaining candidates; with smaller lists
// one more data pass runs.
inline size_t em_workspace_bytes_for(int64_t n_max)
{
    int64_t cand = n_max / 1024;
    cand = cand < kMaeCand ? kMaeCand : (cand > kMaeCandMax ? kMaeCandMax : cand);
    return kEmMaeOffset + align_up(kEmMaeStateBytes + 2 * kEmMaeHistBytes + (size_t)16 * (size_t)cand * 8, 256);
}
// Entries per level that the candidate lists of a workspace of ws_bytes hold.
inline uint32_t mae_cand_capacity(size_t ws_bytes)
{
    const size_t fixed = kEmMaeOffset + kEmMaeStateBytes + 2 * kEmMaeHistBytes;
    const size_t cap = ws_bytes > fixed ? (ws_bytes - fixed) / (16 * 8) : 0;
    return (uint32_t)(cap > (size_t)kMaeCandMax ? (size_t)kMaeCandMax : cap);
}

// ---------------------------------------------------------------- OPQ workspace
// The weights are cut into tiles of kOpqTile elements (one warp iteration).  Each tile has a
// count and a staging slot of kOpqStage outliers; tiles are scanned in chunks of kOpqChunk.
constexpr int kOpqTile = 512;
constexpr int kOpqStage = 16;
constexpr int kOpqChunk = 2048;

struct OpqLayout {
    int64_t tiles, chunks;
    size_t counts, chunk_off, stage_idx, stage_val, total;
};

inline OpqLayout opq_layout(int64_t n)
{
    OpqLayout L;
    L.tiles = (n + kOpqTile - 1) / kOpqTile;
    L.chunks = (L.tiles + kOpqChunk - 1) / kOpqChunk;
    size_t off = 0;
    L.counts = off;
    off = align_up(off + (size_t)L.tiles * 4, 256);
    L.chunk_off = off;
    off = align_up(off + (size_t)(L.chunks + 1) * 8, 256);
    L.stage_idx = off;
    off = align_up(off + (size_t)L.tiles * kOpqStage * 4, 256);
    L.stage_val = off;
    off = align_up(off + (size_t)L.tiles * kOpqStage * 2, 256);
    L.total = off < 256 ? 256 : off;
    return L;
}

}  // namespace bof4
