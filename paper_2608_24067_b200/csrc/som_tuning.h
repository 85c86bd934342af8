// Geometry tunables of the row-table search kernel, set through som_set_option (include/som.h).
// They exist for benchmarking and for the tests that walk every template instance; 0 always means
// "the measured default".  A reusable plan (som_plan_create) is tied to their values at its creation.
//
//   key 1  hot rows kept in shared memory beside the 16 mask rows (default: 330 rows of 512 bytes, 720 (fp16 wide rows: 676) of
//          256 bytes, 1376 / 1456 of 128 bytes: what keeps table + slot rings under 196 KB, so that the
//          SM keeps a 60 KB L1)
//   key 2  block size: 512, 576 (wide fp32 layout only), 640, 768, 896, 1024
//   key 3  neurons per lane: fp32 storage 4, 8 (needs M % 64 == 0), 16 (M % 128 == 0); fp16 storage 8,
//          16 (M % 128 == 0); default: the widest that divides M (fp32 with the two-stage search: 8)
//   key 4  sample parts per neuron range (default: see som_table_default_parts in som_plan.cuh)
//   key 8  how many of the 16 most frequent features of a batch are handled as mask bits (1..16); default:
//          floor(log2(samples)) - 8, less floor((floor(log2(ranges of 128 neurons)) - 3) / 2) (at most 4) where the
//          search prunes; at least 4, at most 16 (see plan_split in som_plan.cu)
//   key 9  slot and key stream loaded with the L2 "evict last" policy: 0 = when the stream is at most 24 MB (then
//          it stays L2-resident from one neuron range to the next: 1024 x 1024 with 250k samples moves 223 GB
//          instead of 257 GB and runs 0.4 % faster), 1 = always, 2 = never
//   key 10 pruning by range maxima in the row-table kernel (M % 128 == 0; exact, see k_bmu_table): 0 = on
//          maps of at least 32 ranges of 128 neurons, 1 = wherever som_norms has written the maxima, 2 = off
//          (set before the first som_norms, it also spares the V * M / 128 floats of the maxima)
#pragma once
#define SOM_OPT_HOT_ROWS 1
#define SOM_OPT_THREADS 2
#define SOM_OPT_LANE_NEURONS 3
#define SOM_OPT_PARTS 4
#define SOM_OPT_MASK_BITS 8
#define SOM_OPT_FEED_KEEP 9
#define SOM_OPT_PRUNE 10
