// Numbering of the output tiles of the tensor-core kernel, shared by the kernel and by the
// kernel that adds the pieces of stream-K tiles.
#pragma once
#include <stdint.h>

#include "gett_dims.h"

#define GETT_RASTER_M 16 // tile rows per rasterisation panel

// Tile number t -> (tile row, tile column).  Tiles are numbered panel by panel: a panel is
// GETT_RASTER_M tile rows high and spans all tile columns, and inside it the row index runs
// fastest, so the tiles in flight at any time share few rows of A and columns of B.
GETT_HD void gett_raster_tile(uint32_t t, uint32_t tiles_m, uint32_t tiles_n, uint32_t& tm, uint32_t& tn)
{
    const uint32_t per_panel = GETT_RASTER_M * tiles_n;
    const uint32_t panel = t / per_panel;
    const uint32_t first_m = panel * GETT_RASTER_M;
    const uint32_t left = tiles_m - first_m;
    const uint32_t rows = left < GETT_RASTER_M ? left : GETT_RASTER_M;
    const uint32_t in_panel = t - panel * per_panel;
    tn = in_panel / rows;
    tm = first_m + (in_panel - tn * rows);
}
