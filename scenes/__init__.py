"""Seeded synthetic input generators shared by the oracle tests and the CUDA path (inputs only)."""
from .generate import (Scene, make_config, make_actions, make_rig, focal_px, custom_scene, grid_map, disk_triangles, make_paper_rig, make_paper_workload, default_palette,
                       CLASS_SKY, CLASS_GROUND, CLASS_ROAD, CLASS_MARKING, CLASS_VEHICLE, CLASS_SIGNAL, CLASS_CYCLIST, CLASS_PEDESTRIAN,
                       NOMINAL_DIMS, MOUNT, DT, WHEELBASE, V_MAX)
