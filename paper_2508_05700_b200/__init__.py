"""B200 (sm_100a) implementation of the multi-faceted embedding-table lookup path.

`paper_2508_05700_b200.mfet` binds the C-ABI library (`include/mfet.h`); it is
imported on first use so that `paper_2508_05700_b200.inputs` (numpy only) can be
used without the CUDA library.
"""


def __getattr__(name):
    if name == "mfet":
        import importlib
        return importlib.import_module(".mfet", __name__)
    raise AttributeError(name)
