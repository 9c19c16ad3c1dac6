"""B200-native save/restore of a text block's KV state (pack, verify, commit).

The package is a thin Python layer over ``libgk.so`` (CUDA, sm_100a): see
``include/gk.h`` for the C ABI and ``binding.py`` for the marshalling.
"""
from .binding import (GK_BF16, GK_FLAG_HEAD_MAJOR, GK_FLAG_SINGLE_PASS, GK_FLAG_SKIP_VERIFY, GK_FP8_E4M3, JOB_CHECKSUM, JOB_MISSING, JOB_OK,
                      JOB_PAGE_TABLE, JOB_TIMEOUT, Cache, Context, Geom, GkError, Job, JobArray, WindowBlock, gk_blob_size,
                      gk_debug_range_ok, gk_page_checksums_noalloc, load_library)

__all__ = ["GK_BF16", "GK_FP8_E4M3", "GK_FLAG_SKIP_VERIFY", "GK_FLAG_HEAD_MAJOR", "GK_FLAG_SINGLE_PASS", "JOB_OK", "JOB_CHECKSUM", "JOB_PAGE_TABLE",
           "JOB_MISSING", "JOB_TIMEOUT", "Cache", "Context", "Geom", "GkError", "Job", "JobArray", "WindowBlock", "gk_blob_size",
           "gk_debug_range_ok", "gk_page_checksums_noalloc", "load_library"]
