"""The Python binding mirrors include/detox.h: enum values, limits and the pipeline struct layout."""
import ctypes
import os
import re

import paper_1907_12205_b200 as dx
from paper_1907_12205_b200 import binding

HEADER = open(os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "detox.h")).read()


def enum_values(prefix):
    return {name: int(val) for name, val in re.findall(r"\b(%s[A-Z_]+)\s*=\s*(\d+)" % prefix, HEADER)}


def test_aggregator_codes_match():
    codes = enum_values("DETOX_AGG_")
    assert codes == {"DETOX_AGG_NONE": dx.AGG_NONE, "DETOX_AGG_MEAN": dx.AGG_MEAN,
                     "DETOX_AGG_COORD_MEDIAN": dx.AGG_COORD_MEDIAN, "DETOX_AGG_MULTIKRUM": dx.AGG_MULTIKRUM,
                     "DETOX_AGG_BULYAN": dx.AGG_BULYAN, "DETOX_AGG_TRIMMED_MEAN": dx.AGG_TRIMMED_MEAN,
                     "DETOX_AGG_GEOMETRIC_MEDIAN": dx.AGG_GEOMETRIC_MEDIAN,
                     "DETOX_AGG_SIGN_MAJORITY": dx.AGG_SIGN_MAJORITY}


def test_split_modes_match():
    modes = {name: int(val) for name, val in re.findall(r"\b(DETOX_SPLIT_[A-Z0-9_]+)\s*=\s*(\d+)", HEADER)}
    assert modes == {"DETOX_SPLIT_AUTO": dx.SPLIT_AUTO, "DETOX_SPLIT_TF32": dx.SPLIT_TF32}


def test_limits_and_status_codes_match():
    defs = {k: int(v) for k, v in re.findall(r"#define\s+(DETOX_[A-Z_]+)\s+(\d+)", HEADER)}
    assert defs["DETOX_MAX_ROWS"] == binding.MAX_ROWS and defs["DETOX_MAX_R"] == binding.MAX_R
    assert defs["DETOX_NOALLOC_MAX_GROUPS"] == binding.NOALLOC_MAX_GROUPS
    status = {name: int(val) for name, val in re.findall(r"\b(DETOX_OK|DETOX_ERR_[A-Z_]+)\s*=\s*(\d+)", HEADER)}
    assert status["DETOX_OK"] == 0 and status["DETOX_ERR_TIMEOUT"] == 5 and len(status) == 6


def test_pipeline_struct_fields_in_header_order():
    body = re.search(r"typedef struct \{(.*?)\} detox_pipeline_desc;", HEADER, re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    names = re.findall(r"\b(\w+);", body)
    assert names == [f[0] for f in binding.PipelineDesc._fields_]
    assert ctypes.sizeof(binding.PipelineDesc) == 72       # two 8-byte-aligned blocks of pointers and ints
