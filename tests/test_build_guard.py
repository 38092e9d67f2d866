"""The build's check on ptxas' resource report: a hot tensor-core kernel whose accumulator array has left the
register file (a large stack frame) fails the build; the variants that spill by design do not."""
from paper_2607_20501_b200 import build as B

REPORT = """\
ptxas info    : Compiling entry function '_ZN2mk4_x_14gemm_tc_kernelILi2ELb0ELb0ELb0ELb0EEEv14CUtensorMap_st' for 'sm_100a'
ptxas info    : Function properties for _ZN2mk4_x_14gemm_tc_kernelILi2ELb0ELb0ELb0ELb0EEEv14CUtensorMap_st
    {frame} bytes stack frame, 0 bytes spill stores, 0 bytes spill loads
ptxas info    : Used 128 registers, used 1 barriers
ptxas info    : Compiling entry function '_ZN2mk4_x_14gemm_tc_kernelILi2ELb0ELb1ELb0ELb0EEEv14CUtensorMap_st' for 'sm_100a'
ptxas info    : Function properties for _ZN2mk4_x_14gemm_tc_kernelILi2ELb0ELb1ELb0ELb0EEEv14CUtensorMap_st
    184 bytes stack frame, 40 bytes spill stores, 40 bytes spill loads
"""


def test_stack_frames_are_read_per_kernel():
    f = B.stack_frames(REPORT.format(frame=16))
    assert sorted(f.values()) == [16, 184] and all("gemm_tc_kernel" in k for k in f)


def test_a_large_frame_in_a_default_instantiation_fails_and_the_row_norm_variant_does_not():
    assert B.check_stack("/x/csrc/gemm_tc.cu", REPORT.format(frame=16)) == []
    bad = B.check_stack("/x/csrc/gemm_tc.cu", REPORT.format(frame=160))
    assert len(bad) == 1 and "160-byte" in bad[0] and "ELb0ELb0ELb0ELb0E" in bad[0]
    assert B.check_stack("/x/csrc/other.cu", REPORT.format(frame=160)) == []
