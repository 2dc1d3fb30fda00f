"""Device microbenchmarks behind the design choices of the kernels (issue rates of the candidate inner operations of the
binary product; cost of an exchange of small words between CTAs through L2).  Not part of the library:

    python -m paper_1802_00150_b200.microbench        # compiles both with nvcc for sm_100a and runs them on cuda:0
"""
