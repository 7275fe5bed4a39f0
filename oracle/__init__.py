"""Plain CPU oracle for the zip2zip dynamic-vocabulary path, written from the paper.

TEST INFRASTRUCTURE ONLY.  Imported by tests/, by the smoke check and by the benchmark's
CPU-baseline / reference legs.  The product package never imports it, and it imports nothing from
the product package: the two share no code.  Each module cites the passage it follows and names
the tests that pin it.
"""
